"""The two-call dispatches (bicache_attend_layer, bicache_attend_step) check everything the host can check,
and place both schedules in the workspace, before they launch anything: a failure of the second half
leaves the outputs of the first half untouched too.  The failure is made on the host: a workspace that
holds the small schedule of the reusing requests but not the schedule of a (claimed) multi-million-row
recompute request, whose rows are never touched because nothing is launched.  Also: the schedule cache
uploads nothing once a step has been seen."""
import ctypes as C

import numpy as np
import pytest
import torch

import __graft_entry__ as entry
from paper_2606_07571_b200 import binding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    binding.load_library()


def small_context(Hq=4, Hkv=4, D=128, L=2, npages=16):
    lib = binding.load_library()
    cfg = binding.Config(L, Hq, Hkv, D, 16, npages, binding.BF16, 0)
    floor = lib.bicache_workspace_bytes(C.byref(cfg), 0, 0)          # the smallest arena the library asks for
    bc = binding.BiCache(L, Hq, Hkv, D, npages, torch.bfloat16, 0, 0, workspace_bytes=floor)
    bc.set_depth_table(workloads.standin_depth_table(L))
    return bc


def test_attend_layer_second_half_failure_leaves_outputs_untouched():
    bc = small_context()
    gen = torch.Generator(device="cuda").manual_seed(1)
    m, n = 40, 24
    kc = torch.randn(2, m, 4, 128, generator=gen, device="cuda").to(torch.bfloat16)
    pid, _, _ = bc.put_prefix(77, kc, kc)
    rows = 2 * (m + n)
    q = torch.randn(rows, 4, 128, generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.full_like(q, 3.0)
    # request 0 reuses (depth 2 > layer 0): a small schedule.  Request 1 recomputes and claims 8M rows:
    # its schedule (125 000 work items) cannot fit the minimal workspace.
    launches, uploads = bc.launch_count(), bc.schedule_uploads()
    with pytest.raises(binding.BiCacheError) as err:
        bc.attend_layer(0, [2, 0], [pid, pid], [0, m + n], [m + n, 8_000_000], q, q, q, out)
    assert err.value.status == binding.ERR_NOMEM
    assert bc.device_status() == binding.OK
    assert bc.launch_count() == launches                      # neither half was launched
    assert (out == 3.0).all()
    # the same call with an honest second request runs, and its reuse half finds its schedule cached
    uploads = bc.schedule_uploads()
    bc.attend_layer(0, [2, 0], [pid, pid], [0, m + n], [m + n, m + n], q, q, q, out)
    assert bc.device_status() == binding.OK
    assert bc.launch_count() == launches + 2
    assert bc.schedule_uploads() == uploads + 1               # only the recompute half was new
    assert not (out[m:m + n] == 3.0).all() and not (out[m + n:] == 3.0).all()
    assert (out[:m] == 3.0).all()                             # prefix rows of the reusing request: not computed
    bc.close()


def test_attend_step_second_half_failure_leaves_outputs_untouched():
    bc = small_context(npages=32)
    gen = torch.Generator(device="cuda").manual_seed(2)
    m, n = 40, 24
    kc = torch.randn(2, m, 4, 128, generator=gen, device="cuda").to(torch.bfloat16)
    pid, _, _ = bc.put_prefix(78, kc, kc)
    priv, _, _ = bc.reserve_prefix(79, m)
    q = torch.randn(2 * (m + n), 4, 128, generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.full_like(q, 3.0)
    launches = bc.launch_count()
    with pytest.raises(binding.BiCacheError) as err:       # step 1 is a refresh step: request 1 recomputes
        bc.attend_step(0, 1, 16, [2, 0], [pid, pid], [-1, priv], [0, m + n], [m + n, 8_000_000], q, q, q, out)
    assert err.value.status == binding.ERR_NOMEM
    assert bc.device_status() == binding.OK
    assert bc.launch_count() == launches                      # no attention, no layer update
    assert (out == 3.0).all()
    bc.close()


def test_a_step_seen_once_uploads_nothing_again():
    """Per-request depths change the reuse / recompute membership from layer to layer; every (kind,
    membership) pair is uploaded once and found again in all later steps."""
    w = workloads.scaled_down(workloads.config4(), num_layers=8, max_requests=12, prefix_div=16, suffix_div=8)
    bc = binding.BiCache(w.num_layers, w.num_q_heads, w.num_kv_heads, w.head_dim, w.pages_needed() + 1, w.dtype,
                         w.total_rows, w.num_requests)
    bc.set_depth_table(workloads.standin_depth_table(w.num_layers))
    pid = []
    for g in range(len(w.prefix_lens)):
        kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
        pid.append(bc.put_prefix(workloads.prefix_key(w, g), kc, vc)[0])
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    out = torch.empty_like(q)
    depth = np.array([(3 * i) % (w.num_layers + 1) for i in range(w.num_requests)], dtype=np.int32)
    req_pid = [pid[g] for g in w.req_prefix]

    def step():
        for l in range(w.num_layers):
            bc.attend_layer(l, depth, req_pid, w.full_row_off, w.full_lens, q, k, v, out, None, w.softmax_scale)

    step()
    first = bc.schedule_uploads()
    assert 2 <= first <= 2 * w.num_layers
    step()
    step()
    assert bc.schedule_uploads() == first
    assert bc.device_status() == binding.OK
    bc.close()
