"""The give-up path of the device-side waits, exercised without any barrier that could never complete:
with a budget of one SM cycle, ordinary waits (for a tile in flight, for the tensor pipe) run out; the
CTAs must drain, release their tensor memory and exit, the status must read TIMEOUT, and the context
must work again once the status is cleared."""
import numpy as np
import pytest
import torch

import oracle
import __graft_entry__ as entry
from paper_2606_07571_b200 import binding, workloads

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _built():
    entry.build()
    binding.load_library()


@pytest.mark.parametrize("Hq,Hkv,lens", [(2, 2, [300]), (32, 8, [700, 130, 256, 513, 64, 900])])
def test_tiny_wait_budget_reports_timeout_and_context_recovers(Hq, Hkv, lens):
    D, dtype = 128, torch.bfloat16
    rows = sum(lens)
    off = np.concatenate([[0], np.cumsum(lens)[:-1]]).tolist()
    bc = binding.BiCache(1, Hq, Hkv, D, 4, dtype, rows, len(lens))
    bc.set_path(binding.PATH_TENSOR)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(2)
    q = torch.randn(rows, Hq, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    k = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    v = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    out = torch.zeros_like(q)
    bc.set_wait_budget(1)                                   # every wait that is not already complete gives up
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)
    assert bc.device_status() == binding.ERR_TIMEOUT        # sticky until cleared
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)   # a launch on a flagged context does no work
    assert bc.device_status(clear=True) == binding.ERR_TIMEOUT
    assert bc.device_status() == binding.OK
    bc.set_wait_budget(0)                                   # the default again
    out.zero_()
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)
    assert bc.device_status() == binding.OK
    ref, _ = oracle.attend_full(off, lens, *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    err = np.abs(workloads.to_f64(out) - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    bc.close()


def test_projection_tiny_wait_budget_reports_timeout_and_context_recovers():
    """The same for the projection kernel, whose CTAs work in pairs: both CTAs of a pair give up,
    wait for their loads, meet at the pair's barrier and release the pair's tensor memory."""
    Hkv, D, m, d_model = 4, 128, 700, 512
    bc = binding.BiCache(1, Hkv, Hkv, D, (m + 15) // 16 + 1, torch.bfloat16, 16, 1)
    pid, _, _ = bc.reserve_prefix(3, m)
    h, w_k, w_v = workloads.draw_hidden_and_weights(m, d_model, Hkv, D, 9, device="cuda")
    bc.set_wait_budget(1)
    bc.project_prefix_layer(pid, 0, h, w_k, w_v)
    assert bc.device_status() == binding.ERR_TIMEOUT
    bc.project_prefix_layer(pid, 0, h, w_k, w_v)            # a launch on a flagged context does no work
    assert bc.device_status(clear=True) == binding.ERR_TIMEOUT
    assert bc.device_status() == binding.OK
    bc.set_wait_budget(0)
    bc.project_prefix_layer(pid, 0, h, w_k, w_v)
    assert bc.device_status() == binding.OK
    rk, rv = oracle.project_kv(workloads.to_f64(h)[None], workloads.to_f64(w_k)[None], workloads.to_f64(w_v)[None],
                               Hkv, D)
    gk = torch.empty(m, Hkv, D, dtype=torch.bfloat16, device="cuda")
    gv = torch.empty_like(gk)
    bc.read_prefix_layer(pid, 0, gk, gv)
    for got, ref in ((gk, rk[0]), (gv, rv[0])):
        assert np.all(np.abs(workloads.to_f64(got) - ref) <= np.abs(ref) * 2.0 ** -8 + 1e-3)
    bc.close()


def test_key_range_kernel_tiny_wait_budget_reports_timeout_and_context_recovers():
    """The same for the kernel that serves few query rows against a long cached prefix."""
    Hq, Hkv, D, m, n = 4, 2, 128, 2000, [7, 12]
    w = workloads.Workload("kr-timeout", 1, Hq, Hkv, D, torch.bfloat16, 16, [m], [0, 0], n, softmax_scale=D ** -0.5)
    bc = binding.BiCache(1, Hq, Hkv, D, w.pages_needed() + 1, torch.bfloat16, w.total_rows, 2)
    st = oracle.PagedPrefixStore(1, Hkv, D, 16, w.pages_needed() + 1)
    kc, vc = workloads.draw_prefix_kv(w, 0, "cuda")
    pid = bc.put_prefix(1, kc, vc)[0]
    opid = st.put(1, workloads.to_f64(kc), workloads.to_f64(vc))[0]
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    out = torch.zeros_like(q)
    args = (0, [pid, pid], w.suffix_row_off, w.suffix_lens, q, k, v, out, None, w.softmax_scale)
    bc.set_wait_budget(1)
    bc.attend(*args)
    assert bc.last_attention_kernel() == binding.KERNEL_KEY_RANGES
    assert bc.device_status() == binding.ERR_TIMEOUT
    bc.attend(*args)                                        # a launch on a flagged context does no work
    assert bc.device_status(clear=True) == binding.ERR_TIMEOUT
    assert bc.device_status() == binding.OK
    bc.set_wait_budget(0)
    out.zero_()
    bc.attend(*args)
    assert bc.device_status() == binding.OK
    ref, _ = oracle.attend(st, 0, [opid, opid], w.suffix_row_off, w.suffix_lens,
                           *(workloads.to_f64(x) for x in (q, k, v)), w.softmax_scale)
    mask = np.zeros(w.total_rows, dtype=bool)
    for o, nn in zip(w.suffix_row_off, w.suffix_lens):
        mask[o:o + nn] = True
    err = np.abs(workloads.to_f64(out)[mask] - ref[mask])
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    bc.close()
