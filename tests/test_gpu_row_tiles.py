"""Row tiles shared by the requests of a prefix group (bicache_attend on the tensor-core kernel): the
query rows of several requests are packed into one 256-row tile, every row masked to the own keys of
its own request.  Element-by-element against the oracle's definition (Eq. 2 over [cached prefix | own
suffix], per request), with the edge cases of the packing: more requests than a tile has segments,
requests that span tiles, lengths that are not multiples of 8, head groupings 1 / 2 / 4 / 8 (shared
tiles) and 7 (tiles per request), requests without a prefix and empty requests between the groups,
peaked logits (the rescale path next to masked rows), more work items than SMs."""
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


def run_case(name, Hq, Hkv, ms, req_prefix, ns, scale=128 ** -0.5, no_prefix=(), order=None, layers=1, layer=0):
    """req_prefix: prefix index per request (grouped); no_prefix: requests dispatched with prefix id -1."""
    w = workloads.Workload(name, layers, Hq, Hkv, 128, torch.bfloat16, 16, ms, req_prefix, ns,
                           softmax_scale=scale, seed=len(ns) + Hq)
    npages = w.pages_needed() + 1
    bc = binding.BiCache(layers, Hq, Hkv, 128, npages, torch.bfloat16, w.total_rows, w.num_requests, free_order=order)
    st = oracle.PagedPrefixStore(layers, Hkv, 128, 16, npages, free_order=order)
    pid = []
    for g in range(len(ms)):
        kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
        p, _, pages = bc.put_prefix(500 + g, kc, vc)
        op, _, opages = st.put(500 + g, workloads.to_f64(kc), workloads.to_f64(vc))
        assert (p, pages) == (op, opages)
        pid.append(p)
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    req_pid = [-1 if i in no_prefix else pid[g] for i, g in enumerate(req_prefix)]
    out = torch.full_like(q, 7.0)
    lse = torch.full(q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
    bc.set_path(binding.PATH_TENSOR)
    bc.attend(layer, req_pid, w.suffix_row_off, w.suffix_lens, q, k, v, out, lse, w.softmax_scale)
    assert bc.device_status() == binding.OK
    assert bc.last_attention_kernel() == binding.KERNEL_TENSOR
    ref, ref_lse = oracle.attend(st, layer, req_pid, w.suffix_row_off, w.suffix_lens,
                                 *(workloads.to_f64(x) for x in (q, k, v)), w.softmax_scale)
    got, got_lse = workloads.to_f64(out), workloads.to_f64(lse)
    mask = np.zeros(w.total_rows, dtype=bool)
    for o, n in zip(w.suffix_row_off, w.suffix_lens):
        mask[o:o + n] = True
    err = np.abs(got[mask] - ref[mask])
    assert np.isfinite(got).all(), name
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (name, float(err.max()), float(err.mean()))
    assert np.abs(got_lse[mask] - ref_lse[mask]).max() <= 1e-3, name
    assert (got[~mask] == 7.0).all() and (got_lse[~mask] == 7.0).all(), name + ": rows outside the requests"
    bc.close()


def test_many_short_requests_more_than_a_tile_has_segments():
    rng = np.random.default_rng(5)
    ns = [int(x) for x in rng.integers(1, 41, size=24)]
    run_case("short", 2, 2, [300], [0] * 24, ns)


def test_requests_spanning_tiles_with_four_heads_per_kv_head():
    run_case("span", 8, 2, [130], [0] * 6, [70, 3, 64, 129, 5, 200])


def test_two_groups_a_request_without_prefix_and_an_empty_one():
    run_case("mixed", 4, 2, [77, 200], [0, 0, 0, 1, 1, 1, 1], [33, 0, 90, 41, 12, 0, 150], no_prefix=(2,))


def test_eight_heads_per_kv_head_single_token_requests():
    run_case("g8", 8, 1, [100], [0] * 5, [1, 1, 1, 50, 17])


def test_seven_heads_per_kv_head_keeps_tiles_per_request():
    run_case("g7", 7, 1, [100], [0] * 4, [40, 3, 100, 9])


def test_peaked_logits_next_to_masked_rows():
    run_case("peaked", 2, 1, [150], [0] * 5, [20, 140, 7, 64, 100], scale=0.75)


def test_more_items_than_sms_scattered_pages_second_layer():
    rng = np.random.default_rng(9)
    ns = [int(x) for x in rng.integers(10, 301, size=40)]
    ms = [260, 90]
    npages = sum((m + 15) // 16 for m in ms) + 1
    run_case("many", 8, 8, ms, [0] * 25 + [1] * 15, ns, order=workloads.shuffled_page_order(npages, 3), layers=2,
             layer=1)


@pytest.mark.parametrize("seed", [31, 32, 33, 34])
def test_large_random_batches_against_the_cuda_core_path(seed):
    """Many requests in several groups, more work items than SMs (every CTA walks through many shared
    and plain tiles in a row), random head groupings that do and do not share tiles: the tensor-core path
    against the CUDA-core path of the same library on the same inputs (both are checked against the
    oracle elsewhere; here the point is volume)."""
    rng = np.random.default_rng(seed)
    G = int(rng.choice([1, 2, 4, 8, 3]))
    Hkv = int(rng.choice([2, 4, 8])) if G <= 2 else int(rng.choice([1, 2]))
    Hq = G * Hkv
    ngroups = int(rng.integers(2, 6))
    ms = [int(rng.integers(17, 900)) for _ in range(ngroups)]
    R = int(rng.integers(40, 120))
    rp = sorted(int(rng.integers(0, ngroups)) for _ in range(R))
    ns = [int(rng.choice([0, 1, 5, 8, 9, 31, 64, 100, 127, 128, 130, 257, 300])) for _ in range(R)]
    w = workloads.Workload("big%d" % seed, 1, Hq, Hkv, 128, torch.bfloat16, 16, ms, rp, ns,
                           softmax_scale=128 ** -0.5, seed=seed)
    bc = binding.BiCache(1, Hq, Hkv, 128, w.pages_needed() + 1, torch.bfloat16, w.total_rows, R)
    pids = []
    for g in range(ngroups):
        kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
        pids.append(bc.put_prefix(100 + g, kc, vc)[0])
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    req_pid = [pids[g] for g in rp]
    # a few requests go without a prefix (between the groups)
    for i in range(0, R, 17):
        req_pid[i] = -1
    ok_groups = all(req_pid[i] == req_pid[i - 1] or req_pid[i] not in req_pid[:i] for i in range(1, R))
    if not ok_groups:                         # a -1 in the middle of a group splits it: ids must stay grouped
        req_pid = [pids[g] for g in rp]
    res = []
    for path in (binding.PATH_TENSOR, binding.PATH_SIMT):
        bc.set_path(path)
        out = torch.full_like(q, 3.0)
        lse = torch.full(q.shape[:2], 3.0, dtype=torch.float32, device="cuda")
        bc.attend(0, req_pid, w.suffix_row_off, w.suffix_lens, q, k, v, out, lse, w.softmax_scale)
        assert bc.device_status() == binding.OK
        res.append((out.float(), lse))
    what = "seed %d G %d Hkv %d groups %s R %d" % (seed, G, Hkv, ms, R)
    assert torch.isfinite(res[0][0]).all(), what
    assert (res[0][0] - res[1][0]).abs().max().item() <= 2e-2, what
    assert (res[0][1] - res[1][1]).abs().max().item() <= 1e-3, what
    bc.close()
