"""GPU parity of the key-range kernel (few query rows against long cached prefixes: the rows of a
prefix group share tiles, the prefix keys are split into ranges, each request's own keys are one
more range, a merge kernel combines them) against the oracle's attend (Eq. 2 over the key set of
Eq. 4), element by element through the C ABI.  Every case asserts that this kernel was the one
that ran.  Tolerances as in test_gpu_parity (bf16: max abs 2e-2, mean abs 2e-3; lse 1e-2)."""
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


def _run(Hq, Hkv, prefix_lens, req_prefix, suffix_lens, reqs=None, shuffle=False, scale=None, std=1.0,
         expect=binding.KERNEL_KEY_RANGES):
    D = 128
    w = workloads.Workload("key-ranges", 1, Hq, Hkv, D, torch.bfloat16, 16, prefix_lens, req_prefix, suffix_lens,
                           softmax_scale=(D ** -0.5 if scale is None else scale), value_std=std, shuffle_pages=shuffle)
    npages = w.pages_needed() + 1
    order = workloads.shuffled_page_order(npages, 7) if shuffle else None
    bc = binding.BiCache(1, Hq, Hkv, D, npages, torch.bfloat16, w.total_rows, w.num_requests, free_order=order)
    st = oracle.PagedPrefixStore(1, Hkv, D, 16, npages, free_order=order)
    pid, opid = [], []
    for g in range(len(prefix_lens)):
        kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
        pid.append(bc.put_prefix(workloads.prefix_key(w, g), kc, vc)[0])
        opid.append(st.put(workloads.prefix_key(w, g), workloads.to_f64(kc), workloads.to_f64(vc))[0])
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    reqs = list(range(w.num_requests)) if reqs is None else reqs
    out = torch.full_like(q, 7.0)
    lse = torch.full(q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
    offs = [w.suffix_row_off[i] for i in reqs]
    lens = [w.suffix_lens[i] for i in reqs]
    bc.attend(0, [pid[w.req_prefix[i]] for i in reqs], offs, lens, q, k, v, out, lse, w.softmax_scale)
    assert bc.device_status() == binding.OK
    assert bc.last_attention_kernel() == expect
    ref, ref_lse = oracle.attend(st, 0, [opid[w.req_prefix[i]] for i in reqs], offs, lens,
                                 *(workloads.to_f64(x) for x in (q, k, v)), w.softmax_scale)
    got, got_lse = workloads.to_f64(out), workloads.to_f64(lse)
    mask = np.zeros(w.total_rows, dtype=bool)
    for o, n in zip(offs, lens):
        mask[o:o + n] = True
    err = np.abs(got[mask] - ref[mask])
    assert err.max() <= 2e-2 and err.mean() <= 2e-3, (float(err.max()), float(err.mean()))
    assert np.abs(got_lse[mask] - ref_lse[mask]).max() <= 1e-3
    assert (got[~mask] == 7.0).all() and (got_lse[~mask] == 7.0).all()          # untouched rows
    bc.close()


def test_two_groups_ragged_prefixes_gqa():
    """Two prefix groups of different, ragged lengths (the last key tile and the last page are
    partial), requests of 0, 1 and a few tokens, four query heads per KV head: the rows of a group
    (requests NOT adjacent in memory: each request's prefix rows lie between) share one tile."""
    _run(8, 2, [1500, 2049], [0, 0, 0, 1, 1], [5, 0, 17, 1, 30], shuffle=True)


def test_group_of_two_row_tiles():
    """180 packed rows per KV head: two 128-row tiles per range, the second one ragged; a request's
    rows straddle the tile boundary."""
    _run(2, 2, [1100], [0, 0, 0], [60, 60, 60])


def test_gqa_seven_heads_per_kv_head_many_ranges():
    """Dream-shaped head grouping (28 / 4): 16 tokens x 7 heads = 112 packed rows, few CTAs per range,
    so the prefix is cut into many ranges (more than 32: the merge spreads them over a block's warps)."""
    _run(28, 4, [9000], [0], [16])


def test_minimal_prefix_and_single_token():
    _run(4, 4, [1024], [0], [1])


def test_subset_of_requests_and_peaked_scores():
    """Only some requests of the batch are passed (as the per-layer dispatch does); large scores make
    the row maximum move between key tiles and ranges (the rescaling path and the merge weights)."""
    _run(4, 2, [1300, 1200], [0, 0, 1, 1], [9, 20, 3, 40], reqs=[1, 2, 3], scale=1.0, std=1.0)


def test_outside_the_regime_the_general_kernel_runs():
    """A short prefix, or a request with more than 128 packed rows, keeps the general tensor-core kernel."""
    _run(4, 2, [700], [0, 0], [10, 10], expect=binding.KERNEL_TENSOR)
    _run(2, 2, [1100], [0, 0], [200, 100], expect=binding.KERNEL_TENSOR)


def test_group_of_many_short_requests_several_row_tiles():
    """Seven requests of up to 100 tokens in one group: 470 packed rows per KV head = four row tiles
    per key range, requests straddling the tile boundaries; a second group of one request."""
    _run(4, 4, [1400, 1100], [0, 0, 0, 0, 0, 0, 0, 1], [100, 64, 1, 90, 15, 100, 100, 128], shuffle=True)


@pytest.mark.parametrize("seed", [0, 1, 2, 3, 4, 5])
def test_seeded_random_shapes(seed):
    rng = np.random.default_rng(500 + seed)
    Hkv = int(rng.choice([1, 2, 4]))
    G = int(rng.choice([1, 2, 4, 7]))
    groups = int(rng.integers(1, 4))
    prefix_lens = [int(rng.integers(1024, 2600)) for _ in range(groups)]
    req_prefix, suffix_lens = [], []
    for g in range(groups):
        for _ in range(int(rng.integers(1, 7))):
            req_prefix.append(g)
            suffix_lens.append(int(rng.integers(0, 128 // G + 1)))   # a request: at most 128 packed rows
    if sum(suffix_lens) == 0:
        suffix_lens[0] = 1
    _run(Hkv * G, Hkv, prefix_lens, req_prefix, suffix_lens, shuffle=bool(rng.integers(0, 2)))
