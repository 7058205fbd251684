"""The tensor-core kernel on pairs of SMs (`PATH_TENSOR_PAIRS`, full attention only) through the C ABI:
against the oracle, against the default one-CTA kernel (same arithmetic in the same order: equal bits),
head groupings that take the gather and copy-out paths, and its give-up path."""
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


def _inputs(lens, Hq, Hkv, seed, scale_q=1.0):
    D, dtype = 128, torch.bfloat16
    rows = sum(lens)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(seed)
    q = (scale_q * torch.randn(rows, Hq, D, generator=gen, device="cuda", dtype=torch.float32)).to(dtype)
    k = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    v = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    off = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64).tolist()
    return q, k, v, off


def _run(bc, path, off, lens, q, k, v, scale):
    bc.set_path(path)
    out = torch.full_like(q, 3.0)
    lse = torch.full(q.shape[:2], 3.0, dtype=torch.float32, device="cuda")
    bc.attend_full(0, off, lens, q, k, v, out, lse, scale)
    assert bc.device_status() == binding.OK
    return out, lse, bc.last_attention_kernel()


# one request of 1 row (the second CTA and tile B idle), requests that end inside a tile, a 16-key tile,
# items whose second CTA has no rows (n G <= 256), several items per request, more items than pairs of SMs
CASES = [
    (2, 2, [1]),
    (2, 2, [300]),
    (4, 4, [513, 127, 640, 16, 1025]),
    (8, 2, [130, 64, 259, 1, 700]),            # four query heads per KV head
    (8, 1, [33, 200, 65]),                     # eight
    (32, 1, [17, 40]),                         # thirty-two: a token is a whole 32-row output box
    (14, 2, [300, 40, 513]),                   # seven: Q by gathers, output rows copied out by the warps
    (3, 1, [129, 700]),                        # three: gathers and copy-out as well
    (32, 32, [1100] * 6),                      # 96 items of 512 rows on 74 pairs
    (16, 16, [896, 600, 777] * 4),             # 192 items, no key splits in the default kernel: equal bits
]


@pytest.mark.parametrize("Hq,Hkv,lens", CASES)
def test_pairs_kernel_matches_oracle_and_default_kernel(Hq, Hkv, lens):
    D = 128
    q, k, v, off = _inputs(lens, Hq, Hkv, seed=5 + len(lens))
    bc = binding.BiCache(1, Hq, Hkv, D, 4, torch.bfloat16, sum(lens), len(lens))
    scale = D ** -0.5
    out_p, lse_p, kern_p = _run(bc, binding.PATH_TENSOR_PAIRS, off, lens, q, k, v, scale)
    out_s, lse_s, kern_s = _run(bc, binding.PATH_TENSOR, off, lens, q, k, v, scale)
    assert kern_p == binding.KERNEL_TENSOR_PAIRS and kern_s == binding.KERNEL_TENSOR
    if max(lens) <= 7 * 128:
        # the default kernel never splits the keys of such a batch: same arithmetic, same order
        assert torch.equal(out_p, out_s) and torch.equal(lse_p, lse_s)
    else:
        assert (out_p.float() - out_s.float()).abs().max().item() <= 1e-2
        assert (lse_p - lse_s).abs().max().item() <= 1e-4
    if sum(n * n for n in lens) * Hq <= 40_000_000:
        ref, ref_lse = oracle.attend_full(off, lens, *(workloads.to_f64(x) for x in (q, k, v)), scale)
        err = np.abs(workloads.to_f64(out_p) - ref)
        assert err.max() <= 2e-2 and err.mean() <= 2e-3
        assert np.abs(workloads.to_f64(lse_p) - ref_lse).max() <= 1e-3
    bc.close()


def test_pairs_kernel_rescales_when_the_row_maximum_jumps():
    # large scores late in the key range: the lazy reference maximum has to move, O is rescaled
    D, Hq, Hkv, lens = 128, 2, 2, [700, 260]
    q, k, v, off = _inputs(lens, Hq, Hkv, seed=9)
    k[500:, :, :] *= 6.0
    bc = binding.BiCache(1, Hq, Hkv, D, 4, torch.bfloat16, sum(lens), len(lens))
    scale = 0.5
    out_p, lse_p, kern_p = _run(bc, binding.PATH_TENSOR_PAIRS, off, lens, q, k, v, scale)
    assert kern_p == binding.KERNEL_TENSOR_PAIRS
    ref, ref_lse = oracle.attend_full(off, lens, *(workloads.to_f64(x) for x in (q, k, v)), scale)
    err = np.abs(workloads.to_f64(out_p) - ref)
    assert err.max() <= 3e-2 and err.mean() <= 2e-3
    assert np.abs(workloads.to_f64(lse_p) - ref_lse).max() <= 2e-3 * max(1.0, np.abs(ref_lse).max() / 100)
    bc.close()


def test_pairs_path_leaves_attend_to_the_default_kernel():
    D = 128
    # attention over a cached prefix stays on the default kernels
    w = workloads.Workload("pairs_attend", 1, 4, 4, 128, torch.bfloat16, 16, [200], [0, 0], [300, 70],
                           softmax_scale=D ** -0.5, seed=77)
    bc = binding.BiCache(1, 4, 4, D, w.pages_needed() + 1, torch.bfloat16, w.total_rows, 2)
    kc, vc = workloads.draw_prefix_kv(w, 0, "cuda")
    pid = bc.put_prefix(1, kc, vc)[0]
    q, k, v = workloads.draw_full_qkv(w, "cuda")
    bc.set_path(binding.PATH_TENSOR_PAIRS)
    out = torch.zeros_like(q)
    bc.attend(0, [pid, pid], w.suffix_row_off, w.suffix_lens, q, k, v, out, None, w.softmax_scale)
    assert bc.device_status() == binding.OK and bc.last_attention_kernel() == binding.KERNEL_TENSOR
    bc.close()


def test_pairs_kernel_tiny_wait_budget_reports_timeout_and_context_recovers():
    D, Hq, Hkv, lens = 128, 8, 8, [700, 130, 513, 900]
    q, k, v, off = _inputs(lens, Hq, Hkv, seed=2)
    bc = binding.BiCache(1, Hq, Hkv, D, 4, torch.bfloat16, sum(lens), len(lens))
    bc.set_path(binding.PATH_TENSOR_PAIRS)
    out = torch.zeros_like(q)
    bc.set_wait_budget(1)                                   # every wait that is not already complete gives up
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)
    assert bc.last_attention_kernel() == binding.KERNEL_TENSOR_PAIRS
    assert bc.device_status() == binding.ERR_TIMEOUT
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)   # a launch on a flagged context does no work
    assert bc.device_status(clear=True) == binding.ERR_TIMEOUT
    assert bc.device_status() == binding.OK
    bc.set_wait_budget(0)
    out.zero_()
    bc.attend_full(0, off, lens, q, k, v, out, None, D ** -0.5)
    assert bc.device_status() == binding.OK
    ref, _ = oracle.attend_full(off, lens, *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    err = np.abs(workloads.to_f64(out) - ref)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    bc.close()
