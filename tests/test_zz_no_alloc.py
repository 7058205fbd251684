"""The allocation-free entry point against the regular one and against the oracle.

bicache_attend_full_static serves callers that cannot allocate device memory (its scratch is a
fixed array inside the library).  It must give what bicache_attend_full gives, call after call:
the array keeps the previous call's contents, so the second call (other sizes, other data) would
expose any stale value that leaked through.  This file sorts last on purpose: a run that stops at
the first failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import __graft_entry__ as entry
import oracle
from paper_2606_07571_b200 import binding, workloads

pytestmark = pytest.mark.gpu


def reference(q, k, v, scale):
    """The regular entry point (context + workspace) on the same tensors."""
    n, Hq, D = q.shape
    bc = binding.BiCache(1, Hq, k.shape[1], D, 1, q.dtype, n, 1)
    out = torch.zeros_like(q)
    bc.attend_full(0, [0], [n], q, k, v, out, None, scale)
    assert bc.device_status() == binding.OK
    bc.close()
    return out


@pytest.mark.parametrize("dtype,tol", [(torch.bfloat16, 2e-2), (torch.float32, 1e-4)])
def test_static_entry_point_matches_regular_one_twice_in_a_row(dtype, tol):
    entry.build()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(3)
    # second call: fewer rows, other head layout, other data -> stale partials would show
    for n, Hq, Hkv, D in ((125, 8, 2, 128), (37, 4, 4, 64)):
        q = torch.randn(n, Hq, D, generator=gen, device="cuda").to(dtype)
        k = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(dtype)
        v = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(dtype)
        out = torch.full_like(q, 5.0)
        assert binding.attend_full_static(q, k, v, out, D ** -0.5) == binding.OK
        torch.cuda.synchronize()
        ref = reference(q, k, v, D ** -0.5)
        err = (out.double() - ref.double()).abs()
        assert torch.isfinite(out).all()
        assert err.max().item() <= tol and err.mean().item() <= tol / 10
        # and against the definition itself (Eq. 2 over the request's own rows)
        want, _ = oracle.attend_full([0], [n], *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
        err = np.abs(workloads.to_f64(out) - want)
        assert err.max() <= tol and err.mean() <= tol / 10


@pytest.mark.parametrize("D", [32, 96])
def test_static_entry_point_other_head_dims_match_the_oracle(D):
    entry.build()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11 + D)
    n, Hq, Hkv = 70, 6, 3
    q = torch.randn(n, Hq, D, generator=gen, device="cuda").to(torch.bfloat16)
    k = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(torch.bfloat16)
    v = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.full_like(q, 5.0)
    assert binding.attend_full_static(q, k, v, out, D ** -0.5) == binding.OK
    torch.cuda.synchronize()
    want, _ = oracle.attend_full([0], [n], *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    err = np.abs(workloads.to_f64(out) - want)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3


def test_static_entry_point_capacity_edge():
    """Exactly BICACHE_STATIC_MAX_ROW_HEADS row-heads are served (and correct), one more is refused."""
    entry.build()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    n, Hq, Hkv, D = 128, 32, 8, 64                                            # 128 * 32 = 4096 row-heads
    assert n * Hq == binding.STATIC_MAX_ROW_HEADS
    q = torch.randn(n, Hq, D, generator=gen, device="cuda").to(torch.bfloat16)
    k = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(torch.bfloat16)
    v = torch.randn(n, Hkv, D, generator=gen, device="cuda").to(torch.bfloat16)
    out = torch.full_like(q, 5.0)
    assert binding.attend_full_static(q, k, v, out, D ** -0.5) == binding.OK
    torch.cuda.synchronize()
    want, _ = oracle.attend_full([0], [n], *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    err = np.abs(workloads.to_f64(out) - want)
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    q1 = torch.zeros(4097, 1, D, dtype=torch.bfloat16, device="cuda")         # 4097 row-heads
    out1 = torch.full_like(q1, 5.0)
    assert binding.attend_full_static(q1, q1, q1, out1) == binding.ERR_NOMEM
    torch.cuda.synchronize()
    assert (out1 == 5.0).all()


def test_static_entry_point_rejects_what_does_not_fit():
    entry.build()
    q = torch.zeros(129, 32, 128, dtype=torch.bfloat16, device="cuda")        # 4128 row-heads > 4096
    out = torch.full_like(q, 5.0)
    assert binding.attend_full_static(q, q, q, out) == binding.ERR_NOMEM
    q2 = torch.zeros(4, 2, 48, dtype=torch.bfloat16, device="cuda")           # head_dim not supported
    assert binding.attend_full_static(q2, q2, q2, torch.zeros_like(q2)) == binding.ERR_UNSUPPORTED
    torch.cuda.synchronize()
    assert (out == 5.0).all()
