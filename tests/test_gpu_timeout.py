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
