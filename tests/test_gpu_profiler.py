"""GPU parity of the profiler reduction (Eq. 3) through the C ABI against the oracle, and the rule
chain similarity -> depth -> table on the same numbers.  Similarities within 1e-5 (fp32 products of
exact inputs summed in fp64; the result is rounded to fp32)."""
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


@pytest.mark.parametrize("dtype,L,Hq,Hkv,D,m,shuffle", [
    (torch.bfloat16, 4, 4, 2, 128, 1000, True),      # swizzled page images, ragged last page
    (torch.bfloat16, 2, 8, 8, 128, 16, False),       # one page
    (torch.bfloat16, 3, 2, 1, 64, 77, True),         # plain [slot][dim] pages
    (torch.float32, 3, 2, 2, 64, 301, True),
])
def test_similarity_matches_oracle(dtype, L, Hq, Hkv, D, m, shuffle):
    npages = (m + 15) // 16 + 3
    order = workloads.shuffled_page_order(npages, 5) if shuffle else None
    bc = binding.BiCache(L, Hq, Hkv, D, npages, dtype, 64, 1, free_order=order)
    st = oracle.PagedPrefixStore(L, Hkv, D, 16, npages, free_order=order)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(21)
    kc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    vc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    pid, _, pages = bc.put_prefix(9, kc, vc)
    opid, _, opages = st.put(9, workloads.to_f64(kc), workloads.to_f64(vc))
    assert pages == opages
    # reference K/V: the cached ones plus layer-dependent noise, so that the similarity falls with depth
    noise_k = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32)
    noise_v = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32)
    amp = torch.linspace(0.0, 0.6, L, device="cuda").view(L, 1, 1, 1)
    # a padded layer stride exercises the stride argument
    big_k = torch.zeros(L, m + 3, Hkv, D, device="cuda", dtype=dtype)
    big_v = torch.zeros(L, m + 3, Hkv, D, device="cuda", dtype=dtype)
    big_k[:, :m] = (kc.float() + amp * noise_k).to(dtype)
    big_v[:, :m] = (vc.float() + amp * noise_v).to(dtype)
    kr, vr = big_k[:, :m], big_v[:, :m]
    sim = bc.prefix_similarity(pid, kr, vr)
    ref = oracle.kv_similarity(st, opid, workloads.to_f64(kr), workloads.to_f64(vr))
    assert np.abs(sim - ref).max() <= 1e-5, (sim, ref)
    assert sim[0] == pytest.approx(1.0, abs=1e-6)           # layer 0 has no noise
    sim_dev = torch.full((L,), 7.0, dtype=torch.float32, device="cuda")
    bc.prefix_similarity_async(pid, kr, vr, sim_dev)        # same numbers without the host copy
    assert (sim_dev.cpu().numpy() == sim).all()
    for tau in (0.97, 0.9, 0.5):
        assert binding.depth_from_similarity(sim, tau) == oracle.depth_from_similarity(np.float32(ref), np.float32(tau))
    # identical / negated / zero references
    assert np.abs(bc.prefix_similarity(pid, kc, vc) - 1.0).max() <= 1e-6
    assert np.abs(bc.prefix_similarity(pid, -kc, -vc) + 1.0).max() <= 1e-6
    assert (bc.prefix_similarity(pid, torch.zeros_like(kc), torch.zeros_like(vc)) == 0).all()
    # the attention calls still work on the workspace afterwards
    q, k, v = (torch.randn(64, h, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype) for h in (Hq, Hkv, Hkv))
    out = torch.zeros_like(q)
    bc.attend(0, [pid], [0], [64], q, k, v, out, None, D ** -0.5)
    assert bc.device_status() == binding.OK
    o_ref, _ = oracle.attend(st, 0, [opid], [0], [64], *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    assert np.abs(workloads.to_f64(out) - o_ref).max() <= (2e-2 if dtype == torch.bfloat16 else 1e-4)
    bc.close()


def test_profile_to_table_chain():
    """A toy profiling run: several 'requests' (reference K/V with noise growing with the layer and
    shrinking with the prefix ratio) -> similarities -> depths -> table, library against oracle."""
    L, Hq, Hkv, D, m = 6, 2, 2, 128, 64
    bc = binding.BiCache(L, Hq, Hkv, D, 8, torch.bfloat16, 64, 1)
    st = oracle.PagedPrefixStore(L, Hkv, D, 16, 8)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(4)
    kc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    vc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    pid, _, _ = bc.put_prefix(1, kc, vc)
    opid, _, _ = st.put(1, workloads.to_f64(kc), workloads.to_f64(vc))
    idx, got_b, ref_b = [], [], []
    for ratio in (30, 30, 60, 60, 90, 90, 90):
        amp = (torch.arange(L, device="cuda").float() * (1.0 - ratio / 100.0) * 0.25).view(L, 1, 1, 1)
        kr = (kc.float() + amp * torch.randn(L, m, Hkv, D, generator=gen, device="cuda")).to(torch.bfloat16)
        vr = (vc.float() + amp * torch.randn(L, m, Hkv, D, generator=gen, device="cuda")).to(torch.bfloat16)
        sim = bc.prefix_similarity(pid, kr, vr)
        ref = oracle.kv_similarity(st, opid, workloads.to_f64(kr), workloads.to_f64(vr))
        assert np.abs(sim - ref).max() <= 1e-5
        idx.append(ratio)
        got_b.append(binding.depth_from_similarity(sim, 0.97))
        ref_b.append(oracle.depth_from_similarity(ref, 0.97))
    assert got_b == ref_b
    table = binding.build_depth_table(idx, got_b, L)
    assert table == oracle.build_depth_table(idx, ref_b, L)
    assert table[90] >= table[60] >= table[30] >= 1          # more prefix, deeper reuse
    bc.set_depth_table(table)                                # and the table drives the depth rule
    assert bc.reuse_depth([90], [10]).tolist() == [table[90]]
    bc.close()
