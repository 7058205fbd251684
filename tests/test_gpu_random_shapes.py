"""Seeded random shapes through the C ABI: the tensor-core path against the CUDA-core path on the same
inputs (every case), and against the oracle (the small cases).  The draw covers what the fixed
configurations do not: head groupings of 1..32 query heads per KV head (7 and 16/32 leave the TMA
paths), several prefix groups, suffixes of one row up to several tiles, prefixes that end inside a
page or a tile, batches with more work items than SMs and with fewer (key splits + merge)."""
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


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_tensor_path_matches_simt_path_and_oracle(seed):
    rng = np.random.default_rng(seed)
    checked_oracle = 0
    for it in range(14):
        G = int(rng.choice([1, 1, 2, 4, 7, 8, 16, 32]))
        Hkv = int(rng.choice([1, 2, 4])) if G <= 8 else 1
        Hq = G * Hkv
        ngroups = int(rng.integers(1, 4))
        ms = [int(rng.choice([1, 15, 16, 100, 128, 129, 500, 1024])) for _ in range(ngroups)]
        R = int(rng.integers(1, 16))
        rp = sorted(int(rng.integers(0, ngroups)) for _ in range(R))
        ns = [int(rng.choice([1, 2, 31, 33, 64, 127, 128, 129, 200, 256, 257, 400])) for _ in range(R)]
        full = bool(rng.integers(0, 2))
        w = workloads.Workload("r%d_%d" % (seed, it), 1, Hq, Hkv, 128, torch.bfloat16, 16, ms, rp, ns,
                               softmax_scale=128 ** -0.5, seed=100 * seed + it)
        bc = binding.BiCache(1, Hq, Hkv, 128, w.pages_needed() + 1, torch.bfloat16, w.total_rows, R)
        small = w.total_rows * Hq * (max(ms) + max(ns)) < 20_000_000
        st = oracle.PagedPrefixStore(1, Hkv, 128, 16, w.pages_needed() + 1) if small else None
        pids = []
        for g in range(ngroups):
            kc, vc = workloads.draw_prefix_kv(w, g, "cuda")
            pids.append(bc.put_prefix(100 + g, kc, vc)[0])
            if small:
                assert st.put(100 + g, workloads.to_f64(kc), workloads.to_f64(vc))[0] == pids[-1]
        q, k, v = workloads.draw_full_qkv(w, "cuda")
        res = []
        for path in (binding.PATH_TENSOR, binding.PATH_SIMT):
            bc.set_path(path)
            out = torch.full_like(q, 3.0)
            lse = torch.full(q.shape[:2], 3.0, dtype=torch.float32, device="cuda")
            if full:
                bc.attend_full(0, w.full_row_off, w.full_lens, q, k, v, out, lse, w.softmax_scale)
            else:
                bc.attend(0, [pids[g] for g in rp], w.suffix_row_off, w.suffix_lens, q, k, v, out, lse, w.softmax_scale)
            assert bc.device_status() == binding.OK
            res.append((workloads.to_f64(out), workloads.to_f64(lse)))
        what = "seed %d case %d G %d Hkv %d m %s n %s full %s" % (seed, it, G, Hkv, ms, ns, full)
        assert np.isfinite(res[0][0]).all(), what
        assert np.abs(res[0][0] - res[1][0]).max() <= 2e-2, what
        assert np.abs(res[0][1] - res[1][1]).max() <= 1e-3, what
        if small:
            qd, kd, vd = (workloads.to_f64(x) for x in (q, k, v))
            if full:
                ref, rl = oracle.attend_full(w.full_row_off, w.full_lens, qd, kd, vd, w.softmax_scale)
                rows = np.arange(w.total_rows)
            else:
                ref, rl = oracle.attend(st, 0, [pids[g] for g in rp], w.suffix_row_off, w.suffix_lens, qd, kd, vd,
                                        w.softmax_scale)
                rows = np.concatenate([np.arange(o, o + n) for o, n in zip(w.suffix_row_off, w.suffix_lens)])
            err = np.abs(res[0][0][rows] - ref[rows])
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, what
            assert np.abs(res[0][1][rows] - rl[rows]).max() <= 1e-3, what
            untouched = np.setdiff1d(np.arange(w.total_rows), rows)
            assert (res[0][0][untouched] == 3.0).all(), what
            checked_oracle += 1
        bc.close()
    assert checked_oracle >= 2
