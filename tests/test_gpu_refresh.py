"""GPU parity of the deep-layer reuse with periodic refresh (Eq. 5) through the C ABI: several
denoising steps with fresh Q/K/V each, shared prefixes in shallow layers, per-request kept prefix
K/V in deep layers, against the oracle's attend_step.  Tolerances as in test_gpu_parity."""
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


def _draw(gen, rows, Hq, Hkv, D, dtype):
    q = torch.randn(rows, Hq, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    k = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    v = torch.randn(rows, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    return q, k, v


@pytest.mark.parametrize("dtype,Hq,Hkv,D,path", [
    (torch.bfloat16, 4, 2, 128, binding.PATH_AUTO),
    (torch.bfloat16, 4, 2, 128, binding.PATH_SIMT),
    (torch.float32, 2, 1, 64, binding.PATH_AUTO),
])
def test_steps_with_refresh_match_oracle(dtype, Hq, Hkv, D, path):
    L, delta, S = 3, 3, 5
    prefix_lens = [150, 40]
    req_prefix = [0, 1, 0, 1, 0]                    # requests of one shared prefix are NOT contiguous
    suffix = [70, 33, 200, 1, 129]
    depth = [2, 1, 0, 3, 1]
    N = [prefix_lens[g] + n for g, n in zip(req_prefix, suffix)]
    row_off = np.concatenate([[0], np.cumsum(N)[:-1]]).tolist()
    rows = int(sum(N))
    R = len(N)
    npages = sum((m + 15) // 16 for m in prefix_lens) + sum((prefix_lens[g] + 15) // 16 for g in req_prefix) + 1
    bc = binding.BiCache(L, Hq, Hkv, D, npages, dtype, rows, R)
    bc.set_path(path)
    st = oracle.PagedPrefixStore(L, Hkv, D, 16, npages)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(11)
    shared, oshared = [], []
    for g, m in enumerate(prefix_lens):
        kc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
        vc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
        pid, _, pages = bc.put_prefix(100 + g, kc, vc)
        opid, _, opages = st.put(100 + g, workloads.to_f64(kc), workloads.to_f64(vc))
        assert (pid, pages) == (opid, opages)
        shared.append(pid)
    private = []
    for i in range(R):
        pid, hit, pages = bc.reserve_prefix(1000 + i, prefix_lens[req_prefix[i]])
        opid, ohit, opages = st.reserve(1000 + i, prefix_lens[req_prefix[i]])
        assert (pid, hit, pages) == (opid, ohit, opages)
        private.append(pid)
    sid = [shared[g] for g in req_prefix]
    scale = D ** -0.5
    max_tol, mean_tol, lse_tol = (2e-2, 2e-3, 1e-3) if dtype == torch.bfloat16 else (1e-4, 1e-5, 1e-5)
    for t in range(1, S + 1):
        q, k, v = _draw(gen, rows, Hq, Hkv, D, dtype)
        qd, kd, vd = (workloads.to_f64(x) for x in (q, k, v))
        assert bc.is_refresh_step(t, delta) == int(oracle.is_refresh_step(t, delta))
        for l in range(L):
            out = torch.full_like(q, 7.0)
            lse = torch.full(q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
            bc.attend_step(l, t, delta, depth, sid, private, row_off, N, q, k, v, out, lse, scale)
            assert bc.device_status() == binding.OK
            ref, rl = oracle.attend_step(st, l, t, delta, depth, sid, private, row_off, N, qd, kd, vd, scale)
            got, gl = workloads.to_f64(out), workloads.to_f64(lse)
            computed = np.isfinite(rl[:, 0])
            err = np.abs(got[computed] - ref[computed])
            assert np.isfinite(got).all()
            assert err.max() <= max_tol and err.mean() <= mean_tol, (t, l, err.max(), err.mean())
            assert np.abs(gl[computed] - rl[computed]).max() <= lse_tol
            assert (got[~computed] == 7.0).all() and (gl[~computed] == 7.0).all()   # rows not computed stay untouched
    # which rows a step computes: suffix rows under reuse, every row on a refresh step
    assert oracle.is_refresh_step(4, delta) and not oracle.is_refresh_step(5, delta)
    bc.close()


def test_update_prefix_layer_then_attend_reads_the_new_kv():
    """A layer written with update_prefix_layer is what attend reads afterwards (strided source rows)."""
    L, Hq, Hkv, D, m, n = 2, 2, 2, 128, 37, 50
    dtype = torch.bfloat16
    bc = binding.BiCache(L, Hq, Hkv, D, 8, dtype, m + n, 1)
    st = oracle.PagedPrefixStore(L, Hkv, D, 16, 8)
    pid, _, _ = bc.reserve_prefix(5, m)
    opid, _, _ = st.reserve(5, m)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(3)
    q, k, v = _draw(gen, m + n, Hq, Hkv, D, dtype)
    wide_k = torch.randn(m, 2 * Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    wide_v = torch.randn(m, 2 * Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
    src_k, src_v = wide_k[:, :Hkv], wide_v[:, :Hkv]          # row stride 2 * Hkv * D elements
    bc.update_prefix_layer(pid, 1, src_k, src_v)
    st.update_layer(opid, 1, workloads.to_f64(src_k), workloads.to_f64(src_v))
    out = torch.zeros_like(q)
    bc.attend(1, [pid], [m], [n], q, k, v, out, None, D ** -0.5)
    assert bc.device_status() == binding.OK
    ref, _ = oracle.attend(st, 1, [opid], [m], [n], *(workloads.to_f64(x) for x in (q, k, v)), D ** -0.5)
    err = np.abs(workloads.to_f64(out)[m:] - ref[m:])
    assert err.max() <= 2e-2 and err.mean() <= 2e-3
    bc.close()


def test_kept_prefixes_own_only_their_deep_layers():
    """Eq. 5 with per-layer storage: request i keeps its own prefix K/V only in the layers from depth[i]
    on (reserve with first_layer = depth[i]); the shallow layers' pools are smaller; a shared prefix put
    AFTER those reservations gets a different page list in every layer.  Page lists of every layer equal
    the oracle's, and three steps (refresh, reuse, reuse) match oracle.attend_step."""
    dtype, Hq, Hkv, D = torch.bfloat16, 4, 2, 128
    L, delta, S = 3, 4, 3
    prefix_lens = [150, 40]
    req_prefix = [0, 1, 0, 1, 0]
    suffix = [70, 33, 200, 1, 129]
    depth = [2, 1, 0, 3, 1]                        # request 3 reuses the shared cache in every layer
    N = [prefix_lens[g] + n for g, n in zip(req_prefix, suffix)]
    row_off = np.concatenate([[0], np.cumsum(N)[:-1]]).tolist()
    rows, R = int(sum(N)), len(N)
    need = [(m + 15) // 16 for m in prefix_lens]
    shared_pages = sum(need)
    caps = [shared_pages + sum(need[g] for g, d in zip(req_prefix, depth) if d <= l) for l in range(L)]
    npages = max(caps)
    bc = binding.BiCache(L, Hq, Hkv, D, npages, dtype, rows, R, layer_pages=caps)
    st = oracle.PagedPrefixStore(L, Hkv, D, 16, npages, layer_pages=caps)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(21)

    def put_shared(key, m):
        kc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
        vc = torch.randn(L, m, Hkv, D, generator=gen, device="cuda", dtype=torch.float32).to(dtype)
        pid, _, pages = bc.put_prefix(key, kc, vc)
        opid, _, opages = st.put(key, workloads.to_f64(kc), workloads.to_f64(vc))
        assert (pid, pages) == (opid, opages)
        for l in range(L):
            assert bc.prefix_pages(pid, l) == st.pages(opid, l)
        return pid

    shared = [put_shared(100, prefix_lens[0]), None]
    private = []
    for i in range(R):
        if depth[i] >= L:
            private.append(-1)
            continue
        pid, hit, pages = bc.reserve_prefix(1000 + i, prefix_lens[req_prefix[i]], first_layer=depth[i])
        opid, ohit, opages = st.reserve(1000 + i, prefix_lens[req_prefix[i]], first_layer=depth[i])
        assert (pid, hit, pages) == (opid, ohit, opages)
        for l in range(depth[i], L):
            assert bc.prefix_pages(pid, l) == st.pages(opid, l)
        private.append(pid)
    shared[1] = put_shared(101, prefix_lens[1])    # after the reservations: the layers' queues differ
    assert len({tuple(bc.prefix_pages(shared[1], l)) for l in range(L)}) > 1
    sid = [shared[g] for g in req_prefix]
    scale = D ** -0.5
    for t in range(1, S + 1):
        q, k, v = _draw(gen, rows, Hq, Hkv, D, dtype)
        qd, kd, vd = (workloads.to_f64(x) for x in (q, k, v))
        for l in range(L):
            out = torch.full_like(q, 7.0)
            lse = torch.full(q.shape[:2], 7.0, dtype=torch.float32, device="cuda")
            bc.attend_step(l, t, delta, depth, sid, private, row_off, N, q, k, v, out, lse, scale)
            assert bc.device_status() == binding.OK
            ref, rl = oracle.attend_step(st, l, t, delta, depth, sid, private, row_off, N, qd, kd, vd, scale)
            got, gl = workloads.to_f64(out), workloads.to_f64(lse)
            computed = np.isfinite(rl[:, 0])
            err = np.abs(got[computed] - ref[computed])
            assert np.isfinite(got).all()
            assert err.max() <= 2e-2 and err.mean() <= 2e-3, (t, l, err.max(), err.mean())
            assert np.abs(gl[computed] - rl[computed]).max() <= 1e-3
            assert (got[~computed] == 7.0).all()
    # a kept prefix cannot be read or written below its first layer
    deep = private[0]                               # first layer 2
    kk = torch.zeros(prefix_lens[0], Hkv, D, dtype=dtype, device="cuda")
    with pytest.raises(binding.BiCacheError) as e:
        bc.update_prefix_layer(deep, 0, kk, kk)
    assert e.value.status == binding.ERR_INVALID
    with pytest.raises(binding.BiCacheError) as e:
        bc.attend(1, [deep], [row_off[0] + prefix_lens[0]], [suffix[0]], q, k, v, out)
    assert e.value.status == binding.ERR_INVALID
    # read-back of one deep layer equals the oracle's kept K/V (bit-exact)
    ko, vo = torch.empty_like(kk), torch.empty_like(kk)
    bc.read_prefix_layer(deep, 2, ko, vo)
    torch.cuda.synchronize()
    rk, rv = st.prefix_kv(2, deep)
    assert np.array_equal(workloads.to_f64(ko), rk) and np.array_equal(workloads.to_f64(vo), rv)
    bc.close()
