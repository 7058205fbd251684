"""Pins for the oracle's attention, merge and layer dispatch (CPU only).

Each test checks the oracle against something other than itself: scalar brute
force over the concatenated key list, a library routine, closed forms,
invariants of softmax attention, or an inequality the paper proves.
"""
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# -- scalar brute force, written over plain Python lists ---------------------

def brute_row(q_row, keys, vals, scale):
    """Eq. 2 for one query: explicit loops, no max subtraction."""
    scores = [scale * sum(a * b for a, b in zip(q_row, kj)) for kj in keys]
    w = [math.exp(s) for s in scores]
    z = sum(w)
    d = len(vals[0])
    o = [sum(w[j] * vals[j][c] for j in range(len(keys))) / z for c in range(d)]
    return o, math.log(z)


def brute_attend(cached, layer, prefix_of, row_off, seqlen, q, k, v, scale, Hq, Hkv):
    """cached[g] = (K [L][m][Hkv][D], V) as nested lists.  Concatenate, then Eq. 2."""
    out = {}
    grp = Hq // Hkv
    for i, (off, n) in enumerate(zip(row_off, seqlen)):
        for h in range(Hq):
            hk = h // grp
            keys, vals = [], []
            if prefix_of[i] >= 0:
                Kc, Vc = cached[prefix_of[i]]
                keys += [Kc[layer][t][hk] for t in range(len(Kc[layer]))]
                vals += [Vc[layer][t][hk] for t in range(len(Vc[layer]))]
            keys += [k[off + j][hk] for j in range(n)]
            vals += [v[off + j][hk] for j in range(n)]
            for a in range(n):
                out[(i, h, a)] = brute_row(q[off + a][h], keys, vals, scale)
    return out


def rand(rng, *shape):
    return rng.standard_normal(shape)


@pytest.mark.parametrize("seed,L,Hq,Hkv,D,ms,ns,P", [
    (0, 1, 2, 2, 8, [5], [3, 4], 4),
    (1, 2, 4, 2, 8, [17, 1], [1, 6, 2], 16),
    (2, 1, 6, 3, 4, [33], [0, 7], 16),
    (3, 2, 1, 1, 8, [16, 32, 7], [5, 5, 5, 5], 16),
])
def test_attend_matches_scalar_brute_force(seed, L, Hq, Hkv, D, ms, ns, P):
    rng = np.random.default_rng(seed)
    npages = sum((m + P - 1) // P for m in ms) + 2
    order = rng.permutation(npages)
    store = oracle.PagedPrefixStore(L, Hkv, D, P, npages, free_order=order)
    cached, ids = [], []
    for g, m in enumerate(ms):
        Kc, Vc = rand(rng, L, m, Hkv, D), rand(rng, L, m, Hkv, D)
        pid, hit, _ = store.put(100 + g, Kc, Vc)
        assert not hit
        cached.append((Kc.tolist(), Vc.tolist()))
        ids.append(pid)
    prefix_of = [i % len(ms) for i in range(len(ns))]
    prefix_of.sort()
    prefix_of[-1] = -1 if len(ns) > 2 else prefix_of[-1]      # one request without prefix
    row_off, off = [], 2                                      # leading gap rows
    for n in ns:
        row_off.append(off)
        off += n + 1                                          # a gap row between requests
    q, k, v = rand(rng, off, Hq, D), rand(rng, off, Hkv, D), rand(rng, off, Hkv, D)
    scale = 0.7
    for layer in range(L):
        o, lse = oracle.attend(store, layer, [ids[g] if g >= 0 else -1 for g in prefix_of],
                               row_off, ns, q, k, v, scale)
        ref = brute_attend(cached, layer, prefix_of, row_off, ns,
                           q.tolist(), k.tolist(), v.tolist(), scale, Hq, Hkv)
        for (i, h, a), (ro, rl) in ref.items():
            np.testing.assert_allclose(o[row_off[i] + a, h], ro, rtol=1e-11, atol=1e-12)
            assert abs(lse[row_off[i] + a, h] - rl) < 1e-11
        # sampled-row entry point gives the same numbers
        samples = list(ref.keys())[::3]
        if samples:
            so, sl = oracle.attend_rows(store, layer, [ids[g] if g >= 0 else -1 for g in prefix_of],
                                        row_off, ns, q, k, v, scale, samples)
            for j, (i, h, a) in enumerate(samples):
                np.testing.assert_allclose(so[j], ref[(i, h, a)][0], rtol=1e-11, atol=1e-12)
                assert abs(sl[j] - ref[(i, h, a)][1]) < 1e-11


def test_attend_full_matches_scalar_brute_force():
    rng = np.random.default_rng(5)
    Hq, Hkv, D = 4, 2, 8
    lens, offs = [6, 1, 9], [0, 6, 7]
    q, k, v = rand(rng, 16, Hq, D), rand(rng, 16, Hkv, D), rand(rng, 16, Hkv, D)
    o, lse = oracle.attend_full(offs, lens, q, k, v, 0.5)
    ref = brute_attend([], 0, [-1] * 3, offs, lens, q.tolist(), k.tolist(), v.tolist(), 0.5, Hq, Hkv)
    for (i, h, a), (ro, rl) in ref.items():
        np.testing.assert_allclose(o[offs[i] + a, h], ro, rtol=1e-11, atol=1e-12)
        assert abs(lse[offs[i] + a, h] - rl) < 1e-11
    so, sl = oracle.attend_full_rows(offs, lens, q, k, v, 0.5, [(2, 3, 8), (0, 0, 0)])
    np.testing.assert_allclose(so[0], ref[(2, 3, 8)][0], rtol=1e-11)
    assert abs(sl[1] - ref[(0, 0, 0)][1]) < 1e-11


def test_attention_matches_torch_sdpa_fp64():
    """Third opinion: a library's non-causal scaled-dot-product attention."""
    rng = np.random.default_rng(7)
    nq, nk, H, D = 9, 21, 3, 16
    q, k, v = rand(rng, nq, H, D), rand(rng, nk, H, D), rand(rng, nk, H, D)
    o, _ = oracle.attention(q, k, v, 0.3)
    tq, tk, tv = (torch.from_numpy(x).permute(1, 0, 2)[None] for x in (q, k, v))
    ref = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=False, scale=0.3)
    np.testing.assert_allclose(o, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_rational_weight_golden_cases():
    """Eq. 2 with scores ln(a_j): weights a_j / sum a, lse = ln sum a."""
    with open(os.path.join(GOLDEN, "rational_softmax.txt")) as f:
        lines = [ln for ln in f if ln.strip() and not ln.startswith("#")]
    assert len(lines) >= 5
    for ln in lines:
        a_s, v_s, o_s, s_s = [x.strip() for x in ln.split(";")]
        a = [int(x) for x in a_s.split()]
        vals = np.array([[float(c) for c in t.split(",")] for t in v_s.split()])
        want = [float(Fraction(x)) for x in o_s.split()]
        scale = 0.25
        q = np.zeros((1, 1, 2))
        q[0, 0, 0] = 1.0 / scale                      # score_j = k_j[0]
        k = np.zeros((len(a), 1, 2))
        k[:, 0, 0] = np.log(a)
        k[:, 0, 1] = 123.0                            # orthogonal to q: must not matter
        o, lse = oracle.attention(q, k, vals[:, None, :], scale)
        np.testing.assert_allclose(o[0, 0], want, rtol=1e-13, atol=1e-13)
        assert abs(lse[0, 0] - math.log(int(s_s))) < 1e-13


def test_closed_forms():
    rng = np.random.default_rng(11)
    m, n, H, D, P = 37, 5, 2, 8, 16
    store = oracle.PagedPrefixStore(1, H, D, P, 4)
    Kc, Vc = rand(rng, 1, m, H, D), rand(rng, 1, m, H, D)
    pid, _, _ = store.put(1, Kc, Vc)
    k, v = rand(rng, n, H, D), rand(rng, n, H, D)
    # Q = 0: uniform weights -> mean of all m + n value rows, lse = ln(m + n)
    o, lse = oracle.attend(store, 0, [pid], [0], [n], np.zeros((n, H, D)), k, v, 1.0)
    mean = np.concatenate([Vc[0], v]).mean(axis=0)
    np.testing.assert_allclose(o, np.broadcast_to(mean, o.shape), rtol=1e-12)
    np.testing.assert_allclose(lse, math.log(m + n), rtol=1e-13)
    # constant V -> output is that constant whatever the scores are
    c = rng.standard_normal(D)
    store2 = oracle.PagedPrefixStore(1, H, D, P, 4)
    pid2, _, _ = store2.put(1, Kc, np.broadcast_to(c, Vc.shape))
    q = rand(rng, n, H, D)
    o, _ = oracle.attend(store2, 0, [pid2], [0], [n], q, k, np.broadcast_to(c, v.shape), 2.0)
    np.testing.assert_allclose(o, np.broadcast_to(c, o.shape), rtol=1e-12)
    # one dominant key (in the last, partial page of the prefix): output -> its value row
    Kd = np.zeros_like(Kc)
    Kd[0, m - 1, :, 0] = 1.0
    qd = np.zeros((n, H, D))
    qd[:, :, 0] = 1.0
    store3 = oracle.PagedPrefixStore(1, H, D, P, 4)
    pid3, _, _ = store3.put(1, Kd, Vc)
    o, lse = oracle.attend(store3, 0, [pid3], [0], [n], qd, np.zeros_like(k), v, 60.0)
    np.testing.assert_allclose(o, np.broadcast_to(Vc[0, m - 1], o.shape), atol=1e-20 + 1e-12)
    np.testing.assert_allclose(lse, 60.0, atol=1e-12)


def test_invariances():
    rng = np.random.default_rng(13)
    nq, nk, Hq, Hkv, D = 4, 19, 4, 2, 8
    q, k, v = rand(rng, nq, Hq, D), rand(rng, nk, Hkv, D), rand(rng, nk, Hkv, D)
    o, lse = oracle.attention(q, k, v, 0.9)
    # permuting the keys changes nothing
    perm = rng.permutation(nk)
    o2, lse2 = oracle.attention(q, k[perm], v[perm], 0.9)
    np.testing.assert_allclose(o2, o, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse2, lse, rtol=1e-13)
    # shifting every score of a row by a constant: K += u with <q, u> = c for all q
    # (q has a constant coordinate) leaves o unchanged and shifts lse by scale * c
    q1 = q.copy()
    q1[:, :, 0] = 2.0
    u = np.zeros(D)
    u[0] = 1.5
    o3, lse3 = oracle.attention(q1, k, v, 0.9)
    o4, lse4 = oracle.attention(q1, k + u, v, 0.9)
    np.testing.assert_allclose(o4, o3, rtol=1e-11, atol=1e-13)
    np.testing.assert_allclose(lse4 - lse3, 0.9 * 3.0, rtol=1e-11)
    # GQA equals MHA with the KV heads replicated
    o5, lse5 = oracle.attention(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1), 0.9)
    np.testing.assert_allclose(o5, o, rtol=1e-13)
    np.testing.assert_allclose(lse5, lse, rtol=1e-13)
    # transposed-operand tripwire: swapping K and V must change the result
    o6, _ = oracle.attention(q, v, k, 0.9)
    assert np.abs(o6 - o).max() > 1e-3


def test_physical_page_assignment_is_invisible():
    rng = np.random.default_rng(17)
    L, H, D, P, m, n = 2, 2, 8, 16, 45, 6
    Kc, Vc = rand(rng, L, m, H, D), rand(rng, L, m, H, D)
    q, k, v = rand(rng, n, H, D), rand(rng, n, H, D), rand(rng, n, H, D)
    outs = []
    for order in (None, rng.permutation(9), rng.permutation(9)):
        st = oracle.PagedPrefixStore(L, H, D, P, 9, free_order=order)
        pid, _, pages = st.put(5, Kc, Vc)
        kk, vv = st.prefix_kv(1, pid)
        assert np.array_equal(kk, Kc[1]) and np.array_equal(vv, Vc[1])
        outs.append(oracle.attend(st, 1, [pid], [0], [n], q, k, v, 0.4))
    for o, lse in outs[1:]:
        assert np.array_equal(o, outs[0][0]) and np.array_equal(lse, outs[0][1])


@pytest.mark.parametrize("seed", range(6))
def test_merge_of_any_split_equals_direct(seed):
    rng = np.random.default_rng(100 + seed)
    nq, nk, Hq, Hkv, D = 5, 23, 2, 1, 8
    q, k, v = rand(rng, nq, Hq, D), rand(rng, nk, Hkv, D) * 3, rand(rng, nk, Hkv, D)
    direct = oracle.attention(q, k, v, 1.1)
    nparts = 2 + seed % 3
    cuts = sorted(rng.integers(0, nk + 1, size=nparts - 1).tolist())
    if seed == 0:
        cuts = [0]                   # an empty first part
    if seed == 1:
        cuts = [nk, nk]              # empty trailing parts
    bounds = [0] + cuts + [nk]
    perm = rng.permutation(nk)       # arbitrary (not only contiguous) subsets
    parts = [oracle.attention(q, k[perm[a:b]], v[perm[a:b]], 1.1)
             for a, b in zip(bounds[:-1], bounds[1:])]
    o, lse = oracle.merge(parts)
    np.testing.assert_allclose(o, direct[0], rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse, direct[1], rtol=1e-12)
    assert np.isfinite(o).all()
    # commutative and associative
    o2, lse2 = oracle.merge(parts[::-1])
    np.testing.assert_allclose(o2, o, rtol=1e-12, atol=1e-14)
    if len(parts) >= 3:
        o3, lse3 = oracle.merge([oracle.merge(parts[:2])] + parts[2:])
        np.testing.assert_allclose(o3, o, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(lse3, lse, rtol=1e-12)


def test_merge_all_empty_is_empty():
    o, lse = oracle.merge([(np.zeros((2, 3)), np.full(2, -np.inf))] * 2)
    assert (o == 0).all() and np.isneginf(lse).all()


def _stack_inputs(rng, L, Hq, Hkv, D, ms, req_prefix, ns):
    offs, lens, off = [], [], 0
    for g, n in zip(req_prefix, ns):
        offs.append(off)
        lens.append(ms[g] + n)
        off += ms[g] + n
    q = [rand(rng, off, Hq, D) for _ in range(L)]
    k = [rand(rng, off, Hkv, D) for _ in range(L)]
    v = [rand(rng, off, Hkv, D) for _ in range(L)]
    return offs, lens, q, k, v


def test_stack_depth0_is_full_recompute_and_depthL_is_all_reuse():
    rng = np.random.default_rng(21)
    L, Hq, Hkv, D, P = 3, 2, 1, 8, 16
    ms, req_prefix, ns = [20, 9], [0, 0, 1], [4, 7, 3]
    offs, lens, q, k, v = _stack_inputs(rng, L, Hq, Hkv, D, ms, req_prefix, ns)
    store = oracle.PagedPrefixStore(L, Hkv, D, P, 8)
    ids = [store.put(g, rand(rng, L, m, Hkv, D), rand(rng, L, m, Hkv, D))[0] for g, m in enumerate(ms)]
    pid = [ids[g] for g in req_prefix]
    pm = [ms[g] for g in req_prefix]
    # depth 0 everywhere: every layer is Eq. 2 over the request's own rows (= "no caching")
    res = oracle.stack(store, [0] * 3, pid, pm, offs, lens, q, k, v, 0.6)
    for l in range(L):
        ref = brute_attend([], 0, [-1] * 3, offs, lens, q[l].tolist(), k[l].tolist(), v[l].tolist(),
                           0.6, Hq, Hkv)
        for (i, h, a), (ro, rl) in ref.items():
            np.testing.assert_allclose(res[l][0][offs[i] + a, h], ro, rtol=1e-11, atol=1e-12)
    # depth L everywhere: every layer is `attend`; prefix rows are not computed
    res = oracle.stack(store, [L] * 3, pid, pm, offs, lens, q, k, v, 0.6)
    for l in range(L):
        o, lse = oracle.attend(store, l, pid, [o_ + m for o_, m in zip(offs, pm)], ns, q[l], k[l], v[l], 0.6)
        assert np.array_equal(res[l][0], o) and np.array_equal(res[l][1], lse)
        assert np.isneginf(res[l][1][offs[0]:offs[0] + pm[0]]).all()
    # mixed depths: layer l of request i is reuse iff l < depth_i
    depth = [1, 3, 2]
    res = oracle.stack(store, depth, pid, pm, offs, lens, q, k, v, 0.6)
    for l in range(L):
        for i in range(3):
            first_prefix_row = res[l][1][offs[i]]
            assert np.isneginf(first_prefix_row).all() == (l < depth[i])


def test_cached_equal_to_fresh_prefix_makes_depth_irrelevant():
    """If the cached prefix KVs equal the request's own prefix KVs (the
    causal-model situation the paper describes, and layer 1 of a DLM), reuse is
    exact: suffix rows of `attend` == suffix rows of `attend_full`."""
    rng = np.random.default_rng(23)
    L, Hq, Hkv, D, P, m = 2, 4, 2, 8, 16, 19
    ns = [5, 2]
    offs, lens, q, k, v = _stack_inputs(rng, L, Hq, Hkv, D, [m], [0, 0], ns)
    for l in range(L):                  # both requests carry the same prefix KVs
        k[l][offs[1]:offs[1] + m] = k[l][offs[0]:offs[0] + m]
        v[l][offs[1]:offs[1] + m] = v[l][offs[0]:offs[0] + m]
    store = oracle.PagedPrefixStore(L, Hkv, D, P, 4)
    pid, _, _ = store.put(9, np.stack([k[l][:m] for l in range(L)]), np.stack([v[l][:m] for l in range(L)]))
    base = oracle.stack(store, [0, 0], [pid] * 2, [m] * 2, offs, lens, q, k, v, 0.8)
    for depth in ([1, 2], [2, 0], [2, 2]):
        res = oracle.stack(store, depth, [pid] * 2, [m] * 2, offs, lens, q, k, v, 0.8)
        for l in range(L):
            for i in range(2):
                s = slice(offs[i] + m, offs[i] + lens[i])
                np.testing.assert_allclose(res[l][0][s], base[l][0][s], rtol=1e-12, atol=1e-14)
                np.testing.assert_allclose(res[l][1][s], base[l][1][s], rtol=1e-12)


def test_dropping_keys_perturbation_bound():
    """Appendix B, Lemma 1: attention over a subset of the keys (renormalised)
    differs from attention over all keys by at most 2 * max|v| * rho, rho being
    the softmax mass of the dropped keys."""
    rng = np.random.default_rng(29)
    nq, m, n, D = 6, 30, 9, 8
    q, k, v = rand(rng, nq, 1, D), rand(rng, m + n, 1, D), rand(rng, m + n, 1, D)
    full, lse_full = oracle.attention(q, k, v, 0.5)
    pre, lse_pre = oracle.attention(q, k[:m], v[:m], 0.5)
    rho = 1.0 - np.exp(lse_pre - lse_full)                 # mass on the n dropped keys
    bv = np.linalg.norm(v[:, 0, :], axis=1).max()
    gap = np.linalg.norm(full[:, 0] - pre[:, 0], axis=1)
    assert (gap <= 2 * bv * rho[:, 0] + 1e-12).all()
    assert (rho > 0).all() and (rho < 1).all()


def test_argument_errors():
    with pytest.raises(oracle.InvalidArgument):
        oracle.attention(np.zeros((1, 3, 4)), np.zeros((1, 2, 4)), np.zeros((1, 2, 4)), 1.0)
    with pytest.raises(oracle.InvalidArgument):
        oracle.attend_full([0], [5], np.zeros((4, 1, 4)), np.zeros((4, 1, 4)), np.zeros((4, 1, 4)), 1.0)
