"""Pins for the oracle's profiler pieces (Eq. 3 similarity, depth under a threshold, table), CPU only."""
import math

import numpy as np
import pytest

import oracle


def _store_with(k, v, page_size=4, order=None):
    L, m, Hkv, D = k.shape
    npages = (m + page_size - 1) // page_size + 2
    st = oracle.PagedPrefixStore(L, Hkv, D, page_size, npages, free_order=order)
    pid, _, _ = st.put(1, k, v)
    return st, pid


def test_similarity_closed_forms():
    rng = np.random.default_rng(1)
    L, m, Hkv, D = 3, 9, 2, 4
    k, v = rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D))
    st, pid = _store_with(k, v, order=[3, 0, 4, 2, 1])
    assert np.allclose(oracle.kv_similarity(st, pid, k, v), 1.0, atol=1e-15)
    assert np.allclose(oracle.kv_similarity(st, pid, -k, -v), -1.0, atol=1e-15)
    assert np.allclose(oracle.kv_similarity(st, pid, 3.5 * k, 3.5 * v), 1.0, atol=1e-15)     # scale-free
    # reference = a * cached + b * (unit-norm-matched part orthogonal to cached): cos = a / sqrt(a^2 + b^2)
    a, b = 0.8, 0.6
    kr, vr = np.empty_like(k), np.empty_like(v)
    for l in range(L):
        c = np.concatenate([k[l].ravel(), v[l].ravel()])
        z = rng.standard_normal(c.shape)
        z -= (z @ c) / (c @ c) * c
        z *= np.linalg.norm(c) / np.linalg.norm(z)
        r = a * c + b * z
        kr[l] = r[:k[l].size].reshape(k[l].shape)
        vr[l] = r[k[l].size:].reshape(v[l].shape)
    assert np.allclose(oracle.kv_similarity(st, pid, kr, vr), a / math.hypot(a, b), atol=1e-12)
    # K and V count as ONE vector: flipping only V changes the value to (|K|^2 - |V|^2) / (|K|^2 + |V|^2)
    sim = oracle.kv_similarity(st, pid, k, -v)
    for l in range(L):
        kk, vv = float((k[l] ** 2).sum()), float((v[l] ** 2).sum())
        assert abs(sim[l] - (kk - vv) / (kk + vv)) < 1e-12
    assert np.all(oracle.kv_similarity(st, pid, np.zeros_like(k), np.zeros_like(v)) == 0.0)
    with pytest.raises(oracle.InvalidArgument):
        oracle.kv_similarity(st, pid, k[:, :-1], v[:, :-1])


def test_similarity_scalar_brute_force():
    rng = np.random.default_rng(2)
    L, m, Hkv, D = 2, 5, 1, 3
    k, v = rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D))
    kr, vr = rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D))
    st, pid = _store_with(k, v)
    sim = oracle.kv_similarity(st, pid, kr, vr)
    for l in range(L):
        dot = na = nb = 0.0
        for t in range(m):
            for d in range(D):
                for x, y in ((k[l, t, 0, d], kr[l, t, 0, d]), (v[l, t, 0, d], vr[l, t, 0, d])):
                    dot += x * y
                    na += x * x
                    nb += y * y
        assert abs(sim[l] - dot / math.sqrt(na * nb)) < 1e-13


def test_depth_under_threshold_hand_cases():
    """b counts the leading layers with sim >= tau (Sec. 4.2: 'all layers from 1 to b')."""
    assert oracle.depth_from_similarity([1.0, 0.99, 0.98, 0.96, 0.99], 0.97) == 3   # a later 0.99 does not count
    assert oracle.depth_from_similarity([1.0, 0.97, 0.97], 0.97) == 3               # >= is inclusive
    assert oracle.depth_from_similarity([0.5, 1.0], 0.97) == 0
    assert oracle.depth_from_similarity([], 0.97) == 0
    assert oracle.depth_from_similarity([1.0, float("nan"), 1.0], 0.97) == 1


def test_table_from_profiled_depths_hand_case():
    """Per ratio bin the floored mean of the b_i; gaps take the nearest filled bin below."""
    idx = [85, 85, 85, 90, 90, 100, 3]
    b = [16, 17, 16, 20, 23, 32, 1]
    t = oracle.build_depth_table(idx, b, 32)
    assert len(t) == 101
    assert t[85] == 16 and t[90] == 21 and t[100] == 32 and t[3] == 1       # floor(49/3), floor(43/2)
    assert t[0] == 1 and t[2] == 1 and t[4] == 1 and t[84] == 1 and t[86] == 16 and t[99] == 21
    assert oracle.build_depth_table([], [], 32) == [1] * 101
    assert oracle.build_depth_table([], [], 0) == [0] * 101
    with pytest.raises(oracle.InvalidArgument):
        oracle.build_depth_table([101], [1], 32)
    with pytest.raises(oracle.InvalidArgument):
        oracle.build_depth_table([5], [33], 32)


def test_similarity_distance_bound():
    """1 - cos(a, b) <= |a - b|^2 / (2 |a| |b|), with equality when |a| = |b| (the paper's auxiliary
    lemma on cosine similarity and distance): an inequality and an identity the oracle's similarity
    must satisfy, computed here from norms of differences only."""
    rng = np.random.default_rng(3)
    L, m, Hkv, D = 4, 11, 2, 8
    k, v = rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D))
    st, pid = _store_with(k, v)
    kr = k + 0.3 * rng.standard_normal(k.shape)
    vr = 1.7 * v + 0.1 * rng.standard_normal(v.shape)
    sim = oracle.kv_similarity(st, pid, kr, vr)
    for l in range(L):
        a = np.concatenate([k[l].ravel(), v[l].ravel()])
        b = np.concatenate([kr[l].ravel(), vr[l].ravel()])
        bound = np.linalg.norm(a - b) ** 2 / (2 * np.linalg.norm(a) * np.linalg.norm(b))
        assert 1 - sim[l] <= bound + 1e-12
        assert 1 - sim[l] > 0
    # equal norms: the bound is attained
    for l in range(L):
        a = np.concatenate([k[l].ravel(), v[l].ravel()])
        b = np.concatenate([kr[l].ravel(), vr[l].ravel()])
        s = np.linalg.norm(a) / np.linalg.norm(b)
        kr[l] *= s
        vr[l] *= s
    sim = oracle.kv_similarity(st, pid, kr, vr)
    for l in range(L):
        a = np.concatenate([k[l].ravel(), v[l].ravel()])
        b = np.concatenate([kr[l].ravel(), vr[l].ravel()])
        assert abs((1 - sim[l]) - np.linalg.norm(a - b) ** 2 / (2 * np.linalg.norm(a) * np.linalg.norm(b))) < 1e-12


def test_rope_rotate_pins():
    """The rotary rotation of keys that the projection may apply (the angles are an input): identity at
    angle 0, a quarter turn maps (a, b) to (-b, a), a scalar loop, norms of pairs, and the property the
    encoding exists for: <rot(q, p), rot(k, p')> depends on p - p' only."""
    rng = np.random.default_rng(8)
    m, H, D = 6, 3, 8
    x = rng.standard_normal((m, H, D))
    zero = np.zeros((m, D // 2))
    assert np.array_equal(oracle.rope_rotate(x, np.ones((m, D // 2)), zero), x)
    quarter = oracle.rope_rotate(x, zero, np.ones((m, D // 2)))
    assert np.allclose(quarter[..., :D // 2], -x[..., D // 2:]) and np.allclose(quarter[..., D // 2:], x[..., :D // 2])
    ang = rng.uniform(-3, 3, (m, D // 2))
    got = oracle.rope_rotate(x, np.cos(ang), np.sin(ang))
    for t in range(m):
        for h in range(H):
            for d in range(D // 2):
                a, b = x[t, h, d], x[t, h, d + D // 2]
                assert abs(got[t, h, d] - (a * math.cos(ang[t, d]) - b * math.sin(ang[t, d]))) < 1e-12
                assert abs(got[t, h, d + D // 2] - (b * math.cos(ang[t, d]) + a * math.sin(ang[t, d]))) < 1e-12
                assert abs(math.hypot(got[t, h, d], got[t, h, d + D // 2]) - math.hypot(a, b)) < 1e-12
    # relative positions: angles pos * theta_d
    theta = 10000.0 ** (-np.arange(D // 2) / (D // 2))
    q, k = rng.standard_normal((1, 1, D)), rng.standard_normal((1, 1, D))

    def at(v, pos):
        return oracle.rope_rotate(v, np.cos(pos * theta)[None], np.sin(pos * theta)[None])[0, 0]

    base = at(q, 7.0) @ at(k, 3.0)
    assert abs(at(q, 104.0) @ at(k, 100.0) - base) < 1e-9
    assert abs(at(q, 4.0) @ k[0, 0] - base) < 1e-9
    assert abs(at(q, 8.0) @ at(k, 3.0) - base) > 1e-3          # another difference, another value
    with pytest.raises(oracle.InvalidArgument):
        oracle.rope_rotate(x, zero[:, :-1], zero[:, :-1])
    # project_kv applies it to the keys only
    L, d = 1, 5
    hdn = rng.standard_normal((L, m, d))
    wk, wv = rng.standard_normal((L, H * D, d)), rng.standard_normal((L, H * D, d))
    k0, v0 = oracle.project_kv(hdn, wk, wv, H, D)
    k1, v1 = oracle.project_kv(hdn, wk, wv, H, D, rope=(np.cos(ang), np.sin(ang)))
    assert np.array_equal(v0, v1) and np.allclose(k1[0], oracle.rope_rotate(k0[0], np.cos(ang), np.sin(ang)))
