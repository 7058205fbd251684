"""Pins for the oracle's deep-layer reuse with periodic refresh (Eq. 5), CPU only."""
import numpy as np
import pytest

import oracle


def test_refresh_steps_enumerated():
    """Eq. 5: step t recomputes iff (t - 1) mod Delta = 0.  For Delta = 16 and 64 steps that is
    t = 1, 17, 33, 49 (written out by hand); Delta = 1 refreshes every step."""
    assert [t for t in range(1, 65) if oracle.is_refresh_step(t, 16)] == [1, 17, 33, 49]
    assert all(oracle.is_refresh_step(t, 1) for t in range(1, 20))
    assert [t for t in range(1, 12) if oracle.is_refresh_step(t, 5)] == [1, 6, 11]
    with pytest.raises(oracle.InvalidArgument):
        oracle.is_refresh_step(0, 16)
    with pytest.raises(oracle.InvalidArgument):
        oracle.is_refresh_step(1, 0)


def _softmax_rows(qr, ks, vs, hk, scale):
    """Scalar loops: one query row over an explicit key list (written separately from the oracle)."""
    s = [scale * sum(float(qr[d]) * float(ks[j][hk][d]) for d in range(len(qr))) for j in range(len(ks))]
    mx = max(s)
    w = [np.exp(x - mx) for x in s]
    z = sum(w)
    return np.array([sum(w[j] * float(vs[j][hk][d]) for j in range(len(ks))) / z for d in range(len(qr))])


def _steps(rng, S, rows, Hq, Hkv, D):
    return [(rng.standard_normal((rows, Hq, D)), rng.standard_normal((rows, Hkv, D)),
             rng.standard_normal((rows, Hkv, D))) for _ in range(S)]


def _run(store_args, L, depth, shared_kv, m, N, S, delta, steps, scale):
    """Drive attend_step over S steps and all layers; returns per step, per layer outputs."""
    st = oracle.PagedPrefixStore(*store_args)
    sid, _, _ = st.put(7, *shared_kv)
    pid, _, _ = st.reserve(8, m)
    outs = []
    for t in range(1, S + 1):
        q, k, v = steps[t - 1]
        outs.append([oracle.attend_step(st, l, t, delta, [depth], [sid], [pid], [0], [N], q, k, v, scale)[0]
                     for l in range(L)])
    return outs


def test_attend_step_against_closed_form_brute_force():
    """The prefix KVs a deep layer uses at step t are those of step 1 + Delta * floor((t - 1) / Delta)
    (Eq. 5 unrolled); a shallow layer uses the shared cached ones (Eq. 4).  Brute force by
    concatenating exactly those rows, with scalar loops."""
    rng = np.random.default_rng(5)
    L, Hq, Hkv, D, m, n, S, delta, depth = 3, 2, 1, 4, 5, 3, 7, 3, 1
    N = m + n
    scale = 0.5
    shared = (rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D)))
    steps = _steps(rng, S, N, Hq, Hkv, D)
    outs = _run((L, Hkv, D, 4, 8), L, depth, shared, m, N, S, delta, steps, scale)
    for t in range(1, S + 1):
        q, k, v = steps[t - 1]
        src = 1 + delta * ((t - 1) // delta)               # the step whose prefix KVs are in use
        for l in range(L):
            if l < depth:
                kp, vp = shared[0][l], shared[1][l]
                rows = range(m, N)
            elif src == t:
                kp, vp = k[:m], v[:m]
                rows = range(0, N)                         # a refresh step recomputes every row
            else:
                kp, vp = steps[src - 1][1][:m], steps[src - 1][2][:m]
                rows = range(m, N)
            ks = list(kp) + list(k[m:])
            vs = list(vp) + list(v[m:])
            for a in rows:
                for h in range(Hq):
                    ref = _softmax_rows(q[a, h], ks, vs, h // (Hq // Hkv), scale)
                    assert np.allclose(outs[t - 1][l][a, h], ref, atol=1e-12), (t, l, a, h)
            if rows.start == m:
                assert np.all(outs[t - 1][l][:m] == 0)     # prefix rows are not computed under reuse


def test_delta_one_is_full_recompute_every_step():
    rng = np.random.default_rng(6)
    L, Hq, Hkv, D, m, n, S = 2, 2, 2, 8, 6, 4, 4
    N = m + n
    shared = (rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D)))
    steps = _steps(rng, S, N, Hq, Hkv, D)
    outs = _run((L, Hkv, D, 4, 8), L, 0, shared, m, N, S, 1, steps, 0.3)
    for t in range(S):
        q, k, v = steps[t]
        full, _ = oracle.attend_full([0], [N], q, k, v, 0.3)
        for l in range(L):
            assert np.array_equal(outs[t][l], full)


def test_constant_prefix_kv_makes_delta_irrelevant():
    """If the prefix rows of K and V do not change over the steps, reusing them equals recomputing
    them: the suffix rows then do not depend on Delta (the autoregressive special case)."""
    rng = np.random.default_rng(7)
    L, Hq, Hkv, D, m, n, S = 2, 4, 2, 8, 7, 5, 6
    N = m + n
    shared = (rng.standard_normal((L, m, Hkv, D)), rng.standard_normal((L, m, Hkv, D)))
    steps = _steps(rng, S, N, Hq, Hkv, D)
    for t in range(1, S):
        steps[t][1][:m] = steps[0][1][:m]
        steps[t][2][:m] = steps[0][2][:m]
    a = _run((L, Hkv, D, 4, 8), L, 0, shared, m, N, S, 1, steps, 0.4)
    b = _run((L, Hkv, D, 4, 8), L, 0, shared, m, N, S, 4, steps, 0.4)
    for t in range(S):
        for l in range(L):
            assert np.allclose(a[t][l][m:], b[t][l][m:], atol=1e-12)


def test_reserve_and_update_layer_follow_the_store_rules():
    st = oracle.PagedPrefixStore(2, 1, 2, 4, 3)
    pid, hit, pages = st.reserve(1, 6)
    assert (hit, pages) == (False, [0, 1])
    k = np.arange(12, dtype=np.float64).reshape(6, 1, 2)
    st.update_layer(pid, 1, k, -k)
    k1, v1 = st.prefix_kv(1, pid)
    assert np.array_equal(k1, k) and np.array_equal(v1, -k)
    k0, _ = st.prefix_kv(0, pid)
    assert np.all(k0 == 0)                                   # the other layer is untouched
    with pytest.raises(oracle.InvalidArgument):
        st.update_layer(pid, 2, k, k)
    with pytest.raises(oracle.InvalidArgument):
        st.update_layer(pid, 0, k[:5], k[:5])
    st.reserve(2, 8)                                         # evicts the first entry (FIFO)
    with pytest.raises(oracle.NotFound):
        st.update_layer(pid, 0, k, k)
