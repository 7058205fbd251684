"""Pins for the oracle's reuse-depth rule and paged FIFO prefix store (CPU)."""
import os

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
from paper_2606_07571_b200 import workloads

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _depth_cases():
    with open(os.path.join(GOLDEN, "depth_cases.txt")) as f:
        return [tuple(int(x) for x in ln.split()) for ln in f if ln.strip() and not ln.startswith("#")]


def test_depth_rule_hand_cases():
    """An identity table turns the rule into its ratio-bin index."""
    table = list(range(101))
    for m, n, idx in _depth_cases():
        assert oracle.reuse_depth([m], [n], table, 1000)[0] == idx
    # clamped into [0, L]; no prefix -> 0
    assert oracle.reuse_depth([99, 0, 50], [1, 10, 50], table, 32).tolist() == [32, 0, 32]
    assert oracle.reuse_depth([10], [10], [-3] * 101, 32)[0] == 0
    with pytest.raises(oracle.InvalidArgument):
        oracle.reuse_depth([1], [1], list(range(100)), 32)
    with pytest.raises(oracle.InvalidArgument):
        oracle.reuse_depth([1], [-1], table, 32)


@given(st.integers(1, 5000), st.integers(0, 5000), st.integers(1, 64))
@settings(max_examples=200, deadline=None)
def test_depth_rule_ranges_and_monotonicity(m, n, L):
    t = workloads.standin_depth_table(L)
    d = oracle.reuse_depth([m, m + 1, m], [n, n, n + 1], t, L)
    assert 1 <= d[0] <= L                      # a shared prefix always allows layer 1
    assert d[1] >= d[0] >= d[2]                # more prefix -> deeper; more suffix -> shallower
    # the bin index is the floor of 100 r, never beyond the true ratio
    idx = oracle.reuse_depth([m], [n], list(range(101)), 1000)[0]
    assert idx * (m + n) <= 100 * m < (idx + 1) * (m + n)


def test_standin_table_shape():
    t = workloads.standin_depth_table(32)
    assert len(t) == 101 and t[100] == 32 and t[85] == 16 and t[0] == 1
    assert (np.diff(t) >= 0).all() and t.min() >= 1


# -- store: an independent trace simulation -----------------------------------

class ModelStore:
    """Deliberately different bookkeeping: a flat owner array plus an explicit
    arrival list, re-deriving the free queue by replaying events."""

    def __init__(self, num_pages, P, order):
        self.P = P
        self.queue = list(order)
        self.live = []          # [key, m, pages] in arrival order
        self.count = 0

    def put(self, key, m):
        for e in self.live:
            if e[0] == key:
                return ("hit", e[3], e[2]) if e[1] == m else ("invalid",)
        need = -(-m // self.P)
        if need > len(self.queue) + sum(len(e[2]) for e in self.live):
            return ("nomem",)
        while len(self.queue) < need:
            self.queue.extend(self.live.pop(0)[2])
        pages, self.queue = self.queue[:need], self.queue[need:]
        self.live.append([key, m, pages, self.count])
        self.count += 1
        return ("miss", self.count - 1, pages)


@given(st.lists(st.tuples(st.integers(0, 6), st.integers(1, 70)), min_size=1, max_size=40),
       st.integers(1, 12), st.integers(0, 3))
@settings(max_examples=150, deadline=None)
def test_store_traces_against_model(trace, num_pages, seed):
    P, L, H, D = 8, 1, 1, 2
    order = list(range(num_pages)) if seed == 0 else np.random.default_rng(seed).permutation(num_pages).tolist()
    real = oracle.PagedPrefixStore(L, H, D, P, num_pages, free_order=order)
    model = ModelStore(num_pages, P, order)
    key_len = {}
    for key, m in trace:
        m = key_len.setdefault(key, m) if seed % 2 == 0 else m
        want = model.put(key, m)
        kv = np.full((L, m, H, D), float(key))
        if want[0] == "invalid":
            with pytest.raises(oracle.InvalidArgument):
                real.put(key, kv, kv)
        elif want[0] == "nomem":
            with pytest.raises(oracle.OutOfPages):
                real.put(key, kv, kv)
        else:
            pid, hit, pages = real.put(key, kv, kv)
            assert (hit, pid, pages) == (want[0] == "hit", want[1], want[2])
        # conservation: every page is free or owned exactly once
        owned = [p for pid in real.entries for p in real.pages(pid)]
        assert sorted(owned + list(real.free[0])) == list(range(num_pages))
        # live keys agree, evicted keys are gone
        live = {e[0] for e in model.live}
        for k in range(7):
            if k in live:
                pid, mm = real.lookup(k)
                kk, _ = real.prefix_kv(0, pid)
                assert kk.shape[0] == mm and (kk == float(k)).all()
            else:
                with pytest.raises(oracle.NotFound):
                    real.lookup(k)


def test_store_fifo_not_lru_and_ids_never_reused():
    s = oracle.PagedPrefixStore(1, 1, 2, 16, 4)
    kv = lambda m: np.ones((1, m, 1, 2))
    a, _, pa = s.put(10, kv(32), kv(32))       # pages 0,1
    b, _, pb = s.put(11, kv(16), kv(16))       # page 2
    assert (a, b, pa, pb) == (0, 1, [0, 1], [2])
    assert s.put(10, kv(32), kv(32))[1] is True            # a hit does not refresh age
    c, hit, pc = s.put(12, kv(32), kv(32))     # needs 2, 1 free -> evict oldest (key 10)
    assert (c, hit, pc) == (2, False, [3, 0])  # free queue was [3] + evicted [0, 1]
    with pytest.raises(oracle.NotFound):
        s.lookup(10)
    with pytest.raises(oracle.NotFound):
        s.pages(a)
    d, _, pd = s.put(10, kv(16), kv(16))       # re-put after eviction: new id, next free page
    assert (d, pd) == (3, [1])
    with pytest.raises(oracle.OutOfPages):
        s.put(13, kv(16 * 5), kv(16 * 5))
    with pytest.raises(oracle.InvalidArgument):
        s.put(11, kv(17), kv(17))
    with pytest.raises(oracle.InvalidArgument):
        oracle.PagedPrefixStore(1, 1, 2, 16, 4, free_order=[0, 1, 1, 2])


# -- store with per-layer page lists (a kept deep-layer prefix owns layers first_layer .. L-1 only) ------

class LayeredModel:
    """Independent model of the per-layer store: an owner array per layer (which prefix holds each page)
    and, per layer, the order in which pages became free, replayed from the events."""

    def __init__(self, L, caps, P, order):
        self.L, self.P = L, P
        self.caps = caps
        self.freed_at = [{p: i for i, p in enumerate(q for q in order if q < caps[l])} for l in range(L)]
        self.tick = len(order)
        self.live = []          # [key, m, first, {layer: pages}, id]
        self.count = 0

    def free_list(self, l):
        return [p for p, _ in sorted(self.freed_at[l].items(), key=lambda kv: kv[1])]

    def insert(self, key, m, first):
        for e in self.live:
            if e[0] == key:
                return ("hit", e[4], e[3][first]) if (e[1], e[2]) == (m, first) else ("invalid",)
        need = -(-m // self.P)
        if any(need > self.caps[l] for l in range(first, self.L)):
            return ("nomem",)
        while any(len(self.freed_at[l]) < need for l in range(first, self.L)):
            old = self.live.pop(0)
            for l, pages in old[3].items():
                for p in pages:
                    self.freed_at[l][p] = self.tick
                    self.tick += 1
        got = {}
        for l in range(first, self.L):
            got[l] = self.free_list(l)[:need]
            for p in got[l]:
                del self.freed_at[l][p]
        self.live.append([key, m, first, got, self.count])
        self.count += 1
        return ("miss", self.count - 1, got[first])


@given(st.lists(st.tuples(st.integers(0, 7), st.integers(1, 40), st.integers(0, 2)), min_size=1, max_size=40),
       st.integers(2, 10), st.integers(0, 3), st.booleans())
@settings(max_examples=150, deadline=None)
def test_layered_store_traces_against_model(trace, num_pages, seed, shrink_shallow):
    P, L, H, D = 8, 3, 1, 2
    order = list(range(num_pages)) if seed == 0 else np.random.default_rng(seed).permutation(num_pages).tolist()
    caps = [max(1, num_pages // 2), max(1, (3 * num_pages) // 4), num_pages] if shrink_shallow else [num_pages] * L
    real = oracle.PagedPrefixStore(L, H, D, P, num_pages, free_order=order, layer_pages=caps)
    model = LayeredModel(L, caps, P, order)
    for key, m, first in trace:
        want = model.insert(key, m, first)
        if want[0] == "invalid":
            with pytest.raises(oracle.InvalidArgument):
                real.reserve(key, m, first)
        elif want[0] == "nomem":
            with pytest.raises(oracle.OutOfPages):
                real.reserve(key, m, first)
        else:
            pid, hit, pages = real.reserve(key, m, first)
            assert (hit, pid, pages) == (want[0] == "hit", want[1], want[2])
        # per layer: every page below the layer's capacity is free or owned exactly once, and the
        # free queue has the model's order
        for l in range(L):
            owned = [p for e in model.live if l in e[3] for p in e[3][l]]
            assert sorted(owned + list(real.free[l])) == list(range(caps[l]))
            assert list(real.free[l]) == model.free_list(l)
        for e in model.live:
            for l in range(L):
                if l in e[3]:
                    assert real.pages(e[4], l) == e[3][l]
                else:
                    with pytest.raises(oracle.InvalidArgument):
                        real.pages(e[4], l)


def test_layered_store_hand_sequence():
    """Three layers of four pages.  A full-depth prefix, then a deep-only one (layers 1-2), then a
    full-depth one that no longer fits layer 1 without evicting the oldest prefix: FIFO order is by
    insertion, whatever layers a prefix owns, and the lists of the third prefix differ by layer."""
    s = oracle.PagedPrefixStore(3, 1, 2, 16, 4)
    a, _, pa = s.reserve(1, 32)                  # pages 0, 1 in every layer
    b, _, pb = s.reserve(2, 32, first_layer=1)   # pages 2, 3 in layers 1 and 2; layer 0 untouched
    assert (a, pa, b, pb) == (0, [0, 1], 1, [2, 3])
    assert [list(q) for q in s.free] == [[2, 3], [], []]
    with pytest.raises(oracle.InvalidArgument):
        s.pages(b, 0)
    with pytest.raises(oracle.InvalidArgument):
        s.prefix_kv(0, b)
    assert s.reserve(2, 32, first_layer=1)[1] is True
    with pytest.raises(oracle.InvalidArgument):
        s.reserve(2, 32, first_layer=2)          # same key, another first layer
    c, hit, pc = s.reserve(3, 32)                # layers 1, 2 are full: the oldest prefix (key 1) goes
    assert (c, hit) == (2, False)
    assert [s.pages(c, l) for l in range(3)] == [[2, 3], [0, 1], [0, 1]]
    assert [list(q) for q in s.free] == [[0, 1], [], []]
    with pytest.raises(oracle.NotFound):
        s.lookup(1)
    # values written to one layer are read back from that layer only
    kv = np.arange(32 * 2, dtype=np.float64).reshape(32, 1, 2)
    s.update_layer(b, 2, kv, kv + 1)
    k2, v2 = s.prefix_kv(2, b)
    assert (k2 == kv).all() and (v2 == kv + 1).all()
    k1, _ = s.prefix_kv(1, b)
    assert (k1 == 0).all()
    with pytest.raises(oracle.InvalidArgument):
        s.update_layer(b, 0, kv, kv)
    with pytest.raises(oracle.InvalidArgument):
        oracle.PagedPrefixStore(3, 1, 2, 16, 4, layer_pages=[4, 5, 4])
    small = oracle.PagedPrefixStore(2, 1, 2, 16, 4, layer_pages=[1, 4])
    with pytest.raises(oracle.OutOfPages):
        small.reserve(9, 32)                      # two pages do not fit layer 0's single page
    assert small.reserve(9, 32, first_layer=1)[2] == [0, 1]


def test_workload_recipes_are_deterministic_and_shaped():
    w = workloads.config4()
    w2 = workloads.config4()
    assert w.prefix_lens == w2.prefix_lens and w.suffix_lens == w2.suffix_lens
    assert len(w.prefix_lens) == 8 and w.num_requests == 256
    assert all(512 <= m <= 4096 for m in w.prefix_lens)
    assert all(32 <= n <= 1024 for n in w.suffix_lens)
    assert w.req_prefix == sorted(w.req_prefix)
    w3 = workloads.config3()
    assert w3.num_requests == 64 and all(64 <= n <= 512 for n in w3.suffix_lens)
    q, k, v = workloads.draw_full_qkv(workloads.config1())
    q2, _, _ = workloads.draw_full_qkv(workloads.config1())
    assert q.shape == (4 * 96, 4, 64) and (q == q2).all()
    small = workloads.scaled_down(w, num_layers=2, max_requests=12, prefix_div=16, suffix_div=8)
    assert small.num_requests == 12 and small.req_prefix == sorted(small.req_prefix)


def test_prefix_key_is_xxh64_of_the_token_ids():
    """Pins for the oracle's hash: the published XXH64 digests of the empty input and of "a", and the
    xxhash library (a third party's implementation) on inputs of every tail length."""
    xxhash = pytest.importorskip("xxhash")
    assert oracle.xxh64(b"") == 0xEF46DB3751D8E999
    assert oracle.xxh64(b"a") == 0xD24EC4F1A98C6E5B
    rng = np.random.default_rng(0)
    for n in list(range(0, 80)) + [255, 256, 1000]:
        data = rng.integers(0, 256, n, dtype=np.uint8).tobytes()
        assert oracle.xxh64(data) == xxhash.xxh64(data).intdigest(), n
        assert oracle.xxh64(data, 12345) == xxhash.xxh64(data, seed=12345).intdigest(), n
    toks = [1, 2, 3, -1, 2 ** 31 - 1]
    assert oracle.prefix_key(toks) == xxhash.xxh64(np.asarray(toks, dtype="<i4").tobytes()).intdigest()


def test_project_kv_is_eq1():
    """k = W^K h, v = W^V h per token and layer: scalar loops, selector weights, linearity."""
    rng = np.random.default_rng(4)
    L, m, d, Hkv, D = 2, 5, 7, 2, 3
    h = rng.standard_normal((L, m, d))
    wk, wv = rng.standard_normal((L, Hkv * D, d)), rng.standard_normal((L, Hkv * D, d))
    k, v = oracle.project_kv(h, wk, wv, Hkv, D)
    assert k.shape == v.shape == (L, m, Hkv, D)
    for l in range(L):
        for t in range(m):
            for hd in range(Hkv):
                for j in range(D):
                    o = hd * D + j
                    assert abs(k[l, t, hd, j] - sum(wk[l, o, c] * h[l, t, c] for c in range(d))) < 1e-12
                    assert abs(v[l, t, hd, j] - sum(wv[l, o, c] * h[l, t, c] for c in range(d))) < 1e-12
    # a weight row that is a unit vector copies that hidden component
    sel = np.zeros((L, Hkv * D, d))
    for o in range(Hkv * D):
        sel[:, o, o % d] = 1.0
    k2, _ = oracle.project_kv(h, sel, sel, Hkv, D)
    for o in range(Hkv * D):
        assert np.array_equal(k2[:, :, o // D, o % D], h[:, :, o % d])
    # linear in the hidden states
    h2 = rng.standard_normal((L, m, d))
    ka, va = oracle.project_kv(2.0 * h + h2, wk, wv, Hkv, D)
    kb, vb = oracle.project_kv(h2, wk, wv, Hkv, D)
    assert np.allclose(ka, 2.0 * k + kb, atol=1e-12) and np.allclose(va, 2.0 * v + vb, atol=1e-12)
    with pytest.raises(oracle.InvalidArgument):
        oracle.project_kv(h, wk[:, :-1], wv, Hkv, D)
