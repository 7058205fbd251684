"""CPU tests of the C-ABI library: it builds, loads, exports every declared symbol, and its host
logic (store bookkeeping, FIFO eviction, depth rule) matches the oracle bit-exactly through a
host-only context.  No compute call is made here."""
import ctypes as C
import os
import re

import numpy as np
import pytest
from hypothesis import given, settings, strategies as st

import oracle
import __graft_entry__ as entry
from paper_2606_07571_b200 import binding, workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return binding.load_library()


def test_every_declared_symbol_is_exported(lib):
    hdr = open(os.path.join(ROOT, "include", "bicache.h")).read()
    declared = set(re.findall(r"\b(bicache_[a-z_]+)\s*\(", hdr))
    assert declared == set(binding.EXPORTED)
    for name in declared:
        assert hasattr(lib, name), name


def host_ctx(lib, L=2, Hq=4, Hkv=2, D=128, pages=8, dtype=binding.BF16, order=None):
    cfg = binding.Config(L, Hq, Hkv, D, 16, pages, dtype, -1)
    keep = None
    if order is not None:
        keep = np.ascontiguousarray(order, dtype=np.int32)
        cfg.initial_free_order = keep.ctypes.data_as(C.POINTER(C.c_int32))
    ctx = C.c_void_p()
    assert lib.bicache_create(C.byref(cfg), C.byref(ctx)) == binding.OK
    return ctx


def put(lib, ctx, key, m, cap=None):
    pid, hit = C.c_int32(-1), C.c_int32(-1)
    cap = (m + 15) // 16 if cap is None else cap
    pages = np.full(max(cap, 1), -1, dtype=np.int32)
    st_ = lib.bicache_put_prefix(ctx, C.c_uint64(key), m, None, None, m * 2 * 128, None, C.byref(pid), C.byref(hit),
                                 pages.ctypes.data_as(C.POINTER(C.c_int32)), cap)
    return st_, pid.value, hit.value, pages[:cap].tolist()


def test_sizes_and_create_errors(lib):
    cfg = binding.Config(32, 32, 32, 128, 16, 128, binding.BF16, -1)
    assert lib.bicache_pool_bytes(C.byref(cfg)) == 32 * 128 * 32 * 16 * 128 * 2
    assert lib.bicache_workspace_bytes(C.byref(cfg), 4096, 16) > 0
    ctx = C.c_void_p()
    bad = binding.Config(32, 32, 5, 128, 16, 128, binding.BF16, -1)        # Hq % Hkv != 0
    assert lib.bicache_create(C.byref(bad), C.byref(ctx)) == binding.ERR_INVALID
    bad = binding.Config(32, 32, 32, 128, 32, 128, binding.BF16, -1)       # page size
    assert lib.bicache_create(C.byref(bad), C.byref(ctx)) == binding.ERR_UNSUPPORTED
    bad = binding.Config(32, 32, 32, 128, 16, 128, 7, -1)                  # dtype
    assert lib.bicache_create(C.byref(bad), C.byref(ctx)) == binding.ERR_UNSUPPORTED
    order = np.array([0, 1, 1, 2], dtype=np.int32)
    bad = binding.Config(1, 1, 1, 128, 16, 4, binding.BF16, -1)
    bad.initial_free_order = order.ctypes.data_as(C.POINTER(C.c_int32))
    assert lib.bicache_create(C.byref(bad), C.byref(ctx)) == binding.ERR_INVALID
    dev = binding.Config(1, 1, 1, 128, 16, 4, binding.BF16, 0)             # device context needs buffers
    assert lib.bicache_create(C.byref(dev), C.byref(ctx)) == binding.ERR_INVALID


def test_depth_rule_matches_oracle(lib):
    ctx = host_ctx(lib, L=32, Hq=32, Hkv=32, pages=4)
    m = np.array([2048, 85, 1, 5, 0, 1024, 512], dtype=np.int32)
    n = np.array([362, 15, 1000, 0, 9, 256, 1024], dtype=np.int32)
    out = np.zeros(7, dtype=np.int32)
    p = lambda a: a.ctypes.data_as(C.POINTER(C.c_int32))
    assert lib.bicache_reuse_depth(ctx, 7, p(m), p(n), p(out)) == binding.ERR_INVALID     # no table yet
    t = workloads.standin_depth_table(32)
    assert lib.bicache_set_depth_table(ctx, p(t), 100) == binding.ERR_INVALID
    assert lib.bicache_set_depth_table(ctx, p(t), 101) == binding.OK
    assert lib.bicache_reuse_depth(ctx, 7, p(m), p(n), p(out)) == binding.OK
    assert out.tolist() == oracle.reuse_depth(m, n, t, 32).tolist()
    ident = np.arange(101, dtype=np.int32)
    lib.bicache_set_depth_table(ctx, p(ident), 101)
    lib.bicache_reuse_depth(ctx, 7, p(m), p(n), p(out))
    assert out.tolist() == [32, 32, 0, 32, 0, 32, 32] and oracle.reuse_depth(m, n, ident, 32).tolist() == out.tolist()
    n[2] = -1
    assert lib.bicache_reuse_depth(ctx, 7, p(m), p(n), p(out)) == binding.ERR_INVALID
    rng = np.random.default_rng(0)
    m = rng.integers(0, 20000, 4000).astype(np.int32)
    n = rng.integers(0, 20000, 4000).astype(np.int32)
    out = np.zeros(4000, dtype=np.int32)
    lib.bicache_set_depth_table(ctx, p(t), 101)
    assert lib.bicache_reuse_depth(ctx, 4000, p(m), p(n), p(out)) == binding.OK
    assert (out == oracle.reuse_depth(m, n, t, 32)).all()
    lib.bicache_destroy(ctx)


def test_store_fifo_sequence_matches_oracle(lib):
    ctx = host_ctx(lib, L=1, Hq=2, Hkv=2, pages=4)
    assert put(lib, ctx, 10, 32) == (binding.OK, 0, 0, [0, 1])
    assert put(lib, ctx, 11, 16) == (binding.OK, 1, 0, [2])
    assert put(lib, ctx, 10, 32) == (binding.OK, 0, 1, [0, 1])                  # hit, age not refreshed
    assert put(lib, ctx, 10, 31)[0] == binding.ERR_INVALID                     # same key, other length
    assert put(lib, ctx, 12, 32) == (binding.OK, 2, 0, [3, 0])                  # evicts key 10 (oldest)
    pid, m = C.c_int32(), C.c_int32()
    assert lib.bicache_lookup_prefix(ctx, C.c_uint64(10), C.byref(pid), C.byref(m)) == binding.ERR_NOTFOUND
    assert lib.bicache_lookup_prefix(ctx, C.c_uint64(12), C.byref(pid), C.byref(m)) == binding.OK
    assert (pid.value, m.value) == (2, 32)
    n = C.c_int32()
    assert lib.bicache_prefix_pages(ctx, 0, None, 0, C.byref(n)) == binding.ERR_NOTFOUND
    assert put(lib, ctx, 10, 16) == (binding.OK, 3, 0, [1])                     # new id after eviction
    assert put(lib, ctx, 13, 16 * 5)[0] == binding.ERR_NOMEM
    assert put(lib, ctx, 14, 0)[0] == binding.ERR_INVALID
    assert put(lib, ctx, 15, 32, cap=1)[0] == binding.ERR_INVALID               # pages_out too small, nothing changes
    assert lib.bicache_lookup_prefix(ctx, C.c_uint64(11), C.byref(pid), C.byref(m)) == binding.OK
    # attention on a host-only context is refused, not emulated
    z = np.zeros(1, dtype=np.int64)
    assert lib.bicache_attend_full(ctx, 0, 1, z.ctypes.data_as(C.POINTER(C.c_int64)),
                                   np.ones(1, np.int32).ctypes.data_as(C.POINTER(C.c_int32)),
                                   None, None, None, 256, 256, None, 256, None, C.c_float(1.0), None) \
        == binding.ERR_UNSUPPORTED
    lib.bicache_destroy(ctx)


@given(st.lists(st.tuples(st.integers(0, 6), st.integers(1, 130)), min_size=1, max_size=40),
       st.integers(1, 12), st.integers(0, 3))
@settings(max_examples=100, deadline=None)
def test_store_traces_match_oracle_bit_exactly(trace, num_pages, seed):
    entry.build()
    lib = binding.load_library()
    order = None if seed == 0 else workloads.shuffled_page_order(num_pages, seed)
    ctx = host_ctx(lib, L=1, Hq=1, Hkv=1, pages=num_pages, order=order)
    ref = oracle.PagedPrefixStore(1, 1, 2, 16, num_pages, free_order=order)
    for key, m in trace:
        kv = np.zeros((1, m, 1, 2))
        try:
            want = (binding.OK,) + tuple(ref.put(key, kv, kv))
        except oracle.InvalidArgument:
            want = (binding.ERR_INVALID,)
        except oracle.OutOfPages:
            want = (binding.ERR_NOMEM,)
        got = put(lib, ctx, key, m)
        if want[0] == binding.OK:
            assert got == (binding.OK, want[1], int(want[2]), want[3])
        else:
            assert got[0] == want[0]
        for k in range(7):
            pid, mm = C.c_int32(), C.c_int32()
            stt = lib.bicache_lookup_prefix(ctx, C.c_uint64(k), C.byref(pid), C.byref(mm))
            try:
                assert (stt, pid.value, mm.value) == (binding.OK,) + tuple(ref.lookup(k))
            except oracle.NotFound:
                assert stt == binding.ERR_NOTFOUND
    lib.bicache_destroy(ctx)


def test_refresh_rule_and_reserve_on_host_context(lib):
    """Eq. 5's step rule and the page bookkeeping of a reserved (per-request) prefix, no GPU."""
    for t in range(1, 70):
        for delta in (1, 3, 16):
            assert lib.bicache_is_refresh_step(t, delta) == int(oracle.is_refresh_step(t, delta))
    assert lib.bicache_is_refresh_step(0, 16) == -1
    assert lib.bicache_is_refresh_step(5, 0) == -1
    ctx = host_ctx(lib, L=2, Hq=2, Hkv=2, pages=4)
    ref = oracle.PagedPrefixStore(2, 2, 2, 16, 4)
    pid, hit = C.c_int32(-1), C.c_int32(-1)
    pages = np.full(8, -1, dtype=np.int32)
    pp = pages.ctypes.data_as(C.POINTER(C.c_int32))
    assert put(lib, ctx, 10, 20) == (binding.OK, 0, 0, [0, 1])
    ref.put(10, np.zeros((2, 20, 2, 2)), np.zeros((2, 20, 2, 2)))
    assert lib.bicache_reserve_prefix(ctx, C.c_uint64(77), 17, C.byref(pid), C.byref(hit), pp, 8) == binding.OK
    want = ref.reserve(77, 17)
    assert (pid.value, bool(hit.value), pages[:2].tolist()) == want
    assert lib.bicache_reserve_prefix(ctx, C.c_uint64(77), 17, C.byref(pid), C.byref(hit), pp, 8) == binding.OK
    assert hit.value == 1
    assert lib.bicache_reserve_prefix(ctx, C.c_uint64(77), 18, C.byref(pid), C.byref(hit), pp, 8) == binding.ERR_INVALID
    # update: id, layer and stride are checked on the host
    assert lib.bicache_update_prefix_layer(ctx, 99, 0, None, None, 256, None) == binding.ERR_NOTFOUND
    assert lib.bicache_update_prefix_layer(ctx, pid.value, 2, None, None, 256, None) == binding.ERR_INVALID
    assert lib.bicache_update_prefix_layer(ctx, pid.value, 0, None, None, 255, None) == binding.ERR_INVALID
    assert lib.bicache_update_prefix_layer(ctx, pid.value, 1, None, None, 256, None) == binding.OK   # host-only: no copy
    # a third prefix evicts the oldest (key 10), the reserved one stays
    assert put(lib, ctx, 11, 20)[0] == binding.OK
    m = C.c_int32()
    assert lib.bicache_lookup_prefix(ctx, C.c_uint64(10), C.byref(pid), C.byref(m)) == binding.ERR_NOTFOUND
    assert lib.bicache_lookup_prefix(ctx, C.c_uint64(77), C.byref(pid), C.byref(m)) == binding.OK
    # the step dispatch validates before it would launch
    i32 = lambda *a: np.asarray(a, dtype=np.int32).ctypes.data_as(C.POINTER(C.c_int32))
    i64 = lambda *a: np.asarray(a, dtype=np.int64).ctypes.data_as(C.POINTER(C.c_int64))
    args = (None, None, None, 256, 256, None, 256, None, C.c_float(1.0), None)
    assert lib.bicache_attend_step(ctx, 0, 0, 16, 1, i32(1), i32(-1), i32(-1), i64(0), i32(4), *args) == binding.ERR_INVALID
    assert lib.bicache_attend_step(ctx, 5, 1, 16, 1, i32(1), i32(-1), i32(-1), i64(0), i32(4), *args) == binding.ERR_INVALID
    assert lib.bicache_attend_step(ctx, 0, 2, 16, 1, i32(0), i32(-1), i32(55), i64(0), i32(40), *args) == binding.ERR_NOTFOUND
    assert lib.bicache_attend_step(ctx, 0, 2, 16, 1, i32(0), i32(-1), i32(pid.value), i64(0), i32(5), *args) \
        == binding.ERR_INVALID                                                   # shorter than its kept prefix
    lib.bicache_destroy(ctx)


def test_profiler_host_pieces_match_oracle(lib):
    """Depth under a threshold and the table from profiled depths: pure host functions."""
    from hypothesis import strategies as hst
    cases = [([1.0, 0.99, 0.98, 0.96, 0.99], 0.97), ([1.0, 0.97, 0.97], 0.97), ([0.5, 1.0], 0.97), ([], 0.5),
             ([1.0, float("nan"), 1.0], 0.97)]
    for sim, tau in cases:
        assert binding.depth_from_similarity(sim, tau) == oracle.depth_from_similarity(np.float32(sim), np.float32(tau))
    rng = np.random.default_rng(0)
    for _ in range(50):
        n = int(rng.integers(0, 60))
        L = int(rng.integers(0, 40))
        idx = rng.integers(0, 101, n).tolist()
        b = rng.integers(0, L + 1, n).tolist()
        assert binding.build_depth_table(idx, b, L) == oracle.build_depth_table(idx, b, L)
    with pytest.raises(binding.BiCacheError):
        binding.build_depth_table([101], [1], 32)
    with pytest.raises(binding.BiCacheError):
        binding.build_depth_table([5], [33], 32)
    ctx = host_ctx(lib)
    sim = np.zeros(2, dtype=np.float32)
    sp = sim.ctypes.data_as(C.POINTER(C.c_float))
    assert lib.bicache_prefix_similarity(ctx, 0, None, None, 1 << 20, sp, None) == binding.ERR_NOTFOUND
    assert put(lib, ctx, 1, 20)[0] == binding.OK
    assert lib.bicache_prefix_similarity(ctx, 0, None, None, 8, sp, None) == binding.ERR_INVALID        # stride < m rows
    assert lib.bicache_prefix_similarity(ctx, 0, None, None, 1 << 20, sp, None) == binding.ERR_UNSUPPORTED
    lib.bicache_destroy(ctx)


def test_hash_tokens_matches_oracle(lib):
    """k = h(p): the library's key of a token sequence against the oracle's XXH64, every tail length."""
    rng = np.random.default_rng(3)
    for n in list(range(0, 40)) + [127, 128, 129, 2048, 16385]:
        toks = rng.integers(-2 ** 31, 2 ** 31, n, dtype=np.int64).astype(np.int32)
        assert binding.hash_tokens(toks) == oracle.prefix_key(toks.tolist()), n
    assert binding.hash_tokens([]) == 0xEF46DB3751D8E999
    a, b = binding.hash_tokens([5, 6, 7]), binding.hash_tokens([5, 6, 8])
    assert a != b                                             # one token apart, another key
    # the key drives the store: same tokens hit, other tokens miss
    ctx = host_ctx(lib, L=1, Hq=1, Hkv=1, pages=4)
    assert put(lib, ctx, a, 16)[:3] == (binding.OK, 0, 0)
    assert put(lib, ctx, binding.hash_tokens([5, 6, 7]), 16)[:3] == (binding.OK, 0, 1)
    assert put(lib, ctx, b, 16)[:3] == (binding.OK, 1, 0)
    lib.bicache_destroy(ctx)


def test_projection_and_read_back_argument_checks_on_host_context(lib):
    """Eq. 1 into the store / layer read-back: ids, layers, shapes and strides are checked on the
    host, before anything would launch."""
    ctx = host_ctx(lib, L=2, Hq=4, Hkv=2, D=128, pages=4)
    pid, hit = C.c_int32(-1), C.c_int32(-1)
    pages = np.full(4, -1, dtype=np.int32)
    pp = pages.ctypes.data_as(C.POINTER(C.c_int32))
    assert lib.bicache_reserve_prefix(ctx, C.c_uint64(5), 40, C.byref(pid), C.byref(hit), pp, 4) == binding.OK
    proj = lib.bicache_project_prefix_layer
    assert proj(ctx, pid.value + 9, 0, None, 512, None, None, 512, None) == binding.ERR_NOTFOUND
    assert proj(ctx, pid.value, 2, None, 512, None, None, 512, None) == binding.ERR_INVALID      # layer
    assert proj(ctx, pid.value, 0, None, 512, None, None, 508, None) == binding.ERR_INVALID      # d_model % 8
    assert proj(ctx, pid.value, 0, None, 504, None, None, 512, None) == binding.ERR_INVALID      # stride < d_model
    assert proj(ctx, pid.value, 0, None, 516, None, None, 512, None) == binding.ERR_INVALID      # stride % 8
    assert proj(ctx, pid.value, 0, None, 0, None, None, 0, None) == binding.ERR_INVALID
    assert proj(ctx, pid.value, 1, None, 520, None, None, 512, None) == binding.OK               # host-only: no launch
    read = lib.bicache_read_prefix_layer
    assert read(ctx, pid.value + 9, 0, None, None, 256, None) == binding.ERR_NOTFOUND
    assert read(ctx, pid.value, 2, None, None, 256, None) == binding.ERR_INVALID
    assert read(ctx, pid.value, 0, None, None, 255, None) == binding.ERR_INVALID
    assert read(ctx, pid.value, 0, None, None, 256, None) == binding.ERR_UNSUPPORTED             # nothing to read from
    lib.bicache_destroy(ctx)
    # only bf16 with head_dim 128 has the projection
    f32 = host_ctx(lib, L=1, Hq=2, Hkv=2, D=64, pages=4, dtype=binding.F32)
    assert lib.bicache_reserve_prefix(f32, C.c_uint64(5), 40, C.byref(pid), C.byref(hit), pp, 4) == binding.OK
    assert proj(f32, pid.value, 0, None, 512, None, None, 512, None) == binding.ERR_UNSUPPORTED
    lib.bicache_destroy(f32)


@given(st.lists(st.tuples(st.integers(0, 7), st.integers(1, 80), st.integers(0, 2)), min_size=1, max_size=40),
       st.integers(2, 10), st.integers(0, 3), st.booleans())
@settings(max_examples=120, deadline=None)
def test_layered_store_traces_match_oracle_bit_exactly(trace, num_pages, seed, shrink_shallow):
    """Prefixes that own only the layers from a first layer on (the kept deep-layer K/V of Eq. 5), with
    per-layer free queues and, optionally, smaller pools in the shallow layers: ids, hit flags, error
    codes and the page list of EVERY layer equal the oracle's after every call."""
    entry.build()
    lib = binding.load_library()
    L = 3
    order = list(range(num_pages)) if seed == 0 else np.random.default_rng(seed).permutation(num_pages).tolist()
    caps = [max(1, num_pages // 2), max(1, (3 * num_pages) // 4), num_pages] if shrink_shallow else None
    cfg = binding.Config(L, 2, 1, 128, 16, num_pages, binding.BF16, -1)
    keep = np.ascontiguousarray(order, dtype=np.int32)
    cfg.initial_free_order = keep.ctypes.data_as(C.POINTER(C.c_int32))
    keep2 = None
    if caps is not None:
        keep2 = np.ascontiguousarray(caps, dtype=np.int32)
        cfg.layer_pages = keep2.ctypes.data_as(C.POINTER(C.c_int32))
    ctx = C.c_void_p()
    assert lib.bicache_create(C.byref(cfg), C.byref(ctx)) == binding.OK
    ref = oracle.PagedPrefixStore(L, 1, 128, 16, num_pages, free_order=order, layer_pages=caps)
    i32p = C.POINTER(C.c_int32)
    live = {}
    for key, m, first in trace:
        pid, hit = C.c_int32(-1), C.c_int32(-1)
        cap = (m + 15) // 16
        pages = np.full(cap, -1, dtype=np.int32)
        st_ = lib.bicache_reserve_prefix_layers(ctx, C.c_uint64(key), m, first, C.byref(pid), C.byref(hit),
                                                pages.ctypes.data_as(i32p), cap)
        try:
            opid, ohit, opages = ref.reserve(key, m, first)
        except oracle.InvalidArgument:
            assert st_ == binding.ERR_INVALID
            continue
        except oracle.OutOfPages:
            assert st_ == binding.ERR_NOMEM
            continue
        assert st_ == binding.OK and (pid.value, bool(hit.value), pages.tolist()) == (opid, ohit, opages)
        live[opid] = first
        for p_id in list(live):
            if p_id not in ref.entries:                     # evicted by this call
                n = C.c_int32(0)
                assert lib.bicache_prefix_pages(ctx, p_id, None, 0, C.byref(n)) == binding.ERR_NOTFOUND
                del live[p_id]
                continue
            for l in range(L):
                n = C.c_int32(0)
                buf = np.full(16, -1, dtype=np.int32)
                st2 = lib.bicache_prefix_pages_layer(ctx, p_id, l, buf.ctypes.data_as(i32p), 16, C.byref(n))
                if l < live[p_id]:
                    assert st2 == binding.ERR_INVALID
                else:
                    assert st2 == binding.OK and buf[:n.value].tolist() == ref.pages(p_id, l)
    lib.bicache_destroy(ctx)


def test_pool_bytes_with_layer_capacities(lib):
    cfg = binding.Config(3, 2, 1, 128, 16, 8, binding.BF16, -1)
    full = lib.bicache_pool_bytes(C.byref(cfg))
    assert full == 3 * 8 * 1 * 16 * 128 * 2
    caps = np.array([2, 5, 8], dtype=np.int32)
    cfg.layer_pages = caps.ctypes.data_as(C.POINTER(C.c_int32))
    assert lib.bicache_pool_bytes(C.byref(cfg)) == (2 + 5 + 8) * 16 * 128 * 2
    bad = np.array([2, 9, 8], dtype=np.int32)
    cfg.layer_pages = bad.ctypes.data_as(C.POINTER(C.c_int32))
    assert lib.bicache_pool_bytes(C.byref(cfg)) == 0
    ctx = C.c_void_p()
    assert lib.bicache_create(C.byref(cfg), C.byref(ctx)) == binding.ERR_INVALID
