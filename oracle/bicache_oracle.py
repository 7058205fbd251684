"""Plain fp64 definition of the BiCache per-denoising-step attention.

TEST INFRASTRUCTURE ONLY: never imported by the product path.

Everything here is written from the paper's statement of the method:

  * Eq. 2  (bidirectional softmax attention over all tokens of the input),
  * Eq. 4  (shallow layers l <= b use the cached shared-prefix KVs),
  * Sec. 5.1/5.2 (ratio r of shared-prefix tokens to all tokens -> lookup
    table T -> shallow depth b; layer l reuses iff l <= b, else recomputes),
  * Sec. 5.2 + implementation appendix (hash-indexed KV store H holding the
    prefix KVs of all L layers; first-in-first-out eviction),
  * Eq. 5  (deep layers l > b: the prefix KVs computed within the request are
    kept and reused across denoising steps, recomputed every Delta steps),
  * Eq. 3 + Sec. 4.2/5.1 (profiler: cosine similarity between cached and
    reference prefix KVs per layer -> depth b_i under threshold tau -> table T),
  * Sec. 5.2 + implementation appendix (k = h(p): a deterministic 64-bit hash,
    XXH64, of the prefix's token ids is the cache key),
  * Eq. 1  (k = W^K h, v = W^V h: the prefix KVs a miss computes and stores).

All floating-point work is numpy float64.  A matrix product (numpy matmul) is
used as a library step; there is no tiling, fusion, online softmax or any
other reordering, so each function can be compared with the paper by eye.
Inputs arrive as float64 arrays that are exact widenings of the bytes the GPU
gets (bf16 or fp32 -> fp64 is exact).

Conventions (0-based, as in the C API): layer index l in [0, L); a request
with depth b reuses the cache in layers l < b (the paper's 1-based l <= b).
Tensors: q [rows, Hq, D]; k, v [rows, Hkv, D]; query head h reads KV head
h // (Hq // Hkv).
"""
from __future__ import annotations

import math
from collections import OrderedDict, deque

import numpy as np


class OracleError(Exception):
    """Base class; subclasses mirror the library's status codes."""


class InvalidArgument(OracleError):
    pass


class OutOfPages(OracleError):
    pass


class NotFound(OracleError):
    pass


# ---------------------------------------------------------------------------
# Reuse-depth rule (Sec. 5.1 "profiling dataset": r = shared-prefix tokens /
# all tokens of the input string; Sec. 5.2: r -> T -> b).
# ---------------------------------------------------------------------------

def reuse_depth(prefix_len, nonshared_len, table, num_layers):
    """Per-request shallow depth b in [0, L].

    r = m / (m + n) is quantised DOWN to the table's 1/100 grid in integer
    arithmetic (the paper profiles r in {0.01, ..., 1.00}; it does not state
    the rounding; flooring is the conservative reading because b grows with
    r).  table has 101 entries, table[idx] for idx = floor(100 m / (m + n)).
    m <= 0 (no shared prefix) gives depth 0.
    """
    table = [int(x) for x in table]
    if len(table) != 101:
        raise InvalidArgument("depth table must have 101 entries")
    out = []
    for m, n in zip(prefix_len, nonshared_len):
        m = int(m)
        n = int(n)
        if n < 0:
            raise InvalidArgument("negative non-shared length")
        if m <= 0:
            out.append(0)
            continue
        idx = (100 * m) // (m + n)
        b = table[idx]
        b = max(0, min(int(num_layers), b))
        out.append(b)
    return np.asarray(out, dtype=np.int32)


# ---------------------------------------------------------------------------
# KV store H (Sec. 5.2: hit -> load the cached KVs of all L layers; miss ->
# insert; implementation appendix: FIFO eviction).  Storage is paged.
# ---------------------------------------------------------------------------

class PagedPrefixStore:
    """Prefix-KV store over fixed-size pages with FIFO eviction.

    Every layer has its own pages and its own free queue (a FIFO: pages are
    taken from its head; an evicted prefix's pages are appended to its tail in
    page-table order).  A prefix owns pages in the layers first_layer .. L-1
    only: a shared prefix (put) in all of them, a request's kept deep-layer
    prefix (reserve, Eq. 5) from its shallow depth on - the shallow layers of
    such a request never read its own prefix KVs.  Token t of a prefix lives, in
    layer l, in page pages_l[t // P], slot t % P.  As long as every prefix owns
    all layers the queues move in lockstep and a prefix has the same page list
    in every layer.  Layer l holds layer_pages[l] pages (default: num_pages in
    every layer).  Prefix ids come from a counter that is never reused.
    """

    def __init__(self, num_layers, num_kv_heads, head_dim, page_size, num_pages,
                 free_order=None, layer_pages=None):
        self.L = int(num_layers)
        self.Hkv = int(num_kv_heads)
        self.D = int(head_dim)
        self.P = int(page_size)
        self.num_pages = int(num_pages)
        if free_order is None:
            free_order = range(self.num_pages)
        free_order = [int(p) for p in free_order]
        if sorted(free_order) != list(range(self.num_pages)):
            raise InvalidArgument("free_order must be a permutation of the pages")
        if layer_pages is None:
            layer_pages = [self.num_pages] * self.L
        self.layer_pages = [int(c) for c in layer_pages]
        if len(self.layer_pages) != self.L or any(c < 1 or c > self.num_pages for c in self.layer_pages):
            raise InvalidArgument("layer_pages needs one capacity in 1..num_pages per layer")
        # layer l's queue: the pages below its capacity, in the given order
        self.free = [deque(p for p in free_order if p < c) for c in self.layer_pages]
        # [layer][page][slot][kv head][dim]
        shape = (self.L, self.num_pages, self.P, self.Hkv, self.D)
        self.k_pool = np.zeros(shape, dtype=np.float64)
        self.v_pool = np.zeros(shape, dtype=np.float64)
        self.by_key = OrderedDict()   # key -> prefix id, in insertion order
        self.entries = {}             # prefix id -> (key, m, first_layer, [pages of layer first_layer, ...])
        self.next_id = 0

    def pages_needed(self, m):
        return (int(m) + self.P - 1) // self.P

    def _insert(self, key, m, first_layer):
        """Hit / miss / FIFO eviction / allocation in the layers first_layer .. L-1.
        Returns (prefix_id, was_hit, pages of layer first_layer)."""
        m = int(m)
        first_layer = int(first_layer)
        if m < 1:
            raise InvalidArgument("empty prefix")
        if not 0 <= first_layer < self.L:
            raise InvalidArgument("first layer out of range")
        key = int(key)
        if key in self.by_key:
            pid = self.by_key[key]
            if self.entries[pid][1] != m or self.entries[pid][2] != first_layer:
                raise InvalidArgument("key already present with another length or first layer")
            return pid, True, list(self.entries[pid][3][0])
        need = self.pages_needed(m)
        layers = range(first_layer, self.L)
        if any(need > self.layer_pages[l] for l in layers):
            raise OutOfPages("prefix larger than a layer's pool")
        while any(len(self.free[l]) < need for l in layers):
            old_key, old_id = next(iter(self.by_key.items()))   # oldest insertion
            del self.by_key[old_key]
            _, _, old_first, old_pages = self.entries.pop(old_id)
            for j, plist in enumerate(old_pages):
                for p in plist:
                    self.free[old_first + j].append(p)
        pages = [[self.free[l].popleft() for _ in range(need)] for l in layers]
        pid = self.next_id
        self.next_id += 1
        self.by_key[key] = pid
        self.entries[pid] = (key, m, first_layer, pages)
        return pid, False, list(pages[0])

    def put(self, key, k, v):
        """Insert prefix KVs k, v of shape [L, m, Hkv, D] (all layers).  Returns
        (prefix_id, was_hit, pages of layer 0)."""
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        if k.shape != v.shape or k.ndim != 4 or k.shape[0] != self.L \
                or k.shape[2] != self.Hkv or k.shape[3] != self.D:
            raise InvalidArgument("bad prefix KV shape")
        m = k.shape[1]
        pid, hit, pages0 = self._insert(key, m, 0)
        if not hit:
            pages = self.entries[pid][3]
            for l in range(self.L):
                for t in range(m):
                    self.k_pool[l, pages[l][t // self.P], t % self.P] = k[l, t]
                    self.v_pool[l, pages[l][t // self.P], t % self.P] = v[l, t]
        return pid, hit, pages0

    def reserve(self, key, m, first_layer=0):
        """Allocate pages for a prefix of m tokens in the layers first_layer .. L-1
        without writing any KV (the per-request deep-layer cache of Eq. 5, which
        only layers past the request's shallow depth keep; filled layer by layer
        at refresh steps).  Same hit / miss / eviction rules as `put`.  Returns
        (prefix_id, was_hit, pages of layer first_layer)."""
        pid, hit, pages0 = self._insert(key, m, first_layer)
        if not hit:
            pages = self.entries[pid][3]
            for j, plist in enumerate(pages):
                for p in plist:
                    self.k_pool[first_layer + j, p] = 0.0
                    self.v_pool[first_layer + j, p] = 0.0
        return pid, hit, pages0

    def _layer_pages(self, prefix_id, layer):
        if prefix_id not in self.entries:
            raise NotFound("unknown or evicted prefix id")
        _, _, first, pages = self.entries[prefix_id]
        if not first <= layer < self.L:
            raise InvalidArgument("the prefix owns no pages in this layer")
        return pages[layer - first]

    def update_layer(self, prefix_id, layer, k, v):
        """Overwrite one layer of an existing prefix with k, v [m, Hkv, D]
        (Eq. 5, refresh step: KV^use <- KV^ref of the current step)."""
        if not 0 <= layer < self.L:
            raise InvalidArgument("layer out of range")
        pages = self._layer_pages(prefix_id, layer)
        m = self.entries[prefix_id][1]
        k = np.asarray(k, dtype=np.float64)
        v = np.asarray(v, dtype=np.float64)
        if k.shape != (m, self.Hkv, self.D) or v.shape != k.shape:
            raise InvalidArgument("bad layer KV shape")
        for t in range(m):
            self.k_pool[layer, pages[t // self.P], t % self.P] = k[t]
            self.v_pool[layer, pages[t // self.P], t % self.P] = v[t]

    def lookup(self, key):
        key = int(key)
        if key not in self.by_key:
            raise NotFound("unknown key")
        pid = self.by_key[key]
        return pid, self.entries[pid][1]

    def first_layer(self, prefix_id):
        if prefix_id not in self.entries:
            raise NotFound("unknown or evicted prefix id")
        return self.entries[prefix_id][2]

    def pages(self, prefix_id, layer=None):
        """Page list of a live prefix in `layer` (default: its first layer)."""
        if prefix_id not in self.entries:
            raise NotFound("unknown or evicted prefix id")
        if layer is None:
            layer = self.entries[prefix_id][2]
        return list(self._layer_pages(prefix_id, int(layer)))

    def prefix_len(self, prefix_id):
        if prefix_id not in self.entries:
            raise NotFound("unknown or evicted prefix id")
        return self.entries[prefix_id][1]

    def prefix_kv(self, layer, prefix_id):
        """Cached K, V of one layer, read back through the page table:
        two arrays [m, Hkv, D]."""
        if not 0 <= layer < self.L:
            raise InvalidArgument("layer out of range")
        pages = self._layer_pages(prefix_id, layer)
        m = self.entries[prefix_id][1]
        k = np.empty((m, self.Hkv, self.D), dtype=np.float64)
        v = np.empty((m, self.Hkv, self.D), dtype=np.float64)
        for t in range(m):
            k[t] = self.k_pool[layer, pages[t // self.P], t % self.P]
            v[t] = self.v_pool[layer, pages[t // self.P], t % self.P]
        return k, v


# ---------------------------------------------------------------------------
# Eq. 2: o = sum_j softmax_j(q . k_j * scale) v_j over ALL keys, no mask.
# ---------------------------------------------------------------------------

def attention(q, k, v, scale):
    """q [nq, Hq, D]; k, v [nk, Hkv, D] -> (o [nq, Hq, D], lse [nq, Hq]).

    lse is the natural log of sum_j exp(scale * q.k_j).  With no keys the
    output is 0 and lse is -inf (the empty partial result of a merge).
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    nq, Hq, D = q.shape
    nk, Hkv, _ = k.shape
    if Hq % Hkv:
        raise InvalidArgument("query heads must be a multiple of KV heads")
    group = Hq // Hkv
    o = np.zeros((nq, Hq, D), dtype=np.float64)
    lse = np.full((nq, Hq), -np.inf, dtype=np.float64)
    if nq == 0 or nk == 0:
        return o, lse
    for h in range(Hq):
        hk = h // group
        s = float(scale) * (q[:, h, :] @ k[:, hk, :].T)          # [nq, nk]
        mx = s.max(axis=1, keepdims=True)
        p = np.exp(s - mx)
        z = p.sum(axis=1, keepdims=True)
        o[:, h, :] = (p @ v[:, hk, :]) / z
        lse[:, h] = (mx + np.log(z))[:, 0]
    return o, lse


def merge(parts):
    """Log-sum-exp merge of partial results over disjoint key sets.

    parts: sequence of (o [.., D], lse [..]).  Returns (o, lse) equal to Eq. 2
    over the union of the key sets:  lse = log sum_i exp(lse_i),
    o = sum_i exp(lse_i - lse) o_i.  A part with lse = -inf weighs 0.
    """
    parts = [(np.asarray(o, dtype=np.float64), np.asarray(l, dtype=np.float64))
             for o, l in parts]
    lses = np.stack([l for _, l in parts])                       # [parts, ...]
    mx = lses.max(axis=0)
    safe = np.where(np.isfinite(mx), mx, 0.0)
    w = np.exp(lses - safe)                                       # exp(-inf) = 0
    tot = w.sum(axis=0)
    with np.errstate(divide="ignore"):
        lse = safe + np.log(tot)
    lse = np.where(tot > 0, lse, -np.inf)
    o = np.zeros_like(parts[0][0])
    for (oi, _), wi in zip(parts, w):
        frac = np.where(tot > 0, wi / np.where(tot > 0, tot, 1.0), 0.0)
        o = o + frac[..., None] * oi
    return o, lse


# ---------------------------------------------------------------------------
# The two calls of the hot path.
# ---------------------------------------------------------------------------

def _check_batch(row_off, seqlen, rows):
    for off, n in zip(row_off, seqlen):
        if n < 0 or off < 0 or off + n > rows:
            raise InvalidArgument("request rows out of range")


def attend(store, layer, prefix_id, row_off, seqlen, q, k, v, scale):
    """Shallow-layer attention (Eq. 2 with the key set Eq. 4 prescribes).

    For request i with suffix rows row_off[i] .. row_off[i] + seqlen[i] of
    q/k/v: every suffix query attends, without any mask, over
    [cached prefix K/V of prefix_id[i] at `layer` | the request's own suffix
    K/V].  prefix_id[i] = -1 means no prefix.  Returns (out, lse) shaped like
    q and q[..., 0]; rows that belong to no request are left at 0 / -inf.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    _check_batch(row_off, seqlen, q.shape[0])
    out = np.zeros_like(q)
    lse = np.full(q.shape[:2], -np.inf)
    for pid, off, n in zip(prefix_id, row_off, seqlen):
        off = int(off)
        n = int(n)
        if n == 0:
            continue
        ks, vs = k[off:off + n], v[off:off + n]
        if pid >= 0:
            kc, vc = store.prefix_kv(layer, int(pid))
            ks = np.concatenate([kc, ks], axis=0)
            vs = np.concatenate([vc, vs], axis=0)
        out[off:off + n], lse[off:off + n] = attention(q[off:off + n], ks, vs, scale)
    return out, lse


def attend_full(row_off, seqlen, q, k, v, scale):
    """Deep-layer fallback: full bidirectional attention (Eq. 2) of each
    request over its own N_i fresh rows; all N_i rows are queries."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    _check_batch(row_off, seqlen, q.shape[0])
    out = np.zeros_like(q)
    lse = np.full(q.shape[:2], -np.inf)
    for off, n in zip(row_off, seqlen):
        off = int(off)
        n = int(n)
        if n == 0:
            continue
        out[off:off + n], lse[off:off + n] = attention(
            q[off:off + n], k[off:off + n], v[off:off + n], scale)
    return out, lse


def _one_row(q_row, ks, vs, hk, scale):
    s = float(scale) * (ks[:, hk, :] @ q_row)
    mx = s.max()
    p = np.exp(s - mx)
    z = p.sum()
    return (p @ vs[:, hk, :]) / z, mx + math.log(z)


def attend_rows(store, layer, prefix_id, row_off, seqlen, q, k, v, scale, samples):
    """Same definition as `attend`, evaluated only at the sampled
    (request, head, row-within-suffix) triples, each over ALL its keys.
    Returns (o [len(samples), D], lse [len(samples)])."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    Hq, Hkv = q.shape[1], k.shape[1]
    o = np.zeros((len(samples), q.shape[2]))
    lse = np.zeros(len(samples))
    cache = {}
    for si, (i, h, a) in enumerate(samples):
        off, n, pid = int(row_off[i]), int(seqlen[i]), int(prefix_id[i])
        if not 0 <= a < n:
            raise InvalidArgument("sampled row outside the request")
        if i not in cache:
            ks, vs = k[off:off + n], v[off:off + n]
            if pid >= 0:
                kc, vc = store.prefix_kv(layer, pid)
                ks = np.concatenate([kc, ks], axis=0)
                vs = np.concatenate([vc, vs], axis=0)
            cache = {i: (ks, vs)}
        ks, vs = cache[i]
        o[si], lse[si] = _one_row(q[off + a, h], ks, vs, h // (Hq // Hkv), scale)
    return o, lse


def attend_full_rows(row_off, seqlen, q, k, v, scale, samples):
    """`attend_full` at sampled (request, head, row) triples."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    Hq, Hkv = q.shape[1], k.shape[1]
    o = np.zeros((len(samples), q.shape[2]))
    lse = np.zeros(len(samples))
    for si, (i, h, a) in enumerate(samples):
        off, n = int(row_off[i]), int(seqlen[i])
        if not 0 <= a < n:
            raise InvalidArgument("sampled row outside the request")
        o[si], lse[si] = _one_row(q[off + a, h], k[off:off + n], v[off:off + n],
                                  h // (Hq // Hkv), scale)
    return o, lse


def stack(store, depth, prefix_id, prefix_len, full_row_off, full_len, q, k, v, scale):
    """One denoising step's attention over all L layers (Sec. 5.2 dispatch).

    Request i owns rows full_row_off[i] .. + full_len[i] of q/k/v (its whole
    input: prefix_len[i] prefix tokens then the suffix).  q, k, v are lists
    with one [rows, H, D] array per layer.  In layer l, requests with
    l < depth[i] go through `attend` on their suffix rows (the tail of their
    row range); the others go through `attend_full` on all their rows.
    Returns a list of per-layer (out, lse); rows not computed in a layer
    (prefix rows of reusing requests) stay 0 / -inf.
    """
    R = len(depth)
    results = []
    for l in range(store.L if store is not None else len(q)):
        reuse = [i for i in range(R) if l < depth[i]]
        full = [i for i in range(R) if l >= depth[i]]
        out = np.zeros_like(np.asarray(q[l], dtype=np.float64))
        lse = np.full(out.shape[:2], -np.inf)
        if reuse:
            offs = [full_row_off[i] + prefix_len[i] for i in reuse]
            lens = [full_len[i] - prefix_len[i] for i in reuse]
            o1, l1 = attend(store, l, [prefix_id[i] for i in reuse], offs, lens,
                            q[l], k[l], v[l], scale)
            for off, n in zip(offs, lens):
                out[off:off + n] = o1[off:off + n]
                lse[off:off + n] = l1[off:off + n]
        if full:
            offs = [full_row_off[i] for i in full]
            lens = [full_len[i] for i in full]
            o2, l2 = attend_full(offs, lens, q[l], k[l], v[l], scale)
            for off, n in zip(offs, lens):
                out[off:off + n] = o2[off:off + n]
                lse[off:off + n] = l2[off:off + n]
        results.append((out, lse))
    return results


# ---------------------------------------------------------------------------
# Eq. 5: deep layers reuse the request's own prefix KVs across steps and
# recompute them every Delta steps.
# ---------------------------------------------------------------------------

def is_refresh_step(t, delta):
    """Eq. 5's condition (t - 1) mod Delta = 0 for the 1-based step t."""
    if t < 1 or delta < 1:
        raise InvalidArgument("t and delta start at 1")
    return (t - 1) % delta == 0


def attend_step(store, layer, t, delta, depth, shared_id, private_id, full_row_off, full_len,
                q, k, v, scale):
    """One layer of denoising step t with both kinds of reuse (Sec. 5.2).

    Request i owns rows full_row_off[i] .. + full_len[i] of q/k/v (prefix
    tokens first).  Per request, in this order:
      * layer < depth[i] and shared_id[i] >= 0: the suffix queries attend over
        [shared cached prefix KVs | own suffix KVs]              (Eq. 4);
      * else, private_id[i] >= 0 and t is not a refresh step: the suffix
        queries attend over [the request's own prefix KVs kept from the last
        refresh step | own suffix KVs]                           (Eq. 5, 2nd case);
      * else: full attention over all the request's rows; if private_id[i] >= 0
        (a refresh step) the fresh prefix KVs of this layer, rows
        0 .. m of the request, replace the kept ones             (Eq. 5, 1st case).
    Returns (out, lse); rows not computed stay 0 / -inf.
    """
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    _check_batch(full_row_off, full_len, q.shape[0])
    refresh = is_refresh_step(t, delta)
    out = np.zeros_like(q)
    lse = np.full(q.shape[:2], -np.inf)
    for i in range(len(depth)):
        off, N = int(full_row_off[i]), int(full_len[i])
        if layer < depth[i] and shared_id[i] >= 0:
            pid = int(shared_id[i])
        elif private_id[i] >= 0 and not refresh:
            pid = int(private_id[i])
        else:
            pid = -1
        if pid >= 0:
            m = store.prefix_len(pid)
            if N < m:
                raise InvalidArgument("request shorter than its prefix")
            kc, vc = store.prefix_kv(layer, pid)
            ks = np.concatenate([kc, k[off + m:off + N]], axis=0)
            vs = np.concatenate([vc, v[off + m:off + N]], axis=0)
            if N > m:
                out[off + m:off + N], lse[off + m:off + N] = attention(q[off + m:off + N], ks, vs, scale)
        else:
            if N > 0:
                out[off:off + N], lse[off:off + N] = attention(q[off:off + N], k[off:off + N], v[off:off + N], scale)
            if private_id[i] >= 0:
                m = store.prefix_len(int(private_id[i]))
                if N < m:
                    raise InvalidArgument("request shorter than its prefix")
                store.update_layer(int(private_id[i]), layer, k[off:off + m], v[off:off + m])
    return out, lse


# ---------------------------------------------------------------------------
# Profiler (Sec. 4.1 Eq. 3, Sec. 4.2, Sec. 5.1): similarity of the cached prefix
# KVs to the ones a request computes itself, per layer; the depth it allows;
# the lookup table built from many requests.
# ---------------------------------------------------------------------------

def kv_similarity(store, prefix_id, k_ref, v_ref):
    """sim_l = cos(KV$_l, KVref_l) for every layer l (Eq. 3).

    The flattening the Sec. 4.1 footnote speaks of is read as: layer l's keys
    and values of all prefix positions and heads, concatenated, form one vector
    per side.  k_ref, v_ref:
    [L, m, Hkv, D].  A zero vector on either side gives similarity 0.
    """
    k_ref = np.asarray(k_ref, dtype=np.float64)
    v_ref = np.asarray(v_ref, dtype=np.float64)
    m = store.prefix_len(prefix_id)
    if k_ref.shape != (store.L, m, store.Hkv, store.D) or v_ref.shape != k_ref.shape:
        raise InvalidArgument("bad reference KV shape")
    sim = np.zeros(store.L)
    for l in range(store.L):
        kc, vc = store.prefix_kv(l, prefix_id)
        a = np.concatenate([kc.reshape(-1), vc.reshape(-1)])
        b = np.concatenate([k_ref[l].reshape(-1), v_ref[l].reshape(-1)])
        na, nb = math.sqrt(float(a @ a)), math.sqrt(float(b @ b))
        sim[l] = float(a @ b) / (na * nb) if na > 0 and nb > 0 else 0.0
    return sim


def depth_from_similarity(sim, tau):
    """Sec. 4.2 / 5.1: b = the largest layer count such that every layer
    1 .. b has sim_l >= tau, i.e. the number of leading layers at or above the
    threshold."""
    b = 0
    for x in sim:
        if not x >= tau:
            break
        b += 1
    return b


def build_depth_table(ratio_idx, depths, num_layers):
    """Sec. 5.1 "lookup table T": for each ratio bin, the average of the b_i of
    the requests profiled at that ratio, as an integer (floored: the smaller,
    safer depth).  Returns 101 entries.  A bin without samples takes the value
    of the nearest filled bin below it (b does not decrease with the ratio, so
    this never overstates it); bins below the first filled one take min(1, L)
    (layer 1's KVs do not depend on the rest of the input, Sec. 4.2 footnote).
    """
    sums = [0] * 101
    cnts = [0] * 101
    for idx, b in zip(ratio_idx, depths):
        if not 0 <= idx <= 100 or not 0 <= b <= num_layers:
            raise InvalidArgument("ratio bin or depth out of range")
        sums[idx] += int(b)
        cnts[idx] += 1
    table = []
    last = min(1, num_layers)
    for idx in range(101):
        if cnts[idx]:
            last = sums[idx] // cnts[idx]
        table.append(last)
    return table


# ---------------------------------------------------------------------------
# Cache key (Sec. 5.2 "k = h(p)"; implementation appendix: a 64-bit xxHash of the
# tokenised prefix).  XXH64 with seed 0 over the token ids as little-endian
# 32-bit integers, written out from the algorithm's published description.
# ---------------------------------------------------------------------------

_M64 = (1 << 64) - 1
_XP1, _XP2, _XP3 = 0x9E3779B185EBCA87, 0xC2B2AE3D27D4EB4F, 0x165667B19E3779F9
_XP4, _XP5 = 0x85EBCA77C2B2AE63, 0x27D4EB2F165667C5


def _rotl(x, r):
    return ((x << r) | (x >> (64 - r))) & _M64


def _xround(acc, lane):
    return (_rotl((acc + lane * _XP2) & _M64, 31) * _XP1) & _M64


def xxh64(data, seed=0):
    """XXH64 of a bytes object."""
    n = len(data)
    pos = 0
    if n >= 32:
        v = [(seed + _XP1 + _XP2) & _M64, (seed + _XP2) & _M64, seed & _M64, (seed - _XP1) & _M64]
        while pos + 32 <= n:
            for i in range(4):
                v[i] = _xround(v[i], int.from_bytes(data[pos + 8 * i:pos + 8 * i + 8], "little"))
            pos += 32
        h = (_rotl(v[0], 1) + _rotl(v[1], 7) + _rotl(v[2], 12) + _rotl(v[3], 18)) & _M64
        for i in range(4):
            h = ((h ^ _xround(0, v[i])) * _XP1 + _XP4) & _M64
    else:
        h = (seed + _XP5) & _M64
    h = (h + n) & _M64
    while pos + 8 <= n:
        h ^= _xround(0, int.from_bytes(data[pos:pos + 8], "little"))
        h = (_rotl(h, 27) * _XP1 + _XP4) & _M64
        pos += 8
    if pos + 4 <= n:
        h ^= (int.from_bytes(data[pos:pos + 4], "little") * _XP1) & _M64
        h = (_rotl(h, 23) * _XP2 + _XP3) & _M64
        pos += 4
    while pos < n:
        h ^= (data[pos] * _XP5) & _M64
        h = (_rotl(h, 11) * _XP1) & _M64
        pos += 1
    h ^= h >> 33
    h = (h * _XP2) & _M64
    h ^= h >> 29
    h = (h * _XP3) & _M64
    h ^= h >> 32
    return h


def prefix_key(tokens):
    """k = h(p): the 64-bit key of a prefix given as a sequence of token ids."""
    raw = b"".join(int(t).to_bytes(4, "little", signed=True) for t in tokens)
    return xxh64(raw, 0)


# ---------------------------------------------------------------------------
# Eq. 1: the key and value vectors of a token are linear projections of its
# hidden state, k = W^K h, v = W^V h (W^K, W^V of shape [d_k, d] per layer).
# ---------------------------------------------------------------------------

def rope_rotate(x, cos, sin):
    """Rotary position encoding of keys (or queries) in the half-split pairing:
    for token t and every head, the pair (x[d], x[d + D/2]), d < D/2, is rotated
    by the angle whose cosine and sine are cos[t, d], sin[t, d]:

        x'[d]       = x[d] cos - x[d + D/2] sin
        x'[d + D/2] = x[d + D/2] cos + x[d] sin

    x [m, H, D]; cos, sin [m, D/2] (the caller's table: the paper names no
    position encoding, so angles are an input, not computed here).
    """
    x = np.asarray(x, dtype=np.float64)
    cos = np.asarray(cos, dtype=np.float64)
    sin = np.asarray(sin, dtype=np.float64)
    m, _, D = x.shape
    if D % 2 or cos.shape != (m, D // 2) or sin.shape != cos.shape:
        raise InvalidArgument("bad rotary table shape")
    half = D // 2
    out = np.empty_like(x)
    for t in range(m):
        lo, hi = x[t, :, :half], x[t, :, half:]
        out[t, :, :half] = lo * cos[t] - hi * sin[t]
        out[t, :, half:] = hi * cos[t] + lo * sin[t]
    return out


def project_kv(h, wk, wv, num_kv_heads, head_dim, rope=None):
    """Prefix KVs from hidden states, every layer (Eq. 1).

    h [L, m, d]; wk, wv [L, Hkv * D, d] (row o of a weight produces output
    component o; components are ordered head-major: o = head * D + dim).
    rope: None (Eq. 1 as printed) or (cos, sin), each [m, D/2]: the keys (not
    the values) are then rotated per token with `rope_rotate` after the
    projection, the form in which a rotary model caches them.
    Returns k, v of shape [L, m, Hkv, D], ready for `PagedPrefixStore.put`.
    """
    h = np.asarray(h, dtype=np.float64)
    wk = np.asarray(wk, dtype=np.float64)
    wv = np.asarray(wv, dtype=np.float64)
    L, m, d = h.shape
    out = num_kv_heads * head_dim
    if wk.shape != (L, out, d) or wv.shape != (L, out, d):
        raise InvalidArgument("bad projection weight shape")
    k = np.empty((L, m, num_kv_heads, head_dim))
    v = np.empty((L, m, num_kv_heads, head_dim))
    for l in range(L):
        k[l] = (h[l] @ wk[l].T).reshape(m, num_kv_heads, head_dim)
        v[l] = (h[l] @ wv[l].T).reshape(m, num_kv_heads, head_dim)
        if rope is not None:
            k[l] = rope_rotate(k[l], rope[0], rope[1])
    return k, v
