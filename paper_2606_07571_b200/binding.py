"""ctypes binding of libbicache.so: same names as the C ABI, argument marshalling only.

Every step of the path runs inside the shared library's CUDA kernels; PyTorch is used for device
buffers and streams.  A missing or unloadable library raises at first use: there is no fallback.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

OK, ERR_INVALID, ERR_NOMEM, ERR_NOTFOUND, ERR_CUDA, ERR_TIMEOUT, ERR_UNSUPPORTED = range(7)
F32, BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR, PATH_TENSOR_PAIRS = 0, 1, 2, 3
KERNEL_SIMT, KERNEL_TENSOR, KERNEL_KEY_RANGES, KERNEL_TENSOR_PAIRS = 1, 2, 3, 4
_STATUS_NAMES = ["OK", "INVALID", "NOMEM", "NOTFOUND", "CUDA", "TIMEOUT", "UNSUPPORTED"]

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libbicache.so")

EXPORTED = [
    "bicache_pool_bytes", "bicache_workspace_bytes", "bicache_create", "bicache_destroy",
    "bicache_set_path", "bicache_set_depth_table", "bicache_put_prefix", "bicache_lookup_prefix",
    "bicache_prefix_pages", "bicache_prefix_pages_layer", "bicache_reserve_prefix_layers", "bicache_reuse_depth", "bicache_attend", "bicache_attend_full",
    "bicache_attend_layer", "bicache_attend_full_static",
    "bicache_is_refresh_step", "bicache_reserve_prefix", "bicache_update_prefix_layer", "bicache_attend_step",
    "bicache_read_prefix_layer", "bicache_project_prefix_layer", "bicache_project_prefix_layer_rope",
    "bicache_prefix_similarity", "bicache_prefix_similarity_async", "bicache_depth_from_similarity",
    "bicache_build_depth_table",
    "bicache_hash_tokens", "bicache_device_status", "bicache_set_wait_budget", "bicache_launch_count", "bicache_schedule_uploads", "bicache_last_attention_kernel", "bicache_last_error",
]


class BiCacheError(RuntimeError):
    def __init__(self, status, where, detail=""):
        self.status = status
        name = _STATUS_NAMES[status] if 0 <= status < len(_STATUS_NAMES) else str(status)
        super().__init__("%s: BICACHE_ERR_%s %s" % (where, name, detail))


class Config(C.Structure):
    _fields_ = [
        ("num_layers", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
        ("head_dim", C.c_int32), ("page_size", C.c_int32), ("num_pages", C.c_int32),
        ("dtype", C.c_int32), ("device", C.c_int32),
        ("initial_free_order", C.POINTER(C.c_int32)),
        ("layer_pages", C.POINTER(C.c_int32)),
        ("k_pool", C.c_void_p), ("v_pool", C.c_void_p),
        ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
    ]


_lib = None


def load_library():
    """Load libbicache.so (built in-tree by __graft_entry__.build()).  Raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libbicache.so is not built (run __graft_entry__.build()); "
                           "there is no fallback path: " + LIB_PATH)
    lib = C.CDLL(LIB_PATH)
    i32p, i64p, vp = C.POINTER(C.c_int32), C.POINTER(C.c_int64), C.c_void_p
    lib.bicache_pool_bytes.restype = C.c_size_t
    lib.bicache_pool_bytes.argtypes = [C.POINTER(Config)]
    lib.bicache_workspace_bytes.restype = C.c_size_t
    lib.bicache_workspace_bytes.argtypes = [C.POINTER(Config), C.c_int64, C.c_int32]
    lib.bicache_create.restype = C.c_int32
    lib.bicache_create.argtypes = [C.POINTER(Config), C.POINTER(vp)]
    lib.bicache_destroy.restype = C.c_int32
    lib.bicache_destroy.argtypes = [vp]
    lib.bicache_set_path.restype = C.c_int32
    lib.bicache_set_path.argtypes = [vp, C.c_int32]
    lib.bicache_set_depth_table.restype = C.c_int32
    lib.bicache_set_depth_table.argtypes = [vp, i32p, C.c_int32]
    lib.bicache_put_prefix.restype = C.c_int32
    lib.bicache_put_prefix.argtypes = [vp, C.c_uint64, C.c_int32, vp, vp, C.c_int64, vp, i32p, i32p, i32p, C.c_int32]
    lib.bicache_lookup_prefix.restype = C.c_int32
    lib.bicache_lookup_prefix.argtypes = [vp, C.c_uint64, i32p, i32p]
    lib.bicache_prefix_pages.restype = C.c_int32
    lib.bicache_prefix_pages.argtypes = [vp, C.c_int32, i32p, C.c_int32, i32p]
    lib.bicache_prefix_pages_layer.restype = C.c_int32
    lib.bicache_prefix_pages_layer.argtypes = [vp, C.c_int32, C.c_int32, i32p, C.c_int32, i32p]
    lib.bicache_reserve_prefix_layers.restype = C.c_int32
    lib.bicache_reserve_prefix_layers.argtypes = [vp, C.c_uint64, C.c_int32, C.c_int32, i32p, i32p, i32p, C.c_int32]
    lib.bicache_reuse_depth.restype = C.c_int32
    lib.bicache_reuse_depth.argtypes = [vp, C.c_int32, i32p, i32p, i32p]
    lib.bicache_attend.restype = C.c_int32
    lib.bicache_attend.argtypes = [vp, C.c_int32, C.c_int32, i32p, i64p, i32p, vp, vp, vp, C.c_int64, C.c_int64,
                                   vp, C.c_int64, vp, C.c_float, vp]
    lib.bicache_attend_full.restype = C.c_int32
    lib.bicache_attend_full.argtypes = [vp, C.c_int32, C.c_int32, i64p, i32p, vp, vp, vp, C.c_int64, C.c_int64,
                                        vp, C.c_int64, vp, C.c_float, vp]
    lib.bicache_attend_layer.restype = C.c_int32
    lib.bicache_attend_layer.argtypes = [vp, C.c_int32, C.c_int32, i32p, i32p, i64p, i32p, vp, vp, vp, C.c_int64,
                                         C.c_int64, vp, C.c_int64, vp, C.c_float, vp]
    lib.bicache_is_refresh_step.restype = C.c_int32
    lib.bicache_is_refresh_step.argtypes = [C.c_int32, C.c_int32]
    lib.bicache_reserve_prefix.restype = C.c_int32
    lib.bicache_reserve_prefix.argtypes = [vp, C.c_uint64, C.c_int32, i32p, i32p, i32p, C.c_int32]
    lib.bicache_update_prefix_layer.restype = C.c_int32
    lib.bicache_update_prefix_layer.argtypes = [vp, C.c_int32, C.c_int32, vp, vp, C.c_int64, vp]
    lib.bicache_read_prefix_layer.restype = C.c_int32
    lib.bicache_read_prefix_layer.argtypes = [vp, C.c_int32, C.c_int32, vp, vp, C.c_int64, vp]
    lib.bicache_project_prefix_layer.restype = C.c_int32
    lib.bicache_project_prefix_layer.argtypes = [vp, C.c_int32, C.c_int32, vp, C.c_int64, vp, vp, C.c_int32, vp]
    lib.bicache_project_prefix_layer_rope.restype = C.c_int32
    lib.bicache_project_prefix_layer_rope.argtypes = [vp, C.c_int32, C.c_int32, vp, C.c_int64, vp, vp, C.c_int32, vp, vp]
    lib.bicache_attend_step.restype = C.c_int32
    lib.bicache_attend_step.argtypes = [vp, C.c_int32, C.c_int32, C.c_int32, C.c_int32, i32p, i32p, i32p, i64p, i32p,
                                        vp, vp, vp, C.c_int64, C.c_int64, vp, C.c_int64, vp, C.c_float, vp]
    f32p = C.POINTER(C.c_float)
    lib.bicache_prefix_similarity.restype = C.c_int32
    lib.bicache_prefix_similarity.argtypes = [vp, C.c_int32, vp, vp, C.c_int64, f32p, vp]
    lib.bicache_prefix_similarity_async.restype = C.c_int32
    lib.bicache_prefix_similarity_async.argtypes = [vp, C.c_int32, vp, vp, C.c_int64, vp, vp]
    lib.bicache_depth_from_similarity.restype = C.c_int32
    lib.bicache_depth_from_similarity.argtypes = [f32p, C.c_int32, C.c_float, i32p]
    lib.bicache_build_depth_table.restype = C.c_int32
    lib.bicache_build_depth_table.argtypes = [i32p, i32p, C.c_int32, C.c_int32, i32p]
    lib.bicache_attend_full_static.restype = C.c_int32
    lib.bicache_attend_full_static.argtypes = [C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.c_int32, vp, vp, vp,
                                               C.c_int64, C.c_int64, vp, C.c_int64, C.c_float, vp]
    lib.bicache_device_status.restype = C.c_int32
    lib.bicache_device_status.argtypes = [vp, vp, C.c_int32]
    lib.bicache_hash_tokens.restype = C.c_uint64
    lib.bicache_hash_tokens.argtypes = [i32p, C.c_int64]
    lib.bicache_set_wait_budget.restype = C.c_int32
    lib.bicache_set_wait_budget.argtypes = [vp, C.c_int64]
    lib.bicache_launch_count.restype = C.c_int64
    lib.bicache_launch_count.argtypes = [vp]
    lib.bicache_schedule_uploads.restype = C.c_int64
    lib.bicache_schedule_uploads.argtypes = [vp]
    lib.bicache_last_error.restype = C.c_char_p
    lib.bicache_last_error.argtypes = [vp]
    lib.bicache_last_attention_kernel.restype = C.c_int32
    lib.bicache_last_attention_kernel.argtypes = [vp]
    _lib = lib
    return lib


def _i32(a):
    a = np.ascontiguousarray(a, dtype=np.int32)
    return a, a.ctypes.data_as(C.POINTER(C.c_int32))


def _i64(a):
    a = np.ascontiguousarray(a, dtype=np.int64)
    return a, a.ctypes.data_as(C.POINTER(C.c_int64))


def _dtype_code(dtype):
    if dtype == torch.float32:
        return F32
    if dtype == torch.bfloat16:
        return BF16
    raise BiCacheError(ERR_UNSUPPORTED, "dtype", str(dtype))


class BiCache:
    """One library context plus the torch-owned device buffers it needs."""

    def __init__(self, num_layers, num_q_heads, num_kv_heads, head_dim, num_pages, dtype,
                 max_total_rows, max_requests, device=0, page_size=16, free_order=None, workspace_bytes=None,
                 layer_pages=None):
        self.lib = load_library()
        if not torch.cuda.is_available():
            raise RuntimeError("BiCache needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", device)
        self.dtype = dtype
        self.L, self.Hq, self.Hkv, self.D = num_layers, num_q_heads, num_kv_heads, head_dim
        cfg = Config(num_layers, num_q_heads, num_kv_heads, head_dim, page_size, num_pages,
                     _dtype_code(dtype), device)
        self._layer_pages = None
        if layer_pages is not None:              # per-layer pool capacities
            self._layer_pages, ptr = _i32(layer_pages)
            assert len(self._layer_pages) == num_layers
            cfg.layer_pages = ptr
        pool_bytes = self.lib.bicache_pool_bytes(C.byref(cfg))
        ws_bytes = self.lib.bicache_workspace_bytes(C.byref(cfg), int(max_total_rows), int(max_requests))
        if workspace_bytes is not None:          # a caller that sizes the workspace itself
            ws_bytes = int(workspace_bytes)
        if pool_bytes == 0 or ws_bytes == 0:
            raise BiCacheError(ERR_INVALID, "bicache_pool_bytes/workspace_bytes")
        # torch allocations are 512-byte aligned
        self.k_pool = torch.empty(pool_bytes, dtype=torch.uint8, device=self.device)
        self.v_pool = torch.empty(pool_bytes, dtype=torch.uint8, device=self.device)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=self.device)
        self._order = None
        if free_order is not None:
            self._order, ptr = _i32(free_order)
            cfg.initial_free_order = ptr
        cfg.k_pool, cfg.v_pool = self.k_pool.data_ptr(), self.v_pool.data_ptr()
        cfg.workspace, cfg.workspace_bytes = self.workspace.data_ptr(), ws_bytes
        self.ctx = C.c_void_p()
        self._check(self.lib.bicache_create(C.byref(cfg), C.byref(self.ctx)), "bicache_create", use_ctx=False)

    # -- helpers ---------------------------------------------------------------------------
    def _check(self, status, where, use_ctx=True):
        if status != OK:
            detail = ""
            if use_ctx and self.ctx:
                detail = (self.lib.bicache_last_error(self.ctx) or b"").decode()
            raise BiCacheError(status, where, detail)

    @staticmethod
    def _stream():
        return C.c_void_p(torch.cuda.current_stream().cuda_stream)

    def close(self):
        if getattr(self, "ctx", None) and self.ctx:
            self.lib.bicache_destroy(self.ctx)
            self.ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the C ABI, one method per call -----------------------------------------------------
    def set_path(self, path):
        self._check(self.lib.bicache_set_path(self.ctx, path), "bicache_set_path")

    def set_depth_table(self, table):
        arr, ptr = _i32(table)
        self._check(self.lib.bicache_set_depth_table(self.ctx, ptr, len(arr)), "bicache_set_depth_table")

    def put_prefix(self, key, k, v):
        """k, v: [L, m, Hkv, D] device tensors.  Returns (prefix_id, was_hit, pages)."""
        assert k.is_cuda and v.is_cuda and k.dtype == self.dtype and k.shape == v.shape
        assert k.stride()[1:] == (self.Hkv * self.D, self.D, 1) and v.stride() == k.stride()
        m = k.shape[1]
        pid, hit = C.c_int32(-1), C.c_int32(0)
        cap = (m + 15) // 16
        pages = np.zeros(max(cap, 1), dtype=np.int32)
        st = self.lib.bicache_put_prefix(self.ctx, C.c_uint64(key), m, k.data_ptr(), v.data_ptr(),
                                         k.stride(0), self._stream(), C.byref(pid), C.byref(hit),
                                         pages.ctypes.data_as(C.POINTER(C.c_int32)), cap)
        self._check(st, "bicache_put_prefix")
        return pid.value, bool(hit.value), pages[:cap].tolist()

    def reserve_prefix(self, key, m, first_layer=0):
        """Pages for a prefix of m tokens in the layers first_layer .. L-1, no K/V written (Eq. 5's
        per-request cache).  Returns (prefix_id, was_hit, pages of layer first_layer)."""
        pid, hit = C.c_int32(-1), C.c_int32(0)
        cap = (m + 15) // 16
        pages = np.zeros(max(cap, 1), dtype=np.int32)
        st = self.lib.bicache_reserve_prefix_layers(self.ctx, C.c_uint64(key), m, first_layer, C.byref(pid),
                                                    C.byref(hit), pages.ctypes.data_as(C.POINTER(C.c_int32)), cap)
        self._check(st, "bicache_reserve_prefix_layers")
        return pid.value, bool(hit.value), pages[:cap].tolist()

    def update_prefix_layer(self, prefix_id, layer, k, v):
        """k, v: [m, Hkv, D] device tensors (rows may be strided) that replace one layer of a prefix."""
        assert k.is_cuda and v.is_cuda and k.dtype == self.dtype and k.shape == v.shape
        assert k.stride()[1:] == (self.D, 1) and v.stride() == k.stride()
        st = self.lib.bicache_update_prefix_layer(self.ctx, prefix_id, layer, k.data_ptr(), v.data_ptr(),
                                                  k.stride(0), self._stream())
        self._check(st, "bicache_update_prefix_layer")

    def read_prefix_layer(self, prefix_id, layer, k_out, v_out):
        """One layer of a stored prefix as dense rows: k_out, v_out [m, Hkv, D] (rows may be strided)."""
        assert k_out.is_cuda and v_out.is_cuda and k_out.dtype == self.dtype and k_out.shape == v_out.shape
        assert k_out.stride()[1:] == (self.D, 1) and v_out.stride() == k_out.stride()
        st = self.lib.bicache_read_prefix_layer(self.ctx, prefix_id, layer, k_out.data_ptr(), v_out.data_ptr(),
                                                k_out.stride(0), self._stream())
        self._check(st, "bicache_read_prefix_layer")

    def project_prefix_layer(self, prefix_id, layer, h, w_k, w_v, rope=None):
        """Eq. 1 into the store: h [m, d_model] (rows may be strided), w_k, w_v [Hkv * D, d_model].
        rope: None, or a device fp32 tensor [m, 64, 2] of (cos, sin) per token and pair of head dims
        (d, d + 64) by which the keys are rotated before they are stored."""
        assert h.is_cuda and w_k.is_cuda and w_v.is_cuda and h.dtype == w_k.dtype == w_v.dtype == self.dtype
        assert h.dim() == 2 and h.stride(1) == 1 and w_k.is_contiguous() and w_v.is_contiguous()
        assert w_k.shape == w_v.shape == (self.Hkv * self.D, h.shape[1])
        rp = None
        if rope is not None:
            assert rope.is_cuda and rope.dtype == torch.float32 and rope.is_contiguous()
            assert tuple(rope.shape) == (h.shape[0], 64, 2)
            rp = rope.data_ptr()
        st = self.lib.bicache_project_prefix_layer_rope(self.ctx, prefix_id, layer, h.data_ptr(), h.stride(0),
                                                        w_k.data_ptr(), w_v.data_ptr(), h.shape[1], rp,
                                                        self._stream())
        self._check(st, "bicache_project_prefix_layer_rope")

    def prefix_similarity(self, prefix_id, k_ref, v_ref):
        """Eq. 3 per layer: cosine between the cached K/V of a prefix and k_ref, v_ref [L, m, Hkv, D]."""
        assert k_ref.is_cuda and v_ref.is_cuda and k_ref.dtype == self.dtype and k_ref.shape == v_ref.shape
        assert k_ref.stride()[1:] == (self.Hkv * self.D, self.D, 1) and v_ref.stride() == k_ref.stride()
        sim = np.zeros(self.L, dtype=np.float32)
        st = self.lib.bicache_prefix_similarity(self.ctx, prefix_id, k_ref.data_ptr(), v_ref.data_ptr(),
                                                k_ref.stride(0), sim.ctypes.data_as(C.POINTER(C.c_float)),
                                                self._stream())
        self._check(st, "bicache_prefix_similarity")
        return sim

    def prefix_similarity_async(self, prefix_id, k_ref, v_ref, sim_dev):
        """As prefix_similarity, result into the device tensor sim_dev [L] (float32), no synchronisation."""
        assert k_ref.is_cuda and v_ref.is_cuda and k_ref.dtype == self.dtype and k_ref.shape == v_ref.shape
        assert k_ref.stride()[1:] == (self.Hkv * self.D, self.D, 1) and v_ref.stride() == k_ref.stride()
        assert sim_dev.is_cuda and sim_dev.dtype == torch.float32 and sim_dev.numel() >= self.L and sim_dev.is_contiguous()
        st = self.lib.bicache_prefix_similarity_async(self.ctx, prefix_id, k_ref.data_ptr(), v_ref.data_ptr(),
                                                      k_ref.stride(0), sim_dev.data_ptr(), self._stream())
        self._check(st, "bicache_prefix_similarity_async")

    def is_refresh_step(self, t, delta):
        return int(self.lib.bicache_is_refresh_step(t, delta))

    def attend_step(self, layer, t, delta, depth, shared_id, private_id, row_off, seqlen, q, k, v, out, lse=None,
                    scale=None):
        d, pd = _i32(depth)
        sid, psid = _i32(shared_id)
        prid, pprid = _i32(private_id)
        off, poff = _i64(row_off)
        n, pn = _i32(seqlen)
        qp, kp, vp_, qs, ks, op, os_, lp = self._tensor_args(q, k, v, out, lse)
        scale = self.D ** -0.5 if scale is None else scale
        st = self.lib.bicache_attend_step(self.ctx, layer, t, delta, len(n), pd, psid, pprid, poff, pn, qp, kp, vp_,
                                          qs, ks, op, os_, lp, C.c_float(scale), self._stream())
        self._check(st, "bicache_attend_step")

    def lookup_prefix(self, key):
        pid, m = C.c_int32(-1), C.c_int32(0)
        self._check(self.lib.bicache_lookup_prefix(self.ctx, C.c_uint64(key), C.byref(pid), C.byref(m)),
                    "bicache_lookup_prefix")
        return pid.value, m.value

    def prefix_pages(self, prefix_id, layer=-1):
        """Page list of a prefix in `layer` (default: its first layer)."""
        n = C.c_int32(0)
        self._check(self.lib.bicache_prefix_pages_layer(self.ctx, prefix_id, layer, None, 0, C.byref(n)),
                    "bicache_prefix_pages_layer")
        pages = np.zeros(max(n.value, 1), dtype=np.int32)
        self._check(self.lib.bicache_prefix_pages_layer(self.ctx, prefix_id, layer,
                                                        pages.ctypes.data_as(C.POINTER(C.c_int32)), n.value,
                                                        C.byref(n)), "bicache_prefix_pages_layer")
        return pages[:n.value].tolist()

    def reuse_depth(self, prefix_len, nonshared_len):
        a, pa = _i32(prefix_len)
        b, pb = _i32(nonshared_len)
        out = np.zeros(max(len(a), 1), dtype=np.int32)
        self._check(self.lib.bicache_reuse_depth(self.ctx, len(a), pa, pb, out.ctypes.data_as(C.POINTER(C.c_int32))),
                    "bicache_reuse_depth")
        return out[:len(a)]

    def _tensor_args(self, q, k, v, out, lse):
        for t in (q, k, v, out):
            assert t.is_cuda and t.dtype == self.dtype and t.dim() == 3 and t.stride(2) == 1 and t.stride(1) == self.D
        assert lse is None or (lse.dtype == torch.float32 and lse.is_contiguous())
        return (q.data_ptr(), k.data_ptr(), v.data_ptr(), q.stride(0), k.stride(0),
                out.data_ptr(), out.stride(0), lse.data_ptr() if lse is not None else None)

    def attend(self, layer, prefix_id, row_off, seqlen, q, k, v, out, lse=None, scale=None):
        pid, ppid = _i32(prefix_id)
        off, poff = _i64(row_off)
        n, pn = _i32(seqlen)
        qp, kp, vp_, qs, ks, op, os_, lp = self._tensor_args(q, k, v, out, lse)
        scale = self.D ** -0.5 if scale is None else scale
        st = self.lib.bicache_attend(self.ctx, layer, len(n), ppid, poff, pn, qp, kp, vp_, qs, ks, op, os_, lp,
                                     C.c_float(scale), self._stream())
        self._check(st, "bicache_attend")

    def attend_full(self, layer, row_off, seqlen, q, k, v, out, lse=None, scale=None):
        off, poff = _i64(row_off)
        n, pn = _i32(seqlen)
        qp, kp, vp_, qs, ks, op, os_, lp = self._tensor_args(q, k, v, out, lse)
        scale = self.D ** -0.5 if scale is None else scale
        st = self.lib.bicache_attend_full(self.ctx, layer, len(n), poff, pn, qp, kp, vp_, qs, ks, op, os_, lp,
                                          C.c_float(scale), self._stream())
        self._check(st, "bicache_attend_full")

    def attend_layer(self, layer, depth, prefix_id, row_off, seqlen, q, k, v, out, lse=None, scale=None):
        d, pd = _i32(depth)
        pid, ppid = _i32(prefix_id)
        off, poff = _i64(row_off)
        n, pn = _i32(seqlen)
        qp, kp, vp_, qs, ks, op, os_, lp = self._tensor_args(q, k, v, out, lse)
        scale = self.D ** -0.5 if scale is None else scale
        st = self.lib.bicache_attend_layer(self.ctx, layer, len(n), pd, ppid, poff, pn, qp, kp, vp_, qs, ks, op, os_,
                                           lp, C.c_float(scale), self._stream())
        self._check(st, "bicache_attend_layer")

    def device_status(self, clear=False):
        return self.lib.bicache_device_status(self.ctx, self._stream(), 1 if clear else 0)

    def set_wait_budget(self, sm_cycles):
        self._check(self.lib.bicache_set_wait_budget(self.ctx, sm_cycles), "bicache_set_wait_budget")

    def last_attention_kernel(self):
        return self.lib.bicache_last_attention_kernel(self.ctx)

    def launch_count(self):
        return int(self.lib.bicache_launch_count(self.ctx))

    def schedule_uploads(self):
        return int(self.lib.bicache_schedule_uploads(self.ctx))


STATIC_MAX_ROW_HEADS = 4096


def attend_full_static(q, k, v, out, scale=None):
    """bicache_attend_full_static: full attention of one request without a context or workspace.

    For callers that may not allocate device memory: the scratch is a fixed array inside the
    library.  q, out [n, Hq, D]; k, v [n, Hkv, D] on the current CUDA device.  Returns the status
    code (0 = OK); n * Hq above STATIC_MAX_ROW_HEADS is refused with ERR_NOMEM."""
    lib = load_library()
    n, Hq, D = q.shape
    Hkv = k.shape[1]
    for t in (q, k, v, out):
        assert t.is_cuda and t.device == q.device and t.dtype == q.dtype and t.dim() == 3
        assert t.stride(2) == 1 and t.stride(1) == D, "heads must be dense within a row"
    assert k.shape == v.shape == (n, Hkv, D) and out.shape == q.shape
    assert q.device.index == torch.cuda.current_device(), "the call runs on the current device"
    scale = D ** -0.5 if scale is None else scale
    return lib.bicache_attend_full_static(_dtype_code(q.dtype), Hq, Hkv, D, n, q.data_ptr(), k.data_ptr(),
                                          v.data_ptr(), q.stride(0), k.stride(0), out.data_ptr(), out.stride(0),
                                          C.c_float(scale), C.c_void_p(torch.cuda.current_stream().cuda_stream))


def depth_from_similarity(sim, tau):
    """bicache_depth_from_similarity: leading layers with similarity >= tau."""
    lib = load_library()
    a = np.ascontiguousarray(sim, dtype=np.float32)
    d = C.c_int32(-1)
    st = lib.bicache_depth_from_similarity(a.ctypes.data_as(C.POINTER(C.c_float)), len(a), C.c_float(tau), C.byref(d))
    if st != OK:
        raise BiCacheError(st, "bicache_depth_from_similarity")
    return d.value


def build_depth_table(ratio_idx, depth, num_layers):
    """bicache_build_depth_table: the 101-entry lookup table from profiled (ratio bin, depth) pairs."""
    lib = load_library()
    r = np.ascontiguousarray(ratio_idx, dtype=np.int32)
    d = np.ascontiguousarray(depth, dtype=np.int32)
    out = np.zeros(101, dtype=np.int32)
    i32p = C.POINTER(C.c_int32)
    st = lib.bicache_build_depth_table(r.ctypes.data_as(i32p), d.ctypes.data_as(i32p), len(r), num_layers,
                                       out.ctypes.data_as(i32p))
    if st != OK:
        raise BiCacheError(st, "bicache_build_depth_table")
    return out.tolist()


def hash_tokens(tokens):
    """bicache_hash_tokens: the 64-bit store key of a prefix given as token ids."""
    lib = load_library()
    a = np.ascontiguousarray(tokens, dtype=np.int32)
    return int(lib.bicache_hash_tokens(a.ctypes.data_as(C.POINTER(C.c_int32)), len(a)))
