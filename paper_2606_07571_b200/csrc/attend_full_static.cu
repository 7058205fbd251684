// bicache_attend_full_static: full bidirectional attention of one request that needs neither a
// context nor a caller-provided workspace.
//
// Who needs this: code that is not allowed to allocate device memory at the point where it wants
// attention - a plugin running inside another framework's memory plan, a real-time serving loop
// that must not touch the allocator after start-up, or a process whose memory budget was fixed
// before this library was loaded.  The regular calls take their scratch (partial results of the
// key splits, schedules) from a workspace the caller allocates; here the scratch is a fixed array
// that lives in the library's device image, so nothing is allocated by anybody.
//
// The kernels are a variant of the key-split CUDA-core attention + log-sum-exp merge used by the
// regular path: the keys of the request are cut into kStaticSplits ranges, every (row, head, range)
// is computed by one warp with an online softmax, the partial (o, lse) go to the static array, and
// a second kernel merges the ranges.
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/bicache.h"

namespace {

constexpr int kStaticSplits = 4;
constexpr int kStaticMaxRowHeads = BICACHE_STATIC_MAX_ROW_HEADS;      // n_rows * num_q_heads
constexpr int kStaticMaxD = 128;
constexpr int kStaticFloatsPerPartial = kStaticMaxD + 1;              // o[D] and lse
constexpr size_t kStaticScratchFloats = (size_t)kStaticMaxRowHeads * kStaticSplits * kStaticFloatsPerPartial;
constexpr int kMaxDevices = 64;

// The scratch itself: 4096 x 4 x 129 floats = 8,454,144 bytes (8.06 MiB) of every GPU that loads this
// library's device code, until the process exits.  With CUDA's lazy module loading the device code of
// this file is loaded, and the array backed, by the first call on a device (the address lookup below).
// In host code this name is only a handle; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

// Device address of the array, per device, looked up once.  Plain host state: not synchronised between
// host threads, and stale after a cudaDeviceReset of that device (a process that resets a device must not
// call this entry point on it again).
float* g_scratch_addr[kMaxDevices] = {nullptr};

template <typename T> __device__ __forceinline__ float ld_elem(const T* p);
template <> __device__ __forceinline__ float ld_elem<float>(const float* p) { return *p; }
template <> __device__ __forceinline__ float ld_elem<__nv_bfloat16>(const __nv_bfloat16* p) { return __bfloat162float(*p); }
template <typename T> __device__ __forceinline__ void st_elem(T* p, float x);
template <> __device__ __forceinline__ void st_elem<float>(float* p, float x) { *p = x; }
template <> __device__ __forceinline__ void st_elem<__nv_bfloat16>(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }

__device__ __forceinline__ float wmax(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float wsum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// One warp per (row, head, key range): lane j scores key j of each 32-key chunk; maximum and sum
// are reduced with shuffles; each lane accumulates dims lane, lane + 32, ...
template <typename T>
__global__ void __launch_bounds__(128)
static_partial_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                      long long q_stride, long long kv_stride, int n_rows, int Hq, int Hkv, int D,
                      float scale, float* __restrict__ scratch) {
  __shared__ float qs[4][kStaticMaxD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rh = blockIdx.x * 4 + warp;                   // row * Hq + head
  const int split = blockIdx.y;
  if (rh >= n_rows * Hq) return;
  const int row = rh / Hq, h = rh - row * Hq, hk = h / (Hq / Hkv);
  const int per = (n_rows + kStaticSplits - 1) / kStaticSplits;
  const int key_begin = min(n_rows, split * per), key_end = min(n_rows, key_begin + per);
  for (int d = lane; d < D; d += 32) qs[warp][d] = ld_elem(q + row * q_stride + (long long)h * D + d);
  __syncwarp();
  float m_run = -INFINITY, l_run = 0.f, acc[kStaticMaxD / 32];
#pragma unroll
  for (int i = 0; i < kStaticMaxD / 32; ++i) acc[i] = 0.f;
  for (int key0 = key_begin; key0 < key_end; key0 += 32) {
    const int j = key0 + lane;
    const bool valid = j < key_end;
    float sc = -INFINITY;
    if (valid) {
      const T* kr = k + j * kv_stride + (long long)hk * D;
      float dot = 0.f;
      for (int d = 0; d < D; ++d) dot = fmaf(ld_elem(kr + d), qs[warp][d], dot);
      sc = scale * dot;
    }
    const float m_new = fmaxf(m_run, wmax(sc));
    const float pj = valid ? expf(sc - m_new) : 0.f;
    const float alpha = expf(m_run - m_new);
    l_run = l_run * alpha + wsum(pj);
#pragma unroll
    for (int i = 0; i < kStaticMaxD / 32; ++i) acc[i] *= alpha;
    m_run = m_new;
    const int cnt = min(32, key_end - key0);
    for (int jj = 0; jj < cnt; ++jj) {
      const float w = __shfl_sync(0xffffffffu, pj, jj);
      const T* vr = v + (long long)(key0 + jj) * kv_stride + (long long)hk * D;
#pragma unroll
      for (int i = 0; i < kStaticMaxD / 32; ++i)
        if (lane + 32 * i < D) acc[i] = fmaf(w, ld_elem(vr + lane + 32 * i), acc[i]);
    }
  }
  const bool any = key_end > key_begin;
  float* part = scratch + ((size_t)split * kStaticMaxRowHeads + rh) * kStaticFloatsPerPartial;
#pragma unroll
  for (int i = 0; i < kStaticMaxD / 32; ++i)
    if (lane + 32 * i < D) part[lane + 32 * i] = any ? acc[i] / l_run : 0.f;
  if (lane == 0) part[kStaticMaxD] = any ? m_run + logf(l_run) : -INFINITY;
}

// Merge of the key ranges: lse = log sum_s exp(lse_s), o = sum_s exp(lse_s - lse) o_s.
template <typename T>
__global__ void __launch_bounds__(128)
static_merge_kernel(T* __restrict__ out, long long out_stride, int n_rows, int Hq, int D,
                    const float* __restrict__ scratch) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rh = blockIdx.x * 4 + warp;
  if (rh >= n_rows * Hq) return;
  const int row = rh / Hq, h = rh - row * Hq;
  float lse[kStaticSplits], mx = -INFINITY;
#pragma unroll
  for (int s = 0; s < kStaticSplits; ++s) {
    lse[s] = scratch[((size_t)s * kStaticMaxRowHeads + rh) * kStaticFloatsPerPartial + kStaticMaxD];
    mx = fmaxf(mx, lse[s]);
  }
  float tot = 0.f;
#pragma unroll
  for (int s = 0; s < kStaticSplits; ++s) tot += expf(lse[s] - mx);
  for (int d = lane; d < D; d += 32) {
    float o = 0.f;
#pragma unroll
    for (int s = 0; s < kStaticSplits; ++s)
      o = fmaf(expf(lse[s] - mx) / tot,
               scratch[((size_t)s * kStaticMaxRowHeads + rh) * kStaticFloatsPerPartial + d], o);
    st_elem(out + row * out_stride + (long long)h * D + d, o);
  }
}

template <typename T>
cudaError_t launch_static(const void* q, const void* k, const void* v, long long qs, long long kvs, void* out,
                          long long os, int n, int Hq, int Hkv, int D, float scale, float* scratch,
                          cudaStream_t stream) {
  const dim3 grid((n * Hq + 3) / 4, kStaticSplits);
  static_partial_kernel<T><<<grid, 128, 0, stream>>>(static_cast<const T*>(q), static_cast<const T*>(k),
                                                     static_cast<const T*>(v), qs, kvs, n, Hq, Hkv, D, scale, scratch);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  static_merge_kernel<T><<<grid.x, 128, 0, stream>>>(static_cast<T*>(out), os, n, Hq, D, scratch);
  return cudaGetLastError();
}

}  // namespace

extern "C" int32_t bicache_attend_full_static(int32_t dtype, int32_t num_q_heads, int32_t num_kv_heads,
                                              int32_t head_dim, int32_t n_rows, const void* q, const void* k,
                                              const void* v, int64_t q_row_stride, int64_t kv_row_stride,
                                              void* out, int64_t out_row_stride, float softmax_scale,
                                              void* stream) {
  if (dtype != BICACHE_F32 && dtype != BICACHE_BF16) return BICACHE_ERR_UNSUPPORTED;
  if (head_dim < 32 || head_dim > kStaticMaxD || head_dim % 32) return BICACHE_ERR_UNSUPPORTED;
  if (num_kv_heads < 1 || num_q_heads < num_kv_heads || num_q_heads % num_kv_heads || n_rows < 0)
    return BICACHE_ERR_INVALID;
  // The static array holds kStaticMaxRowHeads partial rows per key range: larger problems are refused.
  if ((int64_t)n_rows * num_q_heads > kStaticMaxRowHeads) return BICACHE_ERR_NOMEM;
  if (n_rows == 0) return BICACHE_OK;
  if (!q || !k || !v || !out) return BICACHE_ERR_INVALID;
  if (q_row_stride < (int64_t)num_q_heads * head_dim || out_row_stride < (int64_t)num_q_heads * head_dim ||
      kv_row_stride < (int64_t)num_kv_heads * head_dim)
    return BICACHE_ERR_INVALID;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return BICACHE_ERR_CUDA;
  if (g_scratch_addr[dev] == nullptr) {
    // First call on this device: resolve the device address of the static array.  The symbol name
    // itself is not a device pointer in host code.
    float* p = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_static_scratch) != cudaSuccess || p == nullptr)
      return BICACHE_ERR_CUDA;
    g_scratch_addr[dev] = p;
  }
  float* scratch = g_scratch_addr[dev];
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  cudaError_t e = dtype == BICACHE_F32
      ? launch_static<float>(q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, n_rows, num_q_heads,
                             num_kv_heads, head_dim, softmax_scale, scratch, s)
      : launch_static<__nv_bfloat16>(q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, n_rows,
                                     num_q_heads, num_kv_heads, head_dim, softmax_scale, scratch, s);
  return e == cudaSuccess ? BICACHE_OK : BICACHE_ERR_CUDA;
}
