// Plain CUDA-core kernels: the page scatter of put_prefix, a straightforward fp32-accumulating
// attention (one warp per query row, online softmax with warp-shuffle reductions) that serves
// fp32 inputs and head dims the tensor-core path does not cover, and the log-sum-exp merge of
// partial results over disjoint key ranges.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"

namespace bicache {

struct TensorArgs {
  const char* q;
  const char* k;
  const char* v;
  char* out;
  float* lse;            // [rows][Hq] or nullptr
  long long q_stride;    // elements between rows
  long long kv_stride;
  long long out_stride;
  int Hq, Hkv, D;
  int layer;
  float scale;
  float* part_o;         // [splits][tokens][Hq][D] fp32, used when the keys are split
  float* part_lse;       // [splits][tokens][Hq]
  int total_tokens;      // sum of n over the call's requests
};

template <typename T> struct ElemTraits;
template <> struct ElemTraits<float> {
  static constexpr int kPerChunk = 4;
  static __device__ __forceinline__ void unpack(const uint4& c, float* f) {
    f[0] = __uint_as_float(c.x); f[1] = __uint_as_float(c.y);
    f[2] = __uint_as_float(c.z); f[3] = __uint_as_float(c.w);
  }
  static __device__ __forceinline__ float load(const char* p) { return *reinterpret_cast<const float*>(p); }
  static __device__ __forceinline__ void store(char* p, float x) { *reinterpret_cast<float*>(p) = x; }
};
template <> struct ElemTraits<__nv_bfloat16> {
  static constexpr int kPerChunk = 8;
  static __device__ __forceinline__ void unpack(const uint4& c, float* f) {
    const unsigned w[4] = {c.x, c.y, c.z, c.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      f[2 * i] = __uint_as_float(w[i] << 16);
      f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ float load(const char* p) {
    return __bfloat162float(*reinterpret_cast<const __nv_bfloat16*>(p));
  }
  static __device__ __forceinline__ void store(char* p, float x) {
    *reinterpret_cast<__nv_bfloat16*>(p) = __float2bfloat16_rn(x);
  }
};

// ---------------------------------------------------------------------------------------------
// put_prefix: scatter [L][m][Hkv][D] rows into pool pages (both K and V), zero-filling the unused
// slots of the last page so that a tile which covers them multiplies weight 0 by a finite value.
// One thread moves one 16-byte chunk.
// ---------------------------------------------------------------------------------------------
__global__ void scatter_prefix_kernel(const char* __restrict__ src_k, const char* __restrict__ src_v,
                                      char* __restrict__ pool_k, char* __restrict__ pool_v,
                                      const int* __restrict__ pages, int num_prefix_pages, int m,
                                      int num_layers, int num_kv_heads, int chunks_per_row,
                                      long long layer_stride_bytes, long long src_row_stride_bytes,
                                      long long pool_layer_bytes, int page_bytes, int swizzled) {
  const long long per_layer = (long long)num_prefix_pages * kPageSize * num_kv_heads * chunks_per_row;
  const long long total = per_layer * num_layers;
  const int row_bytes = chunks_per_row * 16;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int layer = (int)(idx / per_layer);
    long long rem = idx - (long long)layer * per_layer;
    const int c16 = (int)(rem % chunks_per_row); rem /= chunks_per_row;
    const int hk = (int)(rem % num_kv_heads); rem /= num_kv_heads;
    const int t = (int)rem;                        // token index, may be >= m inside the last page
    const int page = pages[t / kPageSize];
    const int slot = t % kPageSize;
    uint4 ck = make_uint4(0, 0, 0, 0), cv = ck;
    if (t < m) {
      const long long so = (long long)layer * layer_stride_bytes + (long long)t * src_row_stride_bytes +
                           (long long)hk * row_bytes + c16 * 16;
      ck = *reinterpret_cast<const uint4*>(src_k + so);
      cv = *reinterpret_cast<const uint4*>(src_v + so);
    }
    const long long po = (long long)layer * pool_layer_bytes +
                         ((long long)page * num_kv_heads + hk) * page_bytes +
                         page_chunk_offset(swizzled != 0, slot, c16, row_bytes);
    *reinterpret_cast<uint4*>(pool_k + po) = ck;
    *reinterpret_cast<uint4*>(pool_v + po) = cv;
  }
}

// ---------------------------------------------------------------------------------------------
// The inverse for one layer: pool pages -> dense rows [m][Hkv][D] (K and V).  One thread moves one
// 16-byte chunk of each.
// ---------------------------------------------------------------------------------------------
__global__ void gather_prefix_kernel(const char* __restrict__ pool_k, const char* __restrict__ pool_v,
                                     char* __restrict__ dst_k, char* __restrict__ dst_v,
                                     const int* __restrict__ pages, int m, int num_kv_heads, int chunks_per_row,
                                     long long dst_row_stride_bytes, int page_bytes, int swizzled) {
  const long long total = (long long)m * num_kv_heads * chunks_per_row;
  const int row_bytes = chunks_per_row * 16;
  for (long long idx = blockIdx.x * (long long)blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    long long rem = idx;
    const int c16 = (int)(rem % chunks_per_row); rem /= chunks_per_row;
    const int hk = (int)(rem % num_kv_heads); rem /= num_kv_heads;
    const int t = (int)rem;
    const long long po = ((long long)pages[t / kPageSize] * num_kv_heads + hk) * page_bytes +
                         page_chunk_offset(swizzled != 0, t % kPageSize, c16, row_bytes);
    const long long d = (long long)t * dst_row_stride_bytes + (long long)hk * row_bytes + c16 * 16;
    *reinterpret_cast<uint4*>(dst_k + d) = *reinterpret_cast<const uint4*>(pool_k + po);
    *reinterpret_cast<uint4*>(dst_v + d) = *reinterpret_cast<const uint4*>(pool_v + po);
  }
}

// ---------------------------------------------------------------------------------------------
// Profiler reduction (Eq. 3): for every layer the three sums behind
//   sim_l = cos(KV$_l, KVref_l) = <a, b> / (|a| |b|),
// a = the cached prefix's K and V of layer l read through the page table, b = the reference K and V
// [L][m][Hkv][D], each side taken as one vector.  HBM bound: both sides are read once, 16 bytes per
// thread and step; consecutive threads walk the reference in memory order (the page image holds the
// same chunks permuted inside 128-byte rows).  Products and squares are summed in fp32 inside a
// chunk, in fp64 across chunks; each block writes its three partial sums and a second kernel adds
// them in a fixed order, so the result does not depend on scheduling.
// ---------------------------------------------------------------------------------------------
constexpr int kSimBlocksPerLayer = 128;
constexpr int kSimThreads = 256;

template <typename T>
__device__ __forceinline__ void chunk_sums(const uint4& a, const uint4& b, float& dot, float& na, float& nb);
template <>
__device__ __forceinline__ void chunk_sums<float>(const uint4& a, const uint4& b, float& dot, float& na, float& nb) {
  const float* x = reinterpret_cast<const float*>(&a);
  const float* y = reinterpret_cast<const float*>(&b);
  dot = na = nb = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    dot = fmaf(x[i], y[i], dot);
    na = fmaf(x[i], x[i], na);
    nb = fmaf(y[i], y[i], nb);
  }
}
template <>
__device__ __forceinline__ void chunk_sums<__nv_bfloat16>(const uint4& a, const uint4& b, float& dot, float& na,
                                                           float& nb) {
  const __nv_bfloat162* x = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* y = reinterpret_cast<const __nv_bfloat162*>(&b);
  dot = na = nb = 0.f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 xf = __bfloat1622float2(x[i]), yf = __bfloat1622float2(y[i]);
    dot = fmaf(xf.x, yf.x, fmaf(xf.y, yf.y, dot));
    na = fmaf(xf.x, xf.x, fmaf(xf.y, xf.y, na));
    nb = fmaf(yf.x, yf.x, fmaf(yf.y, yf.y, nb));
  }
}

template <typename T>
__global__ void __launch_bounds__(kSimThreads)
kv_similarity_partial_kernel(const char* __restrict__ pool_k, const char* __restrict__ pool_v,
                             const char* __restrict__ ref_k, const char* __restrict__ ref_v,
                             const int* __restrict__ pages, int m, int num_kv_heads, int chunks_per_row,
                             long long ref_layer_stride_bytes, long long pool_layer_bytes, int page_bytes,
                             int swizzled, double* __restrict__ partials) {
  // Rows of the layer: the m K rows, then the m V rows; a block takes a contiguous range of them.
  // A thread keeps its chunk column(s) of the row and walks down the rows, so the per-chunk work is
  // two loads, a handful of integer operations and the sums (no division in the loop).
  const int layer = blockIdx.y;
  const int row_bytes = chunks_per_row * 16;
  const int row_chunks = num_kv_heads * chunks_per_row;     // 16-byte chunks of one token row
  const int tpr = min(row_chunks, (int)blockDim.x);         // threads that share a row
  const int rpp = (int)blockDim.x / tpr;                    // rows in flight per pass
  const int r_local = (int)threadIdx.x / tpr, c0 = (int)threadIdx.x - r_local * tpr;
  const int rows = 2 * m;
  const int per_block = (rows + (int)gridDim.x - 1) / (int)gridDim.x;
  const int row_begin = (int)blockIdx.x * per_block, row_end = min(rows, row_begin + per_block);
  const char* pool_k_l = pool_k + (long long)layer * pool_layer_bytes;
  const char* pool_v_l = pool_v + (long long)layer * pool_layer_bytes;
  const char* ref_k_l = ref_k + (long long)layer * ref_layer_stride_bytes;
  const char* ref_v_l = ref_v + (long long)layer * ref_layer_stride_bytes;
  const long long page_stride = (long long)num_kv_heads * page_bytes;
  double dot = 0.0, na = 0.0, nb = 0.0;
  constexpr int kUnroll = 4;                      // loads of four rows in flight before any arithmetic
  if (r_local < rpp) {
    for (int c = c0; c < row_chunks; c += tpr) {
      const int hk = c / chunks_per_row, c16 = c - hk * chunks_per_row;
      const long long slice = (long long)hk * page_bytes;
      for (int base = row_begin + r_local; base < row_end; base += kUnroll * rpp) {
        uint4 a[kUnroll], b[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
          const int row = base + u * rpp;
          a[u] = make_uint4(0, 0, 0, 0);
          b[u] = a[u];
          if (row < row_end) {
            const bool is_v = row >= m;
            const int t = is_v ? row - m : row;
            const int page = pages[t / kPageSize];
            const char* pa = (is_v ? pool_v_l : pool_k_l) + page * page_stride + slice +
                             page_chunk_offset(swizzled != 0, t % kPageSize, c16, row_bytes);
            const char* pb = (is_v ? ref_v_l : ref_k_l) + ((long long)t * row_chunks + c) * 16;
            a[u] = *reinterpret_cast<const uint4*>(pa);
            b[u] = *reinterpret_cast<const uint4*>(pb);
          }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {       // rows past the end are zeros and add nothing
          float d, x, y;
          chunk_sums<T>(a[u], b[u], d, x, y);
          dot += d;
          na += x;
          nb += y;
        }
      }
    }
  }
  // block reduction in a fixed order: shuffles inside a warp, then warp 0 over the warps' sums
  __shared__ double red[3][kSimThreads / 32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    dot += __shfl_down_sync(0xffffffffu, dot, o);
    na += __shfl_down_sync(0xffffffffu, na, o);
    nb += __shfl_down_sync(0xffffffffu, nb, o);
  }
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    red[0][warp] = dot;
    red[1][warp] = na;
    red[2][warp] = nb;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    double s0 = 0.0, s1 = 0.0, s2 = 0.0;
    for (int w = 0; w < kSimThreads / 32; ++w) {
      s0 += red[0][w];
      s1 += red[1][w];
      s2 += red[2][w];
    }
    double* out = partials + ((long long)layer * gridDim.x + blockIdx.x) * 3;
    out[0] = s0;
    out[1] = s1;
    out[2] = s2;
  }
}

// One thread per layer adds the blocks' partial sums in block order and forms the cosine.
__global__ void kv_similarity_final_kernel(const double* __restrict__ partials, int blocks_per_layer, int num_layers,
                                           float* __restrict__ sim) {
  const int layer = blockIdx.x * blockDim.x + threadIdx.x;
  if (layer >= num_layers) return;
  double dot = 0.0, na = 0.0, nb = 0.0;
  for (int b = 0; b < blocks_per_layer; ++b) {
    const double* p = partials + ((long long)layer * blocks_per_layer + b) * 3;
    dot += p[0];
    na += p[1];
    nb += p[2];
  }
  sim[layer] = (na > 0.0 && nb > 0.0) ? (float)(dot / (sqrt(na) * sqrt(nb))) : 0.f;
}

// ---------------------------------------------------------------------------------------------
// SIMT attention.  One block = one work item (128 packed rows of one request and KV head); each
// warp takes packed rows warp, warp + nwarps, ...  Keys are visited 32 at a time: lane j scores
// key j, the chunk maximum and sum are reduced with shuffles, and P.V is accumulated with each lane
// owning dims lane, lane + 32, ...
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

constexpr int kSimtWarps = 4;
constexpr int kSimtMaxD = 256;

template <typename T>
__global__ void __launch_bounds__(kSimtWarps * 32)
simt_attention_kernel(ScheduleView s, PoolView pool, TensorArgs t) {
  using Tr = ElemTraits<T>;
  constexpr int kEsize = (int)sizeof(T);
  __shared__ float qs[kSimtWarps][kSimtMaxD];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const WorkItem item = s.items[blockIdx.x];
  const ReqMeta req = s.reqs[item.req];
  const int G = t.Hq / t.Hkv;
  const int D = t.D;
  const int row_bytes = D * kEsize;
  const int chunks = row_bytes / 16;
  const int dims_per_lane = D / 32;
  // Key tiles: ceil(m/128) tiles of cached prefix keys, then ceil(n/128) tiles of own keys; a key
  // split covers a contiguous range of tiles.
  const int prefix_tiles = (req.m + kTileKeys - 1) / kTileKeys;
  const int all_tiles = prefix_tiles + (req.n + kTileKeys - 1) / kTileKeys;
  int tile_begin = 0, tile_end = all_tiles;
  if (s.num_splits > 1) {
    tile_begin = min(all_tiles, item.split * s.tiles_per_split);
    tile_end = min(all_tiles, tile_begin + s.tiles_per_split);
  }
  const int pre_begin = min(req.m, tile_begin * kTileKeys), pre_end = min(req.m, tile_end * kTileKeys);
  const int own_begin = min(req.n, max(0, tile_begin - prefix_tiles) * kTileKeys);
  const int own_end = min(req.n, max(0, tile_end - prefix_tiles) * kTileKeys);
  const int* pages = s.pages + req.page_off;
  const int row_end = min(item.row0 + kTileRows, req.n * G);

  for (int p = item.row0 + warp; p < row_end; p += kSimtWarps) {
    const int a = p / G;
    const int h = item.kv_head * G + (p - a * G);
    const char* qrow = t.q + ((req.row_off + a) * t.q_stride + (long long)h * D) * kEsize;
    __syncwarp();
    for (int d = lane; d < D; d += 32) qs[warp][d] = Tr::load(qrow + d * kEsize);
    __syncwarp();

    float m_run = -INFINITY, l_run = 0.f;
    float acc[kSimtMaxD / 32];
#pragma unroll
    for (int i = 0; i < kSimtMaxD / 32; ++i) acc[i] = 0.f;

    for (int part = 0; part < 2; ++part) {
      const bool paged = part == 0;
      const int key_begin = paged ? pre_begin : own_begin;
      const int key_end = paged ? pre_end : own_end;
      for (int key0 = key_begin; key0 < key_end; key0 += 32) {
        const int j = key0 + lane;
        const bool valid = j < key_end;
        float sc = -INFINITY;
        if (valid) {
          const char* base;
          int slot = 0;
          if (paged) {
            base = pool.k + pool_slice_offset(pool, t.layer, pages[j / kPageSize], item.kv_head);
            slot = j % kPageSize;
          } else {
            base = t.k + ((req.row_off + j) * t.kv_stride + (long long)item.kv_head * D) * kEsize;
          }
          float dot = 0.f;
          for (int c = 0; c < chunks; ++c) {
            const char* cp = paged ? base + page_chunk_offset(pool.swizzled != 0, slot, c, row_bytes)
                                   : base + c * 16;
            const uint4 raw = *reinterpret_cast<const uint4*>(cp);
            float f[Tr::kPerChunk];
            Tr::unpack(raw, f);
#pragma unroll
            for (int e = 0; e < Tr::kPerChunk; ++e) dot = fmaf(f[e], qs[warp][c * Tr::kPerChunk + e], dot);
          }
          sc = t.scale * dot;
        }
        const float m_new = fmaxf(m_run, warp_max(sc));
        const float pj = valid ? expf(sc - m_new) : 0.f;
        const float alpha = expf(m_run - m_new);          // exp(-inf) = 0 on the first chunk
        l_run = l_run * alpha + warp_sum(pj);
#pragma unroll
        for (int i = 0; i < kSimtMaxD / 32; ++i) acc[i] *= alpha;
        m_run = m_new;
        const int cnt = min(32, key_end - key0);
        for (int jj = 0; jj < cnt; ++jj) {
          const float w = __shfl_sync(0xffffffffu, pj, jj);
          const int key = key0 + jj;
          const char* base;
          int slot = 0;
          if (paged) {
            base = pool.v + pool_slice_offset(pool, t.layer, pages[key / kPageSize], item.kv_head);
            slot = key % kPageSize;
          } else {
            base = t.v + ((req.row_off + key) * t.kv_stride + (long long)item.kv_head * D) * kEsize;
          }
#pragma unroll
          for (int i = 0; i < kSimtMaxD / 32; ++i) {
            if (i < dims_per_lane) {
              const int d = lane + 32 * i;
              const int c = d / Tr::kPerChunk, e = d % Tr::kPerChunk;
              const char* ep = paged ? base + page_chunk_offset(pool.swizzled != 0, slot, c, row_bytes) + e * kEsize
                                     : base + d * kEsize;
              acc[i] = fmaf(w, Tr::load(ep), acc[i]);
            }
          }
        }
      }
    }

    const bool any = pre_end > pre_begin || own_end > own_begin;
    const float inv = any ? 1.f / l_run : 0.f;
    const float lse = any ? m_run + logf(l_run) : -INFINITY;
    if (s.num_splits > 1) {
      const long long pr = ((long long)item.split * t.total_tokens + req.tok_off + a) * t.Hq + h;
#pragma unroll
      for (int i = 0; i < kSimtMaxD / 32; ++i)
        if (i < dims_per_lane) t.part_o[pr * D + lane + 32 * i] = acc[i] * inv;
      if (lane == 0) t.part_lse[pr] = lse;
    } else {
      char* orow = t.out + ((req.row_off + a) * t.out_stride + (long long)h * D) * kEsize;
#pragma unroll
      for (int i = 0; i < kSimtMaxD / 32; ++i)
        if (i < dims_per_lane) Tr::store(orow + (lane + 32 * i) * kEsize, acc[i] * inv);
      if (lane == 0 && t.lse != nullptr) t.lse[(req.row_off + a) * t.Hq + h] = lse;
    }
  }
}

// ---------------------------------------------------------------------------------------------
// Log-sum-exp merge of the partial results of `num_splits` disjoint key ranges:
//   lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s.
// An empty part carries lse = -inf and weighs 0.  One block per split-0 work item, one warp per
// packed row.
// ---------------------------------------------------------------------------------------------
constexpr int kMergeRowsPerBlock = 8;   // packed rows per block of the merge kernel (one warp each)

template <typename T>
__global__ void __launch_bounds__(kMergeRowsPerBlock * 32)
merge_partials_kernel(ScheduleView s, TensorArgs t) {
  using Tr = ElemTraits<T>;
  constexpr int kEsize = (int)sizeof(T);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // blockIdx.x enumerates (split-0 work item, group of kMergeRowsPerBlock packed rows); the first
  // num_items / num_splits items of the schedule are the split-0 items.
  constexpr int kBlocksPerItem = kTileRows / kMergeRowsPerBlock;
  const WorkItem item = s.items[blockIdx.x / kBlocksPerItem];
  const ReqMeta req = s.reqs[item.req];
  const int G = t.Hq / t.Hkv;
  const int D = t.D;
  const int p = item.row0 + (blockIdx.x % kBlocksPerItem) * kMergeRowsPerBlock + warp;
  if (p >= req.n * G) return;
  const int a = p / G;
  const int h = item.kv_head * G + (p - a * G);
  const long long pr0 = ((long long)req.tok_off + a) * t.Hq + h;
  const long long split_stride = (long long)t.total_tokens * t.Hq;
  // lane sp holds the lse of split sp (+32, ...): maximum and total weight by shuffles
  float mx = -INFINITY;
  for (int sp = lane; sp < s.num_splits; sp += 32) mx = fmaxf(mx, t.part_lse[pr0 + sp * split_stride]);
  mx = warp_max(mx);
  float tot = 0.f;
  for (int sp = lane; sp < s.num_splits; sp += 32) tot += expf(t.part_lse[pr0 + sp * split_stride] - mx);
  tot = warp_sum(tot);
  const bool any = mx > -INFINITY;
  const float inv_tot = any ? 1.f / tot : 0.f;
  char* orow = t.out + ((req.row_off + a) * t.out_stride + (long long)h * D) * kEsize;
  float acc[kSimtMaxD / 32];
#pragma unroll
  for (int i = 0; i < kSimtMaxD / 32; ++i) acc[i] = 0.f;
  if (any) {
    // Lane l holds the weights of splits l, l + 32, ...; the partial rows of eight splits are
    // loaded before any is used, so that their latencies overlap.
    for (int base = 0; base < s.num_splits; base += 32) {
      const int mine = base + lane;
      const float w_lane = mine < s.num_splits ? expf(t.part_lse[pr0 + mine * split_stride] - mx) * inv_tot : 0.f;
      const int cnt = min(32, s.num_splits - base);
      for (int s0 = 0; s0 < cnt; s0 += 8) {
        float v[8][kSimtMaxD / 32];
        float w[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const int sp = min(s0 + u, cnt - 1);               // a clamped repeat gets weight 0 below
          const float w_sp = __shfl_sync(0xffffffffu, w_lane, sp);
          w[u] = s0 + u < cnt ? w_sp : 0.f;
          const float* po = t.part_o + (pr0 + (long long)(base + sp) * split_stride) * D;
#pragma unroll
          for (int i = 0; i < kSimtMaxD / 32; ++i) v[u][i] = lane + 32 * i < D ? po[lane + 32 * i] : 0.f;
        }
#pragma unroll
        for (int u = 0; u < 8; ++u)
#pragma unroll
          for (int i = 0; i < kSimtMaxD / 32; ++i) acc[i] = fmaf(w[u], v[u][i], acc[i]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < kSimtMaxD / 32; ++i)
    if (lane + 32 * i < D) Tr::store(orow + (lane + 32 * i) * kEsize, acc[i]);
  if (lane == 0 && t.lse != nullptr)
    t.lse[(req.row_off + a) * t.Hq + h] = any ? mx + logf(tot) : -INFINITY;
}

}  // namespace bicache
