// Tensor-core attention for bf16, head_dim 128, on sm_100a: tcgen05.mma with TMEM accumulators.
//
// One CTA computes one work item: 128 packed query rows (one request, one KV head) against a
// range of key tiles of 128 keys - first the cached prefix (pages of 16 tokens, staged with
// cp.async.bulk because a pool page already is the shared-memory image the MMA reads), then the
// request's own rows (16-byte cp.async gathers from the caller's row-major K/V, zero-filled past
// the end).  Per tile: S = Q K^T (tcgen05, fp32 in TMEM) -> online softmax in registers
// (one thread per row) -> P as bf16 back to TMEM -> O += P V (tcgen05, A operand from TMEM).
// The running maximum only moves when it grew by more than 2^8, so rescaling O is rare; the
// final normalisation uses the same reference, which keeps the result exact.
//
// Roles: warps 0-3 softmax / correction / epilogue, warp 4 MMA issue and TMEM ownership,
// warps 5-8 loads.  All waits are bounded; a wait that gives up raises a sticky status word
// and the CTA drains and exits.
#pragma once
#include <cuda_bf16.h>
#include "common.cuh"
#include "simt_kernels.cuh"

namespace bicache {

constexpr bool kTensorPathBuilt = true;

namespace tc {

constexpr int kStages = 3;                       // K/V ring depth
constexpr int kTileBytes = kTileKeys * 128 * 2;  // 32 KB: one 128 x 128 bf16 tile
constexpr int kPageBytes = 4096;
constexpr int kThreads = 288;
constexpr int kSoftmaxThreads = 128;
constexpr int kLoadThreads = 128;
constexpr unsigned kMaxPolls = 1u << 21;         // bounded waits: about a quarter of a second

// shared-memory layout (dynamic, 1024-byte aligned by hand)
struct alignas(8) Barriers {
  unsigned long long q_full;
  unsigned long long kv_full[kStages];
  unsigned long long kv_free[kStages];
  unsigned long long s_full[2];
  unsigned long long s_free[2];
  unsigned long long p_full[2];
  unsigned long long o_done;
  unsigned long long drain;
  unsigned tmem_base;
  int abort_flag;
};
constexpr int kSmemBytes = 1024 + kTileBytes * (1 + 2 * kStages) + (int)sizeof(Barriers) + 64;

// ----- raw PTX wrappers --------------------------------------------------------------------
__device__ __forceinline__ unsigned smem_u32(const void* p) {
  return (unsigned)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(unsigned bar, unsigned count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned bar, unsigned bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false (and raises the CTA's abort flag) if the phase never completes.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
  for (unsigned it = 0; it < kMaxPolls; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it >= 32) {
      __nanosleep(64);
      if (*abort_flag) return false;
    }
  }
  *abort_flag = 1;
  return false;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_barrier_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void cp_async16(unsigned dst, const void* src, unsigned src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

__device__ __forceinline__ void bulk_copy_g2s(unsigned dst, const void* src, unsigned bytes, unsigned bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst), "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}

__device__ __forceinline__ void tmem_alloc(unsigned smem_slot, unsigned cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
__device__ __forceinline__ void mma_commit(unsigned bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem] * B[smem]
__device__ __forceinline__ void mma_ss(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                       unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem]
__device__ __forceinline__ void mma_ts(unsigned d_tmem, unsigned a_tmem, unsigned long long b_desc,
                                       unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_ld32(unsigned taddr, unsigned* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_st32(unsigned taddr, const unsigned* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
      "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
        "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
        "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st16(unsigned taddr, const unsigned* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
      ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
        "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ unsigned pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);     // .x = lo (low 16 bits), .y = hi
  return *reinterpret_cast<unsigned*>(&v);
}

// Shared-memory matrix descriptor, 128-byte swizzle, for the tile image used everywhere here:
// 16-row blocks of 4 KB = [rows 0-7, dims 0-63 | rows 0-7, dims 64-127 | rows 8-15, dims 0-63 |
// rows 8-15, dims 64-127]; 8-row groups are 2048 bytes apart, the two 64-dim halves 1024 bytes.
//   K-major operand (Q, K: the contraction runs over dims): stride-dimension offset = 2048
//   (between 8-row groups); a K step of 16 dims is 32 bytes inside the swizzled 128-byte row.
//   MN-major operand (V: the contraction runs over keys = rows): leading-dimension offset = 1024
//   (between the two 64-dim halves), stride-dimension offset = 2048 (between 8-key groups).
__device__ __forceinline__ unsigned long long make_desc(unsigned smem_addr, unsigned lbo_bytes, unsigned sbo_bytes) {
  unsigned long long d = 0;
  d |= (unsigned long long)((smem_addr & 0x3FFFFu) >> 4);
  d |= (unsigned long long)(lbo_bytes >> 4) << 16;
  d |= (unsigned long long)(sbo_bytes >> 4) << 32;
  d |= 1ull << 46;                 // descriptor version of this architecture
  d |= 2ull << 61;                 // 128-byte swizzle
  return d;
}
// Instruction descriptor: fp32 accumulate, bf16 A and B, M = 128, N = 128.
constexpr unsigned kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);
constexpr unsigned kIdescQK = kIdescBase;                 // A, B both K-major
constexpr unsigned kIdescPV = kIdescBase | (1u << 16);    // B (= V) MN-major

// byte offset of 16-byte chunk c16 (0..15) of row r (0..127) inside a tile image
__device__ __forceinline__ unsigned tile_chunk_offset(int r, int c16) {
  return (unsigned)((r >> 4) * kPageBytes) + page_chunk_offset(true, r & 15, c16, 256);
}

}  // namespace tc

__global__ void __launch_bounds__(tc::kThreads, 1)
tc_attention_kernel(ScheduleView s, PoolView pool, TensorArgs t, int* status) {
  using namespace tc;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Barriers* bars = reinterpret_cast<Barriers*>(smem + kTileBytes * (1 + 2 * kStages));
  volatile int* abort_flag = &bars->abort_flag;
  const unsigned q_smem = smem_u32(smem);
  const unsigned kv_smem = q_smem + kTileBytes;             // stage i: K at 2i, V at 2i + 1

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const WorkItem item = s.items[blockIdx.x];
  const ReqMeta req = s.reqs[item.req];
  const int G = t.Hq / t.Hkv;
  const int prefix_tiles = (req.m + kTileKeys - 1) / kTileKeys;
  const int all_tiles = prefix_tiles + (req.n + kTileKeys - 1) / kTileKeys;
  int tile_begin = 0, tile_end = all_tiles;
  if (s.num_splits > 1) {
    tile_begin = min(all_tiles, item.split * s.tiles_per_split);
    tile_end = min(all_tiles, tile_begin + s.tiles_per_split);
  }
  const int T = tile_end - tile_begin;
  const int packed_rows = req.n * G;

  if (tid == 0) {
    bars->abort_flag = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    mbar_init(smem_u32(&bars->q_full), kLoadThreads);
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&bars->kv_full[i]), kLoadThreads);
      mbar_init(smem_u32(&bars->kv_free[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->s_full[i]), 1);
      mbar_init(smem_u32(&bars->s_free[i]), kSoftmaxThreads);
      mbar_init(smem_u32(&bars->p_full[i]), kSoftmaxThreads);
    }
    mbar_init(smem_u32(&bars->o_done), 1);
    mbar_init(smem_u32(&bars->drain), 1);
    fence_barrier_init();
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&bars->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&bars->tmem_base);
  const unsigned tmem_o = tmem + 256;
  const bool dead = *abort_flag != 0;        // an earlier CTA already gave up: do no work

  if (!dead && warp < 4) {
    // =========================== softmax / correction / epilogue ===========================
    const unsigned lane_base = (unsigned)(warp * 32) << 16;  // this warp's quarter of the TMEM lanes
    const float sl2 = t.scale * 1.4426950408889634f;         // scores are handled in the log2 domain
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    for (int j = 0; j < T; ++j) {
      const int b = j & 1;
      const unsigned tmem_s = tmem + b * 128 + lane_base;
      const unsigned tmem_p = tmem + 384 + b * 64 + lane_base;
      const int jg = tile_begin + j;
      const int cnt = jg < prefix_tiles ? min(kTileKeys, req.m - jg * kTileKeys)
                                        : min(kTileKeys, req.n - (jg - prefix_tiles) * kTileKeys);
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->s_full[b]), (j >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      // pass 1: row maximum of the scaled scores (columns >= cnt do not exist)
      float mx = -INFINITY;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        unsigned r[32];
        tmem_ld32(tmem_s + c * 32, r);
        tmem_wait_ld();
        if (cnt >= kTileKeys) {
#pragma unroll
          for (int i = 0; i < 32; ++i) mx = fmaxf(mx, __uint_as_float(r[i]) * sl2);
        } else {
#pragma unroll
          for (int i = 0; i < 32; ++i)
            if (c * 32 + i < cnt) mx = fmaxf(mx, __uint_as_float(r[i]) * sl2);
        }
      }
      // The reference maximum moves only when the row maximum outgrew it by more than 2^8.
      float alpha = 1.f;
      if (j == 0) {
        m_ref = mx;
      } else if (mx > m_ref + 8.f) {
        alpha = ex2(m_ref - mx);
        m_ref = mx;
      }
      if (j > 0) {
        // P[b] was read by the P.V product of tile j-2 and O is accumulated by that of tile j-1:
        // both have finished once o_done completed its phase for tile j-1.
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->o_done), (j - 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            unsigned r[32];
            tmem_ld32(tmem_o + lane_base + c * 32, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
            tmem_st32(tmem_o + lane_base + c * 32, r);
          }
          tmem_wait_st();
        }
      }
      // pass 2: p = 2^(s - m_ref), row sum, P as bf16 into TMEM (two values per 32-bit column)
      float psum = 0.f;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        unsigned r[32];
        tmem_ld32(tmem_s + c * 32, r);
        tmem_wait_ld();
        unsigned pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          float p0 = ex2(fmaf(__uint_as_float(r[2 * i]), sl2, -m_ref));
          float p1 = ex2(fmaf(__uint_as_float(r[2 * i + 1]), sl2, -m_ref));
          if (cnt < kTileKeys) {
            if (c * 32 + 2 * i >= cnt) p0 = 0.f;
            if (c * 32 + 2 * i + 1 >= cnt) p1 = 0.f;
          }
          psum += p0 + p1;
          pk[i] = pack_bf16(p0, p1);
        }
        tmem_st16(tmem_p + c * 16, pk);
      }
      tmem_wait_st();
      l_sum = l_sum * alpha + psum;
      tc_fence_before();
      mbar_arrive(smem_u32(&bars->s_free[b]));      // S[b] may be overwritten by tile j + 2
      mbar_arrive(smem_u32(&bars->p_full[b]));      // P[b] is complete, O is rescaled
    }
    // ------------------------------- epilogue -------------------------------------------
    const int prow = item.row0 + tid;                // packed row of this thread
    const bool row_valid = prow < packed_rows;
    const int a = prow / G;
    const int h = item.kv_head * G + (prow - a * G);
    if (ok && T > 0) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->o_done), (T - 1) & 1, abort_flag));
      if (ok) tc_fence_after();
    }
    if (ok) {
      const float inv = T > 0 ? 1.f / l_sum : 0.f;
      const float lse = T > 0 ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
      if (s.num_splits > 1) {
        const long long pr = ((long long)item.split * t.total_tokens + req.tok_off + a) * t.Hq + h;
        float* po = t.part_o + pr * 128;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          unsigned r[32];
          if (T > 0) {
            tmem_ld32(tmem_o + lane_base + c * 32, r);
            tmem_wait_ld();
          } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) r[i] = 0u;
          }
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) {
              float4 v4 = make_float4(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv,
                                      __uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
              *reinterpret_cast<float4*>(po + c * 32 + i) = v4;
            }
          }
        }
        if (row_valid) t.part_lse[pr] = lse;
      } else if (T > 0) {
        char* orow = t.out + ((req.row_off + a) * t.out_stride + (long long)h * 128) * 2;
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          unsigned r[32];
          tmem_ld32(tmem_o + lane_base + c * 32, r);
          tmem_wait_ld();
          if (row_valid) {
#pragma unroll
            for (int i = 0; i < 32; i += 8) {
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(r[i]) * inv, __uint_as_float(r[i + 1]) * inv);
              v4.y = pack_bf16(__uint_as_float(r[i + 2]) * inv, __uint_as_float(r[i + 3]) * inv);
              v4.z = pack_bf16(__uint_as_float(r[i + 4]) * inv, __uint_as_float(r[i + 5]) * inv);
              v4.w = pack_bf16(__uint_as_float(r[i + 6]) * inv, __uint_as_float(r[i + 7]) * inv);
              *reinterpret_cast<uint4*>(orow + (c * 32 + i) * 2) = v4;
            }
          }
        }
        if (row_valid && t.lse != nullptr) t.lse[(req.row_off + a) * t.Hq + h] = lse;
      }
    }
    tc_fence_before();
  } else if (!dead && warp == 4) {
    // ===================================== MMA issue =====================================
    if (lane == 0 && T > 0) {
      bool ok = mbar_wait(smem_u32(&bars->q_full), 0, abort_flag);
      // software pipeline: S(j) = Q K_j^T is issued before O += P(j-1) V_(j-1)
      for (int j = 0; j <= T && ok; ++j) {
        if (j < T) {
          const int st = j % kStages, b = j & 1;
          ok = mbar_wait(smem_u32(&bars->kv_full[st]), (j / kStages) & 1, abort_flag);
          if (ok) ok = mbar_wait(smem_u32(&bars->s_free[b]), ((j >> 1) & 1) ^ 1, abort_flag);
          if (!ok) break;
          fence_proxy_async();
          tc_fence_after();
          const unsigned k_smem = kv_smem + (2 * st) * kTileBytes;
#pragma unroll
          for (int k = 0; k < 8; ++k) {
            const unsigned off = (k >> 2) * 1024 + (k & 3) * 32;
            mma_ss(tmem + b * 128, make_desc(q_smem + off, 16, 2048), make_desc(k_smem + off, 16, 2048),
                   kIdescQK, k > 0 ? 1u : 0u);
          }
          mma_commit(smem_u32(&bars->s_full[b]));
        }
        if (j >= 1) {
          const int jp = j - 1, st = jp % kStages, b = jp & 1;
          const int jg = tile_begin + jp;
          const int cnt = jg < prefix_tiles ? min(kTileKeys, req.m - jg * kTileKeys)
                                            : min(kTileKeys, req.n - (jg - prefix_tiles) * kTileKeys);
          const int ksteps = (cnt + 15) >> 4;
          ok = mbar_wait(smem_u32(&bars->p_full[b]), (jp >> 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          const unsigned v_smem = kv_smem + (2 * st + 1) * kTileBytes;
          for (int k = 0; k < ksteps; ++k) {
            mma_ts(tmem_o, tmem + 384 + b * 64 + k * 8, make_desc(v_smem + k * kPageBytes, 1024, 2048),
                   kIdescPV, (jp > 0 || k > 0) ? 1u : 0u);
          }
          mma_commit(smem_u32(&bars->kv_free[st]));
          mma_commit(smem_u32(&bars->o_done));
        }
      }
      // Whatever happened, let every MMA issued so far finish before TMEM is released.
      mma_commit(smem_u32(&bars->drain));
      mbar_wait(smem_u32(&bars->drain), 0, abort_flag);
    }
    __syncwarp();
  } else if (!dead && warp >= 5) {
    // ====================================== loads =======================================
    const int lt = tid - 5 * 32;                      // 0..127
    const int G_ = G;
    // Q tile: 128 packed rows x 256 bytes; 16 consecutive threads fetch one row; rows past the
    // request's end are zero-filled.
#pragma unroll 4
    for (int i = 0; i < 16; ++i) {
      const int idx = i * kLoadThreads + lt;
      const int r = idx >> 4, c16 = idx & 15;
      const int prow = item.row0 + r;
      const bool valid = prow < packed_rows;
      const int a = valid ? prow / G_ : 0;
      const int h = item.kv_head * G_ + (valid ? prow - a * G_ : 0);
      const char* src = t.q + ((req.row_off + a) * t.q_stride + (long long)h * 128) * 2 + c16 * 16;
      cp_async16(q_smem + tile_chunk_offset(r, c16), src, valid ? 16u : 0u);
    }
    cp_async_commit();
    cp_async_wait<0>();
    fence_proxy_async();
    mbar_arrive(smem_u32(&bars->q_full));

    const int* pages = s.pages + req.page_off;
    bool ok = true;
    int pending_async = -1;                           // tile whose cp.async group is still in flight
    for (int j = 0; j < T; ++j) {
      const int st = j % kStages;
      const int jg = tile_begin + j;
      ok = mbar_wait(smem_u32(&bars->kv_free[st]), ((j / kStages) & 1) ^ 1, abort_flag);
      if (!ok) break;
      const unsigned k_smem = kv_smem + (2 * st) * kTileBytes;
      const unsigned v_smem = k_smem + kTileBytes;
      const unsigned full = smem_u32(&bars->kv_full[st]);
      if (jg < prefix_tiles) {
        // cached prefix tile: one bulk copy per page and tensor; a page is already the image
        const int cnt = min(kTileKeys, req.m - jg * kTileKeys);
        const int npages = (cnt + kPageSize - 1) / kPageSize;
        if (lt == 0) {
          mbar_arrive_expect_tx(full, (unsigned)(2 * npages * kPageBytes));
          for (int pg = 0; pg < npages; ++pg) {
            const long long off = pool_slice_offset(pool, t.layer, pages[jg * 8 + pg], item.kv_head);
            bulk_copy_g2s(k_smem + pg * kPageBytes, pool.k + off, kPageBytes, full);
            bulk_copy_g2s(v_smem + pg * kPageBytes, pool.v + off, kPageBytes, full);
          }
        } else {
          mbar_arrive(full);
        }
      } else {
        // own rows: 16-byte gathers from row-major K/V into the image, zero-filled past the end
        const int key0 = (jg - prefix_tiles) * kTileKeys;
        const int cnt = min(kTileKeys, req.n - key0);
#pragma unroll 4
        for (int i = 0; i < 16; ++i) {
          const int idx = i * kLoadThreads + lt;
          const int r = idx >> 4, c16 = idx & 15;
          const bool valid = r < cnt;
          const long long roff = ((req.row_off + key0 + (valid ? r : 0)) * t.kv_stride +
                                  (long long)item.kv_head * 128) * 2 + c16 * 16;
          const unsigned dst = tile_chunk_offset(r, c16);
          cp_async16(k_smem + dst, t.k + roff, valid ? 16u : 0u);
          cp_async16(v_smem + dst, t.v + roff, valid ? 16u : 0u);
        }
        cp_async_commit();
        if (pending_async >= 0) {
          cp_async_wait<1>();                         // the previous gathered tile has landed
          fence_proxy_async();
          mbar_arrive(smem_u32(&bars->kv_full[pending_async % kStages]));
        }
        pending_async = j;
      }
    }
    cp_async_wait<0>();
    if (pending_async >= 0) {
      fence_proxy_async();
      mbar_arrive(smem_u32(&bars->kv_full[pending_async % kStages]));
    }
    // On the normal path every tile loaded has been consumed by the time the CTA ends (the
    // epilogue waits for the last P.V).  After a give-up, bulk copies may still be in flight:
    // wait (bounded) for the stages this thread armed.
    if (!ok || *abort_flag) {
      if (lt == 0) {
        for (int j = max(0, T - kStages); j < T; ++j)
          if (tile_begin + j < prefix_tiles)
            for (unsigned it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bars->kv_full[j % kStages]), (j / kStages) & 1); ++it)
              __nanosleep(256);
      }
    }
  }

  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && !dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
}

inline cudaError_t configure_tc_attention() {
  return cudaFuncSetAttribute(tc_attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
}

inline cudaError_t launch_tc_attention(const ScheduleView& s, const PoolView& pool, const TensorArgs& t,
                                       int* status, cudaStream_t stream) {
  tc_attention_kernel<<<s.num_items, tc::kThreads, tc::kSmemBytes, stream>>>(s, pool, t, status);
  return cudaGetLastError();
}

}  // namespace bicache
