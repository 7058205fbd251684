// Prefix K/V projection written straight into the paged store (Eq. 1): for one layer,
//   K = H W_K^T, V = H W_V^T,   H [m][d] hidden states of the prefix tokens, W [Hkv * D][d],
// bf16 in, fp32 accumulate, bf16 out, D = 128.  The output never exists as a dense [m][Hkv][D]
// tensor: every (page, kv head) slice of the pool is produced as the 4 KB operand image the
// attention kernel reads and leaves shared memory as one bulk copy.
//
// A persistent tcgen05 GEMM.  One output tile is 128 tokens x 256 output features (two KV heads
// of K, or two of V); the contraction runs over d in blocks of 64 (one 128-byte swizzled row per
// token / feature and block).  Warp 0 feeds a four-stage ring of (H tile 16 KB, W tile 32 KB) by
// TMA, warp 1 issues the MMAs (M = 128, N = 256, K = 16) into one of two 256-column TMEM
// accumulators, warps 2-5 drain the other accumulator: TMEM -> registers -> bf16 -> page images
// in shared memory -> eight 4 KB bulk copies per head.  Tiles are handed out statically
// (tile = block + i * grid) with all tiles of a token block adjacent, so that the H tile is
// shared through L2 by the CTAs working on it.
//
// Every wait is bounded (SM clock); a wait that gives up raises the CTA's abort flag, the roles
// leave their loops, loads and MMAs in flight are waited for, TMEM is released and the context's
// sticky status word is set.
#pragma once

#include "tc_attention.cuh"

namespace bicache {
namespace proj {

using namespace tc;

constexpr int kBM = 128;                       // tokens per tile
constexpr int kBN = 256;                       // output features per tile (two heads of 128 dims)
constexpr int kBK = 64;                        // contraction block: 64 bf16 = one 128-byte row
constexpr int kStages = 4;
constexpr int kABytes = kBM * kBK * 2;         // 16 KB
constexpr int kBBytes = kBN * kBK * 2;         // 32 KB
constexpr int kProjStageBytes = kABytes + kBBytes;
constexpr int kOutBytes = 8 * kPageBytes;      // 128 tokens of one head = eight page images
constexpr int kProjThreads = 192;
constexpr int kEpiWarps = 4;
// fp32 accumulate, bf16 A and B (both K-major), M = 128, N = 256
constexpr unsigned kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((128u >> 4) << 24);

struct Sync {
  unsigned long long full[kStages];      // stage holds its two tiles
  unsigned long long empty[kStages];     // the MMAs reading the stage have completed
  unsigned long long acc_full[2];        // the accumulator holds a finished tile
  unsigned long long acc_empty[2];       // the epilogue has read the accumulator
  unsigned long long epi;                // barrier of the four epilogue warps
  unsigned long long drain;
  long long wait_cycles;                 // budget of every wait; directly before abort_flag (mbar_wait reads it)
  int abort_flag;
  unsigned tmem_base;
  int dead;
};
constexpr int kProjSmemBytes = 1024 + kStages * kProjStageBytes + kOutBytes + (int)sizeof(Sync);
static_assert(kProjSmemBytes <= 232448, "shared memory of one CTA");

struct ProjArgs {
  char* pool_k;              // the layer's slice of the K pool
  char* pool_v;
  const int* pages;          // page list of the prefix (device)
  int m;                     // prefix tokens
  int d_model;
  int num_kv_heads;
  int m_tiles;               // ceil(m / 128)
  int n_tiles;               // per matrix: ceil(Hkv / 2)
};

__device__ __forceinline__ void tma_load_2d(unsigned dst, const void* tmap, int c0, int c1, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(tmap)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
__device__ __forceinline__ void bulk_copy_s2g(void* dst, unsigned src, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes)
               : "memory");
}

struct TileCoord {
  int mt, nt, which;         // token block, feature block of the matrix, 0: K, 1: V
};
__device__ __forceinline__ TileCoord tile_coord(int tile, int n_tiles) {
  TileCoord c;
  c.mt = tile / (2 * n_tiles);
  const int rem = tile - c.mt * 2 * n_tiles;
  c.which = rem / n_tiles;
  c.nt = rem - c.which * n_tiles;
  return c;
}

}  // namespace proj

__global__ void __launch_bounds__(proj::kProjThreads, 1)
project_kv_kernel(proj::ProjArgs a, int* status, const __grid_constant__ CUtensorMap tm_h,
                  const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                  long long wait_cycles) {
  using namespace proj;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* const out_stage = smem + kStages * kProjStageBytes;
  Sync* sy = reinterpret_cast<Sync*>(out_stage + kOutBytes);
  volatile int* abort_flag = &sy->abort_flag;
  const unsigned ring = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;

  if (tid == 0) {
    sy->wait_cycles = wait_cycles;
    sy->dead = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    sy->abort_flag = (sy->dead || wait_cycles < kStrictBudget) ? 1 : 0;
    for (int i = 0; i < kStages; ++i) {
      mbar_init(smem_u32(&sy->full[i]), 1);
      mbar_init(smem_u32(&sy->empty[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&sy->acc_full[i]), 1);
      mbar_init(smem_u32(&sy->acc_empty[i]), kEpiWarps);
    }
    mbar_init(smem_u32(&sy->epi), kEpiWarps);
    mbar_init(smem_u32(&sy->drain), 1);
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(&sy->tmem_base), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&sy->tmem_base);
  const bool dead = *reinterpret_cast<volatile int*>(&sy->dead) != 0;
  const int total_tiles = a.m_tiles * 2 * a.n_tiles;
  const int KB = (a.d_model + kBK - 1) / kBK;

  if (warp == 0) {
    // ===================================== TMA producer =====================================
    bool ok = !dead;
    int it = 0;                              // stage uses over the life of the CTA
    int armed[kStages] = {-1, -1, -1, -1};
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x) {
      const TileCoord c = tile_coord(tile, a.n_tiles);
      const void* tm_w = c.which ? (const void*)&tm_wv : (const void*)&tm_wk;
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % kStages;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->empty[s]), ((it / kStages) & 1) ^ 1, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const unsigned full = smem_u32(&sy->full[s]);
          const unsigned dst = ring + s * kProjStageBytes;
          mbar_arrive_expect_tx(full, (unsigned)kProjStageBytes);
          tma_load_2d(dst, &tm_h, kb * kBK, c.mt * kBM, full);
          tma_load_2d(dst + kABytes, tm_w, kb * kBK, c.nt * kBN, full);
          armed[s] = it;
        }
      }
    }
    // After a give-up, loads may still be in flight: wait (bounded) for the barriers armed last.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      for (int s = 0; s < kStages; ++s)
        if (armed[s] >= 0)
          for (unsigned n = 0; n < 4096 && !mbar_try_wait(smem_u32(&sy->full[s]), (armed[s] / kStages) & 1); ++n)
            __nanosleep(256);
    }
  } else if (warp == 1) {
    // ====================================== MMA issue ======================================
    bool ok = !dead;
    if (ok) {
      int it = 0, tl = 0;
      for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tl) {
        const int buf = tl & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->acc_empty[buf]), ((tl >> 1) & 1) ^ 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        const unsigned d_tmem = tmem + buf * kBN;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kStages;
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->full[s]), (it / kStages) & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          // both operands K-major, rows of 128 bytes, 8-row groups 1024 bytes apart; a K step of
          // 16 elements is 32 bytes inside the swizzled row
          const unsigned long long a_desc = make_desc(ring + s * kProjStageBytes, 16, 1024);
          const unsigned long long b_desc = make_desc(ring + s * kProjStageBytes + kABytes, 16, 1024);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            mma_ss_elect(d_tmem, a_desc + 2 * k, b_desc + 2 * k, kIdesc, (kb | k) ? 1u : 0u);
          mma_commit_elect(smem_u32(&sy->empty[s]));
        }
        if (!ok) break;
        mma_commit_elect(smem_u32(&sy->acc_full[buf]));
      }
      // Whatever happened, let every MMA issued so far finish before TMEM is released.
      __syncwarp();
      mma_commit_elect(smem_u32(&sy->drain));
      mbar_wait_issued(smem_u32(&sy->drain), 0);
    }
    __syncwarp();
  } else {
    // ====================================== epilogue =======================================
    // Warp w reads TMEM lanes 32 (w & 3) .. + 31: thread = one token of the tile.  Per head:
    // 128 fp32 -> bf16, written as 16-byte chunks into the token's slot of its page image
    // (page = token / 16); when all four warps are done, eight threads copy one page each.
    const int q = warp & 3;
    const int e = q * 32 + lane;                             // token within the tile
    const unsigned lane_base = (unsigned)(q * 32) << 16;
    unsigned char* const my_row = out_stage + (e >> 4) * kPageBytes;
    const int slot = e & 15;
    bool ok = !dead;
    int sync_n = 0;
    auto epi_sync = [&]() {
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&sy->epi));
      const bool done = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->epi), sync_n & 1, abort_flag));
      ++sync_n;
      return done;
    };
    int tl = 0;
    for (int tile = blockIdx.x; tile < total_tiles && ok; tile += gridDim.x, ++tl) {
      const TileCoord c = tile_coord(tile, a.n_tiles);
      const int buf = tl & 1;
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->acc_full[buf]), (tl >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int hh = 0; hh < 2; ++hh) {
        const int head = c.nt * 2 + hh;
        const bool head_valid = head < a.num_kv_heads;
        if (e < 8) bulk_wait_read();                         // the previous copies have read the staging pages
        ok = epi_sync();
        if (!ok) break;
        if (head_valid) {
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            unsigned r[32];
            tmem_ld32(tmem + buf * kBN + hh * 128 + cc * 32 + lane_base, r);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(r[8 * i]), __uint_as_float(r[8 * i + 1]));
              v4.y = pack_bf16(__uint_as_float(r[8 * i + 2]), __uint_as_float(r[8 * i + 3]));
              v4.z = pack_bf16(__uint_as_float(r[8 * i + 4]), __uint_as_float(r[8 * i + 5]));
              v4.w = pack_bf16(__uint_as_float(r[8 * i + 6]), __uint_as_float(r[8 * i + 7]));
              *reinterpret_cast<uint4*>(my_row + page_chunk_offset(true, slot, cc * 4 + i, 256)) = v4;
            }
          }
        }
        if (hh == 1) {
          // the accumulator has been read: the MMAs of the tile after next may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) mbar_arrive(smem_u32(&sy->acc_empty[buf]));
        }
        fence_proxy_async();                                 // the bulk copies read what the threads wrote
        ok = epi_sync();
        if (!ok) break;
        if (e < 8) {
          const int tok0 = c.mt * kBM + e * kPageSize;
          if (head_valid && tok0 < a.m) {
            const int page = a.pages[c.mt * 8 + e];
            char* dst = (c.which ? a.pool_v : a.pool_k) + ((long long)page * a.num_kv_heads + head) * kPageBytes;
            bulk_copy_s2g(dst, smem_u32(out_stage + e * kPageBytes), kPageBytes);
          }
          bulk_commit_group();
        }
      }
    }
    if (e < 8) bulk_wait_all();                              // this thread's page copies have completed
    tc_fence_before();
  }

  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
  if (tid == 0 && !dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
}

inline cudaError_t configure_project_kv() {
  return cudaFuncSetAttribute(project_kv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, proj::kProjSmemBytes);
}

inline cudaError_t launch_project_kv(const proj::ProjArgs& a, int* status, int num_sms, const CUtensorMap& tm_h,
                                     const CUtensorMap& tm_wk, const CUtensorMap& tm_wv, long long wait_cycles,
                                     cudaStream_t stream) {
  const int total = a.m_tiles * 2 * a.n_tiles;
  if (total <= 0) return cudaSuccess;
  const int grid = total < num_sms ? total : num_sms;
  project_kv_kernel<<<grid, proj::kProjThreads, proj::kProjSmemBytes, stream>>>(
      a, status, tm_h, tm_wk, tm_wv, wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  return cudaGetLastError();
}

}  // namespace bicache
