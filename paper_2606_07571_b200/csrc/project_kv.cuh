// Prefix K/V projection written straight into the paged store (Eq. 1): for one layer,
//   K = H W_K^T, V = H W_V^T,   H [m][d] hidden states of the prefix tokens, W [Hkv * D][d],
// bf16 in, fp32 accumulate, bf16 out, D = 128.  The output never exists as a dense [m][Hkv][D]
// tensor: every (page, kv head) slice of the pool is produced as the 4 KB operand image the
// attention kernel reads and leaves shared memory as one bulk copy.
//
// A persistent tcgen05 GEMM on CTA pairs (clusters of two, the two-SM MMA).  One output tile of
// a pair is 256 tokens x 256 output features (two KV heads of K, or two of V): CTA r of the pair
// owns tokens 128 r .. 128 r + 127 of the tile (its rows of A and of the accumulator, in its own
// TMEM) and stages rows 128 r .. 128 r + 127 of the W tile (its half of B), so every SM stages
// and reads half of the B operand a one-CTA tile would.  The contraction runs over d in blocks of
// 64 (one 128-byte swizzled row per token / feature and block).  Per CTA: warp 0 feeds a
// six-stage ring of (H tile 16 KB, W half tile 16 KB) by TMA, the loads of both CTAs completing
// on one barrier in CTA 0; warp 1 of CTA 0 issues the MMAs (cta_group::2, M = 256, N = 256,
// K = 16) into one of two 256-column TMEM accumulators; warps 2-5 drain the other accumulator:
// TMEM -> registers -> bf16 -> page images in shared memory -> eight 4 KB bulk copies per head.
// One tcgen05.commit with a CTA mask releases a stage, or hands over an accumulator, in both
// CTAs; the epilogue warps of CTA 1 release the accumulator on CTA 0's barrier through the
// cluster's shared address space.  Tiles are handed out statically (tile = pair + i * pairs) with
// all tiles of a token block adjacent, so that the H tile is shared through L2.
//
// Every wait is bounded (SM clock) and on a barrier of the waiting CTA; a wait that gives up
// raises the CTA's abort flag, the roles leave their loops (the partner's waits then run out
// too), loads and MMAs in flight are waited for, the pair meets at a cluster barrier, TMEM is
// released and the context's sticky status word is set.
#pragma once

#include <cooperative_groups.h>

#include "tc_attention.cuh"

namespace bicache {
namespace proj {

using namespace tc;

constexpr int kBM = 128;                       // tokens per tile and CTA (256 per pair)
constexpr int kBN = 256;                       // output features per tile (two heads of 128 dims)
constexpr int kBK = 64;                        // contraction block: 64 bf16 = one 128-byte row
constexpr int kStages = 6;
constexpr int kABytes = kBM * kBK * 2;         // 16 KB: this CTA's tokens
constexpr int kBBytes = (kBN / 2) * kBK * 2;   // 16 KB: this CTA's half of the W tile
constexpr int kProjStageBytes = kABytes + kBBytes;
constexpr int kOutBytes = 8 * kPageBytes;      // 128 tokens of one head = eight page images
constexpr int kProjThreads = 192;
constexpr int kEpiWarps = 4;
// fp32 accumulate, bf16 A and B (both K-major), M = 256 (over the pair), N = 256
constexpr unsigned kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((256u >> 3) << 17) | ((256u >> 4) << 24);
// the same with N = 128: one head (the tiles of the last, partial round are split in two)
constexpr unsigned kIdescHalf = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);

struct Sync {
  unsigned long long full[kStages];      // CTA 0 only: the stage holds its tiles in BOTH CTAs
  unsigned long long empty[kStages];     // the MMAs reading the stage (in both CTAs) have completed
  unsigned long long acc_full[2];        // the accumulator holds a finished tile
  unsigned long long acc_empty[2];       // CTA 0 only: the epilogues of both CTAs have read the accumulator
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
  const float2* rope;        // nullptr, or (cos, sin) of the rotation of the keys: [m][64], pair d = dims (d, d + 64)
  int m;                     // prefix tokens
  int d_model;
  int num_kv_heads;
  int m_tiles;               // ceil(m / 256): token blocks of a CTA pair
  int n_tiles;               // per matrix: ceil(Hkv / 2)
  int full_tiles;            // tiles 0 .. full_tiles - 1 are worked on whole (whole rounds of the grid);
                             // each tile after them is split into its two heads, so that the last
                             // round takes half the time
};

__device__ __forceinline__ void tma_load_2d(unsigned dst, const void* tmap, int c0, int c1, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(tmap)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
// The same load issued by either CTA of a pair, completing on the barrier at `bar`'s offset in the
// pair's FIRST CTA (bit 24 of a shared-window address is the CTA's rank in the pair): one barrier
// there collects the bytes of both CTAs' stages.  No multicast: each CTA's data goes to its own
// shared memory.
__device__ __forceinline__ void tma_load_2d_pair(unsigned dst, const void* tmap, int c0, int c1, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(tmap)), "r"(c0), "r"(c1), "r"(bar & 0xFEFFFFFFu)
      : "memory");
}
__device__ __forceinline__ void bulk_copy_s2g(void* dst, unsigned src, unsigned bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes)
               : "memory");
}

// arrive on the barrier at the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ void mbar_arrive_remote(unsigned local_bar, unsigned rank) {
  unsigned raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local_bar), "r"(rank));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(raddr) : "memory");
}
// The two-SM MMA, issued by one elected lane of a converged warp of the pair's first CTA.  The
// descriptors name the same shared-memory offsets in both CTAs: CTA r supplies rows 128 r .. of A
// and rows N/2 r .. of B and receives rows 128 r .. of D in its own TMEM.
__device__ __forceinline__ void mma2_ss_elect(unsigned d_tmem, unsigned long long a_desc, unsigned long long b_desc,
                                              unsigned idesc, unsigned accumulate) {
  asm volatile(
      "{\n\t.reg .pred P, Q;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "setp.ne.b32 Q, %4, 0;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5, %5, %5, %5, %5}, Q;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// commit of the two-SM MMAs issued so far by this thread: arrives on the barrier at this offset in
// both CTAs of the pair
__device__ __forceinline__ void mma2_commit_both_elect(unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "@P tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;\n\t}"
      ::"r"(bar), "h"((unsigned short)3)
      : "memory");
}
// the same, arriving in this CTA only
__device__ __forceinline__ void mma2_commit_local_elect(unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "@P tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar)
      : "memory");
}
__device__ __forceinline__ void tmem_alloc2(unsigned smem_slot, unsigned cols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish2() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(unsigned taddr, unsigned cols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}

struct TileCoord {
  int mt, nt, which;         // token block, feature block of the matrix, 0: K, 1: V
  int half;                  // -1: both heads of the feature block; 0 / 1: that head only
  int valid;
};
// work unit `idx` of the launch (a pair takes idx = pair, pair + pairs, ...)
__device__ __forceinline__ TileCoord tile_coord(int idx, const ProjArgs& a) {
  TileCoord c;
  const int total = a.m_tiles * 2 * a.n_tiles;
  int tile = idx;
  c.half = -1;
  if (idx >= a.full_tiles) {
    const int j = idx - a.full_tiles;
    tile = a.full_tiles + (j >> 1);
    c.half = j & 1;
  }
  c.valid = tile < total;
  c.mt = tile / (2 * a.n_tiles);
  const int rem = tile - c.mt * 2 * a.n_tiles;
  c.which = rem / a.n_tiles;
  c.nt = rem - c.which * a.n_tiles;
  return c;
}

}  // namespace proj

// kRope: the epilogue rotates the keys (a second instantiation, so that the plain projection keeps its
// register count and its epilogue as they were: with the rotation compiled in, 210 registers instead of
// 152 and 10-17 % less throughput on launches that never rotate).
template <bool kRope>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(proj::kProjThreads, 1)
project_kv_kernel(proj::ProjArgs a, int* status, const __grid_constant__ CUtensorMap tm_h,
                  const __grid_constant__ CUtensorMap tm_wk, const __grid_constant__ CUtensorMap tm_wv,
                  long long wait_cycles) {
  using namespace proj;
  namespace cg = cooperative_groups;
  extern __shared__ unsigned char smem_raw[];
  // the same offsets in both CTAs of the pair: the MMA descriptors name them once for both
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* const out_stage = smem + kStages * kProjStageBytes;
  Sync* sy = reinterpret_cast<Sync*>(out_stage + kOutBytes);
  volatile int* abort_flag = &sy->abort_flag;
  const unsigned ring = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster.block_rank();              // 0: issues the pair's MMAs
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

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
      mbar_init(smem_u32(&sy->acc_empty[i]), 2 * kEpiWarps);
    }
    mbar_init(smem_u32(&sy->epi), kEpiWarps);
    mbar_init(smem_u32(&sy->drain), 1);
    fence_barrier_init();
  }
  if (warp == 1) {                                          // the same warp in both CTAs
    tmem_alloc2(smem_u32(&sy->tmem_base), 512);
    tmem_relinquish2();
  }
  tc_fence_before();
  cluster.sync();                                           // barriers of both CTAs exist before any remote arrival
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&sy->tmem_base);
  const bool dead = *reinterpret_cast<volatile int*>(&sy->dead) != 0;
  const int KB = (a.d_model + kBK - 1) / kBK;

  if (warp == 0) {
    // ===================================== TMA producer =====================================
    // this CTA's 128 tokens of the H tile and its 128 rows of the W tile
    bool ok = !dead;
    int it = 0;                              // stage uses over the life of the CTA
    int armed[kStages];
#pragma unroll
    for (int i = 0; i < kStages; ++i) armed[i] = -1;
    for (int idx = pair; ok; idx += num_pairs) {
      const TileCoord c = tile_coord(idx, a);
      if (!c.valid) break;
      const void* tm_w = c.which ? (const void*)&tm_wv : (const void*)&tm_wk;
      // rows of W this CTA stages: its half of the tile's features (64-row boxes)
      const int w_row = c.nt * kBN + (c.half < 0 ? (int)rank * 128 : c.half * 128 + (int)rank * 64);
      const unsigned stage_tx = c.half < 0 ? 2u * kProjStageBytes : 2u * (kABytes + kBBytes / 2);
      for (int kb = 0; kb < KB; ++kb, ++it) {
        const int s = it % kStages;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->empty[s]), ((it / kStages) & 1) ^ 1, abort_flag));
        if (!ok) break;
        if (lane == 0) {
          const unsigned full = smem_u32(&sy->full[s]);
          const unsigned dst = ring + s * kProjStageBytes;
          if (rank == 0) mbar_arrive_expect_tx(full, stage_tx);               // the bytes of both CTAs
          tma_load_2d_pair(dst, &tm_h, kb * kBK, (c.mt * 2 + (int)rank) * kBM, full);
          tma_load_2d_pair(dst + kABytes, tm_w, kb * kBK, w_row, full);
          if (c.half < 0) tma_load_2d_pair(dst + kABytes + kBBytes / 2, tm_w, kb * kBK, w_row + 64, full);
          armed[s] = it;
        }
      }
    }
    // After a give-up, loads may still be in flight.  CTA 0 waits (bounded) for the barriers it
    // armed last, which count the bytes of both CTAs.  CTA 1 cannot see those barriers: if it has
    // issued loads it waits out the same limit before it joins the pair's last barrier.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      for (int s = 0; s < kStages; ++s)
        if (armed[s] >= 0) {
          if (rank == 0) {
            for (unsigned n = 0; n < 4096 && !mbar_try_wait(smem_u32(&sy->full[s]), (armed[s] / kStages) & 1); ++n)
              __nanosleep(256);
          } else {
            for (unsigned n = 0; n < 4096; ++n) __nanosleep(256);
            break;
          }
        }
    }
  } else if (warp == 1 && rank == 1) {
    // CTA 1's warp 1 only owns the pair's TMEM allocation with its counterpart
  } else if (warp == 1) {
    // ================================== CTA 0: MMA issue ===================================
    bool ok = !dead;
    if (ok) {
      int it = 0, tl = 0;
      for (int idx = pair; ok; idx += num_pairs, ++tl) {
        const TileCoord c = tile_coord(idx, a);
        if (!c.valid) break;
        const unsigned idesc = c.half < 0 ? kIdesc : kIdescHalf;
        const int buf = tl & 1;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->acc_empty[buf]), ((tl >> 1) & 1) ^ 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        const unsigned d_tmem = tmem + buf * kBN;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const int s = it % kStages;
          const unsigned ph = (it / kStages) & 1;
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->full[s]), ph, abort_flag));
          if (!ok) break;
          tc_fence_after();
          // both operands K-major, rows of 128 bytes, 8-row groups 1024 bytes apart; a K step of
          // 16 elements is 32 bytes inside the swizzled row
          const unsigned long long a_desc = make_desc(ring + s * kProjStageBytes, 16, 1024);
          const unsigned long long b_desc = make_desc(ring + s * kProjStageBytes + kABytes, 16, 1024);
#pragma unroll
          for (int k = 0; k < kBK / 16; ++k)
            mma2_ss_elect(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) ? 1u : 0u);
          mma2_commit_both_elect(smem_u32(&sy->empty[s]));
        }
        if (!ok) break;
        mma2_commit_both_elect(smem_u32(&sy->acc_full[buf]));
      }
      // Whatever happened, let every MMA issued so far finish before the pair's TMEM is released.
      __syncwarp();
      mma2_commit_local_elect(smem_u32(&sy->drain));
      mbar_wait_issued(smem_u32(&sy->drain), 0);
    }
    __syncwarp();
  } else {
    // ====================================== epilogue =======================================
    // Warp w reads TMEM lanes 32 (w & 3) .. + 31: thread = one token of this CTA's half of the
    // tile.  Per head: 128 fp32 -> bf16, written as 16-byte chunks into the token's slot of its
    // page image (page = token / 16); when all four warps are done, eight threads copy one page each.
    const int q = warp & 3;
    const int e = q * 32 + lane;                             // token within this CTA's 128
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
    for (int idx = pair; ok; idx += num_pairs, ++tl) {
      const TileCoord c = tile_coord(idx, a);
      if (!c.valid) break;
      const int hh_begin = c.half < 0 ? 0 : c.half, hh_end = c.half < 0 ? 2 : c.half + 1;
      const int buf = tl & 1;
      const int tok_base = (c.mt * 2 + (int)rank) * kBM;     // first token of this CTA's half
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->acc_full[buf]), (tl >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
#pragma unroll 1
      for (int hh = hh_begin; hh < hh_end; ++hh) {
        const int head = c.nt * 2 + hh;
        const int col = buf * kBN + (c.half < 0 ? hh * 128 : 0);   // a split tile's head sits in the first columns
        const bool head_valid = head < a.num_kv_heads;
        if (e < 8) bulk_wait_read();                         // the previous copies have read the staging pages
        ok = epi_sync();
        if (!ok) break;
        if (kRope && head_valid && c.which == 0) {
          // Keys with a rotary position encoding: dims d and d + 64 of the head form a pair, rotated by
          // the token's angle for pair d (the caller's table).  Chunk cc (dims 32 cc ..) and chunk cc + 2
          // are read together; tokens past the end keep their zeros.
          const int tok = tok_base + e;
          const float4* tab = reinterpret_cast<const float4*>(a.rope + (long long)min(tok, a.m - 1) * 64);
          const bool rot = tok < a.m;
#pragma unroll 1
          for (int cc = 0; cc < 2; ++cc) {
            unsigned lo[32], hi[32];
            tmem_ld32(tmem + col + cc * 32 + lane_base, lo);
            tmem_ld32(tmem + col + (cc + 2) * 32 + lane_base, hi);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float4 cs = rot ? tab[cc * 16 + i] : make_float4(1.f, 0.f, 1.f, 0.f);   // (cos, sin) of two pairs
              const float a0 = __uint_as_float(lo[2 * i]), b0 = __uint_as_float(hi[2 * i]);
              const float a1 = __uint_as_float(lo[2 * i + 1]), b1 = __uint_as_float(hi[2 * i + 1]);
              lo[2 * i] = __float_as_uint(a0 * cs.x - b0 * cs.y);
              hi[2 * i] = __float_as_uint(b0 * cs.x + a0 * cs.y);
              lo[2 * i + 1] = __float_as_uint(a1 * cs.z - b1 * cs.w);
              hi[2 * i + 1] = __float_as_uint(b1 * cs.z + a1 * cs.w);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(lo[8 * i]), __uint_as_float(lo[8 * i + 1]));
              v4.y = pack_bf16(__uint_as_float(lo[8 * i + 2]), __uint_as_float(lo[8 * i + 3]));
              v4.z = pack_bf16(__uint_as_float(lo[8 * i + 4]), __uint_as_float(lo[8 * i + 5]));
              v4.w = pack_bf16(__uint_as_float(lo[8 * i + 6]), __uint_as_float(lo[8 * i + 7]));
              *reinterpret_cast<uint4*>(my_row + page_chunk_offset(true, slot, cc * 4 + i, 256)) = v4;
              v4.x = pack_bf16(__uint_as_float(hi[8 * i]), __uint_as_float(hi[8 * i + 1]));
              v4.y = pack_bf16(__uint_as_float(hi[8 * i + 2]), __uint_as_float(hi[8 * i + 3]));
              v4.z = pack_bf16(__uint_as_float(hi[8 * i + 4]), __uint_as_float(hi[8 * i + 5]));
              v4.w = pack_bf16(__uint_as_float(hi[8 * i + 6]), __uint_as_float(hi[8 * i + 7]));
              *reinterpret_cast<uint4*>(my_row + page_chunk_offset(true, slot, (cc + 2) * 4 + i, 256)) = v4;
            }
          }
        } else if (head_valid) {
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            unsigned r[32];
            tmem_ld32(tmem + col + cc * 32 + lane_base, r);
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
        if (hh == hh_end - 1) {
          // the accumulator has been read: the MMAs of the tile after next may overwrite it
          tc_fence_before();
          __syncwarp();
          if (lane == 0) {
            if (rank == 0) mbar_arrive(smem_u32(&sy->acc_empty[buf]));
            else mbar_arrive_remote(smem_u32(&sy->acc_empty[buf]), 0);
          }
        }
        fence_proxy_async();                                 // the bulk copies read what the threads wrote
        ok = epi_sync();
        if (!ok) break;
        if (e < 8) {
          const int tok0 = tok_base + e * kPageSize;
          if (head_valid && tok0 < a.m) {
            const int page = a.pages[tok0 / kPageSize];
            char* dst = (c.which ? a.pool_v : a.pool_k) + ((long long)page * a.num_kv_heads + head) * kPageBytes;
            bulk_copy_s2g(dst, smem_u32(out_stage + e * kPageBytes), kPageBytes);
          }
          bulk_commit_group();
        }
      }
    }
    if (e < 8) bulk_wait_all();                              // this thread's page copies have completed
  }

  // The pair leaves together: CTA 0's MMAs read CTA 1's shared memory and write its TMEM.
  tc_fence_before();
  cluster.sync();
  tc_fence_after();
  if (warp == 1) tmem_dealloc2(tmem, 512);
  if (tid == 0 && !dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
}

// Sets the kernel's shared-memory limit and returns how many CTA pairs the device runs at once.
inline cudaError_t configure_project_kv(int* max_pairs) {
  cudaError_t e =
      cudaFuncSetAttribute(project_kv_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, proj::kProjSmemBytes);
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(project_kv_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, proj::kProjSmemBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(proj::kProjThreads, 1, 1);
  cfg.dynamicSmemBytes = proj::kProjSmemBytes;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, project_kv_kernel<false>, &cfg);
  if (e != cudaSuccess) return e;
  *max_pairs = n;
  return n > 0 ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

inline cudaError_t launch_project_kv(const proj::ProjArgs& a, int* status, int max_pairs, const CUtensorMap& tm_h,
                                     const CUtensorMap& tm_wk, const CUtensorMap& tm_wv, long long wait_cycles,
                                     cudaStream_t stream) {
  const int total = a.m_tiles * 2 * a.n_tiles;
  if (total <= 0) return cudaSuccess;
  // Whole rounds of the grid work on whole tiles.  If the tiles left for the last round occupy at
  // most half of the pairs they are split in two (one head each), which halves that round; a
  // fuller last round is better off with whole tiles (a split tile stages H for half the work).
  proj::ProjArgs b = a;
  const int left = total % max_pairs;
  b.full_tiles = 2 * left <= max_pairs ? total - left : total;
  const int units = b.full_tiles + 2 * (total - b.full_tiles);
  const int pairs = units < max_pairs ? units : max_pairs;
  if (b.rope != nullptr)
    project_kv_kernel<true><<<2 * pairs, proj::kProjThreads, proj::kProjSmemBytes, stream>>>(
        b, status, tm_h, tm_wk, tm_wv, wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  else
    project_kv_kernel<false><<<2 * pairs, proj::kProjThreads, proj::kProjSmemBytes, stream>>>(
        b, status, tm_h, tm_wk, tm_wv, wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  return cudaGetLastError();
}

}  // namespace bicache
