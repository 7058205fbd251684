// The tensor-core attention kernel on CTA pairs (clusters of two, the two-SM tcgen05 MMA), bf16,
// head_dim 128, for launches whose requests bring at least 512 packed query rows per KV head.
//
// A work item is up to 512 packed query rows of one request and one KV head: CTA r of the pair owns rows
// 256 r .. 256 r + 255 as its two 128-row tiles A and B, with its own Q tiles, S/P/O in its own tensor
// memory, its own softmax warps and its own epilogue - all as in the one-CTA kernel.  What changes is
// the B operand: for S = Q K^T each CTA stages the K rows of 64 of a tile's 128 keys, for O += P V the V
// columns of 64 of the 128 dims for all of its keys, and one MMA of M = 256 issued by the first CTA
// computes tile X of both CTAs from the two halves.  Every SM therefore writes half of the K/V bytes
// into shared memory and its tensor core reads half of the B operand from there: the shared-memory
// port, which is what the one-CTA kernel runs into, carries 160 KB per key tile instead of 256 KB.
//
// Barriers: the MMA warp of the first CTA waits on barriers of its own CTA only.  Loads of both CTAs
// complete on the first CTA's `full` / `q_full` barriers (tiled TMA loads with .cta_group::2; gathered
// tiles by a remote arrival of the loading warp), the softmax threads of the second CTA arrive on the
// first CTA's `p_half` / `o_free` barriers through the cluster's shared address space, and one
// tcgen05.commit with a CTA mask signals `s_full` / `free_` / `q_free` / `o_done` in both CTAs.  The first
// CTA takes the items from the launch's counter and passes each index on to its partner.
// Every wait is bounded, as in the one-CTA kernel; the pair leaves through a cluster barrier, after
// which the pair's tensor memory is released.
#pragma once
#include <cooperative_groups.h>

#include "project_kv.cuh"
#include "tc_attention.cuh"

namespace bicache {
namespace tcp {

using namespace tc;
using proj::mbar_arrive_remote;
using proj::tmem_alloc2;
using proj::tmem_dealloc2;
using proj::tmem_relinquish2;

constexpr int kPairRows = 2 * kTileRows;         // query rows of one item of a pair
constexpr int kHalfBytes = kTileBytes / 2;       // 16 KB: this CTA's half of a K or V tile
constexpr int kRing2 = 8;                        // ring slots of half a tile each: K0 V0 K1 V1 K2 V2 K3 V3
constexpr unsigned kSlotUnits2 = kHalfBytes >> 4;

struct alignas(8) PairBarriers {
  unsigned long long info_full[2];
  unsigned long long info_free[2];
  unsigned long long idx_full[2];        // second CTA: the first CTA has written the index of the item
  unsigned long long q_full[2];          // first CTA: the Q tiles X of BOTH CTAs are in shared memory
  unsigned long long q_free[2];
  unsigned long long full[kRing2];       // first CTA: the slot holds its half tile in BOTH CTAs
  unsigned long long free_[kRing2];
  unsigned long long s_full[2];
  unsigned long long p_half[2][2];       // first CTA: the softmax threads of BOTH CTAs have stored this half of P
  unsigned long long o_done[2];
  unsigned long long o_free[2];          // first CTA: the epilogues of BOTH CTAs have read O
  unsigned long long drain;
  int idx[2];                            // second CTA: item indices handed over by the first
  long long wait_cycles;                 // directly before abort_flag (mbar_wait reads it)
  int abort_flag;
  unsigned tmem_base;
  int dead;
  ItemInfo info[2];
};
constexpr int kPairSmemBytes = 1024 + kTileBytes * 2 + kHalfBytes * kRing2 + kStageBytes + (int)sizeof(PairBarriers) + 64;
static_assert(kPairSmemBytes <= 232448, "shared memory of one CTA");

// fp32 accumulate, bf16 A and B, M = 256 over the pair, N = 128
constexpr unsigned kIdescBase2 = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((256u >> 4) << 24);
constexpr unsigned kIdescQK2 = kIdescBase2;
constexpr unsigned kIdescPV2 = kIdescBase2 | (1u << 16);

__device__ __forceinline__ unsigned cluster_rank() {
  unsigned r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of `local` (a shared-memory address of this CTA) in CTA `rank` of the cluster
__device__ __forceinline__ unsigned map_to_rank(unsigned local, unsigned rank) {
  unsigned raddr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(raddr) : "r"(local), "r"(rank));
  return raddr;
}
// Arrival on a barrier named by a cluster address (this CTA's or the partner's), without a cluster-scope
// release (which costs a memory barrier on the arriving warp): for hand-overs whose data lives in tensor
// memory and is ordered by the tcgen05 fences, not by this arrival.
__device__ __forceinline__ void mbar_arrive_cluster_plain(unsigned cluster_bar) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_bar) : "memory");
}
__device__ __forceinline__ void st_cluster_u32(unsigned cluster_addr, unsigned v) {
  asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
// bounded wait that also makes the partner's earlier writes to this CTA's shared memory visible
__device__ __forceinline__ bool mbar_try_wait_cluster(unsigned bar, unsigned parity) {
  unsigned ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster(unsigned bar, unsigned parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t_end = clock64() + *reinterpret_cast<const volatile long long*>(abort_flag - 2);
#pragma unroll 1
  while (!*abort_flag && clock64() < t_end)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  *abort_flag = 1;
  return false;
}
// Tiled TMA load issued by either CTA of the pair into its own shared memory, completing on the barrier
// at `bar`'s offset in the pair's first CTA.  No multicast.
__device__ __forceinline__ void tma_load_3d_pair(unsigned dst, const void* tmap, int c0, int c1, int c2, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(tmap)), "r"(c0), "r"(c1), "r"(c2), "r"(bar & 0xFEFFFFFFu)
      : "memory");
}
// Batches of two-SM MMAs issued by the elected lane of the first CTA's MMA warp (see mma_ss_batch8).
__device__ __forceinline__ void mma2_ss_batch8(unsigned el, unsigned d_tmem, const unsigned long long (&a)[8],
                                               const unsigned long long (&b)[8], unsigned idesc) {
  asm volatile(
      "{\n\t.reg .pred P, T, F;\n\t"
      "setp.ne.b32 P, %18, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.u32 F, 0, 0;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %9, %17, F;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %2, %10, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %3, %11, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %4, %12, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %5, %13, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %6, %14, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %7, %15, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], %8, %16, %17, T;\n\t}"
      ::"r"(d_tmem), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(a[4]), "l"(a[5]), "l"(a[6]), "l"(a[7]),
        "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "l"(b[6]), "l"(b[7]), "r"(idesc), "r"(el)
      : "memory");
}
__device__ __forceinline__ void mma2_ts_batch4(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                               const unsigned long long (&b)[4], unsigned idesc, unsigned acc0) {
  asm volatile(
      "{\n\t.reg .pred P, T, Q;\n\t.reg .b32 p1, p2, p3;\n\t"
      "setp.ne.b32 P, %8, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "add.u32 p2, %1, 16;\n\t"
      "add.u32 p3, %1, 24;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %6, Q;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], [p1], %3, %6, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], [p2], %4, %6, T;\n\t"
      "@P tcgen05.mma.cta_group::2.kind::f16 [%0], [p3], %5, %6, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "r"(idesc), "r"(acc0), "r"(el)
      : "memory");
}
__device__ __forceinline__ void mma2_ts_batch4_first(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                                     const unsigned long long (&b)[4], unsigned idesc, unsigned acc0,
                                                     int n_on) {
  asm volatile(
      "{\n\t.reg .pred P, T, Q, E0, E1, E2, E3;\n\t.reg .b32 p1, p2, p3;\n\t"
      "setp.ne.b32 P, %8, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.b32 Q, %7, 0;\n\t"
      "setp.gt.s32 E0, %9, 0;\n\t"
      "setp.gt.s32 E1, %9, 1;\n\t"
      "setp.gt.s32 E2, %9, 2;\n\t"
      "setp.gt.s32 E3, %9, 3;\n\t"
      "and.pred E0, E0, P;\n\t"
      "and.pred E1, E1, P;\n\t"
      "and.pred E2, E2, P;\n\t"
      "and.pred E3, E3, P;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "add.u32 p2, %1, 16;\n\t"
      "add.u32 p3, %1, 24;\n\t"
      "@E0 tcgen05.mma.cta_group::2.kind::f16 [%0], [%1], %2, %6, Q;\n\t"
      "@E1 tcgen05.mma.cta_group::2.kind::f16 [%0], [p1], %3, %6, T;\n\t"
      "@E2 tcgen05.mma.cta_group::2.kind::f16 [%0], [p2], %4, %6, T;\n\t"
      "@E3 tcgen05.mma.cta_group::2.kind::f16 [%0], [p3], %5, %6, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "r"(idesc), "r"(acc0), "r"(el), "r"(n_on)
      : "memory");
}
// commit of the two-SM MMAs this thread has issued: arrives on the barrier at this offset in both CTAs
__device__ __forceinline__ void mma2_commit_both_pred(unsigned el, unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "setp.ne.b32 P, %1, 0;\n\t"
      "@P tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %2;\n\t}"
      ::"r"(bar), "r"(el), "h"((unsigned short)3)
      : "memory");
}
// the same, arriving in this CTA only
__device__ __forceinline__ void mma2_commit_local_pred(unsigned el, unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "setp.ne.b32 P, %1, 0;\n\t"
      "@P tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar), "r"(el)
      : "memory");
}

}  // namespace tcp

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(tc::kThreads, 1)
tc_attention_pair_kernel(ScheduleView s, TensorArgs t, int* status, const __grid_constant__ CUtensorMap tm_q,
                         const __grid_constant__ CUtensorMap tm_k64, const __grid_constant__ CUtensorMap tm_v,
                         const __grid_constant__ CUtensorMap tm_o, int q_tma, int o_tma, long long wait_cycles) {
  using namespace tcp;
  namespace cg = cooperative_groups;
  extern __shared__ unsigned char smem_raw[];
  // the same offsets in both CTAs of the pair: the MMA descriptors name them once for both
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  unsigned char* const stage_base = smem + kTileBytes * 2 + kHalfBytes * kRing2;
  PairBarriers* bars = reinterpret_cast<PairBarriers*>(stage_base + kStageBytes);
  volatile int* abort_flag = &bars->abort_flag;
  const unsigned q_smem = smem_u32(smem);                  // Q_A, then Q_B
  const unsigned ring_smem = q_smem + 2 * kTileBytes;
  int* const next_item = status + 16;                      // items handed out beyond the first one of every pair
  int* const ctas_done = status + 17;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = t.Hq / t.Hkv;
  cg::cluster_group cluster = cg::this_cluster();
  const unsigned rank = cluster_rank();                    // 0: issues the pair's MMAs, takes the items
  const int pair = blockIdx.x >> 1, num_pairs = gridDim.x >> 1;

  if (tid == 0) {
    bars->wait_cycles = wait_cycles;
    bars->dead = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    bars->abort_flag = (bars->dead || wait_cycles < kStrictBudget) ? 1 : 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->info_full[i]), 1);
      mbar_init(smem_u32(&bars->info_free[i]), rank == 0 ? kInfoReaders : kInfoReaders - 1);   // no MMA warp in CTA 1
      mbar_init(smem_u32(&bars->idx_full[i]), 1);
      mbar_init(smem_u32(&bars->q_full[i]), 2);                        // one arrival per CTA's Q loader
      mbar_init(smem_u32(&bars->q_free[i]), 1);
      mbar_init(smem_u32(&bars->s_full[i]), 1);
      mbar_init(smem_u32(&bars->p_half[i][0]), 8);                     // one arrival per softmax warp of tile i, both CTAs
      mbar_init(smem_u32(&bars->p_half[i][1]), 8);
      mbar_init(smem_u32(&bars->o_done[i]), 1);
      mbar_init(smem_u32(&bars->o_free[i]), 8);
    }
    for (int i = 0; i < kRing2; ++i) {
      mbar_init(smem_u32(&bars->full[i]), 2);                          // one arrival per CTA's load warp
      mbar_init(smem_u32(&bars->free_[i]), 1);
    }
    mbar_init(smem_u32(&bars->drain), 1);
    fence_barrier_init();
  }
  if (warp == kMmaWarp) {                                   // the same warp in both CTAs
    tmem_alloc2(smem_u32(&bars->tmem_base), kTmemCols);
    tmem_relinquish2();
  }
  tc_fence_before();
  cluster.sync();                                           // barriers of both CTAs exist before any remote arrival
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&bars->tmem_base);
  const bool dead = *reinterpret_cast<volatile int*>(&bars->dead) != 0;

  if (warp < 8) {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
  }
  if (warp < 8) {
    // ====================== softmax / correction / epilogue of one query tile ======================
    // As in the one-CTA kernel, except that the hand-over of P and the release of O arrive on the first
    // CTA's barriers.
    const int X = warp >> 2;
    const int gt = tid & 127;
    const unsigned lane_base = (unsigned)((warp & 3) * 32) << 16;
    const unsigned tmem_s = tmem + X * 128 + lane_base;
    const unsigned tmem_o = tmem + 256 + X * 128 + lane_base;
    const float sl2 = t.scale * 1.4426950408889634f;
    const unsigned long long sl2_2 = pack2(sl2, sl2);
    unsigned char* const stage = stage_base + warp * 4096;
    const unsigned bar_p0 = map_to_rank(smem_u32(&bars->p_half[X][0]), 0);
    const unsigned bar_p1 = map_to_rank(smem_u32(&bars->p_half[X][1]), 0);
    const unsigned bar_of = map_to_rank(smem_u32(&bars->o_free[X]), 0);
    // one arrival per warp (the tcgen05 stores and loads before it are warp-wide): on the own CTA's
    // barrier directly, on the first CTA's through the cluster
    auto warp_arrive = [&](unsigned local_bar, unsigned cluster_bar) {
      __syncwarp();
      if (lane == 0) {
        if (rank == 0) mbar_arrive(local_bar);
        else mbar_arrive_cluster_plain(cluster_bar);
      }
    };
    const unsigned loc_p0 = smem_u32(&bars->p_half[X][0]), loc_p1 = smem_u32(&bars->p_half[X][1]);
    const unsigned loc_of = smem_u32(&bars->o_free[X]);
    bool ok = !dead;
    int n_it = 0, c_tile = 0, e_item = 0;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_full[n_it & 1]), (n_it >> 1) & 1, abort_flag));
      if (!ok) break;
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, 1, 0);
      if (!g.valid) break;
      const int T = g.T;
      const bool active = X == 0 || g.b_active;              // of the pair: both CTAs run tile B or neither
      const int vseg = seg_of_row(inf, g.nseg, X * 128 + gt);   // -1: a row past the end of the request
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int j = 0; j < T && active; ++j) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->s_full[X]), c_tile & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        bool dense_unused;
        const int cnt = tile_keys_single(g, j, dense_unused);
        unsigned r[128];
        tmem_ld32(tmem_s, r);
        tmem_ld32(tmem_s + 32, r + 32);
        tmem_ld32(tmem_s + 64, r + 64);
        tmem_ld32(tmem_s + 96, r + 96);
        tmem_wait_ld();

        float alpha = 1.f;
        unsigned long long acc_a = pack2(0.f, 0.f), acc_b = pack2(0.f, 0.f);
        bool stored = false;
        if (cnt < kTileKeys) {
#pragma unroll
          for (int i = 0; i < 128; ++i)
            if (i >= cnt) r[i] = 0xff800000u;
        }
        if (j == 0) {
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
          for (int i = 0; i < 128; i += 8) {
            mx0 = max3(mx0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
            mx1 = max3(mx1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            mx2 = max3(mx2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
            mx3 = max3(mx3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
          }
          m_ref = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sl2;
        }
        {
          const unsigned long long neg_m2 = pack2(-m_ref, -m_ref);
          float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            mx0 = max3(mx0, __uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1]));
            mx1 = max3(mx1, __uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3]));
            mx0 = max3(mx0, __uint_as_float(r[64 + 4 * i]), __uint_as_float(r[64 + 4 * i + 1]));
            mx1 = max3(mx1, __uint_as_float(r[64 + 4 * i + 2]), __uint_as_float(r[64 + 4 * i + 3]));
            const unsigned long long xa =
                fma2(pack2(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1])), sl2_2, neg_m2);
            const unsigned long long xb =
                fma2(pack2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), sl2_2, neg_m2);
            float xa0, xa1, xb0, xb1;
            unpack2(xa, xa0, xa1);
            unpack2(xb, xb0, xb1);
            const float p0 = ex2(xa0), p1 = ex2(xa1), p2 = ex2(xb0), p3 = ex2(xb1);
            acc_a = add2(acc_a, pack2(p0, p1));
            acc_b = add2(acc_b, pack2(p2, p3));
            r[2 * i] = pack_bf16(p0, p1);
            r[2 * i + 1] = pack_bf16(p2, p3);
          }
          const float mx = fmaxf(mx0, mx1) * sl2;
          if (!__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
            tmem_st32(tmem_s, r);
            tmem_wait_st();
            tc_fence_before();
            warp_arrive(loc_p0, bar_p0);
#pragma unroll
            for (int i = 16; i < 32; ++i) {
              const unsigned long long xa =
                  fma2(pack2(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1])), sl2_2, neg_m2);
              const unsigned long long xb =
                  fma2(pack2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), sl2_2, neg_m2);
              float xa0, xa1, xb0, xb1;
              unpack2(xa, xa0, xa1);
              unpack2(xb, xb0, xb1);
              const float p0 = ex2(xa0), p1 = ex2(xa1), p2 = ex2(xb0), p3 = ex2(xb1);
              acc_a = add2(acc_a, pack2(p0, p1));
              acc_b = add2(acc_b, pack2(p2, p3));
              r[2 * i] = pack_bf16(p0, p1);
              r[2 * i + 1] = pack_bf16(p2, p3);
            }
            tmem_st32(tmem_s + 32, r + 32);
            tmem_wait_st();
            tc_fence_before();
            warp_arrive(loc_p1, bar_p1);
            stored = true;
          } else {
            // redo with the new reference: S is still intact in TMEM
            if (mx > m_ref + 8.f) {
              alpha = ex2(m_ref - mx);
              m_ref = mx;
            }
            unsigned s4[32];
            const float neg_m = -m_ref;
            float ps = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              tmem_ld32(tmem_s + c * 32, s4);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                const float p0 = c * 32 + 2 * i < cnt ? ex2(fmaf(__uint_as_float(s4[2 * i]), sl2, neg_m)) : 0.f;
                const float p1 = c * 32 + 2 * i + 1 < cnt ? ex2(fmaf(__uint_as_float(s4[2 * i + 1]), sl2, neg_m)) : 0.f;
                ps += p0 + p1;
                r[c * 16 + i] = pack_bf16(p0, p1);
              }
            }
            acc_a = pack2(ps, 0.f);
            acc_b = pack2(0.f, 0.f);
#pragma unroll 1
            for (int c = 0; c < 4; ++c) {
              tmem_ld32(tmem_o + c * 32, s4);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) s4[i] = __float_as_uint(__uint_as_float(s4[i]) * alpha);
              tmem_st32(tmem_o + c * 32, s4);
            }
          }
        }
        if (!stored) {
          tmem_st32(tmem_s, r);
          tmem_st32(tmem_s + 32, r + 32);
          tmem_wait_st();
          tc_fence_before();
          warp_arrive(loc_p0, bar_p0);
          warp_arrive(loc_p1, bar_p1);
        }
        {
          float s0, s1, s2, s3;
          unpack2(acc_a, s0, s1);
          unpack2(acc_b, s2, s3);
          l_sum = l_sum * alpha + ((s0 + s1) + (s2 + s3));
        }
        ++c_tile;
      }
      if (!ok) break;
      // ------------------------------- epilogue -------------------------------------------
      if (active) {
        const int kv_head = inf->kv_head;
        const bool row_valid = vseg >= 0;
        const SegInfo* sg = &inf->seg[0];
        const long long row_off = sg->row_off;
        const int prow = sg->prow0 + (X * 128 + gt);            // packed row of this thread within its request
        const int a = prow / G;
        const int h = kv_head * G + (prow - a * G);
        unsigned o[128];
        if (T > 0) {
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->o_done[X]), e_item & 1, abort_flag));
          if (!ok) break;
          tc_fence_after();
          ++e_item;
          tmem_ld32(tmem_o, o);
          tmem_ld32(tmem_o + 32, o + 32);
          tmem_ld32(tmem_o + 64, o + 64);
          tmem_ld32(tmem_o + 96, o + 96);
          tmem_wait_ld();
          tc_fence_before();
          warp_arrive(loc_of, bar_of);                        // the next item may overwrite O
          const float inv = 1.f / l_sum;
          const float lse = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
          const int seg_first = __shfl_sync(0xffffffffu, vseg, 0), seg_last = __shfl_sync(0xffffffffu, vseg, 31);
          const int prow_first = __shfl_sync(0xffffffffu, prow, 0);
          const bool by_tma = o_tma && seg_first >= 0 && seg_last >= 0 && prow_first % G == 0;
          const int tok_first = (int)row_off + prow_first / G;
          const long long my_dst = row_valid ? ((row_off + a) * t.out_stride + (long long)h * 128) * 2 : -1;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (lane == 0) bulk_wait_read();
            __syncwarp();
#pragma unroll
            for (int c = 0; c < 8; ++c) {
              const int i = hh * 64 + c * 8;
              uint4 v4;
              v4.x = pack_bf16(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv);
              v4.y = pack_bf16(__uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
              v4.z = pack_bf16(__uint_as_float(o[i + 4]) * inv, __uint_as_float(o[i + 5]) * inv);
              v4.w = pack_bf16(__uint_as_float(o[i + 6]) * inv, __uint_as_float(o[i + 7]) * inv);
              *reinterpret_cast<uint4*>(stage + lane * 128 + ((c ^ (lane & 7)) << 4)) = v4;
            }
            if (by_tma) {
              fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                tma_store_3d(&tm_o, smem_u32(stage), hh * 64, kv_head * G, tok_first);
                bulk_commit_group();
              }
            } else {
              __syncwarp();
              const int ch = lane & 7;
#pragma unroll 2
              for (int it = 0; it < 8; ++it) {
                const int row = it * 4 + (lane >> 3);
                const long long dst_off = __shfl_sync(0xffffffffu, my_dst, row);
                if (dst_off >= 0)
                  *reinterpret_cast<uint4*>(t.out + dst_off + hh * 128 + ch * 16) =
                      *reinterpret_cast<const uint4*>(stage + row * 128 + ((ch ^ (row & 7)) << 4));
              }
              __syncwarp();
            }
          }
          if (row_valid && t.lse != nullptr) t.lse[(row_off + a) * t.Hq + h] = lse;
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->info_free[n_it & 1]));
      ++n_it;
    }
    if (lane == 0) bulk_wait_all();
    tc_fence_before();
  } else if (warp == 9) {
    // ============================== item fetch and Q loads ===============================
    // The first CTA takes item indices from the launch's counter and hands each one to its partner
    // (a store into the partner's shared memory, then an arrival on its `idx_full` barrier); either CTA
    // writes its own record: the same key tiles, its own 256 of the item's 512 rows.
    bool ok = !dead;
    int n_it = 0;
    int eq[2] = {0, 0};
    auto write_info = [&](ItemInfo* dst, int idx) {
      if (lane == 0) {
        if (idx < s.num_items) {
          const WorkItem wi = s.items[idx];
          const ReqMeta rq = s.reqs[wi.req];
          const int own = (rq.n + kTileKeys - 1) / kTileKeys;
          const int pair_rows = min(kPairRows, rq.n * G - wi.row0);
          SegInfo si;
          si.row_off = rq.row_off;
          si.n = rq.n;
          si.prow0 = wi.row0 + (int)rank * kTileRows;
          si.begin = 0;
          si.count = max(0, min(kTileRows, pair_rows - (int)rank * kTileRows));
          si.tok_off = rq.tok_off;
          si.tile_end = own;
          dst->seg[0] = si;
          dst->kv_head = wi.kv_head;
          dst->split = 0;
          dst->m = 0;
          dst->page_off = 0;
          dst->nseg = 1;
          dst->nrows = pair_rows;                          // of the pair: tile B runs in both CTAs or in neither
          dst->all_tiles = own;
          dst->valid = 1;
        } else {
          dst->valid = 0;
        }
      }
      __syncwarp();
    };
    if (ok) {
      write_info(&bars->info[0], pair);
      if (lane == 0) mbar_arrive(smem_u32(&bars->info_full[0]));
    }
    __syncwarp();
    while (ok) {
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, 1, 0);
      if (!g.valid) break;
      for (int x = 0; x < 2 && ok; ++x) {
        if (x == 1 && !g.b_active) break;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->q_free[x]), (eq[x] & 1) ^ 1, abort_flag));
        if (!ok) break;
        ++eq[x];
        const unsigned qf = smem_u32(&bars->q_full[x]);
        const unsigned q_dst = q_smem + x * kTileBytes;
        const SegInfo* s0 = &inf->seg[0];
        if (q_tma) {
          if (lane == 0) {
            const int tok = (int)s0->row_off + (s0->prow0 + x * 128) / G;
            if (rank == 0) mbar_arrive_expect_tx(qf, 2u * kTileBytes);      // the Q tiles of both CTAs
            tma_load_3d_pair(q_dst, &tm_q, 0, inf->kv_head * G, tok, qf);
            tma_load_3d_pair(q_dst + kTileBytes / 2, &tm_q, 64, inf->kv_head * G, tok, qf);
            if (rank != 0) mbar_arrive_remote(qf, 0);
          }
        } else {
          // gathers into the page-image layout (the heads of a KV group do not divide 128): packed row
          // p = token a * G + head jj of the group; rows past the end are zero-filled
          const int packed_rows = s0->n * G;
          const int r0 = lane >> 4, c16 = lane & 15;
          int prow = s0->prow0 + x * 128 + r0;
          const int a0 = prow / G;
          int jj = prow - a0 * G;
          const long long q_row_bytes = t.q_stride * 2;
          const char* q_base = t.q + (s0->row_off * t.q_stride + (long long)inf->kv_head * G * 128) * 2 + c16 * 16;
          const char* src_row = q_base + a0 * q_row_bytes;
#pragma unroll 4
          for (int i = 0; i < 64; ++i) {
            const bool valid = prow < packed_rows;
            cp_async16(q_dst + tile_chunk_offset(r0 + 2 * i, c16), valid ? src_row + jj * 256 : q_base, valid ? 16u : 0u);
            prow += 2;
            jj += 2;
            while (jj >= G) {
              jj -= G;
              src_row += q_row_bytes;
            }
          }
          cp_async_commit();
          cp_async_wait<0>();
          fence_proxy_async();
          __syncwarp();
          if (lane == 0) {
            if (rank == 0) mbar_arrive(qf);
            else mbar_arrive_remote(qf, 0);
          }
        }
        __syncwarp();
      }
      if (!ok) break;
      {
        const int nn = n_it + 1;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_free[nn & 1]), ((nn >> 1) & 1) ^ 1, abort_flag));
        if (!ok) break;
        int idx = 0;
        if (rank == 0) {
          if (lane == 0) {
            idx = num_pairs + atomicAdd(next_item, 1);
            st_cluster_u32(map_to_rank(smem_u32(&bars->idx[nn & 1]), 1), (unsigned)idx);
            mbar_arrive_remote(smem_u32(&bars->idx_full[nn & 1]), 1);
          }
        } else {
          // item nn is the (nn / 2)-th use of this slot after the pair's first item (which needs no message)
          ok = __all_sync(0xffffffffu,
                          mbar_wait_cluster(smem_u32(&bars->idx_full[nn & 1]), ((nn - 1) >> 1) & 1, abort_flag));
          if (!ok) break;
          if (lane == 0) idx = *reinterpret_cast<volatile int*>(&bars->idx[nn & 1]);
        }
        idx = __shfl_sync(0xffffffffu, idx, 0);
        write_info(&bars->info[nn & 1], idx);
        if (lane == 0) mbar_arrive(smem_u32(&bars->info_full[nn & 1]));
      }
      __syncwarp();
      ++n_it;
    }
    // After a give-up the Q loads issued last may still be in flight (they complete on the first CTA's
    // barrier): the first CTA waits (bounded) for them, the second waits out the same limit.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      if (rank == 0) {
        for (int x = 0; x < 2; ++x)
          if (eq[x] > 0)
            for (unsigned it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bars->q_full[x]), (eq[x] - 1) & 1); ++it)
              __nanosleep(256);
      } else if (eq[0] > 0) {
        for (unsigned it = 0; it < 4096; ++it) __nanosleep(256);
      }
    }
  } else if (warp >= 10) {
    // ====================================== loads =======================================
    // Warp 10 stages this CTA's half of every K tile (the rows of keys 64 r .. 64 r + 63), warp 11 its
    // half of every V tile (dims 64 r .. 64 r + 63 of all 128 keys), each running ahead of the MMAs by
    // the depth of the ring.  Ring use u = 2 * (key tiles before) + (0: K, 1: V).
    const int is_v = warp - 10;
    bool ok = !dead;
    int n_it = 0, U = 0;
    int last_armed = -1;
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_full[n_it & 1]), (n_it >> 1) & 1, abort_flag));
      if (!ok) break;
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, 1, 0);
      if (!g.valid) break;
      const int kv_head = inf->kv_head;
      const long long row_off = inf->seg[0].row_off;
      for (int j = 0; j < g.T; ++j) {
        const int u = U + 2 * j + is_v;
        const int slot = u % kRing2;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->free_[slot]), ((u / kRing2) & 1) ^ 1, abort_flag));
        if (!ok) break;
        const unsigned dst = ring_smem + slot * kHalfBytes;
        const unsigned full = smem_u32(&bars->full[slot]);
        const int key0 = j * kTileKeys, cnt = min(kTileKeys, g.n0 - key0);
        if (cnt >= kTileKeys) {
          if (lane == 0) {
            const int row = (int)row_off + key0;
            if (rank == 0) mbar_arrive_expect_tx(full, (unsigned)kTileBytes);   // both CTAs' halves
            if (!is_v) {
              // 64 keys x 128 dims: two boxes of 64 rows, the 64-dim halves 8 KB apart
              tma_load_3d_pair(dst, &tm_k64, 0, kv_head, row + 64 * (int)rank, full);
              tma_load_3d_pair(dst + kHalfBytes / 2, &tm_k64, 64, kv_head, row + 64 * (int)rank, full);
            } else {
              // 128 keys x 64 dims: one box
              tma_load_3d_pair(dst, &tm_v, 64 * (int)rank, kv_head, row, full);
            }
            if (rank != 0) mbar_arrive_remote(full, 0);
            last_armed = u;
          }
          __syncwarp();
          continue;
        }
        // ragged last tile: 16-byte gathers, zero-filled past the end
        if (!is_v) {
          // page-image layout of 64 rows (see tile_chunk_offset): keys 64 r + i
          const int r0 = lane >> 4, c16 = lane & 15;
          const char* first = t.k + ((row_off + key0) * t.kv_stride + (long long)kv_head * 128) * 2 + c16 * 16;
          const long long row_bytes = t.kv_stride * 2;
          const char* rowp = first + 64 * (int)rank * row_bytes;
#pragma unroll 4
          for (int i = 0; i < 32; ++i) {
            const int rr = r0 + 2 * i;
            const bool valid = 64 * (int)rank + rr < cnt;
            cp_async16(dst + tile_chunk_offset(rr, c16), valid ? rowp + rr * row_bytes : first, valid ? 16u : 0u);
          }
        } else {
          // 128 keys x 64 dims, rows of 128 bytes, 16-byte chunks XOR-placed by the row (the 128-byte swizzle)
          const int r0 = lane >> 3, c8 = lane & 7;
          const char* rowp = t.v + ((row_off + key0) * t.kv_stride + (long long)kv_head * 128 + 64 * (int)rank) * 2 + c8 * 16;
          const long long row_bytes = t.kv_stride * 2;
#pragma unroll 4
          for (int i = 0; i < 32; ++i) {
            const int rr = r0 + 4 * i;
            const bool valid = rr < cnt;
            cp_async16(dst + rr * 128 + ((c8 ^ (rr & 7)) << 4), valid ? rowp + rr * row_bytes : rowp, valid ? 16u : 0u);
          }
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          if (rank == 0) mbar_arrive(full);
          else mbar_arrive_remote(full, 0);
        }
      }
      if (!ok) break;
      U += 2 * g.T;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->info_free[n_it & 1]));
      ++n_it;
    }
    cp_async_wait<0>();
    if (!dead && (!ok || *abort_flag) && lane == 0 && last_armed >= 0) {
      if (rank == 0) {
        for (unsigned it = 0;
             it < 4096 && !mbar_try_wait(smem_u32(&bars->full[last_armed % kRing2]), (last_armed / kRing2) & 1); ++it)
          __nanosleep(256);
      } else {
        for (unsigned it = 0; it < 4096; ++it) __nanosleep(256);
      }
    }
  } else if (warp == kMmaWarp && rank == 0) {
    // ===================================== MMA issue =====================================
    // The issue order of the one-CTA kernel, every MMA for tile X of both CTAs at once:
    //   S_A(0) S_B(0) | O_A(0) S_A(1) | O_B(0) S_B(1) | ...
    bool ok = !dead;
    if (ok) {
      const unsigned bar_full = smem_u32(&bars->full[0]), bar_free = smem_u32(&bars->free_[0]);   // slot i: + 8 i
      const unsigned bar_p = smem_u32(&bars->p_half[0][0]);     // [x][half]: + 16 x + 8 half
      const unsigned bar_s = smem_u32(&bars->s_full[0]), bar_qfull = smem_u32(&bars->q_full[0]);   // [x]: + 8 x
      const unsigned bar_qfree = smem_u32(&bars->q_free[0]), bar_odone = smem_u32(&bars->o_done[0]);
      const unsigned bar_ofree = smem_u32(&bars->o_free[0]);
      // Layouts of this CTA's half tiles (the same in the partner).  K half, 64 keys x 128 dims: the page
      // image of a gathered ragged tile (8-row groups 2048 bytes apart, the 64-dim halves 1024 bytes) or
      // the dense layout TMA writes (8-row groups 1024 bytes apart, halves 8 KB).  V half, 128 keys x 64
      // dims, one layout: rows of 128 bytes, 8-key groups 1024 bytes apart.  Q as in the one-CTA kernel.
      const unsigned q_hi = q_tma ? 1024u : 64u;
      const unsigned long long q_desc0 = make_desc(q_smem, 16, q_tma ? 1024u : 2048u);
      const unsigned long long q_desc1 = q_desc0 + (kTileBytes >> 4);
      const unsigned long long kb_img = make_desc(ring_smem, 16, 2048), kb_dense = make_desc(ring_smem, 16, 1024);
      const unsigned long long vb = make_desc(ring_smem, 1024, 1024);
      constexpr unsigned kVStep = 128;                         // 16 keys further, in 16-byte units
      const unsigned tmem_u = __shfl_sync(0xffffffffu, tmem, 0);
      const unsigned tmem_s1 = tmem_u + 128, tmem_o0 = tmem_u + 256, tmem_o1 = tmem_u + 384;
#define BICACHE_WAIT(bar, parity) __all_sync(0xffffffffu, mbar_wait((bar), (parity), abort_flag))
      const unsigned el = elect_one() ? 1u : 0u;
      auto issue_s = [&](unsigned d_tmem, unsigned long long qd, unsigned long long kd, unsigned k_hi) {
        unsigned long long a[8], b[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          a[k] = qd + (k >> 2) * q_hi + (k & 3) * 2;
          b[k] = kd + (k >> 2) * k_hi + (k & 3) * 2;
        }
        mma2_ss_batch8(el, d_tmem, a, b, kIdescQK2);
      };
      auto issue_pv = [&](unsigned o_tmem, unsigned p_tmem, unsigned long long vd, int half, unsigned acc0, int ksteps) {
        unsigned long long b[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) b[k] = vd + (half * 4 + k) * kVStep;
        if (ksteps == 8) mma2_ts_batch4(el, o_tmem, p_tmem + half * 32, b, kIdescPV2, half ? 1u : acc0);
        else mma2_ts_batch4_first(el, o_tmem, p_tmem + half * 32, b, kIdescPV2, half ? 1u : acc0, ksteps - half * 4);
      };
      int n_it = 0;
      int c0 = 0, c1 = 0;
      int e0 = 0, e1 = 0;
      unsigned u = 0;
      ok = BICACHE_WAIT(smem_u32(&bars->info_full[0]), 0);
      Geo cur = read_geo_uniform(&bars->info[0], 1, 0);
      bool dn = false;
      int ksteps = 8;
      bool pre = false;
      while (ok && cur.valid) {
        Geo nxt;
        nxt.valid = 0;
        bool have_next = false, can_pre = false;
        const int T = cur.T;
        if (T > 0) {
          const bool b_on = cur.b_active;
          if (!pre) {
            ok = BICACHE_WAIT(bar_full + (u & 7) * 8, (u >> 3) & 1) && BICACHE_WAIT(bar_qfull, e0 & 1);
            if (!ok) break;
            tc_fence_after();
            ksteps = (tile_keys_single(cur, 0, dn) + 15) >> 4;
            const unsigned long long kd0 = (dn ? kb_dense : kb_img) + (u & 7) * kSlotUnits2;
            issue_s(tmem_u, q_desc0, kd0, dn ? 512u : 64u);
            mma2_commit_both_pred(el, bar_s);
            if (T == 1) mma2_commit_both_pred(el, bar_qfree);
            if (b_on) {
              ok = BICACHE_WAIT(bar_p, c0 & 1) && BICACHE_WAIT(bar_qfull + 8, e1 & 1);
              if (!ok) break;
              issue_s(tmem_s1, q_desc1, kd0, dn ? 512u : 64u);
              mma2_commit_both_pred(el, bar_s + 8);
              if (T == 1) mma2_commit_both_pred(el, bar_qfree + 8);
            }
            mma2_commit_both_pred(el, bar_free + (u & 7) * 8);
          }
          ok = BICACHE_WAIT(bar_full + ((u + 1) & 7) * 8, ((u + 1) >> 3) & 1) && BICACHE_WAIT(bar_ofree, (e0 & 1) ^ 1);
          if (!ok) break;
          auto tile_iter = [&](auto last_c, int j) {
            constexpr bool last = decltype(last_c)::value;
            const unsigned sv = (u + 1) & 7, sn = (u + 2) & 7;
            const unsigned long long v_desc = vb + sv * kSlotUnits2;
            const unsigned acc0 = j > 0 ? 1u : 0u;
            ok = BICACHE_WAIT(bar_p, c0 & 1);
            if (!ok) return;
            tc_fence_after();
            issue_pv(tmem_o0, tmem_u, v_desc, 0, acc0, ksteps);
            bool s_on0 = true, s_on1 = b_on;
            bool q_last = j + 2 == T;
            bool dn_next = false;
            int ks_next = 8;
            if (!last) {
              ks_next = (tile_keys_single(cur, j + 1, dn_next) + 15) >> 4;
            } else {
              const int nn = n_it + 1;
              ok = BICACHE_WAIT(smem_u32(&bars->info_full[nn & 1]), (nn >> 1) & 1);
              if (!ok) return;
              nxt = read_geo_uniform(&bars->info[nn & 1], 1, 0);
              have_next = true;
              can_pre = nxt.valid && nxt.T > 0;
              s_on0 = can_pre;
              s_on1 = can_pre && nxt.b_active;
              q_last = nxt.T == 1;
              if (can_pre) ks_next = (tile_keys_single(nxt, 0, dn_next) + 15) >> 4;
            }
            if (s_on0) {
              ok = BICACHE_WAIT(bar_full + sn * 8, ((u + 2) >> 3) & 1);
              if (!ok) return;
            }
            const unsigned long long k_desc = (dn_next ? kb_dense : kb_img) + sn * kSlotUnits2;
            const unsigned k_hi = dn_next ? 512u : 64u;
            ok = BICACHE_WAIT(bar_p + 8, c0 & 1);
            if (!ok) return;
            tc_fence_after();
            issue_pv(tmem_o0, tmem_u, v_desc, 1, acc0, ksteps);
            ++c0;
            if (last) {
              mma2_commit_both_pred(el, bar_odone);
              ++e0;
            }
            if (s_on0) {
              if (last) {
                ok = BICACHE_WAIT(bar_qfull, e0 & 1);
                if (!ok) return;
              }
              issue_s(tmem_u, q_desc0, k_desc, k_hi);
              mma2_commit_both_pred(el, bar_s);
              if (q_last) mma2_commit_both_pred(el, bar_qfree);
            }
            if (b_on) {
              if (j == 0) {
                ok = BICACHE_WAIT(bar_ofree + 8, (e1 & 1) ^ 1);
                if (!ok) return;
              }
              ok = BICACHE_WAIT(bar_p + 16, c1 & 1);
              if (!ok) return;
              tc_fence_after();
              issue_pv(tmem_o1, tmem_s1, v_desc, 0, acc0, ksteps);
            }
            if (b_on) {
              ok = BICACHE_WAIT(bar_p + 24, c1 & 1);
              if (!ok) return;
              tc_fence_after();
              issue_pv(tmem_o1, tmem_s1, v_desc, 1, acc0, ksteps);
              ++c1;
              if (last) {
                mma2_commit_both_pred(el, bar_odone + 8);
                ++e1;
              }
            }
            if (s_on1) {
              if (last) {
                ok = BICACHE_WAIT(bar_qfull + 8, e1 & 1);
                if (!ok) return;
              }
              issue_s(tmem_s1, q_desc1, k_desc, k_hi);
              mma2_commit_both_pred(el, bar_s + 8);
              if (q_last) mma2_commit_both_pred(el, bar_qfree + 8);
            }
            mma2_commit_both_pred(el, bar_free + sv * 8);
            if (s_on0) mma2_commit_both_pred(el, bar_free + sn * 8);
            u += 2;
            dn = dn_next;
            ksteps = ks_next;
            if (!last) {
              ok = BICACHE_WAIT(bar_full + ((u + 1) & 7) * 8, ((u + 1) >> 3) & 1);
              if (!ok) return;
            }
          };
          for (int j = 0; j + 1 < T && ok; ++j) tile_iter(std::false_type{}, j);
          if (ok) tile_iter(std::true_type{}, T - 1);
          if (!ok) break;
        }
        if (!have_next) {
          const int nn = n_it + 1;
          ok = BICACHE_WAIT(smem_u32(&bars->info_full[nn & 1]), (nn >> 1) & 1);
          if (!ok) break;
          nxt = read_geo_uniform(&bars->info[nn & 1], 1, 0);
        }
        if (elect_one()) mbar_arrive(smem_u32(&bars->info_free[n_it & 1]));
        __syncwarp();
        pre = can_pre;
        cur = nxt;
        ++n_it;
      }
#undef BICACHE_WAIT
      // Whatever happened, let every MMA issued so far finish before the pair's TMEM is released.
      __syncwarp();
      mma2_commit_local_pred(el, smem_u32(&bars->drain));
      mbar_wait_issued(smem_u32(&bars->drain), 0);
    }
    __syncwarp();
  }

  // The pair leaves together: the first CTA's MMAs read the partner's shared memory and write its TMEM.
  tc_fence_before();
  cluster.sync();
  tc_fence_after();
  if (warp == kMmaWarp) tmem_dealloc2(tmem, kTmemCols);
  if (tid == 0) {
    if (!dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
    __threadfence();
    if (atomicAdd(ctas_done, 1) == (int)gridDim.x - 1) {
      *next_item = 0;
      *ctas_done = 0;
      __threadfence();
    }
  }
}

// Sets the kernel's limits and returns how many CTA pairs the device runs at once.
inline cudaError_t configure_tc_attention_pair(int* max_pairs) {
  cudaFuncAttributes attr;
  cudaError_t e = cudaFuncGetAttributes(&attr, tc_attention_pair_kernel);
  if (e != cudaSuccess) return e;
  if (attr.numRegs * tc::kThreads < 2 * tc::kGroupThreads * tc::kSoftmaxRegs + 128 * tc::kOtherRegs)
    return cudaErrorLaunchOutOfResources;
  e = cudaFuncSetAttribute(tc_attention_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, tcp::kPairSmemBytes);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(2, 1, 1);
  cfg.blockDim = dim3(tc::kThreads, 1, 1);
  cfg.dynamicSmemBytes = tcp::kPairSmemBytes;
  int n = 0;
  e = cudaOccupancyMaxActiveClusters(&n, tc_attention_pair_kernel, &cfg);
  if (e != cudaSuccess) return e;
  *max_pairs = n;
  return n > 0 ? cudaSuccess : cudaErrorLaunchOutOfResources;
}

// Tensor maps of a launch on CTA pairs: q and o (and their flags) as in TcTensorMaps; k64: [rows][Hkv][128]
// with a box of (64 dims, 1 head, 64 rows); v: the box of (64 dims, 1 head, 128 rows) of TcTensorMaps.
inline cudaError_t launch_tc_attention_pair(const ScheduleView& s, const TensorArgs& t, int* status, int max_pairs,
                                            const CUtensorMap& tm_q, const CUtensorMap& tm_k64, const CUtensorMap& tm_v,
                                            const CUtensorMap& tm_o, int q_tma, int o_tma, long long wait_cycles,
                                            cudaStream_t stream) {
  const int pairs = s.num_items < max_pairs ? s.num_items : max_pairs;
  tc_attention_pair_kernel<<<2 * pairs, tc::kThreads, tcp::kPairSmemBytes, stream>>>(
      s, t, status, tm_q, tm_k64, tm_v, tm_o, q_tma, o_tma, wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  return cudaGetLastError();
}

}  // namespace bicache
