// Tensor-core attention for bf16, head_dim 128, on sm_100a: tcgen05.mma with TMEM accumulators.
//
// Persistent kernel: one CTA per SM takes work items from a shared counter (longest items first).
// A work item is up to 256 packed query rows (one request, one KV head) as two 128-row tiles A
// and B that share every K/V tile, against a range of key tiles of 128 keys - first the cached
// prefix (pages of 16 tokens, staged with cp.async.bulk because a pool page already is the
// shared-memory image the MMA reads), then the request's own rows (full tiles by tiled TMA loads
// through tensor maps of the caller's row-major K/V; the ragged last tile by 16-byte cp.async
// gathers, zero-filled past the end).  Q tiles come by TMA as well when the query heads of a KV
// group divide 128, else by gathers.
// Per key tile and query tile: S = Q K^T (tcgen05, fp32 in TMEM) -> online softmax in registers
// (one thread per row) -> P as bf16 written over S in TMEM -> O += P V (tcgen05, A from TMEM).
// The MMA warp issues  O_A(j), S_A(j+1), O_B(j), S_B(j+1)  so that each softmax warpgroup works
// while the other tile's MMAs run, and the stream of key tiles runs on across item boundaries:
// after the last O_X of an item comes the first S_X of the next item, whose Q, K and V were
// fetched while the current item was computed, so only the epilogue of a query tile (TMEM ->
// registers -> bf16 -> shared memory -> TMA store) stands between two items.  The running maximum
// only moves when it grew by more than 2^8, so rescaling O is rare; the final normalisation uses
// the same reference, which keeps the result exact.
//
// Roles: warps 0-3 softmax/correction/epilogue of tile A, warps 4-7 of tile B (one thread per
// row), warp 8 MMA issue and TMEM ownership, warp 9 item fetch and Q loads, warp 10 K tiles,
// warp 11 V tiles.  The softmax uses packed fp32 instructions and 3-input maxima; MMAs are issued
// branch-free by an elected lane of a converged warp.  All waits are bounded; a wait that gives
// up raises a sticky status word and the CTA drains and exits.
#pragma once
#include <cuda.h>
#include <type_traits>
#include <cuda_bf16.h>
#include "common.cuh"
#include "simt_kernels.cuh"

namespace bicache {

constexpr bool kTensorPathBuilt = true;

namespace tc {

constexpr int kTileBytes = kTileKeys * 128 * 2;  // 32 KB: one 128 x 128 bf16 tile
constexpr int kPageBytes = 4096;
constexpr int kRing = 4;                         // K/V ring slots of one tile each: K0 V0 K1 V1
constexpr int kThreads = 384;
constexpr int kGroupThreads = 128;               // softmax threads of one query tile (one per row)
constexpr int kLoadThreads = 32;                 // one warp loads a whole tile
constexpr int kSoftmaxRegs = 184;                // registers per thread after setmaxnreg
constexpr int kOtherRegs = 136;
constexpr int kMmaWarp = 8;
#ifndef BICACHE_POLY_PERIOD
#define BICACHE_POLY_PERIOD 0
#endif
constexpr int kPolyPeriod = BICACHE_POLY_PERIOD;                   // of every kPolyPeriod groups of 4 scores, one sends 2 scores to the FMA-pipe cubic (0: none)
constexpr long long kWaitCycles = 400000000LL;   // default budget of a bounded wait: about 0.2 s of SM clocks

// shared-memory layout (dynamic, 1024-byte aligned by hand): Q_A, Q_B, ring, output staging
// (4 KB per softmax warp), barriers and item records
// One work item as the roles see it, written by warp 9.  Its query rows are `nseg` segments; segment k
// is rows [begin, begin + count) of the item = packed rows prow0 .. of one request.  An item of a plain
// schedule has one segment; an item of a tiled schedule has one per request with rows in its row tile
// (all of one prefix group).  Key tiles: the cached prefix's, then every segment's request's own rows.
struct SegInfo {
  long long row_off;                     // first row of the request in q / k / v / out
  int n;                                 // its rows: queries and own keys
  int prow0, begin, count;
  int tok_off;                           // its first token in the call's token numbering (key-split partials)
  int tile_end;                          // key tiles of the item up to and including this request's own tiles
};
struct ItemInfo {
  int valid;                             // 0: the items are exhausted
  int kv_head, split;
  int m, page_off;
  int nseg, nrows;                       // segments; end of the last one
  int all_tiles;                         // ceil(m / 128) + sum over the segments of ceil(n / 128)
  SegInfo seg[kMaxSegs];
};
struct alignas(8) Barriers {
  unsigned long long info_full[2];       // item record (double-buffered by item parity) is written
  unsigned long long info_free[2];       // every role is done with the record
  unsigned long long q_full[2];          // Q tile of the item is in shared memory (per query tile)
  unsigned long long q_free[2];          // the last S of the item has been computed: Q may be replaced
  unsigned long long full[kRing];        // ring slot holds its tile
  unsigned long long free_[kRing];       // the MMAs reading the slot have completed
  unsigned long long s_full[2];          // S = Q K^T of the current key tile is in TMEM (per query tile)
  unsigned long long p_half[2][2];       // P of keys 0-95 / 96-127 is in TMEM and O is rescaled (per query tile)
  unsigned long long o_done[2];          // the last O += P V of the item has completed (per query tile)
  unsigned long long o_free[2];          // the epilogue has read O out of TMEM (per query tile)
  unsigned long long drain;
  // What the K loader found out about the key tiles, for the MMA warp and the softmax warps (which
  // then need no per-tile arithmetic of their own): entry (t & 7) describes the t-th key tile the CTA
  // has staged: keys | dense layout << 8 | (segment + 1) << 16 (segment -1: cached prefix).  A ring
  // of 8 is deep enough: the loaders run at most two tiles ahead of the MMAs, the softmax less than
  // one tile behind them.
  int tile_meta[8];
  long long wait_cycles;                 // SM-clock budget of every wait; directly before abort_flag (mbar_wait reads it)
  int abort_flag;
  unsigned tmem_base;
  int dead;                              // the context's status word was already set when the CTA started
  ItemInfo info[2];
};
constexpr int kInfoReaders = 8 + 1 + 2;  // arrivals on info_free: softmax warps, the MMA warp, the two load warps
constexpr int kStageBytes = 8 * 4096;
constexpr int kTmemCols = 512;           // S_A 0-127, S_B 128-255 (P over the first 64 of each), O_A 256-383, O_B 384-511
constexpr int kSmemBytes = 1024 + kTileBytes * (2 + kRing) + kStageBytes + (int)sizeof(Barriers) + 64;
static_assert(kSmemBytes <= 232448, "shared memory of one CTA");

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
// Bounded wait.  try_wait suspends the thread in hardware until the phase completes or a short
// system time limit passes, so the loop itself needs no sleep; the SM clock bounds the total.
// Returns false if the CTA's abort flag is up or (raising it) if the budget runs out.  Kept small:
// the kernels wait at some sixty places, every one an inlined copy, and their code has to stay in
// the instruction cache.
__device__ __forceinline__ bool mbar_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  // the budget sits in shared memory directly before the abort flag
  const long long t_end = clock64() + *reinterpret_cast<const volatile long long*>(abort_flag - 2);
#pragma unroll 1
  while (!*abort_flag && clock64() < t_end)
    if (mbar_try_wait(bar, parity)) return true;
  *abort_flag = 1;
  return false;
}
// A budget below this is the tests' way to walk the give-up path with barriers that all complete:
// the abort flag is up from the start, so every wait that is not over at its first poll gives up,
// and the launch reports a timeout.
constexpr long long kStrictBudget = 1024;
// Wait for work that is certain to finish (MMAs already issued): the default budget, whatever the
// per-wait budget or the abort flag say, because tensor memory must not be released under them.
__device__ __forceinline__ bool mbar_wait_issued(unsigned bar, unsigned parity) {
  const long long t0 = clock64();
  for (unsigned it = 0;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((it & 63u) == 63u && clock64() - t0 > kWaitCycles) return false;
  }
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

// Tiled TMA load of a 3-D box (dims innermost first: head dim, head, row) into shared memory.
// The innermost coordinate times the element size must be a multiple of 16 bytes.
__device__ __forceinline__ void tma_load_3d(unsigned dst, const void* tmap, int c0, int c1, int c2, unsigned bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(reinterpret_cast<unsigned long long>(tmap)), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}
// Tiled TMA store of a 3-D box from shared memory (bulk async-group completion).
__device__ __forceinline__ void tma_store_3d(const void* tmap, unsigned src, int c0, int c1, int c2) {
  asm volatile("cp.async.bulk.tensor.3d.global.shared::cta.tile.bulk_group [%0, {%2, %3, %4}], [%1];"
               ::"l"(reinterpret_cast<unsigned long long>(tmap)), "r"(src), "r"(c0), "r"(c1), "r"(c2)
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// the shared-memory source of every committed bulk store has been read
__device__ __forceinline__ void bulk_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// every committed bulk store has completed
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void tmem_alloc(unsigned smem_slot, unsigned cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_slot), "r"(cols) : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(unsigned taddr, unsigned cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(cols) : "memory");
}
// tcgen05.commit issued by one elected lane of a converged warp, without a branch
__device__ __forceinline__ void mma_commit_elect(unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "elect.sync _|P, 0xffffffff;\n\t"
      "@P tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar)
      : "memory");
}
// Batches of MMAs issued by the elected lane (`el` = elect_one() of a converged warp) under one
// predicate, every descriptor computed by the caller (warp-uniform values stay in the uniform
// datapath): the issuing warp then spends two instructions per MMA instead of five.
// S = Q K^T: eight K steps of 16 dims; the first overwrites, the rest accumulate.
__device__ __forceinline__ void mma_ss_batch8(unsigned el, unsigned d_tmem, const unsigned long long (&a)[8],
                                              const unsigned long long (&b)[8], unsigned idesc) {
  asm volatile(
      "{\n\t.reg .pred P, T, F;\n\t"
      "setp.ne.b32 P, %18, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.u32 F, 0, 0;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %9, %17, F;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %2, %10, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %3, %11, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %4, %12, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %5, %13, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %6, %14, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %7, %15, %17, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], %8, %16, %17, T;\n\t}"
      ::"r"(d_tmem), "l"(a[0]), "l"(a[1]), "l"(a[2]), "l"(a[3]), "l"(a[4]), "l"(a[5]), "l"(a[6]), "l"(a[7]),
        "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "l"(b[6]), "l"(b[7]), "r"(idesc), "r"(el)
      : "memory");
}
// O (+)= P V, up to four K steps of 16 keys (the key-range kernel's 64-key tiles): P read from TMEM at p + 8 k; the
// first accumulates iff acc0; only the first n_on steps are issued.
__device__ __forceinline__ void mma_ts_batch4_first(unsigned el, unsigned o_tmem, unsigned p_tmem,
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
      "@E0 tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %6, Q;\n\t"
      "@E1 tcgen05.mma.cta_group::1.kind::f16 [%0], [p1], %3, %6, T;\n\t"
      "@E2 tcgen05.mma.cta_group::1.kind::f16 [%0], [p2], %4, %6, T;\n\t"
      "@E3 tcgen05.mma.cta_group::1.kind::f16 [%0], [p3], %5, %6, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "r"(idesc), "r"(acc0), "r"(el), "r"(n_on)
      : "memory");
}
// The split of O += P V that the kernel uses: P is handed over as keys 0-95 and keys 96-127, so that only
// two K steps follow the last exponentials of a tile.  Six K steps; step k is issued iff k < n_on.
__device__ __forceinline__ void mma_ts_batch6(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                              const unsigned long long (&b)[6], unsigned idesc, unsigned acc0, int n_on) {
  asm volatile(
      "{\n\t.reg .pred P, T, Q, E0, E1, E2, E3, E4, E5;\n\t.reg .b32 p1, p2, p3, p4, p5;\n\t"
      "setp.ne.b32 P, %10, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.b32 Q, %9, 0;\n\t"
      "setp.gt.s32 E0, %11, 0;\n\t"
      "setp.gt.s32 E1, %11, 1;\n\t"
      "setp.gt.s32 E2, %11, 2;\n\t"
      "setp.gt.s32 E3, %11, 3;\n\t"
      "setp.gt.s32 E4, %11, 4;\n\t"
      "setp.gt.s32 E5, %11, 5;\n\t"
      "and.pred E0, E0, P;\n\t"
      "and.pred E1, E1, P;\n\t"
      "and.pred E2, E2, P;\n\t"
      "and.pred E3, E3, P;\n\t"
      "and.pred E4, E4, P;\n\t"
      "and.pred E5, E5, P;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "add.u32 p2, %1, 16;\n\t"
      "add.u32 p3, %1, 24;\n\t"
      "add.u32 p4, %1, 32;\n\t"
      "add.u32 p5, %1, 40;\n\t"
      "@E0 tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %8, Q;\n\t"
      "@E1 tcgen05.mma.cta_group::1.kind::f16 [%0], [p1], %3, %8, T;\n\t"
      "@E2 tcgen05.mma.cta_group::1.kind::f16 [%0], [p2], %4, %8, T;\n\t"
      "@E3 tcgen05.mma.cta_group::1.kind::f16 [%0], [p3], %5, %8, T;\n\t"
      "@E4 tcgen05.mma.cta_group::1.kind::f16 [%0], [p4], %6, %8, T;\n\t"
      "@E5 tcgen05.mma.cta_group::1.kind::f16 [%0], [p5], %7, %8, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "r"(idesc),
        "r"(acc0), "r"(el), "r"(n_on)
      : "memory");
}
// the same for a full key tile: no per-step predicates
__device__ __forceinline__ void mma_ts_batch6_full(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                                   const unsigned long long (&b)[6], unsigned idesc, unsigned acc0) {
  asm volatile(
      "{\n\t.reg .pred P, T, Q;\n\t.reg .b32 p1, p2, p3, p4, p5;\n\t"
      "setp.ne.b32 P, %10, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.ne.b32 Q, %9, 0;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "add.u32 p2, %1, 16;\n\t"
      "add.u32 p3, %1, 24;\n\t"
      "add.u32 p4, %1, 32;\n\t"
      "add.u32 p5, %1, 40;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %8, Q;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p1], %3, %8, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p2], %4, %8, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p3], %5, %8, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p4], %6, %8, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p5], %7, %8, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "l"(b[2]), "l"(b[3]), "l"(b[4]), "l"(b[5]), "r"(idesc),
        "r"(acc0), "r"(el)
      : "memory");
}
__device__ __forceinline__ void mma_ts_batch2_full(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                                   const unsigned long long (&b)[2], unsigned idesc) {
  asm volatile(
      "{\n\t.reg .pred P, T;\n\t.reg .b32 p1;\n\t"
      "setp.ne.b32 P, %5, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %4, T;\n\t"
      "@P tcgen05.mma.cta_group::1.kind::f16 [%0], [p1], %3, %4, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "r"(idesc), "r"(el)
      : "memory");
}
// The last two K steps (keys 96-111, 112-127), always accumulating; step k is issued iff k < n_on.
__device__ __forceinline__ void mma_ts_batch2(unsigned el, unsigned o_tmem, unsigned p_tmem,
                                              const unsigned long long (&b)[2], unsigned idesc, int n_on) {
  asm volatile(
      "{\n\t.reg .pred P, T, E0, E1;\n\t.reg .b32 p1;\n\t"
      "setp.ne.b32 P, %5, 0;\n\t"
      "setp.eq.u32 T, 0, 0;\n\t"
      "setp.gt.s32 E0, %6, 0;\n\t"
      "setp.gt.s32 E1, %6, 1;\n\t"
      "and.pred E0, E0, P;\n\t"
      "and.pred E1, E1, P;\n\t"
      "add.u32 p1, %1, 8;\n\t"
      "@E0 tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %4, T;\n\t"
      "@E1 tcgen05.mma.cta_group::1.kind::f16 [%0], [p1], %3, %4, T;\n\t}"
      ::"r"(o_tmem), "r"(p_tmem), "l"(b[0]), "l"(b[1]), "r"(idesc), "r"(el), "r"(n_on)
      : "memory");
}
// tcgen05.commit by the same elected lane (a commit covers the MMAs its own thread issued)
__device__ __forceinline__ void mma_commit_pred(unsigned el, unsigned bar) {
  asm volatile(
      "{\n\t.reg .pred P;\n\t"
      "setp.ne.b32 P, %1, 0;\n\t"
      "@P tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];\n\t}"
      ::"r"(bar), "r"(el)
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

// One lane of a converged warp (all 32 lanes must call this together).
__device__ __forceinline__ bool elect_one() {
  unsigned pred;
  asm volatile("{\n\t.reg .pred P;\n\telect.sync _|P, 0xffffffff;\n\tselp.u32 %0, 1, 0, P;\n\t}" : "=r"(pred));
  return pred != 0;
}
__device__ __forceinline__ float ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float max3(float a, float b, float c) {
  float d;
  asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(a), "f"(b), "f"(c));
  return d;
}
// two fp32 values in one 64-bit register, for the packed fp32 instructions
__device__ __forceinline__ unsigned long long pack2(float lo, float hi) {
  unsigned long long d;
  asm("mov.b64 %0, {%1, %2};" : "=l"(d) : "f"(lo), "f"(hi));
  return d;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long d;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
  return d;
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long d;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
  return d;
}
// 2^x for a pair of arguments on the FMA pipe (the exp unit is the scarce resource of the softmax):
// x = n + f with n = round(x), f in [-0.5, 0.5]; 2^f by a cubic (relative error 7.5e-5, far below
// the bf16 rounding of P); 2^n by adding n to the exponent field.  x is clamped at -126.
__device__ __forceinline__ void ex2_poly2(unsigned long long x2, float& p0, float& p1) {
  float x0, x1;
  unpack2(x2, x0, x1);
  x2 = pack2(fmaxf(x0, -126.f), fmaxf(x1, -126.f));
  const unsigned long long magic = pack2(12582912.f, 12582912.f);          // 1.5 * 2^23
  const unsigned long long t2 = add2(x2, magic);                            // low mantissa bits = round(x)
  const unsigned long long neg_n2 = fma2(t2, pack2(-1.f, -1.f), magic);     // -(round(x))
  const unsigned long long f2 = add2(x2, neg_n2);
  unsigned long long q2 = fma2(f2, pack2(0.055171650f, 0.055171650f), pack2(0.24261113f, 0.24261113f));
  q2 = fma2(q2, f2, pack2(0.69326097f, 0.69326097f));
  q2 = fma2(q2, f2, pack2(0.99992806f, 0.99992806f));
  float q0, q1, t0, t1;
  unpack2(q2, q0, q1);
  unpack2(t2, t0, t1);
  p0 = __int_as_float(__float_as_int(q0) + (__float_as_int(t0) << 23));
  p1 = __int_as_float(__float_as_int(q1) + (__float_as_int(t1) << 23));
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

// Geometry of one work item, derived from its record.  n0 / end0: rows of the first segment's request
// and the end of its own key tiles, kept in registers because most items have one segment and their
// per-tile arithmetic must not touch shared memory.
struct Geo {
  int valid, m, nseg, prefix_tiles, tile_begin, T, b_active, n0, end0;
};
__device__ __forceinline__ Geo read_geo(const ItemInfo* inf, int num_splits, int tiles_per_split) {
  Geo g;
  g.valid = inf->valid;
  g.m = inf->m;
  g.nseg = inf->nseg;
  g.prefix_tiles = (g.m + kTileKeys - 1) / kTileKeys;
  const int all_tiles = inf->all_tiles;
  int tb = 0, te = all_tiles;
  if (num_splits > 1) {
    tb = min(all_tiles, inf->split * tiles_per_split);
    te = min(all_tiles, tb + tiles_per_split);
  }
  g.tile_begin = tb;
  g.T = g.valid ? te - tb : 0;
  g.b_active = inf->nrows > 128;                            // the item has a second query tile
  g.n0 = inf->seg[0].n;
  g.end0 = inf->seg[0].tile_end;
  return g;
}
// The same, with every field broadcast from lane 0 of a converged warp: the compiler then knows the
// values to be warp-uniform and keeps what derives from them (loop counters, MMA descriptors) in
// the uniform datapath, which the MMA issue path needs to run at full rate.
__device__ __forceinline__ Geo read_geo_uniform(const ItemInfo* inf, int num_splits, int tiles_per_split) {
  Geo g = read_geo(inf, num_splits, tiles_per_split);
  g.valid = __shfl_sync(0xffffffffu, g.valid, 0);
  g.m = __shfl_sync(0xffffffffu, g.m, 0);
  g.nseg = __shfl_sync(0xffffffffu, g.nseg, 0);
  g.prefix_tiles = __shfl_sync(0xffffffffu, g.prefix_tiles, 0);
  g.tile_begin = __shfl_sync(0xffffffffu, g.tile_begin, 0);
  g.T = __shfl_sync(0xffffffffu, g.T, 0);
  g.b_active = __shfl_sync(0xffffffffu, g.b_active, 0);
  g.n0 = __shfl_sync(0xffffffffu, g.n0, 0);
  g.end0 = __shfl_sync(0xffffffffu, g.end0, 0);
  return g;
}
// Key tile j of the item: which keys it holds.  seg < 0: keys key0 .. of the cached prefix; else own
// rows key0 .. of segment seg's request.  Tiles of the prefix and of the first segment are resolved from
// registers; only the later segments of a shared row tile read the item record.
struct TileRef {
  int seg, key0, cnt;
};
__device__ __forceinline__ TileRef tile_ref(const ItemInfo* inf, const Geo& g, int j) {
  const int jg = g.tile_begin + j;
  TileRef r;
  if (jg < g.prefix_tiles) {
    r.seg = -1;
    r.key0 = jg * kTileKeys;
    r.cnt = min(kTileKeys, g.m - r.key0);
    return r;
  }
  if (jg < g.end0) {
    r.seg = 0;
    r.key0 = (jg - g.prefix_tiles) * kTileKeys;
    r.cnt = min(kTileKeys, g.n0 - r.key0);
    return r;
  }
  int k = 1, start = g.end0;
  while (k + 1 < g.nseg && jg >= inf->seg[k].tile_end) {
    start = inf->seg[k].tile_end;
    ++k;
  }
  r.seg = k;
  r.key0 = (jg - start) * kTileKeys;
  r.cnt = min(kTileKeys, inf->seg[k].n - r.key0);
  return r;
}
// The same for a converged warp, the result warp-uniform to the compiler as well: what comes from the
// item record is broadcast from lane 0 (see read_geo_uniform).
__device__ __forceinline__ TileRef tile_ref_uniform(const ItemInfo* inf, const Geo& g, int j) {
  const int jg = g.tile_begin + j;
  TileRef r;
  if (jg < g.end0) {
    const bool pre = jg < g.prefix_tiles;
    r.seg = pre ? -1 : 0;
    r.key0 = (pre ? jg : jg - g.prefix_tiles) * kTileKeys;
    r.cnt = min(kTileKeys, (pre ? g.m : g.n0) - r.key0);
    return r;
  }
  r = tile_ref(inf, g, j);
  r.seg = __shfl_sync(0xffffffffu, r.seg, 0);
  r.key0 = __shfl_sync(0xffffffffu, r.key0, 0);
  r.cnt = __shfl_sync(0xffffffffu, r.cnt, 0);
  return r;
}
// Keys of key tile j of an item with ONE segment, from registers only; dense: a full tile of own rows.
__device__ __forceinline__ int tile_keys_single(const Geo& g, int j, bool& dense) {
  const int jg = g.tile_begin + j;
  const bool pre = jg < g.prefix_tiles;
  const int cnt = min(kTileKeys, pre ? g.m - jg * kTileKeys : g.n0 - (jg - g.prefix_tiles) * kTileKeys);
  dense = !pre && cnt >= kTileKeys;
  return cnt;
}
// the segment that holds row p of the item, or -1
__device__ __forceinline__ int seg_of_row(const ItemInfo* inf, int nseg, int p) {
  int k = -1;
  for (int i = 0; i < nseg; ++i)
    if (p >= inf->seg[i].begin && p < inf->seg[i].begin + inf->seg[i].count) k = i;
  return k;
}


}  // namespace tc


// kShared: the schedule holds row tiles with several segments (requests of a prefix group sharing a
// tile); that instantiation takes its per-tile key counts from the K loader's notes.  The plain one keeps
// them in registers and carries none of the shared-tile code in its loops.
template <bool kShared>
__global__ void __launch_bounds__(tc::kThreads, 1)
tc_attention_kernel(ScheduleView s, PoolView pool, TensorArgs t, int* status,
                    const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
                    const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_o,
                    const __grid_constant__ CUtensorMap tm_q8, int q_tma, int o_tma, long long wait_cycles) {
  using namespace tc;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem =
      reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  Barriers* bars = reinterpret_cast<Barriers*>(smem + kTileBytes * (2 + kRing) + kStageBytes);
  volatile int* abort_flag = &bars->abort_flag;
  const unsigned q_smem = smem_u32(smem);                  // Q_A, then Q_B
  const unsigned ring_smem = q_smem + 2 * kTileBytes;
  int* const next_item = status + 16;                      // items handed out beyond the first gridDim.x
  int* const ctas_done = status + 17;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int G = t.Hq / t.Hkv;

  if (tid == 0) {
    bars->wait_cycles = wait_cycles;
    bars->dead = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    bars->abort_flag = (bars->dead || wait_cycles < kStrictBudget) ? 1 : 0;
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&bars->info_full[i]), 1);
      mbar_init(smem_u32(&bars->info_free[i]), kInfoReaders);
      mbar_init(smem_u32(&bars->q_full[i]), kLoadThreads);
      mbar_init(smem_u32(&bars->q_free[i]), 1);
      mbar_init(smem_u32(&bars->s_full[i]), 1);
      mbar_init(smem_u32(&bars->p_half[i][0]), kGroupThreads);
      mbar_init(smem_u32(&bars->p_half[i][1]), kGroupThreads);
      mbar_init(smem_u32(&bars->o_done[i]), 1);
      mbar_init(smem_u32(&bars->o_free[i]), kGroupThreads);
    }
    for (int i = 0; i < kRing; ++i) {
      mbar_init(smem_u32(&bars->full[i]), kLoadThreads);
      mbar_init(smem_u32(&bars->free_[i]), 1);
    }
    mbar_init(smem_u32(&bars->drain), 1);
    fence_barrier_init();
  }
  if (warp == kMmaWarp) {
    tmem_alloc(smem_u32(&bars->tmem_base), kTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&bars->tmem_base);
  const bool dead = *reinterpret_cast<volatile int*>(&bars->dead) != 0;   // an earlier launch or CTA gave up: do no work

  // Registers move from the MMA/load warpgroup to the two softmax warpgroups, which hold a whole
  // row of S (128 values) per thread.  The counts must fit the CTA's launch allocation:
  // 256 * kSoftmaxRegs + 128 * kOtherRegs <= 384 * (registers per thread at launch); the host
  // checks this before the first launch, because an increase that cannot be met never returns.
  if (warp < 8) {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
  } else {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
  }
  if (warp < 8) {
    // ====================== softmax / correction / epilogue of one query tile ======================
    const int X = warp >> 2;                                 // 0: tile A, 1: tile B
    const int gt = tid & 127;                                // row of the tile = TMEM lane
    const unsigned lane_base = (unsigned)((warp & 3) * 32) << 16;
    const unsigned tmem_s = tmem + X * 128 + lane_base;      // S, and P written over its first 64 columns
    const unsigned tmem_o = tmem + 256 + X * 128 + lane_base;
    const float sl2 = t.scale * 1.4426950408889634f;         // scores are handled in the log2 domain
    const unsigned long long sl2_2 = pack2(sl2, sl2);
    unsigned char* const stage = smem + kTileBytes * (2 + kRing) + warp * 4096;   // this warp's 32 rows x 128 bytes
    bool ok = !dead;
    int n_it = 0;                // items seen by this CTA
    int c_tile = 0;              // key tiles this query tile has processed (phase of s_full / p_half)
    int e_item = 0;              // items this query tile has taken part in (phase of o_done)
    int tg = 0;                  // key tiles of all items so far (index into the tile descriptions)
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_full[n_it & 1]), (n_it >> 1) & 1, abort_flag));
      if (!ok) break;
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, s.num_splits, s.tiles_per_split);
      if (!g.valid) break;
      const int T = g.T;
      const bool active = X == 0 || g.b_active;
      // The segment (request) this thread's row belongs to; -1: a padding row.  With several segments a
      // row takes part only in the own-key tiles of its own request (the prefix tiles come first, so its
      // reference maximum is finite by then); with one segment padding rows just run along.
      const int vseg = seg_of_row(inf, g.nseg, X * 128 + gt);
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int j = 0; j < T && active; ++j) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->s_full[X]), c_tile & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // Keys of the tile.  The plain kernel works them out from registers; the kernel for row tiles
        // shared by several requests reads what the K loader wrote down (two code paths side by side in
        // this loop cost more than either alone, hence two kernels).  In a shared tile a row takes part only in the own keys of its own request: for the
        // other rows the reference maximum used below is +inf, which makes every exponential exactly 0
        // (and the row's own maximum -inf, so it never asks for a rescale): no branch, no code of its
        // own in this loop.
        int cnt;
        bool mine = true;
        if (!kShared) {
          bool dense_unused;
          cnt = tile_keys_single(g, j, dense_unused);
        } else {
          const int meta = __shfl_sync(0xffffffffu, *reinterpret_cast<volatile int*>(&bars->tile_meta[(tg + j) & 7]), 0);
          cnt = meta & 255;
          const int tseg = (meta >> 16) - 1;
          mine = tseg < 0 || tseg == vseg;
        }
        // the whole row of S into registers: four loads in flight, one wait
        unsigned r[128];
        tmem_ld32(tmem_s, r);
        tmem_ld32(tmem_s + 32, r + 32);
        tmem_ld32(tmem_s + 64, r + 64);
        tmem_ld32(tmem_s + 96, r + 96);
        tmem_wait_ld();

        float alpha = 1.f;
        unsigned long long acc_a = pack2(0.f, 0.f), acc_b = pack2(0.f, 0.f);
        bool stored = false;                                   // P already stored and signalled
        // A ragged tile: columns past the last key become -inf (their exponentials are exactly 0).
        if (cnt < kTileKeys) {
#pragma unroll
          for (int i = 0; i < 128; ++i)
            if (i >= cnt) r[i] = 0xff800000u;
        }
        // The first tile of an item takes its own row maximum as the reference (a short extra pass);
        // everything else is one code path for every tile: this code runs once per key tile and
        // must stay in the instruction cache, which a separate first-tile path (11 KB of straight-
        // line code met once per item) did not.
        if (j == 0) {
          float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
          for (int i = 0; i < 128; i += 8) {
            mx0 = max3(mx0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
            mx1 = max3(mx1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
            mx2 = max3(mx2, __uint_as_float(r[i + 4]), __uint_as_float(r[i + 5]));
            mx3 = max3(mx3, __uint_as_float(r[i + 6]), __uint_as_float(r[i + 7]));
          }
          m_ref = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * sl2;   // scale > 0; finite: a tile has a key
        }
        {
          // The exponentials use the reference maximum of
          // the earlier tiles and do not wait for this tile's maximum, which is computed alongside.
          // P of the first 96 keys is handed to the tensor pipe before the last 32 exponentials are computed
          // (a 64 / 64 split left four K steps of P V behind the last exponential, 2 % slower; 112 / 16 is
          // slower again: the first part then starts too late).
          // If the row maximum turns out to exceed the reference by more than 2^8 (rare: checked per
          // warp before anything is handed over), the tile is redone below with the new reference.
          const float neg_m_eff = mine ? -m_ref : -INFINITY;
          const unsigned long long neg_m2 = pack2(neg_m_eff, neg_m_eff);
          float mx0 = -INFINITY, mx1 = -INFINITY;
          // the first 64 exponentials, with the maximum over all 128 scores computed alongside
          // (independent instructions that fill the exp unit's latency)
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
            float xa0, xa1, p2, p3;
            unpack2(xa, xa0, xa1);
            const float p0 = ex2(xa0), p1 = ex2(xa1);
            if (kPolyPeriod > 0 && i % (kPolyPeriod > 0 ? kPolyPeriod : 1) == 0) {
              ex2_poly2(xb, p2, p3);                            // this pair on the FMA pipe
            } else {
              float xb0, xb1;
              unpack2(xb, xb0, xb1);
              p2 = ex2(xb0);
              p3 = ex2(xb1);
            }
            acc_a = add2(acc_a, pack2(p0, p1));
            acc_b = add2(acc_b, pack2(p2, p3));
            r[2 * i] = pack_bf16(p0, p1);
            r[2 * i + 1] = pack_bf16(p2, p3);
          }
          const float mx = mine ? fmaxf(mx0, mx1) * sl2 : -INFINITY;   // scale > 0

          if (!__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
            // keys 64-95 join the first hand-over, so that only two K steps of P V follow the last exponentials
#pragma unroll
            for (int i = 16; i < 24; ++i) {
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
            tmem_st32(tmem_s, r);
            tmem_st16(tmem_s + 32, r + 32);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bars->p_half[X][0]));

#pragma unroll
            for (int i = 24; i < 32; ++i) {
              const unsigned long long xa =
                  fma2(pack2(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1])), sl2_2, neg_m2);
              const unsigned long long xb =
                  fma2(pack2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), sl2_2, neg_m2);
              float xa0, xa1, p2, p3;
              unpack2(xa, xa0, xa1);
              const float p0 = ex2(xa0), p1 = ex2(xa1);
              if (kPolyPeriod > 0 && i % (kPolyPeriod > 0 ? kPolyPeriod : 1) == 0) {
                ex2_poly2(xb, p2, p3);                            // this pair on the FMA pipe
              } else {
                float xb0, xb1;
                unpack2(xb, xb0, xb1);
                p2 = ex2(xb0);
                p3 = ex2(xb1);
              }
              acc_a = add2(acc_a, pack2(p0, p1));
              acc_b = add2(acc_b, pack2(p2, p3));
              r[2 * i] = pack_bf16(p0, p1);
              r[2 * i + 1] = pack_bf16(p2, p3);
            }
            tmem_st16(tmem_s + 48, r + 48);
            tmem_wait_st();
            tc_fence_before();
            mbar_arrive(smem_u32(&bars->p_half[X][1]));
            stored = true;
          } else {
            // redo with the new reference: S is still intact in TMEM
            if (mx > m_ref + 8.f) {
              alpha = ex2(m_ref - mx);
              m_ref = mx;
            }
            unsigned s4[32];
            const float neg_m = mine ? -m_ref : -INFINITY;
            float ps = 0.f;
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              tmem_ld32(tmem_s + c * 32, s4);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) {
                // (the scores come from TMEM again: columns past the last key of a ragged tile are masked here)
                const float p0 = c * 32 + 2 * i < cnt ? ex2(fmaf(__uint_as_float(s4[2 * i]), sl2, neg_m)) : 0.f;
                const float p1 = c * 32 + 2 * i + 1 < cnt ? ex2(fmaf(__uint_as_float(s4[2 * i + 1]), sl2, neg_m)) : 0.f;
                ps += p0 + p1;
                r[c * 16 + i] = pack_bf16(p0, p1);
              }
            }
            acc_a = pack2(ps, 0.f);
            acc_b = pack2(0.f, 0.f);
            // S(j) was committed after O += P V of tile j-1 was issued, so O is quiescent here.
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
          mbar_arrive(smem_u32(&bars->p_half[X][0]));
          mbar_arrive(smem_u32(&bars->p_half[X][1]));
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
        const SegInfo* sg = &inf->seg[row_valid ? vseg : 0];
        const long long row_off = sg->row_off;
        const int prow = sg->prow0 + (X * 128 + gt - sg->begin);   // packed row of this thread within its request
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
          mbar_arrive(smem_u32(&bars->o_free[X]));           // the next item may overwrite O
        } else {
#pragma unroll
          for (int i = 0; i < 128; ++i) o[i] = 0u;
        }
        const float inv = T > 0 ? 1.f / l_sum : 0.f;
        const float lse = T > 0 ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
        if (s.num_splits > 1) {
          // key-split call: normalised fp32 partial and its lse, merged by a second kernel
          if (row_valid) {
            const long long pr = ((long long)inf->split * t.total_tokens + sg->tok_off + a) * t.Hq + h;
            float* po = t.part_o + pr * 128;
#pragma unroll
            for (int i = 0; i < 128; i += 4)
              *reinterpret_cast<float4*>(po + i) =
                  make_float4(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv,
                              __uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
            t.part_lse[pr] = lse;
          }
        } else if (T > 0) {
          // Each thread holds one output row.  The warp stages its 32 rows, one 64-dim half at a
          // time (128 bytes per row, 16-byte chunks XOR-placed by row: the 128-byte swizzle), and
          // one TMA store writes the half out; a warp whose rows are not all valid, or a head
          // grouping the box cannot express, copies the staged rows out itself, four rows per
          // instruction.
          // (a warp whose 32 rows lie in one segment on whole tokens; else every row finds its own place)
          const int seg_first = __shfl_sync(0xffffffffu, vseg, 0), seg_last = __shfl_sync(0xffffffffu, vseg, 31);
          const int prow_first = __shfl_sync(0xffffffffu, prow, 0);
          const bool by_tma = o_tma && seg_first >= 0 && seg_first == seg_last && prow_first % G == 0;
          const int tok_first = (int)__shfl_sync(0xffffffffu, (int)row_off, 0) + prow_first / G;
          // byte offset of this thread's output row (one 64-dim half is added below); -1: a padding row
          const long long my_dst = row_valid ? ((row_off + a) * t.out_stride + (long long)h * 128) * 2 : -1;
#pragma unroll
          for (int hh = 0; hh < 2; ++hh) {
            if (lane == 0) bulk_wait_read();                 // the previous store has read the staging rows
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
      tg += T;
    }
    if (lane == 0) bulk_wait_all();                          // the output stores of this warp have completed
    tc_fence_before();
  } else if (warp == 9) {
    // ============================== item fetch and Q loads ===============================
    // Lane 0 writes the record of the CTA's first item (its block index) and, while item n is
    // computed, fetches item n + 1 from the shared counter.  The warp loads the Q tiles of item n
    // as soon as the last S of item n - 1 has been computed.
    bool ok = !dead;
    int n_it = 0;
    int eq[2] = {0, 0};          // items each query tile has taken part in (phase of q_free / q_full)
    // The record of item `idx` (the whole warp works on it; lane k fills segment k).
    auto write_info = [&](ItemInfo* dst, int idx) {
      if (idx < s.num_items) {
        const WorkItem wi = s.items[idx];
        if (s.tiles != nullptr) {
          const RowTile* tl = s.tiles + wi.req;
          const int nseg = tl->nseg, m = tl->m;
          const int pt = (m + kTileKeys - 1) / kTileKeys;
          SegInfo si;
          int own = 0;
          if (lane < nseg) {
            const RowSeg sg = tl->seg[lane];
            const ReqMeta rq = s.reqs[sg.req];
            si.row_off = rq.row_off;
            si.n = rq.n;
            si.prow0 = sg.prow0;
            si.begin = sg.begin;
            si.count = sg.count;
            si.tok_off = rq.tok_off;
            own = (rq.n + kTileKeys - 1) / kTileKeys;
          }
          int scan = own;                                 // inclusive prefix sum over the segments
#pragma unroll
          for (int o = 1; o < kMaxSegs; o <<= 1) {
            const int up = __shfl_up_sync(0xffffffffu, scan, o);
            if (lane >= o) scan += up;
          }
          if (lane < nseg) {
            si.tile_end = pt + scan;
            dst->seg[lane] = si;
          }
          const int all_tiles = pt + __shfl_sync(0xffffffffu, scan, nseg - 1);
          if (lane == 0) {
            dst->kv_head = wi.kv_head;
            dst->split = wi.split;
            dst->m = m;
            dst->page_off = tl->page_off;
            dst->nseg = nseg;
            dst->nrows = tl->nrows;
            dst->all_tiles = all_tiles;
            dst->valid = 1;
          }
        } else if (lane == 0) {
          const ReqMeta rq = s.reqs[wi.req];
          const int pt = (rq.m + kTileKeys - 1) / kTileKeys, own = (rq.n + kTileKeys - 1) / kTileKeys;
          SegInfo si;
          si.row_off = rq.row_off;
          si.n = rq.n;
          si.prow0 = wi.row0;
          si.begin = 0;
          si.count = min(kTileRows, rq.n * G - wi.row0);
          si.tok_off = rq.tok_off;
          si.tile_end = pt + own;
          dst->seg[0] = si;
          dst->kv_head = wi.kv_head;
          dst->split = wi.split;
          dst->m = rq.m;
          dst->page_off = rq.page_off;
          dst->nseg = 1;
          dst->nrows = si.count;
          dst->all_tiles = pt + own;
          dst->valid = 1;
        }
      } else if (lane == 0) {
        dst->valid = 0;
      }
      __syncwarp();                                       // every lane's part is written before lane 0 signals
    };
    if (ok) {
      write_info(&bars->info[0], (int)blockIdx.x);
      if (lane == 0) mbar_arrive(smem_u32(&bars->info_full[0]));
    }
    __syncwarp();
    while (ok) {
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, s.num_splits, s.tiles_per_split);
      if (!g.valid) break;
      if (g.T > 0) {
        for (int x = 0; x < 2 && ok; ++x) {
          if (x == 1 && !g.b_active) break;
          ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->q_free[x]), (eq[x] & 1) ^ 1, abort_flag));
          if (!ok) break;
          ++eq[x];
          const unsigned qf = smem_u32(&bars->q_full[x]);
          const unsigned q_dst = q_smem + x * kTileBytes;
          const SegInfo* s0 = &inf->seg[0];
          if (kShared && g.nseg > 1) {
            // Rows of several requests (only built when the heads of a KV group divide 8): 16 boxes of 8
            // packed rows per 64-dim half, one per lane, each from the request that owns its rows
            // (segments start on multiples of 8 rows); a box past the last segment is filled with zeros
            // (a coordinate outside the tensor).  Dense swizzled layout: row r at r * 128 bytes, halves
            // 16 KB apart.
            const int box = lane & 15, half = lane >> 4;
            const int k = seg_of_row(inf, g.nseg, x * 128 + box * 8);
            int tok = 0x3fffffff;
            if (k >= 0) tok = (int)inf->seg[k].row_off + (inf->seg[k].prow0 + x * 128 + box * 8 - inf->seg[k].begin) / G;
            tma_load_3d(q_dst + half * (kTileBytes / 2) + box * 1024, &tm_q8, half * 64, inf->kv_head * G, tok, qf);
            if (lane == 0) mbar_arrive_expect_tx(qf, (unsigned)kTileBytes);
            else mbar_arrive(qf);
          } else if (q_tma) {
            // 128 packed rows = 128 / G tokens x G heads of the KV group (the schedule starts such an
            // item on a whole token): one TMA box per 64-dim half, in the dense swizzled layout (row r
            // at r * 128 bytes, halves 16 KB apart)
            if (lane == 0) {
              const int tok = (int)s0->row_off + (s0->prow0 + x * 128) / G;
              mbar_arrive_expect_tx(qf, (unsigned)kTileBytes);
              tma_load_3d(q_dst, &tm_q, 0, inf->kv_head * G, tok, qf);
              tma_load_3d(q_dst + kTileBytes / 2, &tm_q, 64, inf->kv_head * G, tok, qf);
            } else {
              mbar_arrive(qf);
            }
          } else {
            // gathers into the page-image layout: packed row p = token a * G + head jj of the KV
            // group; rows past the end are zero-filled
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
              while (jj >= G) {                         // at most twice (G >= 1)
                jj -= G;
                src_row += q_row_bytes;
              }
            }
            cp_async_commit();
            cp_async_wait<0>();
            fence_proxy_async();
            mbar_arrive(qf);
          }
        }
        if (!ok) break;
      }
      // the next item: its record slot must have been released by every role (item n - 1)
      {
        const int nn = n_it + 1;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_free[nn & 1]), ((nn >> 1) & 1) ^ 1, abort_flag));
        if (ok) {
          int idx = 0;
          if (lane == 0) idx = (int)gridDim.x + atomicAdd(next_item, 1);
          idx = __shfl_sync(0xffffffffu, idx, 0);
          write_info(&bars->info[nn & 1], idx);
          if (lane == 0) mbar_arrive(smem_u32(&bars->info_full[nn & 1]));
        }
      }
      __syncwarp();
      ++n_it;
    }
    cp_async_wait<0>();
    // After a give-up, the Q loads issued last may still be in flight: wait (bounded) for them.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      for (int x = 0; x < 2; ++x)
        if (eq[x] > 0)
          for (unsigned it = 0; it < 4096 && !mbar_try_wait(smem_u32(&bars->q_full[x]), (eq[x] - 1) & 1); ++it)
            __nanosleep(256);
    }
  } else if (warp >= 10) {
    // ====================================== loads =======================================
    // Warp 10 stages the K tiles, warp 11 the V tiles, each running ahead of the MMAs by the depth
    // of the ring (K0 V0 K1 V1) and on into the next item.  Ring uses are counted over the whole
    // life of the CTA: use u = 2 * (key tiles before) + (0: K, 1: V).
    const int is_v = warp - 10;
    // A gathered 128-row tile is fetched as 64 passes of 2 rows: lane l takes 16-byte chunk (l & 15)
    // of rows (l >> 4) + 2 i.  In the tile image, rows r, r + 8, r + 16, ... are 2048 bytes apart.
    const int r0 = lane >> 4, c16 = lane & 15;
    unsigned dst_q[4];
#pragma unroll
    for (int q = 0; q < 4; ++q) dst_q[q] = tile_chunk_offset(r0 + 2 * q, c16);
    bool ok = !dead;
    int n_it = 0, U = 0;
    int armed[kRing] = {-1, -1, -1, -1};     // the last use armed with bulk copies, per slot
    while (ok) {
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->info_full[n_it & 1]), (n_it >> 1) & 1, abort_flag));
      if (!ok) break;
      const ItemInfo* inf = &bars->info[n_it & 1];
      const Geo g = read_geo_uniform(inf, s.num_splits, s.tiles_per_split);
      if (!g.valid) break;
      const int kv_head = inf->kv_head;
      const int* pages = s.pages + inf->page_off;
      for (int j = 0; j < g.T; ++j) {
        const int u = U + 2 * j + is_v;
        const int slot = u % kRing;
        const int jg = g.tile_begin + j;
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bars->free_[slot]), ((u / kRing) & 1) ^ 1, abort_flag));
        if (!ok) break;
        const unsigned dst = ring_smem + slot * kTileBytes;
        const unsigned full = smem_u32(&bars->full[slot]);
        const TileRef tr = tile_ref_uniform(inf, g, j);
        if (kShared && !is_v && lane == 0)       // before this lane's arrival on `full`, which publishes it
          bars->tile_meta[(u >> 1) & 7] = tr.cnt | ((tr.seg >= 0 && tr.cnt >= kTileKeys) ? 256 : 0) | ((tr.seg + 1) << 16);
        if (jg < g.prefix_tiles) {
          // cached prefix tile: one bulk copy per page (a pool page already is the tile image), each
          // issued by its own lane so that the page-table reads overlap
          const int cnt = min(kTileKeys, g.m - jg * kTileKeys);
          const int npages = (cnt + kPageSize - 1) / kPageSize;
          if (lane < npages) {
            const char* pool_base = is_v ? pool.v : pool.k;
            bulk_copy_g2s(dst + lane * kPageBytes,
                          pool_base + pool_slice_offset(pool, t.layer, pages[jg * 8 + lane], kv_head), kPageBytes, full);
          }
          // every lane arrives, so the phase cannot complete before lane 0 has announced the bytes
          if (lane == 0) {
            mbar_arrive_expect_tx(full, (unsigned)(npages * kPageBytes));
            armed[slot] = u;
          } else {
            mbar_arrive(full);
          }
          continue;
        }
        // own rows of one of the item's requests
        const long long row_off = inf->seg[tr.seg].row_off;
        const int key0 = tr.key0, cnt = tr.cnt;
        if (cnt >= kTileKeys) {
          // a full tile of the request's own rows: two TMA boxes (dense swizzled layout)
          if (lane == 0) {
            const int row = (int)row_off + key0;
            const void* tm = is_v ? (const void*)&tm_v : (const void*)&tm_k;
            mbar_arrive_expect_tx(full, (unsigned)kTileBytes);
            tma_load_3d(dst, tm, 0, kv_head, row, full);
            tma_load_3d(dst + kTileBytes / 2, tm, 64, kv_head, row, full);
            armed[slot] = u;
          } else {
            mbar_arrive(full);
          }
          continue;
        }
        // ragged last tile: 16-byte gathers into the page-image layout, zero-filled past the end
        const char* rowp = (is_v ? t.v : t.k) + ((row_off + key0) * t.kv_stride + (long long)kv_head * 128) * 2 + c16 * 16;
        const long long row_bytes = t.kv_stride * 2;
        const char* src = rowp + r0 * row_bytes;
#pragma unroll 4
        for (int i = 0; i < 64; ++i) {
          const bool valid = r0 + 2 * i < cnt;
          cp_async16(dst + dst_q[i & 3] + (i >> 2) * 2048, valid ? src : rowp, valid ? 16u : 0u);
          src += 2 * row_bytes;
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        mbar_arrive(full);
      }
      if (!ok) break;
      U += 2 * g.T;
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bars->info_free[n_it & 1]));
      ++n_it;
    }
    cp_async_wait<0>();
    // On the normal path every tile loaded has been consumed by the time the CTA ends (the
    // epilogue waits for the last MMA).  After a give-up, bulk copies may still be in flight:
    // wait (bounded) for the last barriers this lane armed.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      for (int i = 0; i < kRing; ++i)
        if (armed[i] >= 0)
          for (unsigned it = 0;
               it < 4096 && !mbar_try_wait(smem_u32(&bars->full[armed[i] % kRing]), (armed[i] / kRing) & 1); ++it)
            __nanosleep(256);
    }
  } else if (warp == kMmaWarp) {
    // ===================================== MMA issue =====================================
    // The whole warp runs this control flow converged and one elected lane issues each batch of
    // tcgen05 instructions.  Issue order inside an item:
    //   S_A(0) S_B(0) | O_A(0) S_A(1) | O_B(0) S_B(1) | O_A(1) S_A(2) | ...
    // O_X(j) += P_X V is issued in two parts as P arrives (six K steps, then two), and the next S_X = Q_X K^T follows it
    // back to back (it overwrites P_X; the tensor pipe runs MMAs in issue order).  After the last
    // O_X of an item the next S_X is the first one of the next item.  Alternating between the two
    // tiles keeps their softmaxes half a period apart, which the exp unit they share needs.
    // This warp shares its scheduler with two busy softmax warps and gets through its own
    // instructions slowly, so everything but the MMAs - waits for K/V tiles, descriptors, what
    // follows each O - sits in the shadow of the waits for the second part of P.
    bool ok = !dead;
    if (ok) {
      const unsigned bar_full = smem_u32(&bars->full[0]), bar_free = smem_u32(&bars->free_[0]);   // slot i: + 8 i
      const unsigned bar_p = smem_u32(&bars->p_half[0][0]);     // [x][half]: + 16 x + 8 half
      const unsigned bar_s = smem_u32(&bars->s_full[0]), bar_qfull = smem_u32(&bars->q_full[0]);   // [x]: + 8 x
      const unsigned bar_qfree = smem_u32(&bars->q_free[0]), bar_odone = smem_u32(&bars->o_done[0]);
      const unsigned bar_ofree = smem_u32(&bars->o_free[0]);
      // Two shared-memory layouts occur (see make_desc): the page image (cached tiles, gathered ragged
      // tiles, gathered Q) and the dense layout TMA writes (full own-row tiles, TMA-loaded Q): 8-row
      // groups 1024 bytes apart, the two 64-dim halves 16 KB apart.  Descriptors of ring slot 0 in
      // both layouts; slot i adds i * (tile bytes / 16) to the address field.
      const unsigned q_hi = q_tma ? 1024u : 64u;
      const unsigned long long q_desc0 = make_desc(q_smem, 16, q_tma ? 1024u : 2048u);
      const unsigned long long q_desc1 = q_desc0 + (kTileBytes >> 4);
      const unsigned long long kb_img = make_desc(ring_smem, 16, 2048), kb_dense = make_desc(ring_smem, 16, 1024);
      const unsigned long long vb_img = make_desc(ring_smem, 1024, 2048), vb_dense = make_desc(ring_smem, 16384, 1024);
      constexpr unsigned kSlotUnits = kTileBytes >> 4;
      const unsigned tmem_u = __shfl_sync(0xffffffffu, tmem, 0);   // warp-uniform copy of the TMEM base
      const unsigned tmem_s1 = tmem_u + 128, tmem_o0 = tmem_u + 256, tmem_o1 = tmem_u + 384;
#define BICACHE_WAIT(bar, parity) __all_sync(0xffffffffu, mbar_wait((bar), (parity), abort_flag))
      const unsigned el = elect_one() ? 1u : 0u;               // the lane that issues every MMA of this warp
      // the eight MMAs (K steps of 16 dims) of S_X = Q_X K^T
      auto issue_s = [&](unsigned d_tmem, unsigned long long qd, unsigned long long kd, unsigned k_hi) {
        unsigned long long a[8], b[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          a[k] = qd + (k >> 2) * q_hi + (k & 3) * 2;
          b[k] = kd + (k >> 2) * k_hi + (k & 3) * 2;
        }
        mma_ss_batch8(el, d_tmem, a, b, kIdescQK);
      };
      // one part of the eight MMAs (K steps of 16 keys) of O_X += P_X V: half 0 = keys 0-95, half 1 = keys 96-127
      auto issue_pv = [&](unsigned o_tmem, unsigned p_tmem, unsigned long long vd, unsigned v_step, int half,
                          unsigned acc0, int ksteps) {
        if (half == 0) {
          unsigned long long b[6];
#pragma unroll
          for (int k = 0; k < 6; ++k) b[k] = vd + k * v_step;
          if (ksteps == 8) mma_ts_batch6_full(el, o_tmem, p_tmem, b, kIdescPV, acc0);
          else mma_ts_batch6(el, o_tmem, p_tmem, b, kIdescPV, acc0, ksteps);
        } else {
          unsigned long long b[2];
#pragma unroll
          for (int k = 0; k < 2; ++k) b[k] = vd + (6 + k) * v_step;
          if (ksteps == 8) mma_ts_batch2_full(el, o_tmem, p_tmem + 48, b, kIdescPV);
          else mma_ts_batch2(el, o_tmem, p_tmem + 48, b, kIdescPV, ksteps - 6);
        }
      };
      int n_it = 0;
      int c0 = 0, c1 = 0;        // key tiles each query tile has been through (phase of p_half)
      int e0 = 0, e1 = 0;        // items each query tile has taken part in (phase of q_full / o_free)
      unsigned u = 0;            // ring use of the current key tile's K; its V is u + 1, the next tile's K u + 2
      ok = BICACHE_WAIT(smem_u32(&bars->info_full[0]), 0);
      Geo cur = read_geo_uniform(&bars->info[0], s.num_splits, s.tiles_per_split);
      // keys | dense << 8 of the key tile whose K has ring use uu, as the K loader described it (valid once
      // that slot's `full` barrier has been waited for); warp-uniform like the geometry
      auto read_meta = [&](unsigned uu) -> int {
        return __shfl_sync(0xffffffffu, *reinterpret_cast<volatile int*>(&bars->tile_meta[(uu >> 1) & 7]), 0);
      };
      bool dn = false;           // layout of the current key tile
      int ksteps = 8;            // its keys, in steps of 16
      bool pre = false;          // the first S of the current item was issued at the end of the previous one
      while (ok && cur.valid) {
        Geo nxt;
        nxt.valid = 0;
        bool have_next = false, can_pre = false;
        const int T = cur.T;
        if (T > 0) {
          const bool b_on = cur.b_active;
          if (!pre) {
            // the first S of an item that could not be issued ahead (the CTA's first item)
            ok = BICACHE_WAIT(bar_full + (u & 3) * 8, (u >> 2) & 1) && BICACHE_WAIT(bar_qfull, e0 & 1);
            if (!ok) break;
            tc_fence_after();
            if (!kShared) {
              ksteps = (tile_keys_single(cur, 0, dn) + 15) >> 4;
            } else {
              const int meta = read_meta(u);
              dn = (meta & 256) != 0;
              ksteps = ((meta & 255) + 15) >> 4;
            }
            const unsigned long long kd0 = (dn ? kb_dense : kb_img) + (u & 3) * kSlotUnits;
            issue_s(tmem_u, q_desc0, kd0, dn ? 1024u : 64u);
            mma_commit_pred(el, bar_s);
            if (T == 1) mma_commit_pred(el, bar_qfree);
            if (b_on) {
              // Stagger the two query tiles: tile B starts when tile A's softmax has handed over its
              // first part of P (started together, the two softmaxes share the exp unit and the MMAs of
              // both tiles then queue behind each other).
              ok = BICACHE_WAIT(bar_p, c0 & 1) && BICACHE_WAIT(bar_qfull + 8, e1 & 1);
              if (!ok) break;
              issue_s(tmem_s1, q_desc1, kd0, dn ? 1024u : 64u);
              mma_commit_pred(el, bar_s + 8);
              if (T == 1) mma_commit_pred(el, bar_qfree + 8);
            }
            mma_commit_pred(el, bar_free + (u & 3) * 8);
          }
          // V of the first key tile; the previous item's epilogue must have read O_A out of TMEM
          ok = BICACHE_WAIT(bar_full + ((u + 1) & 3) * 8, ((u + 1) >> 2) & 1) && BICACHE_WAIT(bar_ofree, (e0 & 1) ^ 1);
          if (!ok) break;
          // One key tile.  The body exists twice: the lean one for every tile but the last, and the
          // one for the last tile, which also looks at the next item.
          auto tile_iter = [&](auto last_c, int j) {
            constexpr bool last = decltype(last_c)::value;
            const unsigned sv = (u + 1) & 3, sn = (u + 2) & 3;  // ring slots: V of this tile, K of the next
            const unsigned long long v_desc = (dn ? vb_dense : vb_img) + sv * kSlotUnits;
            const unsigned v_step = dn ? 128u : 256u;           // 16 keys further, in 16-byte units
            const unsigned acc0 = j > 0 ? 1u : 0u;
            // ---- tile A: first part of O += P V as soon as P of keys 0-95 is there ----
            ok = BICACHE_WAIT(bar_p, c0 & 1);
            if (!ok) return;
            tc_fence_after();
                        issue_pv(tmem_o0, tmem_u, v_desc, v_step, 0, acc0, ksteps);
            // ---- shadow of A's last exponentials: what follows the O of this iteration ----
            bool s_on0 = true, s_on1 = b_on;                   // an S follows O_A / O_B
            bool q_last = j + 2 == T;                           // ... and it is the last S of its item
            bool dn_next = false;
            int ks_next = 8;
            if (!last) {
              if (!kShared) ks_next = (tile_keys_single(cur, j + 1, dn_next) + 15) >> 4;
            } else {
              // the next item (fetched long ago): its first S follows this item's last O
              const int nn = n_it + 1;
              ok = BICACHE_WAIT(smem_u32(&bars->info_full[nn & 1]), (nn >> 1) & 1);
              if (!ok) return;
              nxt = read_geo_uniform(&bars->info[nn & 1], s.num_splits, s.tiles_per_split);
              have_next = true;
              can_pre = nxt.valid && nxt.T > 0;
              s_on0 = can_pre;
              s_on1 = can_pre && nxt.b_active;
              q_last = nxt.T == 1;
              if (!kShared && can_pre) ks_next = (tile_keys_single(nxt, 0, dn_next) + 15) >> 4;
            }
            if (s_on0) {
              ok = BICACHE_WAIT(bar_full + sn * 8, ((u + 2) >> 2) & 1);
              if (!ok) return;
              if (kShared) {
                const int meta = read_meta(u + 2);
                dn_next = (meta & 256) != 0;
                ks_next = ((meta & 255) + 15) >> 4;
              }
            }
            const unsigned long long k_desc = (dn_next ? kb_dense : kb_img) + sn * kSlotUnits;
            const unsigned k_hi = dn_next ? 1024u : 64u;
            // ---- tile A: second part, then the next S_A back to back ----
            ok = BICACHE_WAIT(bar_p + 8, c0 & 1);
            if (!ok) return;
            tc_fence_after();
                        issue_pv(tmem_o0, tmem_u, v_desc, v_step, 1, acc0, ksteps);
            ++c0;
            if (last) {
              mma_commit_pred(el, bar_odone);
              ++e0;
            }
            if (s_on0) {
              if (last) {
                ok = BICACHE_WAIT(bar_qfull, e0 & 1);           // the next item's Q tile must have landed
                if (!ok) return;
              }
              issue_s(tmem_u, q_desc0, k_desc, k_hi);
              mma_commit_pred(el, bar_s);
              if (q_last) mma_commit_pred(el, bar_qfree);
            }
            // ---- tile B: first part ----
            if (b_on) {
              if (j == 0) {
                ok = BICACHE_WAIT(bar_ofree + 8, (e1 & 1) ^ 1);  // the previous epilogue has read O_B
                if (!ok) return;
              }
              ok = BICACHE_WAIT(bar_p + 16, c1 & 1);
              if (!ok) return;
              tc_fence_after();
                            issue_pv(tmem_o1, tmem_s1, v_desc, v_step, 0, acc0, ksteps);
            }
            // ---- tile B: second part, then the next S_B ----
            if (b_on) {
              ok = BICACHE_WAIT(bar_p + 24, c1 & 1);
              if (!ok) return;
              tc_fence_after();
                            issue_pv(tmem_o1, tmem_s1, v_desc, v_step, 1, acc0, ksteps);
              ++c1;
              if (last) {
                mma_commit_pred(el, bar_odone + 8);
                ++e1;
              }
            }
            if (s_on1) {
              if (last) {
                ok = BICACHE_WAIT(bar_qfull + 8, e1 & 1);
                if (!ok) return;
              }
              issue_s(tmem_s1, q_desc1, k_desc, k_hi);
              mma_commit_pred(el, bar_s + 8);
              if (q_last) mma_commit_pred(el, bar_qfree + 8);
            }
            // release V of this tile and K of the next
            mma_commit_pred(el, bar_free + sv * 8);
            if (s_on0) mma_commit_pred(el, bar_free + sn * 8);
            u += 2;
            dn = dn_next;
            ksteps = ks_next;
            // V of the next key tile (its slot was released one iteration ago: it lands about now)
            if (!last) {
              ok = BICACHE_WAIT(bar_full + ((u + 1) & 3) * 8, ((u + 1) >> 2) & 1);
              if (!ok) return;
            }
          };
          for (int j = 0; j + 1 < T && ok; ++j) tile_iter(std::false_type{}, j);
          if (ok) tile_iter(std::true_type{}, T - 1);
          if (!ok) break;
        }
        // done with this item's record; move on
        if (!have_next) {
          const int nn = n_it + 1;
          ok = BICACHE_WAIT(smem_u32(&bars->info_full[nn & 1]), (nn >> 1) & 1);
          if (!ok) break;
          nxt = read_geo_uniform(&bars->info[nn & 1], s.num_splits, s.tiles_per_split);
        }
        if (elect_one()) mbar_arrive(smem_u32(&bars->info_free[n_it & 1]));
        __syncwarp();
        pre = can_pre;
        cur = nxt;
        ++n_it;
      }
#undef BICACHE_WAIT
      // Whatever happened, let every MMA issued so far finish before TMEM is released.
      __syncwarp();
      mma_commit_elect(smem_u32(&bars->drain));               // elect.sync names the same lane as `el`
      mbar_wait_issued(smem_u32(&bars->drain), 0);
    }
    __syncwarp();
  }

  __syncthreads();
  if (warp == kMmaWarp) {
    tc_fence_after();
    tmem_dealloc(tmem, kTmemCols);
  }
  if (tid == 0) {
    if (!dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
    // the last CTA to finish rewinds the item counter for the next launch
    __threadfence();
    if (atomicAdd(ctas_done, 1) == (int)gridDim.x - 1) {
      *next_item = 0;
      *ctas_done = 0;
      __threadfence();
    }
  }
}

inline cudaError_t configure_tc_attention() {
  cudaFuncAttributes attr;
  for (int shared = 0; shared < 2; ++shared) {
    const void* fn = shared ? (const void*)tc_attention_kernel<true> : (const void*)tc_attention_kernel<false>;
    cudaError_t e = cudaFuncGetAttributes(&attr, fn);
    if (e != cudaSuccess) return e;
    // the register pool the kernel redistributes is the launch allocation of the CTA
    if (attr.numRegs * tc::kThreads < 2 * tc::kGroupThreads * tc::kSoftmaxRegs + 128 * tc::kOtherRegs)
      return cudaErrorLaunchOutOfResources;
    e = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, tc::kSmemBytes);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

// Tensor maps of one call: q [rows][Hq][128] with a box of (64 dims, G heads, 128 / G rows) so that
// a box is 128 packed rows; k, v [rows][Hkv][128] with a box of (64 dims, 1 head, 128 rows); out like
// q with a box of 32 packed rows (the rows of one softmax warp).
struct TcTensorMaps {
  CUtensorMap q, k, v, o;
  CUtensorMap q8;            // q again with a box of 8 packed rows (row tiles made of several segments)
  int q8_tma;                // 0: G does not divide 8
  int q_tma;                 // 0: G does not divide 128, Q is gathered instead
  int o_tma;                 // 0: G does not divide 32, the output rows are copied out by the warps
};

// `status` points at the context's status area: word 0 is the sticky device status, words 16 and 17
// are the item counter and the count of finished CTAs (both zero between launches).
inline cudaError_t launch_tc_attention(const ScheduleView& s, const PoolView& pool, const TensorArgs& t,
                                       int* status, int num_sms, const TcTensorMaps& maps, long long wait_cycles,
                                       cudaStream_t stream) {
  const int grid = s.num_items < num_sms ? s.num_items : num_sms;
  if (s.tiles != nullptr && s.shared_tiles)
    tc_attention_kernel<true><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(
        s, pool, t, status, maps.q, maps.k, maps.v, maps.o, maps.q8, maps.q_tma, maps.o_tma,
        wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  else
    tc_attention_kernel<false><<<grid, tc::kThreads, tc::kSmemBytes, stream>>>(
        s, pool, t, status, maps.q, maps.k, maps.v, maps.o, maps.q8, maps.q_tma, maps.o_tma,
        wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  return cudaGetLastError();
}

}  // namespace bicache
