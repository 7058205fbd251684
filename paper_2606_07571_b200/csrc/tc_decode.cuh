// Few query rows against many keys (block-query decoding shapes): the bandwidth-bound form of
// Eq. 2 / Eq. 4.  One CTA computes, for up to 128 packed query rows of one KV head and one RANGE of
// keys, the normalised partial result and its log-sum-exp; a merge kernel combines the ranges
// (the identity behind the log-sum-exp merge: softmax over a union of key sets).  The query rows of
// ALL requests of a prefix group share tiles (token t of the group is row tok_rows[t] of q), so the
// cached prefix is read once per group, not once per request.  The requests' own keys ride along
// with the first range: after its prefix tiles that CTA runs over the own rows of the requests in its
// row tile, every query row masked to the keys of its own request (a block-diagonal mask: Eq. 2
// per request).
//
// Why a second kernel: with one 128-row tile per CTA the big kernel's chain S -> softmax -> P V
// runs once per 128 keys with nothing to overlap it, and one CTA per SM cannot keep HBM busy.
// Here a CTA is small (112 KB of shared memory, 256 TMEM columns: two CTAs per SM), key tiles are
// 64 keys, and S is double-buffered in TMEM: S(j+1) = Q K(j+1)^T is issued before the softmax of
// tile j ends.  Roles: warps 0-3 softmax (one thread per row; they also gather the Q tile before
// their first key tile), warp 4 MMA issue and TMEM, warp 5 stages K tiles, warp 6 stages V tiles
// (cached pages: one 4 KB bulk copy per page, a pool page already is the operand image; own rows:
// 16-byte gathers into the same image).  Every wait is bounded, as in the big kernel.
#pragma once

#include "tc_attention.cuh"

namespace bicache {
namespace dec {

using namespace tc;

constexpr int kKeys = 64;                          // keys per tile
constexpr int kKvTileBytes = kKeys * 128 * 2;      // 16 KB
constexpr int kQBytes = 128 * 128 * 2;             // 32 KB
constexpr int kKStages = 3;                        // K tiles are consumed one tile early (S is double-buffered)
constexpr int kVStages = 2;
constexpr int kDecThreads = 224;
constexpr int kDecTmemCols = 256;                  // S0 0-63, S1 64-127 (P over the first 32 of each), O 128-255
// fp32 accumulate, bf16 A and B (both K-major), M = 128, N = 64
constexpr unsigned kIdescS64 = (1u << 4) | (1u << 7) | (1u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);

struct DecodeItem {
  int n;                 // tokens in the row space: all requests of a prefix group, concatenated
  int tok_off;           // index of the row space's first token among the call's tokens
  int kv_head;
  int row0;              // first packed row of the item (multiple of 128)
  int key_begin;         // first cached prefix key of the range (multiple of 64)
  int key_count;         // cached keys in the range (0: none)
  int page_off;          // index of the prefix's first page id in the schedule's page list
  int slot;              // which partial this range is
  int own_begin;         // range 0 only: the own keys it also covers are tokens tok_off + own_begin ..
  int own_count;         // .. + own_count - 1 of the call (the requests that have rows in this row tile)
};

struct DecSync {
  unsigned long long q_full;
  unsigned long long k_full[kKStages], k_free[kKStages];
  unsigned long long v_full[kVStages], v_free[kVStages];
  unsigned long long s_full[2];          // S of a key tile is in TMEM
  unsigned long long p_full[2];          // P of the tile is in TMEM (and O rescaled if it had to be)
  unsigned long long pv_done;            // O += P V of a tile has completed (one phase per tile)
  unsigned long long o_done;             // O += P V of the LAST tile has completed
  unsigned long long drain;
  long long wait_cycles;                 // directly before abort_flag (mbar_wait reads it)
  int abort_flag;
  unsigned tmem_base;
  int dead;
};
constexpr int kDecSmemBytes = kQBytes + (kKStages + kVStages) * kKvTileBytes + (int)sizeof(DecSync);
static_assert(2 * (kDecSmemBytes + 1024) <= 233472, "two CTAs per SM");
static_assert(128 * 528 <= (kKStages + kVStages) * kKvTileBytes, "the partial rows are staged over the K/V rings");


}  // namespace dec

__global__ void __launch_bounds__(dec::kDecThreads, 2)
tc_decode_kernel(const dec::DecodeItem* __restrict__ items, const long long* __restrict__ tok_rows,
                 const int2* __restrict__ tok_span, const int* __restrict__ pages, PoolView pool, TensorArgs t,
                 int* status, long long wait_cycles) {
  using namespace dec;
  // No room for alignment slack with two CTAs per SM: the kernel has no static shared memory, the
  // dynamic window starts 1024-byte aligned (the swizzled tiles need that), and a CTA that finds
  // otherwise reports an error instead of computing.
  extern __shared__ __align__(1024) unsigned char smem_raw[];
  unsigned char* const smem = smem_raw;
  DecSync* sy = reinterpret_cast<DecSync*>(smem + kQBytes + (kKStages + kVStages) * kKvTileBytes);
  volatile int* abort_flag = &sy->abort_flag;
  const unsigned q_smem = smem_u32(smem);
  const unsigned k_ring = q_smem + kQBytes, v_ring = k_ring + kKStages * kKvTileBytes;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // the merge kernel that follows may be placed on the SMs from now on (it waits for this grid's end)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  const DecodeItem it = items[blockIdx.x];
  const int G = t.Hq / t.Hkv;
  // key tiles: the cached range first, then (range 0) the own keys
  const int T_pre = (it.key_count + kKeys - 1) / kKeys;
  const int T = T_pre + (it.own_count + kKeys - 1) / kKeys;
  auto tile_cnt = [&](int j) {
    return j < T_pre ? min(kKeys, it.key_count - j * kKeys) : min(kKeys, it.own_count - (j - T_pre) * kKeys);
  };

  if (tid == 0) {
    sy->wait_cycles = wait_cycles;
    if ((q_smem & 1023u) != 0) atomicCAS(status, kDevOk, kDevInternal);
    sy->dead = (*reinterpret_cast<volatile int*>(status) != 0) ? 1 : 0;
    sy->abort_flag = (sy->dead || wait_cycles < kStrictBudget) ? 1 : 0;
    mbar_init(smem_u32(&sy->q_full), 128);
    for (int i = 0; i < kKStages; ++i) {
      mbar_init(smem_u32(&sy->k_full[i]), 32);
      mbar_init(smem_u32(&sy->k_free[i]), 1);
    }
    for (int i = 0; i < kVStages; ++i) {
      mbar_init(smem_u32(&sy->v_full[i]), 32);
      mbar_init(smem_u32(&sy->v_free[i]), 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(smem_u32(&sy->s_full[i]), 1);
      mbar_init(smem_u32(&sy->p_full[i]), 128);
    }
    mbar_init(smem_u32(&sy->pv_done), 1);
    mbar_init(smem_u32(&sy->o_done), 1);
    mbar_init(smem_u32(&sy->drain), 1);
    fence_barrier_init();
  }
  if (warp == 4) {
    tmem_alloc(smem_u32(&sy->tmem_base), kDecTmemCols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const unsigned tmem = *reinterpret_cast<volatile unsigned*>(&sy->tmem_base);
  const bool dead = *reinterpret_cast<volatile int*>(&sy->dead) != 0;
  const unsigned tmem_o = tmem + 128;

  if (warp < 4) {
    // ================================ softmax and epilogue =================================
    const int row = warp * 32 + lane;                        // row of the tile = TMEM lane
    const unsigned lane_base = (unsigned)(warp * 32) << 16;
    const float sl2 = t.scale * 1.4426950408889634f;         // scores are handled in the log2 domain
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = !dead;
    // the call's tokens that are this row's own keys (its request); none for a row past the end
    int2 span = make_int2(0, 0);
    if (T > T_pre && it.row0 + row < it.n * G) span = tok_span[it.tok_off + (it.row0 + row) / G];
    if (ok && T > 0) {
      // The Q tile, gathered by the 128 threads that have nothing else to do yet: warp w fetches rows
      // 32 w .. 32 w + 31, lane l the 16-byte chunk (l & 15) of rows 32 w + (l >> 4) + 2 i.  Packed row
      // p = token a * G + head jj of the KV group; rows past the end are zero-filled.
      const int r0 = warp * 32 + (lane >> 4), c16 = lane & 15;
      const int packed_rows = it.n * G;
      const char* const q_head = t.q + ((long long)it.kv_head * G * 128) * 2 + c16 * 16;
      int prow = it.row0 + r0;
      int a = prow / G, jj = prow - a * G;
#pragma unroll 4
      for (int i = 0; i < 16; ++i) {
        const bool valid = prow < packed_rows;
        const char* src = q_head;
        if (valid) src = q_head + (tok_rows[it.tok_off + a] * t.q_stride + jj * 128) * 2;
        cp_async16(q_smem + tile_chunk_offset(r0 + 2 * i, c16), src, valid ? 16u : 0u);
        prow += 2;
        jj += 2;
        while (jj >= G) {                           // at most twice (G >= 1)
          jj -= G;
          ++a;
        }
      }
      cp_async_commit();
      cp_async_wait<0>();
      fence_proxy_async();
      mbar_arrive(smem_u32(&sy->q_full));
    }
    for (int j = 0; j < T && ok; ++j) {
      const int b = j & 1;
      const int cnt = tile_cnt(j);
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->s_full[b]), (j >> 1) & 1, abort_flag));
      if (!ok) break;
      tc_fence_after();
      unsigned r[64];
      tmem_ld32(tmem + b * 64 + lane_base, r);
      tmem_ld32(tmem + b * 64 + 32 + lane_base, r + 32);
      tmem_wait_ld();
      if (j >= T_pre) {
        // own keys: column i is token tok_off + own_begin + 64 (j - T_pre) + i of the call; a row
        // sees the tokens of its own request only (every row has seen a cached tile before, so its
        // reference maximum is finite even if this whole tile is masked for it)
        const int tok0 = it.tok_off + it.own_begin + (j - T_pre) * kKeys;
        const int lo = span.x - tok0, hi = span.y - tok0;
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i < lo || i >= hi) r[i] = 0xff800000u;
      } else if (cnt < kKeys) {
#pragma unroll
        for (int i = 0; i < 64; ++i)
          if (i >= cnt) r[i] = 0xff800000u;                  // -inf: columns past the last key
      }
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int i = 0; i < 64; i += 4) {
        mx0 = max3(mx0, __uint_as_float(r[i]), __uint_as_float(r[i + 1]));
        mx1 = max3(mx1, __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
      }
      const float mx = fmaxf(mx0, mx1) * sl2;                // scale > 0
      if (j == 0) {
        m_ref = mx;
      } else if (__any_sync(0xffffffffu, mx > m_ref + 8.f)) {
        // Rare: a row's maximum exceeds the reference by more than 2^8.  O must be rescaled, and
        // S of this tile was issued before O += P V of the previous one: wait for that first.
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->pv_done), (j - 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        float alpha = 1.f;
        if (mx > m_ref + 8.f) {
          alpha = ex2(m_ref - mx);
          m_ref = mx;
        }
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          unsigned o[32];
          tmem_ld32(tmem_o + c * 32 + lane_base, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
          tmem_st32(tmem_o + c * 32 + lane_base, o);
        }
        tmem_wait_st();
        l_sum *= alpha;
      }
      const unsigned long long sl2_2 = pack2(sl2, sl2), neg_m2 = pack2(-m_ref, -m_ref);
      unsigned long long acc_a = pack2(0.f, 0.f), acc_b = pack2(0.f, 0.f);
#pragma unroll
      for (int i = 0; i < 16; ++i) {
        const unsigned long long xa =
            fma2(pack2(__uint_as_float(r[4 * i]), __uint_as_float(r[4 * i + 1])), sl2_2, neg_m2);
        const unsigned long long xb =
            fma2(pack2(__uint_as_float(r[4 * i + 2]), __uint_as_float(r[4 * i + 3])), sl2_2, neg_m2);
        float x0, x1, x2, x3;
        unpack2(xa, x0, x1);
        unpack2(xb, x2, x3);
        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
        acc_a = add2(acc_a, pack2(p0, p1));
        acc_b = add2(acc_b, pack2(p2, p3));
        r[2 * i] = pack_bf16(p0, p1);
        r[2 * i + 1] = pack_bf16(p2, p3);
      }
      tmem_st32(tmem + b * 64 + lane_base, r);               // P over the first 32 columns of this S
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(smem_u32(&sy->p_full[b]));
      float s0, s1, s2, s3;
      unpack2(acc_a, s0, s1);
      unpack2(acc_b, s2, s3);
      l_sum += (s0 + s1) + (s2 + s3);
    }
    // -------- epilogue: the normalised partial of this key range and its log-sum-exp --------
    if (ok) {
      const int p = it.row0 + row;                           // packed row of the row space
      const bool row_valid = p < it.n * G;
      const int a = p / G;
      const int h = it.kv_head * G + (p - a * G);
      const long long pr = ((long long)it.slot * t.total_tokens + it.tok_off + a) * t.Hq + h;
      if (T > 0) {
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->o_done), 0, abort_flag));
        if (ok) {
          tc_fence_after();
          // Each thread holds one row of the partial (128 fp32 = 512 bytes, contiguous in the
          // workspace).  Written from registers, a warp's stores would touch 32 rows at a time; so
          // the row goes to shared memory first (the K/V rings are free by now: every tile has been
          // consumed; rows 528 bytes apart keep the 16-byte stores conflict-free) and leaves as one
          // 512-byte bulk copy per row.
          const float inv = 1.f / l_sum;
          unsigned char* const stage_row = smem + kQBytes + row * 528;
#pragma unroll 1
          for (int c = 0; c < 4; ++c) {
            unsigned o[32];
            tmem_ld32(tmem_o + c * 32 + lane_base, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; i += 4)
              *reinterpret_cast<float4*>(stage_row + (c * 32 + i) * 4) =
                  make_float4(__uint_as_float(o[i]) * inv, __uint_as_float(o[i + 1]) * inv,
                              __uint_as_float(o[i + 2]) * inv, __uint_as_float(o[i + 3]) * inv);
          }
          fence_proxy_async();
          if (row_valid) {
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], 512;"
                         ::"l"(t.part_o + pr * 128), "r"(smem_u32(stage_row)) : "memory");
            bulk_commit_group();
            t.part_lse[pr] = (m_ref + log2f(l_sum)) * 0.6931471805599453f;
            bulk_wait_all();
          }
        }
      } else if (row_valid) {
        float* po = t.part_o + pr * 128;
#pragma unroll 4
        for (int i = 0; i < 128; i += 4) *reinterpret_cast<float4*>(po + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        t.part_lse[pr] = -INFINITY;
      }
    }
    tc_fence_before();
  } else if (warp == 4) {
    // ====================================== MMA issue ======================================
    bool ok = !dead && T > 0;
    if (ok) {
      const unsigned long long q_desc = make_desc(q_smem, 16, 2048);
      const unsigned el = elect_one() ? 1u : 0u;               // the lane that issues every MMA of this warp
      // a K step of 16 dims: 32 bytes inside the swizzled row; dims 64.. sit 1024 bytes further
      auto kstep = [](int k) { return (unsigned long long)((k & 3) * 2 + (k >> 2) * 64); };
      auto issue_s = [&](int j) {
        const int b = j & 1, ks = j % kKStages;
        bool good = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->k_full[ks]), (j / kKStages) & 1, abort_flag));
        if (!good) return false;
        tc_fence_after();
        const unsigned long long k_desc = make_desc(k_ring + ks * kKvTileBytes, 16, 2048);
        unsigned long long qa[8], kb[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          qa[k] = q_desc + kstep(k);
          kb[k] = k_desc + kstep(k);
        }
        mma_ss_batch8(el, tmem + b * 64, qa, kb, kIdescS64);   // one predicated group instead of eight elections
        mma_commit_pred(el, smem_u32(&sy->s_full[b]));
        mma_commit_pred(el, smem_u32(&sy->k_free[ks]));
        return true;
      };
      ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->q_full), 0, abort_flag));
      if (ok) ok = issue_s(0);
      for (int j = 0; j < T && ok; ++j) {
        const int b = j & 1;
        if (j + 1 < T) {
          ok = issue_s(j + 1);
          if (!ok) break;
        }
        ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->p_full[b]), (j >> 1) & 1, abort_flag));
        if (ok) ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&sy->v_full[b]), (j >> 1) & 1, abort_flag));
        if (!ok) break;
        tc_fence_after();
        // V is the MN-major operand: 64-dim halves 1024 bytes apart, 8-key groups 2048 bytes; a K
        // step of 16 keys is one page image (4096 bytes).  Steps past the last key are skipped.
        const unsigned long long v_desc = make_desc(v_ring + b * kKvTileBytes, 1024, 2048);
        const int cnt = tile_cnt(j);
        const int ksteps = (cnt + 15) >> 4;
        const unsigned long long vb[4] = {v_desc, v_desc + 256ull, v_desc + 512ull, v_desc + 768ull};
        mma_ts_batch4_first(el, tmem_o, tmem + b * 64, vb, kIdescPV, j > 0 ? 1u : 0u, ksteps);
        mma_commit_pred(el, smem_u32(&sy->v_free[b]));
        mma_commit_pred(el, smem_u32(&sy->pv_done));
        if (j == T - 1) mma_commit_pred(el, smem_u32(&sy->o_done));
      }
      // Whatever happened, let every MMA issued so far finish before TMEM is released.
      __syncwarp();
      mma_commit_elect(smem_u32(&sy->drain));
      mbar_wait_issued(smem_u32(&sy->drain), 0);
    }
    __syncwarp();
  } else {
    // ======================================= loads ========================================
    // Warp 5 stages the K tiles, warp 6 the V tiles.
    const int is_v = warp - 5;
    const int r0 = lane >> 4, c16 = lane & 15;
    bool ok = !dead;
    const int stages = is_v ? kVStages : kKStages;
    int armed[kKStages] = {-1, -1, -1};      // the last tile armed with bulk copies, per stage
    const unsigned ring = is_v ? v_ring : k_ring;
    for (int j = 0; j < T && ok; ++j) {
      const int b = j % stages;
      const unsigned free_bar = smem_u32(is_v ? &sy->v_free[b] : &sy->k_free[b]);
      const unsigned full = smem_u32(is_v ? &sy->v_full[b] : &sy->k_full[b]);
      ok = __all_sync(0xffffffffu, mbar_wait(free_bar, ((j / stages) & 1) ^ 1, abort_flag));
      if (!ok) break;
      const unsigned dst = ring + b * kKvTileBytes;
      const int key0 = it.key_begin + j * kKeys;
      const int cnt = tile_cnt(j);
      if (j < T_pre) {
        // cached prefix: one bulk copy per page (a pool page already is the tile image), each issued
        // by its own lane so that the page-table reads overlap
        const int npages = (cnt + kPageSize - 1) / kPageSize;
        if (lane < npages) {
          const char* pool_base = is_v ? pool.v : pool.k;
          bulk_copy_g2s(dst + lane * kPageBytes,
                        pool_base + pool_slice_offset(pool, t.layer, pages[it.page_off + key0 / kPageSize + lane],
                                                      it.kv_head),
                        kPageBytes, full);
        }
        // every lane arrives, so the phase cannot complete before lane 0 has announced the bytes
        if (lane == 0) {
          mbar_arrive_expect_tx(full, (unsigned)(npages * kPageBytes));
          armed[b] = j;
        } else {
          mbar_arrive(full);
        }
      } else {
        // own keys: 16-byte gathers into the page-image layout, zero-filled past the end; key r of the
        // tile is token tok0 + r of the call, row tok_rows[tok0 + r] of k / v
        const int tok0 = it.tok_off + it.own_begin + (j - T_pre) * kKeys;
        const char* const base = (is_v ? t.v : t.k) + ((long long)it.kv_head * 128) * 2 + c16 * 16;
#pragma unroll 4
        for (int i = 0; i < kKeys / 2; ++i) {
          const int r = r0 + 2 * i;
          const bool valid = r < cnt;
          const char* src = base;
          if (valid) src = base + tok_rows[tok0 + r] * t.kv_stride * 2;
          cp_async16(dst + tile_chunk_offset(r, c16), src, valid ? 16u : 0u);
        }
        cp_async_commit();
        cp_async_wait<0>();
        fence_proxy_async();
        mbar_arrive(full);
      }
    }
    cp_async_wait<0>();
    // After a give-up, bulk copies may still be in flight: wait (bounded) for the barriers armed last.
    if (!dead && (!ok || *abort_flag) && lane == 0) {
      for (int b = 0; b < stages; ++b)
        if (armed[b] >= 0) {
          const unsigned full = smem_u32(is_v ? &sy->v_full[b] : &sy->k_full[b]);
          for (unsigned n = 0; n < 4096 && !mbar_try_wait(full, (armed[b] / stages) & 1); ++n) __nanosleep(256);
        }
    }
  }

  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, kDecTmemCols);
  }
  if (tid == 0 && !dead && *abort_flag) atomicCAS(status, kDevOk, kDevTimeout);
}

// ---------------------------------------------------------------------------------------------
// Merge of the key ranges (the log-sum-exp merge): for every (token, query head) of the call,
//   lse = log sum_s exp(lse_s),  o = sum_s exp(lse_s - lse) o_s
// over the num_slots partials, written as the bf16 output row.  One warp per (token, head), one
// float4 of the 128 dims per lane; the rows of eight ranges are loaded before any is used.
// Launched as a programmatic dependent of the key-range kernel: the grid is placed while that
// kernel still runs and waits here for its memory to be visible.
// ---------------------------------------------------------------------------------------------
constexpr int kMergeWarps = 8;

// kSlotWarps = 1: one warp per (token, head), eight per block.  kSlotWarps = 8: the eight warps of a
// block share one (token, head), warp w taking ranges w, w + 8, ...; for many ranges and few rows.
template <int kSlotWarps>
__global__ void __launch_bounds__(kMergeWarps * 32)
merge_ranges_kernel(const float* __restrict__ part_o, const float* __restrict__ part_lse,
                    const long long* __restrict__ tok_rows, int total_tokens, int Hq, int num_slots,
                    char* __restrict__ out, long long out_stride, float* __restrict__ lse_out) {
  __shared__ float4 red[kSlotWarps == 1 ? 1 : kMergeWarps][32];
  asm volatile("griddepcontrol.wait;" ::: "memory");
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long pr = kSlotWarps == 1 ? (long long)blockIdx.x * kMergeWarps + warp : (long long)blockIdx.x;   // token * Hq + head
  if (pr >= (long long)total_tokens * Hq) return;
  const int tg = (int)(pr / Hq), h = (int)(pr - (long long)tg * Hq);
  const long long slot_stride = (long long)total_tokens * Hq;
  // Up to 16 ranges (the common case): every range's row is requested before anything else, so that the
  // row loads, the lse loads and the row-table load are one round trip instead of three.
  const bool few = kSlotWarps == 1 && num_slots <= 16;
  float4 pre[16];
  if (few) {
#pragma unroll
    for (int u = 0; u < 16; ++u)
      pre[u] = *reinterpret_cast<const float4*>(part_o + (pr + min(u, num_slots - 1) * slot_stride) * 128 + lane * 4);
  }
  const long long row = tok_rows[tg];
  const float l0 = lane < num_slots ? part_lse[pr + lane * slot_stride] : -INFINITY;
  const float l1 = lane + 32 < num_slots ? part_lse[pr + (lane + 32) * slot_stride] : -INFINITY;
  const float mx = warp_max(fmaxf(l0, l1));
  const bool any = mx > -INFINITY;
  float w0 = any ? expf(l0 - mx) : 0.f, w1 = any ? expf(l1 - mx) : 0.f;
  const float tot = warp_sum(w0 + w1);
  const float inv = any ? 1.f / tot : 0.f;
  w0 *= inv;
  w1 *= inv;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  // this warp's ranges: first, first + kSlotWarps, ...; eight of them are loaded before any is used
  const int first = kSlotWarps == 1 ? 0 : warp;
  if (few) {
#pragma unroll
    for (int u = 0; u < 16; ++u) {
      const float w = u < num_slots ? __shfl_sync(0xffffffffu, w0, u) : 0.f;
      acc.x = fmaf(w, pre[u].x, acc.x);
      acc.y = fmaf(w, pre[u].y, acc.y);
      acc.z = fmaf(w, pre[u].z, acc.z);
      acc.w = fmaf(w, pre[u].w, acc.w);
    }
  }
  for (int s0 = few ? num_slots : first; s0 < num_slots; s0 += 8 * kSlotWarps) {
    float4 v[8];
    float w[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int want = s0 + u * kSlotWarps;
      const int sl = min(want, num_slots - 1);               // a clamped repeat gets weight 0
      const float ws = __shfl_sync(0xffffffffu, sl < 32 ? w0 : w1, sl & 31);
      w[u] = want < num_slots ? ws : 0.f;
      v[u] = *reinterpret_cast<const float4*>(part_o + (pr + sl * slot_stride) * 128 + lane * 4);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      acc.x = fmaf(w[u], v[u].x, acc.x);
      acc.y = fmaf(w[u], v[u].y, acc.y);
      acc.z = fmaf(w[u], v[u].z, acc.z);
      acc.w = fmaf(w[u], v[u].w, acc.w);
    }
  }
  if (kSlotWarps > 1) {
    red[warp][lane] = acc;
    __syncthreads();
    if (warp != 0) return;
#pragma unroll
    for (int w = 1; w < kMergeWarps; ++w) {
      const float4 o = red[w][lane];
      acc.x += o.x;
      acc.y += o.y;
      acc.z += o.z;
      acc.w += o.w;
    }
  }
  uint2 o2;
  o2.x = tc::pack_bf16(acc.x, acc.y);
  o2.y = tc::pack_bf16(acc.z, acc.w);
  *reinterpret_cast<uint2*>(out + (row * out_stride + (long long)h * 128) * 2 + lane * 8) = o2;
  if (lane == 0 && lse_out != nullptr) lse_out[row * Hq + h] = any ? mx + logf(tot) : -INFINITY;
}

inline cudaError_t launch_merge_ranges(const TensorArgs& t, const long long* tok_rows, int num_slots,
                                       cudaStream_t stream) {
  const long long row_heads = (long long)t.total_tokens * t.Hq;
  if (row_heads <= 0) return cudaSuccess;
  const bool slot_warps = num_slots > 16;                   // many ranges: spread them over the block's warps
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)(slot_warps ? row_heads : (row_heads + kMergeWarps - 1) / kMergeWarps), 1, 1);
  cfg.blockDim = dim3(kMergeWarps * 32, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (slot_warps)
    return cudaLaunchKernelEx(&cfg, merge_ranges_kernel<8>, (const float*)t.part_o, (const float*)t.part_lse, tok_rows,
                              t.total_tokens, t.Hq, num_slots, t.out, t.out_stride, t.lse);
  return cudaLaunchKernelEx(&cfg, merge_ranges_kernel<1>, (const float*)t.part_o, (const float*)t.part_lse, tok_rows,
                            t.total_tokens, t.Hq, num_slots, t.out, t.out_stride, t.lse);
}

inline cudaError_t configure_tc_decode() {
  return cudaFuncSetAttribute(tc_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, dec::kDecSmemBytes);
}

inline cudaError_t launch_tc_decode(const dec::DecodeItem* items, int num_items, const long long* tok_rows,
                                    const int2* tok_span, const int* pages, const PoolView& pool,
                                    const TensorArgs& t, int* status, long long wait_cycles, cudaStream_t stream) {
  if (num_items <= 0) return cudaSuccess;
  tc_decode_kernel<<<num_items, dec::kDecThreads, dec::kDecSmemBytes, stream>>>(
      items, tok_rows, tok_span, pages, pool, t, status, wait_cycles > 0 ? wait_cycles : tc::kWaitCycles);
  return cudaGetLastError();
}

}  // namespace bicache
