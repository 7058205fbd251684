// Host runtime and C ABI of the BiCache attention library (see include/bicache.h).
//
// Host side: the prefix KV store's bookkeeping (key map, FIFO eviction, free-page queue), the
// reuse-depth rule, and the per-call schedule (which 128-row work items exist, which keys they
// cover), cached across the layers of a denoising step.  Device side: kernels in the .cuh files.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <deque>
#include <list>
#include <new>
#include <string>
#include <unordered_map>
#include <vector>

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/bicache.h"
#include "common.cuh"
#include "simt_kernels.cuh"
#include "tc_attention.cuh"
#include "project_kv.cuh"
#include "tc_attention_pair.cuh"
#include "tc_decode.cuh"

using namespace bicache;

namespace {

constexpr bool kTiledAttend = true;           // row tiles shared by the requests of a prefix group
constexpr int kMaxCached = 192;              // cached schedules a context keeps track of
constexpr int kStageBufs = 4;                // pinned staging buffers of the schedule uploads
constexpr size_t kStatusBytes = 256;
constexpr int kTargetCtas = 296;             // two waves of 148 SMs: aim of the key split
constexpr long long kMaxPartialRowHeads = (long long)kTargetCtas * kTileRows;

size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// A stored prefix owns ceil(m / 16) pages in each of the layers first_layer .. L-1 (a shared prefix in all
// of them; a request's kept deep-layer prefix, Eq. 5, from its shallow depth on).  Every layer has its own
// free queue; as long as all prefixes own all layers the queues move in lockstep and a prefix has ONE
// page list (`uniform`); otherwise `layer_pages[l - first_layer]` is the list of layer l.
struct PrefixEntry {
  uint64_t key;
  int32_t id;
  int32_t m;
  int32_t first_layer = 0;
  bool uniform = true;
  std::vector<int32_t> pages;                         // the list of layer first_layer
  std::vector<std::vector<int32_t>> layer_pages;      // only if !uniform
};
inline const std::vector<int32_t>& pages_of(const PrefixEntry& e, int layer) {
  return e.uniform ? e.pages : e.layer_pages[layer - e.first_layer];
}

// A schedule kept on the device: where it lives in the schedule arena and what batch it describes.
struct CachedSchedule {
  bool valid = false;
  uint64_t last_use = 0;                      // API-call counter of the last use (entries of the running call are pinned)
  uint64_t hash = 0;                          // of (kind, R, row_off, seqlen, prefix_id)
  int kind = 0;                               // 0 attend, 1 attend_full, 2 attend through the key-range kernel
  std::vector<int32_t> prefix_id;
  std::vector<int64_t> row_off;
  std::vector<int32_t> seqlen;
  int num_items = 0, num_splits = 1, tiles_per_split = 0, total_tokens = 0;
  size_t off = 0, bytes = 0;                  // place in the arena
  size_t reqs_off = 0, pages_off = 0, items_off = 0;   // byte offsets inside the schedule
  size_t ditems_off = 0;                      // kind 2: the key-range items
  size_t tok_rows_off = 0;                    // kind 2: row of every token of the call
  size_t tok_span_off = 0;                    // kind 2: the tokens of every token's own request
  int num_ditems = 0;
  int num_tiles = 0;                          // tiled schedules: row tiles behind the items (at ditems_off)
  bool shared_tiles = false;                  // ... and some tile holds rows of several requests
};
constexpr int kMaxDecodeItems = 4096;
constexpr int kMaxDecodeTokens = 4096;        // tokens of a call served by the key-range kernel

}  // namespace

struct bicache_ctx {
  bicache_config cfg;
  int esize = 2;
  bool swizzled = false;
  bool tensor_ok = false;
  int last_kernel = 0;                                            // which attention kernel the last call launched
  int attn_pairs = 0;                                             // CTA pairs of the attention kernel on pairs the device runs at once
  int proj_pairs = 0;                                             // CTA pairs of the projection kernel the device runs at once
  bool host_only = false;                                         // cfg.device < 0: bookkeeping only
  int path = BICACHE_PATH_AUTO;
  std::vector<std::deque<int32_t>> free_pages;                   // one queue per layer
  std::vector<int32_t> layer_cap;                                 // pages of each layer's pool
  std::vector<long long> layer_off;                               // byte offset of each layer inside a pool
  bool uniform_caps = true;                                       // every layer holds cfg.num_pages pages
  std::list<PrefixEntry> fifo;                                    // insertion order, oldest first
  std::unordered_map<uint64_t, std::list<PrefixEntry>::iterator> by_key;
  std::unordered_map<int32_t, std::list<PrefixEntry>::iterator> by_id;
  int32_t next_id = 0;
  std::vector<int32_t> depth_table;
  // workspace carving
  int* d_status = nullptr;
  long long wait_cycles = 0;       // SM-clock budget of the device-side waits (0: the kernel's default)
  // Schedule arena (the part of the workspace behind the fixed areas): schedules are placed one after
  // the other and the place wraps around, evicting what it overwrites.
  char* d_arena = nullptr;
  size_t arena_bytes = 0, arena_head = 0;
  // Pinned staging for the uploads, so that a schedule miss never makes the host wait for the stream.
  char* h_stage[kStageBufs] = {nullptr, nullptr, nullptr, nullptr};
  cudaEvent_t stage_ev[kStageBufs] = {nullptr, nullptr, nullptr, nullptr};
  bool stage_used[kStageBufs] = {false, false, false, false};
  size_t stage_bytes = 0;
  int stage_next = 0;
  int64_t schedule_uploads = 0;
  float* d_part_o = nullptr;
  float* d_part_lse = nullptr;
  long long part_capacity_rowheads = 0;
  int* d_put_pages = nullptr;                                     // page list staging for put_prefix
  std::vector<CachedSchedule> sched;                              // kMaxCached entries
  uint64_t use_counter = 0;                                       // one tick per API call
  int64_t launches = 0;
  int sm_count = 148;
  std::string last_error;
};

namespace {

int fail(const bicache_ctx* ctx, int code, const std::string& msg) {
  if (ctx) const_cast<bicache_ctx*>(ctx)->last_error = msg;
  return code;
}

bool supported(const bicache_config* c, int* esize, bool* swz, bool* tensor_ok) {
  if (c->dtype != BICACHE_F32 && c->dtype != BICACHE_BF16) return false;
  if (c->page_size != kPageSize) return false;
  if (c->head_dim < 32 || c->head_dim > kSimtMaxD || c->head_dim % 32) return false;
  *esize = c->dtype == BICACHE_F32 ? 4 : 2;
  *swz = c->dtype == BICACHE_BF16 && c->head_dim == 128;
  *tensor_ok = *swz && kTensorPathBuilt;
  return true;
}

bool sane(const bicache_config* c) {
  return c && c->num_layers >= 1 && c->num_kv_heads >= 1 && c->num_q_heads >= c->num_kv_heads &&
         c->num_q_heads % c->num_kv_heads == 0 && c->num_pages >= 1 && c->head_dim >= 1;
}

// Upper bound of the bytes of one schedule of at most max_req requests and max_rows rows.
size_t schedule_bytes_for(const bicache_config* c, int64_t max_rows, int32_t max_req) {
  const int G = c->num_q_heads / c->num_kv_heads;
  const long long tiles = (max_rows * G + kTileRows - 1) / kTileRows + max_req;
  const long long max_items = std::max<long long>(tiles * c->num_kv_heads, 1) + 2LL * kTargetCtas;
  return align_up((size_t)max_req * sizeof(ReqMeta) + 16, 256) +
         align_up((size_t)c->num_pages * sizeof(int) + 16, 256) +
         align_up((size_t)max_items * sizeof(WorkItem) + 16, 256) +
         std::max(align_up((size_t)kMaxDecodeItems * sizeof(dec::DecodeItem) + 16, 256),
                  align_up((size_t)tiles * sizeof(RowTile) + 16, 256)) +
         align_up((size_t)kMaxDecodeTokens * sizeof(long long) + 16, 256) +
         align_up((size_t)kMaxDecodeTokens * sizeof(int2) + 16, 256);
}

// How many schedules of the largest size the arena is asked to hold: a denoising step alternates
// between at most two schedules per distinct depth value (the reuse set and the recompute set change
// membership only there), and a set's schedule is smaller than the bound above, so this holds a step.
int arena_schedules_for(const bicache_config* c) { return std::min(2 * c->num_layers + 4, 72); }

size_t partial_bytes_for(const bicache_config* c) {
  return align_up((size_t)kMaxPartialRowHeads * (c->head_dim + 1) * sizeof(float), 256);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// The whole pools (layer stride = a full layer: only meaningful when every layer has the same capacity).
PoolView pool_view(const bicache_ctx* ctx) {
  PoolView p;
  p.k = static_cast<const char*>(ctx->cfg.k_pool);
  p.v = static_cast<const char*>(ctx->cfg.v_pool);
  p.page_bytes = kPageSize * ctx->cfg.head_dim * ctx->esize;
  p.num_kv_heads = ctx->cfg.num_kv_heads;
  p.layer_bytes = (long long)ctx->cfg.num_pages * ctx->cfg.num_kv_heads * p.page_bytes;
  p.swizzled = ctx->swizzled ? 1 : 0;
  return p;
}
// One layer of the pools, addressed as layer 0 of the view.
PoolView pool_view_layer(const bicache_ctx* ctx, int layer) {
  PoolView p = pool_view(ctx);
  p.k += ctx->layer_off[layer];
  p.v += ctx->layer_off[layer];
  return p;
}

// cuTensorMapEncodeTiled, fetched through the runtime so that the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeTiledFn encode_tiled_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 tensor [rows][heads][128] with `row_stride` elements between rows; box = (64 dims, box_heads,
// box_rows), 128-byte swizzle, zero fill outside.
bool encode_map(CUtensorMap* m, const void* base, long long rows, int heads, long long row_stride, int box_heads,
                int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, (cuuint64_t)heads, (cuuint64_t)rows};
  const cuuint64_t strides[2] = {256, (cuuint64_t)row_stride * 2};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

uint64_t fnv1a(uint64_t h, const void* data, size_t bytes) {
  const unsigned char* p = static_cast<const unsigned char*>(data);
  for (size_t i = 0; i < bytes; ++i) h = (h ^ p[i]) * 0x100000001b3ull;
  return h;
}

// A pinned staging buffer of at least `bytes` bytes whose previous upload has completed.
char* staging_buffer(bicache_ctx* ctx, size_t bytes, int* index) {
  if (bytes > ctx->stage_bytes) {
    // grow: rare (the first batches of a context); every upload in flight must finish first
    for (int i = 0; i < kStageBufs; ++i) {
      if (ctx->stage_used[i]) cudaEventSynchronize(ctx->stage_ev[i]);
      ctx->stage_used[i] = false;
      if (ctx->h_stage[i]) cudaFreeHost(ctx->h_stage[i]);
      ctx->h_stage[i] = nullptr;
    }
    const size_t want = align_up(bytes + bytes / 2, 4096);
    for (int i = 0; i < kStageBufs; ++i)
      if (cudaHostAlloc(reinterpret_cast<void**>(&ctx->h_stage[i]), want, cudaHostAllocDefault) != cudaSuccess) {
        ctx->h_stage[i] = nullptr;
        ctx->stage_bytes = 0;
        return nullptr;
      }
    ctx->stage_bytes = want;
  }
  const int i = ctx->stage_next;
  ctx->stage_next = (i + 1) % kStageBufs;
  if (ctx->stage_used[i]) cudaEventSynchronize(ctx->stage_ev[i]);   // kStageBufs uploads ago: long done
  *index = i;
  return ctx->h_stage[i];
}

// Room for `bytes` in the schedule arena: schedules follow one another and the place wraps around;
// what the new schedule would overwrite is dropped from the cache, except schedules of the running API
// call (they are about to be launched), which are stepped over.  Returns the offset or (size_t)-1.
size_t arena_place(bicache_ctx* ctx, size_t bytes) {
  bytes = align_up(bytes, 256);
  if (bytes > ctx->arena_bytes) return (size_t)-1;
  size_t head = ctx->arena_head;
  for (int attempt = 0; attempt < 8; ++attempt) {
    if (head + bytes > ctx->arena_bytes) head = 0;
    bool moved = false;
    for (CachedSchedule& c : ctx->sched) {
      if (!c.valid || c.off >= head + bytes || c.off + c.bytes <= head) continue;
      if (c.last_use == ctx->use_counter) {               // pinned: try behind it
        head = c.off + c.bytes;
        moved = true;
        break;
      }
      c.valid = false;
    }
    if (!moved) {
      ctx->arena_head = head + bytes;
      return head;
    }
  }
  return (size_t)-1;
}

// Build (or find) the device-resident schedule for this batch.  Returns its index in ctx->sched or -1.
// `tiled`: kind 0 on the tensor path - the query rows of a prefix group are packed into row tiles.
// `pairs`: kind 1 for the kernel on CTA pairs - items of 512 packed rows, the keys never split.
int prepare_schedule(bicache_ctx* ctx, int kind, bool tiled, bool pairs, int layer, int R, const int32_t* prefix_id,
                     const int64_t* row_off, const int32_t* seqlen, cudaStream_t stream, int* status) {
  *status = BICACHE_OK;
  // A schedule holds the page lists of its prefixes.  They are the same in every layer unless some
  // prefix has per-layer lists; only then is the schedule tied to the layer it was built for.
  int layer_tag = 0;
  if (kind != 1)
    for (int i = 0; i < R; ++i)
      if (prefix_id[i] >= 0 && (i == 0 || prefix_id[i] != prefix_id[i - 1]) && !ctx->by_id.at(prefix_id[i])->uniform)
        layer_tag = layer + 1;
  const int key_kind = kind + (tiled ? 8 : 0) + (pairs ? 16 : 0) + 32 * layer_tag;
  uint64_t hash = fnv1a(0xcbf29ce484222325ull, &key_kind, sizeof(key_kind));
  hash = fnv1a(hash, &R, sizeof(R));
  hash = fnv1a(hash, row_off, sizeof(int64_t) * R);
  hash = fnv1a(hash, seqlen, sizeof(int32_t) * R);
  if (kind != 1) hash = fnv1a(hash, prefix_id, sizeof(int32_t) * R);
  for (size_t s = 0; s < ctx->sched.size(); ++s) {
    CachedSchedule& c = ctx->sched[s];
    if (!c.valid || c.hash != hash || c.kind != key_kind || (int)c.seqlen.size() != R) continue;
    if (std::memcmp(c.row_off.data(), row_off, sizeof(int64_t) * R) != 0) continue;
    if (std::memcmp(c.seqlen.data(), seqlen, sizeof(int32_t) * R) != 0) continue;
    if (kind != 1 && std::memcmp(c.prefix_id.data(), prefix_id, sizeof(int32_t) * R) != 0) continue;
    c.last_use = ctx->use_counter;
    return (int)s;
  }
  const int Hkv = ctx->cfg.num_kv_heads, G = ctx->cfg.num_q_heads / Hkv;
  std::vector<ReqMeta> reqs(R);
  std::vector<int> pages;
  long long tok = 0;
  int max_key_tiles = 0;
  long long unsplit_items = 0;
  int last_pid = -1, last_page_off = 0;
  for (int i = 0; i < R; ++i) {
    ReqMeta& r = reqs[i];
    r.row_off = row_off[i];
    r.n = seqlen[i];
    r.m = 0;
    r.page_off = 0;
    r.tok_off = (int)tok;
    tok += seqlen[i];
    if (kind != 1 && prefix_id[i] >= 0) {
      const PrefixEntry& e = *ctx->by_id.at(prefix_id[i]);
      r.m = e.m;
      if (prefix_id[i] != last_pid) {
        last_pid = prefix_id[i];
        last_page_off = (int)pages.size();
        const std::vector<int32_t>& pl = pages_of(e, layer);
        pages.insert(pages.end(), pl.begin(), pl.end());
      }
      r.page_off = last_page_off;
    }
    if (r.n > 0) {
      max_key_tiles = std::max(max_key_tiles, (r.m + kTileKeys - 1) / kTileKeys + (r.n + kTileKeys - 1) / kTileKeys);
      unsplit_items += (long long)((r.n * (long long)G + kTileRows - 1) / kTileRows) * Hkv;
    }
  }
  // Split the keys across CTAs when the batch has too few row tiles to fill the GPU.  The number of
  // splits minimises a simple cost model: waves of CTAs (one CTA per SM) times the time of one CTA
  // (a fixed prologue/epilogue plus a per-key-tile cost), plus the merge pass over the partials.
  int num_splits = 1, tiles_per_split = 0;
  if (kind != 2 && !pairs && unsplit_items > 0 && unsplit_items < 2LL * ctx->sm_count && max_key_tiles >= 8) {
    const int key_tiles = max_key_tiles;
    const double c_tile = 3300.0, c_cta = 12000.0;         // SM clocks, fitted on the small-suffix shapes
    auto cost = [&](int nsplit, int tps) {
      const long long ctas = unsplit_items * nsplit;
      const double waves = (double)((ctas + ctx->sm_count - 1) / ctx->sm_count);
      double c = waves * (c_cta + c_tile * tps);
      if (nsplit > 1) c += 6000.0 + (double)tok * ctx->cfg.num_q_heads * nsplit * 516.0 / 3300.0;
      return c;
    };
    double best = cost(1, key_tiles);
    for (int want = 2; want <= std::min(64, key_tiles / 2); ++want) {
      if (tok * ctx->cfg.num_q_heads * want > ctx->part_capacity_rowheads) break;
      const int tps = (key_tiles + want - 1) / want;
      const int ns = (key_tiles + tps - 1) / tps;
      const double c = cost(ns, tps);
      if (ns > 1 && c < best) {
        best = c;
        num_splits = ns;
        tiles_per_split = tps;
      }
    }
  }
  std::vector<WorkItem> items;
  std::vector<RowTile> tiles;
  std::vector<dec::DecodeItem> ditems;
  if (kind == 2) {
    // Key-range kernel (few query rows against long cached prefixes).  Row space: all requests of a
    // prefix group, their tokens concatenated.  Ranges 0 .. sp-1 split the prefix keys; the CTAs of
    // range 0 also cover the own keys of the requests that have rows in their row tile.
    struct Group { int first, last; int n, tok_off; };
    std::vector<Group> groups;
    for (int i = 0; i < R; ++i) {
      if (groups.empty() || prefix_id[i] != prefix_id[groups.back().first])
        groups.push_back(Group{i, i, 0, reqs[i].tok_off});
      Group& g = groups.back();
      g.last = i;
      g.n += seqlen[i];
    }
    long long base_items = 0;
    int tiles64_max = 1;
    for (const Group& g : groups) {
      if (g.n <= 0) continue;
      base_items += (long long)((g.n * (long long)G + 127) / 128) * Hkv;
      tiles64_max = std::max(tiles64_max, (reqs[g.first].m + 63) / 64);
    }
    // ranges per prefix: what fills the two CTA slots of every SM once, at least 4 key tiles each
    int sp = (int)std::max<long long>(1, 2LL * ctx->sm_count / std::max<long long>(1, base_items));
    sp = std::min(sp, std::max(1, tiles64_max / 4));
    sp = std::min(sp, 64);
    while (sp > 1 && tok * ctx->cfg.num_q_heads * sp > ctx->part_capacity_rowheads) --sp;
    if (tok * ctx->cfg.num_q_heads * sp > ctx->part_capacity_rowheads) {
      *status = fail(ctx, BICACHE_ERR_NOMEM, "the partial results of this batch do not fit the workspace");
      return -1;                                          // the caller falls back to the general kernel
    }
    for (const Group& g : groups) {
      if (g.n <= 0) continue;
      const ReqMeta& r0m = reqs[g.first];
      const int ktiles = (r0m.m + 63) / 64, tps = (ktiles + sp - 1) / sp;
      for (int s = 0; s < sp; ++s) {
        const int kb = s * tps * 64;
        const int kc = std::max(0, std::min(r0m.m - kb, tps * 64));
        for (int hk = 0; hk < Hkv; ++hk)
          for (int r0 = 0; r0 < g.n * G; r0 += 128) {
            int own_begin = 0, own_count = 0;
            if (s == 0) {
              // the requests that own tokens r0 / G .. (last row of the tile) / G of the group
              const int a_first = r0 / G, a_last = (std::min(r0 + 128, g.n * G) - 1) / G;
              int lo = -1, hi = -1;
              for (int i = g.first; i <= g.last; ++i) {
                const int b0 = reqs[i].tok_off - g.tok_off, b1 = b0 + reqs[i].n;
                if (reqs[i].n <= 0 || b1 <= a_first || b0 > a_last) continue;
                if (lo < 0) lo = b0;
                hi = b1;
              }
              own_begin = lo;
              own_count = hi - lo;
            }
            ditems.push_back(dec::DecodeItem{g.n, g.tok_off, hk, r0, kc > 0 ? kb : 0, kc, r0m.page_off, s, own_begin,
                                             own_count});
          }
      }
    }
    // long ranges first
    std::stable_sort(ditems.begin(), ditems.end(), [](const dec::DecodeItem& a, const dec::DecodeItem& b) {
      return a.key_count + a.own_count > b.key_count + b.own_count;
    });
    num_splits = sp;                                       // what the merge kernel combines
    tiles_per_split = 0;
  }
  if (tiled && num_splits == 1) {
    // Row tiles of up to 256 packed rows.  The requests of a prefix group (consecutive requests with the
    // same cached prefix) share tiles: a tile is a list of segments, each a run of one request's packed
    // rows, so that a staged prefix tile serves the rows of several requests and ragged suffixes do
    // not leave tile rows empty.  Segments start on multiples of 8 rows (what the 8-row TMA boxes of the
    // Q tile need), which is why requests share tiles only when the query heads of a KV group divide 8;
    // a request without a cached prefix gets tiles of its own.
    const bool pack = 8 % G == 0;                          // else every request keeps tiles of its own
    const int seg_align = 8;
    std::vector<int> tile_cost;                            // key tiles of every row tile
    RowTile cur = RowTile{};
    int fill = 0, cur_cost = 0;
    auto flush = [&]() {
      if (cur.nseg > 0) {
        cur.nrows = cur.seg[cur.nseg - 1].begin + cur.seg[cur.nseg - 1].count;
        tiles.push_back(cur);
        tile_cost.push_back(cur_cost);
      }
      cur = RowTile{};
      fill = 0;
      cur_cost = 0;
    };
    for (int i = 0; i < R; ++i) {
      if (reqs[i].n <= 0) continue;
      const bool joins = pack && cur.nseg > 0 && reqs[i].m > 0 && prefix_id[i] == prefix_id[cur.seg[0].req];
      if (!joins) flush();
      int prow = 0, left = reqs[i].n * G;
      while (left > 0) {
        if (cur.nseg == kMaxSegs || fill >= kTileRows) flush();
        if (cur.nseg == 0) {
          cur.m = reqs[i].m;
          cur.page_off = reqs[i].page_off;
          cur_cost = (reqs[i].m + kTileKeys - 1) / kTileKeys;
        }
        const int take = std::min(left, kTileRows - fill);
        cur.seg[cur.nseg++] = RowSeg{i, prow, fill, take};
        cur_cost += (reqs[i].n + kTileKeys - 1) / kTileKeys;
        fill = (int)align_up((size_t)(fill + take), (size_t)seg_align);
        prow += take;
        left -= take;
      }
    }
    flush();
    // Items in the order (run of tiles with one prefix, KV head, tile): CTAs that run side by side then
    // read the same cached K/V tiles and share them in L2.  Then longest key range first (in steps of
    // four key tiles, so that neighbours mostly stay neighbours): the tail of the launch is made of
    // short items.
    items.reserve(tiles.size() * Hkv);
    for (size_t t0 = 0; t0 < tiles.size();) {
      size_t t1 = t0 + 1;
      while (t1 < tiles.size() && tiles[t1].m > 0 && tiles[t1].page_off == tiles[t0].page_off && tiles[t1].m == tiles[t0].m)
        ++t1;
      for (int hk = 0; hk < Hkv; ++hk)
        for (size_t tI = t0; tI < t1; ++tI) items.push_back(WorkItem{(int)tI, hk, 0, 0});
      t0 = t1;
    }
    std::stable_sort(items.begin(), items.end(), [&](const WorkItem& a, const WorkItem& b) {
      return tile_cost[a.req] / 4 > tile_cost[b.req] / 4;
    });
  } else {
    tiled = false;
    const int item_rows = pairs ? 2 * kTileRows : kTileRows;
    items.reserve((size_t)unsplit_items * num_splits);
    for (int sp = 0; sp < (kind == 2 ? 1 : num_splits); ++sp) {
      const size_t first = items.size();
      for (int i = 0; i < R; ++i) {
        if (reqs[i].n <= 0) continue;
        const int prow = reqs[i].n * G;
        for (int hk = 0; hk < Hkv; ++hk)
          for (int r0 = 0; r0 < prow; r0 += item_rows) items.push_back(WorkItem{i, hk, r0, sp});
      }
      // Longest key range first (the tail of the launch is then made of short items); items of one
      // KV head and request stay adjacent so that concurrently running CTAs share K/V tiles in L2.
      std::stable_sort(items.begin() + first, items.end(), [&](const WorkItem& a, const WorkItem& b) {
        const int ka = reqs[a.req].m + reqs[a.req].n, kb = reqs[b.req].m + reqs[b.req].n;
        return ka > kb;
      });
    }
  }
  const size_t reqs_off = 0;
  const size_t pages_off = align_up(reqs_off + reqs.size() * sizeof(ReqMeta) + 16, 256);
  const size_t items_off = align_up(pages_off + pages.size() * sizeof(int) + 16, 256);
  // the key-range items (kind 2) or the row tiles (tiled schedules) follow the items
  const size_t ditems_off = align_up(items_off + items.size() * sizeof(WorkItem) + 16, 256);
  std::vector<long long> tok_rows;
  std::vector<int2> tok_span;                              // per token: the call's tokens of its own request
  if (kind == 2) {
    tok_rows.reserve((size_t)tok);
    tok_span.reserve((size_t)tok);
    for (int i = 0; i < R; ++i)
      for (int a = 0; a < reqs[i].n; ++a) {
        tok_rows.push_back(reqs[i].row_off + a);
        tok_span.push_back(make_int2(reqs[i].tok_off, reqs[i].tok_off + reqs[i].n));
      }
  }
  const size_t second_bytes = kind == 2 ? ditems.size() * sizeof(dec::DecodeItem) : tiles.size() * sizeof(RowTile);
  const size_t tok_rows_off = align_up(ditems_off + second_bytes + 16, 256);
  const size_t tok_span_off = align_up(tok_rows_off + tok_rows.size() * sizeof(long long) + 16, 256);
  const size_t total = tok_span_off + tok_span.size() * sizeof(int2);
  if ((int)ditems.size() > kMaxDecodeItems || (long long)tok_rows.size() > kMaxDecodeTokens) {
    *status = fail(ctx, BICACHE_ERR_NOMEM, "batch too large for the key-range kernel's tables");
    return -1;
  }
  int victim = -1;
  for (size_t s = 0; s < ctx->sched.size(); ++s)
    if (!ctx->sched[s].valid) { victim = (int)s; break; }
  if (victim < 0) {                                        // every entry in use: drop the least recently used
    victim = 0;
    for (size_t s = 0; s < ctx->sched.size(); ++s)
      if (ctx->sched[s].last_use < ctx->sched[victim].last_use) victim = (int)s;
    if (ctx->sched[victim].last_use == ctx->use_counter) {
      *status = fail(ctx, BICACHE_ERR_NOMEM, "workspace too small for this batch's schedule");
      return -1;
    }
    ctx->sched[victim].valid = false;
  }
  const size_t place = arena_place(ctx, total);
  if (place == (size_t)-1) {
    *status = fail(ctx, BICACHE_ERR_NOMEM, "workspace too small for this batch's schedule");
    return -1;
  }
  CachedSchedule& c = ctx->sched[victim];
  c.valid = false;
  if (total > 0) {
    int sb = 0;
    char* blob = staging_buffer(ctx, total, &sb);
    if (!blob) {
      *status = fail(ctx, BICACHE_ERR_NOMEM, "no pinned host memory for the schedule upload");
      return -1;
    }
    if (!reqs.empty()) std::memcpy(blob + reqs_off, reqs.data(), reqs.size() * sizeof(ReqMeta));
    if (!pages.empty()) std::memcpy(blob + pages_off, pages.data(), pages.size() * sizeof(int));
    if (!items.empty()) std::memcpy(blob + items_off, items.data(), items.size() * sizeof(WorkItem));
    if (!ditems.empty()) std::memcpy(blob + ditems_off, ditems.data(), ditems.size() * sizeof(dec::DecodeItem));
    if (!tiles.empty()) std::memcpy(blob + ditems_off, tiles.data(), tiles.size() * sizeof(RowTile));
    if (!tok_rows.empty()) std::memcpy(blob + tok_rows_off, tok_rows.data(), tok_rows.size() * sizeof(long long));
    if (!tok_span.empty()) std::memcpy(blob + tok_span_off, tok_span.data(), tok_span.size() * sizeof(int2));
    cudaError_t e = cudaMemcpyAsync(ctx->d_arena + place, blob, total, cudaMemcpyHostToDevice, stream);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->stage_ev[sb], stream);
    if (e != cudaSuccess) {
      *status = fail(ctx, BICACHE_ERR_CUDA, std::string("schedule upload: ") + cudaGetErrorString(e));
      return -1;
    }
    ctx->stage_used[sb] = true;
    ctx->schedule_uploads++;
  }
  c.kind = key_kind;
  c.hash = hash;
  c.off = place;
  c.bytes = align_up(total, 256);
  c.prefix_id.assign(prefix_id ? prefix_id : nullptr, prefix_id ? prefix_id + R : nullptr);
  c.row_off.assign(row_off, row_off + R);
  c.seqlen.assign(seqlen, seqlen + R);
  c.num_items = (int)items.size() * (kind == 2 ? num_splits : 1);   // kind 2 stores the first range's items only
  c.ditems_off = ditems_off;
  c.tok_rows_off = tok_rows_off;
  c.tok_span_off = tok_span_off;
  c.num_ditems = (int)ditems.size();
  c.num_tiles = (int)tiles.size();
  c.shared_tiles = false;
  for (const RowTile& tl : tiles) c.shared_tiles = c.shared_tiles || tl.nseg > 1;
  c.num_splits = num_splits;
  c.tiles_per_split = tiles_per_split;
  c.total_tokens = (int)tok;
  c.reqs_off = reqs_off;
  c.pages_off = pages_off;
  c.items_off = items_off;
  c.last_use = ctx->use_counter;
  c.valid = true;
  return victim;
}

void drop_schedules(bicache_ctx* ctx) {
  for (CachedSchedule& c : ctx->sched) c.valid = false;
}

// The pinned staging buffers and their events (the only non-heap host resources of a context).
void destroy_host_resources(bicache_ctx* ctx) {
  for (int i = 0; i < kStageBufs; ++i) {
    if (ctx->stage_ev[i]) cudaEventDestroy(ctx->stage_ev[i]);
    if (ctx->h_stage[i]) cudaFreeHost(ctx->h_stage[i]);
    ctx->stage_ev[i] = nullptr;
    ctx->h_stage[i] = nullptr;
  }
}

// One attention call, validated and with its schedule on the device, not yet launched.
struct PreparedCall {
  bool empty = true;           // nothing to launch
  int entry = -1;              // index in ctx->sched
  bool key_ranges = false, use_tensor = false;
  bool pairs = false;          // the tensor-core kernel on CTA pairs
  TcTensorMaps maps;
  CUtensorMap k64;             // pairs: k with a box of 64 rows
};

// Everything the host can check, then the schedule (found in the cache or built and uploaded) and the
// tensor maps.  Launches no kernel and writes no output.
int prepare_attention(bicache_ctx* ctx, int kind, int32_t layer, int32_t R, const int32_t* prefix_id,
                      const int64_t* row_off, const int32_t* seqlen, const void* q, const void* k, const void* v,
                      int64_t q_row_stride, int64_t kv_row_stride, void* out, int64_t out_row_stride,
                      float* lse_out, float softmax_scale, void* stream_, PreparedCall* pc) {
  *pc = PreparedCall();
  if (!ctx) return BICACHE_ERR_INVALID;
  if (ctx->host_only) return fail(ctx, BICACHE_ERR_UNSUPPORTED, "host-only context has no device path");
  const bicache_config& cfg = ctx->cfg;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if (layer < 0 || layer >= cfg.num_layers) return fail(ctx, BICACHE_ERR_INVALID, "layer out of range");
  if (R < 0) return fail(ctx, BICACHE_ERR_INVALID, "negative request count");
  if (R == 0) return BICACHE_OK;
  if (!row_off || !seqlen || (kind == 0 && !prefix_id))
    return fail(ctx, BICACHE_ERR_INVALID, "null metadata array");
  if (!q || !k || !v || !out) return fail(ctx, BICACHE_ERR_INVALID, "null tensor pointer");
  if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) ||
      (lse_out && (reinterpret_cast<uintptr_t>(lse_out) & 3)))
    return fail(ctx, BICACHE_ERR_INVALID, "tensor pointer not 16-byte aligned");
  const int D = cfg.head_dim;
  if (q_row_stride < (int64_t)cfg.num_q_heads * D || out_row_stride < (int64_t)cfg.num_q_heads * D ||
      kv_row_stride < (int64_t)cfg.num_kv_heads * D || (q_row_stride * ctx->esize) % 16 ||
      (kv_row_stride * ctx->esize) % 16 || (out_row_stride * ctx->esize) % 16)
    return fail(ctx, BICACHE_ERR_INVALID, "bad row stride");
  long long total = 0;
  for (int i = 0; i < R; ++i) {
    if (seqlen[i] < 0 || row_off[i] < 0) return fail(ctx, BICACHE_ERR_INVALID, "negative length or offset");
    total += seqlen[i];
  }
  if (total > 0x7fffffffLL / std::max(1, cfg.num_q_heads / cfg.num_kv_heads))
    return fail(ctx, BICACHE_ERR_INVALID, "batch too large");
  if (kind == 0) {
    // equal ids contiguous; every id live
    std::vector<int32_t> seen;
    for (int i = 0; i < R; ++i) {
      const int32_t p = prefix_id[i];
      if (p < -1) return fail(ctx, BICACHE_ERR_INVALID, "bad prefix id");
      if (i > 0 && p == prefix_id[i - 1]) continue;
      if (p >= 0) {
        if (std::find(seen.begin(), seen.end(), p) != seen.end())
          return fail(ctx, BICACHE_ERR_INVALID, "requests of one prefix are not contiguous");
        seen.push_back(p);
        auto found = ctx->by_id.find(p);
        if (found == ctx->by_id.end())
          return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
        if (found->second->first_layer > layer)
          return fail(ctx, BICACHE_ERR_INVALID, "the prefix owns no pages in this layer");
      }
    }
  }
  if (total == 0) return BICACHE_OK;

  // the tensor-core kernels take the row maximum before scaling, which needs a positive scale
  pc->use_tensor = ctx->tensor_ok && ctx->path != BICACHE_PATH_SIMT && softmax_scale > 0.f;
  // Few query rows per prefix group against a long cached prefix (block-query decoding): the
  // bandwidth-bound regime, served by the key-range kernel.  Conditions: every request has a cached
  // prefix of at least 1024 tokens and at most 128 packed rows per KV head (a request with more fills
  // the general kernel's tiles by itself), and the call's tokens fit the kernel's tables.
  bool key_ranges = kind == 0 && pc->use_tensor;
  if (key_ranges) {
    const int G = cfg.num_q_heads / cfg.num_kv_heads;
    for (int i = 0; i < R && key_ranges; ++i) {
      if (prefix_id[i] < 0) { key_ranges = false; break; }
      if (ctx->by_id.at(prefix_id[i])->m < 1024) key_ranges = false;
      if ((long long)seqlen[i] * G > 128) key_ranges = false;
    }
    if (total > kMaxDecodeTokens) key_ranges = false;
  }
  // The kernel on CTA pairs serves full attention only when asked for (it is the slower of the two on
  // every shape measured: the hand-over between the two SMs lengthens the per-tile chain by more than
  // the halved shared-memory traffic shortens it).
  pc->pairs = kind == 1 && pc->use_tensor && ctx->path == BICACHE_PATH_TENSOR_PAIRS && ctx->attn_pairs > 0;
  int st = BICACHE_OK;
  int entry = -1;
  if (key_ranges) {
    entry = prepare_schedule(ctx, 2, false, false, layer, R, prefix_id, row_off, seqlen, stream, &st);
    if (entry < 0) {                                     // does not fit: the general path
      key_ranges = false;
      ctx->last_error.clear();
    }
  }
  if (entry < 0)
    entry = prepare_schedule(ctx, kind, kind == 0 && pc->use_tensor && kTiledAttend, pc->pairs, layer, R, prefix_id,
                             row_off, seqlen, stream, &st);
  if (entry < 0) return st;
  pc->entry = entry;
  pc->key_ranges = key_ranges;
  if (pc->use_tensor && !key_ranges) {
    // rows the tensors are known to have: up to the end of the last request
    long long rows_total = 0;
    for (int i = 0; i < R; ++i) rows_total = std::max<long long>(rows_total, row_off[i] + seqlen[i]);
    const int G = cfg.num_q_heads / cfg.num_kv_heads;
    TcTensorMaps& maps = pc->maps;
    maps.q_tma = (128 % G == 0) ? 1 : 0;
    maps.q8_tma = (8 % G == 0) ? 1 : 0;
    bool okm = encode_map(&maps.k, k, rows_total, cfg.num_kv_heads, kv_row_stride, 1, 128) &&
               encode_map(&maps.v, v, rows_total, cfg.num_kv_heads, kv_row_stride, 1, 128) &&
               encode_map(&maps.q, q, rows_total, cfg.num_q_heads, q_row_stride, maps.q_tma ? G : 1,
                          maps.q_tma ? 128 / G : 128) &&
               encode_map(&maps.q8, q, rows_total, cfg.num_q_heads, q_row_stride, maps.q8_tma ? G : 1,
                          maps.q8_tma ? 8 / G : 8);
    maps.o_tma = (32 % G == 0) ? 1 : 0;
    okm = okm && encode_map(&maps.o, out, rows_total, cfg.num_q_heads, out_row_stride, maps.o_tma ? G : 1,
                            maps.o_tma ? 32 / G : 32);
    if (pc->pairs) okm = okm && encode_map(&pc->k64, k, rows_total, cfg.num_kv_heads, kv_row_stride, 1, 64);
    if (!okm) return fail(ctx, BICACHE_ERR_CUDA, "tensor map encoding failed");
  }
  pc->empty = false;
  return BICACHE_OK;
}

// The kernel launches of a prepared call.
int launch_attention(bicache_ctx* ctx, const PreparedCall& pc, int32_t layer, const void* q, const void* k,
                     const void* v, int64_t q_row_stride, int64_t kv_row_stride, void* out, int64_t out_row_stride,
                     float* lse_out, float softmax_scale, void* stream_) {
  if (pc.empty) return BICACHE_OK;
  const bicache_config& cfg = ctx->cfg;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const CachedSchedule& c = ctx->sched[pc.entry];
  char* base = ctx->d_arena + c.off;
  ScheduleView sv;
  sv.reqs = reinterpret_cast<const ReqMeta*>(base + c.reqs_off);
  sv.pages = reinterpret_cast<const int*>(base + c.pages_off);
  sv.items = reinterpret_cast<const WorkItem*>(base + c.items_off);
  sv.tiles = c.num_tiles > 0 ? reinterpret_cast<const RowTile*>(base + c.ditems_off) : nullptr;
  sv.shared_tiles = c.shared_tiles ? 1 : 0;
  sv.num_items = c.num_items;
  sv.num_splits = c.num_splits;
  sv.tiles_per_split = c.tiles_per_split;

  TensorArgs t;
  t.q = static_cast<const char*>(q);
  t.k = static_cast<const char*>(k);
  t.v = static_cast<const char*>(v);
  t.out = static_cast<char*>(out);
  t.lse = lse_out;
  t.q_stride = q_row_stride;
  t.kv_stride = kv_row_stride;
  t.out_stride = out_row_stride;
  t.Hq = cfg.num_q_heads;
  t.Hkv = cfg.num_kv_heads;
  t.D = cfg.head_dim;
  t.layer = 0;                                  // the pool view below starts at this call's layer
  t.scale = softmax_scale;
  t.part_o = ctx->d_part_o;
  t.part_lse = ctx->d_part_lse;
  t.total_tokens = c.total_tokens;
  const PoolView pool = pool_view_layer(ctx, layer);

  cudaError_t e;
  ctx->last_kernel = pc.key_ranges ? BICACHE_KERNEL_KEY_RANGES
                     : pc.pairs    ? BICACHE_KERNEL_TENSOR_PAIRS
                     : pc.use_tensor ? BICACHE_KERNEL_TENSOR
                                     : BICACHE_KERNEL_SIMT;
  if (pc.key_ranges) {
    e = launch_tc_decode(reinterpret_cast<const dec::DecodeItem*>(base + c.ditems_off), c.num_ditems,
                         reinterpret_cast<const long long*>(base + c.tok_rows_off),
                         reinterpret_cast<const int2*>(base + c.tok_span_off), sv.pages, pool, t, ctx->d_status,
                         ctx->wait_cycles, stream);
  } else if (pc.pairs) {
    e = launch_tc_attention_pair(sv, t, ctx->d_status, ctx->attn_pairs, pc.maps.q, pc.k64, pc.maps.v, pc.maps.o,
                                 pc.maps.q_tma, pc.maps.o_tma, ctx->wait_cycles, stream);
  } else if (pc.use_tensor) {
    e = launch_tc_attention(sv, pool, t, ctx->d_status, ctx->sm_count, pc.maps, ctx->wait_cycles, stream);
  } else if (cfg.dtype == BICACHE_F32) {
    simt_attention_kernel<float><<<c.num_items, kSimtWarps * 32, 0, stream>>>(sv, pool, t);
    e = cudaGetLastError();
  } else {
    simt_attention_kernel<__nv_bfloat16><<<c.num_items, kSimtWarps * 32, 0, stream>>>(sv, pool, t);
    e = cudaGetLastError();
  }
  ctx->launches++;
  if (e != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(e));
  if (pc.key_ranges) {
    e = launch_merge_ranges(t, reinterpret_cast<const long long*>(base + c.tok_rows_off), c.num_splits, stream);
    ctx->launches++;
    if (e != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("merge launch: ") + cudaGetErrorString(e));
  } else if (c.num_splits > 1) {
    const int grid = c.num_items / c.num_splits * (kTileRows / kMergeRowsPerBlock);
    if (cfg.dtype == BICACHE_F32)
      merge_partials_kernel<float><<<grid, kMergeRowsPerBlock * 32, 0, stream>>>(sv, t);
    else
      merge_partials_kernel<__nv_bfloat16><<<grid, kMergeRowsPerBlock * 32, 0, stream>>>(sv, t);
    ctx->launches++;
    e = cudaGetLastError();
    if (e != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("merge launch: ") + cudaGetErrorString(e));
  }
  return BICACHE_OK;
}

int run_attention(bicache_ctx* ctx, int kind, int32_t layer, int32_t R, const int32_t* prefix_id,
                  const int64_t* row_off, const int32_t* seqlen, const void* q, const void* k, const void* v,
                  int64_t q_row_stride, int64_t kv_row_stride, void* out, int64_t out_row_stride,
                  float* lse_out, float softmax_scale, void* stream) {
  if (ctx) ctx->use_counter++;
  PreparedCall pc;
  const int st = prepare_attention(ctx, kind, layer, R, prefix_id, row_off, seqlen, q, k, v, q_row_stride,
                                   kv_row_stride, out, out_row_stride, lse_out, softmax_scale, stream, &pc);
  if (st != BICACHE_OK) return st;
  return launch_attention(ctx, pc, layer, q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                          softmax_scale, stream);
}

}  // namespace

extern "C" {

size_t bicache_pool_bytes(const bicache_config* cfg) {
  if (!sane(cfg)) return 0;
  const size_t es = cfg->dtype == BICACHE_F32 ? 4 : 2;
  size_t pages = 0;
  for (int l = 0; l < cfg->num_layers; ++l) {
    const int32_t c = cfg->layer_pages ? cfg->layer_pages[l] : cfg->num_pages;
    if (c < 1 || c > cfg->num_pages) return 0;
    pages += (size_t)c;
  }
  return pages * cfg->num_kv_heads * cfg->page_size * cfg->head_dim * es;
}

size_t bicache_workspace_bytes(const bicache_config* cfg, int64_t max_total_rows, int32_t max_requests) {
  if (!sane(cfg) || max_total_rows < 0 || max_requests < 0) return 0;
  return kStatusBytes + (size_t)arena_schedules_for(cfg) * schedule_bytes_for(cfg, max_total_rows, max_requests) +
         partial_bytes_for(cfg) + align_up((size_t)cfg->num_pages * sizeof(int) + 16, 256);
}

int32_t bicache_create(const bicache_config* cfg, bicache_ctx** out) {
  if (!out) return BICACHE_ERR_INVALID;
  *out = nullptr;
  if (!sane(cfg)) return BICACHE_ERR_INVALID;
  int esize;
  bool swz, tensor_ok;
  if (!supported(cfg, &esize, &swz, &tensor_ok)) return BICACHE_ERR_UNSUPPORTED;
  const bool host_only = cfg->device < 0;
  const size_t part = partial_bytes_for(cfg);
  const size_t put_pages = align_up((size_t)cfg->num_pages * sizeof(int) + 16, 256);
  if (cfg->layer_pages)
    for (int l = 0; l < cfg->num_layers; ++l)
      if (cfg->layer_pages[l] < 1 || cfg->layer_pages[l] > cfg->num_pages) return BICACHE_ERR_INVALID;
  if (!host_only) {
    if (!cfg->k_pool || !cfg->v_pool || !cfg->workspace) return BICACHE_ERR_INVALID;
    if ((reinterpret_cast<uintptr_t>(cfg->k_pool) & 255) || (reinterpret_cast<uintptr_t>(cfg->v_pool) & 255) ||
        (reinterpret_cast<uintptr_t>(cfg->workspace) & 255))
      return BICACHE_ERR_INVALID;
    if (cfg->workspace_bytes < kStatusBytes + part + put_pages + 2 * schedule_bytes_for(cfg, 0, 0))
      return BICACHE_ERR_NOMEM;
  }
  std::vector<int32_t> order(cfg->num_pages);
  if (cfg->initial_free_order) {
    std::vector<char> seen(cfg->num_pages, 0);
    for (int i = 0; i < cfg->num_pages; ++i) {
      const int32_t p = cfg->initial_free_order[i];
      if (p < 0 || p >= cfg->num_pages || seen[p]) return BICACHE_ERR_INVALID;
      seen[p] = 1;
      order[i] = p;
    }
  } else {
    for (int i = 0; i < cfg->num_pages; ++i) order[i] = i;
  }
  if (!host_only && cudaSetDevice(cfg->device) != cudaSuccess) return BICACHE_ERR_CUDA;
  bicache_ctx* ctx = new (std::nothrow) bicache_ctx();
  if (!ctx) return BICACHE_ERR_NOMEM;
  ctx->host_only = host_only;
  ctx->cfg = *cfg;
  ctx->cfg.initial_free_order = nullptr;
  ctx->cfg.layer_pages = nullptr;
  ctx->esize = esize;
  ctx->swizzled = swz;
  ctx->tensor_ok = tensor_ok;
  // per layer: capacity, place inside a pool, and the free queue (the pages below the layer's capacity,
  // in the initial order)
  ctx->free_pages.resize(cfg->num_layers);
  ctx->layer_cap.resize(cfg->num_layers);
  ctx->layer_off.resize(cfg->num_layers);
  long long off = 0;
  const long long slice = (long long)cfg->num_kv_heads * kPageSize * cfg->head_dim * esize;
  for (int l = 0; l < cfg->num_layers; ++l) {
    const int32_t cap = cfg->layer_pages ? cfg->layer_pages[l] : cfg->num_pages;
    ctx->layer_cap[l] = cap;
    ctx->layer_off[l] = off;
    off += (long long)cap * slice;
    if (cap != cfg->num_pages) ctx->uniform_caps = false;
    for (int32_t pg : order)
      if (pg < cap) ctx->free_pages[l].push_back(pg);
  }
  if (host_only) {
    *out = ctx;
    return BICACHE_OK;
  }
  char* ws = static_cast<char*>(cfg->workspace);
  ctx->d_status = reinterpret_cast<int*>(ws);
  ctx->d_part_o = reinterpret_cast<float*>(ws + kStatusBytes);
  ctx->d_part_lse = ctx->d_part_o + (size_t)kMaxPartialRowHeads * cfg->head_dim;
  ctx->part_capacity_rowheads = kMaxPartialRowHeads;
  ctx->d_put_pages = reinterpret_cast<int*>(ws + kStatusBytes + part);
  ctx->d_arena = ws + kStatusBytes + part + put_pages;
  ctx->arena_bytes = (cfg->workspace_bytes - (kStatusBytes + part + put_pages)) / 256 * 256;
  ctx->sched.resize(kMaxCached);
  for (int i = 0; i < kStageBufs; ++i)
    if (cudaEventCreateWithFlags(&ctx->stage_ev[i], cudaEventDisableTiming) != cudaSuccess) {
      destroy_host_resources(ctx);
      delete ctx;
      return BICACHE_ERR_CUDA;
    }
  int sms = 0;
  if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device) == cudaSuccess && sms > 0)
    ctx->sm_count = sms;
  if (cudaMemset(ws, 0, kStatusBytes) != cudaSuccess) {
    destroy_host_resources(ctx);
    delete ctx;
    return BICACHE_ERR_CUDA;
  }
  if (tensor_ok) {
    cudaError_t e = configure_tc_attention();
    if (e == cudaSuccess) e = configure_project_kv(&ctx->proj_pairs);
    if (e == cudaSuccess) e = configure_tc_attention_pair(&ctx->attn_pairs);
    if (e == cudaSuccess) e = configure_tc_decode();
    if (e != cudaSuccess) {
      destroy_host_resources(ctx);
      delete ctx;
      return BICACHE_ERR_CUDA;
    }
  }
  *out = ctx;
  return BICACHE_OK;
}

int32_t bicache_destroy(bicache_ctx* ctx) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (ctx->host_only) {
    delete ctx;
    return BICACHE_OK;
  }
  cudaSetDevice(ctx->cfg.device);
  cudaError_t e = cudaDeviceSynchronize();
  destroy_host_resources(ctx);
  delete ctx;
  return e == cudaSuccess ? BICACHE_OK : BICACHE_ERR_CUDA;
}

int32_t bicache_set_path(bicache_ctx* ctx, int32_t path) {
  if (!ctx || path < BICACHE_PATH_AUTO || path > BICACHE_PATH_TENSOR_PAIRS) return BICACHE_ERR_INVALID;
  if ((path == BICACHE_PATH_TENSOR || path == BICACHE_PATH_TENSOR_PAIRS) && !ctx->tensor_ok)
    return fail(ctx, BICACHE_ERR_UNSUPPORTED, "tensor-core path needs bf16 and head_dim 128");
  ctx->path = path;
  return BICACHE_OK;
}

int32_t bicache_set_depth_table(bicache_ctx* ctx, const int32_t* table, int32_t n) {
  if (!ctx || !table || n != 101) return fail(ctx, BICACHE_ERR_INVALID, "depth table must have 101 entries");
  ctx->depth_table.assign(table, table + n);
  return BICACHE_OK;
}

}  // extern "C"

namespace {
// Insert a prefix that owns the layers first_layer .. L-1: hit / miss / FIFO eviction / page allocation
// per layer, and (write = true, first_layer = 0) the scatter of all layers' K/V into the page images.
int32_t put_impl(bicache_ctx* ctx, uint64_t key, int32_t m, const void* k, const void* v, int64_t layer_stride,
                 void* stream_, int32_t* prefix_id, int32_t* was_hit, int32_t* pages_out, int32_t pages_cap,
                 bool write, int32_t first_layer) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (!prefix_id) return fail(ctx, BICACHE_ERR_INVALID, "prefix_id is required");
  if (m < 1) return fail(ctx, BICACHE_ERR_INVALID, "empty prefix");
  const bicache_config& cfg = ctx->cfg;
  const int L = cfg.num_layers;
  if (first_layer < 0 || first_layer >= L) return fail(ctx, BICACHE_ERR_INVALID, "first layer out of range");
  const int need = (m + kPageSize - 1) / kPageSize;
  auto found = ctx->by_key.find(key);
  if (found != ctx->by_key.end()) {
    const PrefixEntry& e = *found->second;
    if (e.m != m || e.first_layer != first_layer)
      return fail(ctx, BICACHE_ERR_INVALID, "key already present with another length or first layer");
    if (pages_out && pages_cap < need) return fail(ctx, BICACHE_ERR_INVALID, "pages_out too small");
    *prefix_id = e.id;
    if (was_hit) *was_hit = 1;
    if (pages_out) std::copy(e.pages.begin(), e.pages.end(), pages_out);
    return BICACHE_OK;
  }
  write = write && !ctx->host_only;
  if (write && (!k || !v || !aligned16(k) || !aligned16(v))) return fail(ctx, BICACHE_ERR_INVALID, "bad k/v pointer");
  const int64_t row_elems = (int64_t)cfg.num_kv_heads * cfg.head_dim;
  if (write && (layer_stride < (int64_t)m * row_elems || (layer_stride * ctx->esize) % 16))
    return fail(ctx, BICACHE_ERR_INVALID, "bad layer stride");
  for (int l = first_layer; l < L; ++l)
    if (need > ctx->layer_cap[l]) return fail(ctx, BICACHE_ERR_NOMEM, "prefix larger than a layer's pool");
  if (pages_out && pages_cap < need) return fail(ctx, BICACHE_ERR_INVALID, "pages_out too small");
  auto lacking = [&]() {
    for (int l = first_layer; l < L; ++l)
      if ((int)ctx->free_pages[l].size() < need) return true;
    return false;
  };
  while (lacking()) {
    PrefixEntry& old = ctx->fifo.front();
    for (int l = old.first_layer; l < L; ++l)
      for (int32_t pg : pages_of(old, l)) ctx->free_pages[l].push_back(pg);
    ctx->by_key.erase(old.key);
    ctx->by_id.erase(old.id);
    ctx->fifo.pop_front();
    drop_schedules(ctx);
  }
  PrefixEntry e;
  e.key = key;
  e.m = m;
  e.first_layer = first_layer;
  e.id = ctx->next_id++;
  std::vector<std::vector<int32_t>> lists(L - first_layer, std::vector<int32_t>(need));
  for (int l = first_layer; l < L; ++l)
    for (int i = 0; i < need; ++i) {
      lists[l - first_layer][i] = ctx->free_pages[l].front();
      ctx->free_pages[l].pop_front();
    }
  e.uniform = true;
  for (size_t j = 1; j < lists.size(); ++j) e.uniform = e.uniform && lists[j] == lists[0];
  e.pages = lists[0];
  if (!e.uniform) e.layer_pages = lists;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  cudaError_t ce = cudaSuccess;
  if (write) {
    const int chunks_per_row = cfg.head_dim * ctx->esize / 16;
    const int threads = 256;
    const PoolView pv = pool_view(ctx);
    if (e.uniform && ctx->uniform_caps) {
      // one page list and one layer stride: all layers in one launch
      ce = cudaMemcpyAsync(ctx->d_put_pages, e.pages.data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
      if (ce == cudaSuccess) {
        const long long total = (long long)L * need * kPageSize * cfg.num_kv_heads * chunks_per_row;
        const int blocks = (int)std::min<long long>((total + threads - 1) / threads, (long long)ctx->sm_count * 16);
        scatter_prefix_kernel<<<blocks, threads, 0, stream>>>(
            static_cast<const char*>(k), static_cast<const char*>(v), static_cast<char*>(cfg.k_pool),
            static_cast<char*>(cfg.v_pool), ctx->d_put_pages, need, m, L, cfg.num_kv_heads, chunks_per_row,
            layer_stride * ctx->esize, (long long)row_elems * ctx->esize, pv.layer_bytes, pv.page_bytes, pv.swizzled);
        ctx->launches++;
        ce = cudaGetLastError();
      }
    } else {
      // the lists or the layers' places differ: one launch per layer (the staging of the list is reused in
      // stream order)
      const long long total = (long long)need * kPageSize * cfg.num_kv_heads * chunks_per_row;
      const int blocks = (int)std::min<long long>((total + threads - 1) / threads, (long long)ctx->sm_count * 16);
      for (int l = 0; l < L && ce == cudaSuccess; ++l) {
        ce = cudaMemcpyAsync(ctx->d_put_pages, lists[l].data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
        if (ce != cudaSuccess) break;
        scatter_prefix_kernel<<<blocks, threads, 0, stream>>>(
            static_cast<const char*>(k) + (long long)l * layer_stride * ctx->esize,
            static_cast<const char*>(v) + (long long)l * layer_stride * ctx->esize,
            static_cast<char*>(cfg.k_pool) + ctx->layer_off[l], static_cast<char*>(cfg.v_pool) + ctx->layer_off[l],
            ctx->d_put_pages, need, m, 1, cfg.num_kv_heads, chunks_per_row, 0, (long long)row_elems * ctx->esize,
            pv.layer_bytes, pv.page_bytes, pv.swizzled);
        ctx->launches++;
        ce = cudaGetLastError();
      }
    }
  }
  if (ce != cudaSuccess) {
    for (int l = first_layer; l < L; ++l) {
      const std::vector<int32_t>& pl = lists[l - first_layer];
      for (auto it = pl.rbegin(); it != pl.rend(); ++it) ctx->free_pages[l].push_front(*it);
    }
    ctx->next_id--;
    return fail(ctx, BICACHE_ERR_CUDA, std::string("put_prefix: ") + cudaGetErrorString(ce));
  }
  *prefix_id = e.id;
  if (was_hit) *was_hit = 0;
  if (pages_out) std::copy(e.pages.begin(), e.pages.end(), pages_out);
  ctx->fifo.push_back(std::move(e));
  auto it = std::prev(ctx->fifo.end());
  ctx->by_key[key] = it;
  ctx->by_id[it->id] = it;
  return BICACHE_OK;
}
}  // namespace

extern "C" {

int32_t bicache_put_prefix(bicache_ctx* ctx, uint64_t key, int32_t m, const void* k, const void* v,
                           int64_t layer_stride, void* stream, int32_t* prefix_id, int32_t* was_hit,
                           int32_t* pages_out, int32_t pages_cap) {
  return put_impl(ctx, key, m, k, v, layer_stride, stream, prefix_id, was_hit, pages_out, pages_cap, true, 0);
}

int32_t bicache_reserve_prefix(bicache_ctx* ctx, uint64_t key, int32_t m, int32_t* prefix_id, int32_t* was_hit,
                               int32_t* pages_out, int32_t pages_cap) {
  return put_impl(ctx, key, m, nullptr, nullptr, 0, nullptr, prefix_id, was_hit, pages_out, pages_cap, false, 0);
}

int32_t bicache_reserve_prefix_layers(bicache_ctx* ctx, uint64_t key, int32_t m, int32_t first_layer,
                                      int32_t* prefix_id, int32_t* was_hit, int32_t* pages_out, int32_t pages_cap) {
  return put_impl(ctx, key, m, nullptr, nullptr, 0, nullptr, prefix_id, was_hit, pages_out, pages_cap, false,
                  first_layer);
}

int32_t bicache_update_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* k,
                                    const void* v, int64_t kv_row_stride, void* stream_) {
  if (!ctx) return BICACHE_ERR_INVALID;
  const bicache_config& cfg = ctx->cfg;
  auto found = ctx->by_id.find(prefix_id);
  if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
  if (layer < 0 || layer >= cfg.num_layers) return fail(ctx, BICACHE_ERR_INVALID, "layer out of range");
  const PrefixEntry& e = *found->second;
  if (layer < e.first_layer) return fail(ctx, BICACHE_ERR_INVALID, "the prefix owns no pages in this layer");
  const int64_t row_elems = (int64_t)cfg.num_kv_heads * cfg.head_dim;
  if (kv_row_stride < row_elems || (kv_row_stride * ctx->esize) % 16)
    return fail(ctx, BICACHE_ERR_INVALID, "bad row stride");
  if (ctx->host_only) return BICACHE_OK;
  if (!k || !v || !aligned16(k) || !aligned16(v)) return fail(ctx, BICACHE_ERR_INVALID, "bad k/v pointer");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int need = (int)e.pages.size();
  cudaError_t ce =
      cudaMemcpyAsync(ctx->d_put_pages, pages_of(e, layer).data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
  if (ce == cudaSuccess) {
    const int chunks_per_row = cfg.head_dim * ctx->esize / 16;
    const long long total = (long long)need * kPageSize * cfg.num_kv_heads * chunks_per_row;
    const int threads = 256;
    const int blocks = (int)std::min<long long>((total + threads - 1) / threads, (long long)ctx->sm_count * 16);
    const PoolView pv = pool_view(ctx);
    scatter_prefix_kernel<<<blocks, threads, 0, stream>>>(
        static_cast<const char*>(k), static_cast<const char*>(v),
        static_cast<char*>(cfg.k_pool) + ctx->layer_off[layer],
        static_cast<char*>(cfg.v_pool) + ctx->layer_off[layer], ctx->d_put_pages, need, e.m, 1,
        cfg.num_kv_heads, chunks_per_row, 0, kv_row_stride * ctx->esize, pv.layer_bytes, pv.page_bytes, pv.swizzled);
    ctx->launches++;
    ce = cudaGetLastError();
  }
  if (ce != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("update_prefix_layer: ") + cudaGetErrorString(ce));
  return BICACHE_OK;
}

int32_t bicache_read_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, void* k_out, void* v_out,
                                  int64_t kv_row_stride, void* stream_) {
  if (!ctx) return BICACHE_ERR_INVALID;
  const bicache_config& cfg = ctx->cfg;
  auto found = ctx->by_id.find(prefix_id);
  if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
  if (layer < 0 || layer >= cfg.num_layers) return fail(ctx, BICACHE_ERR_INVALID, "layer out of range");
  const PrefixEntry& e = *found->second;
  if (layer < e.first_layer) return fail(ctx, BICACHE_ERR_INVALID, "the prefix owns no pages in this layer");
  const int64_t row_elems = (int64_t)cfg.num_kv_heads * cfg.head_dim;
  if (kv_row_stride < row_elems || (kv_row_stride * ctx->esize) % 16)
    return fail(ctx, BICACHE_ERR_INVALID, "bad row stride");
  if (ctx->host_only) return fail(ctx, BICACHE_ERR_UNSUPPORTED, "host-only context");
  if (!k_out || !v_out || !aligned16(k_out) || !aligned16(v_out))
    return fail(ctx, BICACHE_ERR_INVALID, "bad k/v pointer");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int need = (int)e.pages.size();
  cudaError_t ce =
      cudaMemcpyAsync(ctx->d_put_pages, pages_of(e, layer).data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
  if (ce == cudaSuccess && e.m > 0) {
    const int chunks_per_row = cfg.head_dim * ctx->esize / 16;
    const long long total = (long long)e.m * cfg.num_kv_heads * chunks_per_row;
    const int threads = 256;
    const int blocks = (int)std::min<long long>((total + threads - 1) / threads, (long long)ctx->sm_count * 16);
    const PoolView pv = pool_view(ctx);
    gather_prefix_kernel<<<blocks, threads, 0, stream>>>(
        pv.k + ctx->layer_off[layer], pv.v + ctx->layer_off[layer],
        static_cast<char*>(k_out), static_cast<char*>(v_out), ctx->d_put_pages, e.m, cfg.num_kv_heads,
        chunks_per_row, kv_row_stride * ctx->esize, pv.page_bytes, pv.swizzled);
    ctx->launches++;
    ce = cudaGetLastError();
  }
  if (ce != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("read_prefix_layer: ") + cudaGetErrorString(ce));
  return BICACHE_OK;
}

// bf16 matrix [rows][cols] with `row_stride` elements between rows; box = (64 columns, box_rows),
// 128-byte swizzle, zero fill outside.
static bool encode_map_2d(CUtensorMap* m, const void* base, long long rows, long long cols, long long row_stride,
                          int box_rows) {
  EncodeTiledFn fn = encode_tiled_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)row_stride * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int32_t bicache_project_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* h,
                                     int64_t h_row_stride, const void* w_k, const void* w_v, int32_t d_model,
                                     void* stream_) {
  return bicache_project_prefix_layer_rope(ctx, prefix_id, layer, h, h_row_stride, w_k, w_v, d_model, nullptr,
                                           stream_);
}

int32_t bicache_project_prefix_layer_rope(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* h,
                                          int64_t h_row_stride, const void* w_k, const void* w_v, int32_t d_model,
                                          const float* rope_cos_sin, void* stream_) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (rope_cos_sin && (reinterpret_cast<uintptr_t>(rope_cos_sin) & 15))
    return fail(ctx, BICACHE_ERR_INVALID, "the rotary table must be 16-byte aligned");
  const bicache_config& cfg = ctx->cfg;
  if (!ctx->tensor_ok && !(ctx->host_only && cfg.dtype == BICACHE_BF16 && cfg.head_dim == 128))
    return fail(ctx, BICACHE_ERR_UNSUPPORTED, "projection needs a bf16 context with head_dim 128");
  auto found = ctx->by_id.find(prefix_id);
  if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
  if (layer < 0 || layer >= cfg.num_layers) return fail(ctx, BICACHE_ERR_INVALID, "layer out of range");
  if (d_model <= 0 || d_model % 8 || h_row_stride < d_model || h_row_stride % 8)
    return fail(ctx, BICACHE_ERR_INVALID, "d_model and the row stride must be positive multiples of 8");
  const PrefixEntry& e = *found->second;
  if (layer < e.first_layer) return fail(ctx, BICACHE_ERR_INVALID, "the prefix owns no pages in this layer");
  if (ctx->host_only) return BICACHE_OK;
  if (!h || !w_k || !w_v || !aligned16(h) || !aligned16(w_k) || !aligned16(w_v))
    return fail(ctx, BICACHE_ERR_INVALID, "bad h/w pointer");
  if (e.m == 0) return BICACHE_OK;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int need = (int)e.pages.size();
  CUtensorMap tm_h, tm_wk, tm_wv;
  const long long out_rows = (long long)cfg.num_kv_heads * cfg.head_dim;
  if (!encode_map_2d(&tm_h, h, e.m, d_model, h_row_stride, proj::kBM) ||
      !encode_map_2d(&tm_wk, w_k, out_rows, d_model, d_model, 64) ||
      !encode_map_2d(&tm_wv, w_v, out_rows, d_model, d_model, 64))
    return fail(ctx, BICACHE_ERR_CUDA, "project_prefix_layer: tensor map encoding failed");
  cudaError_t ce =
      cudaMemcpyAsync(ctx->d_put_pages, pages_of(e, layer).data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
  if (ce == cudaSuccess) {
    const PoolView pv = pool_view(ctx);
    proj::ProjArgs a;
    a.pool_k = static_cast<char*>(cfg.k_pool) + ctx->layer_off[layer];
    a.pool_v = static_cast<char*>(cfg.v_pool) + ctx->layer_off[layer];
    a.pages = ctx->d_put_pages;
    a.rope = reinterpret_cast<const float2*>(rope_cos_sin);
    a.m = e.m;
    a.d_model = d_model;
    a.num_kv_heads = cfg.num_kv_heads;
    a.m_tiles = (e.m + 2 * proj::kBM - 1) / (2 * proj::kBM);
    a.n_tiles = (cfg.num_kv_heads + 1) / 2;
    a.full_tiles = 0;                                   // set by the launcher
    ce = launch_project_kv(a, ctx->d_status, ctx->proj_pairs, tm_h, tm_wk, tm_wv, ctx->wait_cycles, stream);
    ctx->launches++;
  }
  if (ce != cudaSuccess)
    return fail(ctx, BICACHE_ERR_CUDA, std::string("project_prefix_layer: ") + cudaGetErrorString(ce));
  return BICACHE_OK;
}

int32_t bicache_prefix_similarity_async(bicache_ctx* ctx, int32_t prefix_id, const void* k_ref, const void* v_ref,
                                        int64_t layer_stride, float* sim_dev, void* stream_) {
  if (!ctx) return BICACHE_ERR_INVALID;
  const bicache_config& cfg = ctx->cfg;
  auto found = ctx->by_id.find(prefix_id);
  if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
  if (!sim_dev) return fail(ctx, BICACHE_ERR_INVALID, "the output array is required");
  const PrefixEntry& e = *found->second;
  const int64_t row_elems = (int64_t)cfg.num_kv_heads * cfg.head_dim;
  if (layer_stride < (int64_t)e.m * row_elems || (layer_stride * ctx->esize) % 16)
    return fail(ctx, BICACHE_ERR_INVALID, "bad layer stride");
  if (ctx->host_only) return fail(ctx, BICACHE_ERR_UNSUPPORTED, "host-only context");
  if (e.first_layer != 0 || !e.uniform || !ctx->uniform_caps)
    return fail(ctx, BICACHE_ERR_UNSUPPORTED, "the similarity needs a prefix with one page list for all layers");
  if (!k_ref || !v_ref || !aligned16(k_ref) || !aligned16(v_ref))
    return fail(ctx, BICACHE_ERR_INVALID, "bad k/v pointer");
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  const int need = (int)e.pages.size();
  // scratch: the key-split partials area (no attention call of this context can be running on it:
  // calls on one context are stream-ordered)
  double* partials = reinterpret_cast<double*>(ctx->d_part_o);
  cudaError_t ce =
      cudaMemcpyAsync(ctx->d_put_pages, e.pages.data(), sizeof(int) * need, cudaMemcpyHostToDevice, stream);
  if (ce == cudaSuccess) {
    const int chunks_per_row = cfg.head_dim * ctx->esize / 16;
    const PoolView pv = pool_view(ctx);
    const int bpl = std::max(1, std::min(kSimBlocksPerLayer, 2 * e.m));       // a block takes whole rows
    const dim3 grid(bpl, cfg.num_layers);
    if (cfg.dtype == BICACHE_F32)
      kv_similarity_partial_kernel<float><<<grid, kSimThreads, 0, stream>>>(
          pv.k, pv.v, static_cast<const char*>(k_ref), static_cast<const char*>(v_ref), ctx->d_put_pages, e.m,
          cfg.num_kv_heads, chunks_per_row, layer_stride * ctx->esize, pv.layer_bytes, pv.page_bytes, pv.swizzled,
          partials);
    else
      kv_similarity_partial_kernel<__nv_bfloat16><<<grid, kSimThreads, 0, stream>>>(
          pv.k, pv.v, static_cast<const char*>(k_ref), static_cast<const char*>(v_ref), ctx->d_put_pages, e.m,
          cfg.num_kv_heads, chunks_per_row, layer_stride * ctx->esize, pv.layer_bytes, pv.page_bytes, pv.swizzled,
          partials);
    kv_similarity_final_kernel<<<(cfg.num_layers + 63) / 64, 64, 0, stream>>>(partials, bpl, cfg.num_layers, sim_dev);
    ctx->launches += 2;
    ce = cudaGetLastError();
  }
  if (ce != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("prefix_similarity: ") + cudaGetErrorString(ce));
  return BICACHE_OK;
}

int32_t bicache_prefix_similarity(bicache_ctx* ctx, int32_t prefix_id, const void* k_ref, const void* v_ref,
                                  int64_t layer_stride, float* sim_out, void* stream_) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (!sim_out) return fail(ctx, BICACHE_ERR_INVALID, "sim_out is required");
  // device copy of the result: behind the block partials in the key-split scratch area
  float* d_sim = reinterpret_cast<float*>(reinterpret_cast<double*>(ctx->d_part_o) +
                                          (size_t)ctx->cfg.num_layers * kSimBlocksPerLayer * 3);
  const int32_t st = bicache_prefix_similarity_async(ctx, prefix_id, k_ref, v_ref, layer_stride, d_sim, stream_);
  if (st != BICACHE_OK) return st;
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  cudaError_t ce = cudaMemcpyAsync(sim_out, d_sim, sizeof(float) * ctx->cfg.num_layers, cudaMemcpyDeviceToHost, stream);
  if (ce == cudaSuccess) ce = cudaStreamSynchronize(stream);
  if (ce != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, std::string("prefix_similarity: ") + cudaGetErrorString(ce));
  return BICACHE_OK;
}

int32_t bicache_depth_from_similarity(const float* sim, int32_t num_layers, float tau, int32_t* depth) {
  if (num_layers < 0 || (num_layers > 0 && !sim) || !depth) return BICACHE_ERR_INVALID;
  int32_t b = 0;
  while (b < num_layers && sim[b] >= tau) ++b;          // NaN compares false: it ends the run
  *depth = b;
  return BICACHE_OK;
}

int32_t bicache_build_depth_table(const int32_t* ratio_idx, const int32_t* depth, int32_t n, int32_t num_layers,
                                  int32_t* table_out) {
  if (n < 0 || num_layers < 0 || !table_out || (n > 0 && (!ratio_idx || !depth))) return BICACHE_ERR_INVALID;
  long long sums[101] = {0};
  long long cnts[101] = {0};
  for (int i = 0; i < n; ++i) {
    if (ratio_idx[i] < 0 || ratio_idx[i] > 100 || depth[i] < 0 || depth[i] > num_layers) return BICACHE_ERR_INVALID;
    sums[ratio_idx[i]] += depth[i];
    cnts[ratio_idx[i]] += 1;
  }
  int32_t last = num_layers < 1 ? num_layers : 1;
  for (int idx = 0; idx <= 100; ++idx) {
    if (cnts[idx]) last = (int32_t)(sums[idx] / cnts[idx]);
    table_out[idx] = last;
  }
  return BICACHE_OK;
}

// XXH64 (seed 0) of the token ids taken as little-endian 32-bit integers: the 64-bit identifier of a
// tokenised prefix (Sec. 5.2 "k = h(p)").  Input length is a multiple of four bytes, so the tail is at
// most one 8-byte lane, one 4-byte lane and no single bytes.
uint64_t bicache_hash_tokens(const int32_t* tokens, int64_t n) {
  constexpr uint64_t P1 = 0x9E3779B185EBCA87ull, P2 = 0xC2B2AE3D27D4EB4Full, P3 = 0x165667B19E3779F9ull,
                     P4 = 0x85EBCA77C2B2AE63ull, P5 = 0x27D4EB2F165667C5ull;
  auto rotl = [](uint64_t x, int r) { return (x << r) | (x >> (64 - r)); };
  auto round = [&](uint64_t acc, uint64_t lane) { return rotl(acc + lane * P2, 31) * P1; };
  auto lane64 = [&](int64_t i) {                     // tokens i, i + 1 as one little-endian 64-bit lane
    return (uint64_t)(uint32_t)tokens[i] | ((uint64_t)(uint32_t)tokens[i + 1] << 32);
  };
  if (n < 0 || (n > 0 && !tokens)) return 0;
  const uint64_t bytes = (uint64_t)n * 4;
  int64_t i = 0;
  uint64_t h;
  if (n >= 8) {
    uint64_t v1 = P1 + P2, v2 = P2, v3 = 0, v4 = 0 - P1;
    for (; i + 8 <= n; i += 8) {
      v1 = round(v1, lane64(i));
      v2 = round(v2, lane64(i + 2));
      v3 = round(v3, lane64(i + 4));
      v4 = round(v4, lane64(i + 6));
    }
    h = rotl(v1, 1) + rotl(v2, 7) + rotl(v3, 12) + rotl(v4, 18);
    h = (h ^ round(0, v1)) * P1 + P4;
    h = (h ^ round(0, v2)) * P1 + P4;
    h = (h ^ round(0, v3)) * P1 + P4;
    h = (h ^ round(0, v4)) * P1 + P4;
  } else {
    h = P5;
  }
  h += bytes;
  for (; i + 2 <= n; i += 2) {
    h ^= round(0, lane64(i));
    h = rotl(h, 27) * P1 + P4;
  }
  if (i < n) {
    h ^= (uint64_t)(uint32_t)tokens[i] * P1;
    h = rotl(h, 23) * P2 + P3;
  }
  h ^= h >> 33;
  h *= P2;
  h ^= h >> 29;
  h *= P3;
  h ^= h >> 32;
  return h;
}

int32_t bicache_is_refresh_step(int32_t t, int32_t delta) {
  if (t < 1 || delta < 1) return -1;
  return (t - 1) % delta == 0 ? 1 : 0;
}

int32_t bicache_lookup_prefix(const bicache_ctx* ctx, uint64_t key, int32_t* prefix_id, int32_t* m) {
  if (!ctx) return BICACHE_ERR_INVALID;
  auto found = ctx->by_key.find(key);
  if (found == ctx->by_key.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown key");
  if (prefix_id) *prefix_id = found->second->id;
  if (m) *m = found->second->m;
  return BICACHE_OK;
}

int32_t bicache_prefix_pages_layer(const bicache_ctx* ctx, int32_t prefix_id, int32_t layer, int32_t* pages_out,
                                   int32_t cap, int32_t* n) {
  if (!ctx) return BICACHE_ERR_INVALID;
  auto found = ctx->by_id.find(prefix_id);
  if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
  const PrefixEntry& e = *found->second;
  if (layer < 0) layer = e.first_layer;
  if (layer < e.first_layer || layer >= ctx->cfg.num_layers)
    return fail(ctx, BICACHE_ERR_INVALID, "the prefix owns no pages in this layer");
  const std::vector<int32_t>& pl = pages_of(e, layer);
  if (n) *n = (int32_t)pl.size();
  if (pages_out) {
    if (cap < (int32_t)pl.size()) return fail(ctx, BICACHE_ERR_INVALID, "pages_out too small");
    std::copy(pl.begin(), pl.end(), pages_out);
  }
  return BICACHE_OK;
}

int32_t bicache_prefix_pages(const bicache_ctx* ctx, int32_t prefix_id, int32_t* pages_out, int32_t cap,
                             int32_t* n) {
  return bicache_prefix_pages_layer(ctx, prefix_id, -1, pages_out, cap, n);
}

int32_t bicache_reuse_depth(const bicache_ctx* ctx, int32_t R, const int32_t* prefix_len,
                            const int32_t* nonshared_len, int32_t* depth_out) {
  if (!ctx || R < 0 || (R > 0 && (!prefix_len || !nonshared_len || !depth_out)))
    return fail(ctx, BICACHE_ERR_INVALID, "bad arguments");
  if (ctx->depth_table.size() != 101) return fail(ctx, BICACHE_ERR_INVALID, "no depth table installed");
  for (int i = 0; i < R; ++i)
    if (nonshared_len[i] < 0) return fail(ctx, BICACHE_ERR_INVALID, "negative non-shared length");
  for (int i = 0; i < R; ++i) {
    const int64_t m = prefix_len[i], n = nonshared_len[i];
    int32_t b = 0;
    if (m > 0) {
      const int64_t idx = (100 * m) / (m + n);
      b = ctx->depth_table[(size_t)idx];
      b = std::max<int32_t>(0, std::min<int32_t>(ctx->cfg.num_layers, b));
    }
    depth_out[i] = b;
  }
  return BICACHE_OK;
}

int32_t bicache_attend(bicache_ctx* ctx, int32_t layer, int32_t R, const int32_t* prefix_id,
                       const int64_t* row_off, const int32_t* seqlen, const void* q, const void* k,
                       const void* v, int64_t q_row_stride, int64_t kv_row_stride, void* out,
                       int64_t out_row_stride, float* lse_out, float softmax_scale, void* stream) {
  return run_attention(ctx, 0, layer, R, prefix_id, row_off, seqlen, q, k, v, q_row_stride, kv_row_stride, out,
                       out_row_stride, lse_out, softmax_scale, stream);
}

int32_t bicache_attend_full(bicache_ctx* ctx, int32_t layer, int32_t R, const int64_t* row_off,
                            const int32_t* seqlen, const void* q, const void* k, const void* v,
                            int64_t q_row_stride, int64_t kv_row_stride, void* out, int64_t out_row_stride,
                            float* lse_out, float softmax_scale, void* stream) {
  return run_attention(ctx, 1, layer, R, nullptr, row_off, seqlen, q, k, v, q_row_stride, kv_row_stride, out,
                       out_row_stride, lse_out, softmax_scale, stream);
}

int32_t bicache_attend_layer(bicache_ctx* ctx, int32_t layer, int32_t R, const int32_t* depth,
                             const int32_t* prefix_id, const int64_t* row_off, const int32_t* seqlen,
                             const void* q, const void* k, const void* v, int64_t q_row_stride,
                             int64_t kv_row_stride, void* out, int64_t out_row_stride, float* lse_out,
                             float softmax_scale, void* stream) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (R < 0 || (R > 0 && (!depth || !prefix_id || !row_off || !seqlen)))
    return fail(ctx, BICACHE_ERR_INVALID, "null metadata array");
  // Layer-partitioned dispatch: request i reuses the cached prefix in this layer iff layer < depth[i].
  std::vector<int32_t> r_pid, r_len, f_len;
  std::vector<int64_t> r_off, f_off;
  for (int i = 0; i < R; ++i) {
    if (seqlen[i] < 0 || row_off[i] < 0) return fail(ctx, BICACHE_ERR_INVALID, "negative length or offset");
    if (layer < depth[i] && prefix_id[i] >= 0) {
      auto found = ctx->by_id.find(prefix_id[i]);
      if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
      const int32_t m = found->second->m;
      if (seqlen[i] < m) return fail(ctx, BICACHE_ERR_INVALID, "request shorter than its prefix");
      r_pid.push_back(prefix_id[i]);
      r_off.push_back(row_off[i] + m);
      r_len.push_back(seqlen[i] - m);
    } else {
      f_off.push_back(row_off[i]);
      f_len.push_back(seqlen[i]);
    }
  }
  // Both halves are validated and their schedules prepared before either is launched, so that an error
  // the host can detect leaves the outputs untouched.
  ctx->use_counter++;
  PreparedCall pr, pf;
  if (!r_len.empty()) {
    for (size_t i = 1; i < r_pid.size(); ++i)
      if (r_pid[i] != r_pid[i - 1] &&
          std::find(r_pid.begin(), r_pid.begin() + i, r_pid[i]) != r_pid.begin() + i)
        return fail(ctx, BICACHE_ERR_INVALID, "requests of one prefix are not contiguous");
    const int32_t st = prepare_attention(ctx, 0, layer, (int32_t)r_len.size(), r_pid.data(), r_off.data(),
                                         r_len.data(), q, k, v, q_row_stride, kv_row_stride, out, out_row_stride,
                                         lse_out, softmax_scale, stream, &pr);
    if (st != BICACHE_OK) return st;
  }
  if (!f_len.empty()) {
    const int32_t st = prepare_attention(ctx, 1, layer, (int32_t)f_len.size(), nullptr, f_off.data(), f_len.data(),
                                         q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                                         softmax_scale, stream, &pf);
    if (st != BICACHE_OK) return st;
  }
  int32_t st = launch_attention(ctx, pr, layer, q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                                softmax_scale, stream);
  if (st != BICACHE_OK) return st;
  return launch_attention(ctx, pf, layer, q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                          softmax_scale, stream);
}

int32_t bicache_attend_step(bicache_ctx* ctx, int32_t layer, int32_t t, int32_t delta, int32_t R,
                            const int32_t* depth, const int32_t* shared_id, const int32_t* private_id,
                            const int64_t* row_off, const int32_t* seqlen, const void* q, const void* k,
                            const void* v, int64_t q_row_stride, int64_t kv_row_stride, void* out,
                            int64_t out_row_stride, float* lse_out, float softmax_scale, void* stream) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (R < 0 || (R > 0 && (!depth || !shared_id || !private_id || !row_off || !seqlen)))
    return fail(ctx, BICACHE_ERR_INVALID, "null metadata array");
  const int refresh = bicache_is_refresh_step(t, delta);
  if (refresh < 0) return fail(ctx, BICACHE_ERR_INVALID, "t and delta start at 1");
  if (layer < 0 || layer >= ctx->cfg.num_layers) return fail(ctx, BICACHE_ERR_INVALID, "layer out of range");
  // Per request: which cached prefix (if any) its suffix rows read in this layer at this step.
  struct Reuse { int32_t pid; int64_t off; int32_t len; int order; };
  std::vector<Reuse> reuse;
  std::vector<int32_t> f_len, upd_id;
  std::vector<int64_t> f_off, upd_off;
  std::unordered_map<int32_t, int> first_seen;
  for (int i = 0; i < R; ++i) {
    if (seqlen[i] < 0 || row_off[i] < 0) return fail(ctx, BICACHE_ERR_INVALID, "negative length or offset");
    int32_t pid = -1;
    if (layer < depth[i] && shared_id[i] >= 0) pid = shared_id[i];
    else if (private_id[i] >= 0 && !refresh) pid = private_id[i];
    if (pid >= 0) {
      auto found = ctx->by_id.find(pid);
      if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
      const int32_t m = found->second->m;
      if (seqlen[i] < m) return fail(ctx, BICACHE_ERR_INVALID, "request shorter than its prefix");
      const int order = first_seen.emplace(pid, (int)first_seen.size()).first->second;
      reuse.push_back(Reuse{pid, row_off[i] + m, seqlen[i] - m, order});
    } else {
      f_off.push_back(row_off[i]);
      f_len.push_back(seqlen[i]);
      if (private_id[i] >= 0) {
        auto found = ctx->by_id.find(private_id[i]);
        if (found == ctx->by_id.end()) return fail(ctx, BICACHE_ERR_NOTFOUND, "unknown or evicted prefix id");
        if (seqlen[i] < found->second->m) return fail(ctx, BICACHE_ERR_INVALID, "request shorter than its prefix");
        upd_id.push_back(private_id[i]);
        upd_off.push_back(row_off[i]);
      }
    }
  }
  // requests of one prefix side by side, in order of first appearance
  std::stable_sort(reuse.begin(), reuse.end(), [](const Reuse& a, const Reuse& b) { return a.order < b.order; });
  // Everything the host can check comes before the first launch: both attention calls are validated and
  // prepared, and the arguments of the layer updates are the same tensors and strides.
  ctx->use_counter++;
  PreparedCall pr, pf;
  std::vector<int32_t> r_pid, r_len;
  std::vector<int64_t> r_off;
  if (!reuse.empty()) {
    for (const Reuse& r : reuse) {
      r_pid.push_back(r.pid);
      r_off.push_back(r.off);
      r_len.push_back(r.len);
    }
    const int32_t st = prepare_attention(ctx, 0, layer, (int32_t)r_len.size(), r_pid.data(), r_off.data(),
                                         r_len.data(), q, k, v, q_row_stride, kv_row_stride, out, out_row_stride,
                                         lse_out, softmax_scale, stream, &pr);
    if (st != BICACHE_OK) return st;
  }
  if (!f_len.empty()) {
    const int32_t st = prepare_attention(ctx, 1, layer, (int32_t)f_len.size(), nullptr, f_off.data(), f_len.data(),
                                         q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                                         softmax_scale, stream, &pf);
    if (st != BICACHE_OK) return st;
  }
  int32_t st = launch_attention(ctx, pr, layer, q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                                softmax_scale, stream);
  if (st != BICACHE_OK) return st;
  st = launch_attention(ctx, pf, layer, q, k, v, q_row_stride, kv_row_stride, out, out_row_stride, lse_out,
                        softmax_scale, stream);
  if (st != BICACHE_OK) return st;
  // refresh: the prefix rows just used become the kept K/V of this layer (Eq. 5, first case)
  for (size_t i = 0; i < upd_id.size(); ++i) {
    const char* kp = static_cast<const char*>(k) + upd_off[i] * kv_row_stride * ctx->esize;
    const char* vp = static_cast<const char*>(v) + upd_off[i] * kv_row_stride * ctx->esize;
    st = bicache_update_prefix_layer(ctx, upd_id[i], layer, kp, vp, kv_row_stride, stream);
    if (st != BICACHE_OK) return st;
  }
  return BICACHE_OK;
}

int32_t bicache_device_status(bicache_ctx* ctx, void* stream, int32_t clear) {
  if (!ctx) return BICACHE_ERR_INVALID;
  if (ctx->host_only) return BICACHE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cudaStreamSynchronize(s) != cudaSuccess) return fail(ctx, BICACHE_ERR_CUDA, "stream synchronize failed");
  int word = 0;
  if (cudaMemcpy(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess)
    return fail(ctx, BICACHE_ERR_CUDA, "status read failed");
  if (clear && word != 0) cudaMemset(ctx->d_status, 0, kStatusBytes);
  if (word == kDevOk) return BICACHE_OK;
  if (word == kDevTimeout) return fail(ctx, BICACHE_ERR_TIMEOUT, "device-side wait gave up");
  return fail(ctx, BICACHE_ERR_CUDA, "a kernel reported an internal error");
}

int32_t bicache_set_wait_budget(bicache_ctx* ctx, int64_t sm_cycles) {
  if (!ctx || sm_cycles < 0) return BICACHE_ERR_INVALID;
  ctx->wait_cycles = sm_cycles;
  return BICACHE_OK;
}

int64_t bicache_launch_count(const bicache_ctx* ctx) { return ctx ? ctx->launches : 0; }

int64_t bicache_schedule_uploads(const bicache_ctx* ctx) { return ctx ? ctx->schedule_uploads : 0; }

int32_t bicache_last_attention_kernel(const bicache_ctx* ctx) { return ctx ? ctx->last_kernel : 0; }

const char* bicache_last_error(const bicache_ctx* ctx) { return ctx ? ctx->last_error.c_str() : "null context"; }

}  // extern "C"
