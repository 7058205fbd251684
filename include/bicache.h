/*
 * bicache.h - C ABI of the BiCache attention hot path for NVIDIA B200 (sm_100a).
 *
 * BiCache serves diffusion language models with a shared-prefix KV cache: in
 * the shallow layers 1..b of a request the cached KVs of the shared prefix are
 * reused (Eq. 4), in the deep layers they are recomputed (Sec. 5.2).  This
 * library is the attention of one denoising step under that scheme:
 *
 *   bicache_put_prefix    KV store H: insert the prefix KVs of all L layers
 *                         under the prefix's key (Sec. 5.2, the miss case),
 *                         paged, with first-in-first-out eviction
 *                         (implementation appendix).
 *   bicache_reuse_depth   r = shared-prefix tokens / all tokens of the input
 *                         string -> lookup table T -> shallow depth b
 *                         (Sec. 5.1, Sec. 5.2 first paragraph).
 *   bicache_attend        layers l < b: suffix queries attend, without a
 *                         causal mask, over [cached prefix K/V | own suffix
 *                         K/V] (Eq. 2 with the key set of Eq. 4).
 *   bicache_attend_full   layers l >= b: full bidirectional attention of a
 *                         request over its own freshly computed rows (Eq. 2).
 *
 * General rules
 *   - Every function returns a bicache_status.  Nothing aborts, throws or
 *     traps the device.  Host-detectable errors return before any launch and
 *     leave all outputs untouched.
 *   - The caller owns every device buffer (pools, workspace, tensors) and the
 *     CUDA stream.  The library allocates no device memory; it owns host
 *     bookkeeping only (key map, FIFO list, free-page queue, schedules).
 *   - Pointers documented "device" must be device pointers on cfg.device and
 *     16-byte aligned; row strides are in elements and must keep every row
 *     16-byte aligned.  Pointers documented "host" are ordinary host memory.
 *   - Calls enqueue work on `stream` and return without synchronising (except
 *     bicache_destroy and bicache_device_status).  One stream per context at a
 *     time; a context is not thread-safe.  Evicting a prefix while work that
 *     reads it is still enqueued is safe only because everything is ordered on
 *     that one stream.
 *   - Layers are 0-based: layer l reuses the cache iff l < depth (the paper's
 *     1-based l <= b).
 */
#ifndef BICACHE_H_
#define BICACHE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct bicache_ctx bicache_ctx;

typedef enum {
  BICACHE_OK = 0,
  BICACHE_ERR_INVALID = 1,     /* bad argument (null/unaligned pointer, range, ungrouped ids, ...) */
  BICACHE_ERR_NOMEM = 2,       /* prefix larger than the pool, or workspace too small             */
  BICACHE_ERR_NOTFOUND = 3,    /* unknown or evicted key / prefix id                              */
  BICACHE_ERR_CUDA = 4,        /* a CUDA runtime call failed                                      */
  BICACHE_ERR_TIMEOUT = 5,     /* a bounded device-side wait gave up (see bicache_device_status)  */
  BICACHE_ERR_UNSUPPORTED = 6  /* dtype / head_dim / page size outside what is built              */
} bicache_status;

enum { BICACHE_F32 = 0, BICACHE_BF16 = 1 };

/* Which kernels serve bf16 head_dim-128 attention.  AUTO picks the tensor-core
 * path when it applies; SIMT forces the plain CUDA-core kernels (used as an
 * on-device cross-check).  fp32 and other head dims always run SIMT.
 * TENSOR_PAIRS is TENSOR with bicache_attend_full on the variant of the tensor-core
 * kernel that runs on pairs of SMs (one MMA over 256 query rows, each SM staging half
 * of every K/V tile); it gives the same bits as the default kernel and is slower, so
 * AUTO never picks it (it exists as a measured alternative and a cross-check). */
enum { BICACHE_PATH_AUTO = 0, BICACHE_PATH_SIMT = 1, BICACHE_PATH_TENSOR = 2, BICACHE_PATH_TENSOR_PAIRS = 3 };

typedef struct {
  int32_t num_layers;        /* L >= 1                                                         */
  int32_t num_q_heads;       /* Hq, a multiple of num_kv_heads                                 */
  int32_t num_kv_heads;      /* Hkv                                                            */
  int32_t head_dim;          /* D: 128 for the tensor-core path; any multiple of 32 up to 256
                                on the SIMT path                                               */
  int32_t page_size;         /* tokens per page; must be 16                                    */
  int32_t num_pages;         /* pages per layer (see layer_pages for layers that hold fewer)   */
  int32_t dtype;             /* BICACHE_F32 or BICACHE_BF16: type of q/k/v/out and the pools   */
  int32_t device;            /* CUDA device ordinal.  A negative value creates a host-only
                                context: the store's bookkeeping and the depth rule work (pools
                                and workspace may be NULL, put_prefix moves no data), the
                                attention calls return UNSUPPORTED.  It exists so that the host
                                logic can be exercised on a machine without a GPU; it computes
                                nothing.                                                       */
  const int32_t* initial_free_order; /* host, num_pages entries, a permutation of 0..num_pages-1
                                giving the initial order of the free-page queue; NULL = 0,1,2,...
                                Read during bicache_create only.                               */
  const int32_t* layer_pages; /* host, num_layers entries, or NULL: pages of each layer's pool,
                                1 .. num_pages (NULL: num_pages everywhere).  Shallow layers may hold
                                fewer: the kept deep-layer prefixes of Eq. 5 own no pages there.
                                Layer l's free queue starts as the pages below its capacity in the
                                initial order.  Read during bicache_create only.                 */
  void* k_pool;              /* device, bicache_pool_bytes() bytes, caller-owned               */
  void* v_pool;              /* device, same size                                              */
  void* workspace;           /* device scratch, caller-owned, 256-byte aligned                 */
  size_t workspace_bytes;    /* >= bicache_workspace_bytes() for the batches to be run         */
} bicache_config;

/* Bytes of ONE pool (K or V): (sum over the layers of their pages) * Hkv * page_size * D elements,
 * the layers one after the other.  The order of elements inside a page is private to the library:
 * only the library writes pools.  0 for an invalid configuration. */
size_t bicache_pool_bytes(const bicache_config* cfg);

/* Workspace needed to run batches of at most max_requests requests and max_total_rows query rows
 * per call (bicache_attend: suffix rows; bicache_attend_full: all rows).  Besides the fixed areas
 * (status, partial results of key-split calls, page-list staging) it holds the schedule arena: the
 * device-resident descriptions of the batches seen so far, kept so that the layers of a denoising step
 * and the following steps upload nothing.  The size asked for holds min(2 L + 4, 72) schedules of the
 * largest batch; a smaller workspace still works as long as two schedules fit (more uploads). */
size_t bicache_workspace_bytes(const bicache_config* cfg, int64_t max_total_rows, int32_t max_requests);

/* Create a context.  Clears the library's part of the workspace with a synchronous memset.
 * INVALID for inconsistent sizes/pointers, UNSUPPORTED for page_size != 16 or an unsupported
 * dtype/head_dim, NOMEM if the workspace cannot hold even an empty batch. */
int32_t bicache_create(const bicache_config* cfg, bicache_ctx** out);

/* Synchronises the device and frees host state.  Device buffers stay the caller's. */
int32_t bicache_destroy(bicache_ctx* ctx);

/* Select the kernel family (BICACHE_PATH_*).  UNSUPPORTED if TENSOR is asked for a
 * dtype/head_dim it does not cover. */
int32_t bicache_set_path(bicache_ctx* ctx, int32_t path);

/* Install the lookup table T (Sec. 5.1): table[idx] is the shallow depth for ratio bin
 * idx = floor(100 * m / (m + n)), idx in 0..100.  n must be 101.  Host pointer; copied. */
int32_t bicache_set_depth_table(bicache_ctx* ctx, const int32_t* table, int32_t n);

/* (1) KV store insert (Sec. 5.2).  k, v: device, [L][m][Hkv][D] with `layer_stride` elements
 * between layers (>= m*Hkv*D), rows dense.  m >= 1.
 *   key present with the same m : hit, nothing is written, *was_hit = 1.
 *   key present with another m  : INVALID.
 *   ceil(m/16) > a layer's pages : NOMEM, nothing evicted.
 *   otherwise: every layer has its own free queue.  Evict whole prefixes, oldest insertion first
 *   (hits do not refresh age), until every layer has enough free pages (an evicted prefix's pages
 *   join the tail of their layer's queue in page-table order), take ceil(m/16) pages from the head of
 *   every layer's queue, and enqueue the scatter of all L layers on `stream`.  The caller may free
 *   k, v once the stream has passed this point.  While every prefix owns all layers (no
 *   bicache_reserve_prefix_layers with a first layer > 0, no layer_pages) the queues move in
 *   lockstep and a prefix has the same page list in every layer.
 * prefix_id (host, required) receives an id that is never reused.  was_hit (host, optional).
 * pages_out (host, optional, capacity pages_cap) receives the page ids of layer 0 in token order;
 * INVALID if pages_cap is too small (checked before anything changes). */
int32_t bicache_put_prefix(bicache_ctx* ctx, uint64_t key, int32_t m, const void* k, const void* v,
                           int64_t layer_stride, void* stream,
                           int32_t* prefix_id, int32_t* was_hit, int32_t* pages_out, int32_t pages_cap);

/* k = h(p) (Sec. 5.2): the 64-bit identifier of a tokenised prefix, for use as the `key` of the store
 * calls.  XXH64 with seed 0 over the n token ids taken as little-endian 32-bit integers (the paper's
 * implementation hashes the token id sequence with xxHash).  Host array, no context; n = 0 gives the
 * hash of the empty input; a negative n or a null array with n > 0 gives 0. */
uint64_t bicache_hash_tokens(const int32_t* tokens, int64_t n);

/* KV store lookup (Sec. 5.2 "On a cache hit").  NOTFOUND if the key is absent or evicted. */
int32_t bicache_lookup_prefix(const bicache_ctx* ctx, uint64_t key, int32_t* prefix_id, int32_t* m);

/* Page list of a live prefix in its first layer, in token order.  *n receives the page count; pages_out
 * (host) may be NULL to query the count only.  NOTFOUND for an evicted id, INVALID if cap is too small. */
int32_t bicache_prefix_pages(const bicache_ctx* ctx, int32_t prefix_id, int32_t* pages_out, int32_t cap,
                             int32_t* n);

/* The same for one layer (a negative layer: the prefix's first layer).  INVALID if the prefix owns no
 * pages in that layer. */
int32_t bicache_prefix_pages_layer(const bicache_ctx* ctx, int32_t prefix_id, int32_t layer, int32_t* pages_out,
                                   int32_t cap, int32_t* n);

/* (2) Per-request shallow depth (Sec. 5.1/5.2).  Host arrays of length R.  prefix_len[i] = m_i
 * shared-prefix tokens, nonshared_len[i] = n_i = every other token of the input string (prompt
 * and all mask positions).  depth_out[i] = clamp(T[floor(100 m / (m + n))], 0, L); m <= 0 gives 0.
 * Pure integer arithmetic, no device work.  INVALID if no table is installed or n_i < 0. */
int32_t bicache_reuse_depth(const bicache_ctx* ctx, int32_t R, const int32_t* prefix_len,
                            const int32_t* nonshared_len, int32_t* depth_out);

/* (3) Shallow-layer attention of a ragged batch grouped by prefix, one layer (Eq. 2 + Eq. 4).
 * Host metadata arrays of length R:
 *   prefix_id[i]  live prefix id, or -1 for "no prefix"; equal ids must be contiguous (INVALID
 *                 otherwise); NOTFOUND for an evicted id.
 *   row_off[i]    first row of request i's suffix inside q, k, v, out, lse_out.
 *   seqlen[i]     n_i >= 0 suffix rows (0 contributes nothing).
 * Device tensors: q, out [rows][Hq][D] with q_row_stride / out_row_stride elements between rows;
 * k, v [rows][Hkv][D] with kv_row_stride.  Heads are dense within a row.  Query head h reads KV
 * head h / (Hq / Hkv).  lse_out: device fp32 [rows][Hq] (dense) or NULL; natural log of the sum of
 * exp(softmax_scale * q.k) over all keys.  Each suffix row i,a attends over the prefix's m cached
 * keys of `layer` and the request's own n_i suffix keys (itself included), no mask.  Only rows that
 * belong to a request are written.  out is rounded to the context dtype (round to nearest even). */
int32_t bicache_attend(bicache_ctx* ctx, int32_t layer, int32_t R, const int32_t* prefix_id,
                       const int64_t* row_off, const int32_t* seqlen,
                       const void* q, const void* k, const void* v,
                       int64_t q_row_stride, int64_t kv_row_stride,
                       void* out, int64_t out_row_stride, float* lse_out,
                       float softmax_scale, void* stream);

/* (4) Deep-layer fallback: full bidirectional attention (Eq. 2) of each request over its own
 * seqlen[i] = N_i rows starting at row_off[i]; every row is a query.  Same tensor conventions as
 * bicache_attend; `layer` is only range-checked (no cache is read). */
int32_t bicache_attend_full(bicache_ctx* ctx, int32_t layer, int32_t R,
                            const int64_t* row_off, const int32_t* seqlen,
                            const void* q, const void* k, const void* v,
                            int64_t q_row_stride, int64_t kv_row_stride,
                            void* out, int64_t out_row_stride, float* lse_out,
                            float softmax_scale, void* stream);

/* Layer-partitioned dispatch of one layer (Sec. 5.2: the per-layer test l <= b of the online phase):
 * request i, whose whole input (prefix rows, then suffix rows) occupies seqlen[i] = N_i rows from
 * row_off[i], goes through bicache_attend on its suffix rows (row_off[i] + m_i, N_i - m_i rows, m_i =
 * length of prefix_id[i]) if layer < depth[i] and prefix_id[i] >= 0, and through bicache_attend_full
 * on all its rows otherwise.  depth, prefix_id, row_off, seqlen: host arrays of length R; the reusing
 * requests' prefix ids must be grouped.  Tensor arguments as for bicache_attend.  Outputs: suffix rows
 * of reusing requests, all rows of the others.  INVALID if a reusing request is shorter than its
 * prefix; other errors as for the two calls.  Both halves are validated and their schedules placed in the
 * workspace before either is launched: an error the host can detect (bad arguments, an evicted id, a
 * schedule that does not fit the workspace) leaves out and lse_out untouched and launches no kernel. */
int32_t bicache_attend_layer(bicache_ctx* ctx, int32_t layer, int32_t R, const int32_t* depth,
                             const int32_t* prefix_id, const int64_t* row_off, const int32_t* seqlen,
                             const void* q, const void* k, const void* v,
                             int64_t q_row_stride, int64_t kv_row_stride,
                             void* out, int64_t out_row_stride, float* lse_out,
                             float softmax_scale, void* stream);

/* ---- Deep layers: reuse within a request with periodic refresh (Sec. 5.2, Eq. 5) ------------------
 * In layers l >= depth a request does not read the shared cache; it keeps the prefix K/V it computed
 * itself and reuses them across denoising steps, recomputing them every delta steps.  The kept K/V
 * live in the same paged store under a per-request key ("private" prefix). */

/* Eq. 5's condition for the 1-based denoising step t: 1 if (t - 1) mod delta == 0 (recompute), 0 if
 * not (reuse the kept K/V), -1 if t < 1 or delta < 1.  Pure integer, no context. */
int32_t bicache_is_refresh_step(int32_t t, int32_t delta);

/* Allocate pages for a prefix of m tokens under `key` without writing K/V: same hit / miss / FIFO
 * eviction rules, outputs and errors as bicache_put_prefix, no kernel is launched.  The content of
 * the pages is unspecified until bicache_update_prefix_layer has written a layer. */
int32_t bicache_reserve_prefix(bicache_ctx* ctx, uint64_t key, int32_t m, int32_t* prefix_id,
                               int32_t* was_hit, int32_t* pages_out, int32_t pages_cap);

/* The same for a prefix that only the layers first_layer .. L-1 keep (Eq. 5: a request's own prefix K/V
 * are kept in the layers past its shallow depth, so first_layer = depth[i]): pages are taken from, and
 * on eviction returned to, the queues of those layers only; the shallow layers' pages stay free for
 * other prefixes.  pages_out receives the list of layer first_layer.  A hit needs the same m and the
 * same first_layer (INVALID otherwise).  Every call that names a layer for this prefix (update, read,
 * project, the attention calls) answers INVALID for a layer below first_layer. */
int32_t bicache_reserve_prefix_layers(bicache_ctx* ctx, uint64_t key, int32_t m, int32_t first_layer,
                                      int32_t* prefix_id, int32_t* was_hit, int32_t* pages_out,
                                      int32_t pages_cap);

/* Overwrite ONE layer of an existing prefix (Eq. 5, refresh step: the kept K/V become the ones just
 * computed).  k, v: device, rows [m][Hkv][D] of the context's dtype, `kv_row_stride` elements between
 * consecutive rows (so k may point at the request's first row inside a packed [rows][Hkv][D] tensor),
 * 16-byte aligned rows.  Copies on `stream`; unused slots of the last page are zero-filled.
 * NOTFOUND for an unknown or evicted id, INVALID for a bad layer, pointer or stride. */
int32_t bicache_update_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* k,
                                    const void* v, int64_t kv_row_stride, void* stream);

/* Read ONE layer of a stored prefix back as dense rows (the inverse of bicache_update_prefix_layer; the
 * store's in-page element order is private, this call is how a caller sees the values): k_out, v_out
 * device, rows [m][Hkv][D] of the context's dtype, `kv_row_stride` elements between rows, 16-byte
 * aligned.  Copies on `stream`; bit-exact.  NOTFOUND / INVALID as for the update call. */
int32_t bicache_read_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, void* k_out, void* v_out,
                                  int64_t kv_row_stride, void* stream);

/* Compute ONE layer's prefix K/V from the layer's input hidden states and write them into the pages
 * of an existing prefix (Eq. 1: k = W^K h, v = W^V h per token, feeding the store H[k] of Sec. 5.2):
 *   K[t][o] = sum_c h[t][c] * w_k[o][c],  V likewise,  o = head * D + dim,
 * bf16 inputs, fp32 accumulation, one rounding to bf16.  h: device, [m][d_model] bf16 with
 * `h_row_stride` elements between rows; w_k, w_v: device, [Hkv * D][d_model] bf16, rows contiguous.
 * All 16-byte aligned; d_model and h_row_stride multiples of 8.  The dense K/V never exist in memory:
 * the kernel (tensor cores) writes page images directly; unused slots of the last page become zero.
 * Runs on `stream`.  UNSUPPORTED unless the context is bf16 with head_dim 128; NOTFOUND / INVALID as
 * for the update call; a device-side wait that gives up is reported by bicache_device_status. */
int32_t bicache_project_prefix_layer(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* h,
                                     int64_t h_row_stride, const void* w_k, const void* w_v, int32_t d_model,
                                     void* stream);

/* The same with a rotary position encoding of the KEYS applied before they are stored (Eq. 1 has no
 * position encoding and the paper names none; the attention calls take K as it is cached, so a model
 * with rotary keys caches them rotated).  rope_cos_sin: device, fp32 [m][64][2]: for token t and pair d
 * the cosine and the sine of the token's angle; the pair is head dims (d, d + 64) of every KV head
 * (the half-split pairing):  k'[d] = k[d] cos - k[d + 64] sin,  k'[d + 64] = k[d + 64] cos + k[d] sin,
 * in fp32 on the accumulator, before the one rounding to bf16.  The table is the caller's (base,
 * scaling and position offset are the model's business); 16-byte aligned.  NULL: no rotation, the call
 * above.  Values are not rotated.  Errors as above. */
int32_t bicache_project_prefix_layer_rope(bicache_ctx* ctx, int32_t prefix_id, int32_t layer, const void* h,
                                          int64_t h_row_stride, const void* w_k, const void* w_v, int32_t d_model,
                                          const float* rope_cos_sin, void* stream);

/* One layer of denoising step t with both kinds of reuse.  Request i owns seqlen[i] = N_i rows from
 * row_off[i] (prefix rows first).  Per request, in this order:
 *   layer < depth[i] and shared_id[i] >= 0      -> suffix rows attend over [shared cached prefix | own
 *                                                  suffix]                              (Eq. 4);
 *   else private_id[i] >= 0 and not a refresh step -> suffix rows attend over [kept prefix K/V of
 *                                                  private_id[i] | own suffix]          (Eq. 5, reuse);
 *   else                                         -> full attention over all N_i rows; on a refresh
 *                                                  step with private_id[i] >= 0, rows 0 .. m_i of k, v
 *                                                  then replace the kept K/V of this layer
 *                                                                                       (Eq. 5, recompute).
 * depth, shared_id, private_id, row_off, seqlen: host arrays of length R (requests of one shared prefix
 * need not be contiguous here: the call groups them).  Tensor arguments, outputs and errors as for
 * bicache_attend_layer; INVALID also if t < 1 or delta < 1.  Everything the host can check (both
 * attention calls and the ids, lengths and strides of the layer updates) is checked, and both schedules
 * are placed in the workspace, before the first launch. */
int32_t bicache_attend_step(bicache_ctx* ctx, int32_t layer, int32_t t, int32_t delta, int32_t R,
                            const int32_t* depth, const int32_t* shared_id, const int32_t* private_id,
                            const int64_t* row_off, const int32_t* seqlen,
                            const void* q, const void* k, const void* v,
                            int64_t q_row_stride, int64_t kv_row_stride,
                            void* out, int64_t out_row_stride, float* lse_out,
                            float softmax_scale, void* stream);

/* ---- Profiler pieces (Sec. 4.1 Eq. 3, Sec. 4.2, Sec. 5.1) -------------------------------------------
 * How close the cached K/V of a prefix are to the K/V a request computes for the same tokens, per
 * layer; the depth that allows under a threshold; the lookup table from many profiled requests. */

/* sim_out[l] = cos(KV$_l, KVref_l), l = 0 .. L-1 (Eq. 3): per layer, the cached keys and values of all
 * prefix positions and heads form one vector, the reference ones the other.  k_ref, v_ref: device,
 * [L][m][Hkv][D] of the context's dtype, `layer_stride` elements between layers (m = the prefix's
 * length).  sim_out: HOST array of L floats.  Runs on `stream` and synchronises it before returning
 * (an offline call).  A zero vector on either side gives 0.  Uses the context's workspace as scratch.
 * NOTFOUND for an unknown or evicted id, INVALID for a bad pointer or stride, UNSUPPORTED on a
 * host-only context and for a prefix whose page list differs between layers (profile shared prefixes
 * before any partial-depth reservation, or in a context of their own). */
int32_t bicache_prefix_similarity(bicache_ctx* ctx, int32_t prefix_id, const void* k_ref, const void* v_ref,
                                  int64_t layer_stride, float* sim_out, void* stream);

/* The same reduction without the copy to the host and without the synchronisation: sim_dev is a DEVICE
 * array of L floats, written on `stream`. */
int32_t bicache_prefix_similarity_async(bicache_ctx* ctx, int32_t prefix_id, const void* k_ref,
                                        const void* v_ref, int64_t layer_stride, float* sim_dev, void* stream);

/* *depth = the number of leading layers whose similarity is >= tau (Sec. 4.2: the largest b such that
 * every layer 1 .. b is at or above the threshold; tau = 0.97 in the paper).  Host arrays, no context;
 * a NaN ends the run. */
int32_t bicache_depth_from_similarity(const float* sim, int32_t num_layers, float tau, int32_t* depth);

/* table_out[0..100] from n profiled requests (ratio_idx[i] = floor(100 r_i) in 0..100, depth[i] in
 * 0..num_layers): per ratio bin the mean of the depths, floored; a bin without samples takes the
 * value of the nearest filled bin below it, bins below the first filled one take min(1, num_layers)
 * (Sec. 5.1 "lookup table").  Host arrays, no context; INVALID for values out of range. */
int32_t bicache_build_depth_table(const int32_t* ratio_idx, const int32_t* depth, int32_t n,
                                  int32_t num_layers, int32_t* table_out);

/* Synchronises `stream` and returns the sticky device status: OK, or TIMEOUT if a kernel gave up
 * on a bounded wait (its outputs are then undefined), or CUDA for a runtime error.  `clear` != 0
 * resets the word. */
int32_t bicache_device_status(bicache_ctx* ctx, void* stream, int32_t clear);

/* Budget, in SM clock cycles, of every device-side wait of the tensor-core kernel (on a barrier that a
 * copy, an MMA or another warp completes).  A wait that exceeds it gives up: the CTA drains its copies
 * and MMAs, releases its tensor memory and exits, and bicache_device_status reports TIMEOUT; outputs of
 * that call are then undefined, the context stays usable once the status is cleared.  0 restores the
 * default (about 0.2 s).  A tiny budget makes ordinary waits run out: that is how the tests exercise
 * the give-up path without any barrier that could never complete.  INVALID for a negative value. */
int32_t bicache_set_wait_budget(bicache_ctx* ctx, int64_t sm_cycles);

/* Allocation-free full attention of ONE request (the paper has no counterpart: this entry point
 * exists for callers, not for the method).
 *
 * Some callers cannot allocate device memory where they need attention: code embedded in another
 * framework's fixed memory plan, a serving loop that must stay clear of the allocator once it is
 * running, a process whose GPU budget was handed out before this library was loaded.  The calls
 * above need a context and a caller-allocated workspace; this one needs neither.  Its scratch
 * (partial results of BICACHE_STATIC_KEY_SPLITS key ranges) is a fixed array inside the library's
 * device image: 4096 x 4 x 129 floats = 8,454,144 bytes (8.06 MiB) on every GPU that runs this entry
 * point, held until the process exits.  The call itself allocates and frees nothing, on the host or
 * on the device.  One caveat for callers with a fixed memory budget: CUDA loads a library's device
 * code lazily, so the FIRST call on a device is when the driver loads this entry point's module and
 * backs the array; make that call at start-up, where an out-of-memory answer (BICACHE_ERR_CUDA) can
 * still be handled, and count the 8.06 MiB into the budget.
 *
 * Computes what bicache_attend_full computes for a single request occupying rows 0..n_rows-1:
 * every row attends, without a mask, over all n_rows keys.  dtype: BICACHE_F32 or BICACHE_BF16;
 * head_dim: 32, 64, 96 or 128; q, out: device [n_rows][Hq][D]; k, v: device [n_rows][Hkv][D]; row
 * strides in elements; heads dense within a row.  Runs on the current device, on `stream`.
 *   NOMEM        n_rows * num_q_heads > BICACHE_STATIC_MAX_ROW_HEADS (the array's capacity)
 *   UNSUPPORTED  dtype or head_dim outside the list above
 *   INVALID      null pointers, bad strides or head counts
 * The first call on each device looks up the array's device address (a host-side set-up step that
 * enqueues nothing and is cached in plain, unsynchronised host state: make the first call from one
 * thread, before starting any stream capture, and do not call again on a device after resetting it).  All calls on a
 * device share the one array and every call overwrites the part it uses, so nothing has to be
 * cleared between calls - but two calls whose kernels may overlap on the GPU (different streams,
 * or different threads) race on it.  Issue them on one stream, or serialise them yourself. */
#define BICACHE_STATIC_MAX_ROW_HEADS 4096
#define BICACHE_STATIC_KEY_SPLITS 4
int32_t bicache_attend_full_static(int32_t dtype, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim,
                                   int32_t n_rows, const void* q, const void* k, const void* v,
                                   int64_t q_row_stride, int64_t kv_row_stride,
                                   void* out, int64_t out_row_stride, float softmax_scale, void* stream);

/* Number of kernels this context has launched so far (for benchmarks' launch accounting). */
int64_t bicache_launch_count(const bicache_ctx* ctx);

/* Number of schedules this context has uploaded to the device so far.  A batch whose metadata
 * (request offsets, lengths, prefix ids) equals that of an earlier call reuses the cached schedule, so
 * in steady state a denoising step uploads none.  An upload goes through pinned host memory owned by
 * the context and does not make the host wait for the stream. */
int64_t bicache_schedule_uploads(const bicache_ctx* ctx);

/* Which attention kernel the context's last attention call launched (for tests and benchmarks):
 * 0 none yet; BICACHE_KERNEL_SIMT the CUDA-core kernel (fp32, head dims other than 128, forced);
 * BICACHE_KERNEL_TENSOR the tensor-core kernel over two 128-row query tiles per work item;
 * BICACHE_KERNEL_KEY_RANGES the tensor-core kernel for few query rows against a long cached prefix
 * (bicache_attend only; chosen when every request has a cached prefix of at least 1024 tokens and at
 * most 128 * Hkv / Hq suffix tokens, and the call is small enough for the kernel's tables): the group's
 * rows share tiles, the prefix keys are split into ranges over the CTAs, each request's own keys are
 * one more range, and a merge kernel applies the log-sum-exp merge (exact up to rounding);
 * BICACHE_KERNEL_TENSOR_PAIRS the tensor-core kernel on pairs of SMs (BICACHE_PATH_TENSOR_PAIRS). */
enum { BICACHE_KERNEL_SIMT = 1, BICACHE_KERNEL_TENSOR = 2, BICACHE_KERNEL_KEY_RANGES = 3, BICACHE_KERNEL_TENSOR_PAIRS = 4 };
int32_t bicache_last_attention_kernel(const bicache_ctx* ctx);

/* Human-readable text for the last error of this context (host string, valid until next call). */
const char* bicache_last_error(const bicache_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* BICACHE_H_ */
