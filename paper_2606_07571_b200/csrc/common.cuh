// Shared host/device definitions of the BiCache attention library: the device-side batch
// description ("schedule") and the private element order of a cache page.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace bicache {

constexpr int kPageSize = 16;          // tokens per page
constexpr int kTileRows = 256;         // query rows of one work item (two tensor-core M tiles of 128)
constexpr int kTileKeys = 128;         // keys per K/V tile

// One request of a call.  Rows are rows of the caller's q/k/v/out tensors.
struct ReqMeta {
  long long row_off;   // first row of the request (suffix rows for attend, all rows for attend_full)
  int n;               // number of rows = number of queries = number of own keys
  int m;               // cached prefix length (0: none)
  int page_off;        // index of the prefix's first page id inside the schedule's page list
  int tok_off;         // sum of n over the earlier requests of the call (row index into partials)
};

// Up to 256 packed query rows of one request and one KV head, over a range of its keys.  Packed row p of
// a request enumerates (token a, query head j within the KV head's group of G = Hq / Hkv):
// p = a * G + j.  Keys are numbered 0..m-1 (cached prefix) then m..m+n-1 (own rows).
struct WorkItem {
  int req;
  int kv_head;
  int row0;            // first packed row of the item
  int split;           // index of the key split this item covers (0 when the keys are not split)
};

// Row tiles (tensor-core `attend` schedules): up to 256 packed query rows that share every key tile of a
// cached prefix.  A tile is a list of segments; segment k is rows [begin, begin + count) of the tile =
// packed rows prow0 .. of request `req`.  All requests of a tile have the same cached prefix; after the
// prefix tiles the tile walks the own rows of every segment's request in turn, and a query row takes part
// only in the key tiles of its own request.  In a tiled schedule WorkItem::req is the index of the row tile.
constexpr int kMaxSegs = 8;
struct RowSeg {
  int req;
  int prow0;
  int begin;
  int count;
};
struct RowTile {
  int m;               // cached prefix length of the tile's requests (0: a request without prefix, one segment)
  int page_off;        // index of the prefix's first page id inside the schedule's page list
  int nrows;           // end of the last segment
  int nseg;
  RowSeg seg[kMaxSegs];
};

// Device view of a schedule: everything a kernel needs besides the tensors.
struct ScheduleView {
  const ReqMeta* reqs;
  const int* pages;          // concatenated page lists
  const WorkItem* items;
  const RowTile* tiles;      // nullptr: items name (request, first packed row) themselves
  int shared_tiles;          // some row tile holds rows of more than one request
  int num_items;
  int num_splits;            // > 1: item covers key tiles [split * tiles_per_split, (split + 1) * tiles_per_split)
  int tiles_per_split;       // key tiles: ceil(m/128) prefix tiles followed by ceil(n/128) own tiles
};

// Bytes from the start of a (page, kv head) slice to the 16-byte chunk `c16` of token slot `slot`.
// For bf16 with D = 128 a page is stored as the shared-memory image the tensor-core descriptors
// read: four 1 KB blocks [slots 0-7, dims 0-63 | slots 0-7, dims 64-127 | slots 8-15, dims 0-63 |
// slots 8-15, dims 64-127], each 8 rows of 128 bytes with the 16-byte chunks of row r XOR-permuted
// by r (the 128-byte swizzle).  Every other dtype/D keeps plain [slot][dim] order.
__host__ __device__ inline unsigned page_chunk_offset(bool swizzled, int slot, int c16, int row_bytes) {
  if (swizzled) {
    const int g = slot >> 3, r = slot & 7, h = c16 >> 3, c = c16 & 7;
    return (unsigned)(g * 2048 + h * 1024 + r * 128 + ((c ^ r) << 4));
  }
  return (unsigned)(slot * row_bytes + c16 * 16);
}

struct PoolView {
  const char* k;
  const char* v;
  long long layer_bytes;     // num_pages * Hkv * page_bytes
  int page_bytes;            // kPageSize * D * elem size (bytes of one (page, head) slice)
  int num_kv_heads;
  int swizzled;
};

__host__ __device__ inline long long pool_slice_offset(const PoolView& p, int layer, int page, int hk) {
  return (long long)layer * p.layer_bytes + ((long long)page * p.num_kv_heads + hk) * p.page_bytes;
}

// Sticky device status word codes (first error wins).
constexpr int kDevOk = 0;
constexpr int kDevTimeout = 5;
constexpr int kDevInternal = 6;   // a kernel found its own launch state wrong (shared-memory alignment)

}  // namespace bicache
