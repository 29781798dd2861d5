// Shared declarations of the mfet library: handle layout, kernel parameter
// blocks, and the small device helpers (hash, exact modulo, cache-hinted
// loads/stores) that several kernels use.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <vector>

#include "../../include/mfet.h"

namespace mfet {

// ------------------------------------------------------------ host side -----

struct CacheInfo {
  const int64_t* keys = nullptr;         // dev i64[n], ascending
  const uint32_t* bucket_start = nullptr;// dev u32[n_buckets + 1]
  const uint8_t* data = nullptr;         // dev [n, row_bytes]
  int64_t n = 0;
  uint32_t bucket_shift = 0;             // bucket = key >> bucket_shift
  uint32_t n_buckets = 0;
};

struct TableHost {
  mfet_table_desc_t desc;
  uint64_t row_bytes = 0;
  uint64_t stride = 0;
  uint64_t magic = 0;        // floor((2^64 - 1) / rows)
  const uint8_t* dev_ptr = nullptr;  // device-visible address of the rows
  void* host_ptr = nullptr;
  bool registered = false;   // host table: memory supplied
  bool pinned_by_us = false;
  CacheInfo cache;
};

}  // namespace mfet

struct mfet_tables {
  int device = 0;
  std::vector<mfet::TableHost> tables;
  uint32_t* err_host = nullptr;  // pinned + mapped status word
  uint32_t* err_dev = nullptr;   // its device-visible address
  cudaStream_t side = nullptr;   // host-table slots: hash + dedup + cache probe, and the pooling, run here
  cudaStream_t fetch = nullptr;  // ... and the reads of the missed rows from host memory here, so that the
                                 // dedup of the next batch runs while the rows of this one cross PCIe
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  cudaEvent_t ev_dedup[2] = {nullptr, nullptr}, ev_fetch[2] = {nullptr, nullptr};  // per result set
  int last_set = 0;              // result set of the most recent host-table batch
  uint64_t last_row_bytes = 16;  // row bytes that laid out the workspace for it
  void* ws = nullptr;
  uint64_t ws_bytes = 0;
  int64_t ws_max_ids = 0;
  uint64_t launches = 0;
  int32_t group_policy = 0;
  uint64_t version = 0;  // caller's tag of this table set (model version)
  uint64_t prefetched = 0, consumed = 0;  // batches handed to mfet_host_prefetch / pooled from a prefetch
  int32_t tile = 0;  // bags per block; 0 = chosen from the batch size
  int32_t stage_cap = 0;  // IDs staged per window of the pooling kernel; 0 = default
  int32_t overlap = 0;    // 1: pooling launches may begin while the stream's previous kernel still runs
  int32_t profile = 0;             // 1: time the stages of the host-table path with events
  cudaEvent_t prof_ev[4] = {nullptr, nullptr, nullptr, nullptr};
  bool prof_valid = false;
};

namespace mfet {

// ----------------------------------------------------------- kernel params --

// One (feature, table) slot as the pooling kernel sees it. Rows wider than 512
// bytes are split on the host into several entries of at most 32 chunks.
struct SlotDev {
  const uint8_t* table;  // first byte of the slot's column block in row 0
  uint64_t rows;
  uint64_t magic;
  uint64_t seed;
  uint64_t stride;       // bytes between rows
  uint32_t feature;
  uint32_t col_off;      // first output column
  uint16_t chunks;       // 16-byte chunks of the row that this entry covers (1..32)
  uint8_t dtype;
  uint8_t pooling;
  uint8_t lpr_log2;      // lanes per row = 1 << lpr_log2 >= chunks
  uint8_t narrow;        // 1: row indices and the stride fit 32 bits
  uint16_t pad;
  uint32_t meta_off;     // INT4: byte offset of the row's fp16 scale/bias pair from `table`
};
static_assert(sizeof(SlotDev) == 64, "SlotDev must stay 64 bytes");

constexpr int kMaxSlotsPerLaunch = 56;
constexpr int kMaxTile = 128;
// IDs of a tile that the pooling kernel stages in shared memory at a time
// (4 bytes each, 8 with weights, 12 with weights and 64-bit row indices).
constexpr int kStageDefault = 4096;
constexpr int kStageMax = 8192;

struct BagParams {
  const uint64_t* ids;
  const int64_t* offsets;
  const float* weights;
  float* out;
  uint32_t* err;
  int64_t out_ld;
  int32_t batch;
  int32_t n_slots;
  int32_t tiles_per_slot;
  int32_t tile;          // bags per block, <= kMaxTile
  uint32_t flags;        // bit0: ids are rows; bit1: out allows 16-byte vector stores;
                         // set at launch: bit2 weights are staged, bit3 upper row-index halves are staged;
                         // bit4: the launch may begin before the stream's previous kernel has finished
  int32_t group_policy;  // 0 auto, 1 one row-group per bag, 2 one warp per bag
  int32_t stage_cap;     // IDs staged per window, 32 .. kStageMax (0: default)
  int32_t n_features;    // offsets has n_features * batch + 1 entries (used by the bounds-checked build)
  SlotDev slot[kMaxSlotsPerLaunch];
};
static_assert(sizeof(BagParams) <= 4000, "BagParams must fit the kernel parameter space");

// ---------------------------------------------------------- device helpers --

// Bounds-checked build (-DMFET_CHECKED, `python -m paper_2508_05700_b200.build --checked`): every
// index that a kernel forms from the caller's data or from its own arithmetic is tested against
// the extent of the array right before the access; a violation sets MFET_DEV_BOUNDS in the device
// error word and the access is skipped (no trap, no assert: the context stays usable). The normal
// build compiles the tests away.
#ifdef MFET_CHECKED
#define MFET_IN_BOUNDS(err, cond) ((cond) ? true : (atomicOr((err), (uint32_t)MFET_DEV_BOUNDS), false))
#else
#define MFET_IN_BOUNDS(err, cond) true
#endif

// splitmix64 output function (public domain; Steele, Lea, Flood).
__host__ __device__ __forceinline__ uint64_t splitmix64(uint64_t x) {
  x += 0x9E3779B97F4A7C15ULL;
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ULL;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBULL;
  return x ^ (x >> 31);
}

// Exact h mod d for a runtime divisor d >= 1, with magic = floor((2^64-1)/d). Let e = 2^64 - magic*d:
// 0 < e <= d (e = d exactly when d is a power of two). Then h*magic/2^64 = h/d - h*e/(d*2^64), and the
// last term lies in [0, 1) because h < 2^64 and e <= d. So q = floor(h*magic / 2^64) is floor(h/d) or
// one less, the remainder estimate is below 2d, and ONE conditional subtraction finishes it.
__device__ __forceinline__ uint64_t mod_rows(uint64_t h, uint64_t d, uint64_t magic) {
  uint64_t q = __umul64hi(h, magic);
  uint64_t r = h - q * d;
  if (r >= d) r -= d;
  return r;
}

inline uint64_t host_magic(uint64_t rows) { return 0xFFFFFFFFFFFFFFFFULL / rows; }

// Number of SMs of the current device (asked once per device; grids are sized by it).
int sm_count();

// 16-byte row load through the read-only path. Rows may allocate in L1: with Zipf-distributed
// IDs an SM re-reads the head rows of a table hundreds of times per batch, and serving those
// from L1 measured 2-8 % faster than keeping rows out of it (no allocation, evict-first and
// evict-last hints were all slower).
__device__ __forceinline__ uint4 ld_row16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ uint32_t ld_row4(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}

__device__ __forceinline__ float bf16lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16hi(uint32_t x) { return __uint_as_float(x & 0xFFFF0000u); }

// ------------------------------------------------- host-table path params --

// Element count of a pass: immediate, or the ID count of one feature read from
// the CSR offsets on the device (the host never learns it).
struct NSrc {
  const int64_t* offsets;  // nullptr => n_imm
  int64_t idx_lo, idx_hi;  // n = offsets[idx_hi] - offsets[idx_lo]
  int64_t n_imm;
  int64_t cap;             // counts above cap (or negative) degrade to 0
};

struct CacheDev {
  const int64_t* keys;
  const uint32_t* bucket_start;
  const uint8_t* data;
  int64_t n;
  uint32_t bucket_shift;
  uint32_t pad;
};

struct WsLayout {
  uint64_t keys_a, keys_b, idx_a, idx_b, hist, tile_counts, counters, uniq, inverse, src, miss_rows,
      staging, total;
  uint64_t inverse2, src2, staging2, miss_rows2;  // second result set: a prefetched batch waits here
  int nblk_sort, nblk_scan;
};

struct HashArgs {
  const uint64_t* ids;
  uint64_t seed, rows, magic;
  uint32_t pre_hashed;
};

struct DedupArgs {
  NSrc ns;
  const uint64_t* first_keys;  // pass-0 input when hash == nullptr
  const HashArgs* hash;        // non-null: pass 0 hashes the slot's raw IDs
  uint64_t max_key;            // largest possible key (sets the number of passes)
  void* ws;
  WsLayout layout;
  const CacheDev* cache;       // non-null: probe + miss compaction
  int64_t* uniq;
  int32_t* inverse;
  int64_t* n_unique;
  int32_t* src;
  int64_t* miss_rows;
  int64_t* n_miss;
  uint32_t* err;
  const uint32_t** sorted_pos_out;  // optional: receives the array of original positions in sorted order
};

// Where the pooling kernel finds the rows of a host-table slot.
struct IndirectParams {
  const int32_t* inverse;     // [n] position in uniq of every lookup of the slot
  const int32_t* src;         // [n_unique] >= 0: cache slot; < 0: -1 - staging index
  const uint8_t* cache_data;
  const uint8_t* staging;
  uint64_t row_bytes;
  int64_t cap;
  int64_t cache_n;            // rows in the cache (used by the bounds-checked build)
};

struct CacheLayout {
  uint64_t keys, bucket_start, data, total;
  uint32_t bucket_shift, n_buckets;
};

uint64_t workspace_layout(int64_t max_ids, uint64_t max_row_bytes, WsLayout* L);
void cache_layout(uint64_t rows, int64_t n, uint64_t row_bytes, CacheLayout* L);
cudaError_t launch_dedup(const DedupArgs& a, uint64_t* launches, cudaStream_t s);
// table_rows, cap: the table's rows and the capacity (in rows) of rows_list / dst, for the bounds-checked build
cudaError_t launch_fetch(const uint8_t* table, uint64_t stride, uint32_t chunks, const int64_t* rows_list,
                         const int64_t* n_ptr, int64_t n_imm, uint8_t* dst, uint64_t table_rows, int64_t cap,
                         uint32_t* err, cudaStream_t s);
cudaError_t launch_bag_indirect(const BagParams& p, const IndirectParams& ip, cudaStream_t s);
// stage bit0: hash + dedup + probe + fetch into result set `set`; bit1: pool from it
int run_host_slot(mfet_tables* t, const TableHost& tb, const BagParams& base, int32_t feature, int32_t pooling,
                  uint32_t col, cudaStream_t side, int stage, int set);

cudaError_t launch_backward(const uint32_t* sorted_pos, const int32_t* inverse, const int32_t* seg_start,
                            const int64_t* n_unique, NSrc ns, const int64_t* offsets_f, int32_t batch,
                            const float* weights, int32_t pooling, const float* grad_out, int64_t out_ld, uint32_t col,
                            uint32_t dim, int32_t chunk, float* partial, float* grad_vals, uint32_t* err,
                            cudaStream_t s);

// launch helpers implemented in the kernel files
cudaError_t launch_hash(const uint64_t* ids, int64_t n, uint64_t seed, uint64_t rows, uint64_t magic,
                        int64_t* rows_out, cudaStream_t s);
cudaError_t launch_fill(void* data, uint64_t row0, uint64_t n_rows, uint32_t dim, uint32_t dtype,
                        uint64_t stride, uint64_t key, uint32_t mode, cudaStream_t s);
cudaError_t launch_bag(const BagParams& p, cudaStream_t s);

}  // namespace mfet
