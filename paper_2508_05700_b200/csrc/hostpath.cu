// Host-resident tables: zero-copy row fetch over PCIe (K-host-fetch), the HBM
// hot-row cache (build + lookup index), and the orchestration of one
// host-table slot: hash -> dedup -> cache probe -> fetch misses -> pool.
#include <cstring>

#include "common.cuh"

using namespace mfet;

namespace mfet {

namespace {

inline uint64_t align256(uint64_t x) { return (x + 255u) & ~255ULL; }

constexpr int kFetchUnroll = 4;

// dst[m] = table[rows_list[m]] for m < n, rows as 16-byte chunks. Consecutive
// threads take consecutive chunks, so a 128-byte row is one fully coalesced
// request; every thread keeps kFetchUnroll independent loads in flight because
// the source may be pinned host memory behind PCIe (about 2 us per request).
__global__ void __launch_bounds__(256) fetch_rows_kernel(const uint8_t* __restrict__ table, uint64_t stride,
                                                         uint32_t chunks, const int64_t* __restrict__ rows_list,
                                                         const int64_t* __restrict__ n_ptr, int64_t n_imm,
                                                         uint8_t* __restrict__ dst, uint64_t table_rows, int64_t cap,
                                                         uint32_t* err) {
  int64_t n = n_ptr ? *n_ptr : n_imm;
  if (!MFET_IN_BOUNDS(err, n >= 0 && n <= cap)) n = 0;
  const int64_t total = n * chunks;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t q0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q0 < total; q0 += step * kFetchUnroll) {
    uint4 v[kFetchUnroll];
#pragma unroll
    for (int k = 0; k < kFetchUnroll; ++k) {
      const int64_t q = q0 + k * step;
      if (q < total) {
        const int64_t m = q / chunks;
        const uint32_t c = (uint32_t)(q - m * chunks);
        const uint64_t row = (uint64_t)rows_list[m];
        v[k] = MFET_IN_BOUNDS(err, row < table_rows) ? ld_row16(table + row * stride + (uint64_t)c * 16)
                                                     : make_uint4(0u, 0u, 0u, 0u);
      }
    }
#pragma unroll
    for (int k = 0; k < kFetchUnroll; ++k) {
      const int64_t q = q0 + k * step;
      if (q < total) *reinterpret_cast<uint4*>(dst + q * 16) = v[k];
    }
  }
}

// bucket_start[b] = first position whose key is >= b << shift (b = n_buckets: n).
__global__ void __launch_bounds__(256) cache_index_kernel(const int64_t* __restrict__ keys, int64_t n,
                                                          uint32_t shift, uint32_t n_buckets,
                                                          uint32_t* __restrict__ bucket_start) {
  const uint64_t b = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (b > n_buckets) return;
  const uint64_t bound = b << shift;
  int64_t lo = 0, hi = n;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if ((uint64_t)keys[mid] < bound) lo = mid + 1;
    else hi = mid;
  }
  bucket_start[b] = (uint32_t)lo;
}

}  // namespace

cudaError_t launch_fetch(const uint8_t* table, uint64_t stride, uint32_t chunks, const int64_t* rows_list,
                         const int64_t* n_ptr, int64_t n_imm, uint8_t* dst, uint64_t table_rows, int64_t cap,
                         uint32_t* err, cudaStream_t s) {
  // A small footprint on purpose: one warp per multiprocessor with kFetchUnroll loads per lane keeps about
  // 2 400 rows in flight, far more than the host link needs (random rows arrive at 50-60 million a second,
  // 2-3 us each). With 4 x 256 threads per multiprocessor (a) random rows came 20 % slower (6.2 instead of
  // 7.8 GB/s on a 128 GB table: the hundreds of thousands of pending host reads get in one another's way),
  // and (b) every other kernel that ran next to the fetch crawled behind them (a 20 us copy kernel took
  // 1.1 ms; now 57 us) - and in the lookup path the pooling of one batch and the dedup of the next run
  // next to it. Consecutive rows still arrive at 43 GB/s (48 with the large footprint).
  fetch_rows_kernel<<<sm_count(), 32, 0, s>>>(table, stride, chunks, rows_list, n_ptr, n_imm, dst, table_rows, cap, err);
  return cudaGetLastError();
}

void cache_layout(uint64_t rows, int64_t n, uint64_t row_bytes, CacheLayout* L) {
  // buckets of 2^shift consecutive row ids; about 4-8 cached rows per bucket
  uint32_t shift = 0;
  const uint64_t want = n / 4 > 1 ? (uint64_t)n / 4 : 1;
  while ((((rows - 1) >> shift) + 1) > want || (((rows - 1) >> shift) + 1) > (1ULL << 28)) ++shift;
  L->bucket_shift = shift;
  L->n_buckets = (uint32_t)(((rows - 1) >> shift) + 1);
  uint64_t off = 0;
  L->keys = off;
  off = align256(off + (uint64_t)n * 8);
  L->bucket_start = off;
  off = align256(off + ((uint64_t)L->n_buckets + 1) * 4);
  L->data = off;
  off = align256(off + (uint64_t)n * row_bytes);
  L->total = off;
}

int run_host_slot(mfet_tables* t, const TableHost& tb, const BagParams& base, int32_t feature, int32_t pooling,
                  uint32_t col, cudaStream_t side, int stage, int set) {
  WsLayout L;
  const uint64_t need = workspace_layout(t->ws_max_ids, tb.row_bytes, &L);
  if (need > t->ws_bytes) return MFET_ERR_WORKSPACE;
  uint8_t* ws = (uint8_t*)t->ws;
  int64_t* counters = (int64_t*)(ws + L.counters);

  HashArgs h{base.ids, tb.desc.hash_seed, tb.desc.rows, tb.magic, base.flags & 1u};
  CacheDev cd{tb.cache.keys, tb.cache.bucket_start, tb.cache.data, tb.cache.n, tb.cache.bucket_shift, 0};
  DedupArgs a;
  std::memset(&a, 0, sizeof(a));
  a.ns = NSrc{base.offsets, (int64_t)feature * base.batch, (int64_t)(feature + 1) * base.batch, 0, t->ws_max_ids};
  a.hash = &h;
  a.max_key = tb.desc.rows - 1;
  a.ws = ws;
  a.layout = L;
  a.cache = &cd;
  a.uniq = (int64_t*)(ws + L.uniq);
  a.inverse = (int32_t*)(ws + (set ? L.inverse2 : L.inverse));
  a.n_unique = counters;
  a.src = (int32_t*)(ws + (set ? L.src2 : L.src));
  uint8_t* staging = ws + (set ? L.staging2 : L.staging);
  a.miss_rows = (int64_t*)(ws + (set ? L.miss_rows2 : L.miss_rows));
  a.n_miss = counters + 1 + set;
  a.err = t->err_dev;
  const bool prof = t->profile != 0 && stage == 3;
  const uint32_t chunks = (uint32_t)(tb.row_bytes / 16);
  if (prof) cudaEventRecord(t->prof_ev[0], side);
  if (stage & 1) {
    // hash + dedup + probe on the side stream; the reads of the missed rows on the fetch stream, which
    // the next batch's dedup does not wait for (it writes the other result set)
    if (launch_dedup(a, &t->launches, side) != cudaSuccess) return MFET_ERR_CUDA;
    if (prof) cudaEventRecord(t->prof_ev[1], side);
    if (cudaEventRecord(t->ev_dedup[set], side) != cudaSuccess) return MFET_ERR_CUDA;
    if (cudaStreamWaitEvent(t->fetch, t->ev_dedup[set], 0) != cudaSuccess) return MFET_ERR_CUDA;
    if (launch_fetch(tb.dev_ptr, tb.stride, chunks, a.miss_rows, a.n_miss, 0, staging, tb.desc.rows, t->ws_max_ids,
                     t->err_dev, t->fetch) != cudaSuccess)
      return MFET_ERR_CUDA;
    t->launches += 1;
    if (prof) cudaEventRecord(t->prof_ev[2], t->fetch);
    if (cudaEventRecord(t->ev_fetch[set], t->fetch) != cudaSuccess) return MFET_ERR_CUDA;
    t->last_set = set;
    t->last_row_bytes = tb.row_bytes;
  }
  if (!(stage & 2)) return MFET_OK;

  // the pooling follows on the side stream once the set's rows have arrived; a later dedup into the
  // same set is behind it in that stream
  if (cudaStreamWaitEvent(side, t->ev_fetch[set], 0) != cudaSuccess) return MFET_ERR_CUDA;
  IndirectParams ip{a.inverse, a.src, tb.cache.data, staging, tb.row_bytes, t->ws_max_ids, tb.cache.n};
  BagParams p = base;
  p.flags &= ~1u;  // the indirect path never hashes
  p.flags |= base.flags & 2u;
  const uint32_t epc = tb.desc.dtype == MFET_F32 ? 4u : 8u;
  const bool int4 = tb.desc.dtype == MFET_INT4;
  const uint32_t chunk_bytes = int4 ? 4u : 16u;
  const uint32_t pool_chunks = int4 ? tb.desc.dim / 8u : chunks;  // a lane's chunk: 16 bytes, INT4: 4 bytes of codes
  int n = 0;
  for (uint32_t c0 = 0; c0 < pool_chunks; c0 += 32) {
    SlotDev& sd = p.slot[n++];
    std::memset(&sd, 0, sizeof(sd));
    const uint32_t ch = pool_chunks - c0 < 32 ? pool_chunks - c0 : 32;
    sd.table = reinterpret_cast<const uint8_t*>((uintptr_t)c0 * chunk_bytes);  // byte offset inside the row
    sd.meta_off = int4 ? tb.desc.dim / 2u - c0 * chunk_bytes : 0u;
    sd.rows = tb.desc.rows;
    sd.stride = tb.row_bytes;
    sd.feature = (uint32_t)feature;
    sd.col_off = col + c0 * epc;
    sd.chunks = (uint16_t)ch;
    sd.dtype = (uint8_t)tb.desc.dtype;
    sd.pooling = (uint8_t)pooling;
    uint8_t lg = 1;
    while ((1u << lg) < ch) ++lg;
    sd.lpr_log2 = lg;
    if (n == kMaxSlotsPerLaunch || c0 + 32 >= pool_chunks) {
      p.n_slots = n;
      if (launch_bag_indirect(p, ip, side) != cudaSuccess) return MFET_ERR_CUDA;
      t->launches += 1;
      n = 0;
    }
  }
  if (prof) {
    cudaEventRecord(t->prof_ev[3], side);
    t->prof_valid = true;
  }
  return MFET_OK;
}

}  // namespace mfet

extern "C" {

int mfet_dedup_rows(mfet_tables_t* t, const int64_t* rows, int64_t n, int64_t* uniq, int32_t* inverse,
                    int64_t* n_unique, int64_t max_row, mfet_stream_t stream_) {
  if (!t || n < 0 || !n_unique || max_row < 0) return MFET_ERR_INVALID_ARG;
  cudaStream_t stream = (cudaStream_t)stream_;
  if (n > 0 && (!rows || !uniq || !inverse)) return MFET_ERR_INVALID_ARG;
  if (n > 0 && (!t->ws || n > t->ws_max_ids || n > 0x7FFFFFFF)) return MFET_ERR_WORKSPACE;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  WsLayout L;
  int rc = MFET_OK;
  if (n == 0) {
    if (cudaMemsetAsync(n_unique, 0, sizeof(int64_t), stream) != cudaSuccess) rc = MFET_ERR_CUDA;
  } else if (workspace_layout(t->ws_max_ids, 16, &L) > t->ws_bytes) {
    rc = MFET_ERR_WORKSPACE;
  } else {
    DedupArgs a;
    std::memset(&a, 0, sizeof(a));
    a.ns = NSrc{nullptr, 0, 0, n, n};
    a.first_keys = reinterpret_cast<const uint64_t*>(rows);
    a.max_key = max_row > 0 ? (uint64_t)max_row - 1 : 0x7FFFFFFFFFFFFFFFULL;
    a.ws = t->ws;
    a.layout = L;
    a.uniq = uniq;
    a.inverse = inverse;
    a.n_unique = n_unique;
    a.err = t->err_dev;
    if (launch_dedup(a, &t->launches, stream) != cudaSuccess) rc = MFET_ERR_CUDA;
  }
  if (prev != t->device) cudaSetDevice(prev);
  return rc;
}

int mfet_host_path_counts(mfet_tables_t* t, int64_t* n_unique, int64_t* n_miss) {
  if (!t || !n_unique || !n_miss) return MFET_ERR_INVALID_ARG;
  if (!t->ws) return MFET_ERR_WORKSPACE;
  WsLayout L;
  workspace_layout(t->ws_max_ids, 16, &L);
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  int64_t c[3] = {0, 0, 0};  // n_unique, n_miss of result set 0, of result set 1
  bool ok = cudaStreamSynchronize(t->side) == cudaSuccess && cudaStreamSynchronize(t->fetch) == cudaSuccess &&
            cudaMemcpy(c, static_cast<uint8_t*>(t->ws) + L.counters, sizeof(c), cudaMemcpyDeviceToHost) == cudaSuccess;
  if (prev != t->device) cudaSetDevice(prev);
  if (!ok) return MFET_ERR_CUDA;
  *n_unique = c[0];
  *n_miss = c[1 + (t->last_set & 1)];
  return MFET_OK;
}

int mfet_host_path_result(mfet_tables_t* t, int64_t* uniq, int32_t* src, int64_t* miss_rows, int64_t capacity) {
  if (!t || capacity < 0) return MFET_ERR_INVALID_ARG;
  if (!t->ws) return MFET_ERR_WORKSPACE;
  WsLayout L;
  workspace_layout(t->ws_max_ids, t->last_row_bytes, &L);
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  const uint8_t* ws = static_cast<const uint8_t*>(t->ws);
  const int set = t->last_set & 1;
  int64_t c[3] = {0, 0, 0};  // n_unique, n_miss of result set 0, of result set 1
  bool ok = cudaStreamSynchronize(t->side) == cudaSuccess && cudaStreamSynchronize(t->fetch) == cudaSuccess &&
            cudaMemcpy(c, ws + L.counters, sizeof(c), cudaMemcpyDeviceToHost) == cudaSuccess;
  int rc = MFET_OK;
  if (ok && (c[0] > capacity || c[1 + set] > capacity)) rc = MFET_ERR_INVALID_ARG;
  if (ok && rc == MFET_OK) {
    if (uniq && c[0] > 0) ok = ok && cudaMemcpy(uniq, ws + L.uniq, (size_t)c[0] * 8, cudaMemcpyDeviceToDevice) == cudaSuccess;
    if (src && c[0] > 0)
      ok = ok && cudaMemcpy(src, ws + (set ? L.src2 : L.src), (size_t)c[0] * 4, cudaMemcpyDeviceToDevice) == cudaSuccess;
    if (miss_rows && c[1 + set] > 0)
      ok = ok && cudaMemcpy(miss_rows, ws + (set ? L.miss_rows2 : L.miss_rows), (size_t)c[1 + set] * 8,
                            cudaMemcpyDeviceToDevice) == cudaSuccess;
    ok = ok && cudaDeviceSynchronize() == cudaSuccess;
  }
  if (prev != t->device) cudaSetDevice(prev);
  if (!ok) return MFET_ERR_CUDA;
  return rc;
}

int mfet_host_fetch_rows(mfet_tables_t* t, int32_t table_id, const int64_t* rows, int64_t n, void* dst,
                         mfet_stream_t stream_) {
  if (!t || n < 0 || table_id < 0 || table_id >= (int32_t)t->tables.size()) return MFET_ERR_INVALID_ARG;
  const TableHost& tb = t->tables[(size_t)table_id];
  if (tb.desc.location != MFET_LOC_HOST) return MFET_ERR_INVALID_ARG;
  if (!tb.registered) return MFET_ERR_NOT_REGISTERED;
  if (n == 0) return MFET_OK;
  if (!rows || !dst) return MFET_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(dst) & 15u) return MFET_ERR_ALIGNMENT;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  const bool ok = launch_fetch(tb.dev_ptr, tb.stride, (uint32_t)(tb.row_bytes / 16), rows, nullptr, n,
                               static_cast<uint8_t*>(dst), tb.desc.rows, n, t->err_dev,
                               (cudaStream_t)stream_) == cudaSuccess;
  if (ok) t->launches += 1;
  if (prev != t->device) cudaSetDevice(prev);
  return ok ? MFET_OK : MFET_ERR_CUDA;
}

int mfet_cache_bytes(const mfet_tables_t* t, int32_t table_id, int64_t n, uint64_t* bytes) {
  if (!t || !bytes || n < 0 || table_id < 0 || table_id >= (int32_t)t->tables.size()) return MFET_ERR_INVALID_ARG;
  const TableHost& tb = t->tables[(size_t)table_id];
  if ((uint64_t)n > tb.desc.rows || n > 0x7FFFFFFF) return MFET_ERR_INVALID_ARG;
  CacheLayout L;
  cache_layout(tb.desc.rows, n, tb.row_bytes, &L);
  *bytes = L.total;
  return MFET_OK;
}

int mfet_cache_build(mfet_tables_t* t, int32_t table_id, const int64_t* rows_sorted, int64_t n, void* cache_mem,
                     uint64_t cache_bytes, mfet_stream_t stream_) {
  if (!t || n < 0 || table_id < 0 || table_id >= (int32_t)t->tables.size()) return MFET_ERR_INVALID_ARG;
  TableHost& tb = t->tables[(size_t)table_id];
  if (tb.desc.location != MFET_LOC_HOST) return MFET_ERR_INVALID_ARG;
  if (n == 0) {
    tb.cache = CacheInfo();
    return MFET_OK;
  }
  if (!tb.registered) return MFET_ERR_NOT_REGISTERED;
  if (!rows_sorted || !cache_mem || (uint64_t)n > tb.desc.rows || n > 0x7FFFFFFF) return MFET_ERR_INVALID_ARG;
  if (reinterpret_cast<uintptr_t>(cache_mem) & 255u) return MFET_ERR_ALIGNMENT;
  for (int64_t i = 0; i < n; ++i) {
    if (rows_sorted[i] < 0 || (uint64_t)rows_sorted[i] >= tb.desc.rows) return MFET_ERR_INVALID_ARG;
    if (i > 0 && rows_sorted[i] <= rows_sorted[i - 1]) return MFET_ERR_INVALID_ARG;
  }
  CacheLayout L;
  cache_layout(tb.desc.rows, n, tb.row_bytes, &L);
  if (cache_bytes < L.total) return MFET_ERR_WORKSPACE;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_;
  uint8_t* mem = (uint8_t*)cache_mem;
  int64_t* keys = (int64_t*)(mem + L.keys);
  uint32_t* bucket_start = (uint32_t*)(mem + L.bucket_start);
  bool ok = cudaMemcpyAsync(keys, rows_sorted, (size_t)n * 8, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (ok) {
    const unsigned blocks = (unsigned)(((uint64_t)L.n_buckets + 1 + 255) / 256);
    cache_index_kernel<<<blocks, 256, 0, stream>>>(keys, n, L.bucket_shift, L.n_buckets, bucket_start);
    ok = cudaGetLastError() == cudaSuccess;
  }
  ok = ok && launch_fetch(tb.dev_ptr, tb.stride, (uint32_t)(tb.row_bytes / 16), keys, nullptr, n, mem + L.data,
                          tb.desc.rows, n, t->err_dev, stream) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  if (ok) {
    t->launches += 2;
    tb.cache.keys = keys;
    tb.cache.bucket_start = bucket_start;
    tb.cache.data = mem + L.data;
    tb.cache.n = n;
    tb.cache.bucket_shift = L.bucket_shift;
    tb.cache.n_buckets = L.n_buckets;
  } else {
    cudaGetLastError();
  }
  if (prev != t->device) cudaSetDevice(prev);
  return ok ? MFET_OK : MFET_ERR_CUDA;
}

static inline uint64_t a256(uint64_t x) { return (x + 255u) & ~255ULL; }

int mfet_host_io_bytes(const mfet_tables_t* t, const mfet_batch_shape_t* shape, const int32_t* table_ids,
                       int64_t nnz, uint64_t* bytes) {
  if (!t || !shape || !table_ids || !bytes || nnz < 0 || shape->batch < 0 || shape->n_features < 1 ||
      shape->n_slots < 1)
    return MFET_ERR_INVALID_ARG;
  int64_t total_dim = 0;
  for (int32_t s = 0; s < shape->n_slots; ++s) {
    if (table_ids[s] < 0 || table_ids[s] >= (int32_t)t->tables.size()) return MFET_ERR_INVALID_ARG;
    total_dim += t->tables[(size_t)table_ids[s]].desc.dim;
  }
  const int64_t out_ld = shape->out_ld ? shape->out_ld : total_dim;
  if (out_ld < total_dim) return MFET_ERR_INVALID_ARG;
  *bytes = a256((uint64_t)nnz * 8) + a256(((uint64_t)shape->n_features * shape->batch + 1) * 8) +
           a256((uint64_t)nnz * 4) + a256((uint64_t)shape->batch * out_ld * 4);
  return MFET_OK;
}

static int forward_host_impl(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids_host,
                             const int64_t* offsets_host, const float* weights_host, int64_t nnz,
                             const int32_t* table_ids, const int32_t* pooling, float* out_host, void* dev_io,
                             uint64_t dev_io_bytes, mfet_stream_t stream_, bool wait) {
  uint64_t need = 0;
  int rc = mfet_host_io_bytes(t, shape, table_ids, nnz, &need);
  if (rc != MFET_OK) return rc;
  if (!dev_io || dev_io_bytes < need) return MFET_ERR_WORKSPACE;
  if (reinterpret_cast<uintptr_t>(dev_io) & 255u) return MFET_ERR_ALIGNMENT;
  if (shape->batch == 0) return MFET_OK;
  if (!offsets_host || !out_host || (nnz > 0 && !ids_host)) return MFET_ERR_INVALID_ARG;
  int64_t total_dim = 0;
  for (int32_t s = 0; s < shape->n_slots; ++s) total_dim += t->tables[(size_t)table_ids[s]].desc.dim;
  const int64_t out_ld = shape->out_ld ? shape->out_ld : total_dim;
  cudaStream_t stream = (cudaStream_t)stream_;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  uint8_t* io = (uint8_t*)dev_io;
  uint64_t* d_ids = (uint64_t*)io;
  int64_t* d_off = (int64_t*)(io + a256((uint64_t)nnz * 8));
  const uint64_t n_off = (uint64_t)shape->n_features * shape->batch + 1;
  float* d_w = (float*)((uint8_t*)d_off + a256(n_off * 8));
  float* d_out = (float*)((uint8_t*)d_w + a256((uint64_t)nnz * 4));
  bool ok = true;
  if (nnz > 0) ok = cudaMemcpyAsync(d_ids, ids_host, (size_t)nnz * 8, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(d_off, offsets_host, n_off * 8, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (ok && weights_host && nnz > 0)
    ok = cudaMemcpyAsync(d_w, weights_host, (size_t)nnz * 4, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (ok) {
    rc = mfet_embedding_bag_forward(t, shape, d_ids, d_off, weights_host ? d_w : nullptr, table_ids, pooling, d_out,
                                    stream_);
    if (rc == MFET_OK) {
      ok = cudaMemcpyAsync(out_host, d_out, (size_t)shape->batch * out_ld * 4, cudaMemcpyDeviceToHost, stream) ==
           cudaSuccess;
      if (wait) ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
    }
  }
  if (prev != t->device) cudaSetDevice(prev);
  if (rc != MFET_OK) return rc;
  return ok ? MFET_OK : MFET_ERR_CUDA;
}

int mfet_embedding_bag_forward_host(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids_host,
                                    const int64_t* offsets_host, const float* weights_host, int64_t nnz,
                                    const int32_t* table_ids, const int32_t* pooling, float* out_host, void* dev_io,
                                    uint64_t dev_io_bytes, mfet_stream_t stream) {
  return forward_host_impl(t, shape, ids_host, offsets_host, weights_host, nnz, table_ids, pooling, out_host, dev_io,
                           dev_io_bytes, stream, true);
}

int mfet_embedding_bag_forward_host_async(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids_host,
                                          const int64_t* offsets_host, const float* weights_host, int64_t nnz,
                                          const int32_t* table_ids, const int32_t* pooling, float* out_host,
                                          void* dev_io, uint64_t dev_io_bytes, mfet_stream_t stream) {
  return forward_host_impl(t, shape, ids_host, offsets_host, weights_host, nnz, table_ids, pooling, out_host, dev_io,
                           dev_io_bytes, stream, false);
}

}  // extern "C"
