// C-ABI boundary: argument checking, descriptor bookkeeping and launch
// orchestration. No arithmetic of the lookup path happens on the host.
#include <algorithm>
#include <atomic>
#include <cstring>
#include <new>

#include "common.cuh"
#include "dedup_layout.cuh"

using namespace mfet;

namespace {

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
    changed = prev != dev;
  }
  ~DeviceGuard() {
    if (changed && prev >= 0) cudaSetDevice(prev);
  }
  bool changed = false;
};

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

namespace mfet {

int sm_count() {
  static std::atomic<int> cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  int sms = cached[dev].load(std::memory_order_relaxed);
  if (sms == 0) {
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) {
      cudaGetLastError();
      return 148;  // not cached: asked again next time
    }
    cached[dev].store(sms, std::memory_order_relaxed);
  }
  return sms;
}

}  // namespace mfet

extern "C" {

uint64_t mfet_row_bytes(uint32_t dim, uint32_t dtype) {
  switch (dtype) {
    case MFET_F32: return (uint64_t)dim * 4;
    case MFET_F16:
    case MFET_BF16: return (uint64_t)dim * 2;
    case MFET_INT4: return ((uint64_t)dim / 2 + 4 + 15) / 16 * 16;
    default: return 0;
  }
}

const char* mfet_status_string(int status) {
  switch (status) {
    case MFET_OK: return "ok";
    case MFET_ERR_INVALID_ARG: return "invalid argument";
    case MFET_ERR_NOT_REGISTERED: return "host table memory not registered";
    case MFET_ERR_ALIGNMENT: return "pointer or stride not 16-byte aligned";
    case MFET_ERR_UNSUPPORTED_DIM: return "row bytes not a multiple of 16";
    case MFET_ERR_WORKSPACE: return "workspace missing or too small";
    case MFET_ERR_CUDA: return "CUDA runtime error";
    case MFET_ERR_TIMEOUT: return "device-side wait timed out";
    default: return "unknown status";
  }
}

int mfet_tables_create(const mfet_table_desc_t* descs, int32_t n_tables, int32_t device,
                       mfet_tables_t** out) {
  if (!descs || !out || n_tables < 1) return MFET_ERR_INVALID_ARG;
  *out = nullptr;
  std::vector<TableHost> tabs((size_t)n_tables);
  for (int32_t i = 0; i < n_tables; ++i) {
    const mfet_table_desc_t& d = descs[i];
    if (d.rows == 0 || d.rows >= (1ULL << 63) || d.dim == 0 || d.flags != 0) return MFET_ERR_INVALID_ARG;
    if (d.dtype > MFET_INT4 || d.location > MFET_LOC_HOST) return MFET_ERR_INVALID_ARG;
    if (d.dtype == MFET_INT4 && (d.dim % 8u) != 0) return MFET_ERR_UNSUPPORTED_DIM;
    const uint64_t rb = mfet_row_bytes(d.dim, d.dtype);
    if (rb == 0 || rb % 16 != 0) return MFET_ERR_UNSUPPORTED_DIM;
    const uint64_t stride = d.row_stride_bytes ? d.row_stride_bytes : rb;
    if (stride < rb) return MFET_ERR_INVALID_ARG;
    if (stride % 16 != 0) return MFET_ERR_ALIGNMENT;
    if (d.rows > 0xFFFFFFFFFFFFFFFFULL / (stride >> 4)) return MFET_ERR_INVALID_ARG;  // row offsets are kept in 16-byte units
    TableHost& t = tabs[(size_t)i];
    t.desc = d;
    t.row_bytes = rb;
    t.stride = stride;
    t.magic = host_magic(d.rows);
    if (d.location == MFET_LOC_DEVICE) {
      if (!d.data) return MFET_ERR_INVALID_ARG;
      if (!aligned16(d.data)) return MFET_ERR_ALIGNMENT;
      t.dev_ptr = static_cast<const uint8_t*>(d.data);
      t.registered = true;
    }
  }
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess) return MFET_ERR_CUDA;
  if (device < 0 || device >= ndev) return MFET_ERR_INVALID_ARG;
  DeviceGuard g(device);
  if (!g.ok) return MFET_ERR_CUDA;
  mfet_tables* h = new (std::nothrow) mfet_tables();
  if (!h) return MFET_ERR_CUDA;
  h->device = device;
  h->tables = std::move(tabs);
  bool ok = cudaHostAlloc((void**)&h->err_host, 64, cudaHostAllocMapped | cudaHostAllocPortable) == cudaSuccess;
  if (ok) {
    *h->err_host = 0;
    ok = cudaHostGetDevicePointer((void**)&h->err_dev, h->err_host, 0) == cudaSuccess;
  }
  // host-table slots are the long pole of a hybrid batch (their rows cross PCIe), so their
  // kernels get the SMs first when they compete with the pooling of the device tables
  int prio_lo = 0, prio_hi = 0;
  ok = ok && cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess;
  ok = ok && cudaStreamCreateWithPriority(&h->side, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
  ok = ok && cudaStreamCreateWithPriority(&h->fetch, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
  for (int i = 0; i < 2; ++i) {
    ok = ok && cudaEventCreateWithFlags(&h->ev_dedup[i], cudaEventDisableTiming) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&h->ev_fetch[i], cudaEventDisableTiming) == cudaSuccess;
  }
  ok = ok && cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) == cudaSuccess;
  ok = ok && cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) == cudaSuccess;
  if (!ok) {
    mfet_tables_destroy(h);
    return MFET_ERR_CUDA;
  }
  *out = h;
  return MFET_OK;
}

int mfet_tables_destroy(mfet_tables_t* t) {
  if (!t) return MFET_OK;
  DeviceGuard g(t->device);
  if (t->side) {
    cudaStreamSynchronize(t->side);
    cudaStreamDestroy(t->side);
  }
  if (t->fetch) {
    cudaStreamSynchronize(t->fetch);
    cudaStreamDestroy(t->fetch);
  }
  for (int i = 0; i < 2; ++i) {
    if (t->ev_dedup[i]) cudaEventDestroy(t->ev_dedup[i]);
    if (t->ev_fetch[i]) cudaEventDestroy(t->ev_fetch[i]);
  }
  if (t->ev_fork) cudaEventDestroy(t->ev_fork);
  if (t->ev_join) cudaEventDestroy(t->ev_join);
  for (int i = 0; i < 4; ++i)
    if (t->prof_ev[i]) cudaEventDestroy(t->prof_ev[i]);
  for (TableHost& tb : t->tables)
    if (tb.pinned_by_us && tb.host_ptr) cudaHostUnregister(tb.host_ptr);
  if (t->err_host) cudaFreeHost(t->err_host);
  delete t;
  return MFET_OK;
}

int mfet_host_tables_register(mfet_tables_t* t, int32_t table_id, void* host_ptr, uint64_t bytes,
                              uint32_t flags) {
  if (!t || !host_ptr || table_id < 0 || table_id >= (int32_t)t->tables.size() || (flags & ~1u))
    return MFET_ERR_INVALID_ARG;
  TableHost& tb = t->tables[(size_t)table_id];
  if (tb.desc.location != MFET_LOC_HOST || tb.registered) return MFET_ERR_INVALID_ARG;
  if (!aligned16(host_ptr)) return MFET_ERR_ALIGNMENT;
  const uint64_t need = (tb.desc.rows - 1) * tb.stride + tb.row_bytes;
  if (bytes < need) return MFET_ERR_INVALID_ARG;
  DeviceGuard g(t->device);
  if (!g.ok) return MFET_ERR_CUDA;
  if (!(flags & 1u)) {
    if (cudaHostRegister(host_ptr, bytes, cudaHostRegisterMapped | cudaHostRegisterPortable) != cudaSuccess) {
      cudaGetLastError();
      return MFET_ERR_CUDA;
    }
    tb.pinned_by_us = true;
  }
  void* dptr = nullptr;
  if (cudaHostGetDevicePointer(&dptr, host_ptr, 0) != cudaSuccess) {
    cudaGetLastError();
    if (tb.pinned_by_us) cudaHostUnregister(host_ptr);
    tb.pinned_by_us = false;
    return MFET_ERR_CUDA;
  }
  tb.host_ptr = host_ptr;
  tb.dev_ptr = static_cast<const uint8_t*>(dptr);
  tb.registered = true;
  return MFET_OK;
}

int mfet_hash_ids(const mfet_tables_t* t, int32_t table_id, const uint64_t* ids, int64_t n,
                  int64_t* rows_out, mfet_stream_t stream) {
  if (!t || table_id < 0 || table_id >= (int32_t)t->tables.size() || n < 0) return MFET_ERR_INVALID_ARG;
  if (n == 0) return MFET_OK;
  if (!ids || !rows_out) return MFET_ERR_INVALID_ARG;
  const TableHost& tb = t->tables[(size_t)table_id];
  DeviceGuard g(t->device);
  if (!g.ok) return MFET_ERR_CUDA;
  if (launch_hash(ids, n, tb.desc.hash_seed, tb.desc.rows, tb.magic, rows_out, (cudaStream_t)stream) != cudaSuccess)
    return MFET_ERR_CUDA;
  const_cast<mfet_tables_t*>(t)->launches += 1;
  return MFET_OK;
}

int mfet_table_fill(void* data, uint64_t row0, uint64_t n_rows, uint32_t dim, uint32_t dtype,
                    uint64_t row_stride_bytes, uint64_t value_key, uint32_t value_mode,
                    mfet_stream_t stream) {
  if (!data || dim == 0 || dtype > MFET_INT4 || value_mode > MFET_VAL_GRID) return MFET_ERR_INVALID_ARG;
  if (dtype == MFET_INT4 && (dim % 8u) != 0) return MFET_ERR_UNSUPPORTED_DIM;
  const uint64_t rb = mfet_row_bytes(dim, dtype);
  if (rb == 0 || rb % 16 != 0) return MFET_ERR_UNSUPPORTED_DIM;
  const uint64_t stride = row_stride_bytes ? row_stride_bytes : rb;
  if (stride < rb) return MFET_ERR_INVALID_ARG;
  if (stride % 16 != 0 || !aligned16(data)) return MFET_ERR_ALIGNMENT;
  if (launch_fill(data, row0, n_rows, dim, dtype, stride, value_key, value_mode, (cudaStream_t)stream) != cudaSuccess)
    return MFET_ERR_CUDA;
  return MFET_OK;
}

int mfet_query_status(mfet_tables_t* t, uint32_t* device_error_bits, int32_t clear) {
  if (!t || !device_error_bits) return MFET_ERR_INVALID_ARG;
  *device_error_bits = *(volatile uint32_t*)t->err_host;
  if (clear) *(volatile uint32_t*)t->err_host = 0;
  return MFET_OK;
}

int mfet_tables_set_version(mfet_tables_t* t, uint64_t version) {
  if (!t) return MFET_ERR_INVALID_ARG;
  t->version = version;
  return MFET_OK;
}

int mfet_tables_version(const mfet_tables_t* t, uint64_t* version) {
  if (!t || !version) return MFET_ERR_INVALID_ARG;
  *version = t->version;
  return MFET_OK;
}

int mfet_launch_count(const mfet_tables_t* t, uint64_t* launches) {
  if (!t || !launches) return MFET_ERR_INVALID_ARG;
  *launches = t->launches;
  return MFET_OK;
}

int mfet_set_option(mfet_tables_t* t, int32_t option, int64_t value) {
  if (!t) return MFET_ERR_INVALID_ARG;
  switch (option) {
    case MFET_OPT_GROUP_POLICY:
      if (value < 0 || value > 2) return MFET_ERR_INVALID_ARG;
      t->group_policy = (int32_t)value;
      return MFET_OK;
    case MFET_OPT_PROFILE:
      if (value != 0 && value != 1) return MFET_ERR_INVALID_ARG;
      if (value == 1 && !t->prof_ev[0]) {
        DeviceGuard g(t->device);
        for (int i = 0; i < 4; ++i)
          if (cudaEventCreate(&t->prof_ev[i]) != cudaSuccess) return MFET_ERR_CUDA;
      }
      t->profile = (int32_t)value;
      t->prof_valid = false;
      return MFET_OK;
    case MFET_OPT_TILE:
      if (value != 0 && (value < 8 || value > kMaxTile)) return MFET_ERR_INVALID_ARG;
      t->tile = (int32_t)value;
      return MFET_OK;
    case MFET_OPT_OVERLAP_LAUNCHES:
      if (value != 0 && value != 1) return MFET_ERR_INVALID_ARG;
      t->overlap = (int32_t)value;
      return MFET_OK;
    case MFET_OPT_STAGE_IDS:
      if (value != 0 && (value < 32 || value > kStageMax)) return MFET_ERR_INVALID_ARG;
      t->stage_cap = (int32_t)value;
      return MFET_OK;
    default: return MFET_ERR_INVALID_ARG;
  }
}

int mfet_profile_read(mfet_tables_t* t, float* stage_ms) {
  if (!t || !stage_ms) return MFET_ERR_INVALID_ARG;
  if (!t->profile || !t->prof_valid) return MFET_ERR_INVALID_ARG;
  DeviceGuard g(t->device);
  if (cudaEventSynchronize(t->prof_ev[3]) != cudaSuccess) return MFET_ERR_CUDA;
  for (int i = 0; i < 3; ++i)
    if (cudaEventElapsedTime(&stage_ms[i], t->prof_ev[i], t->prof_ev[i + 1]) != cudaSuccess) return MFET_ERR_CUDA;
  return MFET_OK;
}

int mfet_workspace_bytes(const mfet_tables_t* t, int64_t max_ids, uint64_t* bytes) {
  if (!t || !bytes || max_ids < 0 || max_ids >= (1ll << 30) - 1) return MFET_ERR_INVALID_ARG;
  uint64_t max_row_bytes = 16;
  for (const TableHost& tb : t->tables)
    if (tb.desc.location == MFET_LOC_HOST && tb.row_bytes > max_row_bytes) max_row_bytes = tb.row_bytes;
  *bytes = workspace_layout(max_ids, max_row_bytes, nullptr);
  return MFET_OK;
}

int mfet_set_workspace(mfet_tables_t* t, void* dev_ptr, uint64_t bytes, int64_t max_ids) {
  if (!t || max_ids < 0 || max_ids >= (1ll << 30) - 1) return MFET_ERR_INVALID_ARG;
  if (!dev_ptr) {
    t->ws = nullptr;
    t->ws_bytes = 0;
    t->ws_max_ids = 0;
    return MFET_OK;
  }
  if (reinterpret_cast<uintptr_t>(dev_ptr) & 255u) return MFET_ERR_ALIGNMENT;
  uint64_t need = 0;
  int rc = mfet_workspace_bytes(t, max_ids, &need);
  if (rc != MFET_OK) return rc;
  if (bytes < need) return MFET_ERR_WORKSPACE;
  {
    // the dedup's digit totals inside the workspace must start at zero (its kernels leave them at zero)
    WsLayout L;
    workspace_layout(max_ids, 16, &L);
    DeviceGuard g(t->device);
    if (!g.ok || cudaMemset(static_cast<uint8_t*>(dev_ptr) + L.counters, 0, 64) != cudaSuccess ||
        cudaMemset(static_cast<uint8_t*>(dev_ptr) + L.hist, 0, kDedupTotalsBytes) != cudaSuccess)
      return MFET_ERR_CUDA;
  }
  t->ws = dev_ptr;
  t->ws_bytes = bytes;
  t->ws_max_ids = max_ids;
  return MFET_OK;
}

int mfet_host_prefetch(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids,
                       const int64_t* offsets, const int32_t* table_ids, mfet_stream_t stream_) {
  if (!t || !shape || !table_ids || !shape->slot_feature || !ids || !offsets) return MFET_ERR_INVALID_ARG;
  const int32_t B = shape->batch, F = shape->n_features, L = shape->n_slots;
  if (B < 1 || F < 1 || L < 1 || (shape->flags & ~3)) return MFET_ERR_INVALID_ARG;
  int host_slot = -1, n_host = 0;
  for (int32_t s = 0; s < L; ++s) {
    const int32_t ti = table_ids[s], f = shape->slot_feature[s];
    if (ti < 0 || ti >= (int32_t)t->tables.size() || f < 0 || f >= F) return MFET_ERR_INVALID_ARG;
    const TableHost& tb = t->tables[(size_t)ti];
    if (!tb.registered) return MFET_ERR_NOT_REGISTERED;
    if (tb.desc.location == MFET_LOC_HOST) {
      host_slot = s;
      ++n_host;
    }
  }
  if (n_host != 1) return MFET_ERR_INVALID_ARG;
  if (!t->ws || t->ws_max_ids <= 0) return MFET_ERR_WORKSPACE;
  if (t->prefetched - t->consumed >= 2) return MFET_ERR_INVALID_ARG;  // both result sets are taken
  if ((reinterpret_cast<uintptr_t>(ids) & 7u) || (reinterpret_cast<uintptr_t>(offsets) & 7u)) return MFET_ERR_ALIGNMENT;
  DeviceGuard g(t->device);
  if (!g.ok) return MFET_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_;
  BagParams p;
  std::memset(&p, 0, sizeof(p));
  p.ids = ids;
  p.offsets = offsets;
  p.err = t->err_dev;
  p.batch = B;
  p.n_features = F;
  p.flags = (uint32_t)(shape->flags & 1);
  // the internal stream starts after what `stream` holds now (the batch's inputs) and is not joined back
  if (cudaEventRecord(t->ev_fork, stream) != cudaSuccess) return MFET_ERR_CUDA;
  if (cudaStreamWaitEvent(t->side, t->ev_fork, 0) != cudaSuccess) return MFET_ERR_CUDA;
  const TableHost& tb = t->tables[(size_t)table_ids[host_slot]];
  int rc = run_host_slot(t, tb, p, shape->slot_feature[host_slot], MFET_POOL_SUM, 0, t->side, 1,
                         (int)(t->prefetched & 1u));
  if (rc != MFET_OK) return rc;
  t->prefetched += 1;
  return MFET_OK;
}

int mfet_embedding_bag_forward(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids,
                               const int64_t* offsets, const float* weights, const int32_t* table_ids,
                               const int32_t* pooling, float* out, mfet_stream_t stream_) {
  if (!t || !shape || !table_ids || !pooling || !shape->slot_feature) return MFET_ERR_INVALID_ARG;
  const int32_t B = shape->batch, F = shape->n_features, L = shape->n_slots;
  if (B < 0 || F < 1 || L < 1 || (shape->flags & ~3)) return MFET_ERR_INVALID_ARG;
  const bool use_prefetch = (shape->flags & MFET_BATCH_PREFETCHED) != 0;
  cudaStream_t stream = (cudaStream_t)stream_;

  // validate slots, lay out the output columns
  int64_t total_dim = 0;
  bool any_wsum = false, any_host = false;
  int n_host_slots = 0;
  for (int32_t s = 0; s < L; ++s) {
    const int32_t ti = table_ids[s], f = shape->slot_feature[s];
    if (ti < 0 || ti >= (int32_t)t->tables.size() || f < 0 || f >= F) return MFET_ERR_INVALID_ARG;
    if (pooling[s] < MFET_POOL_SUM || pooling[s] > MFET_POOL_WSUM) return MFET_ERR_INVALID_ARG;
    const TableHost& tb = t->tables[(size_t)ti];
    if (!tb.registered) return MFET_ERR_NOT_REGISTERED;
    any_wsum |= pooling[s] == MFET_POOL_WSUM;
    any_host |= tb.desc.location == MFET_LOC_HOST;
    n_host_slots += tb.desc.location == MFET_LOC_HOST;
    total_dim += tb.desc.dim;
  }
  const int64_t out_ld = shape->out_ld ? shape->out_ld : total_dim;
  if (out_ld < total_dim) return MFET_ERR_INVALID_ARG;
  if (B == 0) return MFET_OK;
  if (!ids || !offsets || !out) return MFET_ERR_INVALID_ARG;
  if (any_wsum && !weights) return MFET_ERR_INVALID_ARG;
  if (any_host && (!t->ws || t->ws_max_ids <= 0)) return MFET_ERR_WORKSPACE;
  // a prefetched batch has exactly one host-table slot and an unconsumed prefetch; a plain
  // batch with a host-table slot must not cut in between a prefetch and its forward
  if (use_prefetch && (n_host_slots != 1 || t->consumed >= t->prefetched)) return MFET_ERR_INVALID_ARG;
  if (!use_prefetch && any_host && t->consumed != t->prefetched) return MFET_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(ids) & 7u) || (reinterpret_cast<uintptr_t>(offsets) & 7u) ||
      (reinterpret_cast<uintptr_t>(out) & 3u) || (reinterpret_cast<uintptr_t>(weights) & 3u))
    return MFET_ERR_ALIGNMENT;

  DeviceGuard g(t->device);
  if (!g.ok) return MFET_ERR_CUDA;

  BagParams p;
  std::memset(&p, 0, sizeof(p));
  p.ids = ids;
  p.offsets = offsets;
  p.weights = weights;
  p.out = out;
  p.err = t->err_dev;
  p.out_ld = out_ld;
  p.batch = B;
  p.n_features = F;
  p.flags = (uint32_t)(shape->flags & 1);
  if (aligned16(out) && out_ld % 4 == 0) p.flags |= 2u;
  if (t->overlap) p.flags |= 16u;
  p.group_policy = t->group_policy;
  // samples per block and staging capacity: the caller's options, else chosen at launch (0)
  p.tile = t->tile;
  p.stage_cap = t->stage_cap;

  // host-table slots go to the side stream, forked from and joined to `stream`
  bool forked = false;
  int64_t col = 0;
  int n = 0;
  auto flush = [&]() -> int {
    if (n == 0) return MFET_OK;
    // widest rows first: their blocks run longest, so they should not be the last to start
    std::stable_sort(p.slot, p.slot + n, [](const SlotDev& a, const SlotDev& b) {
      return (uint32_t)a.chunks * (a.dtype == MFET_INT4 ? 4u : 16u) > (uint32_t)b.chunks * (b.dtype == MFET_INT4 ? 4u : 16u);
    });
    p.n_slots = n;
    if (launch_bag(p, stream) != cudaSuccess) return MFET_ERR_CUDA;
    t->launches += 1;
    n = 0;
    return MFET_OK;
  };
  for (int32_t s = 0; s < L; ++s) {
    const TableHost& tb = t->tables[(size_t)table_ids[s]];
    if (tb.desc.location == MFET_LOC_HOST) {
      if (!forked) {
        if (cudaEventRecord(t->ev_fork, stream) != cudaSuccess) return MFET_ERR_CUDA;
        if (cudaStreamWaitEvent(t->side, t->ev_fork, 0) != cudaSuccess) return MFET_ERR_CUDA;
        forked = true;
      }
      int rc = run_host_slot(t, tb, p, shape->slot_feature[s], pooling[s], (uint32_t)col, t->side,
                             use_prefetch ? 2 : 3, (int)((use_prefetch ? t->consumed : t->prefetched) & 1u));
      if (rc != MFET_OK) return rc;
      if (use_prefetch) t->consumed += 1;
    } else {
      // rows wider than 512 bytes are covered by several entries of <= 32 chunks
      // a lane's chunk: 16 bytes, or 4 bytes of codes for INT4 rows
      const bool int4 = tb.desc.dtype == MFET_INT4;
      const uint32_t chunk_bytes = int4 ? 4u : 16u;
      const uint32_t chunks_total = int4 ? tb.desc.dim / 8u : (uint32_t)(tb.row_bytes / 16);
      const uint32_t epc = tb.desc.dtype == MFET_F32 ? 4u : 8u;  // elements per chunk
      for (uint32_t c0 = 0; c0 < chunks_total; c0 += 32) {
        if (n == kMaxSlotsPerLaunch) {
          int rc = flush();
          if (rc != MFET_OK) return rc;
        }
        SlotDev& sd = p.slot[n++];
        const uint32_t ch = chunks_total - c0 < 32 ? chunks_total - c0 : 32;
        sd.table = tb.dev_ptr + (uint64_t)c0 * chunk_bytes;
        sd.meta_off = int4 ? tb.desc.dim / 2u - c0 * chunk_bytes : 0u;
        sd.rows = tb.desc.rows;
        sd.magic = tb.magic;
        sd.seed = tb.desc.hash_seed;
        sd.stride = tb.stride;
        sd.feature = (uint32_t)shape->slot_feature[s];
        sd.col_off = (uint32_t)(col + (uint64_t)c0 * epc);
        sd.chunks = (uint16_t)ch;
        sd.dtype = (uint8_t)tb.desc.dtype;
        sd.pooling = (uint8_t)pooling[s];
        uint8_t lg = 1;
        while ((1u << lg) < ch) ++lg;
        sd.lpr_log2 = lg;
        sd.narrow = (tb.desc.rows <= 0xFFFFFFFFULL && tb.stride <= 0xFFFFFFFFULL) ? 1 : 0;
      }
    }
    col += tb.desc.dim;
  }
  int rc = flush();
  if (rc != MFET_OK) return rc;
  if (forked) {
    if (cudaEventRecord(t->ev_join, t->side) != cudaSuccess) return MFET_ERR_CUDA;
    if (cudaStreamWaitEvent(stream, t->ev_join, 0) != cudaSuccess) return MFET_ERR_CUDA;
  }
  return MFET_OK;
}

}  // extern "C"
