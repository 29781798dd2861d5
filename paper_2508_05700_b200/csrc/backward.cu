// K-backward: gradient of the pooled output with respect to the rows of one slot's
// table, as a sparse list (ascending distinct rows + one fp32 gradient vector each).
// The lookups of the slot are hashed and sorted by row with the dedup machinery; every
// distinct row then sums coef * grad_out[bag] over its run of lookups in input order
// (the sort is stable), so the result does not depend on timing.
#include <cstring>

#include "common.cuh"

using namespace mfet;

namespace mfet {

namespace {

constexpr int kBwdRegs = 4;  // gradient columns per lane per pass (32 lanes x 4 = 128 columns)

// One warp per distinct row u: its run is sorted positions [seg_start[u], seg_start[u+1])
// (or n for the last row). For every lookup of the run: find its bag by bisection in the
// feature's offsets, take coef = 1 (SUM), 1/len (MEAN) or weights[i] (WSUM), and add
// coef * grad_out[bag, col + d]. Lanes own columns d = lane, lane + 32, ...
__global__ void __launch_bounds__(256) backward_rows_kernel(const uint32_t* __restrict__ sorted_pos,
                                                            const int32_t* __restrict__ seg_start,
                                                            const int64_t* __restrict__ n_unique, NSrc ns,
                                                            const int64_t* __restrict__ offsets_f, int32_t batch,
                                                            const float* __restrict__ weights, int32_t pooling,
                                                            const float* __restrict__ grad_out, int64_t out_ld,
                                                            uint32_t col, uint32_t dim, float* __restrict__ grad_vals) {
  const int64_t feat_lo = offsets_f[0];
  int64_t n = offsets_f[batch] - feat_lo;
  if (n < 0 || n > ns.cap) n = 0;
  const int64_t nu = *n_unique;
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t u = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5; u < nu; u += warps) {
    const int64_t j0 = seg_start[u];
    const int64_t j1 = (u + 1 < nu) ? (int64_t)seg_start[u + 1] : n;
    for (uint32_t d0 = 0; d0 < dim; d0 += 32 * kBwdRegs) {
      float acc[kBwdRegs];
#pragma unroll
      for (int k = 0; k < kBwdRegs; ++k) acc[k] = 0.f;
      for (int64_t j = j0; j < j1; ++j) {
        const int64_t i = feat_lo + sorted_pos[j];  // position of the lookup in ids / weights
        // bag of i: the last b with offsets_f[b] <= i
        int lo = 0, hi = batch;
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (offsets_f[mid] <= i) lo = mid;
          else hi = mid;
        }
        float coef = 1.f;
        if (pooling == MFET_POOL_MEAN) coef = __fdiv_rn(1.f, (float)(offsets_f[lo + 1] - offsets_f[lo]));
        else if (pooling == MFET_POOL_WSUM) coef = weights[i];
        const float* g = grad_out + (int64_t)lo * out_ld + col + d0;
#pragma unroll
        for (int k = 0; k < kBwdRegs; ++k) {
          const uint32_t d = d0 + lane + 32 * k;
          if (d < dim) acc[k] = fmaf(coef, g[lane + 32 * k], acc[k]);
        }
      }
#pragma unroll
      for (int k = 0; k < kBwdRegs; ++k) {
        const uint32_t d = d0 + lane + 32 * k;
        if (d < dim) grad_vals[u * dim + d] = acc[k];
      }
    }
  }
}

}  // namespace

cudaError_t launch_backward(const uint32_t* sorted_pos, const int32_t* seg_start, const int64_t* n_unique, NSrc ns,
                            const int64_t* offsets_f, int32_t batch, const float* weights, int32_t pooling,
                            const float* grad_out, int64_t out_ld, uint32_t col, uint32_t dim, float* grad_vals,
                            cudaStream_t s) {
  backward_rows_kernel<<<sm_count() * 8, 256, 0, s>>>(sorted_pos, seg_start, n_unique, ns, offsets_f, batch, weights, pooling,
                                               grad_out, out_ld, col, dim, grad_vals);
  return cudaGetLastError();
}

}  // namespace mfet

extern "C" int mfet_embedding_bag_backward(mfet_tables_t* t, const mfet_batch_shape_t* shape, const uint64_t* ids,
                                           const int64_t* offsets, const float* weights, const int32_t* table_ids,
                                           const int32_t* pooling, const float* grad_out, int32_t slot,
                                           int64_t* grad_rows, float* grad_vals, int64_t* n_rows,
                                           mfet_stream_t stream_) {
  if (!t || !shape || !table_ids || !pooling || !shape->slot_feature) return MFET_ERR_INVALID_ARG;
  const int32_t B = shape->batch, F = shape->n_features, L = shape->n_slots;
  if (B < 1 || F < 1 || L < 1 || (shape->flags & ~1) || slot < 0 || slot >= L) return MFET_ERR_INVALID_ARG;
  if (!ids || !offsets || !grad_out || !grad_rows || !grad_vals || !n_rows) return MFET_ERR_INVALID_ARG;
  int64_t total_dim = 0, col = 0;
  for (int32_t s = 0; s < L; ++s) {
    const int32_t ti = table_ids[s], f = shape->slot_feature[s];
    if (ti < 0 || ti >= (int32_t)t->tables.size() || f < 0 || f >= F) return MFET_ERR_INVALID_ARG;
    if (pooling[s] < MFET_POOL_SUM || pooling[s] > MFET_POOL_WSUM) return MFET_ERR_INVALID_ARG;
    if (s == slot) col = total_dim;
    total_dim += t->tables[(size_t)ti].desc.dim;
  }
  const int64_t out_ld = shape->out_ld ? shape->out_ld : total_dim;
  if (out_ld < total_dim) return MFET_ERR_INVALID_ARG;
  if (pooling[slot] == MFET_POOL_WSUM && !weights) return MFET_ERR_INVALID_ARG;
  if (!t->ws || t->ws_max_ids <= 0) return MFET_ERR_WORKSPACE;
  if (t->consumed != t->prefetched) return MFET_ERR_INVALID_ARG;  // the workspace holds a prefetched batch
  const TableHost& tb = t->tables[(size_t)table_ids[slot]];
  const int32_t f = shape->slot_feature[slot];
  WsLayout Lw;
  if (workspace_layout(t->ws_max_ids, 16, &Lw) > t->ws_bytes) return MFET_ERR_WORKSPACE;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != t->device && cudaSetDevice(t->device) != cudaSuccess) return MFET_ERR_CUDA;
  cudaStream_t stream = (cudaStream_t)stream_;
  uint8_t* ws = (uint8_t*)t->ws;
  HashArgs h{ids, tb.desc.hash_seed, tb.desc.rows, tb.magic, (uint32_t)(shape->flags & 1)};
  const uint32_t* sorted_pos = nullptr;
  DedupArgs a;
  std::memset(&a, 0, sizeof(a));
  a.ns = NSrc{offsets, (int64_t)f * B, (int64_t)(f + 1) * B, 0, t->ws_max_ids};
  a.hash = &h;
  a.max_key = tb.desc.rows - 1;
  a.ws = ws;
  a.layout = Lw;
  a.uniq = grad_rows;
  a.inverse = (int32_t*)(ws + Lw.inverse);
  a.n_unique = n_rows;
  a.src = (int32_t*)(ws + Lw.src);  // run starts
  a.err = t->err_dev;
  a.sorted_pos_out = &sorted_pos;
  int rc = MFET_OK;
  if (launch_dedup(a, &t->launches, stream) != cudaSuccess) rc = MFET_ERR_CUDA;
  if (rc == MFET_OK &&
      launch_backward(sorted_pos, a.src, n_rows, a.ns, offsets + (int64_t)f * B, B, weights, pooling[slot], grad_out,
                      out_ld, (uint32_t)col, tb.desc.dim, grad_vals, stream) != cudaSuccess)
    rc = MFET_ERR_CUDA;
  if (rc == MFET_OK) t->launches += 1;
  if (prev != t->device) cudaSetDevice(prev);
  return rc;
}
