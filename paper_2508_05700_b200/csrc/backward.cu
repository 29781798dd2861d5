// K-backward: gradient of the pooled output with respect to the rows of one slot's
// table, as a sparse list (ascending distinct rows + one fp32 gradient vector each).
// The lookups of the slot are hashed and sorted by row with the dedup machinery; every
// distinct row then sums coef * grad_out[bag] over its run of lookups (the sort is stable:
// a run is in input order), long runs in pieces that are combined in a fixed order, so the
// result does not depend on timing.
#include <cstring>

#include "common.cuh"

using namespace mfet;

static constexpr int32_t kBwdChunkDefault = 256;  // most sorted lookups per warp of the gradient pass

namespace mfet {

namespace {

constexpr int kBwdRegs = 4;      // gradient columns per lane per pass (32 lanes x 4 = 128 columns)
constexpr int kBwdBatch = 8;     // gradient rows that a warp requests together

// The lookups of the slot, sorted by table row (stably, so a row's run is in input order), are
// cut into CHUNKS of `chunk` consecutive sorted positions, one warp per chunk; a hot row's run of
// thousands of lookups is thereby spread over many warps instead of being one warp's serial loop.
// Inside a chunk the warp works on 32 lookups at a time: every lane finds the bag of one lookup
// (bisection in the feature's offsets) and its coefficient - 1 (SUM), 1/len (MEAN) or weights[i]
// (WSUM) -, then the 32 lookups are added one after the other, lanes owning the columns
// d = lane, lane + 32, ... of grad_out[bag, col + d]. A row whose run lies inside the chunk is
// stored directly. A run that crosses a chunk boundary leaves a partial sum in the chunk's HEAD
// slot (the run began before the chunk) or TAIL slot (it goes on after it);
// backward_combine_kernel adds the partial sums of such a row in chunk order. The order of the
// additions depends only on the inputs and the chunk length.
__global__ void __launch_bounds__(256) backward_chunks_kernel(const uint32_t* __restrict__ sorted_pos,
                                                              const int32_t* __restrict__ inverse,
                                                              const int32_t* __restrict__ seg_start,
                                                              const int64_t* __restrict__ n_unique, NSrc ns,
                                                              const int64_t* __restrict__ offsets_f, int32_t batch,
                                                              const float* __restrict__ weights, int32_t pooling,
                                                              const float* __restrict__ grad_out, int64_t out_ld,
                                                              uint32_t col, uint32_t dim, int32_t chunk,
                                                              float* __restrict__ partial, float* __restrict__ grad_vals,
                                                              uint32_t* err) {
  const int64_t feat_lo = offsets_f[0];
  int64_t n = offsets_f[batch] - feat_lo;
  if (n < 0 || n > ns.cap) n = 0;
  const int64_t nu = *n_unique;
  const int lane = threadIdx.x & 31;
  const int64_t k = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;  // this warp's chunk
  const int64_t c0 = k * chunk;
  if (c0 >= n) return;
  const int64_t c1 = c0 + chunk < n ? c0 + chunk : n;
  float* head = partial + (size_t)(2 * k) * dim;
  float* tail = head + dim;
  for (uint32_t d0 = 0; d0 < dim; d0 += 32 * kBwdRegs) {
    float acc[kBwdRegs];
#pragma unroll
    for (int r = 0; r < kBwdRegs; ++r) acc[r] = 0.f;
    int32_t cur = -1;  // distinct-row index of the run that acc belongs to
    auto flush = [&](int32_t u) {
      if (!MFET_IN_BOUNDS(err, u >= 0 && (int64_t)u < nu)) return;
      // run of row u: sorted positions [j0, j1)
      const int64_t j0 = seg_start[u];
      const int64_t j1 = ((int64_t)u + 1 < nu) ? (int64_t)seg_start[u + 1] : n;
      float* dst = (j0 >= c0 && j1 <= c1) ? grad_vals + (size_t)u * dim : (j0 < c0 ? head : tail);
#pragma unroll
      for (int r = 0; r < kBwdRegs; ++r) {
        const uint32_t d = d0 + lane + 32 * r;
        if (d < dim) dst[d] = acc[r];
        acc[r] = 0.f;
      }
    };
    for (int64_t j32 = c0; j32 < c1; j32 += 32) {
      // every lane: one lookup's row, bag and coefficient
      const int64_t j = j32 + lane;
      int32_t u = -1, bag = 0;
      float coef = 0.f;
      if (j < c1) {
        uint32_t pos = sorted_pos[j];
        if (!MFET_IN_BOUNDS(err, (int64_t)pos < n)) pos = 0;
        const int64_t i = feat_lo + pos;  // position of the lookup in ids / weights
        u = inverse[pos];
        int lo = 0, hi = batch;  // the last b with offsets_f[b] <= i
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (offsets_f[mid] <= i) lo = mid;
          else hi = mid;
        }
        bag = lo;
        coef = 1.f;
        if (pooling == MFET_POOL_MEAN) coef = __fdiv_rn(1.f, (float)(offsets_f[lo + 1] - offsets_f[lo]));
        else if (pooling == MFET_POOL_WSUM) coef = weights[i];
      }
      const int cnt = (int)(c1 - j32 < 32 ? c1 - j32 : 32);
      for (int t0 = 0; t0 < cnt; t0 += kBwdBatch) {
        float g[kBwdBatch][kBwdRegs];
#pragma unroll
        for (int t = 0; t < kBwdBatch; ++t) {  // the loads of a batch do not depend on one another
          const int32_t bt = __shfl_sync(0xFFFFFFFFu, bag, (t0 + t) & 31);
          const float* row = grad_out + (int64_t)bt * out_ld + col + d0;
#pragma unroll
          for (int r = 0; r < kBwdRegs; ++r) {
            const uint32_t d = d0 + lane + 32 * r;
            g[t][r] = (t0 + t < cnt && d < dim) ? __ldg(row + lane + 32 * r) : 0.f;
          }
        }
#pragma unroll
        for (int t = 0; t < kBwdBatch; ++t) {
          const int32_t ut = __shfl_sync(0xFFFFFFFFu, u, (t0 + t) & 31);
          const float ct = __shfl_sync(0xFFFFFFFFu, coef, (t0 + t) & 31);
          if (t0 + t < cnt) {
            if (ut != cur) {
              if (cur >= 0) flush(cur);
              cur = ut;
            }
#pragma unroll
            for (int r = 0; r < kBwdRegs; ++r) acc[r] = fmaf(ct, g[t][r], acc[r]);
          }
        }
      }
    }
    if (cur >= 0) flush(cur);
  }
}

// Rows whose run crosses a chunk boundary: the gradient is the TAIL slot of the chunk where the run
// begins, the HEAD slots of the chunks it covers entirely, and the HEAD slot of the chunk where it
// ends, added in that order. A warp looks at 32 rows at a time (one per lane: most runs lie inside
// one chunk and need nothing), then works through the ones that do with all its lanes on the
// columns. chunk = 1 << chunk_shift.
__global__ void __launch_bounds__(256) backward_combine_kernel(const int32_t* __restrict__ seg_start,
                                                               const int64_t* __restrict__ n_unique, NSrc ns,
                                                               const int64_t* __restrict__ offsets_f, int32_t batch,
                                                               uint32_t dim, int32_t chunk_shift,
                                                               const float* __restrict__ partial,
                                                               float* __restrict__ grad_vals) {
  int64_t n = offsets_f[batch] - offsets_f[0];
  if (n < 0 || n > ns.cap) n = 0;
  const int64_t nu = *n_unique;
  const int lane = threadIdx.x & 31;
  const int64_t warps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  for (int64_t u0 = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5) * 32; u0 < nu; u0 += warps * 32) {
    const int64_t u = u0 + lane;
    int64_t k0 = 0, k1 = 0;
    if (u < nu) {
      const int64_t j0 = seg_start[u];
      const int64_t j1 = (u + 1 < nu) ? (int64_t)seg_start[u + 1] : n;
      k0 = j0 >> chunk_shift;
      k1 = (j1 - 1) >> chunk_shift;
    }
    uint32_t todo = __ballot_sync(0xFFFFFFFFu, k0 != k1);  // runs inside one chunk were stored by the chunk's warp
    while (todo) {
      const int t = __ffs(todo) - 1;
      todo &= todo - 1;
      const int64_t a0 = __shfl_sync(0xFFFFFFFFu, k0, t), a1 = __shfl_sync(0xFFFFFFFFu, k1, t);
      // the loads of 8 chunks x 4 column groups are requested together (a hot row spans hundreds of
      // chunks); the additions of a column stay in chunk order
      for (uint32_t d0 = 0; d0 < dim; d0 += 32 * kBwdRegs) {
        float s[kBwdRegs];
#pragma unroll
        for (int r = 0; r < kBwdRegs; ++r) {
          const uint32_t d = d0 + lane + 32 * r;
          s[r] = d < dim ? partial[(size_t)(2 * a0 + 1) * dim + d] : 0.f;
        }
        for (int64_t kb = a0 + 1; kb <= a1; kb += 8) {
          float v[8][kBwdRegs];
#pragma unroll
          for (int j = 0; j < 8; ++j)
#pragma unroll
            for (int r = 0; r < kBwdRegs; ++r) {
              const uint32_t d = d0 + lane + 32 * r;
              v[j][r] = (kb + j <= a1 && d < dim) ? __ldcg(partial + (size_t)(2 * (kb + j)) * dim + d) : 0.f;
            }
#pragma unroll
          for (int j = 0; j < 8; ++j)
            if (kb + j <= a1) {
#pragma unroll
              for (int r = 0; r < kBwdRegs; ++r) s[r] += v[j][r];
            }
        }
#pragma unroll
        for (int r = 0; r < kBwdRegs; ++r) {
          const uint32_t d = d0 + lane + 32 * r;
          if (d < dim) grad_vals[(size_t)(u0 + t) * dim + d] = s[r];
        }
      }
    }
  }
}

}  // namespace

// partial: room for 2 * dim floats per chunk of `chunk` sorted lookups, capacity ns.cap lookups.
cudaError_t launch_backward(const uint32_t* sorted_pos, const int32_t* inverse, const int32_t* seg_start,
                            const int64_t* n_unique, NSrc ns, const int64_t* offsets_f, int32_t batch,
                            const float* weights, int32_t pooling, const float* grad_out, int64_t out_ld, uint32_t col,
                            uint32_t dim, int32_t chunk, float* partial, float* grad_vals, uint32_t* err,
                            cudaStream_t s) {
  const int64_t chunks = (ns.cap + chunk - 1) / chunk;
  const int64_t blocks = (chunks + 7) / 8;  // 8 warps per block, one chunk per warp
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  backward_chunks_kernel<<<(unsigned)(blocks > 0 ? blocks : 1), 256, 0, s>>>(
      sorted_pos, inverse, seg_start, n_unique, ns, offsets_f, batch, weights, pooling, grad_out, out_ld, col, dim, chunk,
      partial, grad_vals, err);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  if (chunks <= 1) return cudaSuccess;  // one chunk holds every run: nothing to combine
  int shift = 0;
  while ((1 << shift) < chunk) ++shift;  // chunk is a power of two whenever there is more than one
  int64_t cblocks = (ns.cap + 32 * 8 - 1) / (32 * 8);  // 8 warps per block, 32 rows per warp and round
  if (cblocks > (int64_t)sm_count() * 8) cblocks = (int64_t)sm_count() * 8;
  backward_combine_kernel<<<(unsigned)(cblocks > 0 ? cblocks : 1), 256, 0, s>>>(seg_start, n_unique, ns, offsets_f, batch,
                                                                            dim, shift, partial, grad_vals);
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
  // partial sums of runs that cross a chunk boundary go to the part of the workspace that the
  // sort does not use (from the miss list to the end): two vectors per chunk; a workspace too
  // small for that (tiny capacities) gets one chunk = one warp for everything
  float* partial = reinterpret_cast<float*>(ws + Lw.miss_rows);
  const uint64_t room = Lw.total - Lw.miss_rows;
  // short chunks spread the work over more warps, long ones keep a hot row's list of partial sums short:
  // 64 lookups per chunk up to 128 k lookups, 256 from 512 k; at least the shortest whose partial sums fit
  int32_t chunk = t->ws_max_ids > 512 * 1024 ? 256 : (t->ws_max_ids > 128 * 1024 ? 128 : 64);
  auto fits = [&](int32_t c) {
    return ((uint64_t)(t->ws_max_ids + c - 1) / c) * 2ull * tb.desc.dim * sizeof(float) <= room;
  };
  while (chunk < kBwdChunkDefault && !fits(chunk)) chunk *= 2;
  if (!fits(chunk)) {
    if (t->ws_max_ids > 0x7FFFFFE0LL) rc = MFET_ERR_WORKSPACE;
    else chunk = (int32_t)((t->ws_max_ids + 31) / 32 * 32);  // every run lies inside the one chunk: no partial sums
  }
  if (rc == MFET_OK &&
      launch_backward(sorted_pos, a.inverse, a.src, n_rows, a.ns, offsets + (int64_t)f * B, B, weights, pooling[slot],
                      grad_out, out_ld, (uint32_t)col, tb.desc.dim, chunk, partial, grad_vals, t->err_dev,
                      stream) != cudaSuccess)
    rc = MFET_ERR_CUDA;
  if (rc == MFET_OK) t->launches += 2;
  if (prev != t->device) cudaSetDevice(prev);
  return rc;
}
