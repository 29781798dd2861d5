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
constexpr int kBwdBatch = 8;     // gradient rows that a warp requests together (16: twice the registers, fewer warps resident)
constexpr int kBwdThreads = 64;   // two warps = two chunks per block (the kernel needs about 200 registers a thread)
constexpr int kBwdCoarse = 1024;   // offsets that the bag search keeps in shared memory
constexpr int kBwdOwn = 4;       // lookups whose row, bag and coefficient a lane works out side by side

// The lookups of the slot, sorted by table row (stably, so a row's run is in input order), are
// cut into CHUNKS of `chunk` consecutive sorted positions, one warp per chunk; a hot row's run of
// thousands of lookups is thereby spread over many warps instead of being one warp's serial loop.
// The warp takes its chunk 128 lookups at a time. First every lane finds, for up to four lookups
// of its own, the distinct-row index, the bag (bisection in the feature's offsets, the four
// searches side by side) and the coefficient - 1 (SUM), 1/len (MEAN) or weights[i] (WSUM). Then
// the lookups are added one after the other, lanes owning the columns d = lane, lane + 32, ... of
// grad_out[bag, col + d], eight gradient rows requested at a time; nothing in that loop waits for
// anything but those rows. A row whose run lies inside the chunk is stored directly. Only the
// chunk's first run can have begun before the chunk and only its last can go on after it (looked up
// once, ahead of the loop): such a run leaves a partial sum in the chunk's HEAD slot (it began
// before the chunk) or TAIL slot (it goes on after it); backward_combine_kernel adds the partial
// sums of such a row in chunk order. The order of the additions depends only on the inputs and
// the chunk length.
__global__ void __launch_bounds__(kBwdThreads) backward_chunks_kernel(const uint32_t* sorted_pos, const int32_t* inverse,
                                                              const int32_t* seg_start, const int64_t* n_unique, NSrc ns,
                                                              const int64_t* __restrict__ offsets_f, int32_t batch,
                                                              const float* __restrict__ weights, int32_t pooling,
                                                              const float* __restrict__ grad_out, int64_t out_ld,
                                                              uint32_t col, uint32_t dim, int32_t chunk,
                                                              float* __restrict__ partial, float* __restrict__ grad_vals,
                                                              uint32_t* err) {
  // Launched programmatically after the sort's last kernel: what that sort wrote (sorted_pos,
  // inverse, seg_start, n_unique) is read only after this wait, and through L2.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // The search for a lookup's bag starts in shared memory: all warps of the
  // GPU would otherwise ask L2 for the same few offsets (the middle one, the quartiles, ...) at
  // the same moment, one dependent step after the other. coarse[i] = offsets_f[i << coarse_shift].
  __shared__ int64_t coarse[kBwdCoarse + 1];
  int coarse_shift = 0;
  while ((batch >> coarse_shift) > kBwdCoarse) ++coarse_shift;
  const int n_coarse = ((batch - 1) >> coarse_shift) + 1;  // entries 0 .. n_coarse - 1 start a stretch of bags
  for (int i = threadIdx.x; i < n_coarse; i += kBwdThreads) coarse[i] = offsets_f[(int64_t)i << coarse_shift];
  __syncthreads();
  const int64_t feat_lo = offsets_f[0];
  int64_t n = offsets_f[batch] - feat_lo;
  if (n < 0 || n > ns.cap) n = 0;
  const int64_t nu = __ldcg(reinterpret_cast<const long long*>(n_unique));
  const int lane = threadIdx.x & 31;
  const int64_t k = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;  // this warp's chunk
  const int64_t c0 = k * chunk;
  if (c0 < n) {
    const int64_t c1 = c0 + chunk < n ? c0 + chunk : n;
    float* head = partial + (size_t)(2 * k) * dim;
    float* tail = head + dim;
    // the chunk's first and last run: do they reach beyond the chunk?
    int32_t u_first = -1, u_last = -1;
    bool first_began_before = false, last_goes_on = false;
    {
      int32_t ue = -1;
      if (lane < 2) {
        uint32_t pos = __ldcg(sorted_pos + (lane == 0 ? c0 : c1 - 1));
        if (!MFET_IN_BOUNDS(err, (int64_t)pos < n)) pos = 0;
        ue = __ldcg(inverse + pos);
        if (!MFET_IN_BOUNDS(err, ue >= 0 && (int64_t)ue < nu)) ue = 0;
      }
      bool beyond = false;
      if (lane == 0) beyond = (int64_t)__ldcg(seg_start + ue) < c0;
      if (lane == 1) beyond = ((int64_t)ue + 1 < nu ? (int64_t)__ldcg(seg_start + ue + 1) : n) > c1;
      u_first = __shfl_sync(0xFFFFFFFFu, ue, 0);
      u_last = __shfl_sync(0xFFFFFFFFu, ue, 1);
      first_began_before = __shfl_sync(0xFFFFFFFFu, (int)beyond, 0) != 0;
      last_goes_on = __shfl_sync(0xFFFFFFFFu, (int)beyond, 1) != 0;
    }
    for (uint32_t d0 = 0; d0 < dim; d0 += 32 * kBwdRegs) {
      float acc[kBwdRegs];
#pragma unroll
      for (int r = 0; r < kBwdRegs; ++r) acc[r] = 0.f;
      int32_t cur = -1;  // distinct-row index of the run that acc belongs to
      auto flush = [&](int32_t u) {
        float* dst = (u == u_first && first_began_before) ? head
                     : (u == u_last && last_goes_on)      ? tail
                                                          : grad_vals + (size_t)u * dim;
#pragma unroll
        for (int r = 0; r < kBwdRegs; ++r) {
          const uint32_t d = d0 + lane + 32 * r;
          if (d < dim) dst[d] = acc[r];
          acc[r] = 0.f;
        }
      };
      for (int64_t base = c0; base < c1; base += 32 * kBwdOwn) {
        // every lane: row, bag and coefficient of up to kBwdOwn lookups (lookup base + 32 q + lane)
        int32_t u[kBwdOwn], bag[kBwdOwn];
        float coef[kBwdOwn];
        int64_t at[kBwdOwn];  // position of the lookup in ids / weights
        int lo[kBwdOwn], hi[kBwdOwn];
#pragma unroll
        for (int q = 0; q < kBwdOwn; ++q) {
          const int64_t j = base + 32 * q + lane;
          uint32_t pos = j < c1 ? __ldcg(sorted_pos + j) : 0u;
          if (!MFET_IN_BOUNDS(err, (int64_t)pos < n)) pos = 0;
          at[q] = feat_lo + pos;
          u[q] = j < c1 ? __ldcg(inverse + pos) : -1;
          if (!MFET_IN_BOUNDS(err, j >= c1 || (u[q] >= 0 && (int64_t)u[q] < nu))) u[q] = 0;
          lo[q] = 0;
          hi[q] = j < c1 ? n_coarse : 1;  // the last coarse entry <= at ...
        }
        for (int step = n_coarse; step > 1; step = (step + 1) >> 1) {  // enough halvings for the widest search
#pragma unroll
          for (int q = 0; q < kBwdOwn; ++q)
            if (hi[q] - lo[q] > 1) {
              const int mid = (lo[q] + hi[q]) >> 1;
              if (coarse[mid] <= at[q]) lo[q] = mid;
              else hi[q] = mid;
            }
        }
#pragma unroll
        for (int q = 0; q < kBwdOwn; ++q) {  // ... then the last b with offsets_f[b] <= at inside its stretch
          const int64_t j = base + 32 * q + lane;
          lo[q] <<= coarse_shift;
          hi[q] = j < c1 ? min(lo[q] + (1 << coarse_shift), batch) : lo[q] + 1;
        }
        for (int step = 1 << coarse_shift; step > 1; step = (step + 1) >> 1) {
#pragma unroll
          for (int q = 0; q < kBwdOwn; ++q)
            if (hi[q] - lo[q] > 1) {
              const int mid = (lo[q] + hi[q]) >> 1;
              if (offsets_f[mid] <= at[q]) lo[q] = mid;
              else hi[q] = mid;
            }
        }
#pragma unroll
        for (int q = 0; q < kBwdOwn; ++q) {
          const int64_t j = base + 32 * q + lane;
          bag[q] = lo[q];
          coef[q] = j < c1 ? 1.f : 0.f;
          if (j < c1) {
            if (pooling == MFET_POOL_MEAN) coef[q] = __fdiv_rn(1.f, (float)(offsets_f[lo[q] + 1] - offsets_f[lo[q]]));
            else if (pooling == MFET_POOL_WSUM) coef[q] = weights[at[q]];
          }
        }
#pragma unroll
        for (int q = 0; q < kBwdOwn; ++q) {
          const int64_t j32 = base + 32 * q;
          if (j32 < c1) {  // the same for all lanes
            const int cnt = (int)(c1 - j32 < 32 ? c1 - j32 : 32);
            for (int t0 = 0; t0 < cnt; t0 += kBwdBatch) {
              float g[kBwdBatch][kBwdRegs];
#pragma unroll
              for (int t = 0; t < kBwdBatch; ++t) {
                // The loads of a batch do not depend on one another, and none is conditional: beyond
                // the chunk's end a lane's bag is 0 and its coefficient 0, and a column beyond the
                // row's end reads the row's last column instead (never stored).
                const int32_t bt = __shfl_sync(0xFFFFFFFFu, bag[q], (t0 + t) & 31);
                const float* row = grad_out + (int64_t)bt * out_ld + col;
#pragma unroll
                for (int r = 0; r < kBwdRegs; ++r) g[t][r] = __ldg(row + min(d0 + lane + 32 * r, dim - 1));
              }
#pragma unroll
              for (int t = 0; t < kBwdBatch; ++t) {
                const int32_t ut = __shfl_sync(0xFFFFFFFFu, u[q], (t0 + t) & 31);
                const float ct = __shfl_sync(0xFFFFFFFFu, coef[q], (t0 + t) & 31);
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
        }
      }
      if (cur >= 0) flush(cur);
    }
  }
  asm volatile("griddepcontrol.launch_dependents;");  // the combine kernel may be set up
}

// Rows whose run crosses a chunk boundary: the gradient is the TAIL slot of the chunk where the run
// begins, the HEAD slots of the chunks it covers entirely, and the HEAD slot of the chunk where it
// ends. A warp owns 32 rows and one group of 32 columns (lane = column). It looks at its rows
// (one per lane: most runs lie inside one chunk and need nothing) and adds up the ones that do in
// chunk order. A hot row spans hundreds of chunks, and one warp keeps only a few loads in flight:
// rows of more than kCombineLong chunks are left to the whole block, whose warps each add a
// stretch of the chunks in order before the stretches are added in order. Either way the order of
// the additions depends only on the inputs and the chunk length. chunk = 1 << chunk_shift.
constexpr int kCombineBatch = 16;
constexpr int kCombineLong = 32;
constexpr int kCombineWarps = 8;

// s + partial[first .. last] (HEAD slots, column dc) in chunk order
__device__ __forceinline__ float add_heads(float s, const float* partial, int64_t first, int64_t last, uint32_t dim,
                                           uint32_t dc) {
  for (int64_t kb = first; kb <= last; kb += kCombineBatch) {
    float v[kCombineBatch];
#pragma unroll
    for (int j = 0; j < kCombineBatch; ++j) {
      const int64_t kk = kb + j <= last ? kb + j : last;  // unconditional loads; the surplus is not added
      v[j] = __ldcg(partial + (size_t)(2 * kk) * dim + dc);
    }
#pragma unroll
    for (int j = 0; j < kCombineBatch; ++j)
      if (kb + j <= last) s += v[j];
  }
  return s;
}

__global__ void __launch_bounds__(32 * kCombineWarps) backward_combine_kernel(
    const int32_t* __restrict__ seg_start, const int64_t* __restrict__ n_unique, NSrc ns,
    const int64_t* __restrict__ offsets_f, int32_t batch, uint32_t dim, int32_t chunk_shift, const float* partial,
    float* __restrict__ grad_vals) {
  __shared__ int64_t long_u[kCombineWarps * 32], long_a0[kCombineWarps * 32], long_a1[kCombineWarps * 32];
  __shared__ int n_long;
  __shared__ float stretch[kCombineWarps][32];
  // launched programmatically after backward_chunks_kernel, whose partial sums are read through L2
  asm volatile("griddepcontrol.wait;" ::: "memory");
  int64_t n = offsets_f[batch] - offsets_f[0];
  if (n < 0 || n > ns.cap) n = 0;
  const int64_t nu = *n_unique;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t col_groups = (dim + 31) / 32;
  const int64_t jobs = ((nu + 31) / 32) * col_groups;  // (32 rows, 32 columns)
  // the jobs of a block are consecutive, so that the warps that hold the column groups of one row sit in
  // one block (if 8 is a multiple of the number of column groups; otherwise a long row may be met twice,
  // which only repeats work)
  for (int64_t job0 = (int64_t)blockIdx.x * kCombineWarps; job0 < jobs; job0 += (int64_t)gridDim.x * kCombineWarps) {
    if (threadIdx.x == 0) n_long = 0;
    __syncthreads();
    const int64_t job = job0 + warp;
    if (job < jobs) {
      const int64_t u0 = (job / col_groups) * 32;
      const int64_t cg = job % col_groups;
      const uint32_t d = (uint32_t)cg * 32 + lane;
      const uint32_t dc = d < dim ? d : dim - 1;  // a lane beyond the row's end reads its last column and stores nothing
      const int64_t u = u0 + lane;
      int64_t k0 = 0, k1 = 0;
      if (u < nu) {
        const int64_t j0 = seg_start[u];
        const int64_t j1 = (u + 1 < nu) ? (int64_t)seg_start[u + 1] : n;
        k0 = j0 >> chunk_shift;
        k1 = (j1 - 1) >> chunk_shift;
      }
      // runs inside one chunk were stored by the chunk's warp; long ones go on the block's list (once:
      // by the warp that holds the row's first column group in this block)
      const bool is_long = k1 - k0 > kCombineLong;
      if (is_long && (cg == 0 || warp == 0)) {
        const int at = atomicAdd(&n_long, 1);
        long_u[at] = u;
        long_a0[at] = k0;
        long_a1[at] = k1;
      }
      uint32_t todo = __ballot_sync(0xFFFFFFFFu, k0 != k1 && !is_long);
      while (todo) {
        const int t = __ffs(todo) - 1;
        todo &= todo - 1;
        const int64_t a0 = __shfl_sync(0xFFFFFFFFu, k0, t), a1 = __shfl_sync(0xFFFFFFFFu, k1, t);
        const float s = add_heads(__ldcg(partial + (size_t)(2 * a0 + 1) * dim + dc), partial, a0 + 1, a1, dim, dc);
        if (d < dim) grad_vals[(size_t)(u0 + t) * dim + d] = s;
      }
    }
    __syncthreads();
    // the long rows of this round: every warp adds one stretch of the row's chunks, for one column group after another
    const int longs = n_long;
    for (int i = 0; i < longs; ++i) {
      const int64_t u = long_u[i], a0 = long_a0[i], a1 = long_a1[i];
      const int64_t heads = a1 - a0;                                   // HEAD slots a0+1 .. a1
      const int64_t per = (heads + kCombineWarps - 1) / kCombineWarps;  // per warp
      const int64_t first = a0 + 1 + warp * per, last = min(a1, first + per - 1);
      for (int64_t cg = 0; cg < col_groups; ++cg) {
        const uint32_t d = (uint32_t)cg * 32 + lane;
        const uint32_t dc = d < dim ? d : dim - 1;
        stretch[warp][lane] = first <= last ? add_heads(0.f, partial, first, last, dim, dc) : 0.f;
        __syncthreads();
        if (warp == 0) {
          float s = __ldcg(partial + (size_t)(2 * a0 + 1) * dim + dc);
#pragma unroll
          for (int w = 0; w < kCombineWarps; ++w) s += stretch[w][lane];
          if (d < dim) grad_vals[(size_t)u * dim + d] = s;
        }
        __syncthreads();
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
  const int64_t blocks = (chunks + kBwdThreads / 32 - 1) / (kBwdThreads / 32);  // one chunk per warp
  if (blocks > 0x7FFFFFFF) return cudaErrorInvalidValue;
  // both kernels may be set up while the kernel before them still runs; they wait inside
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(kBwdThreads);
  cfg.gridDim = dim3((unsigned)(blocks > 0 ? blocks : 1));
  cfg.stream = s;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaLaunchKernelEx(&cfg, backward_chunks_kernel, sorted_pos, inverse, seg_start, n_unique, ns, offsets_f,
                                     batch, weights, pooling, grad_out, out_ld, col, dim, chunk, partial, grad_vals, err);
  if (e != cudaSuccess) return e;
  if (chunks <= 1) return cudaSuccess;  // one chunk holds every run: nothing to combine
  int shift = 0;
  while ((1 << shift) < chunk) ++shift;  // chunk is a power of two whenever there is more than one
  // 8 warps per block; a warp's job is 32 rows x 32 columns
  int64_t cblocks = ((ns.cap + 31) / 32 * ((dim + 31) / 32) + 7) / 8;
  if (cblocks > (int64_t)sm_count() * 8) cblocks = (int64_t)sm_count() * 8;
  cfg.blockDim = dim3(256);
  cfg.gridDim = dim3((unsigned)(cblocks > 0 ? cblocks : 1));
  return cudaLaunchKernelEx(&cfg, backward_combine_kernel, seg_start, n_unique, ns, offsets_f, batch, dim, shift,
                            (const float*)partial, grad_vals);
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
