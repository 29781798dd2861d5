// K-dedup: in-batch dedup of hashed rows = stable LSD radix sort of (row, index)
// pairs, then adjacent-unique with an inverse map. For a host-table slot the
// same pass also probes the HBM hot-row cache and compacts the misses, so that
// only distinct, uncached rows are fetched over PCIe.
//
// Every kernel here is a plain data-parallel pass; the passes are ordered by the
// stream, so no kernel ever waits on another block. Results are canonical
// (ascending unique rows), hence bit-reproducible.
#include <cstring>
#include <mutex>

#include "common.cuh"

namespace mfet {

namespace {

constexpr int kSortThreads = 256;
constexpr int kSortRounds = 8;
constexpr int kSortTile = kSortThreads * kSortRounds;  // keys per block per pass
constexpr int kScanThreads = 256;
constexpr int kScanItems = 4;
constexpr int kScanTile = kScanThreads * kScanItems;

// Number of elements: either immediate, or the ID count of feature f taken
// from the CSR offsets on the device. Out-of-capacity or negative counts
// degrade to 0 (the caller flags MFET_DEV_CAPACITY once).
__device__ __forceinline__ int64_t resolve_n(const NSrc& s, int64_t* lo) {
  if (s.offsets == nullptr) {
    *lo = 0;
    return s.n_imm;
  }
  const int64_t a = s.offsets[s.idx_lo], b = s.offsets[s.idx_hi];
  *lo = a;
  const int64_t n = b - a;
  return (n < 0 || n > s.cap) ? 0 : n;
}

// ---- pass kernels --------------------------------------------------------

// True in exactly one block of the grid: the one whose arrival is the last. That block may
// then read what all other blocks wrote before they arrived. Nobody waits for anybody.
__device__ __forceinline__ bool last_block_arrives(uint32_t* ticket) {
  __shared__ bool last;
  __threadfence();
  __syncthreads();
  if (threadIdx.x == 0) last = atomicAdd(ticket, 1u) == gridDim.x - 1;
  __syncthreads();
  if (last) __threadfence();
  return last;
}

// The histogram kernel runs 1024 threads per tile (the scatter kernel 256): the block that arrives
// last scans tiles x 256 counters, and its critical path is the number of dependent memory round
// trips of one thread, so four threads share a digit's column.
constexpr int kHistThreads = 1024;
constexpr int kHistRounds = kSortTile / kHistThreads;
constexpr int kHistGroups = kHistThreads / 256;  // threads that share one digit in the scan

// Turns the per-tile digit counts hist[tile][digit] into the global start position of every
// (digit, tile) pair in digit-major order: start(d, b) = all counts of smaller digits + counts
// of digit d in tiles before b. Run by the 1024 threads of one block: thread (g, d) owns digit d in
// the g-th quarter of the tiles, so loads and stores are coalesced across the digits, and a
// thread's loads are independent of one another (batches of 16 are issued together).
__device__ __forceinline__ void scan_digit_counts(uint32_t* hist, int nblk) {
  __shared__ uint32_t part[kHistGroups][256];  // keys of digit d in the tiles of group g
  __shared__ uint32_t dstart[256];             // keys of all smaller digits
  __shared__ uint32_t warp_tot[8];
  const int d = threadIdx.x & 255, g = threadIdx.x >> 8;
  const int per = (nblk + kHistGroups - 1) / kHistGroups;
  const int b0 = g * per, b1 = min(nblk, b0 + per);
  uint32_t tot = 0;
  for (int b = b0; b < b1; b += 16) {
    uint32_t v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = b + j < b1 ? __ldcg(hist + (size_t)(b + j) * 256 + d) : 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) tot += v[j];
  }
  part[g][d] = tot;
  __syncthreads();
  if (g == 0) {
    uint32_t all = 0;
#pragma unroll
    for (int q = 0; q < kHistGroups; ++q) all += part[q][d];
    const int lane = d & 31;
    uint32_t inc = all;
#pragma unroll
    for (int k = 1; k < 32; k <<= 1) {
      const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, k);
      if (lane >= k) inc += t;
    }
    if (lane == 31) warp_tot[d >> 5] = inc;
    dstart[d] = inc - all;  // exclusive inside the warp; the warps before are added below
  }
  __syncthreads();
  uint32_t run = dstart[d];
  for (int w = 0; w < (d >> 5); ++w) run += warp_tot[w];
#pragma unroll
  for (int q = 0; q < kHistGroups; ++q) run += q < g ? part[q][d] : 0u;
  for (int b = b0; b < b1; b += 16) {
    uint32_t v[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) v[j] = b + j < b1 ? __ldcg(hist + (size_t)(b + j) * 256 + d) : 0u;
#pragma unroll
    for (int j = 0; j < 16; ++j) {
      if (b + j < b1) hist[(size_t)(b + j) * 256 + d] = run;
      run += v[j];
    }
  }
}

// Digit histogram of one tile; the block that finishes last turns all histograms into
// scatter positions. With HASH the keys are produced here from the raw IDs (first pass of
// a host-table slot) and stored for the later passes.
template <bool HASH>
__global__ void __launch_bounds__(kHistThreads) hist_kernel(NSrc ns, const uint64_t* __restrict__ keys_in,
                                                            uint64_t* __restrict__ keys_store,
                                                            const uint64_t* __restrict__ ids, uint64_t seed,
                                                            uint64_t rows, uint64_t magic, uint32_t pre_hashed,
                                                            int shift, uint32_t* hist, int nblk,
                                                            uint32_t* err, uint32_t* ticket) {
  __shared__ uint32_t h[256];
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  if (HASH && blockIdx.x == 0 && threadIdx.x == 0 && ns.offsets) {
    const int64_t raw = ns.offsets[ns.idx_hi] - ns.offsets[ns.idx_lo];
    if (raw < 0) atomicOr(err, (uint32_t)MFET_DEV_OFFSETS);
    if (raw > ns.cap) atomicOr(err, (uint32_t)MFET_DEV_CAPACITY);
  }
  if (threadIdx.x < 256) h[threadIdx.x] = 0;
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kSortTile;
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int r = 0; r < kHistRounds; ++r) {
    const int64_t i = base + r * kHistThreads + threadIdx.x;
    const bool valid = i < n;
    uint64_t k = 0;
    if (valid) {
      if (HASH) {
        const uint64_t id = __ldcs(reinterpret_cast<const unsigned long long*>(ids) + lo + i);
        k = pre_hashed ? id : mod_rows(splitmix64(id ^ seed), rows, magic);
        if (k >= rows) {  // only possible for pre-hashed input
          atomicOr(err, (uint32_t)MFET_DEV_ROW_RANGE);
          k = rows - 1;
        }
        keys_store[i] = k;
      } else {
        k = keys_in[i];
      }
    }
    // one shared-memory add per distinct digit of the warp: Zipf heads repeat the same row
    // thousands of times, and per-thread adds on one counter would serialise
    const uint32_t d = (uint32_t)(k >> shift) & 255u;
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, valid ? d : 256u + (uint32_t)lane);
    if (valid && (peers & ((1u << lane) - 1u)) == 0) atomicAdd(&h[d], (uint32_t)__popc(peers));
  }
  __syncthreads();
  if (threadIdx.x < 256) hist[(size_t)blockIdx.x * 256 + threadIdx.x] = h[threadIdx.x];  // block-major: coalesced
  if (last_block_arrives(ticket)) {
    scan_digit_counts(hist, nblk);
    if (threadIdx.x == 0) *ticket = 0;  // ready for the next pass
  }
}

// Stable scatter of one tile by the current digit. A thread holds one key of each of the
// tile's rounds (round r = keys r*256 .. r*256+255 of the tile, so (round, warp, lane) is the
// input order). Phase 1: per (round, warp) digit counts and every key's rank among the equal
// digits of its warp, through match_any. Phase 2: thread d turns the 64 counts of digit d into
// running offsets. Phase 3: position = tile's start for the digit + offset of (round, warp) +
// rank. Two block barriers in all.
__global__ void __launch_bounds__(kSortThreads) scatter_kernel(NSrc ns, const uint64_t* __restrict__ keys_in,
                                                               const uint32_t* __restrict__ idx_in,
                                                               uint64_t* __restrict__ keys_out,
                                                               uint32_t* __restrict__ idx_out, int shift,
                                                               const uint32_t* __restrict__ hist, int nblk,
                                                               uint32_t* err) {
  constexpr int kWarps = kSortThreads / 32;
  __shared__ uint16_t wcnt[kSortRounds][kWarps][256];  // counts, then offsets inside the tile (< 2048)
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t tile0 = (int64_t)blockIdx.x * kSortTile;
  if (tile0 >= n) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t base = hist[(size_t)blockIdx.x * 256 + threadIdx.x];  // start of digit threadIdx.x for this tile
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(&wcnt[0][0][0]);
#pragma unroll
    for (int j = 0; j < kSortRounds * kWarps * 256 / 2 / kSortThreads; ++j) z[j * kSortThreads + threadIdx.x] = 0u;
  }
  __syncthreads();
  uint64_t k[kSortRounds];
  uint32_t src[kSortRounds];
  uint32_t dr[kSortRounds];  // digit | rank << 8 | valid << 16
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    const int64_t i = tile0 + r * kSortThreads + threadIdx.x;
    const bool valid = i < n;
    k[r] = 0;
    src[r] = 0;
    if (valid) {
      k[r] = keys_in[i];
      src[r] = idx_in ? idx_in[i] : (uint32_t)i;
    }
  }
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    const bool valid = tile0 + r * kSortThreads + threadIdx.x < n;
    const uint32_t d = (uint32_t)(k[r] >> shift) & 255u;
    const uint32_t peers = __match_any_sync(0xFFFFFFFFu, valid ? d : (256u + (uint32_t)lane));  // invalid lanes match nobody
    const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
    if (valid && rank == 0) wcnt[r][warp][d] = (uint16_t)__popc(peers);
    dr[r] = d | (rank << 8) | (valid ? 1u << 16 : 0u);
  }
  __syncthreads();
  {
    uint32_t run = 0;  // thread d: exclusive running sum of digit d over (round, warp)
#pragma unroll
    for (int r = 0; r < kSortRounds; ++r)
#pragma unroll
      for (int w = 0; w < kWarps; ++w) {
        const uint32_t c = wcnt[r][w][threadIdx.x];
        wcnt[r][w][threadIdx.x] = (uint16_t)run;
        run += c;
      }
  }
  __shared__ uint32_t sbase[256];
  sbase[threadIdx.x] = base;
  __syncthreads();
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    if (dr[r] >> 16) {
      const uint32_t d = dr[r] & 255u;
      const uint32_t pos = sbase[d] + wcnt[r][warp][d] + ((dr[r] >> 8) & 255u);
      if (MFET_IN_BOUNDS(err, (int64_t)pos < n)) {
        keys_out[pos] = k[r];
        idx_out[pos] = src[r];
      }
    }
  }
}

// ---- unique / inverse / probe ---------------------------------------------

__device__ __forceinline__ int32_t cache_probe(const CacheDev& c, int64_t key) {
  if (c.n == 0) return -1;
  const uint32_t b = (uint32_t)((uint64_t)key >> c.bucket_shift);
  uint32_t lo = c.bucket_start[b], hi = c.bucket_start[b + 1];
  while (lo < hi) {
    const uint32_t mid = (lo + hi) >> 1;
    const int64_t v = c.keys[mid];
    if (v == key) return (int32_t)mid;
    if (v < key) lo = mid + 1;
    else hi = mid;
  }
  return -1;
}

// Block-wide exclusive scan of one value per thread (256 threads); returns the
// exclusive prefix and the block total.
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* total, uint32_t* sh /*[8]*/) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  uint32_t inc = v;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, d);
    if (lane >= d) inc += t;
  }
  __syncthreads();  // sh may still be in use by a previous call
  if (lane == 31) sh[warp] = inc;
  __syncthreads();
  uint32_t before = 0, all = 0;
#pragma unroll
  for (int w = 0; w < kScanThreads / 32; ++w) {
    const uint32_t s = sh[w];
    if (w < warp) before += s;
    all += s;
  }
  *total = all;
  return before + inc - v;
}

// Pass 1: count heads (first of each run of equal keys) per tile; with PROBE
// also look every head up in the cache, remember the answer per sorted
// position and count the misses.
template <bool PROBE>
__global__ void __launch_bounds__(kScanThreads) unique_count_kernel(NSrc ns, const uint64_t* __restrict__ keys,
                                                                    CacheDev cache, int32_t* __restrict__ probe_tmp,
                                                                    uint32_t* tile_counts, int nblk, uint32_t* ticket,
                                                                    int64_t* __restrict__ n_unique,
                                                                    int64_t* __restrict__ n_miss) {
  __shared__ uint32_t sh[8];
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t i0 = ((int64_t)blockIdx.x * kScanThreads + threadIdx.x) * kScanItems;
  uint32_t heads = 0, misses = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    if (i < n) {
      const uint64_t k = keys[i];
      const bool head = (i == 0) || (keys[i - 1] != k);
      if (head) {
        ++heads;
        if (PROBE) {
          const int32_t slot = cache_probe(cache, (int64_t)k);
          probe_tmp[i] = slot;
          if (slot < 0) ++misses;
        }
      }
    }
  }
  uint32_t th, tm;
  block_excl_scan(heads, &th, sh);
  if (PROBE) block_excl_scan(misses, &tm, sh);
  if (threadIdx.x == 0) {
    tile_counts[blockIdx.x] = th;
    if (PROBE) tile_counts[nblk + blockIdx.x] = tm;
  }
  // the block that finishes last scans the per-tile counts and publishes the totals
  if (last_block_arrives(ticket)) {
    for (int a = 0; a < (PROBE ? 2 : 1); ++a) {
      uint32_t* arr = tile_counts + (size_t)a * nblk;
      uint32_t run = 0;
      for (int i0 = 0; i0 < nblk; i0 += kScanThreads) {
        const int i = i0 + threadIdx.x;
        const uint32_t v = i < nblk ? __ldcg(arr + i) : 0u;
        uint32_t tot;
        const uint32_t ex = block_excl_scan(v, &tot, sh);
        if (i < nblk) arr[i] = run + ex;
        run += tot;
      }
      if (threadIdx.x == 0) {
        if (a == 0) *n_unique = (int64_t)run;
        else *n_miss = (int64_t)run;
      }
    }
    if (threadIdx.x == 0) *ticket = 0;
  }
}

// Pass 2: write uniq, inverse and (PROBE) the per-unique source and the list of
// missed rows.
template <bool PROBE>
__global__ void __launch_bounds__(kScanThreads) unique_write_kernel(NSrc ns, const uint64_t* __restrict__ keys,
                                                                    const uint32_t* __restrict__ idx,
                                                                    const int32_t* __restrict__ probe_tmp,
                                                                    const uint32_t* __restrict__ tile_counts, int nblk,
                                                                    int64_t* __restrict__ uniq, int32_t* __restrict__ inverse,
                                                                    int32_t* __restrict__ src, int64_t* __restrict__ miss_rows,
                                                                    uint32_t* err) {
  __shared__ uint32_t sh[8];
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t i0 = ((int64_t)blockIdx.x * kScanThreads + threadIdx.x) * kScanItems;
  uint64_t k[kScanItems];
  bool head[kScanItems];
  int32_t slot[kScanItems];
  uint32_t heads = 0, misses = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    head[j] = false;
    slot[j] = 0;
    k[j] = 0;
    if (i < n) {
      k[j] = keys[i];
      head[j] = (i == 0) || (keys[i - 1] != k[j]);
      if (head[j]) {
        ++heads;
        if (PROBE) {
          slot[j] = probe_tmp[i];
          if (slot[j] < 0) ++misses;
        }
      }
    }
  }
  uint32_t tot;
  uint32_t u = tile_counts[blockIdx.x] + block_excl_scan(heads, &tot, sh);
  uint32_t m = 0;
  if (PROBE) m = tile_counts[nblk + blockIdx.x] + block_excl_scan(misses, &tot, sh);
  // u = number of heads strictly before this thread's first element
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    if (i < n && MFET_IN_BOUNDS(err, (int64_t)u - (head[j] ? 0 : 1) < n && (int64_t)m <= n && (int64_t)idx[i] < n)) {
      if (head[j]) {
        uniq[u] = (int64_t)k[j];
        if (!PROBE && src) src[u] = (int32_t)i;  // where this row's run starts in the sorted order
        if (PROBE) {
          if (slot[j] < 0) {
            src[u] = -1 - (int32_t)m;
            miss_rows[m] = (int64_t)k[j];
            ++m;
          } else {
            src[u] = slot[j];
          }
        }
        ++u;
      }
      inverse[idx[i]] = (int32_t)(u - 1);
    }
  }
}

inline uint64_t align256(uint64_t x) { return (x + 255u) & ~255ULL; }

}  // namespace

uint64_t workspace_layout(int64_t max_ids, uint64_t max_row_bytes, WsLayout* L) {
  WsLayout l;
  const uint64_t n = (uint64_t)(max_ids > 0 ? max_ids : 0);
  l.nblk_sort = (int)((n + kSortTile - 1) / kSortTile);
  l.nblk_scan = (int)((n + kScanTile - 1) / kScanTile);
  if (l.nblk_sort < 1) l.nblk_sort = 1;
  if (l.nblk_scan < 1) l.nblk_scan = 1;
  uint64_t off = 0;
  auto take = [&](uint64_t bytes) {
    const uint64_t at = off;
    off = align256(off + bytes);
    return at;
  };
  l.keys_a = take(n * 8);
  l.keys_b = take(n * 8);
  l.idx_a = take(n * 4);
  l.idx_b = take(n * 4);
  l.hist = take((uint64_t)l.nblk_sort * 256 * 4);
  l.tile_counts = take((uint64_t)l.nblk_scan * 2 * 4);
  l.counters = take(64);
  l.uniq = take(n * 8);
  l.inverse = take(n * 4);
  l.src = take(n * 4);
  l.miss_rows = take(n * 8);
  l.staging = take(n * max_row_bytes);
  l.inverse2 = take(n * 4);
  l.src2 = take(n * 4);
  l.staging2 = take(n * max_row_bytes);
  l.miss_rows2 = take(n * 8);
  l.total = off;
  if (L) *L = l;
  return off;
}

// Sort + unique + inverse (+ cache probe). `first_keys` is the array that pass 0
// reads when hash == nullptr; with hash != nullptr pass 0 hashes the slot's raw
// IDs into the workspace instead. On return (in stream order) uniq / inverse /
// n_unique hold the dedup result; with `cache` non-null also src / miss_rows /
// n_miss.
cudaError_t launch_dedup(const DedupArgs& a, uint64_t* launches, cudaStream_t s) {
  uint8_t* ws = (uint8_t*)a.ws;
  const WsLayout& L = a.layout;
  uint64_t* ka = (uint64_t*)(ws + L.keys_a);
  uint64_t* kb = (uint64_t*)(ws + L.keys_b);
  uint32_t* ia = (uint32_t*)(ws + L.idx_a);
  uint32_t* ib = (uint32_t*)(ws + L.idx_b);
  uint32_t* hist = (uint32_t*)(ws + L.hist);
  uint32_t* tile_counts = (uint32_t*)(ws + L.tile_counts);
  uint32_t* tickets = (uint32_t*)(ws + L.counters + 32);  // two arrival counters, zero between launches

  const int64_t cap = a.ns.offsets ? a.ns.cap : a.ns.n_imm;
  const int nblk = (int)((cap + kSortTile - 1) / kSortTile) > 0 ? (int)((cap + kSortTile - 1) / kSortTile) : 1;
  const int nblk2 = (int)((cap + kScanTile - 1) / kScanTile) > 0 ? (int)((cap + kScanTile - 1) / kScanTile) : 1;
  int bits = 1;
  while (bits < 63 && (a.max_key >> bits) != 0) ++bits;
  const int passes = (bits + 7) / 8;

  const uint64_t* kin = a.hash ? ka : a.first_keys;
  const uint32_t* iin = nullptr;
  uint64_t* kout = a.hash ? kb : ka;
  uint32_t* iout = ia;
  for (int p = 0; p < passes; ++p) {
    const int shift = 8 * p;
    if (p == 0 && a.hash)
      hist_kernel<true><<<nblk, kHistThreads, 0, s>>>(a.ns, nullptr, ka, a.hash->ids, a.hash->seed, a.hash->rows,
                                                      a.hash->magic, a.hash->pre_hashed, shift, hist, nblk, a.err, tickets);
    else
      hist_kernel<false><<<nblk, kHistThreads, 0, s>>>(a.ns, kin, nullptr, nullptr, 0, 0, 0, 0, shift, hist, nblk, a.err, tickets);
    scatter_kernel<<<nblk, kSortThreads, 0, s>>>(a.ns, kin, iin, kout, iout, shift, hist, nblk, a.err);
    *launches += 2;
    // next pass reads what this one wrote
    kin = kout;
    iin = iout;
    kout = (kout == ka) ? kb : ka;
    iout = (iout == ia) ? ib : ia;
  }
  // kin / iin: sorted keys and their original positions; iout is free
  int32_t* probe_tmp = (int32_t*)iout;
  if (a.cache) {
    unique_count_kernel<true><<<nblk2, kScanThreads, 0, s>>>(a.ns, kin, *a.cache, probe_tmp, tile_counts, nblk2,
                                                             tickets + 1, a.n_unique, a.n_miss);
    unique_write_kernel<true><<<nblk2, kScanThreads, 0, s>>>(a.ns, kin, iin, probe_tmp, tile_counts, nblk2, a.uniq,
                                                            a.inverse, a.src, a.miss_rows, a.err);
  } else {
    CacheDev none{};
    unique_count_kernel<false><<<nblk2, kScanThreads, 0, s>>>(a.ns, kin, none, nullptr, tile_counts, nblk2, tickets + 1,
                                                              a.n_unique, nullptr);
    unique_write_kernel<false><<<nblk2, kScanThreads, 0, s>>>(a.ns, kin, iin, nullptr, tile_counts, nblk2, a.uniq,
                                                             a.inverse, a.src, nullptr, a.err);
  }
  if (a.sorted_pos_out) *a.sorted_pos_out = iin;
  *launches += 2;
  return cudaGetLastError();
}

}  // namespace mfet

// ---- dedup without any caller- or library-side allocation -------------------
//
// The sort's ping-pong buffers and counters live in a fixed device array that
// is part of the library image: every GPU that loads the library holds these
// bytes until the process exits, which is why the capacity is kept modest.

namespace {

constexpr int64_t kStaticMaxIds = MFET_STATIC_DEDUP_MAX_IDS;
constexpr uint64_t kStaticSortBlocks = (kStaticMaxIds + mfet::kSortTile - 1) / mfet::kSortTile;
constexpr uint64_t kStaticScanBlocks = (kStaticMaxIds + mfet::kScanTile - 1) / mfet::kScanTile;
constexpr uint64_t pad256(uint64_t x) { return (x + 255u) & ~255ULL; }
constexpr uint64_t kOffKeysA = 0;
constexpr uint64_t kOffKeysB = kOffKeysA + pad256(kStaticMaxIds * 8);
constexpr uint64_t kOffIdxA = kOffKeysB + pad256(kStaticMaxIds * 8);
constexpr uint64_t kOffIdxB = kOffIdxA + pad256(kStaticMaxIds * 4);
constexpr uint64_t kOffHist = kOffIdxB + pad256(kStaticMaxIds * 4);
constexpr uint64_t kOffTiles = kOffHist + pad256(kStaticSortBlocks * 256 * 4);
constexpr uint64_t kOffCounters = kOffTiles + pad256(kStaticScanBlocks * 2 * 4);
constexpr uint64_t kStaticScratchBytes = kOffCounters + 256;

// In host code this name is only a handle of the symbol, not a device address:
// the address is asked from the runtime once per device (below).
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
void* g_scratch_addr[kMaxDevices];  // device address of g_static_scratch, per GPU
bool g_scratch_ready[kMaxDevices];
std::mutex g_scratch_mutex;

}  // namespace

extern "C" int mfet_dedup_rows_static(int32_t device, const int64_t* rows, int64_t n, int64_t* uniq,
                                      int32_t* inverse, int64_t* n_unique, int64_t max_row,
                                      mfet_stream_t stream_) {
  if (device < 0 || device >= kMaxDevices || n < 0 || !n_unique || max_row < 0) return MFET_ERR_INVALID_ARG;
  if (n > kStaticMaxIds) return MFET_ERR_WORKSPACE;  // beyond the built-in scratch: use mfet_dedup_rows
  if (n > 0 && (!rows || !uniq || !inverse)) return MFET_ERR_INVALID_ARG;
  int prev = 0;
  if (cudaGetDevice(&prev) != cudaSuccess) return MFET_ERR_CUDA;
  if (prev != device && cudaSetDevice(device) != cudaSuccess) {
    cudaGetLastError();
    return MFET_ERR_INVALID_ARG;
  }
  cudaStream_t stream = (cudaStream_t)stream_;
  int rc = MFET_OK;
  void* scratch = nullptr;
  {
    // first call on this GPU: look the array's device address up, with this GPU current
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_ready[device]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) {
        cudaGetLastError();
        rc = MFET_ERR_CUDA;
      } else {
        g_scratch_addr[device] = p;
        g_scratch_ready[device] = true;
      }
    }
    scratch = g_scratch_addr[device];
  }
  if (rc == MFET_OK) {
    if (n == 0) {
      if (cudaMemsetAsync(n_unique, 0, sizeof(int64_t), stream) != cudaSuccess) rc = MFET_ERR_CUDA;
    } else {
      // every scratch region that a pass reads is written in full by an earlier pass of the
      // same call, so nothing left over from the previous call needs clearing
      mfet::DedupArgs a;
      std::memset(&a, 0, sizeof(a));
      a.ns = mfet::NSrc{nullptr, 0, 0, n, n};
      a.first_keys = reinterpret_cast<const uint64_t*>(rows);
      a.max_key = max_row > 0 ? (uint64_t)max_row - 1 : 0x7FFFFFFFFFFFFFFFULL;
      a.ws = scratch;
      a.layout.keys_a = kOffKeysA;
      a.layout.keys_b = kOffKeysB;
      a.layout.idx_a = kOffIdxA;
      a.layout.idx_b = kOffIdxB;
      a.layout.hist = kOffHist;
      a.layout.tile_counts = kOffTiles;
      a.layout.counters = kOffCounters;
      a.uniq = uniq;
      a.inverse = inverse;
      a.n_unique = n_unique;
      uint64_t launches = 0;
      if (mfet::launch_dedup(a, &launches, stream) != cudaSuccess) rc = MFET_ERR_CUDA;
    }
  }
  if (prev != device) cudaSetDevice(prev);
  return rc;
}
