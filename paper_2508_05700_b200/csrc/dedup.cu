// K-dedup: in-batch dedup of hashed rows = stable LSD radix sort of (row, index)
// pairs, then adjacent-unique with an inverse map. For a host-table slot the
// same pass also probes the HBM hot-row cache and compacts the misses, so that
// only distinct, uncached rows are fetched over PCIe.
//
// One launch counts the digits of all passes, one launch per 8-bit digit scatters, two launches
// count and write the unique rows and the inverse map. Inside a scatter launch a tile learns the
// counts of the tiles before it from status words in global memory (see below) instead of from a
// separate scan launch. Results are canonical (ascending unique rows), hence bit-reproducible.
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "dedup_layout.cuh"

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
//
// Tiles of one launch hand their counts to the tiles after them through status words in global
// memory, one per (tile, digit): value and flag travel in one word, so no fence is needed. Tiles
// form groups of kGroup. A tile publishes its own counts (kFlagLocal) as soon as they are known;
// the last tile of a group adds up its group and publishes the group's counts. A tile then needs
// the counts of the tiles before it in its own group and of the groups before its own: two
// rounds of loads after the tiles have published, however many tiles there are. All tiles of a
// small input start together, so a walk from tile to tile would cost one memory round trip per
// step. A tile only ever waits for tiles of lower block index, which the hardware starts first;
// every wait is bounded all the same (kStallNs), after which the block raises MFET_DEV_STALLED
// and returns without writing its keys.
constexpr uint32_t kFlagLocal = 1u << 30, kValueMask = (1u << 30) - 1u;
constexpr uint64_t kStallNs = 2000000000ull;
constexpr int kGroup = 16;      // tiles per group
constexpr int kLookBatch = 16;  // status words of one digit that a thread asks for at once
constexpr int kMaxPasses = 8;
constexpr int kCountGroup = 256;  // tiles of the unique kernels whose counts are also added up into one group sum
static_assert(kDedupTotalsBytes == (uint64_t)kMaxPasses * 256 * 4, "digit totals: one counter per pass and digit");

__device__ __forceinline__ uint32_t ld_status(const uint32_t* p) {
  uint32_t v;
  asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ void st_status(uint32_t* p, uint32_t v) {
  asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// What an earlier kernel of the same call wrote is read through L2 (ld.global.cg): a kernel that
// is launched programmatically begins before that earlier kernel has ended, so the data is not
// constant over its lifetime, which the read-only path (const __restrict__) would require.
__device__ __forceinline__ uint64_t ld_l2(const uint64_t* p) {
  return (uint64_t)__ldcg(reinterpret_cast<const unsigned long long*>(p));
}
__device__ __forceinline__ uint32_t ld_l2(const uint32_t* p) { return __ldcg(p); }
__device__ __forceinline__ int32_t ld_l2(const int32_t* p) { return __ldcg(p); }

__device__ __forceinline__ uint64_t now_ns() {
  uint64_t t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}

// A bounded wait: pause() after every look that found a word missing; over() once the waits have
// lasted longer than kStallNs.
struct Patience {
  uint32_t looks = 0;
  uint64_t t_first = 0;
  bool gone = false;
  __device__ __forceinline__ void pause() {
    __nanosleep(32);  // a short breath between looks
    if (((++looks) & 63u) == 0) {
      const uint64_t now = now_ns();
      if (t_first == 0) t_first = now;
      else if (now - t_first > kStallNs) gone = true;
    }
  }
  __device__ __forceinline__ bool over() const { return gone; }
};

constexpr int kHistThreads = 1024;
constexpr int kHistRounds = kSortTile / kHistThreads;

// Digit counts of the whole input for every pass at once (the keys do not change from pass to
// pass, only their order), added into total[pass][digit], which every call leaves at zero. With
// HASH the keys are produced here from the raw IDs (a host-table slot) and stored for the passes.
// Also clears the status words that the first pass polls and the group sums of the unique kernels.
template <bool HASH>
__global__ void __launch_bounds__(kHistThreads) digit_totals_kernel(NSrc ns, const uint64_t* __restrict__ keys_in,
                                                                    uint64_t* __restrict__ keys_store,
                                                                    const uint64_t* __restrict__ ids, uint64_t seed,
                                                                    uint64_t rows, uint64_t magic, uint32_t pre_hashed,
                                                                    int passes, uint32_t* total, uint32_t* status0,
                                                                    uint32_t* group_status0, uint64_t* ustatus,
                                                                    int nblk2, uint32_t* err) {
  __shared__ uint32_t h[kMaxPasses][256];
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  if (HASH && blockIdx.x == 0 && threadIdx.x == 0 && ns.offsets) {
    const int64_t raw = ns.offsets[ns.idx_hi] - ns.offsets[ns.idx_lo];
    if (raw < 0) atomicOr(err, (uint32_t)MFET_DEV_OFFSETS);
    if (raw > ns.cap) atomicOr(err, (uint32_t)MFET_DEV_CAPACITY);
  }
  for (int j = threadIdx.x; j < passes * 256; j += kHistThreads) (&h[0][0])[j] = 0;
  if (threadIdx.x < 256) status0[(size_t)blockIdx.x * 256 + threadIdx.x] = 0;
  else if (threadIdx.x < 512 && blockIdx.x * kGroup < gridDim.x) group_status0[(size_t)blockIdx.x * 256 + threadIdx.x - 256] = 0;
  for (int j = blockIdx.x * kHistThreads + threadIdx.x; j < (nblk2 + kCountGroup - 1) / kCountGroup; j += gridDim.x * kHistThreads)
    ustatus[nblk2 + j] = 0;  // the group sums of the unique kernels
  __syncthreads();
  const int64_t base = (int64_t)blockIdx.x * kSortTile;
  if (base >= n) return;
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
    // a warp whose keys all carry the same digit (the high digits of small tables, a run of one
    // hot row) adds once; otherwise every lane adds for itself
    for (int p = 0; p < passes; ++p) {
      const uint32_t d = (uint32_t)(k >> (8 * p)) & 255u;
      const uint32_t d0 = __shfl_sync(0xFFFFFFFFu, d, 0);  // by every lane, valid or not
      if (__all_sync(0xFFFFFFFFu, valid && d == d0)) {
        if (lane == 0) atomicAdd(&h[p][d], 32u);
      } else if (valid) {
        atomicAdd(&h[p][d], 1u);
      }
    }
  }
  __syncthreads();
  for (int j = threadIdx.x; j < passes * 256; j += kHistThreads) {
    const uint32_t c = (&h[0][0])[j];
    if (c) atomicAdd(total + j, c);
  }
  // The kernel after this one is launched programmatically: it may be set up from here on, and
  // waits inside until this one is complete. (Letting it in earlier gains nothing: its blocks
  // would crowd onto the multiprocessors that this kernel leaves free and run several to one
  // of them, the rest idle.)
  asm volatile("griddepcontrol.launch_dependents;");
}

// One pass: stable scatter of one tile by the current digit. A thread holds one key of each of
// the tile's rounds (round r = keys r*256 .. r*256+255 of the tile, so (round, warp, lane) is the
// input order). Phase 1: per (round, warp) digit counts and every key's rank among the equal
// digits of its warp, through match_any. Phase 2: thread d turns the 64 counts of digit d into
// running offsets, publishes the tile's count of digit d and collects the counts of the tiles
// before it. Phase 3: position = keys of smaller digits (from the totals) + keys of digit d in
// earlier tiles + offset of (round, warp) + rank.
__global__ void __launch_bounds__(kSortThreads) sort_pass_kernel(NSrc ns, const uint64_t* __restrict__ keys_in,
                                                                 const uint32_t* __restrict__ idx_in,
                                                                 uint64_t* __restrict__ keys_out,
                                                                 uint32_t* __restrict__ idx_out, int shift,
                                                                 const uint32_t* __restrict__ total, uint32_t* status,
                                                                 uint32_t* group_status, uint32_t* status_next,
                                                                 uint32_t* group_status_next, uint32_t* err) {
  constexpr int kWarps = kSortThreads / 32;
  __shared__ uint16_t wcnt[kSortRounds][kWarps][256];  // counts, then offsets inside the tile (< 2048)
  __shared__ uint32_t sbase[256];
  __shared__ uint32_t warp_tot[kWarps];
  {
    uint32_t* z = reinterpret_cast<uint32_t*>(&wcnt[0][0][0]);
#pragma unroll
    for (int j = 0; j < kSortRounds * kWarps * 256 / 2 / kSortThreads; ++j) z[j * kSortThreads + threadIdx.x] = 0u;
  }
  // Launched with programmatic stream serialization, this block may have started before the
  // stream's earlier kernel is complete: nothing of global memory is touched before the wait.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t tile0 = (int64_t)blockIdx.x * kSortTile;
  if (status_next) {  // the next pass polls these
    status_next[(size_t)blockIdx.x * 256 + threadIdx.x] = 0;
    if (blockIdx.x * kGroup < gridDim.x) group_status_next[(size_t)blockIdx.x * 256 + threadIdx.x] = 0;
  }
  if (tile0 >= n) return;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const uint32_t all_d = __ldcg(total + threadIdx.x);  // keys of digit threadIdx.x in the whole input
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
      k[r] = ld_l2(keys_in + i);
      src[r] = idx_in ? ld_l2(idx_in + i) : (uint32_t)i;
    }
  }
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    const bool valid = tile0 + r * kSortThreads + threadIdx.x < n;
    const uint32_t d = (uint32_t)(k[r] >> shift) & 255u;
    // the lanes of the warp that hold the same digit: one vote per bit of the digit (eight votes
    // cost far less here than the match instruction)
    uint32_t peers = __ballot_sync(0xFFFFFFFFu, valid);
#pragma unroll
    for (int b = 0; b < 8; ++b) {
      const bool bit = (d >> b) & 1u;
      const uint32_t with = __ballot_sync(0xFFFFFFFFu, bit);
      peers &= bit ? with : ~with;
    }
    const uint32_t rank = __popc(peers & ((1u << lane) - 1u));
    if (valid && rank == 0) wcnt[r][warp][d] = (uint16_t)__popc(peers);
    dr[r] = d | (rank << 8) | (valid ? 1u << 16 : 0u);
  }
  // keys of all smaller digits: exclusive scan of the totals over the 256 digits
  uint32_t inc = all_d;
#pragma unroll
  for (int j = 1; j < 32; j <<= 1) {
    const uint32_t t = __shfl_up_sync(0xFFFFFFFFu, inc, j);
    if (lane >= j) inc += t;
  }
  if (lane == 31) warp_tot[warp] = inc;
  __syncthreads();
  uint32_t mine = 0;  // keys of digit threadIdx.x in this tile
#pragma unroll
  for (int r = 0; r < kSortRounds; ++r) {
    uint32_t c[kWarps];
#pragma unroll
    for (int w = 0; w < kWarps; ++w) c[w] = wcnt[r][w][threadIdx.x];
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      wcnt[r][w][threadIdx.x] = (uint16_t)mine;
      mine += c[w];
    }
  }
  st_status(status + (size_t)blockIdx.x * 256 + threadIdx.x, kFlagLocal | mine);
  uint32_t start = inc - all_d;
  for (int w = 0; w < warp; ++w) start += warp_tot[w];
  // keys of this digit in the tiles before this one: first the tiles of this tile's group ...
  const int group = (int)blockIdx.x / kGroup, in_group = (int)blockIdx.x % kGroup;
  uint32_t before = 0;
  Patience patience;
  {
    const uint32_t* w0 = status + (size_t)group * kGroup * 256 + threadIdx.x;
    bool ready = in_group == 0;
    while (!ready && !patience.over()) {
      uint32_t v[kGroup - 1];
#pragma unroll
      for (int j = 0; j < kGroup - 1; ++j) v[j] = j < in_group ? ld_status(w0 + (size_t)j * 256) : kFlagLocal;
      uint32_t all = kFlagLocal, sum = 0;
#pragma unroll
      for (int j = 0; j < kGroup - 1; ++j) {
        all &= v[j];
        sum += v[j] & kValueMask;
      }
      ready = (all & kFlagLocal) != 0;
      if (ready) before = sum;
      else patience.pause();
    }
  }
  if (in_group == kGroup - 1 && !patience.over()) st_status(group_status + (size_t)group * 256 + threadIdx.x, kFlagLocal | (before + mine));
  // ... then the groups before this tile's group
  for (int g0 = 0; g0 < group && !patience.over(); g0 += kLookBatch) {
    const uint32_t* w0 = group_status + (size_t)g0 * 256 + threadIdx.x;
    bool ready = false;
    while (!ready && !patience.over()) {
      uint32_t v[kLookBatch];
#pragma unroll
      for (int j = 0; j < kLookBatch; ++j) v[j] = g0 + j < group ? ld_status(w0 + (size_t)j * 256) : kFlagLocal;
      uint32_t all = kFlagLocal, sum = 0;
#pragma unroll
      for (int j = 0; j < kLookBatch; ++j) {
        all &= v[j];
        sum += v[j] & kValueMask;
      }
      ready = (all & kFlagLocal) != 0;
      if (ready) before += sum;
      else patience.pause();
    }
  }
  const bool stalled = patience.over();
  sbase[threadIdx.x] = start + before;
  if (__syncthreads_or(stalled)) {
    if (threadIdx.x == 0) atomicOr(err, (uint32_t)MFET_DEV_STALLED);
    return;
  }
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
  asm volatile("griddepcontrol.launch_dependents;");  // see digit_totals_kernel
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

// Adjacent-unique over the sorted keys, in two launches, neither of which waits for another block.
// A head is the first of a run of equal keys. Counts travel as one 64-bit word: heads in bits
// 0..30, cache misses in bits 31..61 (both below 2^30).

// Launch 1: a tile counts its heads; with PROBE it also looks every head up in the cache, remembers
// the answer per sorted position and counts the misses. The tile stores its counts and adds them
// to the sum of its group of kCountGroup tiles (zeroed by digit_totals_kernel).
template <bool PROBE>
__global__ void __launch_bounds__(kScanThreads) unique_count_kernel(NSrc ns, const uint64_t* __restrict__ keys,
                                                                    CacheDev cache, int32_t* __restrict__ probe_tmp,
                                                                    uint64_t* __restrict__ tile_counts,
                                                                    unsigned long long* group_sums) {
  __shared__ uint32_t sh[8];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // see sort_pass_kernel
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t tile0 = (int64_t)blockIdx.x * kScanTile;
  if (tile0 >= n) return;
  const int64_t i0 = tile0 + (int64_t)threadIdx.x * kScanItems;
  uint32_t heads = 0, misses = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    if (i < n) {
      const uint64_t k = ld_l2(keys + i);
      if ((i == 0) || (ld_l2(keys + i - 1) != k)) {
        ++heads;
        if (PROBE) {
          const int32_t slot = cache_probe(cache, (int64_t)k);
          probe_tmp[i] = slot;
          if (slot < 0) ++misses;
        }
      }
    }
  }
  uint32_t th = 0, tm = 0;
  block_excl_scan(heads, &th, sh);
  if (PROBE) block_excl_scan(misses, &tm, sh);
  if (threadIdx.x == 0) {
    const uint64_t mine = (uint64_t)th | ((uint64_t)tm << 31);
    tile_counts[blockIdx.x] = mine;
    atomicAdd(group_sums + blockIdx.x / kCountGroup, (unsigned long long)mine);
  }
  asm volatile("griddepcontrol.launch_dependents;");  // see digit_totals_kernel
}

// Launch 2: a tile adds up the counts of the tiles before it (those of its own group one by one,
// the groups before it by their sums) and writes uniq, inverse and (PROBE) the per-unique source
// and the list of missed rows. The tile that holds the last key publishes the totals.
template <bool PROBE>
__global__ void __launch_bounds__(kScanThreads) unique_write_kernel(NSrc ns, const uint64_t* __restrict__ keys,
                                                                    const uint32_t* __restrict__ idx,
                                                                    const int32_t* __restrict__ probe_tmp,
                                                                    const uint64_t* __restrict__ tile_counts,
                                                                    const unsigned long long* __restrict__ group_sums,
                                                                    int64_t* __restrict__ uniq, int32_t* __restrict__ inverse,
                                                                    int32_t* __restrict__ src, int64_t* __restrict__ miss_rows,
                                                                    int64_t* __restrict__ n_unique,
                                                                    int64_t* __restrict__ n_miss, uint32_t* total,
                                                                    uint32_t* err) {
  __shared__ uint32_t sh[8];
  __shared__ uint64_t sh_part[kScanThreads / 32];
  asm volatile("griddepcontrol.wait;" ::: "memory");  // see sort_pass_kernel
  int64_t lo;
  const int64_t n = resolve_n(ns, &lo);
  const int64_t tile0 = (int64_t)blockIdx.x * kScanTile;
  if (blockIdx.x == 0) {
    // the passes are done with the digit totals: leave them at zero for the next call
    for (int j = threadIdx.x; j < kMaxPasses * 256; j += kScanThreads) total[j] = 0;
    if (n == 0 && threadIdx.x == 0) {
      *n_unique = 0;
      if (PROBE) *n_miss = 0;
    }
  }
  if (tile0 >= n) return;
  // counts of the tiles before this one: asked for first, needed last
  const int group = (int)blockIdx.x / kCountGroup, in_group = (int)blockIdx.x % kCountGroup;
  uint64_t part = (int)threadIdx.x < in_group ? ld_l2(tile_counts + group * kCountGroup + threadIdx.x) : 0ull;
  for (int g = threadIdx.x; g < group; g += kScanThreads) part += (uint64_t)__ldcg(group_sums + g);
  const int64_t i0 = tile0 + (int64_t)threadIdx.x * kScanItems;
  uint64_t k[kScanItems];
  uint32_t pos[kScanItems];
  bool head[kScanItems];
  int32_t slot[kScanItems];
  uint32_t heads = 0, misses = 0;
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    head[j] = false;
    slot[j] = 0;
    k[j] = 0;
    pos[j] = 0;
    if (i < n) {
      k[j] = ld_l2(keys + i);
      pos[j] = ld_l2(idx + i);
      head[j] = (i == 0) || (ld_l2(keys + i - 1) != k[j]);
      if (head[j]) {
        ++heads;
        if (PROBE) {
          slot[j] = ld_l2(probe_tmp + i);
          if (slot[j] < 0) ++misses;
        }
      }
    }
  }
  uint32_t th = 0, tm = 0;
  uint32_t u = block_excl_scan(heads, &th, sh);
  uint32_t m = 0;
  if (PROBE) m = block_excl_scan(misses, &tm, sh);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xFFFFFFFFu, part, o);
  if ((threadIdx.x & 31) == 0) sh_part[threadIdx.x >> 5] = part;
  __syncthreads();
  uint64_t before = 0;
#pragma unroll
  for (int w = 0; w < kScanThreads / 32; ++w) before += sh_part[w];
  if (threadIdx.x == 0 && tile0 + kScanTile >= n) {
    const uint64_t all = before + ((uint64_t)th | ((uint64_t)tm << 31));
    *n_unique = (int64_t)(all & 0x7FFFFFFFull);
    if (PROBE) *n_miss = (int64_t)(all >> 31);
  }
  u += (uint32_t)(before & 0x7FFFFFFFull);
  m += (uint32_t)(before >> 31);
  // u = number of heads strictly before this thread's first element
#pragma unroll
  for (int j = 0; j < kScanItems; ++j) {
    const int64_t i = i0 + j;
    if (i < n && MFET_IN_BOUNDS(err, (int64_t)u - (head[j] ? 0 : 1) < n && (int64_t)m <= n && (int64_t)pos[j] < n)) {
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
      inverse[pos[j]] = (int32_t)(u - 1);
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
  l.hist = take(((uint64_t)(l.nblk_sort + (l.nblk_sort + kGroup - 1) / kGroup) * 2 + kMaxPasses) * 256 * 4);  // digit totals + two sets of status words
  l.tile_counts = take((uint64_t)(l.nblk_scan + (l.nblk_scan + kCountGroup - 1) / kCountGroup) * 8);  // the unique kernels' tile counts and group sums
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
  // status words of the passes (two sets, used in turn), then the digit totals of every pass
  const int64_t cap = a.ns.offsets ? a.ns.cap : a.ns.n_imm;
  if (cap >= (int64_t)kValueMask) return cudaErrorInvalidValue;  // counts travel in 30 bits
  const int nblk = (int)((cap + kSortTile - 1) / kSortTile) > 0 ? (int)((cap + kSortTile - 1) / kSortTile) : 1;
  const int nblk2 = (int)((cap + kScanTile - 1) / kScanTile) > 0 ? (int)((cap + kScanTile - 1) / kScanTile) : 1;
  // the digit totals of every pass (zero between calls), then two sets of status words, used in turn
  uint32_t* total = (uint32_t*)(ws + L.hist);
  const int ngroups = (nblk + kGroup - 1) / kGroup;
  uint32_t* status[2] = {total + kMaxPasses * 256, total + kMaxPasses * 256 + (size_t)nblk * 256};
  uint32_t* group_status[2] = {status[1] + (size_t)nblk * 256, status[1] + (size_t)(nblk + ngroups) * 256};
  uint64_t* ustatus = (uint64_t*)(ws + L.tile_counts);
  int bits = 1;
  while (bits < 63 && (a.max_key >> bits) != 0) ++bits;
  const int passes = (bits + 7) / 8;

  if (a.hash)
    digit_totals_kernel<true><<<nblk, kHistThreads, 0, s>>>(a.ns, nullptr, ka, a.hash->ids, a.hash->seed, a.hash->rows,
                                                            a.hash->magic, a.hash->pre_hashed, passes, total, status[0],
                                                            group_status[0], ustatus, nblk2, a.err);
  else
    digit_totals_kernel<false><<<nblk, kHistThreads, 0, s>>>(a.ns, a.first_keys, nullptr, nullptr, 0, 0, 0, 0, passes, total,
                                                             status[0], group_status[0], ustatus, nblk2, a.err);
  *launches += 1;
  // Every later kernel of the call may start while the one before it still runs (it waits
  // inside, before it touches global memory), which hides the launch latency between them.
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.blockDim = dim3(kSortThreads);
  cfg.gridDim = dim3((unsigned)nblk);
  cfg.stream = s;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  cudaError_t e = cudaSuccess;
  const uint64_t* kin = a.hash ? ka : a.first_keys;
  const uint32_t* iin = nullptr;
  uint64_t* kout = a.hash ? kb : ka;
  uint32_t* iout = ia;
  for (int p = 0; p < passes; ++p) {
    e = cudaLaunchKernelEx(&cfg, sort_pass_kernel, a.ns, kin, iin, kout, iout, 8 * p, (const uint32_t*)(total + p * 256),
                           status[p & 1], group_status[p & 1], p + 1 < passes ? status[(p + 1) & 1] : (uint32_t*)nullptr,
                           group_status[(p + 1) & 1], a.err);
    if (e != cudaSuccess) return e;
    *launches += 1;
    // next pass reads what this one wrote
    kin = kout;
    iin = iout;
    kout = (kout == ka) ? kb : ka;
    iout = (iout == ia) ? ib : ia;
  }
  // kin / iin: sorted keys and their original positions; iout is free
  int32_t* probe_tmp = (int32_t*)iout;
  uint64_t* tile_counts = ustatus;
  unsigned long long* group_sums = (unsigned long long*)(ustatus + nblk2);
  cfg.blockDim = dim3(kScanThreads);
  cfg.gridDim = dim3((unsigned)nblk2);
  if (a.cache) {
    e = cudaLaunchKernelEx(&cfg, unique_count_kernel<true>, a.ns, kin, *a.cache, probe_tmp, tile_counts, group_sums);
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, unique_write_kernel<true>, a.ns, kin, iin, (const int32_t*)probe_tmp,
                           (const uint64_t*)tile_counts, (const unsigned long long*)group_sums, a.uniq, a.inverse, a.src,
                           a.miss_rows, a.n_unique, a.n_miss, total, a.err);
  } else {
    CacheDev none{};
    e = cudaLaunchKernelEx(&cfg, unique_count_kernel<false>, a.ns, kin, none, (int32_t*)nullptr, tile_counts, group_sums);
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, unique_write_kernel<false>, a.ns, kin, iin, (const int32_t*)nullptr,
                           (const uint64_t*)tile_counts, (const unsigned long long*)group_sums, a.uniq, a.inverse, a.src,
                           (int64_t*)nullptr, a.n_unique, (int64_t*)nullptr, total, a.err);
  }
  if (e != cudaSuccess) return e;
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
constexpr uint64_t kOffTiles = kOffHist + pad256(((kStaticSortBlocks + (kStaticSortBlocks + mfet::kGroup - 1) / mfet::kGroup) * 2 + mfet::kMaxPasses) * 256 * 4);
constexpr uint64_t kOffCounters = kOffTiles + pad256((kStaticScanBlocks + (kStaticScanBlocks + mfet::kCountGroup - 1) / mfet::kCountGroup) * 8);
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
      // The status words that a pass polls are cleared by an earlier kernel of the same call.
      // The digit totals must be zero on entry: the array starts out zero (device memory of the
      // library image), and every call leaves them at zero.
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
