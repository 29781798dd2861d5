// K-bag: fused hash -> gather -> pool -> concatenated store, all device-table
// slots of a batch in one launch.
//
// Work split. A block takes one (slot, tile of up to 128 consecutive samples).
// The IDs of a tile are one contiguous range of the CSR arrays, so the block
// first STAGES them: all 256 threads stream the range with coalesced loads, hash
// every ID to its table row and park the 32-bit row index (and the weight) in
// shared memory. The hashing of the whole tile therefore runs with full memory
// parallelism and before any row is requested; the gather that follows has no
// load that depends on another global load, and its inner loop is little more
// than shared-memory read, address, 16-byte load and the fp32 adds.
//
// Gather. A table row is 16-byte chunks; LPR lanes (a ROW GROUP) read one row
// with one 16-byte load each. The tile's bags are ordered: long bags first, then
// the others by falling length (counting sort). A long bag gets a whole warp
// (its 32/LPR row groups stride over the bag's rows and are combined by a
// shuffle reduce-scatter, so that every lane ends with a distinct piece of the
// output row); every other bag is owned by one row group (32/LPR bags of nearly
// equal length per warp, no cross-lane reduction at all). Warps take their next
// bags from a shared counter. The steps that all lanes of a warp have in common
// run without predicates in batches of U loads per lane; accumulation is fp32
// (packed two-wide FMA).
//
// A tile whose IDs do not fit the staging buffer is processed in WINDOWS of the
// buffer's capacity; a bag cut by a window boundary continues from the partial
// sum that its earlier piece left in the output row. The order of additions
// depends only on the inputs, the tile size and the staging capacity, never on
// timing.
#include <algorithm>
#include <atomic>
#include <functional>
#include <mutex>
#include <queue>
#include <vector>

#include "common.cuh"

namespace mfet {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kLongBag = 64;      // bags at least this long get a whole warp (32: measured slower)
constexpr int kGatherLoads = 8;  // row loads that a lane keeps in flight (4 with 48 registers: slower)
constexpr int kMinBlocks = 4;    // resident blocks per SM that the register budget allows (3, 5: slower)
// the ordering of the shorter bags has one lane per length class: classes of kClassW lengths
constexpr int kClassW = (kLongBag + 31) / 32;
constexpr int kClasses = (kLongBag + kClassW - 1) / kClassW;  // <= 32; class kClasses = long bags
static_assert(kLongBag >= 1 && kClasses <= 32, "one lane per class of shorter bags");

// A lane's piece of a row: 16 bytes (4 fp32 or 8 fp16/bf16 values), or for INT4 rows
// 4 bytes (8 four-bit codes) plus the row's fp16 scale/bias pair.
template <int DT>
struct ChunkElems {
  static constexpr int value = (DT == MFET_F32) ? 4 : 8;
  static constexpr int bytes = (DT == MFET_INT4) ? 4 : 16;
};

template <int DT>
__device__ __forceinline__ uint4 load_chunk(const uint8_t* chunk, const uint8_t* meta) {
  if constexpr (DT == MFET_INT4) return make_uint4(ld_row4(chunk), ld_row4(meta), 0u, 0u);
  else return ld_row16(chunk);
}

__device__ __forceinline__ unsigned long long pack2(uint32_t lo, uint32_t hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "r"(lo), "r"(hi));
  return r;
}

// a += x * w on two packed fp32 lanes (each lane one IEEE fused multiply-add).
__device__ __forceinline__ void fma2(unsigned long long& a, unsigned long long x, unsigned long long w) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a) : "l"(x), "l"(w));
}

// acc (E fp32 values as E/2 packed pairs) += w * (the 16-byte chunk v decoded to
// fp32). The up-conversion of fp16 / bf16 is exact.
template <int DT>
__device__ __forceinline__ void accumulate(unsigned long long* acc, const uint4& v, float w) {
  if constexpr (DT == MFET_INT4) {
    // value = fma(code, scale, bias) in fp32 (one rounding), then acc += w * value
    const float2 sb = __half22float2(*reinterpret_cast<const __half2*>(&v.y));
    const unsigned long long s2 = pack2(__float_as_uint(sb.x), __float_as_uint(sb.x));
    const unsigned long long b2 = pack2(__float_as_uint(sb.y), __float_as_uint(sb.y));
    const unsigned long long w2 = pack2(__float_as_uint(w), __float_as_uint(w));
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      // codes 2j, 2j+1 -> exact floats through the 2^23 mantissa trick
      const uint32_t lo = 0x4B000000u | ((v.x >> (8 * j)) & 15u), hi = 0x4B000000u | ((v.x >> (8 * j + 4)) & 15u);
      const float c0 = __uint_as_float(lo) - 8388608.f, c1 = __uint_as_float(hi) - 8388608.f;
      unsigned long long val = b2;
      fma2(val, pack2(__float_as_uint(c0), __float_as_uint(c1)), s2);
      fma2(acc[j], val, w2);
    }
    return;
  }
  const uint32_t x[4] = {v.x, v.y, v.z, v.w};
  const unsigned long long w2 = pack2(__float_as_uint(w), __float_as_uint(w));
  if constexpr (DT == MFET_F32) {
    fma2(acc[0], pack2(x[0], x[1]), w2);
    fma2(acc[1], pack2(x[2], x[3]), w2);
  } else if constexpr (DT == MFET_F16) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&x[j]));
      fma2(acc[j], pack2(__float_as_uint(f.x), __float_as_uint(f.y)), w2);
    }
  } else {
#pragma unroll
    for (int j = 0; j < 4; ++j) fma2(acc[j], pack2(x[j] << 16, x[j] & 0xFFFF0000u), w2);
  }
}

// Combine the GG row groups of a bag group. While a lane holds more than one
// value, each step halves what it keeps (reduce-scatter); afterwards plain
// butterfly adds, with only one lane of each pair left as the writer.
template <int N, int K, int GG, int LPR>
struct ReduceScatter {
  static __device__ __forceinline__ void run(float* v, int sub, int& off, bool& writer) {
    if constexpr ((1 << K) < GG) {
      const int dist = LPR << K;
      const bool bit = (sub >> K) & 1;
      if constexpr (N > 1) {
        constexpr int H = N / 2;
#pragma unroll
        for (int i = 0; i < H; ++i) {
          const float send = bit ? v[i] : v[i + H];
          const float keep = bit ? v[i + H] : v[i];
          v[i] = keep + __shfl_xor_sync(kFull, send, dist);
        }
        off += bit ? H : 0;
        ReduceScatter<H, K + 1, GG, LPR>::run(v, sub, off, writer);
      } else {
        v[0] += __shfl_xor_sync(kFull, v[0], dist);
        writer = writer && !bit;
        ReduceScatter<1, K + 1, GG, LPR>::run(v, sub, off, writer);
      }
    }
  }
};


// What a warp needs to know about the block's staging window. The window's bags
// are listed long ones first, then by falling length: entry q has the window
// position of the bag's first staged row, the number of its rows in the window
// and the bag's index in the tile (plus kNotFirst when an earlier window held the
// start of the bag and kNotLast when a later one holds its end).
constexpr int kNotFirst = 0x100, kNotLast = 0x200;
struct Win {
  const uint32_t* srow;   // staged row index (IND: dedup source index) per window position
  const uint32_t* shi;    // its upper half, for tables of more than 2^32-1 rows
  const float* sw;        // staged weight per window position (weighted slots)
  const int* spos;        // per listed bag, see above
  const int* slen;
  const int* sbag;
  int* next;              // shared work counter
  const int64_t* soff;    // the tile's CSR offsets
  int nbw;                // bags listed
  int n_long;             // the first n_long of them get a whole warp
  int b0;                 // first sample of the tile
};

// Where this lane's chunk (and, INT4, the scale/bias pair) of a staged row is.
// Direct tables: base + row * stride. IND: the dedup source index selects the
// cache (>= 0) or the staging buffer of fetched rows (< 0: -1 - index).
template <bool IND>
struct RowAddr {
  const uint8_t* tbase;   // table (IND: cache rows) + this lane's chunk offset
  const uint8_t* mbase;   // same + the offset of the scale/bias pair
  const uint8_t* tbase2;  // IND: the fetched-rows variants
  const uint8_t* mbase2;
  uint64_t stride;
  uint32_t stride32;
  bool wide;              // row index or stride beyond 32 bits
#ifdef MFET_CHECKED
  uint64_t rows, rows2;   // rows of the table (IND: of the cache), IND: of the fetched-rows buffer
  uint32_t* err;
  __device__ __forceinline__ bool row_ok(uint32_t lo, uint32_t hi) const {
    if constexpr (IND) {
      const bool cached = (int32_t)lo >= 0;
      return MFET_IN_BOUNDS(err, (uint64_t)(cached ? lo : ~lo) < (cached ? rows : rows2));
    } else {
      return MFET_IN_BOUNDS(err, (wide ? (((uint64_t)hi << 32) | lo) : (uint64_t)lo) < rows);
    }
  }
#else
  __device__ __forceinline__ bool row_ok(uint32_t, uint32_t) const { return true; }
#endif
  // the common case: row index and stride fit 32 bits
  __device__ __forceinline__ void get_narrow(uint32_t lo, const uint8_t*& chunk, const uint8_t*& meta) const {
    if constexpr (IND) {
      get(lo, 0u, chunk, meta);
    } else {
      const uint64_t off = (uint64_t)lo * stride32;
      chunk = tbase + off;
      meta = mbase + off;
    }
  }
  __device__ __forceinline__ void get(uint32_t lo, uint32_t hi, const uint8_t*& chunk, const uint8_t*& meta) const {
    if constexpr (IND) {
      const bool cached = (int32_t)lo >= 0;
      const uint64_t off = (uint64_t)(cached ? lo : ~lo) * stride32;
      chunk = (cached ? tbase : tbase2) + off;
      meta = (cached ? mbase : mbase2) + off;
    } else {
      const uint64_t off = wide ? (((uint64_t)hi << 32) | lo) * stride : (uint64_t)lo * stride32;
      chunk = tbase + off;
      meta = mbase + off;
    }
  }
};

// N consecutive steps of a lane: N row chunks are requested, then added to acc.
// srow/shi/sw point at the lane's first of these steps; a step is GG staged
// entries further than the one before. WS: the slot is weighted (a compile-time
// copy of the flag for the common path). PRED = false: every lane has all N
// steps, the table is narrow and every staged row is a row. PRED = true: the
// lane has only `left` of the N steps (possibly none or all of them), and a
// staged row may be the "no row" sentinel or lie outside this lane's chunks;
// what is not loaded counts as zeros.
template <int DT, int GG, bool IND, int N, bool PRED, bool WS, bool PLAIN = false>
__device__ __forceinline__ void run_steps(const uint32_t* srow, const uint32_t* shi, const float* sw,
                                          const RowAddr<IND>& ra, bool wsum, int left, bool chunk_ok,
                                          unsigned long long* acc) {
  uint4 v[N];
#pragma unroll
  for (int j = 0; j < N; ++j) {
    const uint8_t *a, *m;
    if constexpr (PRED && PLAIN) {
      // predicated, but the table is narrow, every staged row is a row and every lane has a chunk
      v[j] = make_uint4(0u, 0u, 0u, 0u);
      if (j < left) {
        const uint32_t lo = srow[j * GG];
        if (ra.row_ok(lo, 0u)) {
          ra.get_narrow(lo, a, m);
          v[j] = load_chunk<DT>(a, m);
        }
      }
    } else if constexpr (PRED) {
      v[j] = make_uint4(0u, 0u, 0u, 0u);
      if (j < left && chunk_ok) {
        const uint32_t lo = srow[j * GG];
        const uint32_t hi = (!IND && ra.wide) ? shi[j * GG] : 0u;
        if ((IND || (ra.wide ? (lo & hi) != 0xFFFFFFFFu : lo != 0xFFFFFFFFu)) && ra.row_ok(lo, hi)) {
          ra.get(lo, hi, a, m);
          v[j] = load_chunk<DT>(a, m);
        }
      }
    } else {
      const uint32_t lo = srow[j * GG];
      v[j] = make_uint4(0u, 0u, 0u, 0u);
      if (ra.row_ok(lo, 0u)) {
        ra.get_narrow(lo, a, m);
        v[j] = load_chunk<DT>(a, m);
      }
    }
  }
#pragma unroll
  for (int j = 0; j < N; ++j) {
    float wj = 1.f;
    if constexpr (PRED) {
      if (wsum && j < left) wj = sw[j * GG];
    } else if constexpr (WS) {
      wj = sw[j * GG];
    }
    accumulate<DT>(acc, v[j], wj);
  }
}

// The steps that every lane of the warp has, without predicates, in batches of U, then 4;
// up to 3 of them are left to the predicated batches.
template <int DT, int GG, bool IND, bool WS>
__device__ __forceinline__ int run_common(const uint32_t* srow, const float* sw, const RowAddr<IND>& ra,
                                          int min_steps, unsigned long long* acc) {
  constexpr int U = kGatherLoads;
  int t = 0;
  for (; t + U <= min_steps; t += U)
    run_steps<DT, GG, IND, U, false, WS>(srow + t * GG, nullptr, sw + t * GG, ra, WS, 0, true, acc);
  if constexpr (U > 4) {
    if (t + 4 <= min_steps) {
      run_steps<DT, GG, IND, 4, false, WS>(srow + t * GG, nullptr, sw + t * GG, ra, WS, 0, true, acc);
      t += 4;
    }
  }
  return t;
}

// One bag piece per bag group of GG row groups: the staged rows pos0 + sub,
// pos0 + sub + GG, ... below pos0 + len are added to acc. GG == 1: every row
// group of the warp has its own (pos0, len); GG > 1: the warp shares them.
// The steps that every lane of the warp has run without predicates in batches
// of U and 4; the last few, and those that only some lanes have (the bags of a
// warp are of nearly the same length), run in predicated batches of 4: every
// batch is one round trip to memory, so the remainder is not split further.
template <int DT, int LPR, int GG, bool IND>
__device__ __forceinline__ void gather_piece(const Win& w, const RowAddr<IND>& ra, int pos0, int len, int sub,
                                             bool fast_ok, bool chunk_ok, bool wsum, unsigned long long* acc) {
  // row loads (steps) of this lane, of the warp's busiest lane and of its idlest one
  int steps, max_steps, min_steps;
  if constexpr (GG == 1) {
    steps = len;
    max_steps = __reduce_max_sync(kFull, len);
    min_steps = fast_ok ? __reduce_min_sync(kFull, len) : 0;
  } else {
    steps = (len - sub + GG - 1) / GG;
    max_steps = (len + GG - 1) / GG;
    min_steps = fast_ok ? len / GG : 0;
  }
  const uint32_t* srow = w.srow + pos0 + sub;
  const uint32_t* shi = w.shi + pos0 + sub;
  const float* sw = w.sw + pos0 + sub;
  int t;
  if (wsum) t = run_common<DT, GG, IND, true>(srow, sw, ra, min_steps, acc);
  else t = run_common<DT, GG, IND, false>(srow, sw, ra, min_steps, acc);
  // what is left: fewer than 4 common steps and the steps that only some lanes have
  if (fast_ok) {
    for (; t < max_steps; t += 4)
      run_steps<DT, GG, IND, 4, true, false, true>(srow + t * GG, shi + t * GG, sw + t * GG, ra, wsum, steps - t, true,
                                                   acc);
  } else {
    for (; t < max_steps; t += 4)
      run_steps<DT, GG, IND, 4, true, false>(srow + t * GG, shi + t * GG, sw + t * GG, ra, wsum, steps - t, chunk_ok,
                                             acc);
  }
}

// Listed bag q of the window (or no bag: q < 0), pooled by a bag group of GG row
// groups and stored (first piece), or added to what the earlier pieces left in
// the output row.
template <int DT, int LPR, int GG, bool IND>
__device__ __forceinline__ void pool_bag(const BagParams& p, const SlotDev& s, const Win& w,
                                         const RowAddr<IND>& ra, int q, int sub, int c, bool fast_ok,
                                         bool chunk_ok, bool wsum) {
  constexpr int E = ChunkElems<DT>::value;
  constexpr int NF = (E / GG) > 0 ? (E / GG) : 1;  // values a lane stores
  int pos0 = 0, len = 0, bag = -1;
  if (q >= 0) {
    pos0 = w.spos[q];
    len = w.slen[q];
    bag = w.sbag[q];
  }
  unsigned long long acc[E / 2];
#pragma unroll
  for (int j = 0; j < E / 2; ++j) acc[j] = 0ull;
  gather_piece<DT, LPR, GG, IND>(w, ra, pos0, len, sub, fast_ok, chunk_ok, wsum, acc);

  float a[E];
#pragma unroll
  for (int j = 0; j < E / 2; ++j) {
    a[2 * j] = __uint_as_float((uint32_t)acc[j]);
    a[2 * j + 1] = __uint_as_float((uint32_t)(acc[j] >> 32));
  }
  int off = 0;
  bool writer = bag >= 0 && chunk_ok;
  ReduceScatter<E, 0, GG, LPR>::run(a, sub, off, writer);
  if (!writer) return;
  const int bi = bag & 0xFF;
  if (!MFET_IN_BOUNDS(p.err, w.b0 + bi < p.batch && (int64_t)s.col_off + c * E + off + NF <= p.out_ld)) return;
  float* o = p.out + (int64_t)(w.b0 + bi) * p.out_ld + s.col_off + c * E + off;
  if (bag & kNotFirst) {
#pragma unroll
    for (int j = 0; j < NF; ++j) a[j] += __ldcg(o + j);
  }
  if (s.pooling == MFET_POOL_MEAN && !(bag & kNotLast)) {
    const int64_t blen = w.soff[bi + 1] - w.soff[bi];
    if (blen > 0) {
      const float inv = __frcp_rn((float)blen);  // correctly rounded reciprocal, then one rounding per product
#pragma unroll
      for (int j = 0; j < NF; ++j) a[j] *= inv;
    }
  }
  if (p.flags & 2u) {
    if constexpr (NF >= 4) {
#pragma unroll
      for (int j = 0; j < NF; j += 4)
        __stcs(reinterpret_cast<float4*>(o + j), make_float4(a[j], a[j + 1], a[j + 2], a[j + 3]));
    } else if constexpr (NF == 2) {
      __stcs(reinterpret_cast<float2*>(o), make_float2(a[0], a[1]));
    } else {
      __stcs(o, a[0]);
    }
  } else {
#pragma unroll
    for (int j = 0; j < NF; ++j) __stcs(o + j, a[j]);
  }
}

// The warps of the block pool the window's bags: the long ones first, one warp
// each, then the others, one row group each, handed out through the shared counter.
template <int DT, int LPR, bool IND>
__device__ __forceinline__ void pool_window(const BagParams& p, const SlotDev& s, const Win& w,
                                            const IndirectParams& ip) {
  constexpr int BPW = 32 / LPR;
  const int lane = threadIdx.x & 31;
  const int rg = lane / LPR;
  const int c = lane & (LPR - 1);
  const bool chunk_ok = c < (int)s.chunks;
  const bool wsum = s.pooling == MFET_POOL_WSUM;
  const bool fast_ok = (int)s.chunks == LPR && !(p.flags & 1u) && (IND || s.narrow != 0);
  RowAddr<IND> ra;
  const uint64_t coff = (uint64_t)c * ChunkElems<DT>::bytes;
  if constexpr (IND) {
    const uint64_t slot_off = reinterpret_cast<uint64_t>(s.table);  // byte offset of the column block in the row
    ra.tbase = ip.cache_data + slot_off + coff;
    ra.mbase = ip.cache_data + slot_off + s.meta_off;
    ra.tbase2 = ip.staging + slot_off + coff;
    ra.mbase2 = ip.staging + slot_off + s.meta_off;
    ra.stride = ip.row_bytes;
    ra.stride32 = (uint32_t)ip.row_bytes;
    ra.wide = false;
#ifdef MFET_CHECKED
    ra.rows = (uint64_t)ip.cache_n;
    ra.rows2 = (uint64_t)ip.cap;
    ra.err = p.err;
#endif
  } else {
    ra.tbase = s.table + coff;
    ra.mbase = s.table + s.meta_off;
    ra.tbase2 = ra.mbase2 = nullptr;
    ra.stride = s.stride;
    ra.stride32 = (uint32_t)s.stride;
    ra.wide = s.narrow == 0;
#ifdef MFET_CHECKED
    ra.rows = s.rows;
    ra.rows2 = 0;
    ra.err = p.err;
#endif
  }
  const int n_long = BPW > 1 ? w.n_long : 0;
  while (true) {
    int u = 0;
    if (lane == 0) u = atomicAdd(w.next, 1);
    u = __shfl_sync(kFull, u, 0);
    if constexpr (BPW > 1) {
      if (u < n_long) {
        pool_bag<DT, LPR, BPW, IND>(p, s, w, ra, u, rg, c, fast_ok, chunk_ok, wsum);
        continue;
      }
    }
    const int q0 = n_long + (u - n_long) * BPW;
    if (q0 >= w.nbw) break;
    const int q = q0 + rg;
    pool_bag<DT, LPR, 1, IND>(p, s, w, ra, q < w.nbw ? q : -1, 0, c, fast_ok, chunk_ok, wsum);
  }
}

template <int DT, bool IND>
__device__ __forceinline__ void pool_window_dt(const BagParams& p, const SlotDev& s, const Win& w,
                                               const IndirectParams& ip) {
  switch (s.lpr_log2) {
    case 1: pool_window<DT, 2, IND>(p, s, w, ip); break;
    case 2: pool_window<DT, 4, IND>(p, s, w, ip); break;
    case 3: pool_window<DT, 8, IND>(p, s, w, ip); break;
    case 4: pool_window<DT, 16, IND>(p, s, w, ip); break;
    default: pool_window<DT, 32, IND>(p, s, w, ip); break;
  }
}

// IDs (and weights) a thread requests before the tile's bags are ordered, so
// that their latency overlaps the ordering.
constexpr int kEarly = 8;

// Q4 = true: the build of the kernel that also decodes INT4 rows (kept apart so that the
// common kernels stay small).
template <bool IND, bool Q4>
__device__ __forceinline__ void bag_body(const BagParams& p, const IndirectParams& ip) {
  extern __shared__ __align__(16) uint32_t dyn[];
  __shared__ int64_t soff[kMaxTile + 1];
  __shared__ int64_t sfeat[2];
  __shared__ int spos[kMaxTile], slen[kMaxTile], sbag[kMaxTile];
  constexpr int kSortWarps = kMaxTile / 32;  // warps whose threads own one bag each in the ordering
  constexpr int kCnt = kSortWarps * (kClasses + 1);  // per sorting warp: the classes of shorter bags, long bags
  static_assert(kCnt <= 256, "one thread clears one counter");
  __shared__ int scnt[kSortWarps][kClasses + 1];
  __shared__ int snext;
  const int tid = threadIdx.x;
  // Launched with programmatic stream serialisation (flag bit 4), the blocks of the NEXT launch on the
  // stream may start as soon as every block of this one has got here; they read and hash their own
  // inputs, then wait below until this launch is complete. Without that launch attribute both
  // instructions do nothing.
  asm volatile("griddepcontrol.launch_dependents;");
  const int slot = blockIdx.x / p.tiles_per_slot;
  const int tile = blockIdx.x - slot * p.tiles_per_slot;
  const SlotDev& s = p.slot[slot];
  const int b0 = tile * p.tile;
  const int nb = min(p.tile, p.batch - b0);
  const int C = p.stage_cap;
  uint32_t* srow = dyn;
  float* sw = reinterpret_cast<float*>(dyn + ((p.flags & 4u) ? C : 0));
  uint32_t* shi = dyn + ((p.flags & 8u) ? ((p.flags & 4u) ? 2 * C : C) : 0);
  const long long* offs = reinterpret_cast<const long long*>(p.offsets) + (int64_t)s.feature * p.batch;
  if (tid <= nb) {
    soff[tid] = MFET_IN_BOUNDS(p.err, (int64_t)s.feature * p.batch + b0 + tid <= (int64_t)p.n_features * p.batch)
                    ? __ldcs(offs + b0 + tid) : 0;
  }
#ifdef MFET_CHECKED
  __shared__ int64_t snnz;  // number of IDs in the batch: the extent of ids and weights
  if (tid == 0) snnz = p.offsets[(int64_t)p.n_features * p.batch];
#endif
  if (IND && tid < 2) sfeat[tid] = offs[tid ? p.batch : 0];
  if (tid < kCnt) (&scnt[0][0])[tid] = 0;
  if (tid == 255) snext = 0;
  __syncthreads();
  int64_t feat_lo = 0;
  if constexpr (IND) {
    // a slot whose ID count exceeds the workspace capacity was not deduplicated:
    // every bag of it is written as zeros (the capacity error bit is already set)
    feat_lo = sfeat[0];
    const int64_t n_feat = sfeat[1] - sfeat[0];
    if (n_feat < 0 || n_feat > ip.cap) {
      __syncthreads();
      if (tid <= nb) soff[tid] = feat_lo;
      __syncthreads();
    }
  }
  const int64_t t0 = soff[0];
  int64_t n_tile = soff[nb] - t0;
  if (n_tile < 0) {
    if (tid == 0) atomicOr(p.err, (uint32_t)MFET_DEV_OFFSETS);
    n_tile = 0;
  }
  const bool wsum = s.pooling == MFET_POOL_WSUM;
  const bool pre = (p.flags & 1u) != 0;
  const bool wide = !IND && s.narrow == 0;
  const unsigned long long* ids = reinterpret_cast<const unsigned long long*>(p.ids);

  // the ID (IND: the position in the dedup list) of a lookup -> staged value of window position pos
  auto stage = [&](int pos, uint64_t id) {
    if (!MFET_IN_BOUNDS(p.err, pos >= 0 && pos < C)) return;
    if constexpr (IND) {
      srow[pos] = MFET_IN_BOUNDS(p.err, (int64_t)(uint32_t)id < ip.cap) ? (uint32_t)__ldg(ip.src + (uint32_t)id) : 0u;
    } else {
      uint64_t row = mod_rows(splitmix64(id ^ s.seed), s.rows, s.magic);
      if (pre) {  // the caller's row indices are used as they are, and checked
        row = id;
        if (row >= s.rows) {
          atomicOr(p.err, (uint32_t)MFET_DEV_ROW_RANGE);
          row = ~0ULL;  // sentinel: no row
        }
      }
      srow[pos] = (uint32_t)row;
      if (wide) shi[pos] = (uint32_t)(row >> 32);
    }
  };
#ifdef MFET_CHECKED
  const int64_t nnz = snnz;
#endif
  auto fetch_id = [&](int64_t i) -> uint64_t {
    if constexpr (IND) {
      if (!MFET_IN_BOUNDS(p.err, i - feat_lo >= 0 && i - feat_lo < ip.cap)) return 0;
      return (uint32_t)__ldg(ip.inverse + (i - feat_lo));
    } else {
#ifdef MFET_CHECKED
      if (!MFET_IN_BOUNDS(p.err, i >= 0 && i < nnz)) return 0;
#endif
      return __ldcs(ids + i);
    }
  };
  auto fetch_w = [&](int64_t i) -> float {
#ifdef MFET_CHECKED
    if (!MFET_IN_BOUNDS(p.err, i >= 0 && i < nnz)) return 0.f;
#endif
    return __ldcs(p.weights + i);
  };

  for (int64_t w0 = 0;; w0 += C) {
    const int wn = (int)(n_tile - w0 < (int64_t)C ? n_tile - w0 : (int64_t)C);
    const int64_t g0 = t0 + w0;  // global index of window position 0
    // ---- request the first IDs of the window --------------------------------
    uint64_t eid[kEarly];
    float ew[kEarly];
#pragma unroll
    for (int k = 0; k < kEarly; ++k) {
      const int pos = tid + k * 256;
      eid[k] = 0;
      ew[k] = 1.f;
      if (pos < wn) {
        eid[k] = fetch_id(g0 + pos);
        if (wsum) ew[k] = fetch_w(g0 + pos);
      }
    }
    // ---- order the bags that have a piece in this window: the long pieces first (a whole
    // warp each), then the others by falling length class (counting sort, stable inside a
    // class), so that the row groups of one warp get pieces of nearly the same length.
    // Empty bags belong to window 0.
    const int lane_ = tid & 31, warp_ = tid >> 5;
    bool have = false;
    int cls = 0, in_warp = 0, plen = 0, ppos = 0, pbag = tid;
    if (warp_ < kSortWarps) {  // threads 0..kMaxTile-1 own one bag each
      if (tid < nb) {
        const int64_t lo = soff[tid] - t0;
        int64_t hi = soff[tid + 1] - t0;
        if (hi < lo) {
          if (w0 == 0) atomicOr(p.err, (uint32_t)MFET_DEV_OFFSETS);
          hi = lo;
        }
        const int64_t a = lo > w0 ? lo : w0;
        const int64_t b = hi < w0 + wn ? hi : w0 + wn;
        if (b > a) {
          plen = (int)(b - a);
          ppos = (int)(a - w0);
        }
        have = plen > 0 || (w0 == 0 && hi == lo);
        if (lo < w0 && w0 != 0) pbag |= kNotFirst;
        if (hi > w0 + wn) pbag |= kNotLast;
        cls = plen < kLongBag ? plen / kClassW : kClasses;
      }
      const unsigned peers = __match_any_sync(kFull, have ? cls : 64 + lane_);
      in_warp = __popc(peers & ((1u << lane_) - 1u));
      if (have && in_warp == 0) scnt[warp_][cls] = __popc(peers);
    }
    const int nbw = __syncthreads_count(have);
    int n_long = 0;
#pragma unroll
    for (int w2 = 0; w2 < kSortWarps; ++w2) n_long += scnt[w2][kClasses];
    if (warp_ < kSortWarps) {
      // lane c of every sorting warp: the bags of class c in all warps, and in the warps before this one
      int tot = 0, before = 0, before_long = 0;
      if (lane_ < kClasses) {
#pragma unroll
        for (int w2 = 0; w2 < kSortWarps; ++w2) {
          const int n = scnt[w2][lane_];
          tot += n;
          before += w2 < warp_ ? n : 0;
        }
      }
#pragma unroll
      for (int w2 = 0; w2 < kSortWarps; ++w2) before_long += w2 < warp_ ? scnt[w2][kClasses] : 0;
      // shorter bags of a higher class than c: suffix sum over the lanes
      int longer = tot;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int o = __shfl_down_sync(kFull, longer, d);
        if (lane_ + d < 32) longer += o;
      }
      const int start = n_long + longer - tot + before;  // first listed position of this warp's bags of class c
      int rank = __shfl_sync(kFull, start, cls & 31);
      if (cls == kClasses) rank = before_long;
      if (have) {
        rank += in_warp;
        spos[rank] = ppos;
        slen[rank] = plen;
        sbag[rank] = pbag;
      }
    }
    // ---- hash the window's IDs into the staging buffer ------------------------
#pragma unroll
    for (int k = 0; k < kEarly; ++k) {
      const int pos = tid + k * 256;
      if (pos < wn) {
        stage(pos, eid[k]);
        if (wsum && MFET_IN_BOUNDS(p.err, pos < C)) sw[pos] = ew[k];
      }
    }
    // the rest of a large window, again with the loads of a batch requested before any of them is used
    for (int base = tid + kEarly * 256; base < wn; base += kEarly * 256) {
#pragma unroll
      for (int k = 0; k < kEarly; ++k) {
        const int pos = base + k * 256;
        if (pos < wn) {
          eid[k] = fetch_id(g0 + pos);
          if (wsum) ew[k] = fetch_w(g0 + pos);
        }
      }
#pragma unroll
      for (int k = 0; k < kEarly; ++k) {
        const int pos = base + k * 256;
        if (pos < wn) {
          stage(pos, eid[k]);
          if (wsum && MFET_IN_BOUNDS(p.err, pos < C)) sw[pos] = ew[k];
        }
      }
    }
    __syncthreads();
    // nothing of the stream's earlier kernel is touched before this point, nothing is written before it
    if (w0 == 0) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (p.group_policy == 1) n_long = 0;
    if (p.group_policy == 2) n_long = nbw;

    const Win w{srow, shi, sw, spos, slen, sbag, &snext, soff, nbw, n_long, b0};
    bool done = false;
    if constexpr (Q4) {
      if (s.dtype == MFET_INT4) {
        pool_window_dt<MFET_INT4, IND>(p, s, w, ip);
        done = true;
      }
    }
    if (!done) {
      switch (s.dtype) {
        case MFET_F32: pool_window_dt<MFET_F32, IND>(p, s, w, ip); break;
        case MFET_F16: pool_window_dt<MFET_F16, IND>(p, s, w, ip); break;
        default: pool_window_dt<MFET_BF16, IND>(p, s, w, ip); break;
      }
    }
    if (w0 + C >= n_tile) break;
    // ---- another window: everyone is done with the staging buffer and the bag list
    __syncthreads();
    if (tid < kCnt) (&scnt[0][0])[tid] = 0;
    if (tid == 255) snext = 0;
    __syncthreads();
  }
}

__global__ void __launch_bounds__(256, kMinBlocks) bag_kernel(const __grid_constant__ BagParams p) {
  const IndirectParams none{};
  bag_body<false, false>(p, none);
}

__global__ void __launch_bounds__(256, kMinBlocks) bag_q4_kernel(const __grid_constant__ BagParams p) {
  const IndirectParams none{};
  bag_body<false, true>(p, none);
}

__global__ void __launch_bounds__(256, kMinBlocks) bag_indirect_kernel(const __grid_constant__ BagParams p,
                                                           const __grid_constant__ IndirectParams ip) {
  bag_body<true, false>(p, ip);
}

__global__ void __launch_bounds__(256, kMinBlocks) bag_indirect_q4_kernel(const __grid_constant__ BagParams p,
                                                              const __grid_constant__ IndirectParams ip) {
  bag_body<true, true>(p, ip);
}

}  // namespace

static bool any_int4(const BagParams& p) {
  for (int i = 0; i < p.n_slots; ++i)
    if (p.slot[i].dtype == MFET_INT4) return true;
  return false;
}

// Samples per block when the caller has not fixed them. The blocks of a launch are handed to
// the SMs in index order (slots with the widest rows first), kMinBlocks at a time per SM; a
// block costs a fixed part (offsets, IDs, hashing, barriers) plus a part that grows with
// samples x lanes per row. The launch ends when the last block does, so for grids of one or
// two waves the tile decides how full the last wave is (4096 samples x 8 slots: 56-sample
// tiles make exactly 592 blocks = one block slot each on 148 SMs, 64-sample tiles leave 80
// slots idle and every block 14 % longer). For every candidate tile the order of dispatch is
// played through on the host (a heap of block-slot free times) and the shortest wins; the
// result is remembered per launch shape. When all slots have the same row width, only tiles
// that fit one wave compete with the size-based default: equal blocks in two or more whole
// waves run in lockstep (all hashing, then all gathering), which measured 5-8 % slower than a
// ragged last wave. Large grids take full tiles without the exercise.
static int choose_tile(const BagParams& p) {
  constexpr double kFixed = 20.0;  // fixed cost of a block, in samples of a 128-byte-row slot
  static std::mutex mu;
  struct Entry { int dev, batch, n, cnt[8], tile; };
  static std::vector<Entry> memo;
  int dev = 0;
  cudaGetDevice(&dev);
  const int slots = sm_count() * kMinBlocks;
  if ((int64_t)p.n_slots * ((p.batch + kMaxTile - 1) / kMaxTile) >= 6LL * slots) return kMaxTile;
  Entry key{};
  key.dev = dev;
  key.batch = p.batch;
  key.n = p.n_slots;
  for (int i = 0; i < p.n_slots; ++i) key.cnt[p.slot[i].lpr_log2 & 7] += 1;
  {
    std::lock_guard<std::mutex> g(mu);
    for (const Entry& e : memo)
      if (e.dev == key.dev && e.batch == key.batch && e.n == key.n && std::equal(e.cnt, e.cnt + 8, key.cnt)) return e.tile;
  }
  bool same_width = true;
  for (int i = 1; i < p.n_slots; ++i) same_width &= p.slot[i].lpr_log2 == p.slot[0].lpr_log2;
  const int64_t bags = (int64_t)p.batch * p.n_slots;
  const int by_size = bags >= 16384 ? 64 : (bags >= 4096 ? 32 : 16);
  int best = by_size;
  double best_t = 1e300;
  for (int tile = kMaxTile; tile >= 16; tile -= 8) {
    const int tiles = (p.batch + tile - 1) / tile;
    if ((int64_t)tiles * p.n_slots > 8LL * slots) break;  // many waves: the tile no longer matters
    if (same_width && (int64_t)tiles * p.n_slots > slots && tile != by_size) continue;
    std::priority_queue<double, std::vector<double>, std::greater<double>> free_at;
    double end = 0.0;
    int running = 0;
    for (int i = 0; i < p.n_slots; ++i) {
      const double full = kFixed + tile * (double)(1 << p.slot[i].lpr_log2) / 8.0;
      for (int k = 0; k < tiles; ++k) {
        const int nb = std::min(tile, p.batch - k * tile);
        const double cost = kFixed + (full - kFixed) * nb / tile;
        double start = 0.0;
        if (running < slots) {
          ++running;
        } else {
          start = free_at.top();
          free_at.pop();
        }
        free_at.push(start + cost);
        end = std::max(end, start + cost);
      }
    }
    if (end < best_t) {
      best_t = end;
      best = tile;
    }
  }
  key.tile = best;
  std::lock_guard<std::mutex> g(mu);
  if (memo.size() < 256) memo.push_back(key);
  return best;
}

// Tile, grid and dynamic shared memory of a launch: the staged row indices, plus the
// weights when a slot is weighted, plus the upper index halves when a table needs them.
// Sets the matching flag bits (4: weights staged, 8: upper halves staged).
static size_t stage_bytes(BagParams& p, bool indirect) {
  bool w = false, wide = false;
  for (int i = 0; i < p.n_slots; ++i) {
    w |= p.slot[i].pooling == MFET_POOL_WSUM;
    wide |= !indirect && p.slot[i].narrow == 0;
  }
  p.flags &= ~12u;
  if (w) p.flags |= 4u;
  if (wide) p.flags |= 8u;
  if (p.tile <= 0) p.tile = choose_tile(p);
  if (p.tile > kMaxTile) p.tile = kMaxTile;
  p.tiles_per_slot = (p.batch + p.tile - 1) / p.tile;
  // staging capacity: room for the IDs of a typical tile (a tile with more is pooled in several passes)
  if (p.stage_cap < 32) p.stage_cap = kStageDefault;
  if (p.stage_cap > kStageMax) p.stage_cap = kStageMax;
  return (size_t)p.stage_cap * 4u * (1u + (w ? 1u : 0u) + (wide ? 1u : 0u));
}

// Shared-memory set-up of a kernel for a launch with `smem` dynamic bytes, redone only when
// that size changes (per kernel and device): the opt-in that a block needs for more than 48 KB
// of shared memory (static and dynamic together), and a carve-out of just what the resident
// blocks need, so that the rest of the SM's array stays L1 for the rows.
template <typename K>
static cudaError_t prepare(K kernel, int which, size_t smem) {
  static std::atomic<long long> configured[4][64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  const long long want = (long long)smem + 1;
  if (configured[which][dev].load(std::memory_order_relaxed) == want) return cudaSuccess;
  cudaFuncAttributes fa{};
  cudaError_t e = cudaFuncGetAttributes(&fa, kernel);
  if (e != cudaSuccess) return e;
  if (smem + fa.sharedSizeBytes > 48 * 1024) {
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStageMax * 12);
    if (e != cudaSuccess) return e;
  }
  const size_t per_block = smem + fa.sharedSizeBytes + 1024;  // dynamic + static + the system's share
  size_t pct = (kMinBlocks * per_block * 100 + 228 * 1024 - 1) / (228 * 1024);
  if (pct > 100) pct = 100;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, (int)pct);
  if (e != cudaSuccess) return e;
  configured[which][dev].store(want, std::memory_order_relaxed);
  return cudaSuccess;
}

// Launch with or without permission to start before the stream's previous kernel has finished.
template <typename K, typename... Args>
static cudaError_t launch(K kernel, int64_t blocks, size_t smem, cudaStream_t s, bool overlap, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)blocks);
  cfg.blockDim = dim3(256);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = s;
  cudaLaunchAttribute attr{};
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = overlap ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, args...);
}

cudaError_t launch_bag_indirect(const BagParams& p_, const IndirectParams& ip, cudaStream_t s) {
  BagParams p = p_;
  if (p.n_slots == 0 || p.batch <= 0) return cudaSuccess;
  const size_t smem = stage_bytes(p, true);
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  cudaError_t e;
  if (any_int4(p)) {
    if ((e = prepare(bag_indirect_q4_kernel, 0, smem)) != cudaSuccess) return e;
    return launch(bag_indirect_q4_kernel, blocks, smem, s, false, p, ip);
  }
  if ((e = prepare(bag_indirect_kernel, 1, smem)) != cudaSuccess) return e;
  return launch(bag_indirect_kernel, blocks, smem, s, false, p, ip);
}

cudaError_t launch_bag(const BagParams& p_, cudaStream_t s) {
  BagParams p = p_;
  if (p.n_slots == 0 || p.batch <= 0) return cudaSuccess;
  const size_t smem = stage_bytes(p, false);
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  const bool overlap = (p.flags & 16u) != 0;
  cudaError_t e;
  if (any_int4(p)) {
    if ((e = prepare(bag_q4_kernel, 2, smem)) != cudaSuccess) return e;
    return launch(bag_q4_kernel, blocks, smem, s, overlap, p);
  }
  if ((e = prepare(bag_kernel, 3, smem)) != cudaSuccess) return e;
  return launch(bag_kernel, blocks, smem, s, overlap, p);
}

}  // namespace mfet
