// K-bag: fused hash -> gather -> pool -> concatenated store, all device-table
// slots of a batch in one launch.
//
// Work split. A block takes one (slot, tile of up to 64 consecutive samples);
// the tile's CSR offsets are staged in shared memory and its bags are ordered by
// falling length class. Inside the block a BAG GROUP of GL lanes owns one bag at
// a time. A table row is 16-byte chunks; LPR lanes (a ROW GROUP) read one row
// with one 16-byte load each, so a bag group reads GL/LPR rows per load
// instruction. Long bags get GL = 32 (the whole warp streams one bag), all other
// bags GL = LPR (several bags per warp, no cross-lane reduction at all); thanks
// to the ordering the bag groups of a warp work on bags of similar length.
//
// The work of a bag group is a sequence of ROUNDS of GL IDs. In a round every
// lane hashes one ID (coalesced 8-byte loads, prefetched one round ahead so the
// ID latency hides behind the previous round's rows), the row offsets travel by
// shuffle to the row group that loads them, U loads are in flight per lane, and
// batches of loads whose rows exist in every bag group of the warp run without
// predicates. Accumulation is fp32 (packed two-wide FMA); row groups are
// combined by a shuffle reduce-scatter so that every lane ends with a distinct
// piece of the output row and the store is one coalesced segment. The order of
// additions depends only on the inputs and the tile configuration, never on
// timing.
#include "common.cuh"

// Tunables (overridable at build time for sweeps): row loads kept in flight per
// lane, the length from which a bag gets a whole warp and the minimum number of
// resident blocks per SM (caps registers).
#ifndef MFET_BAG_U
#define MFET_BAG_U 4
#endif
#ifndef MFET_BAG_LONG
#define MFET_BAG_LONG 64
#endif
#ifndef MFET_BAG_MINB
#define MFET_BAG_MINB 5
#endif

namespace mfet {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kLongBag = MFET_BAG_LONG;  // bags at least this long get a whole warp

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

// One bag of a bag group, as the round loop sees it.
struct BagCur {
  int64_t lo;   // first ID of the bag
  int len;      // its length (0 when this group has no bag)
  int bi;       // index inside the tile
  int maxlen;   // longest / shortest bag among the warp's bag groups: the warp
  int minlen;   // runs maxlen rows, the first minlen of them without predicates
  bool have;
};

// IND = false: rows come from the slot's table by hashing the ID.
// IND = true : rows of a host-table slot come from the HBM cache or the staging
//              buffer, through the dedup inverse map (feat_lo = first ID of the
//              slot's feature, so that positions are slot-local).
template <int DT, int LPR, int GL, bool IND>
__device__ __forceinline__ void pool_tile(const BagParams& p, const SlotDev& s, const int64_t* soff,
                                          int b0, const uint8_t* perm, int q0, int q1,
                                          const IndirectParams& ip, int64_t feat_lo) {
  constexpr int E = ChunkElems<DT>::value;
  constexpr int GG = GL / LPR;          // row groups per bag group
  constexpr int NG = 256 / GL;          // bag groups per block
  constexpr int U = LPR < MFET_BAG_U ? LPR : MFET_BAG_U;  // row loads in flight per lane
  constexpr int NF = (E / GG) > 0 ? (E / GG) : 1;         // values a lane stores

  const int lane = threadIdx.x & 31;
  const int gl = lane & (GL - 1);
  const int sub = gl / LPR;
  const int c = gl & (LPR - 1);
  const int grp = threadIdx.x / GL;
  const bool all_chunks = (int)s.chunks == LPR;  // no idle chunk lanes
  const bool chunk_ok = c < (int)s.chunks;
  const bool wsum = s.pooling == MFET_POOL_WSUM;
  const bool pre = (p.flags & 1u) != 0;
  const bool narrow = !IND && s.narrow != 0;
  const uint8_t* tbase = s.table + c * ChunkElems<DT>::bytes;  // IND: s.table = byte offset of the column block
  const uint8_t* mbase = s.table + s.meta_off;               // INT4: the row's scale/bias pair
  const uint64_t stride16 = s.stride >> 4;
  const unsigned long long* ids = reinterpret_cast<const unsigned long long*>(p.ids);

  // bags perm[q0 .. q1) of the tile, NG at a time
  auto open_bag = [&](int qb, BagCur& b) {
    // bags come in falling length: every other pass hands them out in reverse group order, so
    // that no warp collects the longest bag of every pass
    const int q = qb + ((((qb - q0) / NG) & 1) ? NG - 1 - grp : grp);
    b.have = q < q1;
    b.bi = b.have ? (int)perm[q] : 0;
    b.lo = 0;
    b.len = 0;
    if (b.have) {
      b.lo = soff[b.bi];
      int64_t l = soff[b.bi + 1] - b.lo;
      if (l < 0) {
        if (gl == 0) atomicOr(p.err, (uint32_t)MFET_DEV_OFFSETS);
        l = 0;
      }
      b.len = l > 0x7FFFFFFF ? 0x7FFFFFFF : (int)l;
    }
    b.maxlen = __reduce_max_sync(kFull, b.len);
    b.minlen = __reduce_min_sync(kFull, b.len);
  };
  // the ID (or, IND, the row location) and weight of position base+gl of a bag
  auto fetch = [&](const BagCur& b, int base, uint64_t& id, float& w) {
    id = 0;
    w = 1.f;
    if (base + gl < b.len) {
      const int64_t i = b.lo + base + gl;
      if constexpr (IND) id = (uint32_t)__ldg(ip.inverse + (i - feat_lo));
      else id = __ldcs(ids + i);
      if (wsum) w = __ldcs(p.weights + i);
    }
  };

  if (q0 >= q1) return;
  BagCur cur;
  open_bag(q0, cur);
  int qb = q0, base = 0;
  uint64_t id_c;
  float w_c;
  fetch(cur, 0, id_c, w_c);

  unsigned long long acc[E / 2];
#pragma unroll
  for (int j = 0; j < E / 2; ++j) acc[j] = 0ull;

  while (true) {
    // ---- what comes after this round; its IDs are requested now -------------
    const bool last_round = base + GL >= cur.maxlen;  // warp-uniform
    BagCur nxt = cur;
    int nbase = base + GL, nqb = qb;
    bool more = true;
    if (last_round) {
      nqb = qb + NG;
      nbase = 0;
      more = nqb < q1;
      if (more) open_bag(nqb, nxt);
    }
    uint64_t id_n = 0;
    float w_n = 1.f;
    if (more) fetch(nxt, nbase, id_n, w_n);

    // ---- this round: every lane of the bag group resolves one row ------------
    uint64_t off16 = ~0ULL;  // sentinel: no row
    if (base + gl < cur.len) {
      if constexpr (IND) {
        const int32_t sidx = __ldg(ip.src + (uint32_t)id_c);
        const uint8_t* rowp = sidx >= 0 ? ip.cache_data + (uint64_t)sidx * ip.row_bytes
                                        : ip.staging + (uint64_t)(-1 - sidx) * ip.row_bytes;
        off16 = reinterpret_cast<uint64_t>(rowp) >> 4;
      } else {
        const uint64_t row = pre ? id_c : mod_rows(splitmix64(id_c ^ s.seed), s.rows, s.magic);
        if (row < s.rows) off16 = row * stride16;
        else atomicOr(p.err, (uint32_t)MFET_DEV_ROW_RANGE);
      }
    }
    const uint32_t off_lo = (uint32_t)off16, off_hi = (uint32_t)(off16 >> 32);
    const int cnt = min(GL, cur.maxlen - base);                 // IDs of the longest group
    const int full = all_chunks ? min(GL, cur.minlen - base) : 0;  // IDs that every group has
#pragma unroll
    for (int u0 = 0; u0 < LPR; u0 += U) {
      if (u0 * GG >= cnt) break;
      uint4 v[U];
      float wk[U];
      if ((u0 + U) * GG <= full && !pre) {
        // every lane has a row in each of the U steps: no predicates
#pragma unroll
        for (int k = 0; k < U; ++k) {
          const int src = (u0 + k) * GG + sub;
          const uint32_t o_lo = __shfl_sync(kFull, off_lo, src, GL);
          const uint32_t o_hi = narrow ? 0u : __shfl_sync(kFull, off_hi, src, GL);
          wk[k] = wsum ? __shfl_sync(kFull, w_c, src, GL) : 1.f;
          const uint64_t ro = (((uint64_t)o_hi << 32) | o_lo) << 4;
          v[k] = load_chunk<DT>(tbase + ro, mbase + ro);
        }
      } else {
#pragma unroll
        for (int k = 0; k < U; ++k) {
          const int src = (u0 + k) * GG + sub;
          const uint32_t o_lo = __shfl_sync(kFull, off_lo, src, GL);
          uint32_t o_hi = 0;
          bool valid;
          if (narrow) {
            valid = o_lo != 0xFFFFFFFFu;
          } else {
            o_hi = __shfl_sync(kFull, off_hi, src, GL);
            valid = (o_lo & o_hi) != 0xFFFFFFFFu;
          }
          wk[k] = wsum ? __shfl_sync(kFull, w_c, src, GL) : 1.f;
          v[k] = make_uint4(0u, 0u, 0u, 0u);
          const uint64_t ro = (((uint64_t)o_hi << 32) | o_lo) << 4;
          if (valid && chunk_ok) v[k] = load_chunk<DT>(tbase + ro, mbase + ro);
        }
      }
#pragma unroll
      for (int k = 0; k < U; ++k) accumulate<DT>(acc, v[k], wk[k]);
    }

    // ---- end of the bag: combine row groups, scale, store ---------------------
    if (last_round) {
      float a[E];
#pragma unroll
      for (int j = 0; j < E / 2; ++j) {
        a[2 * j] = __uint_as_float((uint32_t)acc[j]);
        a[2 * j + 1] = __uint_as_float((uint32_t)(acc[j] >> 32));
        acc[j] = 0ull;
      }
      int off = 0;
      bool writer = cur.have && chunk_ok;
      ReduceScatter<E, 0, GG, LPR>::run(a, sub, off, writer);
      if (s.pooling == MFET_POOL_MEAN && cur.len > 0) {
        const float fl = (float)cur.len;
#pragma unroll
        for (int j = 0; j < NF; ++j) a[j] = __fdiv_rn(a[j], fl);
      }
      if (writer) {
        float* o = p.out + (int64_t)(b0 + cur.bi) * p.out_ld + s.col_off + c * E + off;
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
    }
    if (!more) break;
    cur = nxt;
    qb = nqb;
    base = nbase;
    id_c = id_n;
    w_c = w_n;
  }
}


#define MFET_POOL_ARGS p, s, soff, b0, perm, ip, feat_lo

// Bags perm[0 .. n_long) are long: one warp each. The rest: one row group each.
template <int DT, int LPR, bool IND>
__device__ __forceinline__ void pool_tile_lpr(const BagParams& p, const SlotDev& s, const int64_t* soff,
                                              int b0, const uint8_t* perm, const IndirectParams& ip,
                                              int64_t feat_lo, int n_long, int nb) {
  if constexpr (LPR == 32) {
    pool_tile<DT, 32, 32, IND>(p, s, soff, b0, perm, 0, nb, ip, feat_lo);
  } else {
    if (n_long > 0) pool_tile<DT, LPR, 32, IND>(p, s, soff, b0, perm, 0, n_long, ip, feat_lo);
    if (n_long < nb) pool_tile<DT, LPR, LPR, IND>(p, s, soff, b0, perm, n_long, nb, ip, feat_lo);
  }
}

template <int DT, bool IND>
__device__ __forceinline__ void pool_tile_dt(const BagParams& p, const SlotDev& s, const int64_t* soff,
                                             int b0, const uint8_t* perm, const IndirectParams& ip,
                                             int64_t feat_lo, int n_long, int nb) {
  switch (s.lpr_log2) {
    case 1: pool_tile_lpr<DT, 2, IND>(MFET_POOL_ARGS, n_long, nb); break;
    case 2: pool_tile_lpr<DT, 4, IND>(MFET_POOL_ARGS, n_long, nb); break;
    case 3: pool_tile_lpr<DT, 8, IND>(MFET_POOL_ARGS, n_long, nb); break;
    case 4: pool_tile_lpr<DT, 16, IND>(MFET_POOL_ARGS, n_long, nb); break;
    default: pool_tile_lpr<DT, 32, IND>(MFET_POOL_ARGS, n_long, nb); break;
  }
}

// Q4 = true: the build of the kernel that also decodes INT4 rows (kept apart so that the
// common kernels stay small).
template <bool IND, bool Q4>
__device__ __forceinline__ void bag_body(const BagParams& p, const IndirectParams& ip) {
  __shared__ int64_t soff[kMaxTile + 1];
  __shared__ int64_t sfeat[2];
  __shared__ uint8_t perm[kMaxTile];
  constexpr int kSortWarps = kMaxTile / 32;  // warps whose threads own one bag each in the ordering
  __shared__ int scnt[kSortWarps][16];
  const int slot = blockIdx.x / p.tiles_per_slot;
  const int tile = blockIdx.x - slot * p.tiles_per_slot;
  const SlotDev& s = p.slot[slot];
  const int b0 = tile * p.tile;
  const int nb = min(p.tile, p.batch - b0);
  const long long* offs = reinterpret_cast<const long long*>(p.offsets) + (int64_t)s.feature * p.batch;
  if ((int)threadIdx.x <= nb) soff[threadIdx.x] = __ldcs(offs + b0 + threadIdx.x);
  if (IND && threadIdx.x < 2) sfeat[threadIdx.x] = offs[threadIdx.x ? p.batch : 0];
  if (threadIdx.x >= 128 && threadIdx.x < 128 + kSortWarps * 16) (&scnt[0][0])[threadIdx.x - 128] = 0;
  __syncthreads();
  int64_t feat_lo = 0;
  if constexpr (IND) {
    // a slot whose ID count exceeds the workspace capacity was not deduplicated:
    // every bag of it is written as zeros (the capacity error bit is already set)
    feat_lo = sfeat[0];
    const int64_t n_feat = sfeat[1] - sfeat[0];
    if (n_feat < 0 || n_feat > ip.cap) {
      __syncthreads();
      if ((int)threadIdx.x <= nb) soff[threadIdx.x] = feat_lo;
      __syncthreads();
    }
  }

  // Order the tile's bags by falling length class (counting sort over 16 classes, stable
  // inside a class): class 15 = long bags (a whole warp each), classes 0..14 = shorter ones
  // in steps of kLongBag/15, so that the bag groups of one warp get bags of similar length.
  const int lane_ = threadIdx.x & 31, warp_ = threadIdx.x >> 5;
  bool have = false;
  int cls = 0, in_warp = 0;
  if (warp_ < kSortWarps) {  // threads 0..kMaxTile-1 own one bag each
    have = (int)threadIdx.x < nb;
    if (have) {
      const int64_t l = soff[threadIdx.x + 1] - soff[threadIdx.x];
      const int len = l < 0 ? 0 : (l > 0x7FFFFFFF ? 0x7FFFFFFF : (int)l);
      cls = len >= kLongBag ? 15 : (len * 15) / kLongBag;
    }
    const unsigned peers = __match_any_sync(kFull, have ? cls : 16 + lane_);
    in_warp = __popc(peers & ((1u << lane_) - 1u));
    if (have && in_warp == 0) scnt[warp_][cls] = __popc(peers);
  }
  __syncthreads();
  if (have) {
    int rank = in_warp;
    for (int w2 = 0; w2 < warp_; ++w2) rank += scnt[w2][cls];
    for (int c2 = cls + 1; c2 < 16; ++c2)
#pragma unroll
      for (int w2 = 0; w2 < kSortWarps; ++w2) rank += scnt[w2][c2];
    perm[rank] = (uint8_t)threadIdx.x;
  }
  __syncthreads();
  int n_long = 0;
#pragma unroll
  for (int w2 = 0; w2 < kSortWarps; ++w2) n_long += scnt[w2][15];
  if (p.group_policy == 1) n_long = 0;
  if (p.group_policy == 2) n_long = nb;

  if constexpr (Q4) {
    if (s.dtype == MFET_INT4) {
      pool_tile_dt<MFET_INT4, IND>(MFET_POOL_ARGS, n_long, nb);
      return;
    }
  }
  switch (s.dtype) {
    case MFET_F32: pool_tile_dt<MFET_F32, IND>(MFET_POOL_ARGS, n_long, nb); break;
    case MFET_F16: pool_tile_dt<MFET_F16, IND>(MFET_POOL_ARGS, n_long, nb); break;
    default: pool_tile_dt<MFET_BF16, IND>(MFET_POOL_ARGS, n_long, nb); break;
  }
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_kernel(const __grid_constant__ BagParams p) {
  const IndirectParams none{};
  bag_body<false, false>(p, none);
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_q4_kernel(const __grid_constant__ BagParams p) {
  const IndirectParams none{};
  bag_body<false, true>(p, none);
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_indirect_kernel(const __grid_constant__ BagParams p,
                                                           const __grid_constant__ IndirectParams ip) {
  bag_body<true, false>(p, ip);
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_indirect_q4_kernel(const __grid_constant__ BagParams p,
                                                              const __grid_constant__ IndirectParams ip) {
  bag_body<true, true>(p, ip);
}

}  // namespace

static bool any_int4(const BagParams& p) {
  for (int i = 0; i < p.n_slots; ++i)
    if (p.slot[i].dtype == MFET_INT4) return true;
  return false;
}

cudaError_t launch_bag_indirect(const BagParams& p, const IndirectParams& ip, cudaStream_t s) {
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  if (blocks == 0) return cudaSuccess;
  if (any_int4(p)) bag_indirect_q4_kernel<<<(unsigned)blocks, 256, 0, s>>>(p, ip);
  else bag_indirect_kernel<<<(unsigned)blocks, 256, 0, s>>>(p, ip);
  return cudaGetLastError();
}

cudaError_t launch_bag(const BagParams& p, cudaStream_t s) {
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  if (blocks == 0) return cudaSuccess;
  if (any_int4(p)) bag_q4_kernel<<<(unsigned)blocks, 256, 0, s>>>(p);
  else bag_kernel<<<(unsigned)blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace mfet
