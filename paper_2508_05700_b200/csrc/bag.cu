// K-bag: fused hash -> gather -> pool -> concatenated store, all device-table
// slots of a batch in one launch.
//
// Work split. A block takes one (slot, tile of up to 64 consecutive samples);
// the tile's CSR offsets are staged in shared memory. Inside the block a BAG
// GROUP of GL lanes owns one bag at a time. A row of the table is 16-byte
// chunks; LPR lanes (a ROW GROUP) read one row with one 16-byte load each, so a
// bag group reads GL/LPR rows per load instruction. GL is either LPR (short
// bags: no cross-lane reduction at all, several bags per warp) or 32 (long
// bags: the whole warp streams one bag), chosen per tile from its mean length.
//
// Per round a bag group takes GL IDs: every lane loads and hashes one ID
// (coalesced 8-byte loads, all lanes busy), then the row offsets travel by
// shuffle to the row group that loads them, U loads in flight per lane.
// Accumulation is fp32; row groups are combined by a shuffle reduce-scatter so
// that every lane ends with a distinct piece of the output row and the store is
// one coalesced segment. The order of additions depends only on the inputs and
// the tile configuration, never on timing.
#include "common.cuh"

// Tunables (overridable at build time for sweeps): row loads kept in flight per
// lane, and the minimum number of resident blocks per SM that caps registers.
#ifndef MFET_BAG_U
#define MFET_BAG_U 4
#endif
#ifndef MFET_BAG_LONG
#define MFET_BAG_LONG 64
#endif
#ifndef MFET_BAG_MINB
#define MFET_BAG_MINB 4
#endif

namespace mfet {

namespace {

constexpr unsigned kFull = 0xFFFFFFFFu;
constexpr int kLongBag = MFET_BAG_LONG;  // bags at least this long get a whole warp

template <int DT>
struct ChunkElems {
  static constexpr int value = (DT == MFET_F32) ? 4 : 8;
};

// acc += w * (the 16-byte chunk v decoded to fp32); exact up-conversion.
template <int DT>
__device__ __forceinline__ void accumulate(float* acc, const uint4& v, float w) {
  if constexpr (DT == MFET_F32) {
    acc[0] = fmaf(w, __uint_as_float(v.x), acc[0]);
    acc[1] = fmaf(w, __uint_as_float(v.y), acc[1]);
    acc[2] = fmaf(w, __uint_as_float(v.z), acc[2]);
    acc[3] = fmaf(w, __uint_as_float(v.w), acc[3]);
  } else if constexpr (DT == MFET_F16) {
    const uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&x[j]));
      acc[2 * j] = fmaf(w, f.x, acc[2 * j]);
      acc[2 * j + 1] = fmaf(w, f.y, acc[2 * j + 1]);
    }
  } else {
    const uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      acc[2 * j] = fmaf(w, bf16lo(x[j]), acc[2 * j]);
      acc[2 * j + 1] = fmaf(w, bf16hi(x[j]), acc[2 * j + 1]);
    }
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
  constexpr int NF = (E / GG) > 0 ? (E / GG) : 1;  // values a lane stores

  const int lane = threadIdx.x & 31;
  const int gl = lane & (GL - 1);
  const int sub = gl / LPR;
  const int c = gl & (LPR - 1);
  const int grp = threadIdx.x / GL;
  const bool chunk_ok = c < (int)s.chunks;
  const bool wsum = s.pooling == MFET_POOL_WSUM;
  const bool pre = (p.flags & 1u) != 0;
  const bool narrow = !IND && s.narrow != 0;
  const uint8_t* tbase = s.table + c * 16;  // IND: s.table = byte offset of the column block
  const uint64_t stride16 = s.stride >> 4;
  const unsigned long long* ids = reinterpret_cast<const unsigned long long*>(p.ids);

  // bags perm[q0 .. q1) of the tile, NG at a time (perm orders the tile by falling length,
  // so the bag groups of one warp work on bags of similar length)
  for (int qb = q0; qb < q1; qb += NG) {
    const int q = qb + grp;
    const bool have = q < q1;
    const int bi = have ? (int)perm[q] : 0;
    int64_t lo = 0;
    int len = 0;
    if (have) {
      lo = soff[bi];
      int64_t l = soff[bi + 1] - lo;
      if (l < 0) {
        if (gl == 0) atomicOr(p.err, (uint32_t)MFET_DEV_OFFSETS);
        l = 0;
      }
      len = l > 0x7FFFFFFF ? 0x7FFFFFFF : (int)l;
    }
    const int maxlen = __reduce_max_sync(kFull, len);

    float acc[E];
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = 0.f;

    for (int base = 0; base < maxlen; base += GL) {
      // every lane of the bag group hashes one ID of this round
      uint64_t off16 = ~0ULL;  // sentinel: no row
      float w = 1.f;
      if (base + gl < len) {
        const int64_t i = lo + base + gl;
        if constexpr (IND) {
          const int32_t j = __ldg(ip.inverse + (i - feat_lo));
          const int32_t sidx = __ldg(ip.src + j);
          const uint8_t* rowp = sidx >= 0 ? ip.cache_data + (uint64_t)sidx * ip.row_bytes
                                          : ip.staging + (uint64_t)(-1 - sidx) * ip.row_bytes;
          off16 = reinterpret_cast<uint64_t>(rowp) >> 4;
        } else {
          const uint64_t id = __ldcs(ids + i);
          const uint64_t row = pre ? id : mod_rows(splitmix64(id ^ s.seed), s.rows, s.magic);
          if (row < s.rows) off16 = row * stride16;
          else atomicOr(p.err, (uint32_t)MFET_DEV_ROW_RANGE);
        }
        if (wsum) w = __ldcs(p.weights + i);
      }
      const uint32_t off_lo = (uint32_t)off16, off_hi = (uint32_t)(off16 >> 32);
      const int cnt = min(GL, maxlen - base);  // warp-uniform
#pragma unroll
      for (int u0 = 0; u0 < LPR; u0 += U) {
        if (u0 * GG >= cnt) break;
        uint4 v[U];
        float wk[U];
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
          wk[k] = wsum ? __shfl_sync(kFull, w, src, GL) : 1.f;
          v[k] = make_uint4(0u, 0u, 0u, 0u);
          if (valid && chunk_ok)
            v[k] = ld_row16(tbase + ((((uint64_t)o_hi << 32) | o_lo) << 4));
        }
#pragma unroll
        for (int k = 0; k < U; ++k) accumulate<DT>(acc, v[k], wk[k]);
      }
    }

    int off = 0;
    bool writer = have && chunk_ok;
    ReduceScatter<E, 0, GG, LPR>::run(acc, sub, off, writer);
    if (s.pooling == MFET_POOL_MEAN && len > 0) {
      const float fl = (float)len;
#pragma unroll
      for (int j = 0; j < NF; ++j) acc[j] = __fdiv_rn(acc[j], fl);
    }
    if (writer) {
      float* o = p.out + (int64_t)(b0 + bi) * p.out_ld + s.col_off + c * E + off;
      if (p.flags & 2u) {
        if constexpr (NF >= 4) {
#pragma unroll
          for (int j = 0; j < NF; j += 4)
            __stcs(reinterpret_cast<float4*>(o + j), make_float4(acc[j], acc[j + 1], acc[j + 2], acc[j + 3]));
        } else if constexpr (NF == 2) {
          __stcs(reinterpret_cast<float2*>(o), make_float2(acc[0], acc[1]));
        } else {
          __stcs(o, acc[0]);
        }
      } else {
#pragma unroll
        for (int j = 0; j < NF; ++j) __stcs(o + j, acc[j]);
      }
    }
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

template <bool IND>
__device__ __forceinline__ void bag_body(const BagParams& p, const IndirectParams& ip) {
  __shared__ int64_t soff[kMaxTile + 1];
  __shared__ int64_t sfeat[2];
  __shared__ uint8_t perm[kMaxTile];
  __shared__ int scnt[2][16];
  const int slot = blockIdx.x / p.tiles_per_slot;
  const int tile = blockIdx.x - slot * p.tiles_per_slot;
  const SlotDev& s = p.slot[slot];
  const int b0 = tile * p.tile;
  const int nb = min(p.tile, p.batch - b0);
  const long long* offs = reinterpret_cast<const long long*>(p.offsets) + (int64_t)s.feature * p.batch;
  if ((int)threadIdx.x <= nb) soff[threadIdx.x] = __ldcs(offs + b0 + threadIdx.x);
  if (IND && threadIdx.x < 2) sfeat[threadIdx.x] = offs[threadIdx.x ? p.batch : 0];
  if (threadIdx.x >= 128 && threadIdx.x < 160) (&scnt[0][0])[threadIdx.x - 128] = 0;
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
  if (warp_ < 2) {  // threads 0..63 own one bag each
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
    int rank = in_warp + (warp_ ? scnt[0][cls] : 0);
    for (int c2 = cls + 1; c2 < 16; ++c2) rank += scnt[0][c2] + scnt[1][c2];
    perm[rank] = (uint8_t)threadIdx.x;
  }
  __syncthreads();
  int n_long = scnt[0][15] + scnt[1][15];
  if (p.group_policy == 1) n_long = 0;
  if (p.group_policy == 2) n_long = nb;

  switch (s.dtype) {
    case MFET_F32: pool_tile_dt<MFET_F32, IND>(MFET_POOL_ARGS, n_long, nb); break;
    case MFET_F16: pool_tile_dt<MFET_F16, IND>(MFET_POOL_ARGS, n_long, nb); break;
    default: pool_tile_dt<MFET_BF16, IND>(MFET_POOL_ARGS, n_long, nb); break;
  }
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_kernel(const __grid_constant__ BagParams p) {
  const IndirectParams none{};
  bag_body<false>(p, none);
}

__global__ void __launch_bounds__(256, MFET_BAG_MINB) bag_indirect_kernel(const __grid_constant__ BagParams p,
                                                           const __grid_constant__ IndirectParams ip) {
  bag_body<true>(p, ip);
}

}  // namespace

cudaError_t launch_bag_indirect(const BagParams& p, const IndirectParams& ip, cudaStream_t s) {
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  if (blocks == 0) return cudaSuccess;
  bag_indirect_kernel<<<(unsigned)blocks, 256, 0, s>>>(p, ip);
  return cudaGetLastError();
}

cudaError_t launch_bag(const BagParams& p, cudaStream_t s) {
  const int64_t blocks = (int64_t)p.n_slots * p.tiles_per_slot;
  if (blocks == 0) return cudaSuccess;
  bag_kernel<<<(unsigned)blocks, 256, 0, s>>>(p);
  return cudaGetLastError();
}

}  // namespace mfet
