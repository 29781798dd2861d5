// CPU oracle for the multi-faceted embedding-table lookup path.
//
// TEST INFRASTRUCTURE ONLY. This file is the slow, single-threaded, obviously
// correct restatement of what the lookup path computes. It is compiled with a
// plain host compiler, contains no CUDA, and shares no source, header, table or
// constant generator with the GPU library. Only the tests, the smoke check and
// the benchmark's CPU-baseline leg may load it; the product never does.
//
// What it follows in the paper:
//   * Section 2.2 ("Large Embedding Tables"): high-cardinality categorical IDs
//     are mapped to dense vectors through hashed lookup tables; collisions
//     appear once the number of distinct IDs exceeds the table's row count.
//     The paper names no hash function; this build's reading is the public
//     splitmix64 output function, reduced modulo the row count.
//   * Section 1 / Section 4.1.1 ("Multi-facet Pretraining"): one ID feature is
//     looked up in several independently pretrained tables (facets) and every
//     facet feeds the ranking model; reading: facet outputs are concatenated.
//   * Section 3.3 ("CPU-GPU Hybrid Serving"): the largest tables live in host
//     memory. Placement and caching are transparent to the result, so the
//     oracle ignores them.
//   * Section 4.1.2 ("Model Quantization"): INT4 post-training quantisation of
//     table rows. The paper gives no format; the row format decoded here is
//     this build's own (parity unpinned by the paper, pinned by a round-trip
//     error bound).
//
// The pooling itself (sum / mean / per-sample-weighted sum over a ragged bag)
// is the textbook embedding-bag definition, accumulated in double precision in
// input order.

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

extern "C" {

// ---------------------------------------------------------------- hashing ---

// splitmix64 output function (public domain, Steele/Lea/Flood; Vigna's
// reference): advance the state by the golden-ratio increment, then mix.
uint64_t orc_splitmix64(uint64_t x) {
  uint64_t z = x + 0x9E3779B97F4A7C15ULL;
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ULL;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBULL;
  return z ^ (z >> 31);
}

// Section 2.2: row = hash(id) mod rows. The per-table seed is XORed into the
// raw ID first, so facets of one feature collide differently.
int64_t orc_hash_row(uint64_t id, uint64_t seed, uint64_t rows) {
  return (int64_t)(orc_splitmix64(id ^ seed) % rows);
}

void orc_hash_ids(const uint64_t* ids, int64_t n, uint64_t seed, uint64_t rows,
                  int64_t* rows_out) {
  for (int64_t i = 0; i < n; ++i) rows_out[i] = orc_hash_row(ids[i], seed, rows);
}

// ------------------------------------------------------- number formats -----

// IEEE binary16 -> binary32, integer manipulation only.
uint32_t orc_f16_bits_to_f32_bits(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  uint32_t exp = (h >> 10) & 0x1Fu;
  uint32_t man = h & 0x3FFu;
  if (exp == 0x1Fu) return sign | 0x7F800000u | (man << 13);  // inf / nan
  if (exp == 0) {
    if (man == 0) return sign;  // signed zero
    // subnormal: value = man * 2^-24; normalise
    int shift = 0;
    while ((man & 0x400u) == 0) {
      man <<= 1;
      ++shift;
    }
    man &= 0x3FFu;
    uint32_t e32 = (uint32_t)(127 - 15 - shift + 1);
    return sign | (e32 << 23) | (man << 13);
  }
  return sign | ((exp + (127 - 15)) << 23) | (man << 13);
}

// bfloat16 is the upper half of binary32.
uint32_t orc_bf16_bits_to_f32_bits(uint16_t b) { return (uint32_t)b << 16; }

// binary32 -> bfloat16, round to nearest even.
uint16_t orc_f32_bits_to_bf16_bits(uint32_t f) {
  if ((f & 0x7F800000u) == 0x7F800000u) {  // inf / nan
    uint16_t hi = (uint16_t)(f >> 16);
    if ((f & 0x007FFFFFu) != 0) hi |= 0x0040u;  // keep it a nan
    return hi;
  }
  uint32_t lsb = (f >> 16) & 1u;
  f += 0x7FFFu + lsb;
  return (uint16_t)(f >> 16);
}

// binary32 -> binary16, round to nearest even, integer manipulation only.
uint16_t orc_f32_bits_to_f16_bits(uint32_t f) {
  uint16_t sign = (uint16_t)((f >> 16) & 0x8000u);
  uint32_t exp = (f >> 23) & 0xFFu;
  uint32_t man = f & 0x007FFFFFu;
  if (exp == 0xFFu) return sign | 0x7C00u | (man ? (0x0200u | (man >> 13)) : 0);
  int e = (int)exp - 127 + 15;
  if (e >= 0x1F) return sign | 0x7C00u;  // overflow -> inf
  if (e <= 0) {
    // result is subnormal or zero: value = (1.man) * 2^(exp-127), unit 2^-24
    if (e < -10) return sign;  // below half the smallest subnormal
    man |= 0x00800000u;
    int shift = 14 - e;  // 14..24
    uint32_t q = man >> shift;
    uint32_t rem = man & ((1u << shift) - 1u);
    uint32_t half = 1u << (shift - 1);
    if (rem > half || (rem == half && (q & 1u))) ++q;
    return sign | (uint16_t)q;  // q may carry into the exponent: still correct
  }
  uint32_t q = ((uint32_t)e << 10) | (man >> 13);
  uint32_t rem = man & 0x1FFFu;
  if (rem > 0x1000u || (rem == 0x1000u && (q & 1u))) ++q;  // carry may reach inf
  return sign | (uint16_t)q;
}

static inline float bits_to_float(uint32_t b) {
  float f;
  std::memcpy(&f, &b, 4);
  return f;
}
static inline uint32_t float_to_bits(float f) {
  uint32_t b;
  std::memcpy(&b, &f, 4);
  return b;
}

// ------------------------------------------------------ table descriptors ---

enum { ORC_F32 = 0, ORC_F16 = 1, ORC_BF16 = 2, ORC_INT4 = 3 };
enum { ORC_POOL_SUM = 0, ORC_POOL_MEAN = 1, ORC_POOL_WSUM = 2 };
enum { ORC_VAL_NORMAL = 0, ORC_VAL_GRID = 1 };

typedef struct {
  const void* data;     // materialised rows, or NULL for procedural values
  uint64_t rows;        // >= 1
  uint32_t dim;         // elements per row
  uint32_t dtype;       // ORC_F32 / ORC_F16 / ORC_BF16 / ORC_INT4
  uint64_t hash_seed;   // XORed into the raw ID before hashing
  uint64_t row_stride;  // bytes between rows of `data`; 0 = dense
  uint64_t value_key;   // procedural tables: key of the value generator
  uint32_t value_mode;  // ORC_VAL_NORMAL / ORC_VAL_GRID
  uint32_t reserved;
} orc_table_t;

static inline uint32_t elem_bytes(uint32_t dtype) { return dtype == ORC_F32 ? 4u : 2u; }

// Bytes of one row as stored. INT4 rows: dim/2 packed nibbles followed by an
// fp16 scale and an fp16 bias, padded up to a multiple of 16 bytes.
uint64_t orc_row_bytes(uint32_t dim, uint32_t dtype) {
  if (dtype == ORC_INT4) return (((uint64_t)dim / 2 + 4) + 15) / 16 * 16;
  return (uint64_t)dim * elem_bytes(dtype);
}

// Procedural table entry: a pure function of (key, row, column), so that
// tables of 80-130 GB never have to exist on the host. The table contents are
// INPUTS of the method (the paper's tables are pretrained weights that are
// not available); this is a counter-based generator:
//   k = r*dim + d;  u = splitmix64(key + k)
//   NORMAL: s = sum of the four 16-bit fields of u (Irwin-Hall, mean 131070,
//           std 37837.227); v = float(s - 131070) * c, c = 0.01/std, giving
//           an approximately N(0, 0.01^2) value (tails end at +-3.46 sigma).
//   GRID:   v = float((u & 255) - 128) * 2^-13 (exact in every dtype; any
//           unweighted sum of up to 2^11 of them is exact in fp32).
// v is then rounded to nearest-even into the table's dtype.
float orc_table_value_f32(uint64_t key, uint32_t mode, uint32_t dim, uint64_t r, uint32_t d) {
  uint64_t k = r * (uint64_t)dim + d;
  uint64_t u = orc_splitmix64(key + k);
  if (mode == ORC_VAL_GRID) {
    int32_t g = (int32_t)(u & 0xFFu) - 128;
    return (float)g * 0x1p-13f;
  }
  int32_t s = (int32_t)((u & 0xFFFFu) + ((u >> 16) & 0xFFFFu) + ((u >> 32) & 0xFFFFu) + (u >> 48));
  return (float)(s - 131070) * 0x1.1bc77ap-22f;  // 0.01 / 37837.227 to fp32
}

// The same entry as the raw bits stored in a table of the given dtype
// (fp32: 32 bits; fp16/bf16: 16 bits).
uint32_t orc_table_value_bits(uint64_t key, uint32_t mode, uint32_t dim, uint32_t dtype,
                              uint64_t r, uint32_t d) {
  uint32_t fb = float_to_bits(orc_table_value_f32(key, mode, dim, r, d));
  if (dtype == ORC_F16) return orc_f32_bits_to_f16_bits(fb);
  if (dtype == ORC_BF16) return orc_f32_bits_to_bf16_bits(fb);
  return fb;
}

// INT4 row format of this build (Section 4.1.2 gives no format): for a row x
// of `dim` fp32 values, lo = min x, hi = max x, scale = fp16_rne((hi-lo)/15),
// bias = fp16_rne(lo); code_d = clamp(rint((x_d - bias)/scale), 0, 15) with
// scale and bias taken AFTER their rounding to fp16 (scale 0 -> all codes 0);
// element d is the low (d even) or high (d odd) nibble of byte d/2; the two
// fp16 values follow the nibbles (scale first, little endian); zero padding
// to a multiple of 16 bytes. Decoded value = float(code) * scale + bias in
// fp32 with one fused rounding.
void orc_int4_quantize_row(const float* x, uint32_t dim, uint8_t* out) {
  uint64_t rb = orc_row_bytes(dim, ORC_INT4);
  std::memset(out, 0, rb);
  float lo = x[0], hi = x[0];
  for (uint32_t d = 1; d < dim; ++d) {
    lo = std::min(lo, x[d]);
    hi = std::max(hi, x[d]);
  }
  uint16_t sb = orc_f32_bits_to_f16_bits(float_to_bits((hi - lo) / 15.0f));
  uint16_t bb = orc_f32_bits_to_f16_bits(float_to_bits(lo));
  float scale = bits_to_float(orc_f16_bits_to_f32_bits(sb));
  float bias = bits_to_float(orc_f16_bits_to_f32_bits(bb));
  for (uint32_t d = 0; d < dim; ++d) {
    int code = 0;
    if (scale > 0.0f) {
      double q = std::nearbyint(((double)x[d] - (double)bias) / (double)scale);
      code = (int)std::min(15.0, std::max(0.0, q));
    }
    out[d / 2] |= (uint8_t)(code << ((d & 1u) * 4));
  }
  std::memcpy(out + dim / 2, &sb, 2);
  std::memcpy(out + dim / 2 + 2, &bb, 2);
}

// One stored row -> dim doubles (exact up-conversion; INT4: code*scale+bias
// evaluated in fp32 with a single rounding, i.e. fmaf).
static void decode_row(const orc_table_t* t, uint64_t r, double* dst) {
  const uint32_t D = t->dim;
  if (t->data == nullptr) {
    if (t->dtype == ORC_INT4) {
      std::vector<float> x(D);
      for (uint32_t d = 0; d < D; ++d) x[d] = orc_table_value_f32(t->value_key, t->value_mode, D, r, d);
      std::vector<uint8_t> q(orc_row_bytes(D, ORC_INT4));
      orc_int4_quantize_row(x.data(), D, q.data());
      orc_table_t tmp = *t;
      tmp.data = q.data();
      tmp.row_stride = 0;
      tmp.rows = 1;
      decode_row(&tmp, 0, dst);
      return;
    }
    for (uint32_t d = 0; d < D; ++d) {
      uint32_t b = orc_table_value_bits(t->value_key, t->value_mode, D, t->dtype, r, d);
      if (t->dtype == ORC_F16) b = orc_f16_bits_to_f32_bits((uint16_t)b);
      if (t->dtype == ORC_BF16) b = orc_bf16_bits_to_f32_bits((uint16_t)b);
      dst[d] = (double)bits_to_float(b);
    }
    return;
  }
  uint64_t stride = t->row_stride ? t->row_stride : orc_row_bytes(D, t->dtype);
  const uint8_t* p = (const uint8_t*)t->data + r * stride;
  if (t->dtype == ORC_F32) {
    for (uint32_t d = 0; d < D; ++d) {
      uint32_t b;
      std::memcpy(&b, p + 4ull * d, 4);
      dst[d] = (double)bits_to_float(b);
    }
  } else if (t->dtype == ORC_F16 || t->dtype == ORC_BF16) {
    for (uint32_t d = 0; d < D; ++d) {
      uint16_t h;
      std::memcpy(&h, p + 2ull * d, 2);
      uint32_t b = t->dtype == ORC_F16 ? orc_f16_bits_to_f32_bits(h) : orc_bf16_bits_to_f32_bits(h);
      dst[d] = (double)bits_to_float(b);
    }
  } else {  // ORC_INT4
    uint16_t sb, bb;
    std::memcpy(&sb, p + D / 2, 2);
    std::memcpy(&bb, p + D / 2 + 2, 2);
    float scale = bits_to_float(orc_f16_bits_to_f32_bits(sb));
    float bias = bits_to_float(orc_f16_bits_to_f32_bits(bb));
    for (uint32_t d = 0; d < D; ++d) {
      int code = (p[d / 2] >> ((d & 1u) * 4)) & 0xF;
      dst[d] = (double)std::fmaf((float)code, scale, bias);
    }
  }
}

// Materialise rows [r0, r1) of a procedural table into `dst` (dense rows).
void orc_table_fill(const orc_table_t* t, uint64_t r0, uint64_t r1, void* dst) {
  const uint32_t D = t->dim;
  uint64_t rb = orc_row_bytes(D, t->dtype);
  uint8_t* out = (uint8_t*)dst;
  std::vector<float> x(D);
  for (uint64_t r = r0; r < r1; ++r, out += rb) {
    if (t->dtype == ORC_INT4) {
      for (uint32_t d = 0; d < D; ++d) x[d] = orc_table_value_f32(t->value_key, t->value_mode, D, r, d);
      orc_int4_quantize_row(x.data(), D, out);
      continue;
    }
    for (uint32_t d = 0; d < D; ++d) {
      uint32_t b = orc_table_value_bits(t->value_key, t->value_mode, D, t->dtype, r, d);
      if (t->dtype == ORC_F32) std::memcpy(out + 4ull * d, &b, 4);
      else {
        uint16_t h = (uint16_t)b;
        std::memcpy(out + 2ull * d, &h, 2);
      }
    }
  }
}

// Decode one stored row to fp32 (exposed so tests can pin the decoders).
void orc_decode_row_f32(const orc_table_t* t, uint64_t r, float* dst) {
  std::vector<double> tmp(t->dim);
  decode_row(t, r, tmp.data());
  for (uint32_t d = 0; d < t->dim; ++d) dst[d] = (float)tmp[d];
}

// ------------------------------------------------------- embedding bag ------

// The whole path for samples [b0, b1): for every slot s (feature f =
// slot_feature[s], table t = table_ids[s], D = dim_t) and sample b, the bag is
// ids[offsets[f*B+b] .. offsets[f*B+b+1]); each ID is hashed to a row of table
// t, rows are summed (weighted by weights[i] for WSUM; divided by the bag
// length for MEAN) in double precision in input order, and the result is
// written as fp32 to out[b*out_ld + col_off_s + d], col_off_s being the sum of
// the dims of the slots before s (facets of a feature are adjacent slots, so
// their outputs are concatenated). An empty bag gives zeros. When
// ids_are_rows != 0 the IDs are taken as row indices and not hashed.
// Returns 0, or -1 on an invalid argument (bad pooling, row out of range,
// decreasing offsets, WSUM without weights).
int orc_embedding_bag(const orc_table_t* tables, int32_t n_tables, int32_t batch,
                      int32_t n_features, int32_t n_slots, const int32_t* slot_feature,
                      const int32_t* table_ids, const int32_t* pooling, int64_t out_ld,
                      int32_t ids_are_rows, const uint64_t* ids, const int64_t* offsets,
                      const float* weights, int32_t b0, int32_t b1, float* out) {
  int64_t total_dim = 0;
  for (int32_t s = 0; s < n_slots; ++s) {
    if (table_ids[s] < 0 || table_ids[s] >= n_tables) return -1;
    if (slot_feature[s] < 0 || slot_feature[s] >= n_features) return -1;
    total_dim += tables[table_ids[s]].dim;
  }
  if (out_ld == 0) out_ld = total_dim;
  if (out_ld < total_dim) return -1;
  std::vector<double> acc, row;
  int64_t col_off = 0;
  for (int32_t s = 0; s < n_slots; ++s) {
    const orc_table_t* t = &tables[table_ids[s]];
    const int32_t f = slot_feature[s];
    const uint32_t D = t->dim;
    const int32_t pool = pooling[s];
    if (pool != ORC_POOL_SUM && pool != ORC_POOL_MEAN && pool != ORC_POOL_WSUM) return -1;
    if (pool == ORC_POOL_WSUM && weights == nullptr) return -1;
    acc.assign(D, 0.0);
    row.assign(D, 0.0);
    for (int32_t b = b0; b < b1; ++b) {
      const int64_t lo = offsets[(int64_t)f * batch + b];
      const int64_t hi = offsets[(int64_t)f * batch + b + 1];
      if (hi < lo) return -1;
      std::fill(acc.begin(), acc.end(), 0.0);
      for (int64_t i = lo; i < hi; ++i) {
        uint64_t r = ids_are_rows ? ids[i] : (uint64_t)orc_hash_row(ids[i], t->hash_seed, t->rows);
        if (r >= t->rows) return -1;
        decode_row(t, r, row.data());
        const double w = pool == ORC_POOL_WSUM ? (double)weights[i] : 1.0;
        for (uint32_t d = 0; d < D; ++d) acc[d] += w * row[d];
      }
      if (pool == ORC_POOL_MEAN && hi > lo) {
        const double len = (double)(hi - lo);
        for (uint32_t d = 0; d < D; ++d) acc[d] /= len;
      }
      float* o = out + (int64_t)b * out_ld + col_off;
      for (uint32_t d = 0; d < D; ++d) o[d] = (float)acc[d];
    }
    col_off += D;
  }
  return 0;
}

// Gradient of the pooled output with respect to the table rows (the paper
// fine-tunes the pretrained tables inside the ranking model, Section 4.3):
// grad_table[r][d] += coef * grad_out[b][col_off + d] for every lookup of row
// r, coef = 1 (SUM), 1/len (MEAN) or weights[i] (WSUM). `grad_table` is a
// dense double [rows, dim] array for ONE slot `s`, accumulated in input order.
int orc_embedding_bag_backward_slot(const orc_table_t* tables, int32_t batch,
                                    const int32_t* slot_feature, const int32_t* table_ids,
                                    const int32_t* pooling, int32_t s, int64_t out_ld,
                                    int64_t col_off, int32_t ids_are_rows, const uint64_t* ids,
                                    const int64_t* offsets, const float* weights,
                                    const float* grad_out, double* grad_table) {
  const orc_table_t* t = &tables[table_ids[s]];
  const int32_t f = slot_feature[s];
  const uint32_t D = t->dim;
  const int32_t pool = pooling[s];
  for (int32_t b = 0; b < batch; ++b) {
    const int64_t lo = offsets[(int64_t)f * batch + b];
    const int64_t hi = offsets[(int64_t)f * batch + b + 1];
    for (int64_t i = lo; i < hi; ++i) {
      uint64_t r = ids_are_rows ? ids[i] : (uint64_t)orc_hash_row(ids[i], t->hash_seed, t->rows);
      if (r >= t->rows) return -1;
      double coef = 1.0;
      if (pool == ORC_POOL_MEAN) coef = 1.0 / (double)(hi - lo);
      if (pool == ORC_POOL_WSUM) coef = (double)weights[i];
      const float* g = grad_out + (int64_t)b * out_ld + col_off;
      for (uint32_t d = 0; d < D; ++d) grad_table[r * D + d] += coef * (double)g[d];
    }
  }
  return 0;
}

// ---------------------------------------------------------------- dedup -----

// In-batch dedup of hashed rows before host reads: uniq = ascending distinct
// values of rows[0..n); inverse[i] = position of rows[i] in uniq. Returns the
// number of distinct values.
int64_t orc_dedup(const int64_t* rows, int64_t n, int64_t* uniq, int32_t* inverse) {
  std::vector<int64_t> v(rows, rows + n);
  std::sort(v.begin(), v.end());
  v.erase(std::unique(v.begin(), v.end()), v.end());
  for (size_t j = 0; j < v.size(); ++j) uniq[j] = v[j];
  for (int64_t i = 0; i < n; ++i)
    inverse[i] = (int32_t)(std::lower_bound(v.begin(), v.end(), rows[i]) - v.begin());
  return (int64_t)v.size();
}

}  // extern "C"
