// K-hash: raw IDs -> table rows.  K-fill: synthetic table contents.
#include "common.cuh"

namespace mfet {

// rows_out[i] = splitmix64(ids[i] ^ seed) mod rows, grid-stride, streaming hints (each value
// is touched once). PAIRS: a thread takes two neighbouring IDs with one 16-byte load and one
// 16-byte store, two such pairs in flight (the arrays must be 16-byte aligned; an odd last ID
// is left to the first thread). Otherwise one ID per thread and 8-byte accesses.
template <bool PAIRS>
__global__ void __launch_bounds__(256) hash_kernel(const uint64_t* __restrict__ ids, int64_t n,
                                                   uint64_t seed, uint64_t rows, uint64_t magic,
                                                   int64_t* __restrict__ rows_out) {
  const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  if constexpr (PAIRS) {
    const int64_t np = n >> 1;
    const ulonglong2* in2 = reinterpret_cast<const ulonglong2*>(ids);
    longlong2* out2 = reinterpret_cast<longlong2*>(rows_out);
    int64_t i = first;
    for (; i + step < np; i += 2 * step) {
      const ulonglong2 a = __ldcs(in2 + i), b = __ldcs(in2 + i + step);
      longlong2 ra, rb;
      ra.x = (long long)mod_rows(splitmix64(a.x ^ seed), rows, magic);
      ra.y = (long long)mod_rows(splitmix64(a.y ^ seed), rows, magic);
      rb.x = (long long)mod_rows(splitmix64(b.x ^ seed), rows, magic);
      rb.y = (long long)mod_rows(splitmix64(b.y ^ seed), rows, magic);
      __stcs(out2 + i, ra);
      __stcs(out2 + i + step, rb);
    }
    if (i < np) {
      const ulonglong2 a = __ldcs(in2 + i);
      longlong2 ra;
      ra.x = (long long)mod_rows(splitmix64(a.x ^ seed), rows, magic);
      ra.y = (long long)mod_rows(splitmix64(a.y ^ seed), rows, magic);
      __stcs(out2 + i, ra);
    }
    if ((n & 1) && first == 0)
      rows_out[n - 1] = (int64_t)mod_rows(splitmix64(ids[n - 1] ^ seed), rows, magic);
  } else {
    for (int64_t i = first; i < n; i += step) {
      uint64_t id = __ldcs(reinterpret_cast<const unsigned long long*>(ids) + i);
      uint64_t r = mod_rows(splitmix64(id ^ seed), rows, magic);
      __stcs(reinterpret_cast<long long*>(rows_out) + i, (long long)r);
    }
  }
}

cudaError_t launch_hash(const uint64_t* ids, int64_t n, uint64_t seed, uint64_t rows, uint64_t magic,
                        int64_t* rows_out, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  const bool pairs = n >= 2 && ((reinterpret_cast<uintptr_t>(ids) | reinterpret_cast<uintptr_t>(rows_out)) & 15u) == 0;
  const int64_t items = pairs ? (n >> 1) : n;
  int64_t blocks = (items + 255) / 256;
  if (blocks > sm_count() * 8) blocks = sm_count() * 8;
  if (pairs) hash_kernel<true><<<(unsigned)blocks, 256, 0, s>>>(ids, n, seed, rows, magic, rows_out);
  else hash_kernel<false><<<(unsigned)blocks, 256, 0, s>>>(ids, n, seed, rows, magic, rows_out);
  return cudaGetLastError();
}

// Synthetic table value before rounding to the table's dtype.
__device__ __forceinline__ float table_value(uint64_t key, uint32_t mode, uint64_t k) {
  uint64_t u = splitmix64(key + k);
  if (mode == MFET_VAL_GRID) return __int2float_rn((int)(u & 0xFFu) - 128) * 0x1p-13f;
  int s = (int)((u & 0xFFFFu) + ((u >> 16) & 0xFFFFu) + ((u >> 32) & 0xFFFFu) + (u >> 48));
  return __fmul_rn(__int2float_rn(s - 131070), 0x1.1bc77ap-22f);
}

// One thread writes one 16-byte chunk of a row (4 fp32 or 8 fp16/bf16 values),
// so that stores are 16-byte vectors, coalesced along the row.
__global__ void __launch_bounds__(256) fill_kernel(uint8_t* __restrict__ data, uint64_t row0,
                                                   uint64_t n_rows, uint32_t dim, uint32_t dtype,
                                                   uint64_t stride, uint64_t key, uint32_t mode,
                                                   uint32_t chunks) {
  const uint64_t total = n_rows * chunks;
  uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const uint64_t step = (uint64_t)gridDim.x * blockDim.x;
  for (; i < total; i += step) {
    const uint64_t r = row0 + i / chunks;
    const uint32_t c = (uint32_t)(i % chunks);
    uint4 v;
    if (dtype == MFET_F32) {
      const uint64_t k = r * dim + c * 4u;
      v.x = __float_as_uint(table_value(key, mode, k + 0));
      v.y = __float_as_uint(table_value(key, mode, k + 1));
      v.z = __float_as_uint(table_value(key, mode, k + 2));
      v.w = __float_as_uint(table_value(key, mode, k + 3));
    } else {
      const uint64_t k = r * dim + c * 8u;
      uint32_t w[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        float a = table_value(key, mode, k + 2 * j), b = table_value(key, mode, k + 2 * j + 1);
        uint32_t lo, hi;
        if (dtype == MFET_F16) {
          lo = __half_as_ushort(__float2half_rn(a));
          hi = __half_as_ushort(__float2half_rn(b));
        } else {
          lo = __bfloat16_as_ushort(__float2bfloat16_rn(a));
          hi = __bfloat16_as_ushort(__float2bfloat16_rn(b));
        }
        w[j] = lo | (hi << 16);
      }
      v = make_uint4(w[0], w[1], w[2], w[3]);
    }
    *reinterpret_cast<uint4*>(data + r * stride + (uint64_t)c * 16u) = v;
  }
}

// INT4 rows (one thread per row; not a hot kernel): the row's fp32 values are generated,
// scale = fp16((max-min)/15) and bias = fp16(min) are fixed, every value becomes the code
// clamp(rint((x - bias) / scale), 0, 15) - the quotient in double precision, so that every
// implementation of this definition rounds the same way -, two codes per byte, low nibble
// first, then scale and bias, then zero padding up to a multiple of 16 bytes.
__global__ void __launch_bounds__(128) fill_int4_kernel(uint8_t* __restrict__ data, uint64_t row0, uint64_t n_rows,
                                                        uint32_t dim, uint64_t stride, uint64_t row_bytes,
                                                        uint64_t key, uint32_t mode) {
  const uint64_t i = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_rows) return;
  const uint64_t r = row0 + i;
  float lo = table_value(key, mode, r * dim), hi = lo;
  for (uint32_t d = 1; d < dim; ++d) {
    const float x = table_value(key, mode, r * dim + d);
    lo = fminf(lo, x);
    hi = fmaxf(hi, x);
  }
  const __half sh = __float2half_rn(__fdiv_rn(__fsub_rn(hi, lo), 15.0f)), bh = __float2half_rn(lo);
  const double scale = (double)__half2float(sh), bias = (double)__half2float(bh);
  uint8_t* row = data + r * stride;
  for (uint32_t d = 0; d < dim; d += 8) {
    uint32_t word = 0;
    for (uint32_t j = 0; j < 8; ++j) {
      int code = 0;
      if (scale > 0.0) {
        const double q = rint(((double)table_value(key, mode, r * dim + d + j) - bias) / scale);
        code = (int)fmin(15.0, fmax(0.0, q));
      }
      word |= (uint32_t)code << (4 * j);
    }
    *reinterpret_cast<uint32_t*>(row + d / 2) = word;
  }
  *reinterpret_cast<uint32_t*>(row + dim / 2) = (uint32_t)__half_as_ushort(sh) | ((uint32_t)__half_as_ushort(bh) << 16);
  for (uint64_t b = dim / 2 + 4; b < row_bytes; b += 4) *reinterpret_cast<uint32_t*>(row + b) = 0u;
}

cudaError_t launch_fill(void* data, uint64_t row0, uint64_t n_rows, uint32_t dim, uint32_t dtype,
                        uint64_t stride, uint64_t key, uint32_t mode, cudaStream_t s) {
  if (n_rows == 0) return cudaSuccess;
  if (dtype == MFET_INT4) {
    const uint64_t blocks = (n_rows + 127) / 128;
    if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidValue;
    fill_int4_kernel<<<(unsigned)blocks, 128, 0, s>>>((uint8_t*)data, row0, n_rows, dim, stride,
                                                      mfet_row_bytes(dim, dtype), key, mode);
    return cudaGetLastError();
  }
  const uint32_t chunks = (uint32_t)(mfet_row_bytes(dim, dtype) / 16);
  uint64_t total = n_rows * chunks;
  uint64_t blocks = (total + 255) / 256;
  if (blocks > (uint64_t)sm_count() * 32) blocks = (uint64_t)sm_count() * 32;
  fill_kernel<<<(unsigned)blocks, 256, 0, s>>>((uint8_t*)data, row0, n_rows, dim, dtype, stride, key,
                                               mode, chunks);
  return cudaGetLastError();
}

}  // namespace mfet
