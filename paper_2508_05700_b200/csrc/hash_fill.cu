// K-hash: raw IDs -> table rows.  K-fill: synthetic table contents.
#include "common.cuh"

namespace mfet {

// rows_out[i] = splitmix64(ids[i] ^ seed) mod rows. One ID per thread,
// grid-stride; 8-byte coalesced loads and stores, streaming hints (each value is
// touched once).
__global__ void __launch_bounds__(256) hash_kernel(const uint64_t* __restrict__ ids, int64_t n,
                                                   uint64_t seed, uint64_t rows, uint64_t magic,
                                                   int64_t* __restrict__ rows_out) {
  int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (; i < n; i += step) {
    uint64_t id = __ldcs(reinterpret_cast<const unsigned long long*>(ids) + i);
    uint64_t r = mod_rows(splitmix64(id ^ seed), rows, magic);
    __stcs(reinterpret_cast<long long*>(rows_out) + i, (long long)r);
  }
}

cudaError_t launch_hash(const uint64_t* ids, int64_t n, uint64_t seed, uint64_t rows, uint64_t magic,
                        int64_t* rows_out, cudaStream_t s) {
  if (n == 0) return cudaSuccess;
  int64_t blocks = (n + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  hash_kernel<<<(unsigned)blocks, 256, 0, s>>>(ids, n, seed, rows, magic, rows_out);
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

cudaError_t launch_fill(void* data, uint64_t row0, uint64_t n_rows, uint32_t dim, uint32_t dtype,
                        uint64_t stride, uint64_t key, uint32_t mode, cudaStream_t s) {
  if (n_rows == 0) return cudaSuccess;
  const uint32_t chunks = (uint32_t)(mfet_row_bytes(dim, dtype) / 16);
  uint64_t total = n_rows * chunks;
  uint64_t blocks = (total + 255) / 256;
  if (blocks > 148ull * 32) blocks = 148ull * 32;
  fill_kernel<<<(unsigned)blocks, 256, 0, s>>>((uint8_t*)data, row0, n_rows, dim, dtype, stride, key,
                                               mode, chunks);
  return cudaGetLastError();
}

}  // namespace mfet
