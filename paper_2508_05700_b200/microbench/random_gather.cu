// Microbenchmark: achievable random 128-byte row gather bandwidth on this GPU.
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <vector>
#include <cstdlib>
#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); exit(1);} } while (0)
template <int U, int ROWB>
__global__ void gather(const uint8_t* __restrict__ table, const uint32_t* __restrict__ rows, int64_t n, uint32_t* out) {
  constexpr int LPR = ROWB / 16, RPW = 32 / LPR;
  const int lane = threadIdx.x & 31, c = lane % LPR, sub = lane / LPR;
  int64_t warp = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
  uint32_t acc = 0;
  for (int64_t base = warp * (RPW * U); base < n; base += nwarps * (RPW * U)) {
    uint4 v[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      int64_t i = base + k * RPW + sub;
      uint32_t r = i < n ? __ldg(rows + i) : 0;
      const uint4* p = reinterpret_cast<const uint4*>(table + (uint64_t)r * ROWB + c * 16);
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(p));
    }
#pragma unroll
    for (int k = 0; k < U; ++k) acc ^= v[k].x ^ v[k].y ^ v[k].z ^ v[k].w;
  }
  if (acc == 0x12345678u) out[0] = acc;
}
template <int U, int ROWB>
void run(const uint8_t* table, const uint32_t* rows, int64_t n, uint32_t* out, int blocks_per_sm, int threads) {
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  int grid = 148 * blocks_per_sm;
  for (int i = 0; i < 3; ++i) gather<U, ROWB><<<grid, threads>>>(table, rows, n, out);
  CK(cudaDeviceSynchronize());
  cudaEventRecord(e0);
  for (int i = 0; i < 10; ++i) gather<U, ROWB><<<grid, threads>>>(table, rows, n, out);
  cudaEventRecord(e1); CK(cudaDeviceSynchronize());
  float ms; cudaEventElapsedTime(&ms, e0, e1); ms /= 10;
  printf("rowB=%d U=%d blocks/SM=%d threads=%d warps/SM=%d : %.1f us  %.0f GB/s\n", ROWB, U, blocks_per_sm, threads, blocks_per_sm * threads / 32, ms * 1e3, n * (double)ROWB / ms / 1e6);
}
int main(int argc, char** argv) {
  // table size in MiB (default 40 GiB: no L2 reuse; 64 MiB: every row read hits the 126 MB L2)
  const uint64_t table_bytes = (argc > 1 ? (uint64_t)atoll(argv[1]) : 40960ull) << 20;
  const int64_t n = 16 << 20;  // rows gathered per launch (2 GiB at 128 B)
  uint8_t* table; uint32_t* rows; uint32_t* out;
  CK(cudaMalloc(&table, table_bytes)); CK(cudaMemset(table, 1, table_bytes));
  CK(cudaMalloc(&rows, n * 4)); CK(cudaMalloc(&out, 4));
  std::vector<uint32_t> h(n);
  uint64_t s = 88172645463325252ull;
  for (int64_t i = 0; i < n; ++i) { s ^= s << 13; s ^= s >> 7; s ^= s << 17; h[i] = (uint32_t)(s % (table_bytes / 256)); }
  CK(cudaMemcpy(rows, h.data(), n * 4, cudaMemcpyHostToDevice));
  for (int bps : {2, 4, 6, 8}) {
    run<1, 128>(table, rows, n, out, bps, 256);
    run<2, 128>(table, rows, n, out, bps, 256);
    run<4, 128>(table, rows, n, out, bps, 256);
    run<8, 128>(table, rows, n, out, bps, 256);
  }
  run<4, 64>(table, rows, n, out, 8, 256);
  run<8, 64>(table, rows, n, out, 8, 256);
  run<4, 256>(table, rows, n, out, 8, 256);
  run<8, 256>(table, rows, n, out, 8, 256);
  return 0;
}
