// Microbenchmark: zero-copy reads of random 128-byte rows from pinned host memory.
#include <cuda_runtime.h>
#include <cstdio>
#include <cstdint>
#include <vector>
#include <cstdlib>
#define CK(x) do { cudaError_t e = (x); if (e != cudaSuccess) { printf("err %s line %d\n", cudaGetErrorString(e), __LINE__); exit(1);} } while (0)
enum { NC16 = 0, PLAIN16 = 1, VOL16 = 2, W4 = 3, W8 = 4 };
template <int MODE, int U>
__global__ void fetch(const uint8_t* __restrict__ table, const int64_t* __restrict__ rows, int64_t n, uint8_t* __restrict__ dst) {
  constexpr int BPL = MODE == W4 ? 4 : (MODE == W8 ? 8 : 16);   // bytes per lane
  constexpr int CH = 128 / BPL;                                  // lanes per row
  const int64_t total = n * CH;
  const int64_t step = (int64_t)gridDim.x * blockDim.x;
  for (int64_t q0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; q0 < total; q0 += step * U) {
    uint4 v[U];
#pragma unroll
    for (int k = 0; k < U; ++k) {
      int64_t q = q0 + k * step;
      if (q < total) {
        int64_t m = q / CH; int c = (int)(q % CH);
        const uint8_t* p = table + (uint64_t)rows[m] * 128 + c * BPL;
        if (MODE == NC16) asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(p));
        else if (MODE == PLAIN16) v[k] = *reinterpret_cast<const uint4*>(p);
        else if (MODE == VOL16) asm volatile("ld.volatile.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v[k].x), "=r"(v[k].y), "=r"(v[k].z), "=r"(v[k].w) : "l"(p));
        else if (MODE == W4) v[k].x = *reinterpret_cast<const uint32_t*>(p);
        else { uint2 t = *reinterpret_cast<const uint2*>(p); v[k].x = t.x; v[k].y = t.y; }
      }
    }
#pragma unroll
    for (int k = 0; k < U; ++k) {
      int64_t q = q0 + k * step;
      if (q < total) {
        if (BPL == 16) *reinterpret_cast<uint4*>(dst + q * 16) = v[k];
        else if (BPL == 8) *reinterpret_cast<uint2*>(dst + q * 8) = make_uint2(v[k].x, v[k].y);
        else *reinterpret_cast<uint32_t*>(dst + q * 4) = v[k].x;
      }
    }
  }
}
// one bulk async copy (TMA) per row, straight into HBM is not possible (bulk copies go global<->shared):
// rows land in shared memory, then are written out with vector stores.
__global__ void fetch_bulk(const uint8_t* __restrict__ table, const int64_t* __restrict__ rows, int64_t n, uint8_t* __restrict__ dst, int* err) {
  extern __shared__ __align__(128) uint8_t sm[];
  const int RPB = blockDim.x;  // rows per block round (one per thread)
  uint64_t* barp = reinterpret_cast<uint64_t*>(sm + (size_t)RPB * 128);
  uint32_t bar = (uint32_t)__cvta_generic_to_shared(barp), base = (uint32_t)__cvta_generic_to_shared(sm);
  if (threadIdx.x == 0) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(1)); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  __syncthreads();
  uint32_t parity = 0;
  for (int64_t r0 = (int64_t)blockIdx.x * RPB; r0 < n; r0 += (int64_t)gridDim.x * RPB) {
    int cnt = (int)min((int64_t)RPB, n - r0);
    if (threadIdx.x == 0) asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(cnt * 128) : "memory");
    if ((int)threadIdx.x < cnt)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(base + threadIdx.x * 128), "l"(table + (uint64_t)rows[r0 + threadIdx.x] * 128), "r"(128), "r"(bar) : "memory");
    uint32_t ok = 0; int tries = 0;
    while (!ok && tries++ < (1 << 22))
      asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.b32 %0, 1, 0, p; }" : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    if (!ok) { *err = 1; return; }
    parity ^= 1;
    for (int q = threadIdx.x; q < cnt * 8; q += blockDim.x)
      *reinterpret_cast<uint4*>(dst + (r0 * 8 + q) * 16) = *reinterpret_cast<const uint4*>(sm + q * 16);
    __syncthreads();
  }
}
template <int MODE, int U>
void run(const char* name, const uint8_t* table, const int64_t* rows, int64_t n, uint8_t* dst, int blocks) {
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  for (int i = 0; i < 2; ++i) fetch<MODE, U><<<blocks, 256>>>(table, rows, n, dst);
  CK(cudaDeviceSynchronize());
  cudaEventRecord(e0);
  for (int i = 0; i < 5; ++i) fetch<MODE, U><<<blocks, 256>>>(table, rows, n, dst);
  cudaEventRecord(e1); CK(cudaDeviceSynchronize());
  float ms; cudaEventElapsedTime(&ms, e0, e1); ms /= 5;
  printf("%-8s U=%d blocks=%5d n=%8lld : %9.1f us  %6.2f GB/s\n", name, U, blocks, (long long)n, ms * 1e3, n * 128.0 / ms / 1e6);
}
int main() {
  const uint64_t host_bytes = 8ull << 30;
  uint8_t* host; CK(cudaHostAlloc((void**)&host, host_bytes, cudaHostAllocMapped));
  for (uint64_t i = 0; i < host_bytes; i += 4096) host[i] = (uint8_t)i;
  uint8_t* dtab; CK(cudaHostGetDevicePointer((void**)&dtab, host, 0));
  const int64_t nmax = 4 << 20;
  std::vector<int64_t> h(nmax), hseq(nmax);
  uint64_t s = 88172645463325252ull;
  for (int64_t i = 0; i < nmax; ++i) { s ^= s << 13; s ^= s >> 7; s ^= s << 17; h[i] = (int64_t)(s % (host_bytes / 128)); hseq[i] = i; }
  int64_t *rows, *rseq; uint8_t* dst; int* err;
  CK(cudaMalloc(&rows, nmax * 8)); CK(cudaMalloc(&rseq, nmax * 8)); CK(cudaMalloc(&dst, nmax * 128)); CK(cudaMalloc(&err, 4)); CK(cudaMemset(err, 0, 4));
  CK(cudaMemcpy(rows, h.data(), nmax * 8, cudaMemcpyHostToDevice)); CK(cudaMemcpy(rseq, hseq.data(), nmax * 8, cudaMemcpyHostToDevice));
  // DMA reference
  { cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1); uint8_t* big; CK(cudaMalloc(&big, 1ull << 30));
    CK(cudaMemcpy(big, host, 1ull << 30, cudaMemcpyHostToDevice));
    cudaEventRecord(e0); for (int i = 0; i < 5; ++i) cudaMemcpyAsync(big, host, 1ull << 30, cudaMemcpyHostToDevice); cudaEventRecord(e1); CK(cudaDeviceSynchronize());
    float ms; cudaEventElapsedTime(&ms, e0, e1); printf("cudaMemcpyAsync H2D 1 GiB: %.2f GB/s\n", 5 * 1.0737 / (ms / 1e3)); cudaFree(big); }
  for (int64_t n : {(int64_t)57000, (int64_t)(1 << 20)}) {
    for (int blocks : {148, 592, 2368}) {
      run<NC16, 4>("nc16", dtab, rows, n, dst, blocks);
      run<PLAIN16, 4>("plain16", dtab, rows, n, dst, blocks);
    }
    run<NC16, 1>("nc16", dtab, rows, n, dst, 2368);
    run<NC16, 8>("nc16", dtab, rows, n, dst, 592);
    run<VOL16, 4>("vol16", dtab, rows, n, dst, 592);
    run<W4, 4>("w4", dtab, rows, n, dst, 592);
    run<W8, 4>("w8", dtab, rows, n, dst, 592);
    run<NC16, 4>("seq-nc16", dtab, rseq, n, dst, 592);
    for (int blocks : {148, 592}) for (int threads : {128, 256}) {
      cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
      size_t sm = (size_t)threads * 128 + 64;
      fetch_bulk<<<blocks, threads, sm>>>(dtab, rows, n, dst, err); CK(cudaDeviceSynchronize());
      cudaEventRecord(e0); for (int i = 0; i < 5; ++i) fetch_bulk<<<blocks, threads, sm>>>(dtab, rows, n, dst, err); cudaEventRecord(e1); CK(cudaDeviceSynchronize());
      float ms; cudaEventElapsedTime(&ms, e0, e1); ms /= 5; int herr; cudaMemcpy(&herr, err, 4, cudaMemcpyDeviceToHost);
      printf("bulk128  blocks=%5d threads=%d n=%8lld : %9.1f us  %6.2f GB/s err=%d\n", blocks, threads, (long long)n, ms * 1e3, n * 128.0 / ms / 1e6, herr);
    }
  }
  return 0;
}
