// Instruction-rate ceilings measured on the device that runs the kernels; they
// are the roofline denominators of the two integer-ALU paths.  Each kernel
// issues one instruction kind from 8 independent chains per thread, enough
// resident warps hiding the latency, and the host divides results by time.
#include "snn_internal.h"

namespace snn {

constexpr int MB_ITERS = 2048;
constexpr int MB_CHAINS = 8;

template <int KIND>
__global__ void __launch_bounds__(256) microbench_kernel(uint32_t* sink, uint32_t seed) {
  __shared__ uint32_t ring[256 * MB_CHAINS];
  uint32_t v[MB_CHAINS];
#pragma unroll
  for (int c = 0; c < MB_CHAINS; ++c) v[c] = seed * (threadIdx.x + 1) + c * 0x9e3779b9u;
  uint32_t k1 = seed | 1u, k2 = ~seed;
  if (KIND == 3) {
    // every slot points at itself: a dependent, conflict-free load chain
#pragma unroll
    for (int c = 0; c < MB_CHAINS; ++c) {
      uint32_t slot = c * 256 + threadIdx.x;
      uint32_t addr = (uint32_t)__cvta_generic_to_shared(&ring[slot]);
      ring[slot] = addr;
      v[c] = addr;
    }
    __syncthreads();
  }
  for (int it = 0; it < MB_ITERS; ++it) {
#pragma unroll
    for (int c = 0; c < MB_CHAINS; ++c) {
      if (KIND == 0) asm volatile("popc.b32 %0, %0;" : "+r"(v[c]));
      if (KIND == 1) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(v[c]) : "r"(k1), "r"(k2));
      if (KIND == 2) asm volatile("add.u32 %0, %0, %1;" : "+r"(v[c]) : "r"(k1));
      if (KIND == 3) asm volatile("ld.shared.u32 %0, [%0];" : "+r"(v[c]));
      if (KIND == 4) {
        uint32_t x, pc;
        asm volatile("xor.b32 %0, %1, %2;" : "=r"(x) : "r"(v[c]), "r"(k2));
        asm volatile("popc.b32 %0, %1;" : "=r"(pc) : "r"(x));
        asm volatile("add.u32 %0, %0, %1;" : "+r"(v[c]) : "r"(pc));
      }
    }
  }
  uint32_t r = 0;
#pragma unroll
  for (int c = 0; c < MB_CHAINS; ++c) r ^= v[c];
  if (r == 0x12345u) sink[0] = r;  // keeps the chains alive; practically never taken
}

template <int KIND>
static cudaError_t run_kind(double* rate) {
  uint32_t* sink = nullptr;
  cudaError_t e = cudaMalloc(&sink, 64);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int blocks = sms * 8;
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  microbench_kernel<KIND><<<blocks, 256>>>(sink, 12345u);  // warm-up
  const int reps = 3;
  cudaEventRecord(e0);
  for (int r = 0; r < reps; ++r) microbench_kernel<KIND><<<blocks, 256>>>(sink, 777u + r);
  cudaEventRecord(e1);
  e = cudaEventSynchronize(e1);
  float ms = 0.f;
  cudaEventElapsedTime(&ms, e0, e1);
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(sink);
  if (e != cudaSuccess) return e;
  double results = (double)reps * blocks * 256.0 * MB_ITERS * MB_CHAINS;
  *rate = results / (ms * 1e-3);
  return cudaGetLastError();
}

cudaError_t microbench(int kind, double* rate) {
  switch (kind) {
    case 0: return run_kind<0>(rate);
    case 1: return run_kind<1>(rate);
    case 2: return run_kind<2>(rate);
    case 3: return run_kind<3>(rate);
    default: return run_kind<4>(rate);
  }
}

}  // namespace snn
