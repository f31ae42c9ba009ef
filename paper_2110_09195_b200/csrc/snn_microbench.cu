// Instruction-rate ceilings measured on the device that runs the kernels; they
// are the roofline denominators of the two integer-ALU paths.  Each kernel
// issues one instruction kind from 8 independent chains per thread, enough
// resident warps hiding the latency, and the host divides results by time.
#include "snn_tc_common.cuh"

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

// ---------------------------------------------------------------------------------------------
// Tensor-pipe ceiling as this library uses the tensor cores: one thread per SM issues a long run of
// tcgen05.mma (M = 128, both operands from shared memory in the K-major layout without swizzle, accumulator
// in tensor memory), alternating between two accumulators and walking through eight operand slices, and the
// cycles until the last one has completed are counted.  Operand contents do not matter (zeros).
//   FP4 = true : kind::mxf4, e2m1 operands with unit block scales, K = 64 per MMA
//   FP4 = false: kind::f16, fp16 operands, K = 16 per MMA
// ---------------------------------------------------------------------------------------------
constexpr int MMA_ITERS = 4096;

template <bool FP4>
__global__ void __launch_bounds__(128, 1) mma_rate_kernel(int N, long long* cycles, int* status) {
  extern __shared__ __align__(128) uint8_t smem[];
  __shared__ uint64_t bar;
  __shared__ uint32_t tslot;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t a_bytes = 8 * 4096, b_bytes = 8u * (uint32_t)N * 32u;   // eight K steps of A (128 rows) and of B (N rows)
  for (uint32_t i = tid; i < (a_bytes + b_bytes) / 16; i += 128) reinterpret_cast<uint4*>(smem)[i] = make_uint4(0, 0, 0, 0);
  if (tid == 0) mbar_init(smem_u32(&bar), 1);
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tslot)), "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  fence_proxy_async();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tb = tslot;
  if (FP4) tmem_fill32(tb + ((uint32_t)(warp * 32) << 16) + 480, 0x7f7f7f7fu);   // unit block scales
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) {
    const bool leader = elect_one();
    const uint64_t a0 = make_desc(smem_u32(smem), 128 * 16, 128);
    const uint64_t b0 = make_desc(smem_u32(smem + a_bytes), (uint32_t)N * 16, 128);
    const uint32_t idesc = FP4 ? ((1u << 7) | (1u << 10) | ((uint32_t)(N >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24))
                               : ((1u << 4) | ((uint32_t)(N >> 3) << 17) | ((128u >> 4) << 24));
    const int nacc = 2 * N <= (FP4 ? 480 : 512) ? 2 : 1;
    const long long t0 = clock64();
    for (int it = 0; it < MMA_ITERS; ++it) {
      if (leader) {
        const uint32_t d = tb + (uint32_t)((it & (nacc - 1)) * N);
        const uint64_t ad = a0 + (uint64_t)(((it >> 1) & 7) * 256);
        const uint64_t bd = b0 + (uint64_t)(((it >> 1) & 7) * (N * 2));
        if (FP4) mma_ss_fp4(d, ad, bd, idesc, it >= nacc ? 1u : 0u, tb + 480, tb + 496);
        else mma_ss_f16(d, ad, bd, idesc, it >= nacc ? 1u : 0u);
      }
    }
    if (leader) tc_commit(smem_u32(&bar));
    const bool ok = mbar_wait(smem_u32(&bar), 0);
    const long long t1 = clock64();
    if (lane == 0) {
      cycles[blockIdx.x] = t1 - t0;
      if (!ok) *status = 1;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tb), "r"(512) : "memory");
}

// results = multiply-accumulates per second over all SMs (measured cycles at the measured duration's clock)
template <bool FP4>
static cudaError_t run_mma_rate(int N, double* rate) {
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  long long* cyc = nullptr;
  int* status = nullptr;
  cudaError_t e = cudaMalloc(&cyc, sizeof(long long) * sms);
  if (e == cudaSuccess) e = cudaMalloc(&status, sizeof(int));
  if (e == cudaSuccess) e = cudaMemset(status, 0, sizeof(int));
  const size_t smem = 8 * 4096 + 8 * (size_t)N * 32;
  if (e == cudaSuccess) e = cudaFuncSetAttribute(mma_rate_kernel<FP4>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  float ms = 0.f;
  if (e == cudaSuccess) {
    mma_rate_kernel<FP4><<<sms, 128, smem>>>(N, cyc, status);   // warm-up
    cudaEventRecord(e0);
    mma_rate_kernel<FP4><<<sms, 128, smem>>>(N, cyc, status);
    cudaEventRecord(e1);
    e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) cudaEventElapsedTime(&ms, e0, e1);
  }
  int st = 0;
  if (e == cudaSuccess) e = cudaMemcpy(&st, status, sizeof(int), cudaMemcpyDeviceToHost);
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  cudaFree(cyc);
  cudaFree(status);
  if (e != cudaSuccess) return e;
  if (st || ms <= 0.f) return cudaErrorUnknown;   // a bounded wait ran out
  const double macs = (double)sms * MMA_ITERS * 128.0 * N * (FP4 ? 64.0 : 16.0);
  *rate = macs / (ms * 1e-3);
  return cudaGetLastError();
}

// Write-only stream: every thread writes 16 bytes per step, consecutive threads consecutive addresses, over a
// buffer far larger than L2; the best of several grid sizes.  Result: bytes per second.
__global__ void __launch_bounds__(256) store_stream_kernel(uint4* dst, size_t n16, uint32_t val) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  const uint4 v = make_uint4(val, val + 1, val + 2, val + 3);
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += stride) dst[i] = v;
}

static cudaError_t run_store_stream(double* rate) {
  const size_t bytes = (size_t)1 << 30;
  uint4* buf = nullptr;
  cudaError_t e = cudaMalloc(&buf, bytes);
  if (e != cudaSuccess) return e;
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  cudaEvent_t e0, e1;
  cudaEventCreate(&e0);
  cudaEventCreate(&e1);
  float best = 0.f;
  for (int mult : {1, 2, 4, 8, 16, 64}) {
    const int grid = sms * mult;
    store_stream_kernel<<<grid, 256>>>(buf, bytes / 16, 1u);   // warm-up
    for (int rep = 0; rep < 3; ++rep) {
      cudaEventRecord(e0);
      store_stream_kernel<<<grid, 256>>>(buf, bytes / 16, 2u + rep);
      cudaEventRecord(e1);
      e = cudaEventSynchronize(e1);
      if (e != cudaSuccess) break;
      float ms = 0.f;
      cudaEventElapsedTime(&ms, e0, e1);
      if (ms > 0.f && (best == 0.f || ms < best)) best = ms;
    }
    if (e != cudaSuccess) break;
  }
  cudaEventDestroy(e0);
  cudaEventDestroy(e1);
  cudaFree(buf);
  if (e != cudaSuccess) return e;
  if (best <= 0.f) return cudaErrorUnknown;
  *rate = (double)bytes / (best * 1e-3);
  return cudaGetLastError();
}

// Self-test of the bounded waits: one thread waits, with the helper every kernel of the library uses, on a
// barrier nothing ever arrives on.  The wait must give up after its attempt limit and raise the status word
// in mapped host memory, exactly as a convolution kernel would; the kernel then ends normally and the
// context stays usable.
__global__ void wait_selftest_kernel(int* status, long long* cycles) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const long long t0 = clock64();
    if (!mbar_wait(smem_u32(&bar), 0)) raise_status(status, 7);
    *cycles = clock64() - t0;
  }
}

// cudaErrorTimeout = the wait gave up and said so (the expected outcome); *rate = seconds the kernel took
cudaError_t run_wait_selftest(double* rate) {
  int* status_host = nullptr;
  int* status_dev = nullptr;
  long long* cycles = nullptr;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaHostAlloc((void**)&status_host, sizeof(int), cudaHostAllocMapped);
  if (e == cudaSuccess) {
    *status_host = 0;
    e = cudaHostGetDevicePointer((void**)&status_dev, status_host, 0);
  }
  if (e == cudaSuccess) e = cudaMalloc((void**)&cycles, sizeof(long long));
  if (e == cudaSuccess) e = cudaEventCreate(&e0);
  if (e == cudaSuccess) e = cudaEventCreate(&e1);
  float ms = 0.f;
  if (e == cudaSuccess) {
    cudaEventRecord(e0);
    wait_selftest_kernel<<<1, 32>>>(status_dev, cycles);
    cudaEventRecord(e1);
    e = cudaEventSynchronize(e1);
    if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
  }
  const int code = status_host ? *status_host : 0;
  if (e0) cudaEventDestroy(e0);
  if (e1) cudaEventDestroy(e1);
  if (cycles) cudaFree(cycles);
  if (status_host) cudaFreeHost(status_host);
  if (e != cudaSuccess) return e;
  *rate = (double)ms * 1e-3;
  return code == 7 ? cudaErrorTimeout : cudaSuccess;
}

cudaError_t microbench(int kind, double* rate) {
  switch (kind) {
    case 9: return run_wait_selftest(rate);
    case 5: return run_mma_rate<true>(240, rate);
    case 6: return run_store_stream(rate);
    case 7: return run_mma_rate<false>(256, rate);
    case 8: return run_mma_rate<true>(128, rate);
    case 0: return run_kind<0>(rate);
    case 1: return run_kind<1>(rate);
    case 2: return run_kind<2>(rate);
    case 3: return run_kind<3>(rate);
    default: return run_kind<4>(rate);
  }
}

}  // namespace snn
