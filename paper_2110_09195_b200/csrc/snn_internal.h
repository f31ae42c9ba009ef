// Internal declarations shared by the translation units of libsnnconv.
// Nothing here is part of the public ABI (see include/snn_conv.h).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "snn_conv.h"

namespace snn {

// Geometry of one forward call.
struct Geom {
  int N, H, W;        // input batch and map
  int C, K, Cw;       // channels in / out, ceil(C/32)
  int stride, pad;
  int Ho, Wo;         // output map
  int tau, T;         // index width, codebook size 2^tau
  int ksize;          // 3, or 1 for the 1x1 extension (8-input-channel vectors, pad 0)
};

// Device-resident layer data derived at create time (Sec. 4.4 storage -> compute form).
struct LayerDev {
  uint16_t* idx = nullptr;       // [K][C] unpacked 0-based indices
  uint16_t* codebook = nullptr;  // [T] 9-bit codes
  float* alpha = nullptr;        // [K]
  float* shift = nullptr;        // [K] added to alpha*S before the sign is taken (packed-sign output), zeros if none
  uint32_t* wplanes = nullptr;   // [9][Cw][K] bit-planes of the decoded +/-1 weights (bit = +1)
  int32_t* corr = nullptr;       // [16][K] border corrections, see snn_decode.cu
  uint8_t* match9 = nullptr;     // [T/16 or 1][512][16] matching-tap counts per (window, codebook kernel)
};

struct Launch {
  const void* act;
  void* out;
  int out_i32;   // 0: write fp32 alpha*S, 1: write int32 S, 2: packed signs of alpha*S (tensor-core path only)
  cudaStream_t stream;
};

// Each returns cudaSuccess / an error from the launch; *launched += kernels launched.
// `supported` variants return false when the path cannot run the shape.
cudaError_t decode_layer(const LayerDev& L, const uint8_t* idx_packed_dev, const Geom& g, int act_type,
                         cudaStream_t s, int* launched);

bool popc_supported(const Geom& g, int act_type);
cudaError_t popc_forward(const LayerDev& L, const Geom& g, const Launch& l, int* launched);

bool reuse_supported(const Geom& g, int act_type);
cudaError_t reuse_forward(const LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched);
// the same sharing with fp16 activations (snn_reuse_f16.cu); reuse_supported / reuse_forward dispatch to these
bool reuse_f16_supported(const Geom& g);
cudaError_t reuse_f16_forward(const LayerDev& L, const Geom& g, const Launch& l, int* launched);

// The tensor-core kernel (snn_tcg.cu) runs one layer, several independent layers, or a chain of dependent
// layers as ONE persistent launch; a single layer is a group of one.
// Several independent problems in one persistent tensor-core launch (snn_tcg.cu).
struct GroupDev;
// What a launch is planned for: the tile shapes and the number of accumulator buffers differ between the kinds.
//   TCG_WORDS  independent problems, fp32 / int32 outputs
//   TCG_CHAIN  member i + 1 reads the packed signs member i writes (binary activations; the members' shapes must
//              follow from one another); tcg_forward then takes the first member's input in act[0] and the last
//              member's output in out[0], and out_type is the last member's
//   TCG_SIGNS  independent problems, packed-sign outputs (binary activations)
// tcg_forward refuses an output type the plan was not made for.
enum { TCG_WORDS = 0, TCG_CHAIN = 1, TCG_SIGNS = 2 };
cudaError_t tcg_create(const LayerDev* const* layers, const Geom* geoms, int count, int act_type, int kind,
                       cudaStream_t s, GroupDev** out, int* launched);
cudaError_t tcg_forward(GroupDev* G, const void* const* act, void* const* out, int out_type, cudaStream_t s,
                        int* status_dev, int* launched);
void tcg_destroy(GroupDev* G);
int tcg_count(const GroupDev* G);
bool tcg_supported(const Geom& g, int act_type);   // can the tensor-core kernel run this layer at this shape?

cudaError_t microbench(int kind, double* rate);

// Largest dynamic shared memory a CTA may ask for on sm_100 (227 KB).
constexpr int kMaxDynSmem = 227 * 1024;

// Raises a kernel's dynamic shared-memory limit (and the shared-memory carve-out) to the maximum, once per device.
template <typename Kernel>
inline cudaError_t allow_max_smem(Kernel kernel, unsigned long long* done_mask) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  const unsigned long long bit = 1ull << (dev & 63);
  if (__atomic_load_n(done_mask, __ATOMIC_ACQUIRE) & bit) return cudaSuccess;
  e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem);
  // all of the SM's memory as shared memory, so that two CTAs of half its size fit side by side
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared);
  if (e == cudaSuccess) __atomic_fetch_or(done_mask, bit, __ATOMIC_RELEASE);
  return e;
}

}  // namespace snn
