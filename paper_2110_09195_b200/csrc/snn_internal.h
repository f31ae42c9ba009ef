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
};

// Device-resident layer data derived at create time (Sec. 4.4 storage -> compute form).
struct LayerDev {
  uint16_t* idx = nullptr;       // [K][C] unpacked 0-based indices
  uint16_t* codebook = nullptr;  // [T] 9-bit codes
  float* alpha = nullptr;        // [K]
  uint32_t* wplanes = nullptr;   // [9][Cw][K] bit-planes of the decoded +/-1 weights (bit = +1)
  int32_t* corr = nullptr;       // [16][K] border corrections, see snn_decode.cu
  uint8_t* match9 = nullptr;     // [T/16 or 1][512][16] matching-tap counts per (window, codebook kernel)
  int8_t* w8 = nullptr;          // tensor-core operand: +/-1 int8 weights, tiled (snn_tc.cu)
  uint16_t* w16 = nullptr;       // tensor-core operand: +/-1 fp16 weights, tiled (fp16 activations)
  void* wcm = nullptr;           // channel-major tensor-core operand, [channel tile][K step][half][128][16 B] (snn_tcm.cu)
  int Kpad = 0;                  // K rounded up for the tensor-core tiling
  int Cpad = 0;                  // C rounded up for the tensor-core tiling
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

bool tc_supported(const Geom& g, int act_type);
// Tile variants of the tensor-core kernel (sub-tiles per CTA, weight-stage size, CTAs per SM);
// variant 0 is the heuristic choice, the others are what snn_conv_tune sweeps.
int tc_variant_count();
bool tc_variant_ok(const Geom& g, int act_type, int variant);
cudaError_t tc_forward(LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched, int* status_dev,
                       int variant);
size_t tc_weight_bytes(const Geom& g, int act_type, int* Kpad, int* Cpad);
cudaError_t tc_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched);

// Channel-major tensor-core kernel (weights in tensor memory); its variants are the positions
// per tile.  tc_variant_count()/tc_variant_ok()/tc_forward() present them after the
// position-major kernel's variants.
int cm_variant_count();
bool cm_variant_ok(const Geom& g, int act_type, int variant);
cudaError_t cm_forward(LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched, int* status_dev,
                       int variant);
size_t cm_weight_bytes(const Geom& g, int act_type);
cudaError_t cm_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched);

// Tensor-core weight operand of the position-major layout with a caller-chosen channel block and
// layout tile, written to `dst` (9 * n_chunks * Kpad * 16 bytes); used by the grouped kernel.
cudaError_t tc_expand_weights_custom(const uint32_t* wplanes, void* dst, int C, int K, int Cw, int Kpad, int n_chunks,
                                     int cb_chunks, int NtL, bool f16, cudaStream_t s);

// Several independent problems in one persistent tensor-core launch (snn_tcg.cu).
struct GroupDev;
cudaError_t tcg_create(const LayerDev* const* layers, const Geom* geoms, int count, int act_type, cudaStream_t s,
                       GroupDev** out, int* launched);
cudaError_t tcg_forward(GroupDev* G, const void* const* act, void* const* out, int out_i32, cudaStream_t s,
                        int* status_dev, int* launched);
void tcg_destroy(GroupDev* G);
int tcg_count(const GroupDev* G);

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
