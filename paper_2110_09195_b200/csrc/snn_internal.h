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
  int Kpad = 0;                  // K rounded up for the tensor-core tiling
  int Cpad = 0;                  // C rounded up for the tensor-core tiling
};

struct Launch {
  const void* act;
  void* out;
  int out_i32;   // 1: write int32 S, 0: write fp32 alpha*S
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
cudaError_t tc_forward(const LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched,
                       int* dev_status_host);
size_t tc_weight_bytes(const Geom& g, int act_type, int* Kpad, int* Cpad);
cudaError_t tc_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched);

cudaError_t microbench(int kind, double* rate);

}  // namespace snn
