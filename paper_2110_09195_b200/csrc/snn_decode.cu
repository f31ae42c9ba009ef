// Create-time decode (Sec. 4.4 storage -> compute form), all on the device:
//   tau-bit index stream -> idx[K][C]
//   idx + codebook       -> bit-planes of the +/-1 weights, [tap][word][co]
//   bit-planes           -> border corrections corr[class][co]
//   codebook             -> matching-tap table for the codebook-reuse path
#include "snn_internal.h"

namespace snn {

// One thread per (co, ci): pull tau bits out of the LSB-first stream.
__global__ void unpack_idx_kernel(const uint8_t* __restrict__ stream, uint16_t* __restrict__ idx,
                                  long long n_elem, int tau, long long n_bytes) {
  long long e = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (e >= n_elem) return;
  long long bit = e * tau;
  long long byte = bit >> 3;
  uint32_t v = 0;
#pragma unroll
  for (int i = 0; i < 3; ++i) {
    long long b = byte + i;
    if (b < n_bytes) v |= (uint32_t)stream[b] << (8 * i);
  }
  idx[e] = (uint16_t)((v >> (bit & 7)) & ((1u << tau) - 1u));
}

// One thread per (co, word): gather the 9-bit codes of 32 input channels and
// transpose them into nine 32-bit planes (plane t, bit b = weight of tap t for
// channel 32*word+b is +1).  Tap t = 3*ky + kx is bit 8-t of a code (Sec. 4.1).
// Channels beyond C get 0 bits, matching the zero padding bits of the activations.
__global__ void decode_planes_kernel(const uint16_t* __restrict__ idx, const uint16_t* __restrict__ codebook,
                                     uint32_t* __restrict__ wplanes, int C, int K, int Cw) {
  int co = blockIdx.x * blockDim.x + threadIdx.x;
  int wd = blockIdx.y;
  if (co >= K) return;
  uint32_t plane[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) plane[t] = 0;
  for (int b = 0; b < 32; ++b) {
    int ci = wd * 32 + b;
    if (ci >= C) break;
    uint32_t code = codebook[idx[(size_t)co * C + ci]];
#pragma unroll
    for (int t = 0; t < 9; ++t) plane[t] |= ((code >> (8 - t)) & 1u) << b;
  }
#pragma unroll
  for (int t = 0; t < 9; ++t) wplanes[((size_t)t * Cw + wd) * K + co] = plane[t];
}

// 1x1 extension (appendix "Extending to Bottleneck with 1x1 Kernels"): an index names an 8-input-channel vector;
// element j of the vector (channel 8g + j) is bit 7 - j of its 8-bit code.  One plane, [word][co].
__global__ void decode_planes1x1_kernel(const uint16_t* __restrict__ idx, const uint16_t* __restrict__ codebook,
                                        uint32_t* __restrict__ wplanes, int C, int K, int Cw) {
  int co = blockIdx.x * blockDim.x + threadIdx.x;
  int wd = blockIdx.y;
  if (co >= K) return;
  const int G = C / 8;
  uint32_t plane = 0;
  for (int g4 = 0; g4 < 4; ++g4) {
    int g = wd * 4 + g4;
    if (g >= G) break;
    uint32_t code = codebook[idx[(size_t)co * G + g]];
#pragma unroll
    for (int e = 0; e < 8; ++e) plane |= ((code >> (7 - e)) & 1u) << (8 * g4 + e);
  }
  wplanes[(size_t)wd * K + co] = plane;
}

// Border corrections.  The integer kernels read a zero activation word where a
// tap falls outside the image, which the +/-1 arithmetic takes for -1; the true
// contribution of such a tap is 0 (zero padding).  Adding back
//   sum_{ci} w(co,ci,t)  for every outside tap t
// repairs the sum.  A pixel's outside taps are the union of whole kernel rows /
// columns, so 4 bits name the case: bit0 top row, bit1 bottom row, bit2 left
// column, bit3 right column.  One thread per co.
__global__ void corr_kernel(const uint32_t* __restrict__ wplanes, int32_t* __restrict__ corr, int C, int K,
                            int Cw) {
  int co = blockIdx.x * blockDim.x + threadIdx.x;
  if (co >= K) return;
  int wsum[9];
#pragma unroll
  for (int t = 0; t < 9; ++t) {
    int plus = 0;
    for (int wd = 0; wd < Cw; ++wd) plus += __popc(wplanes[((size_t)t * Cw + wd) * K + co]);
    wsum[t] = 2 * plus - C;
  }
  for (int cls = 0; cls < 16; ++cls) {
    int acc = 0;
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      int ky = t / 3, kx = t % 3;
      bool outside = ((cls & 1) && ky == 0) || ((cls & 2) && ky == 2) || ((cls & 4) && kx == 0) ||
                     ((cls & 8) && kx == 2);
      if (outside) acc += wsum[t];
    }
    corr[(size_t)cls * K + co] = acc;
  }
}

// match9[(k/16)][w][k%16] = number of the 9 taps at which window code w agrees
// with codebook kernel k (XNOR + bitcount of Sec. 3 on one 3x3 slice); the
// slice's +/-1 dot product with kernel k is 2*match - 9.
__global__ void match9_kernel(const uint16_t* __restrict__ codebook, uint8_t* __restrict__ match9, int T) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  int Tp = (T + 15) / 16 * 16;
  if (i >= 512 * Tp) return;
  int k = i % Tp, w = i / Tp;
  uint8_t m = 0;
  if (k < T) m = (uint8_t)(9 - __popc((uint32_t)(w ^ codebook[k]) & 0x1ffu));
  match9[((size_t)(k / 16) * 512 + w) * 16 + (k % 16)] = m;
}

cudaError_t decode_layer(const LayerDev& L, const uint8_t* idx_packed_dev, const Geom& g, int act_type,
                         cudaStream_t s, int* launched) {
  (void)act_type;
  long long n_elem = (long long)g.K * (g.ksize == 1 ? g.C / 8 : g.C);
  long long n_bytes = (n_elem * g.tau + 7) / 8;
  unpack_idx_kernel<<<(unsigned)((n_elem + 255) / 256), 256, 0, s>>>(idx_packed_dev, L.idx, n_elem, g.tau, n_bytes);
  dim3 grid((g.K + 127) / 128, g.Cw);
  if (g.ksize == 1) {
    // only the tensor-core path runs 1x1 layers: no border corrections (no padding), no matching-tap table
    decode_planes1x1_kernel<<<grid, 128, 0, s>>>(L.idx, L.codebook, L.wplanes, g.C, g.K, g.Cw);
    *launched += 2;
    return cudaGetLastError();
  }
  decode_planes_kernel<<<grid, 128, 0, s>>>(L.idx, L.codebook, L.wplanes, g.C, g.K, g.Cw);
  corr_kernel<<<(g.K + 127) / 128, 128, 0, s>>>(L.wplanes, L.corr, g.C, g.K, g.Cw);
  int Tp = (g.T + 15) / 16 * 16;
  match9_kernel<<<(512 * Tp + 255) / 256, 256, 0, s>>>(L.codebook, L.match9, g.T);
  *launched += 4;
  return cudaGetLastError();
}

}  // namespace snn
