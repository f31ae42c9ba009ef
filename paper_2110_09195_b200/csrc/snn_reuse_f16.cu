// Codebook reuse with fp16 activations: the weights-only variant the paper deploys (Sec. 5.3: activations
// are not binarised) computed the way the paper shares work (Sec. 4.5, Fig. 6; accelerator of Sec. 4.6):
//   stage 1   P[ci][k][pixel] = sum over the nine taps of  K_k[tap] * a[pixel + tap][ci]      (+/- additions)
//             for every kernel k of the layer's codebook, once per input channel and pixel,
//   stage 2   S[co][pixel] = sum over ci of P[ci][idx[co][ci]][pixel]                           (index-driven)
// and Y = alpha[co] * S.  Sums are fp32, in the order of the two stages.
//
// One CTA owns 16 consecutive output pixels and all output channels.  Input channels go through in chunks
// of CC = min(8, 512 / 2^tau): the chunk's 3x3 windows are converted to fp32 in shared memory, stage 1 fills
// a table of CC * 2^tau rows of 16 pixels, stage 2 has one thread per output channel add the row its index
// names (four 16-byte reads) to 16 accumulators in registers.  P never leaves the SM.
#include <cuda_fp16.h>

#include "snn_internal.h"

namespace snn {

namespace {

constexpr int RF_PT = 16;        // output pixels per CTA
constexpr int RF_THREADS = 256;
constexpr int RF_ROWS = 512;     // table rows per chunk = CC * 2^tau at most
constexpr int RF_CC_MAX = 8;

struct RFParams {
  const __half* act;
  const uint16_t* idx;
  const uint16_t* codebook;
  const float* alpha;
  float* out;
  int N, H, W, C, K, stride, pad, Ho, Wo, T, CC;
  long long pixels;
};

template <int KJ>
__global__ void __launch_bounds__(RF_THREADS) reuse_f16_kernel(const RFParams p) {
  __shared__ __align__(16) float win[RF_CC_MAX * 9 * RF_PT];    // [cc][tap][pixel]
  __shared__ __align__(16) float tab[RF_ROWS * RF_PT];          // [cc * T + k][pixel]
  __shared__ uint16_t codes[512];
  __shared__ int pix_in[RF_PT * 9];                             // input pixel of (pixel, tap), or -1 (padding, past the end)

  const int tid = threadIdx.x;
  const long long pix0 = (long long)blockIdx.x * RF_PT;
  const int T = p.T, CC = p.CC, C = p.C, K = p.K;

  for (int k = tid; k < T; k += RF_THREADS) codes[k] = p.codebook[k];
  if (tid < RF_PT * 9) {
    const int pp = tid / 9, t = tid - pp * 9;
    const long long q = pix0 + pp;
    int src = -1;
    if (q < p.pixels) {
      const int x = (int)(q % p.Wo);
      const long long rest = q / p.Wo;
      const int y = (int)(rest % p.Ho);
      const int n = (int)(rest / p.Ho);
      const int r = y * p.stride + t / 3 - p.pad, c = x * p.stride + t % 3 - p.pad;
      if (r >= 0 && r < p.H && c >= 0 && c < p.W) src = (n * p.H + r) * p.W + c;
    }
    pix_in[tid] = src;
  }
  float acc[KJ][RF_PT];
#pragma unroll
  for (int j = 0; j < KJ; ++j)
#pragma unroll
    for (int e = 0; e < RF_PT; ++e) acc[j][e] = 0.f;
  const bool vec = CC == 8 && (C & 7) == 0 && (reinterpret_cast<uintptr_t>(p.act) & 15) == 0 &&
                   (reinterpret_cast<uintptr_t>(p.idx) & 15) == 0;
  __syncthreads();

  for (int ci0 = 0; ci0 < C; ci0 += CC) {
    // the chunk's windows, fp16 -> fp32 (zero padding is a literal 0)
    if (tid < RF_PT * 9) {
      const int pp = tid / 9, t = tid - pp * 9;
      const int src = pix_in[tid];
      if (vec) {
        uint4 raw = make_uint4(0, 0, 0, 0);
        if (src >= 0) raw = __ldg(reinterpret_cast<const uint4*>(p.act + (size_t)src * C + ci0));
        const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __half22float2(h[e]);
          win[((2 * e) * 9 + t) * RF_PT + pp] = f.x;
          win[((2 * e + 1) * 9 + t) * RF_PT + pp] = f.y;
        }
      } else {
        for (int cc = 0; cc < CC; ++cc) {
          float v = 0.f;
          if (src >= 0 && ci0 + cc < C) v = __half2float(p.act[(size_t)src * C + ci0 + cc]);
          win[(cc * 9 + t) * RF_PT + pp] = v;
        }
      }
    }
    __syncthreads();
    // stage 1: every codebook kernel on every channel of the chunk (nine signed additions each)
    for (int e = tid; e < CC * T * RF_PT; e += RF_THREADS) {
      const int pp = e % RF_PT, row = e / RF_PT;
      const int cc = row / T, k = row - cc * T;
      const uint32_t code = codes[k];
      const float* w = win + cc * 9 * RF_PT + pp;
      float v = 0.f;
#pragma unroll
      for (int t = 0; t < 9; ++t) {
        const float a = w[t * RF_PT];
        v += ((code >> (8 - t)) & 1u) ? a : -a;   // bit 8 - tap of a code: +1 (Sec. 4.1 numbering)
      }
      tab[e] = v;
    }
    __syncthreads();
    // stage 2: a thread is an output channel; its index picks the row to add
#pragma unroll
    for (int j = 0; j < KJ; ++j) {
      const int co = tid + j * RF_THREADS;
      if (co >= K) continue;
      uint16_t kk[RF_CC_MAX];
      if (vec) {
        const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p.idx + (size_t)co * C + ci0));
        kk[0] = (uint16_t)(raw.x & 0xffff); kk[1] = (uint16_t)(raw.x >> 16);
        kk[2] = (uint16_t)(raw.y & 0xffff); kk[3] = (uint16_t)(raw.y >> 16);
        kk[4] = (uint16_t)(raw.z & 0xffff); kk[5] = (uint16_t)(raw.z >> 16);
        kk[6] = (uint16_t)(raw.w & 0xffff); kk[7] = (uint16_t)(raw.w >> 16);
      } else {
#pragma unroll
        for (int cc = 0; cc < RF_CC_MAX; ++cc) kk[cc] = (cc < CC && ci0 + cc < C) ? p.idx[(size_t)co * C + ci0 + cc] : 0;
      }
#pragma unroll
      for (int cc = 0; cc < RF_CC_MAX; ++cc) {
        if (cc >= CC || ci0 + cc >= C) break;
        const float4* r = reinterpret_cast<const float4*>(tab + (size_t)(cc * T + kk[cc]) * RF_PT);
#pragma unroll
        for (int e = 0; e < RF_PT / 4; ++e) {
          const float4 v = r[e];
          acc[j][4 * e] += v.x;
          acc[j][4 * e + 1] += v.y;
          acc[j][4 * e + 2] += v.z;
          acc[j][4 * e + 3] += v.w;
        }
      }
    }
    __syncthreads();
  }
  // epilogue: one fp32 multiply per output (Sec. 3: channel-wise scale)
#pragma unroll
  for (int j = 0; j < KJ; ++j) {
    const int co = tid + j * RF_THREADS;
    if (co >= K) continue;
    const float a = p.alpha[co];
#pragma unroll
    for (int e = 0; e < RF_PT; ++e)
      if (pix0 + e < p.pixels) p.out[(size_t)(pix0 + e) * K + co] = __fmul_rn(a, acc[j][e]);
  }
}

}  // namespace

bool reuse_f16_supported(const Geom& g) {
  return g.K <= 4 * RF_THREADS && (long long)g.N * g.H * g.W < (1ll << 31) && (long long)g.N * g.Ho * g.Wo < (1ll << 31);
}

cudaError_t reuse_f16_forward(const LayerDev& L, const Geom& g, const Launch& l, int* launched) {
  if (l.out_i32 != 0) return cudaErrorInvalidValue;   // fp32 outputs only
  RFParams p;
  p.act = (const __half*)l.act;
  p.idx = L.idx;
  p.codebook = L.codebook;
  p.alpha = L.alpha;
  p.out = (float*)l.out;
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  p.T = g.T;
  int cc = RF_ROWS / g.T;
  p.CC = cc < 1 ? 1 : (cc > RF_CC_MAX ? RF_CC_MAX : cc);
  p.pixels = (long long)g.N * g.Ho * g.Wo;
  const long long blocks = (p.pixels + RF_PT - 1) / RF_PT;
  if (blocks <= 0) return cudaSuccess;
  if (blocks > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
  const int kj = (g.K + RF_THREADS - 1) / RF_THREADS;
  *launched += 1;
  if (kj <= 1) reuse_f16_kernel<1><<<(unsigned)blocks, RF_THREADS, 0, l.stream>>>(p);
  else if (kj == 2) reuse_f16_kernel<2><<<(unsigned)blocks, RF_THREADS, 0, l.stream>>>(p);
  else reuse_f16_kernel<4><<<(unsigned)blocks, RF_THREADS, 0, l.stream>>>(p);
  return cudaGetLastError();
}

}  // namespace snn
