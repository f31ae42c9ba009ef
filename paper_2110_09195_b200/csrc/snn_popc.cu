// Decoded-weight path on the integer ALUs: implicit GEMM with XOR + popcount
// (Sec. 3: the +/-1 dot product of 32 channels is 32 - 2*popc(a XOR w)).
//
// A CTA owns a tile of TH x TW output pixels (TH "global rows" = rows of the
// batch stacked image after image) and KT output channels.  The three input
// rows of every tile row are staged in shared memory as [word][row][col] so a
// warp's 32 pixels read consecutive words; the decoded bit-planes of the KT
// channels sit beside them as [tap][word][co] and are read as broadcasts.
// Taps outside the image read 0 words, which the arithmetic takes for -1; the
// per-(case, co) corrections from create time repair the sum (snn_decode.cu).
#include "snn_internal.h"

namespace snn {

struct PopcParams {
  const uint32_t* act;
  const uint32_t* wplanes;
  const int32_t* corr;
  const float* alpha;
  void* out;
  int out_i32;
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int TH, TW, RL;   // tile rows / cols, staged row length (TW-1)*stride+3
  int tiles_x;
  int rows_total;   // N*Ho
  int cwc;          // channel words per shared-memory chunk
};

template <int PM, int PN>
__global__ void __launch_bounds__(256) popc_conv_kernel(const PopcParams p) {
  constexpr int KT = 4 * PN;
  extern __shared__ __align__(16) uint32_t smem[];
  const int TH3 = p.TH * 3;
  uint32_t* As = smem;                                  // [cwc][TH3][RL]
  uint32_t* Ws = smem + (size_t)p.cwc * TH3 * p.RL;     // [9][cwc][KT]
  // keep Ws 16-byte aligned for the vector reads
  Ws = (uint32_t*)(((uintptr_t)Ws + 15) & ~(uintptr_t)15);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int pw = warp & 1, cg = warp >> 1;
  const int tile_x = blockIdx.x % p.tiles_x, tile_y = blockIdx.x / p.tiles_x;
  const int row0 = tile_y * p.TH, col0 = tile_x * p.TW;
  const int co0 = blockIdx.y * KT;

  int base[PM];
  bool valid[PM];
  int gy[PM], ox[PM];
#pragma unroll
  for (int j = 0; j < PM; ++j) {
    int pj = pw * 32 + lane + 64 * j;
    int ty = pj / p.TW, tx = pj - ty * p.TW;
    gy[j] = row0 + ty;
    ox[j] = col0 + tx;
    valid[j] = (ty < p.TH) && (gy[j] < p.rows_total) && (ox[j] < p.Wo);
    if (!valid[j]) { ty = 0; tx = 0; }
    base[j] = ty * 3 * p.RL + tx * p.stride;
  }

  int acc[PM][PN];
#pragma unroll
  for (int j = 0; j < PM; ++j)
#pragma unroll
    for (int n = 0; n < PN; ++n) acc[j][n] = 0;

  const int in_c0 = col0 * p.stride - p.pad;
  for (int w0 = 0; w0 < p.Cw; w0 += p.cwc) {
    const int cw = min(p.cwc, p.Cw - w0);
    // ---- stage activations
    const int n_a = cw * TH3 * p.RL;
    for (int i = tid; i < n_a; i += 256) {
      int wd = i % cw, pos = i / cw;
      int col = pos % p.RL, rs = pos / p.RL;
      int ky = rs % 3, ty = rs / 3;
      int g = row0 + ty;
      uint32_t v = 0;
      if (g < p.rows_total) {
        int n = g / p.Ho, y = g - n * p.Ho;
        int r = y * p.stride - p.pad + ky, c = in_c0 + col;
        if (r >= 0 && r < p.H && c >= 0 && c < p.W)
          v = __ldg(p.act + (((size_t)n * p.H + r) * p.W + c) * p.Cw + w0 + wd);
      }
      As[(wd * TH3 + rs) * p.RL + col] = v;
    }
    // ---- stage weight planes
    const int n_w = 9 * cw * KT;
    for (int i = tid; i < n_w; i += 256) {
      int col = i % KT, tw = i / KT;
      int wd = tw % cw, t = tw / cw;
      int co = co0 + col;
      uint32_t v = 0;
      if (co < p.K) v = __ldg(p.wplanes + ((size_t)t * p.Cw + w0 + wd) * p.K + co);
      Ws[(t * p.cwc + wd) * KT + col] = v;
    }
    __syncthreads();
    // ---- contraction
#pragma unroll
    for (int t = 0; t < 9; ++t) {
      const int toff = (t / 3) * p.RL + (t % 3);
      for (int wd = 0; wd < cw; ++wd) {
        uint32_t a[PM];
#pragma unroll
        for (int j = 0; j < PM; ++j) a[j] = As[wd * TH3 * p.RL + base[j] + toff];
        const uint4* wp = reinterpret_cast<const uint4*>(Ws + (t * p.cwc + wd) * KT + cg * PN);
#pragma unroll
        for (int q = 0; q < PN / 4; ++q) {
          uint4 w4 = wp[q];
#pragma unroll
          for (int j = 0; j < PM; ++j) {
            acc[j][4 * q + 0] += __popc(a[j] ^ w4.x);
            acc[j][4 * q + 1] += __popc(a[j] ^ w4.y);
            acc[j][4 * q + 2] += __popc(a[j] ^ w4.z);
            acc[j][4 * q + 3] += __popc(a[j] ^ w4.w);
          }
        }
      }
    }
    __syncthreads();
  }

  // ---- epilogue: S = 9*C - 2*mismatches + border correction; Y = float(S)*alpha (Sec. 3)
  const int cobase = co0 + cg * PN;
#pragma unroll
  for (int j = 0; j < PM; ++j) {
    if (!valid[j]) continue;
    int n = gy[j] / p.Ho, y = gy[j] - n * p.Ho;
    int r0 = y * p.stride - p.pad, c0 = ox[j] * p.stride - p.pad;
    int cls = (r0 < 0 ? 1 : 0) | (r0 + 2 >= p.H ? 2 : 0) | (c0 < 0 ? 4 : 0) | (c0 + 2 >= p.W ? 8 : 0);
    size_t o = ((size_t)gy[j] * p.Wo + ox[j]) * p.K + cobase;
    const int32_t* cr = p.corr + (size_t)cls * p.K + cobase;
    if ((p.K & 3) == 0 && cobase + PN <= p.K) {
#pragma unroll
      for (int q = 0; q < PN / 4; ++q) {
        int4 s;
        int4 c4 = cls ? __ldg(reinterpret_cast<const int4*>(cr) + q) : make_int4(0, 0, 0, 0);
        s.x = 9 * p.C - 2 * acc[j][4 * q + 0] + c4.x;
        s.y = 9 * p.C - 2 * acc[j][4 * q + 1] + c4.y;
        s.z = 9 * p.C - 2 * acc[j][4 * q + 2] + c4.z;
        s.w = 9 * p.C - 2 * acc[j][4 * q + 3] + c4.w;
        if (p.out_i32) {
          reinterpret_cast<int4*>((int32_t*)p.out + o)[q] = s;
        } else {
          float4 al = __ldg(reinterpret_cast<const float4*>(p.alpha + cobase) + q);
          float4 yv;
          yv.x = __fmul_rn((float)s.x, al.x);
          yv.y = __fmul_rn((float)s.y, al.y);
          yv.z = __fmul_rn((float)s.z, al.z);
          yv.w = __fmul_rn((float)s.w, al.w);
          reinterpret_cast<float4*>((float*)p.out + o)[q] = yv;
        }
      }
    } else {
#pragma unroll
      for (int n2 = 0; n2 < PN; ++n2) {
        if (cobase + n2 >= p.K) break;
        int s = 9 * p.C - 2 * acc[j][n2] + (cls ? __ldg(cr + n2) : 0);
        if (p.out_i32) ((int32_t*)p.out)[o + n2] = s;
        else ((float*)p.out)[o + n2] = __fmul_rn((float)s, __ldg(p.alpha + cobase + n2));
      }
    }
  }
}

bool popc_supported(const Geom& g, int act_type) { return act_type == SNN_ACT_BIN && g.N >= 0; }

// Tile shape: TH*TW <= TP pixels, chosen to waste the fewest lanes.
static void pick_tile(int TP, int Wo, long long rows, int* TH, int* TW) {
  double best = -1.0;
  int bh = 1, bw = TP;
  for (int tw = 1; tw <= TP; ++tw) {
    int th = TP / tw;
    if (th < 1) continue;
    long long tx = (Wo + tw - 1) / tw, ty = (rows + th - 1) / th;
    double eff = (double)Wo * (double)rows / ((double)tx * ty * TP);
    eff -= 1e-3 / tw;  // prefer wide tiles: fewer halo columns to stage
    if (tw > Wo + 8) continue;
    if (eff > best) { best = eff; bh = th; bw = tw; }
  }
  *TH = bh;
  *TW = bw;
}

template <int PM, int PN>
static cudaError_t launch_popc(PopcParams p, cudaStream_t s) {
  constexpr int KT = 4 * PN;
  constexpr int TP = 64 * PM;
  pick_tile(TP, p.Wo, p.rows_total, &p.TH, &p.TW);
  p.RL = (p.TW - 1) * p.stride + 3;
  p.tiles_x = (p.Wo + p.TW - 1) / p.TW;
  int tiles_y = (p.rows_total + p.TH - 1) / p.TH;
  // words per chunk: keep shared memory under 96 KB
  int per_word = (p.TH * 3 * p.RL + 9 * KT) * 4;
  int cwc = (96 * 1024 - 64) / per_word;
  if (cwc < 1) return cudaErrorInvalidConfiguration;
  if (cwc > p.Cw) cwc = p.Cw;
  if (cwc > 16) cwc = 16;
  p.cwc = cwc;
  size_t smem = (size_t)cwc * per_word + 64;
  static unsigned long long done = 0;
  cudaError_t e = allow_max_smem(popc_conv_kernel<PM, PN>, &done);
  if (e != cudaSuccess) return e;
  dim3 grid((unsigned)(p.tiles_x * tiles_y), (unsigned)((p.K + KT - 1) / KT));
  popc_conv_kernel<PM, PN><<<grid, 256, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t popc_forward(const LayerDev& L, const Geom& g, const Launch& l, int* launched) {
  PopcParams p;
  p.act = (const uint32_t*)l.act;
  p.wplanes = L.wplanes;
  p.corr = L.corr;
  p.alpha = L.alpha;
  p.out = l.out;
  p.out_i32 = l.out_i32;
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K; p.Cw = g.Cw;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  p.rows_total = g.N * g.Ho;
  p.TH = p.TW = p.RL = p.tiles_x = p.cwc = 0;
  *launched += 1;
  if (g.K <= 16) return launch_popc<2, 4>(p, l.stream);
  return launch_popc<2, 8>(p, l.stream);
}

}  // namespace snn
