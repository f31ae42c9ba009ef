// Codebook-reuse path (Sec. 4.5 "Acceleration", Fig. 6; Sec. 4.6 dataflow):
// every 1x3x3 activation slice is evaluated once against each of the 2^tau
// codebook kernels, and an output channel adds, along c_in, the entry its
// index selects -- the look-up table of the paper's accumulator unit.
//
// Mapping used here.  A CTA owns a run of consecutive output pixels (batch,
// row, column flattened) and up to 256 output channels, and walks c_in in
// chunks of 16 channels:
//   stage 0  one thread per pixel reads the nine activation words of its 3x3 window once
//            and turns the chunk's 16 channels into sixteen 9-bit window codes in shared
//            memory (a word is read once per chunk, not once per channel);
//   stage 1  for every (4-pixel group, channel) of the chunk build the table
//            tab[k] = matching-tap counts of the four slices against kernel k,
//            one byte per pixel, from the 512 x 2^tau table made at create
//            time (a slice's dot product is 2*match - 9);
//   stage 2  lane = output channel: acc += tab[idx[co][ci]] -- one shared-memory
//            read and one packed add serve four pixels.  A table of up to 32
//            words covers each bank once, so any index pattern is conflict-free.
// Byte lanes hold at most 16*9 = 144 before they are widened to 16 bits.
// Taps outside the image enter as -1 and are repaired by the create-time
// corrections, exactly as in the popcount path.
#include "snn_internal.h"

namespace snn {

constexpr int RC = 16;  // channels per chunk (byte lanes stay <= 16*9)

struct ReuseParams {
  const uint32_t* act;
  const uint16_t* idx;      // [K][C]
  const uint8_t* match9;    // [NH][512][16]
  const int32_t* corr;
  const float* alpha;
  void* out;
  int out_i32;
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int T, Tp, NH;            // codebook size, rounded to 16, Tp/16
  int KW, QG;               // co-warps and quad-groups per CTA (KW*QG warps)
  int KT;                   // channels per CTA = 32*KW
  long long pixels;         // N*Ho*Wo
  int match_in_smem;
  int CS;                   // table stride between channels, in words
};

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t s) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(s));
  return r;
}

template <int Q>
__global__ void __launch_bounds__(256) reuse_conv_kernel(const ReuseParams p) {
  extern __shared__ __align__(16) uint8_t smem_raw[];
  const int nthreads = blockDim.x;
  const int NQ = p.QG * Q;          // quads per CTA
  const int PT = NQ * 4;            // pixels per CTA
  // shared-memory carve-up
  uint32_t* tab = reinterpret_cast<uint32_t*>(smem_raw);                 // [RC][CS]
  uint16_t* idxs = reinterpret_cast<uint16_t*>(tab + (size_t)RC * p.CS); // [RC][KT]
  int* pix_base = reinterpret_cast<int*>(idxs + (size_t)RC * p.KT);      // [PT] n*H*W or -1
  int* pix_r0 = pix_base + PT;
  int* pix_c0 = pix_r0 + PT;
  uint16_t* codes = reinterpret_cast<uint16_t*>(pix_c0 + PT);            // [RC][PT] window code of (channel, pixel)
  uint8_t* m9s = reinterpret_cast<uint8_t*>(codes + (size_t)RC * PT);    // [NH][512][16] (optional)
  m9s = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(m9s) + 15) & ~(uintptr_t)15);

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int kw = warp % p.KW, qg = warp / p.KW;
  const long long g0 = (long long)blockIdx.x * PT;
  const int cob = blockIdx.y * p.KT;
  const int co_l = kw * 32 + lane;
  const int co = cob + co_l;

  for (int i = tid; i < PT; i += nthreads) {
    long long g = g0 + i;
    if (g < p.pixels) {
      int x = (int)(g % p.Wo);
      long long gy = g / p.Wo;
      int y = (int)(gy % p.Ho), n = (int)(gy / p.Ho);
      pix_base[i] = n * p.H * p.W;
      pix_r0[i] = y * p.stride - p.pad;
      pix_c0[i] = x * p.stride - p.pad;
    } else {
      pix_base[i] = -1;
      pix_r0[i] = 0;
      pix_c0[i] = 0;
    }
  }
  if (p.match_in_smem) {
    const uint4* src = reinterpret_cast<const uint4*>(p.match9);
    uint4* dst = reinterpret_cast<uint4*>(m9s);
    for (int i = tid; i < p.NH * 512; i += nthreads) dst[i] = __ldg(src + i);
  }
  const uint8_t* m9 = p.match_in_smem ? m9s : p.match9;

  uint32_t lo[Q], hi[Q];
#pragma unroll
  for (int q = 0; q < Q; ++q) lo[q] = hi[q] = 0;

  for (int c0 = 0; c0 < p.C; c0 += RC) {
    const int cc = min(RC, p.C - c0);
    __syncthreads();  // previous chunk's readers are done; coordinates / match table are visible
    // ---- indices of this chunk, [ci][co]
    for (int i = tid; i < RC * p.KT; i += nthreads) {
      int ci = i % RC, cl = i / RC;
      uint16_t v = 0;
      if (ci < cc && cob + cl < p.K) v = __ldg(p.idx + (size_t)(cob + cl) * p.C + c0 + ci);
      idxs[ci * p.KT + cl] = v;
    }
    // ---- stage 0: window codes of the chunk's channels, one thread per pixel
    {
      const int wd = c0 >> 5, sh = c0 & 31;   // the chunk's 16 channels are one half of a 32-channel word
      for (int pi = tid; pi < PT; pi += nthreads) {
        const int nb = pix_base[pi], r0 = pix_r0[pi], cc0 = pix_c0[pi];
        uint32_t half[9];
#pragma unroll
        for (int t = 0; t < 9; ++t) {
          const int r = r0 + t / 3, cx = cc0 + t % 3;
          half[t] = 0;   // outside the image: read as -1, repaired by the border corrections
          if (nb >= 0 && r >= 0 && r < p.H && cx >= 0 && cx < p.W)
            half[t] = (__ldg(p.act + ((size_t)nb + (size_t)r * p.W + cx) * p.Cw + wd) >> sh) & 0xffffu;
        }
#pragma unroll
        for (int ci = 0; ci < RC; ++ci) {
          uint32_t code = 0;
#pragma unroll
          for (int t = 0; t < 9; ++t) code |= ((half[t] >> ci) & 1u) << (8 - t);
          codes[ci * PT + pi] = (uint16_t)code;
        }
      }
    }
    __syncthreads();
    // ---- stage 1: tables for every (quad, channel) of the chunk
    for (int item = tid; item < NQ * RC; item += nthreads) {
      const int ci = item % RC, quad = item / RC;
      if (ci >= cc) continue;
      uint32_t w9[4];
      {
        const uint2 cq = *reinterpret_cast<const uint2*>(codes + ci * PT + quad * 4);   // four pixels' codes
        w9[0] = cq.x & 0xffffu; w9[1] = cq.x >> 16; w9[2] = cq.y & 0xffffu; w9[3] = cq.y >> 16;
      }
      uint32_t* row = tab + (size_t)ci * p.CS + (size_t)quad * p.Tp;
      for (int h = 0; h < p.NH; ++h) {
        uint4 m[4];
#pragma unroll
        for (int j = 0; j < 4; ++j)
          m[j] = *reinterpret_cast<const uint4*>(m9 + ((size_t)h * 512 + w9[j]) * 16);
        // 4x4 byte transposes: word k = (pixel0, pixel1, pixel2, pixel3) counts for kernel k
        const uint32_t a0[4] = {m[0].x, m[0].y, m[0].z, m[0].w};
        const uint32_t a1[4] = {m[1].x, m[1].y, m[1].z, m[1].w};
        const uint32_t a2[4] = {m[2].x, m[2].y, m[2].z, m[2].w};
        const uint32_t a3[4] = {m[3].x, m[3].y, m[3].z, m[3].w};
#pragma unroll
        for (int g4 = 0; g4 < 4; ++g4) {
          uint32_t t0 = prmt(a0[g4], a1[g4], 0x5140u), t1 = prmt(a2[g4], a3[g4], 0x5140u);
          uint32_t t2 = prmt(a0[g4], a1[g4], 0x7362u), t3 = prmt(a2[g4], a3[g4], 0x7362u);
          uint4 o;
          o.x = prmt(t0, t1, 0x5410u);
          o.y = prmt(t0, t1, 0x7632u);
          o.z = prmt(t2, t3, 0x5410u);
          o.w = prmt(t2, t3, 0x7632u);
          *reinterpret_cast<uint4*>(row + h * 16 + g4 * 4) = o;
        }
      }
    }
    __syncthreads();
    // ---- stage 2: lane = output channel, index-driven accumulate (Sec. 4.6 accumulator unit)
    {
      uint32_t acc8[Q];
#pragma unroll
      for (int q = 0; q < Q; ++q) acc8[q] = 0;
      const uint32_t* tb = tab + (size_t)qg * Q * p.Tp;
      for (int ci = 0; ci < cc; ++ci) {
        const uint32_t id = idxs[ci * p.KT + co_l];
        const uint32_t* e = tb + (size_t)ci * p.CS + id;
#pragma unroll
        for (int q = 0; q < Q; ++q) acc8[q] += e[q * p.Tp];
      }
#pragma unroll
      for (int q = 0; q < Q; ++q) {
        lo[q] += acc8[q] & 0x00ff00ffu;
        hi[q] += (acc8[q] >> 8) & 0x00ff00ffu;
      }
    }
  }

  // ---- epilogue: S = 2*matches - 9*C + border correction; Y = float(S)*alpha (Sec. 3)
  if (co < p.K) {
    const float al = p.out_i32 ? 0.f : __ldg(p.alpha + co);
#pragma unroll
    for (int q = 0; q < Q; ++q) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int pi = (qg * Q + q) * 4 + j;
        if (pix_base[pi] < 0) continue;
        const uint32_t src = (j & 1) ? hi[q] : lo[q];
        const int match = (j & 2) ? (int)(src >> 16) : (int)(src & 0xffffu);
        const int r0 = pix_r0[pi], c0 = pix_c0[pi];
        const int cls = (r0 < 0 ? 1 : 0) | (r0 + 2 >= p.H ? 2 : 0) | (c0 < 0 ? 4 : 0) | (c0 + 2 >= p.W ? 8 : 0);
        int s = 2 * match - 9 * p.C;
        if (cls) s += __ldg(p.corr + (size_t)cls * p.K + co);
        const size_t o = (size_t)(g0 + pi) * p.K + co;
        if (p.out_i32) ((int32_t*)p.out)[o] = s;
        else ((float*)p.out)[o] = __fmul_rn((float)s, al);
      }
    }
  }
}

bool reuse_supported(const Geom& g, int act_type) {
  if (act_type == SNN_ACT_F16) return reuse_f16_supported(g);
  if (act_type != SNN_ACT_BIN) return false;
  // 16-bit lanes hold the matching-tap total 9*C
  return (long long)9 * g.C <= 65535;
}

static int pow2_floor(int v) {
  int r = 1;
  while (r * 2 <= v) r *= 2;
  return r;
}

template <int Q>
static cudaError_t launch_reuse(const ReuseParams& p, size_t smem, dim3 grid, int threads, cudaStream_t s) {
  static unsigned long long done = 0;
  cudaError_t e = allow_max_smem(reuse_conv_kernel<Q>, &done);
  if (e != cudaSuccess) return e;
  reuse_conv_kernel<Q><<<grid, threads, smem, s>>>(p);
  return cudaGetLastError();
}

cudaError_t reuse_forward(const LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched) {
  if (act_type == SNN_ACT_F16) return reuse_f16_forward(L, g, l, launched);
  ReuseParams p;
  p.act = (const uint32_t*)l.act;
  p.idx = L.idx;
  p.match9 = L.match9;
  p.corr = L.corr;
  p.alpha = L.alpha;
  p.out = l.out;
  p.out_i32 = l.out_i32;
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K; p.Cw = g.Cw;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  p.T = g.T;
  p.Tp = (g.T + 15) / 16 * 16;
  p.NH = p.Tp / 16;
  p.pixels = (long long)g.N * g.Ho * g.Wo;
  int kw = (g.K + 31) / 32;
  p.KW = kw >= 8 ? 8 : (kw > 4 ? 8 : (kw > 2 ? 4 : (kw > 1 ? 2 : 1)));
  p.KT = 32 * p.KW;
  // quads per CTA bounded by the table budget: RC * NQ * Tp words <= 64 KB
  int nq_max = 1024 / p.Tp;
  if (nq_max < 1) nq_max = 1;
  int qg = 8 / p.KW;
  if (qg > nq_max) qg = pow2_floor(nq_max);
  int q = nq_max / qg;
  if (q > 16) q = 16;
  q = pow2_floor(q);
  p.QG = qg;
  const int NQ = qg * q;
  p.CS = NQ * p.Tp + 4;
  const size_t match_bytes = (size_t)p.NH * 512 * 16;
  p.match_in_smem = match_bytes <= 64 * 1024;
  size_t smem = (size_t)RC * p.CS * 4 + (size_t)RC * p.KT * 2 + (size_t)NQ * 4 * 3 * 4 + (size_t)RC * NQ * 4 * 2 + 16 +
                (p.match_in_smem ? match_bytes : 0);
  const int threads = 32 * p.KW * p.QG;
  const int PT = NQ * 4;
  dim3 grid((unsigned)((p.pixels + PT - 1) / PT), (unsigned)((g.K + p.KT - 1) / p.KT));
  *launched += 1;
  switch (q) {
    case 16: return launch_reuse<16>(p, smem, grid, threads, l.stream);
    case 8: return launch_reuse<8>(p, smem, grid, threads, l.stream);
    case 4: return launch_reuse<4>(p, smem, grid, threads, l.stream);
    case 2: return launch_reuse<2>(p, smem, grid, threads, l.stream);
    default: return launch_reuse<1>(p, smem, grid, threads, l.stream);
  }
}

}  // namespace snn
