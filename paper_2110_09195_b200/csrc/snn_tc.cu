// Decoded-weight path on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// The +/-1 weights of Sec. 3 become int8 (binary activations, exact int32
// accumulation) or fp16 (fp16 activations, fp32 accumulation) operands and the
// 3x3 convolution runs as an implicit GEMM:
//   M = 128 consecutive positions of a padded, flattened copy of the input,
//   N = a tile of output channels, K = (tap, input channel).
//
// Implicit im2col without copies.  The input tile is expanded once into shared
// memory as [16-byte channel chunk][position][16 B], the K-major layout without
// swizzle in which consecutive rows are 16 bytes apart.  The A operand of tap
// (ky, kx) is then the same buffer read from a start address shifted by
// ky*pitch + kx rows, so the nine taps reuse one staged tile.  The flattened
// space keeps one zero column per row and one zero row per image (shared by
// neighbours), which makes zero padding literal zeros (a zero byte contributes
// 0, as the definition requires; no border correction is needed here).
// Stride 2 splits the padded input into its four row/column parity planes, in
// each of which the taps are again plain shifts.
//
// Per CTA (192 threads): warps 0-3 expand activations and later run the
// epilogue (TMEM -> registers -> alpha scale -> global), warp 4 issues the
// MMAs, warp 5 streams the weight stages with bulk async copies through an
// mbarrier ring.  Every wait is bounded; a wait that runs out raises a status
// word the host reads, and the CTA still frees its TMEM and returns.
#include <cuda_fp16.h>

#include <cstdlib>

#include "snn_internal.h"

namespace snn {

namespace {

constexpr int TC_THREADS = 192;
constexpr int TC_WORKERS = 128;
constexpr int NS = 4;                     // weight stages in flight
constexpr uint32_t WAIT_LIMIT = 1u << 20; // try_wait attempts before giving up (each suspends up to ~us)

struct TcParams {
  const void* act;        // uint32 [N][H][W][Cw] or half [N][H][W][C]
  const uint8_t* wt;      // tiled weights, 16-byte chunks: [tap][chunk][Kpad][16 B]
  const float* alpha;
  void* out;
  int* status;            // mapped host word, set on a timed-out wait
  int out_i32;
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int Kpad, n_chunks;     // chunks of 16 B along the (padded) channel dimension
  int Hq, Wq;             // rows per image / row pitch of the flattened position space
  int n_planes;           // 1 (stride 1) or 4 (stride 2)
  int halo;               // largest tap shift in rows
  int Rr;                 // staged rows per plane = 128*MT + halo
  int MT, Nt;             // M sub-tiles per CTA, channels per CTA
  int cb_chunks;          // chunks per channel block (A staged per block)
  int n_cb;               // channel blocks
  int ks_chunks;          // chunks per weight stage
  long long Qtot;         // flattened positions to cover
  uint32_t tmem_cols;     // power of two >= MT*Nt
  uint32_t a_bytes;       // bytes of the staged activation block
  uint32_t stage_bytes;   // bytes of one weight stage
};

// ---------------------------------------------------------------- PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// Bounded wait for the phase with the given parity; false when the limit ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint32_t limit = WAIT_LIMIT) {
  for (uint32_t it = 0; it < limit; ++it) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(src), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void raise_status(int* status, int code) {
  *reinterpret_cast<volatile int*>(status) = code;
  __threadfence_system();
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}

// Shared-memory matrix descriptor, K-major, no swizzle: rows 16 B apart inside an
// 8-row group, groups `sbo` bytes apart, the two 16-byte K chunks `lbo` bytes apart.
__device__ __forceinline__ uint64_t make_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3ffffu) >> 4);
  d |= (uint64_t)((lbo >> 4) & 0x3fffu) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3fffu) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version for this architecture
  return d;
}

template <bool F16>
__device__ __forceinline__ void mma_ss(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                       uint32_t accumulate) {
  if (F16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
        "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
        "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 4 activation bits -> 4 bytes of +1 (0x01) / -1 (0xff)
__device__ __forceinline__ uint32_t nibble_to_pm1(uint32_t nib) {
  uint32_t t = (nib * 0x00204081u) & 0x01010101u;
  return ~(t * 0xfeu);
}
__device__ __forceinline__ uint32_t nibble_to_mask(uint32_t nib) {
  uint32_t t = (nib * 0x00204081u) & 0x01010101u;
  return t * 0xffu;
}

// Flattened position of plane (pa, pb) -> input pixel, or -1 when it is padding.
__device__ __forceinline__ long long position_to_pixel(const TcParams& p, long long q, int pa, int pb) {
  if (q < 0) return -1;
  long long rg = q / p.Wq;
  int j = (int)(q - rg * p.Wq);
  long long n = rg / p.Hq;
  int i = (int)(rg - n * p.Hq);
  if (n >= p.N) return -1;
  int r = p.stride * i + pa - p.pad, c = p.stride * j + pb - p.pad;
  if (r < 0 || r >= p.H || c < 0 || c >= p.W) return -1;
  return (n * p.H + r) * p.W + c;
}

}  // namespace

template <bool F16>
__global__ void __launch_bounds__(TC_THREADS) tc_conv_kernel(const TcParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  // carve-up: [A block][NS weight stages][barriers]
  uint8_t* a_smem = smem;
  uint8_t* b_smem = smem + p.a_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(b_smem + (size_t)NS * p.stage_bytes);
  // bars: full[NS], empty[NS], a_ready, a_free, accum
  const uint32_t bar_full = smem_u32(bars), bar_empty = smem_u32(bars + NS);
  const uint32_t bar_aready = smem_u32(bars + 2 * NS), bar_afree = smem_u32(bars + 2 * NS + 1);
  const uint32_t bar_accum = smem_u32(bars + 2 * NS + 2);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * NS + 3);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long Q0 = (long long)blockIdx.x * (128 * p.MT);
  const int n0 = blockIdx.y * p.Nt;
  const int esz_chunk_ch = F16 ? 8 : 16;  // channels per 16-byte chunk

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(bar_full + 8 * s, 1);
      mbar_init(bar_empty + 8 * s, 1);
    }
    mbar_init(bar_aready, TC_WORKERS);
    mbar_init(bar_afree, 1);
    mbar_init(bar_accum, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  const int stages_per_cb_tap = p.cb_chunks / p.ks_chunks;      // weight stages per (block, tap)
  const int stages_per_cb = 9 * stages_per_cb_tap;
  const int n_stages = p.n_cb * stages_per_cb;
  const uint32_t plane_bytes = (uint32_t)p.cb_chunks * p.Rr * 16;

  if (warp == 5) {
    // ------------------------------------------------ weight producer (one lane)
    if (lane == 0) {
      int issued = 0;
      for (int i = 0; i < n_stages; ++i) {
        if (*abort_flag) break;
        const int s = i % NS;
        if (i >= NS && !mbar_wait(bar_empty + 8 * s, ((i / NS) - 1) & 1)) {
          *abort_flag = 1;
          raise_status(p.status, 1);
          break;
        }
        const int cb = i / stages_per_cb, rem = i - cb * stages_per_cb;
        const int t = rem / stages_per_cb_tap, g = rem - t * stages_per_cb_tap;
        const int chunk0 = cb * p.cb_chunks + g * p.ks_chunks;
        const uint32_t dst = smem_u32(b_smem + (size_t)s * p.stage_bytes);
        mbar_expect_tx(bar_full + 8 * s, p.stage_bytes);
        for (int c = 0; c < p.ks_chunks; ++c) {
          const uint8_t* src = p.wt + (((size_t)t * p.n_chunks + chunk0 + c) * p.Kpad + n0) * 16;
          bulk_g2s(dst + (uint32_t)c * p.Nt * 16, src, (uint32_t)p.Nt * 16, bar_full + 8 * s);
        }
        issued = i + 1;
      }
      // never leave with copies in flight: wait (bounded) for the last load of every slot
      for (int s = 0; s < NS; ++s) {
        int last = -1;
        for (int i = s; i < issued; i += NS) last = i;
        if (last >= 0) mbar_wait(bar_full + 8 * s, (last / NS) & 1);
      }
    }
    __syncwarp();
  } else if (warp == 4) {
    // ------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      // instruction descriptor: D format, A/B formats, K-major both, N>>3, M>>4
      const uint32_t idesc = F16 ? ((1u << 4) | ((uint32_t)(p.Nt >> 3) << 17) | ((128u >> 4) << 24))
                                 : ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.Nt >> 3) << 17) |
                                    ((128u >> 4) << 24));
      const uint32_t a_lbo = (uint32_t)p.Rr * 16, b_lbo = (uint32_t)p.Nt * 16;
      bool ok = true;
      int i = 0;
      for (int cb = 0; cb < p.n_cb && ok; ++cb) {
        if (!mbar_wait(bar_aready, cb & 1)) { ok = false; break; }
        tc_fence_after();
        for (int t = 0; t < 9 && ok; ++t) {
          const int ky = t / 3, kx = t % 3;
          int plane, off;
          if (p.stride == 1) { plane = 0; off = ky * p.Wq + kx; }
          else { plane = (ky & 1) * 2 + (kx & 1); off = (ky >> 1) * p.Wq + (kx >> 1); }
          for (int g = 0; g < stages_per_cb_tap; ++g, ++i) {
            const int s = i % NS;
            if (*abort_flag || !mbar_wait(bar_full + 8 * s, (i / NS) & 1)) { ok = false; break; }
            tc_fence_after();
            const uint32_t b_base = smem_u32(b_smem + (size_t)s * p.stage_bytes);
            for (int mt = 0; mt < p.MT; ++mt) {
              for (int j = 0; j < p.ks_chunks / 2; ++j) {
                const uint32_t a_addr = smem_u32(a_smem) + plane * plane_bytes +
                                        (uint32_t)(((g * p.ks_chunks + 2 * j) * p.Rr) + mt * 128 + off) * 16;
                const uint32_t b_addr = b_base + (uint32_t)(2 * j) * p.Nt * 16;
                mma_ss<F16>(tmem_base + (uint32_t)(mt * p.Nt), make_desc(a_addr, a_lbo, 128),
                            make_desc(b_addr, b_lbo, 128), idesc, (i > 0 || j > 0) ? 1u : 0u);
              }
            }
            tc_commit(bar_empty + 8 * s);  // the slot is free once these MMAs have read it
          }
        }
        if (ok && cb + 1 < p.n_cb) tc_commit(bar_afree);  // activation block may be overwritten
      }
      if (!ok) {
        *abort_flag = 1;
        raise_status(p.status, 2);
      }
      tc_commit(bar_accum);  // fires when everything issued so far is complete
    }
    __syncwarp();
  } else {
    // ------------------------------------------------ workers: expand activations, then epilogue
    const int cw_pad = F16 ? 0 : (p.n_chunks / 2);  // 32-bit words covering the padded channels (int8 path)
    for (int cb = 0; cb < p.n_cb; ++cb) {
      if (cb > 0 && !mbar_wait(bar_afree, (cb - 1) & 1)) {
        *abort_flag = 1;
        raise_status(p.status, 3);
      }
      if (!*abort_flag) {
        for (int pl = 0; pl < p.n_planes; ++pl) {
          const int pa = pl >> 1, pb = pl & 1;
          uint8_t* a_plane = a_smem + (size_t)pl * plane_bytes;
          for (int r = tid; r < p.Rr; r += TC_WORKERS) {
            const long long pix = position_to_pixel(p, Q0 + r, pa, pb);
            if (F16) {
              const int ch0 = cb * p.cb_chunks * esz_chunk_ch;
              const __half* src = pix >= 0 ? (const __half*)p.act + (size_t)pix * p.C + ch0 : nullptr;
              const bool vec = pix >= 0 && ((p.C & 7) == 0);
              for (int c = 0; c < p.cb_chunks; ++c) {
                uint4 v = make_uint4(0, 0, 0, 0);
                const int ch = ch0 + c * 8;
                if (vec && ch + 8 <= p.C) {
                  v = __ldg(reinterpret_cast<const uint4*>(src + c * 8));
                } else if (pix >= 0) {
                  __align__(16) __half tmp[8];
#pragma unroll
                  for (int e = 0; e < 8; ++e) tmp[e] = (ch + e < p.C) ? src[c * 8 + e] : __float2half(0.f);
                  v = *reinterpret_cast<uint4*>(tmp);
                }
                *reinterpret_cast<uint4*>(a_plane + ((size_t)c * p.Rr + r) * 16) = v;
              }
            } else {
              const int w0 = cb * (p.cb_chunks / 2);
              const uint32_t* src = pix >= 0 ? (const uint32_t*)p.act + (size_t)pix * p.Cw : nullptr;
              for (int w = 0; w < p.cb_chunks / 2; ++w) {
                const int wg = w0 + w;
                uint4 lo = make_uint4(0, 0, 0, 0), hi = make_uint4(0, 0, 0, 0);
                if (pix >= 0 && wg < p.Cw && wg < cw_pad) {
                  const uint32_t bits = __ldg(src + wg);
                  lo.x = nibble_to_pm1(bits & 15u);
                  lo.y = nibble_to_pm1((bits >> 4) & 15u);
                  lo.z = nibble_to_pm1((bits >> 8) & 15u);
                  lo.w = nibble_to_pm1((bits >> 12) & 15u);
                  hi.x = nibble_to_pm1((bits >> 16) & 15u);
                  hi.y = nibble_to_pm1((bits >> 20) & 15u);
                  hi.z = nibble_to_pm1((bits >> 24) & 15u);
                  hi.w = nibble_to_pm1(bits >> 28);
                  const int left = p.C - wg * 32;  // channels of this word that exist
                  if (left < 32) {
                    const uint32_t vm = (1u << left) - 1u;
                    lo.x &= nibble_to_mask(vm & 15u);
                    lo.y &= nibble_to_mask((vm >> 4) & 15u);
                    lo.z &= nibble_to_mask((vm >> 8) & 15u);
                    lo.w &= nibble_to_mask((vm >> 12) & 15u);
                    hi.x &= nibble_to_mask((vm >> 16) & 15u);
                    hi.y &= nibble_to_mask((vm >> 20) & 15u);
                    hi.z &= nibble_to_mask((vm >> 24) & 15u);
                    hi.w &= nibble_to_mask(vm >> 28);
                  }
                }
                *reinterpret_cast<uint4*>(a_plane + ((size_t)(2 * w) * p.Rr + r) * 16) = lo;
                *reinterpret_cast<uint4*>(a_plane + ((size_t)(2 * w + 1) * p.Rr + r) * 16) = hi;
              }
            }
          }
        }
      }
      fence_proxy_async();      // generic-proxy writes -> visible to the tensor core's reads
      mbar_arrive(bar_aready);
    }

    // ---- epilogue: row m of sub-tile mt lives in TMEM lane m, columns mt*Nt ..
    bool done = mbar_wait(bar_accum, 0);
    if (!done) {
      *abort_flag = 1;
      raise_status(p.status, 4);
    }
    tc_fence_after();
    const bool go = __all_sync(0xffffffffu, done && !*abort_flag);  // warp-uniform: the TMEM loads are .aligned
    if (go) {
      for (int mt = 0; mt < p.MT; ++mt) {
        const long long q = Q0 + mt * 128 + tid;
        long long rg = q / p.Wq;
        const int x = (int)(q - rg * p.Wq);
        const long long n = rg / p.Hq;
        const int y = (int)(rg - n * p.Hq);
        const bool valid = (n < p.N) && (y < p.Ho) && (x < p.Wo);
        const size_t obase = (((size_t)n * p.Ho + y) * p.Wo + x) * p.K;
        for (int c0 = 0; c0 < p.Nt; c0 += 16) {
          uint32_t v[16];
          // all lanes of the warp take part in the load; only valid rows store
          tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(mt * p.Nt + c0), v);
          tmem_ld_wait();
          const int co0 = n0 + c0;
          if (!valid || co0 >= p.K) continue;
          const bool vec = ((p.K & 3) == 0) && (co0 + 16 <= p.K);
          if (p.out_i32) {
            int32_t* o = (int32_t*)p.out + obase + co0;
            if (vec) {
#pragma unroll
              for (int e = 0; e < 4; ++e)
                reinterpret_cast<int4*>(o)[e] = make_int4((int)v[4 * e], (int)v[4 * e + 1], (int)v[4 * e + 2],
                                                          (int)v[4 * e + 3]);
            } else {
              for (int e = 0; e < 16 && co0 + e < p.K; ++e) o[e] = (int)v[e];
            }
          } else {
            float* o = (float*)p.out + obase + co0;
            float f[16];
#pragma unroll
            for (int e = 0; e < 16; ++e) {
              const float al = (co0 + e < p.K) ? __ldg(p.alpha + co0 + e) : 0.f;
              const float acc = F16 ? __uint_as_float(v[e]) : (float)(int)v[e];
              f[e] = __fmul_rn(acc, al);
            }
            if (vec) {
#pragma unroll
              for (int e = 0; e < 4; ++e)
                reinterpret_cast<float4*>(o)[e] = make_float4(f[4 * e], f[4 * e + 1], f[4 * e + 2], f[4 * e + 3]);
            } else {
              for (int e = 0; e < 16 && co0 + e < p.K; ++e) o[e] = f[e];
            }
          }
        }
      }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols)
                 : "memory");
  }
}

// ------------------------------------------------------------ create-time operand
// wt[tap][chunk][Kpad][16 B]: chunk = 16 (int8) or 8 (fp16) consecutive input channels
template <bool F16>
__global__ void tc_expand_weights_kernel(const uint32_t* __restrict__ wplanes, uint8_t* __restrict__ wt, int C, int K,
                                         int Cw, int Kpad, int n_chunks) {
  long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  long long total = (long long)9 * n_chunks * Kpad;
  if (i >= total) return;
  int co = (int)(i % Kpad);
  long long r = i / Kpad;
  int chunk = (int)(r % n_chunks), t = (int)(r / n_chunks);
  const int cpc = F16 ? 8 : 16;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (co < K) {
    int ch0 = chunk * cpc;
    int wd = ch0 >> 5, sh = ch0 & 31;
    uint32_t bits = wd < Cw ? wplanes[((size_t)t * Cw + wd) * K + co] >> sh : 0u;
    if (F16) {
      __align__(16) uint16_t h[8];
#pragma unroll
      for (int e = 0; e < 8; ++e) h[e] = (ch0 + e < C) ? (((bits >> e) & 1u) ? 0x3c00 : 0xbc00) : 0;  // +1.0 / -1.0
      v = *reinterpret_cast<uint4*>(h);
    } else {
      __align__(16) int8_t b[16];
#pragma unroll
      for (int e = 0; e < 16; ++e) b[e] = (ch0 + e < C) ? (((bits >> e) & 1u) ? 1 : -1) : 0;
      v = *reinterpret_cast<uint4*>(b);
    }
  }
  reinterpret_cast<uint4*>(wt)[i] = v;
}

static int round_up(int v, int m) { return (v + m - 1) / m * m; }

size_t tc_weight_bytes(const Geom& g, int act_type, int* Kpad, int* Cpad) {
  const bool f16 = act_type == SNN_ACT_F16;
  *Kpad = g.K <= 256 ? round_up(g.K, 16) : round_up(g.K, 256);
  *Cpad = round_up(g.C, f16 ? 16 : 32);
  const int n_chunks = *Cpad / (f16 ? 8 : 16);
  return (size_t)9 * n_chunks * (*Kpad) * 16;
}

cudaError_t tc_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched) {
  const bool f16 = act_type == SNN_ACT_F16;
  const int n_chunks = L.Cpad / (f16 ? 8 : 16);
  long long total = (long long)9 * n_chunks * L.Kpad;
  unsigned blocks = (unsigned)((total + 255) / 256);
  if (f16)
    tc_expand_weights_kernel<true><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.w16, g.C, g.K, g.Cw, L.Kpad, n_chunks);
  else
    tc_expand_weights_kernel<false><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.w8, g.C, g.K, g.Cw, L.Kpad, n_chunks);
  *launched += 1;
  return cudaGetLastError();
}

// ------------------------------------------------------------------ launch plan
struct TcPlan {
  TcParams p;
  size_t smem;
  dim3 grid;
  bool ok;
};

static int env_int(const char* name, int dflt) {
  const char* v = getenv(name);
  return v ? atoi(v) : dflt;
}

static TcPlan make_plan(const Geom& g, int act_type) {
  TcPlan pl{};
  TcParams& p = pl.p;
  const bool f16 = act_type == SNN_ACT_F16;
  pl.ok = false;
  if (g.N < 1) return pl;
  int Kpad, Cpad;
  tc_weight_bytes(g, act_type, &Kpad, &Cpad);
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K; p.Cw = g.Cw;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  p.Kpad = Kpad;
  p.n_chunks = Cpad / (f16 ? 8 : 16);
  if (g.stride == 1) {
    p.Hq = g.H + g.pad; p.Wq = g.W + g.pad; p.n_planes = 1; p.halo = 2 * p.Wq + 2;
  } else {
    p.Hq = g.Ho + 1; p.Wq = g.Wo + 1; p.n_planes = 4; p.halo = p.Wq + 1;
  }
  p.Qtot = (long long)g.N * p.Hq * p.Wq;
  const long long mtiles = (p.Qtot + 127) / 128;
  // channels per CTA
  int Nt = Kpad <= 256 ? Kpad : 256;
  int forced_nt = env_int("SNN_TC_NT", 0);
  if (forced_nt >= 16 && forced_nt <= 256 && forced_nt % 16 == 0 && Kpad % forced_nt == 0) Nt = forced_nt;
  else
    while (Nt > 64 && Nt % 32 == 0 && mtiles * (Kpad / Nt) < 148) Nt /= 2;
  p.Nt = Nt;
  const int ntiles = Kpad / Nt;
  // M sub-tiles per CTA: the largest that keeps the SMs evenly loaded
  int MT = 1;
  {
    double best = -1.0;
    for (int mt = 1; mt <= 4; mt *= 2) {
      if (mt * Nt > 256) break;
      long long ctas = ((mtiles + mt - 1) / mt) * ntiles;
      long long waves = (ctas + 295) / 296;
      double eff = (double)ctas / (double)(waves * 296);
      if (ctas < 148) eff = (double)ctas / 148.0 * 0.5;
      eff += 0.02 * mt;  // a larger tile stages less halo and re-reads fewer weights
      if (eff > best) { best = eff; MT = mt; }
    }
  }
  int forced_mt = env_int("SNN_TC_MT", 0);
  if ((forced_mt == 1 || forced_mt == 2 || forced_mt == 4) && forced_mt * Nt <= 512) MT = forced_mt;
  p.MT = MT;
  p.Rr = 128 * MT + p.halo;
  uint32_t cols = 32;
  while (cols < (uint32_t)(MT * Nt)) cols *= 2;
  p.tmem_cols = cols;
  // weight stage: 64 (int8) / 32 (fp16) channels = 4 chunks, or the whole padded C if smaller
  p.ks_chunks = p.n_chunks < 4 ? p.n_chunks : 4;
  if (p.n_chunks % p.ks_chunks) p.ks_chunks = 2;
  p.stage_bytes = (uint32_t)p.ks_chunks * Nt * 16;
  // channel block: as many stages' worth of chunks as fit the activation budget
  const size_t budget = 200 * 1024 - (size_t)NS * p.stage_bytes - 256;
  const size_t per_chunk = (size_t)p.n_planes * p.Rr * 16;
  int cb_chunks = p.n_chunks;
  if ((size_t)cb_chunks * per_chunk > budget) {
    cb_chunks = (int)(budget / per_chunk) / p.ks_chunks * p.ks_chunks;
    if (cb_chunks < p.ks_chunks) return pl;
    // keep the blocks equal: the largest divisor of n_chunks not above the budget
    while (cb_chunks > p.ks_chunks && (p.n_chunks % cb_chunks)) cb_chunks -= p.ks_chunks;
    if (p.n_chunks % cb_chunks) return pl;
  }
  p.cb_chunks = cb_chunks;
  p.n_cb = p.n_chunks / cb_chunks;
  p.a_bytes = (uint32_t)((size_t)cb_chunks * per_chunk);
  p.a_bytes = (p.a_bytes + 127) & ~127u;
  pl.smem = (size_t)p.a_bytes + (size_t)NS * p.stage_bytes + 256;
  if (pl.smem > 227 * 1024) return pl;
  if ((size_t)p.a_bytes + (size_t)NS * p.stage_bytes >= (1u << 18)) return pl;  // descriptor address range
  if ((uint32_t)p.Rr * 16 >= (1u << 18)) return pl;                                 // LBO field range
  long long gx = (mtiles + MT - 1) / MT;
  if (gx > 0x7fffffffLL) return pl;
  pl.grid = dim3((unsigned)gx, (unsigned)ntiles);
  pl.ok = true;
  return pl;
}

bool tc_supported(const Geom& g, int act_type) {
  if (env_int("SNN_TC_DISABLE", 0)) return false;
  Geom gg = g;
  if (gg.N < 1) gg.N = 1;
  return make_plan(gg, act_type).ok;
}

cudaError_t tc_forward(const LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched,
                       int* status_host) {
  TcPlan pl = make_plan(g, act_type);
  if (!pl.ok) return cudaErrorInvalidConfiguration;
  const bool f16 = act_type == SNN_ACT_F16;
  TcParams& p = pl.p;
  p.act = l.act;
  p.wt = f16 ? (const uint8_t*)L.w16 : (const uint8_t*)L.w8;
  p.alpha = L.alpha;
  p.out = l.out;
  p.out_i32 = l.out_i32;
  int* status_dev = nullptr;
  cudaError_t e = cudaHostGetDevicePointer((void**)&status_dev, status_host, 0);
  if (e != cudaSuccess) return e;
  p.status = status_dev;
  if (f16) {
    e = cudaFuncSetAttribute(tc_conv_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    tc_conv_kernel<true><<<pl.grid, TC_THREADS, pl.smem, l.stream>>>(p);
  } else {
    e = cudaFuncSetAttribute(tc_conv_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);
    if (e != cudaSuccess) return e;
    tc_conv_kernel<false><<<pl.grid, TC_THREADS, pl.smem, l.stream>>>(p);
  }
  *launched += 1;
  return cudaGetLastError();
}

}  // namespace snn
