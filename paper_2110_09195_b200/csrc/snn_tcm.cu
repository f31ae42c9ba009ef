// Decoded-weight path on the tensor cores, channel-major accumulators.
//
// The same implicit GEMM as the position-major kernel (Sec. 3: every 3x3 kernel of
// +/-1 weights decoded from its codebook index, zero padding contributes 0), with
// the operands swapped:
//   M = 128 output channels, their +/-1 weights in TENSOR MEMORY (the A operand),
//   N = a tile of Np consecutive positions of the padded, flattened input, staged in
//       shared memory as  [plane][16-byte channel chunk][row][16 B]  (the B operand),
//   K = (channel block, tap, 32 int8 / 16 fp16 channels).
// Why: one MMA of M=128 reads its shared-memory operands at 32*(128 + N) bytes per
// N/2 cycles, which for N <= 128 is all of the 128 B/clk an SM's shared memory
// delivers; with the weights also arriving there by bulk copy, the position-major
// kernel is bound by shared-memory bandwidth, not by the tensor core.  Here the
// weights never touch shared memory (global -> registers -> tcgen05.st -> TMEM), the
// only shared-memory operand is the activation tile (32*Np bytes per MMA), and tap
// (ky, kx) is again the same staged unit read from a start address shifted by
// ky*pitch + kx rows.  The accumulator holds channels in TMEM lanes and positions in
// columns, so a draining thread owns one channel; 16-position chunks are transposed
// through a small shared-memory tile so that a store instruction writes four full
// 128-byte lines of the [N][Ho][Wo][K] output.
//
//      warp 0        allocates tensor memory
//      warp 1        one thread issues tcgen05.mma (A from TMEM, B from shared memory)
//      warps 2-9     drain the accumulators: TMEM -> registers -> transposition tile ->
//                    alpha -> line stores, for tile i while the MMAs of tile i+1 run
//      warps 10-17   expanders: packed bits -> +1/-1 bytes into the activation ring
//      warps 18-25   weight loaders, two per TMEM lane quarter, each filling half of a
//                    stage of eight K steps: 32 B per thread and K step from global
//                    memory, one tcgen05.st per half stage into a ring of TMEM columns
// When all K steps of a channel tile fit the ring they are loaded once and kept.
// Every wait is bounded; one that runs out raises a status word the host reads, and
// the CTA still frees its tensor memory and returns.
#include "snn_tc_common.cuh"

namespace snn {

namespace {

constexpr int CM_EPI_WARPS = 8, CM_EXP_WARPS = 8, CM_LOAD_WARPS = 8;
constexpr int CM_EXP_THREADS = 32 * CM_EXP_WARPS;
constexpr int CM_FIRST_EXP = 2 + CM_EPI_WARPS, CM_FIRST_LOAD = CM_FIRST_EXP + CM_EXP_WARPS;
constexpr int CM_THREADS = 32 * (CM_FIRST_LOAD + CM_LOAD_WARPS);
constexpr int CM_EXP_ROWS = 3;        // rows of a unit one expander thread loads together
constexpr int CM_WST = 8;             // K steps per weight stage (8 TMEM columns each); a loader warp fills half a stage
constexpr int CM_RING_MAX = 8;        // most weight stages in the ring
constexpr int CM_EPI_STAGE = 2048;    // bytes of an epilogue warp's transposition tile: 16 positions x 32 channels
constexpr int CM_NA_MAX = 8;          // most activation units in flight
constexpr size_t kCmTail = 512;

struct CmParams {
  const void* act;        // uint32 [N][H][W][Cw] or half [N][H][W][C]
  const uint8_t* wa;      // [channel tile][K step][16-byte half][128 channels][16 B]
  const float* alpha;
  void* out;
  int* status;
  int out_i32, act_vec;
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int Hq, Wq;             // rows per image / row pitch of the flattened position space
  FastDiv dWq, dHq, dCt;  // exact division by Wq, Hq and the number of channel tiles
  int n_planes, halo;
  int Np, Rr;             // positions per tile; staged rows per plane = Np + halo
  int n_mgroups, n_cotiles, total_tiles;
  int cb_chunks, n_cb, kpt;
  int KS;                 // K steps per tile = 9 * n_cb * kpt, ordered (block, tap, step)
  int spc;                // weight stages per channel block = ceil(9 * kpt / 4); the last may be short
  int n_wstages;          // weight stages per tile = n_cb * spc
  int NW;                 // stages in the TMEM ring
  int w_resident;         // all stages of the CTA's channel tile stay in the ring
  int NA, n_acc;
  long long Qtot;
  uint32_t ring_col0;     // first TMEM column of the weight ring
  uint32_t a_unit_bytes, off_pix, off_epi, off_tail;
};

__device__ __forceinline__ int cm_input_pixel(const CmParams& p, uint32_t q, int pa, int pb) {
  if ((long long)q >= p.Qtot) return -1;
  const uint32_t rg = fdiv(q, p.dWq);
  const int j = (int)(q - rg * (uint32_t)p.Wq);
  const uint32_t n = fdiv(rg, p.dHq);
  const int i = (int)(rg - n * (uint32_t)p.Hq);
  if ((int)n >= p.N) return -1;
  const int r = p.stride * i + pa - p.pad, c = p.stride * j + pb - p.pad;
  if (r < 0 || r >= p.H || c < 0 || c >= p.W) return -1;
  return ((int)n * p.H + r) * p.W + c;
}

// flattened position -> output pixel (n*Ho + y)*Wo + x, or -1 when it is not an output
__device__ __forceinline__ int cm_output_pixel(const CmParams& p, uint32_t q) {
  if ((long long)q >= p.Qtot) return -1;
  const uint32_t rg = fdiv(q, p.dWq);
  const int x = (int)(q - rg * (uint32_t)p.Wq);
  const uint32_t n = fdiv(rg, p.dHq);
  const int y = (int)(rg - n * (uint32_t)p.Hq);
  if ((int)n >= p.N || y >= p.Ho || x >= p.Wo) return -1;
  return ((int)n * p.Ho + y) * p.Wo + x;
}

// D[tmem] (+)= A[tmem] * B[smem]
template <bool F16>
__device__ __forceinline__ void mma_ts(uint32_t d_tmem, uint32_t a_tmem, uint32_t b_lo, uint32_t b_hi, uint32_t idesc,
                                       uint32_t accumulate) {
  if (F16) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
  } else {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\tsetp.ne.b32 p, %5, 0;\n\tmov.b64 db, {%2, %3};\n\t"
        "tcgen05.mma.cta_group::1.kind::i8 [%0], [%1], db, %4, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "r"(b_lo), "r"(b_hi), "r"(idesc), "r"(accumulate)
        : "memory");
  }
}

// 32 registers of this thread -> 32 consecutive TMEM columns of its lane
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
      "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
      "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]),
      "r"(v[19]), "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]),
      "r"(v[28]), "r"(v[29]), "r"(v[30]), "r"(v[31])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

}  // namespace

// KPT = MMAs per tap and channel block (cb_chunks / 2), a compile-time constant so that the
// issuing thread runs straight-line code.
template <bool F16, int KPT>
__global__ void __launch_bounds__(CM_THREADS, 1) cm_conv_kernel(const CmParams p) {
  extern __shared__ __align__(128) uint8_t smem[];
  uint8_t* a_smem = smem;                                      // [NA activation units]
  int* pix_tab = reinterpret_cast<int*>(smem + p.off_pix);    // [plane][row] input pixel of a staged row
  uint8_t* epi_smem = smem + p.off_epi;                       // [epilogue warp][16 positions][32 channels]
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_tail);
  // barriers: w_full[8] (+4 unused) w_empty[8] (+4 unused) a_full[8] a_empty[8] acc_full[2] acc_empty[2]
  const uint32_t bar_wfull = smem_u32(bars), bar_wempty = smem_u32(bars + 12);
  const uint32_t bar_afull = smem_u32(bars + 24), bar_aempty = smem_u32(bars + 32);
  const uint32_t bar_accfull = smem_u32(bars + 40), bar_accempty = smem_u32(bars + 42);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 44);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* tap_units = tmem_slot + 3;  // [9] row offset of every tap inside a unit

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NA = p.NA, NW = p.NW;

  if (tid < 44) {
    uint32_t count = 1;
    if (tid < 12) count = CM_LOAD_WARPS;              // w_full: every loader warp arrives
    if (tid >= 24 && tid < 32) count = CM_EXP_THREADS;  // a_full: every expander thread arrives
    if (tid >= 42) count = CM_EPI_WARPS;              // acc_empty: one arrival per epilogue warp
    mbar_init(smem_u32(bars + tid), count);
  }
  if (tid == 64) *abort_flag = 0;
  if (tid >= 96 && tid < 105) {
    const int t = tid - 96, ky = t / 3, kx = t % 3;
    uint32_t u;
    if (p.stride == 1) u = (uint32_t)(ky * p.Wq + kx);
    else u = (uint32_t)((ky & 1) * 2 + (kx & 1)) * (uint32_t)(p.cb_chunks * p.Rr) +
             (uint32_t)((ky >> 1) * p.Wq + (kx >> 1));
    tap_units[t] = u;
  }
  if (warp == 0) {
    // the whole tensor memory: accumulators in the first columns, the weight ring behind them
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp >= CM_FIRST_EXP && warp < CM_FIRST_LOAD) {
    // The expanders' table for their first tile (input pixel of every staged row, -1 = padding)
    // depends on nothing but the parameters: it is worked out here, beside the set-up and before
    // the wait for the previous kernel.  A thread reads back only entries it wrote itself.
    const int et0 = tid - CM_FIRST_EXP * 32;
    const uint32_t Q00 = (uint32_t)((int)blockIdx.x / p.n_cotiles) * (uint32_t)p.Np;
    // (plane, row) pairs form one index space f = plane*Rr + row, dealt to the threads at a stride of
    // the expander count, here and in the expanders' loops
    for (int f = et0; f < p.n_planes * p.Rr; f += CM_EXP_THREADS) {
      const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
      pix_tab[f] = cm_input_pixel(p, Q00 + (uint32_t)(f - pl * p.Rr), pl >> 1, pl & 1);
    }
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_launch();

  const int my_tiles = (p.total_tiles - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;

  if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    // The whole warp walks the loops and waits together, so that every address and descriptor is
    // a warp-uniform value; one elected lane issues the MMAs and the commits.
    {
      const bool leader = elect_one();
      const uint32_t idesc = F16 ? ((1u << 4) | ((uint32_t)(p.Np >> 3) << 17) | ((128u >> 4) << 24))
                                 : ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.Np >> 3) << 17) |
                                    ((128u >> 4) << 24));
      const uint64_t b_desc0 = make_desc(smem_u32(a_smem), (uint32_t)p.Rr * 16, 128);
      const uint32_t b_lo0 = (uint32_t)b_desc0, b_hi = (uint32_t)(b_desc0 >> 32);
      const uint32_t unit_units = p.a_unit_bytes >> 4;
      const uint32_t a_step = 2u * (uint32_t)p.Rr;  // two chunks per MMA
      const uint32_t ring = tmem_base + p.ring_col0;
      uint32_t tapu[9];
#pragma unroll
      for (int t = 0; t < 9; ++t) tapu[t] = tap_units[t];
      bool ok = true;
      int a_slot = 0, w_slot = 0, acc_slot = 0;
      uint32_t a_phase = 0, w_phase = 0, acc_phase = 1;
      for (int it = 0; it < my_tiles && ok; ++it) {
        if (it >= p.n_acc) {
          if (!mbar_wait_backoff(bar_accempty + 8 * acc_slot, acc_phase, 20)) { ok = false; break; }
          tc_fence_after();
        }
        const uint32_t d0 = tmem_base + (uint32_t)(acc_slot * p.Np);
        uint32_t acc = 0;
        const bool wait_w = !(p.w_resident && it > 0);
        if (p.w_resident) { w_slot = 0; w_phase = 0; }
        for (int cb = 0; cb < p.n_cb && ok; ++cb) {
          if (!mbar_wait_backoff(bar_afull + 8 * a_slot, a_phase, 20)) { ok = false; break; }
          tc_fence_after();
          const uint32_t unit = b_lo0 + (uint32_t)a_slot * unit_units;
          uint32_t wbase = 0;
          // K step j = tap*KPT + k of this block sits in column group j%4 of weight stage j/4
#pragma unroll
          for (int t = 0; t < 9; ++t) {
            const uint32_t bt = unit + tapu[t];
#pragma unroll
            for (int k = 0; k < KPT; ++k) {
              const int j = t * KPT + k;
              if (j % CM_WST == 0) {
                if (wait_w && ok) {
                  if (!mbar_wait_backoff(bar_wfull + 8 * w_slot, w_phase, 20)) ok = false;
                  tc_fence_after();
                }
                wbase = ring + (uint32_t)(w_slot * (8 * CM_WST));
              }
              if (leader)
                mma_ts<F16>(d0, wbase + (uint32_t)((j % CM_WST) * 8), bt + (uint32_t)k * a_step, b_hi, idesc, acc);
              acc = 1;
              if (j % CM_WST == CM_WST - 1 || j == 9 * KPT - 1) {
                if (!p.w_resident && leader) tc_commit(bar_wempty + 8 * w_slot);  // the ring stage may be overwritten
                if (++w_slot == NW) { w_slot = 0; w_phase ^= 1u; }
              }
            }
          }
          if (leader) tc_commit(bar_aempty + 8 * a_slot);
          if (++a_slot == NA) { a_slot = 0; a_phase ^= 1u; }
        }
        if (leader) tc_commit(bar_accfull + 8 * acc_slot);
        if (++acc_slot == p.n_acc) { acc_slot = 0; acc_phase ^= 1u; }
      }
      if (!ok && leader) {
        *abort_flag = 1;
        raise_status(p.status, 3);
      }
    }
    __syncwarp();
  } else if (warp >= 2 && warp < CM_FIRST_LOAD) {
    // ------------------------------------------------ drain warps (2-9) and expanders (10-17)
    grid_dep_wait();  // activations may come from, and the output may still be read by, the previous kernel
    const int et = tid - CM_FIRST_EXP * 32;  // rank among the expander threads
    int a_slot = 0, a_done = 0;
    uint32_t a_phase = 1;  // parity of the previous use of a slot (valid from the second lap)
    const int nstep = p.cb_chunks / 2;
    // Draining: warp w reads TMEM lanes 32*(w%4).. = 32 channels (one per thread); the warps of a lane
    // quarter take the 16-position chunks in turn.  A chunk is transposed through a 2 KB tile of
    // shared memory (this kernel leaves half of the shared-memory bandwidth unused), so that a
    // thread then holds four consecutive channels of one position and a store instruction writes
    // four full 128-byte lines: the store path takes as long for a 4-byte-per-thread instruction
    // as for a 16-byte one.
    const int qtr = warp & 3, sub = (warp - 2) >> 2;
    const int nchunk = p.Np >> 4;
    uint8_t* stg = epi_smem + (size_t)(warp - 2) * CM_EPI_STAGE;
    const int rpos = lane >> 3, cgrp = lane & 7;  // when storing: position (mod 4) and channel group of this lane
    int acc_slot = 0;
    uint32_t acc_phase = 0;
    auto expand_tile = [&](int it) -> bool {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      const int mg = (int)fdiv((uint32_t)tile, p.dCt);
      const uint32_t Q0 = (uint32_t)mg * (uint32_t)p.Np;
      bool stop = false;
      if (it > 0)  // the first tile's table was made during set-up
        for (int f = et; f < p.n_planes * p.Rr; f += CM_EXP_THREADS) {
          const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
          pix_tab[f] = cm_input_pixel(p, Q0 + (uint32_t)(f - pl * p.Rr), pl >> 1, pl & 1);
        }
      for (int cb = 0; cb < p.n_cb; ++cb) {
        if (a_done >= NA) {
          // every warp polls for itself (one lane, sleeping between attempts): no wait in this
          // kernel depends on another warp having taken the same exit
          int okf = 1;
          if (lane == 0) okf = (!*abort_flag && mbar_wait_backoff(bar_aempty + 8 * a_slot, a_phase, 64)) ? 1 : 0;
          okf = __shfl_sync(0xffffffffu, okf, 0);
          if (!okf) {
            if (lane == 0 && !*abort_flag) {
              *abort_flag = 1;
              raise_status(p.status, 1);
            }
            stop = true;
            break;
          }
        }
        uint8_t* unit = a_smem + (size_t)a_slot * p.a_unit_bytes;
        // A thread has rows of several planes in flight together: a stride-2 unit (four short
        // planes) costs one round trip to memory instead of four.
        const int all_rows = p.n_planes * p.Rr;
        {
          for (int rb = 0; rb < all_rows; rb += CM_EXP_ROWS * CM_EXP_THREADS) {
            int pix[CM_EXP_ROWS];  // -1 padding, -2 past the unit
            uint8_t* dst[CM_EXP_ROWS];  // where the row starts in its plane (chunk 0)
#pragma unroll
            for (int j = 0; j < CM_EXP_ROWS; ++j) {
              const int f = rb + et + j * CM_EXP_THREADS;
              pix[j] = f < all_rows ? pix_tab[f] : -2;
              const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
              dst[j] = unit + ((size_t)pl * p.cb_chunks * p.Rr + (size_t)(f - pl * p.Rr)) * 16;
            }
            if (F16) {
              for (int c0 = 0; c0 < p.cb_chunks; c0 += 2) {
                uint4 v[CM_EXP_ROWS][2];
#pragma unroll
                for (int j = 0; j < CM_EXP_ROWS; ++j) {
#pragma unroll
                  for (int k = 0; k < 2; ++k) {
                    v[j][k] = make_uint4(0, 0, 0, 0);
                    const int ch = (cb * p.cb_chunks + c0 + k) * 8;
                    if (pix[j] >= 0 && ch < p.C) {
                      const __half* src = (const __half*)p.act + wide_mul((uint32_t)pix[j], (uint32_t)p.C) + ch;
                      if (p.act_vec) {
                        v[j][k] = __ldg(reinterpret_cast<const uint4*>(src));
                      } else {
                        uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                          if (ch + e < p.C) w[e >> 1] |= (uint32_t)__half_as_ushort(src[e]) << (16 * (e & 1));
                        v[j][k] = make_uint4(w[0], w[1], w[2], w[3]);
                      }
                    }
                  }
                }
#pragma unroll
                for (int j = 0; j < CM_EXP_ROWS; ++j) {
                  if (pix[j] != -2) {
                    *reinterpret_cast<uint4*>(dst[j] + (size_t)c0 * p.Rr * 16) = v[j][0];
                    *reinterpret_cast<uint4*>(dst[j] + (size_t)(c0 + 1) * p.Rr * 16) = v[j][1];
                  }
                }
              }
            } else {
              const int w0 = cb * nstep;
              uint32_t bits[CM_EXP_ROWS][4];
#pragma unroll
              for (int j = 0; j < CM_EXP_ROWS; ++j) {
                bits[j][0] = bits[j][1] = bits[j][2] = bits[j][3] = 0;
                if (pix[j] >= 0 && w0 < p.Cw) {
                  const uint32_t* src = (const uint32_t*)p.act + wide_mul((uint32_t)pix[j], (uint32_t)p.Cw) + w0;
                  if (p.act_vec && nstep == 4) {
                    const uint4 t = __ldg(reinterpret_cast<const uint4*>(src));
                    bits[j][0] = t.x; bits[j][1] = t.y; bits[j][2] = t.z; bits[j][3] = t.w;
                  } else if (p.act_vec && nstep == 2) {
                    const uint2 t = __ldg(reinterpret_cast<const uint2*>(src));
                    bits[j][0] = t.x; bits[j][1] = t.y;
                  } else {
#pragma unroll
                    for (int k = 0; k < 4; ++k)
                      if (k < nstep && w0 + k < p.Cw) bits[j][k] = __ldg(src + k);
                  }
                }
              }
#pragma unroll
              for (int j = 0; j < CM_EXP_ROWS; ++j) {
                if (pix[j] != -2) {
#pragma unroll
                  for (int k = 0; k < 4; ++k) {
                    if (k < nstep) {
                      uint4 lo, hi;
                      expand_word(bits[j][k], p.C - (w0 + k) * 32, pix[j] >= 0 && w0 + k < p.Cw, lo, hi);
                      *reinterpret_cast<uint4*>(dst[j] + (size_t)(2 * k) * p.Rr * 16) = lo;
                      *reinterpret_cast<uint4*>(dst[j] + (size_t)(2 * k + 1) * p.Rr * 16) = hi;
                    }
                  }
                }
              }
            }
          }
        }
        fence_proxy_async();  // generic-proxy writes -> visible to the tensor core's reads
        mbar_arrive(bar_afull + 8 * a_slot);
        ++a_done;
        if (++a_slot == NA) { a_slot = 0; a_phase ^= 1u; }
      }
      return !stop;
    };
    auto drain_tile = [&](int it) -> bool {
      const int tile = (int)blockIdx.x + it * (int)gridDim.x;
      const int mg = (int)fdiv((uint32_t)tile, p.dCt), ct = tile - mg * p.n_cotiles;
      const uint32_t Q0 = (uint32_t)mg * (uint32_t)p.Np;
      const int co4 = ct * 128 + qtr * 32 + cgrp * 4;  // first of the four channels this lane stores
      float al[4] = {0.f, 0.f, 0.f, 0.f};
      if (!p.out_i32) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (co4 + e < p.K) al[e] = __ldg(p.alpha + co4 + e);
      }
      int okw = 1;
      if (lane == 0) okw = (!*abort_flag && mbar_wait_backoff(bar_accfull + 8 * acc_slot, acc_phase, 100)) ? 1 : 0;
      okw = __shfl_sync(0xffffffffu, okw, 0);
      if (!okw) {
        if (lane == 0 && !*abort_flag) {
          *abort_flag = 1;
          raise_status(p.status, 4);
        }
        return false;
      }
      tc_fence_after();
      const uint32_t d0 = tmem_base + (uint32_t)(acc_slot * p.Np) + ((uint32_t)(qtr * 32) << 16);
      uint32_t* out32 = reinterpret_cast<uint32_t*>(p.out);  // int32 and fp32 outputs share the layout
      const bool vec = (p.K & 3) == 0;  // groups of 4 channels exist together and are 16-byte aligned
      uint32_t v[16];
      if (sub < nchunk) tmem_ld16(d0 + (uint32_t)(sub * 16), v);
#pragma unroll 1
      for (int c = sub; c < nchunk; c += CM_EPI_WARPS / 4) {
        const int mypix = cm_output_pixel(p, Q0 + (uint32_t)(c * 16 + (lane & 15)));
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) *reinterpret_cast<uint32_t*>(stg + j * 128 + lane * 4) = v[j];
        __syncwarp();
        if (c + CM_EPI_WARPS / 4 < nchunk) tmem_ld16(d0 + (uint32_t)((c + CM_EPI_WARPS / 4) * 16), v);  // flies while this chunk is stored
        uint4 w[4];
        int pj[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          w[r] = *reinterpret_cast<const uint4*>(stg + (r * 4 + rpos) * 128 + cgrp * 16);
          pj[r] = __shfl_sync(0xffffffffu, mypix, r * 4 + rpos);
        }
        if (!p.out_i32) {
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            w[r].x = __float_as_uint(__fmul_rn(F16 ? __uint_as_float(w[r].x) : small_int_to_float(w[r].x), al[0]));
            w[r].y = __float_as_uint(__fmul_rn(F16 ? __uint_as_float(w[r].y) : small_int_to_float(w[r].y), al[1]));
            w[r].z = __float_as_uint(__fmul_rn(F16 ? __uint_as_float(w[r].z) : small_int_to_float(w[r].z), al[2]));
            w[r].w = __float_as_uint(__fmul_rn(F16 ? __uint_as_float(w[r].w) : small_int_to_float(w[r].w), al[3]));
          }
        }
        if (vec) {
#pragma unroll
          for (int r = 0; r < 4; ++r)
            if (pj[r] >= 0 && co4 < p.K) *reinterpret_cast<uint4*>(out32 + wide_mul((uint32_t)pj[r], (uint32_t)p.K) + co4) = w[r];
        } else {
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            if (pj[r] >= 0) {
              uint32_t* o = out32 + wide_mul((uint32_t)pj[r], (uint32_t)p.K) + co4;
              if (co4 + 0 < p.K) o[0] = w[r].x;
              if (co4 + 1 < p.K) o[1] = w[r].y;
              if (co4 + 2 < p.K) o[2] = w[r].z;
              if (co4 + 3 < p.K) o[3] = w[r].w;
            }
          }
        }
        __syncwarp();  // the tile is rewritten by the next chunk
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_accempty + 8 * acc_slot);
      if (++acc_slot == p.n_acc) { acc_slot = 0; acc_phase ^= 1u; }
      return true;
    };
    if (warp < CM_FIRST_EXP) {
      for (int it = 0; it < my_tiles; ++it)
        if (!drain_tile(it)) break;
    } else {
      for (int it = 0; it < my_tiles; ++it)
        if (!expand_tile(it)) break;
    }
  } else if (warp >= CM_FIRST_LOAD) {
    // ------------------------------------------------ weight loaders
    // The weights are constants of the layer, so there is no wait for the previous kernel.
    const int lw = warp - CM_FIRST_LOAD;
    const int qtr = warp & 3, pair = lw >> 2;      // lane quarter this warp may write; which half of a stage it fills
    const int row = qtr * 32 + lane;               // channel inside the tile
    const int per_cb = 9 * p.kpt;
    const long long n_stages = p.w_resident ? (long long)p.n_wstages : (long long)my_tiles * p.n_wstages;
    uint32_t v[32];
    // Position of the next stage to load: channel tile of the CTA's current tile, channel block,
    // stage inside the block; kept as counters, because divisions by run-time values are slow.
    int ld_ct = (int)blockIdx.x % p.n_cotiles, ld_cb = 0, ld_si = 0;
    const int ct_step = (int)gridDim.x % p.n_cotiles;  // 0 when the grid is a multiple of the channel tiles
    // this warp's half of the next stage -> registers; returns the number of K steps in it (<= 0: none)
    auto load_half = [&]() -> int {
      const int ct = ld_ct, cb = ld_cb, si = ld_si;
      if (++ld_si == p.spc) {
        ld_si = 0;
        if (++ld_cb == p.n_cb) {
          ld_cb = 0;
          ld_ct += ct_step;
          if (ld_ct >= p.n_cotiles) ld_ct -= p.n_cotiles;
        }
      }
      const int first = si * CM_WST + pair * 4;   // first K step of the half inside the channel block
      const int nks = min(4, per_cb - first);
      // a warp reads 512 contiguous bytes per instruction: the two halves of a K step's rows are stored apart
      const uint8_t* src = p.wa + ((size_t)ct * p.KS + (size_t)cb * per_cb + first) * 4096 + (size_t)row * 16;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        uint4 x = make_uint4(0, 0, 0, 0), y = x;
        if (j < nks) {
          x = __ldg(reinterpret_cast<const uint4*>(src + (size_t)j * 4096));
          y = __ldg(reinterpret_cast<const uint4*>(src + (size_t)j * 4096 + 2048));
        }
        v[8 * j + 0] = x.x; v[8 * j + 1] = x.y; v[8 * j + 2] = x.z; v[8 * j + 3] = x.w;
        v[8 * j + 4] = y.x; v[8 * j + 5] = y.y; v[8 * j + 6] = y.z; v[8 * j + 7] = y.w;
      }
      return nks;
    };
    int nks = n_stages > 0 ? load_half() : 0;
    int slot = 0;
    uint32_t use = 0;  // laps of the ring so far
    for (long long g = 0; g < n_stages; ++g) {
      if (use >= 1) {
        int okw = 1;
        if (lane == 0)
          okw = (!*abort_flag && mbar_wait_backoff(bar_wempty + 8 * slot, (uint32_t)((use - 1) & 1), 32)) ? 1 : 0;
        okw = __shfl_sync(0xffffffffu, okw, 0);
        if (!okw) {
          if (lane == 0 && !*abort_flag) {
            *abort_flag = 1;
            raise_status(p.status, 2);
          }
          break;
        }
        tc_fence_after();
      }
      const bool stored = nks > 0;
      if (stored)
        tmem_st32(tmem_base + p.ring_col0 + (uint32_t)(slot * 8 * CM_WST + pair * 32) + ((uint32_t)(qtr * 32) << 16), v);
      // The store has read its registers once it is issued: the next stage's loads go out now
      // and fly while the store completes and the stage is published.
      if (g + 1 < n_stages) nks = load_half();
      if (stored) tmem_st_wait();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_wfull + 8 * slot);
      if (++slot == NW) { slot = 0; ++use; }
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ------------------------------------------------------------ create-time operand
// wa[channel tile][K step][half][128][16 B]; K step ks = (block*9 + tap)*kpt + k holds the 32 int8
// (16 fp16) channels of chunks 2k (half 0) and 2k+1 (half 1) of channel block `block`; rows past
// c_out are zero.
template <bool F16>
__global__ void cm_expand_weights_kernel(const uint32_t* __restrict__ wplanes, uint8_t* __restrict__ wa, int C, int K,
                                         int Cw, long long total, int cb_chunks, int n_cb) {
  // one thread per 16-byte half row
  long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i >= total) return;
  long long r = i;
  const int row = (int)(r % 128);
  r /= 128;
  const int hf = (int)(r & 1);
  r >>= 1;
  const int kpt = cb_chunks / 2;
  const int KS = 9 * n_cb * kpt;
  const int ks = (int)(r % KS), ct = (int)(r / KS);
  const int k = ks % kpt, t = (ks / kpt) % 9, cb = ks / (kpt * 9);
  const int co = ct * 128 + row;
  const int cpc = F16 ? 8 : 16;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (co < K) {
    const int ch0 = (cb * cb_chunks + 2 * k + hf) * cpc;
    const int wd = ch0 >> 5, sh = ch0 & 31;
    const uint32_t bits = wd < Cw ? wplanes[((size_t)t * Cw + wd) * K + co] >> sh : 0u;
    uint32_t w[4] = {0, 0, 0, 0};
    if (F16) {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (ch0 + e < C) w[e >> 1] |= (((bits >> e) & 1u) ? 0x3c00u : 0xbc00u) << (16 * (e & 1));  // +1.0 / -1.0
    } else {
#pragma unroll
      for (int e = 0; e < 16; ++e)
        if (ch0 + e < C) w[e >> 2] |= (((bits >> e) & 1u) ? 0x01u : 0xffu) << (8 * (e & 3));       // +1 / -1
    }
    v = make_uint4(w[0], w[1], w[2], w[3]);
  }
  reinterpret_cast<uint4*>(wa)[i] = v;
}

size_t cm_weight_bytes(const Geom& g, int act_type) {
  const bool f16 = act_type == SNN_ACT_F16;
  int n_chunks, cb;
  channel_blocks(g.C, f16, &n_chunks, &cb);
  const size_t cotiles = (size_t)(g.K + 127) / 128;
  return cotiles * 9 * (size_t)(n_chunks / 2) * 128 * 32;
}

cudaError_t cm_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched) {
  const bool f16 = act_type == SNN_ACT_F16;
  int n_chunks, cb;
  channel_blocks(g.C, f16, &n_chunks, &cb);
  const long long total = (long long)(cm_weight_bytes(g, act_type) / 16);
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (f16)
    cm_expand_weights_kernel<true><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.wcm, g.C, g.K, g.Cw, total, cb,
                                                         n_chunks / cb);
  else
    cm_expand_weights_kernel<false><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.wcm, g.C, g.K, g.Cw, total, cb,
                                                          n_chunks / cb);
  *launched += 1;
  return cudaGetLastError();
}

// ------------------------------------------------------------------ launch plan
namespace {

struct CmPlan {
  CmParams p;
  size_t smem;
  dim3 grid;
  bool ok;
};

constexpr size_t kCmSmemBudget = 226 * 1024;

// positions per tile offered as variants
const int kCmNp[] = {128, 256, 96, 176, 64, 192};
constexpr int kCmVariants = (int)(sizeof(kCmNp) / sizeof(kCmNp[0]));

CmPlan cm_plan(const Geom& g, int act_type, int Np) {
  CmPlan pl{};
  CmParams& p = pl.p;
  const bool f16 = act_type == SNN_ACT_F16;
  pl.ok = false;
  if (g.N < 1 || Np < 16 || Np > 256 || Np % 16) return pl;
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K; p.Cw = g.Cw;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  int n_chunks;
  channel_blocks(g.C, f16, &n_chunks, &p.cb_chunks);
  p.n_cb = n_chunks / p.cb_chunks;
  p.kpt = p.cb_chunks / 2;
  p.KS = 9 * p.n_cb * p.kpt;
  p.spc = (9 * p.kpt + CM_WST - 1) / CM_WST;
  p.n_wstages = p.n_cb * p.spc;
  if (g.stride == 1) {
    p.Hq = g.H + g.pad; p.Wq = g.W + g.pad; p.n_planes = 1; p.halo = 2 * p.Wq + 2;
  } else {
    p.Hq = g.Ho + 1; p.Wq = g.Wo + 1; p.n_planes = 4; p.halo = p.Wq + 1;
  }
  p.dWq = make_fastdiv((uint32_t)p.Wq);
  p.dHq = make_fastdiv((uint32_t)p.Hq);
  p.Qtot = (long long)g.N * p.Hq * p.Wq;
  if (p.Qtot + 1024 + p.halo >= (1ll << 31)) return pl;  // positions are 32-bit in the kernel
  if (g.C > kMaxChannelsSmallInt) return pl;             // the drain's int -> float shortcut
  if ((long long)g.N * g.H * g.W >= (1ll << 31) || (long long)g.N * g.Ho * g.Wo >= (1ll << 31)) return pl;
  p.Np = Np;
  p.Rr = Np + p.halo;
  const long long mgroups = (p.Qtot + Np - 1) / Np;
  p.n_cotiles = (g.K + 127) / 128;
  p.dCt = make_fastdiv((uint32_t)p.n_cotiles);
  if (mgroups * p.n_cotiles > 0x7fffffffLL) return pl;
  p.n_mgroups = (int)mgroups;
  p.total_tiles = (int)(mgroups * p.n_cotiles);
  const int sms = sm_count();
  int grid = sms;
  if (grid > p.total_tiles) grid = p.total_tiles;
  if (grid >= p.n_cotiles) grid = grid / p.n_cotiles * p.n_cotiles;  // a CTA keeps its channel tile
  const int tiles_per_cta = (p.total_tiles + grid - 1) / grid;
  // tensor memory: accumulators first, the weight ring behind them (32 columns per stage)
  p.n_acc = (tiles_per_cta > 1 && 2 * Np + 2 * 8 * CM_WST <= 512) ? 2 : 1;
  const int acc_cols = (p.n_acc * Np + 31) / 32 * 32;
  int nw = (512 - acc_cols) / (8 * CM_WST);
  if (nw > CM_RING_MAX) nw = CM_RING_MAX;
  if (nw < 2) return pl;
  p.ring_col0 = (uint32_t)acc_cols;
  p.w_resident = (p.n_wstages <= nw && grid % p.n_cotiles == 0 && !env_int("SNN_CM_NO_RESIDENT", 0)) ? 1 : 0;
  p.NW = p.w_resident ? p.n_wstages : nw;
  // shared memory: activation units, pixel table, tail
  const size_t unit_exact = (size_t)p.n_planes * p.cb_chunks * p.Rr * 16;
  p.a_unit_bytes = (uint32_t)((unit_exact + 127) & ~(size_t)127);
  const size_t pix_bytes = ((size_t)p.n_planes * p.Rr * 4 + 127) & ~(size_t)127;
  const size_t epi_bytes = (size_t)CM_EPI_WARPS * CM_EPI_STAGE;
  const size_t fixed = pix_bytes + epi_bytes + kCmTail;
  if (p.a_unit_bytes + fixed > kCmSmemBudget) return pl;
  long long na = (long long)((kCmSmemBudget - fixed) / p.a_unit_bytes);
  const long long units_per_cta = (long long)tiles_per_cta * p.n_cb;
  if (na > units_per_cta) na = units_per_cta;
  if (na > CM_NA_MAX) na = CM_NA_MAX;
  if (int v = env_int("SNN_CM_NA", 0)) if (v >= 1 && v < na) na = v;
  p.NA = (int)na;
  p.off_pix = (uint32_t)((size_t)p.NA * p.a_unit_bytes);
  p.off_epi = p.off_pix + (uint32_t)pix_bytes;
  p.off_tail = p.off_epi + (uint32_t)epi_bytes;
  pl.smem = (size_t)p.off_tail + kCmTail;
  if (pl.smem > (size_t)kMaxDynSmem || pl.smem >= (1u << 18)) return pl;   // descriptor address range
  if ((uint32_t)p.Rr * 16 >= (1u << 18)) return pl;                        // leading-offset field range
  pl.grid = dim3((unsigned)grid);
  pl.ok = true;
  return pl;
}

}  // namespace

int cm_variant_count() { return kCmVariants; }

bool cm_variant_ok(const Geom& g, int act_type, int variant) {
  if (variant < 0 || variant >= kCmVariants) return false;
  if (env_int("SNN_CM_DISABLE", 0)) return false;
  return cm_plan(g, act_type, kCmNp[variant]).ok;
}

cudaError_t cm_forward(LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched, int* status_dev,
                       int variant) {
  if (variant < 0 || variant >= kCmVariants) return cudaErrorInvalidConfiguration;
  CmPlan pl = cm_plan(g, act_type, kCmNp[variant]);
  if (!pl.ok || !L.wcm) return cudaErrorInvalidConfiguration;
  const bool f16 = act_type == SNN_ACT_F16;
  CmParams& p = pl.p;
  p.act = l.act;
  {
    // vector loads of a row's words need the base pointer and the row pitch aligned to the load
    const uintptr_t addr = (uintptr_t)l.act;
    if (f16) p.act_vec = (addr & 15) == 0 && (g.C & 7) == 0;
    else if (p.cb_chunks == 8) p.act_vec = (addr & 15) == 0 && (g.Cw & 3) == 0;
    else if (p.cb_chunks == 4) p.act_vec = (addr & 7) == 0 && (g.Cw & 1) == 0;
    else p.act_vec = 0;
  }
  p.wa = (const uint8_t*)L.wcm;
  p.alpha = L.alpha;
  p.out = l.out;
  p.out_i32 = l.out_i32;
  p.status = status_dev;
  // Launched as a programmatic dependent of its predecessor in the stream: set-up and the first
  // weight loads overlap that kernel's tail; the warps that read activations or write the output
  // wait on the device for it.
  const bool pdl = env_int("SNN_TC_PDL", 1) != 0;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.stream = l.stream;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  cfg.gridDim = pl.grid;
  cfg.blockDim = dim3(CM_THREADS);
  cfg.dynamicSmemBytes = pl.smem;
  cudaError_t e = cudaErrorInvalidConfiguration;
#define SNN_CM_LAUNCH(F, KP)                                                          \
  do {                                                                                \
    static unsigned long long done = 0;                                               \
    e = allow_max_smem(cm_conv_kernel<F, KP>, &done);                                 \
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, cm_conv_kernel<F, KP>, p);     \
  } while (0)
#define SNN_CM_LAUNCH_K(F)                     \
  do {                                         \
    if (p.kpt == 4) SNN_CM_LAUNCH(F, 4);       \
    else if (p.kpt == 3) SNN_CM_LAUNCH(F, 3);  \
    else if (p.kpt == 2) SNN_CM_LAUNCH(F, 2);  \
    else if (p.kpt == 1) SNN_CM_LAUNCH(F, 1);  \
  } while (0)
  if (f16) SNN_CM_LAUNCH_K(true);
  else SNN_CM_LAUNCH_K(false);
#undef SNN_CM_LAUNCH_K
#undef SNN_CM_LAUNCH
  if (e != cudaSuccess) return e;
  *launched += 1;
  return cudaGetLastError();
}

}  // namespace snn
