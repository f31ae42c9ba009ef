// Decoded-weight path on the 5th-generation tensor cores (tcgen05 + TMEM).
//
// The +/-1 weights of Sec. 3 become int8 (binary activations, exact int32
// accumulation) or fp16 (fp16 activations, fp32 accumulation) operands and the
// 3x3 convolution runs as an implicit GEMM:
//   M = 128 consecutive positions of a padded, flattened copy of the input,
//   N = a tile of output channels, K = (tap, input channel).
//
// One persistent, warp-specialised kernel per forward call.
//
// The A operand lives in shared memory as units  [plane][16-byte channel
// chunk][row][16 B]  (one unit = one tile of positions x one channel block), the
// K-major, no-swizzle layout whose rows are 16 bytes apart.  The flattened
// position space keeps one zero column per row and one zero row per image
// (shared by neighbours), so zero padding is a literal zero operand (a zero
// contributes 0, as the definition requires) and the A operand of tap (ky, kx)
// is the same unit read from a start address shifted by ky*pitch + kx rows:
// the nine taps reuse one staged unit, there is no im2col copy.  Stride 2
// splits the padded input into its four row/column parity planes.  The K loop
// runs channel block by channel block (then taps, then chunks), so the MMAs of
// a tile start when its first block is staged.
//      warp 0        one thread streams weight stages (cp.async.bulk onto
//                    mbarriers, a ring of NS stages; resident when they fit)
//      warp 1        one thread issues tcgen05.mma into one of two TMEM
//                    accumulator buffers and commits barriers
//      warps 2-9     epilogue: TMEM -> registers -> per-warp shared-memory
//                    transposition -> alpha scale -> 128-byte row stores, for
//                    tile i while the MMAs of tile i+1 run
//      warps 10-17   expanders: packed bits -> +1/-1 bytes (or fp16 copied)
//                    straight into the A units of a ring of NA, ahead of the MMAs
//    Measured on B200 and shaping this code: a thread alone on its warp retires
//    about one instruction per 5-8 cycles (more when other warps compete) and
//    an mbarrier wait costs ~200 cycles even when it is ready, so the issuing
//    thread runs straight code over large stages from tabulated offsets; warps
//    that wait elect one poller that sleeps between attempts, because many
//    pollers crowd the issuing threads.  Every wait is bounded; one that runs
//    out raises a status word the host reads, and the CTA still frees its
//    TMEM and returns.
#include "snn_tc_common.cuh"

namespace snn {

namespace {

// A CTA has EW epilogue warps and EW expander warps behind the producer and the MMA issuer.
// EW = 8: one CTA per SM with all of its shared and tensor memory.  EW = 4: a CTA of half the
// size (at most half of the shared memory, 256 tensor-memory columns, 320 threads), two of which
// share an SM, so that one's start-up, first loads and last drain run beside the other's MMAs,
// and the CTAs of the next kernel in the stream set themselves up while this one still runs.
constexpr int tc_threads(int ew) { return 64 + 64 * ew; }  // warp 0 producer, 1 MMA issue, EW epilogue, EW expanders
constexpr int EXP_ROWS = 3;                   // rows of a unit one expander thread loads together
constexpr int NS_MAX = 8;                     // most weight stages in flight
constexpr int EPI_PITCH = 128;                // bytes per staged output row; 16-byte columns are XOR-swizzled by row
constexpr int epi_bytes(int ew) { return ew * 32 * EPI_PITCH; }
constexpr size_t kSmemTail = 512;             // barriers, flags, tap offsets

struct TcParams {
  const void* act;        // uint32 [N][H][W][Cw] or half [N][H][W][C]
  const uint8_t* wt;      // tiled weights: [layout tile][block][tap][chunk][NtL][16 B]
  const float* alpha;
  void* out;
  int* status;            // mapped host word, set on a timed-out wait
  int out_i32;            // 0: fp32 alpha*S, 1: int32 S, 2: packed signs of alpha*S
  int act_vec;            // the activation rows may be read with 8/16-byte loads
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int Kpad, n_chunks;     // padded channels out; 16-byte chunks along the padded channels in
  int NtL;                // channels per layout tile of the weight operand
  int Hq, Wq;             // rows per image / row pitch of the flattened position space
  FastDiv dWq, dHq, dNt;  // exact division by Wq, Hq and the number of channel tiles
  int n_planes;           // 1 (stride 1) or 4 (stride 2)
  int halo;               // largest tap shift in rows
  int Rr;                 // staged rows per plane = 128*MT + halo
  int n_mgroups;          // position groups (tiles along M)
  int MT, Nt;             // M sub-tiles per tile, channels per tile
  int cb_chunks, n_cb;    // chunks per channel block (fixed when the layer is created), blocks
  int kpt;                // MMAs per sub-tile and tap within a block (= cb_chunks / 2, at most 4)
  int st_taps;            // taps per weight stage (1, 3 or 9)
  int NS, NA;             // weight stages / activation units in flight
  int n_acc;              // TMEM accumulator buffers (1 or 2)
  int b_resident;         // the whole weight set of the CTA's channel tile stays in the ring
  int n_ntiles;           // channel tiles
  int total_tiles;        // position groups * channel tiles
  long long Qtot;         // flattened positions to cover
  uint32_t tmem_cols;     // power of two >= n_acc*MT*Nt
  uint32_t a_unit_bytes;  // bytes of one staged activation unit
  uint32_t stage_bytes;   // bytes of one weight stage
  uint32_t off_b, off_epi, off_pix, off_tail;  // shared-memory offsets
};

// Flattened position of plane (pa, pb) -> input pixel index, or -1 when it is padding.
__device__ __forceinline__ int position_to_pixel(const TcParams& p, uint32_t q, int pa, int pb) {
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

// One 16/32-column slice of an accumulator row straight from registers (used
// when c_out is not a multiple of 4 or the channel tile not a multiple of 32).
template <bool F16, int NC>
__device__ __forceinline__ void epilogue_slice(const TcParams& p, uint32_t taddr, int c0, int n0, bool valid,
                                               size_t obase) {
  uint32_t v[NC];
  if (NC == 32) tmem_ld32(taddr, reinterpret_cast<uint32_t(&)[32]>(v));
  else tmem_ld16(taddr, reinterpret_cast<uint32_t(&)[16]>(v));
  tmem_ld_wait();
  const int co0 = n0 + c0;
  if (!valid || co0 >= p.K) return;
  if (p.out_i32) {
    int32_t* o = (int32_t*)p.out + obase + co0;
#pragma unroll
    for (int e = 0; e < NC; ++e)
      if (co0 + e < p.K) o[e] = (int)v[e];
  } else {
    float* o = (float*)p.out + obase + co0;
#pragma unroll
    for (int e = 0; e < NC; ++e)
      if (co0 + e < p.K)
        o[e] = __fmul_rn(F16 ? __uint_as_float(v[e]) : small_int_to_float(v[e]), __ldg(p.alpha + co0 + e));
  }
}

}  // namespace

// ------------------------------------------------------------------ GEMM
// KPT = MMAs per sub-tile and tap when known at compile time (2 or 4), 0 = read from the parameters
template <bool F16, int MT, int KPT, int EW>
__global__ void __launch_bounds__(tc_threads(EW), EW == 8 ? 1 : 2) tc_conv_kernel(const TcParams p) {
  constexpr int EPI_WARPS = EW, EXP_THREADS = 32 * EW;
  constexpr int NH = EW / 4;  // epilogue warps per TMEM lane quarter; they take the 32-column slices in turn
  extern __shared__ __align__(128) uint8_t smem[];
  // carve-up: [NA activation units][NS weight stages][epilogue tiles][barriers, flags, table]
  uint8_t* a_smem = smem;
  uint8_t* b_smem = smem + p.off_b;
  uint8_t* epi_smem = smem + p.off_epi;
  int* pix_tab = reinterpret_cast<int*>(smem + p.off_pix);  // [plane][row] input pixel of a staged row
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_tail);
  // barriers: b_full[8] b_empty[8] a_full[4] a_empty[4] acc_full[2] acc_empty[2]
  const uint32_t bar_bfull = smem_u32(bars), bar_bempty = smem_u32(bars + 8);
  const uint32_t bar_afull = smem_u32(bars + 16), bar_aempty = smem_u32(bars + 20);
  const uint32_t bar_accfull = smem_u32(bars + 24), bar_accempty = smem_u32(bars + 26);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 28);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* tap_units = tmem_slot + 3;  // [9] A row offset of every tap inside a unit (tmem_slot[2] = expander flag)

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NS = p.NS, NA = p.NA;

  if (tid < 28) {
    uint32_t count = 1;
    if (tid >= 26) count = EPI_WARPS;                // acc_empty: one arrival per epilogue warp
    if (tid >= 16 && tid < 20) count = EXP_THREADS;  // a_full: every expander thread arrives
    mbar_init(smem_u32(bars + tid), count);
  }
  if (tid == 32) *abort_flag = 0;
  if (tid >= 64 && tid < 73) {
    // rows (16-byte units) from a unit's origin to tap t: plane offset + shift inside the plane
    const int t = tid - 64, ky = t / 3, kx = t % 3;
    uint32_t u;
    if (p.stride == 1) u = (uint32_t)(ky * p.Wq + kx);
    else u = (uint32_t)((ky & 1) * 2 + (kx & 1)) * (uint32_t)(p.cb_chunks * p.Rr) +
             (uint32_t)((ky >> 1) * p.Wq + (kx >> 1));
    tap_units[t] = u;
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(p.tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp >= 2 + EPI_WARPS) {
    // The expanders' table for their first tile (input pixel of every staged row, -1 = padding)
    // depends on nothing but the parameters: it is worked out here, beside the set-up and before
    // the wait for the previous kernel.  A thread reads back only entries it wrote itself.
    const int et0 = tid - (2 + EPI_WARPS) * 32;
    const uint32_t Q00 = (uint32_t)((int)blockIdx.x / p.n_ntiles) * (uint32_t)(128 * MT);
    // (plane, row) pairs form one index space f = plane*Rr + row, dealt to the threads at a stride of
    // the expander count, here and in the expanders' loops
    for (int f = et0; f < p.n_planes * p.Rr; f += EXP_THREADS) {
      const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
      pix_tab[f] = position_to_pixel(p, Q00 + (uint32_t)(f - pl * p.Rr), pl >> 1, pl & 1);
    }
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_launch();  // the next kernel in the stream may be scheduled; it waits for this grid to finish

  // A weight stage holds st_taps whole taps of one channel block.
  const int stages_per_cb = 9 / p.st_taps;
  const int stages_per_tile = p.n_cb * stages_per_cb;
  const uint32_t acc_cols = (uint32_t)(MT * p.Nt);

  if (warp == 0) {
    // ------------------------------------------------ producer (one lane)
    if (lane == 0) {
      int b_slot = 0, b_issued = 0;
      uint32_t b_phase = 1;  // parity of the previous use of a slot (valid from the second lap)
      bool ok = true;
      // Weight stages are issued in the order the MMAs consume them; `w_next` counts the stages
      // already requested, so that the first ones can be requested before the expanded
      // activations exist (the weights are constants of the layer).
      long long w_next = 0;
      int w_cb = 0, w_sg = 0;
      auto issue_weights = [&](int tile, long long upto) -> bool {
        // requests stages [w_next, upto) of this CTA's stage sequence, stopping when the ring is full
        const int nti = tile - (int)fdiv((uint32_t)tile, p.dNt) * p.n_ntiles;
        const int n0 = nti * p.Nt;
        // channel tile -> layout tile of the weight operand (the same thing unless a narrower tile was asked for)
        const int ltile = p.Nt == p.NtL ? nti : n0 / p.NtL;
        const size_t wtile = (size_t)ltile * p.n_cb;
        const int n_in = n0 - ltile * p.NtL;
        while (w_next < upto) {
          const int cb = w_cb, sg = w_sg;  // position inside the tile, kept as counters (no divisions)
          if (++w_sg == stages_per_cb) {
            w_sg = 0;
            if (++w_cb == p.n_cb) w_cb = 0;
          }
          if (b_issued >= NS && !mbar_wait_backoff(bar_bempty + 8 * b_slot, b_phase, 32)) return false;
          const uint32_t dst = smem_u32(b_smem) + (uint32_t)b_slot * p.stage_bytes;
          const uint8_t* src =
              p.wt + ((((wtile + cb) * 9 + (size_t)sg * p.st_taps) * p.cb_chunks) * p.NtL + n_in) * 16;
          mbar_expect_tx(bar_bfull + 8 * b_slot, p.stage_bytes);
          if (p.Nt == p.NtL) {
            bulk_g2s(dst, src, p.stage_bytes, bar_bfull + 8 * b_slot);  // (tap, chunk) blocks are contiguous
          } else {
            const int nchunk = p.st_taps * p.cb_chunks;
            for (int c = 0; c < nchunk; ++c)
              bulk_g2s(dst + (uint32_t)c * p.Nt * 16, src + (size_t)c * p.NtL * 16, (uint32_t)p.Nt * 16,
                       bar_bfull + 8 * b_slot);
          }
          ++b_issued;
          ++w_next;
          if (++b_slot == NS) { b_slot = 0; b_phase ^= 1u; }
        }
        return true;
      };
      long long tiles_seen = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tiles_seen) {
        if (p.b_resident && tiles_seen > 0) break;  // kept from the first tile on
        if (*abort_flag) break;
        if (!issue_weights(tile, (tiles_seen + 1) * stages_per_tile)) {
          *abort_flag = 1;
          raise_status(p.status, 2);
          ok = false;
        }
      }
      // never leave with copies in flight: wait (bounded) for the last load of every slot
      for (int s = 0; s < NS; ++s) {
        int last = -1;
        for (int i = s; i < b_issued; i += NS) last = i;
        if (last >= 0) mbar_wait_backoff(bar_bfull + 8 * s, (last / NS) & 1, 64);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    // The whole warp walks the loops and waits together, so that every address and descriptor is
    // a warp-uniform value (no per-MMA moves into uniform registers); one elected lane issues the
    // MMAs and the commits.
    {
      const bool leader = elect_one();
      // instruction descriptor: D format, A/B formats, K-major both, N>>3, M>>4
      const uint32_t idesc = F16 ? ((1u << 4) | ((uint32_t)(p.Nt >> 3) << 17) | ((128u >> 4) << 24))
                                 : ((2u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(p.Nt >> 3) << 17) |
                                    ((128u >> 4) << 24));
      // Descriptors are built once; every MMA only adds row offsets (16-byte units) to the
      // address field.
      const uint64_t a_desc0 = make_desc(smem_u32(a_smem), (uint32_t)p.Rr * 16, 128);
      const uint64_t b_desc0 = make_desc(smem_u32(b_smem), (uint32_t)p.Nt * 16, 128);
      const uint32_t stage_units = p.stage_bytes >> 4, unit_units = p.a_unit_bytes >> 4;
      const uint32_t a_step = 2u * (uint32_t)p.Rr, b_step = 2u * (uint32_t)p.Nt;  // two chunks per MMA
      const uint32_t nt = (uint32_t)p.Nt;
      const int kpt = KPT ? KPT : p.kpt, st_taps = p.st_taps;
      bool ok = true;
      int a_slot = 0, b_slot = 0, acc_slot = 0;
      uint32_t a_phase = 0, b_phase = 0, acc_phase = 1;
      int tiles_done = 0;
      for (int tile = blockIdx.x; tile < p.total_tiles && ok; tile += gridDim.x, ++tiles_done) {
        // the accumulator buffer must have been drained by the epilogue of its previous tile
        if (tiles_done >= p.n_acc) {
          if (!mbar_wait(bar_accempty + 8 * acc_slot, acc_phase)) { ok = false; break; }
          tc_fence_after();
        }
        const uint32_t d0 = tmem_base + (uint32_t)acc_slot * acc_cols;
        uint32_t acc = 0;  // 0 only for the first MMA of every sub-tile
        const bool wait_b = !(p.b_resident && tiles_done > 0);
        for (int cb = 0; cb < p.n_cb && ok; ++cb) {
          if (!mbar_wait(bar_afull + 8 * a_slot, a_phase)) { ok = false; break; }
          tc_fence_after();
          const uint64_t a_unit = a_desc0 + (uint64_t)((uint32_t)a_slot * unit_units);
          int t = 0;
          for (int sg = 0; sg < stages_per_cb; ++sg) {
            if (wait_b) {
              if (!mbar_wait(bar_bfull + 8 * b_slot, b_phase)) { ok = false; break; }
              tc_fence_after();
            }
            uint64_t bd = b_desc0 + (uint64_t)((uint32_t)b_slot * stage_units);
            for (int tt = 0; tt < st_taps; ++tt, ++t) {
              uint64_t ad = a_unit + (uint64_t)tap_units[t];
#pragma unroll
              for (int k = 0; k < (KPT ? KPT : 4); ++k) {
                if (KPT || k < kpt) {
                  if (leader) {
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt)
                      mma_ss<F16>(d0 + (uint32_t)mt * nt, ad + (uint64_t)(mt * 128), bd, idesc, acc);
                  }
                  acc = 1;
                  ad += a_step;
                  bd += b_step;
                }
              }
            }
            if (!p.b_resident && leader) tc_commit(bar_bempty + 8 * b_slot);  // free once these MMAs have read it
            if (++b_slot == NS) { b_slot = 0; b_phase ^= 1u; }
          }
          if (leader) tc_commit(bar_aempty + 8 * a_slot);  // the activation unit may be overwritten
          if (++a_slot == NA) { a_slot = 0; a_phase ^= 1u; }
        }
        if (leader) tc_commit(bar_accfull + 8 * acc_slot);  // fires when this tile's MMAs are complete
        if (++acc_slot == p.n_acc) { acc_slot = 0; acc_phase ^= 1u; }
      }
      if (!ok && leader) {
        *abort_flag = 1;
        raise_status(p.status, 3);
      }
    }
    __syncwarp();
  } else if (warp < 2 + EPI_WARPS) {
    // ------------------------------------------------ epilogue warps
    grid_dep_wait();  // an earlier kernel in the stream may still read the output buffer
    // Warp w reads TMEM lanes 32*(w%4).. (rows of the tile); the two warps of a lane quarter
    // split the 32-column slices between them.  A slice goes through a per-warp shared-memory
    // tile so that each store instruction writes whole 128-byte rows.
    const int ew = warp - 2;
    const int rq = warp & 3, half = ew >> 2;
    uint8_t* stage = epi_smem + (size_t)ew * (32 * EPI_PITCH);
    const int srow = lane >> 3, scol = lane & 7;  // this lane's (row mod 4, 16-byte column) when storing
    const bool fast = ((p.K & 3) == 0) && ((p.Nt & 31) == 0);
    int acc_slot = 0;
    uint32_t acc_phase = 0;
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      const int mg = (int)fdiv((uint32_t)tile, p.dNt), nti = tile - mg * p.n_ntiles;
      const uint32_t Q0 = (uint32_t)mg * (uint32_t)(128 * MT);
      const int n0 = nti * p.Nt;
      int okw = 1;
      if (lane == 0) okw = (!*abort_flag && mbar_wait_backoff(bar_accfull + 8 * acc_slot, acc_phase, 100)) ? 1 : 0;
      okw = __shfl_sync(0xffffffffu, okw, 0);
      if (!okw) {
        if (lane == 0 && !*abort_flag) {
          *abort_flag = 1;
          raise_status(p.status, 4);
        }
        break;
      }
      tc_fence_after();
      const uint32_t d0 = tmem_base + (uint32_t)acc_slot * acc_cols;
      // row of sub-tile mt this lane owns in TMEM -> is it an output, and where does it go
      // output pixel (n*Ho + y)*Wo + x, or -1 when the row is not an output
      auto row_pixel = [&](int mt) -> int {
        const uint32_t q = Q0 + (uint32_t)(mt * 128 + rq * 32 + lane);
        const uint32_t rg = fdiv(q, p.dWq);
        const int x = (int)(q - rg * (uint32_t)p.Wq);
        const uint32_t n = fdiv(rg, p.dHq);
        const int y = (int)(rg - n * (uint32_t)p.Hq);
        const bool valid = ((long long)q < p.Qtot) && ((int)n < p.N) && (y < p.Ho) && (x < p.Wo);
        return valid ? ((int)n * p.Ho + y) * p.Wo + x : -1;
      };
      if (p.out_i32 == 2) {
        // Packed signs of the scaled output (Algorithm 1: the next layer consumes sign(a)): a thread
        // owns one position and the 32 (or 16) consecutive channels of a slice, i.e. one word (or
        // half-word) of the next layer's binary input.  No transposition, one small store per slice.
        const int Kw = (p.K + 31) >> 5;
        uint32_t* out32 = reinterpret_cast<uint32_t*>(p.out);
        if ((p.Nt & 31) == 0) {
          const int per_mt = (p.Nt - 32 * half + 32 * NH - 1) / (32 * NH);
#pragma unroll 1
          for (int mt = 0; mt < MT; ++mt) {
            const int pix = row_pixel(mt);
#pragma unroll 1
            for (int ci = 0; ci < per_mt; ++ci) {
              const int c0 = 32 * half + 32 * NH * ci, co0 = n0 + c0;
              uint32_t v[32];
              __syncwarp();  // the load is a warp-wide instruction: no lane may still be in the store below
              tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * p.Nt + c0), v);
              tmem_ld_wait();
              if (pix >= 0 && co0 < p.K) {
                uint32_t word = 0;
#pragma unroll
                for (int e = 0; e < 32; ++e) {
                  const float a = co0 + e < p.K ? __ldg(p.alpha + co0 + e) : -1.f;  // a missing channel gives bit 0 ...
                  const float s = co0 + e < p.K ? small_int_to_float(v[e]) : 1.f;   // ... through 1 * -1 < 0
                  word |= (__fmul_rn(s, a) >= 0.f ? 1u : 0u) << e;
                }
                out32[wide_mul((uint32_t)pix, (uint32_t)Kw) + (uint32_t)(co0 >> 5)] = word;
              }
            }
          }
        } else {
          // one channel tile whose width is an odd multiple of 16: half-words; the slice that ends
          // the tile also clears the half-word behind it, so that every word is written in full
          uint16_t* out16 = reinterpret_cast<uint16_t*>(p.out);
#pragma unroll 1
          for (int mt = 0; mt < MT; ++mt) {
            const int pix = row_pixel(mt);
            for (int c0 = 16 * half; c0 < p.Nt; c0 += 16 * NH) {
              uint32_t v[16];
              __syncwarp();
              tmem_ld16(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * p.Nt + c0), v);
              tmem_ld_wait();
              const int co0 = n0 + c0;
              if (pix >= 0) {
                uint32_t hw = 0;
#pragma unroll
                for (int e = 0; e < 16; ++e) {
                  const float a = co0 + e < p.K ? __ldg(p.alpha + co0 + e) : -1.f;
                  const float s = co0 + e < p.K ? small_int_to_float(v[e]) : 1.f;
                  hw |= (__fmul_rn(s, a) >= 0.f ? 1u : 0u) << e;
                }
                const size_t at = wide_mul((uint32_t)pix, (uint32_t)(2 * Kw)) + (uint32_t)(co0 >> 4);
                if ((co0 >> 4) < 2 * Kw) out16[at] = (uint16_t)hw;
                if (c0 + 16 >= p.Nt && (co0 >> 4) + 1 < 2 * Kw) out16[at + 1] = 0;
              }
            }
          }
        }
      } else if (fast) {
        // The warp's slices (sub-tile mt, columns c0..c0+31) form one sequence.  The TMEM load of
        // slice s+1 is issued as soon as slice s sits in the staging tile, so it flies while
        // slice s is converted and stored, and the store path never waits for a TMEM load.
        const int per_mt = (p.Nt - 32 * half + 32 * NH - 1) / (32 * NH);
        const int total = MT * per_mt;
        uint32_t v[32];
        int ro[8];
        if (total > 0) tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(32 * half), v);
        int mt = 0, ci = 0;  // slice = (sub-tile mt, this warp's ci-th slice of it); no divisions in the loop
#pragma unroll 1
        for (int sl = 0; sl < total; ++sl) {
          const int c0 = 32 * half + 32 * NH * ci;
          if (ci == 0) {
            // output pixels of the eight rows this lane stores (row = srow + 4*i), -1 when not an output
            const int mine = row_pixel(mt);
#pragma unroll
            for (int i = 0; i < 8; ++i) ro[i] = __shfl_sync(0xffffffffu, mine, srow + 4 * i);
          }
          const int co = n0 + c0 + scol * 4;
          float4 al = make_float4(0.f, 0.f, 0.f, 0.f);
          if (!p.out_i32 && co < p.K) al = __ldg(reinterpret_cast<const float4*>(p.alpha + co));
          tmem_ld_wait();
#pragma unroll
          for (int e = 0; e < 8; ++e)
            *reinterpret_cast<uint4*>(stage + lane * EPI_PITCH + ((e ^ (lane & 7)) << 4)) =
                make_uint4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
          __syncwarp();
          const int this_mt = mt;
          if (++ci == per_mt) { ci = 0; ++mt; }
          if (sl + 1 < total)
            tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * p.Nt + 32 * half + 32 * NH * ci), v);
          (void)this_mt;
          if (co < p.K) {  // K is a multiple of 4 here, so the four channels exist together
            // loads and conversions first, the (predicated) stores last: no branch sits between
            // the eight independent chains, so their latencies overlap
            uint4 u[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const int row = srow + 4 * i;
              u[i] = *reinterpret_cast<const uint4*>(stage + row * EPI_PITCH + ((scol ^ (row & 7)) << 4));
            }
            if (!p.out_i32) {
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                scale_pair<F16>(u[i].x, u[i].y, al.x, al.y);
                scale_pair<F16>(u[i].z, u[i].w, al.z, al.w);
              }
            }
            uint32_t* obase32 = reinterpret_cast<uint32_t*>(p.out) + co;  // int32 and fp32 outputs share the layout
#pragma unroll
            for (int i = 0; i < 8; ++i)
              if (ro[i] >= 0) *reinterpret_cast<uint4*>(obase32 + wide_mul((uint32_t)ro[i], (uint32_t)p.K)) = u[i];
          }
          __syncwarp();
        }
      } else {
#pragma unroll 1
        for (int mt = 0; mt < MT; ++mt) {
          const int pix = row_pixel(mt);
          const bool valid = pix >= 0;
          const size_t obase = (size_t)(valid ? pix : 0) * (size_t)p.K;
          const uint32_t trow = d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * p.Nt);
          if ((p.Nt & 31) == 0) {
            for (int c0 = 32 * half; c0 < p.Nt; c0 += 32 * NH)
              epilogue_slice<F16, 32>(p, trow + (uint32_t)c0, c0, n0, valid, obase);
          } else {
            for (int c0 = 16 * half; c0 < p.Nt; c0 += 16 * NH)
              epilogue_slice<F16, 16>(p, trow + (uint32_t)c0, c0, n0, valid, obase);
          }
        }
      }
      // this warp has read its part of the accumulator buffer: hand it back to the MMA issuer
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar_accempty + 8 * acc_slot);
      if (++acc_slot == p.n_acc) { acc_slot = 0; acc_phase ^= 1u; }
    }
  }
  else {
    // ------------------------------------------------ expanders (the last EW warps)
    // Fill activation unit (tile, channel block) of the ring: for every plane, row and 32-channel
    // word, bits -> two 16-byte chunks of +1/-1 bytes (fp16: copy two 8-channel chunks).  A thread
    // takes EXP_ROWS rows at a time and issues their loads together.
    grid_dep_wait();  // the activations may come from the previous kernel in the stream
    const int et = tid - (2 + EPI_WARPS) * 32;
    int a_slot = 0, a_done = 0;
    uint32_t a_phase = 1;  // parity of the previous use of a slot (valid from the second lap)
    volatile int* exp_flag = abort_flag + 1;
    const int nstep = p.cb_chunks / 2;  // pairs of chunks per unit
    for (int tile = blockIdx.x; tile < p.total_tiles; tile += gridDim.x) {
      const int mg = (int)fdiv((uint32_t)tile, p.dNt);
      const uint32_t Q0 = (uint32_t)mg * (uint32_t)(128 * MT);
      bool stop = false;
      // input pixel of every staged row, once per tile (the first tile's table was made during set-up)
      if (tile != (int)blockIdx.x)
        for (int f = et; f < p.n_planes * p.Rr; f += EXP_THREADS) {
          const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
          pix_tab[f] = position_to_pixel(p, Q0 + (uint32_t)(f - pl * p.Rr), pl >> 1, pl & 1);
        }
      for (int cb = 0; cb < p.n_cb; ++cb) {
        if (a_done >= NA) {
          // one elected thread polls; the rest wait on a hardware barrier instead of spinning
          if (et == 0) *exp_flag = (!*abort_flag && mbar_wait_backoff(bar_aempty + 8 * a_slot, a_phase, 64)) ? 1 : 0;
          asm volatile("bar.sync 3, %0;" ::"n"(EXP_THREADS) : "memory");
          const int okf = *exp_flag;
          asm volatile("bar.sync 3, %0;" ::"n"(EXP_THREADS) : "memory");
          if (!okf) {
            if (et == 0 && !*abort_flag) {
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
          for (int rb = 0; rb < all_rows; rb += EXP_ROWS * EXP_THREADS) {
            int pix[EXP_ROWS];  // input pixel of each of this thread's rows; -1 padding, -2 past the unit
            uint8_t* dst[EXP_ROWS];  // where the row starts in its plane (chunk 0)
#pragma unroll
            for (int j = 0; j < EXP_ROWS; ++j) {
              const int f = rb + et + j * EXP_THREADS;
              pix[j] = f < all_rows ? pix_tab[f] : -2;
              const int pl = (f >= p.Rr) + (f >= 2 * p.Rr) + (f >= 3 * p.Rr);
              dst[j] = unit + ((size_t)pl * p.cb_chunks * p.Rr + (size_t)(f - pl * p.Rr)) * 16;
            }
            if (F16) {
              for (int c0 = 0; c0 < p.cb_chunks; c0 += 2) {
                uint4 v[EXP_ROWS][2];
#pragma unroll
                for (int j = 0; j < EXP_ROWS; ++j) {
#pragma unroll
                  for (int k = 0; k < 2; ++k) {
                    v[j][k] = make_uint4(0, 0, 0, 0);
                    const int ch = (cb * p.cb_chunks + c0 + k) * 8;  // first channel of the chunk
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
                for (int j = 0; j < EXP_ROWS; ++j) {
                  if (pix[j] != -2) {
                    *reinterpret_cast<uint4*>(dst[j] + (size_t)c0 * p.Rr * 16) = v[j][0];
                    *reinterpret_cast<uint4*>(dst[j] + (size_t)(c0 + 1) * p.Rr * 16) = v[j][1];
                  }
                }
              }
            } else {
              // up to four 32-channel words per row and block, as one vector load when aligned
              const int w0 = cb * nstep;
              uint32_t bits[EXP_ROWS][4];
#pragma unroll
              for (int j = 0; j < EXP_ROWS; ++j) {
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
              for (int j = 0; j < EXP_ROWS; ++j) {
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
      if (stop) break;
    }
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(p.tmem_cols)
                 : "memory");
  }
}

// ------------------------------------------------------------ create-time operand
// wt[layout tile][channel block][tap][chunk][NtL][16 B]: chunk = 16 (int8) or 8 (fp16)
// consecutive input channels, cb_chunks chunks per block, NtL output channels per layout tile.
// A CTA that owns a whole layout tile reads every weight stage (consecutive taps of one channel
// block) as one contiguous piece.
template <bool F16>
__global__ void tc_expand_weights_kernel(const uint32_t* __restrict__ wplanes, uint8_t* __restrict__ wt, int C, int K,
                                         int Cw, long long total, int cb_chunks, int n_cb, int NtL) {
  long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i >= total) return;
  int row = (int)(i % NtL);
  long long r = i / NtL;
  int c = (int)(r % cb_chunks);
  r /= cb_chunks;
  int t = (int)(r % 9);
  r /= 9;
  int cb = (int)(r % n_cb), tile = (int)(r / n_cb);
  int co = tile * NtL + row;
  const int cpc = F16 ? 8 : 16;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (co < K) {
    int ch0 = (cb * cb_chunks + c) * cpc;
    int wd = ch0 >> 5, sh = ch0 & 31;
    uint32_t bits = wd < Cw ? wplanes[((size_t)t * Cw + wd) * K + co] >> sh : 0u;
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
  reinterpret_cast<uint4*>(wt)[i] = v;
}

// Layout tile of the weight operand: all channels when they fit one MMA (N <= 256), else 128.
static int layout_tile(int K) { return K <= 256 ? round_up(K, 16) : 128; }

size_t tc_weight_bytes(const Geom& g, int act_type, int* Kpad, int* Cpad) {
  const bool f16 = act_type == SNN_ACT_F16;
  int n_chunks, cb;
  channel_blocks(g.C, f16, &n_chunks, &cb);
  *Kpad = round_up(g.K, layout_tile(g.K));
  *Cpad = n_chunks * (f16 ? 8 : 16);
  return (size_t)9 * n_chunks * (*Kpad) * 16;
}

cudaError_t tc_expand_weights(const LayerDev& L, const Geom& g, int act_type, cudaStream_t s, int* launched) {
  const bool f16 = act_type == SNN_ACT_F16;
  int n_chunks, cb;
  channel_blocks(g.C, f16, &n_chunks, &cb);
  const long long total = (long long)9 * n_chunks * L.Kpad;
  unsigned blocks = (unsigned)((total + 255) / 256);
  const int NtL = layout_tile(g.K);
  if (f16)
    tc_expand_weights_kernel<true><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.w16, g.C, g.K, g.Cw, total, cb,
                                                         n_chunks / cb, NtL);
  else
    tc_expand_weights_kernel<false><<<blocks, 256, 0, s>>>(L.wplanes, (uint8_t*)L.w8, g.C, g.K, g.Cw, total, cb,
                                                          n_chunks / cb, NtL);
  *launched += 1;
  return cudaGetLastError();
}

cudaError_t tc_expand_weights_custom(const uint32_t* wplanes, void* dst, int C, int K, int Cw, int Kpad, int n_chunks,
                                     int cb_chunks, int NtL, bool f16, cudaStream_t s) {
  const long long total = (long long)9 * n_chunks * Kpad;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (f16)
    tc_expand_weights_kernel<true><<<blocks, 256, 0, s>>>(wplanes, (uint8_t*)dst, C, K, Cw, total, cb_chunks,
                                                         n_chunks / cb_chunks, NtL);
  else
    tc_expand_weights_kernel<false><<<blocks, 256, 0, s>>>(wplanes, (uint8_t*)dst, C, K, Cw, total, cb_chunks,
                                                          n_chunks / cb_chunks, NtL);
  return cudaGetLastError();
}

// ------------------------------------------------------------------ launch plan
struct TcPlan {
  TcParams p;
  int ew;
  size_t smem;
  dim3 grid;
  bool ok;
  double score;
};

// Shared memory a CTA may plan with: the whole SM's, or half of it for the half-size CTAs
// (two of them, plus the 1 KB the system keeps per resident CTA, fit the SM's 228 KB).
static size_t smem_budget(int ew) { return ew == 8 ? (size_t)226 * 1024 : (size_t)112 * 1024; }

// Everything that follows from a choice of sub-tiles per tile (MT), weight-stage size and
// CTA size (ew = 8: one CTA per SM, ew = 4: two half-size CTAs per SM).
static TcPlan plan_for(const Geom& g, int act_type, int MT, int stage_kb, int ew) {
  const size_t kSmemBudget = smem_budget(ew);
  const int EPI_BYTES = epi_bytes(ew);
  const int tmem_limit = ew == 8 ? 512 : 256;
  TcPlan pl{};
  pl.ew = ew;
  TcParams& p = pl.p;
  const bool f16 = act_type == SNN_ACT_F16;
  pl.ok = false;
  int Kpad, Cpad;
  tc_weight_bytes(g, act_type, &Kpad, &Cpad);
  p.N = g.N; p.H = g.H; p.W = g.W; p.C = g.C; p.K = g.K; p.Cw = g.Cw;
  p.stride = g.stride; p.pad = g.pad; p.Ho = g.Ho; p.Wo = g.Wo;
  p.Kpad = Kpad;
  p.NtL = layout_tile(g.K);
  channel_blocks(g.C, f16, &p.n_chunks, &p.cb_chunks);
  p.n_cb = p.n_chunks / p.cb_chunks;
  p.kpt = p.cb_chunks / 2;
  if (g.stride == 1) {
    p.Hq = g.H + g.pad; p.Wq = g.W + g.pad; p.n_planes = 1; p.halo = 2 * p.Wq + 2;
  } else {
    p.Hq = g.Ho + 1; p.Wq = g.Wo + 1; p.n_planes = 4; p.halo = p.Wq + 1;
  }
  p.dWq = make_fastdiv((uint32_t)p.Wq);
  p.dHq = make_fastdiv((uint32_t)p.Hq);
  p.Qtot = (long long)g.N * p.Hq * p.Wq;
  if (p.Qtot + 1024 + p.halo >= (1ll << 31)) return pl;  // positions are 32-bit in the kernels
  if (g.C > kMaxChannelsSmallInt) return pl;             // the drain's int -> float shortcut
  if ((long long)g.N * g.H * g.W >= (1ll << 31)) return pl;
  const long long mtiles = (p.Qtot + 127) / 128;
  const int sms = sm_count();
  // channels per tile: a layout tile, or a part of one on request
  int Nt = p.NtL;
  int forced_nt = env_int("SNN_TC_NT", 0);
  if (forced_nt >= 16 && forced_nt <= 256 && forced_nt % 16 == 0 && p.NtL % forced_nt == 0) Nt = forced_nt;
  if (ew == 4 && Nt > 128 && p.NtL % 128 == 0) Nt = 128;  // two accumulators in 256 tensor-memory columns
  p.Nt = Nt;
  p.n_ntiles = Kpad / Nt;
  p.dNt = make_fastdiv((uint32_t)p.n_ntiles);
  if (MT * Nt > tmem_limit) return pl;
  p.MT = MT;
  p.Rr = 128 * MT + p.halo;
  const long long mgroups = (mtiles + MT - 1) / MT;
  if (mgroups * p.n_ntiles > 0x7fffffffLL || mgroups * p.Rr >= (1ll << 31)) return pl;
  p.n_mgroups = (int)mgroups;
  p.total_tiles = (int)(mgroups * p.n_ntiles);
  // persistent grid: one CTA (two half-size ones) per SM, a multiple of the channel tiles so that a
  // CTA keeps its channel tile
  int grid = ew == 8 ? sms : 2 * sms;
  if (grid > p.total_tiles) grid = p.total_tiles;
  if (grid >= p.n_ntiles) grid = grid / p.n_ntiles * p.n_ntiles;
  const int tiles_per_cta = (p.total_tiles + grid - 1) / grid;
  p.n_acc = (2 * MT * Nt <= tmem_limit && tiles_per_cta > 1) ? 2 : 1;
  uint32_t cols = 32;
  while (cols < (uint32_t)(p.n_acc * MT * Nt)) cols *= 2;
  p.tmem_cols = cols;

  // ---- shared memory: activation units, weight stages, epilogue tiles, tail
  const size_t unit_exact = (size_t)p.n_planes * p.cb_chunks * p.Rr * 16;
  p.a_unit_bytes = (uint32_t)((unit_exact + 127) & ~(size_t)127);
  const size_t kstep_bytes = (size_t)2 * Nt * 16;        // weights of one MMA
  const size_t tap_bytes = (size_t)p.kpt * kstep_bytes;  // weights of one tap of one channel block
  const size_t pix_bytes = ((size_t)p.n_planes * p.Rr * 4 + 127) & ~(size_t)127;
  const size_t fixed = (size_t)EPI_BYTES + pix_bytes + kSmemTail;
  const size_t stage_cap = (size_t)(stage_kb > 0 ? stage_kb : 48) * 1024;
  const long long units_per_cta = (long long)tiles_per_cta * p.n_cb;
  int na = units_per_cta >= 3 && p.n_cb >= 2 ? 3 : (units_per_cta >= 2 ? 2 : 1);
  while (na > 1 && (size_t)na * p.a_unit_bytes + 2 * tap_bytes + fixed > kSmemBudget) --na;
  if ((size_t)na * p.a_unit_bytes + tap_bytes + fixed > kSmemBudget) return pl;
  p.NA = na;
  const size_t b_budget = kSmemBudget - fixed - (size_t)na * p.a_unit_bytes;
  const size_t all_bytes = (size_t)9 * p.n_cb * tap_bytes;  // every weight of a channel tile
  // resident weights: the CTA's channel tile never changes and its weights fit next to the rest
  p.b_resident = 0;
  if (p.n_cb == 1 && tiles_per_cta > 1 && grid % p.n_ntiles == 0 && all_bytes <= b_budget &&
      !env_int("SNN_TC_NO_RESIDENT", 0))
    p.b_resident = 1;
  size_t cap = stage_cap < b_budget / 2 ? stage_cap : b_budget / 2;  // at least two stages in flight
  if (p.b_resident) cap = stage_cap;
  if (cap < tap_bytes) cap = tap_bytes <= b_budget ? tap_bytes : 0;
  if (cap == 0) return pl;
  p.st_taps = 9 * tap_bytes <= cap ? 9 : (3 * tap_bytes <= cap ? 3 : 1);
  p.stage_bytes = (uint32_t)((size_t)p.st_taps * tap_bytes);
  const int stages_per_tile = p.n_cb * (9 / p.st_taps);
  int ns = (int)(b_budget / p.stage_bytes);
  if (ns > NS_MAX) ns = NS_MAX;
  if (p.b_resident) {
    if (stages_per_tile > ns) p.b_resident = 0;
    else ns = stages_per_tile;
  }
  if (!p.b_resident) {
    const long long all_stages = (long long)stages_per_tile * tiles_per_cta;
    if (ns > all_stages) ns = (int)all_stages;
    int forced_ns = env_int("SNN_TC_NS", 0);
    if (forced_ns >= 1 && forced_ns <= ns) ns = forced_ns;
    if (ns < 1) return pl;
  }
  p.NS = ns;
  p.off_b = (uint32_t)((size_t)na * p.a_unit_bytes);
  p.off_epi = p.off_b + (uint32_t)((size_t)ns * p.stage_bytes);
  p.off_pix = p.off_epi + EPI_BYTES;
  p.off_tail = p.off_pix + (uint32_t)pix_bytes;
  pl.smem = (size_t)p.off_tail + kSmemTail;
  if (pl.smem > (size_t)kMaxDynSmem) return pl;
  if (pl.smem >= (1u << 18)) return pl;               // shared-memory descriptor address range
  if ((uint32_t)p.Rr * 16 >= (1u << 18)) return pl;   // leading-offset field range
  if (p.stage_bytes >= (1u << 20) || unit_exact >= (1u << 20)) return pl;  // mbarrier transaction counts
  pl.grid = dim3((unsigned)grid);
  // heuristic score: balance of the persistent CTAs x useful share of the staged rows
  const long long rounds = tiles_per_cta;
  double eff = (double)p.total_tiles / (double)(rounds * grid) * (double)grid / (double)(ew == 8 ? sms : 2 * sms);
  eff *= (double)(128 * MT) / (double)(128 * MT + p.halo);
  if (p.n_acc == 1 && rounds > 1) eff *= 0.8;   // epilogue cannot overlap the next tile's MMAs
  if (p.b_resident) eff *= 1.1;
  pl.score = eff;
  pl.ok = true;
  return pl;
}

constexpr int kPmVariants = 16;  // position-major variants come first, then the channel-major ones,
constexpr int kPmHalfVariants = 8;  // then the position-major kernel's half-size CTAs

// variant: 0 = heuristic; 1..15 = mt_code (1..3 -> 1,2,4) + 4*stage_code (0..3 -> 48,16,32,64 KB);
// half-size CTAs: 0..7 = mt_code' (0,1 -> 1,2) + 2*stage_code' (0..3 -> 8,16,24,32 KB)
static TcPlan make_plan(const Geom& g, int act_type, int variant, bool half_size = false) {
  TcPlan none{};
  none.ok = false;
  if (g.N < 1) return none;
  if (half_size) {
    static const int kbs[4] = {8, 16, 24, 32};
    return plan_for(g, act_type, 1 + (variant & 1), kbs[(variant >> 1) & 3], 4);
  }
  int want_mt = 0, want_stage_kb = 0;
  if (variant > 0) {
    static const int mts[4] = {0, 1, 2, 4};
    static const int kbs[4] = {0, 16, 32, 64};
    want_mt = mts[variant & 3];
    want_stage_kb = kbs[(variant >> 2) & 3];
  }
  if (int v = env_int("SNN_TC_MT", 0)) want_mt = v;
  if (int v = env_int("SNN_TC_STAGE_KB", 0)) want_stage_kb = v;
  if (want_mt == 1 || want_mt == 2 || want_mt == 4) return plan_for(g, act_type, want_mt, want_stage_kb, 8);
  TcPlan best = none;
  for (int mt = 1; mt <= 4; mt *= 2) {
    TcPlan c = plan_for(g, act_type, mt, want_stage_kb, 8);
    if (c.ok && (!best.ok || c.score > best.score)) best = c;
  }
  return best;
}

int tc_variant_count() { return kPmVariants + cm_variant_count() + kPmHalfVariants; }

bool tc_supported(const Geom& g, int act_type) {
  if (env_int("SNN_TC_DISABLE", 0)) return false;
  Geom gg = g;
  if (gg.N < 1) gg.N = 1;
  return make_plan(gg, act_type, 0).ok;
}

bool tc_variant_ok(const Geom& g, int act_type, int variant) {
  if (variant < 0 || variant >= tc_variant_count()) return false;
  if (variant >= kPmVariants + cm_variant_count()) {
    if (env_int("SNN_TC_NO_HALF", 0)) return false;
    return make_plan(g, act_type, variant - kPmVariants - cm_variant_count(), true).ok;
  }
  if (variant >= kPmVariants) return cm_variant_ok(g, act_type, variant - kPmVariants);
  if (variant > 0 && (variant & 3) == 0) return false;  // names no tile size
  return make_plan(g, act_type, variant).ok;
}

cudaError_t tc_forward(LayerDev& L, const Geom& g, int act_type, const Launch& l, int* launched, int* status_dev,
                       int variant) {
  {
    const int forced = env_int("SNN_TC_VARIANT", -1);  // test hook: run one variant regardless of tuning
    if (forced >= 0 && tc_variant_ok(g, act_type, forced)) variant = forced;
  }
  const int first_half = kPmVariants + cm_variant_count();
  if (l.out_i32 == 2 && variant >= kPmVariants && variant < first_half) variant = 0;  // packed signs: this kernel only
  if (variant >= kPmVariants && variant < first_half)
    return cm_forward(L, g, act_type, l, launched, status_dev, variant - kPmVariants);
  TcPlan pl = variant >= first_half ? make_plan(g, act_type, variant - first_half, true) : make_plan(g, act_type, variant);
  if (!pl.ok) return cudaErrorInvalidConfiguration;
  const bool f16 = act_type == SNN_ACT_F16;
  TcParams& p = pl.p;
  p.act = l.act;
  {
    // vector loads of a row's words need the base pointer and the row pitch aligned to the load
    const uintptr_t addr = (uintptr_t)l.act;
    if (f16) p.act_vec = (addr & 15) == 0 && (g.C & 7) == 0;
    else if (p.cb_chunks == 8) p.act_vec = (addr & 15) == 0 && (g.Cw & 3) == 0;
    else if (p.cb_chunks == 4) p.act_vec = (addr & 7) == 0 && (g.Cw & 1) == 0;
    else p.act_vec = 0;
  }
  p.wt = f16 ? (const uint8_t*)L.w16 : (const uint8_t*)L.w8;
  p.alpha = L.alpha;
  p.out = l.out;
  p.out_i32 = l.out_i32;
  p.status = status_dev;
  // The kernel is launched as a programmatic dependent of its predecessor in the stream: its
  // set-up and first weight loads overlap that kernel's tail, and it waits on the device for it
  // before it reads the activations or writes the output.
  const bool pdl = env_int("SNN_TC_PDL", 1) != 0;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg{};
  cfg.stream = l.stream;
  cfg.attrs = attr;
  cfg.numAttrs = pdl ? 1 : 0;
  cudaError_t e = cudaSuccess;
  cfg.gridDim = pl.grid;
  cfg.blockDim = dim3((unsigned)tc_threads(pl.ew));
  cfg.dynamicSmemBytes = pl.smem;
#define SNN_TC_LAUNCH(F, M, KP, E)                                                                 \
  do {                                                                                             \
    static unsigned long long done = 0;                                                            \
    e = allow_max_smem(tc_conv_kernel<F, M, KP, E>, &done);                                        \
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, tc_conv_kernel<F, M, KP, E>, p);            \
  } while (0)
#define SNN_TC_LAUNCH_K(F, M, E)                    \
  do {                                              \
    if (p.kpt == 4) SNN_TC_LAUNCH(F, M, 4, E);      \
    else if (p.kpt == 2) SNN_TC_LAUNCH(F, M, 2, E); \
    else SNN_TC_LAUNCH(F, M, 0, E);                 \
  } while (0)
  if (pl.ew == 4) {
    if (f16) {
      if (p.MT == 1) SNN_TC_LAUNCH_K(true, 1, 4);
      else SNN_TC_LAUNCH_K(true, 2, 4);
    } else {
      if (p.MT == 1) SNN_TC_LAUNCH_K(false, 1, 4);
      else SNN_TC_LAUNCH_K(false, 2, 4);
    }
  } else if (f16) {
    if (p.MT == 1) SNN_TC_LAUNCH_K(true, 1, 8);
    else if (p.MT == 2) SNN_TC_LAUNCH_K(true, 2, 8);
    else SNN_TC_LAUNCH_K(true, 4, 8);
  } else {
    if (p.MT == 1) SNN_TC_LAUNCH_K(false, 1, 8);
    else if (p.MT == 2) SNN_TC_LAUNCH_K(false, 2, 8);
    else SNN_TC_LAUNCH_K(false, 4, 8);
  }
#undef SNN_TC_LAUNCH_K
#undef SNN_TC_LAUNCH
  if (e != cudaSuccess) return e;
  *launched += 1;
  return cudaGetLastError();
}

}  // namespace snn
