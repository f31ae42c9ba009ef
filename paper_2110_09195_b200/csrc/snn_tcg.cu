// The tensor-core kernel: one or several sub-bit convolutions in ONE persistent launch.
//
// Each problem of a launch is the forward pass of Sec. 3 / Algorithm 1 for one layer (3x3, or the 1x1
// extension of the appendix) on its own input: decoded +1/-1 weights as 4-bit e2m1 operands (binary
// activations) or fp16 operands (fp16 activations), implicit GEMM over a padded, flattened position space
// in which the nine taps are the same staged activations read from shifted start addresses.  One CTA per
// SM walks through all problems without any grid-wide step in between: while the MMAs of one problem's
// last tile run, the expander warps already stage the next problem's first activations, the weight
// producer streams its first stages, and the epilogue warps still drain the tile before.  Start-up, first
// loads and last drain, which cost a single-layer launch about as much as its MMAs at batch 64, are paid
// once per launch.  A single layer is a launch of one problem.
//
// Independent problems (a group) need nothing else.  A chain (a stack: problem i + 1 reads the packed signs
// problem i writes) runs in the same launch on per-tile completion counters: the epilogue bumps the counter
// of a tile's row block when its part is written, and the expanders of the successor wait (bounded) until the
// row blocks under a tile's input window are complete.  The launch is cooperative then, so that all CTAs are
// resident while some of them wait.
//
// What makes this possible is a ring geometry that is the same for every problem:
//   activation units  NA slots of a_slot_bytes   (a problem's unit uses a prefix)
//   weight stages     NS slots of b_slot_bytes   (a stage = whole taps of one channel block)
//   accumulators      two or three buffers of tensor-memory columns (by operand mode and output kind:
//                     3 x 160 for word outputs on e2m1 operands, else 2 x 240; 2 x 256 with fp16 operands)
// so slots, barriers and phases simply carry on from one problem to the next.
// Tiles of a problem are dealt to the CTAs round-robin; which CTAs get a problem's odd
// tiles is decided on the host from the time the CTAs have been given so far, so that the
// CTAs end close together.
//
//      warp 0        one thread streams weight stages (cp.async.bulk onto mbarriers)
//      warp 1        issues tcgen05.mma and commits barriers (warp-uniform, one elected lane)
//      warps 2-9     epilogue: TMEM -> registers -> shared-memory transposition -> alpha ->
//                    128-byte row stores; or TMEM -> registers -> threshold -> packed sign words
//      warps 10-19   expanders (13 and 17 idle): packed bits -> e2m1 nibbles (or fp16 copied)
//                    into the activation ring
// The kernel is compiled per operand mode and per output kind (words, the common case of words alone, packed
// signs, chain), so that no variant carries another one's code in its loops; the plan (tile shapes, accumulator
// buffers) is made per output kind as well.
// Every wait is bounded; one that runs out raises a status word the host reads, and
// the CTA still frees its tensor memory and returns.
#include <algorithm>
#include <cstdio>
#include <vector>

#include "snn_tc_common.cuh"

namespace snn {

namespace {

// Operand modes of the kernel.  Binary activations run on 4-bit e2m1 operands (+1 / -1 / 0 are exact, the
// block scales are all 1, and the fp32 accumulators hold the exact integer sums: |S| <= 9 * c_in < 2^24);
// an MMA then covers 64 input channels in the time an 8-bit MMA covers 32.  fp16 activations run on fp16
// operands.  Both accumulate in fp32.
enum { M_F16 = 1, M_FP4 = 2 };
constexpr int G_EW = 8;                       // epilogue warps = expander warps

// Warps 13 and 17 stay idle: a warp's scheduler is warp % 4, and the MMA-issuing warp (1) then
// shares its scheduler with two epilogue warps only instead of two epilogue and two expander warps.
constexpr int G_THREADS = 64 + 64 * G_EW + 64;
constexpr int G_EXP_THREADS = 32 * G_EW;
constexpr int G_XTEAMS = 2;                    // teams of expander warps in the pipelined form
constexpr int G_EXP_ROWS = 3;                 // rows of a unit one expander thread loads together
constexpr int G_EPI_PITCH = 128;
constexpr int G_EPI_ALPHA = 1024;              // per epilogue warp: the scales of a tile's channels (at most 256)
constexpr int G_EPI_WARP = 32 * G_EPI_PITCH + G_EPI_ALPHA;
constexpr int G_EPI_BYTES = G_EW * G_EPI_WARP;
constexpr int G_NS_MAX = 8;
constexpr uint32_t G_ACC_COLS = 256;          // tensor-memory columns of one accumulator buffer
constexpr uint32_t G_ACC_COLS_FP4 = 240;      // 4-bit mode, two buffers: columns 480..511 hold the (unit) block scales
constexpr uint32_t G_ACC_COLS_FP4_3 = 160;    // 4-bit mode, three buffers
// Accumulator buffers.  Word outputs on 4-bit operands use three: the MMAs of the tile after next run while both
// epilogue groups still drain, so a group never waits for them (the epilogue is what bounds that variant).  The
// other variants are bound elsewhere and do better with two larger buffers (larger tiles).
constexpr int G_NACC = 2, G_NACC_WORDS = 3;
constexpr uint32_t G_SCALE_COL = 480;
constexpr size_t kGTail = 512;
constexpr size_t kGSmemBudget = 226 * 1024;
constexpr uint32_t kGASlotMax = 40 * 1024 + 512;   // largest activation unit a problem may stage
constexpr uint32_t kGBSlot = 32 * 1024;            // bytes of a weight-stage slot

// One problem of a group, as the kernel reads it from global memory.
struct GLayer {
  const uint8_t* wt;      // [layout tile][channel block][tap][chunk][NtL][16 B], owned by the group
  const float* alpha;
  const float* shift;     // per-channel constant added to alpha*S before the sign is taken (packed-sign output)
  int N, H, W, C, K, Cw, stride, pad, Ho, Wo;
  int NtL, Nt;            // channels per layout tile of the weight operand / per tile
  int Hq, Wq;             // rows per image / row pitch of the flattened position space
  FastDiv dWq, dHq, dNt;
  int n_planes, halo, Rr; // 1 or 4 planes; largest tap shift; staged rows per plane = 128*MT + halo
  int MT;                 // M sub-tiles of 128 positions per tile
  int cb_chunks, n_cb, kpt;
  int taps;               // 9 (3x3 layers) or 1 (the 1x1 extension)
  int st_taps;            // taps per weight stage (the last stage of a channel block holds taps % st_taps, if not 0)
  uint32_t tap_bytes;     // weights of one tap of one channel block and channel tile = kpt * 2 * Nt * 16
  int n_ntiles, total_tiles;
  const uint16_t* rank;   // [grid] CTA b takes this problem's tiles rank[b], rank[b] + grid, ...
  long long Qtot;
  // A chain (every member reads the packed signs its predecessor writes, all in one launch): a tile may be
  // staged once the predecessor's tiles that hold its input pixels are complete, and says so itself when done.
  const uint2* deps;          // [M groups] first and last M group of the predecessor this M group reads (x > y: none)
  const uint32_t* prev_done;  // the predecessor's completion counters, and the count that means "complete"
  uint32_t prev_target;
  uint32_t* done;             // [M groups] epilogue warps that have finished the group, over all its channel tiles
};

struct GParams {
  const GLayer* layers;
  int n_layers;
  const void* act[SNN_GROUP_MAX];
  void* out[SNN_GROUP_MAX];
  int* status;
  uint8_t out_type[SNN_GROUP_MAX];   // per member: 0 fp32 alpha*S, 1 int32 S, 2 packed signs of alpha*S + shift
  uint32_t acc_cols;      // tensor-memory columns of one accumulator buffer
  int n_acc;              // accumulator buffers (tile seq of a CTA uses buffer seq % n_acc)
  int NA, NS;
  uint32_t a_slot_bytes, b_slot_bytes;
  uint32_t off_b, off_epi, off_pix, off_lay, off_tail;
  uint32_t pix_words;     // entries of one pixel table (the pipelined expanders keep one per team)
};

// Profiling aid (build with -DSNN_TRACE): every role's reporting lane adds up the cycles it spends in its
// waits; the host prints the averages over the CTAs after each launch.  No effect on an ordinary build.
#ifdef SNN_TRACE
__device__ long long g_trace[256 * 16];
#define TR_WAIT(var, expr) ([&]() { const long long _t = clock64(); const bool _r = (expr); var += clock64() - _t; return _r; }())
#define TR_BEGIN(t) const long long t = clock64()
#define TR_END(var, t) var += clock64() - t
#define TR_REPORT(role, total, w0, w1, w2)                         \
  do {                                                             \
    long long* _o = g_trace + (size_t)blockIdx.x * 16 + (role)*4;  \
    _o[0] = (total); _o[1] = (w0); _o[2] = (w1); _o[3] = (w2);     \
  } while (0)
#else
#define TR_WAIT(var, expr) (expr)
#define TR_BEGIN(t) do { } while (0)
#define TR_END(var, t) do { } while (0)
#define TR_REPORT(role, total, w0, w1, w2) do { } while (0)
#endif

__device__ __forceinline__ int g_position_to_pixel(const GLayer& L, uint32_t q, int pa, int pb) {
  if ((long long)q >= L.Qtot) return -1;
  const uint32_t rg = fdiv(q, L.dWq);
  const int j = (int)(q - rg * (uint32_t)L.Wq);
  const uint32_t n = fdiv(rg, L.dHq);
  const int i = (int)(rg - n * (uint32_t)L.Hq);
  if ((int)n >= L.N) return -1;
  const int r = L.stride * i + pa - L.pad, c = L.stride * j + pb - L.pad;
  if (r < 0 || r >= L.H || c < 0 || c >= L.W) return -1;
  return ((int)n * L.H + r) * L.W + c;
}

// Bounded wait until a completion counter another CTA advances has reached `target` (acquire: what that CTA
// wrote before is visible afterwards).  False when the limit ran out or the CTA is giving up.
__device__ __forceinline__ bool g_wait_counter(const uint32_t* ctr, uint32_t target, volatile int* abort_flag) {
  for (uint32_t it = 0; it < (1u << 21); ++it) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if (*abort_flag) return false;
    __nanosleep(100);
  }
  return false;
}
// Activation words: through the read-only path, or - when another CTA of this launch wrote them - from L2.
__device__ __forceinline__ uint32_t g_ld1(const uint32_t* p, bool fresh) { return fresh ? __ldcg(p) : __ldg(p); }
__device__ __forceinline__ uint2 g_ld2(const uint32_t* p, bool fresh) {
  return fresh ? __ldcg(reinterpret_cast<const uint2*>(p)) : __ldg(reinterpret_cast<const uint2*>(p));
}
__device__ __forceinline__ uint4 g_ld4(const uint32_t* p, bool fresh) {
  return fresh ? __ldcg(reinterpret_cast<const uint4*>(p)) : __ldg(reinterpret_cast<const uint4*>(p));
}

// first tile of problem L for this CTA (tiles then follow at a stride of the grid)
__device__ __forceinline__ int g_first_tile(const GLayer& L) {
  return (int)__ldg(L.rank + blockIdx.x);
}

// The MMAs of one channel block of one tile: 9 taps x KPT K steps x MT sub-tiles.  The body of
// a tap is straight-line code; the taps are a loop, because the issuing thread runs alone on
// its warp and nine unrolled taps no longer fit the instruction cache closest to it.
// Weight stages are waited for and released as the K-step counter crosses their boundaries.
template <int MODE, int MT, int KPT>
__device__ __forceinline__ bool g_issue_block(uint64_t a_unit, uint32_t wq, uint32_t plane_units, bool s2, uint32_t a_step,
                                              uint64_t b_desc0, uint32_t b_slot_units, uint32_t b_step, uint32_t d0,
                                              uint32_t nt, uint32_t idesc, uint32_t& acc, int taps, int st_taps, int NS,
                                              uint32_t bar_bfull, uint32_t bar_bempty, int& b_slot, uint32_t& b_phase,
                                              bool leader, uint32_t sf, long long& tr_b) {
  uint32_t ky = 0, kx = 0;
  int t = 0;
#pragma unroll 1
  while (t < taps) {
    // a weight stage holds whole taps: one wait, then nothing but MMAs until its last tap
    if (!TR_WAIT(tr_b, mbar_wait(bar_bfull + 8 * b_slot, b_phase))) return false;
    tc_fence_after();
    uint64_t bd = b_desc0 + (uint64_t)((uint32_t)b_slot * b_slot_units);
    const int t_end = t + st_taps < taps ? t + st_taps : taps;
#pragma unroll 1
    for (; t < t_end; ++t) {
      // rows (16-byte units) from a unit's origin to tap (ky, kx): a shift inside the plane, plus, for stride 2,
      // the offset of the tap's parity plane
      const uint32_t tap = s2 ? ((ky & 1u) * 2u + (kx & 1u)) * plane_units + (ky >> 1) * wq + (kx >> 1) : ky * wq + kx;
      if (++kx == 3) { kx = 0; ++ky; }
      const uint64_t ad_t = a_unit + (uint64_t)tap;
      if (leader) {
#pragma unroll
        for (int k = 0; k < KPT; ++k) {
#pragma unroll
          for (int mt = 0; mt < MT; ++mt) {
            const uint64_t ad = ad_t + (uint64_t)((uint32_t)k * a_step + (uint32_t)(mt * 128));
            const uint64_t bdk = bd + (uint64_t)((uint32_t)k * b_step);
            const uint32_t accum = k == 0 ? acc : 1u;
            if (MODE == M_FP4) mma_ss_fp4(d0 + (uint32_t)mt * nt, ad, bdk, idesc, accum, sf, sf + 16);
            else mma_ss_f16(d0 + (uint32_t)mt * nt, ad, bdk, idesc, accum);
          }
        }
      }
      acc = 1;
      bd += (uint64_t)((uint32_t)KPT * b_step);
    }
    if (leader) tc_commit(bar_bempty + 8 * b_slot);  // the slot is free once these MMAs have read it
    if (++b_slot == NS) { b_slot = 0; b_phase ^= 1u; }
  }
  return true;
}

}  // namespace

// OUTK: what the epilogue is compiled for.  0: fp32 or int32 words for every member; 1: packed signs for every
// member; 2: a chain - packed signs between the members, any type for the last, and the dependency waits and
// completion counters.  Keeping the variants apart keeps each one's registers and code to what it needs.
// 3: the common case of 0 compiled alone - fp32 outputs, 4-bit operands, every member's channel count a multiple
// of 4 and its channel tile a multiple of 32, rows readable two words at a time: the expanders run their
// two-stage load pipeline instead of the plain loop, and the epilogue has its one fast path and no other.  The
// roles share instruction caches; what a variant does not carry makes the rest faster.
enum { OUT_WORDS = 0, OUT_SIGNS = 1, OUT_CHAIN = 2, OUT_WORDS_PIPED = 3 };

template <int MODE, int OUTK>
__global__ void __launch_bounds__(G_THREADS, 1) tcg_conv_kernel(const GParams p) {
  constexpr bool F16 = MODE == M_F16;   // fp16 activations (copied, not expanded)
  constexpr bool FP4 = MODE == M_FP4;   // binary activations as e2m1 nibbles
  constexpr bool CHAIN = OUTK == OUT_CHAIN;
  constexpr bool WORDS = OUTK == OUT_WORDS || OUTK == OUT_WORDS_PIPED;
  constexpr bool PIPED = OUTK == OUT_WORDS_PIPED;
  // Word outputs (fp32 / int32) are bound by the stores: there the epilogue warps form two groups of four (one
  // warp per quarter of the accumulator's lanes) that take the tiles in turn, group g draining accumulator
  // buffer g, so that one group's stores drain while the other reads tensor memory and transposes.  Packed
  // signs are bound by the epilogue's instructions: all eight warps drain every tile together.
  constexpr bool G_EPI_SPLIT = WORDS;
  constexpr int G_EPI_ARRIVALS = G_EPI_SPLIT ? G_EW / 2 : G_EW;   // epilogue warps that drain one tile
  extern __shared__ __align__(128) uint8_t smem[];
  // carve-up: [NA activation slots][NS weight slots][epilogue tiles][pixel table][problem table][barriers, flags]
  uint8_t* a_smem = smem;
  uint8_t* b_smem = smem + p.off_b;
  uint8_t* epi_smem = smem + p.off_epi;
  int* pix_tab = reinterpret_cast<int*>(smem + p.off_pix);
  // The problems' descriptions are read from shared memory where they are needed instead of
  // being held in registers: the roles are at different problems at the same time, and the
  // epilogue's registers are all taken by the slices it transposes.
  const GLayer* lay = reinterpret_cast<const GLayer*>(smem + p.off_lay);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + p.off_tail);
  // barriers: b_full[8] b_empty[8] a_full[4] a_empty[4] acc_full[4] acc_empty[3]
  // acc_full is indexed by the tile's sequence number in the CTA (seq % 4), not by the buffer: an epilogue group
  // that takes every other tile then sees every phase of the barriers it waits on (seq % 4 = g and g + 2), and a
  // barrier's next phase cannot complete before its last one was consumed (tile seq + 3 needs the buffer tile seq
  // releases).  acc_empty is per buffer.
  const uint32_t bar_bfull = smem_u32(bars), bar_bempty = smem_u32(bars + 8);
  const uint32_t bar_afull = smem_u32(bars + 16), bar_aempty = smem_u32(bars + 20);
  const uint32_t bar_accfull = smem_u32(bars + 24), bar_accempty = smem_u32(bars + 28);
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 31);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int NS = p.NS, NA = p.NA;
  const int G = (int)gridDim.x;

  if (tid < 31) {
    uint32_t count = 1;
    if (tid >= 28) count = G_EPI_ARRIVALS;             // acc_empty: one arrival per epilogue warp of the tile
    if (tid >= 16 && tid < 20)   // a_full: every expander thread arrives, or one lane per expander warp (pipelined form)
      count = PIPED ? G_EXP_THREADS / 32 / G_XTEAMS : G_EXP_THREADS;
    mbar_init(smem_u32(bars + tid), count);
  }
  if (tid == 32) *abort_flag = 0;
  {
    const uint32_t* src = reinterpret_cast<const uint32_t*>(p.layers);
    uint32_t* dst = reinterpret_cast<uint32_t*>(smem + p.off_lay);
    const int words = p.n_layers * (int)(sizeof(GLayer) / 4);
    for (int i = tid; i < words; i += G_THREADS) dst[i] = __ldg(src + i);
  }
  if (warp == 2) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"(512)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  grid_dep_launch();
  if (FP4) {
    // unit block scales: every byte of the scale columns is the ue8m0 code of 1.0, in all 128 lanes
    // (warps 2..5 cover the four lane quarters), whatever part of them an MMA reads
    if (warp >= 2 && warp < 6) tmem_fill32(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + G_SCALE_COL, 0x7f7f7f7fu);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
  }

  if (warp == 0) {
    // ------------------------------------------------ weight producer (one lane)
    if (lane == 0) {
      int b_slot = 0;
      long long b_issued = 0;
      uint32_t b_phase = 1;  // parity of the previous use of a slot (valid from the second lap)
      bool ok = true;
      long long tr_w0 = 0, tr_t0 = clock64();
      (void)tr_w0; (void)tr_t0;
      for (int l = 0; l < p.n_layers && ok; ++l) {
        const GLayer& L = lay[l];
        const int Nt = L.Nt, NtL = L.NtL, n_cb = L.n_cb, n_ntiles = L.n_ntiles, total = L.total_tiles;
        const int taps = L.taps, st_taps = L.st_taps, stages_per_cb = (taps + st_taps - 1) / st_taps;
        const int chunks_per_tap = 2 * L.kpt;
        const uint32_t tap_bytes = L.tap_bytes;
        const uint8_t* wt = L.wt;
        const size_t cb_bytes = (size_t)taps * L.cb_chunks * NtL * 16;   // one channel block of one layout tile
        const FastDiv dNt = L.dNt;
        for (int tile = g_first_tile(L); tile < total && ok; tile += G) {
          if (*abort_flag) { ok = false; break; }
          const int nti = tile - (int)fdiv((uint32_t)tile, dNt) * n_ntiles;
          const int n0 = nti * Nt;
          const int ltile = Nt == NtL ? nti : n0 / NtL;
          const int n_in = n0 - ltile * NtL;
          const uint8_t* src_tile = wt + (size_t)ltile * n_cb * cb_bytes + (size_t)n_in * 16;
          for (int cb = 0; cb < n_cb && ok; ++cb) {
            const uint8_t* src = src_tile + (size_t)cb * cb_bytes;
            for (int sg = 0; sg < stages_per_cb; ++sg) {
              const int ntaps = taps - sg * st_taps < st_taps ? taps - sg * st_taps : st_taps;
              const uint32_t stage_bytes = (uint32_t)ntaps * tap_bytes;
              const int chunks_per_stage = ntaps * chunks_per_tap;
              if (b_issued >= NS && !TR_WAIT(tr_w0, mbar_wait_backoff(bar_bempty + 8 * b_slot, b_phase, 32))) { ok = false; break; }
              const uint32_t dst = smem_u32(b_smem) + (uint32_t)b_slot * p.b_slot_bytes;
              mbar_expect_tx(bar_bfull + 8 * b_slot, stage_bytes);
              if (Nt == NtL) {
                bulk_g2s(dst, src, stage_bytes, bar_bfull + 8 * b_slot);  // the stage's chunks are contiguous
              } else {
                for (int c = 0; c < chunks_per_stage; ++c)
                  bulk_g2s(dst + (uint32_t)c * Nt * 16, src + (size_t)c * NtL * 16, (uint32_t)Nt * 16,
                           bar_bfull + 8 * b_slot);
              }
              src += (size_t)chunks_per_stage * NtL * 16;
              ++b_issued;
              if (++b_slot == NS) { b_slot = 0; b_phase ^= 1u; }
            }
          }
        }
      }
      if (!ok && !*abort_flag) {
        *abort_flag = 1;
        raise_status(p.status, 2);
      }
      TR_REPORT(0, clock64() - tr_t0, tr_w0, 0, 0);
      // never leave with copies in flight: wait (bounded) for the last load of every slot
      for (int s = 0; s < NS; ++s) {
        long long last = -1;
        if (b_issued > s) last = s + (b_issued - 1 - s) / NS * NS;
        if (last >= 0) mbar_wait_backoff(bar_bfull + 8 * s, (uint32_t)((last / NS) & 1), 64);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    // The whole warp walks the loops and waits together, so that every address and descriptor
    // is a warp-uniform value; one elected lane issues the MMAs and the commits.
    {
      const bool leader = elect_one();
      bool ok = true;
      int a_slot = 0, b_slot = 0, acc_slot = 0, full_slot = 0;
      uint32_t a_phase = 0, b_phase = 0, acc_phase = 1;
      const int n_acc = p.n_acc;
      long long tiles_done = 0;
      long long tr_w0 = 0, tr_w1 = 0, tr_w2 = 0, tr_t0 = clock64();
      (void)tr_w0; (void)tr_w1; (void)tr_w2; (void)tr_t0;
      const uint32_t a_slot_units = p.a_slot_bytes >> 4, b_slot_units = p.b_slot_bytes >> 4;
      for (int l = 0; l < p.n_layers && ok; ++l) {
        const GLayer& L = lay[l];
        const int Nt = L.Nt, Rr = L.Rr, n_cb = L.n_cb, MT = L.MT, kpt = L.kpt, total = L.total_tiles;
        const int st_taps = L.st_taps;
        // instruction descriptor: D format, A/B formats, K-major both, N>>3, M>>4
        // (4-bit mode: A/B format e2m1, scale format ue8m0, scale ids 0)
        const uint32_t idesc =
            F16 ? ((1u << 4) | ((uint32_t)(Nt >> 3) << 17) | ((128u >> 4) << 24))
                : ((1u << 7) | (1u << 10) | ((uint32_t)(Nt >> 3) << 17) | (1u << 23) | ((128u >> 4) << 24));
        const uint64_t a_desc0 = make_desc(smem_u32(a_smem), (uint32_t)Rr * 16, 128);
        const uint64_t b_desc0 = make_desc(smem_u32(b_smem), (uint32_t)Nt * 16, 128);
        const uint32_t a_step = 2u * (uint32_t)Rr, b_step = 2u * (uint32_t)Nt;  // two chunks per MMA
        for (int tile = g_first_tile(L); tile < total && ok; tile += G, ++tiles_done) {
          if (tiles_done >= n_acc) {
            if (!TR_WAIT(tr_w0, mbar_wait(bar_accempty + 8 * acc_slot, acc_phase))) { ok = false; break; }
            tc_fence_after();
          }
          const uint32_t d0 = tmem_base + (uint32_t)acc_slot * p.acc_cols;
          uint32_t acc = 0;  // 0 only for the first MMA of every sub-tile
          for (int cb = 0; cb < n_cb && ok; ++cb) {
            if (!TR_WAIT(tr_w1, mbar_wait(bar_afull + 8 * a_slot, a_phase))) { ok = false; break; }
            tc_fence_after();
            const uint64_t a_unit = a_desc0 + (uint64_t)((uint32_t)a_slot * a_slot_units);
#define G_ISSUE(M, KP)                                                                                       \
  ok = g_issue_block<MODE, M, KP>(a_unit, (uint32_t)L.Wq, (uint32_t)(L.cb_chunks * Rr), L.stride != 1, a_step, b_desc0, b_slot_units, b_step, d0, (uint32_t)Nt, idesc, acc, \
                                  L.taps, st_taps, NS, bar_bfull, bar_bempty, b_slot, b_phase, leader,                   \
                                  tmem_base + G_SCALE_COL, tr_w2)
#define G_ISSUE_K(M)                   \
  do {                                 \
    if (kpt == 4) G_ISSUE(M, 4);       \
    else if (kpt == 2) G_ISSUE(M, 2);  \
    else if (kpt == 3) G_ISSUE(M, 3);  \
    else G_ISSUE(M, 1);                \
  } while (0)
            if (MT == 4) G_ISSUE_K(4);
            else if (MT == 3) G_ISSUE_K(3);
            else if (MT == 2) G_ISSUE_K(2);
            else G_ISSUE_K(1);
#undef G_ISSUE_K
#undef G_ISSUE
            if (!ok) break;
            if (leader) tc_commit(bar_aempty + 8 * a_slot);  // the activation unit may be overwritten
            if (++a_slot == NA) { a_slot = 0; a_phase ^= 1u; }
          }
          if (!ok) break;
          if (leader) tc_commit(bar_accfull + 8 * full_slot);  // fires when this tile's MMAs are complete
          full_slot = (full_slot + 1) & 3;
          if (++acc_slot == n_acc) { acc_slot = 0; acc_phase ^= 1u; }
        }
      }
      if (!ok && leader && !*abort_flag) {
        *abort_flag = 1;
        raise_status(p.status, 3);
      }
      if (leader) TR_REPORT(1, clock64() - tr_t0, tr_w0, tr_w1, tr_w2);
    }
    __syncwarp();
  } else if (warp < 2 + G_EW) {
    // ------------------------------------------------ epilogue warps
    grid_dep_wait();  // an earlier kernel in the stream may still read the output buffers
    // Warp w reads TMEM lanes 32*(w%4).. (rows of the tile); the two warps of a lane quarter take
    // the 32-column slices in turn.  A slice goes through a per-warp shared-memory tile so that
    // each store instruction writes whole 128-byte rows.
    const int ew = warp - 2;
    const int rq = warp & 3, half = ew >> 2;
    const int cfirst = G_EPI_SPLIT ? 0 : 32 * half, cstep = G_EPI_SPLIT ? 32 : 64;   // this warp's 32-column slices
    long long seq = 0;   // tiles of this CTA so far, over all problems (the MMA issuer alternates the buffers the same way)
    uint8_t* stage = epi_smem + (size_t)ew * G_EPI_WARP;
    const uint32_t a_stage = smem_u32(stage) + 32 * G_EPI_PITCH;   // this warp's copy of the tile's scales
    const int srow = lane >> 3, scol = lane & 7;  // this lane's (row mod 4, 16-byte column) when storing
    // Staging tile: row r, 16-byte chunk c sits at r*128 + ((c ^ (r & 7)) << 4).  A lane writes its own row
    // (chunk e at st_lane ^ (e << 4)) and reads chunk scol of rows srow + 4i.
    const uint32_t st_lane = smem_u32(stage) + (uint32_t)(lane * G_EPI_PITCH + ((lane & 7) << 4));
    const uint32_t ld_even = smem_u32(stage) + (uint32_t)(srow * G_EPI_PITCH + ((scol ^ srow) << 4));
    const uint32_t ld_odd = smem_u32(stage) + (uint32_t)((srow + 4) * G_EPI_PITCH + ((scol ^ (srow + 4)) << 4));
    (void)st_lane; (void)ld_even; (void)ld_odd;
    int acc_slot = 0;   // buffer of tile seq: seq % n_acc, kept in step with seq
    const int n_acc = p.n_acc;
    bool live = true;
    long long tr_w0 = 0, tr_w1 = 0, tr_w2 = 0, tr_t0 = clock64();
    (void)tr_w0; (void)tr_w1; (void)tr_w2; (void)tr_t0;
    for (int l = 0; l < p.n_layers && live; ++l) {
      const GLayer& L = lay[l];
      const int Nt = L.Nt, MT = L.MT, K = L.K;
      const float* alpha = L.alpha;
      const float* shift = L.shift;
      const int out_i32 = PIPED ? 0 : WORDS ? (int)p.out_type[0] : OUTK == OUT_SIGNS ? 2 : (int)p.out_type[l];
      uint32_t* out32 = reinterpret_cast<uint32_t*>(p.out[l]);  // int32 and fp32 outputs share the layout
      const bool fast = PIPED || (((K & 3) == 0) && ((Nt & 31) == 0));   // (checked on the host for variant 3)
      for (int tile = g_first_tile(L); tile < L.total_tiles; tile += G, ++seq, acc_slot = acc_slot + 1 == n_acc ? 0 : acc_slot + 1) {
        if (G_EPI_SPLIT && (int)(seq & 1) != half) continue;   // the other group's tile
        const uint32_t full_bar = bar_accfull + 8u * (uint32_t)(seq & 3), full_phase = (uint32_t)((seq >> 2) & 1);
        const int mg = (int)fdiv((uint32_t)tile, L.dNt), nti = tile - mg * L.n_ntiles;
        const uint32_t Q0 = (uint32_t)mg * (uint32_t)(128 * MT);
        const int n0 = nti * Nt;
        int okw = 1;
        if (lane == 0) okw = (!*abort_flag && TR_WAIT(tr_w0, mbar_wait_backoff(full_bar, full_phase, 100))) ? 1 : 0;
        okw = __shfl_sync(0xffffffffu, okw, 0);
        if (!okw) {
          if (lane == 0 && !*abort_flag) {
            *abort_flag = 1;
            raise_status(p.status, 4);
          }
          live = false;
          break;
        }
        tc_fence_after();
        const uint32_t d0 = tmem_base + (uint32_t)acc_slot * p.acc_cols;
        // output pixel (n*Ho + y)*Wo + x of the row of sub-tile mt this lane owns in TMEM, or -1
        auto row_pixel = [&](int mt) -> int {
          const uint32_t q = Q0 + (uint32_t)(mt * 128 + rq * 32 + lane);
          const uint32_t rg = fdiv(q, L.dWq);
          const int x = (int)(q - rg * (uint32_t)L.Wq);
          const uint32_t n = fdiv(rg, L.dHq);
          const int y = (int)(rg - n * (uint32_t)L.Hq);
          const bool valid = ((long long)q < L.Qtot) && ((int)n < L.N) && (y < L.Ho) && (x < L.Wo);
          return valid ? ((int)n * L.Ho + y) * L.Wo + x : -1;
        };
        if (!WORDS && out_i32 == 2) {
          // Packed signs of the scaled output (Algorithm 1: the next layer consumes sign(a)): a thread
          // owns one position and the 32 (or 16) consecutive channels of a slice, i.e. one word (or
          // half-word) of the next layer's binary input.  No transposition, one small store per slice.
          const int Kw = (K + 31) >> 5;
          // the scale and threshold arrays can be read four at a time (their allocations are; a tile starts at a multiple of 16)
          const bool sign_vec = ((reinterpret_cast<uintptr_t>(alpha) | reinterpret_cast<uintptr_t>(shift)) & 15) == 0;
          if ((Nt & 31) == 0) {
            const int per_mt = (Nt - cfirst + cstep - 1) / cstep;
#pragma unroll 1
            for (int mt = 0; mt < MT; ++mt) {
              const int pix = row_pixel(mt);
#pragma unroll 1
              for (int ci = 0; ci < per_mt; ++ci) {
                const int c0 = cfirst + cstep * ci, co0 = n0 + c0;
                uint32_t v[32];
                __syncwarp();  // the load is a warp-wide instruction: no lane may still be in the store below
                tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * Nt + c0), v);
                tmem_ld_wait();
                if (pix >= 0 && co0 + 32 <= K && sign_vec) {
                  // all 32 channels exist: scales and thresholds four at a time (the same addresses in every
                  // lane), multiply and add as packed fp32 pairs - each half rounds as the scalar instruction does
                  uint32_t word = 0;
#pragma unroll
                  for (int e = 0; e < 32; e += 4) {
                    const float4 a = __ldg(reinterpret_cast<const float4*>(alpha + co0 + e));
                    const float4 t = __ldg(reinterpret_cast<const float4*>(shift + co0 + e));
                    unsigned long long x0, x1, m0, m1, t0, t1;
                    asm("mov.b64 %0, {%1, %2};" : "=l"(x0) : "r"(v[e]), "r"(v[e + 1]));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(x1) : "r"(v[e + 2]), "r"(v[e + 3]));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(m0) : "f"(a.x), "f"(a.y));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(m1) : "f"(a.z), "f"(a.w));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(t0) : "f"(t.x), "f"(t.y));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(t1) : "f"(t.z), "f"(t.w));
                    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(x0) : "l"(m0));
                    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(x1) : "l"(m1));
                    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(x0) : "l"(t0));
                    asm("add.rn.f32x2 %0, %0, %1;" : "+l"(x1) : "l"(t1));
                    float y0, y1, y2, y3;
                    asm("mov.b64 {%0, %1}, %2;" : "=f"(y0), "=f"(y1) : "l"(x0));
                    asm("mov.b64 {%0, %1}, %2;" : "=f"(y2), "=f"(y3) : "l"(x1));
                    word |= (y0 >= 0.f ? 1u : 0u) << e;
                    word |= (y1 >= 0.f ? 1u : 0u) << (e + 1);
                    word |= (y2 >= 0.f ? 1u : 0u) << (e + 2);
                    word |= (y3 >= 0.f ? 1u : 0u) << (e + 3);
                  }
                  out32[wide_mul((uint32_t)pix, (uint32_t)Kw) + (uint32_t)(co0 >> 5)] = word;
                } else if (pix >= 0 && co0 < K) {
                  uint32_t word = 0;
#pragma unroll
                  for (int e = 0; e < 32; ++e) {
                    const float a = co0 + e < K ? __ldg(alpha + co0 + e) : -1.f;  // a missing channel gives bit 0 ...
                    const float s = co0 + e < K ? __uint_as_float(v[e]) : 1.f;     // ... through 1 * -1 + 0 < 0
                    const float t = co0 + e < K ? __ldg(shift + co0 + e) : 0.f;
                    word |= (__fadd_rn(__fmul_rn(s, a), t) >= 0.f ? 1u : 0u) << e;
                  }
                  out32[wide_mul((uint32_t)pix, (uint32_t)Kw) + (uint32_t)(co0 >> 5)] = word;
                }
              }
            }
          } else {
            // one channel tile whose width is an odd multiple of 16: half-words; the slice that ends
            // the tile also clears the half-word behind it, so that every word is written in full
            uint16_t* out16 = reinterpret_cast<uint16_t*>(out32);
#pragma unroll 1
            for (int mt = 0; mt < MT; ++mt) {
              const int pix = row_pixel(mt);
              for (int c0 = G_EPI_SPLIT ? 0 : 16 * half; c0 < Nt; c0 += G_EPI_SPLIT ? 16 : 32) {
                uint32_t v[16];
                __syncwarp();
                tmem_ld16(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * Nt + c0), v);
                tmem_ld_wait();
                const int co0 = n0 + c0;
                if (pix >= 0) {
                  uint32_t hw = 0;
#pragma unroll
                  for (int e = 0; e < 16; ++e) {
                    const float a = co0 + e < K ? __ldg(alpha + co0 + e) : -1.f;
                    const float s = co0 + e < K ? __uint_as_float(v[e]) : 1.f;
                    const float t = co0 + e < K ? __ldg(shift + co0 + e) : 0.f;
                    hw |= (__fadd_rn(__fmul_rn(s, a), t) >= 0.f ? 1u : 0u) << e;
                  }
                  const size_t at = wide_mul((uint32_t)pix, (uint32_t)(2 * Kw)) + (uint32_t)(co0 >> 4);
                  if ((co0 >> 4) < 2 * Kw) out16[at] = (uint16_t)hw;
                  if (c0 + 16 >= Nt && (co0 >> 4) + 1 < 2 * Kw) out16[at + 1] = 0;
                }
              }
            }
          }
        } else if (OUTK == OUT_SIGNS) {
          // (packed signs only: nothing else is compiled into this variant)
        } else if (fast) {
          // The warp's slices (sub-tile mt, columns c0..c0+31) form one sequence; the TMEM load of slice s+1 is
          // issued as soon as slice s sits in the staging tile.  The loop is written for few instructions (this
          // role is bound by how many it issues): shared-memory addresses are fixed per lane, values travel as
          // 64-bit pairs from the staging tile through the packed fp32 multiply to the 16-byte store, and a row's
          // place in the output is one 32-bit element offset per sub-tile.
          const int per_mt = (Nt - cfirst + cstep - 1) / cstep;
          const int total_sl = MT * per_mt;
          uint32_t v[32];
          uint32_t roff[8];   // element offset of (row srow + 4i, this lane's four channels of a slice's first column), or none
          if (total_sl > 0) tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)cfirst, v);
          if (PIPED) {
            // The tile's scales go to shared memory once: a global load issued between the slices' stores waits
            // behind them in the load/store unit's queue, one per slice was a stall of hundreds of cycles each.
            __syncwarp();   // the previous tile's last slice has read its scales
            for (int c = lane * 4; c < Nt; c += 128) {
              float4 al = make_float4(0.f, 0.f, 0.f, 0.f);
              if (n0 + c < K) al = __ldg(reinterpret_cast<const float4*>(alpha + n0 + c));
              asm volatile("st.shared.v4.f32 [%0], {%1,%2,%3,%4};" ::"r"(a_stage + (uint32_t)c * 4u), "f"(al.x), "f"(al.y),
                           "f"(al.z), "f"(al.w)
                           : "memory");
            }
            __syncwarp();
          }
          int mt = 0, ci = 0;
#pragma unroll 1
          for (int sl = 0; sl < total_sl; ++sl) {
            const int c0 = cfirst + cstep * ci;
            if (ci == 0) {
              const int mine = row_pixel(mt);
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                const int r = __shfl_sync(0xffffffffu, mine, srow + 4 * i);
                roff[i] = r >= 0 ? (uint32_t)r * (uint32_t)K + (uint32_t)(n0 + scol * 4) : 0xffffffffu;
              }
            }
            const int co = n0 + c0 + scol * 4;
            unsigned long long alA = 0, alB = 0;   // (alpha[co], alpha[co+1]) and (alpha[co+2], alpha[co+3])
            if (PIPED) {
              asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];" : "=l"(alA), "=l"(alB) : "r"(a_stage + (uint32_t)(c0 + scol * 4) * 4u) : "memory");
            } else if (!out_i32 && co < K) {
              const float4 al = __ldg(reinterpret_cast<const float4*>(alpha + co));
              asm("mov.b64 %0, {%1, %2};" : "=l"(alA) : "f"(al.x), "f"(al.y));
              asm("mov.b64 %0, {%1, %2};" : "=l"(alB) : "f"(al.z), "f"(al.w));
            }
            tmem_ld_wait();
#pragma unroll
            for (int e = 0; e < 8; ++e)
              asm volatile("st.shared.v4.b32 [%0], {%1,%2,%3,%4};" ::"r"(st_lane ^ (uint32_t)(e << 4)), "r"(v[4 * e]),
                           "r"(v[4 * e + 1]), "r"(v[4 * e + 2]), "r"(v[4 * e + 3])
                           : "memory");
            __syncwarp();
            if (++ci == per_mt) { ci = 0; ++mt; }
            if (sl + 1 < total_sl)
              tmem_ld32(d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * Nt + cfirst + cstep * ci), v);
            if (co < K) {  // K is a multiple of 4 here, so the four channels exist together
              const uint32_t* obase = out32 + c0;
#pragma unroll
              for (int hh = 0; hh < 2; ++hh) {   // four rows at a time: 16 registers of values in flight
                unsigned long long ua[4], ub[4];
#pragma unroll
                for (int j = 0; j < 4; ++j) {    // row srow + 4i, i = 4hh + j: even i from ld_even, odd i from ld_odd
                  const int i = 4 * hh + j;
                  asm volatile("ld.shared.v2.b64 {%0,%1}, [%2];"
                               : "=l"(ua[j]), "=l"(ub[j])
                               : "r"(((i & 1) ? ld_odd : ld_even) + (uint32_t)((i >> 1) * 1024))
                               : "memory");
                }
                if (!out_i32) {
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(ua[j]) : "l"(alA));
                    asm("mul.rn.f32x2 %0, %0, %1;" : "+l"(ub[j]) : "l"(alB));
                  }
                } else {
                  // int32 sums asked of fp32 accumulators: the sums are integers, the conversion is exact
#pragma unroll
                  for (int j = 0; j < 4; ++j) {
                    uint32_t x, y, z, w;
                    asm("mov.b64 {%0, %1}, %2;" : "=r"(x), "=r"(y) : "l"(ua[j]));
                    asm("mov.b64 {%0, %1}, %2;" : "=r"(z), "=r"(w) : "l"(ub[j]));
                    x = (uint32_t)__float2int_rn(__uint_as_float(x)); y = (uint32_t)__float2int_rn(__uint_as_float(y));
                    z = (uint32_t)__float2int_rn(__uint_as_float(z)); w = (uint32_t)__float2int_rn(__uint_as_float(w));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(ua[j]) : "r"(x), "r"(y));
                    asm("mov.b64 %0, {%1, %2};" : "=l"(ub[j]) : "r"(z), "r"(w));
                  }
                }
#pragma unroll
                for (int j = 0; j < 4; ++j)
                  if (roff[4 * hh + j] != 0xffffffffu)
                    asm volatile("st.global.v2.b64 [%0], {%1,%2};" ::"l"(obase + roff[4 * hh + j]), "l"(ua[j]), "l"(ub[j])
                                 : "memory");
              }
            }
            __syncwarp();
          }
        } else {
          // c_out not a multiple of 4 or a channel tile not a multiple of 32: 16-column slices
          // straight from registers, element by element
#pragma unroll 1
          for (int mt = 0; mt < MT; ++mt) {
            const int pix = row_pixel(mt);
            const uint32_t trow = d0 + ((uint32_t)(rq * 32) << 16) + (uint32_t)(mt * Nt);
            for (int c0 = G_EPI_SPLIT ? 0 : 16 * half; c0 < Nt; c0 += G_EPI_SPLIT ? 16 : 32) {
              uint32_t v[16];
              tmem_ld16(trow + (uint32_t)c0, v);
              tmem_ld_wait();
              const int co0 = n0 + c0;
              if (pix < 0 || co0 >= K) continue;
              uint32_t* o = out32 + wide_mul((uint32_t)pix, (uint32_t)K) + co0;
              if ((K & 3) == 0 && co0 + 16 <= K) {
                // all 16 channels exist and rows are 16-byte aligned: four channels per load, multiply and store
#pragma unroll
                for (int e = 0; e < 16; e += 4) {
                  uint4 r;
                  if (out_i32) {
                    r.x = (uint32_t)__float2int_rn(__uint_as_float(v[e]));
                    r.y = (uint32_t)__float2int_rn(__uint_as_float(v[e + 1]));
                    r.z = (uint32_t)__float2int_rn(__uint_as_float(v[e + 2]));
                    r.w = (uint32_t)__float2int_rn(__uint_as_float(v[e + 3]));
                  } else {
                    const float4 al = __ldg(reinterpret_cast<const float4*>(alpha + co0 + e));
                    r.x = __float_as_uint(__fmul_rn(__uint_as_float(v[e]), al.x));
                    r.y = __float_as_uint(__fmul_rn(__uint_as_float(v[e + 1]), al.y));
                    r.z = __float_as_uint(__fmul_rn(__uint_as_float(v[e + 2]), al.z));
                    r.w = __float_as_uint(__fmul_rn(__uint_as_float(v[e + 3]), al.w));
                  }
                  *reinterpret_cast<uint4*>(o + e) = r;
                }
                continue;
              }
#pragma unroll
              for (int e = 0; e < 16; ++e) {
                if (co0 + e < K) {
                  if (out_i32) o[e] = (uint32_t)__float2int_rn(__uint_as_float(v[e]));
                  else o[e] = __float_as_uint(__fmul_rn(__uint_as_float(v[e]), __ldg(alpha + co0 + e)));
                }
              }
            }
          }
        }
        // this warp has read its part of the accumulator buffer: hand it back to the MMA issuer
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_accempty + 8 * acc_slot);
        if (CHAIN && L.done) {
          // chain: this warp's part of the tile is written; the successor may read it
          __threadfence();
          __syncwarp();
          if (lane == 0) atomicAdd(L.done + mg, 1u);
        }
      }
    }
    if (warp == 2 && lane == 0) TR_REPORT(2, clock64() - tr_t0, tr_w0, tr_w1, tr_w2);
  } else if (warp != 13 && warp != 17) {
    // ------------------------------------------------ expanders (warps 10-12, 14-16, 18, 19)
    // Fill activation unit (problem, tile, channel block) of the ring: for every plane, row and
    // 32-channel word, bits -> two 16-byte chunks of +1/-1 bytes (fp16: copy two 8-channel chunks).
    grid_dep_wait();  // the activations may come from the previous kernel in the stream
    const int et = (warp - 10 - (warp > 13) - (warp > 17)) * 32 + lane;  // rank among the expander threads
    int a_slot = 0;
    long long a_done = 0;
    uint32_t a_phase = 1;  // parity of the previous use of a slot (valid from the second lap)
    volatile int* exp_flag = abort_flag + 1;
    volatile int* dep_flag = abort_flag + 2;
    bool stop = false;
    long long tr_w0 = 0, tr_t0 = clock64();
    (void)tr_w0; (void)tr_t0; (void)exp_flag; (void)dep_flag;
    if (!CHAIN && FP4) {
      // Independent problems: all inputs exist when the launch starts and are small beside the L2 (1/29 of the
      // outputs; fp16 inputs are not: half of the outputs).  The CTAs pull them into L2 together, once, so that the staging loads below see L2 latency
      // instead of DRAM latency: a unit is one round trip, and the round trip is what the expanders' rate is.
      for (int l = 0; l < p.n_layers; ++l) {
        const GLayer& L = lay[l];
        const size_t bytes = (size_t)L.N * L.H * L.W * (F16 ? (size_t)L.C * 2 : (size_t)L.Cw * 4);
        const char* base = reinterpret_cast<const char*>(p.act[l]);
        for (size_t off = ((size_t)blockIdx.x * G_EXP_THREADS + et) * 128; off < bytes; off += (size_t)G * G_EXP_THREADS * 128)
          asm volatile("prefetch.global.L2 [%0];" ::"l"(base + off));
      }
    }
    // Independent problems on 4-bit operands whose rows can be read two words at a time run a two-stage software
    // pipeline per thread: a "group" is up to three rows of one unit with one vector load each; the loads of
    // group g + 1 are issued (into registers) before group g is expanded into shared memory, so that a unit no
    // longer costs a full round trip to memory - with few words per row the round trip is nearly all of it.
    constexpr bool piped = PIPED;   // (the host has checked the alignment of all inputs)
    if constexpr (PIPED) {
      struct XGroup {
        uint4 t[G_EXP_ROWS];        // the rows' words (two or four of them)
        uint32_t da[G_EXP_ROWS];    // where a row's first chunk goes
        uint32_t cstride;           // bytes from one chunk of a plane to the next
        uint32_t flags;             // bit j: row j exists; bit 4 + j: its pixel is inside the image; 8: four words per
                                    // row; 9: first group of its unit; 10: last group of its unit
      };
      // The expander warps form XG teams that take the units in turn (the ring has a multiple of XG slots, so a
      // slot always belongs to the same team): with few rows per unit a unit is a chain of latencies, and two
      // chains in flight are what doubles the rate.
      constexpr int XG = G_XTEAMS, XT = G_EXP_THREADS / XG;
      const int gx = et / XT, etg = et % XT;
      int* const pix = pix_tab + gx * (int)p.pix_words;
      // issue side: the unit (il, itile, icb) with sequence number iu, and the next group to load in it
      int il = 0, itile = 0, itotal = 0, icb = 0, irb = 0, ik0 = 0, i_slot = 0, iu = 0;
      int Rr = 0, n_planes = 0, n_cb = 0, cbc = 0, Cw = 0, all_rows = 0, kstep = 2;
      int pix_l = -1, pix_t = -1;   // the tile the pixel table holds
      const uint32_t* act = nullptr;
      bool ivalid = false;
      auto enter_layer = [&]() {   // first layer from il on in which this CTA has a tile
        for (; il < p.n_layers; ++il) {
          const GLayer& L = lay[il];
          itile = g_first_tile(L);
          itotal = L.total_tiles;
          if (itile >= itotal) continue;
          Rr = L.Rr; n_planes = L.n_planes; n_cb = L.n_cb; cbc = L.cb_chunks; Cw = L.Cw;
          all_rows = n_planes * Rr;
          act = reinterpret_cast<const uint32_t*>(p.act[il]);
          kstep = ((reinterpret_cast<uintptr_t>(act) & 15) == 0 && (Cw & 3) == 0 && (cbc & 3) == 0) ? 4 : 2;
          icb = 0;
          ivalid = true;
          return;
        }
        ivalid = false;
      };
      auto next_unit = [&]() {     // the unit after (il, itile, icb) in the CTA's sequence
        ++iu;
        i_slot = i_slot + 1 == NA ? 0 : i_slot + 1;
        if (++icb >= n_cb) {
          icb = 0;
          itile += G;
          if (itile >= itotal) {
            ++il;
            enter_layer();
          }
        }
      };
      auto seek_own = [&]() {      // on to this team's next unit; input pixel of each of this thread's rows of its tile
        while (ivalid && (iu % XG) != gx) next_unit();
        if (ivalid && (pix_l != il || pix_t != itile)) {
          const GLayer& L = lay[il];
          const int mg = (int)fdiv((uint32_t)itile, L.dNt);
          const uint32_t Q0 = (uint32_t)mg * (uint32_t)(128 * L.MT);
          for (int f = etg; f < all_rows; f += XT) {
            const int pl = (f >= Rr) + (f >= 2 * Rr) + (f >= 3 * Rr);
            pix[f] = g_position_to_pixel(L, Q0 + (uint32_t)(f - pl * Rr), pl >> 1, pl & 1);
          }
          pix_l = il;
          pix_t = itile;
        }
      };
      auto issue = [&](XGroup& g) {   // loads of the group at the issue position; moves the position on
        const uint32_t cs = (uint32_t)Rr * 16u;
        uint32_t flags = (kstep == 4 ? 0x100u : 0u) | ((irb == 0 && ik0 == 0) ? 0x200u : 0u);
        const uint32_t unit = smem_u32(a_smem) + (uint32_t)i_slot * p.a_slot_bytes;
#pragma unroll
        for (int j = 0; j < G_EXP_ROWS; ++j) {
          const int f = irb + etg + j * XT;
          const int px = f < all_rows ? pix[f] : -2;
          const int pl = (f >= Rr) + (f >= 2 * Rr) + (f >= 3 * Rr);
          g.da[j] = unit + (uint32_t)(pl * cbc * Rr + (f - pl * Rr)) * 16u + (uint32_t)ik0 * cs;
          if (px != -2) flags |= 1u << j;
          g.t[j] = make_uint4(0, 0, 0, 0);
          if (px >= 0) {
            flags |= 0x10u << j;
            const uint32_t* src = act + wide_mul((uint32_t)px, (uint32_t)Cw) + icb * cbc + ik0;
            if (kstep == 4) {
              g.t[j] = __ldg(reinterpret_cast<const uint4*>(src));
            } else {
              const uint2 v = __ldg(reinterpret_cast<const uint2*>(src));
              g.t[j].x = v.x;
              g.t[j].y = v.y;
            }
          }
        }
        g.cstride = cs;
        ik0 += kstep;
        if (ik0 >= cbc) {
          ik0 = 0;
          irb += G_EXP_ROWS * XT;
          if (irb >= all_rows) {   // the unit ends with this group
            irb = 0;
            flags |= 0x400u;
            next_unit();
            seek_own();
          }
        }
        g.flags = flags;
      };
      enter_layer();
      seek_own();
      // completion side: this team's slots gx, gx + XG, ... of the ring
      a_slot = gx;
      XGroup cur, nxt;
      bool nvalid = ivalid;
      if (nvalid) issue(nxt);
      while (nvalid && !stop) {
        cur = nxt;
        nvalid = ivalid;
        if (nvalid) issue(nxt);
        if ((cur.flags & 0x200u) && a_done >= NA / XG) {
          int okf = 1;
          if (lane == 0) okf = (!*abort_flag && TR_WAIT(tr_w0, mbar_wait_backoff(bar_aempty + 8 * a_slot, a_phase, 64))) ? 1 : 0;
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
#pragma unroll
        for (int j = 0; j < G_EXP_ROWS; ++j) {
          if (cur.flags & (1u << j)) {
            const bool on = (cur.flags & (0x10u << j)) != 0;
            const uint32_t d = cur.da[j], cs = cur.cstride;
            sts16(d, expand_word_fp4(cur.t[j].x, on));
            sts16(d + cs, expand_word_fp4(cur.t[j].y, on));
            if (cur.flags & 0x100u) {
              sts16(d + 2 * cs, expand_word_fp4(cur.t[j].z, on));
              sts16(d + 3 * cs, expand_word_fp4(cur.t[j].w, on));
            }
          }
        }
        if (cur.flags & 0x400u) {
          fence_proxy_async();  // generic-proxy writes -> visible to the tensor core's reads
          __syncwarp();
          if (lane == 0) mbar_arrive(bar_afull + 8 * a_slot);
          ++a_done;
          a_slot += XG;
          if (a_slot >= NA) { a_slot -= NA; a_phase ^= 1u; }
        }
      }
    }
    for (int l = 0; l < (piped ? 0 : p.n_layers) && !stop; ++l) {
      const GLayer& L = lay[l];
      const int Rr = L.Rr, n_planes = L.n_planes, n_cb = L.n_cb, cb_chunks = L.cb_chunks, MT = L.MT;
      const int C = L.C, Cw = L.Cw, total = L.total_tiles;
      const FastDiv dNt = L.dNt;
      const void* act = p.act[l];
      const bool fresh = CHAIN && L.deps != nullptr;   // written by other CTAs of this launch: read from L2
      // vector loads of a row's words need the base pointer and the row pitch aligned to the load
      bool vec;
      {
        const uintptr_t addr = (uintptr_t)act;
        if (F16) vec = (addr & 15) == 0 && (C & 7) == 0;
        else if (FP4) vec = (addr & 7) == 0 && (Cw & 1) == 0;  // pairs of words (a block's first word is even)
        else vec = false;
      }
      const bool vec4 = FP4 && vec && ((uintptr_t)act & 15) == 0 && (Cw & 3) == 0 && (cb_chunks & 3) == 0;
      for (int tile = g_first_tile(L); tile < total && !stop; tile += G) {
        const int mg = (int)fdiv((uint32_t)tile, dNt);
        const uint32_t Q0 = (uint32_t)mg * (uint32_t)(128 * MT);
        if (CHAIN && L.deps) {
          // chain: wait until the predecessor has written every input pixel of this tile (one thread polls)
          if (et == 0) {
            const uint2 d = __ldg(L.deps + mg);
            int okd = 1;
            for (uint32_t m = d.x; m <= d.y && okd; ++m) okd = g_wait_counter(L.prev_done + m, L.prev_target, abort_flag) ? 1 : 0;
            *dep_flag = okd;
          }
          asm volatile("bar.sync 3, %0;" ::"n"(G_EXP_THREADS) : "memory");
          const int okd = *dep_flag;
          if (!okd) {
            if (et == 0 && !*abort_flag) {
              *abort_flag = 1;
              raise_status(p.status, 5);
            }
            stop = true;
            break;
          }
        }
        // Input pixel of every staged row, once per tile.  The table is private to the expanders:
        // the barrier keeps a fast thread from overwriting entries another still reads (and, in a chain,
        // the polling thread from setting the next tile's flag before everyone has read this one).
        asm volatile("bar.sync 3, %0;" ::"n"(G_EXP_THREADS) : "memory");
        // (plane, row) pairs form one index space f = plane*Rr + row, dealt to the threads at a stride of
        // the expander count, here and below: a thread reads back only entries it wrote itself
        const int all_rows = n_planes * Rr;
        for (int f = et; f < all_rows; f += G_EXP_THREADS) {
          const int pl = (f >= Rr) + (f >= 2 * Rr) + (f >= 3 * Rr);
          pix_tab[f] = g_position_to_pixel(L, Q0 + (uint32_t)(f - pl * Rr), pl >> 1, pl & 1);
        }
        for (int cb = 0; cb < n_cb; ++cb) {
          if (a_done >= NA) {
            // one elected thread polls; the rest wait on a hardware barrier instead of spinning
            if (et == 0) *exp_flag = (!*abort_flag && TR_WAIT(tr_w0, mbar_wait_backoff(bar_aempty + 8 * a_slot, a_phase, 64))) ? 1 : 0;
            asm volatile("bar.sync 3, %0;" ::"n"(G_EXP_THREADS) : "memory");
            const int okf = *exp_flag;
            asm volatile("bar.sync 3, %0;" ::"n"(G_EXP_THREADS) : "memory");
            if (!okf) {
              if (et == 0 && !*abort_flag) {
                *abort_flag = 1;
                raise_status(p.status, 1);
              }
              stop = true;
              break;
            }
          }
          uint8_t* unit = a_smem + (size_t)a_slot * p.a_slot_bytes;
          // A thread has rows of several planes in flight together: a stride-2 unit (four short
          // planes) costs one round trip to memory instead of four.
          {
            for (int rb = 0; rb < all_rows; rb += G_EXP_ROWS * G_EXP_THREADS) {
              int pix[G_EXP_ROWS];  // input pixel of each of this thread's rows; -1 padding, -2 past the unit
              uint8_t* dst[G_EXP_ROWS];  // where the row starts in its plane (chunk 0)
#pragma unroll
              for (int j = 0; j < G_EXP_ROWS; ++j) {
                const int f = rb + et + j * G_EXP_THREADS;
                pix[j] = f < all_rows ? pix_tab[f] : -2;
                const int pl = (f >= Rr) + (f >= 2 * Rr) + (f >= 3 * Rr);
                dst[j] = unit + ((size_t)pl * cb_chunks * Rr + (size_t)(f - pl * Rr)) * 16;
              }
              if (F16 && vec) {
                // fp16 activations are copied: asynchronous 16-byte copies straight into the unit (zero-filled where
                // the row is padding or the channels end), all of a thread's chunks in flight together; the thread
                // waits for its own copies before it makes them visible to the tensor core and arrives.
#pragma unroll
                for (int j = 0; j < G_EXP_ROWS; ++j) {
                  if (pix[j] == -2) continue;
                  const __half* row = (const __half*)act + wide_mul((uint32_t)(pix[j] < 0 ? 0 : pix[j]), (uint32_t)C);
                  const uint32_t d = smem_u32(dst[j]);
                  for (int c0 = 0; c0 < cb_chunks; ++c0) {
                    const int ch = (cb * cb_chunks + c0) * 8;  // first channel of the chunk
                    const bool on = pix[j] >= 0 && ch < C;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d + (uint32_t)c0 * (uint32_t)Rr * 16u),
                                 "l"(on ? (const void*)(row + ch) : act), "r"(on ? 16 : 0)
                                 : "memory");
                  }
                }
              } else if (F16) {
                for (int c0 = 0; c0 < cb_chunks; c0 += 2) {
                  uint4 v[G_EXP_ROWS][2];
#pragma unroll
                  for (int j = 0; j < G_EXP_ROWS; ++j) {
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                      v[j][k] = make_uint4(0, 0, 0, 0);
                      const int ch = (cb * cb_chunks + c0 + k) * 8;  // first channel of the chunk
                      if (pix[j] >= 0 && ch < C) {
                        const __half* src = (const __half*)act + wide_mul((uint32_t)pix[j], (uint32_t)C) + ch;
                        if (vec) {
                          v[j][k] = __ldg(reinterpret_cast<const uint4*>(src));
                        } else {
                          uint32_t w[4] = {0, 0, 0, 0};
#pragma unroll
                          for (int e = 0; e < 8; ++e)
                            if (ch + e < C) w[e >> 1] |= (uint32_t)__half_as_ushort(src[e]) << (16 * (e & 1));
                          v[j][k] = make_uint4(w[0], w[1], w[2], w[3]);
                        }
                      }
                    }
                  }
#pragma unroll
                  for (int j = 0; j < G_EXP_ROWS; ++j) {
                    if (pix[j] != -2) {
                      *reinterpret_cast<uint4*>(dst[j] + (size_t)c0 * Rr * 16) = v[j][0];
                      *reinterpret_cast<uint4*>(dst[j] + (size_t)(c0 + 1) * Rr * 16) = v[j][1];
                    }
                  }
                }
              } else if (FP4) {
                // A 32-channel word becomes one 16-byte chunk of nibbles.  The common case (an even number of
                // words per pixel, so that a block's words are read two or four at a time) is kept free of
                // per-word conditions: this role, too, is bound by the instructions it issues.
                const int wb = cb * cb_chunks;
                const uint32_t cstride = (uint32_t)Rr * 16u;   // bytes from one chunk of a plane to the next
                uint32_t da[G_EXP_ROWS];
#pragma unroll
                for (int j = 0; j < G_EXP_ROWS; ++j) da[j] = smem_u32(dst[j]);
                if (vec) {
                  const uint32_t* src[G_EXP_ROWS];
#pragma unroll
                  for (int j = 0; j < G_EXP_ROWS; ++j)
                    src[j] = (const uint32_t*)act + wide_mul((uint32_t)(pix[j] < 0 ? 0 : pix[j]), (uint32_t)Cw) + wb;
                  if (vec4) {
                    for (int k0 = 0; k0 < cb_chunks; k0 += 4) {
                      uint4 t[G_EXP_ROWS];
#pragma unroll
                      for (int j = 0; j < G_EXP_ROWS; ++j) {
                        t[j] = make_uint4(0, 0, 0, 0);
                        if (pix[j] >= 0) t[j] = g_ld4(src[j] + k0, fresh);
                      }
#pragma unroll
                      for (int j = 0; j < G_EXP_ROWS; ++j) {
                        if (pix[j] != -2) {
                          const bool on = pix[j] >= 0;
                          const uint32_t d = da[j] + (uint32_t)k0 * cstride;
                          sts16(d, expand_word_fp4(t[j].x, on));
                          sts16(d + cstride, expand_word_fp4(t[j].y, on));
                          sts16(d + 2 * cstride, expand_word_fp4(t[j].z, on));
                          sts16(d + 3 * cstride, expand_word_fp4(t[j].w, on));
                        }
                      }
                    }
                  } else {
                    for (int k0 = 0; k0 < cb_chunks; k0 += 2) {
                      uint2 t[G_EXP_ROWS];
#pragma unroll
                      for (int j = 0; j < G_EXP_ROWS; ++j) {
                        t[j] = make_uint2(0, 0);
                        if (pix[j] >= 0) t[j] = g_ld2(src[j] + k0, fresh);
                      }
#pragma unroll
                      for (int j = 0; j < G_EXP_ROWS; ++j) {
                        if (pix[j] != -2) {
                          const bool on = pix[j] >= 0;
                          const uint32_t d = da[j] + (uint32_t)k0 * cstride;
                          sts16(d, expand_word_fp4(t[j].x, on));
                          sts16(d + cstride, expand_word_fp4(t[j].y, on));
                        }
                      }
                    }
                  }
                } else {
                  // an odd number of words per pixel, or a pointer that is not 8-byte aligned: word by word
                  for (int k = 0; k < cb_chunks; ++k) {
#pragma unroll
                    for (int j = 0; j < G_EXP_ROWS; ++j) {
                      if (pix[j] == -2) continue;
                      const bool on = pix[j] >= 0 && wb + k < Cw;
                      uint32_t w = 0;
                      if (on) w = g_ld1((const uint32_t*)act + wide_mul((uint32_t)pix[j], (uint32_t)Cw) + wb + k, fresh);
                      sts16(da[j] + (uint32_t)k * cstride, expand_word_fp4(w, on));
                    }
                  }
                }
              }
            }
          }
          if (F16) asm volatile("cp.async.wait_all;" ::: "memory");
          fence_proxy_async();  // generic-proxy writes -> visible to the tensor core's reads
          mbar_arrive(bar_afull + 8 * a_slot);
          ++a_done;
          if (++a_slot == NA) { a_slot = 0; a_phase ^= 1u; }
        }
      }
    }
    if (et == 0) TR_REPORT(3, clock64() - tr_t0, tr_w0, 0, 0);
  }

  // ---------------------------------------------------------------- teardown
  tc_fence_before();
  __syncthreads();
  if (warp == 2) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512) : "memory");
  }
}

// ------------------------------------------------------------------ host side
struct GroupDev {
  int count = 0, act_type = 0, mode = M_FP4;
  int kind = TCG_WORDS;           // what the tiles were planned for (word outputs, packed signs, chain)
  bool hot = false;               // planned for the hot variant of the word-output kernel (see tcg_create)
  int chain = 0;                  // 1: member i + 1 reads the packed signs member i writes (one launch, dependency counters)
  uint8_t* chain_buf = nullptr;   // the packed signs between the members, one buffer per boundary
  size_t chain_off[SNN_GROUP_MAX] = {};
  uint32_t* done = nullptr;       // completion counters of all members' M groups
  size_t done_words = 0;
  uint2* deps = nullptr;
  GLayer* layers_dev = nullptr;   // [count]
  uint8_t* weights = nullptr;     // the group's own weight operands, one after the other
  uint16_t* ranks = nullptr;      // [count][grid] tile assignment, see tcg_create
  GParams p{};                    // everything but the per-call pointers
  size_t smem = 0;
  int grid = 0;
};

namespace {

// Tile shape, channel blocks and weight stages of one problem under the group's fixed slot sizes.
// Operand of the weights: wt[layout tile][channel block][tap][chunk][NtL][16 B]; a chunk is 16 bytes along the
// input channels (16 int8, 8 fp16 or 32 e2m1 values), cb_chunks chunks per block, NtL output channels per
// layout tile.  Channels that do not exist are zeros, so whatever the activation operand holds there adds 0.
template <int MODE>
__global__ void g_expand_weights_kernel(const uint32_t* __restrict__ wplanes, uint8_t* __restrict__ wt, int C, int K,
                                        int Cw, long long total, int cb_chunks, int n_cb, int NtL, int taps) {
  long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x;
  if (i >= total) return;
  int row = (int)(i % NtL);
  long long r = i / NtL;
  int c = (int)(r % cb_chunks);
  r /= cb_chunks;
  int t = (int)(r % taps);
  r /= taps;
  int cb = (int)(r % n_cb), tile = (int)(r / n_cb);
  int co = tile * NtL + row;
  constexpr int cpc = MODE == M_F16 ? 8 : 32;
  uint4 v = make_uint4(0, 0, 0, 0);
  if (co < K) {
    int ch0 = (cb * cb_chunks + c) * cpc;
    int wd = ch0 >> 5, sh = ch0 & 31;
    uint32_t bits = wd < Cw ? wplanes[((size_t)t * Cw + wd) * K + co] >> sh : 0u;
    uint32_t w[4] = {0, 0, 0, 0};
    if (MODE == M_F16) {
#pragma unroll
      for (int e = 0; e < 8; ++e)
        if (ch0 + e < C) w[e >> 1] |= (((bits >> e) & 1u) ? 0x3c00u : 0xbc00u) << (16 * (e & 1));  // +1.0 / -1.0
    } else {
#pragma unroll
      for (int e = 0; e < 32; ++e)
        if (ch0 + e < C) w[e >> 3] |= (((bits >> e) & 1u) ? 0x2u : 0xau) << (4 * (e & 7));         // e2m1 +1.0 / -1.0
    }
    v = make_uint4(w[0], w[1], w[2], w[3]);
  }
  reinterpret_cast<uint4*>(wt)[i] = v;
}

cudaError_t g_expand_weights(int mode, const uint32_t* wplanes, void* dst, int C, int K, int Cw, int Kpad, int n_chunks,
                             int cb_chunks, int NtL, int taps, cudaStream_t s) {
  const long long total = (long long)taps * n_chunks * Kpad;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  const int n_cb = n_chunks / cb_chunks;
  if (mode == M_F16)
    g_expand_weights_kernel<M_F16><<<blocks, 256, 0, s>>>(wplanes, (uint8_t*)dst, C, K, Cw, total, cb_chunks, n_cb, NtL, taps);
  else
    g_expand_weights_kernel<M_FP4><<<blocks, 256, 0, s>>>(wplanes, (uint8_t*)dst, C, K, Cw, total, cb_chunks, n_cb, NtL, taps);
  return cudaGetLastError();
}

inline int g_mode_for(int act_type) { return act_type == SNN_ACT_F16 ? M_F16 : M_FP4; }

// Cycles of one MMA of 128 positions x nt channels as measured on B200 (any operand type): half a cycle per
// channel plus a constant that does not overlap the previous MMA.
inline double g_mma_cycles(int nt) { return 0.5 * nt + 33.0; }

// tensor-memory columns of one accumulator buffer when there are n_acc of them
inline int g_acc_cols(int mode, int n_acc) {
  return mode != M_FP4 ? (int)G_ACC_COLS : n_acc == G_NACC_WORDS ? (int)G_ACC_COLS_FP4_3 : (int)G_ACC_COLS_FP4;
}

bool g_plan_layer(const Geom& g, int mode, int n_acc, GLayer* L, int* n_chunks_out, int* Kpad_out) {
  const int cpc = mode == M_F16 ? 8 : 32;
  const int acc_cols = g_acc_cols(mode, n_acc);
  const int raw = round_up(g.C, 2 * cpc) / cpc;  // 16-byte chunks along the channels, even
  GLayer& o = *L;
  o.N = g.N; o.H = g.H; o.W = g.W; o.C = g.C; o.K = g.K; o.Cw = g.Cw;
  o.stride = g.stride; o.pad = g.pad; o.Ho = g.Ho; o.Wo = g.Wo;
  o.taps = g.ksize == 1 ? 1 : 9;
  if (g.ksize == 1) {
    // 1x1 layer: the positions are the output pixels themselves (input pixel = stride * output pixel), no halo
    o.Hq = g.Ho; o.Wq = g.Wo; o.n_planes = 1; o.halo = 0;
  } else if (g.stride == 1) {
    o.Hq = g.H + g.pad; o.Wq = g.W + g.pad; o.n_planes = 1; o.halo = 2 * o.Wq + 2;
  } else {
    o.Hq = g.Ho + 1; o.Wq = g.Wo + 1; o.n_planes = 4; o.halo = o.Wq + 1;
  }
  o.dWq = make_fastdiv((uint32_t)o.Wq);
  o.dHq = make_fastdiv((uint32_t)o.Hq);
  o.Qtot = (long long)g.N * o.Hq * o.Wq;
  if (g.N < 1) return false;
  if (o.Qtot + 1024 + o.halo >= (1ll << 31)) return false;  // positions are 32-bit in the kernel
  if (g.C > (1 << 20)) return false;                        // 9 * c_in stays far below 2^24: exact fp32 sums
  if ((long long)g.N * g.H * g.W >= (1ll << 31) || (long long)g.N * g.Ho * g.Wo >= (1ll << 31)) return false;
  if ((long long)g.N * g.Ho * g.Wo * g.K >= 0xffffffffLL) return false;   // output element offsets are 32-bit
  // layout tile of the weight operand = channels per tile: all of them up to 256; beyond that 256
  // when that pads little (fewer channel tiles re-expand the same activations), else 128
  if (mode == M_FP4) o.NtL = g.K <= acc_cols ? round_up(g.K, 16) : 128;   // (columns 480..511 hold the scales)
  else o.NtL = g.K <= 256 ? round_up(g.K, 16) : (round_up(g.K, 256) - g.K < 64 ? 256 : 128);
  o.Nt = o.NtL;
  const int Kpad = round_up(g.K, o.NtL);
  o.n_ntiles = Kpad / o.Nt;
  o.dNt = make_fastdiv((uint32_t)o.n_ntiles);
  // channel block: the largest of 8/6/4/2 chunks that divides the channels and whose unit fits a slot
  int d = 0;
  for (int c = 8; c >= 2; c -= 2) {
    if (raw % c) continue;
    if ((size_t)o.n_planes * c * (128 + o.halo) * 16 <= kGASlotMax) { d = c; break; }
  }
  if (!d) return false;
  o.cb_chunks = d;
  o.n_cb = raw / d;
  o.kpt = d / 2;
  int MT = 1;
  for (int m = 4; m >= 2; --m)
    if ((size_t)o.n_planes * d * (128 * m + o.halo) * 16 <= kGASlotMax && m * o.Nt <= acc_cols) { MT = m; break; }
  const long long mtiles = (o.Qtot + 127) / 128;
  while (MT > 1 && mtiles < MT) --MT;  // a tiny problem does not need the larger tile
  o.MT = MT;
  o.Rr = 128 * MT + o.halo;
  if ((uint32_t)o.Rr * 16 >= (1u << 18)) return false;  // leading-offset field of the descriptor
  const long long mgroups = (mtiles + MT - 1) / MT;
  if (mgroups * o.n_ntiles > 0x7fffffffLL || mgroups * o.Rr >= (1ll << 31)) return false;
  o.total_tiles = (int)(mgroups * o.n_ntiles);
  // weight stage: as many whole taps of a channel block as fit a slot
  o.tap_bytes = (uint32_t)(o.kpt * 2 * o.Nt * 16);
  int st = (int)(kGBSlot / o.tap_bytes);
  if (st < 1) return false;
  o.st_taps = st > o.taps ? o.taps : st;
  *n_chunks_out = raw;
  *Kpad_out = Kpad;
  return true;
}

}  // namespace

namespace {
// host copy of the kernel's position -> input pixel map
int h_position_to_pixel(const GLayer& L, long long q, int pa, int pb) {
  if (q >= L.Qtot) return -1;
  const long long rg = q / L.Wq;
  const int j = (int)(q - rg * L.Wq);
  const long long n = rg / L.Hq;
  const int i = (int)(rg - n * L.Hq);
  if (n >= L.N) return -1;
  const int r = L.stride * i + pa - L.pad, c = L.stride * j + pb - L.pad;
  if (r < 0 || r >= L.H || c < 0 || c >= L.W) return -1;
  return (int)((n * L.H + r) * L.W + c);
}
}  // namespace

cudaError_t tcg_create(const LayerDev* const* Ls, const Geom* gs, int count, int act_type, int kind, cudaStream_t s,
                       GroupDev** out, int* launched) {
  *out = nullptr;
  if (count < 1 || count > SNN_GROUP_MAX) return cudaErrorInvalidConfiguration;
  if (kind != TCG_WORDS && act_type != SNN_ACT_BIN) return cudaErrorInvalidConfiguration;
  const int chain = kind == TCG_CHAIN;
  const int mode = g_mode_for(act_type);
  GLayer host[SNN_GROUP_MAX];
  int n_chunks[SNN_GROUP_MAX], Kpad[SNN_GROUP_MAX];
  size_t w_off[SNN_GROUP_MAX], w_total = 0;
  size_t a_slot = 0, pix_bytes = 0;
  long long tiles = 0;
  // Word outputs on 4-bit operands get three accumulator buffers where the launch can run its hot variant (every
  // member: c_out a multiple of 4, channel tile a multiple of 32, an even number of activation words per pixel);
  // with the plain expanders two larger buffers measure faster, so everything else is planned with two.
  int n_acc = (mode == M_FP4 && kind == TCG_WORDS) ? G_NACC_WORDS : G_NACC;
  bool hot = n_acc == G_NACC_WORDS;
  if (hot) {
    for (int i = 0; i < count && hot; ++i) {
      if (!g_plan_layer(gs[i], mode, n_acc, &host[i], &n_chunks[i], &Kpad[i])) return cudaErrorInvalidConfiguration;
      if ((gs[i].Cw & 1) || (gs[i].K & 3) || (host[i].Nt & 31)) hot = false;
    }
    if (!hot) n_acc = G_NACC;
  }
  for (int i = 0; i < count; ++i) {
    if (!g_plan_layer(gs[i], mode, n_acc, &host[i], &n_chunks[i], &Kpad[i])) return cudaErrorInvalidConfiguration;
    const size_t unit = (size_t)host[i].n_planes * host[i].cb_chunks * host[i].Rr * 16;
    if (unit > a_slot) a_slot = unit;
    const size_t pb = (size_t)host[i].n_planes * host[i].Rr * 4;
    if (pb > pix_bytes) pix_bytes = pb;
    w_off[i] = w_total;
    w_total += ((size_t)host[i].taps * n_chunks[i] * Kpad[i] * 16 + 255) & ~(size_t)255;
    tiles += host[i].total_tiles;
  }
  a_slot = (a_slot + 127) & ~(size_t)127;
  pix_bytes = (pix_bytes + 127) & ~(size_t)127;
  const size_t pix_one = pix_bytes;
  if (hot) pix_bytes *= G_XTEAMS;   // one table per expander team
  const size_t lay_bytes = ((size_t)count * sizeof(GLayer) + 127) & ~(size_t)127;
  const size_t fixed = (size_t)G_EPI_BYTES + pix_bytes + lay_bytes + kGTail;
  // ring depth: three slots if they fit, else two; the plan for word outputs on 4-bit operands takes two, a
  // multiple of the number of expander teams (four slots never fit beside three weight slots of these sizes)
  int na = hot ? 2 : 3, ns = 0;
  static_assert(G_XTEAMS == 1 || G_XTEAMS == 2, "the ring depth below is a multiple of the team count");
  for (; na >= 2; --na) {
    if ((size_t)na * a_slot + fixed + 3 * (size_t)kGBSlot > kGSmemBudget) continue;
    ns = (int)((kGSmemBudget - fixed - (size_t)na * a_slot) / kGBSlot);
    break;
  }
  if (na < 2 || ns < 3) return cudaErrorInvalidConfiguration;
  if (ns > G_NS_MAX) ns = G_NS_MAX;
  const int sms = sm_count();
  int grid = tiles < sms ? (int)tiles : sms;
  // A chain's CTAs wait for one another, so all of them must be resident together (a cooperative launch
  // checks that); members with fewer tiles than CTAs simply leave some CTAs without work in that member.
  std::vector<uint2> deps;
  std::vector<size_t> deps_off(count, 0), done_off(count, 0);
  size_t done_words = 0, chain_bytes = 0;
  size_t chain_off[SNN_GROUP_MAX] = {};
  if (chain) {
    for (int i = 0; i < count; ++i) {
      if (i > 0 && (gs[i].C != gs[i - 1].K || gs[i].H != gs[i - 1].Ho || gs[i].W != gs[i - 1].Wo || gs[i].N != gs[0].N))
        return cudaErrorInvalidConfiguration;
      const int mgroups = host[i].total_tiles / host[i].n_ntiles;
      done_off[i] = done_words;
      done_words += (size_t)mgroups;
      if (i + 1 < count) {
        chain_off[i] = chain_bytes;
        chain_bytes += (((size_t)gs[i].N * gs[i].Ho * gs[i].Wo * ((gs[i].K + 31) / 32) * 4) + 255) & ~(size_t)255;
      }
      if (i == 0) continue;
      // which M groups of the predecessor hold the input pixels of each of this member's M groups
      const GLayer& L = host[i];
      const GLayer& P = host[i - 1];
      deps_off[i] = deps.size();
      for (int mg = 0; mg < mgroups; ++mg) {
        const long long Q0 = (long long)mg * 128 * L.MT;
        long long lo = -1, hi = -1;
        for (int pl = 0; pl < L.n_planes; ++pl)
          for (int r = 0; r < L.Rr; ++r) {
            const int px = h_position_to_pixel(L, Q0 + r, pl >> 1, pl & 1);
            if (px < 0) continue;
            if (lo < 0 || px < lo) lo = px;
            if (px > hi) hi = px;
          }
        uint2 d = make_uint2(1u, 0u);
        if (lo >= 0) {
          // output pixel of the predecessor -> its position -> its M group
          auto group_of = [&](long long px) {
            const long long n = px / ((long long)P.Ho * P.Wo);
            const long long rem = px - n * (long long)P.Ho * P.Wo;
            const long long y = rem / P.Wo, x = rem - y * P.Wo;
            const long long q = (n * P.Hq + y) * P.Wq + x;
            return (uint32_t)(q / (128 * P.MT));
          };
          d = make_uint2(group_of(lo), group_of(hi));
        }
        deps.push_back(d);
      }
    }
  }
  // Which CTAs take a problem's odd tiles.  Every CTA gets floor(tiles / grid) tiles of a problem
  // and the first (tiles % grid) CTAs in the problem's rank order get one more; the rank order is
  // by the time the CTAs have been given so far, least first, so that the CTAs end close
  // together although a tile of one problem may take six times as long as a tile of another.
  // Time of a tile: the larger of its MMAs (73 cycles each up to 128 channels wide, 128 cycles at
  // 256) and of its fp32 output at the write rate an SM gets (13 bytes per cycle).
  std::vector<uint16_t> ranks((size_t)count * grid);
  {
    std::vector<double> busy(grid, 0.0);
    std::vector<int> order(grid);
    for (int i = 0; i < count; ++i) {
      const GLayer& o = host[i];
      const double mma = (double)o.MT * o.n_cb * o.taps * o.kpt * g_mma_cycles(o.Nt);
      const double wr = 128.0 * o.MT * (o.Nt < o.K ? o.Nt : o.K) * 4 / 13.0;
      const double cost = (mma > wr ? mma : wr) + 300.0;
      for (int b = 0; b < grid; ++b) order[b] = b;
      std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return busy[a] < busy[b]; });
      const int base = o.total_tiles / grid, rem = o.total_tiles % grid;
      for (int r = 0; r < grid; ++r) {
        ranks[(size_t)i * grid + order[r]] = (uint16_t)r;
        busy[order[r]] += cost * (base + (r < rem ? 1 : 0));
      }
    }
  }
  GroupDev* G = new GroupDev();
  G->count = count;
  G->act_type = act_type;
  G->mode = mode;
  G->grid = grid;
  G->chain = chain;
  G->kind = kind;
  G->hot = hot;
  cudaError_t e = cudaMalloc(&G->weights, w_total);
  if (chain) {
    G->done_words = done_words;
    for (int i = 0; i < count; ++i) G->chain_off[i] = chain_off[i];
    if (e == cudaSuccess) e = cudaMalloc(&G->done, done_words * sizeof(uint32_t));
    if (e == cudaSuccess) e = cudaMalloc(&G->chain_buf, chain_bytes ? chain_bytes : 256);
    if (e == cudaSuccess) e = cudaMalloc(&G->deps, (deps.size() ? deps.size() : 1) * sizeof(uint2));
    if (e == cudaSuccess && !deps.empty())
      e = cudaMemcpyAsync(G->deps, deps.data(), deps.size() * sizeof(uint2), cudaMemcpyHostToDevice, s);
  }
  if (e == cudaSuccess) e = cudaMalloc(&G->layers_dev, sizeof(GLayer) * count);
  if (e == cudaSuccess) e = cudaMalloc(&G->ranks, ranks.size() * sizeof(uint16_t));
  if (e == cudaSuccess)
    e = cudaMemcpyAsync(G->ranks, ranks.data(), ranks.size() * sizeof(uint16_t), cudaMemcpyHostToDevice, s);
  for (int i = 0; i < count && e == cudaSuccess; ++i) {
    host[i].rank = G->ranks + (size_t)i * grid;
    host[i].wt = G->weights + w_off[i];
    host[i].alpha = Ls[i]->alpha;
    host[i].shift = Ls[i]->shift;
    host[i].deps = nullptr; host[i].prev_done = nullptr; host[i].prev_target = 0; host[i].done = nullptr;
    if (chain) {
      host[i].done = G->done + done_off[i];
      if (i > 0) {
        host[i].deps = G->deps + deps_off[i];
        host[i].prev_done = G->done + done_off[i - 1];
        host[i].prev_target = (uint32_t)(G_EW * host[i - 1].n_ntiles);   // (all eight warps drain a chain's tiles)
      }
    }
    e = g_expand_weights(mode, Ls[i]->wplanes, G->weights + w_off[i], gs[i].C, gs[i].K, gs[i].Cw, Kpad[i],
                         n_chunks[i], host[i].cb_chunks, host[i].NtL, host[i].taps, s);
    if (e == cudaSuccess) *launched += 1;
  }
  if (e == cudaSuccess) e = cudaMemcpyAsync(G->layers_dev, host, sizeof(GLayer) * count, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);  // `host` and `ranks` live on this stack
  if (e != cudaSuccess) {
    tcg_destroy(G);
    return e;
  }
  GParams& p = G->p;
  p.layers = G->layers_dev;
  p.n_layers = count;
  p.NA = na;
  p.NS = ns;
  p.acc_cols = (uint32_t)g_acc_cols(mode, n_acc);
  p.n_acc = n_acc;
  p.a_slot_bytes = (uint32_t)a_slot;
  p.b_slot_bytes = kGBSlot;
  p.off_b = (uint32_t)((size_t)na * a_slot);
  p.off_epi = p.off_b + (uint32_t)ns * kGBSlot;
  p.off_pix = p.off_epi + G_EPI_BYTES;
  p.off_lay = p.off_pix + (uint32_t)pix_bytes;
  p.pix_words = (uint32_t)(pix_one / 4);
  p.off_tail = p.off_lay + (uint32_t)lay_bytes;
  G->smem = (size_t)p.off_tail + kGTail;
  if (G->smem > (size_t)kMaxDynSmem || G->smem >= (1u << 18)) {
    tcg_destroy(G);
    return cudaErrorInvalidConfiguration;
  }
  *out = G;
  return cudaSuccess;
}

void tcg_destroy(GroupDev* G) {
  if (!G) return;
  cudaFree(G->weights);
  cudaFree(G->layers_dev);
  cudaFree(G->ranks);
  cudaFree(G->done);
  cudaFree(G->chain_buf);
  cudaFree(G->deps);
  delete G;
}

int tcg_count(const GroupDev* G) { return G->count; }

bool tcg_supported(const Geom& g, int act_type) {
  // one problem alone, under every plan a launch may use: two activation slots, the fixed parts and three
  // weight slots must fit
  const int mode = g_mode_for(act_type);
  for (int n_acc = G_NACC; n_acc <= (mode == M_FP4 ? G_NACC_WORDS : G_NACC); ++n_acc) {
    GLayer L;
    int n_chunks = 0, Kpad = 0;
    if (!g_plan_layer(g, mode, n_acc, &L, &n_chunks, &Kpad)) return false;
    const size_t unit = (((size_t)L.n_planes * L.cb_chunks * L.Rr * 16) + 127) & ~(size_t)127;
    const size_t pix = (((size_t)L.n_planes * L.Rr * 4) + 127) & ~(size_t)127;
    const size_t fixed = (size_t)G_EPI_BYTES + G_XTEAMS * pix + 256 + kGTail;
    if (2 * unit + fixed + 3 * (size_t)kGBSlot > kGSmemBudget) return false;
  }
  return true;
}

cudaError_t tcg_forward(GroupDev* G, const void* const* act, void* const* out, int out_type, cudaStream_t s,
                        int* status_dev, int* launched) {
  GParams p = G->p;
  cudaLaunchAttribute attr[1];
  if (G->chain) {
    // act[0] is the first member's input and out[0] the last member's output; the packed signs in between
    // stay in the group's own buffers
    for (int i = 0; i < G->count; ++i) {
      p.act[i] = i == 0 ? act[0] : (const void*)(G->chain_buf + G->chain_off[i - 1]);
      p.out[i] = i + 1 == G->count ? out[0] : (void*)(G->chain_buf + G->chain_off[i]);
      p.out_type[i] = (uint8_t)(i + 1 == G->count ? out_type : 2);
    }
    cudaError_t e0 = cudaMemsetAsync(G->done, 0, G->done_words * sizeof(uint32_t), s);
    if (e0 != cudaSuccess) return e0;
    attr[0].id = cudaLaunchAttributeCooperative;   // the CTAs wait for one another: all must be resident
    attr[0].val.cooperative = 1;
  } else {
    for (int i = 0; i < G->count; ++i) {
      p.act[i] = act[i];
      p.out[i] = out[i];
      p.out_type[i] = (uint8_t)out_type;
    }
    // Launched as a programmatic dependent of its predecessor in the stream: set-up overlaps that
    // kernel's tail; the warps that read activations or write outputs wait on the device for it.
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
  }
  p.status = status_dev;
  cudaLaunchConfig_t cfg{};
  cfg.stream = s;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cfg.gridDim = dim3((unsigned)G->grid);
  cfg.blockDim = dim3(G_THREADS);
  cfg.dynamicSmemBytes = G->smem;
  cudaError_t e;
  const int outk = G->chain ? OUT_CHAIN : (out_type == 2 ? OUT_SIGNS : OUT_WORDS);
  if (!G->chain && (outk == OUT_SIGNS) != (G->kind == TCG_SIGNS)) return cudaErrorInvalidValue;  // planned for the other kind
  bool piped = G->hot && outk == OUT_WORDS && out_type == 0;
  // rows are read two or four words at a time by the pipelined expanders: every input 8-byte aligned
  for (int i = 0; piped && i < G->count; ++i)
    if (reinterpret_cast<uintptr_t>(act[i]) & 7) piped = false;
#define G_LAUNCH(M, O)                                                      \
  do {                                                                      \
    static unsigned long long done = 0;                                     \
    e = allow_max_smem(tcg_conv_kernel<M, O>, &done);                       \
    if (e == cudaSuccess) e = cudaLaunchKernelEx(&cfg, tcg_conv_kernel<M, O>, p); \
  } while (0)
  if (G->mode == M_F16) {
    if (outk == OUT_WORDS) G_LAUNCH(M_F16, OUT_WORDS);
    else return cudaErrorInvalidValue;   // packed signs and chains need binary activations
  } else if (outk == OUT_WORDS && piped) G_LAUNCH(M_FP4, OUT_WORDS_PIPED);
  else if (outk == OUT_WORDS) G_LAUNCH(M_FP4, OUT_WORDS);
  else if (outk == OUT_SIGNS) G_LAUNCH(M_FP4, OUT_SIGNS);
  else G_LAUNCH(M_FP4, OUT_CHAIN);
#undef G_LAUNCH
  if (e != cudaSuccess) return e;
  *launched += 1;
#ifdef SNN_TRACE
  {
    static long long h[256 * 16];
    cudaDeviceSynchronize();
    cudaMemcpyFromSymbol(h, g_trace, sizeof(h));
    static const char* role[4] = {"producer", "mma", "epilogue", "expander"};
    for (int r = 0; r < 4; ++r) {
      double a[4] = {0, 0, 0, 0}, mx = 0;
      for (int b = 0; b < G->grid; ++b) {
        for (int k = 0; k < 4; ++k) a[k] += (double)h[b * 16 + r * 4 + k] / G->grid;
        if ((double)h[b * 16 + r * 4] > mx) mx = (double)h[b * 16 + r * 4];
      }
      fprintf(stderr, "[trace] %-9s total %8.0f (max %8.0f)  waits %8.0f %8.0f %8.0f cycles\n", role[r], a[0], mx, a[1], a[2],
              a[3]);
    }
  }
#endif
  return cudaGetLastError();
}

}  // namespace snn
