/*
 * CPU oracle for the sub-bit binary 3x3 convolution (test infrastructure).
 *
 * THIS IS NOT PART OF THE PRODUCT.  It exists so that tests, the smoke check
 * and the benchmark's host-baseline leg have a plain, slow, obviously correct
 * answer to compare the CUDA library against.  It shares no code, header,
 * table or helper with the CUDA path and is never called from it.
 *
 * What it computes (Sec. 3, a^i = lambda^i * (w_bar^i o a_bar^{i-1}); Sec. 4.4,
 * every (c_out, c_in) kernel is a tau-bit index into a per-layer set of 2^tau
 * binary 3x3 kernels; Sec. 4.1, a binary kernel is numbered by reading its
 * flattened +/-1 entries as a binary sequence, all -1 being the first and all
 * +1 the last of the 512):
 *
 *   S[n,co,y,x] = sum_{ci} sum_{ky<3} sum_{kx<3} w(co,ci,ky,kx) * a(n, y*s+ky-p, x*s+kx-p, ci)
 *   w(co,ci,ky,kx) = +1 if bit (8 - (3*ky+kx)) of codebook[idx[co][ci]] is set, else -1
 *   a(n,r,c,ci)    = 0 outside the image, else +1 / -1 for activation bit 1 / 0
 *   Y[n,co,y,x]    = (float)S * alpha[co]          (one fp32 multiply)
 *
 * The sum is a cross-correlation (no kernel flip), zero padding contributes 0,
 * the scale is per output channel and the output size is floor((H+2p-3)/s)+1.
 * The bit order of a code and the index-stream packing are conventions of
 * this repository (the paper's figures that would fix them are not available):
 * parity unpinned by the paper for those two; everything else is pinned by
 * tests/test_oracle_*.py.
 *
 * The method reaches exactly this result by a cheaper route, so the oracle is
 * the definition written out as seven nested loops over integer +/-1 values.
 * No popcount, no packing tricks, no tables.
 *
 * Layouts: activations uint32 [N][H][W][ceil(C/32)] (channel ci = bit ci%32 of
 * word ci/32) or IEEE binary16 bit patterns [N][H][W][C]; outputs [N][Ho][Wo][K].
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_NO_MEM 2

int snn_oracle_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* tau-bit element e of an LSB-first bit stream (Sec. 4.4 storage). */
static uint32_t stream_get(const uint8_t* stream, int tau, size_t e) {
  uint32_t v = 0;
  for (int b = 0; b < tau; ++b) {
    size_t bit = e * (size_t)tau + (size_t)b;
    uint32_t one = (stream[bit >> 3] >> (bit & 7)) & 1u;
    v |= one << b;
  }
  return v;
}

/* Decode indices + codebook into dense +/-1 weights w[K][C][3][3] (Sec. 4.1 numbering). */
static int8_t* decode_weights(const uint16_t* codebook, int tau, const uint8_t* idx_packed,
                              int C, int K) {
  int8_t* w = (int8_t*)malloc((size_t)K * C * 9);
  if (!w) return NULL;
  for (int co = 0; co < K; ++co)
    for (int ci = 0; ci < C; ++ci) {
      uint32_t j = stream_get(idx_packed, tau, (size_t)co * C + ci);
      uint32_t code = codebook[j];
      for (int ky = 0; ky < 3; ++ky)
        for (int kx = 0; kx < 3; ++kx) {
          int bit = (code >> (8 - (3 * ky + kx))) & 1;
          w[(((size_t)co * C + ci) * 3 + ky) * 3 + kx] = bit ? 1 : -1;
        }
    }
  return w;
}

/* Export the decoded weights (for tests that hand them to a library conv). */
int snn_oracle_decode(const uint16_t* codebook, int tau, const uint8_t* idx_packed, int C, int K,
                      int8_t* w_out) {
  if (!codebook || !idx_packed || !w_out || tau < 1 || tau > 9 || C < 1 || K < 1) return ORACLE_BAD_ARG;
  for (int j = 0; j < (1 << tau); ++j)
    if (codebook[j] >= 512) return ORACLE_BAD_ARG;
  int8_t* w = decode_weights(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
  memcpy(w_out, w, (size_t)K * C * 9);
  free(w);
  return ORACLE_OK;
}

static int check_common(const uint16_t* codebook, int tau, const uint8_t* idx_packed,
                        const float* alpha, int C, int K, int stride, int pad, const void* act,
                        int N, int H, int W) {
  if (!codebook || !idx_packed || !alpha || !act) return ORACLE_BAD_ARG;
  if (tau < 1 || tau > 9 || C < 1 || K < 1 || N < 0 || H < 1 || W < 1) return ORACLE_BAD_ARG;
  if (stride < 1 || pad < 0) return ORACLE_BAD_ARG;
  if (H + 2 * pad < 3 || W + 2 * pad < 3) return ORACLE_BAD_ARG;
  for (int j = 0; j < (1 << tau); ++j)
    if (codebook[j] >= 512) return ORACLE_BAD_ARG;
  return ORACLE_OK;
}

/*
 * Binary activations.  S_out and/or Y_out may be NULL.
 */
int snn_oracle_conv_bin(const uint16_t* codebook, int tau, const uint8_t* idx_packed,
                        const float* alpha, int C, int K, int stride, int pad,
                        const uint32_t* act, int N, int H, int W, int32_t* S_out, float* Y_out) {
  int rc = check_common(codebook, tau, idx_packed, alpha, C, K, stride, pad, act, N, H, W);
  if (rc) return rc;
  const int Ho = (H + 2 * pad - 3) / stride + 1;
  const int Wo = (W + 2 * pad - 3) / stride + 1;
  const int Cw = (C + 31) / 32;
  int8_t* w = decode_weights(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
  /* +/-1 activations as plain integers, a[n][r][c][ci] */
  int8_t* a = (int8_t*)malloc((size_t)N * H * W * C + 1);
  if (!a) { free(w); return ORACLE_NO_MEM; }
  for (size_t px = 0; px < (size_t)N * H * W; ++px)
    for (int ci = 0; ci < C; ++ci) {
      uint32_t word = act[px * Cw + (ci >> 5)];
      a[px * C + ci] = ((word >> (ci & 31)) & 1u) ? 1 : -1;
    }

#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < K; ++co)
      for (int y = 0; y < Ho; ++y)
        for (int x = 0; x < Wo; ++x) {
          int32_t s = 0;
          for (int ci = 0; ci < C; ++ci)
            for (int ky = 0; ky < 3; ++ky)
              for (int kx = 0; kx < 3; ++kx) {
                int r = y * stride + ky - pad;
                int c = x * stride + kx - pad;
                if (r < 0 || r >= H || c < 0 || c >= W) continue; /* zero padding adds 0 */
                int av = a[(((size_t)n * H + r) * W + c) * C + ci];
                int wv = w[(((size_t)co * C + ci) * 3 + ky) * 3 + kx];
                s += wv * av;
              }
          size_t o = (((size_t)n * Ho + y) * Wo + x) * K + co;
          if (S_out) S_out[o] = s;
          if (Y_out) Y_out[o] = (float)s * alpha[co];
        }
  free(a);
  free(w);
  return ORACLE_OK;
}

/* IEEE binary16 bit pattern -> double, exactly. */
static double half_bits_to_double(uint16_t hb) {
  int sign = (hb >> 15) & 1;
  int ex = (hb >> 10) & 0x1f;
  int man = hb & 0x3ff;
  double v;
  if (ex == 0) v = ldexp((double)man, -24);
  else if (ex == 31) v = man ? NAN : INFINITY;
  else v = ldexp((double)(man + 1024), ex - 25);
  return sign ? -v : v;
}

/*
 * Weights-only variant (Sec. 5.3 deployment test: activations not binarised):
 * fp16 activations, +/-1 weights, accumulation in double in the loop order of
 * the definition, Y = (float)(alpha * sum).
 */
int snn_oracle_conv_f16(const uint16_t* codebook, int tau, const uint8_t* idx_packed,
                        const float* alpha, int C, int K, int stride, int pad,
                        const uint16_t* act_half_bits, int N, int H, int W, float* Y_out) {
  int rc = check_common(codebook, tau, idx_packed, alpha, C, K, stride, pad, act_half_bits, N, H, W);
  if (rc) return rc;
  if (!Y_out) return ORACLE_BAD_ARG;
  const int Ho = (H + 2 * pad - 3) / stride + 1;
  const int Wo = (W + 2 * pad - 3) / stride + 1;
  int8_t* w = decode_weights(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
  double* a = (double*)malloc(((size_t)N * H * W * C + 1) * sizeof(double));
  if (!a) { free(w); return ORACLE_NO_MEM; }
  for (size_t i = 0; i < (size_t)N * H * W * C; ++i) a[i] = half_bits_to_double(act_half_bits[i]);

#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < K; ++co)
      for (int y = 0; y < Ho; ++y)
        for (int x = 0; x < Wo; ++x) {
          double s = 0.0;
          for (int ci = 0; ci < C; ++ci)
            for (int ky = 0; ky < 3; ++ky)
              for (int kx = 0; kx < 3; ++kx) {
                int r = y * stride + ky - pad;
                int c = x * stride + kx - pad;
                if (r < 0 || r >= H || c < 0 || c >= W) continue;
                double av = a[(((size_t)n * H + r) * W + c) * C + ci];
                int wv = w[(((size_t)co * C + ci) * 3 + ky) * 3 + kx];
                s += (double)wv * av;
              }
          size_t o = (((size_t)n * Ho + y) * Wo + x) * K + co;
          Y_out[o] = (float)((double)alpha[co] * s);
        }
  free(a);
  free(w);
  return ORACLE_OK;
}

/*
 * ---------------------------------------------------------------------------
 * 1x1 extension (appendix "Extending to Bottleneck with 1x1 Kernels" and its
 * comparison table): the weights of a 1x1 layer are cut into c_out * c_in / 8
 * vectors of 8 consecutive input channels; every vector is a tau'-bit index
 * (1 <= tau' <= 8; tau' = 8 is the full set, i.e. a plain 1-bit layer) into a
 * layer-specific set of 2^tau' vectors from {-1,+1}^8 (256 in all).
 *
 *   S[n,co,y,x] = sum_{ci} w(co,ci) * a(n, y*s, x*s, ci)        (no padding)
 *   w(co, 8g + j) = +1 if bit (7 - j) of codebook[idx[co][g]] is set, else -1
 *   Y = (float)S * alpha[co]
 *
 * The numbering follows the 3x3 kernels' (Sec. 4.1): the flattened vector read
 * as a binary sequence, first element most significant, all -1 first (code 0)
 * and all +1 last (code 255).  The index stream is the same LSB-first tau'-bit
 * stream, element e = co * (c_in/8) + g.  Bit order and packing are conventions
 * of this repository (parity unpinned by the paper for those two).
 * ---------------------------------------------------------------------------
 */
static int8_t* decode_weights1x1(const uint16_t* codebook, int tau, const uint8_t* idx_packed, int C, int K) {
  int8_t* w = (int8_t*)malloc((size_t)K * C);
  if (!w) return NULL;
  const int G = C / 8;
  for (int co = 0; co < K; ++co)
    for (int g = 0; g < G; ++g) {
      uint32_t j = stream_get(idx_packed, tau, (size_t)co * G + g);
      uint32_t code = codebook[j];
      for (int e = 0; e < 8; ++e) w[(size_t)co * C + 8 * g + e] = ((code >> (7 - e)) & 1) ? 1 : -1;
    }
  return w;
}

static int check_1x1(const uint16_t* codebook, int tau, const uint8_t* idx_packed, int C, int K) {
  if (!codebook || !idx_packed || tau < 1 || tau > 8 || C < 8 || (C % 8) || K < 1) return ORACLE_BAD_ARG;
  for (int j = 0; j < (1 << tau); ++j)
    if (codebook[j] >= 256) return ORACLE_BAD_ARG;
  return ORACLE_OK;
}

int snn_oracle_decode1x1(const uint16_t* codebook, int tau, const uint8_t* idx_packed, int C, int K, int8_t* w_out) {
  int rc = check_1x1(codebook, tau, idx_packed, C, K);
  if (rc || !w_out) return ORACLE_BAD_ARG;
  int8_t* w = decode_weights1x1(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
  memcpy(w_out, w, (size_t)K * C);
  free(w);
  return ORACLE_OK;
}

int snn_oracle_conv1x1_bin(const uint16_t* codebook, int tau, const uint8_t* idx_packed, const float* alpha, int C,
                           int K, int stride, const uint32_t* act, int N, int H, int W, int32_t* S_out,
                           float* Y_out) {
  int rc = check_1x1(codebook, tau, idx_packed, C, K);
  if (rc) return rc;
  if (!alpha || !act || N < 0 || H < 1 || W < 1 || stride < 1) return ORACLE_BAD_ARG;
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  const int Cw = (C + 31) / 32;
  int8_t* w = decode_weights1x1(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < K; ++co)
      for (int y = 0; y < Ho; ++y)
        for (int x = 0; x < Wo; ++x) {
          const size_t px = ((size_t)n * H + (size_t)y * stride) * W + (size_t)x * stride;
          int32_t s = 0;
          for (int ci = 0; ci < C; ++ci) {
            uint32_t word = act[px * Cw + (ci >> 5)];
            int av = ((word >> (ci & 31)) & 1u) ? 1 : -1;
            s += (int)w[(size_t)co * C + ci] * av;
          }
          size_t o = (((size_t)n * Ho + y) * Wo + x) * K + co;
          if (S_out) S_out[o] = s;
          if (Y_out) Y_out[o] = (float)s * alpha[co];
        }
  free(w);
  return ORACLE_OK;
}

int snn_oracle_conv1x1_f16(const uint16_t* codebook, int tau, const uint8_t* idx_packed, const float* alpha, int C,
                           int K, int stride, const uint16_t* act_half_bits, int N, int H, int W, float* Y_out) {
  int rc = check_1x1(codebook, tau, idx_packed, C, K);
  if (rc) return rc;
  if (!alpha || !act_half_bits || !Y_out || N < 0 || H < 1 || W < 1 || stride < 1) return ORACLE_BAD_ARG;
  const int Ho = (H - 1) / stride + 1, Wo = (W - 1) / stride + 1;
  int8_t* w = decode_weights1x1(codebook, tau, idx_packed, C, K);
  if (!w) return ORACLE_NO_MEM;
#pragma omp parallel for collapse(2) schedule(static)
  for (int n = 0; n < N; ++n)
    for (int co = 0; co < K; ++co)
      for (int y = 0; y < Ho; ++y)
        for (int x = 0; x < Wo; ++x) {
          const size_t px = ((size_t)n * H + (size_t)y * stride) * W + (size_t)x * stride;
          double s = 0.0;
          for (int ci = 0; ci < C; ++ci)
            s += (double)w[(size_t)co * C + ci] * half_bits_to_double(act_half_bits[px * C + ci]);
          size_t o = (((size_t)n * Ho + y) * Wo + x) * K + co;
          Y_out[o] = (float)((double)alpha[co] * s);
        }
  free(w);
  return ORACLE_OK;
}
