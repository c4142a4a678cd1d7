/*
 * CPU ORACLE for binarized convolution (daBNN, arXiv 1908.05858).
 *
 * THIS FILE IS TEST INFRASTRUCTURE, NOT THE PRODUCT.  It is a plain, slow, scalar
 * statement of what the method computes, written from the paper, so that the CUDA
 * library can be checked against it.  It shares no code, header, table or helper with
 * the CUDA path, and the CUDA path never calls it.  Only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may load it.
 *
 * What each function follows:
 *   oracle_pack_c2 / oracle_bconv_bits_c2   the same packer and Eq. 1 with the activations in the paper's NC1HWC2
 *                                       layout (Section 2.1.2, last paragraph; Fig. 3), C2 = 128 bits.
 *   oracle_pack / oracle_pack_i32 / oracle_pack_weights
 *                                       Section 2.1.1 (bit-packing), the "naive" sequential
 *                                       packer the paper describes as the prior method:
 *                                       test every element, set its bit.
 *   oracle_bconv_pm1                    Section 2.1.2, last paragraph: A = weights (M = C_out),
 *                                       B = im2col'ed input (N = OH*OW): the convolution of
 *                                       the two {-1,+1} tensors, written as the definition.
 *   oracle_bconv_bits                   Eq. 1 (BGEMM: sum_k bitcount(xnor(A_ik, B_kj))) on the
 *                                       packed words, turned into the +-1 dot product
 *                                       2*C_xnor - K  =  K - 2*sum popcount(xor).
 *   oracle_bgemm_xnor                   Eq. 1 as printed: counts of agreeing bit positions, C in N^{M x N}.
 *   oracle_bn_fold / oracle_bn_sign_pack  Section 2.1.1, last sentence (fused BN + binarize).
 *   oracle_bn_add_sign_pack             the same with the real-valued shortcut of Section 2.3 added before the sign.
 *   oracle_bireal18_forward             Section 2.3 / Table 2: Bi-Real Net 18 (a binary
 *                                       ResNet-18; first conv and last fc in full precision).
 *
 * Readings of the paper taken here (the paper is silent or loose on each):
 *   - binarize: v = (x < 0) ? -1 : +1, as an IEEE comparison; +0.0, -0.0 and NaN give +1.
 *     The packed bit is 1 for -1 (the IEEE sign bit of every non-zero, non-NaN value).
 *   - 64-bit words, channel c -> word c>>6, bit c&63 (LSB first); tail bits are 0.
 *   - packed activations are [N][H][W][Cw], packed weights [O][kh][kw][Cw], Cw = ceil(C/64).
 *   - spatial padding has a declared value in {-1,+1}; every output sums K = C*kh*kw terms.
 *   - cross-correlation (no kernel flip), dilation 1, groups 1.
 *   - BN folded in double: sd = gamma / sqrt(var + eps); scale = (float)sd;
 *     shift = (float)(beta - mean*sd); y = fmaf((float)acc, scale, shift); bit = (y < 0).
 *   - every fp32 operation of the network is one correctly rounded IEEE operation in a
 *     stated order (see oracle_bireal18_forward), so the result is single-valued.
 *
 * Parity of oracle_bireal18_forward's TOPOLOGY is unpinned by the paper (it only names
 * the network); its arithmetic is pinned by the tests against fp64 library routines.  The same holds
 * for the STEM module variant (Section 2.3): its figure is missing from the paper's text, so the
 * module's structure is a reading (see stem_module): PARITY UNPINNED by the paper.
 *
 * Build: gcc -O2 -mfma -mpopcnt -ffp-contract=off -fopenmp -shared -fPIC oracle.c -lm
 * (-ffp-contract=off: the only fused multiply-adds are the explicit fmaf calls.)
 */
#include <math.h>
#include <stddef.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define LAYOUT_NCHW 0
#define LAYOUT_NHWC 1

static int g_threads = 1;

void oracle_set_threads(int n) { g_threads = n < 1 ? 1 : n; }
int oracle_get_threads(void) { return g_threads; }
int oracle_max_threads(void) {
#ifdef _OPENMP
  return omp_get_num_procs();
#else
  return 1;
#endif
}

/* ---- binarize (Section 2.1.1) ------------------------------------------------------ */
static int binarize(float x) { return (x < 0.0f) ? -1 : +1; }

static size_t words_per_pixel(int C) { return (size_t)((C + 63) / 64); }

/* bitcount of Eq. 1: the number of set bits of a word.  The compiler's builtin (one POPCNT instruction with -mpopcnt) is
   the default; -DORACLE_BITCOUNT_LOOP selects a bit-by-bit loop instead.  oracle_bitcount exposes it to the pins. */
static int popcount64(uint64_t v) {
#ifdef ORACLE_BITCOUNT_LOOP
  int n = 0;
  while (v) { n += (int)(v & 1u); v >>= 1; }
  return n;
#else
  return __builtin_popcountll(v);
#endif
}
int oracle_bitcount(uint64_t v) { return popcount64(v); }

/* ---- pack (Section 2.1.1, the sequential packer) ----------------------------------- */
void oracle_pack(const float* x, int layout, int N, int C, int H, int W, uint64_t* P) {
  size_t Cw = words_per_pixel(C);
  memset(P, 0, (size_t)N * H * W * Cw * sizeof(uint64_t));
  for (int n = 0; n < N; n++)
    for (int h = 0; h < H; h++)
      for (int w = 0; w < W; w++)
        for (int c = 0; c < C; c++) {
          size_t xi = (layout == LAYOUT_NCHW) ? (((size_t)n * C + c) * H + h) * W + w
                                              : (((size_t)n * H + h) * W + w) * C + c;
          uint64_t bit = (binarize(x[xi]) == -1) ? 1u : 0u;
          P[(((size_t)n * H + h) * W + w) * Cw + (size_t)(c >> 6)] |= bit << (c & 63);
        }
}

/* Section 2.1.1, int32 input: the bit is the sign bit of the integer, i.e. 1 for x < 0 (0 packs as +1). */
void oracle_pack_i32(const int32_t* x, int layout, int N, int C, int H, int W, uint64_t* P) {
  size_t Cw = words_per_pixel(C);
  memset(P, 0, (size_t)N * H * W * Cw * sizeof(uint64_t));
  for (int n = 0; n < N; n++)
    for (int h = 0; h < H; h++)
      for (int w = 0; w < W; w++)
        for (int c = 0; c < C; c++) {
          size_t xi = (layout == LAYOUT_NCHW) ? (((size_t)n * C + c) * H + h) * W + w
                                              : (((size_t)n * H + h) * W + w) * C + c;
          uint64_t bit = (x[xi] < 0) ? 1u : 0u;
          P[(((size_t)n * H + h) * W + w) * Cw + (size_t)(c >> 6)] |= bit << (c & 63);
        }
}

/* Section 2.1.2, last paragraph (Fig. 3): the NC1HWC2 layout with C2 = 128 bits.  P is [N][C1][H][W][2] 64-bit words,
   C1 = ceil(C/128); channel c sets bit c&63 of word (c>>6)&1 of group c>>7.  Same sequential packer. */
void oracle_pack_c2(const float* x, int layout, int N, int C, int H, int W, uint64_t* P) {
  size_t C1 = (size_t)((C + 127) / 128);
  memset(P, 0, (size_t)N * C1 * H * W * 2 * sizeof(uint64_t));
  for (int n = 0; n < N; n++)
    for (int h = 0; h < H; h++)
      for (int w = 0; w < W; w++)
        for (int c = 0; c < C; c++) {
          size_t xi = (layout == LAYOUT_NCHW) ? (((size_t)n * C + c) * H + h) * W + w
                                              : (((size_t)n * H + h) * W + w) * C + c;
          uint64_t bit = (binarize(x[xi]) == -1) ? 1u : 0u;
          P[((((size_t)n * C1 + (size_t)(c >> 7)) * H + h) * W + w) * 2 + (size_t)((c >> 6) & 1)] |= bit << (c & 63);
        }
}

void oracle_pack_weights(const float* w_oihw, int O, int C, int kh, int kw, uint64_t* Wp) {
  size_t Cw = words_per_pixel(C);
  memset(Wp, 0, (size_t)O * kh * kw * Cw * sizeof(uint64_t));
  for (int o = 0; o < O; o++)
    for (int c = 0; c < C; c++)
      for (int i = 0; i < kh; i++)
        for (int j = 0; j < kw; j++) {
          float v = w_oihw[(((size_t)o * C + c) * kh + i) * kw + j];
          uint64_t bit = (binarize(v) == -1) ? 1u : 0u;
          Wp[(((size_t)o * kh + i) * kw + j) * Cw + (size_t)(c >> 6)] |= bit << (c & 63);
        }
}

static int out_dim(int in, int k, int stride, int pad) { return (in + 2 * pad - k) / stride + 1; }

static size_t out_index(int layout, int n, int o, int oh, int ow, int O, int OH, int OW) {
  return (layout == LAYOUT_NCHW) ? (((size_t)n * O + o) * OH + oh) * OW + ow
                                 : (((size_t)n * OH + oh) * OW + ow) * O + o;
}

/* ---- convolution of the +-1 tensors (the definition; Section 2.1.2) ---------------- */
static int32_t pm1_one(const float* x, int C, int H, int W, const float* wt, int kh, int kw,
                       int sh, int sw, int ph, int pw, int pad_value, int n, int o, int oh, int ow) {
  double s = 0.0;
  for (int c = 0; c < C; c++)
    for (int i = 0; i < kh; i++)
      for (int j = 0; j < kw; j++) {
        int ih = oh * sh + i - ph, iw = ow * sw + j - pw;
        double a = (ih < 0 || ih >= H || iw < 0 || iw >= W)
                       ? (double)pad_value
                       : (double)binarize(x[(((size_t)n * C + c) * H + ih) * W + iw]);
        double b = (double)binarize(wt[(((size_t)o * C + c) * kh + i) * kw + j]);
        s += a * b;
      }
  return (int32_t)s;
}

void oracle_bconv_pm1(const float* x_nchw, int N, int C, int H, int W, const float* w_oihw, int O,
                      int kh, int kw, int sh, int sw, int ph, int pw, int pad_value, int32_t* out,
                      int out_layout) {
  int OH = out_dim(H, kh, sh, ph), OW = out_dim(W, kw, sw, pw);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int o = 0; o < O; o++)
      for (int oh = 0; oh < OH; oh++)
        for (int ow = 0; ow < OW; ow++)
          out[out_index(out_layout, n, o, oh, ow, O, OH, OW)] =
              pm1_one(x_nchw, C, H, W, w_oihw, kh, kw, sh, sw, ph, pw, pad_value, n, o, oh, ow);
}

/* The same definition at a list of output coordinates (n, o, oh, ow quadruples). */
void oracle_bconv_pm1_at(const float* x_nchw, int N, int C, int H, int W, const float* w_oihw, int O,
                         int kh, int kw, int sh, int sw, int ph, int pw, int pad_value,
                         const int32_t* coords, int64_t ncoords, int32_t* vals) {
  (void)N; (void)O;
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (int64_t q = 0; q < ncoords; q++)
    vals[q] = pm1_one(x_nchw, C, H, W, w_oihw, kh, kw, sh, sw, ph, pw, pad_value,
                      coords[4 * q], coords[4 * q + 1], coords[4 * q + 2], coords[4 * q + 3]);
}

/* ---- Eq. 1 on the packed words ------------------------------------------------------ */
static uint64_t pad_word(int C, int cw, int pad_value) {
  /* all valid channel bits of word cw hold [pad_value < 0]; tail bits are 0 */
  if (pad_value >= 0) return 0;
  int valid = C - 64 * cw;
  if (valid >= 64) return ~(uint64_t)0;
  return (((uint64_t)1) << valid) - 1;
}

static int32_t bits_one(const uint64_t* A, int C, int H, int W, const uint64_t* Wp, int kh, int kw,
                        int sh, int sw, int ph, int pw, int pad_value, int n, int o, int oh, int ow) {
  int Cw = (int)words_per_pixel(C);
  int K = C * kh * kw;
  int agree = 0; /* C_ij of Eq. 1: number of positions where the two bits are equal */
  for (int i = 0; i < kh; i++)
    for (int j = 0; j < kw; j++)
      for (int cw = 0; cw < Cw; cw++) {
        int ih = oh * sh + i - ph, iw = ow * sw + j - pw;
        uint64_t a = (ih < 0 || ih >= H || iw < 0 || iw >= W)
                         ? pad_word(C, cw, pad_value)
                         : A[(((size_t)n * H + ih) * W + iw) * Cw + cw];
        uint64_t b = Wp[(((size_t)o * kh + i) * kw + j) * Cw + cw];
        int valid = C - 64 * cw;
        if (valid > 64) valid = 64;
        /* xnor counts the equal positions; the tail (both 0) would count too, so only
           the valid positions of the word are looked at */
        uint64_t mask = (valid == 64) ? ~(uint64_t)0 : ((((uint64_t)1) << valid) - 1);
        agree += popcount64(~(a ^ b) & mask);
      }
  return (int32_t)(2 * agree - K);
}

void oracle_bconv_bits(const uint64_t* A, int N, int C, int H, int W, const uint64_t* Wp, int O,
                       int kh, int kw, int sh, int sw, int ph, int pw, int pad_value, int32_t* out,
                       int out_layout) {
  int OH = out_dim(H, kh, sh, ph), OW = out_dim(W, kw, sw, pw);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int oh = 0; oh < OH; oh++)
      for (int ow = 0; ow < OW; ow++)
        for (int o = 0; o < O; o++)
          out[out_index(out_layout, n, o, oh, ow, O, OH, OW)] =
              bits_one(A, C, H, W, Wp, kh, kw, sh, sw, ph, pw, pad_value, n, o, oh, ow);
}

void oracle_bconv_bits_at(const uint64_t* A, int N, int C, int H, int W, const uint64_t* Wp, int O,
                          int kh, int kw, int sh, int sw, int ph, int pw, int pad_value,
                          const int32_t* coords, int64_t ncoords, int32_t* vals) {
  (void)N; (void)O;
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (int64_t q = 0; q < ncoords; q++)
    vals[q] = bits_one(A, C, H, W, Wp, kh, kw, sh, sw, ph, pw, pad_value, coords[4 * q],
                       coords[4 * q + 1], coords[4 * q + 2], coords[4 * q + 3]);
}

/* Eq. 1 on activations in the NC1HWC2 layout (weights stay [O][kh][kw][Cw]): the same sum, words fetched from
   [N][C1][H][W][2]. */
void oracle_bconv_bits_c2(const uint64_t* A, int N, int C, int H, int W, const uint64_t* Wp, int O,
                          int kh, int kw, int sh, int sw, int ph, int pw, int pad_value, int32_t* out,
                          int out_layout) {
  int OH = out_dim(H, kh, sh, ph), OW = out_dim(W, kw, sw, pw);
  int Cw = (int)words_per_pixel(C), C1 = (C + 127) / 128, K = C * kh * kw;
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int oh = 0; oh < OH; oh++)
      for (int ow = 0; ow < OW; ow++)
        for (int o = 0; o < O; o++) {
          int agree = 0;
          for (int i = 0; i < kh; i++)
            for (int j = 0; j < kw; j++)
              for (int cw = 0; cw < Cw; cw++) {
                int ih = oh * sh + i - ph, iw = ow * sw + j - pw;
                uint64_t a = (ih < 0 || ih >= H || iw < 0 || iw >= W)
                                 ? pad_word(C, cw, pad_value)
                                 : A[((((size_t)n * C1 + (size_t)(cw >> 1)) * H + ih) * W + iw) * 2 + (size_t)(cw & 1)];
                uint64_t b = Wp[(((size_t)o * kh + i) * kw + j) * Cw + cw];
                int valid = C - 64 * cw;
                if (valid > 64) valid = 64;
                uint64_t mask = (valid == 64) ? ~(uint64_t)0 : ((((uint64_t)1) << valid) - 1);
                agree += popcount64(~(a ^ b) & mask);
              }
          out[out_index(out_layout, n, o, oh, ow, O, OH, OW)] = (int32_t)(2 * agree - K);
        }
}

/* ---- BGEMM exactly as Eq. 1 prints it: C_ij = sum_k bitcount(xnor(A_ik, B_kj)) ------------------------
 * A is [M][Kw] packed rows, B is given by its columns as [N][Kw] packed rows (column j of the paper's B),
 * Kbits valid bits per row (tail bits 0 in both).  C is [M][N], a count of agreeing positions in 0..Kbits. */
void oracle_bgemm_xnor(const uint64_t* A, int M, const uint64_t* B, int N, int Kbits, int32_t* Cout) {
  int Kw = (int)words_per_pixel(Kbits);
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (int i = 0; i < M; i++)
    for (int j = 0; j < N; j++) {
      int count = 0;
      for (int k = 0; k < Kw; k++) {
        int valid = Kbits - 64 * k;
        if (valid > 64) valid = 64;
        uint64_t mask = (valid == 64) ? ~(uint64_t)0 : ((((uint64_t)1) << valid) - 1);
        count += popcount64(~(A[(size_t)i * Kw + k] ^ B[(size_t)j * Kw + k]) & mask);
      }
      Cout[(size_t)i * N + j] = count;
    }
}

/* ---- fused BN + binarize (Section 2.1.1, last sentence) ----------------------------- */
void oracle_bn_fold(const float* gamma, const float* beta, const float* mean, const float* var,
                    double eps, int O, float* scale, float* shift) {
  for (int o = 0; o < O; o++) {
    double sd = (double)gamma[o] / sqrt((double)var[o] + eps);
    double prod = (double)mean[o] * sd;
    scale[o] = (float)sd;
    shift[o] = (float)((double)beta[o] - prod);
  }
}

/* acc is [npix][O] (NHWC with the pixel axes flattened); out is [npix][ceil(O/64)] */
void oracle_bn_sign_pack(const int32_t* acc, int64_t npix, int O, const float* scale,
                         const float* shift, uint64_t* out) {
  size_t Ow = words_per_pixel(O);
  memset(out, 0, (size_t)npix * Ow * sizeof(uint64_t));
  for (int64_t p = 0; p < npix; p++)
    for (int o = 0; o < O; o++) {
      float y = fmaf((float)acc[(size_t)p * O + o], scale[o], shift[o]);
      uint64_t bit = (binarize(y) == -1) ? 1u : 0u;
      out[(size_t)p * Ow + (size_t)(o >> 6)] |= bit << (o & 63);
    }
}

/* ---- the Bi-Real block epilogue (Section 2.1.1, last sentence, with the real-valued shortcut of Section 2.3) ----
 * y = fmaf((float)acc, scale[o], shift[o]) + r: the BN as one fused multiply-add, then ONE rounded fp32 add of the
 * shortcut value; the packed bit is the sign of y.  acc, r and y are [npix][O]; bits is [npix][ceil(O/64)]. */
void oracle_bn_add_sign_pack(const int32_t* acc, int64_t npix, int O, const float* scale, const float* shift,
                             const float* r, float* y, uint64_t* bits) {
  size_t Ow = words_per_pixel(O);
  memset(bits, 0, (size_t)npix * Ow * sizeof(uint64_t));
  for (int64_t p = 0; p < npix; p++)
    for (int o = 0; o < O; o++) {
      size_t i = (size_t)p * O + o;
      float bn = fmaf((float)acc[i], scale[o], shift[o]);
      float v = bn + r[i];
      y[i] = v;
      uint64_t bit = (binarize(v) == -1) ? 1u : 0u;
      bits[(size_t)p * Ow + (size_t)(o >> 6)] |= bit << (o & 63);
    }
}

/* ---- Bi-Real Net 18 (Section 2.3, Table 2) ------------------------------------------ */
typedef struct {
  const float* stem_w;                       /* [64][3][7][7] */
  const float* stem_bn[4];                   /* gamma, beta, mean, var, each [64] */
  const float* block_w[16];                  /* fp32 OIHW [O][C][3][3]; binarized here */
  const float* block_bn[16][4];              /* each [O] */
  const float* down_w[3];                    /* fp32 [O][C] 1x1, stages 2..4 */
  const float* down_bn[3][4];
  const float* fc_w;                         /* [1000][512] */
  const float* fc_b;                         /* [1000] */
  double bn_eps;
  int conv_form;                             /* 0: +-1 products (definition), 1: Eq. 1 on packed words */
  int use_stem_module;                       /* 0: 7x7 stem conv + max-pool; 1: the STEM module below (Section 2.3, Fig. 6) */
  const float* sm_w[4];                      /* [32][3][3][3], [16][32][1][1], [32][16][3][3], [64][64][1][1] */
  const float* sm_bn[4][4];                  /* gamma, beta, mean, var of the BN after each of the four convolutions */
} oracle_bireal18_params;

/* One fp32 convolution of the STEM module, NCHW, zero padding, no bias, in the pinned order (c, kh, kw ascending, taps
   outside the image skipped), then y = fmaf(acc, scale, shift) and, if relu, y = (y > 0) ? y : +0. */
static void conv_bn_fp32(const float* x, int N, int C, int H, int W, const float* w, int O, int k, int stride, int pad,
                         const float* scale, const float* shift, int relu, float* y) {
  int OH = out_dim(H, k, stride, pad), OW = out_dim(W, k, stride, pad);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int o = 0; o < O; o++)
      for (int oh = 0; oh < OH; oh++)
        for (int ow = 0; ow < OW; ow++) {
          float a = 0.0f;
          for (int c = 0; c < C; c++)
            for (int i = 0; i < k; i++)
              for (int j = 0; j < k; j++) {
                int ih = oh * stride + i - pad, iw = ow * stride + j - pad;
                if (ih < 0 || ih >= H || iw < 0 || iw >= W) continue;
                a = fmaf(x[(((size_t)n * C + c) * H + ih) * W + iw], w[(((size_t)o * C + c) * k + i) * k + j], a);
              }
          float v = fmaf(a, scale[o], shift[o]);
          if (relu) v = (v > 0.0f) ? v : 0.0f;
          y[(((size_t)n * O + o) * OH + oh) * OW + ow] = v;
        }
}

/* The STEM module that replaces the 7x7 convolution and the max-pool (Section 2.3, Fig. 6; the figure is not in the
   paper's text, so this is a READING, after the stem block of PeleeNet that the paper cites: PARITY UNPINNED BY THE PAPER):
     s1  = relu(BN(conv3x3/2, pad 1, 3 -> 32))(image)            224 -> 112
     a   = relu(BN(conv1x1, 32 -> 16))(s1)
     a   = relu(BN(conv3x3/2, pad 1, 16 -> 32))(a)               112 -> 56
     b   = maxpool2x2/2(s1)                                      112 -> 56
     out = BN(conv1x1, 64 -> 64)(concat(a, b))                   no activation: the binary blocks take its sign
   out is fp32 NCHW [N][64][56][56]. */
static void stem_module(const oracle_bireal18_params* p, const float* images, int N, float* out) {
  float scale[64], shift[64];
  float* s1 = (float*)malloc((size_t)N * 32 * 112 * 112 * sizeof(float));
  float* a1 = (float*)malloc((size_t)N * 16 * 112 * 112 * sizeof(float));
  float* cat = (float*)malloc((size_t)N * 64 * 56 * 56 * sizeof(float));
  float* a2 = (float*)malloc((size_t)N * 32 * 56 * 56 * sizeof(float));
  oracle_bn_fold(p->sm_bn[0][0], p->sm_bn[0][1], p->sm_bn[0][2], p->sm_bn[0][3], p->bn_eps, 32, scale, shift);
  conv_bn_fp32(images, N, 3, 224, 224, p->sm_w[0], 32, 3, 2, 1, scale, shift, 1, s1);
  oracle_bn_fold(p->sm_bn[1][0], p->sm_bn[1][1], p->sm_bn[1][2], p->sm_bn[1][3], p->bn_eps, 16, scale, shift);
  conv_bn_fp32(s1, N, 32, 112, 112, p->sm_w[1], 16, 1, 1, 0, scale, shift, 1, a1);
  oracle_bn_fold(p->sm_bn[2][0], p->sm_bn[2][1], p->sm_bn[2][2], p->sm_bn[2][3], p->bn_eps, 32, scale, shift);
  conv_bn_fp32(a1, N, 16, 112, 112, p->sm_w[2], 32, 3, 2, 1, scale, shift, 1, a2);
  for (int n = 0; n < N; n++) {
    /* channels 0..31: the convolution branch; 32..63: the pooled branch */
    memcpy(cat + (size_t)n * 64 * 56 * 56, a2 + (size_t)n * 32 * 56 * 56, (size_t)32 * 56 * 56 * sizeof(float));
    for (int c = 0; c < 32; c++)
      for (int oh = 0; oh < 56; oh++)
        for (int ow = 0; ow < 56; ow++) {
          const float* q = s1 + (((size_t)n * 32 + c) * 112 + 2 * oh) * 112 + 2 * ow;
          float m = q[0];
          if (q[1] > m) m = q[1];
          if (q[112] > m) m = q[112];
          if (q[113] > m) m = q[113];
          cat[(((size_t)n * 64 + 32 + c) * 56 + oh) * 56 + ow] = m;
        }
  }
  oracle_bn_fold(p->sm_bn[3][0], p->sm_bn[3][1], p->sm_bn[3][2], p->sm_bn[3][3], p->bn_eps, 64, scale, shift);
  conv_bn_fp32(cat, N, 64, 56, 56, p->sm_w[3], 64, 1, 1, 0, scale, shift, 0, out);
  free(s1); free(a1); free(cat); free(a2);
}

static const int kStageC[4] = {64, 128, 256, 512};
static const int kStageHW[4] = {56, 28, 14, 7};

/* taps (optional, may be NULL): taps[0] = output of stem+maxpool, taps[1+b] = output of
   block b; each fp32 NCHW, caller-allocated, N*C*H*W floats. */
void oracle_bireal18_forward(const oracle_bireal18_params* p, const float* images, int N,
                             float* logits, float* const* taps) {
  const int IH = 224, IW = 224, SH = 112, SW = 112;
  float* scale = (float*)malloc(512 * sizeof(float));
  float* shift = (float*)malloc(512 * sizeof(float));
  float* stem = (float*)malloc((size_t)N * 64 * SH * SW * sizeof(float));
  size_t act_elems = (size_t)N * 64 * 56 * 56; /* the largest activation after the stem */
  float* cur = (float*)malloc(act_elems * sizeof(float));
  float* nxt = (float*)malloc(act_elems * sizeof(float));
  float* sc = (float*)malloc(act_elems * sizeof(float));
  float* pooled = (float*)malloc(act_elems * sizeof(float));
  int32_t* acc = (int32_t*)malloc(act_elems * sizeof(int32_t));
  uint64_t* pa = (uint64_t*)malloc((size_t)N * 56 * 56 * 8 * sizeof(uint64_t));
  uint64_t* pw = (uint64_t*)malloc((size_t)512 * 9 * 8 * sizeof(uint64_t));

  if (p->use_stem_module) {
    stem_module(p, images, N, cur);
    goto blocks;
  }
  /* 1. stem: conv 7x7, 3 -> 64, stride 2, zero pad 3, no bias; then BN */
  oracle_bn_fold(p->stem_bn[0], p->stem_bn[1], p->stem_bn[2], p->stem_bn[3], p->bn_eps, 64, scale, shift);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int o = 0; o < 64; o++)
      for (int oh = 0; oh < SH; oh++)
        for (int ow = 0; ow < SW; ow++) {
          float a = 0.0f;
          for (int c = 0; c < 3; c++)
            for (int i = 0; i < 7; i++)
              for (int j = 0; j < 7; j++) {
                int ih = oh * 2 + i - 3, iw = ow * 2 + j - 3;
                if (ih < 0 || ih >= IH || iw < 0 || iw >= IW) continue;
                a = fmaf(images[(((size_t)n * 3 + c) * IH + ih) * IW + iw],
                         p->stem_w[((o * 3 + c) * 7 + i) * 7 + j], a);
              }
          stem[(((size_t)n * 64 + o) * SH + oh) * SW + ow] = fmaf(a, scale[o], shift[o]);
        }
  /*    maxpool 3x3, stride 2, pad 1 (taps outside the image are ignored) */
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++)
    for (int c = 0; c < 64; c++)
      for (int oh = 0; oh < 56; oh++)
        for (int ow = 0; ow < 56; ow++) {
          float m = -INFINITY;
          for (int i = 0; i < 3; i++)
            for (int j = 0; j < 3; j++) {
              int ih = oh * 2 + i - 1, iw = ow * 2 + j - 1;
              if (ih < 0 || ih >= SH || iw < 0 || iw >= SW) continue;
              float v = stem[(((size_t)n * 64 + c) * SH + ih) * SW + iw];
              if (v > m) m = v;
            }
          cur[(((size_t)n * 64 + c) * 56 + oh) * 56 + ow] = m;
        }
blocks:
  if (taps && taps[0]) memcpy(taps[0], cur, (size_t)N * 64 * 56 * 56 * sizeof(float));

  /* 2. sixteen blocks: out = BN(bconv3x3(sign(x))) + shortcut(x) */
  int C = 64, HW = 56;
  for (int b = 0; b < 16; b++) {
    int stage = b / 4;
    int O = kStageC[stage], OHW = kStageHW[stage];
    int down = (stage > 0 && b % 4 == 0);
    int stride = down ? 2 : 1;
    /* binary conv, pad 1 with value -1 */
    if (p->conv_form == 0) {
      oracle_bconv_pm1(cur, N, C, HW, HW, p->block_w[b], O, 3, 3, stride, stride, 1, 1, -1, acc, LAYOUT_NCHW);
    } else {
      oracle_pack(cur, LAYOUT_NCHW, N, C, HW, HW, pa);
      oracle_pack_weights(p->block_w[b], O, C, 3, 3, pw);
      oracle_bconv_bits(pa, N, C, HW, HW, pw, O, 3, 3, stride, stride, 1, 1, -1, acc, LAYOUT_NCHW);
    }
    /* shortcut */
    const float* shortcut = cur;
    if (down) {
      int d = stage - 1;
      /* avgpool 2x2 stride 2 */
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
      for (int n = 0; n < N; n++)
        for (int c = 0; c < C; c++)
          for (int oh = 0; oh < OHW; oh++)
            for (int ow = 0; ow < OHW; ow++) {
              const float* q = cur + (((size_t)n * C + c) * HW + 2 * oh) * HW + 2 * ow;
              float s = q[0] + q[1];
              s = s + q[HW];
              s = s + q[HW + 1];
              pooled[(((size_t)n * C + c) * OHW + oh) * OHW + ow] = s * 0.25f;
            }
      /* fp32 conv 1x1, C -> O, then BN */
      oracle_bn_fold(p->down_bn[d][0], p->down_bn[d][1], p->down_bn[d][2], p->down_bn[d][3], p->bn_eps, O, scale, shift);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
      for (int n = 0; n < N; n++)
        for (int o = 0; o < O; o++)
          for (int oh = 0; oh < OHW; oh++)
            for (int ow = 0; ow < OHW; ow++) {
              float a = 0.0f;
              for (int c = 0; c < C; c++)
                a = fmaf(pooled[(((size_t)n * C + c) * OHW + oh) * OHW + ow], p->down_w[d][(size_t)o * C + c], a);
              sc[(((size_t)n * O + o) * OHW + oh) * OHW + ow] = fmaf(a, scale[o], shift[o]);
            }
      shortcut = sc;
    }
    /* BN on the integer result, then one rounded add of the shortcut */
    oracle_bn_fold(p->block_bn[b][0], p->block_bn[b][1], p->block_bn[b][2], p->block_bn[b][3], p->bn_eps, O, scale, shift);
#pragma omp parallel for collapse(2) num_threads(g_threads) schedule(static)
    for (int n = 0; n < N; n++)
      for (int o = 0; o < O; o++)
        for (int q = 0; q < OHW * OHW; q++) {
          size_t idx = ((size_t)n * O + o) * OHW * OHW + q;
          float y = fmaf((float)acc[idx], scale[o], shift[o]);
          nxt[idx] = y + shortcut[idx];
        }
    float* t = cur; cur = nxt; nxt = t;
    C = O; HW = OHW;
    if (taps && taps[1 + b]) memcpy(taps[1 + b], cur, (size_t)N * C * HW * HW * sizeof(float));
  }

  /* 3. head: global average over 7x7, fc 512 -> 1000 */
#pragma omp parallel for num_threads(g_threads) schedule(static)
  for (int n = 0; n < N; n++) {
    float g[512];
    for (int c = 0; c < 512; c++) {
      float s = 0.0f;
      for (int h = 0; h < 7; h++)
        for (int w = 0; w < 7; w++) s = s + cur[(((size_t)n * 512 + c) * 7 + h) * 7 + w];
      g[c] = s / 49.0f;
    }
    for (int j = 0; j < 1000; j++) {
      float a = 0.0f;
      for (int k = 0; k < 512; k++) a = fmaf(g[k], p->fc_w[(size_t)j * 512 + k], a);
      logits[(size_t)n * 1000 + j] = a + p->fc_b[j];
    }
  }
  free(scale); free(shift); free(stem); free(cur); free(nxt); free(sc); free(pooled); free(acc);
  free(pa); free(pw);
}
