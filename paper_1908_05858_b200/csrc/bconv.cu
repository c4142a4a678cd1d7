// Binary convolution on packed words (Section 2.1.2, Eq. 1 of the paper) with fused epilogues
// (Section 2.1.1, last sentence): out = K - 2 * sum popcount(a xor w).
//
// Formulation.  The paper reads the convolution as BGEMM with A = weights (M = C_out rows) and
// B = the im2col'ed input (N = OH*OW columns), and sums the per-lane bit counts in a vector
// accumulator, reducing once at the end (Eq. 6-7).  Here a CTA owns a tile of BP output pixels
// x BO output channels; the im2col rows of its pixels and the weight rows of its channels are
// gathered chunk by chunk into shared memory with cp.async (a 3-stage ring), padded positions are
// written as the declared pad word, and every thread keeps a TP x TO register tile of partial bit
// counts that is turned into K - 2*count once, in the epilogue.
//
// Pipes (measured on B200): POPC issues on the XU pipe at 16 lanes/clk/SM, LOP3 and IADD on the ALU
// pipe at 64 lanes/clk/SM.  The plain loop (xor, popc, add per 32-bit word pair) is therefore
// POPC-bound.  The carry-save loop feeds the two halves of a 64-bit word pair through a full adder
// with a running "ones" word per output -- three 3-input logic ops with the xors folded in, see
// bit_mac -- and popcounts only the carry word: half the POPCs, so the bound doubles to 32 word
// pairs/clk/SM (XU full, ALU at 3/4), and the accumulation is an IMAD on the FMA pipe.
// Both give sum popcount(a xor w) exactly.
#include <stdlib.h>

#include "common.cuh"
#include "bconv_tile.cuh"

namespace dabnn {

namespace {

// ---- host side -----------------------------------------------------------------------------------

int g_conv_variant = 0;
int g_conv_tile = 0;

template <int BP, int BO, int TP, int TO, int MINB, int EPI, bool CSA, bool VEC16, int STAGES>
dabnn_status launch_one(const BConvArgs& g, cudaStream_t st) {
  constexpr int THREADS = (BP / TP) * (BO / TO);
  constexpr size_t SMEM = (size_t)STAGES * (BP + BO) * PITCH * 4 + (size_t)BP * sizeof(RowInfo);
  auto kern = bconv_kernel<BP, BO, TP, TO, MINB, EPI, CSA, VEC16, STAGES>;
  static bool configured[kMaxDevices] = {};  // one attribute call per instantiation and device (idempotent if raced)
  const int dev = current_device();
  if (dev < 0) return DABNN_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    configured[dev] = true;
  }
  const long long gx = (g.M + BP - 1) / BP;
  const int ochan = (EPI == EPI_I32) ? g.O : g.Ow32 * 32;
  const int gy = (ochan + BO - 1) / BO;
  if (gx > 0x7FFFFFFF || gy > 65535) return DABNN_ERR_UNSUPPORTED;
  launch_chain(kern, dim3((unsigned)gx, (unsigned)gy), dim3(THREADS), (size_t)SMEM, st, g);
  return launch_status();
}

// The several-tiles-per-CTA form for short-K pointwise layers (bconv_pointwise_tiles), 128 x 64 tiles.
template <int EPI, bool VEC16>
dabnn_status launch_pointwise(const BConvArgs& g, cudaStream_t st) {
  constexpr int BP = 128, BO = 64, TP = 8, TO = 4, NSUB = 4, THREADS = (BP / TP) * (BO / TO);
  constexpr size_t SMEM = (size_t)(BO + 3 * BP) * PITCH * 4 + (size_t)BP * (BO / 32) * 4;
  auto kern = bconv_pointwise_kernel<BP, BO, TP, TO, 2, EPI, VEC16, NSUB>;
  static bool configured[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return DABNN_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    configured[dev] = true;
  }
  const int ochan = (EPI == EPI_I32) ? g.O : g.Ow32 * 32;
  const long long gx = ((g.M + BP - 1) / BP + NSUB - 1) / NSUB;
  const int gy = (ochan + BO - 1) / BO;
  if (gx > 0x7FFFFFFF || gy > 65535) return DABNN_ERR_UNSUPPORTED;
  kern<<<dim3((unsigned)gx, (unsigned)gy), THREADS, SMEM, st>>>(g);
  return launch_status();
}

template <int BP, int BO, int TP, int TO, int MINB, int EPI, int STAGES = STAGES_DEFAULT>
dabnn_status launch_tile(const BConvArgs& g, bool csa, cudaStream_t st) {
  const bool vec16 = (g.Cw % 2 == 0) && aligned(g.a, 16) && aligned(g.w, 16);
  if (csa)
    return vec16 ? launch_one<BP, BO, TP, TO, MINB, EPI, true, true, STAGES>(g, st)
                 : launch_one<BP, BO, TP, TO, MINB, EPI, true, false, STAGES>(g, st);
  return vec16 ? launch_one<BP, BO, TP, TO, MINB, EPI, false, true, STAGES>(g, st)
               : launch_one<BP, BO, TP, TO, MINB, EPI, false, false, STAGES>(g, st);
}

template <int EPI>
dabnn_status launch_epi(const BConvArgs& g, cudaStream_t st) {
  const bool csa = g_conv_variant != 1;
  const int sms = sm_count();
  const int ochan = (EPI == EPI_I32) ? g.O : g.Ow32 * 32;
  auto ctas = [&](int bp, int bo) { return ((g.M + bp - 1) / bp) * ((ochan + bo - 1) / bo); };
  int tile = g_conv_tile;
  if (tile == 0) {
    // Measured on B200 (batch 64 to 256, the ResNet-18 stage shapes and the 1x1 512 -> 2048 layer): 32 outputs per thread
    // (128 x 64, two CTAs = 16 warps per SM) where that still gives four waves of CTAs, else 16 outputs per thread (64 x 64);
    // the 8 x 8 register tile of 128 x 128 spills at 255 registers, leaves two warps per scheduler and is slower everywhere.
    if (ctas(128, 64) >= 4LL * sms) tile = 2;
    else if (ctas(64, 64) >= 4LL * sms) tile = 3;
    else if (ctas(32, 32) >= sms || g.K64 > 5 * KC64) tile = 4;
    else tile = 5;  // less than one wave of the smallest tile: latency is all that counts
  }
  if constexpr (EPI != EPI_BIREAL) {
    // short-K pointwise layers with at least four waves of four-tile CTAs (DABNN_CONV_POINTWISE=0 in the environment, read
    // once, keeps the one-tile form, for measurements)
    static const bool pw_off = [] { const char* e = getenv("DABNN_CONV_POINTWISE"); return e && atoi(e) == 0; }();
    if (g.pointwise && csa && !pw_off && !g_chain_launch && g.K64 <= KC64 && (g_conv_tile == 0 || g_conv_tile == 2) &&
        ctas(128, 64) >= 16LL * sms)
      return ((g.Cw % 2 == 0) && aligned(g.a, 16) && aligned(g.w, 16)) ? launch_pointwise<EPI, true>(g, st) : launch_pointwise<EPI, false>(g, st);
  }
  switch (tile) {
    case 1: return launch_tile<128, 128, 8, 8, 1, EPI>(g, csa, st);
    case 2: return launch_tile<128, 64, 8, 4, 2, EPI>(g, csa, st);
    case 3: return launch_tile<64, 64, 4, 4, 2, EPI>(g, csa, st);
    case 4: return launch_tile<32, 32, 2, 4, 4, EPI>(g, csa, st);
    // 16 x 32 outputs per CTA and a ring of 6 stages: every chunk of K up to 80 words (a 3x3 filter over 512 channels is
    // 72) is requested before the first one is used, so the CTA waits for memory once
    default: return launch_tile<16, 32, 1, 4, 4, EPI, 6>(g, csa, st);
  }
}

dabnn_status fill_args(BConvArgs& g, const uint64_t* a, dabnn_shape in, const uint64_t* w, int O, dabnn_conv cv,
                       dabnn_packed_layout pl = DABNN_PACKED_NHWC) {
  if (pl != DABNN_PACKED_NHWC && pl != DABNN_PACKED_NC1HWC2) return DABNN_ERR_SHAPE;
  if (!a || !w) return DABNN_ERR_NULL;
  if (in.N <= 0 || in.C <= 0 || in.H <= 0 || in.W <= 0 || O <= 0) return DABNN_ERR_SHAPE;
  if (cv.kh <= 0 || cv.kw <= 0 || cv.stride_h <= 0 || cv.stride_w <= 0 || cv.pad_h < 0 || cv.pad_w < 0)
    return DABNN_ERR_SHAPE;
  if (cv.pad_value != 1 && cv.pad_value != -1) return DABNN_ERR_SHAPE;
  if (!aligned(a, 8) || !aligned(w, 8)) return DABNN_ERR_ALIGNMENT;
  const int OH = dabnn_out_dim(in.H, cv.kh, cv.stride_h, cv.pad_h);
  const int OW = dabnn_out_dim(in.W, cv.kw, cv.stride_w, cv.pad_w);
  if (OH <= 0 || OW <= 0) return DABNN_ERR_SHAPE;
  const long long Kbits = (long long)in.C * cv.kh * cv.kw;
  const long long Cw = (in.C + 63) / 64;
  if (Kbits >= (1LL << 24) || Cw * cv.kh * cv.kw > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
  const long long M = (long long)in.N * OH * OW;
  if (M * O > (1LL << 40) || (long long)in.H * in.W * Cw > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
  g.a = a; g.w = w;
  g.N = in.N; g.H = in.H; g.W = in.W; g.Cw = (int)Cw; g.C = in.C;
  g.O = O; g.kh = cv.kh; g.kw = cv.kw; g.sh = cv.stride_h; g.sw = cv.stride_w; g.ph = cv.pad_h; g.pw = cv.pad_w;
  g.OH = OH; g.OW = OW; g.M = M; g.K64 = (int)(Cw * cv.kh * cv.kw); g.Kbits = (int)Kbits;
  g.pad_neg = cv.pad_value < 0;
  g.tail_mask = (in.C % 64 == 0) ? ~0ull : ((1ull << (in.C % 64)) - 1);
  g.out = nullptr; g.out_nchw = 0; g.scale = g.shift = g.residual = nullptr; g.y_out = nullptr;
  g.out_packed32 = nullptr; g.Ow32 = 2 * ((O + 63) / 64); g.one = 1;
  if (pl == DABNN_PACKED_NC1HWC2) {
    const long long C1 = (in.C + 127) / 128;
    if ((long long)in.H * in.W * C1 * 2 > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
    g.img_stride = C1 * in.H * in.W * 2; g.pix_stride = 2; g.pair_stride = 2 * in.H * in.W;
    if (!aligned(a, 16)) return DABNN_ERR_ALIGNMENT;  // 128-bit vectors
  } else {
    g.img_stride = (long long)in.H * in.W * Cw; g.pix_stride = (int)Cw; g.pair_stride = 2;
  }
  g.magic_ow = OW == 1 ? 0ull : ~0ull / (unsigned long long)OW + 1ull;
  g.magic_oh = OH == 1 ? 0ull : ~0ull / (unsigned long long)OH + 1ull;
  g.pointwise = (pl == DABNN_PACKED_NHWC && cv.kh == 1 && cv.kw == 1 && cv.stride_h == 1 && cv.stride_w == 1 && cv.pad_h == 0 &&
                 cv.pad_w == 0) ? 1 : 0;
  g.magic_cw = Cw == 1 ? 0ull : ~0ull / (unsigned long long)Cw + 1ull;
  g.magic_kw = cv.kw == 1 ? 0ull : ~0ull / (unsigned long long)cv.kw + 1ull;
  return DABNN_OK;
}

}  // namespace

int sm_count() {
  static int cached[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return 148;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      return 148;
    }
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace dabnn

using namespace dabnn;

extern "C" int dabnn_set_conv_variant(int variant) {
  const int prev = g_conv_variant;
  if (variant >= 0 && variant <= 2) g_conv_variant = variant;
  return prev;
}

extern "C" int dabnn_set_conv_tile(int tile) {
  const int prev = g_conv_tile;
  if (tile >= 0 && tile <= 5) g_conv_tile = tile;
  return prev;
}

extern "C" size_t dabnn_words_per_pixel(int C) { return C <= 0 ? 0 : (size_t)((C + 63) / 64); }

extern "C" int dabnn_out_dim(int in, int k, int stride, int pad) {
  if (stride <= 0) return 0;
  const int span = in + 2 * pad - k;
  if (span < 0) return 0;
  return span / stride + 1;
}

extern "C" const char* dabnn_status_string(dabnn_status s) {
  switch (s) {
    case DABNN_OK: return "ok";
    case DABNN_ERR_NULL: return "null pointer";
    case DABNN_ERR_SHAPE: return "invalid shape or convolution parameters";
    case DABNN_ERR_UNSUPPORTED: return "size beyond the supported index range";
    case DABNN_ERR_ALIGNMENT: return "misaligned pointer";
    case DABNN_ERR_WORKSPACE: return "workspace too small";
    case DABNN_ERR_CUDA: return "CUDA launch error";
    case DABNN_ERR_TIMEOUT: return "a bounded wait inside a kernel ran out; the outputs of the launches since the flag was last read are undefined";
    case DABNN_ERR_STATIC_LIMIT: return "request exceeds the library's built-in scratch area (see DABNN_STATIC_MAX_BATCH)";
  }
  return "unknown status";
}

extern "C" dabnn_status dabnn_bconv2d(const uint64_t* a_packed, dabnn_shape in, const uint64_t* w_packed, int O,
                                      dabnn_conv cv, int32_t* out, dabnn_layout out_layout, void* stream) {
  BConvArgs g;
  dabnn_status s = fill_args(g, a_packed, in, w_packed, O, cv);
  if (s != DABNN_OK) return s;
  if (!out) return DABNN_ERR_NULL;
  if (out_layout != DABNN_NCHW && out_layout != DABNN_NHWC) return DABNN_ERR_SHAPE;
  if (!aligned(out, 4)) return DABNN_ERR_ALIGNMENT;
  g.out = out;
  g.out_nchw = out_layout == DABNN_NCHW;
  return launch_epi<EPI_I32>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_bconv2d_from(const uint64_t* a_packed, dabnn_packed_layout a_layout, dabnn_shape in,
                                           const uint64_t* w_packed, int O, dabnn_conv cv, int32_t* out,
                                           dabnn_layout out_layout, void* stream) {
  BConvArgs g;
  dabnn_status s = fill_args(g, a_packed, in, w_packed, O, cv, a_layout);
  if (s != DABNN_OK) return s;
  if (!out) return DABNN_ERR_NULL;
  if (out_layout != DABNN_NCHW && out_layout != DABNN_NHWC) return DABNN_ERR_SHAPE;
  if (!aligned(out, 4)) return DABNN_ERR_ALIGNMENT;
  g.out = out;
  g.out_nchw = out_layout == DABNN_NCHW;
  return launch_epi<EPI_I32>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_bconv2d_bn_sign_pack(const uint64_t* a_packed, dabnn_shape in, const uint64_t* w_packed,
                                                   int O, dabnn_conv cv, const float* scale, const float* shift,
                                                   uint64_t* out_packed, void* stream) {
  BConvArgs g;
  dabnn_status s = fill_args(g, a_packed, in, w_packed, O, cv);
  if (s != DABNN_OK) return s;
  if (!scale || !shift || !out_packed) return DABNN_ERR_NULL;
  if (!aligned(scale, 4) || !aligned(shift, 4) || !aligned(out_packed, 8)) return DABNN_ERR_ALIGNMENT;
  g.scale = scale; g.shift = shift;
  g.out_packed32 = reinterpret_cast<uint32_t*>(out_packed);
  return launch_epi<EPI_BNPACK>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_bconv2d_bn_add_sign_pack(const uint64_t* a_packed, dabnn_shape in,
                                                       const uint64_t* w_packed, int O, dabnn_conv cv,
                                                       const float* scale, const float* shift, const float* residual,
                                                       float* y_out, uint64_t* out_packed, void* stream) {
  BConvArgs g;
  dabnn_status s = fill_args(g, a_packed, in, w_packed, O, cv);
  if (s != DABNN_OK) return s;
  if (!scale || !shift || !residual || !y_out) return DABNN_ERR_NULL;
  if (!aligned(scale, 4) || !aligned(shift, 4) || !aligned(residual, 4) || !aligned(y_out, 4) ||
      !aligned(out_packed, 8))
    return DABNN_ERR_ALIGNMENT;
  g.scale = scale; g.shift = shift; g.residual = residual; g.y_out = y_out;
  g.out_packed32 = reinterpret_cast<uint32_t*>(out_packed);
  return launch_epi<EPI_BIREAL>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_bgemm(const uint64_t* A, int M, const uint64_t* B, int N, int Kbits, int32_t* C,
                                    void* stream) {
  // rows of A are "pixels" of a 1x1 image batch, rows of B the "filters": a 1x1 convolution over Kbits channels
  if (M <= 0 || N <= 0 || Kbits <= 0) return DABNN_ERR_SHAPE;
  const dabnn_shape in = {M, Kbits, 1, 1};
  const dabnn_conv cv = {1, 1, 1, 1, 0, 0, -1};
  return dabnn_bconv2d(A, in, B, N, cv, C, DABNN_NHWC, stream);
}
