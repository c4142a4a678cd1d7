// The STEM module variant of the Bi-Real Net 18 front end (Section 2.3 of the paper: the 7x7 convolution and the
// max-pool replaced by a STEM module, 30 % faster on the paper's phone).  The module's figure is not part of the
// paper's text; the structure built here follows the stem block of the network the paper cites for it:
//     s1  = relu(BN(conv3x3/2, pad 1, 3 -> 32))(image)        224 -> 112
//     a   = relu(BN(conv1x1, 32 -> 16))(s1)
//     a   = relu(BN(conv3x3/2, pad 1, 16 -> 32))(a)           112 -> 56
//     b   = maxpool2x2/2(s1)                                  112 -> 56
//     out = BN(conv1x1, 64 -> 64)(concat(a, b))               no activation: the binary blocks take its sign
// Every value is produced by single IEEE-rounded fp32 operations in a fixed order (fmaf chains over c, kh, kw ascending),
// like the rest of the network's fp32 parts, so the result does not depend on tiling.
#include "common.cuh"

namespace dabnn {

namespace {

// Direct fp32 convolution, zero padding, then y = fmaf(acc, scale, shift) and an optional ReLU.  A thread owns two
// neighbouring output pixels x CO output channels; the CO filters of the CTA (blockIdx.y) sit in shared memory as
// [c][kh][kw][CO], read as broadcast 128-bit loads.  Taps outside the image multiply a zero: fmaf(0, w, acc) = acc.
// x: NCHW (IN_NCHW) or NHWC with CIN channels per pixel; y: NHWC with y_stride channels per pixel, written at channel y_off.
template <int K, int S, int PAD, int CIN, int CO, bool IN_NCHW, bool RELU>
__global__ void __launch_bounds__(128) conv_fp32_pinned(const float* __restrict__ x, int N, int H, int W, int OH, int OW,
                                                        const float* __restrict__ w_oihw, const float* __restrict__ scale,
                                                        const float* __restrict__ shift, float* __restrict__ y,
                                                        int y_stride, int y_off) {
  __shared__ __align__(16) float ws[CIN * K * K * CO];
  const int o0 = blockIdx.y * CO;
  for (int idx = threadIdx.x; idx < CIN * K * K * CO; idx += 128) {
    const int o = idx % CO, k = idx / CO;
    ws[idx] = w_oihw[(size_t)(o0 + o) * (CIN * K * K) + k];
  }
  __syncthreads();
  const int pairs_per_row = (OW + 1) / 2;
  const long long pp = (long long)blockIdx.x * 128 + threadIdx.x;
  if (pp >= (long long)N * OH * pairs_per_row) return;
  const int pw = (int)(pp % pairs_per_row);
  const int oh = (int)((pp / pairs_per_row) % OH);
  const long long n = pp / ((long long)pairs_per_row * OH);
  const int ow0 = 2 * pw;
  const bool second = ow0 + 1 < OW;

  // per tap: offset of the input value of channel 0 and whether the tap lies inside the image, for both pixels
  long long off[2][K * K];
  bool in[2][K * K];
#pragma unroll
  for (int q = 0; q < 2; q++)
#pragma unroll
    for (int i = 0; i < K; i++)
#pragma unroll
      for (int j = 0; j < K; j++) {
        const int ih = oh * S + i - PAD, iw = (ow0 + q) * S + j - PAD;
        const bool ok = ih >= 0 && ih < H && iw >= 0 && iw < W && (q == 0 || second);
        in[q][i * K + j] = ok;
        off[q][i * K + j] = !ok ? 0 : IN_NCHW ? ((n * CIN) * H + ih) * (long long)W + iw : ((n * H + ih) * W + iw) * (long long)CIN;
      }
  constexpr long long CSTEP_NHWC = 1;
  const long long cstep = IN_NCHW ? (long long)H * W : CSTEP_NHWC;

  float acc[2][CO];
#pragma unroll
  for (int q = 0; q < 2; q++)
#pragma unroll
    for (int o = 0; o < CO; o++) acc[q][o] = 0.0f;
#pragma unroll 2
  for (int c = 0; c < CIN; c++) {
#pragma unroll
    for (int t = 0; t < K * K; t++) {
      const float x0 = in[0][t] ? __ldg(x + off[0][t] + c * cstep) : 0.0f;
      const float x1 = in[1][t] ? __ldg(x + off[1][t] + c * cstep) : 0.0f;
      const float4* wv = reinterpret_cast<const float4*>(ws + (c * K * K + t) * CO);
#pragma unroll
      for (int o4 = 0; o4 < CO / 4; o4++) {
        const float4 w4 = wv[o4];
        acc[0][4 * o4] = __fmaf_rn(x0, w4.x, acc[0][4 * o4]);
        acc[0][4 * o4 + 1] = __fmaf_rn(x0, w4.y, acc[0][4 * o4 + 1]);
        acc[0][4 * o4 + 2] = __fmaf_rn(x0, w4.z, acc[0][4 * o4 + 2]);
        acc[0][4 * o4 + 3] = __fmaf_rn(x0, w4.w, acc[0][4 * o4 + 3]);
        acc[1][4 * o4] = __fmaf_rn(x1, w4.x, acc[1][4 * o4]);
        acc[1][4 * o4 + 1] = __fmaf_rn(x1, w4.y, acc[1][4 * o4 + 1]);
        acc[1][4 * o4 + 2] = __fmaf_rn(x1, w4.z, acc[1][4 * o4 + 2]);
        acc[1][4 * o4 + 3] = __fmaf_rn(x1, w4.w, acc[1][4 * o4 + 3]);
      }
    }
  }
#pragma unroll
  for (int q = 0; q < 2; q++) {
    if (q == 1 && !second) break;
    float* dst = y + ((n * OH + oh) * (long long)OW + ow0 + q) * y_stride + y_off + o0;
#pragma unroll
    for (int o4 = 0; o4 < CO / 4; o4++) {
      float v[4];
#pragma unroll
      for (int e = 0; e < 4; e++) {
        const int o = 4 * o4 + e;
        float r = __fmaf_rn(acc[q][o], __ldg(scale + o0 + o), __ldg(shift + o0 + o));
        if (RELU) r = (r > 0.0f) ? r : 0.0f;
        v[e] = r;
      }
      *reinterpret_cast<float4*>(dst + 4 * o4) = make_float4(v[0], v[1], v[2], v[3]);
    }
  }
}

// maxpool 2x2 / 2 of s1 (NHWC, 32 channels, 112 x 112) into channels 32..63 of the concatenated tensor (NHWC, 64
// channels, 56 x 56).  A thread handles 4 channels of one output pixel.
__global__ void __launch_bounds__(256) stem_pool_concat(const float* __restrict__ s1, long long npix, float* __restrict__ cat) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long pix = t >> 3;
  const int c4 = (int)(t & 7);
  if (pix >= npix) return;
  const int ow = (int)(pix % 56), oh = (int)((pix / 56) % 56);
  const long long n = pix / (56 * 56);
  const float* q = s1 + ((n * 112 + 2 * oh) * 112 + 2 * ow) * 32 + c4 * 4;
  float4 m = *reinterpret_cast<const float4*>(q);
  auto take = [&](const float4 v) {
    m.x = (v.x > m.x) ? v.x : m.x; m.y = (v.y > m.y) ? v.y : m.y; m.z = (v.z > m.z) ? v.z : m.z; m.w = (v.w > m.w) ? v.w : m.w;
  };
  take(*reinterpret_cast<const float4*>(q + 32));
  take(*reinterpret_cast<const float4*>(q + 112 * 32));
  take(*reinterpret_cast<const float4*>(q + 113 * 32));
  *reinterpret_cast<float4*>(cat + pix * 64 + 32 + c4 * 4) = m;
}

}  // namespace

// s1: [N][112][112][32], a1: [N][112][112][16], cat: [N][56][56][64] (scratch); out: [N][56][56][64] fp32, bits: its signs.
dabnn_status launch_stem_module(const dabnn_stem_module_params* sm, const float* images, int N, float* s1, float* a1,
                                float* cat, float* out, uint64_t* bits, cudaStream_t st) {
  for (int i = 0; i < 4; i++)
    if (!sm->w[i] || !sm->scale[i] || !sm->shift[i]) return DABNN_ERR_NULL;
  const long long p112 = (long long)N * 112 * 56, p56 = (long long)N * 56 * 28;  // pixel pairs
  conv_fp32_pinned<3, 2, 1, 3, 16, true, true><<<dim3(ceil_div(p112, 128), 2), 128, 0, st>>>(
      images, N, 224, 224, 112, 112, sm->w[0], sm->scale[0], sm->shift[0], s1, 32, 0);
  conv_fp32_pinned<1, 1, 0, 32, 16, false, true><<<dim3(ceil_div(p112, 128), 1), 128, 0, st>>>(
      s1, N, 112, 112, 112, 112, sm->w[1], sm->scale[1], sm->shift[1], a1, 16, 0);
  conv_fp32_pinned<3, 2, 1, 16, 16, false, true><<<dim3(ceil_div(p56, 128), 2), 128, 0, st>>>(
      a1, N, 112, 112, 56, 56, sm->w[2], sm->scale[2], sm->shift[2], cat, 64, 0);
  const long long npix = (long long)N * 56 * 56;
  stem_pool_concat<<<ceil_div(npix * 8, 256), 256, 0, st>>>(s1, npix, cat);
  conv_fp32_pinned<1, 1, 0, 64, 16, false, false><<<dim3(ceil_div(p56, 128), 4), 128, 0, st>>>(
      cat, N, 56, 56, 56, 56, sm->w[3], sm->scale[3], sm->shift[3], out, 64, 0);
  dabnn_status s = launch_status();
  if (s != DABNN_OK) return s;
  const dabnn_shape sh = {N, 64, 56, 56};
  return dabnn_pack(out, DABNN_NHWC, sh, bits, st);
}

}  // namespace dabnn
