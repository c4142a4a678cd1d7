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

// Direct fp32 convolution, zero padding, then y = fmaf(acc, scale, shift) and an optional ReLU, as a register-tiled product
// with a fixed summation order.  A CTA of 256 threads owns 128 consecutive output pixels x BN output channels; K = CIN * k * k
// is walked in chunks of CG channels x all taps (k index = c * taps + tap ascending: the pinned order).  Per chunk the
// im2col values of the CTA's pixels go to shared memory k-major ([k][pixel]: a thread later reads its 4 pixels as one
// 128-bit load) and the filters as [k][channel] (broadcast reads); thread (tx, ty) keeps 4 pixels x TN = BN / 8 channels.
// The loader thread of pixel p fetches CG consecutive channels of a tap with one vector load (NHWC input) or walks the
// channels (NCHW input, lanes along the image row).  Taps outside the image are zeros: fmaf(0, w, acc) = acc.
// x: NCHW (IN_NCHW) or NHWC with CIN channels per pixel; y: NHWC with y_stride channels per pixel, written at channel y_off.
template <int K, int S, int PAD, int CIN, int BN, int CG, bool IN_NCHW, bool RELU>
__global__ void __launch_bounds__(256) conv_fp32_pinned(const float* __restrict__ x, int N, int H, int W, int OH, int OW,
                                                        const float* __restrict__ w_oihw, const float* __restrict__ scale,
                                                        const float* __restrict__ shift, float* __restrict__ y,
                                                        int y_stride, int y_off) {
  constexpr int BM = 128, T = K * K, KC = CG * T, TN = BN / 8, AP = BM + 4, WP = BN + 4;
  static_assert(CIN % CG == 0 && BN % 16 == 0 && (IN_NCHW || (K == 1 ? CG % 8 == 0 : CG == 4)), "tile");
  __shared__ __align__(16) float a_s[KC * AP];
  __shared__ __align__(16) float w_s[KC * WP];
  const int tid = threadIdx.x;
  const long long npix = (long long)N * OH * OW;
  const long long p0 = (long long)blockIdx.x * BM;
  const int o0 = blockIdx.y * BN;
  // loader role: pixel lp, and one half of the chunk's taps (or channels, for a single tap)
  const int lp = tid & (BM - 1), lhalf = tid >> 7;
  const long long pl = p0 + lp;
  int ih0 = 0, iw0 = 0;
  long long xn = -1;  // offset of image n in x, or -1 for a pixel beyond the end
  if (pl < npix) {
    const int ow = (int)(pl % OW), oh = (int)((pl / OW) % OH);
    const long long n = pl / ((long long)OW * OH);
    ih0 = oh * S - PAD;
    iw0 = ow * S - PAD;
    xn = n * (long long)CIN * H * W;
  }
  const int tx = tid & 31, ty = tid >> 5;
  float acc[4][TN];
#pragma unroll
  for (int i = 0; i < 4; i++)
#pragma unroll
    for (int j = 0; j < TN; j++) acc[i][j] = 0.0f;

  for (int c0 = 0; c0 < CIN; c0 += CG) {
    // filters of this chunk: w_s[k][o] = w[o0 + o][c0 * T + k]
    for (int idx = tid; idx < KC * BN; idx += 256) {
      const int o = idx / KC, k = idx - o * KC;  // consecutive threads: consecutive k of one filter (contiguous in OIHW)
      w_s[k * WP + o] = w_oihw[(size_t)(o0 + o) * (CIN * T) + c0 * T + k];
    }
    // im2col values of this chunk
    if (IN_NCHW) {
#pragma unroll
      for (int k = 0; k < KC; k++) {
        if ((k & 1) != lhalf) continue;
        const int cc = k / T, t = k % T, ih = ih0 + t / K, iw = iw0 + t % K;
        float v = 0.0f;
        if (xn >= 0 && ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(x + xn + ((long long)(c0 + cc) * H + ih) * W + iw);
        a_s[k * AP + lp] = v;
      }
    } else if (T == 1) {
      // one tap: the two loader threads of a pixel take half of the chunk's channels each
#pragma unroll
      for (int q = 0; q < CG / 8; q++) {
        const int cc = lhalf * (CG / 2) + 4 * q;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (xn >= 0) v = __ldg(reinterpret_cast<const float4*>(x + xn + ((long long)ih0 * W + iw0) * CIN + c0 + cc));
        a_s[(cc + 0) * AP + lp] = v.x; a_s[(cc + 1) * AP + lp] = v.y; a_s[(cc + 2) * AP + lp] = v.z; a_s[(cc + 3) * AP + lp] = v.w;
      }
    } else {
#pragma unroll
      for (int t = 0; t < T; t++) {
        if ((t & 1) != lhalf) continue;
        const int ih = ih0 + t / K, iw = iw0 + t % K;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (xn >= 0 && ih >= 0 && ih < H && iw >= 0 && iw < W) v = __ldg(reinterpret_cast<const float4*>(x + xn + ((long long)ih * W + iw) * CIN + c0));
        a_s[(0 * T + t) * AP + lp] = v.x; a_s[(1 * T + t) * AP + lp] = v.y; a_s[(2 * T + t) * AP + lp] = v.z; a_s[(3 * T + t) * AP + lp] = v.w;
      }
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < KC; k++) {
      const float4 a = *reinterpret_cast<const float4*>(a_s + k * AP + 4 * tx);
      float wv[TN];
#pragma unroll
      for (int j = 0; j < TN; j += 2) {
        const float2 w2 = *reinterpret_cast<const float2*>(w_s + k * WP + ty * TN + j);
        wv[j] = w2.x; wv[j + 1] = w2.y;
      }
#pragma unroll
      for (int j = 0; j < TN; j++) {
        acc[0][j] = __fmaf_rn(a.x, wv[j], acc[0][j]);
        acc[1][j] = __fmaf_rn(a.y, wv[j], acc[1][j]);
        acc[2][j] = __fmaf_rn(a.z, wv[j], acc[2][j]);
        acc[3][j] = __fmaf_rn(a.w, wv[j], acc[3][j]);
      }
    }
    __syncthreads();
  }
  const int o = o0 + ty * TN;
  float sc[TN], sf[TN];
#pragma unroll
  for (int j = 0; j < TN; j++) { sc[j] = __ldg(scale + o + j); sf[j] = __ldg(shift + o + j); }
#pragma unroll
  for (int i = 0; i < 4; i++) {
    const long long pp = p0 + 4 * tx + i;
    if (pp >= npix) continue;
    float* dst = y + pp * y_stride + y_off + o;
#pragma unroll
    for (int j = 0; j < TN; j += 2) {
      float r0 = __fmaf_rn(acc[i][j], sc[j], sf[j]), r1 = __fmaf_rn(acc[i][j + 1], sc[j + 1], sf[j + 1]);
      if (RELU) { r0 = (r0 > 0.0f) ? r0 : 0.0f; r1 = (r1 > 0.0f) ? r1 : 0.0f; }
      *reinterpret_cast<float2*>(dst + j) = make_float2(r0, r1);
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
  const long long p112 = (long long)N * 112 * 112, p56 = (long long)N * 56 * 56;  // output pixels
  conv_fp32_pinned<3, 2, 1, 3, 32, 3, true, true><<<dim3(ceil_div(p112, 128), 1), 256, 0, st>>>(
      images, N, 224, 224, 112, 112, sm->w[0], sm->scale[0], sm->shift[0], s1, 32, 0);
  conv_fp32_pinned<1, 1, 0, 32, 16, 16, false, true><<<dim3(ceil_div(p112, 128), 1), 256, 0, st>>>(
      s1, N, 112, 112, 112, 112, sm->w[1], sm->scale[1], sm->shift[1], a1, 16, 0);
  conv_fp32_pinned<3, 2, 1, 16, 32, 4, false, true><<<dim3(ceil_div(p56, 128), 1), 256, 0, st>>>(
      a1, N, 112, 112, 56, 56, sm->w[2], sm->scale[2], sm->shift[2], cat, 64, 0);
  const long long npix = (long long)N * 56 * 56;
  stem_pool_concat<<<ceil_div(npix * 8, 256), 256, 0, st>>>(s1, npix, cat);
  conv_fp32_pinned<1, 1, 0, 64, 64, 16, false, false><<<dim3(ceil_div(p56, 128), 1), 256, 0, st>>>(
      cat, N, 56, 56, 56, 56, sm->w[3], sm->scale[3], sm->shift[3], out, 64, 0);
  dabnn_status s = launch_status();
  if (s != DABNN_OK) return s;
  const dabnn_shape sh = {N, 64, 56, 56};
  return dabnn_pack(out, DABNN_NHWC, sh, bits, st);
}

}  // namespace dabnn
