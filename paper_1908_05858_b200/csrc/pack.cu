// Binarize + bit-pack kernels (Section 2.1.1 of the paper): fp32 -> one bit per element, 64 channels
// per word, words of a pixel contiguous (channel-packed NHWC).  Pure HBM streaming: 4 bytes read and
// 1/8 byte written per element.
//
// The paper gathers IEEE sign bits with NEON shift-and-insert instructions spread over several
// registers.  Here the sign test is a compare (so -0.0 and NaN pack as +1), 128-bit loads keep the
// memory system busy, bits are gathered in registers by shift-or, and the words leave through shared
// memory so that global stores are whole, contiguous 16-byte pieces.
#include "common.cuh"

namespace dabnn {

namespace {

constexpr int kPackThreads = 128;

// NCHW, H*W a multiple of 4, 16-byte aligned input.  A CTA covers `pix_per_cta` = 128 * (4 / wc)
// consecutive pixels of one image; wc warps share a 128-pixel group and split its channel words.
// Each lane owns 4 consecutive pixels (one float4 per channel) and walks 64 channels per word.
template <int WC>  // warps per pixel group: 1, 2 or 4
__global__ void __launch_bounds__(kPackThreads) pack_nchw_vec4(const float* __restrict__ x, int C, int HW, int Cw,
                                                               uint64_t* __restrict__ packed) {
  extern __shared__ uint64_t s_words[];  // [pix_per_cta][Cw]
  constexpr int GROUPS = 4 / WC;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int group = warp / WC, wsel = warp % WC;
  const int n = blockIdx.y;
  const int pix0 = blockIdx.x * (128 * GROUPS);
  const int p = pix0 + group * 128 + lane * 4;  // first of this lane's 4 pixels
  const bool live = p < HW;                     // HW % 4 == 0, so all 4 pixels are live together
  const float* xn = x + (size_t)n * C * HW;
  for (int cw = wsel; cw < Cw; cw += WC) {
    uint64_t w0 = 0, w1 = 0, w2 = 0, w3 = 0;
    const int c0 = cw * 64;
    const int cn = min(64, C - c0);
    if (live) {
      const float4* src = reinterpret_cast<const float4*>(xn + (size_t)c0 * HW + p);
      const size_t cstride = (size_t)HW / 4;
      int c = 0;
#pragma unroll 1
      for (; c + 8 <= cn; c += 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; u++) v[u] = __ldcs(src + (size_t)(c + u) * cstride);
        unsigned b0 = 0, b1 = 0, b2 = 0, b3 = 0;  // 8 channels of each of the 4 pixels
#pragma unroll
        for (int u = 0; u < 8; u++) {
          b0 |= (unsigned)(v[u].x < 0.0f) << u;
          b1 |= (unsigned)(v[u].y < 0.0f) << u;
          b2 |= (unsigned)(v[u].z < 0.0f) << u;
          b3 |= (unsigned)(v[u].w < 0.0f) << u;
        }
        w0 |= (uint64_t)b0 << c;
        w1 |= (uint64_t)b1 << c;
        w2 |= (uint64_t)b2 << c;
        w3 |= (uint64_t)b3 << c;
      }
      for (; c < cn; c++) {
        float4 v = __ldcs(src + (size_t)c * cstride);
        w0 |= (uint64_t)(v.x < 0.0f) << c;
        w1 |= (uint64_t)(v.y < 0.0f) << c;
        w2 |= (uint64_t)(v.z < 0.0f) << c;
        w3 |= (uint64_t)(v.w < 0.0f) << c;
      }
    }
    const int lp = group * 128 + lane * 4;
    s_words[(size_t)(lp + 0) * Cw + cw] = w0;
    s_words[(size_t)(lp + 1) * Cw + cw] = w1;
    s_words[(size_t)(lp + 2) * Cw + cw] = w2;
    s_words[(size_t)(lp + 3) * Cw + cw] = w3;
  }
  __syncthreads();
  // contiguous in global memory: pixels pix0 .. pix0+npix-1, all words
  const int npix = min(128 * GROUPS, HW - pix0);
  if (npix <= 0) return;
  uint64_t* dst = packed + ((size_t)n * HW + pix0) * Cw;
  const int total = npix * Cw;
  if ((((size_t)n * HW + pix0) * Cw) % 2 == 0 && (reinterpret_cast<uintptr_t>(packed) & 15) == 0) {
    const int pairs = total / 2;
    const ulonglong2* s2 = reinterpret_cast<const ulonglong2*>(s_words);
    ulonglong2* d2 = reinterpret_cast<ulonglong2*>(dst);
    for (int i = threadIdx.x; i < pairs; i += kPackThreads) d2[i] = s2[i];
    if ((total & 1) && threadIdx.x == 0) dst[total - 1] = s_words[total - 1];
  } else {
    for (int i = threadIdx.x; i < total; i += kPackThreads) dst[i] = s_words[i];
  }
}

// Any layout, any shape: one thread per output word.
__global__ void pack_generic(const float* __restrict__ x, int nhwc, int C, int HW, int Cw, long long total_words,
                             uint64_t* __restrict__ packed) {
  long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total_words) return;
  const int cw = (int)(t % Cw);
  const long long pix = t / Cw;  // n*HW + hw
  const int c0 = cw * 64, cn = min(64, C - c0);
  uint64_t w = 0;
  if (nhwc) {
    const float* src = x + (size_t)pix * C + c0;
    for (int c = 0; c < cn; c++) w |= (uint64_t)(src[c] < 0.0f) << c;
  } else {
    const long long n = pix / HW, hw = pix % HW;
    const float* src = x + ((size_t)n * C + c0) * HW + hw;
    for (int c = 0; c < cn; c++) w |= (uint64_t)(src[(size_t)c * HW] < 0.0f) << c;
  }
  packed[t] = w;
}

// NHWC with C a multiple of 64 and 16-byte aligned input: 16 lanes share one word; each lane tests 4
// channels (one float4), places its nibble, and an OR-reduction over 8-lane groups builds each half.
__global__ void __launch_bounds__(256) pack_nhwc_c64(const float* __restrict__ x, long long total_words,
                                                     uint64_t* __restrict__ packed) {
  const int lane = threadIdx.x & 31;
  const long long warp_global = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const unsigned gmask = 0xFFu << (lane & 24);  // this lane's 8-lane group
  // a warp handles 2 words (128 floats) per step; 4 steps in flight per iteration
  for (long long w0 = warp_global * 8; w0 < total_words; w0 += nwarps * 8) {
    float4 v[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const long long word = w0 + 2 * u + (lane >> 4);
      v[u] = (word < total_words) ? __ldcs(reinterpret_cast<const float4*>(x) + word * 16 + (lane & 15))
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
    }
#pragma unroll
    for (int u = 0; u < 4; u++) {
      unsigned nib = (unsigned)(v[u].x < 0.0f) | ((unsigned)(v[u].y < 0.0f) << 1) |
                     ((unsigned)(v[u].z < 0.0f) << 2) | ((unsigned)(v[u].w < 0.0f) << 3);
      unsigned half = __reduce_or_sync(gmask, nib << (4 * (lane & 7)));  // 32 channels of this 8-lane group
      unsigned other = __shfl_xor_sync(0xFFFFFFFFu, half, 8);            // the other half of the word
      const long long word = w0 + 2 * u + (lane >> 4);
      if ((lane & 15) == 0 && word < total_words) packed[word] = (uint64_t)half | ((uint64_t)other << 32);
    }
  }
}

__global__ void pack_weights_kernel(const float* __restrict__ w, int O, int C, int taps, int Cw,
                                    uint64_t* __restrict__ wp) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const long long total = (long long)O * taps * Cw;
  if (t >= total) return;
  const int cw = (int)(t % Cw);
  const int tap = (int)((t / Cw) % taps);
  const int o = (int)(t / ((long long)Cw * taps));
  const int c0 = cw * 64, cn = min(64, C - c0);
  const float* src = w + ((size_t)o * C + c0) * taps + tap;  // OIHW: channel stride = kh*kw
  uint64_t word = 0;
  for (int c = 0; c < cn; c++) word |= (uint64_t)(src[(size_t)c * taps] < 0.0f) << c;
  wp[t] = word;
}

}  // namespace

}  // namespace dabnn

using namespace dabnn;

extern "C" dabnn_status dabnn_pack(const float* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed,
                                   void* stream) {
  if (!x || !packed) return DABNN_ERR_NULL;
  if (s.N <= 0 || s.C <= 0 || s.H <= 0 || s.W <= 0) return DABNN_ERR_SHAPE;
  if (in_layout != DABNN_NCHW && in_layout != DABNN_NHWC) return DABNN_ERR_SHAPE;
  if (!aligned(x, 4) || !aligned(packed, 8)) return DABNN_ERR_ALIGNMENT;
  const long long HW = (long long)s.H * s.W;
  const long long Cw = (s.C + 63) / 64;
  if (HW > 0x7FFFFFFF || (long long)s.N * HW > 0x7FFFFFFFFFFLL) return DABNN_ERR_UNSUPPORTED;
  const long long total_words = (long long)s.N * HW * Cw;
  cudaStream_t st = as_stream(stream);
  if (in_layout == DABNN_NCHW && HW % 4 == 0 && aligned(x, 16) && ((long long)s.C * HW) % 4 == 0 && s.N <= 65535 &&
      Cw * 512 * 8 <= 48 * 1024) {
    const int wc = Cw >= 4 ? 4 : (Cw >= 2 ? 2 : 1);
    const int pix_per_cta = 128 * (4 / wc);
    dim3 grid(ceil_div(HW, pix_per_cta), s.N);
    const size_t smem = (size_t)pix_per_cta * Cw * 8;
    if (wc == 4) pack_nchw_vec4<4><<<grid, kPackThreads, smem, st>>>(x, s.C, (int)HW, (int)Cw, packed);
    else if (wc == 2) pack_nchw_vec4<2><<<grid, kPackThreads, smem, st>>>(x, s.C, (int)HW, (int)Cw, packed);
    else pack_nchw_vec4<1><<<grid, kPackThreads, smem, st>>>(x, s.C, (int)HW, (int)Cw, packed);
  } else if (in_layout == DABNN_NHWC && s.C % 64 == 0 && aligned(x, 16)) {
    const long long warps_needed = (total_words + 7) / 8;
    long long blocks = (warps_needed + 7) / 8;
    const long long cap = (long long)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    pack_nhwc_c64<<<(unsigned)blocks, 256, 0, st>>>(x, total_words, packed);
  } else {
    const long long blocks = (total_words + 255) / 256;
    if (blocks > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
    pack_generic<<<(unsigned)blocks, 256, 0, st>>>(x, in_layout == DABNN_NHWC, s.C, (int)HW, (int)Cw, total_words,
                                                   packed);
  }
  return launch_status();
}

extern "C" dabnn_status dabnn_pack_weights(const float* w_oihw, int O, int C, int kh, int kw, uint64_t* wpacked,
                                           void* stream) {
  if (!w_oihw || !wpacked) return DABNN_ERR_NULL;
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0) return DABNN_ERR_SHAPE;
  if (!aligned(w_oihw, 4) || !aligned(wpacked, 8)) return DABNN_ERR_ALIGNMENT;
  const long long Cw = (C + 63) / 64;
  const long long total = (long long)O * kh * kw * Cw;
  const long long blocks = (total + 255) / 256;
  if (blocks > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
  pack_weights_kernel<<<(unsigned)blocks, 256, 0, as_stream(stream)>>>(w_oihw, O, C, kh * kw, (int)Cw, wpacked);
  return launch_status();
}
