// Binarize + bit-pack kernels (Section 2.1.1 of the paper): fp32 (or int32) -> one bit per element, 64 channels
// per word, words of a pixel contiguous (channel-packed NHWC).  Pure HBM streaming: 4 bytes read and
// 1/8 byte written per element.
//
// The paper gathers IEEE sign bits with NEON shift-and-insert instructions spread over several
// registers.  Here the sign test is a compare (so -0.0 and NaN pack as +1), 128-bit loads keep the
// memory system busy, bits are gathered in registers by shift-or, and the words leave through shared
// memory so that global stores are whole, contiguous 16-byte pieces.  The int32 form (the paper packs the sign bit
// of 32-bit integers the same way, e.g. a convolution's raw sums) runs the same kernels with an integer compare.
#include "common.cuh"

namespace dabnn {

namespace {

constexpr int kPackThreads = 128;

// Streaming 16-byte load.  Written as volatile asm so that a batch of them is issued back to back, in program
// order, before the first result is consumed (memory-level parallelism is what an HBM-bound kernel lives on).
__device__ __forceinline__ float4 ld_stream_v4(const float4* p) {
  float4 v;
  asm volatile("ld.global.cs.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ int4 ld_stream_v4(const int4* p) {
  int4 v;
  asm volatile("ld.global.cs.v4.s32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
template <typename T> struct Vec4;
template <> struct Vec4<float> { using type = float4; };
template <> struct Vec4<int32_t> { using type = int4; };
// the bit: 1 where the value is negative (a compare: -0.0 and NaN give 0, i.e. +1)
__device__ __forceinline__ unsigned neg(float v) { return (unsigned)(v < 0.0f); }
__device__ __forceinline__ unsigned neg(int32_t v) { return (unsigned)(v < 0); }

// NCHW, H*W a multiple of 4, 16-byte aligned input.  A CTA covers 128 consecutive pixels of the batch (images follow one
// another in the pixel count: a tile may span two or more images, so small images leave no ragged tile per image) and all
// channels.  Each lane owns 4 consecutive pixels of one image (one float4 per channel); the four warps split every word's
// 64 channels into quarters of 16, so a thread has 16 independent 16-byte loads in flight per word, and the 16-bit
// quarters are placed side by side in shared memory, which assembles the 64-bit words without any exchange.
// C2: the words leave in the NC1HWC2 layout instead ([N][C1][H][W][2]: 128-bit vectors of one channel group, pixel after
// pixel; an odd last word gets a zero partner).
template <typename T, bool C2>
__global__ void __launch_bounds__(kPackThreads) pack_nchw_vec4(const T* __restrict__ x, int C, int HW, int Cw, long long npix,
                                                               uint64_t* __restrict__ packed) {
  extern __shared__ __align__(16) uint64_t s_words[];  // [128][Cw]
  uint16_t* s_q = reinterpret_cast<uint16_t*>(s_words);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const long long pix0 = (long long)blockIdx.x * 128;  // in pixels of the whole batch
  const long long p = pix0 + lane * 4;                 // first of this lane's 4 pixels
  const bool live = p < npix;                          // HW % 4 == 0, so all 4 pixels are live together and in one image
  using V4 = typename Vec4<T>::type;
  const long long n = live ? p / HW : 0;
  const int hw = live ? (int)(p - n * HW) : 0;
  const T* xn = x + (size_t)n * C * HW + hw;
  const size_t cstride = (size_t)HW / 4;
  for (int cw = 0; cw < Cw; cw++) {
    const int c0 = cw * 64 + warp * 16;
    unsigned b0 = 0, b1 = 0, b2 = 0, b3 = 0;  // 16 channels of each of the 4 pixels
    if (live && c0 < C) {
      const V4* src = reinterpret_cast<const V4*>(xn + (size_t)c0 * HW);
      if (c0 + 16 <= C) {
        V4 v[16];
#pragma unroll
        for (int u = 0; u < 16; u++) v[u] = ld_stream_v4(src + (size_t)u * cstride);
#pragma unroll
        for (int u = 0; u < 16; u++) {
          b0 |= neg(v[u].x) << u;
          b1 |= neg(v[u].y) << u;
          b2 |= neg(v[u].z) << u;
          b3 |= neg(v[u].w) << u;
        }
      } else {
        for (int u = 0; u < C - c0; u++) {
          const V4 v = __ldcs(src + (size_t)u * cstride);
          b0 |= neg(v.x) << u;
          b1 |= neg(v.y) << u;
          b2 |= neg(v.z) << u;
          b3 |= neg(v.w) << u;
        }
      }
    }
    const int lp = lane * 4;
    s_q[((lp + 0) * Cw + cw) * 4 + warp] = (uint16_t)b0;
    s_q[((lp + 1) * Cw + cw) * 4 + warp] = (uint16_t)b1;
    s_q[((lp + 2) * Cw + cw) * 4 + warp] = (uint16_t)b2;
    s_q[((lp + 3) * Cw + cw) * 4 + warp] = (uint16_t)b3;
  }
  __syncthreads();
  const int npx = (int)min((long long)128, npix - pix0);
  if (npx <= 0) return;
  if (C2) {
    const int C1 = (Cw + 1) / 2;
    ulonglong2* d2 = reinterpret_cast<ulonglong2*>(packed);  // 16-byte aligned: checked on the host
    for (int i = threadIdx.x; i < C1 * npx; i += kPackThreads) {
      const int grp = i / npx, px = i - grp * npx;  // consecutive threads: consecutive pixels of one channel group
      const long long pp = pix0 + px, nn = pp / HW, hh = pp - nn * HW;
      const uint64_t lo = s_words[px * Cw + 2 * grp], hi = (2 * grp + 1 < Cw) ? s_words[px * Cw + 2 * grp + 1] : 0ull;
      d2[((size_t)nn * C1 + grp) * HW + hh] = make_ulonglong2(lo, hi);
    }
    return;
  }
  // contiguous in global memory: pixels pix0 .. pix0+npx-1 of the batch, all words
  uint64_t* dst = packed + (size_t)pix0 * Cw;
  const int total = npx * Cw;
  if (((size_t)pix0 * Cw) % 2 == 0 && (reinterpret_cast<uintptr_t>(packed) & 15) == 0) {
    const int pairs = total / 2;
    const ulonglong2* s2 = reinterpret_cast<const ulonglong2*>(s_words);
    ulonglong2* d2 = reinterpret_cast<ulonglong2*>(dst);
    for (int i = threadIdx.x; i < pairs; i += kPackThreads) d2[i] = s2[i];
    if ((total & 1) && threadIdx.x == 0) dst[total - 1] = s_words[total - 1];
  } else {
    for (int i = threadIdx.x; i < total; i += kPackThreads) dst[i] = s_words[i];
  }
}

// NCHW, any H*W and alignment: a CTA takes 128 consecutive pixels of one image and one 64-channel word.  The
// 64 x 128 sign flags are gathered with coalesced scalar loads (lanes along pixels) into shared memory; each
// thread then assembles 32 channel bits of one pixel and stores that half word.
template <typename T>
__global__ void __launch_bounds__(256) pack_nchw_tile(const T* __restrict__ x, int C, int HW, int Cw,
                                                      uint64_t* __restrict__ packed) {
  __shared__ unsigned char s_sign[64 * 128];
  const int tid = threadIdx.x, lane = tid & 31, ty = tid >> 5;
  const int n = blockIdx.y, p0 = blockIdx.x * 128, cw = blockIdx.z;
  const int npix = min(128, HW - p0);
  const T* xn = x + (size_t)n * C * HW + p0;
  const int c0 = cw * 64, cn = min(64, C - c0);
#pragma unroll
  for (int c = ty; c < 64; c += 8) {
    const T* row = xn + (size_t)(c0 + c) * HW;
#pragma unroll
    for (int q = 0; q < 4; q++) {
      const int p = lane + 32 * q;
      s_sign[c * 128 + p] = (c < cn && p < npix) ? (unsigned char)neg(__ldcs(row + p)) : (unsigned char)0;
    }
  }
  __syncthreads();
  const int p = tid & 127, half = tid >> 7;
  if (p < npix) {
    uint32_t bits = 0;
#pragma unroll
    for (int c = 0; c < 32; c++) bits |= (uint32_t)s_sign[(half * 32 + c) * 128 + p] << c;
    reinterpret_cast<uint32_t*>(packed)[(((size_t)n * HW + p0 + p) * Cw + cw) * 2 + half] = bits;
  }
}

// Any layout, any shape: one thread per output word (c2: the word goes to its place in the NC1HWC2 layout, and the
// thread of an odd last word also writes the zero partner).
template <typename T>
__global__ void pack_generic(const T* __restrict__ x, int nhwc, int C, int HW, int Cw, long long total_words,
                             uint64_t* __restrict__ packed, int c2) {
  long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= total_words) return;
  const int cw = (int)(t % Cw);
  const long long pix = t / Cw;  // n*HW + hw
  const int c0 = cw * 64, cn = min(64, C - c0);
  uint64_t w = 0;
  if (nhwc) {
    const T* src = x + (size_t)pix * C + c0;
    for (int c = 0; c < cn; c++) w |= (uint64_t)neg(src[c]) << c;
  } else {
    const long long n = pix / HW, hw = pix % HW;
    const T* src = x + ((size_t)n * C + c0) * HW + hw;
    for (int c = 0; c < cn; c++) w |= (uint64_t)neg(src[(size_t)c * HW]) << c;
  }
  if (c2) {
    const long long n = pix / HW, hw = pix % HW;
    const int C1 = (Cw + 1) / 2;
    uint64_t* v = packed + (((size_t)n * C1 + (cw >> 1)) * HW + hw) * 2;
    v[cw & 1] = w;
    if (cw == Cw - 1 && (cw & 1) == 0) v[1] = 0;
  } else {
    packed[t] = w;
  }
}

// NHWC with C a multiple of 64 and 16-byte aligned input: 16 lanes share one word; each lane tests 4
// channels (one float4), places its nibble, and an OR-reduction over 8-lane groups builds each half.
template <typename T>
__global__ void __launch_bounds__(256) pack_nhwc_c64(const T* __restrict__ x, long long total_words,
                                                     uint64_t* __restrict__ packed) {
  const int lane = threadIdx.x & 31;
  const long long warp_global = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
  const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
  const unsigned gmask = 0xFFu << (lane & 24);  // this lane's 8-lane group
  using V4 = typename Vec4<T>::type;
  // a warp handles 2 words (128 floats) per step; 4 steps in flight per iteration
  for (long long w0 = warp_global * 8; w0 < total_words; w0 += nwarps * 8) {
    V4 v[4];
#pragma unroll
    for (int u = 0; u < 4; u++) {
      const long long word = w0 + 2 * u + (lane >> 4);
      v[u] = V4{0, 0, 0, 0};
      if (word < total_words) v[u] = __ldcs(reinterpret_cast<const V4*>(x) + word * 16 + (lane & 15));
    }
#pragma unroll
    for (int u = 0; u < 4; u++) {
      unsigned nib = neg(v[u].x) | (neg(v[u].y) << 1) | (neg(v[u].z) << 2) | (neg(v[u].w) << 3);
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

template <typename T>
dabnn_status pack_any(const T* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed, void* stream,
                      dabnn_packed_layout pl = DABNN_PACKED_NHWC) {
  if (!x || !packed) return DABNN_ERR_NULL;
  if (s.N <= 0 || s.C <= 0 || s.H <= 0 || s.W <= 0) return DABNN_ERR_SHAPE;
  if (in_layout != DABNN_NCHW && in_layout != DABNN_NHWC) return DABNN_ERR_SHAPE;
  if (pl != DABNN_PACKED_NHWC && pl != DABNN_PACKED_NC1HWC2) return DABNN_ERR_SHAPE;
  const bool c2 = pl == DABNN_PACKED_NC1HWC2;
  if (!aligned(x, 4) || !aligned(packed, c2 ? 16 : 8)) return DABNN_ERR_ALIGNMENT;
  const long long HW = (long long)s.H * s.W;
  const long long Cw = (s.C + 63) / 64;
  if (HW > 0x7FFFFFFF || (long long)s.N * HW > 0x7FFFFFFFFFFLL) return DABNN_ERR_UNSUPPORTED;
  const long long total_words = (long long)s.N * HW * Cw;
  cudaStream_t st = as_stream(stream);
  if (in_layout == DABNN_NCHW && HW % 4 == 0 && aligned(x, 16) && Cw * 128 * 8 <= 48 * 1024 &&
      (long long)s.N * HW <= 128LL * 0x7FFFFFFF) {
    const long long npix = (long long)s.N * HW;
    const unsigned grid = (unsigned)((npix + 127) / 128);
    if (c2) pack_nchw_vec4<T, true><<<grid, kPackThreads, (size_t)128 * Cw * 8, st>>>(x, s.C, (int)HW, (int)Cw, npix, packed);
    else pack_nchw_vec4<T, false><<<grid, kPackThreads, (size_t)128 * Cw * 8, st>>>(x, s.C, (int)HW, (int)Cw, npix, packed);
  } else if (!c2 && in_layout == DABNN_NCHW && s.N <= 65535 && Cw <= 65535) {
    dim3 grid(ceil_div(HW, 128), s.N, (unsigned)Cw);
    pack_nchw_tile<T><<<grid, 256, 0, st>>>(x, s.C, (int)HW, (int)Cw, packed);
  } else if (!c2 && in_layout == DABNN_NHWC && s.C % 64 == 0 && aligned(x, 16)) {
    const long long warps_needed = (total_words + 7) / 8;
    long long blocks = (warps_needed + 7) / 8;
    const long long cap = (long long)sm_count() * 16;
    if (blocks > cap) blocks = cap;
    pack_nhwc_c64<T><<<(unsigned)blocks, 256, 0, st>>>(x, total_words, packed);
  } else {
    const long long blocks = (total_words + 255) / 256;
    if (blocks > 0x7FFFFFFF) return DABNN_ERR_UNSUPPORTED;
    pack_generic<T><<<(unsigned)blocks, 256, 0, st>>>(x, in_layout == DABNN_NHWC, s.C, (int)HW, (int)Cw, total_words,
                                                   packed, c2 ? 1 : 0);
  }
  return launch_status();
}

extern "C" dabnn_status dabnn_pack(const float* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed,
                                   void* stream) {
  return pack_any<float>(x, in_layout, s, packed, stream);
}

extern "C" dabnn_status dabnn_pack_as(const float* x, dabnn_layout in_layout, dabnn_shape s, dabnn_packed_layout packed_layout,
                                      uint64_t* packed, void* stream) {
  return pack_any<float>(x, in_layout, s, packed, stream, packed_layout);
}

extern "C" size_t dabnn_packed_words(dabnn_shape s, dabnn_packed_layout packed_layout) {
  if (s.N <= 0 || s.C <= 0 || s.H <= 0 || s.W <= 0) return 0;
  const size_t pix = (size_t)s.N * s.H * s.W;
  if (packed_layout == DABNN_PACKED_NC1HWC2) return pix * 2 * (size_t)((s.C + 127) / 128);
  return packed_layout == DABNN_PACKED_NHWC ? pix * (size_t)((s.C + 63) / 64) : 0;
}

extern "C" dabnn_status dabnn_pack_i32(const int32_t* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed,
                                       void* stream) {
  return pack_any<int32_t>(x, in_layout, s, packed, stream);
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
