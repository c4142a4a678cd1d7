// The xor/popcount convolution tile (Section 2.1.2, Eq. 1 of the paper): everything one CTA does for a tile of BP output
// pixels x BO output channels, as a device function, so that the stand-alone kernel (bconv.cu) and the one-launch
// Bi-Real chain for single images (bireal18.cu) run the same code.  See bconv.cu for the formulation.
#pragma once
#include "common.cuh"

namespace dabnn {

namespace {

enum { EPI_I32 = 0, EPI_BNPACK = 1, EPI_BIREAL = 2 };

constexpr int KC64 = 16;             // 64-bit words per K chunk and smem row
constexpr int PITCH = 2 * KC64 + 4;  // 32-bit words per smem row: 144 B, keeps 8 consecutive rows on distinct banks
constexpr int STAGES_DEFAULT = 3;  // ring depth of the throughput tiles; the small-problem tile holds all of K at once

struct BConvArgs {
  const uint64_t* a;
  const uint64_t* w;
  int N, H, W, Cw, C;
  int O, kh, kw, sh, sw, ph, pw, OH, OW;
  long long M;  // N*OH*OW output pixels
  int K64;      // kh*kw*Cw 64-bit words per filter
  int Kbits;    // C*kh*kw
  int pad_neg;  // padded positions hold -1 (bit 1)
  uint64_t tail_mask;  // valid bits of a pixel's last word
  int32_t* out;
  int out_nchw;
  const float* scale;
  const float* shift;
  const float* residual;
  float* y_out;
  uint32_t* out_packed32;  // packed output viewed as 32-bit halves
  int Ow32;                // 2*ceil(O/64)
  int one;                 // the constant 1 (see bit_mac)
  unsigned long long magic_cw, magic_kw;  // ceil(2^64 / Cw), ceil(2^64 / kw) (0 when the divisor is 1): see fast_div
  // Where word cw of pixel (ih, iw) of image n lives, in 64-bit words:  n * img_stride + (ih * W + iw) * pix_stride +
  // (cw >> 1) * pair_stride + (cw & 1).  Channel-packed NHWC [N][H][W][Cw]: pix_stride = Cw, pair_stride = 2.
  // NC1HWC2 with 128-bit vectors [N][C1][H][W][2] (Section 2.1.2, last paragraph): pix_stride = 2, pair_stride = 2*H*W.
  long long img_stride;
  int pix_stride, pair_stride;
  unsigned long long magic_ow, magic_oh;  // ceil(2^64 / OW), ceil(2^64 / OH) (0 for 1), used when M < 2^31
  int pointwise;  // 1x1 filter, stride 1, no padding, channel-packed NHWC words: the im2col row of output pixel m is
                  // simply pixel m's words, so the loader needs no per-row table and no bounds tests
};

struct RowInfo {
  long long base;  // element offset of image n in `a`, or -1 for a row beyond M
  int ih0, iw0;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// floor(q / d) for q < 2^32 with magic = ceil(2^64 / d) (0 for d = 1): one 64-bit multiply-high instead of a division.
__device__ __forceinline__ int fast_div(int q, unsigned long long magic) {
  return magic == 0 ? q : (int)__umul64hi((unsigned long long)(uint32_t)q, magic);
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async8(uint32_t dst, const void* src, int bytes) {
  asm volatile("cp.async.ca.shared.global [%0], [%1], 8, %2;" ::"r"(dst), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() {
  asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory");
}

// `one` is the constant 1 passed through the kernel arguments: multiplying by it keeps the accumulation an
// integer multiply-add, which issues on the FMA pipe and leaves the ALU pipe to the logic operations.
template <bool CSA>
__device__ __forceinline__ void bit_mac(uint32_t a0, uint32_t a1, uint32_t w0, uint32_t w1, int& acc, uint32_t& ones,
                                        int one) {
  if (CSA) {
    // Full adder of (ones, a0 ^ w0, a1 ^ w1) in three 3-input logic ops, the xors folded in:
    //   t = ones ^ a0 ^ w0;  s = t ^ a1 ^ w1 (the sum bit);  carry = t ? ~s : ones
    // (where ones and the first term differ, t = 1 and the majority is the second term, which is s ^ t = ~s; where
    // they agree, t = 0 and the majority is their common value).
    uint32_t t, s, c;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(t) : "r"(ones), "r"(a0), "r"(w0));
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(s) : "r"(t), "r"(a1), "r"(w1));
    asm("lop3.b32 %0, %1, %2, %3, 0x3A;" : "=r"(c) : "r"(t), "r"(s), "r"(ones));  // (t & ~s) | (~t & ones)
    ones = s;
    acc = __popc(c) * one + acc;
  } else {
    acc = __popc(a0 ^ w0) * one + acc;
    acc = __popc(a1 ^ w1) * one + acc;
  }
}

// Two carry-save steps (one 128-bit load of each operand) whose two popcounts join the count in ONE three-input add: 6 LOP3
// + 1 IADD3 on the ALU pipe (7 of the 8 cycles that the two POPCs occupy the XU pipe) and no multiply-add: 4.5 issue slots
// per word-pair step instead of 5.  Measured against the IMAD form: +10 % on the 1x1 512 -> 2048 layer, +0.5 to 3 % on the 3x3 layers.
__device__ __forceinline__ void bit_mac_pair(const uint4 a, const uint4 w, int& acc, uint32_t& ones) {
  uint32_t t, s, c0, c1;
  asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(t) : "r"(ones), "r"(a.x), "r"(w.x));
  asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(s) : "r"(t), "r"(a.y), "r"(w.y));
  asm("lop3.b32 %0, %1, %2, %3, 0x3A;" : "=r"(c0) : "r"(t), "r"(s), "r"(ones));
  ones = s;
  asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(t) : "r"(ones), "r"(a.z), "r"(w.z));
  asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(s) : "r"(t), "r"(a.w), "r"(w.w));
  asm("lop3.b32 %0, %1, %2, %3, 0x3A;" : "=r"(c1) : "r"(t), "r"(s), "r"(ones));
  ones = s;
  acc += __popc(c0) + __popc(c1);
}

// One tile: pixel tile `bx`, channel tile `by`, `smem` = STAGES * (BP + BO) * PITCH words + BP RowInfo.  All threads of
// the CTA call it together.  CHAINED: the stand-alone kernel's hooks for chained launches (see common.cuh).
template <int BP, int BO, int TP, int TO, int EPI, bool CSA, bool VEC16, int STAGES, bool CHAINED>
__device__ __forceinline__ void bconv_tile(const BConvArgs& g, const long long bx, const int by, uint32_t* smem) {
  constexpr int THREADS = (BP / TP) * (BO / TO);
  constexpr int UW = VEC16 ? 2 : 1;         // 64-bit words per copy unit
  constexpr int UNITS = KC64 / UW;          // units per row and chunk
  constexpr int ROWS_PER_PASS = THREADS / UNITS;
  static_assert(THREADS % UNITS == 0 && THREADS % 32 == 0, "thread count");
  static_assert(BP % (8 * TP) == 0 && BO % (4 * TO) == 0, "warp tile");
  static_assert(BP % ROWS_PER_PASS == 0 && BO % ROWS_PER_PASS == 0, "loader passes");
  constexpr int WPN = BP / (8 * TP);        // warps along the pixel axis
  constexpr int UNROLL_K = (TP * TO >= 32) ? 1 : 2;
  constexpr int STAGE_WORDS = (BP + BO) * PITCH;
  // Small tiles serve launches of less than a wave, where latency is all there is: what does not depend on the previous
  // layer (weights, BN vectors) is requested before the wait of a chained launch, and the residual values together with
  // the activation words rather than after the main loop.
  constexpr bool EARLY = TP * TO <= 8;

  uint32_t* ring = smem;                                           // [STAGES][BP + BO][PITCH]
  RowInfo* rows = reinterpret_cast<RowInfo*>(smem + STAGES * STAGE_WORDS);  // [BP]

  const int tid = threadIdx.x;
  const long long m0 = bx * BP;
  const int o0 = by * BO;

  for (int r = tid; r < (g.pointwise ? 0 : BP); r += THREADS) {
    const long long m = m0 + r;
    RowInfo ri;
    if (m < g.M) {
      int ow, oh;
      long long n;
      if (g.M < (1LL << 31)) {  // the usual case: 32-bit coordinates, multiply-high instead of 64-bit divisions
        const int t = fast_div((int)m, g.magic_ow);
        ow = (int)m - t * g.OW;
        const int nn = fast_div(t, g.magic_oh);
        oh = t - nn * g.OH;
        n = nn;
      } else {
        ow = (int)(m % g.OW);
        const long long t = m / g.OW;
        oh = (int)(t % g.OH);
        n = t / g.OH;
      }
      ri.base = n * g.img_stride;
      ri.ih0 = oh * g.sh - g.ph;
      ri.iw0 = ow * g.sw - g.pw;
    } else {
      ri.base = -1;
      ri.ih0 = ri.iw0 = 0;
    }
    rows[r] = ri;
  }

  const int unit = tid % UNITS;
  const int row_first = tid / UNITS;
  const int nchunks = (g.K64 + KC64 - 1) / KC64;

  auto load_chunk = [&](int chunk, int stage, const bool want_a, const bool want_w) {
    uint32_t* As = ring + stage * STAGE_WORDS;
    uint32_t* Ws = As + BP * PITCH;
    const int k = chunk * KC64 + unit * UW;  // first 64-bit word of this thread's unit
    const bool k_live = k < g.K64;
    int tap = 0, cw = 0, ti = 0, tj = 0;
    if (k_live) {
      tap = fast_div(k, g.magic_cw);
      cw = k - tap * g.Cw;
      ti = fast_div(tap, g.magic_kw);
      tj = tap - ti * g.kw;
    }
    // activations: one im2col row per output pixel
#pragma unroll
    for (int it = 0; it < (want_a ? BP / ROWS_PER_PASS : 0); it++) {
      const int r = row_first + it * ROWS_PER_PASS;
      uint32_t* dst = As + r * PITCH + unit * UW * 2;
      if (g.pointwise) {  // (uniform) pixel m's words are the row: k counts channel words
        const bool live = k_live && m0 + r < g.M;
        const uint64_t* src = live ? g.a + ((m0 + r) * g.Cw + k) : g.a;
        if (UW == 2) cp_async16(smem_u32(dst), src, live ? 16 : 0);
        else cp_async8(smem_u32(dst), src, live ? 8 : 0);
        continue;
      }
      const RowInfo ri = rows[r];
      const int ih = ri.ih0 + ti, iw = ri.iw0 + tj;
      const bool live = k_live && ri.base >= 0;
      if (live && (ih < 0 || ih >= g.H || iw < 0 || iw >= g.W)) {
        // padded position: the declared pad word (tail bits of a pixel's last word stay 0)
        uint64_t p0 = 0, p1 = 0;
        if (g.pad_neg) {
          p0 = (cw == g.Cw - 1) ? g.tail_mask : ~0ull;
          if (UW == 2) p1 = (cw + 1 == g.Cw - 1) ? g.tail_mask : ~0ull;
        }
        if (UW == 2) *reinterpret_cast<ulonglong2*>(dst) = make_ulonglong2(p0, p1);
        else *reinterpret_cast<uint64_t*>(dst) = p0;
      } else {
        // (the offset inside one image fits 32 bits: checked on the host)
        const uint64_t* src =
            live ? g.a + (ri.base + (long long)((ih * g.W + iw) * g.pix_stride + (cw >> 1) * g.pair_stride + (cw & 1))) : g.a;
        if (UW == 2) cp_async16(smem_u32(dst), src, live ? 16 : 0);
        else cp_async8(smem_u32(dst), src, live ? 8 : 0);
      }
    }
    // weights: one row per output channel, K contiguous
#pragma unroll
    for (int it = 0; it < (want_w ? BO / ROWS_PER_PASS : 0); it++) {
      const int r = row_first + it * ROWS_PER_PASS;
      const int o = o0 + r;
      uint32_t* dst = Ws + r * PITCH + unit * UW * 2;
      const bool live = k_live && o < g.O;
      const uint64_t* src = live ? g.w + (long long)o * g.K64 + k : g.w;
      if (UW == 2) cp_async16(smem_u32(dst), src, live ? 16 : 0);
      else cp_async8(smem_u32(dst), src, live ? 8 : 0);
    }
  };

  const int one = g.one;
  const int lane = tid & 31, wid = tid >> 5;
  const int pl = lane & 7, ol = lane >> 3;
  const int wp = wid % WPN, wo = wid / WPN;
  const int arow0 = wp * 8 * TP + pl;        // + 8*i
  const int wrow0 = wo * 4 * TO + ol * TO;   // + j

  int acc[TP][TO];
  uint32_t ones[TP][TO];
#pragma unroll
  for (int i = 0; i < TP; i++)
#pragma unroll
    for (int j = 0; j < TO; j++) {
      acc[i][j] = 0;
      ones[i][j] = 0;
    }

  float sc[TO], sf[TO], res[TP][TO];
  const bool res_vec = EPI == EPI_BIREAL && TO % 4 == 0 && o0 + wrow0 + TO <= g.O && (g.O & 3) == 0 &&
                       ((reinterpret_cast<uintptr_t>(g.residual) | reinterpret_cast<uintptr_t>(g.y_out)) & 15) == 0;
  if (EARLY) {
#pragma unroll
    for (int s = 0; s < STAGES - 1; s++)
      if (s < nchunks) load_chunk(s, s, false, true);
    if (EPI != EPI_I32) {
#pragma unroll
      for (int j = 0; j < TO; j++) {
        sc[j] = (o0 + wrow0 + j < g.O) ? g.scale[o0 + wrow0 + j] : 0.f;
        sf[j] = (o0 + wrow0 + j < g.O) ? g.shift[o0 + wrow0 + j] : 0.f;
      }
    }
  }
  __syncthreads();            // rows[] is complete
  if (CHAINED) chain_wait();  // (chained launches: nothing above reads what the previous kernel wrote)
#pragma unroll
  for (int s = 0; s < STAGES - 1; s++) {
    if (s < nchunks) load_chunk(s, s, true, !EARLY);
    cp_async_commit();
  }
  if (EARLY && EPI == EPI_BIREAL) {
#pragma unroll
    for (int i = 0; i < TP; i++) {
      const long long m = m0 + arow0 + 8 * i;
      const float* rs = g.residual + m * g.O + o0 + wrow0;
#pragma unroll
      for (int j = 0; j < TO; j++) res[i][j] = 0.f;
      if (m >= g.M) continue;
      if (res_vec) {
#pragma unroll
        for (int j = 0; j < TO; j += 4) {
          const float4 r4 = __ldcs(reinterpret_cast<const float4*>(rs + j));
          res[i][j] = r4.x; res[i][j + 1] = r4.y; res[i][j + 2] = r4.z; res[i][j + 3] = r4.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < TO; j++)
          if (o0 + wrow0 + j < g.O) res[i][j] = rs[j];
      }
    }
  }

  for (int chunk = 0; chunk < nchunks; chunk++) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();  // chunk's data visible to all; everyone is done with the stage about to be refilled
    {
      const int nxt = chunk + STAGES - 1;
      if (nxt < nchunks) load_chunk(nxt, nxt % STAGES, true, true);
      cp_async_commit();
    }
    const uint32_t* As = ring + (chunk % STAGES) * STAGE_WORDS;
    const uint32_t* Ws = As + BP * PITCH;
    const int kvalid = min(KC64, g.K64 - chunk * KC64);  // 64-bit words in this chunk
    int k = 0;
#pragma unroll UNROLL_K
    for (; k + 2 <= kvalid; k += 2) {
      uint4 w[TO];
#pragma unroll
      for (int j = 0; j < TO; j++) w[j] = *reinterpret_cast<const uint4*>(Ws + (wrow0 + j) * PITCH + 2 * k);
#pragma unroll
      for (int i = 0; i < TP; i++) {  // (activation rows one at a time: a thread never holds all of them)
        const uint4 a = *reinterpret_cast<const uint4*>(As + (arow0 + 8 * i) * PITCH + 2 * k);
#pragma unroll
        for (int j = 0; j < TO; j++) {
          if (CSA) {
            bit_mac_pair(a, w[j], acc[i][j], ones[i][j]);
            continue;
          }
          bit_mac<CSA>(a.x, a.y, w[j].x, w[j].y, acc[i][j], ones[i][j], one);
          bit_mac<CSA>(a.z, a.w, w[j].z, w[j].w, acc[i][j], ones[i][j], one);
        }
      }
    }
    if (k < kvalid) {  // odd tail: one 64-bit word
      uint2 a[TP], w[TO];
#pragma unroll
      for (int i = 0; i < TP; i++) a[i] = *reinterpret_cast<const uint2*>(As + (arow0 + 8 * i) * PITCH + 2 * k);
#pragma unroll
      for (int j = 0; j < TO; j++) w[j] = *reinterpret_cast<const uint2*>(Ws + (wrow0 + j) * PITCH + 2 * k);
#pragma unroll
      for (int i = 0; i < TP; i++)
#pragma unroll
        for (int j = 0; j < TO; j++) bit_mac<CSA>(a[i].x, a[i].y, w[j].x, w[j].y, acc[i][j], ones[i][j], one);
    }
  }
  cp_async_wait<0>();
  if (CHAINED) chain_trigger();

  // ---- epilogue: counts -> K - 2*count, then the selected output form -------------------------
  if (EPI == EPI_I32) {
#pragma unroll
    for (int i = 0; i < TP; i++) {
      const long long m = m0 + arow0 + 8 * i;
      if (m >= g.M) continue;
      int v[TO];
#pragma unroll
      for (int j = 0; j < TO; j++) {
        const int cnt = CSA ? 2 * acc[i][j] + __popc(ones[i][j]) : acc[i][j];
        v[j] = g.Kbits - 2 * cnt;
      }
      const int o = o0 + wrow0;
      // (streaming stores: the int32 sums are read by nothing in this library, and kept out of the way in L2 they do
      // not displace the weights and activations that the following launches read)
      if (!g.out_nchw) {
        int32_t* dst = g.out + m * g.O + o;
        if (TO % 4 == 0 && o + TO <= g.O && (g.O & 3) == 0 && (reinterpret_cast<uintptr_t>(g.out) & 15) == 0) {
#pragma unroll
          for (int j = 0; j < TO; j += 4) __stcs(reinterpret_cast<int4*>(dst + j), make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]));
        } else {
#pragma unroll
          for (int j = 0; j < TO; j++)
            if (o + j < g.O) __stcs(dst + j, v[j]);
        }
      } else {
        const long long ohw = (long long)g.OH * g.OW;
        const long long n = m / ohw, q = m % ohw;
#pragma unroll
        for (int j = 0; j < TO; j++)
          if (o + j < g.O) __stcs(g.out + (n * g.O + o + j) * ohw + q, v[j]);
      }
    }
  } else {
    constexpr int BW = BO / 32;  // 32-bit sign words per pixel row of this tile
    __syncthreads();             // all warps are done reading the ring
    uint32_t* sbits = smem;      // [BP][BW]
    const bool want_bits = g.out_packed32 != nullptr;
    if (want_bits) {
      for (int t = tid; t < BP * BW; t += THREADS) sbits[t] = 0;
      __syncthreads();
    }
    const int o = o0 + wrow0;
    if (!EARLY) {
#pragma unroll
      for (int j = 0; j < TO; j++) {
        sc[j] = (o + j < g.O) ? g.scale[o + j] : 0.f;
        sf[j] = (o + j < g.O) ? g.shift[o + j] : 0.f;
      }
    }
#pragma unroll
    for (int i = 0; i < TP; i++) {
      const long long m = m0 + arow0 + 8 * i;
      if (m >= g.M) continue;
      float y[TO];
#pragma unroll
      for (int j = 0; j < TO; j++) {
        const int cnt = CSA ? 2 * acc[i][j] + __popc(ones[i][j]) : acc[i][j];
        y[j] = __fmaf_rn((float)(g.Kbits - 2 * cnt), sc[j], sf[j]);
      }
      if (EPI == EPI_BIREAL) {
        const float* rs = g.residual + m * g.O + o;
        float* yd = g.y_out + m * g.O + o;
        if (res_vec) {
#pragma unroll
          for (int j = 0; j < TO; j += 4) {
            float4 r4;
            if (EARLY) r4 = make_float4(res[i][j], res[i][j + 1], res[i][j + 2], res[i][j + 3]);
            else r4 = __ldcs(reinterpret_cast<const float4*>(rs + j));  // the residual is read once
            y[j] = __fadd_rn(y[j], r4.x);
            y[j + 1] = __fadd_rn(y[j + 1], r4.y);
            y[j + 2] = __fadd_rn(y[j + 2], r4.z);
            y[j + 3] = __fadd_rn(y[j + 3], r4.w);
            *reinterpret_cast<float4*>(yd + j) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
          }
        } else {
#pragma unroll
          for (int j = 0; j < TO; j++)
            if (o + j < g.O) {
              y[j] = __fadd_rn(y[j], EARLY ? res[i][j] : rs[j]);
              yd[j] = y[j];
            }
        }
      }
      if (want_bits) {
        uint32_t field = 0;
#pragma unroll
        for (int j = 0; j < TO; j++) field |= (uint32_t)((o + j < g.O) && (y[j] < 0.0f)) << j;
        if (field) atomicOr(&sbits[(arow0 + 8 * i) * BW + (wrow0 >> 5)], field << (wrow0 & 31));
      }
    }
    if (want_bits) {
      __syncthreads();
      const int wbase = o0 >> 5;
      for (int t = tid; t < BP * BW; t += THREADS) {
        const int r = t / BW, q = t - r * BW;
        const long long m = m0 + r;
        if (m < g.M && wbase + q < g.Ow32) g.out_packed32[m * g.Ow32 + wbase + q] = sbits[t];
      }
    }
  }
}

// ---- short-K pointwise layers: several pixel tiles per CTA -----------------------------------------------------
// An unpadded 1x1 stride-1 layer whose K fits one chunk (C <= 1024) has no K loop to pipeline: a one-tile CTA is set-up,
// one round of loads, 256 word-pair steps per thread and an epilogue, and a third of its instructions are the fixed part.
// Here a CTA keeps its BO weight rows in shared memory and walks over NSUB consecutive pixel tiles, whose activation rows
// run through the ring: the loads of tile s + 2 are in flight while tile s is multiplied and written.
template <int BP, int BO, int TP, int TO, int EPI, bool VEC16, int NSUB>
__device__ __forceinline__ void bconv_pointwise_tiles(const BConvArgs& g, uint32_t* smem) {
  static_assert(EPI == EPI_I32 || EPI == EPI_BNPACK, "output form");
  constexpr int THREADS = (BP / TP) * (BO / TO);
  constexpr int STAGES = 3;
  constexpr int UW = VEC16 ? 2 : 1;
  constexpr int UNITS = KC64 / UW;
  constexpr int ROWS_PER_PASS = THREADS / UNITS;
  static_assert(THREADS % UNITS == 0 && BP % ROWS_PER_PASS == 0 && BO % ROWS_PER_PASS == 0, "loader passes");
  constexpr int WPN = BP / (8 * TP);
  constexpr int BW = BO / 32;
  uint32_t* Ws = smem;                         // [BO][PITCH]
  uint32_t* ring = smem + BO * PITCH;          // [STAGES][BP][PITCH]
  uint32_t* sbits = ring + STAGES * BP * PITCH;  // [BP][BW]

  const int tid = threadIdx.x;
  const int o0 = blockIdx.y * BO;
  const long long n_bx = (g.M + BP - 1) / BP;
  const long long t_first = (long long)blockIdx.x * NSUB;
  const int nsub = (int)min((long long)NSUB, n_bx - t_first);
  const int unit = tid % UNITS, row_first = tid / UNITS;
  const int k = unit * UW;
  const bool k_live = k < g.K64;

  auto load_a = [&](int sidx, int stage) {
    uint32_t* As = ring + stage * BP * PITCH;
    const long long m0 = (t_first + sidx) * BP;
#pragma unroll
    for (int it = 0; it < BP / ROWS_PER_PASS; it++) {
      const int r = row_first + it * ROWS_PER_PASS;
      const bool live = k_live && m0 + r < g.M;
      const uint64_t* src = live ? g.a + ((m0 + r) * g.Cw + k) : g.a;
      if (UW == 2) cp_async16(smem_u32(As + r * PITCH + unit * UW * 2), src, live ? 16 : 0);
      else cp_async8(smem_u32(As + r * PITCH + unit * UW * 2), src, live ? 8 : 0);
    }
  };
#pragma unroll
  for (int it = 0; it < BO / ROWS_PER_PASS; it++) {  // the CTA's weight rows, once
    const int r = row_first + it * ROWS_PER_PASS;
    const bool live = k_live && o0 + r < g.O;
    const uint64_t* src = live ? g.w + (long long)(o0 + r) * g.K64 + k : g.w;
    if (UW == 2) cp_async16(smem_u32(Ws + r * PITCH + unit * UW * 2), src, live ? 16 : 0);
    else cp_async8(smem_u32(Ws + r * PITCH + unit * UW * 2), src, live ? 8 : 0);
  }
#pragma unroll
  for (int s = 0; s < STAGES - 1; s++) {
    if (s < nsub) load_a(s, s);
    cp_async_commit();
  }

  const int lane = tid & 31, wid = tid >> 5;
  const int pl = lane & 7, ol = lane >> 3;
  const int wp = wid % WPN, wo = wid / WPN;
  const int arow0 = wp * 8 * TP + pl;
  const int wrow0 = wo * 4 * TO + ol * TO;
  const int o = o0 + wrow0;
  const int one = g.one;
  float sc[TO], sf[TO];
  if (EPI == EPI_BNPACK) {
#pragma unroll
    for (int j = 0; j < TO; j++) {
      sc[j] = (o + j < g.O) ? g.scale[o + j] : 0.f;
      sf[j] = (o + j < g.O) ? g.shift[o + j] : 0.f;
    }
  }
  int acc[TP][TO];
  uint32_t ones[TP][TO];
  for (int s = 0; s < nsub; s++) {
#pragma unroll
    for (int i = 0; i < TP; i++)
#pragma unroll
      for (int j = 0; j < TO; j++) {
        acc[i][j] = 0;
        ones[i][j] = 0;
      }
    cp_async_wait<STAGES - 2>();
    __syncthreads();  // tile s (and the weights) visible to all; everyone is done with the stage about to be refilled
    if (s + STAGES - 1 < nsub) load_a(s + STAGES - 1, (s + STAGES - 1) % STAGES);
    cp_async_commit();
    const uint32_t* As = ring + (s % STAGES) * BP * PITCH;
    int kk = 0;
    for (; kk + 2 <= g.K64; kk += 2) {
      uint4 w[TO];
#pragma unroll
      for (int j = 0; j < TO; j++) w[j] = *reinterpret_cast<const uint4*>(Ws + (wrow0 + j) * PITCH + 2 * kk);
#pragma unroll
      for (int i = 0; i < TP; i++) {
        const uint4 a = *reinterpret_cast<const uint4*>(As + (arow0 + 8 * i) * PITCH + 2 * kk);
#pragma unroll
        for (int j = 0; j < TO; j++) bit_mac_pair(a, w[j], acc[i][j], ones[i][j]);
      }
    }
    if (kk < g.K64) {  // odd tail: one 64-bit word
      uint2 w[TO];
#pragma unroll
      for (int j = 0; j < TO; j++) w[j] = *reinterpret_cast<const uint2*>(Ws + (wrow0 + j) * PITCH + 2 * kk);
#pragma unroll
      for (int i = 0; i < TP; i++) {
        const uint2 a = *reinterpret_cast<const uint2*>(As + (arow0 + 8 * i) * PITCH + 2 * kk);
#pragma unroll
        for (int j = 0; j < TO; j++) bit_mac<true>(a.x, a.y, w[j].x, w[j].y, acc[i][j], ones[i][j], one);
      }
    }
    const long long m0 = (t_first + s) * BP;
    if (EPI == EPI_I32) {
#pragma unroll
      for (int i = 0; i < TP; i++) {
        const long long m = m0 + arow0 + 8 * i;
        if (m >= g.M) continue;
        int v[TO];
#pragma unroll
        for (int j = 0; j < TO; j++) v[j] = g.Kbits - 2 * (2 * acc[i][j] + __popc(ones[i][j]));
        if (!g.out_nchw) {
          int32_t* dst = g.out + m * g.O + o;
          if (TO % 4 == 0 && o + TO <= g.O && (g.O & 3) == 0 && (reinterpret_cast<uintptr_t>(g.out) & 15) == 0) {
#pragma unroll
            for (int j = 0; j < TO; j += 4) __stcs(reinterpret_cast<int4*>(dst + j), make_int4(v[j], v[j + 1], v[j + 2], v[j + 3]));
          } else {
#pragma unroll
            for (int j = 0; j < TO; j++)
              if (o + j < g.O) __stcs(dst + j, v[j]);
          }
        } else {
          const long long ohw = (long long)g.OH * g.OW;
          const long long n = m / ohw, q = m % ohw;
#pragma unroll
          for (int j = 0; j < TO; j++)
            if (o + j < g.O) __stcs(g.out + (n * g.O + o + j) * ohw + q, v[j]);
        }
      }
    } else {
      for (int t = tid; t < BP * BW; t += THREADS) sbits[t] = 0;  // (the previous tile's readers passed this tile's barrier)
      __syncthreads();
#pragma unroll
      for (int i = 0; i < TP; i++) {
        const long long m = m0 + arow0 + 8 * i;
        if (m >= g.M) continue;
        uint32_t field = 0;
#pragma unroll
        for (int j = 0; j < TO; j++) {
          const float y = __fmaf_rn((float)(g.Kbits - 2 * (2 * acc[i][j] + __popc(ones[i][j]))), sc[j], sf[j]);
          field |= (uint32_t)((o + j < g.O) && (y < 0.0f)) << j;
        }
        if (field) atomicOr(&sbits[(arow0 + 8 * i) * BW + (wrow0 >> 5)], field << (wrow0 & 31));
      }
      __syncthreads();
      const int wbase = o0 >> 5;
      for (int t = tid; t < BP * BW; t += THREADS) {
        const int r = t / BW, q = t - r * BW;
        const long long m = m0 + r;
        if (m < g.M && wbase + q < g.Ow32) g.out_packed32[m * g.Ow32 + wbase + q] = sbits[t];
      }
    }
  }
  cp_async_wait<0>();
}

template <int BP, int BO, int TP, int TO, int MINB, int EPI, bool VEC16, int NSUB>
__global__ void __launch_bounds__((BP / TP) * (BO / TO), MINB) bconv_pointwise_kernel(const BConvArgs g) {
  extern __shared__ __align__(16) uint32_t bconv_smem[];
  bconv_pointwise_tiles<BP, BO, TP, TO, EPI, VEC16, NSUB>(g, bconv_smem);
}

template <int BP, int BO, int TP, int TO, int MINB, int EPI, bool CSA, bool VEC16, int STAGES>
__global__ void __launch_bounds__((BP / TP) * (BO / TO), MINB) bconv_kernel(const BConvArgs g) {
  extern __shared__ __align__(16) uint32_t bconv_smem[];
  bconv_tile<BP, BO, TP, TO, EPI, CSA, VEC16, STAGES, true>(g, blockIdx.x, blockIdx.y, bconv_smem);
}

}  // namespace

}  // namespace dabnn
