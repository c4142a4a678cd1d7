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
// POPC-bound.  The carry-save loop feeds the two halves of a 64-bit word pair through a 3:2
// compressor with a running "ones" word per output (2 xor + 2 lop3 per two word pairs) and
// popcounts only the carry word: half the POPCs for twice the logic, which balances the two pipes.
// Both give sum popcount(a xor w) exactly.
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
};

struct RowInfo {
  long long base;  // element offset of image n in `a`, or -1 for a row beyond M
  int ih0, iw0;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
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
    const uint32_t x1 = a0 ^ w0, x2 = a1 ^ w1;
    uint32_t s, c;
    asm("lop3.b32 %0, %1, %2, %3, 0x96;" : "=r"(s) : "r"(ones), "r"(x1), "r"(x2));  // sum bit
    asm("lop3.b32 %0, %1, %2, %3, 0xE8;" : "=r"(c) : "r"(ones), "r"(x1), "r"(x2));  // carry bit (majority)
    ones = s;
    acc = __popc(c) * one + acc;
  } else {
    acc = __popc(a0 ^ w0) * one + acc;
    acc = __popc(a1 ^ w1) * one + acc;
  }
}

template <int BP, int BO, int TP, int TO, int MINB, int EPI, bool CSA, bool VEC16, int STAGES>
__global__ void __launch_bounds__((BP / TP) * (BO / TO), MINB) bconv_kernel(const BConvArgs g) {
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

  extern __shared__ __align__(16) uint32_t smem[];
  uint32_t* ring = smem;                                           // [STAGES][BP + BO][PITCH]
  RowInfo* rows = reinterpret_cast<RowInfo*>(smem + STAGES * STAGE_WORDS);  // [BP]

  const int tid = threadIdx.x;
  const long long m0 = (long long)blockIdx.x * BP;
  const int o0 = blockIdx.y * BO;

  for (int r = tid; r < BP; r += THREADS) {
    const long long m = m0 + r;
    RowInfo ri;
    if (m < g.M) {
      const int ow = (int)(m % g.OW);
      const long long t = m / g.OW;
      const int oh = (int)(t % g.OH);
      const long long n = t / g.OH;
      ri.base = n * g.H * g.W * g.Cw;
      ri.ih0 = oh * g.sh - g.ph;
      ri.iw0 = ow * g.sw - g.pw;
    } else {
      ri.base = -1;
      ri.ih0 = ri.iw0 = 0;
    }
    rows[r] = ri;
  }
  __syncthreads();
  chain_wait();  // (chained launches: everything above is index arithmetic)

  const int unit = tid % UNITS;
  const int row_first = tid / UNITS;
  const int nchunks = (g.K64 + KC64 - 1) / KC64;

  auto load_chunk = [&](int chunk, int stage) {
    uint32_t* As = ring + stage * STAGE_WORDS;
    uint32_t* Ws = As + BP * PITCH;
    const int k = chunk * KC64 + unit * UW;  // first 64-bit word of this thread's unit
    const bool k_live = k < g.K64;
    int tap = 0, cw = 0, ti = 0, tj = 0;
    if (k_live) {
      tap = k / g.Cw;
      cw = k - tap * g.Cw;
      ti = tap / g.kw;
      tj = tap - ti * g.kw;
    }
    // activations: one im2col row per output pixel
#pragma unroll
    for (int it = 0; it < BP / ROWS_PER_PASS; it++) {
      const int r = row_first + it * ROWS_PER_PASS;
      const RowInfo ri = rows[r];
      uint32_t* dst = As + r * PITCH + unit * UW * 2;
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
        const uint64_t* src = live ? g.a + ri.base + ((long long)ih * g.W + iw) * g.Cw + cw : g.a;
        if (UW == 2) cp_async16(smem_u32(dst), src, live ? 16 : 0);
        else cp_async8(smem_u32(dst), src, live ? 8 : 0);
      }
    }
    // weights: one row per output channel, K contiguous
#pragma unroll
    for (int it = 0; it < BO / ROWS_PER_PASS; it++) {
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

#pragma unroll
  for (int s = 0; s < STAGES - 1; s++) {
    if (s < nchunks) load_chunk(s, s);
    cp_async_commit();
  }

  for (int chunk = 0; chunk < nchunks; chunk++) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();  // chunk's data visible to all; everyone is done with the stage about to be refilled
    {
      const int nxt = chunk + STAGES - 1;
      if (nxt < nchunks) load_chunk(nxt, nxt % STAGES);
      cp_async_commit();
    }
    const uint32_t* As = ring + (chunk % STAGES) * STAGE_WORDS;
    const uint32_t* Ws = As + BP * PITCH;
    const int kvalid = min(KC64, g.K64 - chunk * KC64);  // 64-bit words in this chunk
    int k = 0;
#pragma unroll UNROLL_K
    for (; k + 2 <= kvalid; k += 2) {
      uint4 a[TP], w[TO];
#pragma unroll
      for (int i = 0; i < TP; i++) a[i] = *reinterpret_cast<const uint4*>(As + (arow0 + 8 * i) * PITCH + 2 * k);
#pragma unroll
      for (int j = 0; j < TO; j++) w[j] = *reinterpret_cast<const uint4*>(Ws + (wrow0 + j) * PITCH + 2 * k);
#pragma unroll
      for (int i = 0; i < TP; i++)
#pragma unroll
        for (int j = 0; j < TO; j++) {
          bit_mac<CSA>(a[i].x, a[i].y, w[j].x, w[j].y, acc[i][j], ones[i][j], one);
          bit_mac<CSA>(a[i].z, a[i].w, w[j].z, w[j].w, acc[i][j], ones[i][j], one);
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
  chain_trigger();

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
    float sc[TO], sf[TO];
#pragma unroll
    for (int j = 0; j < TO; j++) {
      sc[j] = (o + j < g.O) ? g.scale[o + j] : 0.f;
      sf[j] = (o + j < g.O) ? g.shift[o + j] : 0.f;
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
        if (TO % 4 == 0 && o + TO <= g.O && (g.O & 3) == 0 &&
            ((reinterpret_cast<uintptr_t>(g.residual) | reinterpret_cast<uintptr_t>(g.y_out)) & 15) == 0) {
#pragma unroll
          for (int j = 0; j < TO; j += 4) {
            const float4 r4 = __ldcs(reinterpret_cast<const float4*>(rs + j));  // the residual is read once
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
              y[j] = __fadd_rn(y[j], rs[j]);
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

// ---- host side -----------------------------------------------------------------------------------

int g_conv_variant = 0;
int g_conv_tile = 0;

template <int BP, int BO, int TP, int TO, int MINB, int EPI, bool CSA, bool VEC16, int STAGES>
dabnn_status launch_one(const BConvArgs& g, cudaStream_t st) {
  constexpr int THREADS = (BP / TP) * (BO / TO);
  constexpr size_t SMEM = (size_t)STAGES * (BP + BO) * PITCH * 4 + (size_t)BP * sizeof(RowInfo);
  auto kern = bconv_kernel<BP, BO, TP, TO, MINB, EPI, CSA, VEC16, STAGES>;
  static bool configured = false;  // one attribute call per instantiation (idempotent if raced)
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    configured = true;
  }
  const long long gx = (g.M + BP - 1) / BP;
  const int ochan = (EPI == EPI_I32) ? g.O : g.Ow32 * 32;
  const int gy = (ochan + BO - 1) / BO;
  if (gx > 0x7FFFFFFF || gy > 65535) return DABNN_ERR_UNSUPPORTED;
  launch_chain(kern, dim3((unsigned)gx, (unsigned)gy), dim3(THREADS), (size_t)SMEM, st, g);
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
    if (ochan > 64 && ctas(128, 128) >= 2LL * sms) tile = 1;
    else if (ctas(128, 64) >= 4LL * sms) tile = 2;
    else if (ctas(64, 64) >= 2LL * sms) tile = 3;
    else if (ctas(32, 32) >= sms || g.K64 > 5 * KC64) tile = 4;
    else tile = 5;  // less than one wave of the smallest tile: latency is all that counts
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

dabnn_status fill_args(BConvArgs& g, const uint64_t* a, dabnn_shape in, const uint64_t* w, int O, dabnn_conv cv) {
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
  return DABNN_OK;
}

}  // namespace

int sm_count() {
  static int cached = 0;
  if (cached == 0) {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) {
      cudaGetLastError();
      return 148;
    }
    cached = n;
  }
  return cached;
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
