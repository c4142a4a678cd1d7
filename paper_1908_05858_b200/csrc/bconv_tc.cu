// Binary convolution on the 5th-generation tensor cores (tcgen05, kind::i8) -- the same integers as the xor/popcount
// kernel (Section 2.1.2, Eq. 1 of the paper, read as a +-1 dot product), computed as a dense int8 contraction.
//
// sm_100a has no native 1-bit MMA (mma.sync ... b1 is emulated and tcgen05 has no 1-bit kind), so the +-1 values
// are expanded to int8 on chip: HBM still holds one bit per activation and per weight use.
//
//   * Weights: expanded once (dabnn_tc_prepare_weights) to int8 {+1,-1} in the UMMA K-major, no-swizzle core-matrix
//     layout, one contiguous block per tile of NT output channels; a persistent CTA copies its block to shared
//     memory once and keeps it for all its pixel tiles.
//   * Activations: a tile is 128 consecutive "slots" q of the padded image grid (slot pitch SP = W + 2*pad_w,
//     H + 2*pad_h slot rows per image).  The CTA reads the packed bits of the 128 + (kh-1)*SP + (kw-1) slots it
//     needs, expands them to int8 rows of 16 channels ([C/16][slots][16 B]) -- padded slots get the declared pad
//     value -- and every filter tap (i, j) is the SAME array read from a start address shifted by (i*SP + j) rows:
//     with a 16-byte row pitch a shift by one slot is a 16-byte step of the matrix descriptor, so no im2col copy
//     is ever materialised.  Rows that fall on padding columns / rows compute garbage that is never stored.
//   * One thread issues kh*kw*(C/32) tcgen05.mma (M = 128, N = NT, K = 32) per tile into a TMEM accumulator
//     (two buffers), commits to an mbarrier, and the CTA's warps read the previous tile's accumulator with
//     tcgen05.ld while the tensor core works on the current one.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records an error flag, skips the remaining work,
// frees its TMEM and returns.
#include "common.cuh"

namespace dabnn {

namespace {

enum { EPI_I32 = 0, EPI_BNPACK = 1, EPI_BIREAL = 2 };

constexpr int TC_THREADS = 256;
constexpr int TC_SMEM_LIMIT = 232448;     // 227 KB opt-in maximum per CTA
constexpr int TC_SMEM_MISC = 1024;        // barriers, TMEM base, alignment slack
constexpr int TC_WEIGHT_BUDGET = 147456;  // 144 KB of resident weights at most

__device__ int g_tc_error = 0;  // 1: an mbarrier wait ran out

struct TcArgs {
  const uint64_t* a;
  const uint8_t* w_tc;
  int N, H, W, Cw, C;
  int O, kh, kw, ph, pw, OH, OW;
  int SP, HP;          // slot pitch and slot rows per image
  long long total_q;   // N * HP * SP
  int slots;           // slots per tile, multiple of 8
  int ntile, n_ntiles; // output channels per tile, number of channel tiles
  long long m_tiles;
  int pad_neg;
  int32_t* out;
  int out_nchw;
  const float* scale;
  const float* shift;
  const float* residual;
  float* y_out;
  uint32_t* out_packed32;
  int Ow32;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

// Bounded wait for the given phase parity; false if it ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
  for (int tries = 0; tries < (1 << 22); tries++) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 0x10000;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
  }
  return false;
}

// 64-bit shared-memory matrix descriptor: K-major, no swizzle.  Core matrix = 8 rows x 16 bytes, rows 16 bytes
// apart; `sbo` = bytes between core matrices along M/N, `lbo` = bytes between the two core matrices along K.
__device__ __forceinline__ uint64_t make_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr >> 4) & 0x3FFF);
  d |= (uint64_t)((lbo >> 4) & 0x3FFF) << 16;
  d |= (uint64_t)((sbo >> 4) & 0x3FFF) << 32;
  d |= (uint64_t)1 << 46;  // descriptor version for this architecture
  return d;                // base offset 0, layout type 0 (no swizzle)
}

// 16 sign bits -> 16 bytes of {+1 (bit 0), -1 (bit 1)}.
__device__ __forceinline__ uint32_t expand4(uint32_t nib) {
  const uint32_t t = (nib * 0x00204081u) & 0x01010101u;  // bit k of the nibble -> byte k
  return (t * 0xFFu) | 0x01010101u;                      // 1 -> 0xFF (-1), 0 -> 0x01 (+1)
}
__device__ __forceinline__ uint4 expand16(uint32_t bits) {
  return make_uint4(expand4(bits & 0xF), expand4((bits >> 4) & 0xF), expand4((bits >> 8) & 0xF),
                    expand4((bits >> 12) & 0xF));
}

template <int NT, int EPI>
__global__ void __launch_bounds__(TC_THREADS, 1) bconv_tc_kernel(const TcArgs g) {
  extern __shared__ __align__(1024) uint8_t smem[];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = g.kh * g.kw * g.C;  // bytes per weight row
  uint8_t* w_s = smem;                                   // [taps][C/16][NT][16]
  uint8_t* a_s = smem + (size_t)NT * K;                  // [C/16][slots][16]
  uint8_t* misc = a_s + (size_t)g.slots * g.C;
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);    // 2 mbarriers
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 16);
  int* s_fail = reinterpret_cast<int*>(misc + 24);
  constexpr int TMEM_COLS = (2 * NT < 32) ? 32 : 2 * NT;

  const int nt = blockIdx.x % g.n_ntiles;
  const long long mt_first = blockIdx.x / g.n_ntiles;
  const long long mt_step = gridDim.x / g.n_ntiles;

  if (tid == 0) {
    mbar_init(smem_u32(&bars[0]), 1);
    mbar_init(smem_u32(&bars[1]), 1);
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                 "r"((uint32_t)TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // resident weights: one contiguous block per channel tile
  {
    const uint8_t* src = g.w_tc + (size_t)nt * NT * K;
    const int units = NT * K / 16;
    for (int u = tid; u < units; u += TC_THREADS) cp_async16(smem_u32(w_s + (size_t)u * 16), src + (size_t)u * 16);
    asm volatile("cp.async.commit_group;" ::: "memory");
    asm volatile("cp.async.wait_group 0;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  const uint32_t idesc = (2u << 4)                      // accumulator: s32
                         | (1u << 7) | (1u << 10)       // A, B: signed 8-bit
                         | ((uint32_t)(NT >> 3) << 17)  // N
                         | ((uint32_t)(128 >> 4) << 24);  // M = 128; both operands K-major
  const int cgroups = g.C >> 4;  // 16-channel groups
  const uint32_t a_lbo = (uint32_t)g.slots * 16, w_lbo = (uint32_t)NT * 16;
  const uint32_t pad_word4 = g.pad_neg ? 0xFFFFFFFFu : 0x01010101u;

  // ---- epilogue of one finished tile --------------------------------------------------------------------------
  auto epilogue = [&](long long mt, int buf) {
    const int row = 32 * (warp & 3) + lane;      // TMEM lane = slot row of the tile
    const int half = warp >> 2;                  // which half of the NT columns this warp reads
    constexpr int COLS = NT / 2;                 // columns per warp
    const long long Q = mt * 128 + row;
    const int col = (int)(Q % g.SP);
    const long long rr = Q / g.SP;
    const int r = (int)(rr % g.HP);
    const long long n = rr / g.HP;
    const bool valid = n < g.N && r < g.OH && col < g.OW;
    const long long m = (n * g.OH + r) * g.OW + col;
    const int o_base = nt * NT + half * COLS;
#pragma unroll
    for (int c0 = 0; c0 < COLS; c0 += 16) {
      uint32_t v[16];
      const uint32_t taddr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(buf * NT + half * COLS + c0);
      asm volatile(
          "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
          : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
            "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
          : "r"(taddr));
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
      const int o = o_base + c0;
      if (!valid) continue;
      if (EPI == EPI_I32 ? (o >= g.O) : (o >= g.Ow32 * 32)) continue;  // sign words are written whole, tail bits 0
      if (EPI == EPI_I32) {
        if (!g.out_nchw) {
          int32_t* dst = g.out + m * g.O + o;
          if (o + 16 <= g.O && (g.O & 3) == 0 && (reinterpret_cast<uintptr_t>(g.out) & 15) == 0) {
#pragma unroll
            for (int j = 0; j < 16; j += 4)
              *reinterpret_cast<int4*>(dst + j) = make_int4((int)v[j], (int)v[j + 1], (int)v[j + 2], (int)v[j + 3]);
          } else {
#pragma unroll
            for (int j = 0; j < 16; j++)
              if (o + j < g.O) dst[j] = (int)v[j];
          }
        } else {
          const long long ohw = (long long)g.OH * g.OW, q = (long long)r * g.OW + col;
#pragma unroll
          for (int j = 0; j < 16; j++)
            if (o + j < g.O) g.out[(n * g.O + o + j) * ohw + q] = (int)v[j];
        }
      } else {
        float y[16];
#pragma unroll
        for (int j = 0; j < 16; j++)
          y[j] = (o + j < g.O) ? __fmaf_rn((float)(int)v[j], g.scale[o + j], g.shift[o + j]) : 0.0f;
        if (EPI == EPI_BIREAL) {
          const float* rs = g.residual + m * g.O + o;
          float* yd = g.y_out + m * g.O + o;
          if (o + 16 <= g.O && (g.O & 3) == 0 &&
              ((reinterpret_cast<uintptr_t>(g.residual) | reinterpret_cast<uintptr_t>(g.y_out)) & 15) == 0) {
#pragma unroll
            for (int j = 0; j < 16; j += 4) {
              const float4 r4 = *reinterpret_cast<const float4*>(rs + j);
              y[j] = __fadd_rn(y[j], r4.x);
              y[j + 1] = __fadd_rn(y[j + 1], r4.y);
              y[j + 2] = __fadd_rn(y[j + 2], r4.z);
              y[j + 3] = __fadd_rn(y[j + 3], r4.w);
              *reinterpret_cast<float4*>(yd + j) = make_float4(y[j], y[j + 1], y[j + 2], y[j + 3]);
            }
          } else {
#pragma unroll
            for (int j = 0; j < 16; j++)
              if (o + j < g.O) {
                y[j] = __fadd_rn(y[j], rs[j]);
                yd[j] = y[j];
              }
          }
        }
        if (g.out_packed32 != nullptr) {
          uint32_t field = 0;
#pragma unroll
          for (int j = 0; j < 16; j++) field |= (uint32_t)((o + j < g.O) && (y[j] < 0.0f)) << j;
          // 16 channels = half of a 32-bit sign word
          reinterpret_cast<uint16_t*>(g.out_packed32)[(m * g.Ow32 + (o >> 5)) * 2 + ((o >> 4) & 1)] = (uint16_t)field;
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  };

  int it = 0;
  long long prev_mt = -1;
  bool failed = false;
  for (long long mt = mt_first; mt < g.m_tiles; mt += mt_step, it++) {
    if (it > 0) {
      // the previous tile's MMAs must be complete before its A rows are overwritten
      if (!mbar_wait(smem_u32(&bars[(it - 1) & 1]), ((it - 1) >> 1) & 1)) *s_fail = 1;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    // ---- expand this tile's slots: bits -> int8 rows ------------------------------------------------------------
    const long long q0 = mt * 128;
    for (int s = tid; s < g.slots; s += TC_THREADS) {
      const long long Q = q0 + s;
      const int col = (int)(Q % g.SP);
      const long long rr = Q / g.SP;
      const int r = (int)(rr % g.HP);
      const long long n = rr / g.HP;
      const int ih = r - g.ph, iw = col - g.pw;
      const bool beyond = n >= g.N;
      const bool inside = !beyond && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W;
      const uint64_t* src = g.a + ((n * g.H + ih) * g.W + iw) * g.Cw;
      for (int cw = 0; cw < g.Cw; cw++) {
        uint64_t word = 0;
        if (inside) word = src[cw];
#pragma unroll
        for (int q4 = 0; q4 < 4; q4++) {
          const int grp = cw * 4 + q4;
          if (grp >= cgroups) break;
          uint4 bytes;
          if (inside) bytes = expand16((uint32_t)(word >> (16 * q4)) & 0xFFFFu);
          else if (beyond) bytes = make_uint4(0, 0, 0, 0);
          else bytes = make_uint4(pad_word4, pad_word4, pad_word4, pad_word4);
          *reinterpret_cast<uint4*>(a_s + ((size_t)grp * g.slots + s) * 16) = bytes;
        }
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    failed = *s_fail != 0;
    if (failed) break;
    if (tid == 0) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const uint32_t d_tmem = tmem_base + (uint32_t)((it & 1) * NT);
      const uint32_t a_base = smem_u32(a_s), w_base = smem_u32(w_s);
      uint32_t accumulate = 0;
      for (int ti = 0; ti < g.kh; ti++)
        for (int tj = 0; tj < g.kw; tj++) {
          const int tap = ti * g.kw + tj;
          const uint32_t shift = (uint32_t)(ti * g.SP + tj);
          for (int kb = 0; kb < (g.C >> 5); kb++) {
            const uint64_t adesc = make_desc(a_base + ((uint32_t)(2 * kb) * g.slots + shift) * 16, a_lbo, 128);
            const uint64_t bdesc = make_desc(w_base + (uint32_t)((tap * cgroups + 2 * kb) * NT) * 16, w_lbo, 128);
            asm volatile(
                "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                "tcgen05.mma.cta_group::1.kind::i8 [%0], %1, %2, %3, p;\n\t}"
                ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
                : "memory");
            accumulate = 1;
          }
        }
      asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                       smem_u32(&bars[it & 1]))
                   : "memory");
    }
    if (it > 0) epilogue(prev_mt, (it - 1) & 1);  // overlaps the tensor core working on this tile
    prev_mt = mt;
  }
  if (!failed && it > 0) {
    if (mbar_wait(smem_u32(&bars[(it - 1) & 1]), ((it - 1) >> 1) & 1)) {
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      epilogue(prev_mt, (it - 1) & 1);
    } else {
      *s_fail = 1;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (*s_fail != 0 && tid == 0) atomicExch(&g_tc_error, 1);
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TMEM_COLS)
                 : "memory");
  }
}

// Weights: packed bits [O][taps][Cw] -> int8 [n_ntiles][taps][C/16][NT][16].
__global__ void tc_prepare_weights_kernel(const uint64_t* __restrict__ wp, int O, int taps, int Cw, int cgroups, int NT,
                                          long long units, uint4* __restrict__ out) {
  const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= units) return;
  const int n = (int)(u % NT);
  long long t = u / NT;
  const int grp = (int)(t % cgroups);
  t /= cgroups;
  const int tap = (int)(t % taps);
  const int nt = (int)(t / taps);
  const int o = nt * NT + n;
  uint4 bytes = make_uint4(0, 0, 0, 0);  // channels beyond O contribute nothing
  if (o < O) {
    const uint64_t word = wp[((long long)o * taps + tap) * Cw + (grp >> 2)];
    bytes = expand16((uint32_t)(word >> (16 * (grp & 3))) & 0xFFFFu);
  }
  out[u] = bytes;
}

int tc_ntile(int O, int C, int taps) {
  const long long K = (long long)C * taps;
  for (int nt = 128; nt >= 32; nt >>= 1) {
    if (nt * K > TC_WEIGHT_BUDGET) continue;
    if (nt > 32 && nt / 2 >= O) continue;  // do not pad a small O to a wide tile
    return nt;
  }
  return 0;
}

// Channel tiles cover O rounded up to whole 64-bit sign words (rows beyond O hold zero weights).
int tc_n_ntiles(int O, int nt) { return ((O + 63) / 64 * 64 + nt - 1) / nt; }

template <int NT, int EPI>
dabnn_status tc_launch(const TcArgs& g, size_t smem, cudaStream_t st) {
  auto kern = bconv_tc_kernel<NT, EPI>;
  static bool configured = false;
  if (!configured) {
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_LIMIT) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    configured = true;
  }
  long long ctas = (long long)g.n_ntiles * g.m_tiles;
  const long long cap = (long long)sm_count() / g.n_ntiles * g.n_ntiles;
  if (cap <= 0) return DABNN_ERR_UNSUPPORTED;
  if (ctas > cap) ctas = cap;
  kern<<<(unsigned)ctas, TC_THREADS, smem, st>>>(g);
  return launch_status();
}

template <int EPI>
dabnn_status tc_dispatch(TcArgs& g, cudaStream_t st) {
  const size_t smem = (size_t)g.ntile * g.kh * g.kw * g.C + (size_t)g.slots * g.C + TC_SMEM_MISC;
  if (smem > (size_t)TC_SMEM_LIMIT) return DABNN_ERR_UNSUPPORTED;
  switch (g.ntile) {
    case 128: return tc_launch<128, EPI>(g, smem, st);
    case 64: return tc_launch<64, EPI>(g, smem, st);
    case 32: return tc_launch<32, EPI>(g, smem, st);
  }
  return DABNN_ERR_UNSUPPORTED;
}

dabnn_status tc_fill(TcArgs& g, const uint64_t* a, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv) {
  if (!a || !w_tc) return DABNN_ERR_NULL;
  if (in.N <= 0 || in.C <= 0 || in.H <= 0 || in.W <= 0 || O <= 0) return DABNN_ERR_SHAPE;
  if (cv.kh <= 0 || cv.kw <= 0 || cv.stride_h <= 0 || cv.stride_w <= 0 || cv.pad_h < 0 || cv.pad_w < 0)
    return DABNN_ERR_SHAPE;
  if (cv.pad_value != 1 && cv.pad_value != -1) return DABNN_ERR_SHAPE;
  if (!aligned(a, 8) || !aligned(w_tc, 16)) return DABNN_ERR_ALIGNMENT;
  const int OH = dabnn_out_dim(in.H, cv.kh, cv.stride_h, cv.pad_h), OW = dabnn_out_dim(in.W, cv.kw, cv.stride_w, cv.pad_w);
  if (OH <= 0 || OW <= 0) return DABNN_ERR_SHAPE;
  // what this engine covers; everything else is served by the xor/popcount kernel
  if (cv.stride_h != 1 || cv.stride_w != 1 || in.C % 32 != 0) return DABNN_ERR_UNSUPPORTED;
  const int nt = tc_ntile(O, in.C, cv.kh * cv.kw);
  if (nt == 0) return DABNN_ERR_UNSUPPORTED;
  g.a = a; g.w_tc = static_cast<const uint8_t*>(w_tc);
  g.N = in.N; g.H = in.H; g.W = in.W; g.Cw = (in.C + 63) / 64; g.C = in.C;
  g.O = O; g.kh = cv.kh; g.kw = cv.kw; g.ph = cv.pad_h; g.pw = cv.pad_w; g.OH = OH; g.OW = OW;
  g.SP = in.W + 2 * cv.pad_w; g.HP = in.H + 2 * cv.pad_h;
  g.total_q = (long long)in.N * g.HP * g.SP;
  g.slots = (128 + (cv.kh - 1) * g.SP + (cv.kw - 1) + 7) / 8 * 8;
  if (g.slots > 16383) return DABNN_ERR_UNSUPPORTED;
  g.ntile = nt; g.n_ntiles = tc_n_ntiles(O, nt);
  g.m_tiles = (g.total_q + 127) / 128;
  if ((long long)in.N * OH * OW * O > (1LL << 40)) return DABNN_ERR_UNSUPPORTED;
  g.pad_neg = cv.pad_value < 0;
  g.out = nullptr; g.out_nchw = 0; g.scale = g.shift = g.residual = nullptr; g.y_out = nullptr;
  g.out_packed32 = nullptr; g.Ow32 = 2 * ((O + 63) / 64);
  return DABNN_OK;
}

}  // namespace

}  // namespace dabnn

using namespace dabnn;

extern "C" size_t dabnn_tc_weights_bytes(int O, int C, int kh, int kw) {
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0 || C % 32 != 0) return 0;
  const int nt = tc_ntile(O, C, kh * kw);
  if (nt == 0) return 0;
  return (size_t)tc_n_ntiles(O, nt) * nt * kh * kw * C;
}

extern "C" dabnn_status dabnn_tc_prepare_weights(const uint64_t* w_packed, int O, int C, int kh, int kw, void* w_tc,
                                                 void* stream) {
  if (!w_packed || !w_tc) return DABNN_ERR_NULL;
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0) return DABNN_ERR_SHAPE;
  if (C % 32 != 0) return DABNN_ERR_UNSUPPORTED;
  if (!aligned(w_packed, 8) || !aligned(w_tc, 16)) return DABNN_ERR_ALIGNMENT;
  const int nt = tc_ntile(O, C, kh * kw);
  if (nt == 0) return DABNN_ERR_UNSUPPORTED;
  const int taps = kh * kw, cgroups = C / 16, n_nt = tc_n_ntiles(O, nt);
  const long long units = (long long)n_nt * taps * cgroups * nt;
  tc_prepare_weights_kernel<<<ceil_div(units, 256), 256, 0, as_stream(stream)>>>(w_packed, O, taps, (C + 63) / 64, cgroups,
                                                                                 nt, units, static_cast<uint4*>(w_tc));
  return launch_status();
}

extern "C" dabnn_status dabnn_tc_bconv2d(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                                         int32_t* out, dabnn_layout out_layout, void* stream) {
  TcArgs g;
  dabnn_status s = tc_fill(g, a_packed, in, w_tc, O, cv);
  if (s != DABNN_OK) return s;
  if (!out) return DABNN_ERR_NULL;
  if (out_layout != DABNN_NCHW && out_layout != DABNN_NHWC) return DABNN_ERR_SHAPE;
  if (!aligned(out, 4)) return DABNN_ERR_ALIGNMENT;
  g.out = out;
  g.out_nchw = out_layout == DABNN_NCHW;
  return tc_dispatch<EPI_I32>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_tc_bconv2d_bn_sign_pack(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O,
                                                      dabnn_conv cv, const float* scale, const float* shift,
                                                      uint64_t* out_packed, void* stream) {
  TcArgs g;
  dabnn_status s = tc_fill(g, a_packed, in, w_tc, O, cv);
  if (s != DABNN_OK) return s;
  if (!scale || !shift || !out_packed) return DABNN_ERR_NULL;
  if (!aligned(scale, 4) || !aligned(shift, 4) || !aligned(out_packed, 8)) return DABNN_ERR_ALIGNMENT;
  g.scale = scale; g.shift = shift;
  g.out_packed32 = reinterpret_cast<uint32_t*>(out_packed);
  return tc_dispatch<EPI_BNPACK>(g, as_stream(stream));
}

extern "C" dabnn_status dabnn_tc_bconv2d_bn_add_sign_pack(const uint64_t* a_packed, dabnn_shape in, const void* w_tc,
                                                          int O, dabnn_conv cv, const float* scale, const float* shift,
                                                          const float* residual, float* y_out, uint64_t* out_packed,
                                                          void* stream) {
  TcArgs g;
  dabnn_status s = tc_fill(g, a_packed, in, w_tc, O, cv);
  if (s != DABNN_OK) return s;
  if (!scale || !shift || !residual || !y_out) return DABNN_ERR_NULL;
  if (!aligned(scale, 4) || !aligned(shift, 4) || !aligned(residual, 4) || !aligned(y_out, 4) || !aligned(out_packed, 8))
    return DABNN_ERR_ALIGNMENT;
  g.scale = scale; g.shift = shift; g.residual = residual; g.y_out = y_out;
  g.out_packed32 = reinterpret_cast<uint32_t*>(out_packed);
  return tc_dispatch<EPI_BIREAL>(g, as_stream(stream));
}

extern "C" int dabnn_tc_error_flag(void) {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}
