// Bi-Real Net 18 forward (Section 2.3, Table 2 of the paper): fp32 stem and head around sixteen binary
// 3x3 convolutions whose BN + shortcut + sign + re-pack run in the convolution's epilogue.
//
// All activations between layers are NHWC.  Every fp32 value is produced by single IEEE-rounded
// operations in a fixed order (explicit fmaf chains, ascending channel / tap order), never by tensor
// cores or split sums, because the next binary layer takes the SIGN of these values: a different
// rounding order could flip a bit and change integer results downstream.
#include <mutex>

#include "common.cuh"

namespace dabnn {

thread_local bool g_chain_launch = false;  // see launch_chain() in common.cuh

namespace {

// ---- BN fold, in double ---------------------------------------------------------------------------
__global__ void bn_fold_kernel(const float* gamma, const float* beta, const float* mean, const float* var, double eps,
                               int O, float* scale, float* shift) {
  const int o = blockIdx.x * blockDim.x + threadIdx.x;
  if (o >= O) return;
  const double sd = __ddiv_rn((double)gamma[o], __dsqrt_rn(__dadd_rn((double)var[o], eps)));
  scale[o] = (float)sd;
  shift[o] = (float)__dsub_rn((double)beta[o], __dmul_rn((double)mean[o], sd));
}

// ---- stem: conv 7x7 / 2, 3 -> 64, zero pad 3, then BN ----------------------------------------------
// A CTA computes a TS x TS tile of output pixels for 4 * CPT channels (all 64 with CPT = 16; with CPT = 8 two CTAs
// share a tile, which spreads a single image over twice as many CTAs).  The input patch sits in shared
// memory with even and odd columns apart, so that lanes walking along ow (input stride 2) read
// consecutive words.  A thread owns PPT pixels (rows TS/PPT apart... see below) x CPT channels and runs one fmaf
// chain per output over (c, kh, kw) in that order.  Zero padding is held as zeros in the patch:
// fmaf(0, w, acc) returns acc.
constexpr int STEM_K = 147;
// Columns per parity of the input patch, padded: the lanes of a warp read 8 consecutive columns of 4 patch rows that
// are two rows (4 * half words) apart, which fall on distinct banks when 4 * half is 8 or 24 modulo 32.
__host__ __device__ constexpr int stem_half(int ps) {
  int h = (ps + 1) / 2 + 1;
  while ((4 * h) % 32 != 8 && (4 * h) % 32 != 24) h++;
  return h;
}

// Two fp32 fused multiply-adds in one instruction (fma.rn.f32x2): each lane of the pair is the same correctly rounded
// fmaf as the scalar instruction, so results do not change; it halves the issue slots of an FMA-bound loop.
__device__ __forceinline__ unsigned long long pack_f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ void unpack_f32x2(unsigned long long v, float& lo, float& hi) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ void fma_f32x2(unsigned long long& acc, unsigned long long a, unsigned long long b) {
  asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(acc) : "l"(a), "l"(b));
}

template <int TS, int PPT, int CPT>
__global__ void __launch_bounds__((TS * TS / PPT) * 4, 2) stem_conv_bn(const float* __restrict__ img,
                                                                       const float* __restrict__ w,
                                                                       const float* __restrict__ scale,
                                                                       const float* __restrict__ shift, int N,
                                                                       float* __restrict__ out /*[N][112][112][64]*/) {
  constexpr int IH = 224, IW = 224, OHW = 112;
  constexpr int PS = 2 * TS + 5;         // patch side
  constexpr int HALF = stem_half(PS);
  constexpr int PATCH = 3 * PS * 2 * HALF;  // floats per patch buffer
  constexpr int PGROUPS = TS * TS / PPT; // pixel groups = threads per channel group
  constexpr int THREADS = PGROUPS * 4;
  constexpr int RSTEP = TS / PPT;        // a thread's pixels are RSTEP rows apart
  constexpr int TILES = (OHW + TS - 1) / TS;
  constexpr int CB = 4 * CPT;            // channels per CTA (blockIdx.y picks which): four thread groups of CPT channels
  static_assert(CPT == 16 || CPT == 8, "channels per thread");
  extern __shared__ __align__(16) float sm[];
  float* w_s = sm;                       // [147][CB], filled once per CTA
  float* x_s = sm + STEM_K * CB;         // [2 buffers][3][PS][2][HALF]
  float* w_raw = x_s + 2 * PATCH;        // [CB][147] as in global memory, until it has been transposed into w_s
  const int ch0 = blockIdx.y * CB;
  w += (size_t)ch0 * STEM_K;             // this CTA's rows of the [64][147] weight matrix
  const int tid = threadIdx.x;
  if ((reinterpret_cast<uintptr_t>(w) & 15) == 0) {  // one coalesced asynchronous copy, in flight together with the first patch
    for (int t = tid; t < STEM_K * CB / 4; t += THREADS) {
      const uint32_t d = (uint32_t)__cvta_generic_to_shared(w_raw + 4 * t);
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(w + 4 * t) : "memory");
    }
  } else {
    for (int t = tid; t < STEM_K * CB; t += THREADS) w_raw[t] = w[t];
  }
  const long long ntiles = (long long)N * TILES * TILES;
  // asynchronous copy of one tile's zero-padded input patch (even and odd columns apart)
  auto load_patch = [&](long long tile, float* dst) {
    const int n = (int)(tile / (TILES * TILES));
    const int rem = (int)(tile % (TILES * TILES));
    const int ih_base = 2 * (rem / TILES) * TS - 3, iw_base = 2 * (rem % TILES) * TS - 3;
    for (int t = tid; t < 3 * PS * PS; t += THREADS) {
      const int lw = t % PS, lh = (t / PS) % PS, c = t / (PS * PS);
      const int ih = ih_base + lh, iw = iw_base + lw;
      const bool in = ih >= 0 && ih < IH && iw >= 0 && iw < IW;
      const float* src = in ? img + (((size_t)n * 3 + c) * IH + ih) * IW + iw : img;
      const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + ((c * PS + lh) * 2 + (lw & 1)) * HALF + (lw >> 1));
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(in ? 4 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const int cg = tid / PGROUPS;          // channel group: 16 channels
  const int pg = tid % PGROUPS;
  const int low = pg % TS, lohb = pg / TS;  // pixels (lohb + RSTEP*i, low)
  float sc[CPT], sf[CPT];
#pragma unroll
  for (int j = 0; j < CPT; j++) {
    sc[j] = scale[ch0 + cg * CPT + j];
    sf[j] = shift[ch0 + cg * CPT + j];
  }
  long long tile = blockIdx.x;
  int buf = 0;
  if (tile < ntiles) load_patch(tile, x_s);
  asm volatile("cp.async.wait_all;" ::: "memory");
  __syncthreads();
  // [CB][147] -> [147][CB]: lanes walk over o, 147 words apart in w_raw (an odd stride: distinct banks) and consecutive in w_s
  for (int t = tid; t < STEM_K * CB; t += THREADS) w_s[t] = w_raw[(t % CB) * STEM_K + t / CB];
  for (; tile < ntiles; tile += gridDim.x, buf ^= 1) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();  // this tile's patch (and, the first time, the weights) are in place; the other buffer is free
    if (tile + gridDim.x < ntiles) load_patch(tile + gridDim.x, x_s + (buf ^ 1) * PATCH);
    const float* xb = x_s + buf * PATCH;
    unsigned long long acc2[PPT][CPT / 2];  // channel pairs (packed fp32 FMAs, same rounding as scalar fmaf)
#pragma unroll
    for (int i = 0; i < PPT; i++)
#pragma unroll
      for (int j = 0; j < CPT / 2; j++) acc2[i][j] = 0ull;
#pragma unroll 1
    for (int c = 0; c < 3; c++)
#pragma unroll 1
      for (int ki = 0; ki < 7; ki++) {  // one row of taps per iteration keeps the loop body inside the instruction cache
#pragma unroll
        for (int kj = 0; kj < 7; kj++) {
          const int k = (c * 7 + ki) * 7 + kj;
          unsigned long long w2[CPT / 2];
#pragma unroll
          for (int q = 0; q < CPT / 4; q++) {
            const float4 t4 = *reinterpret_cast<const float4*>(w_s + k * CB + cg * CPT + 4 * q);
            w2[2 * q] = pack_f32x2(t4.x, t4.y);
            w2[2 * q + 1] = pack_f32x2(t4.z, t4.w);
          }
#pragma unroll
          for (int i = 0; i < PPT; i++) {
            const int lh = 2 * (lohb + RSTEP * i) + ki;
            const float xv = xb[((c * PS + lh) * 2 + (kj & 1)) * HALF + low + (kj >> 1)];
            const unsigned long long x2 = pack_f32x2(xv, xv);
#pragma unroll
            for (int j = 0; j < CPT / 2; j++) fma_f32x2(acc2[i][j], x2, w2[j]);
          }
        }
      }
    float acc[PPT][CPT];
#pragma unroll
    for (int i = 0; i < PPT; i++)
#pragma unroll
      for (int j = 0; j < CPT / 2; j++) unpack_f32x2(acc2[i][j], acc[i][2 * j], acc[i][2 * j + 1]);
    if (tile + gridDim.x >= ntiles) chain_trigger();  // the CTA's last tile: the next kernel may start its set-up
    const int n = (int)(tile / (TILES * TILES));
    const int rem = (int)(tile % (TILES * TILES));
    const int oh0 = (rem / TILES) * TS, ow0 = (rem % TILES) * TS;
#pragma unroll
    for (int i = 0; i < PPT; i++) {
      const int oh = oh0 + lohb + RSTEP * i, ow = ow0 + low;
      if (oh >= OHW || ow >= OHW) continue;
      float* dst = out + (((size_t)n * OHW + oh) * OHW + ow) * 64 + ch0 + cg * CPT;
#pragma unroll
      for (int j = 0; j < CPT; j += 4)
        *reinterpret_cast<float4*>(dst + j) =
            make_float4(__fmaf_rn(acc[i][j], sc[j], sf[j]), __fmaf_rn(acc[i][j + 1], sc[j + 1], sf[j + 1]),
                        __fmaf_rn(acc[i][j + 2], sc[j + 2], sf[j + 2]), __fmaf_rn(acc[i][j + 3], sc[j + 3], sf[j + 3]));
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// Large batches: the same convolution with an 8 pixels (along a row) x 8 channels register tile.  Per (c, kh) a thread
// loads the 21 input values its 8 pixels need (even and odd columns as 3 + 3 float4) once and reuses them for all 7
// horizontal taps; per tap it loads 8 weights.  Persistent CTAs as above; the order of every output's fmaf chain is
// unchanged: c, then kh, then kw.
__global__ void __launch_bounds__(256, 2) stem_conv_bn_8x8(const float* __restrict__ img, const float* __restrict__ w,
                                                           const float* __restrict__ scale,
                                                           const float* __restrict__ shift, int N,
                                                           float* __restrict__ out /*[N][112][112][64]*/) {
  chain_trigger();  // (a chained successor may set itself up as this grid drains; it waits for all of it before reading)
  constexpr int TS = 16, IH = 224, IW = 224, OHW = 112;
  constexpr int PS = 2 * TS + 5;         // 37
  constexpr int HALF = 20;               // columns per parity (19 / 18 used), a multiple of 4
  constexpr int PATCH = 3 * PS * 2 * HALF;
  constexpr int THREADS = 256;
  constexpr int TILES = OHW / TS;        // 7
  extern __shared__ __align__(16) float sm[];
  float* w_s = sm;                       // [147][64]
  float* x_s = sm + STEM_K * 64;         // [2 buffers][3][PS][2][HALF]
  const int tid = threadIdx.x;
  for (int t = tid; t < STEM_K * 64; t += THREADS) {
    const int o = t % 64, k = t / 64;
    w_s[k * 64 + o] = w[o * STEM_K + k];
  }
  const long long ntiles = (long long)N * TILES * TILES;
  auto load_patch = [&](long long tile, float* dst) {
    const int n = (int)(tile / (TILES * TILES));
    const int rem = (int)(tile % (TILES * TILES));
    const int ih_base = 2 * (rem / TILES) * TS - 3, iw_base = 2 * (rem % TILES) * TS - 3;
    for (int t = tid; t < 3 * PS * 2 * HALF; t += THREADS) {  // every word of the buffer, padding columns included
      const int hc = t % HALF, par = (t / HALF) % 2, lh = (t / (2 * HALF)) % PS, c = t / (2 * HALF * PS);
      const int lw = 2 * hc + par;
      const int ih = ih_base + lh, iw = iw_base + lw;
      const bool in = lw < PS && ih >= 0 && ih < IH && iw >= 0 && iw < IW;
      const float* src = in ? img + (((size_t)n * 3 + c) * IH + ih) * IW + iw : img;
      const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst + t);
      asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(in ? 4 : 0) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  const int chg = tid & 7, pg = tid >> 3;        // 8 channel groups x 32 pixel groups
  const int row = pg >> 1, ow0 = (pg & 1) * 8;   // 8 consecutive pixels of one tile row
  // a thread's 8 channels are chg*4 .. +3 and 32 + chg*4 .. +3, so that the 8 lanes of a quarter-warp read 128 contiguous
  // bytes of weights (no bank conflict) and write 128 contiguous bytes of output
  float sc[8], sf[8];
#pragma unroll
  for (int j = 0; j < 8; j++) {
    const int ch = (j < 4) ? chg * 4 + j : 32 + chg * 4 + (j - 4);
    sc[j] = scale[ch];
    sf[j] = shift[ch];
  }
  long long tile = blockIdx.x;
  int buf = 0;
  if (tile < ntiles) load_patch(tile, x_s);
  for (; tile < ntiles; tile += gridDim.x, buf ^= 1) {
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();
    if (tile + gridDim.x < ntiles) load_patch(tile + gridDim.x, x_s + (buf ^ 1) * PATCH);
    const float* xb = x_s + buf * PATCH;
    unsigned long long acc2[8][4];  // channel pairs (0,1) (2,3) (4,5) (6,7) of each pixel
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) acc2[i][j] = 0ull;  // (+0.0, +0.0)
#pragma unroll 1
    for (int c = 0; c < 3; c++)
#pragma unroll 1
      for (int ki = 0; ki < 7; ki++) {
        const float* xr = xb + ((c * PS + 2 * row + ki) * 2) * HALF + ow0;
        float xe[12], xo[12];  // even / odd input columns 2*(ow0 + t), 2*(ow0 + t) + 1
#pragma unroll
        for (int q = 0; q < 3; q++) {
          const float4 e4 = *reinterpret_cast<const float4*>(xr + 4 * q);
          const float4 o4 = *reinterpret_cast<const float4*>(xr + HALF + 4 * q);
          xe[4 * q] = e4.x; xe[4 * q + 1] = e4.y; xe[4 * q + 2] = e4.z; xe[4 * q + 3] = e4.w;
          xo[4 * q] = o4.x; xo[4 * q + 1] = o4.y; xo[4 * q + 2] = o4.z; xo[4 * q + 3] = o4.w;
        }
        const float* wk = w_s + ((c * 7 + ki) * 7) * 64 + chg * 4;
#pragma unroll
        for (int kj = 0; kj < 7; kj++) {
          const float4 wa = *reinterpret_cast<const float4*>(wk + kj * 64);
          const float4 wb = *reinterpret_cast<const float4*>(wk + kj * 64 + 32);
          const unsigned long long w2[4] = {pack_f32x2(wa.x, wa.y), pack_f32x2(wa.z, wa.w), pack_f32x2(wb.x, wb.y),
                                            pack_f32x2(wb.z, wb.w)};
#pragma unroll
          for (int i = 0; i < 8; i++) {
            const float xv = (kj & 1) ? xo[i + (kj >> 1)] : xe[i + (kj >> 1)];
            const unsigned long long x2 = pack_f32x2(xv, xv);
#pragma unroll
            for (int j = 0; j < 4; j++) fma_f32x2(acc2[i][j], x2, w2[j]);
          }
        }
      }
    float acc[8][8];
#pragma unroll
    for (int i = 0; i < 8; i++)
#pragma unroll
      for (int j = 0; j < 4; j++) unpack_f32x2(acc2[i][j], acc[i][2 * j], acc[i][2 * j + 1]);
    const int n = (int)(tile / (TILES * TILES));
    const int rem = (int)(tile % (TILES * TILES));
    const int oh = (rem / TILES) * TS + row, owb = (rem % TILES) * TS + ow0;
#pragma unroll
    for (int i = 0; i < 8; i++) {
      float* dst = out + (((size_t)n * OHW + oh) * OHW + owb + i) * 64 + chg * 4;
      *reinterpret_cast<float4*>(dst) = make_float4(__fmaf_rn(acc[i][0], sc[0], sf[0]), __fmaf_rn(acc[i][1], sc[1], sf[1]),
                                                    __fmaf_rn(acc[i][2], sc[2], sf[2]), __fmaf_rn(acc[i][3], sc[3], sf[3]));
      *reinterpret_cast<float4*>(dst + 32) = make_float4(__fmaf_rn(acc[i][4], sc[4], sf[4]), __fmaf_rn(acc[i][5], sc[5], sf[5]),
                                                        __fmaf_rn(acc[i][6], sc[6], sf[6]), __fmaf_rn(acc[i][7], sc[7], sf[7]));
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// In the kernels that take part in chained launches, the pointer to the ACTIVATIONS (what the previous kernel of the stream
// wrote) is deliberately neither __restrict__ nor read with __ldg: such loads count as invariant and the compiler may move
// them above the wait for the previous kernel (seen in a trial that chained the fc kernel: it read pooled values before
// they were written).  Where the read-only path matters, ld_nc_f4 (volatile asm) keeps the load behind the wait.
// ---- maxpool 3x3 / 2, pad 1 (64 channels) -> fp32 residual stream + packed signs -------------------
// A thread handles 4 channels of one output pixel; 16 lanes make one 64-bit word.
__global__ void __launch_bounds__(256) maxpool_pack(const float* x /*[N][112][112][64]*/, long long npix,
                                                    float* __restrict__ y /*[N][56][56][64]*/,
                                                    uint64_t* __restrict__ bits /*[N][56][56][1]*/) {
  const long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  const int lane = threadIdx.x & 31;
  const long long pix = t >> 4;
  const int c4 = (int)(t & 15);
  const bool live = pix < npix;
  float4 m = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
  chain_wait();
  chain_trigger();
  if (live) {
    const int ow = (int)(pix % 56), oh = (int)((pix / 56) % 56);
    const long long n = pix / (56 * 56);
#pragma unroll
    for (int i = 0; i < 3; i++)
#pragma unroll
      for (int j = 0; j < 3; j++) {
        const int ih = 2 * oh + i - 1, iw = 2 * ow + j - 1;
        if (ih < 0 || ih >= 112 || iw < 0 || iw >= 112) continue;
        const float4 v = ld_nc_f4(x + ((n * 112 + ih) * 112 + iw) * 64 + c4 * 4);
        m.x = fmaxf(m.x, v.x); m.y = fmaxf(m.y, v.y); m.z = fmaxf(m.z, v.z); m.w = fmaxf(m.w, v.w);
      }
    *reinterpret_cast<float4*>(y + pix * 64 + c4 * 4) = m;
  }
  unsigned nib = 0;
  if (live) nib = (unsigned)(m.x < 0.0f) | ((unsigned)(m.y < 0.0f) << 1) | ((unsigned)(m.z < 0.0f) << 2) | ((unsigned)(m.w < 0.0f) << 3);
  const unsigned gmask = 0xFFu << (lane & 24);
  const unsigned half = __reduce_or_sync(gmask, nib << (4 * (lane & 7)));
  const unsigned other = __shfl_xor_sync(0xFFFFFFFFu, half, 8);
  if (live && (lane & 15) == 0) bits[pix] = (uint64_t)half | ((uint64_t)other << 32);
}

// ---- downsample shortcut: avgpool 2x2 / 2 -> fp32 conv 1x1 (C -> O) -> BN ---------------------------
// A register-tiled matrix product with a fixed summation order: CTA tile BM (64 or 128) output pixels x 128 output
// channels, 256 threads, BM/16 pixels x 8 channels per thread, K (= C) in chunks of 16 through two shared-memory stages.
// The pooled activations are formed on the fly (four loads, three adds, one multiply, in that order) and the weights loaded
// while the previous chunk is being multiplied.  Each output is one fmaf chain over c ascending, as pinned.
constexpr int SC_BM = 128, SC_BN = 128, SC_BK = 16;  // SC_BM: the pixel tile the small-batch crossover below was measured with
template <int BM>
__global__ void __launch_bounds__(256, BM == 128 ? 2 : 3) shortcut_down(const float* __restrict__ x /*[N][HW][HW][C]*/, int HW, int C,
                                                     const float* __restrict__ w /*[O][C]*/, int O,
                                                     const float* __restrict__ scale, const float* __restrict__ shift,
                                                     long long npix_out, float* __restrict__ y /*[N][HW/2][HW/2][O]*/) {
  chain_trigger();  // (as in the stem: lets a chained tensor-engine block start its set-up under this grid's tail)
  constexpr int PV = BM * SC_BK / 256;   // pooled values a thread forms per chunk: 8 or 4 consecutive c of one pixel
  constexpr int TYP = BM / 16;           // pixels per thread in the register tile
  static_assert(BM == 128 || BM == 64, "pixel tile");
  __shared__ __align__(16) float p_s[2][SC_BK][BM + 4];  // [stage][c][pixel]
  __shared__ __align__(16) float w_s[2][SC_BK][SC_BN + 4];  // [stage][c][channel]
  const int tid = threadIdx.x;
  const long long p0 = (long long)blockIdx.x * BM;
  const int o0 = blockIdx.y * SC_BN;
  const int OHW = HW / 2;
  // loader roles: a thread pools PV (pixel, c) pairs per chunk: pixel = tid / (16 / PV), c = (tid % (16 / PV)) * PV .. + PV - 1
  const int lp = tid / (SC_BK / PV), lc = (tid % (SC_BK / PV)) * PV;
  const long long pl = p0 + lp;
  const float* xq = nullptr;
  if (pl < npix_out) {
    const int ow = (int)(pl % OHW), oh = (int)((pl / OHW) % OHW);
    const long long n = pl / ((long long)OHW * OHW);
    xq = x + ((n * HW + 2 * oh) * HW + 2 * ow) * C;
  }
  // weights: 16 c x 128 channels per chunk = 2048 floats: thread copies 8 floats of one channel row: channel = tid / 2
  const int wo = tid >> 1, wc = (tid & 1) * 8;
  const bool c_vec = (C % 8 == 0) && (reinterpret_cast<uintptr_t>(x) % 16 == 0) && (reinterpret_cast<uintptr_t>(w) % 16 == 0);
  float pooled[PV];
  auto pool_load = [&](int c0) {  // registers <- pooled values of chunk c0
#pragma unroll
    for (int k = 0; k < PV; k++) pooled[k] = 0.0f;
    if (xq == nullptr) return;
    const int c = c0 + lc;
    if (c_vec && c + PV <= C) {
      const float4* q00 = reinterpret_cast<const float4*>(xq + c);
      const float4* q01 = reinterpret_cast<const float4*>(xq + C + c);
      const float4* q10 = reinterpret_cast<const float4*>(xq + (size_t)HW * C + c);
      const float4* q11 = reinterpret_cast<const float4*>(xq + (size_t)HW * C + C + c);
#pragma unroll
      for (int h = 0; h < PV / 4; h++) {
        const float4 a = __ldcs(q00 + h), b = __ldcs(q01 + h), cc = __ldcs(q10 + h), d = __ldcs(q11 + h);  // read once
        pooled[4 * h + 0] = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.x, b.x), cc.x), d.x), 0.25f);
        pooled[4 * h + 1] = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.y, b.y), cc.y), d.y), 0.25f);
        pooled[4 * h + 2] = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.z, b.z), cc.z), d.z), 0.25f);
        pooled[4 * h + 3] = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.w, b.w), cc.w), d.w), 0.25f);
      }
    } else {
#pragma unroll
      for (int k = 0; k < PV; k++)
        if (c + k < C) {
          const float* q = xq + c + k;
          pooled[k] = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(q[0], q[C]), q[(size_t)HW * C]), q[(size_t)HW * C + C]), 0.25f);
        }
    }
  };
  auto pool_store = [&](int st) {
#pragma unroll
    for (int k = 0; k < PV; k++) p_s[st][lc + k][lp] = pooled[k];
  };
  float wreg[8];
  auto w_load = [&](int c0) {
    const int o = o0 + wo, c = c0 + wc;
#pragma unroll
    for (int k = 0; k < 8; k++) wreg[k] = 0.0f;
    if (o >= O) return;
    if (c_vec && c + 8 <= C) {
      const float4 a = *reinterpret_cast<const float4*>(w + (size_t)o * C + c);
      const float4 b = *reinterpret_cast<const float4*>(w + (size_t)o * C + c + 4);
      wreg[0] = a.x; wreg[1] = a.y; wreg[2] = a.z; wreg[3] = a.w; wreg[4] = b.x; wreg[5] = b.y; wreg[6] = b.z; wreg[7] = b.w;
    } else {
#pragma unroll
      for (int k = 0; k < 8; k++)
        if (c + k < C) wreg[k] = w[(size_t)o * C + c + k];
    }
  };
  auto w_store = [&](int st) {
#pragma unroll
    for (int k = 0; k < 8; k++) w_s[st][wc + k][wo] = wreg[k];
  };
  // compute roles: 16 x 16 threads; thread (ty, tx) owns pixels ty*TYP..+TYP-1 and channels tx*4..+3 and 64 + tx*4..+3
  const int ty = tid >> 4, tx = tid & 15;
  unsigned long long acc2[TYP][4];  // channel pairs of each pixel (packed fp32 FMAs, same rounding as scalar fmaf)
#pragma unroll
  for (int i = 0; i < TYP; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) acc2[i][j] = 0ull;
  const int nchunks = (C + SC_BK - 1) / SC_BK;
  pool_load(0);
  w_load(0);
  pool_store(0);
  w_store(0);
  __syncthreads();
  for (int ch = 0; ch < nchunks; ch++) {
    const int st = ch & 1;
    if (ch + 1 < nchunks) {  // next chunk's global loads are in flight during this chunk's multiply-adds
      pool_load((ch + 1) * SC_BK);
      w_load((ch + 1) * SC_BK);
    }
    const int cn = min(SC_BK, C - ch * SC_BK);
    const float* pb = &p_s[st][0][ty * TYP];
    const float* wbse = &w_s[st][0][tx * 4];
    auto mac = [&](int cc) {  // one input channel of the chunk for the thread's whole register tile
      float pv[TYP];
#pragma unroll
      for (int i = 0; i < TYP; i += 4) {
        const float4 pa = *reinterpret_cast<const float4*>(pb + cc * (BM + 4) + i);
        pv[i] = pa.x; pv[i + 1] = pa.y; pv[i + 2] = pa.z; pv[i + 3] = pa.w;
      }
      const float4 wa = *reinterpret_cast<const float4*>(wbse + cc * (SC_BN + 4));
      const float4 wb = *reinterpret_cast<const float4*>(wbse + cc * (SC_BN + 4) + 64);
      const unsigned long long w2[4] = {pack_f32x2(wa.x, wa.y), pack_f32x2(wa.z, wa.w), pack_f32x2(wb.x, wb.y),
                                        pack_f32x2(wb.z, wb.w)};
#pragma unroll
      for (int i = 0; i < TYP; i++) {
        const unsigned long long p2 = pack_f32x2(pv[i], pv[i]);
#pragma unroll
        for (int j = 0; j < 4; j++) fma_f32x2(acc2[i][j], p2, w2[j]);
      }
    };
    if (cn == SC_BK) {  // a whole chunk: straight-line code, every address an immediate offset
#pragma unroll
      for (int cc = 0; cc < SC_BK; cc++) mac(cc);
    } else {
      for (int cc = 0; cc < cn; cc++) mac(cc);
    }
    if (ch + 1 < nchunks) {
      pool_store(st ^ 1);
      w_store(st ^ 1);
    }
    __syncthreads();
  }
  float acc[TYP][8];
#pragma unroll
  for (int i = 0; i < TYP; i++)
#pragma unroll
    for (int j = 0; j < 4; j++) unpack_f32x2(acc2[i][j], acc[i][2 * j], acc[i][2 * j + 1]);
#pragma unroll
  for (int h = 0; h < 2; h++) {
    const int o = o0 + 64 * h + tx * 4;
    if (o >= O) continue;
    float sc[4], sf[4];
#pragma unroll
    for (int j = 0; j < 4; j++) {
      sc[j] = (o + j < O) ? scale[o + j] : 0.0f;
      sf[j] = (o + j < O) ? shift[o + j] : 0.0f;
    }
#pragma unroll
    for (int i = 0; i < TYP; i++) {
      const long long p = p0 + ty * TYP + i;
      if (p >= npix_out) continue;
      float* dst = y + p * O + o;
      const float r0 = __fmaf_rn(acc[i][4 * h], sc[0], sf[0]), r1 = __fmaf_rn(acc[i][4 * h + 1], sc[1], sf[1]);
      const float r2 = __fmaf_rn(acc[i][4 * h + 2], sc[2], sf[2]), r3 = __fmaf_rn(acc[i][4 * h + 3], sc[3], sf[3]);
      if (o + 4 <= O && (O & 3) == 0 && (reinterpret_cast<uintptr_t>(y) & 15) == 0) {
        *reinterpret_cast<float4*>(dst) = make_float4(r0, r1, r2, r3);
      } else {
        dst[0] = r0;
        if (o + 1 < O) dst[1] = r1;
        if (o + 2 < O) dst[2] = r2;
        if (o + 3 < O) dst[3] = r3;
      }
    }
  }
}

// Small problems (batch 1): one thread per output, so that a 7x7x512 layer still fills the chip.  A CTA takes 4 output
// pixels x 64 channels; the pooled inputs of its pixels sit in shared memory, each thread walks its weight row.
// Same order of operations as above.
__global__ void __launch_bounds__(256) shortcut_down_small(const float* __restrict__ x, int HW, int C,
                                                           const float* __restrict__ w, int O,
                                                           const float* __restrict__ scale, const float* __restrict__ shift,
                                                           long long npix_out, float* __restrict__ y) {
  __shared__ __align__(16) float pooled[4][512];
  const int tid = threadIdx.x;
  const long long p0 = (long long)blockIdx.x * 4;
  const int OHW = HW / 2;
  for (int t = tid; t < 4 * C; t += 256) {
    const int c = t % C, pp = t / C;
    const long long p = p0 + pp;
    float v = 0.0f;
    if (p < npix_out) {
      const int ow = (int)(p % OHW), oh = (int)((p / OHW) % OHW);
      const long long n = p / ((long long)OHW * OHW);
      const float* q = x + ((n * HW + 2 * oh) * HW + 2 * ow) * C + c;
      float s = __fadd_rn(q[0], q[C]);
      s = __fadd_rn(s, q[(size_t)HW * C]);
      s = __fadd_rn(s, q[(size_t)HW * C + C]);
      v = __fmul_rn(s, 0.25f);
    }
    pooled[pp][c] = v;
  }
  __syncthreads();
  const int pp = tid / 64, o = blockIdx.y * 64 + tid % 64;
  const long long p = p0 + pp;
  if (o >= O || p >= npix_out) return;
  const float* wr = w + (size_t)o * C;
  float a = 0.0f;
  if ((C & 3) == 0 && (reinterpret_cast<uintptr_t>(w) & 15) == 0) {
    for (int c = 0; c < C; c += 4) {
      const float4 wv = __ldg(reinterpret_cast<const float4*>(wr + c));
      const float4 pv = *reinterpret_cast<const float4*>(&pooled[pp][c]);
      a = __fmaf_rn(pv.x, wv.x, a);
      a = __fmaf_rn(pv.y, wv.y, a);
      a = __fmaf_rn(pv.z, wv.z, a);
      a = __fmaf_rn(pv.w, wv.w, a);
    }
  } else {
    for (int c = 0; c < C; c++) a = __fmaf_rn(pooled[pp][c], wr[c], a);
  }
  y[p * O + o] = __fmaf_rn(a, scale[o], shift[o]);
}

// The same for a few images, with every global load issued before the first fmaf: a tile is 16 output pixels x 16
// channels; its 16 weight rows and the pooled inputs of its 16 pixels go through shared memory (coalesced float4 loads,
// all in flight at once), then each thread runs the fmaf chain(s) of its output(s) over c ascending.  C <= 256, C % 4 == 0.
// `sm` holds 2 x 16 x SC16_PITCH floats.  CHAINED: hooks of a kernel launched by launch_chain (see common.cuh).
constexpr int SC16_PITCH = 260;  // floats per row: 16 rows, read as float4, fall on distinct banks
template <int THREADS, bool CHAINED>
__device__ __forceinline__ void shortcut_tile16(const float* x, int HW, int C, const float* __restrict__ w, int O,
                                                const float* __restrict__ scale, const float* __restrict__ shift,
                                                long long npix_out, float* y, const long long bx, const int by, float* sm) {
  constexpr int NOUT = 256 / THREADS;  // outputs per thread, 128 apart in the tile
  float(*pooled)[SC16_PITCH] = reinterpret_cast<float(*)[SC16_PITCH]>(sm);
  float(*ws)[SC16_PITCH] = reinterpret_cast<float(*)[SC16_PITCH]>(sm + 16 * SC16_PITCH);
  const int tid = threadIdx.x;
  const long long p0 = bx * 16;
  const int o0 = by * 16;
  const int OHW = HW / 2, C4 = C / 4;
#pragma unroll 4
  for (int t = tid; t < 16 * C4; t += THREADS) {
    const int row = t / C4, q = t - row * C4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (o0 + row < O) v = __ldg(reinterpret_cast<const float4*>(w + (size_t)(o0 + row) * C) + q);
    *reinterpret_cast<float4*>(&ws[row][4 * q]) = v;
  }
  if (CHAINED) chain_wait();  // (the weights above do not depend on the previous kernel)
#pragma unroll 4
  for (int t = tid; t < 16 * C4; t += THREADS) {
    const int pp = t / C4, q = t - pp * C4;
    const long long p = p0 + pp;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (p < npix_out) {
      const int ow = (int)(p % OHW), oh = (int)((p / OHW) % OHW);
      const long long n = p / ((long long)OHW * OHW);
      const float* src = x + ((n * HW + 2 * oh) * HW + 2 * ow) * C + 4 * q;
      const float4 a = *reinterpret_cast<const float4*>(src);
      const float4 b = *reinterpret_cast<const float4*>(src + C);
      const float4 c = *reinterpret_cast<const float4*>(src + (size_t)HW * C);
      const float4 d = *reinterpret_cast<const float4*>(src + (size_t)HW * C + C);
      v.x = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.x, b.x), c.x), d.x), 0.25f);
      v.y = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.y, b.y), c.y), d.y), 0.25f);
      v.z = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.z, b.z), c.z), d.z), 0.25f);
      v.w = __fmul_rn(__fadd_rn(__fadd_rn(__fadd_rn(a.w, b.w), c.w), d.w), 0.25f);
    }
    *reinterpret_cast<float4*>(&pooled[pp][4 * q]) = v;
  }
  __syncthreads();
  if (CHAINED) chain_trigger();
  const int oo = tid & 15, o = o0 + oo;
  float a[NOUT];
#pragma unroll
  for (int u = 0; u < NOUT; u++) a[u] = 0.0f;
#pragma unroll 4
  for (int c = 0; c < C; c += 4) {
    const float4 wv = *reinterpret_cast<const float4*>(&ws[oo][c]);
#pragma unroll
    for (int u = 0; u < NOUT; u++) {
      const float4 pv = *reinterpret_cast<const float4*>(&pooled[(tid >> 4) + u * (THREADS / 16)][c]);
      a[u] = __fmaf_rn(pv.x, wv.x, a[u]);
      a[u] = __fmaf_rn(pv.y, wv.y, a[u]);
      a[u] = __fmaf_rn(pv.z, wv.z, a[u]);
      a[u] = __fmaf_rn(pv.w, wv.w, a[u]);
    }
  }
  if (o < O) {
    const float sc = scale[o], sf = shift[o];
#pragma unroll
    for (int u = 0; u < NOUT; u++) {
      const long long p = p0 + (tid >> 4) + u * (THREADS / 16);
      if (p < npix_out) y[p * O + o] = __fmaf_rn(a[u], sc, sf);
    }
  }
}
__global__ void __launch_bounds__(256) shortcut_down_tile16(const float* x, int HW, int C, const float* __restrict__ w, int O,
                                                            const float* __restrict__ scale, const float* __restrict__ shift,
                                                            long long npix_out, float* y) {
  __shared__ __align__(16) float sm[2 * 16 * SC16_PITCH];
  shortcut_tile16<256, true>(x, HW, C, w, O, scale, shift, npix_out, y, blockIdx.x, blockIdx.y, sm);
}

// ---- head: global average over 7x7 (sequential sum over (h, w), then /49) into the workspace, then fc 512 -> 1000 as
// one fmaf chain per logit over k ascending, then + bias.  Three forms of the fc, by batch size, below.
__global__ void __launch_bounds__(512) gap_small(const float* __restrict__ x /*[N][7][7][512]*/, float* __restrict__ g) {
  const int n = blockIdx.x, c = threadIdx.x;
  float s = 0.0f;
  for (int q = 0; q < 49; q++) s = __fadd_rn(s, x[((size_t)n * 49 + q) * 512 + c]);
  g[(size_t)n * 512 + c] = __fdiv_rn(s, 49.0f);
}
// One to four images: pooling and fc in one launch.  A 512-thread CTA takes 8 logits of one image: it pools the image's
// 7x7x512 map itself (thread c owns channel c; same sum order and division as gap_small) while its 8 weight rows are in
// flight, then 8 threads run the 8 fmaf chains out of shared memory.
__global__ void __launch_bounds__(512) head_small(const float* x /*[N][7][7][512]*/,
                                                  const float* __restrict__ fw, const float* __restrict__ fb,
                                                  float* __restrict__ logits) {
  constexpr int PITCH = 516;
  __shared__ __align__(16) float gs[512];
  __shared__ __align__(16) float ws[8][PITCH];
  const int n = blockIdx.y, tid = threadIdx.x, j0 = blockIdx.x * 8;
  float4 wv[2];
#pragma unroll
  for (int u = 0; u < 2; u++) {
    const int idx = tid + 512 * u, row = idx >> 7, q = idx & 127;
    wv[u] = (j0 + row < 1000) ? __ldg(reinterpret_cast<const float4*>(fw + (size_t)(j0 + row) * 512) + q)
                              : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  chain_wait();  // (chained launches: the weight rows above do not depend on the previous kernel)
  float s = 0.0f;
#pragma unroll 7
  for (int q = 0; q < 49; q++) s = __fadd_rn(s, x[((size_t)n * 49 + q) * 512 + tid]);
  gs[tid] = __fdiv_rn(s, 49.0f);
#pragma unroll
  for (int u = 0; u < 2; u++) {
    const int idx = tid + 512 * u, row = idx >> 7, q = idx & 127;
    *reinterpret_cast<float4*>(&ws[row][4 * q]) = wv[u];
  }
  __syncthreads();
  const int j = j0 + tid;
  if (tid >= 8 || j >= 1000) return;
  float a = 0.0f;
#pragma unroll 8
  for (int k = 0; k < 512; k += 4) {
    const float4 w4 = *reinterpret_cast<const float4*>(&ws[tid][k]);
    const float4 g4 = *reinterpret_cast<const float4*>(&gs[k]);
    a = __fmaf_rn(g4.x, w4.x, a);
    a = __fmaf_rn(g4.y, w4.y, a);
    a = __fmaf_rn(g4.z, w4.z, a);
    a = __fmaf_rn(g4.w, w4.w, a);
  }
  logits[(size_t)n * 1000 + j] = __fadd_rn(a, fb[j]);
}

// Five to 63 images: pooled vectors come from gap_small; a 64-thread CTA takes 8 logits of up to 8 images.  Its 8 weight
// rows and the images' pooled vectors are staged in shared memory by coalesced loads, all in flight at once; thread
// (image, logit) then runs its fmaf chain over k ascending.
__global__ void __launch_bounds__(64) fc_mid(const float* __restrict__ g /*[N][512]*/, int N, const float* __restrict__ fw,
                                             const float* __restrict__ fb, float* __restrict__ logits) {
  constexpr int PITCH = 516;
  __shared__ __align__(16) float gs[8][PITCH];
  __shared__ __align__(16) float ws[8][PITCH];
  const int tid = threadIdx.x, j0 = blockIdx.x * 8, n0 = blockIdx.y * 8;
  float4 wv[16], gv[16];
#pragma unroll
  for (int u = 0; u < 16; u++) {  // 8 rows x 128 float4 each
    const int idx = tid + 64 * u, row = idx >> 7, q = idx & 127;
    wv[u] = (j0 + row < 1000) ? __ldg(reinterpret_cast<const float4*>(fw + (size_t)(j0 + row) * 512) + q)
                              : make_float4(0.f, 0.f, 0.f, 0.f);
    gv[u] = (n0 + row < N) ? *(reinterpret_cast<const float4*>(g + (size_t)(n0 + row) * 512) + q)
                           : make_float4(0.f, 0.f, 0.f, 0.f);
  }
#pragma unroll
  for (int u = 0; u < 16; u++) {
    const int idx = tid + 64 * u, row = idx >> 7, q = idx & 127;
    *reinterpret_cast<float4*>(&ws[row][4 * q]) = wv[u];
    *reinterpret_cast<float4*>(&gs[row][4 * q]) = gv[u];
  }
  __syncthreads();
  const int jj = tid & 7, im = tid >> 3, j = j0 + jj, n = n0 + im;
  float a = 0.0f;
#pragma unroll 8
  for (int k = 0; k < 512; k += 4) {
    const float4 w4 = *reinterpret_cast<const float4*>(&ws[jj][k]);
    const float4 g4 = *reinterpret_cast<const float4*>(&gs[im][k]);
    a = __fmaf_rn(g4.x, w4.x, a);
    a = __fmaf_rn(g4.y, w4.y, a);
    a = __fmaf_rn(g4.z, w4.z, a);
    a = __fmaf_rn(g4.w, w4.w, a);
  }
  if (j < 1000 && n < N) logits[(size_t)n * 1000 + j] = __fadd_rn(a, fb[j]);
}

// Larger batches: pooled vectors come from gap_small; a 64-thread CTA computes 64 logits for 8 images, so every weight
// it loads is used 8 times and there are 16 x N/8 CTAs.  The weight rows of the 64 logits pass through shared memory in
// chunks of 32 inputs (coalesced 128-byte pieces of each row in, conflict-free columns out), the next chunk in flight
// while the current one is multiplied.  Each logit is still one fmaf chain over the inputs in ascending order.
__global__ void __launch_bounds__(64) fc_batched(const float* __restrict__ g /*[N][512]*/, int N, const float* __restrict__ fw,
                                                 const float* __restrict__ fb, float* __restrict__ logits) {
  __shared__ __align__(16) float gs[8][512];
  __shared__ __align__(16) float ws[64][36];  // (pitch 36: 128-bit rows in and 128-bit columns out, both free of bank conflicts)
  const int tid = threadIdx.x;
  const int n0 = blockIdx.y * 8, nimg = min(8, N - n0);
  for (int t = tid; t < 8 * 128; t += 64) {
    const int im = t / 128;
    reinterpret_cast<float4*>(&gs[0][0])[t] =
        im < nimg ? reinterpret_cast<const float4*>(g + (size_t)n0 * 512)[t] : make_float4(0.f, 0.f, 0.f, 0.f);
  }
  const int j0 = blockIdx.x * 64, j = j0 + tid;
  float4 wreg[8];
  auto w_load = [&](int k0) {  // 64 rows x 32 inputs: piece u of this thread is row (tid + 64u) / 8, float4 (tid + 64u) % 8
#pragma unroll
    for (int u = 0; u < 8; u++) {
      const int idx = tid + 64 * u, row = idx >> 3, q = idx & 7;
      wreg[u] = (j0 + row < 1000) ? __ldg(reinterpret_cast<const float4*>(fw + (size_t)(j0 + row) * 512 + k0) + q)
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
    }
  };
  auto w_store = [&]() {
#pragma unroll
    for (int u = 0; u < 8; u++) {
      const int idx = tid + 64 * u, row = idx >> 3, q = idx & 7;
      *reinterpret_cast<float4*>(&ws[row][4 * q]) = wreg[u];
    }
  };
  float a[8];
#pragma unroll
  for (int im = 0; im < 8; im++) a[im] = 0.0f;
  w_load(0);
  for (int k0 = 0; k0 < 512; k0 += 32) {
    __syncthreads();  // the previous chunk has been read (and, the first time, gs is complete)
    w_store();
    __syncthreads();
    if (k0 + 32 < 512) w_load(k0 + 32);
#pragma unroll 2
    for (int kk = 0; kk < 32; kk += 4) {  // four inputs per 128-bit load; each chain still takes them in ascending order
      const float4 wv = *reinterpret_cast<const float4*>(&ws[tid][kk]);
#pragma unroll
      for (int im = 0; im < 8; im++) {
        const float4 gv = *reinterpret_cast<const float4*>(&gs[im][k0 + kk]);
        a[im] = __fmaf_rn(gv.x, wv.x, a[im]);
        a[im] = __fmaf_rn(gv.y, wv.y, a[im]);
        a[im] = __fmaf_rn(gv.z, wv.z, a[im]);
        a[im] = __fmaf_rn(gv.w, wv.w, a[im]);
      }
    }
  }
  if (j >= 1000) return;
  const float bias = fb[j];
#pragma unroll
  for (int im = 0; im < 8; im++)
    if (im < nimg) logits[(size_t)(n0 + im) * 1000 + j] = __fadd_rn(a[im], bias);
}

constexpr int kStageC[4] = {64, 128, 256, 512};
constexpr int kStageHW[4] = {56, 28, 14, 7};

size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Workspace {
  size_t stem_out, res_a, res_b, bits_a, bits_b, gap, total;
};

Workspace plan(int N) {
  Workspace ws;
  size_t off = 0;
  ws.stem_out = off; off = align_up(off + (size_t)N * 112 * 112 * 64 * 4, 256);
  ws.res_a = off;    off = align_up(off + (size_t)N * 56 * 56 * 64 * 4, 256);
  ws.res_b = off;    off = align_up(off + (size_t)N * 28 * 28 * 128 * 4, 256);
  ws.bits_a = off;   off = align_up(off + (size_t)N * 56 * 56 * 8, 256);
  ws.bits_b = off;   off = align_up(off + (size_t)N * 56 * 56 * 8, 256);
  ws.gap = off;      off = align_up(off + (size_t)N * 512 * 4, 256);
  ws.total = off;
  return ws;
}

dabnn_status launch_stem_8x8(const dabnn_bireal18_params* p, const float* images, int N, float* out, cudaStream_t st) {
  constexpr size_t SMEM = (size_t)(STEM_K * 64 + 2 * 3 * 37 * 2 * 20) * 4;
  static bool configured[kMaxDevices] = {};
  const int dev = current_device();
  if (dev < 0) return DABNN_ERR_CUDA;
  if (!configured[dev]) {
    if (cudaFuncSetAttribute(stem_conv_bn_8x8, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)SMEM) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    configured[dev] = true;
  }
  const long long ntiles = (long long)N * 49, cap = 2LL * sm_count();
  stem_conv_bn_8x8<<<(unsigned)(ntiles < cap ? ntiles : cap), 256, SMEM, st>>>(images, p->stem_w, p->stem_scale,
                                                                             p->stem_shift, N, out);
  return launch_status();
}

template <int TS, int PPT, int CPT>
dabnn_status launch_stem(const dabnn_bireal18_params* p, const float* images, int N, float* out, cudaStream_t st) {
  constexpr int PS = 2 * TS + 5, HALF = stem_half(PS);
  constexpr size_t SMEM = (size_t)(2 * STEM_K * 4 * CPT + 2 * 3 * PS * 2 * HALF) * 4;
  auto kern = stem_conv_bn<TS, PPT, CPT>;
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
  const int tiles = (112 + TS - 1) / TS;
  const long long ntiles = (long long)N * tiles * tiles;
  const long long cap = 2LL * sm_count();  // persistent: two CTAs per SM, each walking over tiles
  kern<<<dim3((unsigned)(ntiles < cap ? ntiles : cap), 16 / CPT), (TS * TS / PPT) * 4, SMEM, st>>>(
      images, p->stem_w, p->stem_scale, p->stem_shift, N, out);  // head of a chain
  return launch_status();
}

}  // namespace

}  // namespace dabnn

using namespace dabnn;

extern "C" dabnn_status dabnn_bn_fold(const float* gamma, const float* beta, const float* mean, const float* var,
                                      double eps, int O, float* scale, float* shift, void* stream) {
  if (!gamma || !beta || !mean || !var || !scale || !shift) return DABNN_ERR_NULL;
  if (O <= 0 || !(eps >= 0.0)) return DABNN_ERR_SHAPE;
  bn_fold_kernel<<<ceil_div(O, 128), 128, 0, as_stream(stream)>>>(gamma, beta, mean, var, eps, O, scale, shift);
  return launch_status();
}

extern "C" size_t dabnn_bireal18_workspace_bytes(int N) { return N <= 0 ? 0 : plan(N).total; }

// sm == nullptr: the 7x7 stem and the max-pool; else the STEM module in their place.
static dabnn_status forward_impl(const dabnn_bireal18_params* p, const dabnn_stem_module_params* sm, const float* images,
                                 int N, float* logits, void* workspace, size_t workspace_bytes, void* stream) {
  if (!p || !images || !logits || !workspace) return DABNN_ERR_NULL;
  if (N <= 0 || N > 65535) return DABNN_ERR_SHAPE;
  if ((!sm && (!p->stem_w || !p->stem_scale || !p->stem_shift)) || !p->fc_w || !p->fc_b) return DABNN_ERR_NULL;
  for (int b = 0; b < 16; b++)
    if (!p->block_w[b] || !p->block_scale[b] || !p->block_shift[b]) return DABNN_ERR_NULL;
  for (int d = 0; d < 3; d++)
    if (!p->down_w[d] || !p->down_scale[d] || !p->down_shift[d]) return DABNN_ERR_NULL;
  if (!aligned(workspace, 256) || !aligned(images, 4) || !aligned(logits, 4) || !aligned(p->fc_w, 16))
    return DABNN_ERR_ALIGNMENT;
  const Workspace ws = plan(N);
  if (workspace_bytes < ws.total) return DABNN_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  // The launches are chained: each kernel that takes part may start its set-up while its predecessor finishes (see
  // launch_chain; DABNN_NO_CHAIN=1 in the environment keeps the ordinary stream order, for measurements).  For one to four
  // images that is a chain of 22 launches shorter than a launch takes; for large batches it hides the start-up of the
  // persistent tensor-engine kernels (tensor memory, barriers, 144 KB of weights per CTA) under the previous kernel's tail.
  static const bool chain_off = getenv("DABNN_NO_CHAIN") != nullptr;
  struct ChainScope {
    explicit ChainScope(bool on) { g_chain_launch = on; }
    ~ChainScope() { g_chain_launch = false; }
  } chain_scope(!chain_off);
  char* base = static_cast<char*>(workspace);
  float* stem_out = reinterpret_cast<float*>(base + ws.stem_out);
  float* cur = reinterpret_cast<float*>(base + ws.res_a);
  float* other = reinterpret_cast<float*>(base + ws.res_b);
  uint64_t* bits_in = reinterpret_cast<uint64_t*>(base + ws.bits_a);
  uint64_t* bits_out = reinterpret_cast<uint64_t*>(base + ws.bits_b);

  dabnn_status s;
  if (sm) {
    // the stem output area holds the module's three scratch tensors: s1 (half of it), a1 and the concatenation (a quarter each)
    float* a1 = stem_out + (size_t)N * 112 * 112 * 32;
    float* cat = a1 + (size_t)N * 112 * 112 * 16;
    if ((s = launch_stem_module(sm, images, N, stem_out, a1, cat, cur, bits_in, st)) != DABNN_OK) return s;
  } else {
    s = (N * 49 >= 2 * sm_count()) ? launch_stem_8x8(p, images, N, stem_out, st)
                                   : (N == 1 ? launch_stem<8, 2, 8>(p, images, N, stem_out, st)  // one image: 392 half-tile CTAs
                                              : launch_stem<8, 2, 16>(p, images, N, stem_out, st));
    if (s != DABNN_OK) return s;
  }
  if (!sm) {
    const long long npix = (long long)N * 56 * 56;
    launch_chain(maxpool_pack, dim3(ceil_div(npix * 16, 256)), dim3(256), (size_t)0, st, stem_out, npix, cur, bits_in);
    if ((s = launch_status()) != DABNN_OK) return s;
  }
  // consecutive tensor-engine blocks are chained (DABNN_NO_CHAIN=1 keeps the ordinary stream order)
  const bool tc_chain = !chain_off;
  int C = 64, HW = 56;
  for (int b = 0; b < 16; b++) {
    const int stage = b / 4, O = kStageC[stage], OHW = kStageHW[stage];
    const bool down = stage > 0 && b % 4 == 0;
    if (down) {
      const long long npo = (long long)N * OHW * OHW;
      // At most one wave of 128 x 128 tiles (whose time is then set by the length of the chain over c alone) and at most
      // three resident rounds of 16 x 16 tiles (about 6 CTAs per SM): one thread per output.  Measured crossover.
      const bool few = (long long)ceil_div(npo, SC_BM) * ceil_div(O, SC_BN) <= sm_count() &&
                       (long long)ceil_div(npo, 16) * ceil_div(O, 16) <= 18LL * sm_count();
      if (few && C <= 256 && C % 4 == 0 && aligned(p->down_w[stage - 1], 16))
        launch_chain(shortcut_down_tile16, dim3(ceil_div(npo, 16), ceil_div(O, 16)), dim3(256), (size_t)0, st, cur, HW, C,
                     p->down_w[stage - 1], O, p->down_scale[stage - 1], p->down_shift[stage - 1], npo, other);
      else if (few && C <= 512)
        shortcut_down_small<<<dim3(ceil_div(npo, 4), ceil_div(O, 64)), 256, 0, st>>>(
            cur, HW, C, p->down_w[stage - 1], O, p->down_scale[stage - 1], p->down_shift[stage - 1], npo, other);
      else  // 64-pixel tiles: 80 registers, three CTAs per SM, and less lost to the last, partly filled round than with 128
        shortcut_down<64><<<dim3(ceil_div(npo, 64), ceil_div(O, SC_BN)), 256, 0, st>>>(
            cur, HW, C, p->down_w[stage - 1], O, p->down_scale[stage - 1], p->down_shift[stage - 1], npo, other);
      if ((s = launch_status()) != DABNN_OK) return s;
      float* t = cur; cur = other; other = t;
    }
    const dabnn_shape in = {N, C, HW, HW};
    const int stride = down ? 2 : 1;
    const dabnn_conv cv = {3, 3, stride, stride, 1, 1, -1};
    s = DABNN_ERR_UNSUPPORTED;
    if (p->block_w_tc[b] != nullptr && tc_worthwhile(in, O, cv))  // tensor-core engine where it covers the layer and pays
      s = tc_bireal_block(bits_in, in, p->block_w_tc[b], O, cv, p->block_scale[b], p->block_shift[b], cur, cur,
                          b == 15 ? nullptr : bits_out, tc_chain, st);
    if (s == DABNN_ERR_UNSUPPORTED)
      s = dabnn_bconv2d_bn_add_sign_pack(bits_in, in, p->block_w[b], O, cv, p->block_scale[b], p->block_shift[b], cur, cur,
                                         b == 15 ? nullptr : bits_out, st);
    if (s != DABNN_OK) return s;
    uint64_t* tb = bits_in; bits_in = bits_out; bits_out = tb;
    C = O; HW = OHW;
  }
  {
    if (N <= 4) {
      launch_chain(head_small, dim3(125, N), dim3(512), (size_t)0, st, cur, p->fc_w, p->fc_b, logits);
      return launch_status();
    }
    float* gbuf = reinterpret_cast<float*>(base + ws.gap);
    gap_small<<<N, 512, 0, st>>>(cur, gbuf);
    if ((s = launch_status()) != DABNN_OK) return s;
    if (N < 64) fc_mid<<<dim3(125, ceil_div(N, 8)), 64, 0, st>>>(gbuf, N, p->fc_w, p->fc_b, logits);
    else fc_batched<<<dim3(ceil_div(1000, 64), ceil_div(N, 8)), 64, 0, st>>>(gbuf, N, p->fc_w, p->fc_b, logits);
  }
  return launch_status();
}

extern "C" dabnn_status dabnn_bireal18_forward(const dabnn_bireal18_params* p, const float* images, int N,
                                               float* logits, void* workspace, size_t workspace_bytes, void* stream) {
  return forward_impl(p, nullptr, images, N, logits, workspace, workspace_bytes, stream);
}

extern "C" dabnn_status dabnn_bireal18_forward_stem_module(const dabnn_bireal18_params* p, const dabnn_stem_module_params* sm,
                                                           const float* images, int N, float* logits, void* workspace,
                                                           size_t workspace_bytes, void* stream) {
  if (!sm) return DABNN_ERR_NULL;
  return forward_impl(p, sm, images, N, logits, workspace, workspace_bytes, stream);
}

// ---- allocation-free variant ---------------------------------------------------------------------------
// Scratch for dabnn_bireal18_forward_static: part of the library image, present on every device that loads
// it.  In host code the symbol below is only a handle; its device address is looked up per device.
static __device__ __align__(256) unsigned char g_static_scratch[DABNN_STATIC_SCRATCH_BYTES];

namespace {
std::mutex g_static_mutex;
void* g_static_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal
}  // namespace

extern "C" dabnn_status dabnn_bireal18_forward_static(const dabnn_bireal18_params* p, const float* images, int N,
                                                      float* logits, void* stream) {
  if (N > DABNN_STATIC_MAX_BATCH) return DABNN_ERR_STATIC_LIMIT;
  if (N <= 0) return DABNN_ERR_SHAPE;
  if (dabnn_bireal18_workspace_bytes(N) > (size_t)DABNN_STATIC_SCRATCH_BYTES) return DABNN_ERR_STATIC_LIMIT;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return DABNN_ERR_CUDA;
  }
  if (dev < 0 || dev >= kMaxDevices) return DABNN_ERR_UNSUPPORTED;
  void* scratch = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_static_mutex);
    scratch = g_static_addr[dev];
    if (scratch == nullptr) {
      // once per device, with that device current: the symbol's address in this device's memory
      if (cudaGetSymbolAddress(&scratch, g_static_scratch) != cudaSuccess || scratch == nullptr) {
        cudaGetLastError();
        return DABNN_ERR_CUDA;
      }
      g_static_addr[dev] = scratch;
    }
  }
  return dabnn_bireal18_forward(p, images, N, logits, scratch, (size_t)DABNN_STATIC_SCRATCH_BYTES, stream);
}
