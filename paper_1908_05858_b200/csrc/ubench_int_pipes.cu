// Register-only micro-benchmarks of the B200 integer pipes: they define the measured roofline of the bit-op
// convolution (how many POPC, LOP3, IADD, IMAD lanes per clock per SM; whether they issue on separate pipes; what
// the plain and carry-save xor/popcount inner loops reach; and what mma.sync ... b1 and s8 reach).
//   ubench_int_pipes          times every kernel with CUDA events (5 launches each) and prints rates
//   ubench_int_pipes once     launches every kernel once (for a profiler's per-pipe instruction counters)
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#define CK(x) do{cudaError_t e=(x); if(e!=cudaSuccess){printf("CUDA error %s at %d\n", cudaGetErrorString(e), __LINE__); return 1;}}while(0)

constexpr int ITERS = 4096;

__global__ void k_popc(uint32_t* out, uint32_t seed) {
  uint32_t x[8];
#pragma unroll
  for (int i = 0; i < 8; i++) x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) asm volatile("popc.b32 %0, %0;" : "+r"(x[i]));
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
__global__ void k_lop3(uint32_t* out, uint32_t seed) {
  uint32_t x[8]; uint32_t y = seed ^ threadIdx.x, z = seed * 3 + 1;
#pragma unroll
  for (int i = 0; i < 8; i++) x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(x[i]) : "r"(y), "r"(z));
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
__global__ void k_iadd(uint32_t* out, uint32_t seed) {
  uint32_t x[8]; uint32_t y = seed ^ threadIdx.x;
#pragma unroll
  for (int i = 0; i < 8; i++) x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) asm volatile("add.u32 %0, %0, %1;" : "+r"(x[i]) : "r"(y));
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
__global__ void k_imad(uint32_t* out, uint32_t seed) {
  uint32_t x[8]; uint32_t y = seed ^ threadIdx.x, z = seed | 1;
#pragma unroll
  for (int i = 0; i < 8; i++) x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(x[i]) : "r"(z), "r"(y));
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
// popc + independent lop3 stream: do they co-issue?
__global__ void k_popc_lop(uint32_t* out, uint32_t seed, int nlop) {
  uint32_t x[8], l[8]; uint32_t y = seed ^ threadIdx.x, z = seed * 3 + 1;
#pragma unroll
  for (int i = 0; i < 8; i++) { x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u; l[i] = x[i] ^ 0x55u; }
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) {
      asm volatile("popc.b32 %0, %0;" : "+r"(x[i]));
      for (int j = 0; j < 4; j++) if (j < nlop) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(l[i]) : "r"(y), "r"(z));
    }
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i] + l[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
template <int NL>
__global__ void k_popc_lopT(uint32_t* out, uint32_t seed) {
  uint32_t x[8], l[8]; uint32_t y = seed ^ threadIdx.x, z = seed * 3 + 1;
#pragma unroll
  for (int i = 0; i < 8; i++) { x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u; l[i] = x[i] ^ 0x55u; }
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) {
      asm volatile("popc.b32 %0, %0;" : "+r"(x[i]));
#pragma unroll
      for (int j = 0; j < NL; j++) asm volatile("lop3.b32 %0, %0, %1, %2, 0x96;" : "+r"(l[i]) : "r"(y), "r"(z));
    }
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i] + l[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
// popc + imad (accumulate on FMA pipe?)
template <int NM>
__global__ void k_popc_imadT(uint32_t* out, uint32_t seed) {
  uint32_t x[8], l[8]; uint32_t y = seed ^ threadIdx.x, z = seed | 1;
#pragma unroll
  for (int i = 0; i < 8; i++) { x[i] = seed * (threadIdx.x + 1) + i * 0x9e3779b9u; l[i] = x[i] ^ 0x55u; }
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) {
      asm volatile("popc.b32 %0, %0;" : "+r"(x[i]));
#pragma unroll
      for (int j = 0; j < NM; j++) asm volatile("mad.lo.u32 %0, %0, %1, %2;" : "+r"(l[i]) : "r"(z), "r"(y));
    }
  }
  uint32_t s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) s += x[i] + l[i];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// Realistic register-tile loops, operands from shared memory. TP x TO tile.
template <int TP, int TO, int MODE>
__global__ void k_tile(uint32_t* out, uint32_t seed, int kwords) {
  extern __shared__ uint32_t sm[];
  // layout: A[k][TP*8 pixels-slots], W[k][TO*8]
  const int KW = 64;
  uint32_t* A = sm; uint32_t* Wt = sm + KW * 64;
  for (int i = threadIdx.x; i < KW * 128; i += blockDim.x) sm[i] = seed * (i + 1) ^ (i * 0x9e3779b9u);
  __syncthreads();
  int lane = threadIdx.x & 31;
  int pg = lane & 3, og = lane >> 2;  // 4 pixel groups x 8 channel groups
  int acc[TP][TO]; uint32_t ones[TP][TO];
#pragma unroll
  for (int i = 0; i < TP; i++)
#pragma unroll
    for (int j = 0; j < TO; j++) { acc[i][j] = 0; ones[i][j] = 0; }
  for (int rep = 0; rep < kwords / KW; rep++) {
#pragma unroll 2
    for (int k = 0; k < KW; k += 4) {
      uint32_t a[TP][4], w[TO][4];
#pragma unroll
      for (int i = 0; i < TP; i++) { uint4 v = *reinterpret_cast<uint4*>(&A[((pg * TP + i) & 15) * 4 * 16 + (k & 63)]); a[i][0]=v.x;a[i][1]=v.y;a[i][2]=v.z;a[i][3]=v.w; }
#pragma unroll
      for (int j = 0; j < TO; j++) { uint4 v = *reinterpret_cast<uint4*>(&Wt[((og * TO + j) & 15) * 4 * 16 + (k & 63)]); w[j][0]=v.x;w[j][1]=v.y;w[j][2]=v.z;w[j][3]=v.w; }
#pragma unroll
      for (int i = 0; i < TP; i++)
#pragma unroll
        for (int j = 0; j < TO; j++) {
          if (MODE == 0) {
#pragma unroll
            for (int q = 0; q < 4; q++) acc[i][j] += __popc(a[i][q] ^ w[j][q]);
          } else if (MODE == 1) {
            // one-level carry-save: 2 words per POPC
#pragma unroll
            for (int q = 0; q < 4; q += 2) {
              uint32_t x1 = a[i][q] ^ w[j][q], x2 = a[i][q + 1] ^ w[j][q + 1];
              uint32_t o = ones[i][j];
              uint32_t s = o ^ x1 ^ x2;
              uint32_t c = (o & x1) | (o & x2) | (x1 & x2);
              ones[i][j] = s;
              acc[i][j] += __popc(c);
            }
          } else {
            // 3:2 on fresh words: 3 words -> 2 popc (uses q=0..2 only, q=3 naive)
            uint32_t x1 = a[i][0] ^ w[j][0], x2 = a[i][1] ^ w[j][1], x3 = a[i][2] ^ w[j][2];
            uint32_t s = x1 ^ x2 ^ x3;
            uint32_t c = (x1 & x2) | (x1 & x3) | (x2 & x3);
            acc[i][j] += __popc(s) + 2 * __popc(c) + __popc(a[i][3] ^ w[j][3]);
          }
        }
    }
  }
  int s = 0;
#pragma unroll
  for (int i = 0; i < TP; i++)
#pragma unroll
    for (int j = 0; j < TO; j++) s += (MODE == 1) ? (2 * acc[i][j] + __popc(ones[i][j])) : acc[i][j];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

// 1-bit MMA chains
template <int OP>
__global__ void k_bmma(int* out, uint32_t seed) {
  uint32_t a[4], b[2];
  for (int i = 0; i < 4; i++) a[i] = seed * (threadIdx.x + 1 + i);
  for (int i = 0; i < 2; i++) b[i] = seed * (threadIdx.x + 7 + i);
  int c[8][4];
#pragma unroll
  for (int i = 0; i < 8; i++) for (int j = 0; j < 4; j++) c[i][j] = 0;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++) {
      if (OP == 0)
        asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.xor.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
          : "+r"(c[i][0]), "+r"(c[i][1]), "+r"(c[i][2]), "+r"(c[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
      else
        asm volatile("mma.sync.aligned.m16n8k256.row.col.s32.b1.b1.s32.and.popc {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
          : "+r"(c[i][0]), "+r"(c[i][1]), "+r"(c[i][2]), "+r"(c[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
    }
  }
  int s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) for (int j = 0; j < 4; j++) s += c[i][j];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}
// int8 mma.sync for comparison (legacy tensor path)
__global__ void k_imma(int* out, uint32_t seed) {
  uint32_t a[4], b[2];
  for (int i = 0; i < 4; i++) a[i] = seed * (threadIdx.x + 1 + i);
  for (int i = 0; i < 2; i++) b[i] = seed * (threadIdx.x + 7 + i);
  int c[8][4];
#pragma unroll
  for (int i = 0; i < 8; i++) for (int j = 0; j < 4; j++) c[i][j] = 0;
  for (int it = 0; it < ITERS; it++) {
#pragma unroll
    for (int i = 0; i < 8; i++)
      asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+r"(c[i][0]), "+r"(c[i][1]), "+r"(c[i][2]), "+r"(c[i][3]) : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b[0]), "r"(b[1]));
  }
  int s = 0;
#pragma unroll
  for (int i = 0; i < 8; i++) for (int j = 0; j < 4; j++) s += c[i][j];
  out[blockIdx.x * blockDim.x + threadIdx.x] = s;
}

static bool g_once = false;
template <typename F>
float timeit(F f) {
  cudaEvent_t e0, e1; cudaEventCreate(&e0); cudaEventCreate(&e1);
  if (g_once) { f(); cudaDeviceSynchronize(); return 1.f; }
  f(); f(); cudaDeviceSynchronize();
  cudaEventRecord(e0); for (int r = 0; r < 5; r++) f(); cudaEventRecord(e1); cudaEventSynchronize(e1);
  float ms; cudaEventElapsedTime(&ms, e0, e1); return ms / 5;
}

int main(int argc, char** argv) {
  g_once = argc > 1;
  cudaDeviceProp p; CK(cudaGetDeviceProperties(&p, 0));
  int sms = p.multiProcessorCount; int clk; cudaDeviceGetAttribute(&clk, cudaDevAttrClockRate, 0);
  printf("device %s SMs %d clockRate %d kHz smem/SM %zu regs/SM %d\n", p.name, sms, clk, p.sharedMemPerMultiprocessor, p.regsPerMultiprocessor);
  uint32_t* out; CK(cudaMalloc(&out, 64 << 20));
  const int TPB = 256; int blocks = sms * 8;
  double thr = (double)blocks * TPB;
  auto rep = [&](const char* name, float ms, double ops_per_thread) {
    double total = thr * ops_per_thread; double per_s = total / (ms * 1e-3);
    printf("%-28s %8.3f ms  %10.2f Gop/s  = %7.2f op/clk/SM @1965MHz (%7.2f @1500)\n", name, ms, per_s / 1e9, per_s / sms / 1.965e9, per_s / sms / 1.5e9);
  };
  rep("popc", timeit([&]{ k_popc<<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("lop3", timeit([&]{ k_lop3<<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("iadd", timeit([&]{ k_iadd<<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("imad", timeit([&]{ k_imad<<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+1lop (popc rate)", timeit([&]{ k_popc_lopT<1><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+2lop (popc rate)", timeit([&]{ k_popc_lopT<2><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+3lop (popc rate)", timeit([&]{ k_popc_lopT<3><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+4lop (popc rate)", timeit([&]{ k_popc_lopT<4><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+6lop (popc rate)", timeit([&]{ k_popc_lopT<6><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+1imad (popc rate)", timeit([&]{ k_popc_imadT<1><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+2imad (popc rate)", timeit([&]{ k_popc_imadT<2><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  rep("popc+4imad (popc rate)", timeit([&]{ k_popc_imadT<4><<<blocks, TPB>>>(out, 12345); }), 8.0 * ITERS);
  CK(cudaGetLastError());
  // tile loops: word-pairs per thread = TP*TO*kwords
  int kwords = 64 * 64; size_t smem = 64 * 128 * 4;
  {
    int b2 = sms * 4;
    double thr2 = (double)b2 * 128;
    auto rep2 = [&](const char* name, float ms, double pairs) {
      double per_s = thr2 * pairs / (ms * 1e-3);
      printf("%-28s %8.3f ms  %10.2f Gwordpair/s = %7.2f pair/clk/SM @1965 ; %8.1f Tbit-op/s\n", name, ms, per_s / 1e9, per_s / sms / 1.965e9, per_s * 64 / 1e12);
    };
    rep2("tile4x4 naive", timeit([&]{ k_tile<4,4,0><<<b2, 128, smem>>>(out, 7, kwords); }), 16.0 * kwords);
    rep2("tile4x4 csa1", timeit([&]{ k_tile<4,4,1><<<b2, 128, smem>>>(out, 7, kwords); }), 16.0 * kwords);
    rep2("tile4x4 csa32", timeit([&]{ k_tile<4,4,2><<<b2, 128, smem>>>(out, 7, kwords); }), 16.0 * kwords);
    rep2("tile8x4 naive", timeit([&]{ k_tile<8,4,0><<<b2, 128, smem>>>(out, 7, kwords); }), 32.0 * kwords);
    rep2("tile8x4 csa1", timeit([&]{ k_tile<8,4,1><<<b2, 128, smem>>>(out, 7, kwords); }), 32.0 * kwords);
    rep2("tile8x4 csa32", timeit([&]{ k_tile<8,4,2><<<b2, 128, smem>>>(out, 7, kwords); }), 32.0 * kwords);
    rep2("tile8x8 naive", timeit([&]{ k_tile<8,8,0><<<b2, 128, smem>>>(out, 7, kwords); }), 64.0 * kwords);
    rep2("tile8x8 csa1", timeit([&]{ k_tile<8,8,1><<<b2, 128, smem>>>(out, 7, kwords); }), 64.0 * kwords);
    b2 = sms * 8; thr2 = (double)b2 * 128;
    rep2("tile4x4 naive x8cta", timeit([&]{ k_tile<4,4,0><<<b2, 128, smem>>>(out, 7, kwords); }), 16.0 * kwords);
    rep2("tile8x4 csa1 x8cta", timeit([&]{ k_tile<8,4,1><<<b2, 128, smem>>>(out, 7, kwords); }), 32.0 * kwords);
    rep2("tile8x8 csa1 x8cta", timeit([&]{ k_tile<8,8,1><<<b2, 128, smem>>>(out, 7, kwords); }), 64.0 * kwords);
  }
  CK(cudaGetLastError());
  // bmma: per warp-instruction 16*8*256 bit-MACs
  {
    auto rep3 = [&](const char* name, float ms, double macs_per_inst) {
      double warps = thr / 32; double total = warps * 8.0 * ITERS * macs_per_inst; double per_s = total / (ms * 1e-3);
      printf("%-28s %8.3f ms  %10.2f T MAC/s = %9.1f MAC/clk/SM @1965\n", name, ms, per_s / 1e12, per_s / sms / 1.965e9);
    };
    rep3("bmma xor.popc m16n8k256", timeit([&]{ k_bmma<0><<<blocks, TPB>>>((int*)out, 3); }), 16.0 * 8 * 256);
    rep3("bmma and.popc m16n8k256", timeit([&]{ k_bmma<1><<<blocks, TPB>>>((int*)out, 3); }), 16.0 * 8 * 256);
    rep3("imma s8 m16n8k32", timeit([&]{ k_imma<<<blocks, TPB>>>((int*)out, 3); }), 16.0 * 8 * 32);
  }
  CK(cudaGetLastError()); CK(cudaDeviceSynchronize());
  printf("done\n");
  return 0;
}
