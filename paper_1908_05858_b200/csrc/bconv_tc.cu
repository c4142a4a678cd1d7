// Binary convolution on the 5th-generation tensor cores (tcgen05) -- the same integers as the xor/popcount kernel
// (Section 2.1.2, Eq. 1 of the paper, read as a +-1 dot product), computed as a dense low-precision contraction.
//
// sm_100a has no native 1-bit MMA (mma.sync ... b1 is emulated and tcgen05 has no 1-bit kind), so the +-1 values
// are expanded on chip to the narrowest type the tensor core takes: 4-bit e2m1 (+1.0 = 0x2, -1.0 = 0xA), used through
// the block-scaled kind::mxf4 with every scale factor set to 1.0 (ue8m0 127).  Products are +-1 and the fp32
// accumulator adds at most K < 2^24 of them, so the result is the exact integer.  HBM still holds one bit per value.
//
//   * Weights: expanded once (dabnn_tc_prepare_weights) to e2m1 rows of 16 bytes = 32 channels, stored in blocks of 32
//     output channels ([O/32][tap][C/32][32][16 B]); a persistent CTA copies the rows of its output channels into the
//     UMMA K-major, no-swizzle core-matrix layout in shared memory once and keeps them for all its pixel tiles -- as
//     many channel tiles as fit, so that a tile of activations is expanded once for all of them.
//   * CTA pairs: where the launch is large enough, two CTAs of a cluster share every MMA (cta_group::2, M = 256: each
//     CTA's 128 rows against N columns of which each CTA holds half).  Per MMA a CTA then reads half the weights from
//     its shared memory -- the tensor pipe's operand reads are what saturates shared memory in the one-CTA form -- and
//     the pair keeps twice the channels resident.  The leader CTA issues; producers and epilogue warps of the peer
//     signal the leader's barriers through the cluster's shared-memory window.
//   * Activations: a tile is 128 consecutive "slots" q of the padded image grid (slot pitch SP and HP slot rows per
//     image: W + pad_w and H + pad_h at stride 1, see below).  The CTA reads the packed bits of the 128 + (kh-1)*SP + (kw-1) slots it
//     needs, expands them to e2m1 rows of 32 channels ([C/32][slots][16 B]) -- padded slots get the declared pad
//     value -- and every filter tap (i, j) is the SAME array read from a start address shifted by (i*SP + j) rows:
//     with a 16-byte row pitch a shift by one slot is a 16-byte step of the matrix descriptor, so no im2col copy
//     is ever materialised.  Rows that fall on padding columns / rows compute garbage that is never stored; at stride 1
//     only the left / top padding has slots of its own (the right / bottom taps read the next row's / image's).
//   * Stride 2 keeps four parity planes of the padded input; tap (i, j) reads plane (i mod 2, j mod 2) shifted by
//     (i div 2, j div 2).
//   * Warp-specialised and mbarrier-driven: four producer warps prefetch the bits two tiles ahead, expand them
//     (table-free, see expand16) into one of up to four A buffers and arrive on `a_full`; one thread of a
//     separate warp waits for it, issues kh*kw*(C/64) tcgen05.mma (M = 128, N = NT, K = 64) into one of up to four
//     TMEM accumulators per resident channel tile and commits to `mma_done` (and, after the tile's last MMA, to `a_free`);
//     four (or eight) epilogue warps wait for that, read the accumulator with tcgen05.ld, write the output form, and hand the
//     accumulator back through `tmem_free`.  The fused BN + sign form is one compare per value against a per-channel
//     integer threshold that each CTA derives from (scale, shift) at start-up.
//
// Every wait on an mbarrier is bounded: on expiry the kernel records an error flag, stops, frees its TMEM and returns.
#include "common.cuh"

#include <cuda.h>  // the tensor-map type and enums only: the one driver function used is looked up at run time

namespace dabnn {

namespace {

enum { EPI_I32 = 0, EPI_BNPACK = 1, EPI_BIREAL = 2 };

constexpr int TC_THREADS = 416;           // warps 0-3 and (optionally) 8-11: epilogue, 4-7: producers, 12: MMA issue
constexpr int TC_SMEM_LIMIT = 232448;     // 227 KB opt-in maximum per CTA
constexpr int TC_MAX_RES = 4;              // channel tiles resident per CTA (pair) at most
constexpr int TC_SMEM_HDR = 512;           // barriers, TMEM base, flags
constexpr int TC_SMEM_MISC = TC_SMEM_HDR + 2 * TC_MAX_RES * 128 * 4;  // ... and this CTA's scale / shift
constexpr int TC_RING_MAX = 4;             // residual chunks in flight per epilogue warp at most
constexpr int TC_RING_CHUNK = 4096;        // one chunk: 32 rows x 32 fp32 channels
constexpr int TC_WEIGHT_BUDGET = 147456;  // 144 KB of resident weights at most
constexpr int TC_MAX_CW = 8;              // words of a row that a producer thread holds: 512 channels per channel group
constexpr int TC_MAX_SPT = 5;             // slots per producer thread: 2 for stride 1, up to 5 for stride 2
constexpr int TC_TMEM_COLS = 512;         // the accumulators' columns + the scale-factor columns
constexpr int TC_WAIT_POLLS = 1 << 20;    // polls of a barrier wait before it gives up (about a second)
constexpr int TC_ACC_COLS = 384;          // columns [0, 384): up to four accumulators (three of 128 columns)
constexpr int TC_SF_COL = 384;            // columns [384, 512) hold scale factors (all 1.0)
constexpr int TC_MAX_BUFS = 4;            // accumulators / activation buffers in flight at most

__device__ int g_tc_error = 0;  // 1: an mbarrier wait ran out (one copy per device; cleared when read by dabnn_last_device_flag)
int g_tc_max_ctas = 0;          // host: CTAs per launch at most (0: one per SM)

struct TcArgs {
  const uint64_t* a;
  const uint8_t* w_tc;
  int N, H, W, Cw, C;
  int O, kh, kw, ph, pw, OH, OW;
  int S;               // stride (1 or 2, both axes)
  int SPin, HPin;      // padded input extent covered by the slot grid: W + 2*pad_w, H + 2*pad_h (one pad each at stride 1)
  int SP, HP;          // slot grid per image: ceil(SPin / S) columns, ceil(HPin / S) rows; output (oh, ow) sits at slot (oh, ow)
  long long total_q;   // N * HP * SP
  unsigned long long magic_sp, magic_hp;  // ceil(2^64 / SP), ceil(2^64 / HP) (0 when the divisor is 1)
  int slots_p;         // slots per parity plane and tile, multiple of 8
  int slots;           // S*S*slots_p: rows of one 32-channel group in an A buffer
  int abufs;           // A buffers in shared memory (1 to 4)
  int nacc;            // accumulators in tensor memory (2 to 4: as many as fit 384 columns)
  int ntile, n_ntiles; // output channels per MMA (N), number of such channel tiles
  int pair;            // 1: CTA pairs (cta_group::2), each CTA holds ntile / 2 weight rows per channel tile
  int nres, n_groups;  // channel tiles resident per CTA (pair), groups of `nres` channel tiles
  int epi2;            // 1: warps 8-11 share the epilogue with warps 0-3
  long long m_tiles;   // tiles of 128 slots (a pair takes two consecutive ones at a time)
  int pad_neg;
  int32_t* out;
  int out_nchw;
  const float* scale;
  const float* shift;
  const float* residual;
  float* y_out;
  uint32_t* out_packed32;
  int Ow32;
  int chained;         // 1: launched with programmatic stream serialization by the Bi-Real forward, whose weights and BN
                       // vectors are constants: the kernel starts while its predecessor's last CTAs still run, sets up
                       // (tensor memory, barriers, thresholds, the weight copy) and only then waits for the predecessor
  int wait_polls;      // polls of a barrier wait before it gives up (TC_WAIT_POLLS; smaller only in the expiry self-test)
  int extra_arrivals;  // 0; the expiry self-test makes `a_full` expect one arrival more than the producers make
  int kgroups, gw;     // channel groups of `gw` 64-bit words (8, or 4 where a thread holds five rows) that a tile's channels
                       // pass through the activation buffers in; 1 group = all channels at once (C <= 512 / 256)
  int res_ring;        // > 0: the residual reaches the epilogue warps as bulk tensor copies into a ring of this many
                       // 4 KB chunks per warp (res_map: [pixels][O] fp32, boxes of 32 rows x 32 channels, 128-byte swizzle)
  alignas(64) CUtensorMap res_map;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Bounded wait for the given phase parity; false if it ran out, or if another role of this CTA has given up (`fail`,
// looked at only now and then: shared-memory reads are slow while the tensor pipe streams its operands).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* fail, int limit) {
  for (int tries = 0; tries < limit; tries++) {  // about a microsecond per poll; then give up
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, 0x400;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if ((tries & 1023) == 1023 && *fail != 0) return false;
  }
  return false;
}
// The same with cluster-scope acquire: the arrivals may come from the peer CTA.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* fail, int limit) {
  for (int tries = 0; tries < limit; tries++) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, 0x400;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity)
        : "memory");
    if (done) return true;
    if ((tries & 1023) == 1023 && *fail != 0) return false;
  }
  return false;
}
// Address of the leader CTA's copy of a shared-memory object, in the cluster's shared window; arrive on it.
__device__ __forceinline__ uint32_t leader_addr(uint32_t local) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, 0;" : "=r"(r) : "r"(local));
  return r;
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
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

// 16 sign bits -> 16 e2m1 nibbles (8 bytes): +1.0 = 0x2 (bit 0), -1.0 = 0xA (bit 1).
// A byte permute whose source register holds the four possible bytes 0x22, 0x2A, 0xA2, 0xAA maps a 2-bit pair value
// to its byte; `h & 0x3333` and `(h >> 2) & 0x3333` already are four valid selector nibbles each, so the expansion is
// three logic ops and two PRMTs, with no table.  Channels land in a permuted order inside their 16-byte row
// (pairs 0,2,4,6 then 1,3,5,7): activations and weights go through this same function, and a dot product does not
// care about the order of its terms.
__device__ __forceinline__ uint2 expand16(uint32_t h) {
  return make_uint2(__byte_perm(0xAAA22A22u, 0u, h & 0x3333u), __byte_perm(0xAAA22A22u, 0u, (h >> 2) & 0x3333u));
}
__device__ __forceinline__ uint4 expand32(uint32_t w) {
  const uint2 lo = expand16(w & 0xFFFFu), hi = expand16(w >> 16);
  return make_uint4(lo.x, lo.y, hi.x, hi.y);
}

// 256-bit global store / load (32-byte aligned): a lane writes a whole 32-byte sector of its output row at once.
// The load (the fp32 residual stream, read once) does not allocate in L1: measured 3 % on the whole Bi-Real forward.
__device__ __forceinline__ void st_global_v8(void* p, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e, uint32_t f,
                                             uint32_t g2, uint32_t h) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(p), "r"(a), "r"(b), "r"(c), "r"(d), "r"(e),
               "r"(f), "r"(g2), "r"(h)
               : "memory");
}
// The same with an evict-first policy in L2 (made once per thread): for output that nothing in this library reads back (the
// int32 sums), so that it drains to DRAM as it is produced instead of displacing the weights and activations that the
// next launches read.
__device__ __forceinline__ uint64_t evict_first_policy() {
  uint64_t pol;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
  return pol;
}
__device__ __forceinline__ void st_global_v8_stream(void* p, uint64_t pol, uint32_t a, uint32_t b, uint32_t c, uint32_t d, uint32_t e,
                                                    uint32_t f, uint32_t g2, uint32_t h) {
  asm volatile("st.global.L2::cache_hint.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8}, %9;" ::"l"(p), "r"(a), "r"(b), "r"(c),
               "r"(d), "r"(e), "r"(f), "r"(g2), "r"(h), "l"(pol)
               : "memory");
}
__device__ __forceinline__ void ld_global_v8(const void* p, float (&r)[8]) {
  asm volatile("ld.global.L1::no_allocate.v8.f32 {%0, %1, %2, %3, %4, %5, %6, %7}, [%8];"
               : "=f"(r[0]), "=f"(r[1]), "=f"(r[2]), "=f"(r[3]), "=f"(r[4]), "=f"(r[5]), "=f"(r[6]), "=f"(r[7])
               : "l"(p));
}

// Read-only-path load of activation bits.  Volatile asm, not __ldg: the compiler treats __ldg as an invariant load that it
// may move anywhere, also above the wait of a chained launch, before which the previous kernel may not have written the bits.
__device__ __forceinline__ uint64_t ld_nc_u64(const uint64_t* p) {
  uint64_t v;
  asm volatile("ld.global.nc.b64 %0, [%1];" : "=l"(v) : "l"(p));
  return v;
}

// The fp32 accumulator holds an exact integer of magnitude <= K < 2^22: adding 1.5 * 2^23 leaves it in the low mantissa
// bits (two full-rate instructions instead of a conversion).
__device__ __forceinline__ uint32_t acc_to_int(uint32_t acc_bits) {
  return __float_as_uint(__fadd_rn(__uint_as_float(acc_bits), 12582912.0f)) - 0x4B400000u;
}

template <int V>
struct IntC { static constexpr int value = V; };

// floor(q / d) for q < 2^32 and 1 <= d < 2^16 with magic = ceil(2^64 / d): one 64-bit multiply-high instead of a division.
__device__ __forceinline__ uint32_t fast_div(uint32_t q, unsigned long long magic) {
  return magic == 0 ? q : (uint32_t)__umul64hi((unsigned long long)q, magic);
}

// KG: more channels than one activation buffer takes (C > 512, or > 256 at stride 2).  The weights stay resident; the
// activations of a tile pass through the ring of activation buffers one channel group (g.gw words per row) at a time and
// the MMAs of all groups add up in the same accumulator.  One channel tile per CTA, no CTA pairs.
template <int NT, int EPI, int SPT, bool PAIR, bool RES_TMA = false, bool KG = false>
__global__ void __launch_bounds__(TC_THREADS, 1) bconv_tc_kernel(const __grid_constant__ TcArgs g) {
  extern __shared__ __align__(1024) uint8_t smem[];
  constexpr int WR = PAIR ? NT / 2 : NT;  // weight rows (output channels) of one channel tile held by this CTA
  constexpr uint32_t PEERS = PAIR ? 2 : 1;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = PAIR ? cluster_ctarank() : 0u;   // 0: the CTA that issues the pair's MMAs
  const int Kb = g.kh * g.kw * (g.C >> 1);               // bytes per weight row
  const int a_bytes = KG ? g.slots * g.gw * 32 : g.slots * (g.C >> 1);  // bytes of one A buffer (one channel group)
  uint8_t* w_s = smem;                                   // [nres][taps][C/32][WR][16]
  uint8_t* a_s = smem + (size_t)g.nres * WR * Kb;        // [abufs][C/32][slots][16]
  uint8_t* misc = a_s + (size_t)g.abufs * a_bytes;
  // [0..3] mma_done  [4..7] tmem_free  [8..11] a_full  [12..15] a_free  [16..18] w_full (thirds of the filter taps);
  // of a pair, the leader's tmem_free, a_full and w_full are used
  uint64_t* bars = reinterpret_cast<uint64_t*>(misc);
  constexpr int B_MMA_DONE = 0, B_TMEM_FREE = 4, B_A_FULL = 8, B_A_FREE = 12, B_W_FULL = 16;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(misc + 160);
  volatile int* s_fail = reinterpret_cast<volatile int*>(misc + 168);
  // [32 + 4 * e ..]: `res_full` of epilogue warp e's ring of residual chunks
  constexpr int B_RES_FULL = 32;
  float* s_scale = reinterpret_cast<float*>(misc + TC_SMEM_HDR);  // [nres][NT] this CTA's channels
  float* s_shift = s_scale + TC_MAX_RES * NT;                // [nres][NT]

  // work: CTA (pair) `unit` takes channel-tile group `ng` and every `unit_step`-th tile (pair of tiles) of 128 slots
  const int unit = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
  const int units = PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x;
  const int ng = unit % g.n_groups;
  const long long mt_first = (long long)(unit / g.n_groups) * PEERS + rank;
  const long long mt_step = (long long)(units / g.n_groups) * PEERS;
  const int nres_here = min(g.nres, g.n_ntiles - ng * g.nres);  // channel tiles of this group that exist
  // a pair runs while its leader has a tile (the peer's last tile may lie beyond the end: pad rows, nothing stored)
  const long long mt_end = PAIR ? (g.m_tiles + 1) / 2 * 2 : g.m_tiles;

  if (g.chained) chain_trigger();  // the successor may start as CTAs of this launch leave (it waits for all of them itself)
  if (EPI == EPI_BIREAL) {
    for (int i = tid; i < nres_here * NT; i += TC_THREADS) {
      const int o = (ng * g.nres + i / NT) * NT + (i % NT);
      s_scale[i] = (o < g.O) ? g.scale[o] : 0.0f;
      s_shift[i] = (o < g.O) ? g.shift[o] : 0.0f;
    }
  }
  if (EPI == EPI_BNPACK) {
    // The sign of fmaf(acc, scale, shift) as a threshold on the integer acc: fmaf is monotone in acc (the exact value is,
    // and rounding keeps order), so { acc in [-K, K] : fmaf(acc, scale, shift) < 0 } is empty, everything, a prefix
    // (scale > 0) or a suffix (scale < 0) of the range -- also for infinite or NaN scale / shift, where the comparison is
    // false wherever the value is NaN.  A bisection with the very fmaf finds the boundary; the epilogue then needs one
    // compare per value: bit = (acc <= T) xor flip, with T in s_scale and one flip bit per channel in s_shift's place.
    uint32_t* s_flip = reinterpret_cast<uint32_t*>(s_shift);
    const int K = g.kh * g.kw * g.C;
    for (int i = tid; i < nres_here * NT; i += TC_THREADS) {  // (whole warps: NT is a multiple of 32)
      const int o = (ng * g.nres + i / NT) * NT + (i % NT);
      const float sc = (o < g.O) ? g.scale[o] : 0.0f, sh = (o < g.O) ? g.shift[o] : 0.0f;
      auto neg = [&](int a) { return __fmaf_rn((float)a, sc, sh) < 0.0f; };
      const bool first = neg(-K), last = neg(K);
      float T;
      uint32_t flip = 0;
      if (first == last) {
        T = first ? (float)(K + 1) : (float)(-K - 1);  // everything / nothing
      } else {
        int lo = -K, hi = K;  // neg(lo) == first, neg(hi) == last
        while (hi - lo > 1) {
          const int mid = lo + ((hi - lo) >> 1);
          if (neg(mid) == first) lo = mid;
          else hi = mid;
        }
        T = (float)lo;        // prefix: negative for acc <= lo; suffix: negative for acc >= hi, i.e. not (acc <= lo)
        flip = first ? 0u : 1u;
      }
      s_scale[i] = T;
      const uint32_t mask = __ballot_sync(0xFFFFFFFFu, flip != 0);
      if (lane == 0) s_flip[i >> 5] = mask;
    }
  }
  if (tid == 0) {
    for (int i = 0; i < TC_MAX_BUFS; i++) {
      mbar_init(smem_u32(&bars[B_MMA_DONE + i]), 1);
      mbar_init(smem_u32(&bars[B_TMEM_FREE + i]), (g.epi2 ? 8 : 4) * PEERS);  // one arrival per epilogue warp
      mbar_init(smem_u32(&bars[B_A_FULL + i]), 4 * PEERS + (uint32_t)g.extra_arrivals);  // one arrival per producer warp
      mbar_init(smem_u32(&bars[B_A_FREE + i]), 1);
    }
    for (int i = 0; i < 3; i++) mbar_init(smem_u32(&bars[B_W_FULL + i]), TC_THREADS * PEERS);
    if (RES_TMA)
      for (int i = 0; i < 8 * TC_RING_MAX; i++) mbar_init(smem_u32(&bars[B_RES_FULL + i]), 1);  // the warp's issuing lane
    *s_fail = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    if (PAIR) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"((uint32_t)TC_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)),
                   "r"((uint32_t)TC_TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  // The start-up barrier: barriers initialised (in both CTAs of a pair, before either signals the other's) and the
  // tensor-memory address published.  Each warp passes it once, as late as its role allows: the weight copy and the
  // producers' first requests for activation bits are already in flight by then.
  auto prologue_sync = [&]() {
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    if (PAIR) cluster_sync_all();
    else __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  };
  const bool is_producer = warp >= 4 && warp < 8;
  uint32_t tmem_base = 0;
  // barriers that both CTAs of a pair signal live in the leader
  const uint32_t bar_tmem_free0 = PAIR ? leader_addr(smem_u32(&bars[B_TMEM_FREE])) : smem_u32(&bars[B_TMEM_FREE]);
  const uint32_t bar_a_full0 = PAIR ? leader_addr(smem_u32(&bars[B_A_FULL])) : smem_u32(&bars[B_A_FULL]);
  const uint32_t bar_w_full = PAIR ? leader_addr(smem_u32(&bars[B_W_FULL])) : smem_u32(&bars[B_W_FULL]);  // + 8, + 16: the later thirds
  auto arrive = [&](uint32_t bar) {
    if (PAIR) mbar_arrive_cluster(bar);
    else mbar_arrive(bar);
  };
  {
    // Resident weights: rows [rank * WR, +WR) of every channel tile of this group, one (tile, tap, 32-channel group)
    // block of WR rows per warp and step; the source holds blocks of 32 output channels.  The producers do not wait
    // for their share until their first tile's rows are out, so the copy overlaps the first expansion.
    // The copy goes in three groups, thirds of the (tap, 32-channel group) blocks in issue order -- for a 3x3 filter
    // one row of taps each -- with a barrier per group: the first MMAs start when the first third has landed.
    const int TG = g.kh * g.kw * (g.C >> 5);
#pragma unroll 1
    for (int j = 0; j < 3; j++) {
      const int lo = TG * j / 3, cnt = TG * (j + 1) / 3 - lo;
      for (int idx = warp; idx < nres_here * cnt; idx += TC_THREADS / 32) {
        const int r = idx / cnt, tg = lo + idx - r * cnt;
        const int col0 = (ng * g.nres + r) * NT + (int)rank * WR;
        uint8_t* dst = w_s + (size_t)(r * TG + tg) * WR * 16;
        for (int n = lane; n < WR; n += 32) {
          const int col = col0 + n;
          cp_async16(smem_u32(dst + n * 16), g.w_tc + (((size_t)(col >> 5) * TG + tg) * 32 + (col & 31)) * 16);
        }
      }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
  }
  // this thread's share of each third has landed -> one arrival on that third's barrier
  auto weights_arrive = [&]() {
    asm volatile("cp.async.wait_group 2;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    arrive(bar_w_full);
    asm volatile("cp.async.wait_group 1;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    arrive(bar_w_full + 8u);
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    arrive(bar_w_full + 16u);
  };
  // (chained launches: nothing above reads or writes what the previous kernel of the stream produces or still reads; the
  // activation bits, the residual and every output come after this point.  A no-op in an ordinary launch.)
  chain_wait();
  if (!is_producer) {
    prologue_sync();
    tmem_base = *tmem_slot;
  }
  if (warp < 4 || warp >= 8) {
    if (warp < 4) {
      // every byte of the scale-factor columns is ue8m0 127 = 1.0, whatever their layout
      const uint32_t one = 0x7F7F7F7Fu;
      for (int c = TC_SF_COL; c < TC_TMEM_COLS; c += 16) {
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * warp) << 16) + (uint32_t)c;
        asm volatile(
            "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1, %1};" ::"r"(taddr),
            "r"(one)
            : "memory");
      }
      asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    weights_arrive();  // one arrival per thread of the CTA (pair) in all: weights (by thirds) and scale factors are in place
  }

  if (warp == 12) {
    // ================= MMA issue: one thread (of the leader CTA) ==================================================
    // The chain below is all there is between two MMAs of this CTA, so it is kept to 32-bit adds: only the start-address
    // field (low 14 bits of a descriptor's low word) changes from one MMA to the next, and shared-memory addresses in
    // 16-byte units never carry out of it.
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 7) | (1u << 10)          // A, B: e2m1
                             | ((uint32_t)(NT >> 3) << 17)   // N
                             | (1u << 23)                    // scale factors: ue8m0
                             | ((uint32_t)((PAIR ? 256 : 128) >> 4) << 24);  // M; both operands K-major; K = 64
      const uint32_t tsfa = tmem_base + TC_SF_COL, tsfb = tmem_base + TC_SF_COL + 64;
      const uint64_t bdesc0 = make_desc(smem_u32(w_s), (uint32_t)WR * 16, 128);
      const uint32_t desc_hi = (uint32_t)(bdesc0 >> 32);  // same for A and B: core matrices 128 bytes apart along M / N
      const uint32_t b_lo0 = (uint32_t)bdesc0;
      const uint32_t a_lo_first = (uint32_t)make_desc(smem_u32(a_s), (uint32_t)g.slots * 16, 128);
      const uint32_t a_buf_units = (uint32_t)a_bytes >> 4;  // one A buffer, in 16-byte units
      const uint32_t a_step = 2u * (uint32_t)g.slots;  // one K = 64 block of A, in 16-byte units
      constexpr uint32_t b_step = 2u * WR;             // weights are laid out in issue order: [tile][tap][C/32][WR][16]
      const uint32_t b_tile = (uint32_t)(g.kh * g.kw * g.Cw) * b_step;  // one resident channel tile
      const int sshift = g.S - 1, smask = g.S - 1;     // stride 1 or 2: masks and shifts instead of divisions
      // tap (ti, tj) reads parity plane (ti % S, tj % S) from a start shifted by (ti / S) slot rows and (tj / S) slots
      auto tap_offset = [&](int ti, int tj) {
        const uint32_t plane = (uint32_t)(((ti & smask) << sshift) + (tj & smask));
        return plane * (uint32_t)g.slots_p + (uint32_t)((ti >> sshift) * g.SP + (tj >> sshift));
      };
      auto mma = [&](uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo, uint32_t accumulate) {
        if (PAIR) {
          asm volatile(
              "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
              "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
              "tcgen05.mma.cta_group::2.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%7], p;\n\t}"
              ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
              : "memory");
        } else {
          asm volatile(
              "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
              "mov.b64 da, {%1, %3};\n\tmov.b64 db, {%2, %3};\n\tsetp.ne.b32 p, %5, 0;\n\t"
              "tcgen05.mma.cta_group::1.kind::mxf4.block_scale.block32 [%0], da, db, %4, [%6], [%7], p;\n\t}"
              ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(desc_hi), "r"(idesc), "r"(accumulate), "r"(tsfa), "r"(tsfb)
              : "memory");
        }
      };
      // completion of everything issued so far -> one arrival on the barrier at this offset (in both CTAs of a pair)
      auto commit = [&](uint32_t bar) {
        if (PAIR)
          asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
                       "h"((uint16_t)3)
                       : "memory");
        else
          asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
      };
      auto wait = [&](uint32_t bar, uint32_t parity) {
        return PAIR ? mbar_wait_cluster(bar, parity, s_fail, g.wait_polls) : mbar_wait(bar, parity, s_fail, g.wait_polls);
      };
      const bool k3 = g.kh == 3 && g.kw == 3;
      uint32_t off9[9];
#pragma unroll
      for (int t = 0; t < 9; t++) off9[t] = k3 ? tap_offset(t / 3, t % 3) : 0u;
      // all MMAs of one tile and channel tile; KB = C / 64 as a compile-time constant, the 3x3 filter fully unrolled
      // (KG: `more` = 1 for every channel group after a tile's first: its MMAs add to what the groups before left; the
      // weights of a tap are g.Cw K blocks apart, of which this group's KB start at b_base)
      auto issue_tile = [&](uint32_t d_tmem, uint32_t a_lo0, uint32_t b_base, uint32_t a_stp, bool first, uint32_t more, auto kbc) {
        constexpr int KB = decltype(kbc)::value;
        const uint32_t tap_blocks = KG ? (uint32_t)g.Cw : (uint32_t)KB;
        if (k3) {
#pragma unroll
          for (int t = 0; t < 9; t++) {
            if (!KG && first && (t == 3 || t == 6) && !wait(smem_u32(&bars[B_W_FULL + t / 3]), 0)) *s_fail = 1;  // that row of taps
            const uint32_t a_lo = a_lo0 + off9[t];
#pragma unroll
            for (int kb = 0; kb < KB; kb++)
              mma(d_tmem, a_lo + (uint32_t)kb * a_stp, b_base + ((uint32_t)t * tap_blocks + (uint32_t)kb) * b_step, (t | kb) ? 1u : more);
          }
        } else {
          if (!KG && first && !(wait(smem_u32(&bars[B_W_FULL + 1]), 0) && wait(smem_u32(&bars[B_W_FULL + 2]), 0))) *s_fail = 1;
          uint32_t b_tap = b_base, accumulate = more;
          for (int ti = 0; ti < g.kh; ti++)
            for (int tj = 0; tj < g.kw; tj++, b_tap += tap_blocks * b_step) {
              const uint32_t a_lo = a_lo0 + tap_offset(ti, tj);
#pragma unroll
              for (int kb = 0; kb < KB; kb++) {
                mma(d_tmem, a_lo + (uint32_t)kb * a_stp, b_tap + (uint32_t)kb * b_step, accumulate);
                accumulate = 1;
              }
            }
        }
      };
      uint32_t ab = 0, a_phase = 0;  // A buffer of this tile and the parity of its `a_full` phase
      uint32_t accb = 0, acc_phase = 0;  // accumulator of this round and the parity of its uses so far
      int ar = 0;                    // accumulator rounds so far: one per (tile, resident channel tile)
      bool ok = wait(smem_u32(&bars[B_W_FULL]), 0);  // first third of the resident weights, and the scale factors
      if (KG) ok = ok && wait(smem_u32(&bars[B_W_FULL + 1]), 0) && wait(smem_u32(&bars[B_W_FULL + 2]), 0);  // ... all of them
      if (!ok) *s_fail = 1;
      if constexpr (KG) {
#pragma unroll 1
        for (long long mt = mt_first; mt < mt_end && ok; mt += mt_step, ar++) {
          if (ar >= g.nacc && !wait(smem_u32(&bars[B_TMEM_FREE + accb]), acc_phase ^ 1u)) { *s_fail = 1; break; }  // accumulator drained
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t d_tmem = tmem_base + accb * (uint32_t)NT;
#pragma unroll 1
          for (int grp = 0; grp < g.kgroups; grp++) {
            if (!wait(smem_u32(&bars[B_A_FULL + ab]), a_phase)) { *s_fail = 1; ok = false; break; }  // this group's rows written
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_lo0 = a_lo_first + ab * a_buf_units;
            const uint32_t b_base = b_lo0 + (uint32_t)(grp * g.gw) * b_step;
            const int kbs = min(g.gw, g.Cw - grp * g.gw);  // K blocks of this group
            const uint32_t more = grp ? 1u : 0u;
            switch (kbs) {
              case 1: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<1>{}); break;
              case 2: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<2>{}); break;
              case 3: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<3>{}); break;
              case 4: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<4>{}); break;
              case 5: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<5>{}); break;
              case 6: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<6>{}); break;
              case 7: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<7>{}); break;
              default: issue_tile(d_tmem, a_lo0, b_base, a_step, false, more, IntC<8>{}); break;
            }
            commit(smem_u32(&bars[B_A_FREE + ab]));  // the group's rows have been read: the A buffer may be refilled
            if (++ab == (uint32_t)g.abufs) { ab = 0; a_phase ^= 1u; }
          }
          if (!ok) break;
          commit(smem_u32(&bars[B_MMA_DONE + accb]));
          if (++accb == (uint32_t)g.nacc) { accb = 0; acc_phase ^= 1u; }
        }
      } else
#pragma unroll 1
      for (long long mt = mt_first; mt < mt_end && ok; mt += mt_step) {
        if (!wait(smem_u32(&bars[B_A_FULL + ab]), a_phase)) { *s_fail = 1; break; }  // rows written
        const uint32_t a_lo0 = a_lo_first + ab * a_buf_units;
        // (opaque to the compiler, so that it does not keep every tap's and K block's offset in a register of its own
        // across tiles: the sums are recomputed per tile, one add each)
        uint32_t a_step_t = a_step;
        asm volatile("" : "+r"(a_step_t));
#pragma unroll 1
        for (int r = 0; r < nres_here; r++, ar++) {
          if (ar >= g.nacc && !wait(smem_u32(&bars[B_TMEM_FREE + accb]), acc_phase ^ 1u)) { *s_fail = 1; ok = false; break; }  // accumulator drained
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t d_tmem = tmem_base + accb * (uint32_t)NT;
          const uint32_t b_base = b_lo0 + (uint32_t)r * b_tile;
          switch (g.Cw) {  // C / 64 = 1..8
            case 1: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<1>{}); break;
            case 2: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<2>{}); break;
            case 3: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<3>{}); break;
            case 4: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<4>{}); break;
            case 5: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<5>{}); break;
            case 6: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<6>{}); break;
            case 7: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<7>{}); break;
            default: issue_tile(d_tmem, a_lo0, b_base, a_step_t, ar == 0, 0u, IntC<8>{}); break;
          }
          commit(smem_u32(&bars[B_MMA_DONE + accb]));
          if (++accb == (uint32_t)g.nacc) { accb = 0; acc_phase ^= 1u; }
        }
        commit(smem_u32(&bars[B_A_FREE + ab]));  // the tile's rows have been read: the A buffer may be refilled
        if (++ab == (uint32_t)g.abufs) { ab = 0; a_phase ^= 1u; }
      }
    }
  } else if (warp >= 4 && warp < 8) {
    // ================= producer warps: packed bits -> e2m1 rows ===================================================
    const int ptid = tid - 128;
    constexpr int PCW = SPT > 2 ? 4 : TC_MAX_CW;  // words per slot held in registers (stride 2 is limited to C <= 256)
    // Registers of one tile's rows.  A row that is padding -- or lies beyond the batch, where no stored output reads
    // it -- carries the pad pattern as its words, so that the expansion is the same straight-line code for every row.
    struct SlotRegs {
      uint64_t words[SPT][PCW];
    };
    const uint64_t pad_bits = g.pad_neg ? ~0ull : 0ull;
    // Slot coordinates (image, slot row, slot column) of this thread's rows in the next tile to request.  Tiles are
    // requested in order, each `mt_step` tiles = a fixed (dn, dr, dc) after the one before: divisions happen once here.
    int co_n[SPT], co_r[SPT], co_c[SPT], co_plane[SPT];
    const uint32_t D = (uint32_t)mt_step * 128u;
    const uint32_t d_rows = fast_div(D, g.magic_sp);
    const int dc = (int)(D - d_rows * (uint32_t)g.SP);
    const int dn = (int)fast_div(d_rows, g.magic_hp);
    const int dr = (int)(d_rows - (uint32_t)dn * (uint32_t)g.HP);
#pragma unroll
    for (int h = 0; h < SPT; h++) {
      int plane = 0, sp = ptid + 128 * h;  // parity plane of this row (always 0 for stride 1)
      while (sp >= g.slots_p && plane < 3) { sp -= g.slots_p; plane++; }
      const uint32_t Q = (uint32_t)mt_first * 128u + (uint32_t)sp;  // total_q < 2^31 is checked on the host
      const uint32_t rr = fast_div(Q, g.magic_sp);
      const uint32_t n = fast_div(rr, g.magic_hp);
      co_c[h] = (int)(Q - rr * (uint32_t)g.SP);
      co_r[h] = (int)(rr - n * (uint32_t)g.HP);
      co_n[h] = (int)n;
      co_plane[h] = plane;
    }
    int pf_grp = 0;  // (KG) channel group of the next request; the slot coordinates move on after a tile's last group
    auto prefetch = [&](SlotRegs& R, auto cwc) {
      constexpr int CW = decltype(cwc)::value;
      const int sshift = g.S - 1;  // stride 1 or 2
      const int w0 = KG ? pf_grp * CW : 0;            // first word of the group
      const int wn = KG ? g.Cw - w0 : g.Cw;           // words from there on (CW of them are taken at most)
      const bool move_on = !KG || pf_grp + 1 == g.kgroups;
#pragma unroll
      for (int h = 0; h < SPT; h++) {
#pragma unroll
        for (int cw = 0; cw < CW; cw++) R.words[h][cw] = pad_bits;
        if (ptid + 128 * h < g.slots) {
          const int ih = (co_r[h] << sshift) + (co_plane[h] >> sshift) - g.ph;  // un-padded input coordinates
          const int iw = (co_c[h] << sshift) + (co_plane[h] & sshift) - g.pw;
          if (co_n[h] < g.N && ih >= 0 && ih < g.H && iw >= 0 && iw < g.W) {
            const uint64_t* src = g.a + (((long long)co_n[h] * g.H + ih) * g.W + iw) * g.Cw + w0;
#pragma unroll
            for (int cw = 0; cw < CW; cw++)
              if (cw < wn) R.words[h][cw] = ld_nc_u64(src + cw);  // (CW is g.Cw rounded up to 1, 2, 4 or 8)
          }
          if (move_on) {
            co_c[h] += dc;
            if (co_c[h] >= g.SP) { co_c[h] -= g.SP; co_r[h]++; }
            co_r[h] += dr;
            if (co_r[h] >= g.HP) { co_r[h] -= g.HP; co_n[h]++; }
            co_n[h] += dn;
          }
        }
      }
      if (KG && ++pf_grp == g.kgroups) pf_grp = 0;
    };
    int ex_grp = 0;  // (KG) channel group of the rows expanded next
    auto expand = [&](const SlotRegs& R, uint8_t* abuf, auto cwc) {
      constexpr int CW = decltype(cwc)::value;
      const int wn = KG ? g.Cw - ex_grp * CW : g.Cw;  // words of this group (CW of them at most)
      if (KG && ++ex_grp == g.kgroups) ex_grp = 0;
#pragma unroll
      for (int h = 0; h < SPT; h++) {
        const int s = ptid + 128 * h;
        if (s >= g.slots) break;
        uint8_t* dst = abuf + (size_t)s * 16;
        const size_t gstride = (size_t)g.slots * 16;  // bytes between consecutive 32-channel groups
#pragma unroll
        for (int cw = 0; cw < CW; cw++) {
          if (cw >= wn) break;  // warp-uniform
          const uint4 lo = expand32((uint32_t)R.words[h][cw]), hi = expand32((uint32_t)(R.words[h][cw] >> 32));
          *reinterpret_cast<uint4*>(dst + (size_t)(2 * cw) * gstride) = lo;
          *reinterpret_cast<uint4*>(dst + (size_t)(2 * cw + 1) * gstride) = hi;
        }
      }
    };

    int it = 0;
    // Per tile: wait until the A buffer is free, expand the rows held in `cur`, hand them over, move the next tile's
    // bits (requested one tile ago, so they have landed) from `nxt` into `cur`, and request the tile after that into
    // `nxt`: registers that a load is still filling are never touched before the next iteration.
    auto run = [&](auto cwc) {  // the words per row (C / 64) as a compile-time constant
      constexpr int CW = decltype(cwc)::value;
      // (stride 2 holds up to five rows per thread: one register set, requested one tile ahead only)
      constexpr bool TWO_SETS = SPT <= 2;
      SlotRegs cur, nxt;
      long long mt = mt_first;
      prefetch(cur, cwc);  // (rows of a tile beyond the last one are beyond the batch: nothing is read for them)
      if (TWO_SETS) prefetch(nxt, cwc);
      prologue_sync();
      uint32_t ab = 0, use_phase = 0;  // A buffer of this tile and the parity of the number of times it has been filled
      bool stop = false;
#pragma unroll 1
      for (; mt < mt_end && !stop; mt += mt_step)
#pragma unroll 1
      for (int grp = 0; grp < (KG ? g.kgroups : 1); grp++, it++) {  // (KG: a tile's channel groups, one A buffer each)
        // its last reader: all MMAs of the tile that used it, signalled through `a_free` (in both CTAs of a pair)
        // (the decision is taken by the warp as a whole, so that its lanes stay together for the warp-wide steps below)
        if (it >= g.abufs && !__all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&bars[B_A_FREE + ab]), use_phase ^ 1u, s_fail, g.wait_polls))) { *s_fail = 1; stop = true; break; }
        expand(cur, a_s + (size_t)ab * a_bytes, cwc);
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the tensor core
        __syncwarp();  // every lane's rows are written and fenced: one arrival stands for the warp
        if (lane == 0) arrive(bar_a_full0 + 8u * (uint32_t)ab);
        if (it == 0) {
          // the first tile's rows went out before anything else: a short launch is all start-up.  Now this thread's
          // share of the weights.
          weights_arrive();
        }
        if (TWO_SETS) {
#pragma unroll
          for (int h = 0; h < SPT; h++) {
#pragma unroll
            for (int cw = 0; cw < CW; cw++) cur.words[h][cw] = nxt.words[h][cw];
          }
          prefetch(nxt, cwc);
        } else {
          prefetch(cur, cwc);
        }
        if (++ab == (uint32_t)g.abufs) { ab = 0; use_phase ^= 1u; }
      }
    };
    // C is a multiple of 64 up to 512: 1..8 words; the common counts get their own straight-line code
    if constexpr (KG) run(IntC<PCW>{});  // groups of 8 words (4 where a thread holds five rows): g.gw == PCW
    else if (g.Cw == 1) run(IntC<1>{});
    else if (g.Cw == 2) run(IntC<2>{});
    else if (g.Cw <= 4) run(IntC<4>{});
    else if constexpr (PCW > 4) run(IntC<8>{});
    else prologue_sync();  // (not reached: the host launches this instance for C <= 256 only)
  } else if (warp < 4 || g.epi2) {
    // ================= epilogue warps: TMEM accumulator -> output ===============================================
    uint32_t accb = 0, acc_phase = 0;  // accumulator of this round (one per tile and resident channel tile), parity of its uses
    bool failed = false;
    // with the second group, two warps share each quarter of the accumulator's rows: warps 0-3 take the even
    // 32-column chunks, warps 8-11 the odd ones
    const int c_first = warp >= 8 ? 32 : 0;
    const int c_step = g.epi2 ? 64 : 32;
    const uint64_t pol_stream = EPI == EPI_I32 ? evict_first_policy() : 0ull;  // (made once, not per store)
    // The residual as bulk tensor copies (g.res_ring > 0): every epilogue warp owns a ring of 4 KB chunks (32 rows x 32
    // channels) and its lane 0 requests the chunks in the order the warp will use them, `res_ring` chunks ahead -- across
    // tiles, which register prefetch cannot afford.  The valid slots of a warp's 32 rows are consecutive output pixels,
    // so a chunk is the box (first channel, first valid pixel) of the [pixels][O] tensor; rows of the box beyond the
    // warp's pixels (or beyond the tensor: zero fill) are read and ignored.  128-byte swizzle: lane = row reads its 16-byte
    // piece j at (j ^ (row & 7)), free of bank conflicts.
    constexpr bool tma_res = RES_TMA;
    const int ew = warp < 4 ? warp : warp - 4;  // epilogue warp 0..7
    const uint32_t ring0 = ((smem_u32(misc) + (uint32_t)TC_SMEM_MISC + 1023u) & ~1023u) + (uint32_t)(ew * g.res_ring) * TC_RING_CHUNK;
    const uint32_t rbar0 = smem_u32(&bars[B_RES_FULL + ew * TC_RING_MAX]);
    long long mt_i = mt_first;                 // the next chunk to request: tile, resident channel tile, first channel
    int r_i = 0, c0_i = warp >= 8 ? 32 : 0;
    uint32_t slot_i = 0, slot_u = 0, phase_u = 0, in_flight = 0;
    auto issue_next = [&]() {  // (warp-uniform state; lane 0 issues)
      if (mt_i >= mt_end) return;
      if (lane == 0) {
        // output pixels before the warp's first slot = the pixel index of its first valid row
        const uint32_t Q0 = (uint32_t)mt_i * 128u + 32u * (uint32_t)(warp & 3);
        const uint32_t rr0 = fast_div(Q0, g.magic_sp);
        const uint32_t col0 = Q0 - rr0 * (uint32_t)g.SP;
        const uint32_t n0 = fast_div(rr0, g.magic_hp);
        const uint32_t r0 = rr0 - n0 * (uint32_t)g.HP;
        uint32_t m0 = (n0 * (uint32_t)g.OH + min(r0, (uint32_t)g.OH)) * (uint32_t)g.OW + (r0 < (uint32_t)g.OH ? min(col0, (uint32_t)g.OW) : 0u);
        if (n0 >= (uint32_t)g.N) m0 = (uint32_t)g.N * (uint32_t)g.OH * (uint32_t)g.OW;  // beyond the batch: an all-zero box
        const uint32_t bar = rbar0 + 8u * slot_i, dst = ring0 + slot_i * TC_RING_CHUNK;
        const uint32_t ch = (uint32_t)((ng * g.nres + r_i) * NT + c0_i);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((uint32_t)TC_RING_CHUNK) : "memory");
        asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(dst),
                     "l"(reinterpret_cast<uint64_t>(&g.res_map)), "r"(ch), "r"(m0), "r"(bar)
                     : "memory");
      }
      in_flight++;
      if (++slot_i == (uint32_t)g.res_ring) slot_i = 0;
      c0_i += g.epi2 ? 64 : 32;
      if (c0_i >= NT) {
        c0_i = warp >= 8 ? 32 : 0;
        if (++r_i >= nres_here) { r_i = 0; mt_i += mt_step; }
      }
    };
    if (tma_res)
      for (int i = 0; i < g.res_ring; i++) issue_next();
    for (long long mt = mt_first; mt < mt_end && !failed; mt += mt_step) {
      const int row = 32 * (warp & 3) + lane;  // TMEM lane = slot row of the tile
      const uint32_t Q = (uint32_t)mt * 128u + (uint32_t)row;
      const uint32_t rr = fast_div(Q, g.magic_sp);
      const int col = (int)(Q - rr * (uint32_t)g.SP);
      const uint32_t n = fast_div(rr, g.magic_hp);
      const int r = (int)(rr - n * (uint32_t)g.HP);
      const int my_valid = (n < (uint32_t)g.N && r < g.OH && col < g.OW) ? 1 : 0;
      const int my_m = (int)((n * (uint32_t)g.OH + (uint32_t)r) * (uint32_t)g.OW + (uint32_t)col);  // < 2^31 (host check)
      // row of this lane's pixel in the warp's residual chunks: its rank among the warp's valid rows
      const uint32_t srow = tma_res ? (uint32_t)__popc(__ballot_sync(0xFFFFFFFFu, my_valid != 0) & ((1u << lane) - 1u)) : 0u;
      // wide outputs: 256-bit accesses when rows are 32-byte multiples at 32-byte aligned addresses
      const bool wide_i32 = EPI == EPI_I32 && !g.out_nchw && (g.O & 7) == 0 && (reinterpret_cast<uintptr_t>(g.out) & 31) == 0;
      const bool wide_y = EPI == EPI_BIREAL && (g.O & 7) == 0 &&
                          ((reinterpret_cast<uintptr_t>(g.residual) | reinterpret_cast<uintptr_t>(g.y_out)) & 31) == 0;
      for (int r = 0; r < nres_here; r++) {
      const uint32_t buf = accb;
      const int nt = ng * g.nres + r;  // this round's channel tile
      const float* r_scale = s_scale + r * NT;
      const float* r_shift = s_shift + r * NT;
      // The residual does not depend on the MMAs: its first 32 channels are requested before waiting for them, and
      // every later chunk one chunk ahead of its use.
      float rpre[32];
      auto load_res = [&](int c0) {
        if (EPI == EPI_BIREAL && wide_y && my_valid && !tma_res) {
          const int o = nt * NT + c0;
          const int nch = min(32, g.O - o);
          const float* rs = g.residual + (long long)my_m * g.O + o;
#pragma unroll
          for (int q = 0; q < 4; q++)
            if (8 * q < nch) ld_global_v8(rs + 8 * q, *reinterpret_cast<float(*)[8]>(&rpre[8 * q]));
        }
      };
      load_res(c_first);
      if (!__all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&bars[B_MMA_DONE + buf]), acc_phase, s_fail, g.wait_polls))) {
        *s_fail = 1;
        failed = true;
        break;
      }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const long long m = my_m;
#pragma unroll 1
      for (int c0 = c_first; c0 < NT; c0 += c_step) {
        __syncwarp();  // the TMEM load is warp-wide: rejoin lanes that took different paths below
        if constexpr (tma_res) {
          // this chunk has landed (requested `res_ring` chunks ago)
          if (!__all_sync(0xFFFFFFFFu, mbar_wait(rbar0 + 8u * slot_u, phase_u, s_fail, g.wait_polls))) {
            *s_fail = 1;
            failed = true;
            break;
          }
          in_flight--;
          uint32_t v[32];
          const uint32_t taddr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(buf * NT + c0);
          asm volatile(
              "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
              "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
              : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
                "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
                "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
                "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
              : "r"(taddr));
          asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
          const int o = nt * NT + c0;
          if (my_valid && o < g.O) {  // (O is a multiple of 32 on this path: a chunk exists whole or not at all)
            const uint32_t src = ring0 + slot_u * TC_RING_CHUNK + srow * 128u;
            float* yd = g.y_out + m * g.O + o;
            uint32_t word = 0;
#pragma unroll
            for (int q = 0; q < 4; q++) {
              float rc[8], y[8];
#pragma unroll
              for (int h = 0; h < 2; h++) {
                const uint32_t ad = src + ((((uint32_t)(2 * q + h)) ^ (srow & 7u)) << 4);
                asm volatile("ld.shared.v4.f32 {%0, %1, %2, %3}, [%4];"
                             : "=f"(rc[4 * h]), "=f"(rc[4 * h + 1]), "=f"(rc[4 * h + 2]), "=f"(rc[4 * h + 3])
                             : "r"(ad));
                const float4 sc = *reinterpret_cast<const float4*>(r_scale + c0 + 8 * q + 4 * h);
                const float4 sh = *reinterpret_cast<const float4*>(r_shift + c0 + 8 * q + 4 * h);
                y[4 * h] = __fmaf_rn(__uint_as_float(v[8 * q + 4 * h]), sc.x, sh.x);
                y[4 * h + 1] = __fmaf_rn(__uint_as_float(v[8 * q + 4 * h + 1]), sc.y, sh.y);
                y[4 * h + 2] = __fmaf_rn(__uint_as_float(v[8 * q + 4 * h + 2]), sc.z, sh.z);
                y[4 * h + 3] = __fmaf_rn(__uint_as_float(v[8 * q + 4 * h + 3]), sc.w, sh.w);
              }
#pragma unroll
              for (int j = 0; j < 8; j++) {
                y[j] = __fadd_rn(y[j], rc[j]);
                word |= (uint32_t)(y[j] < 0.0f) << (8 * q + j);
              }
              st_global_v8(yd + 8 * q, __float_as_uint(y[0]), __float_as_uint(y[1]), __float_as_uint(y[2]), __float_as_uint(y[3]),
                           __float_as_uint(y[4]), __float_as_uint(y[5]), __float_as_uint(y[6]), __float_as_uint(y[7]));
            }
            if (g.out_packed32 != nullptr) g.out_packed32[m * g.Ow32 + (o >> 5)] = word;
          } else if (my_valid && o < g.Ow32 * 32 && g.out_packed32 != nullptr) {
            g.out_packed32[m * g.Ow32 + (o >> 5)] = 0u;  // sign words are written whole: the half beyond O holds zeros
          }
          // the chunk is in registers (or stored): its buffer takes the next request
          if (++slot_u == (uint32_t)g.res_ring) { slot_u = 0; phase_u ^= 1u; }
          __syncwarp();
          issue_next();
          continue;
        }
        float rc[32];
        if (false) {
        } else if (EPI == EPI_BIREAL) {
#pragma unroll
          for (int j = 0; j < 32; j++) rc[j] = rpre[j];
          if (c0 + c_step < NT) load_res(c0 + c_step);
        }
        uint32_t v[32];
        const uint32_t taddr = tmem_base + ((uint32_t)(32 * (warp & 3)) << 16) + (uint32_t)(buf * NT + c0);
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
            "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
              "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
              "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
            : "r"(taddr));
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
        const int o = nt * NT + c0;  // first of the 32 channels of this chunk; the lane owns them all for its row
        if (!my_valid) continue;
        const int nch = min(32, g.O - o);  // channels of this chunk that exist (<= 0: none)
        if (EPI == EPI_I32) {
          if (nch <= 0) continue;
          if (wide_i32) {
            int32_t* dst = g.out + m * g.O + o;
#pragma unroll
            for (int q = 0; q < 4; q++)
              if (8 * q < nch)  // nch is a multiple of 8 here
                st_global_v8_stream(dst + 8 * q, pol_stream, acc_to_int(v[8 * q]),
                             acc_to_int(v[8 * q + 1]),
                             acc_to_int(v[8 * q + 2]),
                             acc_to_int(v[8 * q + 3]),
                             acc_to_int(v[8 * q + 4]),
                             acc_to_int(v[8 * q + 5]),
                             acc_to_int(v[8 * q + 6]),
                             acc_to_int(v[8 * q + 7]));
          } else if (!g.out_nchw) {
            int32_t* dst = g.out + m * g.O + o;
#pragma unroll
            for (int j = 0; j < 32; j++)
              if (j < nch) __stcs(reinterpret_cast<uint32_t*>(dst) + j, acc_to_int(v[j]));
          } else {
            const long long ohw = (long long)g.OH * g.OW;
            const long long nn = m / ohw, q = m - nn * ohw;
#pragma unroll
            for (int j = 0; j < 32; j++)
              if (j < nch) __stcs(reinterpret_cast<uint32_t*>(g.out) + (nn * g.O + o + j) * ohw + q, acc_to_int(v[j]));
          }
        } else if (EPI == EPI_BNPACK) {
          if (o >= g.Ow32 * 32) continue;  // sign words are written whole (tail bits 0), nothing beyond them
          uint32_t word = 0;
#pragma unroll
          for (int q = 0; q < 8; q++) {
            const float4 t4 = *reinterpret_cast<const float4*>(r_scale + c0 + 4 * q);  // thresholds (see the prologue)
            word |= (uint32_t)(__uint_as_float(v[4 * q]) <= t4.x) << (4 * q);
            word |= (uint32_t)(__uint_as_float(v[4 * q + 1]) <= t4.y) << (4 * q + 1);
            word |= (uint32_t)(__uint_as_float(v[4 * q + 2]) <= t4.z) << (4 * q + 2);
            word |= (uint32_t)(__uint_as_float(v[4 * q + 3]) <= t4.w) << (4 * q + 3);
          }
          word ^= reinterpret_cast<const uint32_t*>(s_shift)[(r * NT + c0) >> 5];
          word &= nch >= 32 ? 0xFFFFFFFFu : (nch > 0 ? (1u << nch) - 1u : 0u);  // channels beyond O: bit 0
          g.out_packed32[m * g.Ow32 + (o >> 5)] = word;
        } else {
          if (o >= g.Ow32 * 32) continue;  // sign words are written whole (tail bits 0), nothing beyond them
          float y[32];
#pragma unroll
          for (int q = 0; q < 8; q++) {  // channels beyond O have scale = shift = 0: y = +0
            const float4 sc = *reinterpret_cast<const float4*>(r_scale + c0 + 4 * q);
            const float4 sh = *reinterpret_cast<const float4*>(r_shift + c0 + 4 * q);
            y[4 * q] = __fmaf_rn(__uint_as_float(v[4 * q]), sc.x, sh.x);
            y[4 * q + 1] = __fmaf_rn(__uint_as_float(v[4 * q + 1]), sc.y, sh.y);
            y[4 * q + 2] = __fmaf_rn(__uint_as_float(v[4 * q + 2]), sc.z, sh.z);
            y[4 * q + 3] = __fmaf_rn(__uint_as_float(v[4 * q + 3]), sc.w, sh.w);
          }
          if (EPI == EPI_BIREAL && nch > 0) {
            const float* rs = g.residual + m * g.O + o;
            float* yd = g.y_out + m * g.O + o;
            if (wide_y) {
#pragma unroll
              for (int q = 0; q < 4; q++)
                if (8 * q < nch) {  // nch is a multiple of 8 here
#pragma unroll
                  for (int j = 0; j < 8; j++) y[8 * q + j] = __fadd_rn(y[8 * q + j], rc[8 * q + j]);
                  st_global_v8(yd + 8 * q, __float_as_uint(y[8 * q]), __float_as_uint(y[8 * q + 1]), __float_as_uint(y[8 * q + 2]),
                               __float_as_uint(y[8 * q + 3]), __float_as_uint(y[8 * q + 4]), __float_as_uint(y[8 * q + 5]),
                               __float_as_uint(y[8 * q + 6]), __float_as_uint(y[8 * q + 7]));
                }
            } else {
#pragma unroll
              for (int j = 0; j < 32; j++)
                if (j < nch) {
                  y[j] = __fadd_rn(y[j], rs[j]);
                  yd[j] = y[j];
                }
            }
          }
          if (g.out_packed32 != nullptr) {
            uint32_t word = 0;
#pragma unroll
            for (int j = 0; j < 32; j++) word |= (uint32_t)(j < nch && y[j] < 0.0f) << j;
            g.out_packed32[m * g.Ow32 + (o >> 5)] = word;
          }
        }
      }
      if (failed) break;
      // this accumulator buffer may be overwritten by the tile after next
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();  // (the tensor-memory loads were warp-wide; lanes may have parted since: rejoin, then one arrival per warp)
      if (lane == 0) arrive(bar_tmem_free0 + 8u * buf);
      if (++accb == (uint32_t)g.nacc) { accb = 0; acc_phase ^= 1u; }
      }
    }
    // (only after a wait ran out:) chunks still on their way must land before the CTA gives up its shared memory
    while (tma_res && in_flight > 0) {
      __all_sync(0xFFFFFFFFu, mbar_wait(rbar0 + 8u * slot_u, phase_u, s_fail, g.wait_polls));
      in_flight--;
      if (++slot_u == (uint32_t)g.res_ring) { slot_u = 0; phase_u ^= 1u; }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (PAIR) cluster_sync_all();  // neither CTA leaves, or frees tensor memory, while the other may still use it
  else __syncthreads();
  if (*s_fail != 0 && tid == 0) atomicExch(&g_tc_error, 1);
  if (warp == 0) {
    if (PAIR)
      asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TC_TMEM_COLS)
                   : "memory");
    else
      asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"((uint32_t)TC_TMEM_COLS)
                   : "memory");
  }
}

// Weights: packed bits [O][taps][Cw] -> e2m1 [blocks of 32 output channels][taps][C/32][32][16 bytes = 32 channels];
// the blocks cover O rounded up to 128, rows beyond O are zero (e2m1 0.0: they contribute nothing).
// Channels beyond C in the last 64-channel word (C not a multiple of 64) get 0.0 as well: whatever the activation rows
// hold there, the product is 0 -- exactly as the zero tail bits of the packed words contribute nothing to Eq. 1.
__global__ void tc_prepare_weights_kernel(const uint64_t* __restrict__ wp, int O, int C, int taps, int Cw, int cgroups,
                                          long long units, uint4* __restrict__ out) {
  const long long u = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (u >= units) return;
  const int n = (int)(u & 31);
  long long t = u >> 5;
  const int grp = (int)(t % cgroups);
  t /= cgroups;
  const int tap = (int)(t % taps);
  const int o = (int)(t / taps) * 32 + n;
  uint4 bytes = make_uint4(0, 0, 0, 0);
  if (o < O) {
    const uint32_t half = (uint32_t)(wp[((long long)o * taps + tap) * Cw + (grp >> 1)] >> (32 * (grp & 1)));
    bytes = expand32(half);
    const int live = C - 32 * grp;  // channels of this group that exist
    if (live < 32) {
      // the validity bits go through the same expansion (and so the same channel order): 0xA marks a live nibble
      const uint4 v = expand32(live <= 0 ? 0u : (1u << live) - 1u);
      bytes.x &= ((v.x >> 3) & 0x11111111u) * 0xFu;
      bytes.y &= ((v.y >> 3) & 0x11111111u) * 0xFu;
      bytes.z &= ((v.z >> 3) & 0x11111111u) * 0xFu;
      bytes.w &= ((v.w >> 3) & 0x11111111u) * 0xFu;
    }
  }
  out[u] = bytes;
}

// 0: choose by size; 1: one CTA per tile; 2: CTA pairs wherever they are possible (environment DABNN_TC_MODE, read once).
int tc_mode() {
  static const int mode = [] {
    const char* e = getenv("DABNN_TC_MODE");
    return e ? atoi(e) : 0;
  }();
  return mode;
}

// C rounded up to whole 64-channel words: what the operand layouts are sized for
int tc_cpad(int C) { return (C + 63) / 64 * 64; }

// (any C whose expanded weights fit: more than 512 channels pass through the activation buffers in groups)
bool tc_covers(int O, int C, int taps) {
  return O > 0 && C > 0 && 32LL * (tc_cpad(C) / 2) * taps <= TC_WEIGHT_BUDGET;
}

// Channels per MMA for a launch: the widest of 128 / 64 / 32 whose rows (half of them per CTA of a pair) fit the
// resident budget, without padding a small O to a wide tile.
int tc_ntile(int O, int C, int taps, bool pair) {
  const long long Kb = (long long)tc_cpad(C) / 2 * taps;  // bytes per weight row
  for (int nt = 128; nt >= (pair ? 64 : 32); nt >>= 1) {
    if ((pair ? nt / 2 : nt) * Kb > TC_WEIGHT_BUDGET) continue;
    if (nt > 32 && nt / 2 >= O) continue;
    return nt;
  }
  return 0;
}

// Channel tiles cover O rounded up to whole 64-bit sign words (rows beyond O hold zero weights).
int tc_n_ntiles(int O, int nt) { return ((O + 63) / 64 * 64 + nt - 1) / nt; }

template <int NT, int EPI, int SPT, bool PAIR, bool RES_TMA = false, bool KG = false>
dabnn_status tc_launch(const TcArgs& g, size_t smem, cudaStream_t st) {
  auto kern = bconv_tc_kernel<NT, EPI, SPT, PAIR, RES_TMA, KG>;
  static bool configured[kMaxDevices] = {};
  static int max_units_dev[kMaxDevices] = {};  // CTAs (pairs) that can be resident at once
  const int dev = current_device();
  if (dev < 0) return DABNN_ERR_CUDA;
  int& max_units = max_units_dev[dev];
  if (!configured[dev]) {
    // the largest shared-memory carve-out for every instance, whatever it needs: consecutive launches of different
    // instances then never make the SMs re-partition their L1 / shared memory
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, TC_SMEM_LIMIT) != cudaSuccess ||
        cudaFuncSetAttribute(kern, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxShared) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
    max_units = sm_count();
    if (PAIR) {
      cudaLaunchConfig_t probe = {};
      probe.gridDim = dim3((unsigned)(sm_count() / 2 * 2));
      probe.blockDim = dim3(TC_THREADS);
      probe.dynamicSmemBytes = TC_SMEM_LIMIT;
      cudaLaunchAttribute at;
      at.id = cudaLaunchAttributeClusterDimension;
      at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
      probe.attrs = &at; probe.numAttrs = 1;
      int clusters = 0;
      if (cudaOccupancyMaxActiveClusters(&clusters, kern, &probe) != cudaSuccess || clusters <= 0) {
        cudaGetLastError();
        return DABNN_ERR_UNSUPPORTED;
      }
      max_units = clusters < sm_count() / 2 ? clusters : sm_count() / 2;
    }
    configured[dev] = true;
  }
  const long long m_units = PAIR ? (g.m_tiles + 1) / 2 : g.m_tiles;
  long long units = (long long)g.n_groups * m_units;
  // (a caller that runs several layers side by side may cap the CTAs of a launch: dabnn_tc_set_max_ctas)
  int avail = max_units;
  if (g_tc_max_ctas > 0) {
    const int capped = PAIR ? g_tc_max_ctas / 2 : g_tc_max_ctas;
    if (capped < avail) avail = capped > g.n_groups ? capped : g.n_groups;
  }
  const long long cap = (long long)avail / g.n_groups * g.n_groups;
  if (cap <= 0) return DABNN_ERR_UNSUPPORTED;
  if (units > cap) units = cap;
  if (!PAIR && !g.chained) {
    kern<<<(unsigned)units, TC_THREADS, smem, st>>>(g);
    return launch_status();
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((PAIR ? 2 : 1) * units));
  cfg.blockDim = dim3(TC_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (PAIR) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = 2; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
    na++;
  }
  if (g.chained) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    na++;
  }
  cfg.attrs = at; cfg.numAttrs = na;
  if (cudaLaunchKernelEx(&cfg, kern, g) != cudaSuccess) {
    cudaGetLastError();
    return DABNN_ERR_CUDA;
  }
  return launch_status();
}

// cuTensorMapEncodeTiled, looked up through the runtime (the library does not link against the driver library)
typedef CUresult (*tc_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
tc_encode_fn tc_encoder() {
  static const tc_encode_fn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess) {
      cudaGetLastError();
      p = nullptr;
    }
    return reinterpret_cast<tc_encode_fn>(p);
  }();
  return fn;
}

// The residual of a Bi-Real block as a tensor [pixels][O] of fp32, fetched in boxes of 32 rows x 32 channels (128 bytes,
// 128-byte swizzle); rows beyond the tensor read as zero.
bool tc_residual_map(CUtensorMap* map, const float* residual, long long pixels, int O) {
  const tc_encode_fn enc = tc_encoder();
  if (enc == nullptr) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)O, (cuuint64_t)pixels};
  const cuuint64_t strides[1] = {(cuuint64_t)O * 4};
  const cuuint32_t box[2] = {32, 32}, estr[2] = {1, 1};
  return enc(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(residual), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int EPI, bool PAIR>
dabnn_status tc_dispatch_mode(TcArgs& g, cudaStream_t st) {
  const size_t wr = (size_t)g.ntile / (PAIR ? 2 : 1);
  const size_t wbytes = (size_t)g.nres * wr * g.kh * g.kw * (g.C / 2);
  const size_t abytes = g.kgroups > 1 ? (size_t)g.slots * g.gw * 32 : (size_t)g.slots * (g.C / 2);
  g.abufs = 1;
  while (g.abufs < TC_MAX_BUFS && wbytes + (size_t)(g.abufs + 1) * abytes + TC_SMEM_MISC <= (size_t)TC_SMEM_LIMIT) g.abufs++;
  g.nacc = TC_ACC_COLS / g.ntile < TC_MAX_BUFS ? TC_ACC_COLS / g.ntile : TC_MAX_BUFS;
  size_t smem = wbytes + g.abufs * abytes + TC_SMEM_MISC;
  if (smem > (size_t)TC_SMEM_LIMIT) return DABNN_ERR_UNSUPPORTED;
  g.res_ring = 0;
  if (EPI == EPI_BIREAL) {
    // The residual through a ring of bulk tensor copies, where shared memory has room for it beside every activation
    // buffer and the launch is long enough for the prefetch distance to matter (environment DABNN_TC_RES_RING = 0 turns
    // it off, = n asks for n chunks per warp; read once, for measurements).
    static const int ring_env = [] { const char* e = getenv("DABNN_TC_RES_RING"); return e ? atoi(e) : -1; }();
    const bool wide = (g.O & 31) == 0 && ((reinterpret_cast<uintptr_t>(g.residual) | reinterpret_cast<uintptr_t>(g.y_out)) & 31) == 0;
    if (!PAIR && g.kgroups == 1 && g.slots <= 256 && g.ntile >= 64 && wide && ring_env != 0 && g.m_tiles >= 2LL * sm_count()) {
      const int warps = g.epi2 ? 8 : 4;
      int ring = ring_env > 0 ? (ring_env < TC_RING_MAX ? ring_env : TC_RING_MAX) : 2;
      for (; ring >= 2; ring--)
        if (smem + 1024 + (size_t)warps * ring * TC_RING_CHUNK <= (size_t)TC_SMEM_LIMIT) break;
      if (ring >= 2 && tc_residual_map(&g.res_map, g.residual, (long long)g.N * g.OH * g.OW, g.O)) {
        g.res_ring = ring;
        smem += 1024 + (size_t)warps * ring * TC_RING_CHUNK;
      }
    }
  }
  if constexpr (EPI == EPI_BIREAL && !PAIR) {
    if (g.res_ring > 0) {
      if (g.ntile == 128) return tc_launch<128, EPI, 2, false, true>(g, smem, st);
      return tc_launch<64, EPI, 2, false, true>(g, smem, st);
    }
  }
  if constexpr (!PAIR) {
    if (g.kgroups > 1) {
      if (g.slots <= 256) {
        switch (g.ntile) {
          case 128: return tc_launch<128, EPI, 2, false, false, true>(g, smem, st);
          case 64: return tc_launch<64, EPI, 2, false, false, true>(g, smem, st);
          default: return tc_launch<32, EPI, 2, false, false, true>(g, smem, st);
        }
      }
      switch (g.ntile) {
        case 128: return tc_launch<128, EPI, TC_MAX_SPT, false, false, true>(g, smem, st);
        case 64: return tc_launch<64, EPI, TC_MAX_SPT, false, false, true>(g, smem, st);
        default: return tc_launch<32, EPI, TC_MAX_SPT, false, false, true>(g, smem, st);
      }
    }
  } else if (g.kgroups > 1) {
    return DABNN_ERR_UNSUPPORTED;  // (not reached: tc_plan never pairs CTAs for grouped channels)
  }
  if (g.slots <= 256) {
    switch (g.ntile) {
      case 128: return tc_launch<128, EPI, 2, PAIR>(g, smem, st);
      case 64: return tc_launch<64, EPI, 2, PAIR>(g, smem, st);
      case 32: if constexpr (!PAIR) return tc_launch<32, EPI, 2, false>(g, smem, st);
    }
  } else if (g.Cw <= 4) {
    switch (g.ntile) {
      case 128: return tc_launch<128, EPI, TC_MAX_SPT, PAIR>(g, smem, st);
      case 64: return tc_launch<64, EPI, TC_MAX_SPT, PAIR>(g, smem, st);
      case 32: if constexpr (!PAIR) return tc_launch<32, EPI, TC_MAX_SPT, false>(g, smem, st);
    }
  }
  return DABNN_ERR_UNSUPPORTED;
}

template <int EPI>
dabnn_status tc_dispatch(TcArgs& g, cudaStream_t st) {
  // A second group of epilogue warps (measured): it pays for the residual epilogue, which moves two fp32 rows per
  // output row; elsewhere the extra warps only add contention.
  // (environment DABNN_TC_EPI2 = 0 / 1 overrides, for measurements)
  static const int epi_env = [] { const char* e = getenv("DABNN_TC_EPI2"); return e ? atoi(e) : -1; }();
  // ... and for short-K layers with many output channels (a 1x1 layer: a handful of MMAs per 128 x 128 accumulator, several
  // accumulators per activation tile), where the epilogue is most of the work: +4 % with int32 output, +10 % with sign words
  // on the 1x1 512 -> 2048 layer; 3x3 layers measured the same or slightly slower with it.
  const bool short_k = g.kh * g.kw * g.Cw <= 8 && g.nres >= 2;
  g.epi2 = epi_env >= 0 ? (epi_env != 0) : (EPI == EPI_BIREAL || short_k);
  return g.pair ? tc_dispatch_mode<EPI, true>(g, st) : tc_dispatch_mode<EPI, false>(g, st);
}

// Launch form for a problem: CTA pairs when there are enough tiles to fill the chip with pairs, and as many channel
// tiles resident per CTA (pair) as fit while every CTA (pair) still gets work.
void tc_plan(TcArgs& g, int O, int C, int taps) {
  const long long Kb = (long long)tc_cpad(C) / 2 * taps;
  const int mode = tc_mode();
  const int units1 = sm_count(), units2 = sm_count() / 2;
  const int nt2 = tc_ntile(O, C, taps, true);
  bool pair = nt2 != 0 && mode != 1 && g.kgroups == 1;
  if (pair && mode == 0) {
    // Measured: pairs win where one CTA cannot keep a 128-channel tile resident (C = 512 at 3x3) and there are
    // enough double tiles to go round; elsewhere the one-CTA form is as fast or faster.
    const long long work = (g.m_tiles + 1) / 2 * tc_n_ntiles(O, nt2);
    pair = nt2 > tc_ntile(O, C, taps, false) && 4 * work >= 3LL * units2;
  }
  g.pair = pair ? 1 : 0;
  g.ntile = pair ? nt2 : tc_ntile(O, C, taps, false);
  if (g.ntile == 0) return;
  g.n_ntiles = tc_n_ntiles(O, g.ntile);
  const long long wr = pair ? g.ntile / 2 : g.ntile;
  long long nres = TC_WEIGHT_BUDGET / (wr * Kb);
  if (nres > TC_MAX_RES) nres = TC_MAX_RES;
  if (nres > g.n_ntiles) nres = g.n_ntiles;
  const long long m_units = pair ? (g.m_tiles + 1) / 2 : g.m_tiles;
  while (nres > 1 && (g.n_ntiles + nres - 1) / nres * m_units < (pair ? units2 : units1)) nres--;
  if (g.kgroups > 1) nres = 1;  // (the groups of a tile add up in one accumulator)
  g.nres = (int)nres;
  g.n_groups = (g.n_ntiles + g.nres - 1) / g.nres;
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
  if (cv.stride_h != cv.stride_w || cv.stride_h > 2) return DABNN_ERR_UNSUPPORTED;
  if (!tc_covers(O, in.C, cv.kh * cv.kw)) return DABNN_ERR_UNSUPPORTED;
  g.a = a; g.w_tc = static_cast<const uint8_t*>(w_tc);
  g.N = in.N; g.H = in.H; g.W = in.W; g.Cw = (in.C + 63) / 64; g.C = tc_cpad(in.C);  // (the kernel sizes everything by whole words; see tc_prepare_weights_kernel)
  g.O = O; g.kh = cv.kh; g.kw = cv.kw; g.ph = cv.pad_h; g.pw = cv.pad_w; g.OH = OH; g.OW = OW;
  g.S = cv.stride_h;
  // Stride 1 with pad <= k - 1: the slot grid keeps only the left and top padding of each image.  A tap that reaches the
  // right padding of a slot row reads the first slots of the next row -- that row's left padding -- and one that reaches
  // the bottom padding reads the top padding of the next image (or rows beyond the batch), which hold the same pad value:
  // (W + pad_w) x (H + pad_h) slots per image instead of (W + 2 pad_w) x (H + 2 pad_h), 64 instead of 81 at 7 x 7.
  const bool shared_pad = g.S == 1 && cv.pad_h <= cv.kh - 1 && cv.pad_w <= cv.kw - 1;
  g.SPin = in.W + (shared_pad ? 1 : 2) * cv.pad_w; g.HPin = in.H + (shared_pad ? 1 : 2) * cv.pad_h;
  g.SP = (g.SPin + g.S - 1) / g.S; g.HP = (g.HPin + g.S - 1) / g.S;
  g.total_q = (long long)in.N * g.HP * g.SP;
  if (g.SP >= 65536 || g.HP >= 65536) return DABNN_ERR_UNSUPPORTED;
  g.magic_sp = g.SP == 1 ? 0ull : ~0ull / (unsigned long long)g.SP + 1ull;
  g.magic_hp = g.HP == 1 ? 0ull : ~0ull / (unsigned long long)g.HP + 1ull;
  g.slots_p = (128 + ((cv.kh - 1) / g.S) * g.SP + (cv.kw - 1) / g.S + 7) / 8 * 8;
  g.slots = g.S * g.S * g.slots_p;
  if ((long long)in.C * cv.kh * cv.kw >= (1LL << 22)) return DABNN_ERR_UNSUPPORTED;  // exact fp32 sums and acc_to_int
  if (g.slots > 128 * TC_MAX_SPT || g.total_q + 512 >= (1LL << 31)) return DABNN_ERR_UNSUPPORTED;
  g.m_tiles = (g.total_q + 127) / 128;
  // words per row that a producer thread holds: 8 (4 where it holds five rows, stride 2); more channels go in groups
  g.gw = g.slots <= 256 ? TC_MAX_CW : 4;
  g.kgroups = (g.Cw + g.gw - 1) / g.gw;
  tc_plan(g, O, in.C, cv.kh * cv.kw);
  if (g.ntile == 0) return DABNN_ERR_UNSUPPORTED;
  if ((long long)in.N * OH * OW >= (1LL << 31) || (long long)in.N * OH * OW * O > (1LL << 40)) return DABNN_ERR_UNSUPPORTED;
  g.pad_neg = cv.pad_value < 0;
  g.out = nullptr; g.out_nchw = 0; g.scale = g.shift = g.residual = nullptr; g.y_out = nullptr;
  g.out_packed32 = nullptr; g.Ow32 = 2 * ((O + 63) / 64);
  g.wait_polls = TC_WAIT_POLLS; g.extra_arrivals = 0; g.chained = 0;
  return DABNN_OK;
}

}  // namespace

bool tc_worthwhile(dabnn_shape in, int O, dabnn_conv cv) {
  if (cv.stride_h != cv.stride_w || cv.stride_h > 2 || !tc_covers(O, in.C, cv.kh * cv.kw)) return false;
  const int nt = tc_ntile(O, in.C, cv.kh * cv.kw, false);
  if (nt == 0) return false;
  const int S = cv.stride_h;
  const int pads = (S == 1 && cv.pad_h <= cv.kh - 1 && cv.pad_w <= cv.kw - 1) ? 1 : 2;  // as in tc_fill
  const long long slots_total = (long long)in.N * ((in.H + pads * cv.pad_h + S - 1) / S) * ((in.W + pads * cv.pad_w + S - 1) / S);
  return 2 * (slots_total / 128) * tc_n_ntiles(O, nt) >= (long long)sm_count();  // measured: from half a wave of tiles on
}

}  // namespace dabnn

using namespace dabnn;

extern "C" size_t dabnn_tc_weights_bytes(int O, int C, int kh, int kw) {
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0 || !tc_covers(O, C, kh * kw)) return 0;
  return (size_t)((O + 127) / 128 * 128) * kh * kw * (tc_cpad(C) / 2);
}

extern "C" dabnn_status dabnn_tc_prepare_weights(const uint64_t* w_packed, int O, int C, int kh, int kw, void* w_tc,
                                                 void* stream) {
  if (!w_packed || !w_tc) return DABNN_ERR_NULL;
  if (O <= 0 || C <= 0 || kh <= 0 || kw <= 0) return DABNN_ERR_SHAPE;
  if (!tc_covers(O, C, kh * kw)) return DABNN_ERR_UNSUPPORTED;
  if (!aligned(w_packed, 8) || !aligned(w_tc, 16)) return DABNN_ERR_ALIGNMENT;
  const int taps = kh * kw, cgroups = tc_cpad(C) / 32;
  const long long units = (long long)((O + 127) / 128 * 128) * taps * cgroups;
  tc_prepare_weights_kernel<<<ceil_div(units, 256), 256, 0, as_stream(stream)>>>(w_packed, O, C, taps, (C + 63) / 64, cgroups,
                                                                                 units, static_cast<uint4*>(w_tc));
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

namespace dabnn {
dabnn_status tc_bireal_block(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                             const float* scale, const float* shift, const float* residual, float* y_out,
                             uint64_t* out_packed, bool chained, cudaStream_t st) {
  TcArgs g;
  dabnn_status s = tc_fill(g, a_packed, in, w_tc, O, cv);
  if (s != DABNN_OK) return s;
  if (!scale || !shift || !residual || !y_out) return DABNN_ERR_NULL;
  if (!aligned(scale, 4) || !aligned(shift, 4) || !aligned(residual, 4) || !aligned(y_out, 4) || !aligned(out_packed, 8))
    return DABNN_ERR_ALIGNMENT;
  g.scale = scale; g.shift = shift; g.residual = residual; g.y_out = y_out;
  g.out_packed32 = reinterpret_cast<uint32_t*>(out_packed);
  g.chained = chained ? 1 : 0;
  return tc_dispatch<EPI_BIREAL>(g, st);
}
}  // namespace dabnn

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

extern "C" dabnn_status dabnn_tc_bgemm(const uint64_t* A, int M, const void* b_tc, int N, int Kbits, int32_t* C, void* stream) {
  // rows of A are the "pixels" of a 1x1 image batch, rows of B the "filters" (expanded by dabnn_tc_prepare_weights with
  // O = N, C = Kbits, kh = kw = 1): a 1x1 convolution over Kbits channels
  if (M <= 0 || N <= 0 || Kbits <= 0) return DABNN_ERR_SHAPE;
  const dabnn_shape in = {M, Kbits, 1, 1};
  const dabnn_conv cv = {1, 1, 1, 1, 0, 0, -1};
  return dabnn_tc_bconv2d(A, in, b_tc, N, cv, C, DABNN_NHWC, stream);
}

extern "C" int dabnn_tc_set_max_ctas(int max_ctas) {
  const int prev = g_tc_max_ctas;
  g_tc_max_ctas = max_ctas > 0 ? max_ctas : 0;
  return prev;
}

extern "C" int dabnn_tc_error_flag(void) {
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return v;
}

extern "C" int dabnn_last_device_flag(void* stream) {
  if (cudaStreamSynchronize(as_stream(stream)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  int v = 0;
  if (cudaMemcpyFromSymbol(&v, g_tc_error, sizeof(int)) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  if (v != 0) {
    const int zero = 0;
    if (cudaMemcpyToSymbol(g_tc_error, &zero, sizeof(int)) != cudaSuccess) {
      cudaGetLastError();
      return -1;
    }
  }
  return v;
}

extern "C" dabnn_status dabnn_stream_status(void* stream) {
  const int v = dabnn_last_device_flag(stream);
  if (v < 0) return DABNN_ERR_CUDA;
  return v == 0 ? DABNN_OK : DABNN_ERR_TIMEOUT;
}

extern "C" dabnn_status dabnn_tc_wait_expiry_selftest(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O,
                                                      dabnn_conv cv, int32_t* out, int wait_polls, void* stream) {
  TcArgs g;
  dabnn_status s = tc_fill(g, a_packed, in, w_tc, O, cv);
  if (s != DABNN_OK) return s;
  if (!out) return DABNN_ERR_NULL;
  if (!aligned(out, 4)) return DABNN_ERR_ALIGNMENT;
  if (wait_polls < 1 || wait_polls > 4096) return DABNN_ERR_SHAPE;  // a few milliseconds at most
  g.out = out;
  g.out_nchw = 0;
  g.wait_polls = wait_polls;
  g.extra_arrivals = 1;  // `a_full` never completes: the MMA thread's first wait runs out, every other role follows
  return tc_dispatch<EPI_I32>(g, as_stream(stream));
}

