// Shared host/device helpers of libdabnn_b200 (CUDA path only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "dabnn.h"

namespace dabnn {

inline cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }

inline dabnn_status launch_status() {
  return cudaGetLastError() == cudaSuccess ? DABNN_OK : DABNN_ERR_CUDA;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

inline int ceil_div(long long a, long long b) { return static_cast<int>((a + b - 1) / b); }

// True when the tensor-core engine covers this layer AND the layer has enough pixel tiles for at least half of the SMs
// (below that the integer-pipe kernel, which spreads small problems over many small CTAs, is faster).
bool tc_worthwhile(dabnn_shape in, int O, dabnn_conv cv);

// The Bi-Real block on the tensor-core engine as the forward launches it.  chained: with programmatic stream serialization
// (the kernel sets itself up under its predecessor's tail; its weights and BN vectors must be constants of the stream).
dabnn_status tc_bireal_block(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                             const float* scale, const float* shift, const float* residual, float* y_out,
                             uint64_t* out_packed, bool chained, cudaStream_t st);

// Chained launches for forwards of a few images, where every kernel is shorter than the time it takes to start one.  A
// kernel started by launch_chain() while g_chain_launch is set may begin before its predecessor in the stream has
// finished: it may do what does not depend on the predecessor (index set-up, fetching weights) and must call
// chain_wait() -- which returns once the predecessor has completed and its writes are visible -- before it touches
// anything else.  chain_trigger(), called by every CTA once its main work is done, lets the successor start.  In a
// kernel launched the ordinary way both are no-ops.
extern thread_local bool g_chain_launch;  // per host thread: set by a forward call for the launches it makes itself
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Read-only-path 16-byte load for data that the PREVIOUS kernel of a chain wrote.  Volatile asm, so that it stays behind
// chain_wait(): __ldg and loads through const __restrict__ pointers count as invariant, and the compiler may move those
// above the wait, before which the data may not have been written.
__device__ __forceinline__ float4 ld_nc_f4(const float* p) {
  float4 v;
  asm volatile("ld.global.nc.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p));
  return v;
}

template <typename... KArgs, typename... Args>
inline void launch_chain(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  if (!g_chain_launch) {
    kern<<<grid, block, smem, st>>>(args...);
    return;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}
#endif

// The STEM module front end of Bi-Real Net 18 (stem_module.cu): fp32 [N][56][56][64] and its packed signs from the images.
dabnn_status launch_stem_module(const dabnn_stem_module_params* sm, const float* images, int N, float* s1, float* a1,
                                float* cat, float* out, uint64_t* bits, cudaStream_t st);

// Per-device host caches (function attributes set, SM counts, symbol addresses) are arrays over the device ordinal.
constexpr int kMaxDevices = 64;
// Ordinal of the calling thread's current device, or -1 (no device, or an ordinal beyond kMaxDevices).
inline int current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) {
    cudaGetLastError();
    return -1;
  }
  return (dev >= 0 && dev < kMaxDevices) ? dev : -1;
}

// Number of SMs of the current device (cached per device).
int sm_count();

}  // namespace dabnn
