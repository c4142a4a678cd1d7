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

// True when the tensor-core engine covers this layer AND the layer has enough pixel tiles to keep every SM's resident
// weights busy (below that the integer-pipe kernel, which spreads small problems over many small CTAs, is faster).
bool tc_worthwhile(dabnn_shape in, int O, dabnn_conv cv);

// Number of SMs of the current device (cached per process; the library runs on one device at a time).
int sm_count();

}  // namespace dabnn
