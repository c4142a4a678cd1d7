// Host-buffer entry point: one binary layer end to end (copy in, pack, convolve, copy out).
#include "common.cuh"

using namespace dabnn;

namespace {
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct HostPlan {
  size_t x, a, out, bits, total;
  long long x_elems, a_words, out_elems, bits_words;
};

bool plan_host(dabnn_shape in, int O, dabnn_conv cv, HostPlan& p) {
  if (in.N <= 0 || in.C <= 0 || in.H <= 0 || in.W <= 0 || O <= 0 || cv.stride_h <= 0 || cv.stride_w <= 0) return false;
  const int OH = dabnn_out_dim(in.H, cv.kh, cv.stride_h, cv.pad_h), OW = dabnn_out_dim(in.W, cv.kw, cv.stride_w, cv.pad_w);
  if (OH <= 0 || OW <= 0) return false;
  p.x_elems = (long long)in.N * in.C * in.H * in.W;
  p.a_words = (long long)in.N * in.H * in.W * ((in.C + 63) / 64);
  p.out_elems = (long long)in.N * OH * OW * O;
  p.bits_words = (long long)in.N * OH * OW * ((O + 63) / 64);
  size_t off = 0;
  p.x = off;    off = align_up(off + (size_t)p.x_elems * 4, 256);
  p.a = off;    off = align_up(off + (size_t)p.a_words * 8, 256);
  p.out = off;  off = align_up(off + (size_t)p.out_elems * 4, 256);
  p.bits = off; off = align_up(off + (size_t)p.bits_words * 8, 256);
  p.total = off;
  return true;
}
}  // namespace

extern "C" size_t dabnn_binary_layer_host_workspace_bytes(dabnn_shape in, int O, dabnn_conv cv) {
  HostPlan p;
  return plan_host(in, O, cv, p) ? p.total : 0;
}

extern "C" dabnn_status dabnn_binary_layer_host(const float* x_host, dabnn_shape in, const uint64_t* w_packed, int O,
                                                dabnn_conv cv, const float* scale, const float* shift,
                                                int32_t* out_host, uint64_t* bits_host, void* workspace,
                                                size_t workspace_bytes, void* stream) {
  if (!x_host || !w_packed || !workspace) return DABNN_ERR_NULL;
  if (!out_host && !bits_host) return DABNN_ERR_NULL;
  if (bits_host && (!scale || !shift)) return DABNN_ERR_NULL;
  HostPlan p;
  if (!plan_host(in, O, cv, p)) return DABNN_ERR_SHAPE;
  if (!aligned(workspace, 256)) return DABNN_ERR_ALIGNMENT;
  if (workspace_bytes < p.total) return DABNN_ERR_WORKSPACE;
  cudaStream_t st = as_stream(stream);
  char* base = static_cast<char*>(workspace);
  float* x_dev = reinterpret_cast<float*>(base + p.x);
  uint64_t* a_dev = reinterpret_cast<uint64_t*>(base + p.a);
  int32_t* out_dev = reinterpret_cast<int32_t*>(base + p.out);
  uint64_t* bits_dev = reinterpret_cast<uint64_t*>(base + p.bits);
  if (cudaMemcpyAsync(x_dev, x_host, (size_t)p.x_elems * 4, cudaMemcpyHostToDevice, st) != cudaSuccess) {
    cudaGetLastError();
    return DABNN_ERR_CUDA;
  }
  dabnn_status s = dabnn_pack(x_dev, DABNN_NCHW, in, a_dev, stream);
  if (s != DABNN_OK) return s;
  if (out_host) {
    s = dabnn_bconv2d(a_dev, in, w_packed, O, cv, out_dev, DABNN_NHWC, stream);
    if (s != DABNN_OK) return s;
    if (cudaMemcpyAsync(out_host, out_dev, (size_t)p.out_elems * 4, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
  }
  if (bits_host) {
    s = dabnn_bconv2d_bn_sign_pack(a_dev, in, w_packed, O, cv, scale, shift, bits_dev, stream);
    if (s != DABNN_OK) return s;
    if (cudaMemcpyAsync(bits_host, bits_dev, (size_t)p.bits_words * 8, cudaMemcpyDeviceToHost, st) != cudaSuccess) {
      cudaGetLastError();
      return DABNN_ERR_CUDA;
    }
  }
  return DABNN_OK;
}
