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

namespace {
// Two side streams per device for the copies (created on first use, never destroyed) and a small ring of events.
// The batch is cut into chunks: chunk k's copy-in runs on the copy-in stream, its kernels on the caller's stream, its
// copy-out on the copy-out stream, so host-to-device and device-to-host traffic overlap each other and the kernels.
// The caller's stream waits for the last copy-out before the call's work counts as done (fork / join, so the call can
// also be captured into a CUDA graph).
constexpr int kHostChunks = 4;
constexpr int kEventRing = 64;
struct CopyLanes {
  cudaStream_t in = nullptr, out = nullptr;
  cudaEvent_t ev[kEventRing];
  cudaEvent_t prev_compute;  // the kernels of the previous (uncaptured) call on this device are done
  bool has_prev = false;
  const void* prev_ws = nullptr;  // workspace of that previous call
  int next = 0;
  bool ok = false;
};
CopyLanes* copy_lanes() {
  static CopyLanes lanes[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  CopyLanes& L = lanes[dev];
  if (!L.ok) {
    if (cudaStreamCreateWithFlags(&L.in, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    if (cudaStreamCreateWithFlags(&L.out, cudaStreamNonBlocking) != cudaSuccess) return nullptr;
    for (int i = 0; i < kEventRing; i++)
      if (cudaEventCreateWithFlags(&L.ev[i], cudaEventDisableTiming) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&L.prev_compute, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    L.ok = true;
  }
  return &L;
}
}  // namespace

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
  CopyLanes* L = copy_lanes();
  if (!L) {
    cudaGetLastError();
    return DABNN_ERR_CUDA;
  }
  auto event = [&]() { return L->ev[L->next++ % kEventRing]; };
  auto fail = [&]() {
    cudaGetLastError();
    return DABNN_ERR_CUDA;
  };
  char* base = static_cast<char*>(workspace);
  float* x_dev = reinterpret_cast<float*>(base + p.x);
  uint64_t* a_dev = reinterpret_cast<uint64_t*>(base + p.a);
  int32_t* out_dev = reinterpret_cast<int32_t*>(base + p.out);
  uint64_t* bits_dev = reinterpret_cast<uint64_t*>(base + p.bits);
  // per-image element counts
  const long long x_img = p.x_elems / in.N, a_img = p.a_words / in.N, out_img = p.out_elems / in.N, bits_img = p.bits_words / in.N;
  // When the caller's stream is being captured the copy-in stream forks from it (everything lands in the graph).
  // Otherwise the copies in only wait for the previous call's kernels -- the last readers of the workspace's input area --
  // so that they run under the previous call's copies out (x_host must hold its data when this function is called).
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cap) != cudaSuccess) return fail();
  const bool capturing = cap != cudaStreamCaptureStatusNone;
  // A workspace that the previous call did not use may still be in use by whatever the caller's stream holds (another
  // layer's call, or memory that the caller's allocator has just recycled): then, too, the copies wait for `st`.
  if (capturing || !L->has_prev || L->prev_ws != workspace) {
    cudaEvent_t e_start = event();
    if (cudaEventRecord(e_start, st) != cudaSuccess || cudaStreamWaitEvent(L->in, e_start, 0) != cudaSuccess) return fail();
  }
  if (!capturing && L->has_prev) {
    if (cudaStreamWaitEvent(L->in, L->prev_compute, 0) != cudaSuccess) return fail();
  }
  const int chunks = in.N < kHostChunks ? in.N : kHostChunks;
  cudaEvent_t e_last_out = nullptr;
  for (int k = 0; k < chunks; k++) {
    const int n0 = (int)((long long)in.N * k / chunks), n1 = (int)((long long)in.N * (k + 1) / chunks);
    dabnn_shape part = in;
    part.N = n1 - n0;
    if (cudaMemcpyAsync(x_dev + x_img * n0, x_host + x_img * n0, (size_t)x_img * part.N * 4, cudaMemcpyHostToDevice, L->in) !=
        cudaSuccess)
      return fail();
    cudaEvent_t e_in = event();
    if (cudaEventRecord(e_in, L->in) != cudaSuccess || cudaStreamWaitEvent(st, e_in, 0) != cudaSuccess) return fail();
    dabnn_status s = dabnn_pack(x_dev + x_img * n0, DABNN_NCHW, part, a_dev + a_img * n0, stream);
    if (s != DABNN_OK) return s;
    if (out_host) {
      s = dabnn_bconv2d(a_dev + a_img * n0, part, w_packed, O, cv, out_dev + out_img * n0, DABNN_NHWC, stream);
      if (s != DABNN_OK) return s;
    }
    if (bits_host) {
      s = dabnn_bconv2d_bn_sign_pack(a_dev + a_img * n0, part, w_packed, O, cv, scale, shift, bits_dev + bits_img * n0, stream);
      if (s != DABNN_OK) return s;
    }
    cudaEvent_t e_done = event();
    if (cudaEventRecord(e_done, st) != cudaSuccess || cudaStreamWaitEvent(L->out, e_done, 0) != cudaSuccess) return fail();
    if (out_host && cudaMemcpyAsync(out_host + out_img * n0, out_dev + out_img * n0, (size_t)out_img * part.N * 4,
                                    cudaMemcpyDeviceToHost, L->out) != cudaSuccess)
      return fail();
    if (bits_host && cudaMemcpyAsync(bits_host + bits_img * n0, bits_dev + bits_img * n0, (size_t)bits_img * part.N * 8,
                                     cudaMemcpyDeviceToHost, L->out) != cudaSuccess)
      return fail();
    e_last_out = event();
    if (cudaEventRecord(e_last_out, L->out) != cudaSuccess) return fail();
  }
  if (!capturing) {
    if (cudaEventRecord(L->prev_compute, st) != cudaSuccess) return fail();
    L->has_prev = true;
    L->prev_ws = workspace;
  }
  // join: the caller's stream is done with this call when the last copy-out is
  if (cudaStreamWaitEvent(st, e_last_out, 0) != cudaSuccess) return fail();
  return DABNN_OK;
}
