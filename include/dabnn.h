/*
 * dabnn.h -- C ABI of libdabnn_b200: binarized convolution on NVIDIA B200 (sm_100a).
 *
 * The operations are those of daBNN (arXiv 1908.05858): sign-binarize + bit-pack along the
 * channel axis (Section 2.1.1), binary convolution on the packed words (Section 2.1.2, Eq. 1)
 * and the fused BN + binarize + re-pack that feeds the next binary layer (Section 2.1.1, last
 * sentence), plus a Bi-Real Net 18 forward built from them (Section 2.3, Table 2).
 *
 * Conventions shared by every entry point
 *   - Every data pointer is DEVICE memory owned by the caller unless its name ends in _host.
 *     The library allocates nothing, frees nothing and keeps no pointer after the call's work
 *     on the stream has completed.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Calls only
 *     enqueue work; they do not synchronise.
 *   - Binarization: v = (x < 0) ? -1 : +1 as an IEEE comparison (+0.0, -0.0 and NaN give +1).
 *     A packed bit is 1 for -1.  Words are 64-bit; channel c lives in word c>>6 at bit c&63;
 *     bits beyond C in the last word are 0.
 *   - Packed activations: uint64 [N][H][W][Cw], Cw = ceil(C/64).
 *     Packed weights:     uint64 [O][kh][kw][Cw].
 *   - Convolution is cross-correlation, dilation 1, groups 1;
 *     OH = floor((H + 2*pad_h - kh)/stride_h) + 1, likewise OW.  Spatial padding holds the
 *     declared value pad_value (+1 or -1), so every output sums K = C*kh*kw terms and
 *     out = K - 2*popcount(xor) lies in [-K, K] with the parity of K.
 *   - Errors: argument problems are reported synchronously, before anything is launched
 *     (DABNN_ERR_NULL / _SHAPE / _ALIGNMENT / _WORKSPACE); a failed launch gives DABNN_ERR_CUDA.
 *     Nothing throws; kernels never trap.  Waits inside the tensor-core kernels are bounded: a kernel whose wait runs
 *     out sets a per-device flag, releases what it holds and returns, and its outputs are undefined.  Calls only enqueue
 *     work, so they still return DABNN_OK then; read the flag with dabnn_stream_status / dabnn_last_device_flag.
 *   - Devices: a process may use the library on several devices (cudaSetDevice before the call); caches of function
 *     attributes and SM counts are kept per device ordinal (up to 64).
 *   - Alignment: packed buffers 8 bytes; fp32 buffers 4 bytes (16 bytes enables vector paths,
 *     chosen automatically).
 */
#ifndef DABNN_H_
#define DABNN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DABNN_OK = 0,
  DABNN_ERR_NULL = 1,        /* a required pointer is NULL */
  DABNN_ERR_SHAPE = 2,       /* non-positive dimension, empty output, bad stride / pad_value / layout */
  DABNN_ERR_UNSUPPORTED = 3, /* a size beyond what the index arithmetic supports (>= 2^31 elements per axis product) */
  DABNN_ERR_ALIGNMENT = 4,
  DABNN_ERR_WORKSPACE = 5,   /* workspace too small */
  DABNN_ERR_CUDA = 6,        /* the CUDA runtime reported an error at launch */
  DABNN_ERR_TIMEOUT = 7,     /* a bounded wait inside a kernel ran out (reported by dabnn_stream_status) */
  DABNN_ERR_STATIC_LIMIT = 8 /* the request is larger than the library's built-in scratch area */
} dabnn_status;

typedef enum { DABNN_NCHW = 0, DABNN_NHWC = 1 } dabnn_layout;

/* Logical (unpacked) shape of an activation tensor. */
typedef struct { int N, C, H, W; } dabnn_shape;

/* Convolution geometry.  pad_value is the value (+1 or -1) every padded position holds. */
typedef struct { int kh, kw, stride_h, stride_w, pad_h, pad_w, pad_value; } dabnn_conv;

const char* dabnn_status_string(dabnn_status s);

/* ceil(C/64): 64-bit words per pixel (or per weight tap). */
size_t dabnn_words_per_pixel(int C);
/* floor((in + 2*pad - k)/stride) + 1 (may be <= 0: no output). */
int dabnn_out_dim(int in, int k, int stride, int pad);

/* Section 2.1.1 -- binarize + pack activations.
 * x: fp32, N*C*H*W elements in `in_layout`.  packed: uint64 [N][H][W][Cw], fully overwritten. */
dabnn_status dabnn_pack(const float* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed, void* stream);
/* The same for 32-bit integers (Section 2.1.1: the packer takes the sign bit of int32 values as it does of floats), e.g. a
 * convolution's raw sums binarized without a BN in between.  bit = (x < 0): 0 packs as +1.  Same layouts, output and
 * errors as dabnn_pack; x must be 4-byte aligned (16-byte aligned input takes the vector path). */
dabnn_status dabnn_pack_i32(const int32_t* x, dabnn_layout in_layout, dabnn_shape s, uint64_t* packed, void* stream);

/* Section 2.1.2, last paragraph / Fig. 3 -- the paper's NC1HWC2 activation layout, for comparison with the channel-packed
 * NHWC words above.  C2 = 128 bits (the paper's vector register): uint64 [N][C1][H][W][2] with C1 = ceil(C/128); channel c
 * lives in group c>>7, word (c>>6)&1, bit c&63; a last group of 64 channels or fewer has a zero second word.
 *   dabnn_packed_words   64-bit words of a packed tensor in either layout (0 for an invalid shape or layout)
 *   dabnn_pack_as        dabnn_pack into the chosen layout (packed: 16-byte aligned for NC1HWC2)
 *   dabnn_bconv2d_from   dabnn_bconv2d reading activations in the chosen layout (weights stay [O][kh][kw][Cw]); the
 *                        integers are the same whichever layout the activations are in. */
typedef enum { DABNN_PACKED_NHWC = 0, DABNN_PACKED_NC1HWC2 = 1 } dabnn_packed_layout;
size_t dabnn_packed_words(dabnn_shape s, dabnn_packed_layout packed_layout);
dabnn_status dabnn_pack_as(const float* x, dabnn_layout in_layout, dabnn_shape s, dabnn_packed_layout packed_layout,
                           uint64_t* packed, void* stream);
dabnn_status dabnn_bconv2d_from(const uint64_t* a_packed, dabnn_packed_layout a_layout, dabnn_shape in,
                                const uint64_t* w_packed, int O, dabnn_conv cv, int32_t* out, dabnn_layout out_layout,
                                void* stream);

/* Section 3 (weights are binarized and packed once, 32x smaller).
 * w_oihw: fp32 [O][C][kh][kw].  wpacked: uint64 [O][kh][kw][Cw], fully overwritten. */
dabnn_status dabnn_pack_weights(const float* w_oihw, int O, int C, int kh, int kw, uint64_t* wpacked, void* stream);

/* Section 2.1.2, Eq. 1 -- binary convolution, int32 result.
 * a_packed: [N][H][W][Cw] for in = {N,C,H,W}; w_packed: [O][kh][kw][Cw];
 * out: int32, N*OH*OW*O elements in `out_layout` ([N][OH][OW][O] or [N][O][OH][OW]). */
dabnn_status dabnn_bconv2d(const uint64_t* a_packed, dabnn_shape in, const uint64_t* w_packed, int O, dabnn_conv cv,
                           int32_t* out, dabnn_layout out_layout, void* stream);

/* Eq. 1 -- BGEMM on packed vectors, for binary fully-connected layers and im2col'ed inputs.
 * A: [M][Kw] packed rows; B: [N][Kw] packed rows (row j is column j of the paper's B); Kbits valid bits per row,
 * Kw = ceil(Kbits/64), tail bits 0.  C: int32 [M][N], the +-1 dot product  Kbits - 2*popcount(xor)  of row i of A and
 * row j of B.  The paper's count of agreeing positions is (C + Kbits) / 2. */
dabnn_status dabnn_bgemm(const uint64_t* A, int M, const uint64_t* B, int N, int Kbits, int32_t* C, void* stream);

/* Section 2.1.1 (fused BN-binarization) on top of Eq. 1: the int32 result never leaves the chip.
 * y = fmaf((float)acc, scale[o], shift[o]); bit = (y < 0); out_packed: uint64 [N][OH][OW][ceil(O/64)]. */
dabnn_status dabnn_bconv2d_bn_sign_pack(const uint64_t* a_packed, dabnn_shape in, const uint64_t* w_packed, int O,
                                        dabnn_conv cv, const float* scale, const float* shift, uint64_t* out_packed,
                                        void* stream);

/* The Bi-Real block epilogue (Section 2.3): y = fmaf((float)acc, scale[o], shift[o]) + residual, one rounded
 * add.  residual and y_out are fp32 [N][OH][OW][O] (may alias each other); out_packed as above holds the sign
 * bits of y_out.  out_packed may be NULL when the packed signs are not needed. */
dabnn_status dabnn_bconv2d_bn_add_sign_pack(const uint64_t* a_packed, dabnn_shape in, const uint64_t* w_packed, int O,
                                            dabnn_conv cv, const float* scale, const float* shift,
                                            const float* residual, float* y_out, uint64_t* out_packed, void* stream);

/* BN parameters -> per-channel (scale, shift), evaluated in double on the device with IEEE-rounded operations:
 * sd = gamma/sqrt(var+eps); scale = (float)sd; shift = (float)(beta - mean*sd).  All arrays hold O floats. */
dabnn_status dabnn_bn_fold(const float* gamma, const float* beta, const float* mean, const float* var, double eps,
                           int O, float* scale, float* shift, void* stream);

/* Section 2.3 / Table 2 -- Bi-Real Net 18 (binary ResNet-18; 7x7 stem conv and the final fc in fp32).
 * Stages of 64/128/256/512 channels at 56/28/14/7 pixels, four blocks each; block b:
 * out = BN_b(bconv3x3(sign(x))) + shortcut(x), pad value -1; the first block of stages 2..4 has stride 2
 * and shortcut(x) = BN(conv1x1_fp32(avgpool2x2(x))).  No activation function other than sign.
 * Every fp32 operation is a single IEEE-rounded operation in a fixed order, so results are reproducible. */
typedef struct {
  const float* stem_w;           /* fp32 [64][3][7][7] */
  const float* stem_scale;       /* folded BN, [64] */
  const float* stem_shift;
  const uint64_t* block_w[16];   /* packed [O][3][3][Cw] (dabnn_pack_weights) */
  const float* block_scale[16];  /* folded BN, [O] */
  const float* block_shift[16];
  const float* down_w[3];        /* fp32 [O][C] 1x1 weights for the first block of stages 2, 3, 4 */
  const float* down_scale[3];
  const float* down_shift[3];
  const float* fc_w;             /* fp32 [1000][512] */
  const float* fc_b;             /* fp32 [1000] */
  const void* block_w_tc[16];    /* optional: weights expanded by dabnn_tc_prepare_weights, or NULL.  Where given and the
                                    batch is large enough for the tensor-core engine to pay (all 16 blocks, stride 1 and
                                    stride 2, from about 70 images on; the early stages from 8), that engine runs the
                                    block; results are identical either way */
} dabnn_bireal18_params;

/* Bytes of device workspace dabnn_bireal18_forward needs for a batch of N images (0 if N <= 0). */
size_t dabnn_bireal18_workspace_bytes(int N);

/* p: HOST struct of device pointers.  images: fp32 NCHW [N][3][224][224].  logits: fp32 [N][1000].
 * workspace: device memory, 256-byte aligned, at least dabnn_bireal18_workspace_bytes(N) bytes; its contents
 * are scratch (activations between layers) and are undefined afterwards.
 * Kernels are chosen by batch size (results are the same bits whichever runs).  The launches are chained with programmatic
 * stream serialization: a kernel may begin its set-up (for the tensor-engine blocks also the copy of its weights and BN
 * vectors, which must therefore not be written by work still pending on the stream) while its predecessor finishes, and
 * waits for it before it reads any activation; on the stream the call as a whole is ordered like any other work, and it
 * can be captured into a CUDA graph.  DABNN_NO_CHAIN=1 in the environment (read once) gives ordinary launches.
 * Where blocks run on the tensor-core engine, a wait that ran out inside one of its kernels leaves the logits undefined
 * while this call has long returned DABNN_OK: after synchronising, check dabnn_stream_status(stream). */
dabnn_status dabnn_bireal18_forward(const dabnn_bireal18_params* p, const float* images, int N, float* logits,
                                    void* workspace, size_t workspace_bytes, void* stream);

/* Section 2.3 / Fig. 6 / Table 2, second row -- Bi-Real Net 18 with the STEM module in place of the 7x7 convolution and
 * the max-pool.  The module's figure is not in the paper's text; the structure here is a reading after the stem block of
 * the network the paper cites for it (so its parity is pinned to this library's oracle only, not to the paper):
 *   s1 = relu(BN(conv3x3/2 pad 1, 3 -> 32))(image); a = relu(BN(conv1x1, 32 -> 16))(s1); a = relu(BN(conv3x3/2 pad 1, 16 -> 32))(a);
 *   b = maxpool2x2/2(s1); out = BN(conv1x1, 64 -> 64)(concat(a, b)), fp32 [N][56][56][64], which feeds the sixteen blocks.
 * w[i]: fp32 OIHW weights of the four convolutions ([32][3][3][3], [16][32][1][1], [32][16][3][3], [64][64][1][1]);
 * scale[i], shift[i]: their folded BN vectors.  p's stem_w / stem_scale / stem_shift are not used (may be NULL).
 * Workspace: dabnn_bireal18_workspace_bytes(N), as for dabnn_bireal18_forward; everything else as there. */
typedef struct {
  const float* w[4];
  const float* scale[4];
  const float* shift[4];
} dabnn_stem_module_params;
dabnn_status dabnn_bireal18_forward_stem_module(const dabnn_bireal18_params* p, const dabnn_stem_module_params* sm,
                                                const float* images, int N, float* logits, void* workspace,
                                                size_t workspace_bytes, void* stream);

/* (No counterpart in the paper: a packaging convenience of this library.)
 * dabnn_bireal18_forward for callers that must not allocate device memory.  Some hosts of this library cannot call
 * cudaMalloc: a plug-in inside a server whose framework has reserved the whole device for its own pool, a
 * latency-critical loop that may not take cudaMalloc's implicit device synchronisation, or code running where any
 * allocation is forbidden by policy.  For them the activations between layers live in a scratch area that is part
 * of the library image itself, so the caller passes only inputs and outputs.
 *   - Limit: N <= DABNN_STATIC_MAX_BATCH images per call; a larger N returns DABNN_ERR_STATIC_LIMIT and nothing runs.
 *   - Cost: the scratch area (DABNN_STATIC_SCRATCH_BYTES, about 8.5 MiB) is reserved on every GPU on which the
 *     library is loaded, from load until the process exits, whether or not this entry point is ever called.
 *   - The first call on each device looks up the area's device address (a runtime query; it may also be the moment at
 *     which the CUDA runtime loads this library's device code and reserves the area).  Make that first call once at
 *     start-up, outside any stream capture.  Later calls on that device reuse the address.
 *   - The call itself performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *   - All calls share the one area and it keeps whatever the previous call left in it.  Nothing in it has to start
 *     at zero (every region is fully written before it is read), so no clearing is done.  Two calls whose work
 *     overlaps on the GPU (different streams, or different threads) race on the area: serialise them.
 * Arguments and results are otherwise exactly those of dabnn_bireal18_forward. */
#define DABNN_STATIC_MAX_BATCH 2
#define DABNN_STATIC_SCRATCH_BYTES 8935424
dabnn_status dabnn_bireal18_forward_static(const dabnn_bireal18_params* p, const float* images, int N, float* logits,
                                           void* stream);

/* One binary layer with HOST buffers (Section 2.1.1 + 2.1.2 end to end): copies x_host (fp32 NCHW, in.N*in.C*in.H*in.W
 * elements; pinned memory makes the copies asynchronous) to the device, packs it, and then
 *   - if out_host  != NULL: runs dabnn_bconv2d and copies the int32 NHWC result [N][OH][OW][O] to out_host;
 *   - if bits_host != NULL: runs dabnn_bconv2d_bn_sign_pack (scale, shift: DEVICE, required then) and copies the
 *     packed result [N][OH][OW][ceil(O/64)] to bits_host.
 * w_packed, scale, shift and workspace are DEVICE pointers; workspace must be 256-byte aligned and hold at least
 * dabnn_binary_layer_host_workspace_bytes(in, O, cv) bytes (0 is returned for an invalid geometry).
 * The batch is processed in up to four chunks whose copies run on two internal copy streams (created per device on first
 * use, kept until exit), so that the copy in, the kernels and the copy out of different chunks overlap; `stream` waits for
 * all of it: the host results are complete once `stream` has been synchronised.  x_host must hold its data when the
 * function is called (its copy may start before earlier work on `stream` has finished).  The first copy into the
 * workspace waits for whatever `stream` held when the function was called whenever the workspace is not the one of the
 * previous call on this device; with the same workspace it waits only for that previous call's kernels, so a caller
 * that lets other work use the workspace in between must synchronise that work itself.  Not thread-safe against
 * concurrent calls on the same device; calls that share a workspace belong on one stream.  This entry point uses the
 * integer-pipe kernels only (no bounded waits), so there is no device flag to read after it. */
size_t dabnn_binary_layer_host_workspace_bytes(dabnn_shape in, int O, dabnn_conv cv);
dabnn_status dabnn_binary_layer_host(const float* x_host, dabnn_shape in, const uint64_t* w_packed, int O, dabnn_conv cv,
                                     const float* scale, const float* shift, int32_t* out_host, uint64_t* bits_host,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* ---- tensor-core engine -------------------------------------------------------------------------------------------
 * The same convolutions (Section 2.1.2, Eq. 1 read as a +-1 dot product) computed on the tcgen05 tensor cores with
 * 4-bit {+1,-1} operands (e2m1, block scale 1.0, fp32 accumulation: exact) expanded on chip from the packed bits.
 * Results are identical to dabnn_bconv2d* bit for bit.
 * Covered: stride 1 or 2 (both axes alike); any C whose expanded weights fit (below) -- up to 512 channels (256 at stride 2)
 * a tile's activations are expanded at once, more pass through the activation buffers in groups of 512 (256) channels
 * while the tile's sums stay in one accumulator (channels beyond C in the last 64-channel word
 * are given zero weights, which is what the zero tail bits of the packed words mean in Eq. 1); images narrow enough
 * that the 128 + (kh-1)*SP + kw-1 slots a tile reads fit its activation buffer of 640 rows (SP = W + pad_w slots per
 * image row at stride 1, so W + pad_w <= 255 for a 3x3 filter; wider still at C <= 256, where a thread holds five rows),
 * filters whose expanded weights fit the resident budget: 32 output channels x kh*kw*C/2 bytes <= 144 KB, i.e. C <= 1024 for
 * a 3x3 filter and <= 9216 for 1x1 (dabnn_tc_weights_bytes returns 0 otherwise); C*kh*kw < 2^22; other cases
 * return DABNN_ERR_UNSUPPORTED and are served by dabnn_bconv2d*.
 * A launch takes one of two forms, chosen by the library from the problem size: one CTA per tile of 128 output
 * positions, or pairs of CTAs of a thread-block cluster that share every tensor-core instruction (used where one CTA
 * cannot keep 128 output channels of weights resident: C = 512 with a 3x3 filter).  Both give the same bits.
 * The int32 output is written with a streaming (evict-first) cache policy.
 * Environment, read once, for measurements only: DABNN_TC_MODE = 1 (never pairs) or 2 (pairs wherever possible);
 * DABNN_TC_EPI2 = 0 / 1 (second group of epilogue warps off / on); DABNN_TC_RES_RING = 0 (residual of the Bi-Real epilogue
 * read with ordinary loads everywhere) or 2..4 (chunks per epilogue warp in flight where bulk tensor copies fetch it).
 * The Bi-Real epilogue of a long stride-1 launch whose rows are whole 128-byte chunks (O a multiple of 32, residual and
 * y_out 32-byte aligned) fetches the residual with bulk tensor copies; the library then encodes a tensor map on the host
 * in the call (cuTensorMapEncodeTiled, looked up through the runtime; if it is not there, ordinary loads are used).
 *   dabnn_tc_weights_bytes    bytes of the expanded weight buffer for a filter bank (0 = not covered): O rounded up to
 *                             128 rows of C*kh*kw/2 bytes, the same buffer for every launch form
 *   dabnn_tc_prepare_weights  w_packed [O][kh][kw][Cw] -> w_tc (device, 16-byte aligned, that many bytes); once per model
 *   dabnn_tc_bconv2d*         as dabnn_bconv2d*, with w_tc in place of w_packed
 *   dabnn_tc_error_flag       synchronises nothing itself; copies the current device's error flag (1 if a bounded wait
 *                             inside a kernel ran out since the flag was last cleared, else 0; -1 if it cannot be read)
 *                             and leaves it set.  Call after synchronising the stream.
 *   dabnn_last_device_flag    synchronises `stream`, returns that flag and clears it (one flag per device, shared by all
 *                             streams: a value of 1 says that some tensor-engine launch on this device since the last
 *                             read gave up, and the outputs written since then are undefined).  Not for use during
 *                             stream capture.
 *   dabnn_stream_status       the same as a status: DABNN_OK, DABNN_ERR_TIMEOUT (flag was set; now cleared) or
 *                             DABNN_ERR_CUDA (the stream or the flag could not be read).
 *   dabnn_tc_wait_expiry_selftest   exercises that failure path without any fault: launches dabnn_tc_bconv2d's kernel (NHWC)
 *                             with its "activation rows ready" barrier expecting one arrival more than it will ever get
 *                             and every wait limited to wait_polls polls (1..4096, about a microsecond each).  Each role
 *                             of each CTA gives up in turn, the flag is set, tensor memory is freed and the kernel
 *                             returns by itself; `out` is undefined.  The next ordinary launch is unaffected. */
size_t dabnn_tc_weights_bytes(int O, int C, int kh, int kw);
dabnn_status dabnn_tc_prepare_weights(const uint64_t* w_packed, int O, int C, int kh, int kw, void* w_tc, void* stream);
dabnn_status dabnn_tc_bconv2d(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                              int32_t* out, dabnn_layout out_layout, void* stream);
dabnn_status dabnn_tc_bconv2d_bn_sign_pack(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                                           const float* scale, const float* shift, uint64_t* out_packed, void* stream);
dabnn_status dabnn_tc_bconv2d_bn_add_sign_pack(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O,
                                               dabnn_conv cv, const float* scale, const float* shift, const float* residual,
                                               float* y_out, uint64_t* out_packed, void* stream);
/* Eq. 1 (BGEMM) on the tensor-core engine: dabnn_bgemm with B expanded once by
 * dabnn_tc_prepare_weights(B, N, Kbits, 1, 1, b_tc) (dabnn_tc_weights_bytes(N, Kbits, 1, 1) bytes; Kbits <= 512).  Same integers. */
dabnn_status dabnn_tc_bgemm(const uint64_t* A, int M, const void* b_tc, int N, int Kbits, int32_t* C, void* stream);
int dabnn_tc_error_flag(void);
int dabnn_last_device_flag(void* stream);
dabnn_status dabnn_stream_status(void* stream);
dabnn_status dabnn_tc_wait_expiry_selftest(const uint64_t* a_packed, dabnn_shape in, const void* w_tc, int O, dabnn_conv cv,
                                           int32_t* out, int wait_polls, void* stream);
/* CTAs per tensor-engine launch at most (0 = the default: one persistent CTA, or CTA of a pair, per SM).  A launch takes
 * every SM it is given; a caller that runs independent layers side by side (several streams, or branches of a CUDA graph)
 * gets more out of the chip with launches capped at about half of it (74 on a B200).  Results do not depend on it.
 * Returns the previous setting.  Not thread-safe against concurrent calls into the library. */
int dabnn_tc_set_max_ctas(int max_ctas);

/* Selects the convolution inner loop for measurement runs: 0 = automatic (default),
 * 1 = one POPC per 32-bit word pair, 2 = carry-save (one POPC per two word pairs).  All give identical results.
 * Returns the previous setting.  Not thread-safe against concurrent calls into the library. */
int dabnn_set_conv_variant(int variant);
/* Forces the convolution's CTA tile for measurement runs: 0 = automatic (default), 1 = 128 pixels x 128 channels,
 * 2 = 128 x 64, 3 = 64 x 64, 4 = 32 x 32, 5 = 16 x 32 with all of K in flight (the choice for launches of less than
 * one wave).  All give identical results.  Returns the previous setting.
 * (Environment, read once, for measurements: DABNN_CONV_POINTWISE=0 keeps long unpadded 1x1 stride-1 layers on the
 * one-tile-per-CTA kernel instead of the form that walks four pixel tiles with the weight rows resident.) */
int dabnn_set_conv_tile(int tile);

#ifdef __cplusplus
}
#endif
#endif /* DABNN_H_ */
