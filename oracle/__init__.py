"""CPU oracle for binarized convolution -- TEST INFRASTRUCTURE, not the product.

A thin ctypes wrapper around ``oracle.c`` (plain scalar C written from the paper).
Only the tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library and its Python binding never do, and this package imports
nothing from them.

Every function takes and returns numpy arrays on the host.  Layout constants:
``NCHW = 0``, ``NHWC = 1``.  Packed activations are ``uint64 [N][H][W][ceil(C/64)]``,
packed weights ``uint64 [O][kh][kw][ceil(C/64)]`` (Section 2.1.1: one bit per element,
bit 1 for a negative value, channel c in word c>>6 at bit c&63).
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Sequence

import numpy as np

NCHW = 0
NHWC = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
CFLAGS = ["-O2", "-mfma", "-mpopcnt", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC"]


def build(force: bool = False) -> str:
    """Compile ``oracle.c`` with gcc into ``liboracle.so`` beside it (if stale)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.oracle_get_threads.restype = ctypes.c_int
        _lib.oracle_max_threads.restype = ctypes.c_int
    return _lib


def set_threads(n: int) -> None:
    lib().oracle_set_threads(ctypes.c_int(int(n)))


def get_threads() -> int:
    return int(lib().oracle_get_threads())


def max_threads() -> int:
    """Cores this process may use (its affinity mask), capped by what OpenMP sees."""
    try:
        aff = len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        aff = os.cpu_count() or 1
    return max(1, min(aff, int(lib().oracle_max_threads())))


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.float32)


def words_per_pixel(C: int) -> int:
    return (C + 63) // 64


def out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return (size + 2 * pad - k) // stride + 1


def pack(x: np.ndarray, layout: int = NCHW) -> np.ndarray:
    """Binarize and pack activations (Section 2.1.1).  x: fp32 NCHW or NHWC."""
    x = _f32(x)
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    P = np.empty((N, H, W, words_per_pixel(C)), dtype=np.uint64)
    lib().oracle_pack(_p(x), ctypes.c_int(layout), N, C, H, W, _p(P))
    return P


def pack_c2(x: np.ndarray, layout: int = NCHW) -> np.ndarray:
    """Binarize and pack into the NC1HWC2 layout (Section 2.1.2, last paragraph): uint64 [N][ceil(C/128)][H][W][2]."""
    x = _f32(x)
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    P = np.empty((N, (C + 127) // 128, H, W, 2), dtype=np.uint64)
    lib().oracle_pack_c2(_p(x), ctypes.c_int(layout), N, C, H, W, _p(P))
    return P


def bconv_bits_c2(A: np.ndarray, C: int, Wp: np.ndarray, stride=(1, 1), pad=(0, 0), pad_value=-1,
                  out_layout=NHWC) -> np.ndarray:
    """Eq. 1 with activations in the NC1HWC2 layout ([N][C1][H][W][2]); weights [O][kh][kw][Cw]."""
    A = np.ascontiguousarray(A, dtype=np.uint64)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint64)
    N, C1, H, W, two = A.shape
    O, kh, kw, Cw = Wp.shape
    assert two == 2 and C1 == (C + 127) // 128 and Cw == words_per_pixel(C)
    OH, OW = out_dim(H, kh, stride[0], pad[0]), out_dim(W, kw, stride[1], pad[1])
    out = np.empty(_out_shape(out_layout, N, O, OH, OW), dtype=np.int32)
    lib().oracle_bconv_bits_c2(_p(A), N, C, H, W, _p(Wp), O, kh, kw, stride[0], stride[1], pad[0], pad[1],
                               int(pad_value), _p(out), int(out_layout))
    return out


def pack_i32(x: np.ndarray, layout: int = NCHW) -> np.ndarray:
    """Pack the sign bits of int32 values (Section 2.1.1).  x: int32 NCHW or NHWC."""
    x = np.ascontiguousarray(x, dtype=np.int32)
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    P = np.empty((N, H, W, words_per_pixel(C)), dtype=np.uint64)
    lib().oracle_pack_i32(_p(x), ctypes.c_int(layout), N, C, H, W, _p(P))
    return P


def pack_weights(w_oihw: np.ndarray) -> np.ndarray:
    w = _f32(w_oihw)
    O, C, kh, kw = w.shape
    Wp = np.empty((O, kh, kw, words_per_pixel(C)), dtype=np.uint64)
    lib().oracle_pack_weights(_p(w), O, C, kh, kw, _p(Wp))
    return Wp


def _out_shape(layout, N, O, OH, OW):
    return (N, O, OH, OW) if layout == NCHW else (N, OH, OW, O)


def bconv_pm1(x_nchw, w_oihw, stride=(1, 1), pad=(0, 0), pad_value=-1, out_layout=NHWC) -> np.ndarray:
    """Convolution of the two {-1,+1} tensors, written as the definition (Section 2.1.2)."""
    x = _f32(x_nchw)
    w = _f32(w_oihw)
    N, C, H, W = x.shape
    O, C2, kh, kw = w.shape
    assert C == C2
    OH, OW = out_dim(H, kh, stride[0], pad[0]), out_dim(W, kw, stride[1], pad[1])
    out = np.empty(_out_shape(out_layout, N, O, OH, OW), dtype=np.int32)
    lib().oracle_bconv_pm1(_p(x), N, C, H, W, _p(w), O, kh, kw, stride[0], stride[1], pad[0], pad[1],
                           int(pad_value), _p(out), int(out_layout))
    return out


def bconv_pm1_at(x_nchw, w_oihw, coords, stride=(1, 1), pad=(0, 0), pad_value=-1) -> np.ndarray:
    """The same definition at the output coordinates ``coords`` = int32 [n][4] of (n, o, oh, ow)."""
    x = _f32(x_nchw)
    w = _f32(w_oihw)
    N, C, H, W = x.shape
    O, _, kh, kw = w.shape
    coords = np.ascontiguousarray(coords, dtype=np.int32)
    vals = np.empty(coords.shape[0], dtype=np.int32)
    lib().oracle_bconv_pm1_at(_p(x), N, C, H, W, _p(w), O, kh, kw, stride[0], stride[1], pad[0], pad[1],
                              int(pad_value), _p(coords), ctypes.c_int64(coords.shape[0]), _p(vals))
    return vals


def bconv_bits(A: np.ndarray, C: int, Wp: np.ndarray, stride=(1, 1), pad=(0, 0), pad_value=-1,
               out_layout=NHWC) -> np.ndarray:
    """Eq. 1 on packed words, returned as the +-1 dot product K - 2*popcount(xor)."""
    A = np.ascontiguousarray(A, dtype=np.uint64)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint64)
    N, H, W, Cw = A.shape
    O, kh, kw, Cw2 = Wp.shape
    assert Cw == Cw2 == words_per_pixel(C)
    OH, OW = out_dim(H, kh, stride[0], pad[0]), out_dim(W, kw, stride[1], pad[1])
    out = np.empty(_out_shape(out_layout, N, O, OH, OW), dtype=np.int32)
    lib().oracle_bconv_bits(_p(A), N, C, H, W, _p(Wp), O, kh, kw, stride[0], stride[1], pad[0], pad[1],
                            int(pad_value), _p(out), int(out_layout))
    return out


def bconv_bits_at(A, C, Wp, coords, stride=(1, 1), pad=(0, 0), pad_value=-1) -> np.ndarray:
    A = np.ascontiguousarray(A, dtype=np.uint64)
    Wp = np.ascontiguousarray(Wp, dtype=np.uint64)
    N, H, W, _ = A.shape
    O, kh, kw, _ = Wp.shape
    coords = np.ascontiguousarray(coords, dtype=np.int32)
    vals = np.empty(coords.shape[0], dtype=np.int32)
    lib().oracle_bconv_bits_at(_p(A), N, C, H, W, _p(Wp), O, kh, kw, stride[0], stride[1], pad[0], pad[1],
                               int(pad_value), _p(coords), ctypes.c_int64(coords.shape[0]), _p(vals))
    return vals


def bgemm_xnor(A: np.ndarray, B: np.ndarray, Kbits: int) -> np.ndarray:
    """Eq. 1 as printed: C[i][j] = sum_k bitcount(xnor(A[i][k], B[j][k])) over the Kbits valid positions.
    A: uint64 [M][Kw]; B: uint64 [N][Kw] (row j = column j of the paper's B).  Returns int32 [M][N]."""
    A = np.ascontiguousarray(A, dtype=np.uint64)
    B = np.ascontiguousarray(B, dtype=np.uint64)
    M, Kw = A.shape
    N, Kw2 = B.shape
    assert Kw == Kw2 == words_per_pixel(Kbits)
    C = np.empty((M, N), dtype=np.int32)
    lib().oracle_bgemm_xnor(_p(A), M, _p(B), N, int(Kbits), _p(C))
    return C


def bn_fold(gamma, beta, mean, var, eps: float = 1e-5):
    """BN parameters -> (scale, shift) in double, rounded once to fp32 each."""
    g, b, m, v = (_f32(t) for t in (gamma, beta, mean, var))
    O = g.shape[0]
    scale = np.empty(O, dtype=np.float32)
    shift = np.empty(O, dtype=np.float32)
    lib().oracle_bn_fold(_p(g), _p(b), _p(m), _p(v), ctypes.c_double(eps), O, _p(scale), _p(shift))
    return scale, shift


def bn_sign_pack(acc_nhwc: np.ndarray, scale, shift) -> np.ndarray:
    """y = fmaf(acc, scale, shift); bit = (y < 0); packed along the channel axis."""
    acc = np.ascontiguousarray(acc_nhwc, dtype=np.int32)
    O = acc.shape[-1]
    npix = acc.size // O
    out = np.empty(acc.shape[:-1] + (words_per_pixel(O),), dtype=np.uint64)
    lib().oracle_bn_sign_pack(_p(acc), ctypes.c_int64(npix), O, _p(_f32(scale)), _p(_f32(shift)), _p(out))
    return out


def bn_add_sign_pack(acc_nhwc: np.ndarray, scale, shift, residual: np.ndarray):
    """The Bi-Real block epilogue (Sections 2.1.1 and 2.3): y = fmaf(acc, scale, shift) + residual (one rounded add);
    returns (y fp32, same shape as acc; packed sign bits of y along the channel axis)."""
    acc = np.ascontiguousarray(acc_nhwc, dtype=np.int32)
    r = _f32(residual)
    assert r.shape == acc.shape
    O = acc.shape[-1]
    npix = acc.size // O
    y = np.empty(acc.shape, dtype=np.float32)
    bits = np.empty(acc.shape[:-1] + (words_per_pixel(O),), dtype=np.uint64)
    lib().oracle_bn_add_sign_pack(_p(acc), ctypes.c_int64(npix), O, _p(_f32(scale)), _p(_f32(shift)), _p(r), _p(y), _p(bits))
    return y, bits


def bitcount(v: int) -> int:
    """The bitcount the C code uses for Eq. 1, on one 64-bit word."""
    lib().oracle_bitcount.restype = ctypes.c_int
    return int(lib().oracle_bitcount(ctypes.c_uint64(int(v) & (2**64 - 1))))


class _Bireal18Params(ctypes.Structure):
    _fields_ = [
        ("stem_w", ctypes.c_void_p),
        ("stem_bn", ctypes.c_void_p * 4),
        ("block_w", ctypes.c_void_p * 16),
        ("block_bn", (ctypes.c_void_p * 4) * 16),
        ("down_w", ctypes.c_void_p * 3),
        ("down_bn", (ctypes.c_void_p * 4) * 3),
        ("fc_w", ctypes.c_void_p),
        ("fc_b", ctypes.c_void_p),
        ("bn_eps", ctypes.c_double),
        ("conv_form", ctypes.c_int),
        ("use_stem_module", ctypes.c_int),
        ("sm_w", ctypes.c_void_p * 4),
        ("sm_bn", (ctypes.c_void_p * 4) * 4),
    ]


STAGE_C = (64, 128, 256, 512)
STAGE_HW = (56, 28, 14, 7)


def bireal18_forward(params: dict, images: np.ndarray, conv_form: int = 1, want_taps: bool = False,
                     stem_module: bool = False):
    """Bi-Real Net 18 forward (Section 2.3).

    ``params`` holds fp32 numpy arrays: ``stem_w`` [64,3,7,7]; ``stem_bn`` = (gamma, beta,
    mean, var); ``block_w[b]`` [O,C,3,3]; ``block_bn[b]``; ``down_w[d]`` [O,C];
    ``down_bn[d]``; ``fc_w`` [1000,512]; ``fc_b`` [1000].  ``conv_form`` 0 uses the +-1
    products, 1 uses Eq. 1 on packed words (identical integers).  Returns logits [N,1000]
    (and, if asked, the 17 intermediate activations as fp32 NCHW arrays).  ``stem_module``: the STEM module of
    Section 2.3 (a reading of the missing Fig. 6, see oracle.c) in place of the 7x7 convolution and the max-pool.
    """
    keep = []

    def ptr(a):
        a = _f32(a)
        keep.append(a)
        return a.ctypes.data

    P = _Bireal18Params()
    P.stem_w = ptr(params["stem_w"])
    for i in range(4):
        P.stem_bn[i] = ptr(params["stem_bn"][i])
    for b in range(16):
        P.block_w[b] = ptr(params["block_w"][b])
        for i in range(4):
            P.block_bn[b][i] = ptr(params["block_bn"][b][i])
    for d in range(3):
        P.down_w[d] = ptr(params["down_w"][d])
        for i in range(4):
            P.down_bn[d][i] = ptr(params["down_bn"][d][i])
    P.fc_w = ptr(params["fc_w"])
    P.fc_b = ptr(params["fc_b"])
    P.bn_eps = float(params.get("bn_eps", 1e-5))
    P.conv_form = int(conv_form)
    P.use_stem_module = 1 if stem_module else 0
    if stem_module:  # params["stem_module"] = {"w": [4 arrays OIHW], "bn": [4 x (gamma, beta, mean, var)]} (Section 2.3)
        for i in range(4):
            P.sm_w[i] = ptr(params["stem_module"]["w"][i])
            for j in range(4):
                P.sm_bn[i][j] = ptr(params["stem_module"]["bn"][i][j])
    images = _f32(images)
    N = images.shape[0]
    assert images.shape[1:] == (3, 224, 224)
    logits = np.empty((N, 1000), dtype=np.float32)
    taps = None
    tap_ptrs = None
    if want_taps:
        taps = [np.empty((N, 64, 56, 56), dtype=np.float32)]
        for b in range(16):
            s = b // 4
            taps.append(np.empty((N, STAGE_C[s], STAGE_HW[s], STAGE_HW[s]), dtype=np.float32))
        tap_ptrs = (ctypes.c_void_p * 17)(*[t.ctypes.data for t in taps])
    lib().oracle_bireal18_forward(ctypes.byref(P), _p(images), N, _p(logits), tap_ptrs)
    return (logits, taps) if want_taps else logits
