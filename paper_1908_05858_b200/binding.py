"""Thin ctypes binding over the C ABI of ``libdabnn_b200.so`` (see ``include/dabnn.h``).

Argument marshalling only: every function checks dtypes / devices, allocates the output tensor with
torch (torch owns device memory and the stream) and calls the entry point of the same name.  There
is no CPU path: without the compiled library, or with a tensor that is not on a CUDA device, the
functions raise.

Packed tensors are ``torch.int64`` on the device (the bit pattern of the library's ``uint64`` words).
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

NCHW = 0
NHWC = 1

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdabnn_b200.so")

EXPORTS = (
    "dabnn_status_string", "dabnn_words_per_pixel", "dabnn_out_dim", "dabnn_pack", "dabnn_pack_i32", "dabnn_pack_weights",
    "dabnn_bconv2d", "dabnn_bgemm", "dabnn_bconv2d_bn_sign_pack", "dabnn_bconv2d_bn_add_sign_pack", "dabnn_bn_fold",
    "dabnn_bireal18_workspace_bytes", "dabnn_bireal18_forward", "dabnn_set_conv_variant",
    "dabnn_binary_layer_host_workspace_bytes", "dabnn_binary_layer_host", "dabnn_bireal18_forward_static", "dabnn_set_conv_tile",
    "dabnn_tc_set_max_ctas", "dabnn_tc_weights_bytes", "dabnn_tc_prepare_weights", "dabnn_tc_bconv2d", "dabnn_tc_bconv2d_bn_sign_pack",
    "dabnn_tc_bconv2d_bn_add_sign_pack", "dabnn_tc_error_flag", "dabnn_last_device_flag", "dabnn_stream_status",
    "dabnn_tc_wait_expiry_selftest", "dabnn_packed_words", "dabnn_pack_as", "dabnn_bconv2d_from",
    "dabnn_bireal18_forward_stem_module", "dabnn_tc_bgemm",
)

PACKED_NHWC = 0
PACKED_NC1HWC2 = 1

ERR_TIMEOUT = 7
ERR_STATIC_LIMIT = 8


class DabnnError(RuntimeError):
    pass


class Shape(ctypes.Structure):
    _fields_ = [("N", ctypes.c_int), ("C", ctypes.c_int), ("H", ctypes.c_int), ("W", ctypes.c_int)]


class Conv(ctypes.Structure):
    _fields_ = [("kh", ctypes.c_int), ("kw", ctypes.c_int), ("stride_h", ctypes.c_int), ("stride_w", ctypes.c_int),
                ("pad_h", ctypes.c_int), ("pad_w", ctypes.c_int), ("pad_value", ctypes.c_int)]


class Bireal18Params(ctypes.Structure):
    _fields_ = [
        ("stem_w", ctypes.c_void_p), ("stem_scale", ctypes.c_void_p), ("stem_shift", ctypes.c_void_p),
        ("block_w", ctypes.c_void_p * 16), ("block_scale", ctypes.c_void_p * 16), ("block_shift", ctypes.c_void_p * 16),
        ("down_w", ctypes.c_void_p * 3), ("down_scale", ctypes.c_void_p * 3), ("down_shift", ctypes.c_void_p * 3),
        ("fc_w", ctypes.c_void_p), ("fc_b", ctypes.c_void_p),
        ("block_w_tc", ctypes.c_void_p * 16),
    ]


class StemModuleParams(ctypes.Structure):
    _fields_ = [("w", ctypes.c_void_p * 4), ("scale", ctypes.c_void_p * 4), ("shift", ctypes.c_void_p * 4)]


_lib: Optional[ctypes.CDLL] = None


def lib() -> ctypes.CDLL:
    """Loads the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise DabnnError("libdabnn_b200.so is missing: run `python -m paper_1908_05858_b200.build` "
                             "(or __graft_entry__.build()) first; there is no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        L.dabnn_status_string.restype = ctypes.c_char_p
        L.dabnn_status_string.argtypes = [ci]
        L.dabnn_words_per_pixel.restype = ctypes.c_size_t
        L.dabnn_words_per_pixel.argtypes = [ci]
        L.dabnn_out_dim.restype = ci
        L.dabnn_out_dim.argtypes = [ci, ci, ci, ci]
        L.dabnn_pack.argtypes = [vp, ci, Shape, vp, vp]
        L.dabnn_pack_i32.argtypes = [vp, ci, Shape, vp, vp]
        L.dabnn_pack_i32.restype = ci
        L.dabnn_pack_weights.argtypes = [vp, ci, ci, ci, ci, vp, vp]
        L.dabnn_bconv2d.argtypes = [vp, Shape, vp, ci, Conv, vp, ci, vp]
        L.dabnn_bgemm.argtypes = [vp, ci, vp, ci, ci, vp, vp]
        L.dabnn_bgemm.restype = ci
        L.dabnn_bconv2d_bn_sign_pack.argtypes = [vp, Shape, vp, ci, Conv, vp, vp, vp, vp]
        L.dabnn_bconv2d_bn_add_sign_pack.argtypes = [vp, Shape, vp, ci, Conv, vp, vp, vp, vp, vp, vp]
        L.dabnn_bn_fold.argtypes = [vp, vp, vp, vp, ctypes.c_double, ci, vp, vp, vp]
        L.dabnn_bireal18_workspace_bytes.restype = ctypes.c_size_t
        L.dabnn_bireal18_workspace_bytes.argtypes = [ci]
        L.dabnn_bireal18_forward.argtypes = [ctypes.POINTER(Bireal18Params), vp, ci, vp, vp, ctypes.c_size_t, vp]
        L.dabnn_binary_layer_host_workspace_bytes.restype = ctypes.c_size_t
        L.dabnn_binary_layer_host_workspace_bytes.argtypes = [Shape, ci, Conv]
        L.dabnn_binary_layer_host.argtypes = [vp, Shape, vp, ci, Conv, vp, vp, vp, vp, vp, ctypes.c_size_t, vp]
        L.dabnn_binary_layer_host.restype = ci
        L.dabnn_set_conv_variant.restype = ci
        L.dabnn_set_conv_variant.argtypes = [ci]
        L.dabnn_tc_set_max_ctas.restype = ci
        L.dabnn_tc_set_max_ctas.argtypes = [ci]
        L.dabnn_tc_weights_bytes.restype = ctypes.c_size_t
        L.dabnn_tc_weights_bytes.argtypes = [ci, ci, ci, ci]
        L.dabnn_tc_prepare_weights.argtypes = [vp, ci, ci, ci, ci, vp, vp]
        L.dabnn_tc_bconv2d.argtypes = [vp, Shape, vp, ci, Conv, vp, ci, vp]
        L.dabnn_tc_bconv2d_bn_sign_pack.argtypes = [vp, Shape, vp, ci, Conv, vp, vp, vp, vp]
        L.dabnn_tc_bconv2d_bn_add_sign_pack.argtypes = [vp, Shape, vp, ci, Conv, vp, vp, vp, vp, vp, vp]
        for name in ("dabnn_tc_prepare_weights", "dabnn_tc_bconv2d", "dabnn_tc_bconv2d_bn_sign_pack",
                     "dabnn_tc_bconv2d_bn_add_sign_pack", "dabnn_tc_error_flag"):
            getattr(L, name).restype = ci
        L.dabnn_set_conv_tile.restype = ci
        L.dabnn_set_conv_tile.argtypes = [ci]
        L.dabnn_bireal18_forward_stem_module.restype = ci
        L.dabnn_bireal18_forward_stem_module.argtypes = [ctypes.POINTER(Bireal18Params), ctypes.POINTER(StemModuleParams), vp, ci, vp, vp,
                                                         ctypes.c_size_t, vp]
        L.dabnn_tc_bgemm.restype = ci
        L.dabnn_tc_bgemm.argtypes = [vp, ci, vp, ci, ci, vp, vp]
        L.dabnn_packed_words.restype = ctypes.c_size_t
        L.dabnn_packed_words.argtypes = [Shape, ci]
        L.dabnn_pack_as.restype = ci
        L.dabnn_pack_as.argtypes = [vp, ci, Shape, ci, vp, vp]
        L.dabnn_bconv2d_from.restype = ci
        L.dabnn_bconv2d_from.argtypes = [vp, ci, Shape, vp, ci, Conv, vp, ci, vp]
        L.dabnn_last_device_flag.restype = ci
        L.dabnn_last_device_flag.argtypes = [vp]
        L.dabnn_stream_status.restype = ci
        L.dabnn_stream_status.argtypes = [vp]
        L.dabnn_tc_wait_expiry_selftest.restype = ci
        L.dabnn_tc_wait_expiry_selftest.argtypes = [vp, Shape, vp, ci, Conv, vp, ci, vp]
        L.dabnn_bireal18_forward_static.restype = ci
        L.dabnn_bireal18_forward_static.argtypes = [ctypes.POINTER(Bireal18Params), vp, ci, vp, vp]
        for name in ("dabnn_pack", "dabnn_pack_weights", "dabnn_bconv2d", "dabnn_bconv2d_bn_sign_pack",
                     "dabnn_bconv2d_bn_add_sign_pack", "dabnn_bn_fold", "dabnn_bireal18_forward"):
            getattr(L, name).restype = ci
        _lib = L
    return _lib


def _default_alloc(shape, dtype, device) -> torch.Tensor:
    return torch.empty(tuple(shape), dtype=dtype, device=device)


_alloc = _default_alloc


def set_output_allocator(fn=None):
    """Every output tensor and workspace that this module creates comes from ``fn(shape, dtype, device)`` (default:
    ``torch.empty``).  A caller with its own memory pool passes its allocator; the tests pass one that puts guard
    bytes around each output.  Returns the previous allocator."""
    global _alloc
    prev = _alloc
    _alloc = fn if fn is not None else _default_alloc
    return prev


def _check(status: int) -> None:
    if status != 0:
        raise DabnnError("dabnn status %d: %s" % (status, lib().dabnn_status_string(status).decode()))


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dev(t: torch.Tensor, dtype: torch.dtype, name: str) -> torch.Tensor:
    if not isinstance(t, torch.Tensor) or not t.is_cuda:
        raise DabnnError("%s must be a CUDA tensor (there is no CPU path)" % name)
    if t.dtype != dtype:
        raise DabnnError("%s must have dtype %s, got %s" % (name, dtype, t.dtype))
    return t.contiguous()


def words_per_pixel(C: int) -> int:
    return int(lib().dabnn_words_per_pixel(C))


def out_dim(size: int, k: int, stride: int, pad: int) -> int:
    return int(lib().dabnn_out_dim(size, k, stride, pad))


def _conv(kh, kw, stride, pad, pad_value) -> Conv:
    return Conv(kh, kw, stride[0], stride[1], pad[0], pad[1], pad_value)


def pack(x: torch.Tensor, layout: int = NCHW, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_pack: fp32 NCHW or NHWC -> packed int64 [N][H][W][Cw]."""
    x = _dev(x, torch.float32, "x")
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    if out is None:
        out = _alloc((N, H, W, words_per_pixel(C)), torch.int64, x.device)
    _check(lib().dabnn_pack(x.data_ptr(), layout, Shape(N, C, H, W), out.data_ptr(), _stream()))
    return out


def pack_as(x: torch.Tensor, packed_layout: int, layout: int = NCHW, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_pack_as: PACKED_NHWC gives int64 [N][H][W][Cw]; PACKED_NC1HWC2 gives int64 [N][C1][H][W][2] (Section 2.1.2)."""
    x = _dev(x, torch.float32, "x")
    N, C, H, W = x.shape if layout == NCHW else (x.shape[0], x.shape[3], x.shape[1], x.shape[2])
    if out is None:
        shape = (N, (C + 127) // 128, H, W, 2) if packed_layout == PACKED_NC1HWC2 else (N, H, W, words_per_pixel(C))
        out = _alloc(shape, torch.int64, x.device)
    if out.numel() != int(lib().dabnn_packed_words(Shape(N, C, H, W), packed_layout)):
        raise DabnnError("packed tensor has the wrong size for this layout")
    _check(lib().dabnn_pack_as(x.data_ptr(), layout, Shape(N, C, H, W), packed_layout, out.data_ptr(), _stream()))
    return out


def bconv2d_from(a_packed, packed_layout: int, C: int, w_packed, stride=(1, 1), pad=(0, 0), pad_value: int = -1,
                 out_layout: int = NHWC, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_bconv2d_from: dabnn_bconv2d on activations in either packed layout."""
    a = _dev(a_packed, torch.int64, "a_packed")
    w = _dev(w_packed, torch.int64, "w_packed")
    if packed_layout == PACKED_NC1HWC2:
        N, C1, H, W, two = a.shape
        if two != 2 or C1 != (C + 127) // 128:
            raise DabnnError("NC1HWC2 activations must be [N][ceil(C/128)][H][W][2]")
    else:
        N, H, W, Cw = a.shape
        if Cw != (C + 63) // 64:
            raise DabnnError("packed word counts do not match C")
    O, kh, kw, Cw2 = w.shape
    if Cw2 != (C + 63) // 64:
        raise DabnnError("packed word counts do not match C")
    OH, OW = out_dim(H, kh, stride[0], pad[0]), out_dim(W, kw, stride[1], pad[1])
    if out is None:
        shape = (N, max(OH, 0), max(OW, 0), O) if out_layout == NHWC else (N, O, max(OH, 0), max(OW, 0))
        out = _alloc(shape, torch.int32, a.device)
    _check(lib().dabnn_bconv2d_from(a.data_ptr(), packed_layout, Shape(N, C, H, W), w.data_ptr(), O,
                                    _conv(kh, kw, stride, pad, pad_value), out.data_ptr(), out_layout, _stream()))
    return out


def pack_i32(x: torch.Tensor, layout: int = NCHW, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_pack_i32: int32 NCHW or NHWC -> packed int64 [N][H][W][Cw] (bit = x < 0)."""
    x = _dev(x, torch.int32, "x")
    if layout == NCHW:
        N, C, H, W = x.shape
    else:
        N, H, W, C = x.shape
    if out is None:
        out = _alloc((N, H, W, words_per_pixel(C)), torch.int64, x.device)
    _check(lib().dabnn_pack_i32(x.data_ptr(), layout, Shape(N, C, H, W), out.data_ptr(), _stream()))
    return out


def pack_weights(w_oihw: torch.Tensor) -> torch.Tensor:
    """dabnn_pack_weights: fp32 OIHW -> packed int64 [O][kh][kw][Cw]."""
    w = _dev(w_oihw, torch.float32, "w")
    O, C, kh, kw = w.shape
    out = _alloc((O, kh, kw, words_per_pixel(C)), torch.int64, w.device)
    _check(lib().dabnn_pack_weights(w.data_ptr(), O, C, kh, kw, out.data_ptr(), _stream()))
    return out


def _geom(a_packed, C, w_packed, stride, pad):
    a = _dev(a_packed, torch.int64, "a_packed")
    w = _dev(w_packed, torch.int64, "w_packed")
    N, H, W, Cw = a.shape
    O, kh, kw, Cw2 = w.shape
    if Cw != Cw2 or Cw != (C + 63) // 64:
        raise DabnnError("packed word counts do not match C")
    OH, OW = out_dim(H, kh, stride[0], pad[0]), out_dim(W, kw, stride[1], pad[1])
    return a, w, N, H, W, O, kh, kw, OH, OW


def bconv2d(a_packed, C: int, w_packed, stride=(1, 1), pad=(0, 0), pad_value: int = -1, out_layout: int = NHWC,
            out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_bconv2d: int32 result, NHWC [N][OH][OW][O] or NCHW [N][O][OH][OW]."""
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    if out is None:
        shape = (N, max(OH, 0), max(OW, 0), O) if out_layout == NHWC else (N, O, max(OH, 0), max(OW, 0))
        out = _alloc(shape, torch.int32, a.device)
    _check(lib().dabnn_bconv2d(a.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O, _conv(kh, kw, stride, pad, pad_value),
                               out.data_ptr(), out_layout, _stream()))
    return out


def bgemm(A: torch.Tensor, B: torch.Tensor, Kbits: int) -> torch.Tensor:
    """dabnn_bgemm: A int64 [M][Kw], B int64 [N][Kw] -> int32 [M][N] of +-1 dot products over Kbits positions."""
    A = _dev(A, torch.int64, "A")
    B = _dev(B, torch.int64, "B")
    M, Kw = A.shape
    N, Kw2 = B.shape
    if Kw != Kw2 or Kw != (Kbits + 63) // 64:
        raise DabnnError("packed word counts do not match Kbits")
    out = _alloc((M, N), torch.int32, A.device)
    _check(lib().dabnn_bgemm(A.data_ptr(), M, B.data_ptr(), N, int(Kbits), out.data_ptr(), _stream()))
    return out


def bconv2d_bn_sign_pack(a_packed, C: int, w_packed, scale, shift, stride=(1, 1), pad=(0, 0), pad_value: int = -1,
                         out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_bconv2d_bn_sign_pack: packed int64 [N][OH][OW][ceil(O/64)]."""
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    scale = _dev(scale, torch.float32, "scale")
    shift = _dev(shift, torch.float32, "shift")
    if out is None:
        out = _alloc((N, max(OH, 0), max(OW, 0), words_per_pixel(O)), torch.int64, a.device)
    _check(lib().dabnn_bconv2d_bn_sign_pack(a.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O,
                                            _conv(kh, kw, stride, pad, pad_value), scale.data_ptr(), shift.data_ptr(),
                                            out.data_ptr(), _stream()))
    return out


def bconv2d_bn_add_sign_pack(a_packed, C: int, w_packed, scale, shift, residual, stride=(1, 1), pad=(0, 0),
                             pad_value: int = -1, want_bits: bool = True):
    """dabnn_bconv2d_bn_add_sign_pack: returns (y fp32 NHWC, packed signs of y or None)."""
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    scale = _dev(scale, torch.float32, "scale")
    shift = _dev(shift, torch.float32, "shift")
    residual = _dev(residual, torch.float32, "residual")
    if tuple(residual.shape) != (N, OH, OW, O):
        raise DabnnError("residual must be NHWC [N][OH][OW][O]")
    y = _alloc(residual.shape, torch.float32, a.device)
    bits = _alloc((N, OH, OW, words_per_pixel(O)), torch.int64, a.device) if want_bits else None
    _check(lib().dabnn_bconv2d_bn_add_sign_pack(a.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O,
                                                _conv(kh, kw, stride, pad, pad_value), scale.data_ptr(),
                                                shift.data_ptr(), residual.data_ptr(), y.data_ptr(),
                                                bits.data_ptr() if want_bits else None, _stream()))
    return y, bits


def bn_fold(gamma, beta, mean, var, eps: float = 1e-5):
    """dabnn_bn_fold: (scale, shift) fp32 device tensors."""
    g, b, m, v = (_dev(t, torch.float32, "bn") for t in (gamma, beta, mean, var))
    O = g.numel()
    scale = _alloc((O,), torch.float32, g.device)
    shift = _alloc((O,), torch.float32, g.device)
    _check(lib().dabnn_bn_fold(g.data_ptr(), b.data_ptr(), m.data_ptr(), v.data_ptr(), float(eps), O,
                               scale.data_ptr(), shift.data_ptr(), _stream()))
    return scale, shift


def bireal18_workspace_bytes(N: int) -> int:
    return int(lib().dabnn_bireal18_workspace_bytes(N))


class Bireal18:
    """Device-resident Bi-Real Net 18 parameters, prepared once with the library's own kernels
    (weights packed by dabnn_pack_weights, BN folded by dabnn_bn_fold)."""

    def __init__(self, params: dict, device="cuda", engine: str = "auto"):
        """engine: "auto" / "tc" = tensor-core engine for the blocks it covers, "popc" = integer-pipe kernel only."""
        dev = torch.device(device)

        def up(a):
            return torch.as_tensor(a, dtype=torch.float32).contiguous().to(dev)

        eps = float(params.get("bn_eps", 1e-5))
        self.keep = []
        P = Bireal18Params()
        self.stem_w = up(params["stem_w"])
        self.stem_scale, self.stem_shift = bn_fold(*[up(t) for t in params["stem_bn"]], eps=eps)
        P.stem_w, P.stem_scale, P.stem_shift = self.stem_w.data_ptr(), self.stem_scale.data_ptr(), self.stem_shift.data_ptr()
        for b in range(16):
            wp = pack_weights(up(params["block_w"][b]))
            sc, sh = bn_fold(*[up(t) for t in params["block_bn"][b]], eps=eps)
            self.keep += [wp, sc, sh]
            P.block_w[b], P.block_scale[b], P.block_shift[b] = wp.data_ptr(), sc.data_ptr(), sh.data_ptr()
            O_b, C_b = int(params["block_w"][b].shape[0]), int(params["block_w"][b].shape[1])
            stride_b = 2 if (b % 4 == 0 and b > 0) else 1
            if engine != "popc" and tc_supported(O_b, C_b, 3, 3, (stride_b, stride_b)):
                wt = TcWeights(wp, C_b)
                self.keep.append(wt)
                P.block_w_tc[b] = wt.buf.data_ptr()
        for d in range(3):
            w = up(params["down_w"][d])
            sc, sh = bn_fold(*[up(t) for t in params["down_bn"][d]], eps=eps)
            self.keep += [w, sc, sh]
            P.down_w[d], P.down_scale[d], P.down_shift[d] = w.data_ptr(), sc.data_ptr(), sh.data_ptr()
        self.fc_w, self.fc_b = up(params["fc_w"]), up(params["fc_b"])
        P.fc_w, P.fc_b = self.fc_w.data_ptr(), self.fc_b.data_ptr()
        self.P = P
        self.device = dev
        self._ws = None
        self.SM = None
        if "stem_module" in params:  # Section 2.3: the STEM module variant (forward_stem_module)
            SM = StemModuleParams()
            for i in range(4):
                w = up(params["stem_module"]["w"][i])
                sc, sh = bn_fold(*[up(t) for t in params["stem_module"]["bn"][i]], eps=eps)
                self.keep += [w, sc, sh]
                SM.w[i], SM.scale[i], SM.shift[i] = w.data_ptr(), sc.data_ptr(), sh.data_ptr()
            self.SM = SM

    def workspace(self, N: int) -> torch.Tensor:
        need = bireal18_workspace_bytes(N)
        if self._ws is None or self._ws.numel() < need:
            self._ws = _alloc((need,), torch.uint8, self.device)
        return self._ws

    def forward(self, images: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
        """dabnn_bireal18_forward: images fp32 NCHW [N][3][224][224] -> logits fp32 [N][1000]."""
        images = _dev(images, torch.float32, "images")
        N = images.shape[0]
        if tuple(images.shape[1:]) != (3, 224, 224):
            raise DabnnError("images must be [N][3][224][224]")
        ws = self.workspace(N)
        if logits is None:
            logits = _alloc((N, 1000), torch.float32, images.device)
        _check(lib().dabnn_bireal18_forward(ctypes.byref(self.P), images.data_ptr(), N, logits.data_ptr(),
                                            ws.data_ptr(), ws.numel(), _stream()))
        return logits


def bireal18_forward_stem_module(net: "Bireal18", images: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_bireal18_forward_stem_module: the forward pass with the STEM module (the net's params held "stem_module")."""
    if net.SM is None:
        raise DabnnError("this network was built without STEM module parameters")
    images = _dev(images, torch.float32, "images")
    N = images.shape[0]
    if tuple(images.shape[1:]) != (3, 224, 224):
        raise DabnnError("images must be [N][3][224][224]")
    ws = net.workspace(N)
    if logits is None:
        logits = _alloc((N, 1000), torch.float32, images.device)
    _check(lib().dabnn_bireal18_forward_stem_module(ctypes.byref(net.P), ctypes.byref(net.SM), images.data_ptr(), N,
                                                    logits.data_ptr(), ws.data_ptr(), ws.numel(), _stream()))
    return logits


def binary_layer_host_workspace_bytes(N, C, H, W, O, kh, kw, stride=(1, 1), pad=(0, 0), pad_value=-1) -> int:
    return int(lib().dabnn_binary_layer_host_workspace_bytes(Shape(N, C, H, W), O, _conv(kh, kw, stride, pad, pad_value)))


def binary_layer_host(x_host: torch.Tensor, w_packed: torch.Tensor, workspace: torch.Tensor, stride=(1, 1), pad=(0, 0),
                      pad_value: int = -1, scale=None, shift=None, out_host: Optional[torch.Tensor] = None,
                      bits_host: Optional[torch.Tensor] = None):
    """dabnn_binary_layer_host: x_host / out_host / bits_host are HOST tensors (pin them for asynchronous
    copies); w_packed, scale, shift, workspace are device tensors.  Work is enqueued on the current stream."""
    if x_host.is_cuda or x_host.dtype != torch.float32 or not x_host.is_contiguous():
        raise DabnnError("x_host must be a contiguous fp32 host tensor")
    w = _dev(w_packed, torch.int64, "w_packed")
    N, C, H, W = x_host.shape
    O, kh, kw, _ = w.shape
    for t, dt in ((out_host, torch.int32), (bits_host, torch.int64)):
        if t is not None and (t.is_cuda or t.dtype != dt or not t.is_contiguous()):
            raise DabnnError("host outputs must be contiguous host tensors of the right dtype")
    _check(lib().dabnn_binary_layer_host(
        x_host.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O, _conv(kh, kw, stride, pad, pad_value),
        scale.data_ptr() if scale is not None else None, shift.data_ptr() if shift is not None else None,
        out_host.data_ptr() if out_host is not None else None, bits_host.data_ptr() if bits_host is not None else None,
        workspace.data_ptr(), workspace.numel() * workspace.element_size(), _stream()))


STATIC_MAX_BATCH = 2


def bireal18_forward_static(net: "Bireal18", images: torch.Tensor, logits: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_bireal18_forward_static: the same forward pass for callers that may not allocate device memory
    (the library's built-in scratch area replaces the workspace; at most STATIC_MAX_BATCH images per call).
    Only `logits` is allocated here, by torch, when the caller does not pass it."""
    images = _dev(images, torch.float32, "images")
    N = images.shape[0]
    if tuple(images.shape[1:]) != (3, 224, 224):
        raise DabnnError("images must be [N][3][224][224]")
    if logits is None:
        logits = _alloc((N, 1000), torch.float32, images.device)
    _check(lib().dabnn_bireal18_forward_static(ctypes.byref(net.P), images.data_ptr(), N, logits.data_ptr(), _stream()))
    return logits


# ---- tensor-core engine ---------------------------------------------------------------------------------------------
class TcWeights:
    """Expanded 4-bit (e2m1) weights for the tensor-core engine (dabnn_tc_prepare_weights), with the filter geometry."""

    def __init__(self, w_packed: torch.Tensor, C: int):
        w = _dev(w_packed, torch.int64, "w_packed")
        self.O, self.kh, self.kw, Cw = w.shape
        self.C = C
        nbytes = int(lib().dabnn_tc_weights_bytes(self.O, C, self.kh, self.kw))
        if nbytes == 0:
            raise DabnnError("this filter bank is not covered by the tensor-core engine")
        self.buf = _alloc((nbytes,), torch.uint8, w.device)
        _check(lib().dabnn_tc_prepare_weights(w.data_ptr(), self.O, C, self.kh, self.kw, self.buf.data_ptr(), _stream()))


def tc_supported(O: int, C: int, kh: int, kw: int, stride=(1, 1)) -> bool:
    return tuple(stride) in ((1, 1), (2, 2)) and int(lib().dabnn_tc_weights_bytes(O, C, kh, kw)) > 0


def _tc_geom(a_packed, wt: TcWeights, stride, pad):
    a = _dev(a_packed, torch.int64, "a_packed")
    N, H, W, Cw = a.shape
    if Cw != (wt.C + 63) // 64:
        raise DabnnError("packed word count does not match C")
    OH, OW = out_dim(H, wt.kh, stride[0], pad[0]), out_dim(W, wt.kw, stride[1], pad[1])
    return a, N, H, W, OH, OW


def tc_bconv2d(a_packed, wt: TcWeights, stride=(1, 1), pad=(0, 0), pad_value: int = -1, out_layout: int = NHWC,
               out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_tc_bconv2d."""
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    if out is None:
        shape = (N, OH, OW, wt.O) if out_layout == NHWC else (N, wt.O, OH, OW)
        out = _alloc(shape, torch.int32, a.device)
    _check(lib().dabnn_tc_bconv2d(a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O,
                                  _conv(wt.kh, wt.kw, stride, pad, pad_value), out.data_ptr(), out_layout, _stream()))
    return out


def tc_bconv2d_bn_sign_pack(a_packed, wt: TcWeights, scale, shift, stride=(1, 1), pad=(0, 0), pad_value: int = -1,
                            out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """dabnn_tc_bconv2d_bn_sign_pack."""
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    scale, shift = _dev(scale, torch.float32, "scale"), _dev(shift, torch.float32, "shift")
    if out is None:
        out = _alloc((N, OH, OW, words_per_pixel(wt.O)), torch.int64, a.device)
    _check(lib().dabnn_tc_bconv2d_bn_sign_pack(a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O,
                                               _conv(wt.kh, wt.kw, stride, pad, pad_value), scale.data_ptr(),
                                               shift.data_ptr(), out.data_ptr(), _stream()))
    return out


def tc_bconv2d_bn_add_sign_pack(a_packed, wt: TcWeights, scale, shift, residual, stride=(1, 1), pad=(0, 0),
                                pad_value: int = -1, want_bits: bool = True):
    """dabnn_tc_bconv2d_bn_add_sign_pack."""
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    scale, shift = _dev(scale, torch.float32, "scale"), _dev(shift, torch.float32, "shift")
    residual = _dev(residual, torch.float32, "residual")
    y = _alloc(residual.shape, torch.float32, a.device)
    bits = _alloc((N, OH, OW, words_per_pixel(wt.O)), torch.int64, a.device) if want_bits else None
    _check(lib().dabnn_tc_bconv2d_bn_add_sign_pack(a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O,
                                                   _conv(wt.kh, wt.kw, stride, pad, pad_value), scale.data_ptr(),
                                                   shift.data_ptr(), residual.data_ptr(), y.data_ptr(),
                                                   bits.data_ptr() if want_bits else None, _stream()))
    return y, bits


def tc_bgemm(A: torch.Tensor, Bt: "TcWeights", Kbits: int) -> torch.Tensor:
    """dabnn_tc_bgemm: A int64 [M][Kw] times the rows of B (a TcWeights built from B viewed as [N][1][1][Kw]) -> int32 [M][N]."""
    A = _dev(A, torch.int64, "A")
    M, Kw = A.shape
    if Kw != (Kbits + 63) // 64 or Bt.C != Kbits or Bt.kh != 1 or Bt.kw != 1:
        raise DabnnError("operands do not match Kbits")
    out = _alloc((M, Bt.O), torch.int32, A.device)
    _check(lib().dabnn_tc_bgemm(A.data_ptr(), M, Bt.buf.data_ptr(), Bt.O, int(Kbits), out.data_ptr(), _stream()))
    return out


def tc_set_max_ctas(max_ctas: int) -> int:
    """dabnn_tc_set_max_ctas: cap the CTAs of a tensor-engine launch (0 = all SMs); returns the previous setting."""
    return int(lib().dabnn_tc_set_max_ctas(int(max_ctas)))


def tc_error_flag() -> int:
    return int(lib().dabnn_tc_error_flag())


def last_device_flag() -> int:
    """dabnn_last_device_flag on the current stream: synchronises it, returns the device's error flag and clears it."""
    return int(lib().dabnn_last_device_flag(_stream()))


def stream_status() -> int:
    """dabnn_stream_status on the current stream (0 = ok, ERR_TIMEOUT = a bounded wait inside a kernel ran out)."""
    return int(lib().dabnn_stream_status(_stream()))


def tc_wait_expiry_selftest(a_packed, wt: "TcWeights", stride=(1, 1), pad=(0, 0), pad_value: int = -1, wait_polls: int = 1000):
    """dabnn_tc_wait_expiry_selftest: a launch whose first wait can never be satisfied and gives up after `wait_polls`
    polls.  Returns the (undefined) output tensor."""
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    out = _alloc((N, OH, OW, wt.O), torch.int32, a.device)
    _check(lib().dabnn_tc_wait_expiry_selftest(a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O,
                                               _conv(wt.kh, wt.kw, stride, pad, pad_value), out.data_ptr(), int(wait_polls),
                                               _stream()))
    return out


class Prepared:
    """A library call with its arguments marshalled once (pointers and structs; the stream is torch's current one),
    for loops where the per-call Python overhead of the checked wrappers would rival the kernel time.
    The tensors passed at creation must stay alive and in place; `keep` holds references to them."""

    def __init__(self, fn, args, keep):
        self.fn, self.args, self.keep = fn, args, keep

    def __call__(self):
        st = self.fn(*self.args, torch.cuda.current_stream().cuda_stream)
        if st != 0:
            _check(st)


def prepare_pack(x: torch.Tensor, out: torch.Tensor, layout: int = NCHW) -> Prepared:
    x = _dev(x, torch.float32, "x")
    N, C, H, W = x.shape if layout == NCHW else (x.shape[0], x.shape[3], x.shape[1], x.shape[2])
    return Prepared(lib().dabnn_pack, (x.data_ptr(), layout, Shape(N, C, H, W), out.data_ptr()), (x, out))


def prepare_bconv2d(a_packed, C, w_packed, out, stride=(1, 1), pad=(0, 0), pad_value=-1, out_layout=NHWC) -> Prepared:
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    return Prepared(lib().dabnn_bconv2d, (a.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O,
                                          _conv(kh, kw, stride, pad, pad_value), out.data_ptr(), out_layout),
                    (a, w, out))


def prepare_bconv2d_bn_sign_pack(a_packed, C, w_packed, scale, shift, out, stride=(1, 1), pad=(0, 0),
                                 pad_value=-1) -> Prepared:
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    return Prepared(lib().dabnn_bconv2d_bn_sign_pack,
                    (a.data_ptr(), Shape(N, C, H, W), w.data_ptr(), O, _conv(kh, kw, stride, pad, pad_value),
                     scale.data_ptr(), shift.data_ptr(), out.data_ptr()), (a, w, scale, shift, out))


def prepare_tc_bconv2d(a_packed, wt: TcWeights, out, stride=(1, 1), pad=(0, 0), pad_value=-1, out_layout=NHWC) -> Prepared:
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    return Prepared(lib().dabnn_tc_bconv2d, (a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O,
                                             _conv(wt.kh, wt.kw, stride, pad, pad_value), out.data_ptr(), out_layout),
                    (a, wt, out))


def prepare_tc_bconv2d_bn_sign_pack(a_packed, wt: TcWeights, scale, shift, out, stride=(1, 1), pad=(0, 0),
                                    pad_value=-1) -> Prepared:
    a, N, H, W, OH, OW = _tc_geom(a_packed, wt, stride, pad)
    return Prepared(lib().dabnn_tc_bconv2d_bn_sign_pack,
                    (a.data_ptr(), Shape(N, wt.C, H, W), wt.buf.data_ptr(), wt.O, _conv(wt.kh, wt.kw, stride, pad, pad_value),
                     scale.data_ptr(), shift.data_ptr(), out.data_ptr()), (a, wt, scale, shift, out))


def prepare_bireal_block(a_packed, C, w_packed, wt: Optional[TcWeights], scale, shift, stream_fp32, stride=(1, 1), pad=(0, 0),
                         pad_value=-1) -> Prepared:
    """The Bi-Real block call as the network makes it: y = BN(conv) + residual written over the residual (`stream_fp32`,
    fp32 NHWC [N][OH][OW][O]) plus the packed signs; on the tensor-core engine when `wt` is given."""
    a, w, N, H, W, O, kh, kw, OH, OW = _geom(a_packed, C, w_packed, stride, pad)
    if tuple(stream_fp32.shape) != (N, OH, OW, O):
        raise DabnnError("the fp32 stream must be NHWC [N][OH][OW][O]")
    bits = _alloc((N, OH, OW, words_per_pixel(O)), torch.int64, a.device)
    fn = lib().dabnn_tc_bconv2d_bn_add_sign_pack if wt is not None else lib().dabnn_bconv2d_bn_add_sign_pack
    wptr = wt.buf.data_ptr() if wt is not None else w.data_ptr()
    return Prepared(fn, (a.data_ptr(), Shape(N, C, H, W), wptr, O, _conv(kh, kw, stride, pad, pad_value), scale.data_ptr(),
                         shift.data_ptr(), stream_fp32.data_ptr(), stream_fp32.data_ptr(), bits.data_ptr()),
                    (a, w, wt, scale, shift, stream_fp32, bits))


def set_conv_variant(variant: int) -> int:
    return int(lib().dabnn_set_conv_variant(int(variant)))


def set_conv_tile(tile: int) -> int:
    return int(lib().dabnn_set_conv_tile(int(tile)))
