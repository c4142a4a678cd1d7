"""The C-ABI library loads without a GPU, exports every symbol the header declares, and rejects bad
arguments before launching anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    from paper_1908_05858_b200 import build as b
    from paper_1908_05858_b200 import binding

    b.build()
    return binding.lib()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "dabnn.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dabnn_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(L):
    from paper_1908_05858_b200 import binding

    names = declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(L, n), n
    assert set(binding.EXPORTS) == set(names)


def test_helpers(L):
    assert L.dabnn_words_per_pixel(1) == 1 and L.dabnn_words_per_pixel(64) == 1 and L.dabnn_words_per_pixel(65) == 2
    assert L.dabnn_words_per_pixel(0) == 0
    assert L.dabnn_out_dim(56, 3, 1, 1) == 56 and L.dabnn_out_dim(56, 3, 2, 1) == 28 and L.dabnn_out_dim(7, 3, 2, 1) == 4
    assert L.dabnn_out_dim(2, 5, 1, 0) == 0
    assert L.dabnn_status_string(0) == b"ok"
    assert b"workspace" in L.dabnn_status_string(5)
    assert L.dabnn_bireal18_workspace_bytes(0) == 0
    per1 = L.dabnn_bireal18_workspace_bytes(1)
    assert per1 >= 112 * 112 * 64 * 4 + 56 * 56 * 64 * 4
    assert L.dabnn_bireal18_workspace_bytes(4) <= 4 * per1 + 4096


def test_argument_errors_are_reported_before_any_launch(L):
    from paper_1908_05858_b200.binding import Conv, Shape

    fake = ctypes.c_void_p(0x1000)  # never dereferenced: every call below fails validation first
    odd = ctypes.c_void_p(0x1004)
    s = Shape(1, 64, 4, 4)
    cv = Conv(3, 3, 1, 1, 1, 1, -1)
    assert L.dabnn_pack(None, 0, s, fake, None) == 1
    assert L.dabnn_pack(fake, 0, Shape(1, 0, 4, 4), fake, None) == 2
    assert L.dabnn_pack(fake, 7, s, fake, None) == 2
    assert L.dabnn_pack(fake, 0, s, odd, None) == 4
    assert L.dabnn_pack_weights(fake, 0, 64, 3, 3, fake, None) == 2
    assert L.dabnn_bconv2d(fake, s, None, 8, cv, fake, 1, None) == 1
    assert L.dabnn_bconv2d(fake, s, fake, 8, Conv(3, 3, 1, 1, 1, 1, 0), fake, 1, None) == 2   # pad_value not +-1
    assert L.dabnn_bconv2d(fake, s, fake, 8, Conv(3, 3, 0, 1, 1, 1, -1), fake, 1, None) == 2  # stride 0
    assert L.dabnn_bconv2d(fake, s, fake, 8, Conv(7, 7, 1, 1, 0, 0, -1), fake, 1, None) == 2  # empty output
    assert L.dabnn_bconv2d(odd, s, fake, 8, cv, fake, 1, None) == 4
    assert L.dabnn_bconv2d(fake, s, fake, 8, cv, fake, 5, None) == 2                           # bad layout
    assert L.dabnn_bconv2d_bn_sign_pack(fake, s, fake, 8, cv, None, fake, fake, None) == 1
    assert L.dabnn_bconv2d_bn_add_sign_pack(fake, s, fake, 8, cv, fake, fake, None, fake, fake, None) == 1
    assert L.dabnn_bn_fold(fake, fake, fake, fake, 1e-5, 0, fake, fake, None) == 2
    assert L.dabnn_bireal18_forward(None, fake, 1, fake, fake, 1 << 30, None) == 1
    assert L.dabnn_set_conv_variant(0) in (0, 1, 2)
    assert L.dabnn_pack_as(fake, 0, s, 2, fake, None) == 2            # unknown packed layout
    assert L.dabnn_pack_as(fake, 0, s, 1, ctypes.c_void_p(0x1008), None) == 4  # NC1HWC2 wants 16-byte aligned vectors
    assert L.dabnn_bconv2d_from(fake, 3, s, fake, 8, cv, fake, 1, None) == 2
    assert L.dabnn_packed_words(Shape(2, 130, 3, 4), 0) == 2 * 3 * 4 * 3 and L.dabnn_packed_words(Shape(2, 130, 3, 4), 1) == 2 * 3 * 4 * 4
    assert L.dabnn_packed_words(Shape(2, 130, 3, 4), 5) == 0
    assert L.dabnn_tc_wait_expiry_selftest(fake, Shape(1, 64, 8, 8), fake, 64, cv, None, 100, None) == 1
    assert L.dabnn_tc_wait_expiry_selftest(fake, Shape(1, 64, 8, 8), fake, 64, cv, fake, 0, None) == 2
    assert b"wait" in L.dabnn_status_string(7) and b"built-in scratch" in L.dabnn_status_string(8)


def test_binding_refuses_cpu_tensors():
    import torch

    from paper_1908_05858_b200 import binding

    with pytest.raises(binding.DabnnError):
        binding.pack(torch.zeros(1, 64, 4, 4))
