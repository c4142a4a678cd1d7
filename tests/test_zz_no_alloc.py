"""The allocation-free Bi-Real Net 18 entry point (dabnn_bireal18_forward_static).

It exists for hosts of the library that are not allowed to allocate device memory themselves (for example a
plug-in running inside a server whose framework owns all of the GPU's memory): the activations between layers
go to a scratch area built into the library instead of a caller-provided workspace.  The checks below call it
through the C ABI and compare it with the ordinary entry point, twice in a row, because consecutive calls reuse
the same scratch area with the previous call's contents still in it.

This file is named so that pytest collects it last.
"""
import ctypes

import numpy as np
import pytest
import torch

from paper_1908_05858_b200 import synth


def test_requests_beyond_the_built_in_scratch_are_refused():
    """Needs no GPU: the size check comes before anything touches the device."""
    from paper_1908_05858_b200 import binding as B

    L = B.lib()
    fake = ctypes.c_void_p(0x1000)  # never dereferenced
    P = B.Bireal18Params()
    assert L.dabnn_bireal18_forward_static(ctypes.byref(P), fake, B.STATIC_MAX_BATCH + 1, fake, None) == B.ERR_STATIC_LIMIT
    assert b"built-in scratch" in L.dabnn_status_string(B.ERR_STATIC_LIMIT)
    assert L.dabnn_bireal18_forward_static(ctypes.byref(P), fake, 0, fake, None) == 2
    assert L.dabnn_bireal18_workspace_bytes(B.STATIC_MAX_BATCH) <= 8935424


@pytest.mark.gpu
def test_static_scratch_forward_equals_the_workspace_forward_twice_in_a_row():
    from paper_1908_05858_b200 import binding as B

    assert torch.cuda.is_available()
    net = B.Bireal18(synth.bireal18_params())
    img = torch.from_numpy(synth.bireal18_images(3)).cuda()
    want = net.forward(img).cpu().numpy()  # the existing entry point, caller-provided workspace
    scale = np.max(np.abs(want))
    # first call: two images; second call: a different, single image, on the scratch the first call left behind
    for sl in (slice(0, 2), slice(2, 3), slice(0, 2)):
        got = B.bireal18_forward_static(net, img[sl].contiguous()).cpu().numpy()
        assert np.max(np.abs(got - want[sl])) <= 1e-3 * scale
        assert np.array_equal(got.argmax(axis=1), want[sl].argmax(axis=1))
        assert np.array_equal(got, want[sl])  # same kernels, same order: identical bits
    with pytest.raises(B.DabnnError, match="built-in scratch"):
        B.bireal18_forward_static(net, img)  # three images: over the limit, refused
