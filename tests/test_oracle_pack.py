"""Pins for the oracle's binarize + pack (Section 2.1.1), independent of the oracle itself."""
import numpy as np
import pytest


def unpack_words(P, C):
    """uint64 [..., Cw] -> {0,1} array [..., C] by shifting, written here independently."""
    Cw = P.shape[-1]
    bits = np.zeros(P.shape[:-1] + (Cw * 64,), dtype=np.uint8)
    for c in range(Cw * 64):
        bits[..., c] = ((P[..., c >> 6] >> np.uint64(c & 63)) & np.uint64(1)).astype(np.uint8)
    return bits[..., :C], bits[..., C:]


def test_hand_vectors(oracle_mod):
    o = oracle_mod
    C = 130  # three words, tail of 2 valid bits in the last
    def one(vals):
        x = np.asarray(vals, dtype=np.float32).reshape(1, C, 1, 1)
        return [int(v) for v in o.pack(x, o.NCHW).reshape(-1)]
    assert one([1.0] * C) == [0, 0, 0]
    assert one([-1.0] * C) == [0xFFFFFFFFFFFFFFFF, 0xFFFFFFFFFFFFFFFF, 0x3]
    alt = [(-1.0 if c % 2 else 1.0) for c in range(C)]  # odd channels negative
    assert one(alt) == [0xAAAAAAAAAAAAAAAA, 0xAAAAAAAAAAAAAAAA, 0x2]
    for c, want in ((0, [1, 0, 0]), (63, [1 << 63, 0, 0]), (64, [0, 1, 0]), (127, [0, 1 << 63, 0]),
                    (128, [0, 0, 1]), (129, [0, 0, 2])):
        v = [0.5] * C
        v[c] = -0.5
        assert one(v) == want, c


def test_special_floats(oracle_mod):
    o = oracle_mod
    neg_nan = np.frombuffer(np.uint32(0xFFC00000).tobytes(), dtype=np.float32)[0]
    pos_nan = np.frombuffer(np.uint32(0x7FC00000).tobytes(), dtype=np.float32)[0]
    vals = [0.0, -0.0, 1e-45, -1e-45, np.inf, -np.inf, pos_nan, neg_nan, 1.17549435e-38, -1.17549435e-38]
    want = [0, 0, 0, 1, 0, 1, 0, 0, 0, 1]  # only values that compare below zero give bit 1
    x = np.asarray(vals, dtype=np.float32).reshape(1, len(vals), 1, 1)
    word = int(o.pack(x, o.NCHW).reshape(-1)[0])
    assert [(word >> i) & 1 for i in range(len(vals))] == want


@pytest.mark.parametrize("shape", [(2, 70, 5, 7), (1, 64, 3, 3), (3, 1, 2, 2), (1, 200, 4, 1)])
def test_unpack_matches_comparison(oracle_mod, shape):
    o = oracle_mod
    rng = np.random.default_rng(11)
    x = rng.standard_normal(shape).astype(np.float32)
    x[rng.random(shape) < 0.05] = 0.0
    P = o.pack(x, o.NCHW)
    N, C, H, W = shape
    assert P.shape == (N, H, W, (C + 63) // 64) and P.dtype == np.uint64
    bits, tail = unpack_words(P, C)
    assert np.array_equal(bits, (np.transpose(x, (0, 2, 3, 1)) < 0).astype(np.uint8))
    assert not tail.any()  # tail bits are zero
    # NHWC input gives the same words
    P2 = o.pack(np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1))), o.NHWC)
    assert np.array_equal(P, P2)


def test_int32_sign_bits(oracle_mod):
    """int32 input: the packed bit is the integer's sign bit (two's complement top bit), independently extracted here."""
    o = oracle_mod
    vals = [0, 1, -1, 2**31 - 1, -2**31, 5, -5, 7]
    x = np.asarray(vals, dtype=np.int32).reshape(1, len(vals), 1, 1)
    word = int(o.pack_i32(x, o.NCHW).reshape(-1)[0])
    assert [(word >> i) & 1 for i in range(len(vals))] == [0, 0, 1, 0, 1, 0, 1, 0]
    rng = np.random.default_rng(5)
    shape = (2, 130, 3, 5)
    x = rng.integers(-2**31, 2**31, size=shape, dtype=np.int64).astype(np.int32)
    x[rng.random(shape) < 0.1] = 0
    P = o.pack_i32(x, o.NCHW)
    bits, tail = unpack_words(P, shape[1])
    top_bit = (np.transpose(x, (0, 2, 3, 1)).view(np.uint32) >> np.uint32(31)).astype(np.uint8)
    assert np.array_equal(bits, top_bit) and not tail.any()
    assert np.array_equal(P, o.pack_i32(np.ascontiguousarray(np.transpose(x, (0, 2, 3, 1))), o.NHWC))
    # where floats represent the integers exactly (|x| < 2^24) both packers agree
    small = rng.integers(-1000, 1000, size=shape).astype(np.int32)
    assert np.array_equal(o.pack_i32(small, o.NCHW), o.pack(small.astype(np.float32), o.NCHW))


def test_size_is_32x_smaller(oracle_mod):
    # one bit per fp32 element (Section 3: packed weights are 32x smaller)
    o = oracle_mod
    x = np.ones((2, 256, 4, 4), dtype=np.float32)
    assert o.pack(x).nbytes * 32 == x.nbytes
    w = np.ones((8, 128, 3, 3), dtype=np.float32)
    assert o.pack_weights(w).nbytes * 32 == w.nbytes


def test_pack_weights_layout(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(5)
    w = rng.standard_normal((5, 70, 3, 2)).astype(np.float32)
    Wp = o.pack_weights(w)
    assert Wp.shape == (5, 3, 2, 2)
    bits, tail = unpack_words(Wp, 70)
    assert np.array_equal(bits, (np.transpose(w, (0, 2, 3, 1)) < 0).astype(np.uint8))
    assert not tail.any()


def test_nc1hwc2_layout_places_every_channel_bit(oracle_mod):
    """The NC1HWC2 layout (Section 2.1.2, last paragraph; C2 = 128 bits): channel c is bit c&63 of word (c>>6)&1 of the
    128-bit vector of group c>>7, one vector per pixel and group.  Checked by unpacking every bit independently."""
    o = oracle_mod
    rng = np.random.default_rng(21)
    for shape in ((2, 300, 3, 5), (1, 64, 4, 4), (3, 128, 2, 3), (1, 130, 1, 2)):
        N, C, H, W = shape
        x = rng.standard_normal(shape).astype(np.float32)
        x.reshape(-1)[:4] = [0.0, -0.0, np.nan, -1e-45]
        P = o.pack_c2(x, o.NCHW)
        C1 = (C + 127) // 128
        assert P.shape == (N, C1, H, W, 2) and P.dtype == np.uint64
        bits = np.zeros((N, C1 * 128, H, W), dtype=np.uint8)
        for g in range(C1):
            for j in range(2):
                for b in range(64):
                    bits[:, 128 * g + 64 * j + b] = ((P[:, g, :, :, j] >> np.uint64(b)) & np.uint64(1)).astype(np.uint8)
        assert np.array_equal(bits[:, :C], (x < 0).astype(np.uint8))
        assert not bits[:, C:].any()  # tail bits, and the zero partner word of an odd last group
        # the NHWC-input form packs the same bits
        assert np.array_equal(o.pack_c2(np.ascontiguousarray(x.transpose(0, 2, 3, 1)), o.NHWC), P)
        # and the two packed layouts hold the same words, rearranged
        Q = o.pack(x, o.NCHW)  # [N][H][W][Cw]
        for cw in range(Q.shape[-1]):
            assert np.array_equal(P[:, cw >> 1, :, :, cw & 1], Q[..., cw])


def test_nc1hwc2_hand_vector(oracle_mod):
    x = -np.ones((1, 130, 1, 1), dtype=np.float32)
    P = oracle_mod.pack_c2(x)
    assert P.reshape(-1).tolist() == [2**64 - 1, 2**64 - 1, 3, 0]
