"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded
inputs.  Integer and bit results must be identical; fp32 results of the Bi-Real path are produced by
the same IEEE operations in the same order on both sides, so they are compared bit for bit as well,
and the logits additionally within the stated tolerance (max-abs 1e-3 of the logit scale, same argmax)."""
import numpy as np
import pytest
import torch

from paper_1908_05858_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_1908_05858_b200 import binding

    assert torch.cuda.is_available(), "the parity tests need a CUDA device"
    binding.lib()  # raises if the CUDA library is missing: no fallback
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def u64(t):
    return t.cpu().numpy().view(np.uint64)


# ---- pack ---------------------------------------------------------------------------------------------
PACK_SHAPES = [
    (2, 64, 14, 14),    # vector path, one word
    (3, 256, 56, 56),   # vector path, four warps per pixel group, ragged last tile (3136 = 24.5 * 128)
    (2, 128, 28, 28),   # vector path, two words
    (1, 192, 12, 12),   # three words
    (2, 70, 7, 5),      # generic path (H*W not a multiple of 4), channel tail
    (1, 1, 1, 1),
    (1, 1000, 2, 2),    # 16 words, tail of 40 bits
    (5, 3, 224, 8),
    (4, 512, 7, 7),     # tile path: H*W = 49
    (2, 100, 15, 13),   # tile path, two pixel tiles, channel tail
    (1, 2100, 3, 3),    # more than 32 words: generic path
]


@pytest.mark.parametrize("shape", PACK_SHAPES)
def test_pack_nchw(B, oracle_mod, shape):
    rng = np.random.default_rng(sum(shape))
    x = rng.standard_normal(shape).astype(np.float32)
    x[rng.random(shape) < 0.01] = 0.0
    flat = x.reshape(-1)
    flat[:6] = [0.0, -0.0, np.nan, -np.inf, 1e-45, -1e-45][: min(6, flat.size)]
    got = u64(B.pack(dev(x), B.NCHW))
    assert np.array_equal(got, oracle_mod.pack(x, oracle_mod.NCHW))


@pytest.mark.parametrize("shape", [(2, 14, 14, 64), (3, 9, 7, 256), (2, 5, 5, 70), (1, 3, 3, 4), (4, 31, 17, 128)])
def test_pack_nhwc(B, oracle_mod, shape):
    rng = np.random.default_rng(sum(shape) + 1)
    x = rng.standard_normal(shape).astype(np.float32)
    x[rng.random(shape) < 0.02] = -0.0
    got = u64(B.pack(dev(x), B.NHWC))
    assert np.array_equal(got, oracle_mod.pack(x, oracle_mod.NHWC))


@pytest.mark.parametrize("shape", PACK_SHAPES)
def test_pack_i32_nchw(B, oracle_mod, shape):
    rng = np.random.default_rng(sum(shape) + 2)
    x = rng.integers(-2**31, 2**31, size=shape, dtype=np.int64).astype(np.int32)
    x[rng.random(shape) < 0.05] = 0
    got = u64(B.pack_i32(dev(x), B.NCHW))
    assert np.array_equal(got, oracle_mod.pack_i32(x, oracle_mod.NCHW))


@pytest.mark.parametrize("shape", [(2, 14, 14, 64), (3, 9, 7, 256), (2, 5, 5, 70), (4, 31, 17, 128)])
def test_pack_i32_nhwc(B, oracle_mod, shape):
    rng = np.random.default_rng(sum(shape) + 3)
    x = rng.integers(-50, 50, size=shape).astype(np.int32)
    got = u64(B.pack_i32(dev(x), B.NHWC))
    assert np.array_equal(got, oracle_mod.pack_i32(x, oracle_mod.NHWC))


def test_pack_i32_of_conv_sums_equals_fused_sign(B, oracle_mod):
    """Binarizing a convolution's int32 sums with the int32 packer = the fused epilogue with scale 1, shift 0."""
    x, w = synth.conv_case(1, 2, 128, 9, 11, 128, 3, 3)
    a = B.pack(dev(x))
    wp = B.pack_weights(dev(w))
    sums = B.bconv2d(a, 128, wp, (1, 1), (1, 1), -1, B.NHWC)
    ones = torch.ones(128, device=a.device)
    fused = B.bconv2d_bn_sign_pack(a, 128, wp, ones, torch.zeros_like(ones), (1, 1), (1, 1), -1)
    assert np.array_equal(u64(B.pack_i32(sums, B.NHWC)), u64(fused))


def test_pack_unaligned_input_takes_the_generic_path(B, oracle_mod):
    rng = np.random.default_rng(8)
    buf = rng.standard_normal(1 + 2 * 64 * 8 * 8).astype(np.float32)
    d = dev(buf)
    x = d[1:].view(2, 64, 8, 8)  # 4-byte aligned only
    got = u64(B.pack(x, B.NCHW))
    assert np.array_equal(got, oracle_mod.pack(buf[1:].reshape(2, 64, 8, 8)))


@pytest.mark.parametrize("shape", [(64, 64, 3, 3), (9, 70, 3, 3), (2048, 512, 1, 1), (5, 130, 5, 2)])
def test_pack_weights(B, oracle_mod, shape):
    w = np.random.default_rng(shape[0]).standard_normal(shape).astype(np.float32)
    assert np.array_equal(u64(B.pack_weights(dev(w))), oracle_mod.pack_weights(w))


# ---- binary convolution ---------------------------------------------------------------------------------
CONV_CASES = [
    # N, C, H, W, O, kh, kw, stride, pad, pad_value
    (1, 64, 14, 14, 64, 3, 3, (1, 1), (1, 1), -1),      # BASELINE config 1
    (2, 70, 7, 5, 9, 3, 3, (1, 1), (1, 1), -1),         # channel tail, tiny O
    (2, 70, 7, 5, 9, 3, 3, (1, 1), (1, 1), +1),
    (1, 130, 9, 8, 37, 3, 3, (2, 2), (1, 1), -1),       # three words (8-byte copy units), stride 2
    (3, 128, 13, 11, 100, 3, 3, (1, 1), (1, 1), -1),    # 16-byte copy units, ragged pixel and channel tiles
    (1, 3, 12, 12, 5, 5, 5, (1, 2), (2, 2), -1),
    (2, 128, 6, 6, 130, 1, 1, (1, 1), (0, 0), -1),      # 1x1
    (1, 17, 6, 7, 3, 2, 3, (2, 1), (0, 1), +1),
    (1, 256, 14, 14, 256, 3, 3, (1, 1), (1, 1), -1),    # several K chunks
    (1, 512, 7, 7, 512, 3, 3, (1, 1), (1, 1), -1),      # K = 4608 bits, 5 chunks
    (1, 64, 56, 56, 64, 3, 3, (1, 1), (1, 1), -1),
    (4, 64, 30, 30, 128, 7, 7, (2, 2), (3, 3), -1),     # 49 taps
    (40, 192, 20, 20, 192, 3, 3, (1, 1), (1, 1), -1),   # large enough for the 128x128 tile
    (130, 192, 13, 13, 1000, 1, 1, (1, 1), (0, 0), -1),  # 1x1, enough tiles for the several-tiles-per-CTA form; odd word count,
    (131, 128, 13, 13, 1000, 1, 1, (1, 1), (0, 0), +1),  # ragged last CTA (173 pixel tiles), ragged channel tile; 16-byte units
]


def conv_inputs(case):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    rng = np.random.default_rng(abs(hash(case)) % (2**32))
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, kh, kw)).astype(np.float32)
    return x, w


@pytest.mark.parametrize("variant", [1, 2])
@pytest.mark.parametrize("case", CONV_CASES)
def test_bconv2d_matches_oracle(B, oracle_mod, case, variant):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    o = oracle_mod
    want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), stride, pad, pv, o.NHWC)
    prev = B.set_conv_variant(variant)
    try:
        a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
        got = B.bconv2d(a, C, wp, stride, pad, pv, B.NHWC).cpu().numpy()
        got_nchw = B.bconv2d(a, C, wp, stride, pad, pv, B.NCHW).cpu().numpy()
        again = B.bconv2d(a, C, wp, stride, pad, pv, B.NHWC).cpu().numpy()
    finally:
        B.set_conv_variant(prev)
    assert np.array_equal(got, want)
    assert np.array_equal(got_nchw, np.transpose(want, (0, 3, 1, 2)))
    assert np.array_equal(again, got)  # a second run gives the same bits (no race)
    if N * O * want.shape[1] * want.shape[2] * C * kh * kw < 3e8:  # the definition itself, where it is quick
        assert np.array_equal(want, o.bconv_pm1(x, w, stride, pad, pv, o.NHWC))


@pytest.mark.parametrize("case", CONV_CASES)
def test_fused_bn_sign_pack_matches_oracle(B, oracle_mod, case):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    o = oracle_mod
    rng = np.random.default_rng(O)
    gamma, beta, mean, var = synth.bn_params(rng, O)
    gamma[::5] *= -1.0
    mean *= 30.0  # thresholds spread over the range of the integer results
    scale_o, shift_o = o.bn_fold(gamma, beta, mean, var)
    scale_g, shift_g = B.bn_fold(dev(gamma), dev(beta), dev(mean), dev(var))
    assert np.array_equal(scale_g.cpu().numpy().view(np.uint32), scale_o.view(np.uint32))
    assert np.array_equal(shift_g.cpu().numpy().view(np.uint32), shift_o.view(np.uint32))
    acc = o.bconv_bits(o.pack(x), C, o.pack_weights(w), stride, pad, pv, o.NHWC)
    want = o.bn_sign_pack(acc, scale_o, shift_o)
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    got = u64(B.bconv2d_bn_sign_pack(a, C, wp, scale_g, shift_g, stride, pad, pv))
    assert np.array_equal(got, want)
    assert 0 < np.count_nonzero(got) < got.size * 64 or O < 4


@pytest.mark.parametrize("case", [CONV_CASES[0], CONV_CASES[3], CONV_CASES[4], CONV_CASES[8], CONV_CASES[12]])
def test_bireal_block_epilogue_matches_oracle(B, oracle_mod, case):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    o = oracle_mod
    rng = np.random.default_rng(O + 1)
    scale_o, shift_o = o.bn_fold(*synth.bn_params(rng, O))
    acc = o.bconv_bits(o.pack(x), C, o.pack_weights(w), stride, pad, pv, o.NHWC)
    res = rng.standard_normal(acc.shape).astype(np.float32) * 20
    y, want_bits = o.bn_add_sign_pack(acc, scale_o, shift_o, res)  # one fmaf, one rounded add, sign, pack
    assert np.array_equal(want_bits, o.pack(y, o.NHWC))
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    got_y, got_bits = B.bconv2d_bn_add_sign_pack(a, C, wp, dev(scale_o), dev(shift_o), dev(res), stride, pad, pv)
    assert np.array_equal(got_y.cpu().numpy().view(np.uint32), y.view(np.uint32))
    assert np.array_equal(u64(got_bits), want_bits)


# ---- the paper's NC1HWC2 activation layout (Section 2.1.2, last paragraph) ---------------------------------------------
@pytest.mark.parametrize("shape", [(2, 256, 28, 28), (3, 64, 7, 5), (2, 130, 9, 8), (1, 300, 12, 12), (2, 128, 6, 7), (1, 2100, 3, 3)])
def test_pack_nc1hwc2(B, oracle_mod, shape):
    rng = np.random.default_rng(sum(shape) + 4)
    x = rng.standard_normal(shape).astype(np.float32)
    x[rng.random(shape) < 0.01] = 0.0
    got = u64(B.pack_as(dev(x), B.PACKED_NC1HWC2))
    assert np.array_equal(got, oracle_mod.pack_c2(x))
    xt = np.ascontiguousarray(x.transpose(0, 2, 3, 1))
    assert np.array_equal(u64(B.pack_as(dev(xt), B.PACKED_NC1HWC2, B.NHWC)), oracle_mod.pack_c2(x))
    assert np.array_equal(u64(B.pack_as(dev(x), B.PACKED_NHWC)), oracle_mod.pack(x))


@pytest.mark.parametrize("case", [CONV_CASES[0], CONV_CASES[1], CONV_CASES[3], CONV_CASES[4], CONV_CASES[8], CONV_CASES[9],
                                  CONV_CASES[11], CONV_CASES[12], (2, 300, 10, 9, 40, 3, 3, (1, 1), (1, 1), +1)])
def test_bconv2d_from_nc1hwc2_matches_oracle(B, oracle_mod, case):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    o = oracle_mod
    want = o.bconv_bits_c2(o.pack_c2(x), C, o.pack_weights(w), stride, pad, pv, o.NHWC)
    a2, wp = B.pack_as(dev(x), B.PACKED_NC1HWC2), B.pack_weights(dev(w))
    got = B.bconv2d_from(a2, B.PACKED_NC1HWC2, C, wp, stride, pad, pv, B.NHWC).cpu().numpy()
    assert np.array_equal(got, want)
    assert np.array_equal(B.bconv2d_from(a2, B.PACKED_NC1HWC2, C, wp, stride, pad, pv, B.NCHW).cpu().numpy(), want.transpose(0, 3, 1, 2))
    # the same integers from the channel-packed NHWC words
    assert np.array_equal(B.bconv2d_from(B.pack(dev(x)), B.PACKED_NHWC, C, wp, stride, pad, pv, B.NHWC).cpu().numpy(), want)


def test_nc1hwc2_full_size_3x3_layer(B, oracle_mod):
    """The large-batch 3x3 layer (batch 256, 256 channels, 28x28) from NC1HWC2 activations: the whole tensor against Eq. 1."""
    x, w = synth.conv_case(5, 256, 256, 28, 28, 256, 3, 3, salt=256)
    a2, wp = B.pack_as(dev(x), B.PACKED_NC1HWC2), B.pack_weights(dev(w))
    assert np.array_equal(u64(a2), oracle_mod.pack_c2(x))
    got = B.bconv2d_from(a2, B.PACKED_NC1HWC2, 256, wp, (1, 1), (1, 1), -1, B.NHWC).cpu().numpy()
    want = oracle_mod.bconv_bits(oracle_mod.pack(x), 256, oracle_mod.pack_weights(w), (1, 1), (1, 1), -1, oracle_mod.NHWC)
    assert np.array_equal(got, want)


# ---- full-size configurations, sampled ---------------------------------------------------------------------
def sample_coords(rng, N, O, OH, OW, n):
    c = np.stack([rng.integers(0, N, n), rng.integers(0, O, n), rng.integers(0, OH, n), rng.integers(0, OW, n)], axis=1)
    # always include the corners and edges, where padding matters
    fixed = [(0, 0, 0, 0), (N - 1, O - 1, OH - 1, OW - 1), (N - 1, 0, 0, OW - 1), (0, O - 1, OH - 1, 0), (N // 2, O // 2, 0, OW // 2)]
    return np.concatenate([np.array(fixed), c]).astype(np.int32)


def full_size_bn(C, N, O, K):
    """Per-channel (scale, shift) whose thresholds spread over the attainable sums (standard deviation sqrt(K))."""
    rng = np.random.default_rng(C + N + 1)
    scale = rng.uniform(0.5, 1.5, O).astype(np.float32)
    scale[::7] *= -1.0
    return scale, rng.normal(0, 0.3 * np.sqrt(K), O).astype(np.float32)


FULL = [(64, C, HW, C, 3, 1) for C, HW in synth.SWEEP_SHAPES] + [(256, 256, 28, 256, 3, 1), (256, 512, 14, 2048, 1, 0)]


@pytest.mark.parametrize("cfg", FULL)
def test_full_size_configs_on_sampled_outputs(B, oracle_mod, cfg):
    N, C, HW, O, k, pad = cfg
    x, w = synth.conv_case(2 if N == 64 else 5, N, C, HW, HW, O, k, k, salt=C)
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    got = B.bconv2d(a, C, wp, (1, 1), (pad, pad), -1, B.NHWC)
    K = C * k * k
    # properties that hold for every output
    assert int(got.min()) >= -K and int(got.max()) <= K
    assert bool(((got - K) % 2 == 0).all())
    g = got.cpu().numpy()
    rng = np.random.default_rng(C + N)
    coords = sample_coords(rng, N, O, HW, HW, 100000)
    want = oracle_mod.bconv_pm1_at(x, w, coords, (1, 1), (pad, pad), -1)  # the definition, output by output
    assert np.array_equal(g[coords[:, 0], coords[:, 2], coords[:, 3], coords[:, 1]], want)
    # packed operands too, bit for bit
    ao, wo = oracle_mod.pack(x), oracle_mod.pack_weights(w)
    assert np.array_equal(u64(a), ao)
    # the whole tensor against Eq. 1 on the packed words
    full = oracle_mod.bconv_bits(ao, C, wo, (1, 1), (pad, pad), -1, oracle_mod.NHWC)
    assert np.array_equal(g, full)
    del g
    # and the whole packed output of the fused BN + sign + pack epilogue
    scale, shift = full_size_bn(C, N, O, K)
    bits = B.bconv2d_bn_sign_pack(a, C, wp, dev(scale), dev(shift), (1, 1), (pad, pad), -1)
    assert np.array_equal(u64(bits), oracle_mod.bn_sign_pack(full, scale, shift))


def test_full_size_pack_config(B, oracle_mod):
    x = synth.pack_case(N=128, C=256, H=56, W=56)
    assert abs(float((x == 0).mean()) - 0.01) < 1e-3
    got = u64(B.pack(dev(x)))
    assert got.shape == (128, 56, 56, 4)
    assert np.array_equal(got, oracle_mod.pack(x))


# ---- Bi-Real Net 18 ---------------------------------------------------------------------------------------------
def test_bireal18_forward_matches_oracle(B, oracle_mod):
    p = synth.bireal18_params()
    img = synth.bireal18_images(3)
    want, taps = oracle_mod.bireal18_forward(p, img, conv_form=1, want_taps=True)
    net = B.Bireal18(p)
    got = net.forward(dev(img)).cpu().numpy()
    # the integer-pipe engine alone gives the same bits as the mixed (tensor-core where covered) network
    assert np.array_equal(B.Bireal18(p, engine="popc").forward(dev(img)).cpu().numpy(), got)
    assert sum(1 for b in range(16) if net.P.block_w_tc[b]) == 16 and B.tc_error_flag() == 0
    scale = np.max(np.abs(want))
    assert np.max(np.abs(got - want)) <= 1e-3 * scale
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))
    # the pinned evaluation order makes the two sides agree to the last bit
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # batch 1 gives the same logits for the same image
    got1 = net.forward(dev(img[:1])).cpu().numpy()
    assert np.array_equal(got1, got[:1])


@pytest.mark.parametrize("tile", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("case", [CONV_CASES[1], CONV_CASES[4], CONV_CASES[9],
                                  (1, 640, 6, 5, 40, 3, 3, (1, 1), (1, 1), -1)])  # 90 words of K: every ring wraps
def test_every_conv_tile_gives_the_same_integers(B, oracle_mod, case, tile):
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    o = oracle_mod
    want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), stride, pad, pv, o.NHWC)
    scale_o, shift_o = o.bn_fold(*synth.bn_params(np.random.default_rng(tile), O))
    want_bits = o.bn_sign_pack(want, scale_o, shift_o)
    prev = B.set_conv_tile(tile)
    try:
        a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
        got = B.bconv2d(a, C, wp, stride, pad, pv, B.NHWC).cpu().numpy()
        got_bits = u64(B.bconv2d_bn_sign_pack(a, C, wp, dev(scale_o), dev(shift_o), stride, pad, pv))
    finally:
        B.set_conv_tile(prev)
    assert np.array_equal(got, want)
    assert np.array_equal(got_bits, want_bits)


@pytest.mark.parametrize("shape", [(5, 7, 150), (300, 260, 512), (1, 1000, 4608), (129, 65, 64)])
def test_bgemm_matches_eq1(B, oracle_mod, shape):
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    A = B.pack(dev(a.reshape(M, K, 1, 1))).reshape(M, -1)
    Bm = B.pack(dev(b.reshape(N, K, 1, 1))).reshape(N, -1)
    got = B.bgemm(A, Bm, K).cpu().numpy()
    counts = oracle_mod.bgemm_xnor(u64(A), u64(Bm), K)  # Eq. 1 as printed: agreeing positions
    assert np.array_equal(got, 2 * counts - K)


def test_bireal18_four_and_five_images_match_oracle(B, oracle_mod):
    """Four images take the chained launches, the 16x32 convolution tile and the pooling + fc kernel; five take the
    ordinary stream order and the staged fc kernel.  Both must equal the oracle bit for bit, eagerly and as a CUDA graph."""
    p = synth.bireal18_params()
    img = synth.bireal18_images(5)
    want = oracle_mod.bireal18_forward(p, img, conv_form=1)
    net = B.Bireal18(p)
    x5, x4 = dev(img), dev(img[:4])
    got5 = net.forward(x5).cpu().numpy()
    got4 = net.forward(x4).cpu().numpy()
    assert np.array_equal(got5.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(got4.view(np.uint32), want[:4].view(np.uint32))
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        net.forward(x4)
        side.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            out = net.forward(x4)
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    assert np.array_equal(out.cpu().numpy().view(np.uint32), want[:4].view(np.uint32))


def test_bireal18_stem_weights_at_an_unaligned_address(B):
    """The small stem copies its weights with 16-byte asynchronous copies when it can and element by element when the
    caller's array is only 4-byte aligned; both give the same logits."""
    p = synth.bireal18_params()
    img = synth.bireal18_images(2)
    net = B.Bireal18(p)
    want2 = net.forward(dev(img)).cpu().numpy()
    want1 = net.forward(dev(img[:1])).cpu().numpy()
    flat = net.stem_w.flatten()
    shifted = torch.empty(flat.numel() + 1, dtype=torch.float32, device=flat.device)
    shifted[1:].copy_(flat)
    assert shifted[1:].data_ptr() % 16 == 4
    net.P.stem_w = shifted[1:].data_ptr()
    got2 = net.forward(dev(img)).cpu().numpy()
    got1 = net.forward(dev(img[:1])).cpu().numpy()
    assert np.array_equal(got2.view(np.uint32), want2.view(np.uint32))
    assert np.array_equal(got1.view(np.uint32), want1.view(np.uint32))


def test_bireal18_shortcut_and_block_weights_at_unaligned_addresses(B):
    """The small-batch shortcut kernel with staged weight rows wants 16-byte aligned 1x1 weights, and the convolution's
    16-byte copies 16-byte aligned packed weights; arrays that are only 4- / 8-byte aligned take the other kernels and
    copy units and must give the same logits."""
    p = synth.bireal18_params()
    img = dev(synth.bireal18_images(2))
    net = B.Bireal18(p, engine="popc")
    want = net.forward(img).cpu().numpy()
    keep = []
    for d in range(3):
        n = int(np.prod(p["down_w"][d].shape))
        src = torch.from_numpy(np.ascontiguousarray(p["down_w"][d], dtype=np.float32)).flatten().to(img.device)
        buf = torch.empty(n + 1, dtype=torch.float32, device=img.device)
        buf[1:].copy_(src)
        keep.append(buf)
        net.P.down_w[d] = buf[1:].data_ptr()
    for b in range(16):
        wp = B.pack_weights(dev(p["block_w"][b])).flatten()
        buf = torch.empty(wp.numel() + 1, dtype=torch.int64, device=img.device)
        buf[1:].copy_(wp)
        assert buf[1:].data_ptr() % 16 == 8
        keep.append(buf)
        net.P.block_w[b] = buf[1:].data_ptr()
    got = net.forward(img).cpu().numpy()
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))


def test_forward_and_convolution_from_two_host_threads(B):
    """A batch-1 forward (chained launches, a per-thread setting inside the library) on one host thread and stream while
    another thread launches plain convolutions on its own stream: both keep giving their single-threaded results."""
    import threading
    p = synth.bireal18_params()
    net = B.Bireal18(p, engine="popc")
    img = dev(synth.bireal18_images(1))
    want_logits = net.forward(img).cpu().numpy()
    case = CONV_CASES[8]
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    x, w = conv_inputs(case)
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    want_conv = B.bconv2d(a, C, wp, stride, pad, pv, B.NHWC).cpu().numpy()
    torch.cuda.synchronize()
    errors = []

    def forwards():
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                for _ in range(40):
                    got = net.forward(img)
                s.synchronize()
                if not np.array_equal(got.cpu().numpy().view(np.uint32), want_logits.view(np.uint32)):
                    errors.append("logits differ")
        except Exception as e:  # noqa: BLE001
            errors.append(repr(e))

    def convs():
        try:
            s = torch.cuda.Stream()
            with torch.cuda.stream(s):
                for _ in range(200):
                    got = B.bconv2d(a, C, wp, stride, pad, pv, B.NHWC)
                s.synchronize()
                if not np.array_equal(got.cpu().numpy(), want_conv):
                    errors.append("convolution differs")
        except Exception as e:  # noqa: BLE001
            errors.append(repr(e))

    threads = [threading.Thread(target=forwards), threading.Thread(target=convs)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert errors == []


def test_bireal18_large_batch_kernels_match_oracle(B, oracle_mod):
    """Batch 8 is large enough for the persistent 8x8-tile stem, the tiled shortcut kernel and the tensor-core engine
    on the early stages; the logits must still equal the oracle's bit for bit."""
    p = synth.bireal18_params()
    img = synth.bireal18_images(8)
    want = oracle_mod.bireal18_forward(p, img, conv_form=1)
    got = B.Bireal18(p).forward(dev(img)).cpu().numpy()
    assert np.max(np.abs(got - want)) <= 1e-3 * np.max(np.abs(want))
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert B.tc_error_flag() == 0


def test_bireal18_batch72_all_blocks_on_the_tensor_engine(B, oracle_mod):
    """At batch 72 every binary block runs on the tensor-core engine (CTA pairs in the last stage, stride-2 planes in the
    three downsampling blocks, the second epilogue group) and the head uses the batched fc kernel with a ragged last
    group of images; logits bit for bit against the oracle."""
    p = synth.bireal18_params()
    img = synth.bireal18_images(72)
    want = oracle_mod.bireal18_forward(p, img, conv_form=1)
    net = B.Bireal18(p)
    got = net.forward(dev(img)).cpu().numpy()
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the same images through the integer-pipe engine only
    got_p = B.Bireal18(p, engine="popc").forward(dev(img)).cpu().numpy()
    assert np.array_equal(got_p.view(np.uint32), want.view(np.uint32))
    assert B.tc_error_flag() == 0


def test_bireal18_batch128_matches_oracle(B, oracle_mod):
    """The network configuration as stated (batch 128), in the launch configuration the benchmark times: logits against
    the oracle within the stated tolerance, same argmax, and (pinned evaluation order) the same bits."""
    p = synth.bireal18_params()
    img = synth.bireal18_images(128)
    want = oracle_mod.bireal18_forward(p, img, conv_form=1)
    net = B.Bireal18(p)
    logits = torch.empty((128, 1000), dtype=torch.float32, device="cuda")
    got = net.forward(dev(img), logits).cpu().numpy()
    assert np.max(np.abs(got - want)) <= 1e-3 * np.max(np.abs(want))
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    assert np.array_equal(got[:1], net.forward(dev(img[:1])).cpu().numpy())  # and batch 1 of the same configuration
    assert B.last_device_flag() == 0


@pytest.mark.parametrize("N", [1, 3, 9, 72])
def test_bireal18_with_stem_module_matches_oracle(B, oracle_mod, N):
    """The STEM module variant (Section 2.3; the module's structure is a reading of the missing figure, so this pins the
    CUDA path to the oracle's reading, not to the paper): logits bit for bit, at batch sizes that take the chained
    launches (1, 3), the ordinary order (9) and the tensor-core engine on every block (72)."""
    p = dict(synth.bireal18_params())
    p["stem_module"] = synth.stem_module_params()
    img = synth.bireal18_images(N)
    want = oracle_mod.bireal18_forward(p, img, conv_form=1, stem_module=True)
    net = B.Bireal18(p)
    got = B.bireal18_forward_stem_module(net, dev(img)).cpu().numpy()
    assert np.max(np.abs(got - want)) <= 1e-3 * np.max(np.abs(want))
    assert np.array_equal(got.argmax(axis=1), want.argmax(axis=1))
    assert np.array_equal(got.view(np.uint32), want.view(np.uint32))
    # the 7x7 variant of the same object still gives its own logits
    assert np.array_equal(net.forward(dev(img[:1])).cpu().numpy().view(np.uint32),
                          oracle_mod.bireal18_forward(p, img[:1], conv_form=1).view(np.uint32))
    assert B.last_device_flag() == 0


def test_guard_bytes_catch_a_write_past_an_output(B, guard_outputs):
    """The guarded allocator the GPU tests run under does notice an out-of-bounds write (made here with torch, on
    purpose, one byte past an output)."""
    t = B.pack(torch.zeros((1, 64, 2, 2), device="cuda"))
    raw = guard_outputs.live[-1][0]
    assert raw.numel() == 2 * 256 + t.numel() * 8
    raw[256 + t.numel() * 8] = 0
    with pytest.raises(AssertionError, match="after an output"):
        guard_outputs.check()
    assert guard_outputs.check() == 0


@pytest.mark.parametrize("N,pinned", [(1, True), (3, True), (5, False), (9, True)])
def test_binary_layer_host_matches_oracle(B, oracle_mod, N, pinned):
    """The host-buffer entry point (chunked, copies on side streams): int32 sums and fused sign words against the oracle,
    called twice in a row on the same workspace with different inputs, results read after one stream synchronisation."""
    o = oracle_mod
    C, H, W, O = 128, 9, 11, 70
    rng = np.random.default_rng(N)
    w = rng.standard_normal((O, C, 3, 3)).astype(np.float32)
    scale_np, shift_np = rng.uniform(0.5, 1.5, O).astype(np.float32), rng.normal(0, 5, O).astype(np.float32)
    wp = B.pack_weights(dev(w))
    scale, shift = dev(scale_np), dev(shift_np)
    ws = torch.empty(B.binary_layer_host_workspace_bytes(N, C, H, W, O, 3, 3, (1, 1), (1, 1), -1), dtype=torch.uint8, device="cuda")
    runs = []
    for rep in range(2):
        x = rng.standard_normal((N, C, H, W)).astype(np.float32)
        xh = torch.from_numpy(x)
        out_h = torch.empty((N, H, W, O), dtype=torch.int32)
        bits_h = torch.empty((N, H, W, 2), dtype=torch.int64)
        if pinned:
            xh, out_h, bits_h = xh.pin_memory(), out_h.pin_memory(), bits_h.pin_memory()
        B.binary_layer_host(xh, wp, ws, (1, 1), (1, 1), -1, scale, shift, out_host=out_h, bits_host=bits_h)
        runs.append((x, out_h, bits_h, xh))
    torch.cuda.synchronize()
    for x, out_h, bits_h, _ in runs:
        want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (1, 1), -1, o.NHWC)
        assert np.array_equal(out_h.numpy(), want)
        assert np.array_equal(bits_h.numpy().view(np.uint64), o.bn_sign_pack(want, scale_np, shift_np))
