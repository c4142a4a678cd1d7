"""GPU parity of the tensor-core engine (dabnn_tc_*): identical integers, bits and fp32 values as the CPU oracle,
through every epilogue, on shapes that cover several channel tiles, ragged tiles, channel tails and pad values."""
import numpy as np
import pytest
import torch

from paper_1908_05858_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def B():
    from paper_1908_05858_b200 import binding

    assert torch.cuda.is_available()
    binding.lib()
    return binding


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def u64(t):
    return t.cpu().numpy().view(np.uint64)


TC_CASES = [
    (2, 70, 7, 5, 9, 3, 1, -1),         # channel tail in the only word, tiny O
    (3, 96, 9, 10, 40, 3, 1, +1),       # C = 96: half of the second word
    (2, 130, 9, 8, 37, 3, 1, -1, 2),    # two live channels in the third word, stride 2
    (2, 500, 6, 6, 70, 1, 0, -1),       # 1x1 with a tail in the eighth word
    (2, 3, 12, 12, 5, 5, 2, -1),        # three channels
    # N, C, H, W, O, k, pad, pad_value[, stride]
    (1, 64, 14, 14, 64, 3, 1, -1),      # BASELINE config 1
    (2, 128, 9, 11, 100, 3, 1, +1),     # O not a multiple of 16, pad +1
    (3, 256, 14, 14, 256, 3, 1, -1),    # four channel tiles of 64
    (2, 512, 7, 7, 512, 3, 1, -1),      # channel tiles of 32, K = 4608
    (2, 512, 14, 14, 300, 1, 0, -1),    # 1x1, ragged channel tile
    (1, 64, 56, 56, 64, 3, 1, -1),
    (2, 192, 10, 10, 70, 5, 2, -1),     # three words, 5x5, O just over one sign word
    (5, 64, 6, 7, 33, 3, 1, -1),        # smallest C, O just over a 32-channel tile
    (9, 128, 28, 28, 128, 3, 1, -1),    # many pixel tiles per CTA? (persistent loop over tiles)
    (300, 64, 8, 8, 64, 3, 0, -1),      # no padding, many images per tile
    (3, 64, 56, 56, 128, 3, 1, -1, 2),  # stride 2 (four parity planes): Bi-Real stage 2 entry
    (5, 128, 28, 28, 256, 3, 1, -1, 2),
    (7, 256, 14, 14, 512, 3, 1, +1, 2),
    (2, 64, 13, 11, 70, 3, 1, -1, 2),   # odd sizes, stride 2
    (2, 128, 12, 12, 64, 1, 0, -1, 2),  # 1x1 stride 2
    (2, 64, 16, 16, 64, 5, 2, -1, 2),   # 5x5 stride 2
    (2, 448, 10, 10, 70, 3, 1, -1),     # seven words
    (2, 192, 10, 10, 70, 4, 2, -1),     # even filter size
    (2, 320, 10, 10, 32, 5, 2, -1),     # five words, 5x5, one 32-channel tile
    (40, 256, 14, 14, 256, 3, 1, -1),   # enough tiles for CTA pairs with two resident channel tiles
    (33, 512, 7, 7, 512, 3, 1, +1),     # pairs, odd number of tiles, four channel-tile groups
    (70, 128, 28, 28, 128, 3, 1, -1, 2),  # pairs, stride 2
    # more channels than one activation buffer takes: a tile's channels pass through the buffers in groups
    (3, 576, 9, 9, 70, 3, 1, -1),         # nine words: a group of eight and a group of one
    (2, 1000, 8, 7, 40, 3, 1, +1),        # sixteen words with a channel tail, weights of 32 channels per CTA
    (5, 2048, 6, 6, 200, 1, 0, -1),       # 1x1 over 2048 channels: four groups
    (3, 1500, 5, 5, 96, 1, 0, -1),        # 24 words: three groups, the last with a tail
    (2, 320, 20, 20, 64, 3, 1, -1, 2),    # stride 2 with five words: groups of four
    (4, 512, 14, 14, 128, 3, 1, -1, 2),   # stride 2, C = 512: two groups of four
    (2, 640, 12, 12, 64, 1, 0, +1, 2),    # 1x1 stride 2, ten words
]


def inputs(case):
    N, C, H, W, O, k, pad, pv = case[:8]
    rng = np.random.default_rng(abs(hash(case)) % (2**32))
    return rng.standard_normal((N, C, H, W)).astype(np.float32), rng.standard_normal((O, C, k, k)).astype(np.float32)


@pytest.mark.parametrize("case", TC_CASES)
def test_tc_conv_and_epilogues_match_oracle(B, oracle_mod, case):
    N, C, H, W, O, k, pad, pv = case[:8]
    st = (case[8], case[8]) if len(case) > 8 else (1, 1)
    x, w = inputs(case)
    o = oracle_mod
    acc = o.bconv_bits(o.pack(x), C, o.pack_weights(w), st, (pad, pad), pv, o.NHWC)
    a = B.pack(dev(x))
    wp = B.pack_weights(dev(w))
    assert B.tc_supported(O, C, k, k, st)
    wt = B.TcWeights(wp, C)
    got = B.tc_bconv2d(a, wt, st, (pad, pad), pv, B.NHWC).cpu().numpy()
    assert np.array_equal(got, acc)
    got_nchw = B.tc_bconv2d(a, wt, st, (pad, pad), pv, B.NCHW).cpu().numpy()
    assert np.array_equal(got_nchw, np.transpose(acc, (0, 3, 1, 2)))
    # the xor/popcount kernel gives the same integers
    assert np.array_equal(B.bconv2d(a, C, wp, st, (pad, pad), pv, B.NHWC).cpu().numpy(), acc)
    # fused BN + sign + pack
    rng = np.random.default_rng(O)
    gamma, beta, mean, var = synth.bn_params(rng, O)
    gamma[::5] *= -1.0
    mean *= 30.0
    scale, shift = o.bn_fold(gamma, beta, mean, var)
    want_bits = o.bn_sign_pack(acc, scale, shift)
    got_bits = u64(B.tc_bconv2d_bn_sign_pack(a, wt, dev(scale), dev(shift), st, (pad, pad), pv))
    assert np.array_equal(got_bits, want_bits)
    # Bi-Real block epilogue
    res = rng.standard_normal(acc.shape).astype(np.float32) * 20
    y, want_ybits = o.bn_add_sign_pack(acc, scale, shift, res)
    got_y, got_ybits = B.tc_bconv2d_bn_add_sign_pack(a, wt, dev(scale), dev(shift), dev(res), st, (pad, pad), pv)
    assert np.array_equal(got_y.cpu().numpy().view(np.uint32), y.view(np.uint32))
    assert np.array_equal(u64(got_ybits), want_ybits)
    torch.cuda.synchronize()
    assert B.tc_error_flag() == 0


# Launches long enough for the form of the Bi-Real epilogue that fetches the residual with bulk tensor copies (a ring of
# 32-row x 32-channel chunks per epilogue warp): ragged slot rows, a channel tile that reaches beyond O, several images per
# tile, and the in-place call the network makes (y written over the residual).
RING_CASES = [
    (16, 64, 56, 56, 64, 3, 1, -1),
    (48, 128, 28, 28, 128, 3, 1, +1),
    (50, 64, 30, 27, 96, 3, 1, -1),
    (700, 128, 7, 9, 160, 1, 0, -1),
]


@pytest.mark.parametrize("case", RING_CASES)
def test_tc_bireal_epilogue_with_the_residual_through_bulk_copies(B, oracle_mod, case):
    N, C, H, W, O, k, pad, pv = case
    x, w = inputs(case)
    o = oracle_mod
    acc = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (pad, pad), pv, o.NHWC)
    rng = np.random.default_rng(O + N)
    gamma, beta, mean, var = synth.bn_params(rng, O)
    gamma[::3] *= -1.0
    scale, shift = o.bn_fold(gamma, beta, mean, var)
    res = (rng.standard_normal(acc.shape) * 15).astype(np.float32)
    y, want_bits = o.bn_add_sign_pack(acc, scale, shift, res)
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    wt = B.TcWeights(wp, C)
    got_y, got_bits = B.tc_bconv2d_bn_add_sign_pack(a, wt, dev(scale), dev(shift), dev(res), (1, 1), (pad, pad), pv)
    assert np.array_equal(got_y.cpu().numpy().view(np.uint32), y.view(np.uint32))
    assert np.array_equal(u64(got_bits), want_bits)
    # in place, twice in a row from the same input (the second call must not see anything of the first)
    for _ in range(2):
        stream = dev(res)
        call = B.prepare_bireal_block(a, C, wp, wt, dev(scale), dev(shift), stream, (1, 1), (pad, pad), pv)
        call()
        torch.cuda.synchronize()
        assert np.array_equal(stream.cpu().numpy().view(np.uint32), y.view(np.uint32))
        assert np.array_equal(u64(call.keep[-1]), want_bits)
    assert B.tc_error_flag() == 0


@pytest.mark.parametrize("shape", [(300, 260, 512), (129, 65, 64), (70, 33, 150), (1000, 2048, 500), (700, 300, 4096), (260, 100, 9000)])
def test_tc_bgemm_matches_eq1(B, oracle_mod, shape):
    M, N, K = shape
    rng = np.random.default_rng(M + N + K)
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    A = B.pack(dev(a.reshape(M, K, 1, 1))).reshape(M, -1)
    Bp = B.pack(dev(b.reshape(N, K, 1, 1)))  # [N][1][1][Kw]: the layout of packed 1x1 weights
    got = B.tc_bgemm(A, B.TcWeights(Bp, K), K).cpu().numpy()
    counts = oracle_mod.bgemm_xnor(u64(A), u64(Bp).reshape(N, -1), K)  # Eq. 1 as printed: agreeing positions
    assert np.array_equal(got, 2 * counts - K)
    assert np.array_equal(got, B.bgemm(A, Bp.reshape(N, -1), K).cpu().numpy())


def test_tc_declines_what_it_does_not_cover(B):
    assert not B.tc_supported(64, 64, 3, 3, stride=(3, 3))
    assert B.tc_supported(64, 576, 3, 3)             # more than 512 channels: in groups
    assert not B.tc_supported(64, 1100, 3, 3)        # ... while the weights of 32 output channels still fit the resident budget
    assert not B.tc_supported(64, 2048, 7, 7)        # expanded weights larger than the resident budget
    a = torch.zeros((1, 8, 8, 1), dtype=torch.int64, device="cuda")
    wt = B.TcWeights(torch.zeros((64, 3, 3, 1), dtype=torch.int64, device="cuda"), 64)
    with pytest.raises(B.DabnnError, match="supported"):
        B.tc_bconv2d(a, wt, (2, 1), (1, 1), -1)


@pytest.mark.parametrize("cfg", [(64, 64, 56, 64, 3, 1), (64, 512, 7, 512, 3, 1), (256, 256, 28, 256, 3, 1), (256, 512, 14, 2048, 1, 0)])
def test_tc_full_size_configs_on_sampled_outputs(B, oracle_mod, cfg):
    N, C, HW, O, k, pad = cfg
    x, w = synth.conv_case(2 if N == 64 else 5, N, C, HW, HW, O, k, k, salt=C)
    a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
    got = B.tc_bconv2d(a, B.TcWeights(wp, C), (1, 1), (pad, pad), -1, B.NHWC)
    K = C * k * k
    assert int(got.min()) >= -K and int(got.max()) <= K and bool(((got - K) % 2 == 0).all())
    # the whole tensor against Eq. 1 on the packed words (the oracle), and samples against the definition
    g = got.cpu().numpy()
    full = oracle_mod.bconv_bits(oracle_mod.pack(x), C, oracle_mod.pack_weights(w), (1, 1), (pad, pad), -1, oracle_mod.NHWC)
    assert np.array_equal(g, full)
    rng = np.random.default_rng(C + N)
    coords = np.stack([rng.integers(0, N, 20000), rng.integers(0, O, 20000), rng.integers(0, HW, 20000), rng.integers(0, HW, 20000)], axis=1).astype(np.int32)
    want = oracle_mod.bconv_pm1_at(x, w, coords, (1, 1), (pad, pad), -1)
    assert np.array_equal(g[coords[:, 0], coords[:, 2], coords[:, 3], coords[:, 1]], want)
    # the fused sign epilogue at full size: the whole packed tensor against the oracle's fmaf + sign + pack of its own
    # sums, and the definition on sampled pixels
    rng2 = np.random.default_rng(C + N + 1)
    scale = rng2.uniform(0.5, 1.5, O).astype(np.float32)
    scale[::7] *= -1.0
    shift = rng2.normal(0, 0.3 * np.sqrt(K), O).astype(np.float32)
    bits = B.tc_bconv2d_bn_sign_pack(a, B.TcWeights(wp, C), dev(scale), dev(shift), (1, 1), (pad, pad), -1)
    assert np.array_equal(u64(bits), oracle_mod.bn_sign_pack(full, scale, shift))
    del full
    px = coords[:2000]
    acc_px = oracle_mod.bconv_pm1_at(x, w, np.stack([np.repeat(px[:, 0], O), np.tile(np.arange(O), len(px)), np.repeat(px[:, 2], O),
                                                     np.repeat(px[:, 3], O)], axis=1).astype(np.int32), (1, 1), (pad, pad), -1)
    want_bits = oracle_mod.bn_sign_pack(acc_px.reshape(len(px), 1, 1, O), scale, shift).reshape(len(px), -1)
    got_bits = bits.cpu().numpy().view(np.uint64)[px[:, 0], px[:, 2], px[:, 3]]
    assert np.array_equal(got_bits, want_bits)
    assert B.tc_error_flag() == 0


@pytest.mark.parametrize("C,k,pad", [(64, 3, 1), (128, 3, 1), (256, 1, 0)])
def test_tc_sign_epilogue_is_exact_for_awkward_bn_vectors(B, oracle_mod, C, k, pad):
    """The fused epilogue decides sign(fmaf(acc, scale, shift)) through an integer threshold per channel: negative, zero,
    huge, tiny, infinite and NaN scales and shifts, and shifts that put y exactly on zero, against the oracle's fmaf."""
    o = oracle_mod
    N, H, W, O = 3, 9, 10, 128
    rng = np.random.default_rng(C + k)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, k, k)).astype(np.float32)
    acc = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (pad, pad), -1, o.NHWC)
    scale = rng.uniform(0.5, 1.5, O).astype(np.float32)
    shift = rng.normal(0, 4, O).astype(np.float32)
    scale[0:8] *= -1                                     # decreasing in acc
    scale[8:12] = [0.0, -0.0, 0.0, -0.0]; shift[8:12] = [1.0, -1.0, -0.0, 0.0]
    scale[12:16] = [np.inf, -np.inf, np.inf, -np.inf]; shift[12:16] = [3.0, 3.0, -np.inf, np.inf]
    scale[16:18] = np.nan; shift[18:20] = np.nan
    scale[20:24] = [1e-30, -1e-30, 1e30, -1e30]; shift[20:24] = [1e-31, 1e-31, -1e29, 5e30]
    scale[24:32] = [1, 1, -1, -1, 2, 0.5, -2, -0.5]      # y exactly zero at an attainable acc, and just beside it
    shift[24:32] = [-4, 4, 6, -6, -8, 1, 12, -3]
    scale[32:36] = [1.0000001, 0.99999994, -1.0000001, -0.99999994]; shift[32:36] = [-10, -10, 10, 10]
    shift[36:40] = [np.inf, -np.inf, 1e38, -1e38]
    want = o.bn_sign_pack(acc, scale, shift)
    a = B.pack(dev(x))
    wt = B.TcWeights(B.pack_weights(dev(w)), C)
    got = u64(B.tc_bconv2d_bn_sign_pack(a, wt, dev(scale), dev(shift), (1, 1), (pad, pad), -1))
    assert np.array_equal(got, want)
    # and the integer-pipe engine, which evaluates the fmaf itself
    got2 = u64(B.bconv2d_bn_sign_pack(a, C, B.pack_weights(dev(w)), dev(scale), dev(shift), (1, 1), (pad, pad), -1))
    assert np.array_equal(got2, want)
    assert B.tc_error_flag() == 0


@pytest.mark.parametrize("cap", [1, 10, 74])
def test_tc_results_do_not_depend_on_the_cta_cap(B, oracle_mod, cap):
    o = oracle_mod
    rng = np.random.default_rng(cap)
    try:
        for N, C, H, W, O in ((5, 128, 14, 14, 128), (20, 512, 7, 7, 512), (3, 64, 20, 20, 192)):
            x = rng.standard_normal((N, C, H, W)).astype(np.float32)
            w = rng.standard_normal((O, C, 3, 3)).astype(np.float32)
            want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (1, 1), -1, o.NHWC)
            a, wt = B.pack(dev(x)), B.TcWeights(B.pack_weights(dev(w)), C)
            assert B.tc_set_max_ctas(cap) in (0, cap)
            got = B.tc_bconv2d(a, wt, (1, 1), (1, 1), -1, B.NHWC).cpu().numpy()
            assert np.array_equal(got, want)
    finally:
        B.tc_set_max_ctas(0)
    assert B.tc_error_flag() == 0


@pytest.mark.parametrize("kh,kw,ph,pw", [(1, 3, 0, 1), (3, 1, 1, 0), (3, 5, 1, 2), (3, 3, 0, 1), (3, 3, 2, 2), (2, 2, 1, 1), (3, 3, 3, 3)])
def test_asymmetric_filters_and_paddings_on_both_engines(B, oracle_mod, kh, kw, ph, pw):
    """Filters and paddings that differ between the axes, padding smaller and larger than (k - 1) / 2, and padding beyond
    k - 1 (where the tensor engine keeps both padding columns in its slot grid)."""
    o = oracle_mod
    N, C, H, W, O = 3, 64, 9, 11, 64
    rng = np.random.default_rng(kh * 100 + kw * 10 + ph + pw)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, kh, kw)).astype(np.float32)
    for pv in (-1, 1):
        want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (ph, pw), pv, o.NHWC)
        a, wp = B.pack(dev(x)), B.pack_weights(dev(w))
        assert np.array_equal(B.bconv2d(a, C, wp, (1, 1), (ph, pw), pv, B.NHWC).cpu().numpy(), want)
        assert np.array_equal(B.tc_bconv2d(a, B.TcWeights(wp, C), (1, 1), (ph, pw), pv, B.NHWC).cpu().numpy(), want)
    assert B.tc_error_flag() == 0


def test_a_wait_that_runs_out_sets_the_flag_and_leaves_the_device_usable(B, oracle_mod):
    """The failure path of the bounded waits, made to happen without any fault: a launch whose "rows ready" barrier expects
    one arrival more than it gets, every wait limited to about a millisecond.  The kernel must return by itself, the
    device flag must read 1 once (then 0 again), the call that reports it must say DABNN_ERR_TIMEOUT, and the next ordinary
    launches must give the oracle's integers."""
    import time
    o = oracle_mod
    for case in ((3, 128, 14, 14, 128, 3, 1), (100, 512, 7, 7, 512, 3, 1)):  # one CTA per tile; CTA pairs
        N, C, H, W, O, k, pad = case
        rng = np.random.default_rng(C)
        x = rng.standard_normal((N, C, H, W)).astype(np.float32)
        w = rng.standard_normal((O, C, k, k)).astype(np.float32)
        want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (1, 1), (pad, pad), -1, o.NHWC)
        a, wt = B.pack(dev(x)), B.TcWeights(B.pack_weights(dev(w)), C)
        assert B.last_device_flag() == 0
        t0 = time.perf_counter()
        B.tc_wait_expiry_selftest(a, wt, (1, 1), (pad, pad), -1, wait_polls=1000)
        assert B.last_device_flag() == 1          # synchronises: the kernel came back by itself
        assert time.perf_counter() - t0 < 5.0
        assert B.last_device_flag() == 0          # reading cleared it
        B.tc_wait_expiry_selftest(a, wt, (1, 1), (pad, pad), -1, wait_polls=200)
        assert B.stream_status() == B.ERR_TIMEOUT and B.stream_status() == 0
        for _ in range(2):                        # tensor memory was freed, barriers start afresh: ordinary launches are exact
            got = B.tc_bconv2d(a, wt, (1, 1), (pad, pad), -1, B.NHWC).cpu().numpy()
            assert np.array_equal(got, want)
        assert B.last_device_flag() == 0
    with pytest.raises(B.DabnnError):
        B.tc_wait_expiry_selftest(a, wt, (1, 1), (pad, pad), -1, wait_polls=1 << 20)  # limit beyond a few milliseconds: refused


def tc_matrix_cases():
    """Channel words 1..8 x filter sizes 1, 2, 3, 4, 5, 7 x strides 1, 2: every count of K blocks per tap through the
    unrolled 3x3 issue path and the runtime tap loops of the other filters, at a size with several tiles and a ragged
    channel tile."""
    return [(2, 64 * cw - (17 if (cw + k) % 3 == 0 else 0), 11, 10, 70, k, k // 2, -1 if (cw + k) % 2 else 1, st)
            for cw in range(1, 9) for k in (1, 2, 3, 4, 5, 7) for st in (1, 2)]  # (a third of the cases with a channel tail)


def run_tc_matrix(B, o):
    """Returns (cases run, cases the engine declines); asserts bit equality with Eq. 1 on the packed words for the rest."""
    ran = declined = 0
    for N, C, H, W, O, k, pad, pv, st in tc_matrix_cases():
        if not B.tc_supported(O, C, k, k, (st, st)):
            declined += 1
            continue
        rng = np.random.default_rng(1000 * C + 10 * k + st)
        x = rng.standard_normal((N, C, H, W)).astype(np.float32)
        w = rng.standard_normal((O, C, k, k)).astype(np.float32)
        a = B.pack(torch.from_numpy(x).cuda())
        wt = B.TcWeights(B.pack_weights(torch.from_numpy(w).cuda()), C)
        try:
            got = B.tc_bconv2d(a, wt, (st, st), (pad, pad), pv, B.NHWC).cpu().numpy()
        except B.DabnnError as e:  # (stride 2 beyond 256 channels: declined at launch)
            assert "supported" in str(e), (C, k, st, str(e))
            declined += 1
            continue
        want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (st, st), (pad, pad), pv, o.NHWC)
        assert np.array_equal(got, want), (C, k, st)
        ran += 1
    torch.cuda.synchronize()
    assert B.last_device_flag() == 0
    return ran, declined


def test_tc_matrix_of_channel_words_filters_and_strides(B, oracle_mod):
    ran, declined = run_tc_matrix(B, oracle_mod)
    assert ran >= 60 and ran + declined == 96, (ran, declined)


_FORCED_FORM_SCRIPT = r"""
import sys, numpy as np, torch
from paper_1908_05858_b200 import binding as B
import oracle as o
o.set_threads(o.max_threads())
rng = np.random.default_rng(77)
cases = [(3, 64, 14, 14, 64, 3, 1, -1, 1), (40, 256, 14, 14, 256, 3, 1, -1, 1), (9, 512, 7, 7, 512, 3, 1, +1, 1),
         (2, 192, 10, 10, 70, 5, 2, -1, 1), (6, 128, 28, 28, 256, 3, 1, -1, 2), (2, 448, 10, 10, 70, 3, 1, -1, 1)]
for N, C, H, W, O, k, pad, pv, st in cases:
    x = rng.standard_normal((N, C, H, W)).astype(np.float32); w = rng.standard_normal((O, C, k, k)).astype(np.float32)
    want = o.bconv_bits(o.pack(x), C, o.pack_weights(w), (st, st), (pad, pad), pv, o.NHWC)
    a = B.pack(torch.from_numpy(x).cuda()); wt = B.TcWeights(B.pack_weights(torch.from_numpy(w).cuda()), C)
    got = B.tc_bconv2d(a, wt, (st, st), (pad, pad), pv, B.NHWC).cpu().numpy()
    assert np.array_equal(got, want), (N, C, H, W, O, k)
    sc = torch.from_numpy(rng.uniform(0.5, 1.5, O).astype(np.float32)).cuda(); sh = torch.from_numpy(rng.normal(0, 3, O).astype(np.float32)).cuda()
    bits = B.tc_bconv2d_bn_sign_pack(a, wt, sc, sh, (st, st), (pad, pad), pv).cpu().numpy().view(np.uint64)
    assert np.array_equal(bits, o.bn_sign_pack(want, sc.cpu().numpy(), sh.cpu().numpy())), (N, C, H, W, O, k)
torch.cuda.synchronize()
assert B.tc_error_flag() == 0
sys.path.insert(0, "tests")
import test_gpu_tc
ran, declined = test_gpu_tc.run_tc_matrix(B, o)
assert ran >= 50, (ran, declined)
print("forced form ok")
"""


@pytest.mark.parametrize("mode", ["1", "2"])
def test_both_launch_forms_in_a_child_process(mode):
    """The launch form is chosen by size; DABNN_TC_MODE (read once per process) forces one CTA per tile (1) or CTA
    pairs (2), so each form is run on the same cases in a child process and compared with the oracle."""
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, DABNN_TC_MODE=mode, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", _FORCED_FORM_SCRIPT], env=env, cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "forced form ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]


_RING_SCRIPT = r"""
import sys
sys.path.insert(0, "tests")
import oracle as o
o.set_threads(o.max_threads())
from paper_1908_05858_b200 import binding as B
import test_gpu_tc
for case in test_gpu_tc.RING_CASES:
    test_gpu_tc.test_tc_bireal_epilogue_with_the_residual_through_bulk_copies(B, o, case)
print("ring ok")
"""


@pytest.mark.parametrize("ring", ["0", "4"])
def test_residual_ring_depths_in_a_child_process(ring):
    """DABNN_TC_RES_RING (read once per process): 0 = the epilogue warps load the residual themselves, 4 = the deepest ring
    of bulk copies.  Both must give the oracle's bits on the cases of the default depth."""
    import os, subprocess, sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = dict(os.environ, DABNN_TC_RES_RING=ring, PYTHONPATH=root + os.pathsep + os.environ.get("PYTHONPATH", ""))
    r = subprocess.run([sys.executable, "-c", _RING_SCRIPT], env=env, cwd=root, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0 and "ring ok" in r.stdout, r.stdout[-2000:] + r.stderr[-2000:]
