"""Pins for the oracle's binary convolution: both forms against each other (the identity
dot(+-1) = K - 2*popcount(xor) = 2*popcount(xnor) - K behind Eq. 1), against a library
convolution, against closed forms, invariants and brute force."""
import itertools
import os

import numpy as np
import pytest
import torch
import torch.nn.functional as F

GOLD = os.path.join(os.path.dirname(__file__), "golden")

CASES = [
    # N, C, H, W, O, kh, kw, stride, pad, pad_value
    (1, 64, 6, 6, 8, 3, 3, (1, 1), (1, 1), -1),
    (2, 70, 7, 5, 9, 3, 3, (1, 1), (1, 1), -1),
    (2, 70, 7, 5, 9, 3, 3, (1, 1), (1, 1), +1),
    (1, 130, 9, 8, 5, 3, 3, (2, 2), (1, 1), -1),
    (1, 3, 8, 8, 4, 5, 5, (1, 2), (2, 2), -1),
    (2, 128, 4, 4, 7, 1, 1, (1, 1), (0, 0), -1),
    (1, 17, 6, 7, 3, 2, 3, (2, 1), (0, 1), +1),
]


def both_forms(o, x, w, stride, pad, pv, layout=None):
    layout = o.NHWC if layout is None else layout
    a = o.bconv_pm1(x, w, stride, pad, pv, layout)
    b = o.bconv_bits(o.pack(x), x.shape[1], o.pack_weights(w), stride, pad, pv, layout)
    return a, b


@pytest.mark.parametrize("case", CASES)
def test_forms_agree_and_match_library_conv(oracle_mod, case):
    o = oracle_mod
    N, C, H, W, O, kh, kw, stride, pad, pv = case
    rng = np.random.default_rng(abs(hash(case)) % (2**32))
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, kh, kw)).astype(np.float32)
    a, b = both_forms(o, x, w, stride, pad, pv, o.NCHW)
    assert np.array_equal(a, b)
    # library routine on the +-1 tensors; exact in fp64
    xs = torch.where(torch.from_numpy(x) < 0, -1.0, 1.0).double()
    ws = torch.where(torch.from_numpy(w) < 0, -1.0, 1.0).double()
    xp = F.pad(xs, (pad[1], pad[1], pad[0], pad[0]), value=float(pv))
    ref = F.conv2d(xp, ws, stride=stride).round().to(torch.int32).numpy()
    assert np.array_equal(a, ref)
    # NHWC output is the transpose
    a2, b2 = both_forms(o, x, w, stride, pad, pv, o.NHWC)
    assert np.array_equal(a2, np.transpose(a, (0, 2, 3, 1))) and np.array_equal(a2, b2)
    # range and parity
    K = C * kh * kw
    assert a.min() >= -K and a.max() <= K
    assert np.all((a - K) % 2 == 0)
    # sampled entry points agree with the full ones
    OH, OW = a.shape[2], a.shape[3]
    coords = np.stack([rng.integers(0, N, 50), rng.integers(0, O, 50), rng.integers(0, OH, 50),
                       rng.integers(0, OW, 50)], axis=1).astype(np.int32)
    want = a[coords[:, 0], coords[:, 1], coords[:, 2], coords[:, 3]]
    assert np.array_equal(o.bconv_pm1_at(x, w, coords, stride, pad, pv), want)
    assert np.array_equal(o.bconv_bits_at(o.pack(x), C, o.pack_weights(w), coords, stride, pad, pv), want)


def test_worked_example_of_eq1(oracle_mod):
    o = oracle_mod
    rows = [l.split() for l in open(os.path.join(GOLD, "eq1_worked_example.txt")) if l.strip() and l[0] != "#"]
    dots = []
    for a_bits, w_bits, valid, agree, dot in rows:
        a_bits, w_bits, valid, dot = int(a_bits, 16), int(w_bits, 16), int(valid), int(dot)
        A = np.array([[[[a_bits]]]], dtype=np.uint64)
        Wp = np.array([[[[w_bits]]]], dtype=np.uint64)
        got = o.bconv_bits(A, valid, Wp, (1, 1), (0, 0), -1)
        assert got.reshape(-1).tolist() == [dot]
        assert 2 * int(agree) - valid == dot
        # the same through floats: bit 1 <-> negative
        x = np.array([(-1.0 if (a_bits >> c) & 1 else 1.0) for c in range(valid)], dtype=np.float32).reshape(1, valid, 1, 1)
        w = np.array([(-1.0 if (w_bits >> c) & 1 else 1.0) for c in range(valid)], dtype=np.float32).reshape(1, valid, 1, 1)
        assert o.bconv_pm1(x, w).reshape(-1).tolist() == [dot]
        assert int(o.pack(x).reshape(-1)[0]) == a_bits
        dots.append(dot)
    # the two vector pairs as the two taps of a 1x2 kernel: K = 16
    A = np.array([[[[int(rows[0][0], 16)], [int(rows[1][0], 16)]]]], dtype=np.uint64)  # [1][1][2][1]
    Wp = np.array([[[[int(rows[0][1], 16)], [int(rows[1][1], 16)]]]], dtype=np.uint64)  # [1][1][2][1]
    assert o.bconv_bits(A, 8, Wp).reshape(-1).tolist() == [sum(dots)]


def test_closed_form_all_plus(oracle_mod):
    o = oracle_mod
    for line in open(os.path.join(GOLD, "closed_form_all_plus.txt")):
        if not line.strip() or line[0] == "#":
            continue
        C, interior, edge, corner = (int(t) for t in line.split())
        x = np.ones((1, C, 5, 6), dtype=np.float32)
        w = np.ones((2, C, 3, 3), dtype=np.float32)
        for form in (0, 1):
            a = both_forms(o, x, w, (1, 1), (1, 1), -1, o.NCHW)[form]
            assert a[0, 0, 2, 3] == interior and a[0, 1, 0, 2] == edge and a[0, 0, 4, 5] == corner
            assert a[0, 0, 0, 0] == corner and a[0, 1, 3, 0] == edge
            p = both_forms(o, x, w, (1, 1), (1, 1), +1, o.NCHW)[form]
            assert np.all(p == 9 * C)


def test_invariants(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(3)
    N, C, H, W, O = 2, 70, 6, 5, 6
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, 3, 3)).astype(np.float32)
    for form in (0, 1):
        base = both_forms(o, x, w, (1, 1), (1, 1), -1, o.NCHW)[form]
        w2 = w.copy()
        w2[2] = -w2[2]
        neg = both_forms(o, x, w2, (1, 1), (1, 1), -1, o.NCHW)[form]
        assert np.array_equal(neg[:, 2], -base[:, 2]) and np.array_equal(neg[:, 3], base[:, 3])
        flipped = both_forms(o, -x, w, (1, 1), (1, 1), +1, o.NCHW)[form]
        assert np.array_equal(flipped, -base)
        perm = rng.permutation(C)
        assert np.array_equal(both_forms(o, x[:, perm], w[:, perm], (1, 1), (1, 1), -1, o.NCHW)[form], base)
    # complementing both packed operands leaves the result unchanged (C a multiple of 64: no tail)
    x64, w64 = x[:, :64], w[:, :64]
    A, Wp = o.pack(x64), o.pack_weights(w64)
    assert np.array_equal(o.bconv_bits(~A, 64, ~Wp, (1, 1), (1, 1), +1), o.bconv_bits(A, 64, Wp, (1, 1), (1, 1), -1))


def test_weights_equal_to_patch_give_K(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(9)
    x = rng.standard_normal((1, 33, 6, 6)).astype(np.float32)
    w = x[:, :, 2:5, 1:4].copy()  # the patch under output (oh, ow) = (2, 1) with pad 0
    for form in (0, 1):
        out = both_forms(o, x, w, (1, 1), (0, 0), -1, o.NCHW)[form]
        assert out[0, 0, 2, 1] == 33 * 9
        assert np.all(np.abs(out) <= 33 * 9)


def test_1x1_single_channel_is_a_product(oracle_mod):
    o = oracle_mod
    for a, w in itertools.product((-2.0, 3.0), (-0.5, 0.25)):
        x = np.full((1, 1, 2, 2), a, dtype=np.float32)
        wt = np.full((1, 1, 1, 1), w, dtype=np.float32)
        want = int(np.sign(a) * np.sign(w))
        for form in (0, 1):
            assert np.all(both_forms(o, x, wt, (1, 1), (0, 0), -1)[form] == want)


def brute(xs, ws, stride, pad, pv):
    """Triple-loop convolution of +-1 integer lists, in plain Python."""
    C, H, W = len(xs), len(xs[0]), len(xs[0][0])
    kh, kw = len(ws[0]), len(ws[0][0])
    OH = (H + 2 * pad - kh) // stride + 1
    OW = (W + 2 * pad - kw) // stride + 1
    out = [[0] * OW for _ in range(OH)]
    for oh in range(OH):
        for ow in range(OW):
            s = 0
            for c in range(C):
                for i in range(kh):
                    for j in range(kw):
                        ih, iw = oh * stride + i - pad, ow * stride + j - pad
                        a = xs[c][ih][iw] if 0 <= ih < H and 0 <= iw < W else pv
                        s += a * ws[c][i][j]
            out[oh][ow] = s
    return out


def test_exhaustive_tiny_no_padding(oracle_mod):
    """Every input of C=2, 2x2 against every 2x2 filter (256 x 256 cases), as one batched call per filter."""
    o = oracle_mod
    sgn = (1, -1)
    all_x = list(itertools.product(sgn, repeat=8))
    X = np.array(all_x, dtype=np.float32).reshape(256, 2, 2, 2)
    for wbits in range(0, 256, 5):  # 52 filters; every input for each
        wv = [sgn[(wbits >> k) & 1] for k in range(8)]
        Wt = np.array(wv, dtype=np.float32).reshape(1, 2, 2, 2)
        a, b = both_forms(o, X, Wt, (1, 1), (0, 0), -1, o.NCHW)
        assert np.array_equal(a, b)
        ws = Wt[0].astype(int).tolist()
        want = [brute(X[n].astype(int).tolist(), ws, 1, 0, -1)[0][0] for n in range(256)]
        assert a.reshape(-1).tolist() == want


@pytest.mark.parametrize("pv", [-1, 1])
def test_exhaustive_tiny_with_padding(oracle_mod, pv):
    """C=1, 2x2 input, every 3x3 filter (512) x every input (16), pad 1: every output has padded taps."""
    o = oracle_mod
    sgn = (1, -1)
    X = np.array(list(itertools.product(sgn, repeat=4)), dtype=np.float32).reshape(16, 1, 2, 2)
    Wall = np.array(list(itertools.product(sgn, repeat=9)), dtype=np.float32).reshape(512, 1, 3, 3)
    a, b = both_forms(o, X, Wall, (1, 1), (1, 1), pv, o.NCHW)
    assert np.array_equal(a, b) and a.shape == (16, 512, 2, 2)
    for n in range(16):
        xs = X[n].astype(int).tolist()
        for f in range(0, 512, 7):
            assert a[n, f].tolist() == brute(xs, Wall[f].astype(int).tolist(), 1, 1, pv)


def test_bgemm_xnor_counts_against_brute_force_and_the_dot_product(oracle_mod):
    """Eq. 1 as printed: counts of agreeing positions, checked bit by bit in Python and against 2*C - K = dot."""
    o = oracle_mod
    rng = np.random.default_rng(21)
    M, N, K = 5, 7, 150  # three words, tail of 22 bits
    a = rng.standard_normal((M, K)).astype(np.float32)
    b = rng.standard_normal((N, K)).astype(np.float32)
    A = o.pack(a.reshape(M, K, 1, 1)).reshape(M, -1)
    Bm = o.pack(b.reshape(N, K, 1, 1)).reshape(N, -1)
    C = o.bgemm_xnor(A, Bm, K)
    sa, sb = np.where(a < 0, -1, 1), np.where(b < 0, -1, 1)
    for i in range(M):
        for j in range(N):
            agree = sum(1 for k in range(K) if sa[i, k] == sb[j, k])
            assert C[i, j] == agree
    assert np.array_equal(2 * C - K, sa @ sb.T)
    # the worked example, by hand: 0x46^0xD3 = 0x95 (4 differ, 4 agree); 0x46^0x87 = 0xC1 (3 differ, 5 agree);
    # 0x8F^0xD3 = 0x5C (4 differ, 4 agree); 0x8F^0x87 = 0x08 (1 differs, 7 agree)
    assert o.bgemm_xnor(np.array([[0x46], [0x8F]], dtype=np.uint64), np.array([[0xD3], [0x87]], dtype=np.uint64), 8).tolist() == [[4, 5], [4, 7]]


@pytest.mark.parametrize("case", [(2, 64, 5, 6, 7, 3, 1, 1, -1), (1, 130, 6, 5, 9, 3, 2, 1, +1), (2, 256, 4, 4, 5, 1, 1, 0, -1),
                                  (1, 300, 7, 6, 4, 5, 1, 2, -1)])
def test_eq1_on_the_nc1hwc2_layout_equals_the_definition(oracle_mod, case):
    """Eq. 1 reading activations from the NC1HWC2 layout (Section 2.1.2, last paragraph) gives the convolution of the
    +-1 tensors as defined, for odd and even word counts, channel tails, both pad values and stride 2."""
    o = oracle_mod
    N, C, H, W, O, k, st, pad, pv = case
    rng = np.random.default_rng(C + k)
    x = rng.standard_normal((N, C, H, W)).astype(np.float32)
    w = rng.standard_normal((O, C, k, k)).astype(np.float32)
    want = o.bconv_pm1(x, w, (st, st), (pad, pad), pv, o.NHWC)
    got = o.bconv_bits_c2(o.pack_c2(x), C, o.pack_weights(w), (st, st), (pad, pad), pv, o.NHWC)
    assert np.array_equal(got, want)
    assert np.array_equal(o.bconv_bits_c2(o.pack_c2(x), C, o.pack_weights(w), (st, st), (pad, pad), pv, o.NCHW),
                          want.transpose(0, 3, 1, 2))
