"""Pins for the oracle's BN fold and fused BN + binarize + re-pack (Section 2.1.1, last sentence)."""
from decimal import Decimal, getcontext
from fractions import Fraction

import numpy as np


def test_fold_matches_batchnorm_definition(oracle_mod):
    """scale*x + shift equals gamma*(x-mean)/sqrt(var+eps)+beta, evaluated with 50-digit decimals."""
    o = oracle_mod
    getcontext().prec = 50
    rng = np.random.default_rng(2)
    O = 64
    gamma = rng.uniform(0.5, 1.5, O).astype(np.float32)
    gamma[:4] *= -1  # negative scales too
    beta = rng.normal(0, 0.1, O).astype(np.float32)
    mean = rng.normal(0, 0.1, O).astype(np.float32)
    var = rng.uniform(0.5, 1.5, O).astype(np.float32)
    scale, shift = o.bn_fold(gamma, beta, mean, var, 1e-5)
    assert scale.dtype == np.float32 and shift.dtype == np.float32
    eps = Decimal(1e-5)  # the double nearest to 1e-5, exactly
    for i in range(O):
        sd = Decimal(float(gamma[i])) / (Decimal(float(var[i])) + eps).sqrt()
        sh = Decimal(float(beta[i])) - Decimal(float(mean[i])) * sd
        # one rounding to fp32 each: relative error <= 2^-24 (plus the double rounding underneath)
        assert abs(Decimal(float(scale[i])) - sd) <= abs(sd) * Decimal(2) ** -23
        assert abs(Decimal(float(shift[i])) - sh) <= max(abs(sh), Decimal(1e-30)) * Decimal(2) ** -22
        for x in (-576, -3, 0, 7, 4608):
            bn = Decimal(float(gamma[i])) * (Decimal(x) - Decimal(float(mean[i]))) / (Decimal(float(var[i])) + eps).sqrt() + Decimal(float(beta[i]))
            folded = Decimal(float(scale[i])) * Decimal(x) + Decimal(float(shift[i]))
            assert abs(bn - folded) <= Decimal(1e-6) * (abs(bn) + 1)


def test_sign_decision_is_the_sign_of_the_exact_value(oracle_mod):
    """fmaf rounds the exact scale*acc+shift once, so y<0 iff the exact rational value is <0
    (no underflow in this range).  Checked with exact fractions for every acc of a K=576 layer."""
    o = oracle_mod
    rng = np.random.default_rng(4)
    O, K = 70, 576
    scale = rng.normal(0, 0.05, O).astype(np.float32)
    shift = rng.normal(0, 1.0, O).astype(np.float32)
    scale[0], shift[0] = 0.0, -1.0   # constant negative
    scale[1], shift[1] = 0.0, 2.0    # constant positive
    scale[2], shift[2] = 0.5, -3.0   # exact zero at acc = 6 -> +1
    scale[3], shift[3] = -0.25, 0.0  # exact zero at acc = 0 -> +1
    accs = np.arange(-K, K + 1, 2, dtype=np.int32)
    acc = np.repeat(accs[:, None], O, axis=1)  # [npix][O]
    P = o.bn_sign_pack(acc, scale, shift)
    assert P.shape == (len(accs), 2)
    for ch in range(O):
        fs, fb = Fraction(float(scale[ch])), Fraction(float(shift[ch]))
        bits = (P[:, ch >> 6] >> np.uint64(ch & 63)) & np.uint64(1)
        want = [1 if fs * int(a) + fb < 0 else 0 for a in accs]
        assert bits.astype(int).tolist() == want, ch
        # monotone in acc: at most one change of sign along the sorted acc values
        assert int(np.count_nonzero(np.diff(bits.astype(int)))) <= 1
    # tail bits of the last word are zero
    assert not np.any(P[:, 1] >> np.uint64(O - 64))


def test_sign_of_bn_output_is_a_threshold_on_the_integer_sum(oracle_mod):
    """sign(fmaf(acc, scale, shift)) is monotone in the integer acc (the exact value is, and rounding keeps order), so for
    every channel the sums that give bit 1 form a prefix (scale > 0), a suffix (scale < 0), everything or nothing --
    also for zero, infinite and NaN parameters.  The GPU's fused epilogue relies on it; here it is checked on the oracle
    for every integer in [-K, K]."""
    o = oracle_mod
    K = 600
    rng = np.random.default_rng(3)
    scale = np.concatenate([rng.uniform(-2, 2, 40), [0.0, -0.0, np.inf, -np.inf, np.nan, 1e-30, -1e30, 1.0, -1.0, 0.5]]).astype(np.float32)
    shift = np.concatenate([rng.normal(0, 200, 40), [1.0, -1.0, 5.0, 5.0, 0.0, -1e-31, 1e29, -7.0, -7.0, np.nan]]).astype(np.float32)
    O = scale.size
    acc = np.repeat(np.arange(-K, K + 1, dtype=np.int32)[:, None], O, axis=1).reshape(2 * K + 1, 1, 1, O)
    words = o.bn_sign_pack(acc, scale, shift).reshape(2 * K + 1, -1)
    bits = np.stack([(words[:, c >> 6] >> np.uint64(c & 63)) & np.uint64(1) for c in range(O)], axis=1).astype(np.int8)
    for c in range(O):
        col = bits[:, c]
        changes = np.count_nonzero(np.diff(col))
        assert changes <= 1, (c, scale[c], shift[c])
        if changes == 1:  # a prefix of ones for an increasing y, a suffix for a decreasing one
            assert (col[0] == 1) == (scale[c] > 0), (c, scale[c], shift[c])
    # and the bit is what a direct evaluation in fp64 says wherever that is unambiguous (|y| well away from zero)
    with np.errstate(invalid="ignore"):  # 0 * inf and inf - inf are NaN on purpose
        y = acc.reshape(2 * K + 1, O).astype(np.float64) * scale.astype(np.float64) + shift.astype(np.float64)
    clear = np.isfinite(y) & (np.abs(y) > 1e-3 * (np.abs(shift.astype(np.float64)) + 1))
    assert np.array_equal(bits[clear], (y[clear] < 0).astype(np.int8))


def round_to_fp32(v: Fraction) -> float:
    """Round-to-nearest-even of an exact rational to IEEE binary32 (normal and subnormal range), by integer arithmetic."""
    if v == 0:
        return 0.0
    s, a = (-1 if v < 0 else 1), abs(v)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    assert Fraction(2) ** e <= a < Fraction(2) ** (e + 1)
    ulp = Fraction(2) ** (max(e, -126) - 23)
    q = a / ulp
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    out = n * ulp
    assert out < Fraction(2) ** 128
    return s * float(out)  # exactly representable as a double


def test_round_to_fp32_helper_on_known_values():
    assert round_to_fp32(Fraction(1, 3)) == float(np.float32(1.0) / np.float32(3.0))
    assert round_to_fp32(Fraction(16777217)) == 16777216.0           # tie -> even
    assert round_to_fp32(Fraction(16777219)) == 16777220.0           # tie -> even, upwards
    assert round_to_fp32(Fraction(-5, 2) ** 31) == float(np.float32(float(Fraction(-5, 2) ** 31)))
    assert round_to_fp32(Fraction(1, 2 ** 149)) == float(np.float32(1.4e-45))


def test_block_epilogue_is_one_fma_then_one_rounded_add(oracle_mod):
    """y = RN(RN(acc*scale + shift) + r) with RN = round-to-nearest-even to fp32, from exact fractions: a contracted or
    double-precision evaluation, a missing shortcut term or a swapped operand gives different bits somewhere in 9000 values."""
    o = oracle_mod
    rng = np.random.default_rng(11)
    npix, O, K = 120, 75, 1152
    acc = (rng.integers(0, K + 1, (npix, 1, 1, O)) * 2 - K).astype(np.int32)
    scale = rng.uniform(-1.5, 1.5, O).astype(np.float32)
    shift = rng.normal(0, 3.0, O).astype(np.float32)
    r = (rng.standard_normal((npix, 1, 1, O)) * 20).astype(np.float32)
    # make some sums cancel (y exactly zero or a tiny difference of large terms)
    scale[0], shift[0] = 1.0, 0.0
    r[:, 0, 0, 0] = -acc[:, 0, 0, 0].astype(np.float32)
    r[::7, 0, 0, 1] = 0.0
    y, bits = o.bn_add_sign_pack(acc, scale, shift, r)
    assert y.shape == acc.shape and y.dtype == np.float32 and bits.shape == (npix, 1, 1, 2)
    for p in range(npix):
        for c in range(O):
            bn = round_to_fp32(Fraction(int(acc[p, 0, 0, c])) * Fraction(float(scale[c])) + Fraction(float(shift[c])))
            want = round_to_fp32(Fraction(bn) + Fraction(float(r[p, 0, 0, c])))
            assert float(y[p, 0, 0, c]) == want, (p, c)
            bit = int((bits[p, 0, 0, c >> 6] >> np.uint64(c & 63)) & np.uint64(1))
            assert bit == (1 if want < 0 else 0)
    assert np.all(y[:, 0, 0, 0] == 0.0) and not np.any(bits[:, 0, 0, 0] & np.uint64(1))  # exact zero packs as +1
    assert not np.any(bits[..., 1] >> np.uint64(O - 64))                                  # tail bits zero
    # without a shortcut it is the plain fused BN + sign
    y0, bits0 = o.bn_add_sign_pack(acc, scale, shift, np.zeros_like(r))
    assert np.array_equal(bits0, o.bn_sign_pack(acc, scale, shift))


def test_bitcount_of_eq1_counts_set_bits(oracle_mod):
    o = oracle_mod
    rng = np.random.default_rng(12)
    words = [0, 1, 2 ** 63, 2 ** 64 - 1, 0xAAAAAAAAAAAAAAAA, 0x5555555555555555, 0x8000000000000001, 0xFFFFFFFF00000000]
    words += [int(v) for v in rng.integers(0, 2 ** 63, 200)] + [int(v) | 2 ** 63 for v in rng.integers(0, 2 ** 63, 50)]
    for v in words:
        assert o.bitcount(v) == bin(v).count("1"), hex(v)
