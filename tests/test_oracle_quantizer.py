"""Pins for the oracle's number formats and quantizer (no GPU).

Each test checks the oracle against something other than itself: numpy's IEEE
fp16, exact rational arithmetic, or a property the mathematics fixes.
"""
from fractions import Fraction

import numpy as np
import pytest

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import synth


ALL_BITS = np.arange(65536, dtype=np.uint16)
ALL_HALF = ALL_BITS.view(np.float16)


def test_half_to_double_all_patterns_match_numpy():
    ref = ALL_HALF.astype(np.float64)
    got = np.array([orc.half_to_double(int(b)) for b in ALL_BITS])
    nan = np.isnan(ref)
    assert np.array_equal(np.isnan(got), nan)
    assert np.array_equal(got[~nan], ref[~nan])
    assert np.array_equal(np.signbit(got[~nan]), np.signbit(ref[~nan]))


def test_double_to_half_matches_numpy_rne():
    rng = np.random.default_rng(1)
    finite = ALL_HALF[np.isfinite(ALL_HALF)].astype(np.float64)
    # every representable value, every midpoint between neighbours (the tie cases), and noise
    srt = np.sort(finite)
    mids = (srt[:-1] + srt[1:]) / 2.0
    near = mids * (1 + rng.choice([-1e-12, 1e-12], size=mids.size))
    rand = np.concatenate([rng.normal(0, s, 4000) for s in (1e-7, 1e-4, 1.0, 3e3, 4e4)])
    edge = np.array([65504.0, 65519.999, 65520.0, 65536.0, 1e9, -65520.0, 2.0 ** -24, 2.0 ** -25,
                     2.0 ** -25 * 1.0000001, 0.0, -0.0, np.inf, -np.inf])
    x = np.concatenate([finite, mids, near, rand, edge])
    with np.errstate(over="ignore"):
        ref = x.astype(np.float16).view(np.uint16)
    got = np.array([orc.double_to_half(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, ref)


def _exact_code(v: Fraction, inv: Fraction) -> int:
    """Nearest integer to v*inv with ties to even, in exact rational arithmetic."""
    p = v * inv
    fl = p.numerator // p.denominator
    rem = p - fl
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and fl % 2 == 1):
        fl += 1
    return fl


def _exact_codes_int64(X: np.ndarray, inv32: np.float32) -> np.ndarray:
    """Nearest integer (ties to even) to x * inv for every fp16 x, in exact integer arithmetic: x = mx * 2^ex
    and inv = mi * 2^ei with integer mantissas (11 and 24 bits), so the product is the 35-bit integer mx * mi
    times a power of two, and the rounding is a shift with an explicit look at the bits shifted out."""
    m, e = np.frexp(X.astype(np.float64))
    mx = np.rint(m * 2048.0).astype(np.int64)            # exact: fp16 mantissas have at most 11 bits
    assert np.array_equal(mx.astype(np.float64) * np.exp2(e - 11.0), X.astype(np.float64))
    mi_f, ei = np.frexp(np.float64(inv32))
    mi = int(round(mi_f * 2.0 ** 24))
    assert mi * 2.0 ** (int(ei) - 24) == float(inv32)
    n = np.abs(mx) * mi                                   # |product| = n * 2^sh
    sh = (e.astype(np.int64) - 11) + (int(ei) - 24)
    out = np.zeros(X.shape, np.int64)
    up = sh >= 0
    out[up] = n[up] << np.minimum(sh[up], 20)             # far beyond the clamp either way
    dn = ~up
    s = np.minimum(-sh[dn], 62)                           # n < 2^35: anything shifted further is 0 with a small remainder
    fl = n[dn] >> s
    rem = n[dn] - (fl << s)
    half = np.int64(1) << (s - 1)
    fl = fl + ((rem > half) | ((rem == half) & (fl % 2 == 1)))
    out[dn] = fl
    return np.where(mx < 0, -out, out)


@pytest.mark.parametrize("scale", [0.03125, 0.0371, 1.0 / 127.0, 0.4321, 3.0e-4])
def test_act_codes_all_fp16_patterns_vs_exact_rationals(scale):
    finite = np.isfinite(ALL_HALF)
    X = ALL_HALF[finite]
    got = orc.quantize_acts(X, np.float32(scale), 8)
    inv32 = np.float32(1.0) / np.float32(scale)          # numpy's IEEE fp32 divide
    # every finite pattern, in exact integer arithmetic
    want = np.clip(_exact_codes_int64(X, inv32), -127, 127)
    assert np.array_equal(got.astype(np.int64), want)
    # and the integer routine itself against Python rationals on a strided sample
    inv = Fraction(float(inv32))
    for i in range(0, X.size, 97):
        q = max(-127, min(127, _exact_code(Fraction(float(X[i])), inv)))
        assert int(want[i]) == q, (float(X[i]), scale)


def test_act_codes_ties_round_to_even():
    # scale 0.5 => inv = 2; x = 0.25 -> 0.5 -> 0 ; 0.75 -> 1.5 -> 2 ; 1.25 -> 2.5 -> 2 ; -0.75 -> -2
    X = np.array([0.25, 0.75, 1.25, 1.75, -0.25, -0.75, -1.25], np.float16)
    got = orc.quantize_acts(X, np.float32(0.5), 8)
    assert got.tolist() == [0, 2, 2, 4, 0, -2, -2]


def test_act_codes_clamp_to_restricted_range():
    X = np.array([1000.0, -1000.0, 63.5, -63.6, 65504.0, -65504.0], np.float16)
    got = orc.quantize_acts(X, np.float32(0.5), 8)
    assert got.tolist() == [127, -127, 127, -127, 127, -127]


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("symmetric", [True, False])
def test_weight_quant_error_bound_extremes_and_idempotence(bits, symmetric):
    W = synth.normal_f16((48, 200), 0.02, seed=11 + bits)
    W[3, :] = 0                      # degenerate row
    W[4, :] = np.float16(0.0123)     # constant positive row
    W[5, :] = -np.abs(W[5, :])       # all-negative row
    scale, zero = orc.weight_minmax_params(W, bits, symmetric)
    codes = orc.quantize_weights(W, bits, scale, None if symmetric else zero)
    deq = orc.dequantize_weights(codes, scale, None if symmetric else zero)
    w = W.astype(np.float64)
    s = scale.astype(np.float64)[:, None]
    # |dequant - w| <= s/2, with the slack that inv = fp32(1/s) adds
    assert np.all(np.abs(deq - w) <= s * (0.5 + 2.0 ** -20) + np.abs(w) * 2.0 ** -22)
    if symmetric:
        qmax = 2 ** (bits - 1) - 1
        assert codes.min() >= -qmax and codes.max() <= qmax
        amax = np.abs(w).max(axis=1)
        for n in range(W.shape[0]):
            if amax[n] == 0:
                assert scale[n] == 1.0 and not codes[n].any()
                continue
            k = int(np.argmax(np.abs(w[n])))
            assert abs(int(codes[n, k])) == qmax
            assert scale[n] == np.float32(amax[n]) / np.float32(qmax)
        assert not zero.any()
    else:
        L = 2 ** bits - 1
        assert codes.min() >= 0 and codes.max() <= L
        for n in range(W.shape[0]):
            lo, hi = min(w[n].min(), 0.0), max(w[n].max(), 0.0)
            if hi == lo:
                assert scale[n] == 1.0 and zero[n] == 0 and not codes[n].any()
                continue
            assert scale[n] == (np.float32(hi) - np.float32(lo)) / np.float32(L)
            assert 0 <= zero[n] <= L
            if lo < 0:
                assert codes[n, int(np.argmin(w[n]))] == 0
            if hi > 0:
                assert codes[n, int(np.argmax(w[n]))] == L
            # zero is exactly representable: a zero weight maps to the zero-point
            Wz = W[n:n + 1].copy()
            Wz[0, 0] = 0
            cz = orc.quantize_weights(Wz, bits, scale[n:n + 1], zero[n:n + 1])
            assert cz[0, 0] == zero[n]
    # idempotence: quantizing the dequantized values (when they are fp16-exact) gives the codes
    deq16 = deq.astype(np.float16)
    exact = deq16.astype(np.float64) == deq
    codes2 = orc.quantize_weights(deq16, bits, scale, None if symmetric else zero)
    assert np.array_equal(codes2[exact], codes[exact])


def test_weight_codes_vs_exact_rationals_asymmetric():
    W = synth.normal_f16((6, 64), 0.02, seed=77)
    for bits in (2, 3, 4, 8):
        scale, zero = orc.weight_minmax_params(W, bits, False)
        codes = orc.quantize_weights(W, bits, scale, zero)
        L = 2 ** bits - 1
        for n in range(W.shape[0]):
            inv = Fraction(float(np.float32(1.0) / scale[n]))
            lo = min(float(W[n].astype(np.float64).min()), 0.0)
            z = max(0, min(L, _exact_code(Fraction(-lo), inv)))
            assert z == zero[n]
            for k in range(W.shape[1]):
                q = max(0, min(L, _exact_code(Fraction(float(W[n, k])), inv) + z))
                assert q == codes[n, k]


def test_sqnr_rises_six_db_per_bit():
    W = synth.normal_f16((64, 1024), 0.02, seed=5)
    w = W.astype(np.float64)
    sq = {}
    for bits in (2, 3, 4, 8):
        scale, zero = orc.weight_minmax_params(W, bits, False)
        deq = orc.dequantize_weights(orc.quantize_weights(W, bits, scale, zero), scale, zero)
        sq[bits] = 10 * np.log10((w ** 2).sum() / ((deq - w) ** 2).sum())
    assert 4.5 < sq[4] - sq[3] < 8.0
    assert 3.0 < sq[3] - sq[2] < 9.0     # a 4-level min-max grid on a Gaussian row is far from uniform-noise theory
    assert 22.0 < sq[8] - sq[4] < 26.5   # four more bits: ~24 dB


def test_act_absmax_and_scale():
    X = synth.normal_f16((5 * 77, 64), 1.0, seed=9)
    X[0, 3] = 900.0
    X[77, 5] = -800.0
    X[78, 7] = -6.5
    x = np.abs(X.astype(np.float64))
    assert orc.act_absmax(X) == np.float32(900.0)
    keep = np.arange(X.shape[0]) % 77 != 0
    assert orc.act_absmax(X, skip_rows_mod=77) == np.float32(x[keep].max())
    assert orc.act_scale(np.float32(12.7), 8) == np.float32(12.7) / np.float32(127.0)
    assert orc.act_scale(np.float32(0.0), 8) == np.float32(1.0)


# ------------------------------------------------------------------ asymmetric activations (Sec. 4.1)

def test_asym_act_params_and_codes_vs_exact_rationals():
    rng = np.random.default_rng(21)
    for shift, spread in ((0.0, 1.0), (0.7, 0.5), (-2.0, 3.0), (5.0, 0.1)):
        X = (rng.normal(shift, spread, (7, 96))).astype(np.float16)
        scale, zero = orc.act_minmax_params(X)
        x = X.astype(np.float64)
        lo, hi = min(x.min(), 0.0), max(x.max(), 0.0)
        assert scale == (np.float32(hi) - np.float32(lo)) / np.float32(255.0)
        inv = Fraction(float(np.float32(1.0) / scale))
        assert zero == max(0, min(255, _exact_code(Fraction(-lo), inv)))
        c = orc.quantize_acts_asym(X, scale, zero)
        for v, got in zip(X.ravel()[::5], c.ravel()[::5]):
            q = max(0, min(255, _exact_code(Fraction(float(v)), inv) + zero))
            assert int(got) == q - zero
        # the range is used to its ends and zero is exactly representable
        assert c.min() == -zero or lo == 0.0
        assert c.max() == 255 - zero or hi == 0.0
        assert orc.quantize_acts_asym(np.zeros(3, np.float16), scale, zero).tolist() == [0, 0, 0]
        # |x_hat - x| <= s/2 (plus the slack of inv = fp32(1/s)) for values inside the range
        xh = c.astype(np.float64) * float(scale)
        assert np.all(np.abs(xh - x) <= float(scale) * (0.5 + 2.0 ** -20) + np.abs(x) * 2.0 ** -22 + float(scale) * 0.5 * (zero in (0, 255)))


def test_asym_act_degenerate_and_clamp():
    s, z = orc.act_minmax_params(np.zeros((4, 8), np.float16))
    assert s == 1.0 and z == 0
    X = np.array([0.0, 1.0, 2.0, 300.0, -300.0], np.float16)
    c = orc.quantize_acts_asym(X, np.float32(1.0), 10)       # codes clamp to [0, 255] before centring
    assert c.tolist() == [0, 1, 2, 245, -10]


def test_asym_acts_gain_a_bit_on_one_sided_tensors():
    # post-GELU-like input (almost no negative part): the asymmetric 8-bit grid covers [lo, hi] with 255
    # steps where the symmetric one spends half of its 254 steps on values that do not occur
    rng = np.random.default_rng(5)
    X = np.maximum(rng.normal(0.0, 1.0, (64, 256)), -0.17).astype(np.float16)
    x = X.astype(np.float64)
    s, z = orc.act_minmax_params(X)
    xa = orc.quantize_acts_asym(X, s, z).astype(np.float64) * float(s)
    ss = orc.act_scale(orc.act_absmax(X), 8)
    xs = orc.quantize_acts(X, ss, 8).astype(np.float64) * float(ss)
    sq = lambda xh: 10 * np.log10((x ** 2).sum() / ((xh - x) ** 2).sum())
    assert 4.5 < sq(xa) - sq(xs) < 7.5     # about one bit = 6 dB
