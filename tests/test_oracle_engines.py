"""Pins for the oracle's packer, integer GEMM / conv, epilogue, weight-only and BOS paths (no GPU)."""
import os

import numpy as np
import pytest

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------- packer

def _read_planes():
    out = {}
    with open(os.path.join(GOLDEN, "bitplane_words.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            name, p0, p1, p2 = line.split()
            out[name] = [int(p0, 16), int(p1, 16), int(p2, 16)]
    return out


def _planes_of(codes32):
    packed = orc.pack_codes(np.asarray(codes32, np.int16).reshape(1, 32), 3)
    return packed.view("<u4")[0].tolist()


def test_bitplane_golden_words():
    g = _read_planes()
    assert _planes_of([j % 8 for j in range(32)]) == g["jmod8"]
    assert _planes_of([7] * 32) == g["all7"]
    assert _planes_of([0] * 31 + [5]) == g["last5"]
    assert _planes_of([2] + [0] * 31) == g["first2"]


def test_two_bit_plane_words_by_hand():
    # the first two planes of the 3-bit words: a 2-bit code is a 3-bit code whose top plane is absent
    g = _read_planes()
    two = lambda codes: orc.pack_codes(np.asarray(codes, np.int16).reshape(1, 32), 2).view("<u4")[0].tolist()
    assert two([j % 4 for j in range(32)]) == g["jmod8"][:2]
    assert two([3] * 32) == g["all7"][:2]
    assert two([2] + [0] * 31) == g["first2"][:2]
    assert two([0] * 31 + [1]) == [0x80000000, 0]


def test_nibble_and_byte_layout_by_hand():
    # 4-bit: even k in the low nibble; signed codes as two's-complement nibbles
    packed = orc.pack_codes(np.array([[1, 2, -1, -8 + 1, 7]], np.int16), 4)
    assert packed[0].tolist() == [0x21, 0x9F, 0x07]
    packed = orc.pack_codes(np.array([[-127, -1, 0, 127, 255]], np.int16), 8)
    assert packed[0].tolist() == [0x81, 0xFF, 0x00, 0x7F, 0xFF]


@pytest.mark.parametrize("bits,signed", [(2, False), (3, False), (4, False), (4, True), (8, False), (8, True)])
@pytest.mark.parametrize("K", [1, 31, 32, 33, 64, 77, 320])
def test_pack_roundtrip_and_size_law(bits, signed, K):
    rng = np.random.default_rng(bits * 100 + K)
    lo, hi = (-(2 ** (bits - 1) - 1), 2 ** (bits - 1) - 1) if signed else (0, 2 ** bits - 1)
    codes = rng.integers(lo, hi + 1, size=(5, K)).astype(np.int16)
    pad = rng.integers(0, min(8, 2 ** bits), size=5).astype(np.int32)
    packed = orc.pack_codes(codes, bits, pad)
    want = {8: K, 4: (K + 1) // 2, 3: ((K + 31) // 32) * 12, 2: ((K + 31) // 32) * 8}[bits]
    assert packed.shape == (5, want)
    assert np.array_equal(orc.unpack_codes(packed, K, bits, signed), codes)
    if bits <= 3 and K % 32:
        # the ragged tail holds the pad code (the row's zero-point)
        Kp = ((K + 31) // 32) * 32
        full = orc.unpack_codes(packed, Kp, bits, False)
        assert np.array_equal(full[:, K:], np.repeat(pad[:, None], Kp - K, 1))


def test_every_value_in_every_position():
    for pos in range(32):
        for val in range(8):
            codes = np.zeros((1, 32), np.int16)
            codes[0, pos] = val
            planes = orc.pack_codes(codes, 3).view("<u4")[0]
            for p in range(3):
                assert int(planes[p]) == (((val >> p) & 1) << pos)
    for pos in range(32):
        for val in range(4):
            codes = np.zeros((1, 32), np.int16)
            codes[0, pos] = val
            planes = orc.pack_codes(codes, 2).view("<u4")[0]
            assert planes.shape == (2,)
            for p in range(2):
                assert int(planes[p]) == (((val >> p) & 1) << pos)
    for pos in range(2):
        for val in range(-7, 8):
            codes = np.zeros((1, 2), np.int16)
            codes[0, pos] = val
            b = int(orc.pack_codes(codes, 4)[0, 0])
            assert b == ((val & 0xF) << (4 * pos))


def test_storage_saving_matches_table1():
    # packed bytes of 3/4/8-bit rows are exactly K*b/8 when K is a multiple of 32, so the
    # size ratio to fp16 is 16 / average-bits: compare with the values the paper prints
    rows = np.loadtxt(os.path.join(GOLDEN, "table1_storage_opt.txt"))
    K = 1280
    for bits in (2, 3, 4, 8):
        assert orc.packed_row_bytes(K, bits) * 8 == K * bits
    for avg_bits, printed in rows:
        assert abs(16.0 / avg_bits - printed) <= 0.05 + 1e-9
    layers = synth.unet_layers()
    synth.assign_bits_weight_only(layers)
    packed = sum(l.N * orc.packed_row_bytes(l.K, l.w_bits) for l in layers)
    fp16 = sum(2 * l.params for l in layers)
    assert abs(synth.average_weight_bits(layers) - 3.66) < 0.005
    assert abs(fp16 / packed - 4.4) < 0.06        # Table 1, W3.66A16 row
    assert len(layers) == 794
    assert abs(sum(l.params for l in layers) / 1e9 - 2.566) < 0.005


# ---------------------------------------------------------- integer engines

def test_int_gemm_brute_force_python_ints():
    rng = np.random.default_rng(0)
    qx = rng.integers(-127, 128, size=(5, 37)).astype(np.int8)
    qw = rng.integers(-127, 128, size=(7, 37)).astype(np.int16)
    acc = orc.int_gemm(qx, qw)
    for m in range(5):
        for n in range(7):
            assert int(acc[m, n]) == sum(int(a) * int(b) for a, b in zip(qx[m], qw[n]))
    # transposed-operand mistakes show on non-square shapes: compare with numpy int64 too
    assert np.array_equal(acc, qx.astype(np.int64) @ qw.astype(np.int64).T)


def test_int_gemm_closed_forms():
    K = 333
    ones = np.ones((4, K), np.int8)
    assert np.all(orc.int_gemm(ones, np.ones((3, K), np.int16)) == K)
    rng = np.random.default_rng(1)
    qw = rng.integers(-7, 8, size=(6, K)).astype(np.int16)
    onehot = np.zeros((K, K), np.int8)
    np.fill_diagonal(onehot, 1)
    assert np.array_equal(orc.int_gemm(onehot, qw), qw.T.astype(np.int32))
    # worst-case magnitude stays inside int32 for the longest reduction of the UNet sweep
    K = 23040
    big = orc.int_gemm(np.full((1, K), 127, np.int8), np.full((1, K), -127, np.int16))
    assert int(big[0, 0]) == -127 * 127 * K


def _im2col(qx, stride):
    B, H, W, C = qx.shape
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    xp = np.zeros((B, H + 2, W + 2, C), qx.dtype)
    xp[:, 1:-1, 1:-1, :] = qx
    cols = np.zeros((B, Ho, Wo, 3, 3, C), qx.dtype)
    for kh in range(3):
        for kw in range(3):
            cols[:, :, :, kh, kw, :] = xp[:, kh:kh + stride * Ho:stride, kw:kw + stride * Wo:stride, :]
    return cols.reshape(B * Ho * Wo, 9 * C), (B, Ho, Wo)


@pytest.mark.parametrize("stride", [1, 2])
@pytest.mark.parametrize("H,W", [(6, 6), (5, 8), (7, 4)])
def test_int_conv_equals_gemm_on_im2col(stride, H, W):
    rng = np.random.default_rng(H * 10 + W + stride)
    qx = rng.integers(-127, 128, size=(2, H, W, 5)).astype(np.int8)
    qw = rng.integers(-127, 128, size=(4, 3, 3, 5)).astype(np.int16)
    acc = orc.int_conv3x3(qx, qw, stride)
    cols, (B, Ho, Wo) = _im2col(qx, stride)
    ref = orc.int_gemm(cols, qw.reshape(4, 45)).reshape(B, Ho, Wo, 4)
    assert acc.shape == ref.shape
    assert np.array_equal(acc, ref)


def test_int_conv_brute_force_single_outputs():
    rng = np.random.default_rng(3)
    qx = rng.integers(-127, 128, size=(1, 4, 5, 3)).astype(np.int8)
    qw = rng.integers(-7, 8, size=(2, 3, 3, 3)).astype(np.int16)
    acc = orc.int_conv3x3(qx, qw, 1)
    for ho in range(4):
        for wo in range(5):
            for n in range(2):
                s = 0
                for kh in range(3):
                    for kw in range(3):
                        hi, wi = ho + kh - 1, wo + kw - 1
                        if 0 <= hi < 4 and 0 <= wi < 5:
                            s += sum(int(qx[0, hi, wi, c]) * int(qw[n, kh, kw, c]) for c in range(3))
                assert int(acc[0, ho, wo, n]) == s


def test_int_conv_tap_counts_and_centre_kernel():
    ones = np.ones((1, 6, 7, 1), np.int8)
    acc = orc.int_conv3x3(ones, np.ones((1, 3, 3, 1), np.int16), 1)[0, :, :, 0]
    assert acc[0, 0] == 4 and acc[0, -1] == 4 and acc[-1, 0] == 4 and acc[-1, -1] == 4
    assert np.all(acc[0, 1:-1] == 6) and np.all(acc[1:-1, 0] == 6)
    assert np.all(acc[1:-1, 1:-1] == 9)
    # a kernel with only the centre tap is a 1x1 conv, i.e. a linear layer over pixels
    rng = np.random.default_rng(4)
    qx = rng.integers(-127, 128, size=(2, 5, 5, 8)).astype(np.int8)
    w11 = rng.integers(-127, 128, size=(3, 8)).astype(np.int16)
    qw = np.zeros((3, 3, 3, 8), np.int16)
    qw[:, 1, 1, :] = w11
    assert np.array_equal(orc.int_conv3x3(qx, qw, 1).reshape(-1, 3), orc.int_gemm(qx.reshape(-1, 8), w11))
    # stride 2 picks every other output of stride 1
    qw = rng.integers(-7, 8, size=(3, 3, 3, 8)).astype(np.int16)
    a1 = orc.int_conv3x3(qx, qw, 1)
    a2 = orc.int_conv3x3(qx, qw, 2)
    assert np.array_equal(a2, a1[:, ::2, ::2, :])


@pytest.mark.parametrize("stride", [1, 2])
def test_int_conv_i16_padding_is_the_zero_point(stride):
    # Explicitly padding the UNSIGNED codes with z and running a border-free brute force over the padded
    # image gives the same sums: the padded ring is the real value 0.  (Padding with code 0 would not.)
    rng = np.random.default_rng(17 + stride)
    B, H, W, Cc, N, z = 2, 6, 4, 3, 2, 93
    q = rng.integers(0, 256, size=(B, H, W, Cc))
    qw = rng.integers(-127, 128, size=(N, 3, 3, Cc)).astype(np.int16)
    acc = orc.int_conv3x3_i16((q - z).astype(np.int16), qw, stride)
    qp = np.full((B, H + 2, W + 2, Cc), z, np.int64)
    qp[:, 1:-1, 1:-1, :] = q
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    assert acc.shape == (B, Ho, Wo, N)
    for b in range(B):
        for ho in range(Ho):
            for wo in range(Wo):
                win = qp[b, ho * stride:ho * stride + 3, wo * stride:wo * stride + 3, :] - z
                for n in range(N):
                    assert int(acc[b, ho, wo, n]) == int((win * qw[n].astype(np.int64)).sum())
    # on codes that fit int8 it is the int8 engine
    c8 = rng.integers(-127, 128, size=(B, H, W, Cc)).astype(np.int8)
    assert np.array_equal(orc.int_conv3x3_i16(c8.astype(np.int16), qw, stride), orc.int_conv3x3(c8, qw, stride))


def test_a8_asym_conv_equals_linear_on_im2col():
    rng = np.random.default_rng(23)
    X = synth.one_sided_f16((2, 5, 6, 8), seed=31)
    W = synth.normal_f16((12, 72), 0.05, seed=32)
    b = synth.normal_f16((12,), 0.1, seed=33)
    ws, _ = orc.weight_minmax_params(W, 8, True)
    codes = orc.quantize_weights(W, 8, ws, None)
    sx, zx = orc.act_minmax_params(X)
    for stride in (1, 2):
        acc, y = orc.conv3x3_a8_asym(X, codes.reshape(12, 3, 3, 8), ws, sx, zx, b, stride)
        # im2col of the fp16 image (zero padding = real zeros) through the linear layer of the same scheme
        Xp = np.zeros((2, 7, 8, 8), np.float16)
        Xp[:, 1:-1, 1:-1, :] = X
        Ho, Wo = acc.shape[1:3]
        cols = np.stack([Xp[:, ho * stride:ho * stride + 3, wo * stride:wo * stride + 3, :].reshape(2, 72)
                         for ho in range(Ho) for wo in range(Wo)], axis=1).reshape(-1, 72)
        acc_l, y_l = orc.linear_a8_asym(cols, codes, ws, sx, zx, b)
        assert np.array_equal(acc.reshape(-1, 12), acc_l)
        assert np.array_equal(y.reshape(-1, 12).view(np.uint16), y_l.view(np.uint16))


# ------------------------------------------------ epilogue and layer identities

def _tol(y_ref):
    return 1e-3 * np.abs(y_ref.astype(np.float64)).max() + 1e-3


def test_epilogue_bias_only_and_scaling():
    bias = synth.normal_f16((9,), 0.01, seed=1)
    acc = np.zeros((4, 9), np.int32)
    y = orc.dequant_epilogue(acc, 0.03, np.ones(9, np.float32), bias)
    assert np.array_equal(y.view(np.uint16), np.broadcast_to(bias, (4, 9)).copy().view(np.uint16))
    acc = np.arange(36, dtype=np.int32).reshape(4, 9) - 17
    ws = np.linspace(0.001, 0.002, 9).astype(np.float32)
    y = orc.dequant_epilogue(acc, np.float32(0.05), ws, None)
    ref = (acc.astype(np.float64) * float(np.float32(0.05)) * ws.astype(np.float64)[None, :])
    assert np.array_equal(y.view(np.uint16), ref.astype(np.float16).view(np.uint16))


def test_w8a8_equals_fake_quant_matmul():
    X, W, b = synth.single_linear(seed=0, M=64, K=96, N=40)
    ws, _ = orc.weight_minmax_params(W, 8, True)
    codes = orc.quantize_weights(W, 8, ws, None)
    sx = orc.act_scale(orc.act_absmax(X), 8)
    acc, y = orc.linear_a8(X, codes, ws, sx, b)
    xq = orc.quantize_acts(X, sx, 8).astype(np.float64) * float(sx)
    wq = codes.astype(np.float64) * ws.astype(np.float64)[:, None]
    ref = xq @ wq.T + b.astype(np.float64)[None, :]
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-7)
    # and it approximates the unquantized layer to int8 accuracy
    full = X.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
    assert np.abs(y.astype(np.float64) - full).max() < 0.02 * np.abs(full).max()


def test_int_gemm_i16_brute_force_and_zero_point_identity():
    rng = np.random.default_rng(3)
    z = 77
    q = rng.integers(0, 256, size=(5, 41)).astype(np.int16)
    cx = (q - z).astype(np.int16)
    qw = rng.integers(-127, 128, size=(6, 41)).astype(np.int16)
    acc = orc.int_gemm_i16(cx, qw)
    for m in range(5):
        for n in range(6):
            assert int(acc[m, n]) == sum(int(a) * int(b) for a, b in zip(cx[m], qw[n]))
    # sum_k (q - z) w = sum_k q w - z sum_k w: the form a kernel with unsigned or re-centred codes uses
    raw = q.astype(np.int64) @ qw.astype(np.int64).T
    assert np.array_equal(acc, raw - z * qw.astype(np.int64).sum(axis=1)[None, :])
    # worst case of the longest linear reduction of the UNet stays inside int32
    K = 10240
    big = orc.int_gemm_i16(np.full((1, K), 255, np.int16), np.full((1, K), -127, np.int16))
    assert int(big[0, 0]) == -255 * 127 * K


@pytest.mark.parametrize("bits", [4, 8])
def test_a8_asym_equals_fake_quant_matmul(bits):
    rng = np.random.default_rng(11)
    X = np.maximum(rng.normal(0.3, 1.0, (48, 80)), -0.17).astype(np.float16)   # one-sided, post-GELU-like
    _, W, b = synth.single_linear(seed=2, M=8, K=80, N=24)
    ws, _ = orc.weight_minmax_params(W, bits, True)
    codes = orc.quantize_weights(W, bits, ws, None)
    sx, zx = orc.act_minmax_params(X)
    acc, y = orc.linear_a8_asym(X, codes, ws, sx, zx, b)
    xq = orc.quantize_acts_asym(X, sx, zx).astype(np.float64) * float(sx)
    wq = codes.astype(np.float64) * ws.astype(np.float64)[:, None]
    ref = xq @ wq.T + b.astype(np.float64)[None, :]
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-7)
    # a symmetric tensor with z = 0 falls back to plain signed codes: same accumulators as the int8 engine
    Xs = np.clip(synth.normal_f16((16, 80), 1.0, seed=4), -3, 3)
    c0 = orc.quantize_acts_asym(Xs, np.float32(3.0 / 127), 0)
    assert c0.min() == 0     # negative values clamp away when the zero point is 0
    if bits == 8:
        # asymmetric codes approximate the unquantized layer better than symmetric ones on this input
        full = X.astype(np.float64) @ wq.T + b.astype(np.float64)
        ss = orc.act_scale(orc.act_absmax(X), 8)
        _, ysym = orc.linear_a8(X, codes, ws, ss, b)
        ea = np.abs(y.astype(np.float64) - full).mean()
        es = np.abs(ysym.astype(np.float64) - full).mean()
        assert ea < 0.75 * es


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
def test_weight_only_equals_fake_quant_matmul(bits):
    X = synth.normal_f16((33, 70), 1.0, seed=21)
    W = synth.normal_f16((19, 70), 0.02, seed=22)
    b = synth.normal_f16((19,), 0.01, seed=23)
    s, z = orc.weight_minmax_params(W, bits, False)
    codes = orc.quantize_weights(W, bits, s, z)
    y = orc.linear_a16(X, codes, s, z, b)
    what = (codes.astype(np.float64) - z[:, None]) * s.astype(np.float64)[:, None]
    ref = X.astype(np.float64) @ what.T + b.astype(np.float64)
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-7)
    if bits == 8:
        # 8-bit weights with 16-bit activations stay within 8-bit weight error of the fp layer
        full = X.astype(np.float64) @ W.astype(np.float64).T + b.astype(np.float64)
        assert np.abs(y.astype(np.float64) - full).max() < 0.01 * np.abs(full).max()


def test_weight_only_conv_equals_linear_on_im2col():
    X = synth.normal_f16((2, 5, 6, 8), 1.0, seed=31)
    W = synth.normal_f16((7, 3, 3, 8), 0.02, seed=32)
    s, z = orc.weight_minmax_params(W.reshape(7, 72), 4, False)
    codes = orc.quantize_weights(W.reshape(7, 72), 4, s, z)
    for stride in (1, 2):
        y = orc.conv3x3_a16(X, codes.reshape(7, 3, 3, 8), s, z, None, stride)
        cols, (B, Ho, Wo) = _im2col(X, stride)
        ref = orc.linear_a16(cols, codes, s, z, None).reshape(B, Ho, Wo, 7)
        d = np.abs(y.astype(np.float64) - ref.astype(np.float64))
        assert d.max() <= 2.0 ** -10 * np.abs(ref.astype(np.float64)).max()


def test_a8_conv_equals_linear_on_im2col():
    X = synth.normal_f16((2, 6, 5, 16), 1.0, seed=41)
    W = synth.normal_f16((5, 3, 3, 16), 0.02, seed=42)
    ws, _ = orc.weight_minmax_params(W.reshape(5, -1), 4, True)
    codes = orc.quantize_weights(W.reshape(5, -1), 4, ws, None)
    sx = orc.act_scale(orc.act_absmax(X), 8)
    acc, y = orc.conv3x3_a8(X, codes.reshape(5, 3, 3, 16), ws, sx, None, 1)
    cols, (B, Ho, Wo) = _im2col(X, 1)
    acc2, y2 = orc.linear_a8(cols, codes, ws, sx, None)
    assert np.array_equal(acc.reshape(-1, 5), acc2)
    assert np.array_equal(y.reshape(-1, 5).view(np.uint16), y2.view(np.uint16))


# ------------------------------------------------------- shortcut-splitting (Sec. 4.1)

def _concat_input(M, C_lo, C_hi, seed, ratio=12.0):
    """[hidden | skip]: two tensors of very different ranges side by side."""
    lo = synth.normal_f16((M, C_lo), 1.0, seed=seed)
    hi = synth.normal_f16((M, C_hi), 1.0 / ratio, seed=seed + 1)
    return np.concatenate([lo, hi], axis=1)


def test_split_epilogue_by_hand_and_reduction_to_unsplit():
    a = np.array([[100, -3]], np.int32)
    b = np.array([[7, 50]], np.int32)
    ws = np.array([0.5, 2.0], np.float32)
    y = orc.dequant_epilogue_split(a, b, 0.25, 0.125, ws, np.array([1.0, -1.0], np.float16))
    # (100*0.25 + 7*0.125)*0.5 + 1 = 13.9375 ; (-3*0.25 + 50*0.125)*2 - 1 = 10
    assert y.astype(np.float64).tolist() == [[13.9375, 10.0]]
    # equal scales: the split layer is the unsplit one, accumulators and outputs
    X, W, bias = synth.single_linear(seed=9, M=40, K=96, N=24)
    ws, _ = orc.weight_minmax_params(W, 8, True)
    codes = orc.quantize_weights(W, 8, ws, None)
    sx = orc.act_scale(orc.act_absmax(X), 8)
    acc, y = orc.linear_a8(X, codes, ws, sx, bias)
    a_lo, a_hi, ys = orc.linear_a8_split(X, codes, ws, sx, sx, 32, bias)
    assert np.array_equal(a_lo.astype(np.int64) + a_hi, acc)
    assert np.abs(ys.astype(np.float64) - y.astype(np.float64)).max() <= 2.0 ** -10 * np.abs(y.astype(np.float64)).max()


@pytest.mark.parametrize("bits", [4, 8])
def test_split_linear_equals_fake_quant_matmul_and_gains(bits):
    X = _concat_input(64, 80, 48, seed=50)
    _, W, b = synth.single_linear(seed=3, M=8, K=128, N=40)
    ws, _ = orc.weight_minmax_params(W, bits, True)
    codes = orc.quantize_weights(W, bits, ws, None)
    s_lo = orc.act_scale(orc.act_absmax(X[:, :80]), 8)
    s_hi = orc.act_scale(orc.act_absmax(X[:, 80:]), 8)
    a_lo, a_hi, y = orc.linear_a8_split(X, codes, ws, s_lo, s_hi, 80, b)
    # brute force of one accumulator pair
    q = np.concatenate([orc.quantize_acts(X[:, :80], s_lo, 8), orc.quantize_acts(X[:, 80:], s_hi, 8)], axis=1)
    assert int(a_lo[5, 7]) == sum(int(q[5, k]) * int(codes[7, k]) for k in range(80))
    assert int(a_hi[5, 7]) == sum(int(q[5, k]) * int(codes[7, k]) for k in range(80, 128))
    xq = np.concatenate([q[:, :80] * float(s_lo), q[:, 80:] * float(s_hi)], axis=1).astype(np.float64)
    wq = codes.astype(np.float64) * ws.astype(np.float64)[:, None]
    ref = xq @ wq.T + b.astype(np.float64)
    assert np.all(np.abs(y.astype(np.float64) - ref) <= 2.0 ** -10 * np.abs(ref) + 1e-7)
    if bits == 8:
        # one scale over the concatenation leaves the small-range half with a few levels only
        full = X.astype(np.float64) @ wq.T + b.astype(np.float64)
        s_all = orc.act_scale(orc.act_absmax(X), 8)
        _, y1 = orc.linear_a8(X, codes, ws, s_all, b)
        e_split = np.abs(y.astype(np.float64) - full).mean()
        e_one = np.abs(y1.astype(np.float64) - full).mean()
        # rounding noise per element ~ step^2 / 12: the hi half's step shrinks 12x, the lo half's stays
        predicted = np.sqrt((80 + 48 / 12.0 ** 2) / 128)
        assert abs(e_split / e_one - predicted) < 0.08


@pytest.mark.parametrize("stride", [1, 2])
def test_split_conv_equals_split_linear_on_im2col(stride):
    B, H, W_, C_lo, C_hi, N = 2, 5, 6, 16, 8, 10
    X = _concat_input(B * H * W_, C_lo, C_hi, seed=60).reshape(B, H, W_, C_lo + C_hi)
    Wt = synth.normal_f16((N, 3, 3, C_lo + C_hi), 0.05, seed=61)
    b = synth.normal_f16((N,), 0.1, seed=62)
    ws, _ = orc.weight_minmax_params(Wt.reshape(N, -1), 8, True)
    codes = orc.quantize_weights(Wt.reshape(N, -1), 8, ws, None).reshape(N, 3, 3, C_lo + C_hi)
    s_lo = orc.act_scale(orc.act_absmax(X[..., :C_lo].reshape(-1, C_lo)), 8)
    s_hi = orc.act_scale(orc.act_absmax(X[..., C_lo:].reshape(-1, C_hi)), 8)
    a_lo, a_hi, y = orc.conv3x3_a8_split(X, codes, ws, s_lo, s_hi, C_lo, b, stride)
    # im2col with the columns regrouped as [all lo channels of the 9 taps | all hi channels]
    Xp = np.zeros((B, H + 2, W_ + 2, C_lo + C_hi), np.float16)
    Xp[:, 1:-1, 1:-1, :] = X
    Ho, Wo = a_lo.shape[1:3]
    win = np.stack([Xp[:, ho * stride:ho * stride + 3, wo * stride:wo * stride + 3, :]
                    for ho in range(Ho) for wo in range(Wo)], axis=1)          # [B, Ho*Wo, 3, 3, C]
    cols = np.concatenate([win[..., :C_lo].reshape(B * Ho * Wo, -1), win[..., C_lo:].reshape(B * Ho * Wo, -1)], axis=1)
    wcols = np.concatenate([codes[..., :C_lo].reshape(N, -1), codes[..., C_lo:].reshape(N, -1)], axis=1)
    l_lo, l_hi, y_l = orc.linear_a8_split(cols, wcols, ws, s_lo, s_hi, 9 * C_lo, b)
    assert np.array_equal(a_lo.reshape(-1, N), l_lo) and np.array_equal(a_hi.reshape(-1, N), l_hi)
    assert np.array_equal(y.reshape(-1, N).view(np.uint16), y_l.view(np.uint16))


# ----------------------------------------------------------------------- BOS

def _sqnr(ref, y):
    ref = ref.astype(np.float64)
    return 10 * np.log10((ref ** 2).sum() / ((y.astype(np.float64) - ref) ** 2).sum())


def test_bos_aware_kv():
    B, N = 2, 48
    E = synth.text_embedding(B, seed=4000)
    W = synth.kv_weight(N, seed=4100)
    ws, _ = orc.weight_minmax_params(W, 8, True)
    codes = orc.quantize_weights(W, 8, ws, None)
    bos = orc.bos_row(E[0, 0], W)
    sx = orc.crossattn_act_scale(E)
    acc, y = orc.crossattn_kv(E, codes, ws, sx, bos)
    # row 0 of every prompt is the stored vector, bit for bit
    for b in range(B):
        assert np.array_equal(y[b, 0].view(np.uint16), bos.view(np.uint16))
    # the stored row is the fp projection of the BOS embedding
    ref0 = E[0, 0].astype(np.float64) @ W.astype(np.float64).T
    assert np.abs(bos.astype(np.float64) - ref0).max() <= 2.0 ** -10 * np.abs(ref0).max()
    # the range ignores token 0 ...
    rest = np.abs(E[:, 1:, :].astype(np.float64)).max()
    assert sx == np.float32(rest) / np.float32(127.0)
    # ... and nothing in rows >= 1 depends on what token 0 holds
    E2 = E.copy()
    E2[:, 0, :] = np.float16(1234.0)
    assert orc.crossattn_act_scale(E2) == sx
    acc2, y2 = orc.crossattn_kv(E2, codes, ws, sx, bos)
    assert np.array_equal(acc, acc2) and np.array_equal(y.view(np.uint16), y2.view(np.uint16))
    # quantizing with token 0 inside the range costs about 20*log10(range ratio) dB on the others
    full = E[:, 1:, :].astype(np.float64).reshape(-1, E.shape[-1]) @ W.astype(np.float64).T
    s_naive = orc.act_scale(orc.act_absmax(E), 8)
    _, y_naive = orc.linear_a8(np.ascontiguousarray(E[:, 1:, :]).reshape(-1, E.shape[-1]), codes, ws,
                               s_naive, None)
    gain = _sqnr(full, y[:, 1:, :].reshape(-1, N)) - _sqnr(full, y_naive)
    expect = 20 * np.log10(float(s_naive) / float(sx))
    assert expect > 15.0
    # weight quantization noise is common to both, so the gain falls a little short of the ratio
    assert expect - 6.0 < gain < expect + 1.0
