"""GPU parity of the W8A8 / W4A8 linear path with asymmetric per-tensor activations (Sec. 4.1):
range, parameters, weight code sums and int32 accumulators bit-exact, fp16 outputs within tolerance."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import (assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for)

pytestmark = pytest.mark.gpu


def _run(X, W, b, bits):
    M, K = X.shape
    N = W.shape[0]
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref, zx_ref = orc.act_minmax_params(X)
    acc_ref, y_ref = orc.linear_a8_asym(X, codes, s_ref, sx_ref, zx_ref, b)

    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sums = mixdq.weight_code_sums(packed, N, K, bits)
    assert np.array_equal(host(sums), codes.astype(np.int64).sum(axis=1))
    mm = host(mixdq.act_minmax(Xd))
    x64 = X.astype(np.float64)
    assert mm[0] == min(x64.min(), 0.0) and mm[1] == max(x64.max(), 0.0)
    sx, zx = mixdq.act_asym_params(Xd)
    assert host(sx)[0] == sx_ref and int(host(zx)[0]) == zx_ref
    st = status_word()
    ws = workspace_for(M, N, K, bits)
    acc = mixdq.linear_a8_asym_acc_i32(Xd, packed, N, bits, sums, sx, zx, workspace=ws, status=st)
    y = mixdq.linear_a8_asym(Xd, packed, N, bits, s, sums, sx, zx, None if b is None else dev(b), workspace=ws,
                             status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
    return zx_ref


# one tile per CTA (ragged), cluster split of the reduction, persistent 128- and 256-wide tiles
SHAPES = [(64, 16, 16), (77, 336, 200), (300, 320, 328), (136, 2064, 520),
          (256, 5120, 320), (16, 2560, 1300),
          (2048, 272, 1288), (4096, 384, 1280), (6144, 640, 1536)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_linear_asym_post_gelu_input(bits, M, K, N):
    X = synth.one_sided_f16((M, K), seed=M + K + 11)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 12)
    b = synth.normal_f16((N,), 0.01, seed=N + 2)
    z = _run(X, W, b, bits)
    assert 0 < z < 40     # almost all of the grid lies on the positive side


@pytest.mark.parametrize("bits", [8, 4])
def test_linear_asym_shifted_and_symmetric_inputs(bits):
    M, K, N = 300, 640, 264
    W = synth.normal_f16((N, K), 0.02, seed=5)
    base = synth.normal_f16((M, K), 1.0, seed=6)
    for shift in (0.0, 2.5, -1.0):
        X = (base.astype(np.float32) + shift).astype(np.float16)
        _run(X, W, None, bits)


@pytest.mark.parametrize("bits", [8, 4])
def test_linear_asym_zero_point_at_the_ends(bits):
    # a non-negative tensor has zero-point 0, a non-positive one 255: the largest corrections, of both signs
    M, K, N = 200, 1040, 136
    W = synth.normal_f16((N, K), 0.02, seed=8)
    Xp = np.abs(synth.normal_f16((M, K), 1.0, seed=9))
    assert _run(Xp, W, None, bits) == 0
    assert _run(-Xp, W, None, bits) == 255
    # weights of one sign make the code sums as large as they get
    assert _run(Xp, np.abs(W), None, bits) == 0


def test_linear_asym_all_zero_input_gives_the_bias():
    M, K, N = 130, 256, 72
    W = synth.normal_f16((N, K), 0.02, seed=3)
    b = synth.normal_f16((N,), 0.5, seed=4)
    X = np.zeros((M, K), np.float16)
    # stored codes are all -128 and the zero-point term cancels them: what is left is the bias
    _run(X, W, b, 8)


def test_linear_asym_needs_the_workspace():
    M, K, N = 64, 64, 64
    X = synth.one_sided_f16((M, K), seed=1)
    W = synth.normal_f16((N, K), 0.02, seed=2)
    s, _, packed = device_weights(W, 8, True)
    sums = mixdq.weight_code_sums(packed, N, K, 8)
    sx, zx = mixdq.act_asym_params(dev(X))
    with pytest.raises(mixdq.MixdqError):
        mixdq.linear_a8_asym(dev(X), packed, N, 8, s, sums, sx, zx)


# ----------------------------------------------------------------------------- 3x3 convolution

def _run_conv(X, Wt, b, bits, stride):
    B, H, W, Cin = X.shape
    Cout = Wt.shape[0]
    s_ref, _, codes = oracle_weights(Wt.reshape(Cout, -1), bits, True)
    sx_ref, zx_ref = orc.act_minmax_params(X)
    acc_ref, y_ref = orc.conv3x3_a8_asym(X, codes.reshape(Cout, 3, 3, Cin), s_ref, sx_ref, zx_ref, b, stride)

    Xd = dev(X)
    s, _, packed = device_weights(Wt.reshape(Cout, -1), bits, True)
    sums = mixdq.weight_code_sums(packed, Cout, 9 * Cin, bits)
    sx, zx = mixdq.act_asym_params(Xd)
    assert host(sx)[0] == sx_ref and int(host(zx)[0]) == zx_ref
    st = status_word()
    ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, H, W, Cin, Cout, stride, bits, 8))
    acc = mixdq.conv3x3_a8_asym_acc_i32(Xd, packed, Cout, bits, sums, sx, zx, stride, workspace=ws, status=st)
    y = mixdq.conv3x3_a8_asym(Xd, packed, Cout, bits, s, sums, sx, zx, None if b is None else dev(b), stride,
                              workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
    return zx_ref


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("B,H,W,Cin,Cout,stride", [(1, 16, 16, 320, 136, 1), (3, 8, 8, 32, 40, 1),
                                                    (2, 32, 32, 160, 136, 1), (1, 64, 64, 32, 24, 1),
                                                    (1, 16, 16, 640, 264, 1), (2, 16, 16, 64, 48, 2),
                                                    (1, 64, 64, 64, 40, 2), (2, 32, 32, 160, 136, 2),
                                                    # persistent kernel: 128- and 256-wide tiles
                                                    (4, 64, 64, 64, 264, 1), (5, 64, 64, 32, 512, 1)])
def test_conv3x3_asym_post_silu_input(bits, B, H, W, Cin, Cout, stride):
    X = synth.one_sided_f16((B, H, W, Cin), seed=H * W + Cin + 1)
    Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=Cout + Cin + 2)
    b = synth.normal_f16((Cout,), 0.01, seed=Cout + 3)
    assert 0 < _run_conv(X, Wt, b, bits, stride) < 40


@pytest.mark.parametrize("bits", [8, 4])
def test_conv3x3_asym_border_is_the_zero_point(bits):
    # one-signed images put the zero-point at an end of the grid, where a border filled with any other code
    # (0, or the re-centred 0) would show in every border pixel; positive weights make it add up
    Wt = np.abs(synth.normal_f16((72, 3, 3, 64), 0.02, seed=41))
    Xp = np.abs(synth.normal_f16((2, 16, 16, 64), 1.0, seed=42)) + np.float16(0.5)
    assert _run_conv(Xp, Wt, None, bits, 1) == 0
    assert _run_conv(-Xp, Wt, None, bits, 1) == 255
    assert _run_conv(-Xp, Wt, None, bits, 2) == 255


def test_conv3x3_asym_geometry_outside_the_two_kernel_path():
    B, H, W, Cin, Cout = 2, 12, 10, 32, 48
    X = synth.one_sided_f16((B, H, W, Cin), seed=1)
    Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=2)
    s, _, packed = device_weights(Wt.reshape(Cout, -1), 8, True)
    sums = mixdq.weight_code_sums(packed, Cout, 9 * Cin, 8)
    sx, zx = mixdq.act_asym_params(dev(X))
    ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, H, W, Cin, Cout, 1, 8, 8))
    with pytest.raises(mixdq.MixdqError):
        mixdq.conv3x3_a8_asym(dev(X), packed, Cout, 8, s, sums, sx, zx, workspace=ws)
