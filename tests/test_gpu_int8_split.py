"""GPU parity of shortcut-splitting (Sec. 4.1): a layer fed by a concatenation keeps one activation scale per
branch.  Both int32 sums bit-exact, fp16 outputs within tolerance, linear layers and 3x3 convolutions."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, host, status_word

pytestmark = pytest.mark.gpu


def _concat(rows, C_lo, C_hi, seed, ratio=12.0):
    """[hidden | skip]: two tensors of very different ranges side by side."""
    lo = synth.normal_f16((rows, C_lo), 1.0, seed=seed)
    hi = synth.normal_f16((rows, C_hi), 1.0 / ratio, seed=seed + 1)
    return np.concatenate([lo, hi], axis=1)


def _device_halves(W_lo, W_hi, W_all, bits):
    """Per-channel scale over the whole row, each column range packed with it."""
    s, _ = mixdq.weight_minmax_params(dev(W_all), bits, True)
    return s, mixdq.pack_weights(dev(W_lo), bits, s), mixdq.pack_weights(dev(W_hi), bits, s)


def _run_linear(M, C_lo, C_hi, N, bits, seed, bias=True, ratio=12.0):
    K = C_lo + C_hi
    X = _concat(M, C_lo, C_hi, seed, ratio)
    W = synth.normal_f16((N, K), 0.02, seed=seed + 2)
    b = synth.normal_f16((N,), 0.01, seed=seed + 3) if bias else None
    ws_ref, _ = orc.weight_minmax_params(W, bits, True)
    codes = orc.quantize_weights(W, bits, ws_ref, None)
    s_lo_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[:, :C_lo])), 8)
    s_hi_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[:, C_lo:])), 8)
    a_lo_ref, a_hi_ref, y_ref = orc.linear_a8_split(X, codes, ws_ref, s_lo_ref, s_hi_ref, C_lo, b)

    Xd = dev(X)
    s, p_lo, p_hi = _device_halves(W[:, :C_lo], W[:, C_lo:], W, bits)
    assert np.array_equal(host(s).view(np.uint32), ws_ref.view(np.uint32))
    s_lo, s_hi = mixdq.act_scale(Xd[:, :C_lo].contiguous()), mixdq.act_scale(Xd[:, C_lo:].contiguous())
    assert host(s_lo)[0] == s_lo_ref and host(s_hi)[0] == s_hi_ref
    ws = mixdq.new_workspace(mixdq.split_workspace_bytes(M, K, C_lo, M, N))
    ws.fill_(0xA5)   # the workspace needs no initial content
    st = status_word()
    a_lo, a_hi = mixdq.linear_a8_split_acc_i32(Xd, C_lo, p_lo, p_hi, N, bits, s_lo, s_hi, workspace=ws, status=st)
    y = mixdq.linear_a8_split(Xd, C_lo, p_lo, p_hi, N, bits, s, s_lo, s_hi, None if b is None else dev(b),
                              workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(a_lo), a_lo_ref) and np.array_equal(host(a_hi), a_hi_ref)
    assert_close(host(y), y_ref)
    return host(y), y_ref, X, W, b, codes, ws_ref


# one ragged tile; cluster split of the reduction; persistent kernels (128- and 256-wide tiles); unequal halves
LINEAR_SHAPES = [(64, 16, 16, 16), (77, 160, 176, 200), (300, 640, 320, 328), (256, 2560, 2560, 320),
                 (2048, 640, 640, 1288), (4096, 256, 128, 1280), (6144, 320, 320, 1536)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,C_lo,C_hi,N", LINEAR_SHAPES)
def test_split_linear_parity(bits, M, C_lo, C_hi, N):
    _run_linear(M, C_lo, C_hi, N, bits, seed=M + C_lo + N)


def test_split_linear_without_bias_and_with_odd_width():
    _run_linear(130, 48, 32, 37, 8, seed=5, bias=False)    # N % 4 != 0: scalar epilogue
    _run_linear(130, 48, 32, 36, 4, seed=6, bias=True)


def test_split_keeps_the_small_branch_resolved():
    # one scale over the concatenation leaves the small-range half with a few levels only: the split output is
    # closer to the floating-point product of the dequantized weights (same check as on the oracle)
    y, y_ref, X, W, b, codes, ws_ref = _run_linear(256, 320, 320, 320, 8, seed=21, ratio=20.0)
    wq = codes.astype(np.float64) * ws_ref.astype(np.float64)[:, None]
    full = X.astype(np.float64) @ wq.T + b.astype(np.float64)
    Xd = dev(X)
    s, _ = mixdq.weight_minmax_params(dev(W), 8, True)
    packed = mixdq.pack_weights(dev(W), 8, s)
    ws = mixdq.new_workspace(mixdq.workspace_bytes(256, 320, 640, 8, 8))
    y_one = host(mixdq.linear(Xd, packed, 320, 8, s, None, 8, mixdq.act_scale(Xd), dev(b), ws, status_word()))
    e_split = np.abs(y.astype(np.float64) - full).mean()
    e_one = np.abs(y_one.astype(np.float64) - full).mean()
    assert e_split < 0.8 * e_one


def _run_conv(B, H, W_, C_lo, C_hi, N, bits, stride, seed):
    C = C_lo + C_hi
    X = _concat(B * H * W_, C_lo, C_hi, seed).reshape(B, H, W_, C)
    Wt = synth.normal_f16((N, 3, 3, C), 0.02, seed=seed + 2)
    b = synth.normal_f16((N,), 0.01, seed=seed + 3)
    ws_ref, _ = orc.weight_minmax_params(Wt.reshape(N, -1), bits, True)
    codes = orc.quantize_weights(Wt.reshape(N, -1), bits, ws_ref, None).reshape(N, 3, 3, C)
    s_lo_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[..., :C_lo]).reshape(-1, C_lo)), 8)
    s_hi_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[..., C_lo:]).reshape(-1, C_hi)), 8)
    a_lo_ref, a_hi_ref, y_ref = orc.conv3x3_a8_split(X, codes, ws_ref, s_lo_ref, s_hi_ref, C_lo, b, stride)

    Xd = dev(X)
    W_lo = np.ascontiguousarray(Wt[..., :C_lo]).reshape(N, -1)
    W_hi = np.ascontiguousarray(Wt[..., C_lo:]).reshape(N, -1)
    s, p_lo, p_hi = _device_halves(W_lo, W_hi, Wt.reshape(N, -1), bits)
    X2 = Xd.reshape(-1, C)
    s_lo, s_hi = mixdq.act_scale(X2[:, :C_lo].contiguous()), mixdq.act_scale(X2[:, C_lo:].contiguous())
    assert host(s_lo)[0] == s_lo_ref and host(s_hi)[0] == s_hi_ref
    Ho, Wo = a_lo_ref.shape[1:3]
    ws = mixdq.new_workspace(mixdq.split_workspace_bytes(B * H * W_, C, C_lo, B * Ho * Wo, N))
    ws.fill_(0x5A)
    st = status_word()
    a_lo, a_hi = mixdq.conv3x3_a8_split_acc_i32(Xd, C_lo, p_lo, p_hi, N, bits, s_lo, s_hi, stride, ws, st)
    y = mixdq.conv3x3_a8_split(Xd, C_lo, p_lo, p_hi, N, bits, s, s_lo, s_hi, dev(b), stride, ws, st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(a_lo), a_lo_ref) and np.array_equal(host(a_hi), a_hi_ref)
    assert_close(host(y), y_ref)


# (B, H, W, C_lo, C_hi, Cout, stride): several images per tile, one tile per image row block, unequal halves
# as in the up path (1280 + 640 -> 1920 scaled down), channel tails (C % 128 != 0), stride 2
CONV_SHAPES = [(2, 8, 8, 32, 32, 48, 1), (1, 16, 16, 160, 96, 136, 1), (3, 16, 16, 256, 128, 320, 1),
               (1, 32, 32, 64, 32, 64, 1), (2, 16, 16, 64, 64, 40, 2), (1, 64, 64, 32, 64, 32, 1)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("B,H,W_,C_lo,C_hi,N,stride", CONV_SHAPES)
def test_split_conv_parity(bits, B, H, W_, C_lo, C_hi, N, stride):
    _run_conv(B, H, W_, C_lo, C_hi, N, bits, stride, seed=H + C_lo + N)


def _kb(c):
    return (c + 127) // 128


# Layers large enough for the two-CTA form run both branches in ONE kernel (an accumulator per branch in tensor
# memory, two-scale epilogue): channel counts that are no multiples of 128 (the last k-block of a tap reads past
# the branch), unequal halves, stride 2, ragged rows and columns.
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("B,H,W_,C_lo,C_hi,N,stride", [(4, 64, 64, 160, 96, 328, 1), (8, 64, 64, 96, 160, 320, 2),
                                                       (5, 32, 32, 320, 320, 648, 1)])
def test_split_conv_in_one_kernel(bits, B, H, W_, C_lo, C_hi, N, stride):
    Ho = (H - 1) // stride + 1
    rows, cols = mixdq.int8_tile_plan(B * Ho * Ho, N, 9 * (_kb(C_lo) + _kb(C_hi)), bits)
    assert rows == 256, (rows, cols)
    _run_conv(B, H, W_, C_lo, C_hi, N, bits, stride, seed=H + C_lo + N + 7)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,C_lo,C_hi,N", [(5567, 400, 384, 776), (16384, 320, 320, 320), (4458, 1296, 656, 648)])
def test_split_linear_in_one_kernel(bits, M, C_lo, C_hi, N):
    rows, cols = mixdq.int8_tile_plan(M, N, _kb(C_lo) + _kb(C_hi), bits)
    assert rows == 256, (rows, cols)
    _run_linear(M, C_lo, C_hi, N, bits, seed=M + C_lo + N + 7)


def test_split_argument_errors():
    X = dev(synth.normal_f16((64, 64), 1.0, seed=1))
    W = synth.normal_f16((32, 64), 0.02, seed=2)
    s, p_lo, p_hi = _device_halves(W[:, :32], W[:, 32:], W, 8)
    sx = mixdq.act_scale(X)
    ws = mixdq.new_workspace(mixdq.split_workspace_bytes(64, 64, 32, 64, 32))
    with pytest.raises(mixdq.MixdqError, match="workspace"):
        mixdq.linear_a8_split(X, 32, p_lo, p_hi, 32, 8, s, sx, sx, workspace=None)
    with pytest.raises(mixdq.MixdqError, match="workspace"):
        mixdq.linear_a8_split(X, 32, p_lo, p_hi, 32, 8, s, sx, sx, workspace=ws[:1024])
    with pytest.raises(mixdq.MixdqError, match="unsupported"):
        mixdq.linear_a8_split(X, 24, p_lo, p_hi, 32, 8, s, sx, sx, workspace=ws)     # not a multiple of 16
    with pytest.raises(mixdq.MixdqError, match="invalid"):
        mixdq.linear_a8_split(X, 64, p_lo, p_hi, 32, 8, s, sx, sx, workspace=ws)     # nothing on the hi side


@pytest.mark.parametrize("zero_side", ["lo", "hi"])
def test_split_with_an_all_zero_branch(zero_side):
    # a branch of zeros has the degenerate scale 1 and codes 0: its sum vanishes and the output is the other
    # branch's layer alone
    M, C_lo, C_hi, N = 200, 64, 96, 72
    X = _concat(M, C_lo, C_hi, seed=31)
    if zero_side == "lo":
        X[:, :C_lo] = 0
    else:
        X[:, C_lo:] = 0
    W = synth.normal_f16((N, C_lo + C_hi), 0.02, seed=32)
    b = synth.normal_f16((N,), 0.01, seed=33)
    ws_ref, _ = orc.weight_minmax_params(W, 8, True)
    codes = orc.quantize_weights(W, 8, ws_ref, None)
    s_lo_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[:, :C_lo])), 8)
    s_hi_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(X[:, C_lo:])), 8)
    assert (s_lo_ref if zero_side == "lo" else s_hi_ref) == np.float32(1.0)
    a_lo_ref, a_hi_ref, y_ref = orc.linear_a8_split(X, codes, ws_ref, s_lo_ref, s_hi_ref, C_lo, b)
    assert not (a_lo_ref if zero_side == "lo" else a_hi_ref).any()
    Xd = dev(X)
    s, p_lo, p_hi = _device_halves(W[:, :C_lo], W[:, C_lo:], W, 8)
    s_lo, s_hi = mixdq.act_scale(Xd[:, :C_lo].contiguous()), mixdq.act_scale(Xd[:, C_lo:].contiguous())
    assert host(s_lo)[0] == s_lo_ref and host(s_hi)[0] == s_hi_ref
    ws = mixdq.new_workspace(mixdq.split_workspace_bytes(M, C_lo + C_hi, C_lo, M, N))
    st = status_word()
    a_lo, a_hi = mixdq.linear_a8_split_acc_i32(Xd, C_lo, p_lo, p_hi, N, 8, s_lo, s_hi, workspace=ws, status=st)
    y = mixdq.linear_a8_split(Xd, C_lo, p_lo, p_hi, N, 8, s, s_lo, s_hi, dev(b), workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(a_lo), a_lo_ref) and np.array_equal(host(a_hi), a_hi_ref)
    assert_close(host(y), y_ref)
