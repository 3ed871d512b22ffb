"""GPU parity of the one-kernel form of a W8A8 / W4A8 linear layer, whose GEMM kernel quantizes its own fp16
activation tiles (Sec. 4.1: per-tensor 8-bit activations): the planner sends short reductions on one wave of
tiles there.  Every case first checks that the shape really takes that form.  int32 accumulators must match the
oracle bit for bit (whole tensor) -- any activation code that differs from the oracle's quantizer shows there --
and fp16 outputs within the path's tolerance; the stored-int8 route (quantization kernel + GEMM) must give the
same output bits."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for

pytestmark = pytest.mark.gpu

# the 32 x 32 level's attention projections at image batch 4 and 1, and ragged rows / columns / reduction tails
SHAPES = [(4096, 640, 640, 4), (4096, 640, 640, 8), (4096, 640, 320, 4), (1024, 640, 640, 8), (1024, 640, 640, 4), (3274, 776, 432, 4),
          (2100, 1000, 208, 8), (2049, 40, 16, 4), (5000, 136, 640, 8)]


def _run(X, W, b, bits, sx_ref):
    M, K = X.shape
    N = W.shape[0]
    s_ref, _, codes = oracle_weights(W, bits, True)
    acc_ref, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, b)
    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = dev(np.array([sx_ref], np.float32))
    st = status_word()
    ws = workspace_for(M, N, K, bits)
    acc = mixdq.linear_acc_i32(Xd, packed, N, bits, sx, workspace=ws, status=st)
    y = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, None if b is None else dev(b), workspace=ws, status=st)
    xq = mixdq.quantize_acts(Xd, sx)
    y_q8 = mixdq.linear_q8(xq, packed, N, bits, s, sx, None if b is None else dev(b), st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(xq), orc.quantize_acts(X, sx_ref).astype(np.int8))
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
    assert np.array_equal(host(y_q8).view(np.uint16), host(y).view(np.uint16))


@pytest.mark.parametrize("M,N,K,bits", SHAPES)
def test_linear_fused_quantization(M, N, K, bits):
    bn = mixdq.linear_fused_quant_tile(M, N, K, bits)
    assert bn > 0 and bn % 32 == 0, bn
    X = synth.normal_f16((M, K), 1.0, seed=M + K)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 1)
    b = synth.normal_f16((N,), 0.01, seed=N)
    _run(X, W, b, bits, orc.act_scale(orc.act_absmax(X), 8))


@pytest.mark.parametrize("scale", [0.0123, 2.0 ** -6, 3.3e-4, 0.9, 41.0, 3.0e-8, 700.0])
def test_every_finite_fp16_value_through_the_fused_quantizer(scale):
    """All 63488 finite fp16 bit patterns as activations, with calibrated scales that leave most of them clamped,
    none of them clamped, or lie outside the range in which the kernel clamps in fp16 (tiny and huge scales take
    its other branch): the accumulators only match if every code does."""
    bits16 = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = bits16.view(np.float16)
    vals = vals[np.isfinite(vals)]
    M, K = 2048, 32
    X = np.zeros(M * K, np.float16)
    X[: vals.size] = vals
    X[vals.size:] = vals[: M * K - vals.size]
    X = np.ascontiguousarray(X.reshape(M, K))
    N = 64
    assert mixdq.linear_fused_quant_tile(M, N, K, 8) > 0
    # weights with a single entry per row pick single codes out; the rest are random (kept small where the
    # activation scale is large, so that the fp16 outputs stay finite)
    wstd = 0.02 * min(1.0, 1.0 / scale)
    W = synth.normal_f16((N, K), wstd, seed=5)
    W[:K] = 0
    W[np.arange(K), np.arange(K)] = np.float16(50.0 * wstd)
    _run(X, W, None, 8, np.float32(scale))


def test_two_kernel_shapes_stay_two_kernel():
    for M, N, K in [(1024, 1280, 1280), (1024, 1280, 640), (16384, 320, 640), (4096, 5120, 640), (4096, 640, 2560)]:
        assert mixdq.linear_fused_quant_tile(M, N, K, 4) == 0


@pytest.mark.parametrize("bits", [4, 8])
@pytest.mark.parametrize("M,N,K,tile_cols", [(1024, 1280, 1280, 256), (1024, 1280, 1280, 96), (1000, 1288, 5136, 160),
                                             (130, 72, 48, 32), (4096, 640, 2560, 224), (777, 520, 400, 64)])
def test_explicit_one_kernel_form_equals_the_planned_path(bits, M, N, K, tile_cols):
    """mixdq_linear_a8_fused_quant on shapes the planner keeps on two kernels (long reductions, several waves,
    ragged tiles, every tile width class): the same output bits as mixdq_linear, which the other tests hold
    against the oracle, and the oracle's outputs within tolerance."""
    X = synth.normal_f16((M, K), 1.0, seed=M + K + 3)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 4)
    b = synth.normal_f16((N,), 0.01, seed=N + 5)
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    _, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, b)
    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    st = status_word()
    y_fused = mixdq.linear_a8_fused_quant(Xd, packed, N, bits, s, sx, dev(b), tile_cols, st)
    y = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, dev(b), workspace=workspace_for(M, N, K, bits), status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert_close(host(y_fused), y_ref)
    assert np.array_equal(host(y_fused).view(np.uint16), host(y).view(np.uint16))


def test_explicit_one_kernel_form_rejects_bad_arguments():
    X = dev(synth.normal_f16((128, 64), 1.0, seed=1))
    s, _, packed = device_weights(synth.normal_f16((32, 64), 0.02, seed=2), 8, True)
    sx = mixdq.act_scale(X)
    for bad in (0, 16, 48, 288):
        with pytest.raises(mixdq.MixdqError):
            mixdq.linear_a8_fused_quant(X, packed, 32, 8, s, sx, None, bad)
    X40 = dev(synth.normal_f16((128, 40), 1.0, seed=3))  # rows of 40 codes are not 16-byte multiples
    s40, _, packed40 = device_weights(synth.normal_f16((32, 40), 0.02, seed=4), 8, True)
    with pytest.raises(mixdq.MixdqError):
        mixdq.linear_a8_fused_quant(X40, packed40, 32, 8, s40, sx, None, 64)
