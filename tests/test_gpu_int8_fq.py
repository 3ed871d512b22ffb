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
SHAPES = [(4096, 640, 640, 4), (4096, 640, 640, 8), (4096, 640, 320, 4), (1024, 640, 640, 8), (3274, 776, 432, 4),
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
    assert mixdq.linear_fused_quant_tile(1024, 640, 640, 4) == 0  # int4 at image batch 1: a tie, left as it was
