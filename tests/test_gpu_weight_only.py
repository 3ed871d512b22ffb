"""GPU parity of the weight-only W3/W4/W8-A16 engine against the double-precision oracle."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights

pytestmark = pytest.mark.gpu


def _run(X, W, b, bits, symmetric=False, use_ws=False):
    M, K = X.shape
    N = W.shape[0]
    s_ref, z_ref, codes = oracle_weights(W, bits, symmetric)
    y_ref = orc.linear_a16(X, codes, s_ref, z_ref, b)
    s, z, packed = device_weights(W, bits, symmetric)
    ws = mixdq.new_workspace(mixdq.workspace_bytes(M, N, K, bits, 16)) if use_ws else None
    y = mixdq.linear(dev(X), packed, N, bits, s, z, 16, None, None if b is None else dev(b), ws)
    torch.cuda.synchronize()
    assert_close(host(y), y_ref)


@pytest.mark.parametrize("idx", [0, 1, 2])
@pytest.mark.parametrize("M", [16, 200])
def test_mixed_bitwidth_trio(idx, M):
    X, W, b, bits = synth.weight_only_layer(idx, M)
    _run(X, W, b, bits)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("M,K,N", [(1, 128, 16), (5, 136, 40), (16, 1280, 96), (33, 2560, 72), (8, 4224, 48),
                                   (77, 320, 330)])
def test_ragged_shapes(bits, M, K, N):
    X = synth.normal_f16((M, K), 1.0, seed=M * 3 + K)
    W = synth.normal_f16((N, K), 0.02, seed=N * 5 + K)
    b = synth.normal_f16((N,), 0.01, seed=N)
    _run(X, W, b, bits)


# 64 tokens or more: the tensor-memory (tcgen05) form of the engine, one or several tiles per CTA
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("M,K,N", [(64, 64, 16), (300, 2880, 136), (2100, 320, 1300), (130, 200, 264), (4096, 320, 320)])
def test_many_token_shapes(bits, M, K, N):
    X = synth.normal_f16((M, K), 1.0, seed=M * 7 + K)
    W = synth.normal_f16((N, K), 0.02, seed=N * 11 + K)
    b = synth.normal_f16((N,), 0.01, seed=N + 2)
    _run(X, W, b, bits)


@pytest.mark.parametrize("bits", [4, 8])
def test_symmetric_codes_many_tokens(bits):
    X = synth.normal_f16((256, 640), 1.0, seed=3)
    W = synth.normal_f16((72, 640), 0.02, seed=4)
    _run(X, W, None, bits, symmetric=True)
    _run(X, W, None, bits, symmetric=True, use_ws=True)


# 256 tokens or more and a workspace: the weights are expanded once to fp16 integers in the workspace and a
# two-CTA tcgen05 kind::f16 GEMM reads both operands by TMA (ragged rows, columns and reduction lengths, one
# and several tiles per CTA pair)
@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("M,K,N", [(256, 64, 32), (300, 2888, 136), (2100, 328, 1300), (1000, 1288, 1290), (4096, 320, 1280),
                                   (5000, 200, 264)])
def test_many_token_shapes_with_workspace(bits, M, K, N):
    X = synth.normal_f16((M, K), 1.0, seed=M * 7 + K)
    W = synth.normal_f16((N, K), 0.02, seed=N * 11 + K)
    b = synth.normal_f16((N,), 0.01, seed=N + 2)
    _run(X, W, b, bits, use_ws=True)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("geom", [(2, 16, 16, 64, 40, 1), (1, 32, 32, 200, 136, 1), (3, 32, 32, 192, 136, 1),
                                  (2, 32, 32, 72, 264, 2), (1, 64, 64, 96, 48, 2)])
def test_weight_only_conv3x3_with_workspace(bits, geom):
    B, H, Wd, Cin, Cout, stride = geom
    X = synth.normal_f16((B, H, Wd, Cin), 1.0, seed=17)
    Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=18)
    b = synth.normal_f16((Cout,), 0.01, seed=19)
    s_ref, z_ref, codes = oracle_weights(Wt.reshape(Cout, -1), bits, False)
    y_ref = orc.conv3x3_a16(X, codes.reshape(Cout, 3, 3, Cin), s_ref, z_ref, b, stride)
    s, z, packed = device_weights(Wt.reshape(Cout, -1), bits, False)
    ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, H, Wd, Cin, Cout, stride, bits, 16))
    assert ws is not None
    y = mixdq.conv3x3(dev(X), packed, Cout, bits, s, z, 16, None, dev(b), stride, ws)
    torch.cuda.synchronize()
    assert_close(host(y), y_ref)


@pytest.mark.parametrize("bits", [4, 8])
def test_symmetric_codes_at_a16(bits):
    X = synth.normal_f16((16, 640), 1.0, seed=1)
    W = synth.normal_f16((64, 640), 0.02, seed=2)
    _run(X, W, None, bits, symmetric=True)


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("geom", [(2, 6, 5, 32, 40, 1), (2, 6, 5, 32, 40, 2), (2, 16, 16, 64, 40, 1),
                                  (1, 8, 8, 128, 48, 1), (3, 32, 32, 192, 136, 1)])
def test_weight_only_conv3x3(bits, geom):
    B, H, Wd, Cin, Cout, stride = geom
    X = synth.normal_f16((B, H, Wd, Cin), 1.0, seed=7)
    Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=8)
    b = synth.normal_f16((Cout,), 0.01, seed=9)
    s_ref, z_ref, codes = oracle_weights(Wt.reshape(Cout, -1), bits, False)
    y_ref = orc.conv3x3_a16(X, codes.reshape(Cout, 3, 3, Cin), s_ref, z_ref, b, stride)
    s, z, packed = device_weights(Wt.reshape(Cout, -1), bits, False)
    y = mixdq.conv3x3(dev(X), packed, Cout, bits, s, z, 16, None, dev(b), stride)
    torch.cuda.synchronize()
    assert_close(host(y), y_ref)
