"""The stated benchmark configurations, verbatim, at full size and whole-tensor against the oracle:

* the weight-only mixed bit-width trio (W3 320->320, W4 320->1280, W8 1280->320, asymmetric per-channel
  weights, fp16 activations) on 4096 tokens and on 16;
* the mid-level transformer FFN in W4A8 and W8A8: GEGLU projection 1280 -> 10240 on an input with 1 % of
  its channels scaled x20, the harness's GEGLU, then 5120 -> 1280, at image batch 1 and 4.  The second
  GEMM's input is the GEGLU of the ORACLE's first output on both sides, so that the two implementations
  see identical tensors at every step;
* the BOS-aware cross-attention K and V projections (2048 -> 640 and 2048 -> 1280, W8A8) at prompt batch
  1 and 8.

int32 accumulators bit-exact, fp16 outputs within the path's tolerance."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("idx", [0, 1, 2])
@pytest.mark.parametrize("M", [4096, 16])
def test_weight_only_trio_as_stated(idx, M):
    X, W, b, bits = synth.weight_only_layer(idx, M)
    N = W.shape[0]
    s_ref, z_ref, codes = oracle_weights(W, bits, False)
    y_ref = orc.linear_a16(X, codes, s_ref, z_ref, b)
    s, z, packed = device_weights(W, bits, False)
    st = status_word()
    y = mixdq.linear(dev(X), packed, N, bits, s, z, 16, None, dev(b), None, st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert_close(host(y), y_ref)


def _a8_linear_both_sides(X, W, b, bits):
    """One A8 linear layer through the oracle and through the library: checks the scale, every accumulator
    and every output, and returns the oracle's fp16 output."""
    M, K = X.shape
    N = W.shape[0]
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    acc_ref, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, b)
    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    st = status_word()
    ws = workspace_for(M, N, K, bits)
    acc = mixdq.linear_acc_i32(Xd, packed, N, bits, sx, workspace=ws, status=st)
    y = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, dev(b), workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert host(sx)[0] == sx_ref
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
    return y_ref


@pytest.mark.parametrize("B", [1, 4])
@pytest.mark.parametrize("bits", [4, 8])
def test_ffn_pair_with_outlier_channels_and_geglu(bits, B):
    X = synth.ffn_input(B, seed=3000 + B)
    # the outlier channels set the per-tensor range: most values then use a fraction of the 8-bit grid
    assert np.abs(X.astype(np.float32)).max() > 40.0
    W1 = synth.normal_f16((10240, 1280), 0.02, seed=3100)
    b1 = synth.normal_f16((10240,), 0.01, seed=3101)
    W2 = synth.normal_f16((1280, 5120), 0.02, seed=3102)
    b2 = synth.normal_f16((1280,), 0.01, seed=3103)
    h_ref = _a8_linear_both_sides(X, W1, b1, bits)
    g = synth.geglu(h_ref)
    assert g.shape == (B * 256, 5120)
    _a8_linear_both_sides(g, W2, b2, bits)


@pytest.mark.parametrize("B", [1, 8])
@pytest.mark.parametrize("N", [640, 1280])
def test_bos_aware_kv_as_stated(N, B):
    E = synth.text_embedding(B, seed=4000)
    assert np.abs(E[:, 0].astype(np.float32)).max() >= 49.0 and np.abs(E[:, 1:].astype(np.float32)).max() < 8.0
    W = synth.kv_weight(N, seed=4200 + N)
    s_ref, _, codes = oracle_weights(W, 8, True)
    bos = orc.bos_row(E[0, 0], W)
    sx_ref = orc.crossattn_act_scale(E)
    acc_ref, y_ref = orc.crossattn_kv(E, codes, s_ref, sx_ref, bos)
    Ed = dev(E)
    s, _, packed = device_weights(W, 8, True)
    sx = mixdq.act_scale(Ed.reshape(-1, E.shape[-1]), skip_rows_mod=77)
    st = status_word()
    ws = workspace_for(B * 76, N, 2048, 8)
    acc = mixdq.crossattn_kv_acc_i32(Ed, packed, N, 8, sx, workspace=ws, status=st)
    y = host(mixdq.crossattn_kv(Ed, packed, N, 8, s, sx, dev(bos), workspace=ws, status=st))
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert host(sx)[0] == sx_ref
    assert np.array_equal(host(acc), acc_ref)
    for p in range(B):
        assert np.array_equal(y[p, 0].view(np.uint16), bos.view(np.uint16))
    assert_close(y, y_ref)
