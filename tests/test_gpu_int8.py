"""GPU parity of the W8A8 / W4A8 engine: int32 accumulators bit-exact, fp16 outputs within
the path's tolerance, on linear layers, the BOS-aware K/V projection and 3x3 convs."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import (assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for)

pytestmark = pytest.mark.gpu


def _run_linear(X, W, b, bits, use_ws):
    M, K = X.shape
    N = W.shape[0]
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    acc_ref, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, b)

    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    assert host(sx)[0] == sx_ref
    st = status_word()
    ws = workspace_for(M, N, K, bits) if use_ws else None
    acc = mixdq.linear_acc_i32(Xd, packed, N, bits, sx, workspace=ws, status=st)
    y = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, None if b is None else dev(b), workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)



@pytest.mark.parametrize("use_ws", [False, True])
def test_single_linear_w8a8_seed0(use_ws):
    X, W, b = synth.single_linear(seed=0)
    _run_linear(X, W, b, 8, use_ws)


# without a workspace the fused kernel runs; with one, layers of 64 rows or more take the
# quantize-once + TMA-fed GEMM pair (128- or 256-wide tiles, cluster split of the reduction)
@pytest.mark.parametrize("use_ws", [False, True])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N", [(1, 16, 16), (77, 336, 200), (300, 320, 328), (129, 1040, 136), (256, 2048, 24),
                                   (200, 272, 1032), (136, 2064, 520)])
def test_linear_ragged_tiles(bits, M, K, N, use_ws):
    g = synth.normal_f16((M, K), 1.0, seed=M + K)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 1)
    b = synth.normal_f16((N,), 0.01, seed=N)
    _run_linear(g, W, b, bits, use_ws)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N", [(256, 5120, 320), (130, 1280, 200), (512, 4096, 136), (40, 4096, 136),
                                   (16, 2560, 1300), (256, 5120, 1280)])
def test_linear_split_reduction(bits, M, K, N):
    g = synth.normal_f16((M, K), 1.0, seed=M + K + 7)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 8)
    _run_linear(g, W, None, bits, True)
    _run_linear(g, W, None, bits, True)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N", [(2048, 272, 1288), (4100, 144, 1290), (2500, 1040, 1032),
                                   # three tiles per CTA with an odd number of k-blocks: ring slots and MMA
                                   # issuers must stay in step across tile boundaries
                                   (4096, 384, 1280), (6144, 640, 1536)])
def test_linear_persistent_tiles(bits, M, K, N):
    # at least as many output tiles as SMs: the persistent kernel walks several tiles per CTA
    g = synth.normal_f16((M, K), 1.0, seed=M + K + 3)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 4)
    b = synth.normal_f16((N,), 0.01, seed=N + 1)
    _run_linear(g, W, b, bits, True)


def test_one_workspace_shared_by_different_layers():
    # a model keeps one scratch buffer for all its layers: whatever a layer leaves in it (its int8
    # activations, partial sums) must not disturb the next one, whichever engine that one uses
    lin = (synth.normal_f16((512, 4096), 1.0, 21), synth.normal_f16((136, 4096), 0.02, 22))
    cX = synth.normal_f16((1, 12, 12, 256), 1.0, 23)
    cW = synth.normal_f16((32, 3, 3, 256), 0.02, 24)
    small = (synth.normal_f16((40, 4096), 1.0, 25), synth.normal_f16((136, 4096), 0.02, 26))
    nbytes = max(mixdq.workspace_bytes(512, 136, 4096, 4, 8), mixdq.workspace_bytes(40, 136, 4096, 4, 8),
                 mixdq.conv3x3_workspace_bytes(1, 12, 12, 256, 32, 1, 4, 8))
    ws = torch.full((nbytes,), 0xA5, dtype=torch.uint8, device="cuda")   # no initial content is assumed
    st = status_word()

    def run_lin(X, W):
        s_ref, _, codes = oracle_weights(W, 4, True)
        sx_ref = orc.act_scale(orc.act_absmax(X), 8)
        acc_ref, _ = orc.linear_a8(X, codes, s_ref, sx_ref, None)
        Xd = dev(X)
        _, _, packed = device_weights(W, 4, True)
        acc = mixdq.linear_acc_i32(Xd, packed, W.shape[0], 4, mixdq.act_scale(Xd), workspace=ws, status=st)
        assert np.array_equal(host(acc), acc_ref)

    def run_conv():
        s_ref, _, codes = oracle_weights(cW.reshape(32, -1), 4, True)
        sx_ref = orc.act_scale(orc.act_absmax(cX), 8)
        acc_ref, _ = orc.conv3x3_a8(cX, codes.reshape(32, 3, 3, 256), s_ref, sx_ref, None, 1)
        Xd = dev(cX)
        _, _, packed = device_weights(cW.reshape(32, -1), 4, True)
        acc = mixdq.conv3x3_acc_i32(Xd, packed, 32, 4, mixdq.act_scale(Xd), 1, workspace=ws, status=st)
        assert np.array_equal(host(acc), acc_ref)

    for _ in range(2):
        run_lin(*lin)
        run_conv()
        run_lin(*small)
    assert int(host(st)[0]) == 0


@pytest.mark.parametrize("bits", [8, 4])
def test_few_output_channels_with_workspace(bits):
    # 4 output channels (conv_out-like): the weight tile is mostly out-of-bounds fill
    _run_linear(synth.normal_f16((200, 2880), 1.0, 6), synth.normal_f16((4, 2880), 0.02, 7),
                synth.normal_f16((4,), 0.01, 8), bits, True)


@pytest.mark.parametrize("bits", [8, 4])
def test_linear_corner_shapes_plain_kernel(bits):
    # reduction length not a multiple of 16, and fewer than 16 output channels
    _run_linear(synth.normal_f16((50, 36), 1.0, 1), synth.normal_f16((40, 36), 0.02, 2), None, bits, False)
    _run_linear(synth.normal_f16((70, 64), 1.0, 3), synth.normal_f16((4, 64), 0.02, 4),
                synth.normal_f16((4,), 0.01, 5), bits, False)


def test_ffn_outlier_channels():
    X = synth.ffn_input(1, seed=3000, K=1280)
    W = synth.normal_f16((384, 1280), 0.02, seed=3001)
    _run_linear(X, W, None, 4, True)
    _run_linear(X, W, None, 8, True)


@pytest.mark.parametrize("use_ws", [False, True])
@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("B,N", [(1, 64), (3, 200), (30, 1280)])
def test_bos_aware_kv(bits, B, N, use_ws):
    E = synth.text_embedding(B, seed=4000)
    W = synth.kv_weight(N, seed=4100 + N)
    s_ref, _, codes = oracle_weights(W, bits, True)
    bos = orc.bos_row(E[0, 0], W)
    sx_ref = orc.crossattn_act_scale(E)
    acc_ref, y_ref = orc.crossattn_kv(E, codes, s_ref, sx_ref, bos)

    Ed = dev(E)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Ed.reshape(-1, E.shape[-1]), skip_rows_mod=77)
    assert host(sx)[0] == sx_ref
    st = status_word()
    ws = workspace_for(B * 76, N, 2048, bits) if use_ws else None
    acc = mixdq.crossattn_kv_acc_i32(Ed, packed, N, bits, sx, workspace=ws, status=st)
    y = mixdq.crossattn_kv(Ed, packed, N, bits, s, sx, dev(bos), workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    yh = host(y)
    for b in range(B):
        assert np.array_equal(yh[b, 0].view(np.uint16), bos.view(np.uint16))
    assert_close(yh, y_ref)
    # what token 0 holds changes nothing in rows >= 1
    E2 = E.copy()
    E2[:, 0, :] = np.float16(-777.0)
    y2 = mixdq.crossattn_kv(dev(E2), packed, N, bits, s, sx, dev(bos), workspace=ws, status=st)
    assert np.array_equal(host(y2).view(np.uint16), yh.view(np.uint16))


@pytest.mark.parametrize("bits", [8, 4])
def test_fused_k_and_v_projection_equals_two_calls(bits):
    # K and V of a cross-attention block read the same text embedding with the same scale: one call on
    # the stacked weights [W_k; W_v] (per-channel scales and BOS rows stacked alike) must give, bit for
    # bit, what the two separate calls give
    B, N = 4, 640
    E = synth.text_embedding(B, seed=4200)
    Wk, Wv = synth.kv_weight(N, seed=4300), synth.kv_weight(N, seed=4301)
    Ed = dev(E)
    sx = mixdq.act_scale(Ed.reshape(-1, E.shape[-1]), skip_rows_mod=77)
    st = status_word()
    outs = []
    for W in (Wk, Wv, np.concatenate([Wk, Wv], axis=0)):
        s, _, packed = device_weights(W, bits, True)
        bos = orc.bos_row(E[0, 0], W)
        ws = workspace_for(B * 76, W.shape[0], 2048, bits)
        outs.append(host(mixdq.crossattn_kv(Ed, packed, W.shape[0], bits, s, sx, dev(bos), workspace=ws, status=st)))
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    yk, yv, ykv = outs
    assert np.array_equal(ykv[..., :N].view(np.uint16), yk.view(np.uint16))
    assert np.array_equal(ykv[..., N:].view(np.uint16), yv.view(np.uint16))


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("use_ws", [False, True])
@pytest.mark.parametrize("B,H,W,Cin,Cout,stride", [(1, 8, 8, 16, 16, 1), (2, 12, 10, 32, 48, 1),
                                                    (2, 12, 10, 32, 48, 2), (1, 16, 16, 320, 136, 1),
                                                    (3, 9, 7, 48, 24, 2), (3, 8, 8, 32, 40, 1),
                                                    (2, 32, 32, 160, 136, 1), (1, 64, 64, 32, 24, 1),
                                                    (1, 16, 16, 640, 264, 1), (2, 16, 16, 64, 48, 2),
                                                    (1, 12, 12, 256, 32, 1), (1, 64, 64, 32, 648, 1),
                                                    # stride 2 on the TMA path: boxes of 4 and of 8 output rows
                                                    (1, 64, 64, 64, 40, 2), (2, 32, 32, 160, 136, 2)])
def test_conv3x3(bits, B, H, W, Cin, Cout, stride, use_ws):
    X = synth.normal_f16((B, H, W, Cin), 1.0, seed=H * W + Cin)
    Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=Cout + Cin)
    b = synth.normal_f16((Cout,), 0.01, seed=Cout)
    s_ref, _, codes = oracle_weights(Wt.reshape(Cout, -1), bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    acc_ref, y_ref = orc.conv3x3_a8(X, codes.reshape(Cout, 3, 3, Cin), s_ref, sx_ref, b, stride)

    Xd = dev(X)
    s, _, packed = device_weights(Wt.reshape(Cout, -1), bits, True)
    sx = mixdq.act_scale(Xd)
    st = status_word()
    ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, H, W, Cin, Cout, stride, bits, 8)) if use_ws else None
    acc = mixdq.conv3x3_acc_i32(Xd, packed, Cout, bits, sx, stride, workspace=ws, status=st)
    y = mixdq.conv3x3(Xd, packed, Cout, bits, s, None, 8, sx, dev(b), stride, workspace=ws, status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)


def test_conv_corner_shapes_plain_kernel():
    # conv_in-like (4 input channels) and conv_out-like (4 output channels)
    for Cin, Cout in ((4, 32), (32, 4)):
        X = synth.normal_f16((1, 10, 10, Cin), 1.0, seed=Cin)
        Wt = synth.normal_f16((Cout, 3, 3, Cin), 0.02, seed=Cout)
        s_ref, _, codes = oracle_weights(Wt.reshape(Cout, -1), 8, True)
        sx_ref = orc.act_scale(orc.act_absmax(X), 8)
        acc_ref, y_ref = orc.conv3x3_a8(X, codes.reshape(Cout, 3, 3, Cin), s_ref, sx_ref, None, 1)
        Xd = dev(X)
        s, _, packed = device_weights(Wt.reshape(Cout, -1), 8, True)
        sx = mixdq.act_scale(Xd)
        acc = mixdq.conv3x3_acc_i32(Xd, packed, Cout, 8, sx, 1)
        y = mixdq.conv3x3(Xd, packed, Cout, 8, s, None, 8, sx, None, 1)
        assert np.array_equal(host(acc), acc_ref)
        assert_close(host(y), y_ref)


def test_conv1x1_equals_linear():
    X = synth.normal_f16((2, 8, 8, 64), 1.0, seed=11)
    Wt = synth.normal_f16((48, 64), 0.02, seed=12)
    s_ref, _, codes = oracle_weights(Wt, 4, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    _, y_ref = orc.linear_a8(X.reshape(-1, 64), codes, s_ref, sx_ref, None)
    Xd = dev(X)
    s, _, packed = device_weights(Wt, 4, True)
    y = mixdq.conv1x1(Xd, packed, 48, 4, s, None, 8, mixdq.act_scale(Xd), None)
    assert_close(host(y).reshape(-1, 48), y_ref)


@pytest.mark.parametrize("bits", [8, 4])
def test_pack_then_layer_on_one_stream_without_synchronization(bits):
    """The layer kernels load their weights before they wait for earlier kernels of the stream; the pack entry
    points end with a full stream dependency so that a layer call enqueued right behind them, with no
    synchronization, still reads complete weights.  The same packed buffer is rewritten for every round."""
    M, K, N = 256, 1280, 640
    X = synth.normal_f16((M, K), 1.0, seed=77)
    Xd = dev(X)
    sx = mixdq.act_scale(Xd)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    st = status_word()
    ws = workspace_for(M, N, K, bits)
    packed = torch.zeros(mixdq.packed_bytes(N, K, bits), dtype=torch.uint8, device="cuda")
    s = torch.zeros(N, dtype=torch.float32, device="cuda")
    Ws = [synth.normal_f16((N, K), 0.02 * (1 + r), seed=780 + r) for r in range(6)]
    Wd = [dev(W) for W in Ws]
    outs = [torch.empty((M, N), dtype=torch.float16, device="cuda") for _ in Ws]
    torch.cuda.synchronize()
    for r in range(len(Ws)):
        mixdq.weight_minmax_params(Wd[r], bits, True, scale_out=s)
        mixdq.pack_weights(Wd[r], bits, s, out=packed)
        mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, None, workspace=ws, status=st, out=outs[r])
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    for r, W in enumerate(Ws):
        s_ref, _, codes = oracle_weights(W, bits, True)
        _, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, None)
        assert_close(host(outs[r]), y_ref)
