"""GPU parity of the int8 path on activations kept as int8 between layers: the quantizer's codes bit-exact,
then accumulators bit-exact and fp16 outputs within tolerance from those codes (Sec. 4.1; Sec. 4.3 for the
stored-int8 activations)."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for

pytestmark = pytest.mark.gpu

# one ragged tile; cluster split of the reduction; persistent 128- and 256-wide tiles
SHAPES = [(64, 16, 16), (77, 336, 200), (300, 320, 328), (256, 5120, 320), (16, 2560, 1300),
          (2048, 272, 1288), (4096, 384, 1280), (1024, 1280, 1280)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("M,K,N", SHAPES)
def test_quantize_then_linear_q8(bits, M, K, N):
    X = synth.ffn_input(1, seed=M + K, K=K)[:M] if M <= 256 else synth.normal_f16((M, K), 1.0, seed=M + K)
    W = synth.normal_f16((N, K), 0.02, seed=N + K + 1)
    b = synth.normal_f16((N,), 0.01, seed=N + 2)
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    q_ref = orc.quantize_acts(X, sx_ref, 8)
    acc_ref, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, b)

    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    Xq = mixdq.quantize_acts(Xd, sx)
    st = status_word()
    acc = mixdq.linear_q8_acc_i32(Xq, packed, N, bits, status=st)
    y = mixdq.linear_q8(Xq, packed, N, bits, s, sx, dev(b), status=st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert np.array_equal(host(Xq).astype(np.int64), q_ref.astype(np.int64))
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
    # the one-call form computes the same thing: identical bits
    y_one = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, dev(b), workspace_for(M, N, K, bits), st)
    assert np.array_equal(host(y).view(np.uint16), host(y_one).view(np.uint16))


def test_quantize_acts_strided_rows_and_ties():
    # rows taken out of a wider matrix (row stride > K); values on rounding ties and beyond the clamp
    K, ld = 64, 96
    base = np.zeros((40, ld), np.float16)
    vals = np.array([0.5, 1.5, 2.5, -0.5, -1.5, -2.5, 126.5, 127.5, 300.0, -127.5, -300.0, 0.0], np.float16)
    base[:, :K] = np.resize(vals, (40, K))
    scale = np.float32(1.0)
    q_ref = orc.quantize_acts(np.ascontiguousarray(base[:, :K]), scale, 8)
    assert q_ref[0, :12].tolist() == [0, 2, 2, 0, -2, -2, 126, 127, 127, -127, -127, 0]   # ties to even, clamp
    Xd = dev(base)
    Xq = mixdq.quantize_acts(Xd[:, :K], dev(np.array([scale], np.float32)))
    assert np.array_equal(host(Xq).astype(np.int64), q_ref.astype(np.int64))


def test_three_projections_share_one_quantization():
    # q, k and v of self-attention read the same tensor: one quantization pass, three GEMMs on the stored codes
    M, K, N = 1024, 640, 640
    X = synth.normal_f16((M, K), 1.0, seed=70)
    Xd = dev(X)
    sx = mixdq.act_scale(Xd)
    Xq = mixdq.quantize_acts(Xd, sx)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    for i in range(3):
        W = synth.normal_f16((N, K), 0.02, seed=71 + i)
        s_ref, _, codes = oracle_weights(W, 4, True)
        _, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, None)
        s, _, packed = device_weights(W, 4, True)
        assert_close(host(mixdq.linear_q8(Xq, packed, N, 4, s, sx)), y_ref)


def test_q8_argument_errors():
    Xq = torch.zeros((64, 40), dtype=torch.int8, device="cuda")
    W = synth.normal_f16((32, 40), 0.02, seed=2)
    s, _, packed = device_weights(W, 8, True)
    sx = dev(np.array([1.0], np.float32))
    with pytest.raises(mixdq.MixdqError, match="unsupported"):
        mixdq.linear_q8(Xq, packed, 32, 8, s, sx)            # K % 16 != 0
    with pytest.raises(mixdq.MixdqError, match="unsupported"):
        mixdq.linear_q8(Xq[:, :32].contiguous(), packed, 32, 3, s, sx)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("B,H,C,N,stride", [(2, 8, 32, 48, 1), (1, 16, 160, 136, 1), (3, 16, 256, 320, 1),
                                             (2, 16, 64, 40, 2), (1, 64, 32, 32, 1)])
def test_conv3x3_on_a_stored_int8_image(bits, B, H, C, N, stride):
    X = synth.normal_f16((B, H, H, C), 1.0, seed=H + C)
    Wt = synth.normal_f16((N, 3, 3, C), 0.02, seed=N + C + 1)
    b = synth.normal_f16((N,), 0.01, seed=N + 2)
    s_ref, _, codes = oracle_weights(Wt.reshape(N, -1), bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    _, y_ref = orc.conv3x3_a8(X, codes.reshape(N, 3, 3, C), s_ref, sx_ref, b, stride)
    Xd = dev(X)
    s, _, packed = device_weights(Wt.reshape(N, -1), bits, True)
    sx = mixdq.act_scale(Xd)
    Xq = mixdq.quantize_acts(Xd.reshape(-1, C), sx).reshape(B, H, H, C)
    st = status_word()
    y = mixdq.conv3x3_q8(Xq, packed, N, bits, s, sx, dev(b), stride, st)
    ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, H, H, C, N, stride, bits, 8))
    y_one = mixdq.conv3x3(Xd, packed, N, bits, s, None, 8, sx, dev(b), stride, ws, st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert_close(host(y), y_ref)
    assert np.array_equal(host(y).view(np.uint16), host(y_one).view(np.uint16))
