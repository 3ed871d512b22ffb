"""Parity on every distinct layer shape of the SDXL-turbo-shaped UNet census, at image batch 4 (the
benchmark's launch configuration) and 1 (the paper's), through the entry points and with the
workspace the layer sweep uses.

int8 path (W4A8 / W8A8): the oracle computes the WHOLE tensor; every int32 accumulator must match bit
for bit and every fp16 output within the path's tolerance.  Weight-only path (A16): the oracle works in
double precision and is too slow for whole tensors of this size, so it computes one output row in every
128-row tile, at a position inside the tile that changes from tile to tile, plus the first and last
rows (a 3x3 conv output pixel is a dot product over its gathered window, which the CPU suite pins
against the direct convolution)."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, host, status_word

pytestmark = pytest.mark.gpu


def _distinct_shapes():
    seen, out = set(), []
    for l in synth.unet_layers():
        key = (l.kind, l.M, l.N, l.K, l.H, l.Cin, l.stride, l.per_batch)
        if key not in seen:
            seen.add(key)
            out.append(l)
    return out


_SHAPES = _distinct_shapes()
_BY_NAME = {l.name: l for l in _SHAPES}


def _gmac(l, B):
    return (l.M * B if l.per_batch else l.M) * l.N * l.K / 1e9


def _int8_cases():
    cases = []
    for i, l in enumerate(_SHAPES):
        corner = l.name.startswith("conv_in") or l.name.startswith("conv_out")
        # batch 4: the dominant width of the sweep's table (4 bits; the corner convolutions stay at 8), and
        # 8 bits as well wherever the oracle's second pass is cheap
        cases.append((l.name, 8 if corner else 4, 4))
        if not corner and _gmac(l, 4) <= 16.0:
            cases.append((l.name, 8, 4))
        # batch 1: widths alternate over the shapes
        cases.append((l.name, 8 if corner else (8 if i % 2 else 4), 1))
    return cases


def rows_one_per_tile(total, tile=128):
    """One row of every `tile`-row block, at a position that moves through the block, plus both ends."""
    rows = {0, total - 1}
    for t in range((total + tile - 1) // tile):
        rows.add(min(total - 1, t * tile + (37 * t + 5) % tile))
    return np.array(sorted(rows))


def window_rows(X, rows, stride):
    """Gathered 3x3 windows (zero padding 1) of the given output pixels: [len(rows), 9 * C]."""
    Bn, H, W, C = X.shape
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    out = np.zeros((len(rows), 3, 3, C), X.dtype)
    for i, m in enumerate(rows):
        b, rem = divmod(int(m), Ho * Wo)
        ho, wo = divmod(rem, Wo)
        for kh in range(3):
            for kw in range(3):
                hi, wi = ho * stride + kh - 1, wo * stride + kw - 1
                if 0 <= hi < H and 0 <= wi < W:
                    out[i, kh, kw] = X[b, hi, wi]
    return out.reshape(len(rows), 9 * C)


@pytest.mark.parametrize("name,w_bits,B", _int8_cases())
def test_int8_layer_whole_tensor(name, w_bits, B):
    l = _BY_NAME[name]
    X, W, b = synth.layer_inputs(l, B, seed=7000 + l.index + 100 * B)
    W2 = np.ascontiguousarray(W.reshape(l.N, -1))
    s_ref, _ = orc.weight_minmax_params(W2, w_bits, True)
    codes = orc.quantize_weights(W2, w_bits, s_ref, None)
    Xd, Wd = dev(X), dev(W2)
    s, _ = mixdq.weight_minmax_params(Wd, w_bits, True)
    packed = mixdq.pack_weights(Wd, w_bits, s)
    st = status_word()
    if l.kind == "bos_kv":
        sx_ref = orc.crossattn_act_scale(X)
        bos = orc.bos_row(X[0, 0], W2)
        acc_ref, y_ref = orc.crossattn_kv(X, codes, s_ref, sx_ref, bos)
        sx = mixdq.act_scale(Xd.reshape(-1, l.K), 77)
        ws = mixdq.new_workspace(mixdq.workspace_bytes(B * 76, l.N, l.K, w_bits, 8))
        acc = mixdq.crossattn_kv_acc_i32(Xd, packed, l.N, w_bits, sx, ws, st)
        y = mixdq.crossattn_kv(Xd, packed, l.N, w_bits, s, sx, dev(bos), ws, st)
        assert np.array_equal(host(y)[:, 0, :].view(np.uint16), np.broadcast_to(bos, (B, l.N)).copy().view(np.uint16))
    elif l.kind == "conv3x3":
        sx_ref = orc.act_scale(orc.act_absmax(X), 8)
        acc_ref, y_ref = orc.conv3x3_a8(X, codes.reshape(l.N, 3, 3, l.Cin), s_ref, sx_ref, b, l.stride)
        sx = mixdq.act_scale(Xd)
        ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, l.H, l.H, l.Cin, l.N, l.stride, w_bits, 8))
        acc = mixdq.conv3x3_acc_i32(Xd, packed, l.N, w_bits, sx, l.stride, ws, st)
        y = mixdq.conv3x3(Xd, packed, l.N, w_bits, s, None, 8, sx, dev(b), l.stride, ws, st)
    else:  # linear layers and 1x1 convolutions (a linear layer over the pixels)
        X2 = np.ascontiguousarray(X.reshape(-1, l.K))
        sx_ref = orc.act_scale(orc.act_absmax(X2), 8)
        acc_ref, y_ref = orc.linear_a8(X2, codes, s_ref, sx_ref, b)
        X2d = Xd.reshape(-1, l.K)
        sx = mixdq.act_scale(X2d)
        ws = mixdq.new_workspace(mixdq.workspace_bytes(X2.shape[0], l.N, l.K, w_bits, 8))
        acc = mixdq.linear_acc_i32(X2d, packed, l.N, w_bits, sx, ws, st)
        y = mixdq.linear(X2d, packed, l.N, w_bits, s, None, 8, sx, dev(b), ws, st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert host(sx)[0] == sx_ref
    assert np.array_equal(host(acc).reshape(acc_ref.shape), acc_ref)
    assert_close(host(y).reshape(y_ref.shape), y_ref)


def _a16_cases():
    cases = []
    for i, l in enumerate(_SHAPES):
        corner = l.name.startswith("conv_in") or l.name.startswith("conv_out")
        cases.append((l.name, 8 if corner else (3, 4, 8)[i % 3], 4))
        cases.append((l.name, 8 if corner else (4, 8, 3)[i % 3], 1))
    return cases


@pytest.mark.parametrize("name,w_bits,B", _a16_cases())
def test_weight_only_layer_one_row_per_tile(name, w_bits, B):
    l = _BY_NAME[name]
    X, W, b = synth.layer_inputs(l, B, seed=7500 + l.index + 100 * B)
    W2 = np.ascontiguousarray(W.reshape(l.N, -1))
    s_ref, z_ref = orc.weight_minmax_params(W2, w_bits, False)
    codes = orc.quantize_weights(W2, w_bits, s_ref, z_ref)
    Xd, Wd = dev(X), dev(W2)
    s, z = mixdq.weight_minmax_params(Wd, w_bits, False)
    packed = mixdq.pack_weights(Wd, w_bits, s, z)
    st = status_word()
    # with the workspace the layer sweep passes (256 rows or more: weights expanded once to fp16, two-CTA fp16 GEMM)
    if l.kind == "conv3x3":
        ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, l.H, l.H, l.Cin, l.N, l.stride, w_bits, 16))
        y = host(mixdq.conv3x3(Xd, packed, l.N, w_bits, s, z, 16, None, dev(b), l.stride, ws, st)).reshape(-1, l.N)
        rows = rows_one_per_tile(y.shape[0])
        a_rows = window_rows(X, rows, l.stride)
    else:
        # the weight-only table keeps the text projections in fp16 activations too: a plain linear layer on all rows
        X2 = np.ascontiguousarray(X.reshape(-1, l.K))
        ws = mixdq.new_workspace(mixdq.workspace_bytes(X2.shape[0], l.N, l.K, w_bits, 16))
        y = host(mixdq.linear(Xd.reshape(-1, l.K), packed, l.N, w_bits, s, z, 16, None, dev(b), ws, st))
        rows = rows_one_per_tile(X2.shape[0])
        a_rows = X2[rows]
    y_ref = orc.linear_a16(np.ascontiguousarray(a_rows), codes, s_ref, z_ref, b)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    assert_close(y[rows], y_ref)
