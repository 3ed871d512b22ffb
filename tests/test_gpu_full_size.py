"""Parity at full layer sizes of the SDXL-turbo-shaped UNet sweep (image batch 4) for the cases the census
tests (test_gpu_census.py: every distinct shape, whole tensors on the int8 path) do not cover: the
weight-bound regime of 16 tokens at full layer width, and the shortcut-split layers.  The oracle computes
one output row in every 128-row tile, at a position that moves through the tile, plus the first and last
rows (a 3x3 conv output pixel is a dot product over its gathered window, which the CPU suite pins against
the direct convolution); int32 accumulators of those rows must match bit for bit, fp16 outputs within the
path's tolerance."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import dev, host, status_word

pytestmark = pytest.mark.gpu

B = 4
_SPECS = {l.name: l for l in synth.unet_layers()}


def _sample_rows(total, seed=0):
    """One row of every 128-row tile, at an in-tile position that depends on the tile (and the layer), plus
    the first and last rows and the rows either side of the first tile boundary."""
    rows = {0, total - 1, min(127, total - 1), min(128, total - 1)}
    for t in range((total + 127) // 128):
        rows.add(min(total - 1, t * 128 + (37 * t + 5 + 11 * seed) % 128))
    return np.array(sorted(rows))


def _window_rows(X, rows, stride):
    """Gathered 3x3 windows (zero padding 1) of the sampled output pixels: [len(rows), 9*C]."""
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


def _close(y, y_ref):
    d = np.abs(y.astype(np.float64) - y_ref.astype(np.float64)).max()
    assert d <= 1e-3 * np.abs(y_ref.astype(np.float64)).max() + 1e-3, d


def _check_layer(name, w_bits, a_bits, rows_override=None):
    l = _SPECS[name]
    X, W, b = synth.layer_inputs(l, B, seed=7000 + l.index)
    if rows_override:                      # the weight-bound regime: a few tokens only
        X = np.ascontiguousarray(X[:rows_override])
    W2 = np.ascontiguousarray(W.reshape(l.N, -1))
    sym = a_bits == 8
    s_ref, z_ref = orc.weight_minmax_params(W2, w_bits, sym)
    codes = orc.quantize_weights(W2, w_bits, s_ref, None if sym else z_ref)

    Xd, Wd = dev(X), dev(W2)
    s, z = mixdq.weight_minmax_params(Wd, w_bits, sym)
    packed = mixdq.pack_weights(Wd, w_bits, s, None if sym else z)
    zd = None if sym else z
    st = status_word()
    conv = l.kind == "conv3x3"
    if conv:
        ws = mixdq.new_workspace(mixdq.conv3x3_workspace_bytes(B, l.H, l.H, l.Cin, l.N, l.stride, w_bits, a_bits))
    else:
        rows_total = X.reshape(-1, X.shape[-1]).shape[0]
        ws = mixdq.new_workspace(mixdq.workspace_bytes(rows_total, l.N, l.K, w_bits, a_bits))

    if a_bits == 8:
        if l.kind == "bos_kv":
            sx_ref = orc.crossattn_act_scale(X)
            sx = mixdq.act_scale(Xd.reshape(-1, l.K), 77)
            bos = orc.bos_row(X[0, 0], W2)
            y = host(mixdq.crossattn_kv(Xd, packed, l.N, w_bits, s, sx, dev(bos), ws, st))
            acc = host(mixdq.crossattn_kv_acc_i32(Xd, packed, l.N, w_bits, sx, ws, st)).reshape(-1, l.N)
            rest = np.ascontiguousarray(X[:, 1:, :]).reshape(-1, l.K)
            rows = _sample_rows(rest.shape[0], seed=l.index)
            a_rows = rest[rows]
            y_rows = y[:, 1:, :].reshape(-1, l.N)[rows]
            assert np.array_equal(y[:, 0, :].view(np.uint16), np.broadcast_to(bos, (B, l.N)).copy().view(np.uint16))
            bias = None
        elif conv:
            sx_ref = orc.act_scale(orc.act_absmax(X), 8)
            sx = mixdq.act_scale(Xd)
            y = host(mixdq.conv3x3(Xd, packed, l.N, w_bits, s, None, 8, sx, dev(b), l.stride, ws, st)).reshape(-1, l.N)
            acc = host(mixdq.conv3x3_acc_i32(Xd, packed, l.N, w_bits, sx, l.stride, ws, st)).reshape(-1, l.N)
            rows = _sample_rows(y.shape[0], seed=l.index)
            a_rows = _window_rows(X, rows, l.stride)
            y_rows, bias = y[rows], b
        else:
            X2 = X.reshape(-1, l.K)
            sx_ref = orc.act_scale(orc.act_absmax(X2), 8)
            sx = mixdq.act_scale(Xd.reshape(-1, l.K))
            y = host(mixdq.linear(Xd.reshape(-1, l.K), packed, l.N, w_bits, s, None, 8, sx, dev(b), ws, st))
            acc = host(mixdq.linear_acc_i32(Xd.reshape(-1, l.K), packed, l.N, w_bits, sx, ws, st))
            rows = _sample_rows(X2.shape[0], seed=l.index)
            a_rows, y_rows, bias = X2[rows], y[rows], b
        assert host(sx)[0] == sx_ref
        acc_ref, y_ref = orc.linear_a8(np.ascontiguousarray(a_rows), codes, s_ref, sx_ref, bias)
        torch.cuda.synchronize()
        assert int(host(st)[0]) == 0
        assert np.array_equal(acc[rows], acc_ref)
        _close(y_rows, y_ref)
    else:
        if conv:
            y = host(mixdq.conv3x3(Xd, packed, l.N, w_bits, s, zd, 16, None, dev(b), l.stride, ws, st)).reshape(-1, l.N)
            rows = _sample_rows(y.shape[0], seed=l.index)
            a_rows = _window_rows(X, rows, l.stride)
        else:
            X2 = X.reshape(-1, l.K)
            y = host(mixdq.linear(Xd.reshape(-1, l.K), packed, l.N, w_bits, s, zd, 16, None, dev(b), ws, st))
            rows = _sample_rows(X2.shape[0], seed=l.index)
            a_rows = X2[rows]
        y_ref = orc.linear_a16(np.ascontiguousarray(a_rows), codes, s_ref, z_ref, b)
        torch.cuda.synchronize()
        assert int(host(st)[0]) == 0
        _close(y[rows], y_ref)


@pytest.mark.parametrize("name,w_bits", [("ffn1_1280#0", 3), ("ffn1_1280#0", 4), ("ffn2_1280#0", 4),
                                         ("attn_1280#0", 8)])
def test_weight_only_sixteen_tokens_full_width(name, w_bits):
    _check_layer(name, w_bits, 16, rows_override=16)


@pytest.mark.parametrize("name,w_bits", [("res16_2560_1280#0", 4), ("res32_1920_640#0", 8), ("res64_640_320#0", 4),
                                         ("sc64_960#0", 4), ("sc16_2560#0", 8)])
def test_shortcut_split_layers_full_size(name, w_bits):
    """The concatenation-fed resnet convolutions at image batch 4 with one activation scale per branch
    (Sec. 4.1): both int32 sums of the sampled output pixels bit-exact, outputs within tolerance."""
    l = _SPECS[name]
    split = synth.shortcut_split_at(l)
    assert split > 0
    X, W, b = synth.layer_inputs(l, B, seed=7000 + l.index)
    X = X.copy()
    X[..., split:] = (X[..., split:].astype(np.float32) / 8.0).astype(np.float16)   # the skip branch: a smaller range
    taps = l.K // l.Cin
    W3 = np.ascontiguousarray(W.reshape(l.N, taps, l.Cin))
    W2 = W3.reshape(l.N, -1)
    s_ref, _ = orc.weight_minmax_params(W2, w_bits, True)
    codes = orc.quantize_weights(W2, w_bits, s_ref, None).reshape(l.N, taps, l.Cin)
    x2 = X.reshape(-1, l.Cin)
    s_lo_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(x2[:, :split])), 8)
    s_hi_ref = orc.act_scale(orc.act_absmax(np.ascontiguousarray(x2[:, split:])), 8)

    Xd = dev(X)
    s, _ = mixdq.weight_minmax_params(dev(W2), w_bits, True)
    p_lo = mixdq.pack_weights(dev(W3[:, :, :split].reshape(l.N, -1)), w_bits, s)
    p_hi = mixdq.pack_weights(dev(W3[:, :, split:].reshape(l.N, -1)), w_bits, s)
    xd2 = Xd.reshape(-1, l.Cin)
    s_lo, s_hi = mixdq.act_scale(xd2[:, :split].contiguous()), mixdq.act_scale(xd2[:, split:].contiguous())
    assert host(s_lo)[0] == s_lo_ref and host(s_hi)[0] == s_hi_ref
    Ho = (l.H - 1) // l.stride + 1
    out_rows = B * Ho * Ho
    ws = mixdq.new_workspace(mixdq.split_workspace_bytes(B * l.H * l.H, l.Cin, split, out_rows, l.N))
    st = status_word()
    if l.kind == "conv3x3":
        a_lo, a_hi = mixdq.conv3x3_a8_split_acc_i32(Xd, split, p_lo, p_hi, l.N, w_bits, s_lo, s_hi, l.stride, ws, st)
        y = mixdq.conv3x3_a8_split(Xd, split, p_lo, p_hi, l.N, w_bits, s, s_lo, s_hi, dev(b), l.stride, ws, st)
    else:
        a_lo, a_hi = mixdq.linear_a8_split_acc_i32(xd2, split, p_lo, p_hi, l.N, w_bits, s_lo, s_hi, ws, st)
        y = mixdq.linear_a8_split(xd2, split, p_lo, p_hi, l.N, w_bits, s, s_lo, s_hi, dev(b), ws, st)
    torch.cuda.synchronize()
    assert int(host(st)[0]) == 0
    a_lo, a_hi, y = (host(t).reshape(-1, l.N) for t in (a_lo, a_hi, y))
    rows = _sample_rows(out_rows, seed=l.index)
    if l.kind == "conv3x3":
        win = _window_rows(X, rows, l.stride).reshape(len(rows), 9, l.Cin)
    else:
        win = x2[rows].reshape(len(rows), 1, l.Cin)
    # the sampled pixels as a split linear layer on [all lo channels of the taps | all hi channels]
    cols = np.ascontiguousarray(np.concatenate([win[:, :, :split].reshape(len(rows), -1),
                                                win[:, :, split:].reshape(len(rows), -1)], axis=1))
    wcols = np.ascontiguousarray(np.concatenate([codes[:, :, :split].reshape(l.N, -1),
                                                 codes[:, :, split:].reshape(l.N, -1)], axis=1))
    lo_ref, hi_ref, y_ref = orc.linear_a8_split(cols, wcols, s_ref, s_lo_ref, s_hi_ref, taps * split, b)
    assert np.array_equal(a_lo[rows], lo_ref) and np.array_equal(a_hi[rows], hi_ref)
    _close(y[rows], y_ref)
