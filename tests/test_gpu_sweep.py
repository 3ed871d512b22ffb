"""The layer sweep's wiring, on a handful of small layers named like those of the census: every layer's output
against the oracle fed with the sweep's own tensors (weight codes read back through the unpack hook), in the
default form, with shortcut-splitting and with the shared q/k/v quantization."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from paper_2405_17873_b200.unet_sweep import UNetSweep
from helpers import assert_close, host

pytestmark = pytest.mark.gpu


def _specs():
    L = [synth.LayerSpec(name=f"attn_640#{i}", kind="linear", M=192, N=96, K=160, w_bits=4 if i % 2 else 8)
         for i in range(7)]
    L.append(synth.LayerSpec(name="res64_640_320#0", kind="conv3x3", M=256, N=64, K=9 * 640, H=16, Cin=640, w_bits=4))
    L.append(synth.LayerSpec(name="sc64_640#0", kind="conv1x1", M=256, N=64, K=640, H=16, Cin=640, w_bits=8))
    L.append(synth.LayerSpec(name="res64_320_320#0", kind="conv3x3", M=256, N=320, K=9 * 320, H=16, Cin=320, w_bits=4))
    for i, l in enumerate(L):
        l.index = i
    return L


def _codes(packed, N, K, bits):
    return host(mixdq.unpack_weights(packed, N, K, bits, True)).astype(np.int16)


def _check_layer(sw, pl, B):
    l = pl.spec
    sw.run_layer(pl)
    torch.cuda.synchronize()
    assert int(sw.status.item()) == 0
    x = host(sw.x[pl.x_key])
    y = host(sw.y[pl.y_key])
    ws = host(pl.w_scale)
    b = None if pl.bias is None else host(pl.bias)
    if pl.split_at:
        s = pl.split_at
        taps = l.K // l.Cin
        c_lo = _codes(pl.packed, l.N, taps * s, l.w_bits).reshape(l.N, taps, s)
        c_hi = _codes(pl.packed_hi, l.N, taps * (l.Cin - s), l.w_bits).reshape(l.N, taps, l.Cin - s)
        codes = np.ascontiguousarray(np.concatenate([c_lo, c_hi], axis=2))
        s_lo, s_hi = (np.float32(host(t)[0]) for t in sw.x_split_scale[(pl.x_key, s)])
        if l.kind == "conv3x3":
            _, _, y_ref = orc.conv3x3_a8_split(x, codes.reshape(l.N, 3, 3, l.Cin), ws, s_lo, s_hi, s, b, l.stride)
        else:
            _, _, y_ref = orc.linear_a8_split(x.reshape(-1, l.Cin), codes.reshape(l.N, l.Cin), ws, s_lo, s_hi, s, b)
        assert_close(y.reshape(y_ref.shape), y_ref)
        return
    codes = _codes(pl.packed, l.N, l.K, l.w_bits)
    sx = np.float32(host(sw.x_scale[pl.x_key])[0])
    if l.kind == "bos_kv":
        bos = host(pl.bos_out)
        _, y_ref = orc.crossattn_kv(x, codes, ws, sx, bos)
        assert np.array_equal(y[:, 0].view(np.uint16), np.broadcast_to(bos.view(np.uint16), y[:, 0].shape))
        assert_close(y, y_ref)
        return
    if l.kind == "conv3x3":
        _, y_ref = orc.conv3x3_a8(x, codes.reshape(l.N, 3, 3, l.Cin), ws, sx, b, l.stride)
    else:
        _, y_ref = orc.linear_a8(x.reshape(-1, x.shape[-1]), codes, ws, sx, b)
    assert_close(y.reshape(y_ref.shape), y_ref)


@pytest.mark.parametrize("opts", [{}, {"shortcut_split": True}, {"share_qkv_quant": True}],
                         ids=["default", "shortcut_split", "share_qkv_quant"])
def test_sweep_layers_against_oracle(opts):
    B = 2
    sw = UNetSweep(B, "w4a8", layers=_specs(), **opts)
    roles = [pl.qkv_role for pl in sw.layers]
    splits = [pl.split_at for pl in sw.layers]
    if opts.get("share_qkv_quant"):
        assert roles[:7] == [0, 1, 2, -1, -1, -1, 0]
    else:
        assert all(r == -1 for r in roles)
    if opts.get("shortcut_split"):
        assert splits == [0] * 7 + [320, 320, 0]
    else:
        assert not any(splits)
    for pl in sw.layers:
        _check_layer(sw, pl, B)


def test_shared_quantization_gives_identical_bits():
    B = 2
    a = UNetSweep(B, "w4a8", layers=_specs())
    b = UNetSweep(B, "w4a8", layers=_specs(), share_qkv_quant=True)
    for pa, pb in zip(a.layers[:3], b.layers[:3]):
        a.run_layer(pa)
        b.run_layer(pb)
        torch.cuda.synchronize()
        assert torch.equal(a.x[pa.x_key], b.x[pb.x_key])
        assert torch.equal(a.y[pa.y_key], b.y[pb.y_key])


def test_fused_projections_against_oracle():
    # q, k, v with equal widths become one 3N-wide layer, K and V one 2N-wide BOS-aware layer; a triple with
    # mixed widths stays apart
    L = [synth.LayerSpec(name=f"attn_640#{i}", kind="linear", M=192, N=96, K=160, w_bits=4) for i in range(3)]
    L += [synth.LayerSpec(name=f"attn_640#{i}", kind="linear", M=192, N=96, K=160, w_bits=8 if i == 7 else 4)
          for i in range(3, 9)]
    L += [synth.LayerSpec(name=f"kv_640#{i}", kind="bos_kv", M=synth.TOKENS_PER_PROMPT, N=48, K=synth.TEXT_DIM, w_bits=8)
          for i in range(2)]
    ops = sum(l.ops(2) for l in L)
    sw = UNetSweep(2, "w4a8", layers=L, fuse_projections=True)
    assert [pl.spec.name for pl in sw.layers] == ["qkv_attn_640#0", "attn_640#3", "attn_640#4", "attn_640#5",
                                                  "attn_640#6", "attn_640#7", "attn_640#8", "kv2_kv_640#0"]
    assert [pl.spec.N for pl in sw.layers] == [288, 96, 96, 96, 96, 96, 96, 96]
    assert sw.total_ops() == ops
    for pl in sw.layers:
        _check_layer(sw, pl, 2)
