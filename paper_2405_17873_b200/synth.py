"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no quantization arithmetic: it only draws random tensors
and lists layer shapes, so that the tests can hand the same inputs to the
CUDA library and to the CPU oracle.  It imports neither of them.

The paper evaluates on SDXL-turbo at 512x512 with COCO prompts (Sec. 4.1,
Sec. 4.2); neither the weights nor the prompts are used here.  What is kept
is the shape of every quantizable layer of that UNet, the N(0, 0.02) /
N(0, 1) magnitude of weights / activations, and the outlier structure the
paper describes for the BOS token of the text embedding (Sec. 3.1: one token
whose magnitude dwarfs the others and is identical for every prompt).
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional

import numpy as np
import torch

TOKENS_PER_PROMPT = 77
TEXT_DIM = 2048


def _gen(seed: int) -> torch.Generator:
    return torch.Generator(device="cpu").manual_seed(int(seed))


def normal_f16(shape, std: float, seed: int) -> np.ndarray:
    """fp32 N(0, std) draw from a seeded CPU generator, rounded to fp16."""
    t = torch.randn(tuple(shape), generator=_gen(seed), dtype=torch.float32) * std
    return t.to(torch.float16).numpy()


# ------------------------------------------------------------------ configs

def single_linear(seed: int = 0, M: int = 256, K: int = 320, N: int = 320):
    """One W8A8 linear layer: X ~ N(0,1), W ~ N(0,0.02), bias ~ N(0,0.01)."""
    g = _gen(seed)
    X = torch.randn(M, K, generator=g).to(torch.float16).numpy()
    W = (torch.randn(N, K, generator=g) * 0.02).to(torch.float16).numpy()
    b = (torch.randn(N, generator=g) * 0.01).to(torch.float16).numpy()
    return X, W, b


WEIGHT_ONLY_LAYERS = [  # (K, N, bits) of the mixed bit-width weight-only trio
    (320, 320, 3),
    (320, 1280, 4),
    (1280, 320, 8),
]


def weight_only_layer(idx: int, M: int, seed_base: int = 2000):
    K, N, bits = WEIGHT_ONLY_LAYERS[idx]
    g = _gen(seed_base + idx)
    X = torch.randn(M, K, generator=g).to(torch.float16).numpy()
    W = (torch.randn(N, K, generator=g) * 0.02).to(torch.float16).numpy()
    b = (torch.randn(N, generator=g) * 0.01).to(torch.float16).numpy()
    return X, W, b, bits


def ffn_input(B: int, seed: int = 3000, K: int = 1280, outlier_frac: float = 0.01,
              outlier_gain: float = 20.0) -> np.ndarray:
    """Transformer FFN input [B*256, K] ~ N(0,1) with 1% of channels scaled x20."""
    g = _gen(seed)
    X = torch.randn(B * 256, K, generator=g)
    n_out = max(1, int(round(outlier_frac * K)))
    idx = torch.randperm(K, generator=g)[:n_out]
    X[:, idx] *= outlier_gain
    return X.to(torch.float16).numpy()


def geglu(h: np.ndarray) -> np.ndarray:
    """value * GELU(gate) of an FFN-1 output [M, 2C] -> [M, C] (un-timed glue between the
    two quantized GEMMs; non-linearities are not quantized, Sec. 4.1)."""
    t = torch.from_numpy(h.astype(np.float32))
    v, gate = t.chunk(2, dim=-1)
    return (v * torch.nn.functional.gelu(gate)).to(torch.float16).numpy()


def one_sided_f16(shape, seed: int, shift: float = 0.0, gain: float = 1.0) -> np.ndarray:
    """gain * GELU(N(shift, 1)): the skewed value range (a short negative tail near -0.17 * gain, a long
    positive one) of a tensor that follows a GELU / SiLU, where an asymmetric grid pays (Sec. 4.1)."""
    t = torch.randn(*shape, generator=_gen(seed)) + shift
    return (gain * torch.nn.functional.gelu(t)).to(torch.float16).numpy()


def text_embedding(B: int, seed: int = 4000, n_outlier_ch: int = 8, outlier_mag: float = 50.0):
    """Text embedding [B,77,2048] ~ N(0,1); token 0 is one seeded row shared by every prompt
    with a few fixed channels at +-outlier_mag."""
    g = _gen(seed)
    E = torch.randn(B, TOKENS_PER_PROMPT, TEXT_DIM, generator=_gen(seed + 1 + B))
    bos = torch.randn(TEXT_DIM, generator=g)
    ch = torch.randperm(TEXT_DIM, generator=g)[:n_outlier_ch]
    sign = torch.where(torch.rand(n_outlier_ch, generator=g) < 0.5, -1.0, 1.0)
    bos[ch] = outlier_mag * sign
    E[:, 0, :] = bos[None, :]
    return E.to(torch.float16).numpy()


def bos_projection(e_bos: torch.Tensor, W: torch.Tensor) -> torch.Tensor:
    """The stored BOS row of a K/V projection: the UNQUANTIZED fp16 layer applied to the BOS embedding,
    accumulated in float64 and rounded once to fp16 (Sec. 3.1: this row is computed ahead of time in
    floating point and never quantized).  Works on tensors of any device."""
    return (W.to(torch.float64) @ e_bos.to(torch.float64)).to(torch.float16).contiguous()


def kv_weight(N: int, seed: int) -> np.ndarray:
    return normal_f16((N, TEXT_DIM), 0.02, seed)


# ------------------------------------------------------------ UNet layer census

@dataclass
class LayerSpec:
    """One quantizable layer of the SDXL-turbo-shaped 512px UNet (per image)."""
    name: str
    kind: str            # "linear" | "bos_kv" | "conv3x3" | "conv1x1"
    M: int               # output rows per image (tokens or output pixels); 1 for embeddings
    N: int               # output channels
    K: int               # reduction length (conv: 9 * Cin)
    H: int = 0           # conv input height/width
    Cin: int = 0
    stride: int = 1
    per_batch: bool = True   # False: M does not grow with the image batch
    w_bits: int = 8
    a_bits: int = 8
    index: int = 0

    def rows(self, B: int) -> int:
        return self.M * B

    @property
    def params(self) -> int:
        return self.N * self.K

    def ops(self, B: int) -> int:
        return 2 * self.rows(B) * self.N * self.K


def unet_layers() -> List[LayerSpec]:
    """Every quantizable layer of the UNet: 794 layers, 2.566 G weights."""
    L: List[LayerSpec] = []

    def add(kind, name, M, N, K, count, **kw):
        for i in range(count):
            L.append(LayerSpec(name=f"{name}#{i}", kind=kind, M=M, N=N, K=K, **kw))

    # transformer blocks, 1280-channel level (16x16 tokens) and 640 level (32x32)
    add("linear", "ffn1_1280", 256, 10240, 1280, 60)
    add("linear", "attn_1280", 256, 1280, 1280, 372)
    add("linear", "ffn2_1280", 256, 1280, 5120, 60)
    add("linear", "ffn1_640", 1024, 5120, 640, 10)
    add("linear", "attn_640", 1024, 640, 640, 70)
    add("linear", "ffn2_640", 1024, 640, 2560, 10)
    add("bos_kv", "kv_1280", TOKENS_PER_PROMPT, 1280, TEXT_DIM, 120)
    add("bos_kv", "kv_640", TOKENS_PER_PROMPT, 640, TEXT_DIM, 20)
    # 3x3 convs, stride 1
    for cin, cnt in ((320, 7), (640, 2), (960, 1)):
        add("conv3x3", f"res64_{cin}_320", 4096, 320, 9 * cin, cnt, H=64, Cin=cin)
    add("conv3x3", "up64_640", 4096, 640, 9 * 640, 1, H=64, Cin=640)
    for cin, cnt in ((320, 1), (640, 6), (960, 1), (1280, 1), (1920, 1)):
        add("conv3x3", f"res32_{cin}_640", 1024, 640, 9 * cin, cnt, H=32, Cin=cin)
    add("conv3x3", "up32_1280", 1024, 1280, 9 * 1280, 1, H=32, Cin=1280)
    for cin, cnt in ((640, 1), (1280, 10), (1920, 1), (2560, 2)):
        add("conv3x3", f"res16_{cin}_1280", 256, 1280, 9 * cin, cnt, H=16, Cin=cin)
    # the two stride-2 downsamplers
    add("conv3x3", "down64_320", 1024, 320, 9 * 320, 1, H=64, Cin=320, stride=2)
    add("conv3x3", "down32_640", 256, 640, 9 * 640, 1, H=32, Cin=640, stride=2)
    # 1x1 shortcut convs
    for cin, cnt in ((640, 2), (960, 1)):
        add("conv1x1", f"sc64_{cin}", 4096, 320, cin, cnt, H=64, Cin=cin)
    for cin in (320, 960, 1280, 1920):
        add("conv1x1", f"sc32_{cin}", 1024, 640, cin, 1, H=32, Cin=cin)
    for cin, cnt in ((640, 1), (1920, 1), (2560, 2)):
        add("conv1x1", f"sc16_{cin}", 256, 1280, cin, cnt, H=16, Cin=cin)
    # corner shapes: conv_in 4->320 and conv_out 320->4
    add("conv3x3", "conv_in", 4096, 320, 36, 1, H=64, Cin=4)
    add("conv3x3", "conv_out", 4096, 4, 2880, 1, H=64, Cin=320)
    # embedding / per-resnet time projections: one row per image
    add("linear", "time_emb1", 1, 1280, 320, 1)
    add("linear", "time_emb2", 1, 1280, 1280, 1)
    add("linear", "add_emb1", 1, 1280, 2816, 1)
    add("linear", "add_emb2", 1, 1280, 1280, 1)
    add("linear", "res_time_320", 1, 320, 1280, 5)
    add("linear", "res_time_640", 1, 640, 1280, 5)
    add("linear", "res_time_1280", 1, 1280, 1280, 7)
    for i, l in enumerate(L):
        l.index = i
    return L


def self_attention_role(l: LayerSpec) -> int:
    """0, 1, 2 for the q, k and v projections of a self-attention block -- three layers that read the same
    tensor -- and -1 for every other layer.  The census lists six 1280x1280 (640x640) projections per
    transformer block (self q, k, v, out; cross q, out) before the per-transformer proj_in / proj_out."""
    base, _, idx = l.name.partition("#")
    blocks = {"attn_1280": 60, "attn_640": 10}.get(base)
    if blocks is None or int(idx) >= 6 * blocks:
        return -1
    role = int(idx) % 6
    return role if role < 3 else -1


def fuse_projections(layers: List[LayerSpec]) -> List[LayerSpec]:
    """The census with projections that read the same tensor stacked into one layer where their widths agree:
    q, k and v of a self-attention block (N -> 3N) and the K and V projections of a cross-attention block
    (consecutive pairs of the BOS-aware layers, N -> 2N).  Per-output-channel weight scales and a shared
    activation scale make the stacked layer compute exactly what the separate ones do; the operation count
    is unchanged."""
    out: List[LayerSpec] = []
    i = 0
    while i < len(layers):
        l = layers[i]
        group = 1
        if self_attention_role(l) == 0 and i + 2 < len(layers):
            group = 3
        elif l.kind == "bos_kv" and int(l.name.partition("#")[2]) % 2 == 0 and i + 1 < len(layers):
            group = 2
        members = layers[i:i + group]
        same = all(m.kind == l.kind and (m.N, m.K, m.M, m.w_bits, m.a_bits) == (l.N, l.K, l.M, l.w_bits, l.a_bits)
                   for m in members)
        if group > 1 and same:
            base, _, idx = l.name.partition("#")
            out.append(LayerSpec(name=f"{'qkv' if group == 3 else 'kv2'}_{base}#{idx}", kind=l.kind, M=l.M,
                                 N=group * l.N, K=l.K, per_batch=l.per_batch, w_bits=l.w_bits, a_bits=l.a_bits))
            i += group
        else:
            out.append(l)
            i += 1
    for j, l in enumerate(out):
        l.index = j
    return out


# hidden-state channels of the layers fed by [hidden | skip] concatenations in the up path, by input width
_CONCAT_HIDDEN = {2560: 1280, 1920: 1280, 1280: 640, 960: 640, 640: 320}


def shortcut_split_at(l: LayerSpec) -> int:
    """Channel at which the input of a resnet convolution (3x3 or its 1x1 shortcut) of the up path splits into
    the hidden state and the skip connection it was concatenated with (Sec. 4.1, shortcut-splitting); 0 for a
    layer that is not fed by a concatenation.  In this architecture those are the resnet layers that narrow
    their input (Cin > Cout)."""
    if l.kind not in ("conv3x3", "conv1x1") or not (l.name.startswith("res") or l.name.startswith("sc")):
        return 0
    if l.Cin <= l.N:
        return 0
    return _CONCAT_HIDDEN.get(l.Cin, 0)


def assign_bits_weight_only(layers: List[LayerSpec], seed: int = 5, target: float = 3.66,
                            frac8: float = 0.02, low: int = 3) -> None:
    """Seeded A16 table whose parameter-weighted mean weight width is ~3.66 bits
    (the W3.66A16 row of Table 1): a shuffled ~2% of parameters at 8 bits, then a
    `low`-vs-4 split chosen to land on the target (low = 3, or 2 for the paper's own candidate
    widths {2, 4, 8}, Sec. 3.3).  conv_in / conv_out stay at 8 bits (Sec. 5 lists them as the
    sensitive convolutions)."""
    assert low in (2, 3)
    rng = np.random.default_rng(seed)
    order = rng.permutation(len(layers))
    total = sum(l.params for l in layers)
    for l in layers:
        l.a_bits = 16
        l.w_bits = 0
    p8 = 0
    for l in layers:
        if l.name.startswith("conv_in") or l.name.startswith("conv_out"):
            l.w_bits = 8
            p8 += l.params
    rest = [layers[i] for i in order if layers[i].w_bits == 0]
    for l in rest:
        if p8 + l.params <= frac8 * total:
            l.w_bits = 8
            p8 += l.params
    rest = [l for l in rest if l.w_bits == 0]
    # choose params at `low` bits so that (8*p8 + low*p3 + 4*(total-p8-p3)) / total == target
    want_p3 = (8 * p8 + 4 * (total - p8) - target * total) / (4 - low)
    p3 = 0
    for l in rest:
        if p3 + l.params <= want_p3:
            l.w_bits = low
            p3 += l.params
        else:
            l.w_bits = 4


def assign_bits_w4a8(layers: List[LayerSpec], seed: int = 5, frac_w8: float = 0.10) -> None:
    """Seeded W4A8 table with 10% of the layers (by count) at W8A8."""
    rng = np.random.default_rng(seed)
    n8 = int(round(frac_w8 * len(layers)))
    chosen = set(rng.permutation(len(layers))[:n8].tolist())
    for i, l in enumerate(layers):
        l.a_bits = 8
        l.w_bits = 8 if (i in chosen or l.name.startswith("conv_in")
                         or l.name.startswith("conv_out")) else 4


def average_weight_bits(layers: List[LayerSpec]) -> float:
    return sum(l.w_bits * l.params for l in layers) / sum(l.params for l in layers)


def distinct_shapes(layers: List[LayerSpec]):
    """Group layers that share (kind, M, N, K, H, Cin, stride, bits): returns {key: count}."""
    out = {}
    for l in layers:
        key = (l.kind, l.M, l.N, l.K, l.H, l.Cin, l.stride, l.w_bits, l.a_bits)
        out[key] = out.get(key, 0) + 1
    return out


def layer_inputs(l: LayerSpec, B: int, seed: int):
    """Seeded (X, W, bias) for one census layer at image batch B.
    conv: X NHWC [B,H,H,Cin], W [N,3,3,Cin] (or [N,Cin] for 1x1); linear: X [rows,K]."""
    g = _gen(seed)
    rows = l.M * B if l.per_batch else l.M
    if l.kind in ("conv3x3", "conv1x1"):
        X = torch.randn(B, l.H, l.H, l.Cin, generator=g).to(torch.float16).numpy()
        wshape = (l.N, 3, 3, l.Cin) if l.kind == "conv3x3" else (l.N, l.Cin)
    elif l.kind == "bos_kv":
        X = text_embedding(B, seed=seed)
        wshape = (l.N, l.K)
    else:
        X = torch.randn(rows, l.K, generator=g).to(torch.float16).numpy()
        wshape = (l.N, l.K)
    W = (torch.randn(wshape, generator=g) * 0.02).to(torch.float16).numpy()
    b = (torch.randn(l.N, generator=g) * 0.01).to(torch.float16).numpy()
    return X, W, b
