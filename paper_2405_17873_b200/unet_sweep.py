"""Layer sweep over the SDXL-turbo-shaped UNet: every quantizable layer once, each with the
weight / activation widths its bit table assigns (the granularity of mixed precision is
the layer, paper Sec. 5 "Hardware Friendly").

The sweep owns device buffers only; each layer is one call into the C-ABI library, which
picks the engine from the widths.  Weights are distinct per layer (as in the real model);
layers with the same input shape read the same activation buffer.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Dict, List, Optional

import torch

from . import mixdq, synth


@dataclass
class PackedLayer:
    spec: synth.LayerSpec
    packed: torch.Tensor
    w_scale: torch.Tensor
    w_zero: Optional[torch.Tensor]
    bias: Optional[torch.Tensor]
    bos_out: Optional[torch.Tensor]
    x_key: tuple
    y_key: tuple
    code_sums: Optional[torch.Tensor] = None   # asymmetric activations: per-channel sums of the weight codes
    split_at: int = 0                          # shortcut-splitting: `packed` holds input channels [0, split_at) ...
    packed_hi: Optional[torch.Tensor] = None   # ... and this the rest
    qkv_role: int = -1                         # shared quantization: 0 quantizes the tensor, 1 and 2 reuse the codes


class UNetSweep:
    def __init__(self, batch: int, table: str = "w4a8", seed: int = 5, device: str = "cuda",
                 layers: Optional[List[synth.LayerSpec]] = None, tokens: int = 0, act_asym: bool = False,
                 low_bits: int = 3, shortcut_split: bool = False, share_qkv_quant: bool = False,
                 fuse_projections: bool = False):
        """tokens > 0: the weight-bound regime -- only the linear layers, each on `tokens` rows in all
        (whatever the image size), so that a layer is one stream over its packed weights.
        act_asym: the 8-bit activations of the linear layers and 3x3 convolutions are asymmetric (Sec. 4.1);
        the BOS-aware K/V projections keep symmetric ones.
        low_bits: lowest width of the a16 table (3, or 2 for the paper's candidate widths {2, 4, 8}).
        shortcut_split: the A8 resnet convolutions (3x3 and 1x1) of the up path, whose input is a concatenation
        [hidden | skip], keep one activation scale per branch (Sec. 4.1); symmetric activations.
        share_qkv_quant: the q, k and v projections of a self-attention block read one tensor; it is quantized
        once (by q's call) and the three GEMMs run on the stored int8 codes (symmetric activations).
        fuse_projections: q, k, v of self-attention and K, V of cross-attention run as one stacked layer each where
        the bit table gives them the same widths (synth.fuse_projections)."""
        assert table in ("w4a8", "a16")
        assert not (act_asym and shortcut_split) and not (act_asym and share_qkv_quant)
        self.share_qkv_quant = share_qkv_quant and table == "w4a8" and tokens == 0
        self.xq: Dict[tuple, torch.Tensor] = {}
        self.shortcut_split = shortcut_split
        self.batch = batch
        self.act_asym = act_asym
        self.tokens = tokens
        self.table = table
        self.device = device
        self.specs = layers if layers is not None else synth.unet_layers()
        if tokens > 0:
            self.specs = [l for l in self.specs if l.kind == "linear"]
        if layers is None:
            if table == "w4a8":
                synth.assign_bits_w4a8(self.specs, seed)
            else:
                synth.assign_bits_weight_only(self.specs, seed, low=low_bits)
        if fuse_projections:
            self.specs = synth.fuse_projections(self.specs)
        self.x: Dict[tuple, torch.Tensor] = {}
        self.y: Dict[tuple, torch.Tensor] = {}
        self.x_scale: Dict[tuple, torch.Tensor] = {}
        self.x_asym: Dict[tuple, tuple] = {}
        self.x_split_scale: Dict[tuple, tuple] = {}
        self.layers: List[PackedLayer] = []
        self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self._build(seed)

    # ------------------------------------------------------------------ setup (untimed)
    def _x_shape(self, l: synth.LayerSpec):
        B = self.batch
        if l.kind in ("conv3x3", "conv1x1"):
            return ("nhwc", B, l.H, l.H, l.Cin)
        if l.kind == "bos_kv":
            return ("text", B, synth.TOKENS_PER_PROMPT, l.K)
        return ("rows", self.tokens if self.tokens > 0 else l.M * B, l.K)

    def _y_shape(self, l: synth.LayerSpec):
        B = self.batch
        if l.kind == "conv3x3":
            Ho = (l.H - 1) // l.stride + 1
            return (B, Ho, Ho, l.N)
        if l.kind == "conv1x1":
            return (B, l.H, l.H, l.N)
        if l.kind == "bos_kv":
            return (B, synth.TOKENS_PER_PROMPT, l.N)
        return (self.tokens if self.tokens > 0 else l.M * B, l.N)

    def _build(self, seed: int):
        g = torch.Generator(device=self.device).manual_seed(seed)
        max_ws = 0
        for l in self.specs:
            xk, yk = self._x_shape(l), self._y_shape(l)
            if xk not in self.x:
                if xk[0] == "text":
                    x = torch.from_numpy(synth.text_embedding(self.batch, seed=seed * 1000)).to(self.device)
                else:
                    x = torch.randn(xk[1:], generator=g, device=self.device, dtype=torch.float32).to(torch.float16)
                self.x[xk] = x.contiguous()
                if l.a_bits == 8 or self.table == "w4a8":
                    skip = synth.TOKENS_PER_PROMPT if xk[0] == "text" else 0
                    self.x_scale[xk] = mixdq.act_scale(self.x[xk].reshape(-1, xk[-1]), skip)
            if yk not in self.y:
                self.y[yk] = torch.empty(yk, dtype=torch.float16, device=self.device)
            W = (torch.randn((l.N, l.K), generator=g, device=self.device, dtype=torch.float32) * 0.02).to(torch.float16)
            bias = (torch.randn((l.N,), generator=g, device=self.device, dtype=torch.float32) * 0.01).to(torch.float16)
            symmetric = l.a_bits == 8
            s, z = mixdq.weight_minmax_params(W, l.w_bits, symmetric)
            packed = mixdq.pack_weights(W, l.w_bits, s, None if symmetric else z)
            bos = None
            if l.kind == "bos_kv":
                bias = None
                if l.a_bits == 8:
                    bos = synth.bos_projection(self.x[xk][0, 0], W)
            sums = None
            # convolutions whose geometry the two-kernel path does not take (conv_in: 4 channels) stay symmetric
            if self.act_asym and l.a_bits == 8 and (l.kind in ("linear", "conv1x1") or (l.kind == "conv3x3" and l.Cin % 32 == 0)):
                sums = mixdq.weight_code_sums(packed, l.N, l.K, l.w_bits)
                if xk not in self.x_asym:
                    self.x_asym[xk] = mixdq.act_asym_params(self.x[xk].reshape(-1, xk[-1]))
            split_at = synth.shortcut_split_at(l) if (self.shortcut_split and l.a_bits == 8) else 0
            packed_hi = None
            if split_at:
                # the two channel ranges of the weights, packed apart with the scale of the whole row
                taps = l.K // l.Cin
                W3 = W.view(l.N, taps, l.Cin)
                packed = mixdq.pack_weights(W3[:, :, :split_at].reshape(l.N, -1).contiguous(), l.w_bits, s)
                packed_hi = mixdq.pack_weights(W3[:, :, split_at:].reshape(l.N, -1).contiguous(), l.w_bits, s)
                if (xk, split_at) not in self.x_split_scale:
                    x2 = self.x[xk].reshape(-1, l.Cin)
                    self.x_split_scale[(xk, split_at)] = (mixdq.act_scale(x2[:, :split_at].contiguous()),
                                                          mixdq.act_scale(x2[:, split_at:].contiguous()))
            role = synth.self_attention_role(l) if (self.share_qkv_quant and l.a_bits == 8) else -1
            if role >= 0 and xk not in self.xq:
                self.xq[xk] = torch.empty((xk[1], xk[2]), dtype=torch.int8, device=self.device)
            self.layers.append(PackedLayer(l, packed, s, None if symmetric else z, bias, bos, xk, yk, sums, split_at,
                                           packed_hi, role))
            if split_at:
                out_rows = yk[0] * yk[1] * yk[2]
                need = mixdq.split_workspace_bytes(self.batch * l.H * l.H, l.Cin, split_at, out_rows, l.N)
            elif l.kind == "conv3x3":
                need = mixdq.conv3x3_workspace_bytes(self.batch, l.H, l.H, l.Cin, l.N, l.stride, l.w_bits, l.a_bits)
            else:
                rows = yk[0] * (yk[1] if len(yk) > 2 else 1) * (yk[2] if len(yk) > 3 else 1)
                if l.kind == "bos_kv" and l.a_bits == 8:
                    rows = self.batch * (synth.TOKENS_PER_PROMPT - 1)
                need = mixdq.workspace_bytes(rows, l.N, l.K, l.w_bits, l.a_bits)
            max_ws = max(max_ws, need)
        self.workspace = mixdq.new_workspace(max_ws, self.device)
        torch.cuda.synchronize()

    # ------------------------------------------------------------------ the timed pass
    def run_layer(self, pl: PackedLayer, workspace=None):
        l = pl.spec
        x, y = self.x[pl.x_key], self.y[pl.y_key]
        sx = self.x_scale.get(pl.x_key) if l.a_bits == 8 else None
        ws = workspace if workspace is not None else self.workspace
        if pl.split_at:
            s_lo, s_hi = self.x_split_scale[(pl.x_key, pl.split_at)]
            if l.kind == "conv3x3":
                return mixdq.conv3x3_a8_split(x, pl.split_at, pl.packed, pl.packed_hi, l.N, l.w_bits, pl.w_scale, s_lo,
                                              s_hi, pl.bias, l.stride, ws, self.status, out=y)
            return mixdq.linear_a8_split(x.reshape(-1, l.Cin), pl.split_at, pl.packed, pl.packed_hi, l.N, l.w_bits,
                                         pl.w_scale, s_lo, s_hi, pl.bias, ws, self.status, out=y.reshape(-1, l.N))
        if l.kind == "conv3x3" and pl.code_sums is not None:
            ax, az = self.x_asym[pl.x_key]
            return mixdq.conv3x3_a8_asym(x, pl.packed, l.N, l.w_bits, pl.w_scale, pl.code_sums, ax, az, pl.bias,
                                         l.stride, ws, self.status, out=y)
        if l.kind == "conv3x3":
            return mixdq.conv3x3(x, pl.packed, l.N, l.w_bits, pl.w_scale, pl.w_zero, l.a_bits, sx, pl.bias,
                                 l.stride, ws, self.status, out=y)
        if l.kind == "bos_kv" and l.a_bits == 8:
            return mixdq.crossattn_kv(x, pl.packed, l.N, l.w_bits, pl.w_scale, sx, pl.bos_out, ws, self.status,
                                      out=y)
        x2 = x.reshape(-1, x.shape[-1])
        if pl.qkv_role >= 0:
            xq = self.xq[pl.x_key]
            if pl.qkv_role == 0:
                mixdq.quantize_acts(x2, sx, out=xq)
            return mixdq.linear_q8(xq, pl.packed, l.N, l.w_bits, pl.w_scale, sx, pl.bias, self.status,
                                   out=y.reshape(-1, l.N))
        if pl.code_sums is not None:
            ax, az = self.x_asym[pl.x_key]
            return mixdq.linear_a8_asym(x2, pl.packed, l.N, l.w_bits, pl.w_scale, pl.code_sums, ax, az, pl.bias, ws,
                                        self.status, out=y.reshape(-1, l.N))
        return mixdq.linear(x2, pl.packed, l.N, l.w_bits, pl.w_scale, pl.w_zero, l.a_bits, sx, pl.bias, ws,
                            self.status, out=y.reshape(-1, l.N))

    def step(self, subset=None):
        for pl in (self.layers if subset is None else subset):
            self.run_layer(pl)

    # ------------------------------------------------------------------ accounting
    def total_ops(self, subset=None) -> int:
        group = self.layers if subset is None else subset
        if self.tokens > 0:
            return sum(2 * self.tokens * pl.spec.N * pl.spec.K for pl in group)
        return sum(pl.spec.ops(self.batch) for pl in group)

    def packed_weight_bytes(self) -> int:
        return sum(pl.packed.numel() + (0 if pl.packed_hi is None else pl.packed_hi.numel()) for pl in self.layers)

    def algorithmic_bytes(self, pl: PackedLayer) -> int:
        """Packed weights + per-channel params + input once + output once + bias."""
        l = pl.spec
        x, y = self.x[pl.x_key], self.y[pl.y_key]
        params = l.N * (4 if pl.w_zero is None else 8)
        return pl.packed.numel() + (0 if pl.packed_hi is None else pl.packed_hi.numel()) + params + x.numel() * 2 + y.numel() * 2 + (0 if pl.bias is None else l.N * 2)

    def uses_tensor_int8(self, pl: PackedLayer) -> bool:
        """True when the layer runs on the tcgen05 int8 engine (not the plain corner kernel)."""
        l = pl.spec
        if l.a_bits != 8:
            return False
        unit = l.Cin if l.kind == "conv3x3" else l.K
        return unit % 16 == 0 and l.N >= 16


def _main(argv=None) -> int:
    """Run one layer of the sweep a few times (e.g. under a profiler):

        python -m paper_2405_17873_b200.unet_sweep --layer attn_1280#0 --w-bits 4 --table w4a8 --batch 4

    Prints the layer's shape, the average time of a CUDA-graph replay of `--reps` runs and the
    device status word.
    """
    import argparse

    ap = argparse.ArgumentParser(description=_main.__doc__)
    ap.add_argument("--layer", required=True, help="layer name from synth.unet_layers(), e.g. ffn1_1280#0")
    ap.add_argument("--w-bits", type=int, default=None, help="override the table's weight bit-width")
    ap.add_argument("--table", default="w4a8", choices=["w4a8", "a16"])
    ap.add_argument("--batch", type=int, default=4)
    ap.add_argument("--reps", type=int, default=3)
    ap.add_argument("--tokens", type=int, default=0, help="linear layers only: run on this many rows (weight-bound regime)")
    ap.add_argument("--act-asym", action="store_true", help="asymmetric 8-bit activations (linear layers and 3x3 convolutions)")
    ap.add_argument("--shortcut-split", action="store_true",
                    help="one activation scale per branch for the concatenation-fed resnet convolutions of the up path")
    ap.add_argument("--eager", action="store_true", help="plain launches only, no graph and no timing")
    a = ap.parse_args(argv)

    specs = synth.unet_layers()
    (synth.assign_bits_w4a8 if a.table == "w4a8" else synth.assign_bits_weight_only)(specs)
    pick = [l for l in specs if l.name == a.layer]
    if not pick:
        raise SystemExit(f"no layer named {a.layer!r}")
    if a.w_bits is not None:
        pick[0].w_bits = a.w_bits
    sw = UNetSweep(a.batch, a.table, layers=pick, tokens=a.tokens, act_asym=a.act_asym,
                   shortcut_split=a.shortcut_split)
    pl = sw.layers[0]
    for _ in range(a.reps):
        sw.run_layer(pl)
    torch.cuda.synchronize()
    l = pl.spec
    line = f"{l.name} {l.kind} M={a.tokens if a.tokens > 0 else l.M * a.batch} N={l.N} K={l.K} W{l.w_bits}A{l.a_bits}"
    if not a.eager:
        st = torch.cuda.Stream()
        with torch.cuda.stream(st):
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=st):
                for _ in range(a.reps):
                    sw.run_layer(pl)
            g.replay()
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
        line += f" {e0.elapsed_time(e1) * 1e3 / a.reps:.1f} us/run"
    print(line, "status", int(sw.status.item()))
    return 0


if __name__ == "__main__":
    raise SystemExit(_main())
