"""ctypes binding of the C-ABI CUDA library (``libmixdq.so``).

Argument marshalling only: torch tensors supply device memory and the current stream,
every step of the path runs in the library's kernels.  There is no CPU fallback: if the
shared library is missing the first call raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libmixdq.so")

LAYOUT_CANONICAL = 0
LAYOUT_DEVICE = 1
TOKENS_PER_PROMPT = 77

_i64, _int, _vp, _sz = C.c_int64, C.c_int, C.c_void_p, C.c_size_t

_SIGNATURES = {
    "mixdq_version": (C.c_int, []),
    "mixdq_strerror": (C.c_char_p, [_int]),
    "mixdq_kernel_launches": (C.c_ulonglong, []),
    "mixdq_int8_tile_plan": (_int, [_i64, _i64, _i64, _int, C.POINTER(_int), C.POINTER(_int), C.POINTER(_int)]),
    "mixdq_linear_fused_quant_tile": (_int, [_i64, _i64, _i64, _int]),
    "mixdq_packed_bytes": (_int, [_i64, _i64, _int, _int, C.POINTER(_sz)]),
    "mixdq_weight_minmax_params": (_int, [_vp, _i64, _i64, _int, _int, _vp, _vp, _vp]),
    "mixdq_pack_weights": (_int, [_vp, _i64, _i64, _int, _vp, _vp, _int, _vp, _vp]),
    "mixdq_unpack_weights": (_int, [_vp, _i64, _i64, _int, _int, _int, _vp, _vp]),
    "mixdq_act_absmax": (_int, [_vp, _i64, _i64, _i64, _int, _vp, _vp]),
    "mixdq_act_scale_from_absmax": (_int, [_vp, _vp, _vp]),
    "mixdq_act_minmax": (_int, [_vp, _i64, _i64, _i64, _vp, _vp]),
    "mixdq_act_asym_params_from_minmax": (_int, [_vp, _vp, _vp, _vp]),
    "mixdq_weight_code_sums": (_int, [_vp, _i64, _i64, _int, _vp, _vp]),
    "mixdq_linear_a8_asym": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp, _vp,
                                    _sz, _vp, _vp]),
    "mixdq_linear_a8_asym_acc_i32": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp,
                                            _sz, _vp, _vp]),
    "mixdq_conv3x3_a8_asym": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp,
                                     _vp, _vp, _sz, _vp, _vp]),
    "mixdq_conv3x3_a8_asym_acc_i32": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _int, _vp, _vp, _vp,
                                             _vp, _vp, _sz, _vp, _vp]),
    "mixdq_quantize_acts": (_int, [_vp, _i64, _i64, _i64, _vp, _vp, _vp]),
    "mixdq_linear_q8": (_int, [_vp, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp]),
    "mixdq_conv3x3_q8": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _int, _vp, _vp, _vp, _vp, _vp, _vp]),
    "mixdq_linear_a8_fused_quant": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _i64, _int, _vp, _vp]),
    "mixdq_selftest_abandoned_wait": (_int, [_vp, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _int, _vp, _vp]),
    "mixdq_linear_q8_acc_i32": (_int, [_vp, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp]),
    "mixdq_split_workspace_bytes": (_int, [_i64, _i64, _i64, _i64, _i64, C.POINTER(_sz)]),
    "mixdq_linear_a8_split": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp, _vp,
                                     _sz, _vp, _vp]),
    "mixdq_linear_a8_split_acc_i32": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _int, _vp, _vp, _vp, _vp,
                                             _vp, _sz, _vp, _vp]),
    "mixdq_conv3x3_a8_split": (_int, [_vp, _i64, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _int, _int, _vp, _vp, _vp,
                                      _vp, _vp, _vp, _sz, _vp, _vp]),
    "mixdq_conv3x3_a8_split_acc_i32": (_int, [_vp, _i64, _i64, _i64, _i64, _i64, _vp, _vp, _i64, _int, _int, _vp, _vp,
                                              _vp, _vp, _vp, _sz, _vp, _vp]),
    "mixdq_workspace_bytes": (_int, [_i64, _i64, _i64, _int, _int, C.POINTER(_sz)]),
    "mixdq_conv3x3_workspace_bytes": (_int, [_i64, _i64, _i64, _i64, _i64, _int, _int, _int, C.POINTER(_sz)]),
    "mixdq_linear": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _int, _vp, _vp, _vp, _vp, _sz,
                            _vp, _vp]),
    "mixdq_linear_acc_i32": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _sz, _vp, _vp]),
    "mixdq_conv3x3": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _int, _vp, _vp, _int, _vp, _vp, _vp,
                             _vp, _sz, _vp, _vp]),
    "mixdq_conv3x3_acc_i32": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _int, _vp, _vp, _vp, _sz,
                                     _vp, _vp]),
    "mixdq_conv1x1": (_int, [_vp, _i64, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _int, _vp, _vp, _vp, _vp,
                             _sz, _vp, _vp]),
    "mixdq_crossattn_kv": (_int, [_vp, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp, _sz, _vp, _vp]),
    "mixdq_crossattn_kv_acc_i32": (_int, [_vp, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _sz, _vp, _vp]),
    "mixdq_probe_mma_loop": (_int, [_int, _int, C.POINTER(C.c_double), _vp, _vp]),
    "mixdq_static_scratch_bytes": (_sz, []),
    "mixdq_linear_a8_static_scratch": (_int, [_vp, _i64, _i64, _i64, _vp, _i64, _int, _vp, _vp, _vp, _vp, _vp,
                                              _vp]),
}

EXPORTS = tuple(_SIGNATURES)

_lib = None


class MixdqError(RuntimeError):
    pass


def lib():
    """Load the shared library (once).  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise MixdqError(f"{LIB_PATH} is missing: build it with python -m paper_2405_17873_b200.build")
        L = C.CDLL(LIB_PATH)
        for name, (res, args) in _SIGNATURES.items():
            fn = getattr(L, name)
            fn.restype = res
            fn.argtypes = args
        _lib = L
    return _lib


def _chk(rc: int, what: str):
    if rc != 0:
        raise MixdqError(f"{what}: {lib().mixdq_strerror(rc).decode()} ({rc})")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_cuda and t.is_contiguous(), "device-resident contiguous tensors only"
    return C.c_void_p(t.data_ptr())


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def version() -> int:
    return lib().mixdq_version()


def kernel_launches() -> int:
    return int(lib().mixdq_kernel_launches())


def int8_tile_plan(M: int, N: int, k_blocks: int, w_bits: int, with_splits: bool = False):
    """(tile_rows, tile_cols[, reduction_splits]) of the int8 tensor-core GEMM for this shape on the current device."""
    r, c, sp = _int(0), _int(0), _int(0)
    _chk(lib().mixdq_int8_tile_plan(M, N, k_blocks, w_bits, C.byref(r), C.byref(c), C.byref(sp)), "mixdq_int8_tile_plan")
    return (r.value, c.value, sp.value) if with_splits else (r.value, c.value)


def linear_fused_quant_tile(M: int, N: int, K: int, w_bits: int) -> int:
    """Tile width of the one-kernel (fused quantization) form for this linear layer, 0 when it runs as two kernels."""
    r = lib().mixdq_linear_fused_quant_tile(M, N, K, w_bits)
    if r < 0:
        _chk(r, "mixdq_linear_fused_quant_tile")
    return r


def packed_bytes(N: int, K: int, bits: int, layout: int = LAYOUT_DEVICE) -> int:
    out = _sz(0)
    _chk(lib().mixdq_packed_bytes(N, K, bits, layout, C.byref(out)), "mixdq_packed_bytes")
    return out.value


def workspace_bytes(rows: int, N: int, K: int, w_bits: int, act_bits: int) -> int:
    out = _sz(0)
    _chk(lib().mixdq_workspace_bytes(rows, N, K, w_bits, act_bits, C.byref(out)), "mixdq_workspace_bytes")
    return out.value


def conv3x3_workspace_bytes(B: int, H: int, W: int, Cin: int, Cout: int, stride: int, w_bits: int,
                            act_bits: int) -> int:
    out = _sz(0)
    _chk(lib().mixdq_conv3x3_workspace_bytes(B, H, W, Cin, Cout, stride, w_bits, act_bits, C.byref(out)),
         "mixdq_conv3x3_workspace_bytes")
    return out.value


def new_workspace(nbytes: int, device="cuda") -> Optional[torch.Tensor]:
    """Zero-filled scratch buffer of the size mixdq_workspace_bytes reported."""
    if nbytes == 0:
        return None
    return torch.zeros(nbytes, dtype=torch.uint8, device=device)


def weight_minmax_params(W: torch.Tensor, bits: int, symmetric: bool, scale_out: Optional[torch.Tensor] = None,
                         zero_out: Optional[torch.Tensor] = None):
    N, K = W.shape
    scale = scale_out if scale_out is not None else torch.empty(N, dtype=torch.float32, device=W.device)
    zero = zero_out if zero_out is not None else torch.zeros(N, dtype=torch.int32, device=W.device)
    _chk(lib().mixdq_weight_minmax_params(_ptr(W), N, K, bits, int(symmetric), _ptr(scale), _ptr(zero),
                                          _stream()), "mixdq_weight_minmax_params")
    return scale, zero


def pack_weights(W: torch.Tensor, bits: int, scale: torch.Tensor, zero: Optional[torch.Tensor] = None,
                 layout: int = LAYOUT_DEVICE, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    N, K = W.shape
    if out is None:
        out = torch.zeros(packed_bytes(N, K, bits, layout), dtype=torch.uint8, device=W.device)
    _chk(lib().mixdq_pack_weights(_ptr(W), N, K, bits, _ptr(scale), _ptr(zero), layout, _ptr(out), _stream()),
         "mixdq_pack_weights")
    return out


def unpack_weights(packed: torch.Tensor, N: int, K: int, bits: int, is_signed: bool,
                   layout: int = LAYOUT_DEVICE) -> torch.Tensor:
    codes = torch.empty((N, K), dtype=torch.int16, device=packed.device)
    _chk(lib().mixdq_unpack_weights(_ptr(packed), N, K, bits, int(is_signed), layout, _ptr(codes), _stream()),
         "mixdq_unpack_weights")
    return codes


def act_absmax(X: torch.Tensor, skip_rows_mod: int = 0) -> torch.Tensor:
    X2 = X.reshape(-1, X.shape[-1])
    out = torch.empty(1, dtype=torch.float32, device=X.device)
    _chk(lib().mixdq_act_absmax(_ptr(X2), X2.shape[0], X2.shape[1], X2.shape[1], skip_rows_mod, _ptr(out),
                                _stream()), "mixdq_act_absmax")
    return out


def act_scale_from_absmax(amax: torch.Tensor) -> torch.Tensor:
    out = torch.empty(1, dtype=torch.float32, device=amax.device)
    _chk(lib().mixdq_act_scale_from_absmax(_ptr(amax), _ptr(out), _stream()), "mixdq_act_scale_from_absmax")
    return out


def act_scale(X: torch.Tensor, skip_rows_mod: int = 0) -> torch.Tensor:
    """Dynamic per-tensor int8 scale max|X| / 127, computed on the device."""
    return act_scale_from_absmax(act_absmax(X, skip_rows_mod))


def act_minmax(X: torch.Tensor) -> torch.Tensor:
    """Device fp32 [2]: min(min x, 0), max(max x, 0)."""
    X2 = X.reshape(-1, X.shape[-1])
    out = torch.empty(2, dtype=torch.float32, device=X.device)
    _chk(lib().mixdq_act_minmax(_ptr(X2), X2.shape[0], X2.shape[1], X2.stride(0), _ptr(out), _stream()),
         "mixdq_act_minmax")
    return out


def act_asym_params(X: torch.Tensor):
    """Asymmetric 8-bit activation parameters (device fp32 scale [1], device int32 zero-point [1])."""
    mm = act_minmax(X)
    scale = torch.empty(1, dtype=torch.float32, device=X.device)
    zero = torch.empty(1, dtype=torch.int32, device=X.device)
    _chk(lib().mixdq_act_asym_params_from_minmax(_ptr(mm), _ptr(scale), _ptr(zero), _stream()),
         "mixdq_act_asym_params_from_minmax")
    return scale, zero


def weight_code_sums(packed_W: torch.Tensor, N: int, K: int, bits: int) -> torch.Tensor:
    out = torch.empty(N, dtype=torch.int32, device=packed_W.device)
    _chk(lib().mixdq_weight_code_sums(_ptr(packed_W), N, K, bits, _ptr(out), _stream()), "mixdq_weight_code_sums")
    return out


def _ws(workspace):
    return (_ptr(workspace), workspace.numel() if workspace is not None else 0)


def linear(X, packed_W, N: int, w_bits: int, w_scale, w_zero=None, act_bits: int = 8, act_scale=None,
           bias=None, workspace=None, status=None, out=None):
    M, K = X.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits, _ptr(w_scale), _ptr(w_zero),
                            act_bits, _ptr(act_scale), _ptr(bias), _ptr(Y), wp, wb, _ptr(status), _stream()),
         "mixdq_linear")
    return Y


def linear_acc_i32(X, packed_W, N: int, w_bits: int, act_scale, workspace=None, status=None):
    M, K = X.shape
    acc = torch.empty((M, N), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear_acc_i32(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits, _ptr(act_scale),
                                    _ptr(acc), wp, wb, _ptr(status), _stream()), "mixdq_linear_acc_i32")
    return acc


def linear_a8_asym(X, packed_W, N: int, w_bits: int, w_scale, w_code_sums, act_scale, act_zero, bias=None,
                   workspace=None, status=None, out=None):
    M, K = X.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear_a8_asym(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits, _ptr(w_scale),
                                    _ptr(w_code_sums), _ptr(act_scale), _ptr(act_zero), _ptr(bias), _ptr(Y),
                                    wp, wb, _ptr(status), _stream()), "mixdq_linear_a8_asym")
    return Y


def linear_a8_asym_acc_i32(X, packed_W, N: int, w_bits: int, w_code_sums, act_scale, act_zero, workspace=None,
                           status=None):
    M, K = X.shape
    acc = torch.empty((M, N), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear_a8_asym_acc_i32(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits,
                                            _ptr(w_code_sums), _ptr(act_scale), _ptr(act_zero), _ptr(acc), wp,
                                            wb, _ptr(status), _stream()), "mixdq_linear_a8_asym_acc_i32")
    return acc


def _out_hw(H, W, stride):
    return (H - 1) // stride + 1, (W - 1) // stride + 1


def conv3x3(X, packed_W, Cout: int, w_bits: int, w_scale, w_zero=None, act_bits: int = 8, act_scale=None,
            bias=None, stride: int = 1, workspace=None, status=None, out=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    Y = out if out is not None else torch.empty((B, Ho, Wo, Cout), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3(_ptr(X), B, H, W, Cin, _ptr(packed_W), Cout, stride, w_bits, _ptr(w_scale),
                             _ptr(w_zero), act_bits, _ptr(act_scale), _ptr(bias), _ptr(Y), wp, wb,
                             _ptr(status), _stream()), "mixdq_conv3x3")
    return Y


def conv3x3_a8_asym(X, packed_W, Cout: int, w_bits: int, w_scale, w_code_sums, act_scale, act_zero, bias=None,
                    stride: int = 1, workspace=None, status=None, out=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    Y = out if out is not None else torch.empty((B, Ho, Wo, Cout), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3_a8_asym(_ptr(X), B, H, W, Cin, _ptr(packed_W), Cout, stride, w_bits, _ptr(w_scale),
                                     _ptr(w_code_sums), _ptr(act_scale), _ptr(act_zero), _ptr(bias), _ptr(Y),
                                     wp, wb, _ptr(status), _stream()), "mixdq_conv3x3_a8_asym")
    return Y


def conv3x3_a8_asym_acc_i32(X, packed_W, Cout: int, w_bits: int, w_code_sums, act_scale, act_zero,
                            stride: int = 1, workspace=None, status=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    acc = torch.empty((B, Ho, Wo, Cout), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3_a8_asym_acc_i32(_ptr(X), B, H, W, Cin, _ptr(packed_W), Cout, stride, w_bits,
                                             _ptr(w_code_sums), _ptr(act_scale), _ptr(act_zero), _ptr(acc), wp,
                                             wb, _ptr(status), _stream()), "mixdq_conv3x3_a8_asym_acc_i32")
    return acc


def quantize_acts(X, act_scale, out=None):
    """int8 codes [rows, K] of X fp16 [rows, K] with the per-tensor scale *act_scale (device)."""
    rows, K = X.shape
    Xq = out if out is not None else torch.empty((rows, K), dtype=torch.int8, device=X.device)
    assert X.stride(1) == 1
    _chk(lib().mixdq_quantize_acts(C.c_void_p(X.data_ptr()), rows, K, X.stride(0), _ptr(act_scale), _ptr(Xq),
                                   _stream()), "mixdq_quantize_acts")
    return Xq


def linear_q8(Xq, packed_W, N: int, w_bits: int, w_scale, act_scale, bias=None, status=None, out=None):
    M, K = Xq.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib().mixdq_linear_q8(_ptr(Xq), M, K, _ptr(packed_W), N, w_bits, _ptr(w_scale), _ptr(act_scale),
                               _ptr(bias), _ptr(Y), _ptr(status), _stream()), "mixdq_linear_q8")
    return Y


def linear_a8_fused_quant(X, packed_W, N: int, w_bits: int, w_scale, act_scale, bias=None, tile_cols: int = 128,
                          status=None, out=None):
    """mixdq_linear (8-bit activations) as one kernel on 128 x tile_cols tiles, whatever the planner would choose."""
    M, K = X.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=X.device)
    _chk(lib().mixdq_linear_a8_fused_quant(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits, _ptr(w_scale),
                                           _ptr(act_scale), _ptr(bias), _ptr(Y), Y.stride(0), tile_cols, _ptr(status),
                                           _stream()), "mixdq_linear_a8_fused_quant")
    return Y


def conv3x3_q8(Xq, packed_W, Cout: int, w_bits: int, w_scale, act_scale, bias=None, stride: int = 1, status=None,
               out=None):
    B, H, W, Cin = Xq.shape
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    Y = out if out is not None else torch.empty((B, Ho, Wo, Cout), dtype=torch.float16, device=Xq.device)
    _chk(lib().mixdq_conv3x3_q8(_ptr(Xq), B, H, W, Cin, _ptr(packed_W), Cout, stride, w_bits, _ptr(w_scale),
                                _ptr(act_scale), _ptr(bias), _ptr(Y), _ptr(status), _stream()), "mixdq_conv3x3_q8")
    return Y


def selftest_abandoned_wait(Xq, packed_W, N: int, w_bits: int, w_scale, act_scale, drop_k_block: int, status):
    """mixdq_linear_q8 with one weight tile never requested: *status becomes MIXDQ_ERR_TIMEOUT (-6)."""
    M, K = Xq.shape
    Y = torch.empty((M, N), dtype=torch.float16, device=Xq.device)
    _chk(lib().mixdq_selftest_abandoned_wait(_ptr(Xq), M, K, _ptr(packed_W), N, w_bits, _ptr(w_scale), _ptr(act_scale),
                                             _ptr(Y), drop_k_block, _ptr(status), _stream()),
         "mixdq_selftest_abandoned_wait")
    return Y


def linear_q8_acc_i32(Xq, packed_W, N: int, w_bits: int, status=None):
    M, K = Xq.shape
    acc = torch.empty((M, N), dtype=torch.int32, device=Xq.device)
    _chk(lib().mixdq_linear_q8_acc_i32(_ptr(Xq), M, K, _ptr(packed_W), N, w_bits, _ptr(acc), _ptr(status),
                                       _stream()), "mixdq_linear_q8_acc_i32")
    return acc


def split_workspace_bytes(in_rows: int, row_len: int, split_at: int, out_rows: int, N: int) -> int:
    out = _sz(0)
    _chk(lib().mixdq_split_workspace_bytes(in_rows, row_len, split_at, out_rows, N, C.byref(out)),
         "mixdq_split_workspace_bytes")
    return out.value


def linear_a8_split(X, split_at: int, packed_W_lo, packed_W_hi, N: int, w_bits: int, w_scale, act_scale_lo,
                    act_scale_hi, bias=None, workspace=None, status=None, out=None):
    M, K = X.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear_a8_split(_ptr(X), M, K, X.stride(0), split_at, _ptr(packed_W_lo), _ptr(packed_W_hi), N,
                                     w_bits, _ptr(w_scale), _ptr(act_scale_lo), _ptr(act_scale_hi), _ptr(bias),
                                     _ptr(Y), wp, wb, _ptr(status), _stream()), "mixdq_linear_a8_split")
    return Y


def linear_a8_split_acc_i32(X, split_at: int, packed_W_lo, packed_W_hi, N: int, w_bits: int, act_scale_lo,
                            act_scale_hi, workspace=None, status=None):
    M, K = X.shape
    lo = torch.empty((M, N), dtype=torch.int32, device=X.device)
    hi = torch.empty((M, N), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_linear_a8_split_acc_i32(_ptr(X), M, K, X.stride(0), split_at, _ptr(packed_W_lo),
                                             _ptr(packed_W_hi), N, w_bits, _ptr(act_scale_lo), _ptr(act_scale_hi),
                                             _ptr(lo), _ptr(hi), wp, wb, _ptr(status), _stream()),
         "mixdq_linear_a8_split_acc_i32")
    return lo, hi


def conv3x3_a8_split(X, split_at: int, packed_W_lo, packed_W_hi, Cout: int, w_bits: int, w_scale, act_scale_lo,
                     act_scale_hi, bias=None, stride: int = 1, workspace=None, status=None, out=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    Y = out if out is not None else torch.empty((B, Ho, Wo, Cout), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3_a8_split(_ptr(X), B, H, W, Cin, split_at, _ptr(packed_W_lo), _ptr(packed_W_hi), Cout,
                                      stride, w_bits, _ptr(w_scale), _ptr(act_scale_lo), _ptr(act_scale_hi),
                                      _ptr(bias), _ptr(Y), wp, wb, _ptr(status), _stream()),
         "mixdq_conv3x3_a8_split")
    return Y


def conv3x3_a8_split_acc_i32(X, split_at: int, packed_W_lo, packed_W_hi, Cout: int, w_bits: int, act_scale_lo,
                             act_scale_hi, stride: int = 1, workspace=None, status=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    lo = torch.empty((B, Ho, Wo, Cout), dtype=torch.int32, device=X.device)
    hi = torch.empty((B, Ho, Wo, Cout), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3_a8_split_acc_i32(_ptr(X), B, H, W, Cin, split_at, _ptr(packed_W_lo),
                                              _ptr(packed_W_hi), Cout, stride, w_bits, _ptr(act_scale_lo),
                                              _ptr(act_scale_hi), _ptr(lo), _ptr(hi), wp, wb, _ptr(status),
                                              _stream()), "mixdq_conv3x3_a8_split_acc_i32")
    return lo, hi


def conv3x3_acc_i32(X, packed_W, Cout: int, w_bits: int, act_scale, stride: int = 1, workspace=None,
                    status=None):
    B, H, W, Cin = X.shape
    Ho, Wo = _out_hw(H, W, stride)
    acc = torch.empty((B, Ho, Wo, Cout), dtype=torch.int32, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv3x3_acc_i32(_ptr(X), B, H, W, Cin, _ptr(packed_W), Cout, stride, w_bits,
                                     _ptr(act_scale), _ptr(acc), wp, wb, _ptr(status), _stream()),
         "mixdq_conv3x3_acc_i32")
    return acc


def conv1x1(X, packed_W, Cout: int, w_bits: int, w_scale, w_zero=None, act_bits: int = 8, act_scale=None,
            bias=None, workspace=None, status=None):
    B, H, W, Cin = X.shape
    Y = torch.empty((B, H, W, Cout), dtype=torch.float16, device=X.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_conv1x1(_ptr(X), B, H, W, Cin, _ptr(packed_W), Cout, w_bits, _ptr(w_scale), _ptr(w_zero),
                             act_bits, _ptr(act_scale), _ptr(bias), _ptr(Y), wp, wb, _ptr(status), _stream()),
         "mixdq_conv1x1")
    return Y


def crossattn_kv(text_emb, packed_W, N: int, w_bits: int, w_scale, act_scale, bos_out, workspace=None,
                 status=None, out=None):
    B, T, Kt = text_emb.shape
    assert T == TOKENS_PER_PROMPT
    Y = out if out is not None else torch.empty((B, T, N), dtype=torch.float16, device=text_emb.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_crossattn_kv(_ptr(text_emb), B, Kt, _ptr(packed_W), N, w_bits, _ptr(w_scale),
                                  _ptr(act_scale), _ptr(bos_out), _ptr(Y), wp, wb, _ptr(status), _stream()),
         "mixdq_crossattn_kv")
    return Y


def crossattn_kv_acc_i32(text_emb, packed_W, N: int, w_bits: int, act_scale, workspace=None, status=None):
    B, T, Kt = text_emb.shape
    assert T == TOKENS_PER_PROMPT
    acc = torch.empty((B, T - 1, N), dtype=torch.int32, device=text_emb.device)
    wp, wb = _ws(workspace)
    _chk(lib().mixdq_crossattn_kv_acc_i32(_ptr(text_emb), B, Kt, _ptr(packed_W), N, w_bits, _ptr(act_scale),
                                          _ptr(acc), wp, wb, _ptr(status), _stream()),
         "mixdq_crossattn_kv_acc_i32")
    return acc


def static_scratch_bytes() -> int:
    return lib().mixdq_static_scratch_bytes()


def linear_a8_static_scratch(X, packed_W, N: int, w_bits: int, w_scale, act_scale, bias=None, status=None,
                             out=None):
    """W8A8 / W4A8 linear whose scratch is the library's built-in array: for callers that cannot
    allocate device memory.  The output tensor is still the caller's (``out``, or a fresh one here)."""
    M, K = X.shape
    Y = out if out is not None else torch.empty((M, N), dtype=torch.float16, device=X.device)
    _chk(lib().mixdq_linear_a8_static_scratch(_ptr(X), M, K, X.stride(0), _ptr(packed_W), N, w_bits,
                                              _ptr(w_scale), _ptr(act_scale), _ptr(bias), _ptr(Y), _ptr(status),
                                              _stream()), "mixdq_linear_a8_static_scratch")
    return Y


def probe_mma_loop(kind: int, batches: int, repeats: int = 3) -> float:
    """Tensor-core MMA-loop peak in TOP/s (kind 1: int8, kind 0: fp16), best of ``repeats``."""
    ops = C.c_double(0.0)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    best = 0.0
    for _ in range(repeats + 1):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        _chk(lib().mixdq_probe_mma_loop(kind, batches, C.byref(ops), _ptr(status), _stream()), "mixdq_probe_mma_loop")
        b.record()
        torch.cuda.synchronize()
        if int(status.item()) != 0:
            raise MixdqError("mixdq_probe_mma_loop: device-side wait timed out")
        best = max(best, ops.value / (a.elapsed_time(b) * 1e-3) / 1e12)
    return best
