"""ctypes front end of the MixDQ CPU oracle (test infrastructure, not product code).

The arithmetic lives in ``mixdq_oracle.c``; this file only marshals numpy
arrays and composes the C steps into the layer-level results the CUDA library
is compared with.  fp16 tensors are numpy ``float16`` arrays (passed as their
uint16 bit patterns).  Nothing here imports the CUDA package.

Layer-level compositions and the passages they follow:
  * ``linear_a8`` / ``conv3x3_a8``: quantize activations per tensor, integer
    MACs, per-channel dequantize + bias (Sec. 4.1 "Quantization Scheme",
    Sec. 4.3 "Speedup of model inference").
  * ``linear_a16`` / ``conv3x3_a16``: weight-only rows of Table 1.
  * ``crossattn_kv``: BOS-aware K/V projection of Sec. 3.1.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mixdq_oracle.c")
_LIB = os.path.join(_HERE, "libmixdq_oracle.so")

TOKENS_PER_PROMPT = 77  # CLIP text length used by the paper's models (Sec. 3.1, Fig. 4)


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (baseline x86-64 code so the binary runs on any host)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        cmd = ["gcc", "-O3", "-fopenmp", "-ffp-contract=off", "-fno-fast-math", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        build()
        L = C.CDLL(_LIB)
        L.orc_half_to_double.restype = C.c_double
        L.orc_half_to_double.argtypes = [C.c_uint16]
        L.orc_double_to_half.restype = C.c_uint16
        L.orc_double_to_half.argtypes = [C.c_double]
        L.orc_packed_row_bytes.restype = C.c_int64
        L.orc_packed_row_bytes.argtypes = [C.c_int64, C.c_int]
        _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _f16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.float16, a.dtype
    return a


def _chk(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def num_threads() -> int:
    return int(lib().orc_num_threads())


def half_to_double(bits: int) -> float:
    return float(lib().orc_half_to_double(int(bits)))


def double_to_half(d: float) -> int:
    return int(lib().orc_double_to_half(float(d)))


# ---------------------------------------------------------------- quantizer

def weight_minmax_params(W, bits: int, symmetric: bool):
    """Per-output-channel (scale fp32[N], zero int32[N]) of W fp16 [N,K]."""
    W = _f16(W)
    N, K = W.shape
    scale = np.empty(N, np.float32)
    zero = np.zeros(N, np.int32)
    _chk(lib().orc_weight_minmax_params(_p(W), C.c_int64(N), C.c_int64(K), bits, int(symmetric),
                                        _p(scale), _p(zero)), "weight_minmax_params")
    return scale, zero


def quantize_weights(W, bits: int, scale, zero=None):
    """Integer codes int16 [N,K]; ``zero=None`` selects symmetric signed codes."""
    W = _f16(W)
    N, K = W.shape
    scale = np.ascontiguousarray(scale, np.float32)
    zero = None if zero is None else np.ascontiguousarray(zero, np.int32)
    codes = np.empty((N, K), np.int16)
    _chk(lib().orc_quantize_weights(_p(W), C.c_int64(N), C.c_int64(K), bits, _p(scale), _p(zero),
                                    _p(codes)), "quantize_weights")
    return codes


def dequantize_weights(codes, scale, zero=None):
    codes = np.ascontiguousarray(codes, np.int16)
    N, K = codes.shape
    scale = np.ascontiguousarray(scale, np.float32)
    zero = None if zero is None else np.ascontiguousarray(zero, np.int32)
    out = np.empty((N, K), np.float64)
    _chk(lib().orc_dequantize_weights(_p(codes), C.c_int64(N), C.c_int64(K), _p(scale), _p(zero),
                                      _p(out)), "dequantize_weights")
    return out


def act_absmax(X, skip_rows_mod: int = 0) -> np.float32:
    X = _f16(X)
    X2 = X.reshape(-1, X.shape[-1])
    out = np.zeros(1, np.float32)
    _chk(lib().orc_act_absmax(_p(X2), C.c_int64(X2.shape[0]), C.c_int64(X2.shape[1]),
                              C.c_int64(X2.shape[1]), int(skip_rows_mod), _p(out)), "act_absmax")
    return out[0]


def act_scale(amax, bits: int = 8) -> np.float32:
    out = np.zeros(1, np.float32)
    _chk(lib().orc_act_scale(C.c_float(float(amax)), bits, _p(out)), "act_scale")
    return out[0]


def quantize_acts(X, scale, bits: int = 8):
    X = _f16(X)
    q = np.empty(X.shape, np.int8)
    _chk(lib().orc_quantize_acts(_p(X), C.c_int64(X.size), bits, C.c_float(float(scale)), _p(q)),
         "quantize_acts")
    return q


def act_minmax_params(X):
    """Asymmetric per-tensor 8-bit activation parameters: (scale fp32, zero-point int in [0, 255])."""
    X = _f16(X)
    scale = np.zeros(1, np.float32)
    zero = np.zeros(1, np.int32)
    _chk(lib().orc_act_minmax_params(_p(X), C.c_int64(X.size), _p(scale), _p(zero)), "act_minmax_params")
    return scale[0], int(zero[0])


def quantize_acts_asym(X, scale, zero: int):
    """Centred codes clamp(rne(x / s) + z, 0, 255) - z as int16."""
    X = _f16(X)
    c = np.empty(X.shape, np.int16)
    _chk(lib().orc_quantize_acts_asym(_p(X), C.c_int64(X.size), C.c_float(float(scale)), C.c_int32(int(zero)), _p(c)),
         "quantize_acts_asym")
    return c


def int_gemm_i16(cx, qw):
    cx = np.ascontiguousarray(cx, np.int16)
    qw = np.ascontiguousarray(qw, np.int16)
    M, K = cx.shape
    N, K2 = qw.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    _chk(lib().orc_int_gemm_i16(_p(cx), _p(qw), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(acc)), "int_gemm_i16")
    return acc


# ------------------------------------------------------------------ packing

def packed_row_bytes(K: int, bits: int) -> int:
    return int(lib().orc_packed_row_bytes(C.c_int64(K), bits))


def pack_codes(codes, bits: int, pad_code=None):
    codes = np.ascontiguousarray(codes, np.int16)
    N, K = codes.shape
    pad = None if pad_code is None else np.ascontiguousarray(pad_code, np.int32)
    out = np.zeros((N, packed_row_bytes(K, bits)), np.uint8)
    _chk(lib().orc_pack_codes(_p(codes), C.c_int64(N), C.c_int64(K), bits, _p(pad), _p(out)),
         "pack_codes")
    return out


def unpack_codes(packed, K: int, bits: int, is_signed: bool):
    packed = np.ascontiguousarray(packed, np.uint8)
    N = packed.shape[0]
    out = np.empty((N, K), np.int16)
    _chk(lib().orc_unpack_codes(_p(packed), C.c_int64(N), C.c_int64(K), bits, int(is_signed),
                                _p(out)), "unpack_codes")
    return out


# ----------------------------------------------------------- integer engines

def int_gemm(qx, qw):
    qx = np.ascontiguousarray(qx, np.int8)
    qw = np.ascontiguousarray(qw, np.int16)
    M, K = qx.shape
    N, K2 = qw.shape
    assert K == K2
    acc = np.empty((M, N), np.int32)
    _chk(lib().orc_int_gemm(_p(qx), _p(qw), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(acc)),
         "int_gemm")
    return acc


def int_conv3x3(qx, qw, stride: int = 1):
    """qx int8 NHWC [B,H,W,C]; qw int16 [N,3,3,C] -> int32 [B,Ho,Wo,N]."""
    qx = np.ascontiguousarray(qx, np.int8)
    qw = np.ascontiguousarray(qw, np.int16)
    B, H, W, Cin = qx.shape
    N = qw.shape[0]
    assert qw.shape == (N, 3, 3, Cin)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    acc = np.empty((B, Ho, Wo, N), np.int32)
    _chk(lib().orc_int_conv3x3(_p(qx), _p(qw), C.c_int64(B), C.c_int64(H), C.c_int64(W),
                               C.c_int64(Cin), C.c_int64(N), stride, _p(acc)), "int_conv3x3")
    return acc


def int_conv3x3_i16(cx, qw, stride: int = 1):
    """cx int16 NHWC [B,H,W,C] (centred codes q - z); qw int16 [N,3,3,C] -> int32 [B,Ho,Wo,N]."""
    cx = np.ascontiguousarray(cx, np.int16)
    qw = np.ascontiguousarray(qw, np.int16)
    B, H, W, Cin = cx.shape
    N = qw.shape[0]
    assert qw.shape == (N, 3, 3, Cin)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    acc = np.empty((B, Ho, Wo, N), np.int32)
    _chk(lib().orc_int_conv3x3_i16(_p(cx), _p(qw), C.c_int64(B), C.c_int64(H), C.c_int64(W),
                                   C.c_int64(Cin), C.c_int64(N), stride, _p(acc)), "int_conv3x3_i16")
    return acc


def dequant_epilogue(acc, act_scale_, w_scale, bias=None):
    acc = np.ascontiguousarray(acc, np.int32)
    N = acc.shape[-1]
    M = acc.size // N
    w_scale = np.ascontiguousarray(w_scale, np.float32)
    bias = None if bias is None else _f16(bias)
    Y = np.empty(acc.shape, np.float16)
    _chk(lib().orc_dequant_epilogue(_p(acc), C.c_int64(M), C.c_int64(N), C.c_float(float(act_scale_)),
                                    _p(w_scale), _p(bias), _p(Y)), "dequant_epilogue")
    return Y


def dequant_epilogue_split(acc_lo, acc_hi, s_lo, s_hi, w_scale, bias=None):
    acc_lo = np.ascontiguousarray(acc_lo, np.int32)
    acc_hi = np.ascontiguousarray(acc_hi, np.int32)
    assert acc_lo.shape == acc_hi.shape
    N = acc_lo.shape[-1]
    M = acc_lo.size // N
    w_scale = np.ascontiguousarray(w_scale, np.float32)
    bias = None if bias is None else _f16(bias)
    Y = np.empty(acc_lo.shape, np.float16)
    _chk(lib().orc_dequant_epilogue_split(_p(acc_lo), _p(acc_hi), C.c_int64(M), C.c_int64(N),
                                          C.c_float(float(s_lo)), C.c_float(float(s_hi)), _p(w_scale), _p(bias),
                                          _p(Y)), "dequant_epilogue_split")
    return Y


# --------------------------------------------------------------- weight-only

def weight_only_linear(X, codes, scale, zero=None, bias=None):
    X = _f16(X)
    codes = np.ascontiguousarray(codes, np.int16)
    M, K = X.shape
    N = codes.shape[0]
    assert codes.shape == (N, K)
    scale = np.ascontiguousarray(scale, np.float32)
    zero = None if zero is None else np.ascontiguousarray(zero, np.int32)
    bias = None if bias is None else _f16(bias)
    Y = np.empty((M, N), np.float16)
    _chk(lib().orc_weight_only_linear(_p(X), _p(codes), C.c_int64(M), C.c_int64(N), C.c_int64(K),
                                      _p(scale), _p(zero), _p(bias), _p(Y)), "weight_only_linear")
    return Y


def weight_only_conv3x3(X, codes, scale, zero=None, bias=None, stride: int = 1):
    X = _f16(X)
    codes = np.ascontiguousarray(codes, np.int16)
    B, H, W, Cin = X.shape
    N = codes.shape[0]
    assert codes.shape == (N, 3, 3, Cin)
    scale = np.ascontiguousarray(scale, np.float32)
    zero = None if zero is None else np.ascontiguousarray(zero, np.int32)
    bias = None if bias is None else _f16(bias)
    Ho, Wo = (H - 1) // stride + 1, (W - 1) // stride + 1
    Y = np.empty((B, Ho, Wo, N), np.float16)
    _chk(lib().orc_weight_only_conv3x3(_p(X), _p(codes), C.c_int64(B), C.c_int64(H), C.c_int64(W),
                                       C.c_int64(Cin), C.c_int64(N), stride, _p(scale), _p(zero),
                                       _p(bias), _p(Y)), "weight_only_conv3x3")
    return Y


def fp_linear(X, W):
    X = _f16(X)
    W = _f16(W)
    M, K = X.shape
    N = W.shape[0]
    Y = np.empty((M, N), np.float16)
    _chk(lib().orc_fp_linear(_p(X), _p(W), C.c_int64(M), C.c_int64(N), C.c_int64(K), _p(Y)),
         "fp_linear")
    return Y


# --------------------------------------------------------- layer compositions

def linear_a8(X, codes, w_scale, act_scale_, bias=None):
    """W8A8 / W4A8 linear: returns (int32 accumulators, fp16 output)."""
    X = _f16(X)
    qx = quantize_acts(X, act_scale_, 8)
    acc = int_gemm(qx.reshape(-1, X.shape[-1]), codes)
    return acc, dequant_epilogue(acc, act_scale_, w_scale, bias)


def linear_a8_asym(X, codes, w_scale, act_scale_, act_zero: int, bias=None):
    """W8A8 / W4A8 linear with asymmetric per-tensor activations (Sec. 4.1):
    acc = sum_k (q_x - z_x) q_w (int32), y = fp16(acc * s_x * s_w[n] + bias[n])."""
    X = _f16(X)
    cx = quantize_acts_asym(X, act_scale_, act_zero)
    acc = int_gemm_i16(cx.reshape(-1, X.shape[-1]), codes)
    return acc, dequant_epilogue(acc, act_scale_, w_scale, bias)


def conv3x3_a8(X, codes, w_scale, act_scale_, bias=None, stride: int = 1):
    """X fp16 NHWC, codes int16 [N,3,3,C]: returns (int32 acc, fp16 out), both NHWC."""
    X = _f16(X)
    qx = quantize_acts(X, act_scale_, 8)
    acc = int_conv3x3(qx, codes, stride)
    return acc, dequant_epilogue(acc, act_scale_, w_scale, bias)


def conv3x3_a8_asym(X, codes, w_scale, act_scale_, act_zero: int, bias=None, stride: int = 1):
    """3x3 convolution with asymmetric per-tensor activations (Sec. 4.1): X fp16 NHWC, codes int16
    [N,3,3,C]; the zero padding is the real value 0, i.e. code z.  Returns (int32 acc, fp16 out), NHWC."""
    X = _f16(X)
    cx = quantize_acts_asym(X, act_scale_, act_zero)
    acc = int_conv3x3_i16(cx, codes, stride)
    return acc, dequant_epilogue(acc, act_scale_, w_scale, bias)


def linear_a8_split(X, codes, w_scale, s_lo, s_hi, split_at: int, bias=None):
    """Shortcut-splitting on a linear layer (Sec. 4.1): columns [0, split_at) of X are quantized with s_lo,
    the rest with s_hi; returns (acc_lo, acc_hi, fp16 out)."""
    X = _f16(X)
    codes = np.ascontiguousarray(codes, np.int16)
    q_lo = quantize_acts(np.ascontiguousarray(X[:, :split_at]), s_lo, 8)
    q_hi = quantize_acts(np.ascontiguousarray(X[:, split_at:]), s_hi, 8)
    acc_lo = int_gemm(q_lo, np.ascontiguousarray(codes[:, :split_at]))
    acc_hi = int_gemm(q_hi, np.ascontiguousarray(codes[:, split_at:]))
    return acc_lo, acc_hi, dequant_epilogue_split(acc_lo, acc_hi, s_lo, s_hi, w_scale, bias)


def conv3x3_a8_split(X, codes, w_scale, s_lo, s_hi, split_at: int, bias=None, stride: int = 1):
    """The same on a 3x3 convolution: X fp16 NHWC whose channels [0, split_at) and [split_at, C) come from
    the two concatenated tensors; codes int16 [N,3,3,C]."""
    X = _f16(X)
    codes = np.ascontiguousarray(codes, np.int16)
    q_lo = quantize_acts(np.ascontiguousarray(X[..., :split_at]), s_lo, 8)
    q_hi = quantize_acts(np.ascontiguousarray(X[..., split_at:]), s_hi, 8)
    acc_lo = int_conv3x3(q_lo, np.ascontiguousarray(codes[..., :split_at]), stride)
    acc_hi = int_conv3x3(q_hi, np.ascontiguousarray(codes[..., split_at:]), stride)
    return acc_lo, acc_hi, dequant_epilogue_split(acc_lo, acc_hi, s_lo, s_hi, w_scale, bias)


def linear_a16(X, codes, scale, zero=None, bias=None):
    return weight_only_linear(X, codes, scale, zero, bias)


def conv3x3_a16(X, codes, scale, zero=None, bias=None, stride: int = 1):
    return weight_only_conv3x3(X, codes, scale, zero, bias, stride)


def bos_row(e_bos, W):
    """Stored fp16 output of the BOS token from the unquantized weight (Sec. 3.1)."""
    return fp_linear(_f16(e_bos).reshape(1, -1), W)[0]


def crossattn_kv(text_emb, codes, w_scale, act_scale_, bos_out):
    """BOS-aware K or V projection (Sec. 3.1).

    text_emb fp16 [B,77,Kt]; rows t >= 1 take the int8 path with the given
    per-tensor scale; row t = 0 of every prompt is the stored ``bos_out``
    copied bit for bit.  Returns (int32 acc [B,76,N], fp16 out [B,77,N]).
    """
    text_emb = _f16(text_emb)
    B, T, Kt = text_emb.shape
    assert T == TOKENS_PER_PROMPT
    rest = np.ascontiguousarray(text_emb[:, 1:, :]).reshape(B * (T - 1), Kt)
    acc, y = linear_a8(rest, codes, w_scale, act_scale_, None)
    N = codes.shape[0]
    out = np.empty((B, T, N), np.float16)
    out[:, 0, :] = _f16(bos_out)[None, :]
    out[:, 1:, :] = y.reshape(B, T - 1, N)
    return acc.reshape(B, T - 1, N), out


def crossattn_act_scale(text_emb):
    """Per-tensor int8 scale over tokens 1..76 of every prompt (Sec. 3.1)."""
    text_emb = _f16(text_emb)
    B, T, Kt = text_emb.shape
    return act_scale(act_absmax(text_emb.reshape(B * T, Kt), skip_rows_mod=T), 8)
