"""Shared glue for the GPU parity tests: run one layer through the CUDA library (via the
ctypes binding over the C ABI) and through the CPU oracle on the same seeded inputs."""
import numpy as np
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq

DEV = "cuda"


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


def host(t):
    return t.detach().cpu().numpy()


def tol(y_ref):
    """Output tolerance of the path: |y - y_ref| <= 1e-3 * max|y_ref| + 1e-3."""
    return 1e-3 * float(np.abs(y_ref.astype(np.float64)).max()) + 1e-3


def assert_close(y, y_ref):
    d = np.abs(y.astype(np.float64) - y_ref.astype(np.float64))
    assert np.isfinite(y.astype(np.float64)).all()
    assert d.max() <= tol(y_ref), (d.max(), tol(y_ref))


def oracle_weights(W2d, bits, symmetric):
    """(scale, zero-or-None, codes int16 [N,K]) from the oracle."""
    s, z = orc.weight_minmax_params(W2d, bits, symmetric)
    codes = orc.quantize_weights(W2d, bits, s, None if symmetric else z)
    return s, (None if symmetric else z), codes


def device_weights(W2d, bits, symmetric, layout=mixdq.LAYOUT_DEVICE):
    """(scale, zero-or-None, packed) on the device, through the library's own packer."""
    Wd = dev(W2d)
    s, z = mixdq.weight_minmax_params(Wd, bits, symmetric)
    packed = mixdq.pack_weights(Wd, bits, s, None if symmetric else z, layout)
    return s, (None if symmetric else z), packed


def status_word():
    return torch.zeros(1, dtype=torch.int32, device=DEV)


def workspace_for(rows, N, K, w_bits, act_bits=8):
    return mixdq.new_workspace(mixdq.workspace_bytes(rows, N, K, w_bits, act_bits))
