"""GPU parity of the offline steps: parameters, packed bytes and codes are bit-exact."""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import dev, host

pytestmark = pytest.mark.gpu


def _weights(N, K, seed):
    W = synth.normal_f16((N, K), 0.02, seed)
    W[1, :] = 0
    W[2, :] = np.float16(0.0173)
    W[3, :] = -np.abs(W[3, :])
    return W


@pytest.mark.parametrize("bits", [2, 3, 4, 8])
@pytest.mark.parametrize("symmetric", [True, False])
@pytest.mark.parametrize("N,K", [(37, 77), (64, 320), (130, 1000)])
def test_minmax_params_bit_exact(bits, symmetric, N, K):
    W = _weights(N, K, 100 + bits + N)
    s_ref, z_ref = orc.weight_minmax_params(W, bits, symmetric)
    s, z = mixdq.weight_minmax_params(dev(W), bits, symmetric)
    assert np.array_equal(host(s).view(np.uint32), s_ref.view(np.uint32))
    assert np.array_equal(host(z), z_ref)


@pytest.mark.parametrize("bits,symmetric", [(2, False), (3, False), (4, False), (4, True), (8, False), (8, True)])
@pytest.mark.parametrize("N,K", [(5, 1), (37, 77), (64, 320), (33, 1000), (16, 2048)])
def test_packed_bytes_and_codes_bit_exact(bits, symmetric, N, K):
    W = _weights(max(N, 4), K, 200 + bits + K)[:N] if N >= 4 else _weights(4, K, 200 + bits + K)[:N]
    W = np.ascontiguousarray(W)
    s_ref, z_ref = orc.weight_minmax_params(W, bits, symmetric)
    zr = None if symmetric else z_ref
    codes_ref = orc.quantize_weights(W, bits, s_ref, zr)
    packed_ref = orc.pack_codes(codes_ref, bits, zr)
    Wd, sd = dev(W), dev(s_ref)
    zd = None if symmetric else dev(z_ref)
    canon = mixdq.pack_weights(Wd, bits, sd, zd, mixdq.LAYOUT_CANONICAL)
    assert np.array_equal(host(canon).reshape(N, -1), packed_ref)
    assert np.array_equal(host(mixdq.unpack_weights(canon, N, K, bits, symmetric, mixdq.LAYOUT_CANONICAL)),
                          codes_ref)
    devp = mixdq.pack_weights(Wd, bits, sd, zd, mixdq.LAYOUT_DEVICE)
    assert np.array_equal(host(mixdq.unpack_weights(devp, N, K, bits, symmetric, mixdq.LAYOUT_DEVICE)),
                          codes_ref)


def test_unpack_reads_oracle_packed_bytes():
    rng = np.random.default_rng(3)
    for bits, signed in ((2, False), (3, False), (4, True), (4, False), (8, True), (8, False)):
        lo, hi = (-(2 ** (bits - 1) - 1), 2 ** (bits - 1) - 1) if signed else (0, 2 ** bits - 1)
        codes = rng.integers(lo, hi + 1, size=(9, 75)).astype(np.int16)
        packed = orc.pack_codes(codes, bits, np.zeros(9, np.int32))
        buf = torch.zeros(packed.size + 16, dtype=torch.uint8, device="cuda")
        buf[:packed.size] = dev(packed.reshape(-1))
        got = mixdq.unpack_weights(buf, 9, 75, bits, signed, mixdq.LAYOUT_CANONICAL)
        assert np.array_equal(host(got), codes)


@pytest.mark.parametrize("rows,cols,skip", [(77 * 3, 2048, 77), (300, 320, 0), (5, 7, 0), (154, 64, 77)])
def test_act_absmax_and_scale_exact(rows, cols, skip):
    X = synth.normal_f16((rows, cols), 1.0, seed=rows + cols)
    X[0, 1] = 900.0
    if rows > 77:
        X[77, 2] = -901.0
    amax_ref = orc.act_absmax(X, skip)
    amax = mixdq.act_absmax(dev(X), skip)
    assert host(amax)[0] == amax_ref
    sc = mixdq.act_scale_from_absmax(amax)
    assert host(sc).view(np.uint32)[0] == np.float32(orc.act_scale(amax_ref, 8)).view(np.uint32)
    zero = mixdq.act_scale(torch.zeros(4, 8, dtype=torch.float16, device="cuda"))
    assert host(zero)[0] == 1.0
