"""The allocation-free int8 linear entry point gives the same result as mixdq_linear.

Some users of the library run where device memory cannot be allocated on their behalf (the
GPU's memory is owned by a server's own manager, or an allocation's device-wide
synchronization is not acceptable in their loop).  For them the library keeps the layer's scratch -- the int8 copy
of the activations between the quantization pass and the GEMM -- in a fixed array of its own.
The test calls that entry point through the C ABI twice in a row -- the second call finds the
array as the first one left it -- and compares both results with the ordinary entry point that
takes a caller workspace and with the CPU oracle.
"""
import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bits", [8, 4])
def test_static_scratch_matches_workspace_entry_point(bits):
    M, K, N = 256, 5120, 320          # few output tiles, long reduction: the reduction is split over a cluster
    X = synth.normal_f16((M, K), 1.0, seed=901)
    W = synth.normal_f16((N, K), 0.02, seed=902)
    b = synth.normal_f16((N,), 0.01, seed=903)
    Xd, bd = dev(X), dev(b)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    st = status_word()
    ws = workspace_for(M, N, K, bits)
    assert 0 < mixdq.workspace_bytes(M, N, K, bits, 8) <= mixdq.static_scratch_bytes()
    y_ref = host(mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, bd, workspace=ws, status=st))
    s_o, _, codes = oracle_weights(W, bits, True)
    _, y_oracle = orc.linear_a8(X, codes, s_o, orc.act_scale(orc.act_absmax(X), 8), b)
    out = torch.empty((M, N), dtype=torch.float16, device="cuda")
    for _ in range(2):
        out.zero_()
        mixdq.linear_a8_static_scratch(Xd, packed, N, bits, s, sx, bd, status=st, out=out)
        torch.cuda.synchronize()
        assert int(host(st)[0]) == 0
        assert_close(host(out), y_ref)
        assert_close(host(out), y_oracle)
    # a second shape right after, so that the array is reused with another tiling
    X2 = synth.normal_f16((130, 1280), 1.0, seed=904)
    W2 = synth.normal_f16((200, 1280), 0.02, seed=905)
    s2, _, p2 = device_weights(W2, bits, True)
    X2d = dev(X2)
    sx2 = mixdq.act_scale(X2d)
    y2_ref = host(mixdq.linear(X2d, p2, 200, bits, s2, None, 8, sx2, None, workspace=workspace_for(130, 200, 1280, bits)))
    y2 = host(mixdq.linear_a8_static_scratch(X2d, p2, 200, bits, s2, sx2))
    assert_close(y2, y2_ref)
    s2_o, _, codes2 = oracle_weights(W2, bits, True)
    assert_close(y2, orc.linear_a8(X2, codes2, s2_o, orc.act_scale(orc.act_absmax(X2), 8), None)[1])


def test_static_scratch_rejects_oversized_problem():
    M, N, K = 4096, 2048, 256          # 32 MiB of partial sums: more than the built-in array holds
    assert mixdq.workspace_bytes(M, N, K, 8, 8) > mixdq.static_scratch_bytes()
    Xd = torch.zeros((M, K), dtype=torch.float16, device="cuda")
    packed = torch.zeros(N * K, dtype=torch.uint8, device="cuda")
    s = torch.ones(N, dtype=torch.float32, device="cuda")
    sx = torch.ones(1, dtype=torch.float32, device="cuda")
    with pytest.raises(mixdq.MixdqError, match="workspace"):
        mixdq.linear_a8_static_scratch(Xd, packed, N, 8, s, sx)
