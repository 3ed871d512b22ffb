"""The kernels' bounded waits end in a status word.

Every wait on a shared-memory barrier in the tensor-core kernels has a cycle budget; when it runs out the
kernel raises an abort flag, lets its copies in flight land, reports MIXDQ_ERR_TIMEOUT through the caller's
status word, releases its tensor memory and returns.  The self-test entry point makes that happen without any
fault: one weight tile is announced to its barrier and never requested.  Afterwards the same GPU context runs
an ordinary layer with full parity against the oracle."""
import time

import numpy as np
import pytest
import torch

from oracle import mixdq_oracle as orc
from paper_2405_17873_b200 import mixdq, synth
from helpers import assert_close, dev, device_weights, host, oracle_weights, status_word, workspace_for

pytestmark = pytest.mark.gpu

MIXDQ_ERR_TIMEOUT = -6


@pytest.mark.parametrize("bits,M,N,K,drop", [(8, 128, 128, 512, 2), (4, 256, 384, 1280, 7), (8, 4096, 2048, 512, 1)])
def test_abandoned_wait_reports_timeout_and_context_survives(bits, M, N, K, drop):
    X = synth.normal_f16((M, K), 1.0, seed=61)
    W = synth.normal_f16((N, K), 0.02, seed=62)
    Xd = dev(X)
    s, _, packed = device_weights(W, bits, True)
    sx = mixdq.act_scale(Xd)
    xq = mixdq.quantize_acts(Xd, sx)
    st = status_word()
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    mixdq.selftest_abandoned_wait(xq, packed, N, bits, s, sx, drop, st)
    torch.cuda.synchronize()                     # returns: the kernel gave up by itself
    dt = time.perf_counter() - t0
    assert int(host(st)[0]) == MIXDQ_ERR_TIMEOUT
    assert dt < 20.0, dt
    # the context is intact and tensor memory was released: the same layer, ordinary call, full parity
    st2 = status_word()
    s_ref, _, codes = oracle_weights(W, bits, True)
    sx_ref = orc.act_scale(orc.act_absmax(X), 8)
    acc_ref, y_ref = orc.linear_a8(X, codes, s_ref, sx_ref, None)
    ws = workspace_for(M, N, K, bits)
    acc = mixdq.linear_acc_i32(Xd, packed, N, bits, sx, workspace=ws, status=st2)
    y = mixdq.linear(Xd, packed, N, bits, s, None, 8, sx, None, workspace=ws, status=st2)
    torch.cuda.synchronize()
    assert int(host(st2)[0]) == 0
    assert np.array_equal(host(acc), acc_ref)
    assert_close(host(y), y_ref)
