"""The N > 1 path of the benchmark (independent replicas, max-over-ranks timing) on two
gloo ranks on the CPU."""
import os
import socket
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2405_17873_b200 import replicas
    replicas.barrier()
    # rank 1 is the slow one for the step time, rank 0 for the end-to-end time
    ms = [10.0 + 5.0 * rank, 30.0 - 4.0 * rank]
    step_ms, e2e_ms = replicas.max_over_ranks(ms)
    rate = replicas.whole_job_rate(6.0e12, step_ms)
    out[rank] = (replicas.world(), step_ms, e2e_ms, rate)
    replicas.barrier()
    dist.destroy_process_group()


def test_two_replicas_report_max_time_and_whole_job_rate():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert set(res) == {0, 1}
    for rank in (0, 1):
        w, step_ms, e2e_ms, rate = res[rank]
        assert w == 2
        assert step_ms == 15.0 and e2e_ms == 30.0          # the slowest rank decides
        assert abs(rate - 2 * 6.0e12 / 15.0e-3) < 1e-3 * rate   # both replicas' work in that time


def test_single_process_is_the_identity():
    from paper_2405_17873_b200 import replicas
    assert replicas.world() == 1
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.whole_job_rate(10.0, 1000.0) == 10.0
