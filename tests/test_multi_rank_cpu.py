"""The N>1 path of bench.py on CPU: replicas only, no data-path collective.
Two gloo ranks check the max-over-ranks timing and the whole-job aggregate."""
import os
import socket
import sys

import pytest
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
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    my_ms = 1.0 + 0.5 * rank                      # rank 1 is the slower replica
    dist.barrier()
    ms_max = bench.max_over_ranks(my_ms, dist)
    value = bench.whole_job_tokens_per_s(world, 1, ms_max)
    out[rank] = (ms_max, value)
    dist.barrier()
    dist.destroy_process_group()


def test_two_gloo_ranks_take_the_slowest_rank_and_sum_the_replicas():
    world = 2
    port = _free_port()
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms_max, value = res[0]
    assert ms_max == pytest.approx(1.5)
    assert value == pytest.approx(2 * 1 / 1.5e-3)


def test_single_rank_helpers():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(2.0, None) == 2.0
    assert bench.whole_job_tokens_per_s(1, 64, 2.0) == pytest.approx(32000.0)


def test_algorithmic_bytes_follow_the_realised_gate():
    sys.path.insert(0, ROOT)
    import numpy as np
    import bench
    import synthetic as S
    spec = S.config3("10")
    ng = spec.n_groups
    fired = np.zeros((4, ng), bool)
    ab0 = bench.algorithmic_bytes(spec, fired)
    assert ab0["fast"] == 880803840 and ab0["w"] == 0
    assert ab0["dense"] == 12 * 4096 * 4096 * 2 * 28 + ab0["act"]
    fired[:, 1] = True                      # the attn_out group of layer 0, every step
    ab1 = bench.algorithmic_bytes(spec, fired)
    assert ab1["w"] == 4096 * 4096 * 2
    fired[:] = True
    assert bench.algorithmic_bytes(spec, fired)["w"] == 12 * 4096 * 4096 * 2 * 28
