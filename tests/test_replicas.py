"""The N > 1 policy of the benchmark (independent replicas, max-over-ranks timing) on CPU:
two gloo ranks."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_15018_b200 import replicas, workloads


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    wl = replicas.replica_workload(workloads.CONFIGS["cfg1"], rank)
    h = workloads.hidden_states(wl, 0)
    times = replicas.max_over_ranks([10.0 + rank, 5.0 - rank])
    dist.barrier()
    out[rank] = (wl.seed, float(h.float().sum()), times)
    dist.destroy_process_group()


def test_two_replicas_have_own_inputs_and_agree_on_the_slowest_time():
    world = 2
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, _free_port(), out), nprocs=world, join=True)
    assert out[0][0] != out[1][0] and out[0][1] != out[1][1]          # own seed, own hidden states
    assert out[0][2] == out[1][2] == [11.0, 5.0]                       # max over ranks, on every rank
    v = replicas.aggregate_tokens_per_s(world, 8, 16, 2.0)
    assert v == 2 * 8 * 16 / 2e-3


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert replicas.replica_workload(workloads.CONFIGS["cfg2"], 0).seed == workloads.CONFIGS["cfg2"].seed
