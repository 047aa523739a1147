"""The N>1 path of bench.py on CPU: two gloo ranks, independent replicas, max-over-ranks timing."""
import os

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_26266_b200 import inputs, replicas


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    w = replicas.replica_workload(inputs.WORKLOADS["tiny"], rank)
    q, _, _ = inputs.make_chunk(w, 0, tokens=8)
    mine = [10.0 + rank, 5.0 - rank, float(q[0, 0, 0, 0])]
    red = replicas.max_over_ranks(mine)
    out.put((rank, w.seed, red, int(q.sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_to_the_slowest_and_use_independent_data():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, red0, sum0), (r1, s1, red1, sum1) = res
    assert (r0, r1) == (0, 1) and s1 == s0 + 1000
    assert red0 == red1 and red0[0] == 11.0 and red0[1] == 5.0
    assert sum0 != sum1                                   # different replicas, different data
    w = inputs.WORKLOADS["tiny"]
    assert np.isclose(replicas.aggregate_value(w.flops(), 2, 1.0), 2 * w.flops() / 1e-3 / 1e12)


def test_single_process_is_identity():
    assert replicas.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
