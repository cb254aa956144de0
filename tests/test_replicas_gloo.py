"""The N > 1 path of the benchmark: independent replicas, a barrier, and the slowest rank's time.
Run here as two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2605_15250_b200 import replicas, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 10.0 + 5.0 * rank  # rank 1 is the slow replica
        dist.barrier()
        ms = replicas.max_over_ranks(my_ms)
        # every rank draws its own batch: same shapes, different values
        w = synth.WORKLOADS["C0"].with_(seed=replicas.replica_seed(synth.WORKLOADS["C0"].seed, rank))
        x = synth.make_inputs(w)
        sums = [torch.zeros(1, dtype=torch.float64) for _ in range(world)]
        dist.all_gather(sums, x["q_c"].double().sum().reshape(1))
        out.put((rank, ms, [float(t) for t in sums], tuple(x["q_c"].shape)))
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_rank_and_distinct_batches():
    world, port = 2, _free_port()
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, sums, shape in res:
        assert ms == 15.0  # max over ranks, on every rank
        assert sums[0] != sums[1]  # the replicas decode different batches
        assert shape == res[0][3]
    # whole-job throughput: world * batch * s_q tokens per (slowest) step
    assert replicas.aggregate_tokens_per_s(2, 64, 1, 0.1) == 2 * 64 / 1e-4
    # without a process group the reduction is the identity
    assert replicas.max_over_ranks(3.5) == 3.5
