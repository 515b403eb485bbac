"""The N > 1 path of the benchmark is 'replicas only': ranks do not exchange data, the only collective
is the max-over-ranks of the step time.  Two gloo ranks on CPU check that reduction and the
whole-job throughput formula."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2506_10443_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = 10.0 if rank == 0 else 25.0        # rank 1 is the slow replica
        got = replicas.max_over_ranks([ms, float(rank)])
        agg = replicas.aggregate_throughput(units_per_rank_step=1000.0, steps=5, elapsed_ms_this_rank=ms, world=world)
        out.put((rank, got, agg))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_report_the_slowest_time_and_the_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, agg in res:
        assert got == [25.0, 1.0]
        assert agg["ms"] == 25.0 and agg["ms_per_step"] == 5.0
        assert agg["units_per_s"] == 1000.0 * 5 * 2 / 0.025          # both replicas' work over the max time
        assert agg["units_per_s_one_replica"] == agg["units_per_s"] / 2


def test_single_process_is_the_identity():
    assert replicas.max_over_ranks([3.5, 1.0]) == [3.5, 1.0]
    agg = replicas.aggregate_throughput(100.0, 10, 2.0, 1)
    assert agg["units_per_s"] == 100.0 * 10 / 0.002
