"""The N > 1 path of the benchmark is "replicas only": every rank searches its own batches and
the ranks meet only for the barrier and the max-over-ranks of the timed region.  These tests run
that glue with two gloo ranks on the CPU."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import bench  # noqa: E402
from paper_2608_24067_b200 import synth  # noqa: E402


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        firsts = bench.replica_first_samples(rank, n_batches=2, batch=1000)
        # every rank generates its own samples; they must differ between ranks
        b = synth.sample_csr(50, 200, 7.0, seed=0, first_sample=firsts[0])
        ms_local = 10.0 + 5.0 * rank
        ms = bench.max_over_ranks(ms_local, dist, torch.device("cpu"))
        total = bench.aggregate_samples_per_s(world, 1000, ms)
        gathered = [None] * world
        dist.all_gather_object(gathered, (firsts, b.indices[:20].tolist()))
        if rank == 0:
            out.put((ms, total, gathered))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_replicas_take_disjoint_samples_and_report_the_slowest_rank():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, total, gathered = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert ms == 15.0  # the slower rank defines the step time
    assert abs(total - 2 * 1000 / 15e-3) < 1e-6
    (f0, i0), (f1, i1) = gathered
    assert f0 == [0, 1000] and f1 == [2000, 3000]  # disjoint sample ranges
    assert i0 != i1


def test_single_process_helpers():
    assert bench.replica_first_samples(0, 4, 250000) == [0, 250000, 500000, 750000]
    assert bench.replica_first_samples(3, 1, 10) == [30]
    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5
    assert bench.aggregate_samples_per_s(1, 1000000, 10.0) == 1e8
