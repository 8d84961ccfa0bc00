"""The N > 1 path of bench.py on CPU: two gloo ranks, each an independent replica; the job time
is the maximum over ranks and the throughput the sum over replicas (no data-path collective)."""
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
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        my_ms = 2.0 if rank == 0 else 5.0            # rank 1 is the slow replica
        ms = bench.max_over_ranks_ms(my_ms, world, torch.device("cpu"))
        tops = bench.whole_job_tops(1e12, ms, world)
        # each rank's oracle result on its own seeded batch is independent of the other rank
        import aser_synth as synth
        lay = synth.make_layer(4, 16, 128, seed=synth.seed_for(2, rank), n_cal=8)
        checksum = float(lay.X.astype("float64").sum())
        gathered = [None] * world
        dist.all_gather_object(gathered, checksum)
        out.put((rank, ms, tops, gathered))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_like_replicas():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = [out.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, tops, gathered in results:
        assert ms == 5.0                                  # max over ranks
        assert tops == pytest.approx(2 * 1e12 / 5e-3 / 1e12)   # both replicas' work over that time
        assert gathered[0] != gathered[1]                 # different seeds, different batches
    assert {r[0] for r in results} == {0, 1}


def test_single_rank_needs_no_process_group():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks_ms(3.0, 1) == 3.0
    assert bench.whole_job_tops(2e12, 1.0, 1) == pytest.approx(2000.0)
