"""Host-side logic of the multi-GPU (replicas only) benchmark path, on CPU with gloo, world size 2."""
import os
import sys
from pathlib import Path

import pytest
import torch
import torch.multiprocessing as mp

ROOT = Path(__file__).resolve().parent.parent


def _worker(rank, world, port, out):
    sys.path.insert(0, str(ROOT))
    import torch.distributed as dist
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # rank 0 needs 100 ms of decode per step set, rank 1 needs 250 ms: the job is as slow as rank 1
    dec_ms = 100.0 if rank == 0 else 250.0
    value, e2e, dmax, cmax = bench.aggregate_replicas(dec_ms, dec_ms + 50.0, steps=2, dec_tokens=511, gen_tokens=512,
                                                      world=world, device="cpu")
    out[rank] = (value, e2e, dmax, cmax)
    dist.barrier()
    dist.destroy_process_group()


def test_replica_aggregation_takes_the_slowest_rank():
    world, port = 2, 29517
    mgr = mp.Manager()
    out = mgr.dict()
    mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
    assert len(out) == 2
    for rank in range(world):
        value, e2e, dmax, cmax = out[rank]
        assert dmax == 250.0 and cmax == 300.0
        assert value == pytest.approx(2 * 2 * 511 / 0.250)       # all ranks' tokens over the max time
        assert e2e == pytest.approx(2 * 2 * 512 / 0.300)


def test_single_rank_aggregation_is_plain_throughput():
    sys.path.insert(0, str(ROOT))
    import bench
    value, e2e, _, _ = bench.aggregate_replicas(1000.0, 1250.0, 1, 511, 512, 1, device="cpu")
    assert value == pytest.approx(511.0) and e2e == pytest.approx(512 / 1.25)
