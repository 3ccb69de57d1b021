"""World-size-2 CPU ranks (gloo) through the bookkeeping the multi-GPU benchmark uses:
per-rank seeds, batch split, MAX-over-ranks timing, whole-job throughput."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_24433_b200 import replicas, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world),
                      LOCAL_RANK=str(rank))
    info = replicas.RankInfo.from_env()
    dist.init_process_group("gloo", rank=info.rank, world_size=info.world)
    try:
        # every rank times its own replica: rank r "took" (r + 1) seconds over 10 units of work
        seconds = float(rank + 1)
        slowest = replicas.max_over_ranks(seconds, dist)
        rate = replicas.job_throughput(10.0, seconds, dist)
        # each replica draws its own batch
        site = synth.config1_site()
        x = synth.make_site(site, replicas.replica_seed(2, info.rank)).x
        digest = torch.tensor([float(np.asarray(x, dtype=np.float64).sum())], dtype=torch.float64)
        both = [torch.zeros_like(digest) for _ in range(world)]
        dist.all_gather(both, digest)
        share = list(replicas.split_batches(7, info.world, info.rank))
        out.put((rank, slowest, rate, [float(b.item()) for b in both], share))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(120)
def test_two_cpu_ranks_max_timing_and_job_rate():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=100) for _ in range(world))
    for p in procs:
        p.join(30)
        assert p.exitcode == 0
    shares = []
    for rank, slowest, rate, digests, share in got:
        assert slowest == 2.0                       # the MAX over ranks, on both ranks
        assert rate == pytest.approx(20.0 / 2.0)    # all ranks' units over the slowest rank's time
        assert digests[0] != digests[1]             # the replicas ran different batches
        shares += share
    assert got[0][3] == got[1][3]                   # and agree on what each other drew
    assert sorted(shares) == list(range(7))


def test_single_process_is_identity():
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.job_throughput(8.0, 2.0) == 4.0
    assert replicas.replica_seed(2, 0) == 2
    assert [len(replicas.split_batches(10, 4, r)) for r in range(4)] == [2, 3, 2, 3]
    with pytest.raises(ValueError):
        replicas.split_batches(4, 2, 2)
