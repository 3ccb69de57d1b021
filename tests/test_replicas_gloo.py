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


def _bench(*args, timeout=150):
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    return subprocess.run([sys.executable, os.path.join(root, "bench.py"), *args], capture_output=True, text=True,
                          timeout=timeout, env=env, cwd=root)


@pytest.mark.timeout(200)
def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`bench.py --gpus 2` outside torchrun starts two ranks itself; with --dry-run they are CPU ranks (gloo) that
    run only the MAX-over-ranks bookkeeping, and rank 0 alone prints the line."""
    import json
    r = _bench("--gpus", "2", "--dry-run")
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, r.stdout
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["ms_per_step"] == 2.0            # the slower of the two made-up ranks
    assert out["value"] == pytest.approx(20.0 / 2e-3)                  # both ranks' units over the slowest duration
    assert out["seed_of_last_rank"] == replicas.replica_seed(2, 1)


@pytest.mark.skipif(torch.cuda.is_available() and torch.cuda.device_count() >= 2, reason="needs a machine with fewer than 2 GPUs")
def test_bench_refuses_more_gpus_than_the_machine_has():
    r = _bench("--gpus", "2", "--steps", "1", "--warmup", "1")
    assert r.returncode != 0 and "needs 2 CUDA devices" in r.stderr
    assert not [ln for ln in r.stdout.splitlines() if ln.startswith("{")]   # and prints no result line
