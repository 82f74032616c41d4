"""N > 1 is replicas only: every rank runs its own sessions, there is no
data-path collective.  What the ranks do share is the bench's timing protocol:
barrier, max over ranks of the device time, sum of the units processed.  This
runs that host logic with world_size 2 on the gloo backend (CPU)."""
import os
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    ms = 10.0 + 5.0 * rank                      # rank 1 is slower
    ms_e2e = 20.0 - 3.0 * rank                  # rank 0 is slower end to end
    agg = bench.aggregate_over_ranks(ms, ms_e2e, world, torch.device("cpu"))
    tokens = bench.tokens_processed(steps=4, batch=2, gen_len=256, schedule_steps=256, world=world)
    if rank == 0:
        out.put((agg, tokens))
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_units():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    agg, tokens = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert agg == (15.0, 20.0)                  # max over ranks of each time
    assert tokens == 4 * 2 * 2                  # one token per sequence per step, both replicas


def test_single_rank_is_identity():
    import bench
    assert bench.aggregate_over_ranks(3.5, 7.0, 1, torch.device("cpu")) == (3.5, 7.0)
    assert bench.tokens_processed(256, 1, 256, 256, 1) == 256


def test_gpus_flag_without_a_launcher_spawns_the_ranks(tmp_path):
    """`python bench.py --gpus N` started plainly must itself start N ranks (one per GPU) and report n_gpus = N;
    under a launcher (WORLD_SIZE set) and for the reference arm it must not spawn again."""
    import json
    import bench
    assert bench.wants_spawn(2, "ours", {}) and bench.wants_spawn(8, "ours", {"PATH": "/usr/bin"})
    assert not bench.wants_spawn(1, "ours", {})
    assert not bench.wants_spawn(2, "ours", {"WORLD_SIZE": "2"})
    assert not bench.wants_spawn(2, "reference", {})
    out = tmp_path / "line.json"
    stub = os.path.join(ROOT, "tests", "replica_stub.py")
    env_before = dict(os.environ)
    rc = bench.spawn_ranks(2, ["--out", str(out)], script=stub)          # bench.py's own launcher, CPU ranks
    assert rc == 0 and dict(os.environ) == env_before
    line = json.loads(out.read_text())
    assert line["n_gpus"] == 2 and line["ms"] == 15.0 and line["ms_e2e"] == 20.0 and line["tokens"] == 16
