"""A rank of a replica job with the device work replaced by fixed numbers: what `bench.py --gpus N` starts N
times, minus CUDA.  Used by tests/test_replicas_gloo.py to run bench.py's own launcher (spawn_ranks) and its
aggregation over ranks on CPU with the gloo backend.  Not a benchmark."""
import json
import os
import sys

import torch
import torch.distributed as dist

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)
import bench  # noqa: E402


def main():
    out = sys.argv[sys.argv.index("--out") + 1]
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    assert os.environ["MASTER_ADDR"] == "127.0.0.1"
    dist.init_process_group("gloo", rank=rank, world_size=world)
    dist.barrier()
    ms, ms_e2e = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 20.0 - 3.0 * rank, world, torch.device("cpu"))
    tokens = bench.tokens_processed(steps=4, batch=2, gen_len=256, schedule_steps=256, world=world)
    if rank == 0:
        with open(out, "w") as f:
            json.dump({"n_gpus": world, "ms": ms, "ms_e2e": ms_e2e, "tokens": tokens,
                       "local_ranks_seen": int(os.environ["LOCAL_RANK"]) + 1}, f)
    dist.barrier()
    dist.destroy_process_group()


if __name__ == "__main__":
    main()
