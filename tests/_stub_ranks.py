"""A rank of the multi-process timing protocol with a stand-in step (a short sleep), for the CPU test of
the launcher: started N times by shard.launch_ranks, joins a gloo group, runs shard.timed_job and lets
rank 0 write one JSON line to the file named on the command line."""
import json
import os
import sys
import time

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2406_17276_b200 import shard  # noqa: E402


def main():
    out_path, steps = sys.argv[1], int(sys.argv[2])
    rank, world, local = shard.init_ranks("gloo")
    calls = []

    def step(i):
        calls.append(i)
        time.sleep(0.002 * (rank + 1))          # rank 1 is the slow one

    value, ms = shard.timed_job(step, steps, 2, units_per_step=4.0, timer=shard.HostTimer(), sync=lambda: None)
    if rank == 0:
        with open(out_path, "w") as f:
            json.dump({"value": value, "ms": ms, "n_gpus": world, "calls": len(calls), "local": local}, f)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
