"""The multi-process side of the benchmark on CPU: two gloo ranks, no GPU.

Sequences are independent, so ranks share nothing but the timing protocol: each rank gets its
own seeded workload, the job's time is the slowest rank's, its throughput the trees of all
ranks over that time.  The oracle stands in for the device step here (host logic only).
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2406_17276_b200 import shard, synth


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        w = shard.rank_workload(synth.WORKLOADS["c1"], rank)
        ld, lt = synth.make_tables(w, H=64, V=512)
        roots = synth.root_tokens(2, 512, w.seed + 1)
        dist.barrier()
        r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, -np.inf)      # this rank's two sequences
        dist.barrier()
        ms_local = 10.0 * (rank + 1)                                            # a made-up time per rank
        value, ms = shard.whole_job(units_local=2.0, ms_local=ms_local)
        total_nodes = shard.sum_over_ranks(float(r.n_sel.sum()))
        np.save(os.path.join(out_dir, f"rank{rank}.npy"),
                np.array([value, ms, total_nodes, float(r.n_sel.sum()), float(roots[0]), float(ld.view(np.uint16)[0, :8].sum())]))
    finally:
        dist.destroy_process_group()


@pytest.mark.timeout(300)
def test_two_ranks_share_only_the_clock(tmp_path):
    world = 2
    mp.spawn(_rank_main, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    a = np.load(tmp_path / "rank0.npy"); b = np.load(tmp_path / "rank1.npy")
    # both ranks agree on the job: slowest rank's time, all ranks' units
    assert a[1] == b[1] == 20.0
    assert a[0] == b[0] == pytest.approx(4.0 / 20e-3)
    assert a[2] == b[2] == a[3] + b[3]
    # each rank worked on its own data
    assert (a[4], a[5]) != (b[4], b[5])


def test_rank_workload_keeps_the_shape():
    w = synth.WORKLOADS["c4"]
    w3 = shard.rank_workload(w, 3)
    assert (w3.batch, w3.V, w3.n, w3.k, w3.max_depth, w3.H) == (w.batch, w.V, w.n, w.k, w.max_depth, w.H)
    assert w3.seed != w.seed and shard.rank_workload(w, 0).seed == w.seed


def test_single_process_needs_no_group():
    assert shard.whole_job(8.0, 4.0) == (2000.0, 4.0)


@pytest.mark.timeout(300)
def test_launcher_starts_one_rank_per_gpu_and_the_job_is_timed_over_all_of_them(tmp_path):
    """shard.launch_ranks + shard.timed_job with gloo ranks and a stand-in step: the job's time is the
    slow rank's, its units are both ranks'."""
    import json
    import sys
    out = tmp_path / "line.json"
    stub = os.path.join(os.path.dirname(os.path.abspath(__file__)), "_stub_ranks.py")
    rc = shard.launch_ranks(stub, [str(out), "10"], 2)
    assert rc == 0
    line = json.load(open(out))
    assert line["n_gpus"] == 2 and line["calls"] == 12            # 2 warm-up + 10 timed steps on rank 0
    assert line["ms"] >= 10 * 4.0 * 0.9                           # rank 1 sleeps 4 ms per step
    assert line["value"] == pytest.approx(2 * 4.0 * 10 / (line["ms"] * 1e-3))


@pytest.mark.timeout(300)
def test_bench_asked_for_two_gpus_starts_two_ranks_by_itself():
    """Without a CUDA device the ranks must stop at the "no CUDA device" exit (the CUDA path has no fallback);
    the launcher ends the other rank as soon as the first has failed, so one message is certain, two are not."""
    import subprocess
    import sys
    bench = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "bench.py")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK")}
    if torch.cuda.is_available():
        pytest.skip("needs a machine without a CUDA device")
    p = subprocess.run([sys.executable, bench, "--gpus", "2", "--steps", "1", "--warmup", "0"], env=env,
                       capture_output=True, text=True)
    assert p.returncode != 0
    text = p.stdout + p.stderr
    assert "of 2: no CUDA device" in text                          # a rank of a two-rank job said so
