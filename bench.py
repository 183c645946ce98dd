#!/usr/bin/env python
"""Benchmark of the OPT-Tree decoding-step bookkeeping on B200.

A step = one pass of the whole hot path over one batch: opt_tree_build (Algorithm 1),
opt_tree_mask and opt_tree_verify (Algorithm 2) for B sequences, with the next step's root
tokens taken from this step's verification.  Workload: batch 32, V=32000, n=64, k=10,
max depth 10 ("c4"), threshold off (every layer drafted, so the byte count is fixed).

  python bench.py [--gpus N] [--steps K] [--warmup W]         # CUDA path, one JSON line
  python bench.py --impl reference ...                        # the CPU oracle, same metric

With N > 1 (launched by torch.distributed.run, one rank per GPU) every rank runs its own batch
with its own seeds and tables (weak scaling, no data-path collective); the time is the maximum
over ranks.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2406_17276_b200 import synth  # noqa: E402

METRIC = "opt_tree_builds_per_s"
UNIT = "trees/s"
NEG_INF = -math.inf


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM bytes of one build_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture, see profiles/), keyed by workload, with the digest of the kernel sources the counters
# were taken on: a changed kernel reports no traffic.
NCU_TRAFFIC = {
    "c4": {"bytes": 600.1e6, "csrc_sha256": "6ae3b61f2b8ac64cafa7e6b91a996773f37410eea89561611d0ded1bbae73f33"},
}


def _csrc_digest() -> str:
    import hashlib
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2406_17276_b200", "csrc")
    for name in sorted(os.listdir(d)):
        if name.endswith((".cu", ".cuh")):
            h.update(name.encode())
            h.update(open(os.path.join(d, name), "rb").read())
    return h.hexdigest()


def _ncu_traffic(workload: str, delta: float):
    rec = NCU_TRAFFIC.get(workload)
    if rec is None or delta != NEG_INF or rec["csrc_sha256"] != _csrc_digest():
        return None
    return rec["bytes"]


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index: int, period_s: float = 0.02):
        super().__init__(daemon=True)
        self.index, self.period, self.stop_flag = index, period_s, threading.Event()
        self.sm, self.reasons, self.sm_max = [], set(), None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.sm_max = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {"hw_slowdown": nv.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": nv.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": nv.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": nv.nvmlClocksThrottleReasonSwPowerCap}
        while not self.stop_flag.is_set():
            try:
                self.sm.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            time.sleep(self.period)

    def result(self):
        self.stop_flag.set()
        self.join(timeout=2)
        return {"sm_mhz": float(np.median(self.sm)) if self.sm else None, "sm_max_mhz": self.sm_max,
                "reasons": sorted(self.reasons), "samples": len(self.sm)}


def logical_rows(w, depth_reached):
    """Rows of L_d one build reads: the root row, the min(n,k) first-layer nodes, then n per layer."""
    rows = 0
    for d in depth_reached:
        d = int(d)
        rows += 1 + (min(w.n, w.k) if d >= 2 else 0) + max(0, d - 2) * w.n
    return rows


def run_cuda(args):
    import torch
    from paper_2406_17276_b200 import binding, build, shard

    rank = int(os.environ.get("RANK", 0)); world = int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    torch.cuda.set_device(local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    build.build()
    w = shard.rank_workload(synth.WORKLOADS[args.workload], rank)
    ld, lt = synth.make_tables(w)
    d_ld = torch.from_numpy(ld.view(np.int16)).cuda(); d_lt = torch.from_numpy(lt.view(np.int16)).cuda()
    B, D = w.batch, w.max_depth
    ot = binding.OptTree(w.V, w.H, w.n, w.k, D, B, device=f"cuda:{local}")
    roots0 = torch.from_numpy(synth.root_tokens(B, w.V, w.seed + 1)).cuda()
    base = torch.zeros(B, dtype=torch.int32, device="cuda")
    tree = ot.alloc_tree(B, trace=False)
    mask = torch.empty((B, w.n, ot.W), dtype=torch.int64, device="cuda")
    pos = torch.empty((B, w.n), dtype=torch.int32, device="cuda")
    i32 = dict(dtype=torch.int32, device="cuda")
    vout = [(torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))
            for _ in range(2)]
    delta = args.delta

    def step(i, root):
        ot.build(d_ld, root, delta, tree)
        ot.mask(tree, base, mask, pos)
        o = vout[i & 1]
        ot.verify(tree, d_lt, root, o)
        return o[3]                                  # next_root feeds the next step

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing ----
    root = roots0
    for i in range(args.warmup):
        root = step(i, root)
    barrier()
    sampler = ClockSampler(local); sampler.start()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    bev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    rows_total = 0
    launches0 = ot.launch_count()
    ev0.record()
    for i in range(args.steps):
        bev[i][0].record()
        ot.build(d_ld, root, delta, tree)
        bev[i][1].record()
        ot.mask(tree, base, mask, pos)
        o = vout[i & 1]
        ot.verify(tree, d_lt, root, o)
        root = o[3]
    ev1.record()
    barrier()
    clocks = sampler.result()
    launches = ot.launch_count() - launches0
    ms = ev0.elapsed_time(ev1)
    build_ms = sum(a.elapsed_time(b) for a, b in bev) / args.steps
    status = ot.device_status()
    if status != 0:
        raise SystemExit(f"bench.py: device status {status}")
    # bytes of the last build (all builds are identical in size when the threshold is off)
    rows_last = logical_rows(w, tree.depth_reached.cpu().numpy())
    if delta == NEG_INF:
        rows_total = rows_last
    else:
        rows_total = rows_last            # threshold on: the last build's own count is reported
    algo_bytes = 2.0 * w.V * rows_total
    value, ms = shard.whole_job(B * args.steps, ms, device="cuda")       # all ranks' trees / the slowest rank's time

    # ---- end to end through the host-buffer entry point ----
    ho = ot.alloc_host_out(B)
    h_root = roots0.cpu().pin_memory(); h_base = torch.zeros(B, dtype=torch.int32).pin_memory()
    e2e_steps = max(3, min(args.steps, 200))
    for _ in range(3):
        ot.step_host(d_ld, d_lt, h_root, h_base, delta, ho)
        h_root.copy_(ho["next_root"])
    barrier()
    t0 = time.perf_counter()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        ot.step_host(d_ld, d_lt, h_root, h_base, delta, ho)
        h_root.copy_(ho["next_root"])
    e1.record()
    barrier()
    e2e_ms = max(e0.elapsed_time(e1), (time.perf_counter() - t0) * 1e3) / e2e_steps
    e2e_value, e2e_ms = shard.whole_job(B, e2e_ms, device="cuda")
    h2d = 2 * B * 4
    d2h = sum(int(t.numel() * t.element_size()) for t in ho.values())

    # ---- the bookkeeping after verification (dense mask, cache keep list): timed on its own, not part of a step ----
    pv_out = ot.post_verify(tree, mask, vout[0][0], vout[0][2])
    for _ in range(5):
        ot.post_verify(tree, mask, vout[0][0], vout[0][2], pv_out)
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    p0.record()
    for _ in range(100):
        ot.post_verify(tree, mask, vout[0][0], vout[0][2], pv_out)
    p1.record(); torch.cuda.synchronize()
    post_verify_us = p0.elapsed_time(p1) * 10.0
    if ot.device_status() != 0:
        raise SystemExit("bench.py: device status after post_verify")

    # ---- the pruned draft (same trees from fewer rows): timed on its own, with its own byte count ----
    rows_read = torch.empty(B, dtype=torch.int32, device="cuda")
    for _ in range(5):
        ot.build_pruned(d_ld, roots0, delta, tree, rows_read)
    q0, q1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    q0.record()
    for _ in range(50):
        ot.build_pruned(d_ld, roots0, delta, tree, rows_read)
    q1.record(); torch.cuda.synchronize()
    pruned_ms = q0.elapsed_time(q1) / 50
    pruned_rows = int(rows_read.sum().item())
    if ot.device_status() != 0:
        raise SystemExit("bench.py: device status after build_pruned")

    # ---- the layer-by-layer build (logits handed in per layer, as a real draft model would): timed on its own.
    #      The table plays the model; every layer's logits are gathered beforehand, only the library's calls are timed.
    layers_ms, layer_bufs = None, []
    if 2.0 * w.V * B * (1 + (D - 1) * w.n) <= 4e9:          # the pre-gathered logits of all layers must fit comfortably
        ot.layers_begin(B)
        ltoks = roots0.view(-1, 1).to(torch.int64)
        lcnt = torch.ones(B, dtype=torch.int32, device="cuda")
        for depth in range(D):
            stride = int(lcnt.max().item())
            if stride == 0:
                break
            lrows = (ltoks[:, :stride] * 31 + depth) % w.H
            layer_bufs.append(d_ld[lrows.reshape(-1)].reshape(B, stride, w.V).contiguous())
            nt, _, lcnt = ot.layers_step(layer_bufs[-1], delta, tree)
            ltoks = nt.to(torch.int64)
        lnxt = (torch.empty((B, w.n), **i32), torch.empty((B, w.n), **i32), torch.empty(B, **i32))

        def layers_run():
            ot.layers_begin(B)
            for lg in layer_bufs:
                ot.layers_step(lg, delta, tree, lnxt)

        for _ in range(3):
            layers_run()
        l0, l1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        l0.record()
        for _ in range(20):
            layers_run()
        l1.record(); torch.cuda.synchronize()
        layers_ms = l0.elapsed_time(l1) / 20
        if ot.device_status() != 0:
            raise SystemExit("bench.py: device status after layers_step")
        del layer_bufs[:]

    # ---- verification with sampling (temperature 1): timed on its own ----
    sv_out = ot.verify_sampled(tree, d_lt, roots0, 1.0, 2024, 0)
    for _ in range(3):
        ot.verify_sampled(tree, d_lt, roots0, 1.0, 2024, 0, sv_out)
    s0, s1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    s0.record()
    for i in range(50):
        ot.verify_sampled(tree, d_lt, roots0, 1.0, 2024, i, sv_out)
    s1.record(); torch.cuda.synchronize()
    verify_sampled_us = s0.elapsed_time(s1) * 20.0
    if ot.device_status() != 0:
        raise SystemExit("bench.py: device status after verify_sampled")

    peak, peak_kind = _peaks()
    achieved = algo_bytes / (build_ms * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: batch {B} per GPU, V={w.V}, n={w.n}, k={w.k}, max_depth={D}, "
                               f"delta={'off' if delta == NEG_INF else delta}, H={w.H} bf16 tables "
                               f"(sigma {w.sigma}, Zipf s {w.zipf_s}, {int(w.disagree * 100)}% rows disagree)",
                   "l2": "inputs larger than L2: two 262 MB tables against a 126 MB L2, no explicit flush",
                   "step": "build + mask + verify, next roots from verify"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "pruned_build": {"ms_per_build": pruned_ms, "trees_per_s": B / (pruned_ms * 1e-3), "rows_read": pruned_rows,
                         "rows_of_full_build": int(rows_total), "gbs_of_rows_read": 2.0 * w.V * pruned_rows / (pruned_ms * 1e-3) / 1e9,
                         "note": "opt_tree_build_pruned alone on the first step's roots: the same trees, only rows that can still matter; not the benchmark's metric"},
        "layers_build": {"ms_per_batch": layers_ms, "trees_per_s": (B / (layers_ms * 1e-3)) if layers_ms else None,
                         "note": "opt_tree_layers_begin + one opt_tree_layers_step per layer on pre-gathered logits (two launches per layer; skipped when those logits would not fit); not the benchmark's metric"},
        "verify_sampled": {"us_per_call": verify_sampled_us,
                           "note": "opt_tree_verify_sampled alone at temperature 1 (one double-precision exponential per target logit); not part of the timed step"},
        "post_verify": {"us_per_call": post_verify_us, "bytes_written": int(sum(t.numel() * t.element_size() for t in pv_out)),
                        "note": "opt_tree_post_verify alone, 100 back-to-back calls; not part of the timed step"},
        "roofline": {"bound": "hbm", "kernel": "build_kernel (opt_tree_build: init_build_kernel + one persistent build_kernel)",
                     "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / 8000.0,
                     "algorithmic_bytes_per_build_call": algo_bytes, "build_ms": build_ms,
                     "traffic": args.traffic if args.traffic is not None else _ncu_traffic(args.workload, args.delta)},
    }
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_baseline(w, ld, lt, steps=2)
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_rows(args):
    """The row step alone (fused softmax + top-k of Algorithm 1's expansion) over a list of rows
    larger than L2: its own roofline line.  Not the benchmark's metric; one GPU."""
    import torch
    from paper_2406_17276_b200 import binding, build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    build.build()
    w = synth.WORKLOADS[args.workload]
    ld, _ = synth.make_tables(w)
    d_ld = torch.from_numpy(ld.view(np.int16)).cuda()
    ot = binding.OptTree(w.V, w.H, w.n, w.k, w.max_depth, w.batch)
    nrows = args.rows
    rows = torch.from_numpy(np.random.default_rng(w.seed).integers(0, w.H, nrows).astype(np.int32)).cuda()
    for _ in range(max(3, args.warmup)):
        ot.row_softmax_topk(d_ld, rows)
    torch.cuda.synchronize()
    sampler = ClockSampler(0); sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        ot.row_softmax_topk(d_ld, rows)
    e1.record(); torch.cuda.synchronize()
    clocks = sampler.result()
    if ot.device_status() != 0:
        raise SystemExit(f"bench.py: device status {ot.device_status()}")
    ms = e0.elapsed_time(e1) / args.steps
    peak, peak_kind = _peaks()
    algo = 2.0 * w.V * nrows
    achieved = algo / (ms * 1e-3) / 1e9
    print(json.dumps({
        "metric": "rows_per_s", "value": nrows / (ms * 1e-3), "unit": "rows/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms, "higher_is_better": True, "dtype": "f32", "data": "synthetic",
        "config": {"workload": f"{w.name}: row step alone, {nrows} random rows of V={w.V}, k={w.k}, H={w.H} bf16 table",
                   "l2": "the 262 MB table is larger than L2; rows repeat across the list"},
        "clocks": clocks, "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "kernel": "row_topk_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": algo, "traffic": None},
    }), flush=True)


def cpu_baseline(w, ld, lt, steps, batch=None):
    """The oracle as it stands, single thread, un-memoised, on a bounded sample of the workload."""
    import oracle
    B = batch or w.batch
    roots = synth.root_tokens(B, w.V, w.seed + 1)
    t0 = time.perf_counter()
    for _ in range(steps):
        r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, NEG_INF)
        roots = r.next_root.copy()
    dt = time.perf_counter() - t0
    return {"value": B * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
            "sample": f"{steps} steps of {B} sequences (build + mask + verify), threshold off, no memo", "seconds": dt}


def run_reference(args):
    """The reference arm: the CPU oracle on the same config and metric (rank 0 only)."""
    if int(os.environ.get("RANK", 0)) != 0:
        return
    import oracle
    oracle.build()
    w = synth.WORKLOADS[args.workload]
    ld, lt = synth.make_tables(w)
    sample_b = 8                                        # bounded sample per step: 8 of the 32 sequences
    steps, warm = max(1, min(args.steps, 4)), max(0, min(args.warmup, 1))
    if warm:
        cpu_baseline(w, ld, lt, warm, batch=sample_b)
    cb = cpu_baseline(w, ld, lt, steps, batch=sample_b)
    line = {"impl": "reference", "metric": METRIC, "value": cb["value"], "unit": UNIT, "n_gpus": int(args.gpus),
            "steps": steps, "warmup": warm, "ms_per_step": cb["seconds"] * 1e3 / steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": f"{w.name}: V={w.V}, n={w.n}, k={w.k}, max_depth={w.max_depth}, delta=off; "
                                   f"each step is a sample of {sample_b} of the batch's {w.batch} sequences"},
            "cpu_baseline": {"value": cb["value"], "unit": UNIT, "cores": 1, "kind": "oracle", "sample": cb["sample"]},
            "e2e": {"value": cb["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="cuda", choices=["cuda", "reference"])
    ap.add_argument("--workload", default="c4", choices=sorted(synth.WORKLOADS))
    ap.add_argument("--delta", type=float, default=NEG_INF)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu dram bytes per build call to report in roofline.traffic (default: the recorded capture, if the kernel sources are unchanged)")
    ap.add_argument("--rows", type=int, default=0,
                    help="time the row step alone over this many rows instead of whole steps (its own roofline line)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.rows > 0:
        run_rows(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
