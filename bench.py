#!/usr/bin/env python
"""Benchmark of the OPT-Tree decoding-step bookkeeping on B200.

A step = one pass of the whole hot path over one batch: opt_tree_build (Algorithm 1),
opt_tree_mask and opt_tree_verify (Algorithm 2) for B sequences, with the next step's root
tokens taken from this step's verification.  Workload: batch 32, V=32000, n=64, k=10,
max depth 10 ("c4"), threshold off (every layer drafted, so the byte count is fixed).

  python bench.py [--gpus N] [--steps K] [--warmup W]         # CUDA path, one JSON line
  python bench.py --impl reference ...                        # the CPU oracle, same metric
  python bench.py --rows N                                    # the row step alone (its own roofline line)
  python bench.py --table-rows H                              # the same workload on a table of H rows
  python bench.py --study mal                                 # acceptance lengths of adaptive and fixed trees

With N > 1 every rank (one per GPU; started by torch.distributed.run, or by this program itself
when it was started as a single process) runs its own batch with its own seeds and tables (weak
scaling, no data-path collective); the time is the maximum over ranks.
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

from paper_2406_17276_b200 import shard, synth  # noqa: E402

METRIC = "opt_tree_builds_per_s"
UNIT = "trees/s"
NEG_INF = -math.inf
MIN_TIMED_MS = 500.0          # the timed region is repeated in blocks of --steps until it has lasted this long
BIG_TABLE_ROWS = 32768        # rows of the table that defeats L2 reuse (2.1 GB at V=32000, 17 times the L2)


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


# DRAM bytes of one build_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu
# capture, see profiles/), keyed by workload and table rows, with the digest of the kernel sources the
# counters were taken on: a changed kernel reports no traffic.
NCU_TRAFFIC = {
    ("c4", 4096): {"bytes": 561.9e6, "csrc_sha256": "6046ba6afba2542026022ed2b3a6ad0841d5f20e31012d0f58d293ece0a95543"},
    ("c4", 32768): {"bytes": 1011.0e6, "csrc_sha256": "6046ba6afba2542026022ed2b3a6ad0841d5f20e31012d0f58d293ece0a95543"},
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


def _ncu_traffic(workload: str, H: int, delta: float):
    rec = NCU_TRAFFIC.get((workload, H))
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


def describe(w, H, delta):
    return (f"{w.name}: batch {w.batch} per GPU, V={w.V}, n={w.n}, k={w.k}, max_depth={w.max_depth}, "
            f"delta={'off' if delta == NEG_INF else delta}, H={H} bf16 tables "
            f"(sigma {w.sigma}, Zipf s {w.zipf_s}, {int(w.disagree * 100)}% rows disagree)")


class EventTimer:
    """CUDA events on the current stream, with the interface shard.timed_job expects."""

    def __init__(self):
        import torch
        self.e0, self.e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def start(self):
        self.e0.record()

    def stop(self):
        self.e1.record()

    def elapsed_ms(self):
        return self.e0.elapsed_time(self.e1)


class Stepper:
    """Device buffers of one workload and its decoding step through the binding."""

    def __init__(self, w, ld, lt, local, with_target=True):
        import torch
        from paper_2406_17276_b200 import binding
        self.torch, self.w = torch, w
        self.H = ld.shape[0]
        self.d_ld = torch.from_numpy(ld.view(np.int16)).cuda()
        self.d_lt = torch.from_numpy(lt.view(np.int16)).cuda() if with_target else None
        B, D = w.batch, w.max_depth
        self.ot = binding.OptTree(w.V, self.H, w.n, w.k, D, B, device=f"cuda:{local}")
        self.roots0 = torch.from_numpy(synth.root_tokens(B, w.V, w.seed + 1)).cuda()
        self.base = torch.zeros(B, dtype=torch.int32, device="cuda")
        self.tree = self.ot.alloc_tree(B, trace=False)
        self.mask = torch.empty((B, w.n, self.ot.W), dtype=torch.int64, device="cuda")
        self.pos = torch.empty((B, w.n), dtype=torch.int32, device="cuda")
        i32 = dict(dtype=torch.int32, device="cuda")
        self.vout = [(torch.empty(B, **i32), torch.empty((B, D + 1), **i32), torch.empty((B, D), **i32), torch.empty(B, **i32))
                     for _ in range(2)]
        self.root = self.roots0
        self.build_events = []

    def step(self, i, delta, time_build=False):
        torch, ot = self.torch, self.ot
        if time_build:
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            ot.build(self.d_ld, self.root, delta, self.tree)
            b.record()
            self.build_events.append((a, b))
        else:
            ot.build(self.d_ld, self.root, delta, self.tree)
        ot.mask(self.tree, self.base, self.mask, self.pos)
        o = self.vout[i & 1]
        ot.verify(self.tree, self.d_lt, self.root, o)
        self.root = o[3]                             # next_root feeds the next step

    def build_ms(self):
        ms = [a.elapsed_time(b) for a, b in self.build_events]
        return sum(ms) / len(ms) if ms else None

    def check(self, what):
        st = self.ot.device_status()
        if st != 0:
            raise SystemExit(f"bench.py: device status {st} after {what}")


def _sync():
    import torch
    torch.cuda.synchronize()


def timed_blocks(s: Stepper, steps, warmup, delta, min_ms=MIN_TIMED_MS, max_build_events=4000):
    """Blocks of exactly `steps` timed steps (shard.timed_job: barrier + synchronize on both sides, the
    slowest rank's time) until the timed region has lasted MIN_TIMED_MS.  Returns (trees/s of the whole
    job, ms per step, blocks)."""
    B = s.w.batch
    blocks, tot_ms = 0, 0.0
    units = 0.0
    w_left = warmup
    while True:
        value, ms = shard.timed_job(lambda i: s.step(i, delta, time_build=len(s.build_events) < max_build_events and i >= w_left),
                                    steps, w_left, B, EventTimer(), _sync, device="cuda")
        w_left = 0
        units += value * ms * 1e-3
        tot_ms += ms
        blocks += 1
        if tot_ms >= min_ms or blocks * steps >= 200000:
            break
    return units / (tot_ms * 1e-3), tot_ms / (blocks * steps), blocks


def mal_sample(s: Stepper, delta, steps=64):
    """Mean acceptance length and mean E(A) of the workload's trees over `steps` steps from fresh seeded roots
    (outside every timed region; a chain that follows its own accepted tokens soon cycles on these tables)."""
    torch, w = s.torch, s.w
    a = torch.zeros((), dtype=torch.float64, device="cuda"); e = torch.zeros((), dtype=torch.float64, device="cuda")
    for i in range(steps):
        s.root = torch.from_numpy(synth.root_tokens(w.batch, w.V, w.seed + 5000 + i)).cuda()
        s.step(i, delta)
        a += s.vout[i & 1][0].double().mean(); e += s.tree.expected_len.mean()
    torch.cuda.synchronize()
    return {"mean_acceptance_length": float(a) / steps, "mean_expected_length": float(e) / steps, "steps": steps,
            "trees": steps * w.batch, "note": "A counts the bonus token, E(A) (Eq. 3) does not"}


def quick_config(name, local, delta=NEG_INF):
    """Device-resident steps of another configuration, timed for a fraction of a second."""
    import torch
    w = synth.WORKLOADS[name]
    ld, lt = synth.make_tables(w)
    s = Stepper(w, ld, lt, local)
    del ld, lt
    for i in range(3):
        s.step(i, delta)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(); s.step(0, delta); e1.record(); torch.cuda.synchronize()
    est = max(e0.elapsed_time(e1), 1e-3)
    steps = int(min(2000, max(5, 300.0 / est)))
    s.build_events = []
    t = EventTimer()
    t.start()
    for i in range(steps):
        s.step(i, delta, time_build=True)
    t.stop(); torch.cuda.synchronize()
    s.check(name)
    ms = t.elapsed_ms() / steps
    bms = s.build_ms()
    rows = logical_rows(w, s.tree.depth_reached.cpu().numpy())
    peak, _ = _peaks()
    gbs = 2.0 * w.V * rows / (bms * 1e-3) / 1e9
    out = {"workload": describe(w, w.H, delta), "steps": steps, "trees_per_s": w.batch / (ms * 1e-3), "ms_per_step": ms,
           "build_ms": bms, "rows_per_build_call": rows, "algorithmic_gbs": gbs, "frac": gbs / peak,
           "frac_of_nominal_8000": gbs / 8000.0}
    if w.batch == 1:
        out["latency_ms_one_sequence"] = ms
    out["mal"] = mal_sample(s, delta, steps=8 if name == "c5" else 64)
    del s
    torch.cuda.empty_cache()
    return out


def big_table_build(w, local, H, delta=NEG_INF, calls=40):
    """opt_tree_build alone on the same shape with a draft table of H rows: every row a build reads is then
    a row the L2 does not hold, so the algorithmic bytes are bytes from HBM."""
    import torch
    from paper_2406_17276_b200 import binding
    ld = synth.draft_table(w.V, w.sigma, w.zipf_s, w.seed, H)
    d_ld = torch.from_numpy(ld.view(np.int16)).cuda()
    del ld
    ot = binding.OptTree(w.V, H, w.n, w.k, w.max_depth, w.batch, device=f"cuda:{local}")
    roots = [torch.from_numpy(synth.root_tokens(w.batch, w.V, w.seed + 100 + i)).cuda() for i in range(8)]
    tree = ot.alloc_tree(w.batch, trace=False)
    for i in range(5):
        ot.build(d_ld, roots[i % 8], delta, tree)
    t = EventTimer()
    torch.cuda.synchronize()
    t.start()
    for i in range(calls):
        ot.build(d_ld, roots[i % 8], delta, tree)
    t.stop(); torch.cuda.synchronize()
    if ot.device_status() != 0:
        raise SystemExit("bench.py: device status after the big-table builds")
    ms = t.elapsed_ms() / calls
    rows = logical_rows(w, tree.depth_reached.cpu().numpy())
    peak, kind = _peaks()
    gbs = 2.0 * w.V * rows / (ms * 1e-3) / 1e9
    traffic = _ncu_traffic(w.name, H, delta)
    out = {"table_rows": H, "table_bytes": 2.0 * w.V * H, "build_ms": ms, "calls": calls, "achieved": gbs, "unit": "GB/s",
           "frac": gbs / peak, "peak_kind": f"of {kind}", "frac_of_nominal_8000": gbs / 8000.0, "traffic": traffic,
           "frac_dram": (traffic / (ms * 1e-3) / 1e9 / peak) if traffic else None,
           "note": "opt_tree_build alone, back to back, roots changing from call to call"}
    del ot, d_ld
    torch.cuda.empty_cache()
    return out


def run_cuda(args):
    import torch

    if args.gpus > 1 and not shard.launched_by_torchrun():
        # asked for several GPUs as a single process: become the launcher of one rank per GPU
        raise SystemExit(shard.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
    if not torch.cuda.is_available():
        raise SystemExit(f"bench.py: rank {os.environ.get('RANK', 0)} of {os.environ.get('WORLD_SIZE', 1)}: "
                         "no CUDA device (the CUDA path has no CPU fallback)")
    local = int(os.environ.get("LOCAL_RANK", 0))
    torch.cuda.set_device(local)
    rank, world, local = shard.init_ranks("nccl", torch.device("cuda", local))
    from paper_2406_17276_b200 import build
    build.build()
    w = shard.rank_workload(synth.WORKLOADS[args.workload], rank)
    H = args.table_rows or w.H
    ld, lt = synth.make_tables(w, H=H)
    s = Stepper(w, ld, lt, local)
    ot, B, D, delta = s.ot, w.batch, w.max_depth, args.delta
    warmup = max(3, args.warmup)

    # one step from the first roots, kept for the comparison with the oracle in the cpu_baseline leg
    s.step(0, delta)
    torch.cuda.synchronize()
    first = {f: getattr(s.tree, f).cpu().numpy() for f in ("token", "parent", "depth", "n_sel", "depth_reached")}
    first.update(mask=s.mask.cpu().numpy().view(np.uint64), position_ids=s.pos.cpu().numpy(),
                 accept_len=s.vout[0][0].cpu().numpy(), accept_tokens=s.vout[0][1].cpu().numpy(),
                 accept_nodes=s.vout[0][2].cpu().numpy(), next_root=s.vout[0][3].cpu().numpy(),
                 phat=s.tree.phat.cpu().numpy(), expected_len=s.tree.expected_len.cpu().numpy())
    s.root = s.roots0

    # ---- device-resident timing ----
    sampler = ClockSampler(local); sampler.start()
    launches0 = ot.launch_count()
    value, ms_per_step, blocks = timed_blocks(s, args.steps, warmup, delta, args.min_timed_ms)
    clocks = sampler.result()
    launches = (ot.launch_count() - launches0) * args.steps // (blocks * args.steps + warmup)   # of one block of --steps
    build_ms = s.build_ms()
    s.check("the timed steps")
    rows_total = logical_rows(w, s.tree.depth_reached.cpu().numpy())    # the last build's own count (all equal with the threshold off)
    algo_bytes = 2.0 * w.V * rows_total
    tree, mask, vout, d_ld, d_lt, roots0 = s.tree, s.mask, s.vout, s.d_ld, s.d_lt, s.roots0

    def barrier():
        if world > 1:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize()

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

    peak, peak_kind = _peaks()
    achieved = algo_bytes / (build_ms * 1e-3) / 1e9
    traffic = args.traffic if args.traffic is not None else _ncu_traffic(args.workload, H, args.delta)
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world,
        "steps": args.steps, "warmup": warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": describe(w, H, delta),
                   "l2": f"inputs larger than L2: two {2.0 * w.V * H / 1e6:.0f} MB tables against a 126 MB L2, no explicit flush",
                   "step": "build + mask + verify, next roots from verify",
                   "timed_region": f"{blocks} blocks of {args.steps} steps (repeated until {args.min_timed_ms:.0f} ms), "
                                   "each block between barriers; value and ms_per_step are over all blocks"},
        "clocks": clocks,
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches),
        "roofline": {"bound": "hbm", "kernel": "build_kernel (opt_tree_build: one persistent kernel per call)",
                     "achieved": achieved, "achieved_kind": "algorithmic bytes (rows read once each; with 4096 table rows part of them is served by L2)",
                     "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "peak_kind": f"of {peak_kind}", "frac_of_nominal_8000": achieved / 8000.0,
                     "algorithmic_bytes_per_build_call": algo_bytes, "build_ms": build_ms,
                     "traffic": traffic,
                     "frac_dram": (traffic / (build_ms * 1e-3) / 1e9 / peak) if traffic else None},
    }
    if world == 1 and not args.quick:
        line.update(extras(s, args, local, rows_total))
        line["mal"] = mal_sample(s, delta)
    del s
    if rank == 0:
        if world == 1 and not args.no_cpu_baseline:
            cb, o_first = cpu_baseline(w, ld, lt, steps=2, want_first=True)
            line["cpu_baseline"] = cb
            line["cpu_baseline_all_cores"] = cpu_baseline_all_cores(w, ld, lt)
            line["parity"] = parity_counts(first, o_first)
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()
    if rank == 0 and line.get("parity", {}).get("mismatch", 0):
        raise SystemExit("bench.py: the checked step differs from the oracle beyond the near-tie rule")


def extras(s: Stepper, args, local, rows_total):
    """Entry points outside the timed step, each timed alone, the same workload on a table that defeats L2
    reuse, and the other configurations (one GPU only)."""
    import torch
    ot, w, tree, mask, vout, d_ld, d_lt, roots0 = s.ot, s.w, s.tree, s.mask, s.vout, s.d_ld, s.d_lt, s.roots0
    B, D, delta = w.batch, w.max_depth, args.delta
    i32 = dict(dtype=torch.int32, device="cuda")
    out = {}

    def timed(fn, reps, warm=3):
        for _ in range(warm):
            fn(0)
        t = EventTimer()
        torch.cuda.synchronize()
        t.start()
        for i in range(reps):
            fn(i)
        t.stop(); torch.cuda.synchronize()
        return t.elapsed_ms() / reps

    # bookkeeping after verification (dense mask, cache keep list)
    pv_out = ot.post_verify(tree, mask, vout[0][0], vout[0][2])
    pv_ms = timed(lambda i: ot.post_verify(tree, mask, vout[0][0], vout[0][2], pv_out), 100, 5)
    s.check("post_verify")
    out["post_verify"] = {"us_per_call": pv_ms * 1e3, "bytes_written": int(sum(t.numel() * t.element_size() for t in pv_out)),
                          "note": "opt_tree_post_verify alone, back-to-back calls; not part of the timed step"}

    # the pruned draft (same trees from fewer rows)
    rows_read = torch.empty(B, **i32)
    pruned_ms = timed(lambda i: ot.build_pruned(d_ld, roots0, delta, tree, rows_read), 50, 5)
    pruned_rows = int(rows_read.sum().item())
    s.check("build_pruned")
    out["pruned_build"] = {"ms_per_build": pruned_ms, "trees_per_s": B / (pruned_ms * 1e-3), "rows_read": pruned_rows,
                           "rows_of_full_build": int(rows_total), "gbs_of_rows_read": 2.0 * w.V * pruned_rows / (pruned_ms * 1e-3) / 1e9,
                           "note": "opt_tree_build_pruned alone on the first step's roots: the same trees, only rows that can still matter; not the benchmark's metric"}

    # the layer-by-layer build: the table plays the model; every layer's logits are gathered beforehand
    layers_ms, layer_bufs = None, []
    if 2.0 * w.V * B * (1 + (D - 1) * w.n) <= 4e9:
        ot.layers_begin(B)
        ltoks = roots0.view(-1, 1).to(torch.int64)
        lcnt = torch.ones(B, **i32)
        for depth in range(D):
            stride = int(lcnt.max().item())
            if stride == 0:
                break
            lrows = (ltoks[:, :stride] * 31 + depth) % s.H
            layer_bufs.append(d_ld[lrows.reshape(-1)].reshape(B, stride, w.V).contiguous())
            nt, _, lcnt = ot.layers_step(layer_bufs[-1], delta, tree)
            ltoks = nt.to(torch.int64)
        lnxt = (torch.empty((B, w.n), **i32), torch.empty((B, w.n), **i32), torch.empty(B, **i32))

        def layers_run(_i):
            ot.layers_begin(B)
            for lg in layer_bufs:
                ot.layers_step(lg, delta, tree, lnxt)

        layers_ms = timed(layers_run, 20)
        s.check("layers_step")
        del layer_bufs[:]
    out["layers_build"] = {"ms_per_batch": layers_ms, "trees_per_s": (B / (layers_ms * 1e-3)) if layers_ms else None,
                           "note": "opt_tree_layers_begin + one opt_tree_layers_step per layer on pre-gathered logits; not the benchmark's metric"}

    # verification with sampling (temperature 1)
    ot.build(d_ld, roots0, delta, tree)
    sv_out = ot.verify_sampled(tree, d_lt, roots0, 1.0, 2024, 0)
    sv_ms = timed(lambda i: ot.verify_sampled(tree, d_lt, roots0, 1.0, 2024, i, sv_out), 50)
    s.check("verify_sampled")
    sv_rows = int(tree.n_sel.sum().item()) + B
    out["verify_sampled"] = {"us_per_call": sv_ms * 1e3, "target_rows": sv_rows,
                             "algorithmic_gbs": 2.0 * w.V * sv_rows / (sv_ms * 1e-3) / 1e9,
                             "note": "opt_tree_verify_sampled alone at temperature 1; not part of the timed step"}
    gv_ms = timed(lambda i: ot.verify(tree, d_lt, roots0, vout[0]), 50)
    out["verify_greedy"] = {"us_per_call": gv_ms * 1e3, "target_rows": sv_rows,
                            "algorithmic_gbs": 2.0 * w.V * sv_rows / (gv_ms * 1e-3) / 1e9}

    if args.table_rows == 0 and args.workload == "c4":
        out["big_table"] = big_table_build(w, local, BIG_TABLE_ROWS, delta)
    if args.workload == "c4" and args.table_rows == 0 and not args.no_other_configs:
        out["other_configs"] = {name: quick_config(name, local) for name in ("c1", "c2", "c3", "c5")}
    return out


def run_rows(args):
    """The row step alone (fused softmax + top-k of Algorithm 1's expansion) over a list of rows
    larger than L2: its own roofline line.  Not the benchmark's metric; one GPU."""
    import torch
    from paper_2406_17276_b200 import binding, build

    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    build.build()
    w = synth.WORKLOADS[args.workload]
    H = args.table_rows or w.H
    ld = synth.draft_table(w.V, w.sigma, w.zipf_s, w.seed, H)
    d_ld = torch.from_numpy(ld.view(np.int16)).cuda()
    ot = binding.OptTree(w.V, H, w.n, w.k, w.max_depth, w.batch)
    nrows = args.rows
    rows = torch.from_numpy(np.random.default_rng(w.seed).integers(0, H, nrows).astype(np.int32)).cuda()
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
        "config": {"workload": f"{w.name}: row step alone, {nrows} random rows of V={w.V}, k={w.k}, H={H} bf16 table",
                   "l2": f"the {2.0 * w.V * H / 1e6:.0f} MB table is larger than L2; rows repeat across the list"},
        "clocks": clocks, "gpu_launches": args.steps,
        "roofline": {"bound": "hbm", "kernel": "row_topk_kernel", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "algorithmic_bytes_per_launch": algo, "traffic": None},
    }), flush=True)


def cpu_baseline(w, ld, lt, steps, batch=None, want_first=False):
    """The oracle as it stands, single thread, un-memoised, on a bounded sample of the workload."""
    import oracle
    B = batch or w.batch
    roots = synth.root_tokens(B, w.V, w.seed + 1)
    first = None
    t0 = time.perf_counter()
    for _ in range(steps):
        r = oracle.table_step(ld, lt, roots, w.n, w.k, w.max_depth, NEG_INF)
        first = first or r
        roots = r.next_root.copy()
    dt = time.perf_counter() - t0
    cb = {"value": B * steps / dt, "unit": UNIT, "cores": 1, "kind": "oracle",
          "sample": f"{steps} steps of {B} sequences (build + mask + verify), threshold off, no memo", "seconds": dt}
    return (cb, first) if want_first else cb


def cpu_baseline_all_cores(w, ld, lt, per_thread=2):
    """The same oracle code on every host core: one thread per core, each taking sequences of its own
    (the C routine runs without the interpreter lock)."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    P = os.cpu_count() or 1
    roots = synth.root_tokens(P * per_thread, w.V, w.seed + 2)
    oracle.lib()

    def work(t):
        for j in range(per_thread):
            oracle.table_step(ld, lt, roots[t * per_thread + j:t * per_thread + j + 1], w.n, w.k, w.max_depth, NEG_INF)

    t0 = time.perf_counter()
    with ThreadPoolExecutor(P) as ex:
        list(ex.map(work, range(P)))
    dt = time.perf_counter() - t0
    return {"value": P * per_thread / dt, "unit": UNIT, "cores": P, "kind": "oracle",
            "sample": f"{per_thread} sequences on each of {P} threads (build + mask + verify), threshold off, no memo", "seconds": dt}


def parity_counts(g, o):
    """The checked step (the first roots, threshold off) against the oracle's result for it: sequences whose
    integer outputs are identical; sequences that differ where the oracle reports a selection boundary closer
    than 1e-6 relative (near ties); anything else is a mismatch.  Largest relative errors of the path values
    and of E(A) over the identical ones."""
    B = g["n_sel"].shape[0]
    out = dict(exact=0, near_tie=0, stop_near_tie=0, mismatch=0, max_phat_rel=0.0, max_elen_rel=0.0, sequences=B)
    ints = ("token", "parent", "depth", "n_sel", "depth_reached", "mask", "position_ids", "accept_len", "accept_tokens",
            "accept_nodes", "next_root")
    for b in range(B):
        if all(np.array_equal(np.asarray(g[f][b]), np.asarray(getattr(o, f)[b])) for f in ints):
            out["exact"] += 1
            ns = int(o.n_sel[b])
            rel = float(np.max(np.abs(g["phat"][b, :ns] - o.phat[b, :ns]) / o.phat[b, :ns])) if ns else 0.0
            er = float(abs(g["expected_len"][b] - o.expected_len[b]) / o.expected_len[b])
            out["max_phat_rel"] = max(out["max_phat_rel"], rel)
            out["max_elen_rel"] = max(out["max_elen_rel"], er)
            if rel > 1e-5 or er > 1e-5:
                out["mismatch"] += 1
        elif o.min_gap[b] < 1e-6:
            out["near_tie"] += 1
        else:
            out["mismatch"] += 1
    return out


def run_study(args):
    """--study mal: acceptance length and E(A) of the adaptive tree against fixed trees of the same size on the
    synthetic tables (paper_2406_17276_b200/study.py), one JSON line; the oracle on the first two steps' roots
    beside it."""
    import torch
    from paper_2406_17276_b200 import build, study
    if not torch.cuda.is_available():
        raise SystemExit("bench.py: no CUDA device (the CUDA path has no CPU fallback)")
    build.build()
    line = {"study": "mal", "data": "synthetic", "steps": args.steps,
            "note": "acceptance length A counts the bonus token; E(A) of Eq. 3 does not, so E(A) + 1 is the figure to set against A",
            "workloads": {}}
    for nm in args.study_workloads.split(","):
        res, first = study.run(nm, args.steps, keep_first=2)
        if not args.no_cpu_baseline:
            res["cpu_baseline"] = study_cpu_baseline(first)
        line["workloads"][nm] = res
    if args.budgets:
        line["budget_sweep_c2"] = {str(n): study.run("c2", max(50, args.steps // 10), n=n)[0]["shapes"]
                                   for n in (16, 64, 256, 512, 1000)}
    print(json.dumps(line), flush=True)


def study_cpu_baseline(first):
    """The oracle on the first two steps' roots of a study: its acceptance lengths and E(A) beside the
    library's for the same roots (both follow the same rule, so they agree up to near-ties)."""
    import oracle
    w, n = first["w"], first["n"]
    ld, lt = first["tables"]
    t0 = time.perf_counter()
    oa, oe = [], []
    for r in first["roots"]:
        o = oracle.table_step(ld, lt, r, n, w.k, w.max_depth, NEG_INF)
        oa.append(o.accept_len); oe.append(o.expected_len)
    dt = time.perf_counter() - t0
    oa, oe = np.array(oa), np.array(oe)
    return {"kind": "oracle", "cores": 1, "sample": f"{len(first['roots'])} steps of {oa.shape[1]} sequences", "seconds": dt,
            "value": oa.size / dt, "unit": UNIT,
            "mean_acceptance_length": float(oa.mean()), "library_mean_acceptance_length_same_steps": float(first["A"].mean()),
            "mean_expected_length": float(oe.mean()), "library_mean_expected_length_same_steps": float(first["E"].mean()),
            "sequences_with_equal_acceptance_length": int((oa == first["A"]).sum()), "sequences": int(oa.size)}


def run_reference(args):
    """The reference arm: the CPU oracle on the same config and metric (rank 0 only)."""
    if int(os.environ.get("RANK", 0)) != 0:
        return
    import oracle
    oracle.build()
    w = synth.WORKLOADS[args.workload]
    ld, lt = synth.make_tables(w)
    sample_b = min(8, w.batch)                          # bounded sample per step: 8 of the batch's sequences
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
    ap.add_argument("--no-other-configs", action="store_true", help="skip the other four configurations")
    ap.add_argument("--min-timed-ms", type=float, default=MIN_TIMED_MS,
                    help="repeat the block of --steps timed steps until the timed region has lasted this long (0: one block, for profiler runs)")
    ap.add_argument("--quick", action="store_true", help="only the timed steps and the end-to-end leg")
    ap.add_argument("--table-rows", type=int, default=0,
                    help="rows H of the logit tables (default: the workload's 4096); e.g. 32768 makes every row a build reads come from HBM")
    ap.add_argument("--traffic", type=float, default=None,
                    help="ncu dram bytes per build call to report in roofline.traffic (default: the recorded capture, if the kernel sources are unchanged)")
    ap.add_argument("--rows", type=int, default=0,
                    help="time the row step alone over this many rows instead of whole steps (its own roofline line)")
    ap.add_argument("--study", default=None, choices=["mal"],
                    help="mal: mean acceptance length and E(A) of OPT-Tree against fixed trees of the same size on the synthetic tables")
    ap.add_argument("--study-workloads", default="c2,c4", help="workloads of --study, comma separated")
    ap.add_argument("--budgets", action="store_true", help="--study: also sweep the node budget on c2 (16 ... 1000 nodes)")
    args = ap.parse_args()
    if args.impl == "reference":
        if args.gpus > 1 and not shard.launched_by_torchrun():
            raise SystemExit(shard.launch_ranks(os.path.abspath(__file__), sys.argv[1:], args.gpus))
        run_reference(args)
    elif args.study:
        run_study(args)
    elif args.rows > 0:
        run_rows(args)
    else:
        run_cuda(args)


if __name__ == "__main__":
    main()
