"""Benchmark of the SLO-NN inference path on B200.

One step = one pass of the whole hot path (FreeHash, bucket lookup, top-k% cut, selected nodes layer by
layer, prediction) over one batch of synthetic queries.  Headline workload: the nine-layer 4096-wide bf16
MLP ("c4") with 4096 queries at a 10 % budget -- the only named network whose weights (276 MB) exceed the
L2 cache.  The same line carries a `configs` block with every named network at every named budget.
Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c4] [--queries 4096] [--budget-bp 1000]
  python bench.py --impl reference ...     # the CPU oracle on a bounded sample of the same workload

Timing: the L2 is flushed (a 256 MB buffer is overwritten) before every timed step, each step has its own
CUDA event pair on the launching stream, `ms_per_step` is the median of the K steps (max over ranks).
Multi-GPU: queries are independent, so ranks are replicas that each process their own batch (weak
scaling); there is no data-path collective.
"""
import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2204_08400_b200 import accounting, workloads  # noqa: E402

L2_BYTES = 126 * 1024 * 1024
FLUSH_BYTES = 256 * 1024 * 1024

# calibration rows used when --n-cal is not given: the named count where the CPU oracle can train the same
# tables within a minute (it is timed beside the GPU on the headline workload), fewer rows for the wide networks
DEFAULT_N_CAL = {"c1": 16384, "c2": 16384, "c3": 2048, "c3xl": 2048, "c4": 1024, "c5": 2048}
DEFAULT_QUERIES = {"c1": 1024, "c2": 65536, "c3": 256, "c3xl": 256, "c4": 4096, "c5": 8192}

# dram__bytes_read.sum + dram__bytes_write.sum of ONE launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (same kernel, same workload and launch shape).  Keyed by (kernel, workload,
# queries, budget); anything else reports null.  An entry is set to None when its kernel has changed since.
NCU_TRAFFIC = {
    # profiles/layer_cols_c4_4096q_10pct.md: a launch that starts with cold caches (the profiler's default cache
    # control); with the caches as the previous layer leaves them the same launch moves 1.3 MB
    ("layer_cols_kernel", "c4", 4096, 1000): 21.0e6,
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    return 6650.0, 1590.0, "fallback"


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None

    def start(self):
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                       "-lms", "20", "-i", str(self.gpu)], stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, reasons, mx = [], set(), None
        for line in self.f.read().splitlines():
            parts = [s.strip() for s in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                sm.append(float(parts[1])); mx = float(parts[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        return out


def resolve(args):
    """Query count, calibration rows and budget of the headline workload (identical in both arms)."""
    n = args.queries if args.queries is not None else DEFAULT_QUERIES[args.workload]
    n_cal = args.n_cal if args.n_cal is not None else DEFAULT_N_CAL[args.workload]
    return n, n_cal


def load_workload(args):
    n, n_cal = resolve(args)
    return workloads.load(args.workload, n_queries=n, n_cal=n_cal, budget_bp=args.budget_bp if args.budget_bp else None,
                          free_hash_nodes=args.free_hash_nodes)


def config_block(args, wl, world):
    """`config` of the JSON line; both arms print the same dict."""
    n, n_cal = resolve(args)
    label = (f"{args.workload}: " + "-".join(map(str, wl.dims)) + f" {wl.dtype} weights, {n} queries/GPU, budget " +
             (f"{args.budget_bp} bp" if args.budget_bp else "mixed 5/10/25/50/100 %") + f", K={wl.K} L={wl.L}, " +
             f"tables trained on {n_cal} calibration rows" + (", hash nodes always active" if wl.free_hash_nodes else ""))
    return {"workload": label, "queries_per_step_per_gpu": n, "budget_bp": args.budget_bp, "n_cal": n_cal,
            "l2": "flushed_between_steps", "parallelism": f"replicas x{world}"}


# ---- the CPU oracle (reference arm and cpu_baseline leg) ---------------------------------------

def oracle_sample(wl, target_seconds):
    """The oracle as it stands on a prefix of the workload's queries sized for about target_seconds.
    Returns (queries, seconds, threads, closure that repeats the timed call)."""
    from oracle import oracle as orc
    from oracle.run_workload import oracle_model, oracle_run, take_queries
    om = oracle_model(wl)
    n0 = min(wl.n_queries, 128)
    for _ in range(2):      # the second pass of the pilot sample is the one that sizes the timed sample
        t0 = time.perf_counter()
        oracle_run(om, wl, take_queries(wl, np.arange(n0)), wl.budget_bp[:n0], orc.CANON32)
        dt = max(time.perf_counter() - t0, 1e-4)
    n1 = int(min(wl.n_queries, max(n0, n0 * target_seconds / dt)))
    xs, bp = take_queries(wl, np.arange(n1)), wl.budget_bp[:n1]

    def again():
        t = time.perf_counter()
        oracle_run(om, wl, xs, bp, orc.CANON32)
        return time.perf_counter() - t
    return n1, again, orc.threads()


def run_reference(args, rank, world):
    if rank != 0:
        return
    wl = load_workload(args)
    steps = max(args.steps, 1)
    n1, again, cores = oracle_sample(wl, target_seconds=min(6.0, 90.0 / steps))
    for _ in range(min(args.warmup, 1)):
        again()
    times = [again() for _ in range(steps)]
    ms = 1e3 * float(np.median(times))
    value = n1 / (ms / 1e3)
    line = {
        "impl": "reference", "metric": "queries_per_sec_at_budget", "value": value, "unit": "queries/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": config_block(args, wl, world),
        "cpu_baseline": {"value": value, "unit": "queries/s", "cores": cores, "kind": "oracle",
                         "sample": f"first {n1} of {wl.n_queries} queries per step"},
        "e2e": {"value": value, "unit": "queries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---- GPU arm -------------------------------------------------------------------------------------

class Rig:
    """One device model with the plumbing to time batches on it."""

    def __init__(self, wl, dev, world, n_cal=None):
        import torch
        from paper_2204_08400_b200 import harness
        self.torch, self.wl, self.dev, self.world = torch, wl, dev, world
        self.dm = harness.DeviceModel(wl, device=dev, n_cal=n_cal)
        self.stream = torch.cuda.current_stream(dev)
        self.shape = accounting.NetShape.of(wl)
        self.x_nnz = (wl.x[0][1:] - wl.x[0][:-1]).astype(np.int64) if wl.first_sparse else None

    def barrier(self):
        import torch.distributed as dist
        self.torch.cuda.synchronize(self.dev)
        if self.world > 1:
            dist.barrier()
        self.torch.cuda.synchronize(self.dev)

    def take(self, n):
        """Inputs of the first n queries."""
        wl = self.wl
        if wl.first_sparse:
            ip = wl.x[0][: n + 1]
            return (ip, wl.x[1][: int(ip[-1])], wl.x[2][: int(ip[-1])])
        return wl.x[:n]

    def batch(self, bps, flags=0, kernel_path=0):
        from paper_2204_08400_b200 import harness
        return harness.DeviceBatch(self.dm, self.take(bps.size), bps, max_budget_bp=int(bps.max()), full_outputs=False,
                                   flags=flags, kernel_path=kernel_path)

    def time_steps(self, batch, steps, warmup, flush):
        """Per-step device times (ms): L2 flushed before every step, an event pair around each."""
        torch = self.torch
        for _ in range(warmup):
            batch.run(self.stream)
        self.barrier()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
        for a, b in ev:
            flush.zero_()
            a.record(self.stream)
            batch.run(self.stream)
            b.record(self.stream)
        self.barrier()
        st = batch.status.cpu().numpy()
        assert st[0] == 0, f"device status {st}"
        return np.array([a.elapsed_time(b) for a, b in ev])

    def trace(self, batch, reps=3):
        """Launch records of one step, times averaged over `reps` traced runs."""
        from paper_2204_08400_b200 import binding as sl
        runs = [sl.slonn_run_traced(self.dm.model, batch.batch, batch.ws, batch.ws_bytes, self.stream) for _ in range(reps + 1)][1:]
        recs = [dict(r) for r in runs[0]]
        for i, r in enumerate(recs):
            r["ms"] = float(np.mean([run[i]["ms"] for run in runs]))
        return recs

    def kernels(self, batch, bps):
        """Per-kernel launches, time and byte counts of one step, plus the dominant kernel's roofline entry."""
        recs = self.trace(batch)
        table = accounting.per_kernel(self.shape, recs, bps, self.x_nnz[: bps.size] if self.x_nnz is not None else None)
        return recs, table


def roofline_of(table, workload, n, budget_bp, dense_tc):
    """Roofline entry of the kernel with the largest share of the step's device time."""
    hbm, tflops, kind = measured_peaks()
    name = max(table, key=lambda k: table[k]["ms"])
    k = table[name]
    total_ms = sum(v["ms"] for v in table.values())
    common = {"kernel": name, "launches_per_step": k["launches"], "avg_launch_ms": k["ms"] / max(k["launches"], 1),
              "share_of_step": k["ms"] / total_ms if total_ms else 0.0, "peak_kind": kind}
    if name == "dense_tc_kernel":
        ach = k["flops"] / (k["ms"] / 1e3) / 1e12
        return dict(common, bound="tensor", achieved=ach, peak=tflops, unit="TFLOP/s", frac=ach / tflops, traffic=None,
                    flops_per_step=k["flops"])
    sec = k["ms"] / 1e3
    ach = k["algorithmic"] / sec / 1e9 if sec > 0 else 0.0
    traffic = None if dense_tc else NCU_TRAFFIC.get((name, workload, n, budget_bp))
    # what actually limits the kernel when DRAM is nearly idle: the rows come from L2 / L1 and the issue slots fill up
    dram_share = traffic * k["launches"] / k["algorithmic"] if traffic and k["algorithmic"] else None
    limiter = None
    if dram_share is not None:
        limiter = ("instruction issue with L2-resident data (DRAM moves %.1f %% of the algorithmic bytes)" % (100 * dram_share)
                   if dram_share < 0.25 else "HBM")
    elif ach > hbm:
        limiter = "L2 / L1 / instruction issue (faster than an HBM stream could deliver the bytes)"
    return dict(common, bound="hbm", limiter=limiter, achieved=ach, peak=hbm, unit="GB/s", frac=ach / hbm, traffic=traffic,
                frac_of_nominal_8TBps=ach / 8000.0, bytes_per_step=int(k["algorithmic"]),
                bytes_as_run=int(k["as_run"]), frac_as_run=k["as_run"] / sec / 1e9 / hbm if sec > 0 else 0.0,
                bytes_row_granular=int(k["row_granular"]),
                frac_row_granular=k["row_granular"] / sec / 1e9 / hbm if sec > 0 else 0.0,
                dram_frac=(traffic * k["launches"] / sec / 1e9 / hbm) if traffic else None,
                note="bytes_per_step: hash rows, bucket lists and selected nodes x input entries (the least any form must "
                     "load); bytes_as_run: whole rows where a layer ran row-wise.  A fraction above 1, or a traffic far "
                     "below bytes_per_step, means the rows were served from L2/L1, not HBM")


def measure(rig, bps, flags, steps, warmup, flush, workload, want_table=True):
    """One (batch size, budgets, flags) point: median step time, dominant kernel, byte counts."""
    batch = rig.batch(bps, flags=flags)
    t = rig.time_steps(batch, steps, warmup, flush)
    out = {"ms": float(np.median(t)), "ms_mean": float(np.mean(t)), "queries_per_s": bps.size / (float(np.median(t)) / 1e3)}
    if want_table:
        recs, table = rig.kernels(batch, bps)
        bp_key = int(bps[0]) if np.all(bps == bps[0]) else 0
        roof = roofline_of(table, workload, int(bps.size), bp_key, bool(flags & 1))
        out.update(kernel=roof["kernel"], frac=roof["frac"], share_of_step=roof["share_of_step"], bound=roof["bound"],
                   frac_as_run=roof.get("frac_as_run"), launches=len(recs))
        sb = accounting.step_bytes(rig.shape, bps, rig.x_nnz[: bps.size] if rig.x_nnz is not None else None)
        out["step_GBps_algorithmic"] = sb["algorithmic"] / (out["ms"] / 1e3) / 1e9
        out["step_frac_of_hbm_peak"] = out["step_GBps_algorithmic"] / measured_peaks()[0]
    del batch
    return out


def latency_block(rig, bps, reps, flags=0):
    """p50/p90/p99 of single steps answered one at a time, also as a CUDA-graph replay."""
    torch, dev, stream = rig.torch, rig.dev, rig.stream
    batch = rig.batch(bps, flags=flags)
    for _ in range(5):
        batch.run(stream)
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for a, b_ in evs:
        a.record(stream)
        batch.run(stream)
        b_.record(stream)
        torch.cuda.synchronize(dev)      # a server answers one request before it takes the next
    t = np.array([a.elapsed_time(b_) for a, b_ in evs]) * 1e3
    out = {"unit": "us per batch", "launches": reps, "p50": float(np.percentile(t, 50)),
           "p90": float(np.percentile(t, 90)), "p99": float(np.percentile(t, 99)), "min": float(t.min())}
    gs = torch.cuda.Stream(dev)
    with torch.cuda.stream(gs):
        batch.run(gs)
        gs.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=gs):
            batch.run(torch.cuda.current_stream(dev))
        tg = []
        for _ in range(reps):
            a, b_ = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); graph.replay(); b_.record()
            torch.cuda.synchronize(dev)
            tg.append(a.elapsed_time(b_) * 1e3)
    out["graph_replay_p50"] = float(np.percentile(tg, 50))
    out["graph_replay_p99"] = float(np.percentile(tg, 99))
    return out


def sweep(rig, n, budgets, steps, flush, workload, mixed=None, small=False):
    """Every named budget at n queries, the 100 % budget on the fixed-order kernels and (where the library
    offers it) on the tensor cores, and each budget's speed-up over both -- the paper's own measure
    (Sec. 5.2: speed-up over the full network)."""
    from paper_2204_08400_b200 import binding as sl
    wl = rig.wl
    out = {}
    full = measure(rig, np.full(n, 10000, np.uint16), 0, steps, 3, flush, workload)
    tc_ok = wl.dtype == "bf16" and not wl.first_sparse and not wl.has_act[-1]
    full_tc = measure(rig, np.full(n, 10000, np.uint16), sl.FLAG_DENSE_TC, steps, 3, flush, workload) if tc_ok else None
    points = [(str(bp), np.full(n, bp, np.uint16)) for bp in budgets]
    if mixed is not None:
        points.insert(0, ("mixed", mixed[:n]))
    for key, bps in points:
        if key == "10000":
            m = dict(full)
        else:
            m = measure(rig, bps, 0, steps, 3, flush, workload)
        m["speedup_vs_full"] = full["ms"] / m["ms"]
        m["speedup_vs_full_on_tensor_cores"] = full_tc["ms"] / m["ms"] if full_tc else None
        if small:
            m["latency"] = latency_block(rig, bps, 200)
        out[key] = m
    out["full_budget_ms"] = {"fixed_order_kernels": full["ms"], "tensor_cores": full_tc["ms"] if full_tc else None}
    if small:
        out["full_budget_latency"] = latency_block(rig, np.full(n, 10000, np.uint16), 200)
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c4")
    ap.add_argument("--budget-bp", type=int, default=1000,
                    help="budget of every query in basis points; 0 = the workload's mixed per-query budgets (c5)")
    ap.add_argument("--queries", type=int, default=None, help="override the workload's query count")
    ap.add_argument("--n-cal", type=int, default=None, help="calibration rows the tables are trained on")
    ap.add_argument("--dense-tc", action="store_true",
                    help="route 100 %% budget queries to the tensor-core dense path (not bit-exact for them)")
    ap.add_argument("--free-hash-nodes", action="store_true",
                    help="the variant in which a layer's K*L hash nodes are always active and absent from its lists")
    ap.add_argument("--row-kernels", action="store_true", help="sparse-input layers: force the row kernels")
    ap.add_argument("--column-kernels", action="store_true", help="sparse-input layers: force the input-stationary kernels")
    ap.add_argument("--kernel-path", type=int, default=0, help="0 auto, 1 per-stage kernels, 2 one warp per query, 3 cluster")
    ap.add_argument("--no-configs", action="store_true", help="headline workload only (e.g. under a profiler)")
    ap.add_argument("--configs", default="c1,c2,c3,c4,c5", help="networks of the configs block")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-policy", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank, world)
        return

    import torch
    import torch.distributed as dist
    from paper_2204_08400_b200 import binding as sl, harness, replicas

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=dev)

    # every rank is a replica with its own batch (same law; throughput does not depend on the draw and the
    # parity tests cover the values)
    wl = load_workload(args)
    n = wl.n_queries
    max_bp = int(wl.budget_bp.max())
    rig = Rig(wl, dev, world)
    dm, stream = rig.dm, rig.stream
    flush = torch.empty(FLUSH_BYTES, dtype=torch.uint8, device=dev)
    hbm_peak, _, _ = measured_peaks()

    # ---- headline: device-resident inputs ----
    flags = sl.FLAG_DENSE_TC if args.dense_tc else 0
    flags |= sl.FLAG_ROW_KERNELS if args.row_kernels else 0
    flags |= sl.FLAG_COLUMN_KERNELS if args.column_kernels else 0
    batch = harness.DeviceBatch(dm, wl.x, wl.budget_bp, max_budget_bp=max_bp, full_outputs=False, flags=flags,
                                kernel_path=args.kernel_path)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
        for _ in range(3):      # nvidia-smi needs a moment to start; keep the GPU under load meanwhile
            batch.run(stream)
        torch.cuda.synchronize(dev)
        time.sleep(0.3)
    step_ms = rig.time_steps(batch, args.steps, args.warmup, flush)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = replicas.slowest_rank_ms(float(np.median(step_ms)), dev)
    n_all = replicas.total_units(n, dev)          # queries all ranks processed in one step
    value = n_all / (ms_step / 1e3)

    # ---- per-launch device time of the same step, byte counts per kernel ----
    recs, table = rig.kernels(batch, wl.budget_bp)
    roofline = roofline_of(table, args.workload, n, args.budget_bp, args.dense_tc)
    roofline["kernels"] = {k: {"launches": v["launches"], "ms": v["ms"], "GBps_algorithmic": (v["algorithmic"] / (v["ms"] / 1e3) / 1e9) if v["ms"] else 0.0,
                               "frac": (v["algorithmic"] / (v["ms"] / 1e3) / 1e9 / hbm_peak) if v["ms"] else 0.0}
                           for k, v in table.items()}
    sb = accounting.step_bytes(rig.shape, wl.budget_bp, rig.x_nnz)
    roofline["step"] = {"bytes_algorithmic": int(sb["algorithmic"]), "bytes_row_granular": int(sb["row_granular"]),
                        "GBps_algorithmic": sb["algorithmic"] / (ms_step / 1e3) / 1e9,
                        "frac": sb["algorithmic"] / (ms_step / 1e3) / 1e9 / hbm_peak}
    launches_per_step = len(recs) + sum(1 for r in recs if r["stage"] == "plan")   # the plan record covers two launches

    latency = latency_block(rig, wl.budget_bp, max(args.steps, 1000), flags) if n <= 64 else None

    # ---- end to end through the host-buffer entry point ----
    e2e = None
    if not args.no_e2e:
        x_nnz = int(wl.x[0][-1]) if wl.first_sparse else 0
        stride = sl.slonn_logit_stride(dm.model, max_bp)
        pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
        view = {np.dtype(np.uint16): np.int16, np.dtype(np.uint32): np.int32, np.dtype(np.uint64): np.int64}
        pinv = lambda a: pin(np.ascontiguousarray(a).view(view.get(a.dtype, a.dtype)))
        h_logits = torch.zeros((n, stride), dtype=torch.float32).pin_memory()
        h_pred = torch.zeros(n, dtype=torch.int32).pin_memory()
        h_status = torch.zeros(4, dtype=torch.int32).pin_memory()
        h_bp = pinv(wl.budget_bp)
        h_lids = torch.zeros((n, stride), dtype=torch.int32).pin_memory() if wl.has_act[-1] else None
        if wl.first_sparse:
            h_csr = tuple(pinv(a) for a in wl.x)
            hb = sl.make_batch(n, h_bp, h_logits, h_status, x_csr=h_csr, max_budget_bp=max_bp,
                               logit_ids=h_lids, pred=h_pred, flags=flags)
        else:
            h_x = pin(wl.x)
            hb = sl.make_batch(n, h_bp, h_logits, h_status, x_dense=h_x, max_budget_bp=max_bp,
                               logit_ids=h_lids, pred=h_pred, flags=flags)
        nb = sl.slonn_host_workspace_bytes(dm.model, n, max_bp, x_nnz, flags)
        hws = torch.empty(nb, dtype=torch.uint8, device=dev)
        e_steps = max(3, min(args.steps, 20))
        for _ in range(3):
            up, down = sl.slonn_run_host(dm.model, hb, hws, nb, stream)
        rig.barrier()
        ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(e_steps)]
        for a, b_ in ev:
            a.record(stream)
            up, down = sl.slonn_run_host(dm.model, hb, hws, nb, stream)
            b_.record(stream)
        rig.barrier()
        ms_e = replicas.slowest_rank_ms(float(np.median([a.elapsed_time(b_) for a, b_ in ev])), dev)
        assert int(h_status[0]) == 0
        e2e = {"value": n_all / (ms_e / 1e3), "unit": "queries/s", "h2d_bytes_per_step": int(up),
               "d2h_bytes_per_step": int(down), "ms_per_step": ms_e}
        del hws

    # ---- every named network at every named budget (rank 0 of a single-GPU run) ----
    configs = None
    if rank == 0 and world == 1 and not args.no_configs:
        configs = {}
        cfg_steps = max(5, min(args.steps, 10))
        for name in [c for c in args.configs.split(",") if c]:
            same = (name == args.workload and not args.free_hash_nodes and resolve(args)[1] == DEFAULT_N_CAL[name]
                    and n >= DEFAULT_QUERIES[name])
            if same:
                r2 = rig
            else:
                w2 = workloads.load(name, n_queries=DEFAULT_QUERIES[name], n_cal=DEFAULT_N_CAL[name])
                r2 = Rig(w2, dev, world)
            budgets = list(r2.wl.budgets_named)
            mixed = workloads.draw_mixed_budgets(DEFAULT_QUERIES[name], 4) if name == "c5" else None
            entry = {"network": "-".join(map(str, r2.wl.dims)) + " " + r2.wl.dtype, "n_cal": r2.dm.n_cal,
                     "table_bytes": r2.dm.table_bytes(),
                     "table_build_ms": r2.dm.build_ms}
            entry[f"{DEFAULT_QUERIES[name]}_queries"] = sweep(r2, DEFAULT_QUERIES[name], budgets, cfg_steps, flush, name, mixed)
            if name == "c4":      # the paper serves at batch size 1: per-batch latency of small batches
                for small_n in (64, 1):
                    entry[f"{small_n}_queries"] = sweep(r2, small_n, budgets, cfg_steps, flush, name, small=True)
            configs[name] = entry
            if r2 is not rig:
                r2.dm.free()
                del r2
                torch.cuda.empty_cache()

    # ---- budget policies on the device (outside the timed region): Confidence tables + ACLO lookup ----
    policy = None
    if (rank == 0 and world == 1 and not args.no_policy and wl.has_act[0] and not wl.first_sparse and not wl.has_act[-1]):
        prof = np.array(sorted(set(wl.budgets_named) | {10000}), np.uint16)
        rows = harness._dev(wl.calib[: min(dm.n_cal, 1024)], dev)
        torch.cuda.synchronize(dev)
        t0 = time.perf_counter()
        conf = sl.slonn_confidence_build(dm.model, rows, prof, stream)
        torch.cuda.synchronize(dev)
        conf_ms = (time.perf_counter() - t0) * 1e3
        thr = torch.full((1, prof.size), -1.0, dtype=torch.float32, device=dev)
        xq = harness._dev(wl.x, dev)
        bpo = torch.zeros(n, dtype=torch.int16, device=dev)
        for _ in range(3):
            sl.slonn_aclo_budgets(dm.model, conf, xq, thr, bpo, stream=stream)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record(stream)
        for _ in range(10):
            sl.slonn_aclo_budgets(dm.model, conf, xq, thr, bpo, stream=stream)
        a1.record(stream)
        torch.cuda.synchronize(dev)
        policy = {"confidence_build_ms": conf_ms, "confidence_rows": int(rows.shape[0]), "profile_bp": prof.tolist(),
                  "aclo_budgets_ms_per_batch": a0.elapsed_time(a1) / 10, "queries": n}
        sl.slonn_confidence_free(conf)
        del rows, xq, bpo

    # ---- the CPU oracle beside it (rank 0, single-GPU runs only) ----
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n1, again, cores = oracle_sample(wl, target_seconds=15.0)
        dt = again()
        cpu = {"value": n1 / dt, "unit": "queries/s", "cores": cores, "kind": "oracle",
               "sample": f"first {n1} of {n} queries, {dt:.1f} s, tables trained by the oracle on the same {dm.n_cal} calibration rows"}

    if rank == 0:
        line = {
            "metric": "queries_per_sec_at_budget", "value": value, "unit": "queries/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "f32",   # every sum is accumulated in fp32 (bf16 weights are widened)
            "data": "synthetic",
            "config": config_block(args, wl, world),
            "timing": {"statistic": "median of the timed steps", "ms_per_step_mean": float(np.mean(step_ms)),
                       "ms_per_step_min": float(np.min(step_ms)), "l2_flush_bytes": FLUSH_BYTES},
            "full_budget_route": "tensor cores (bf16 activations)" if args.dense_tc else "fixed-order fp32 kernels",
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": launches_per_step * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "configs": configs, "latency": latency,
            "policy": policy,
            "table_build": {"ms": dm.build_ms, "calibration_rows": dm.n_cal, "table_bytes": dm.table_bytes(),
                            "rows_per_s": dm.n_cal / (dm.build_ms / 1e3), "timing": "host wall clock around slonn_build"},
            "paper_context": "the paper reports only speed-ups over the full network (1.3-56.7x, CPU, NumPy+Numba, batch size 1); "
                             "speedup_vs_full in `configs` is that measure on this GPU",
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
