"""Benchmark of the SLO-NN inference path on B200.

One step = one pass of the whole hot path (plan, hash+select, gather-dot per
layer, argmax) over one batch of synthetic queries.  Default workload: the
784-1024-1024-10 bf16 MLP with 65,536 queries ("c2"), headline budget 10 %,
plus a sweep over the other budgets.  Prints ONE JSON line on rank 0.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload c2] [--budget-bp 1000]
  python bench.py --impl reference ...     # the CPU oracle on a bounded sample

Multi-GPU: queries are independent, so ranks are replicas that each process
their own batch (weak scaling); there is no data-path collective.
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

from paper_2204_08400_b200 import workloads  # noqa: E402

L2_BYTES = 126 * 1024 * 1024

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the dominant kernel, from the ncu captures
# summarised under profiles/ (same workload, same launch shape).  Keyed by (kernel, workload, queries, budget);
# anything else reports null.  Set an entry to None when its kernel changes until the capture is redone.
NCU_TRAFFIC = {
    ("fused_network_kernel", "c2", 65536, 1000): 217.0e6,   # profiles/fused_network_c2_65536q_10pct.md
}


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a kernel timed alone (the burst figure)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        return float(json.load(open(p))["bf16_tflops"]), "measured"
    return 1590.0, "fallback"


def hash_bytes(wl, n):
    """Weight bytes of the FreeHash rows of one step: K*L rows per query and activator layer."""
    esz = 2 if wl.dtype == "bf16" else 4
    return sum(wl.K * wl.L * wl.dims[l] * esz * n for l in range(len(wl.dims) - 1) if wl.has_act[l])


def budget_nodes(bp, N):
    return np.minimum(np.maximum((bp.astype(np.int64) * N + 5000) // 10000, 1), N)


def gathered_bytes(wl, budget_bp, force_rows=False, force_cols=False, cols_max_bp=3500):
    """Algorithmic weight bytes of one step's gather launches, all queries, split by kernel kind:
    (row kernels, gather_cols_kernel, layer_cols_kernel, full_rows_kernel on layers without activator).
    Row kernels (dense input, or a list input that is not sparse enough): every selected weight row
    once per query, whole (row-granular).  Input-stationary kernels (a layer fed by the list of the
    activator layer below, budgets up to cols_max_bp): selected nodes x input list entries
    (B_out * B_in weights), the weights such a query needs at all; the whole-layer kernel of an
    activator layer also reads its K*L hash rows at the list entries."""
    esz = 2 if wl.dtype == "bf16" else 4
    bp = np.asarray(budget_bp)
    rows = cols = layer = grouped = 0
    if bp.size == 0:
        return 0, 0, 0, 0
    for l in range(len(wl.dims) - 1):
        if l == 0 and wl.first_sparse:
            continue
        D, N = wl.dims[l], wl.dims[l + 1]
        b_out = budget_nodes(bp, N) if wl.has_act[l] else np.full(bp.size, N, np.int64)
        list_input = l > 0 and wl.has_act[l - 1]
        use_cols = np.zeros(bp.size, bool)
        if list_input and not force_rows:
            big = bp.size * int(b_out.max()) >= 148 * 1024
            if force_cols:
                use_cols[:] = bp.size * int(b_out.max()) > 148 * 64
            elif big:
                use_cols = bp <= cols_max_bp
            elif bp.size * int(b_out.max()) > 148 * 64 and D >= 2048 and int(bp.max()) <= 1500:
                use_cols = bp <= 1500
        b_in = budget_nodes(bp, D) if list_input else np.full(bp.size, D, np.int64)
        if wl.has_act[l] and wl.K * wl.L <= 32:
            layer += int(((b_out[use_cols] + wl.K * wl.L) * b_in[use_cols]).sum()) * esz
        else:
            cols += int((b_out[use_cols] * b_in[use_cols]).sum()) * esz
        row_bytes = int(b_out[~use_cols].sum()) * D * esz
        # a layer without activator: the row-kernel queries share every row and run four per block
        if (not wl.has_act[l] and bp.size >= 256 and bp.size * N * D >= 2 ** 30 and 16 * D <= 200 * 1024
                and not use_cols.all()):
            grouped += row_bytes
        else:
            rows += row_bytes
    return rows, cols, layer, grouped


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


def oracle_queries_per_sec(wl, budget_bp, target_seconds=12.0):
    """The CPU oracle as it stands, timed on a bounded prefix of the workload's queries."""
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle import oracle as orc
    from parity_util import oracle_model, oracle_run, take_queries
    om = oracle_model(wl)
    n0 = min(wl.n_queries, 256)
    idx = np.arange(n0)
    bp = wl.budget_bp[:n0] if budget_bp is None else np.full(n0, budget_bp, np.uint16)
    t0 = time.perf_counter()
    oracle_run(om, wl, take_queries(wl, idx), bp, orc.CANON32)
    dt = max(time.perf_counter() - t0, 1e-4)
    n1 = int(min(wl.n_queries, max(n0, n0 * target_seconds / dt)))
    idx = np.arange(n1)
    bp = wl.budget_bp[:n1] if budget_bp is None else np.full(n1, budget_bp, np.uint16)
    xs = take_queries(wl, idx)
    t0 = time.perf_counter()
    oracle_run(om, wl, xs, bp, orc.CANON32)
    dt = time.perf_counter() - t0
    return n1 / dt, orc.threads(), n1, dt, (om, xs, bp)


def workload_label(args, wl):
    return (f"{args.workload}: " + "-".join(map(str, wl.dims)) + f" {wl.dtype} weights, {wl.n_queries} queries/GPU, budget " +
            (f"{args.budget_bp} bp" if args.budget_bp else "mixed 5/10/25/50/100 %") + f", K={wl.K} L={wl.L}" +
            (", hash nodes always active" if wl.free_hash_nodes else ""))


def run_reference(args, rank, world):
    if rank != 0:
        return
    wl = workloads.load(args.workload, n_queries=args.queries, n_cal=args.n_cal,
                        budget_bp=args.budget_bp if args.budget_bp else None, free_hash_nodes=args.free_hash_nodes)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    from oracle import oracle as orc
    from parity_util import oracle_run
    qps, cores, n1, dt, (om, xs, bp) = oracle_queries_per_sec(wl, args.budget_bp if args.budget_bp else None,
                                                              target_seconds=6.0)
    for _ in range(args.warmup):
        pass  # the sizing pass above already warmed caches; warm-up steps would only repeat it
    times = []
    for _ in range(args.steps):
        t0 = time.perf_counter()
        oracle_run(om, wl, xs, bp, orc.CANON32)
        times.append(time.perf_counter() - t0)
    ms = 1e3 * float(np.sum(times)) / max(args.steps, 1)
    value = n1 / (ms / 1e3)
    line = {
        "impl": "reference", "metric": "queries_per_sec_at_budget", "value": value, "unit": "queries/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_label(args, wl), "queries_per_step_per_gpu": wl.n_queries,
                   "budget_bp": args.budget_bp, "queries_timed_per_step": n1},
        "cpu_baseline": {"value": value, "unit": "queries/s", "cores": cores, "kind": "oracle",
                         "sample": f"first {n1} of {wl.n_queries} queries per step"},
        "e2e": {"value": value, "unit": "queries/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c2")
    ap.add_argument("--budget-bp", type=int, default=1000,
                    help="budget of every query in basis points; 0 = the workload's mixed per-query budgets (c5)")
    ap.add_argument("--queries", type=int, default=None, help="override the workload's query count")
    ap.add_argument("--n-cal", type=int, default=None)
    ap.add_argument("--dense-tc", action="store_true",
                    help="route 100 %% budget queries to the tensor-core dense path (not bit-exact for them)")
    ap.add_argument("--free-hash-nodes", action="store_true",
                    help="the variant in which a layer's K*L hash nodes are always active and absent from its lists")
    ap.add_argument("--row-kernels", action="store_true", help="sparse-input layers: force the row kernels")
    ap.add_argument("--column-kernels", action="store_true", help="sparse-input layers: force the input-stationary kernels")
    ap.add_argument("--kernel-path", type=int, default=0, help="0 auto, 1 per-stage kernels, 2 one warp per query, 3 cluster")
    ap.add_argument("--no-sweep", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--cpu-baseline", action="store_true", help="time the oracle also for workloads other than c1/c2")
    ap.add_argument("--no-e2e", action="store_true")
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

    # every rank is a replica with its own batch (same law, rank-specific seed is not needed:
    # throughput does not depend on the draw; parity tests cover the values)
    wl = workloads.load(args.workload, n_queries=args.queries, n_cal=args.n_cal,
                        budget_bp=args.budget_bp if args.budget_bp else None, free_hash_nodes=args.free_hash_nodes)
    max_bp = int(wl.budget_bp.max())
    n = wl.n_queries
    dm = harness.DeviceModel(wl, device=dev)
    stream = torch.cuda.current_stream(dev)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(batch, steps, warmup):
        for _ in range(warmup):
            batch.run(stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(steps):
            batch.run(stream)
        e1.record(stream)
        barrier()
        return replicas.slowest_rank_ms(e0.elapsed_time(e1), dev) / steps

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
    ms_step = timed(batch, args.steps, args.warmup)
    clocks = sampler.stop() if rank == 0 else None
    status = batch.status.cpu().numpy()
    assert status[0] == 0, f"device status {status}"
    n_all = replicas.total_units(n, dev)          # queries all ranks processed in one step
    value = n_all / (ms_step / 1e3)
    launches_per_step = None  # counted below from the per-stage launch counters

    # ---- per-query latency for small batches (the paper serves at batch size 1): one event pair per step ----
    latency = None
    if n <= 64:
        reps = max(args.steps, 1000)
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
        for a, b_ in evs:
            a.record(stream)
            batch.run(stream)
            b_.record(stream)
            torch.cuda.synchronize(dev)      # a server answers one request before it takes the next
        t = np.array([a.elapsed_time(b_) for a, b_ in evs]) * 1e3
        latency = {"unit": "us per batch", "launches": reps, "p50": float(np.percentile(t, 50)),
                   "p90": float(np.percentile(t, 90)), "p99": float(np.percentile(t, 99)), "min": float(t.min())}
        # the same step captured once in a CUDA graph and replayed per request
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
        latency["graph_replay_p50"] = float(np.percentile(tg, 50))
        latency["graph_replay_p99"] = float(np.percentile(tg, 99))

    # ---- per-stage device time of the same step (event pair around every launch) ----
    stage_ms = {s: 0.0 for s in sl.STAGES}
    stage_cnt = {s: 0 for s in sl.STAGES}
    prof_steps = max(3, min(args.steps, 10))
    for _ in range(prof_steps):
        ms, cnt = sl.slonn_run_timed(dm.model, batch.batch, batch.ws, batch.ws_bytes, stream)
        for s in sl.STAGES:
            stage_ms[s] += ms[s]; stage_cnt[s] += cnt[s]
    def full_route_active(bps):
        """The library's rule for taking the 100 % queries out of the per-query kernels (four per block)."""
        weights = sum(wl.dims[l] * wl.dims[l + 1] for l in range(len(wl.dims) - 1))
        return (not (flags & sl.FLAG_DENSE_TC) and not wl.first_sparse and bps.size >= 256 and int(bps.max()) == 10000
                and bps.size * weights >= 2 ** 32 and 16 * max(wl.dims[:-1]) <= 200 * 1024)

    def stage_roofline(ms_by_stage, cnt_by_stage, bps, steps):
        """Dominant kernel of the step and its achieved rate on the weight bytes it must touch."""
        esz = 2 if wl.dtype == "bf16" else 4
        n_full = int((bps == 10000).sum()) if bps.size and full_route_active(bps) else 0
        full_b = n_full * sum(wl.dims[l] * wl.dims[l + 1] for l in range(len(wl.dims) - 1)) * esz
        if (flags & sl.FLAG_DENSE_TC) or n_full:     # queries at 100 % leave the per-query kernels
            bps = bps[bps != 10000]
        row_b, col_b, layer_b, grouped_b = gathered_bytes(wl, bps, args.row_kernels, args.column_kernels, sl.COLS_MAX_BP)
        if ms_by_stage["full_rows"] > 0 and ms_by_stage["full_rows"] >= max(ms_by_stage.values()):
            ms, launches = ms_by_stage["full_rows"] / steps, cnt_by_stage["full_rows"] // steps
            nbytes = full_b + (grouped_b if ms_by_stage["fused"] == 0 and ms_by_stage["cluster"] == 0 else 0)
            return "full_rows_kernel", ms, launches, nbytes, nbytes / (ms / 1e3) / 1e9
        cols_ms = ms_by_stage["gather_cols"] + ms_by_stage["layer_cols"]
        if ms_by_stage["fused"] > 0:     # one launch does hash + select + gather for every layer
            row_b = sum(gathered_bytes(wl, bps, force_rows=True)[i] for i in (0, 3))
            kernel, ms, launches, nbytes = "fused_network_kernel", ms_by_stage["fused"], cnt_by_stage["fused"], row_b + hash_bytes(wl, bps.size)
        elif ms_by_stage["cluster"] > 0:
            row_b = sum(gathered_bytes(wl, bps, force_rows=True)[i] for i in (0, 3))
            kernel, ms, launches, nbytes = "cluster_network_kernel", ms_by_stage["cluster"], cnt_by_stage["cluster"], row_b + hash_bytes(wl, bps.size)
        elif cols_ms > ms_by_stage["gather_dot"]:
            # the input-stationary kernels: the whole-layer kernel of the activator layers (hash + selection +
            # nodes) or, if larger, the plain gather of the layers without activator
            if ms_by_stage["layer_cols"] >= ms_by_stage["gather_cols"]:
                kernel, ms, launches, nbytes = "layer_cols_kernel", ms_by_stage["layer_cols"], cnt_by_stage["layer_cols"], layer_b
            else:
                kernel, ms, launches, nbytes = "gather_cols_kernel", ms_by_stage["gather_cols"], cnt_by_stage["gather_cols"], col_b
        else:
            esz = 2 if wl.dtype == "bf16" else 4
            gather_layers = [l for l in range(len(wl.dims) - 1) if not (l == 0 and wl.first_sparse)]
            short = all(wl.dims[l] * esz <= 512 for l in gather_layers)   # rows of one 512-byte round
            kernel = "gather_short_kernel" if short else "gather_dot_kernel"
            ms, launches, nbytes = ms_by_stage["gather_dot"], cnt_by_stage["gather_dot"], row_b
        ms /= steps
        launches //= steps
        ach = nbytes / (ms / 1e3) / 1e9 if ms > 0 else 0.0
        return kernel, ms, launches, nbytes, ach

    peak, peak_kind = measured_peaks()
    kernel, k_ms, k_launches, k_bytes, achieved = stage_roofline(stage_ms, stage_cnt, wl.budget_bp, prof_steps)
    roofline = {"bound": "hbm", "kernel": kernel, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": peak_kind,
                "traffic": NCU_TRAFFIC.get((kernel, args.workload, n, args.budget_bp)) if not args.dense_tc else None,
                "frac_of_nominal_8TBps": achieved / 8000.0,
                "bytes_per_step": int(k_bytes), "launches_per_step": k_launches,
                "avg_launch_ms": k_ms / max(k_launches, 1),
                "stage_ms_per_step": {s: stage_ms[s] / prof_steps for s in sl.STAGES}}
    if stage_ms["dense_tc"] >= max(stage_ms.values()):
        # the step is dominated by the tensor-core route: its roofline is the tensor pipe.  The stage time
        # covers the compaction of the routed queries and the bf16 copy of their inputs as well.
        n_tc = int((wl.budget_bp == 10000).sum())
        flops = sum(2.0 * n_tc * wl.dims[l] * wl.dims[l + 1] for l in range(len(wl.dims) - 1))
        tc_ms = stage_ms["dense_tc"] / prof_steps
        tpeak, tkind = measured_tensor_peak()
        ach = flops / (tc_ms / 1e3) / 1e12
        roofline = {"bound": "tensor", "kernel": "dense_tc_kernel", "achieved": ach, "peak": tpeak, "unit": "TFLOP/s",
                    "frac": ach / tpeak, "peak_kind": tkind, "traffic": None, "flops_per_step": flops,
                    "launches_per_step": len(wl.dims) - 1, "avg_launch_ms": tc_ms / (len(wl.dims) - 1),
                    "stage_ms_per_step": {s: stage_ms[s] / prof_steps for s in sl.STAGES}}

    # ---- budget sweep (the latency profile T(k, isolated) of the paper) ----
    sweep = {}
    if not args.no_sweep and world == 1:
        for bp in wl.budgets_named:
            bps = np.full(n, bp, np.uint16)
            b2 = harness.DeviceBatch(dm, wl.x, bps, max_budget_bp=bp, full_outputs=False, flags=flags,
                                     kernel_path=args.kernel_path)
            ms2 = timed(b2, max(3, args.steps // 4), 3)
            st_ms, st_cnt = sl.slonn_run_timed(dm.model, b2.batch, b2.ws, b2.ws_bytes, stream)
            k2, _, _, _, ach2 = stage_roofline(st_ms, st_cnt, bps, 1)
            sweep[str(bp)] = {"queries_per_s": n / (ms2 / 1e3), "ms_per_step": ms2, "kernel": k2,
                              "weight_GBps": ach2, "frac_of_peak": ach2 / peak}
            del b2

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
        e_steps = max(3, min(args.steps, 10))
        for _ in range(3):
            up, down = sl.slonn_run_host(dm.model, hb, hws, nb, stream)
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e_steps):
            up, down = sl.slonn_run_host(dm.model, hb, hws, nb, stream)
        e1.record(stream)
        barrier()
        ms_e = replicas.slowest_rank_ms(e0.elapsed_time(e1), dev) / e_steps
        assert int(h_status[0]) == 0
        e2e = {"value": n_all / (ms_e / 1e3), "unit": "queries/s", "h2d_bytes_per_step": int(up),
               "d2h_bytes_per_step": int(down), "ms_per_step": ms_e}

    # ---- budget policies on the device (outside the timed region): Confidence tables + ACLO lookup ----
    policy = None
    if rank == 0 and world == 1 and not args.no_sweep and wl.has_act[0] and not wl.first_sparse and not wl.has_act[-1]:
        prof = np.array(sorted(set(wl.budgets_named) | {10000}), np.uint16)
        rows = harness._dev(wl.calib[: min(dm.n_cal, 4096)], dev)
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
    # the oracle builds its own tables from the same calibration rows: seconds for c1/c2, many minutes for
    # the wide networks, so those need --cpu-baseline (and usually --n-cal) to be asked for explicitly
    want_cpu = args.cpu_baseline or (args.workload in ("c1", "c2") and not args.no_cpu_baseline)
    if rank == 0 and world == 1 and want_cpu:
        qps, cores, n1, dt, _ = oracle_queries_per_sec(wl, None if not args.budget_bp else args.budget_bp)
        cpu = {"value": qps, "unit": "queries/s", "cores": cores, "kind": "oracle",
               "sample": f"first {n1} of {n} queries, {dt:.1f} s"}

    if rank == 0:
        esz_name = "f32"  # every sum is accumulated in fp32 (bf16 weights are widened)
        line = {
            "metric": "queries_per_sec_at_budget", "value": value, "unit": "queries/s", "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": esz_name, "data": "synthetic",
            "config": {"workload": workload_label(args, wl),
                       "queries_per_step_per_gpu": n, "budget_bp": args.budget_bp,
                       "l2": "inputs_larger_than_l2" if (wl.x.nbytes if not wl.first_sparse else 0) > L2_BYTES
                             else "weights_and_inputs_l2_resident",
                       "table_bytes": dm.table_bytes(), "parallelism": f"replicas x{world}",
                       "full_budget_route": "tensor cores (bf16 activations)" if args.dense_tc else "fixed-order fp32 kernels"},
            "clocks": clocks, "e2e": e2e,
            "gpu_launches": (sum(stage_cnt.values()) // prof_steps + (1 if stage_cnt["plan"] else 0)) * args.steps,
            "roofline": roofline, "cpu_baseline": cpu, "budget_sweep": sweep, "latency": latency,
            "policy": policy,
            "table_build": {"ms": dm.build_ms, "calibration_rows": dm.n_cal,
                            "rows_per_s": dm.n_cal / (dm.build_ms / 1e3), "timing": "host wall clock around slonn_build"},
        }
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
