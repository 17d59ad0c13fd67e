#!/usr/bin/env python
"""Benchmark of the multi-view attention hot path (plan pre-computed; forward + backward per step).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl mate|reference] [--workload long]

One step = one mate_attn_fwd + one mate_attn_bwd over one synthetic batch of the named workload.
Prints ONE JSON line.  With N > 1 (torchrun) every rank runs its own replica of the workload
(the path has no exchange step); the time is the max over ranks, the value the sum of the work.
`--impl reference` times the CPU oracle instead (rank 0 only).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from workloads import tables  # noqa: E402

METRIC = "MATE attn fwd+bwd useful-pair TFLOP/s at N=8192 (4*d flop/pair fwd, 10*d bwd)"
UNIT = "TFLOP/s"
N_BUFFER_SETS = 4
TRAFFIC_JSON = os.path.join(ROOT, "profiles", "ncu_traffic_long.json")


def kernel_sources_hash():
    """sha1 over the CUDA sources: ties the stored ncu counters to the kernels they were taken on."""
    import glob
    import hashlib
    h = hashlib.sha1()
    for path in sorted(glob.glob(os.path.join(ROOT, "paper_2109_04312_b200", "csrc", "*"))):
        with open(path, "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:12]


def ncu_traffic(kernel, workload):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of `kernel`, from the ncu capture stored
    under profiles/ -- or None when there is none for this workload or the kernels have changed since."""
    try:
        with open(TRAFFIC_JSON) as f:
            t = json.load(f)
    except (OSError, ValueError):
        return None
    if t.get("workload") != workload or t.get("sources_sha1") != kernel_sources_hash():
        return None
    k = t.get("kernels", {}).get(kernel)
    return None if k is None else float(k["dram_bytes_read"]) + float(k["dram_bytes_write"])


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons in the background (read-only queries)."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.samples = []
        self.proc = None
        self.index = index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self):
        if self.proc is not None:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass

    def summary(self, t0, t1):
        rows = [s for (t, s) in self.samples if t0 <= t <= t1] or [s for (_, s) in self.samples[-3:]]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for nm, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm)}


def oracle_step(cfg, rows, cols, vals, hv, scale):
    import oracle
    t0 = time.perf_counter()
    oracle.fwd(vals["Q"], vals["K"], vals["V"], rows, cols, cfg.P, hv, scale)
    t1 = time.perf_counter()
    oracle.bwd(vals["Q"], vals["K"], vals["V"], vals["dO"], rows, cols, cfg.P, hv, scale)
    t2 = time.perf_counter()
    return t1 - t0, t2 - t1


def pair_flops(cfg, pairs):
    return 4.0 * cfg.d * pairs, 10.0 * cfg.d * pairs


def run_reference(args, cfg):
    """CPU oracle arm.  Each step is one forward + backward of a bounded sample of the workload:
    the same table, a subset of the heads (always at least one row head and one column head),
    chosen so that warmup + steps stay within a few minutes on the host cores."""
    import oracle
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows, cols, info = tables.make_structure(cfg, 1234)
    vals = tables.make_values(cfg, info["N"], 5678)
    hv = tables.head_view(cfg)
    scale = 1.0 / np.sqrt(cfg.d)
    row_heads = [h for h in range(cfg.H) if hv[h] == 0]
    col_heads = [h for h in range(cfg.H) if hv[h] == 1]

    def subset(k):  # k heads of each view (all heads of a view when it has fewer)
        return sorted(row_heads[:k] + col_heads[:k])

    def sample_of(hsel):
        return {n: np.ascontiguousarray(v[:, hsel]) for n, v in vals.items()}, hv[hsel]

    # calibrate on the smallest sample, then take the largest sample that fits the time budget
    hsel = subset(1)
    sv, shv = sample_of(hsel)
    t0 = time.perf_counter()
    oracle_step(cfg, rows, cols, sv, shv, scale)
    t_small = time.perf_counter() - t0
    budget = 150.0 / max(args.steps + args.warmup, 1)
    k = max(1, min(max(len(row_heads), len(col_heads)), int(budget / max(t_small, 1e-9))))
    if k > 1:
        hsel = subset(k)
        sv, shv = sample_of(hsel)
    pairs = float(oracle.useful_pairs(rows, cols, cfg.P, shv).sum())
    f_fwd, f_bwd = pair_flops(cfg, pairs)
    # When even the smallest sample (one head of each view) does not fit `steps + warmup` times into the
    # budget, fewer steps are run (at least 3 timed, 1 warm-up) and the line says how many.
    n_warm, n_steps = args.warmup, args.steps
    if k == 1 and (n_warm + n_steps) * t_small > 150.0:
        n_steps = max(3, min(n_steps, int(150.0 / max(t_small, 1e-9)) - 1))
        n_warm = min(n_warm, 1)
    for _ in range(n_warm):
        oracle_step(cfg, rows, cols, sv, shv, scale)
    tf = tb = 0.0
    for _ in range(n_steps):
        a, b = oracle_step(cfg, rows, cols, sv, shv, scale)
        tf += a
        tb += b
    t_step = (tf + tb) / n_steps
    value = (f_fwd + f_bwd) / t_step / 1e12
    sample = "%s workload (B=%d N=%d), heads %s of %d, fwd+bwd per step, fp64" % (
        cfg.name, cfg.B, info["N"], hsel, cfg.H)
    if n_steps != args.steps:
        sample += "; %d of the %d requested steps run (time budget of the CPU arm)" % (n_steps, args.steps)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": n_steps, "warmup": n_warm, "ms_per_step": t_step * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "N": info["N"], "d": cfg.d, "P": cfg.P},
        "fwd": {"ms": tf / n_steps * 1e3, "tflops": f_fwd / (tf / n_steps) / 1e12},
        "bwd": {"ms": tb / n_steps * 1e3, "tflops": f_bwd / (tb / n_steps) / 1e12},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def reduce_over_ranks(times, work, world):
    """Whole-job figures from per-rank ones: every rank runs its own replica (the path has no
    exchange step), so the job's time is the slowest rank's (MAX) and its work the sum (SUM).
    `times` and `work` are float64 tensors on the rank's device (CPU tensors under gloo)."""
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(times, op=dist.ReduceOp.MAX)
        dist.all_reduce(work, op=dist.ReduceOp.SUM)
    return times.tolist(), work.tolist()


def run_mate(args, cfg):
    import torch
    import torch.distributed as dist

    import paper_2109_04312_b200 as mate

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    dev = torch.device("cuda", local_rank)
    peaks = load_peaks()

    # every rank builds its own replica of the workload (different seed per rank): no exchange step
    rows, cols, info = tables.make_structure(cfg, 1234 + rank)
    hv = tables.head_view(cfg)
    N = info["N"]
    scale = 1.0 / np.sqrt(cfg.d)
    tdt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32
    rows_d, cols_d = torch.from_numpy(rows).to(dev), torch.from_numpy(cols).to(dev)
    mate.mate_plan(rows_d, cols_d, cfg.P, hv, cfg.n_rows, cfg.n_cols).destroy()   # first call: library set-up
    torch.cuda.synchronize()
    # the plan is pre-computed (outside the timed step); its cost is reported on its own: wall time of
    # the call (allocations, kernels, work-lists on the host) and device time between two events
    pe0, pe1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_plan0 = time.perf_counter()
    pe0.record()
    plan = mate.mate_plan(rows_d, cols_d, cfg.P, hv, cfg.n_rows, cfg.n_cols)
    pe1.record()
    torch.cuda.synchronize()
    plan_wall_ms = (time.perf_counter() - t_plan0) * 1e3
    plan_dev_ms = pe0.elapsed_time(pe1)
    pairs = float(plan.useful_pairs().sum())
    launches_per_step = 3  # tc_fwd_kernel, rowdot_kernel, tc_bwd_kernel
    n_valid_tokens = float(sum(info["n_valid"]))
    f_fwd, f_bwd = pair_flops(cfg, pairs)

    host = tables.make_values(cfg, N, 5678 + rank)
    pinned = {k: torch.from_numpy(v).to(tdt).pin_memory() for k, v in host.items()}
    sets = []
    for s in range(N_BUFFER_SETS):
        d = {k: pinned[k].to(dev, non_blocking=True).clone() for k in ("Q", "K", "V", "dO")}
        if s:
            for k in d:  # distinct contents per set, same distribution
                d[k] = d[k].roll(s, dims=2).contiguous()
        d["O"] = torch.empty_like(d["Q"])
        d["LSE"] = torch.empty((cfg.B, cfg.H, N), dtype=torch.float32, device=dev)
        sets.append(d)
    torch.cuda.synchronize()
    set_bytes = sum(t.numel() * t.element_size() for t in sets[0].values()) + 3 * sets[0]["Q"].numel() * 2

    fwd_impl = mate.IMPL_AUTO | {"auto": 0, "bulk": mate.FLAG_BULK_TILES, "gather": mate.FLAG_GATHER_TILES}[args.loader]

    def step(d):
        mate.mate_attn_fwd(plan, d["Q"], d["K"], d["V"], scale, fwd_impl, out=d["O"], lse=d["LSE"])
        return mate.mate_attn_bwd(plan, d["Q"], d["K"], d["V"], d["O"], d["LSE"], d["dO"], scale)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()

    for i in range(args.warmup):
        step(sets[i % N_BUFFER_SETS])
    torch.cuda.synchronize()
    plan.status()

    # ---- device-resident timing: K steps, CUDA events on the launching (current) stream
    K = args.steps
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    for i in range(K):
        d = sets[i % N_BUFFER_SETS]
        ev[i][0].record()
        mate.mate_attn_fwd(plan, d["Q"], d["K"], d["V"], scale, fwd_impl, out=d["O"], lse=d["LSE"])
        ev[i][1].record()
        mate.mate_attn_bwd(plan, d["Q"], d["K"], d["V"], d["O"], d["LSE"], d["dO"], scale)
        ev[i][2].record()
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_wall1 = time.time()
    plan.status()
    total_ms = ev[0][0].elapsed_time(ev[K - 1][2])
    fwd_ms = np.asarray([e[0].elapsed_time(e[1]) for e in ev])
    bwd_ms = np.asarray([e[1].elapsed_time(e[2]) for e in ev])

    # ---- the same on ONE buffer set (about 50 MB of inputs: served from the 126 MB L2), for comparison
    warm_ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(min(K, 50))]
    d = sets[0]
    for e in warm_ev:
        e[0].record()
        mate.mate_attn_fwd(plan, d["Q"], d["K"], d["V"], scale, fwd_impl, out=d["O"], lse=d["LSE"])
        e[1].record()
        mate.mate_attn_bwd(plan, d["Q"], d["K"], d["V"], d["O"], d["LSE"], d["dO"], scale)
        e[2].record()
    torch.cuda.synchronize()
    fwd_warm_ms = float(np.median([e[0].elapsed_time(e[1]) for e in warm_ev]))
    bwd_warm_ms = float(np.median([e[1].elapsed_time(e[2]) for e in warm_ev]))

    # ---- the small HBM-bound kernel beside the path: per-cell mean of token logits (Section 4.1).  The
    #      kernel is far shorter than the host's share of one call, so twenty calls are captured in a CUDA
    #      graph and the graph is timed (device time per call, no host gaps).
    logits = torch.randn((cfg.B, N), dtype=torch.float32, device=dev)
    cm_out = mate.mate_cell_mean(plan, logits, cols_d)
    torch.cuda.synchronize()
    cell_ms = None
    try:
        g = torch.cuda.CUDAGraph()
        side = torch.cuda.Stream(dev)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            with torch.cuda.graph(g, stream=side):
                for _ in range(20):
                    mate.mate_cell_mean(plan, logits, cols_d, out=cm_out)
        torch.cuda.current_stream().wait_stream(side)
        g.replay()
        torch.cuda.synchronize()
        c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        c0.record()
        for _ in range(5):
            g.replay()
        c1.record()
        torch.cuda.synchronize()
        cell_ms = c0.elapsed_time(c1) / 100.0
    except Exception:  # no graph capture available: report nothing rather than a host-bound figure
        cell_ms = None
    # algorithmic bytes: logits, column ids and the row view's order read once, means and counts written
    cell_bytes = cfg.B * N * 12.0 + cfg.B * (cfg.n_rows + 1) * (cfg.n_cols + 1) * 8.0

    # ---- end-to-end timing: pinned host inputs -> device, forward + backward, results -> host
    e2e_steps = max(3, min(K, 20))
    res_host = {k: torch.empty_like(pinned["Q"]) for k in ("O", "dQ", "dK", "dV")}
    lse_host = torch.empty((cfg.B, cfg.H, N), dtype=torch.float32).pin_memory()
    for k in res_host:
        res_host[k] = res_host[k].pin_memory()
    h2d = sum(pinned[k].numel() * pinned[k].element_size() for k in ("Q", "K", "V", "dO"))
    d2h = sum(t.numel() * t.element_size() for t in res_host.values()) + lse_host.numel() * 4

    def e2e_step(d):
        for k in ("Q", "K", "V", "dO"):
            d[k].copy_(pinned[k], non_blocking=True)
        dQ, dK, dV = step(d)
        res_host["O"].copy_(d["O"], non_blocking=True)
        lse_host.copy_(d["LSE"], non_blocking=True)
        res_host["dQ"].copy_(dQ, non_blocking=True)
        res_host["dK"].copy_(dK, non_blocking=True)
        res_host["dV"].copy_(dV, non_blocking=True)

    e2e_step(sets[0])
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(e2e_steps):
        e2e_step(sets[i % N_BUFFER_SETS])
    e1.record()
    torch.cuda.synchronize()
    e2e_serial_ms = e0.elapsed_time(e1) / e2e_steps

    # The same steps pipelined the way a caller would run them: uploads, kernels and downloads on three
    # streams over double-buffered device sets, ordered by events, so that the copies of step i + 1 and
    # of step i - 1 run under the kernels of step i.  Every step still moves all its inputs up and all
    # its results down inside the timed region.  All kernels run on one stream (calls on one plan must
    # not overlap).
    s_up, s_run, s_down = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    res_host2 = [{k: torch.empty_like(pinned["Q"]).pin_memory() for k in ("O", "dQ", "dK", "dV")} for _ in range(2)]
    lse_host2 = [torch.empty((cfg.B, cfg.H, N), dtype=torch.float32).pin_memory() for _ in range(2)]
    grads = [None, None]
    up_done = [torch.cuda.Event() for _ in range(2)]
    run_done = [torch.cuda.Event() for _ in range(2)]
    down_done = [torch.cuda.Event() for _ in range(2)]

    def e2e_pipelined(n_steps):
        for i in range(n_steps):
            j = i & 1
            dset = sets[j]
            with torch.cuda.stream(s_up):
                if i >= 2:
                    s_up.wait_event(run_done[j])      # the kernels of step i - 2 have read this set
                for k in ("Q", "K", "V", "dO"):
                    dset[k].copy_(pinned[k], non_blocking=True)
                up_done[j].record(s_up)
            with torch.cuda.stream(s_run):
                s_run.wait_event(up_done[j])
                if i >= 2:
                    s_run.wait_event(down_done[j])    # the results of step i - 2 have left the device
                mate.mate_attn_fwd(plan, dset["Q"], dset["K"], dset["V"], scale, fwd_impl, out=dset["O"], lse=dset["LSE"])
                grads[j] = mate.mate_attn_bwd(plan, dset["Q"], dset["K"], dset["V"], dset["O"], dset["LSE"], dset["dO"],
                                              scale)
                run_done[j].record(s_run)
            with torch.cuda.stream(s_down):
                s_down.wait_event(run_done[j])
                res_host2[j]["O"].copy_(dset["O"], non_blocking=True)
                lse_host2[j].copy_(dset["LSE"], non_blocking=True)
                for nm, g in zip(("dQ", "dK", "dV"), grads[j]):
                    res_host2[j][nm].copy_(g, non_blocking=True)
                down_done[j].record(s_down)

    torch.cuda.synchronize()
    e2e_pipelined(4)
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    t_p0 = time.perf_counter()
    e2e_pipelined(e2e_steps)
    torch.cuda.synchronize()
    e2e_ms = (time.perf_counter() - t_p0) * 1e3 / e2e_steps

    if rank == 0:
        sampler.stop()

    times = torch.tensor([total_ms, float(np.median(fwd_ms)), float(np.median(bwd_ms)), e2e_ms,
                          float(fwd_ms.min()), float(bwd_ms.min()), e2e_serial_ms, fwd_warm_ms, bwd_warm_ms],
                         dtype=torch.float64, device=dev)
    work = torch.tensor([pairs, n_valid_tokens], dtype=torch.float64, device=dev)
    (total_ms, fwd_med, bwd_med, e2e_ms, fwd_min, bwd_min, e2e_serial_ms, fwd_warm_ms, bwd_warm_ms), \
        (pairs_all, tokens_all) = reduce_over_ranks(times, work, world)
    ff, fb = pair_flops(cfg, pairs_all)
    ms_per_step = total_ms / K

    if rank == 0:
        value = (ff + fb) / (ms_per_step * 1e-3) / 1e12
        fwd_tflops = ff / (fwd_med * 1e-3) / 1e12
        bwd_tflops = fb / (bwd_med * 1e-3) / 1e12
        # Roofline of the dominant kernel, tc_bwd_kernel (one launch = the whole backward of one
        # rank).  Its duration is taken as that of the mate_attn_bwd call, which also holds the
        # small row-dot kernel (about 5% by the ncu launch list), so `achieved` is a lower bound
        # for the kernel itself.
        fwd_tflops_rank = f_fwd / (float(np.mean(fwd_ms)) * 1e-3) / 1e12
        bwd_tflops_rank = f_bwd / (float(np.mean(bwd_ms)) * 1e-3) / 1e12
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
            "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "B": cfg.B, "H": cfg.H, "N": N, "d": cfg.d, "P": cfg.P,
                       "useful_pairs": pairs_all, "dense_pairs": float(world * cfg.B * cfg.H * N * N),
                       "l2": "rotating %d buffer sets of %.0f MB (> 126 MB L2)" % (N_BUFFER_SETS, set_bytes / 1e6),
                       "plan": "pre-computed, outside the timed region", "fwd_loader": args.loader},
            "fwd": {"ms_median": fwd_med, "ms_min": fwd_min, "ms_l2_warm": fwd_warm_ms, "tflops": fwd_tflops,
                    "frac_of_bf16_peak": fwd_tflops / (peaks["bf16_tflops"] * world),
                    "tokens_per_s": tokens_all / (fwd_med * 1e-3)},
            "bwd": {"ms_median": bwd_med, "ms_min": bwd_min, "ms_l2_warm": bwd_warm_ms, "tflops": bwd_tflops,
                    "frac_of_bf16_peak": bwd_tflops / (peaks["bf16_tflops"] * world),
                    "tokens_per_s": tokens_all / (bwd_med * 1e-3)},
            "tokens_per_s": tokens_all / (ms_per_step * 1e-3),
            "tokens_per_s_padded": world * cfg.B * N / (ms_per_step * 1e-3),
            "plan": {"wall_ms": plan_wall_ms, "stream_ms": plan_dev_ms,
                     "note": "mate_plan, pre-computed once per table, outside the timed step: wall time of the call "
                             "(two allocations, plan kernel, work-lists built on the host) and time between two "
                             "events on its stream; plan_kernel alone is in the ncu launch list under profiles/"},
            "cell_mean": None if not cell_ms else {
                "ms": cell_ms, "gbs": cell_bytes / (cell_ms * 1e-3) / 1e9, "peak_gbs": peaks["hbm_gbs"],
                "frac": cell_bytes / (cell_ms * 1e-3) / 1e9 / peaks["hbm_gbs"],
                "note": "100 KB of ids and logits: latency-bound at this size, far from the HBM roofline it is named against"},
            "roofline": {"kernel": "tc_bwd_kernel", "bound": "tensor", "achieved": bwd_tflops_rank,
                         "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": bwd_tflops_rank / peaks["bf16_tflops"], "peak_source": peaks["source"],
                         "traffic": ncu_traffic("tc_bwd_kernel", cfg.name)},
            "roofline_fwd": {"kernel": "tc_fwd_kernel", "bound": "tensor", "achieved": fwd_tflops_rank,
                             "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                             "frac": fwd_tflops_rank / peaks["bf16_tflops"], "peak_source": peaks["source"],
                             "traffic": ncu_traffic("tc_fwd_kernel", cfg.name)},
            "e2e": {"value": (ff + fb) / (e2e_ms * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": e2e_ms,
                    "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "how": "uploads, kernels and downloads on three streams over two device sets; wall clock",
                    "serial_ms_per_step": e2e_serial_ms,
                    "serial_value": (ff + fb) / (e2e_serial_ms * 1e-3) / 1e12},
            "gpu_launches": K * launches_per_step,
            "clocks": sampler.summary(t_wall0, t_wall1),
        }
        if world == 1 and not args.no_cpu_baseline:
            runs = [oracle_step(cfg, rows, cols, host, hv, scale) for _ in range(3)]
            tf, tb = min(r[0] for r in runs), min(r[1] for r in runs)
            import oracle
            line["cpu_baseline"] = {
                "value": (f_fwd + f_bwd) / (tf + tb) / 1e12, "unit": UNIT, "cores": oracle.num_threads(),
                "kind": "oracle", "fwd_s": tf, "bwd_s": tb,
                "sample": "whole %s workload (B=%d H=%d N=%d), fwd+bwd, fp64, best of 3 runs" % (cfg.name, cfg.B, cfg.H, N)}
        print(json.dumps(line), flush=True)
    plan.destroy()
    if world > 1:
        dist.destroy_process_group()


FWD_TRACE_LABELS = {
    "softmax warp 0 (half 0)": ["wait S", "wait previous P V", None, "tile: S seen to P handed over", "tiles", "unit set-up",
                               "epilogue", "total"],
    "softmax warp 4 (half 1)": ["wait S", "wait previous P V", None, "tile: S seen to P handed over", "tiles", "unit set-up",
                               "epilogue", "total"],
    "MMA thread of half 0": ["wait Q", "wait P", "issue Q K^T", "issue P V", "tiles", "wait K/V tile", "wait S free", "total"],
    "loader warp 10": ["wait for a free buffer", "flush pending copies", "issue copies", "commit and signal", "tiles", None, None,
                       "total"],
}
BWD_TRACE_LABELS = {
    "arithmetic warp 0": ["wait S/dP", "wait previous gradient MMAs", "arithmetic", "epilogue", "tensor-memory loads", "total",
                          "signal operands", "tiles"],
    "arithmetic warp 4": ["wait S/dP", "wait previous gradient MMAs", "arithmetic", "epilogue", "tensor-memory loads", None,
                          "signal operands", "tiles"],
    "MMA thread": ["wait row operands", "wait column tile", "wait operands from the warps", "issue gradient MMAs", "issue S/dP",
                   "wait S/dP read", None, "tiles"],
    "loader warp": ["wait for a free buffer", None, None, None, None, None, None, None],
}


def run_trace(args, cfg):
    """Per-role cycle counters of the two tensor-core kernels: builds the profiling variant of the library
    (-DMATE_TRACE), runs a few steps and prints the mean over the CTAs of every counter, one JSON line."""
    import ctypes
    from paper_2109_04312_b200 import build as lib_build
    os.environ["MATE_LIB"] = lib_build.build(trace=True)
    import torch
    import paper_2109_04312_b200 as mate
    from paper_2109_04312_b200 import api
    torch.cuda.set_device(0)
    rows, cols, info = tables.make_structure(cfg, 1234)
    hv = tables.head_view(cfg)
    vals = tables.make_values(cfg, info["N"], 5678)
    plan = mate.mate_plan(torch.from_numpy(rows).cuda(), torch.from_numpy(cols).cuda(), cfg.P, hv, cfg.n_rows, cfg.n_cols)
    Q, K, V, dO = (torch.from_numpy(vals[n]).cuda().to(torch.bfloat16) for n in ("Q", "K", "V", "dO"))
    for _ in range(max(args.warmup, 3)):
        O, LSE = mate.mate_attn_fwd(plan, Q, K, V)
        mate.mate_attn_bwd(plan, Q, K, V, O, LSE, dO)
    torch.cuda.synchronize()
    plan.status()
    lib = api._load()
    n_sm = torch.cuda.get_device_properties(0).multi_processor_count
    out = {"trace": cfg.name, "clock": "SM cycles per CTA, mean over %d CTAs of one launch" % n_sm}
    for key, fn, labels in (("tc_fwd_kernel", lib.mate_debug_trace, FWD_TRACE_LABELS),
                            ("tc_bwd_kernel", lib.mate_debug_trace_bwd, BWD_TRACE_LABELS)):
        buf = np.zeros((256, 4, 8), np.int64)
        fn.restype = ctypes.c_int
        assert fn(ctypes.c_void_p(buf.ctypes.data)) == 0
        buf = buf[:n_sm].astype(np.float64)
        out[key] = {}
        for r, (role, names) in enumerate(labels.items()):
            out[key][role] = {nm: round(float(buf[:, r, i].mean())) for i, nm in enumerate(names) if nm}
            if "total" in out[key][role]:
                i = names.index("total")
                out[key][role]["total of the slowest CTA"] = round(float(buf[:, r, i].max()))
    print(json.dumps(out), flush=True)
    plan.destroy()


def spawn_ranks(argv, n, run=subprocess.call):
    """`python bench.py --gpus N` without a launcher: start the N ranks here, one per GPU, through
    torch.distributed.run on the loopback address, and return its exit code."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", str(n),
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + list(argv)
    return run(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="mate", choices=["mate", "reference"])
    ap.add_argument("--workload", default="long", choices=sorted(tables.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--trace", action="store_true",
                    help="print the per-role cycle counters of the profiling build instead of timing")
    ap.add_argument("--loader", default="auto", choices=["auto", "gather", "bulk"],
                    help="forward K/V tiles that are contiguous in the tensors: the library's default (bulk tensor "
                         "copies), row-by-row gathers like every other tile, or bulk tensor copies stated explicitly")
    args = ap.parse_args()
    cfg = tables.CONFIGS[args.workload]
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "mate":
        sys.exit(spawn_ranks(sys.argv[1:], args.gpus))
    if args.trace:
        run_trace(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        args.warmup = max(args.warmup, 3)
        run_mate(args, cfg)


if __name__ == "__main__":
    main()
