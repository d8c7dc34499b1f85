#!/usr/bin/env python
"""Benchmark: one step = one whole aggregation (CenteredClip + verification) of one synthetic
gradient tensor.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

Without --config the workload is configuration 5 (64 peers, d = 2^28, 64 GiB of rows: the largest
one that fits a GPU), run for a fixed 20 updates with the Gram variant timed beside it, and the line
also carries a `per_config` object with configurations 2, 3 and 4.

N > 1 is launched by torchrun (one rank per GPU); the partitions of the method are independent, but
the target of this build is a single GPU, so every rank aggregates its own replica of the workload
(no data-path collective) and the reported value is the sum over ranks ("weak" scaling).
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "CenteredClip+verify input GB/s"
UNIT = "GB/s"
DEFAULT_CONFIG = 5


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def recorded_traffic(kernel, config):
    """DRAM bytes per launch taken from ncu captures, kept as data next to their summaries.  Returns
    (cold, steady, note): cold = caches flushed before the launch (ncu's default), steady = the same
    launch between its neighbours without the flush.  (None, None, why) when no capture covers it."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.json")
    try:
        with open(path) as f:
            table = json.load(f)
    except (OSError, ValueError):
        return None, None, "no capture on record"
    for row in table.get("captures", []):
        if row.get("kernel") == kernel and row.get("config") == config:
            return row.get("cold_bytes_per_launch"), row.get("steady_bytes_per_launch"), row.get("note")
    return None, None, "no capture of this kernel on this workload"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.QUERY,
                 "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                smax.append(float(f[2]))
            except ValueError:
                continue
            for name, val in zip(names, f[5:9]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2] if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(ms, dist, device):
    """The job is as slow as its slowest replica: MAX of a per-rank time over all ranks."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(bytes_per_rank, ms_step, world):
    """Replicas only: every rank aggregates its own copy, the job's throughput is the sum."""
    return world * bytes_per_rank / (ms_step * 1e-3) / 1e9


def algorithmic_bytes(w, iters, gram=False):
    """Bytes the method must move for one aggregation: one init pass, one pass per update and one
    verification pass over each partition's [n][row_stride] rows, each with v read and written.
    The Gram variant needs a Gram pass and a combine-and-verify pass, whatever the number of updates.
    Returns (input bytes only, bytes with v, passes per partition)."""
    n, stride = w.n, w.row_stride
    per_pass = n * stride * 4 * (1.0 + 2.0 / n)
    input_only = n * stride * 4
    passes = [2 for _ in iters] if gram else [2 + int(i) for i in iters]
    return sum(passes) * input_only, sum(passes) * per_pass, passes


def workload_name(cfg, w, P=None):
    return "config %d: n=%d peers, d=%d, P=%d partitions, row_stride=%d" % (cfg, w.n, w.d, w.P if P is None else P,
                                                                           w.row_stride)


class Runner:
    """One workload resident in HBM, with the buffers both algorithms need."""

    def __init__(self, w, btard, torch):
        self.w, self.btard, self.torch = w, btard, torch
        g = w.g
        self.P, self.n, self.stride = g.shape
        dev = g.device
        self.ws_v = torch.empty(btard.verify_projections_workspace(self.n, self.P, self.stride, w.K),
                                dtype=torch.uint8, device=dev)
        self.ws = {}
        self.v = {}
        self.state = {}

    def _buffers(self, algo):
        torch, btard, w = self.torch, self.btard, self.w
        if algo not in self.ws:
            dev = w.g.device
            self.ws[algo] = torch.empty(btard.centered_clip_workspace(self.n, self.P, self.stride, w.stop_mode, algo),
                                        dtype=torch.uint8, device=dev)
            self.v[algo] = torch.empty((self.P, self.stride), dtype=torch.float32, device=dev)
            self.state[algo] = {}
        return self.ws[algo], self.v[algo], self.state[algo]

    def aggregate(self, algo, max_iters=None):
        """One aggregation + verification; the Gram variant goes through the one-call entry point
        (combine and verification passes fused), the direct ones through the two calls."""
        btard, w = self.btard, self.w
        ws, v, st = self._buffers(algo)
        iters = w.max_iters if max_iters is None else max_iters
        ckeys = ("iters", "last_step_norm", "resid_norm", "status")
        vkeys = ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm", "status")
        if algo == btard.ALGO_GRAM:
            r, o = btard.centered_clip_verify(w.g, w.tau, w.zseed, K=w.K, part_len=w.part_len, init_mode=w.init_mode,
                                              v=v, stop_mode=w.stop_mode, max_iters=iters, eps=w.eps, algo=algo,
                                              workspaces=(ws, self.ws_v),
                                              out=(st.get("c"), st.get("v")) if st else None)
        else:
            r = btard.centered_clip(w.g, w.tau, part_len=w.part_len, init_mode=w.init_mode, v=v,
                                    stop_mode=w.stop_mode, max_iters=iters, eps=w.eps, algo=algo,
                                    workspace=ws, out=st.get("c"))
            o = btard.verify_projections(w.g, v, w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                         resid_norm_in=r["resid_norm"], workspace=self.ws_v, out=st.get("v"))
        st["c"] = {k: r[k] for k in ckeys}
        st["v"] = {k: o[k] for k in vkeys}

    def timed(self, algo, steps, warmup, max_iters=None, dist=None):
        """CUDA-event time of `steps` back-to-back aggregations after `warmup` untimed ones: ms per
        aggregation, with nothing but the library's own launches on the stream in between."""
        torch = self.torch
        for _ in range(warmup):
            self.aggregate(algo, max_iters)
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        launches0 = self.btard.kernel_launch_count()
        e0.record()
        for _ in range(steps):
            self.aggregate(algo, max_iters)
        e1.record()
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        return e0.elapsed_time(e1) / steps, self.btard.kernel_launch_count() - launches0

    def iters(self, algo):
        st = self.state[algo]
        return st["c"]["iters"].cpu().numpy(), st["c"]["status"].cpu().numpy()

    def iteration_launch_ms(self, algo, steps, ms_full=None):
        """Duration of one launch of the CenteredClip update pass inside the un-bracketed step, by
        difference: the same steps with I and with I // 2 updates differ by I - I // 2 launches of that
        kernel and nothing else.  I = the smallest number of updates any partition applied (so that every
        partition takes part in every one of them).  Returns (ms per launch, I, I // 2, ms at I, ms at I // 2)."""
        it, _ = self.iters(algo)
        full = int(it.min())
        half = full // 2
        if full < 2:
            return None, full, half, None, None
        if ms_full is None or full != self.w.max_iters:
            ms_full, _ = self.timed(algo, steps, 2, max_iters=full)
        ms_half, _ = self.timed(algo, steps, 2, max_iters=half)
        self.aggregate(algo)                                    # leave the full run's outputs in place
        self.torch.cuda.synchronize()
        return (ms_full - ms_half) / (full - half), full, half, ms_full, ms_half


def config_record(cfg, steps, peak, btard, torch, workloads):
    """Configuration `cfg` in both algorithms: ms per aggregation, input GB/s, fraction of the peak, and the
    roofline record of its dominant kernel (the update pass of the direct algorithm)."""
    w = workloads.make_workload(cfg, device="cuda")
    run = Runner(w, btard, torch)
    out = {"workload": workload_name(cfg, w), "stop": "eps" if w.stop_mode else "fixed", "max_iters": w.max_iters, "K": w.K}
    per_pass = w.n * w.row_stride * 4 * (1.0 + 2.0 / w.n) * w.P
    for name, algo in (("direct", btard.ALGO_DIRECT), ("gram", btard.ALGO_GRAM)):
        used = steps
        ms, launches = run.timed(algo, used, 3)
        if ms * used < 40.0:                      # a sub-millisecond aggregation: time at least 40 ms of them
            used = min(400, int(40.0 / ms) + 1)
            ms, launches = run.timed(algo, used, 0)
        it, status = run.iters(algo)
        in_bytes, _, passes = algorithmic_bytes(w, it, gram=(name == "gram"))
        out[name] = {"ms_per_aggregation": ms, "steps": used, "value": in_bytes / (ms * 1e-3) / 1e9, "unit": UNIT,
                     "fraction_of_hbm_peak": in_bytes / (ms * 1e-3) / 1e9 / peak,
                     "passes_per_partition": [min(passes), max(passes)], "updates": [int(it.min()), int(it.max())],
                     "not_converged_partitions": int((status & 1).sum()), "gpu_launches_per_step": launches / used}
        if name == "direct":
            ms_launch, full, half, ms_full, ms_half = run.iteration_launch_ms(algo, steps, ms_full=ms)
            cold, steady, note = recorded_traffic("cclip_pass_kernel<ITER>", cfg)
            out["roofline"] = {
                "kernel": "cclip_pass_kernel<ITER>", "bound": "hbm", "unit": UNIT, "peak": peak,
                "achieved": per_pass / (ms_launch * 1e-3) / 1e9 if ms_launch else None,
                "frac": per_pass / (ms_launch * 1e-3) / 1e9 / peak if ms_launch else None,
                "avg_launch_ms": ms_launch, "algorithmic_bytes_per_launch": per_pass,
                "how": "difference of the un-bracketed step at %d and %d updates" % (full, half),
                "ms_step_at_full": ms_full, "ms_step_at_half": ms_half,
                "traffic": steady if steady is not None else cold, "traffic_cold": cold, "traffic_note": note}
    vd = run.v[btard.ALGO_DIRECT]
    out["rel_l2_difference_of_v"] = float((run.v[btard.ALGO_GRAM] - vd).norm() / vd.norm())
    del run, w
    torch.cuda.empty_cache()
    return out


def oracle_sample(cfg, workloads, cores, seconds_per_step, device="cpu"):
    """A bounded sample of configuration `cfg` for the float64 oracle on the host cores: whole partitions,
    one per core, for the configurations that fit; for the 64 GiB configuration partitions of the same
    recipe with shorter rows, sized so that one step takes about `seconds_per_step`."""
    meta = workloads.make_workload(cfg, data=False)
    P = meta.P
    parts = list(range(0, P, max(1, P // max(1, min(cores, P)))))[:cores]
    if meta.d >= (1 << 27):
        # one core streams about 0.45 GiB of rows x 22 passes in 16 s: scale the row length to the budget
        shrink = 4 if seconds_per_step >= 8 else 16
        d = meta.d // shrink
        w = workloads.make_workload(cfg, device=device, d=d, partitions=parts)
        text = ("%d partitions of config %d's recipe (same peers, attacks, tau, K) with rows of %d instead of %d "
                "columns, full iteration count + verification" % (len(parts), cfg, w.row_stride, meta.row_stride))
    else:
        w = workloads.make_workload(cfg, device=device, partitions=parts)
        text = "partitions %s of config %d, full iteration count + verification" % (parts, cfg)
    w.g = w.g.cpu()                                          # generated where it is fastest, timed on the host
    return w, text


def oracle_step(w, oracle, np):
    ref = oracle.centered_clip(w.g.numpy(), w.tau, w.part_len, init_mode=w.init_mode, stop_mode=w.stop_mode,
                               max_iters=w.max_iters, eps=w.eps)
    oracle.verify(w.g.numpy(), ref["v"].astype(np.float32), w.tau, w.zseed, K=w.K, part_len=w.part_len,
                  norm_in=ref["resid_norm"])
    return ref["iters"]


def run_ours(args):
    import numpy as np
    import torch
    import workloads
    import paper_2106_11257_b200 as btard
    from paper_2106_11257_b200 import build as lib_build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local)
    if not lib_build.up_to_date():
        if local == 0:
            lib_build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    btard.lib()
    peak, peak_kind = measured_peaks()
    cfg = args.config if args.config else DEFAULT_CONFIG

    # ---- the other configurations first (rank 0 only; they are freed before the main workload) ------
    per_config = None
    if args.config is None and not args.no_per_config and rank == 0:
        per_config = {}
        for c in (2, 3, 4):
            per_config[str(c)] = config_record(c, max(3, min(args.steps, 10)), peak, btard, torch, workloads)
    if dist:
        dist.barrier()

    w = workloads.make_workload(cfg, device="cuda", d=args.d)
    if args.max_iters:
        w.max_iters = args.max_iters
    if args.stop:
        w.stop_mode = {"fixed": btard.STOP_FIXED_ITERS, "eps": btard.STOP_EPS}[args.stop]
    g = w.g
    P, n, stride = g.shape
    dev = g.device
    algo = {"direct": btard.ALGO_DIRECT, "gram": btard.ALGO_GRAM, "cooperative": btard.ALGO_DIRECT_COOPERATIVE}[args.algo]
    run = Runner(w, btard, torch)

    for _ in range(args.warmup):
        run.aggregate(algo)
    torch.cuda.synchronize()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # Timed region: K steps, nothing but the library's own launches on the stream.
    ms_step, launches = run.timed(algo, args.steps, 0, dist=dist)
    clocks = sampler.stop() if rank == 0 else None
    ms_step = max_over_ranks(ms_step, dist, dev)
    iters, status = run.iters(algo)
    in_bytes, alg_bytes, passes = algorithmic_bytes(w, iters, gram=(args.algo == "gram"))
    value = whole_job_value(in_bytes, ms_step, world)

    # ---- the dominant kernel inside the un-bracketed step -------------------------------------------
    per_pass_bytes = n * stride * 4 * (1.0 + 2.0 / n) * P
    roof = None
    if args.algo != "gram":
        k_diff = max(2, min(args.steps, 5))
        ms_launch, full, half, ms_full, ms_half = run.iteration_launch_ms(algo, k_diff, ms_full=ms_step if world == 1 else None)
        cold, steady, note = recorded_traffic("cclip_pass_kernel<ITER>", cfg)
        achieved = per_pass_bytes / (ms_launch * 1e-3) / 1e9 if ms_launch else None
        roof = {"kernel": "cclip_pass_kernel<ITER>", "bound": "hbm", "achieved": achieved, "peak": peak,
                "peak_kind": peak_kind, "unit": UNIT, "frac": achieved / peak if achieved else None,
                "traffic": steady if steady is not None else cold, "traffic_cold": cold, "traffic_note": note,
                "launches_per_step": full, "avg_launch_ms": ms_launch,
                "algorithmic_bytes_per_launch": per_pass_bytes,
                "how": "difference of the un-bracketed timed step at %d and at %d updates, divided by %d launches"
                       % (full, half, full - half),
                "ms_step_at_full": ms_full, "ms_step_at_half": ms_half,
                "kernel_ms_per_step": ms_launch * full if ms_launch else None}
    else:
        # the Gram variant has two passes of about equal weight; its Gram pass is the contraction
        roof = {"kernel": "gram pass + combine-and-verify pass", "bound": "hbm", "unit": UNIT, "peak": peak,
                "peak_kind": peak_kind, "achieved": 2 * per_pass_bytes / (ms_step * 1e-3) / 1e9,
                "frac": 2 * per_pass_bytes / (ms_step * 1e-3) / 1e9 / peak, "traffic": None,
                "algorithmic_bytes_per_launch": per_pass_bytes,
                "how": "two passes of algorithmic bytes over the whole aggregation (median start and "
                       "coefficient iteration counted as time only)"}

    # ---- per-kernel breakdown: a second run with every launch bracketed by events (informational) ----
    kernels = None
    if not args.no_kernel_events:
        k_ev = max(1, min(args.steps, 3))
        btard.profile_collect()
        btard.profile_enable(True)
        for _ in range(k_ev):
            run.aggregate(algo)
        torch.cuda.synchronize()
        btard.profile_enable(False)
        prof = btard.profile_collect()
        kernels = {k: {"ms_per_step": prof[k][0] / k_ev, "launches_per_step": prof[k][1] / k_ev} for k in prof}
        kernels["note"] = ("event-bracketed run: the events stop consecutive launches from overlapping, so these "
                           "sum to more than ms_per_step; the roofline uses the un-bracketed difference instead")

    # ---- the other algorithm on the same tensor, for the side-by-side the configurations ask for ---
    other = None
    if args.side_by_side and w.n <= 128 and args.algo != "cooperative":
        other_algo = btard.ALGO_DIRECT if args.algo == "gram" else btard.ALGO_GRAM
        k3 = max(3, min(args.steps, 10))
        ms_o, launches_o = run.timed(other_algo, k3, 3, dist=dist)
        ms_o = max_over_ranks(ms_o, dist, dev)
        it_o, _ = run.iters(other_algo)
        ob, _, _ = algorithmic_bytes(w, it_o, gram=(other_algo == btard.ALGO_GRAM))
        diff = float((run.v[other_algo] - run.v[algo]).norm() / run.v[algo].norm())
        other = {"algo": "direct" if args.algo == "gram" else "gram", "ms_per_aggregation": ms_o,
                 "value": whole_job_value(ob, ms_o, world), "unit": UNIT,
                 "fraction_of_hbm_peak": ob / (ms_o * 1e-3) / 1e9 / peak,
                 "passes_counted": "2 per partition (Gram pass, combine-and-verify pass); the median start and the "
                                   "coefficient iteration are time without bytes, so this fraction is not comparable "
                                   "with the direct algorithm's" if other_algo == btard.ALGO_GRAM
                                   else "1 init + updates + 1 verify per partition",
                 "gpu_launches_per_step": launches_o / k3, "rel_l2_difference_of_v": diff}

    # ---- end to end: host buffers in, host results out, copies inside the timed region ----------
    e2e = None
    if not args.no_e2e:
        e2e = end_to_end(args, w, btard, torch, dist, dev, world, in_bytes_fn=lambda it, gram: algorithmic_bytes(w, it, gram)[0])

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample of the same workload ---------
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        cores = oracle.max_threads()
        ws, text = oracle_sample(cfg, workloads, cores, seconds_per_step=10, device="cuda")
        if args.max_iters:
            ws.max_iters = args.max_iters
        t0 = time.perf_counter()
        it_ref = oracle_step(ws, oracle, np)
        dt = time.perf_counter() - t0
        cb, _, _ = algorithmic_bytes(ws, it_ref)
        cpu_baseline = {"value": cb / dt / 1e9, "unit": UNIT, "cores": min(cores, ws.P),
                        "kind": "oracle", "seconds": dt, "sample": text}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_name(cfg, w),
                   "algo": args.algo, "init": "coordinate median", "stop": "eps" if w.stop_mode else "fixed",
                   "max_iters": w.max_iters, "eps": w.eps, "K": w.K,
                   "updates_per_partition": [int(iters.min()), int(iters.max())],
                   "not_converged_partitions": int((status & 1).sum()),
                   "passes_counted": ("1 Gram + 1 combine-and-verify per partition" if args.algo == "gram"
                                      else "1 init + updates + 1 verify per partition"),
                   "l2": "input (%.0f MB) larger than L2 (126 MB), no flush" % (g.numel() * 4 / 1e6),
                   "multi_gpu": "replicas only" if world > 1 else "single GPU"},
        "fraction_of_hbm_peak": value / world / peak, "hbm_peak_gbs": peak, "hbm_peak_kind": peak_kind,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": e2e,
        "roofline": roof,
        "kernels_bracketed": kernels,
        "ms_per_aggregation": ms_step,
        "other_algorithm": other,
        "per_config": per_config,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def end_to_end(args, w, btard, torch, dist, dev, world, in_bytes_fn):
    """The same metric through btard_aggregate_host: pinned host rows in, host results out, both copies
    inside the timed region, for the direct algorithm and for the Gram variant.  The headline entry is
    the algorithm of this run; the other one rides along.  Skipped (with the reason) when the rows do not
    fit in host memory."""
    g = w.g
    P, n, stride = g.shape
    need = g.numel() * 4
    try:
        with open("/proc/meminfo") as f:
            avail = [int(l.split()[1]) * 1024 for l in f if l.startswith("MemAvailable")][0]
    except (OSError, IndexError):
        avail = None
    if avail is not None and need > 0.6 * avail:
        return {"value": None, "unit": UNIT, "h2d_bytes_per_step": need, "d2h_bytes_per_step": None,
                "skipped": "the rows (%.1f GB) do not fit in the host memory available to this process (%.1f GB)"
                           % (need / 1e9, avail / 1e9)}
    gh = torch.empty(g.shape, dtype=torch.float32, pin_memory=True)
    gh.copy_(g)
    copy_stream = torch.cuda.Stream()
    out = {}
    main = "gram" if args.algo == "gram" else "direct"
    for name, algo in (("direct", btard.ALGO_DIRECT), ("gram", btard.ALGO_GRAM)):
        if name != main and (not args.side_by_side or w.n > 128):
            continue
        scratch = torch.empty(btard.aggregate_host_scratch(n, P, stride, w.K, algo), dtype=torch.uint8, device=dev)
        hout = None

        def host_step():
            nonlocal hout
            r = btard.aggregate_host(gh, w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                     init_mode=w.init_mode, stop_mode=w.stop_mode,
                                     max_iters=w.max_iters, eps=w.eps, scratch=scratch, out=hout,
                                     copy_stream=copy_stream, algo=algo)
            hout = {k: r[k] for k in r if k != "scratch"}
        for _ in range(max(1, min(args.warmup, 2))):
            host_step()
        torch.cuda.synchronize()
        if dist:
            dist.barrier()
        k2 = max(1, min(args.steps, 5))
        t0 = time.perf_counter()
        for _ in range(k2):
            host_step()
        torch.cuda.synchronize()
        ms = (time.perf_counter() - t0) * 1e3 / k2
        ms = max_over_ranks(ms, dist, dev)
        d2h = sum(hout[k].numel() * hout[k].element_size() for k in hout)
        in_bytes = in_bytes_fn(hout["iters"].numpy(), name == "gram")
        out[name] = {"value": whole_job_value(in_bytes, ms, world), "unit": UNIT, "ms_per_step": ms,
                     "h2d_bytes_per_step": need, "d2h_bytes_per_step": d2h, "algo": name}
        del scratch
    e2e = dict(out[main])
    for name in out:
        if name != main:
            e2e["other_algorithm"] = out[name]
    del gh
    return e2e


def run_reference(args):
    """The reference arm is the float64 oracle on the host cores: each step aggregates a bounded
    sample of the same workload (one partition per core)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    import workloads

    cfg = args.config if args.config else DEFAULT_CONFIG
    cores = oracle.max_threads()
    meta = workloads.make_workload(cfg, data=False)
    w, sample_txt = oracle_sample(cfg, workloads, cores, seconds_per_step=3)
    if args.max_iters:
        w.max_iters = args.max_iters
    iters = None
    for _ in range(args.warmup):
        iters = oracle_step(w, oracle, np)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        iters = oracle_step(w, oracle, np)
    dt = (time.perf_counter() - t0) / args.steps
    in_bytes, _, _ = algorithmic_bytes(w, iters)
    value = in_bytes / dt / 1e9
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(cfg, meta), "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, w.P),
                         "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=None,
                    help="1-5; default: configuration 5 plus a per_config object for 2, 3 and 4")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--algo", default="direct", choices=["direct", "gram", "cooperative"])
    ap.add_argument("--max-iters", type=int, default=None, help="override the configuration's iteration cap")
    ap.add_argument("--d", type=int, default=None,
                    help="override the configuration's vector length (smaller cases for profiler captures)")
    ap.add_argument("--stop", default=None, choices=["fixed", "eps"], help="override the configuration's stop rule")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="skip the event-bracketed run that gives the per-kernel breakdown")
    ap.add_argument("--no-side-by-side", dest="side_by_side", action="store_false",
                    help="do not also time the other algorithm (direct / Gram) on the same tensor")
    ap.add_argument("--no-per-config", action="store_true", help="skip configurations 2-4 in the default run")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
