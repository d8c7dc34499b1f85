#!/usr/bin/env python
"""Benchmark: one step = one whole aggregation (CenteredClip + verification) of one synthetic
gradient tensor.  Prints ONE JSON line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config C] [--impl ours|reference]

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
# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the iteration kernel (ncu capture
# summarised in profiles/cclip_pass_iter_config2.md); set to None whenever that kernel changes.
ITER_TRAFFIC = {(2, "direct"): 791.9e6}
UNIT = "GB/s"


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


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
    The Gram variant needs a Gram pass, a combine pass and the verification pass, whatever the
    number of updates."""
    n, stride = w.n, w.row_stride
    per_pass = n * stride * 4 * (1.0 + 2.0 / n)
    input_only = n * stride * 4
    passes = [2 for _ in iters] if gram else [2 + int(i) for i in iters]   # Gram: combine and verification are one pass
    return sum(passes) * input_only, sum(passes) * per_pass, passes


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

    w = workloads.make_workload(args.config, device="cuda")
    if args.max_iters:
        w.max_iters = args.max_iters
    g = w.g
    P, n, stride = g.shape
    dev = g.device
    algo = {"direct": btard.ALGO_DIRECT, "gram": btard.ALGO_GRAM,
            "cooperative": btard.ALGO_DIRECT_COOPERATIVE, "resident": btard.ALGO_DIRECT_RESIDENT,
            "staged": btard.ALGO_DIRECT_STAGED}[args.algo]
    ws_c = torch.empty(btard.centered_clip_workspace(n, P, stride, w.stop_mode, algo), dtype=torch.uint8, device=dev)
    ws_v = torch.empty(btard.verify_projections_workspace(n, P, stride, w.K), dtype=torch.uint8, device=dev)
    v = torch.empty((P, stride), dtype=torch.float32, device=dev)
    state = {}

    ckeys = ("iters", "last_step_norm", "resid_norm", "status")
    vkeys = ("norm", "weight", "dot", "s", "s_sum", "znorm2", "resid_sum_norm", "status")

    def aggregate(which, vbuf, ws, st):
        """One aggregation + verification with algorithm `which`; the Gram variant goes through the one-call
        entry point (combine and verification passes fused where the library can)."""
        if which == btard.ALGO_GRAM:
            r, o = btard.centered_clip_verify(g, w.tau, w.zseed, K=w.K, part_len=w.part_len, init_mode=w.init_mode,
                                              v=vbuf, stop_mode=w.stop_mode, max_iters=w.max_iters, eps=w.eps,
                                              algo=which, workspaces=(ws, ws_v),
                                              out=(st.get("c"), st.get("v")) if st else None)
        else:
            r = btard.centered_clip(g, w.tau, part_len=w.part_len, init_mode=w.init_mode, v=vbuf,
                                    stop_mode=w.stop_mode, max_iters=w.max_iters, eps=w.eps, algo=which,
                                    workspace=ws, out=st.get("c"))
            o = btard.verify_projections(g, vbuf, w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                         resid_norm_in=r["resid_norm"], workspace=ws_v, out=st.get("v"))
        st["c"] = {k: r[k] for k in ckeys}
        st["v"] = {k: o[k] for k in vkeys}

    def step():
        aggregate(algo, v, ws_c, state)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    # Timed region: K steps, nothing but the library's own launches on the stream.
    launches0 = btard.kernel_launch_count()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    if dist:
        dist.barrier()
    ms_total = e0.elapsed_time(e1)
    launches = btard.kernel_launch_count() - launches0
    # The same K steps once more with every kernel bracketed by CUDA events on the launching stream
    # (per-kernel durations for the roofline).  Kept apart because an event between two launches
    # stops them from running back to back: with the events the step is 3-15 % slower.
    prof = None
    if not args.no_kernel_events:
        btard.profile_collect()
        btard.profile_enable(True)
        for _ in range(args.steps):
            step()
        torch.cuda.synchronize()
        btard.profile_enable(False)
        prof = btard.profile_collect()
    clocks = sampler.stop() if rank == 0 else None

    iters = state["c"]["iters"].cpu().numpy()
    status = state["c"]["status"].cpu().numpy()
    in_bytes, alg_bytes, passes = algorithmic_bytes(w, iters, gram=(args.algo == "gram"))
    ms_step = ms_total / args.steps
    ms_step = max_over_ranks(ms_step, dist, dev)
    value = whole_job_value(in_bytes, ms_step, world)

    # ---- the other algorithm on the same tensor, for the side-by-side the configurations ask for ---
    other = None
    if args.side_by_side and w.n <= 128:
        other_algo = btard.ALGO_DIRECT if args.algo == "gram" else btard.ALGO_GRAM
        ws_o = torch.empty(btard.centered_clip_workspace(n, P, stride, w.stop_mode, other_algo),
                           dtype=torch.uint8, device=dev)
        v_o = torch.empty((P, stride), dtype=torch.float32, device=dev)
        so = {}

        def other_step():
            aggregate(other_algo, v_o, ws_o, so)
        for _ in range(3):
            other_step()
        torch.cuda.synchronize()
        k3 = max(3, min(args.steps, 10))
        o0, o1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        o0.record()
        for _ in range(k3):
            other_step()
        o1.record()
        torch.cuda.synchronize()
        ms_o = max_over_ranks(o0.elapsed_time(o1) / k3, dist, dev)
        diff = float((v_o - v).norm() / v.norm())
        other = {"algo": "direct" if args.algo == "gram" else "gram", "ms_per_aggregation": ms_o,
                 "rel_l2_difference_of_v": diff}
        del ws_o, v_o

    # ---- end to end: host buffers in, host results out, copies inside the timed region ----------
    e2e = None
    if not args.no_e2e and args.algo != "gram":
        gh = torch.empty(g.shape, dtype=torch.float32, pin_memory=True)
        gh.copy_(g)
        scratch = torch.empty(btard.aggregate_host_scratch(n, P, stride, w.K), dtype=torch.uint8, device=dev)
        hout = None
        copy_stream = torch.cuda.Stream()

        def host_step():
            nonlocal hout
            r = btard.aggregate_host(gh, w.tau, w.zseed, K=w.K, part_len=w.part_len,
                                     init_mode=w.init_mode, stop_mode=w.stop_mode,
                                     max_iters=w.max_iters, eps=w.eps, scratch=scratch, out=hout,
                                     copy_stream=copy_stream)
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
        ms_e2e = (time.perf_counter() - t0) * 1e3 / k2
        ms_e2e = max_over_ranks(ms_e2e, dist, dev)
        d2h = sum(hout[k].numel() * hout[k].element_size() for k in hout)
        e2e = {"value": whole_job_value(in_bytes, ms_e2e, world), "unit": UNIT,
               "ms_per_step": ms_e2e, "h2d_bytes_per_step": gh.numel() * 4, "d2h_bytes_per_step": d2h}
        del gh, scratch

    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel (the CenteredClip iteration pass) -----------------------
    peak, peak_kind = measured_peaks()
    if prof is None:
        prof = {k: (0.0, 0) for k in btard.KERNEL_KINDS}
    iter_ms, iter_launches = prof["iter"]
    per_pass_bytes = n * stride * 4 * (1.0 + 2.0 / n)
    iter_bytes = args.steps * sum(int(i) for i in iters) * per_pass_bytes
    achieved = iter_bytes / (iter_ms * 1e-3) / 1e9 if iter_ms > 0 else None
    kernels = {k: {"ms_per_step": prof[k][0] / args.steps, "launches_per_step": prof[k][1] / args.steps}
               for k in prof}
    ver_ms = prof["verify"][0]
    ver_gbs = args.steps * P * per_pass_bytes / (ver_ms * 1e-3) / 1e9 if ver_ms > 0 else None

    # ---- CPU baseline: the oracle, as it stands, on a bounded sample of the same workload ---------
    cpu_baseline = None
    if not args.no_cpu_baseline:
        import oracle
        cores = oracle.max_threads()
        sample = list(range(0, P, max(1, P // max(1, min(cores, P)))))[:cores]
        gs = g[sample].cpu().numpy()
        t0 = time.perf_counter()
        ref = oracle.centered_clip(gs, w.tau[sample], w.part_len[sample], init_mode=w.init_mode,
                                   stop_mode=w.stop_mode, max_iters=w.max_iters, eps=w.eps)
        oracle.verify(gs, ref["v"].astype(np.float32), w.tau[sample], w.zseed, K=w.K,
                      part_len=w.part_len[sample], norm_in=ref["resid_norm"])
        dt = time.perf_counter() - t0
        cb, _, _ = algorithmic_bytes(w, ref["iters"])
        cpu_baseline = {"value": cb / dt / 1e9, "unit": UNIT, "cores": min(cores, len(sample)),
                        "kind": "oracle", "seconds": dt,
                        "sample": "partitions %s of config %d, full iteration count + verification"
                                  % (sample, args.config)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": "config %d: n=%d peers, d=%d, P=%d partitions, row_stride=%d" %
                               (args.config, w.n, w.d, w.P, w.row_stride),
                   "algo": args.algo, "init": "coordinate median", "stop": "eps" if w.stop_mode else "fixed",
                   "max_iters": w.max_iters, "eps": w.eps, "K": w.K,
                   "iters_per_partition": [int(i) for i in iters],
                   "not_converged_partitions": int((status & 1).sum()),
                   "passes_counted": ("1 Gram + 1 combine-and-verify per partition" if args.algo == "gram"
                                      else "1 init + iters + 1 verify per partition"),
                   "l2": "input (%.0f MB) larger than L2 (126 MB), no flush" % (g.numel() * 4 / 1e6),
                   "kernel_events": "per-kernel durations come from a second run of the same K steps",
                   "multi_gpu": "replicas only" if world > 1 else "single GPU"},
        "fraction_of_hbm_peak": value / world / peak, "hbm_peak_gbs": peak, "hbm_peak_kind": peak_kind,
        "gpu_launches": int(launches),
        "clocks": clocks,
        "e2e": e2e,
        "roofline": {"kernel": "cclip_pass_kernel<ITER>", "bound": "hbm", "achieved": achieved,
                     "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                     "frac": achieved / peak if achieved else None,
                     "traffic": ITER_TRAFFIC.get((args.config, args.algo)),
                     "launches": iter_launches, "avg_launch_ms": iter_ms / max(1, iter_launches),
                     "algorithmic_bytes_per_launch": per_pass_bytes * P,
                     "verify_kernel_gbs": ver_gbs},
        "kernels": kernels,
        "ms_per_aggregation": ms_step,
        "other_algorithm": other,
        "cpu_baseline": cpu_baseline,
    }
    print(json.dumps(line))
    if dist:
        dist.destroy_process_group()


def run_reference(args):
    """The reference arm is the float64 oracle on the host cores: each step aggregates a bounded
    sample of the same workload (one partition per core)."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    import oracle
    import workloads

    cores = oracle.max_threads()
    wmeta = workloads.make_workload(args.config, data=False)
    P = wmeta.P
    sample = list(range(0, P, max(1, P // max(1, min(cores, P)))))[:cores]
    w = workloads.make_workload(args.config, device="cpu", partitions=sample)
    if args.max_iters:
        w.max_iters = args.max_iters
    g = w.g.numpy()
    iters = None

    def step():
        nonlocal iters
        ref = oracle.centered_clip(g, w.tau, w.part_len, init_mode=w.init_mode, stop_mode=w.stop_mode,
                                   max_iters=w.max_iters, eps=w.eps)
        oracle.verify(g, ref["v"].astype(np.float32), w.tau, w.zseed, K=w.K, part_len=w.part_len,
                      norm_in=ref["resid_norm"])
        iters = ref["iters"]
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / args.steps
    in_bytes, _, _ = algorithmic_bytes(w, iters)
    value = in_bytes / dt / 1e9
    sample_txt = "partitions %s of config %d per step, full iteration count + verification" % (sample, args.config)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT,
        "n_gpus": int(os.environ.get("WORLD_SIZE", "1")), "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "config %d: n=%d peers, d=%d, P=%d partitions, row_stride=%d" %
                               (args.config, w.n, w.d, wmeta.P, w.row_stride), "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": min(cores, len(sample)),
                         "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", type=int, default=2)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--algo", default="direct", choices=["direct", "gram", "cooperative", "resident", "staged"])
    ap.add_argument("--max-iters", type=int, default=None, help="override the configuration's iteration cap")
    ap.add_argument("--no-kernel-events", action="store_true",
                    help="do not bracket the library's kernels with CUDA events (no roofline object)")
    ap.add_argument("--no-side-by-side", dest="side_by_side", action="store_false",
                    help="do not also time the other algorithm (direct / Gram) on the same tensor")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
