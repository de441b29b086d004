#!/usr/bin/env python
"""Benchmark of the Accordion gradient-compression step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 5] [--impl reference]

One "step" is one pass of the whole hot path over one batch of synthetic worker gradients: the
PowerSGD step and the TopK step of the workload (each with its own error memory, both with error
feedback, the first also accumulating the detector's gradient), plus -- every `check_every` steps --
the layer norms and the regime test that sets the per-layer levels for the following steps.

metric = GB/s of gradient processed: each compressor pass consumes the W workers' gradients once, so a
step processes (number of compressors) x 4 x W x N bytes.  Prints ONE JSON line (rank 0).
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

import numpy as np  # noqa: E402
import torch  # noqa: E402

METRIC = "compression_step_gradient_throughput"
UNIT = "GB/s"
RING = 4  # pre-generated gradient batches cycled through the steps (each far larger than L2)
NOMINAL_HBM_GBS = 8000.0     # the B200's nominal HBM3e bandwidth, the figure the target of this path is stated against
SAMPLE_PARAM_WORKERS = 26e6  # size of the oracle's sample of the workload (parameter-workers per step)


def _peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json hbm_gbs)"
    return 6650.0, "fallback (6.65 TB/s, no MEASURED_PEAKS.json)"


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=2)
        except Exception:
            pass
        rows = [l for (t, l) in self.lines if t0 <= t <= t1 + 0.15] or [l for (_, l) in self.lines]
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(power)) if power else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def _kernel_alg_bytes(name, units, n_workers=None, carries_delta=()):
    """Algorithmic bytes one launch of a streaming kernel must move (fp32), for `units` MATRIX parameter-workers:
    the reads and writes the method itself requires of that pass.  The first pass of a compressor reads g and e and
    writes M (12 B per unit); the one that also accumulates the detector's gradient (the first compressor of the
    step) reads and writes delta for one worker in W (8/W B per unit more).  The selection passes work on the
    subsets their work lists name, so no per-launch figure is given for them."""
    per_unit = {
        "psgd_project_kernel": 12.0,    # read g, read e, write M
        "psgd_residual_kernel": 8.0,    # read M, write e' (eager mode; in lazy mode it only writes out)
        "topk_ef_hist1_kernel": 12.0,   # read g, read e, write M
        "ef_kernel": 12.0,
    }
    b = per_unit.get(name, 0.0)
    if b and name in carries_delta and n_workers:
        b += 8.0 / n_workers
    return b * units


def oracle_sample(w, device):
    """A bounded sample of workload ``w`` for the CPU oracle: every layer cut to its first rows (1/s of them, s the
    smallest power of two that brings W x parameters under SAMPLE_PARAM_WORKERS), filled from the workload's own
    gradient stream (iterations 0 and 1, the values the GPU arm sees), so the sample keeps the layer mix, the value
    distributions and the row-sparse encoder of the full set.  Returns (sub-table, layer tuples, batches, text)."""
    from paper_2010_16248_b200 import workloads as wl
    full, W = w.table, w.n_workers
    s = 1
    while W * full.n_params / s > SAMPLE_PARAM_WORKERS:
        s *= 2
    shapes = []
    for l in range(full.n_layers):
        n, m = int(full.rows[l]), int(full.cols[l])
        if full.kind[l] == wl.MATRIX:
            shapes.append((full.names[l], (max(min(n, 4), -(-n // s)), m)))
        else:
            shapes.append((full.names[l], (max(1, m // s),)))
    sub = wl.make_table(shapes)
    gen = wl.GradientStream(w, device=device)
    batches = []
    for t in range(2):
        g = gen.grads(t)
        b = np.zeros((W, sub.stride), np.float32)
        for l in range(sub.n_layers):
            size = int(sub.rows[l]) * int(sub.cols[l])
            o_full, o_sub = int(full.offset[l]), int(sub.offset[l])
            b[:, o_sub:o_sub + size] = g[:, o_full:o_full + size].cpu().numpy()
        batches.append(b)
        del g
    cut = "every layer whole" if s == 1 else f"the first 1/{s} of the rows of every layer"
    text = (f"{w.name}: {cut} ({sub.n_params} of {full.n_params} parameters, all {W} workers, a row-sparse layer "
            f"included where the set has one), gradients of iterations 0 and 1 of the workload's own stream, every "
            f"compressor of the workload per step")
    return sub, batches, text


def run_reference(args, rank, world):
    """Times the CPU oracle, as it stands, on a bounded sample of the workload (see ``oracle_sample``): with the
    host's default thread pool for the K timed steps, and single-threaded on a few more.  The oracle's products
    run in the BLAS pool; its sort (the TopK half) is one thread whatever the pool size."""
    if rank != 0:
        return
    from oracle import accordion_oracle as orc
    from paper_2010_16248_b200 import workloads as wl
    w = wl.workload(args.config)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    sub, batches, sample = oracle_sample(w, dev)
    layers = [(int(sub.offset[l]), int(sub.rows[l]), int(sub.cols[l]), int(sub.kind[l])) for l in range(sub.n_layers)]
    W = w.n_workers
    q0 = [None if x is None else x.numpy() for x in wl.initial_q(sub, w.rank_low)]
    state = {}

    def reset():
        state.update(err_p=np.zeros((W, sub.stride), np.float32), err_t=np.zeros((W, sub.stride), np.float32),
                     q=[None if x is None else x.copy() for x in q0], level=np.ones(sub.n_layers, np.uint8),
                     delta=np.zeros(sub.stride), prev=-np.ones(sub.n_layers))

    def step(t):
        g = batches[t % 2]
        orc.accumulate(state["delta"], g[0], layers)
        n_comp = 0
        if "powersgd" in w.compressors:
            _, e, qn, _ = orc.powersgd_step(g, state["err_p"], state["q"], state["level"], layers, w.rank_low,
                                            w.rank_high)
            state["err_p"] = e.astype(np.float32)
            state["q"] = [None if x is None else x.astype(np.float32) for x in qn]
            n_comp += 1
        if "topk" in w.compressors:
            _, _, _, _, state["err_t"] = orc.topk_step(g, state["err_t"], state["level"], layers, w.topk_low_bp,
                                                       w.topk_high_bp)
            n_comp += 1
        if (t + 1) % w.check_every == 0:
            state["level"], state["prev"] = orc.detect_regime(orc.layer_norms2(state["delta"], layers), state["prev"],
                                                              0.1, 0.1, w.eta)
            state["delta"][:] = 0
        return n_comp

    def timed(k, warm):
        reset()
        for t in range(warm):
            step(t)
        t0 = time.perf_counter()
        n = 0
        for t in range(k):
            n = step(warm + t)
        dt = time.perf_counter() - t0
        return n * 4.0 * W * sub.n_params * k / dt / 1e9, dt / k * 1e3

    value, ms = timed(args.steps, args.warmup)
    cores, value_1 = 1, None
    try:
        from threadpoolctl import threadpool_info, threadpool_limits
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
        with threadpool_limits(limits=1):
            value_1, _ = timed(min(2, args.steps), 1)
    except Exception:
        pass
    cpu = {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
           "value_single_thread": value_1,
           "threads": f"{cores} BLAS threads for the oracle's matrix products; its sort (TopK) runs on one thread"}
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "sample": sample},
            "cpu_baseline": cpu,
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def cpu_baseline(w):
    """The oracle timed on the host cores on a bounded sample of the workload (the --impl reference leg, 3 steps)."""
    ns = argparse.Namespace(config=w.config_id, warmup=1, steps=3, gpus=1)
    import io
    from contextlib import redirect_stdout
    buf = io.StringIO()
    with redirect_stdout(buf):
        run_reference(ns, 0, 1)
    return json.loads(buf.getvalue().strip().splitlines()[-1])["cpu_baseline"]


def respawn_under_torchrun(n):
    """``--gpus N`` given to a plain ``python bench.py``: start N ranks, one per GPU, under torch.distributed.run
    on this node, with the same arguments, and hand their output and exit code through."""
    import socket
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.abspath(__file__)] + sys.argv[1:]
    return subprocess.call(cmd)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=5, help="benchmark configuration 1..5 (default: 5, the largest gradient set)")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--eager", action="store_true", help="PowerSGD: materialise the error memory every step")
    ap.add_argument("--no-graphs", action="store_true", help="issue the timed steps call by call instead of as CUDA graphs")
    ap.add_argument("--pipeline", default="auto", choices=["auto", "always", "never"],
                    help="first PowerSGD pass: persistent bulk-copy pipeline, direct kernel, or the library's choice")
    ap.add_argument("--share-sms", action="store_true",
                    help="two compressors: the pipelined first PowerSGD pass takes half of the SMs, the TopK step's "
                         "kernels run beside it (faster step, slower kernel; off by default so that the roofline "
                         "entry times the kernel on the whole GPU)")
    ap.add_argument("--no-overlap", action="store_true",
                    help="two-compressor configs: run the TopK step after the PowerSGD step instead of beside it")
    ap.add_argument("--sgd-tail", action="store_true",
                    help="single-compressor configs: apply the Nesterov update inside the step (fused optimiser tail)")
    ap.add_argument("--batch-mode", action="store_true",
                    help="batch-size mode instead of compression: a step is n_accum micro-batch accumulations, the "
                         "uncompressed average with the fused Nesterov update, and (every check_every steps) the "
                         "whole-model detector")
    ap.add_argument("--real-workers", action="store_true",
                    help="every GPU holds the config's W workers and the compressed factors are exchanged between "
                         "GPUs (all-reduce of P and Q, all-gather of the packed TopK sets) instead of independent "
                         "replicas; at --gpus 1 the collectives are the identity")
    ap.add_argument("--groups", type=int, default=1,
                    help="--real-workers: layer groups whose exchanges run on a communication stream beside the next "
                         "group's first pass")
    ap.add_argument("--n-accum", type=int, default=8, help="--batch-mode: micro-batches per step (B_high / micro-batch)")
    ap.add_argument("--force-level", default="auto", choices=["auto", "low", "high"],
                    help="auto: the detector sets the per-layer levels (the method as it runs); low / high: every "
                         "layer held at that compression level for the whole run (the detector still runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup

    if args.impl == "reference":  # the oracle on the host cores: rank 0 alone works, whatever N
        run_reference(args, int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")))
        return
    if "WORLD_SIZE" not in os.environ and args.gpus > 1:
        sys.exit(respawn_under_torchrun(args.gpus))
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world != max(args.gpus, 1):
        raise SystemExit(f"--gpus {args.gpus} but the launcher started {world} rank(s)")

    import torch.distributed as dist
    from paper_2010_16248_b200 import build, dist_util, pipeline, workloads as wl
    if rank == 0:
        build.build_library()
    assert torch.cuda.is_available(), "bench.py needs a CUDA device (there is no CPU path)"
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)
        dist.barrier()

    w = wl.workload(args.config)
    table, W = w.table, w.n_workers
    n_comp = len(w.compressors)
    stream_gen = wl.GradientStream(w, device=dev)
    # independent replicas: every rank draws its own gradient batches
    ring = [stream_gen.grads(dist_util.replica_seed_offset(rank) + t) for t in range(RING)]
    if args.batch_mode:
        run_batch_mode(args, w, ring, dev, rank, world, local_rank)
        return
    if args.real_workers:
        run_real_workers(args, w, ring, dev, rank, world, local_rank)
        return
    optimizer = None
    if args.sgd_tail:
        assert n_comp == 1, "--sgd-tail needs a single-compressor config (2, 3 or 4)"
        optimizer = {"params": torch.zeros(table.stride, device=dev), "lr": 0.1, "momentum": 0.9}
    eng = pipeline.AccordionStep(table, W, w.compressors, w.rank_low, w.rank_high, w.topk_low_bp, w.topk_high_bp,
                                 w.eta, 1e-8, w.check_every, device=dev, lazy_residual=not args.eager,
                                 optimizer=optimizer, extra_flags={"auto": 0, "always": 2, "never": 4}[args.pipeline],
                                 overlap=not args.no_overlap, share_sms=args.share_sms)
    n_mat = table.n_matrix_params
    grad_bytes_step = n_comp * 4.0 * W * table.n_params

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    step_no = 0

    use_graphs = not args.no_graphs
    force = {"auto": None, "low": 1, "high": 0}[args.force_level]
    if force is not None:
        eng.level.fill_(force)
    # the per-layer levels in force during each step, for the per-regime report: the array only changes at a regime
    # check, so a copy is kept (device to device, read back after the timed region) whenever one has run
    level_log = torch.zeros(args.steps // max(w.check_every, 1) + 2, table.n_layers, dtype=torch.uint8, device=dev)
    level_from = []  # (first timed step a logged row applies to, row)

    def run_steps(k, events=None, graphs=False, log=False):
        nonlocal step_no
        if log:
            level_log[0].copy_(eng.level)
            level_from.append((0, 0))
        for i in range(k):
            if events is not None:
                events[i][0].record()
            if graphs:
                eng.step_graph(step_no % RING)
            else:
                eng.step(ring[step_no % RING])
            if events is not None:
                events[i][1].record()
            step_no += 1
            if eng.t % w.check_every == 0:
                if force is not None:
                    eng.level.fill_(force)
                if log:
                    level_log[len(level_from)].copy_(eng.level)
                    level_from.append((i + 1, len(level_from)))

    # ---- warm-up, then the timed region (device-resident inputs)
    run_steps(args.warmup)
    barrier()
    if use_graphs:  # one CUDA graph per gradient buffer and per kind of iteration (with / without regime check)
        eng.capture_graphs(ring)
    K = args.steps
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(K)]
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    barrier()
    launches0 = eng.launches
    t0 = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    run_steps(K, ev, graphs=use_graphs, log=True)
    stop.record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    total_ms = start.elapsed_time(stop)
    gpu_launches = eng.launches - launches0
    per_step = np.array([a.elapsed_time(b) for a, b in ev])
    # regime of every timed step: share of the MATRIX parameters whose layer was at the low compression level
    log_host = level_log.cpu().numpy()
    mat = table.kind == wl.MATRIX
    weight = table.sizes[mat] / table.sizes[mat].sum()
    regime = []
    for i in range(K):
        row = [r for (first, r) in level_from if first <= i][-1]
        share = float((log_host[row][mat] * weight).sum())
        regime.append("low" if share > 1 - 1e-9 else "high" if share < 1e-9 else "mixed")
    total_ms = dist_util.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / K
    value = dist_util.whole_job_throughput(grad_bytes_step, ms_per_step, world) / 1e9

    # ---- same K steps again with per-kernel CUDA events (on the launching stream) for the roofline
    # (the two compressors one after the other here, so that a kernel's events bracket that kernel alone)
    overlap, eng.overlap = eng.overlap, False
    eng.ctx.acc_profile_enable(True)
    run_steps(K)
    torch.cuda.synchronize()
    prof = eng.ctx.acc_profile_read()
    eng.ctx.acc_profile_enable(False)
    eng.overlap = overlap
    peak, peak_src = _peaks()
    units = W * n_mat
    compulsory = n_comp * 12.0 * units  # bytes a step must move: read g, read e, write e', per compressor

    def step_fracs(ms):
        gbs = compulsory / (ms * 1e-3) / 1e9
        return {"of_measured_copy_peak": round(gbs / peak, 4), "of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4)}

    by_regime = {}
    # the stored per-step traffic belongs to the default path (lazy residual, no optimiser tail, the library's choice
    # of first PowerSGD pass, the config's own worker count)
    default_path = not (args.eager or args.sgd_tail or args.share_sms or args.pipeline != "auto")
    for name in ("low", "high", "mixed"):
        ts = per_step[[r == name for r in regime]]
        if len(ts):
            by_regime[name] = {"steps": int(len(ts)), "median_ms": round(float(np.median(ts)), 4),
                               "min_ms": round(float(ts.min()), 4), "max_ms": round(float(ts.max()), 4),
                               "gradient_gbs": round(grad_bytes_step / (float(np.median(ts)) * 1e-3) / 1e9, 1),
                               "frac_of_12B": step_fracs(float(np.median(ts)))}
            # achieved DRAM throughput of the whole step: the bytes ncu counted for one step of this config and level
            # (every kernel of the step, one-pass capture) over this run's median step time
            traffic = STEP_TRAFFIC.get((args.config, name)) if default_path else None
            if traffic:
                gbs = traffic / (float(np.median(ts)) * 1e-3) / 1e9
                by_regime[name]["dram"] = {"bytes_per_step_ncu": traffic, "gbs": round(gbs, 1),
                                           "frac_of_measured_copy_peak": round(gbs / peak, 4),
                                           "frac_of_nominal_8TBs": round(gbs / NOMINAL_HBM_GBS, 4)}
    total_k_ms = sum(ms for ms, _ in prof.values())
    kernels = {}
    # the first compressor of the step carries the detector's accumulation in its first pass
    carries = ("psgd_project_kernel",) if "powersgd" in w.compressors else ("topk_ef_hist1_kernel",)
    for name, (ms, cnt) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
        alg = _kernel_alg_bytes(name, units)
        if name == "psgd_residual_kernel" and not args.eager:
            alg = 0.0  # lazy mode: this slot times the decompress kernel, which only writes out (4/W B per unit)
        avg = ms / cnt
        kernels[name] = {"launches": cnt, "ms_total": round(ms, 4), "share": round(ms / total_k_ms, 4),
                         "avg_ms": round(avg, 5),
                         "alg_gbs": round(alg / (avg * 1e-3) / 1e9, 1) if alg else None}
    dom = next(iter(kernels))
    dom_alg = _kernel_alg_bytes(dom, units)  # 12 B per unit: the fraction is reported against the compulsory bytes
    dom_alg_delta = _kernel_alg_bytes(dom, units, W, carries)  # ... and with the detector's accumulation counted
    dom_avg_ms = prof[dom][0] / prof[dom][1]
    achieved = dom_alg / (dom_avg_ms * 1e-3) / 1e9
    tkey = traffic_key(dom, args, table, W, torch.cuda.get_device_properties(dev).multi_processor_count)
    if default_path and (args.config, tkey) in TRAFFIC_PER_LAUNCH:
        traffic, traffic_src = TRAFFIC_PER_LAUNCH[(args.config, tkey)], "ncu one-pass launch list on this config"
    elif tkey in TRAFFIC_PER_UNIT:
        traffic, traffic_src = TRAFFIC_PER_UNIT[tkey] * units, TRAFFIC_SOURCE.get(tkey)
    else:
        traffic, traffic_src = None, None
    roofline = {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "peak_source": peak_src,
                "peak_nominal": NOMINAL_HBM_GBS, "frac_of_nominal": round(achieved / NOMINAL_HBM_GBS, 4),
                "traffic": traffic,
                "traffic_source": traffic_src,
                "traffic_over_algorithmic": round(traffic / dom_alg, 3) if traffic and dom_alg else None,
                "alg_bytes_per_launch": dom_alg, "alg_bytes_per_unit": round(dom_alg / units, 3),
                "frac_with_detector_bytes": round(dom_alg_delta / (dom_avg_ms * 1e-3) / 1e9 / peak, 4),
                "step_frac_of_12B": step_fracs(ms_per_step)["of_measured_copy_peak"],
                "step_frac_of_12B_nominal": step_fracs(ms_per_step)["of_nominal_8TBs"]}

    # ---- end to end: host (pinned) gradients -> device every step, results read back to the host.
    # Uploads run on a copy stream into two staging buffers and overlap the previous step's kernels.
    ke = max(1, min(args.e2e_steps, K))
    host = [torch.empty(W, table.stride, dtype=torch.float32).pin_memory() for _ in range(2)]
    for i in range(2):
        host[i].copy_(ring[i])
    fed = pipeline.HostFedStep(eng)
    fed.step(host[0])
    fed.synchronize()
    barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for i in range(ke):
        fed.step(host[(i + 1) % 2])
    torch.cuda.current_stream().wait_event(fed.downloaded)
    e2.record()
    fed.synchronize()
    barrier()
    e2e_ms = s2.elapsed_time(e2)
    e2e_ms = dist_util.max_over_ranks(e2e_ms, dev)
    e2e = {"value": dist_util.whole_job_throughput(grad_bytes_step, e2e_ms / ke, world) / 1e9, "unit": UNIT, "steps": ke,
           "ms_per_step": e2e_ms / ke, "h2d_bytes_per_step": int(fed.h2d_bytes_per_step),
           "d2h_bytes_per_step": int(fed.d2h_bytes_per_step),
           "note": "pinned host gradients uploaded every step (copy stream, double-buffered), outputs downloaded"}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(w)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name, "n_workers": W, "params": table.n_params,
                           "compressors": list(w.compressors), "rank_low_high": [w.rank_low, w.rank_high],
                           "topk_bp_low_high": [w.topk_low_bp, w.topk_high_bp], "check_every": w.check_every,
                           "powersgd_residual": "eager" if args.eager else "lazy (applied on the next load)",
                           "optimizer_tail": "Nesterov update fused into the step" if args.sgd_tail else "none",
                           "gradient_bytes_per_step": grad_bytes_step,
                           "l2_policy": f"inputs larger than L2: {RING} gradient batches of "
                                        f"{4 * W * table.stride / 1e6:.0f} MB cycled, no flush",
                           "launch": "CUDA graph replay per step" if use_graphs else "direct calls",
                           "levels": ("set by the detector" if force is None else
                                      f"every layer held at the {args.force_level} compression level"),
                           "regime_of_value": ", ".join(f"{v['steps']} of {K} timed steps at {k}"
                                                        for k, v in by_regime.items()),
                           "streams": (("TopK step beside the PowerSGD step on a second stream" +
                                        ("; pipelined first PowerSGD pass on half of the SMs" if args.share_sms
                                         else ""))
                                       if (n_comp == 2 and not args.no_overlap) else "one stream"),
                           "multi_gpu": "independent replicas, no collective"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches,
                "roofline": roofline, "cpu_baseline": cpu,
                "step_ms": {"median": float(np.median(per_step)), "min": float(per_step.min()),
                            "max": float(per_step.max())},
                "step_ms_by_regime": by_regime,
                "kernels": kernels}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_batch_mode(args, w, ring, dev, rank, world, local_rank):
    """Batch-size mode on the workload's layer table: a step = n_accum accumulations of [W, N] micro-batch
    gradients, one average over workers fused with the Nesterov update, and the whole-model detector every
    check_every steps.  Same timing rules and JSON keys as the compression bench."""
    import torch.distributed as dist
    from paper_2010_16248_b200 import dist_util, pipeline
    table, W, n_accum = w.table, w.n_workers, args.n_accum
    params = torch.zeros(table.stride, device=dev)
    bs = pipeline.BatchSizeStep(table, W, b_low=512, b_high=512 * n_accum, micro_batch=512, eta=w.eta, device=dev,
                                optimizer={"params": params, "lr": 0.1, "momentum": 0.9})
    grad_bytes_step = 4.0 * W * table.n_params * n_accum
    step_no = 0

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step():
        nonlocal step_no
        n = 0
        for j in range(n_accum):
            bs.micro_step(ring[(step_no * n_accum + j) % RING])
            n += bs.ctx.last_launch_count()
        bs.apply()
        n += bs.ctx.last_launch_count()
        step_no += 1
        if step_no % w.check_every == 0:
            bs.ctx.acc_layer_norms(bs.delta, 1, bs.norm2_layers)
            n += bs.ctx.last_launch_count()
            bs.ctx.acc_detect_batch(bs.norm2_layers, bs.norm2_prev, 0.1, 0.1, bs.b_low, bs.b_high, bs.batch,
                                    bs.lr_scale, bs.delta)
            n += bs.ctx.last_launch_count()
        return n

    for _ in range(args.warmup):
        one_step()
    barrier()
    K = args.steps
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    barrier()
    t0 = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    gpu_launches = sum(one_step() for _ in range(K))
    stop.record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    ms_per_step = dist_util.max_over_ranks(start.elapsed_time(stop), dev) / K
    value = dist_util.whole_job_throughput(grad_bytes_step, ms_per_step, world) / 1e9

    bs.ctx.acc_profile_enable(True)
    for _ in range(K):
        one_step()
    torch.cuda.synchronize()
    prof = bs.ctx.acc_profile_read()
    bs.ctx.acc_profile_enable(False)
    peak, peak_src = _peaks()
    # algorithmic bytes per launch: accumulate reads g and acc and writes acc for every worker (the first
    # micro-batch of a step skips the read of acc), plus the decider's read-modify-write of delta;
    # average reads W accumulators, writes out, and reads + writes params and momentum
    n = table.n_params
    alg = {"batch_accumulate_kernel": (12.0 * W - 4.0 * W / n_accum + 8.0) * n,
           "batch_average_kernel": (4.0 * W + 4.0 + 16.0) * n}
    total_k_ms = sum(ms for ms, _ in prof.values())
    kernels = {}
    for name, (ms, cnt) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
        avg = ms / cnt
        a = alg.get(name)
        kernels[name] = {"launches": cnt, "ms_total": round(ms, 4), "share": round(ms / total_k_ms, 4),
                         "avg_ms": round(avg, 5), "alg_gbs": round(a / (avg * 1e-3) / 1e9, 1) if a else None}
    dom = next(iter(kernels))
    achieved = alg[dom] / (prof[dom][0] / prof[dom][1] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "peak_source": peak_src, "traffic": None,
                "alg_bytes_per_launch": alg[dom]}

    # end to end: each micro-batch uploaded from pinned host memory (copy stream, two staging buffers); the
    # step's result (the updated parameters) read back to the host
    ke = max(1, min(args.e2e_steps, K))
    host = [torch.empty(W, table.stride, dtype=torch.float32).pin_memory() for _ in range(2)]
    for i in range(2):
        host[i].copy_(ring[i])
    stage = [torch.empty(W, table.stride, device=dev) for _ in range(2)]
    params_host = torch.empty(table.stride, dtype=torch.float32).pin_memory()
    copy = torch.cuda.Stream(device=dev)
    up = [torch.cuda.Event() for _ in range(2)]
    used = [torch.cuda.Event() for _ in range(2)]
    main = torch.cuda.current_stream(dev)
    barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    i = 0
    for _ in range(ke):
        for j in range(n_accum):
            b = i & 1
            with torch.cuda.stream(copy):
                if i >= 2:
                    copy.wait_event(used[b])
                stage[b].copy_(host[b], non_blocking=True)
                up[b].record(copy)
            main.wait_event(up[b])
            bs.micro_step(stage[b])
            used[b].record(main)
            i += 1
        bs.apply()
        params_host.copy_(params, non_blocking=True)
    e2.record()
    barrier()
    e2e_ms = dist_util.max_over_ranks(s2.elapsed_time(e2), dev)
    e2e = {"value": dist_util.whole_job_throughput(grad_bytes_step, e2e_ms / ke, world) / 1e9, "unit": UNIT,
           "steps": ke, "ms_per_step": e2e_ms / ke, "h2d_bytes_per_step": int(4 * W * table.stride * n_accum),
           "d2h_bytes_per_step": int(4 * table.stride)}
    if rank == 0:
        line = {"metric": "batch_mode_gradient_throughput", "value": value, "unit": UNIT, "n_gpus": world, "steps": K,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name + " layer table, batch-size mode", "n_workers": W,
                           "params": table.n_params, "n_accum": n_accum, "check_every": w.check_every,
                           "optimizer_tail": "Nesterov update fused into the average",
                           "gradient_bytes_per_step": grad_bytes_step,
                           "l2_policy": f"inputs larger than L2: {RING} gradient batches cycled, no flush",
                           "multi_gpu": "independent replicas, no collective"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "roofline": roofline,
                "cpu_baseline": None, "kernels": kernels}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


def run_real_workers(args, w, ring, dev, rank, world, local_rank):
    """The step with the factors exchanged between GPUs: W workers per GPU (weak scaling: N*W workers in all), one
    pipeline.DistributedStep per compressor of the workload.  Same timing rules and JSON keys."""
    import torch.distributed as dist
    from paper_2010_16248_b200 import dist_util, pipeline
    table, W = w.table, w.n_workers
    engines = [pipeline.DistributedStep(table, W, comp, w.rank_low, w.rank_high, w.topk_low_bp, w.topk_high_bp, w.eta,
                                        1e-8, w.check_every, device=dev, lazy_residual=not args.eager,
                                        groups=args.groups)
               for comp in w.compressors]
    n_comp = len(engines)
    grad_bytes_step = n_comp * 4.0 * W * table.n_params
    step_no = 0

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def one_step(g):
        nonlocal step_no
        for e in engines:
            e.step(g)
        step_no += 1

    for _ in range(args.warmup):
        one_step(ring[step_no % RING])
    barrier()
    K = args.steps
    sampler = ClockSampler(local_rank) if rank == 0 else None
    if sampler:
        sampler.start()
        time.sleep(0.25)
    barrier()
    t0 = time.time()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for _ in range(K):
        one_step(ring[step_no % RING])
    stop.record()
    barrier()
    t1 = time.time()
    clocks = sampler.stop(t0, t1) if sampler else None
    ms_per_step = dist_util.max_over_ranks(start.elapsed_time(stop), dev) / K
    value = dist_util.whole_job_throughput(grad_bytes_step, ms_per_step, world) / 1e9

    contexts = list({id(c): c for e in engines for c in [p.ctx for p in e.parts] + [e.ctx]}.values())
    for c in contexts:
        c.acc_profile_enable(True)
    for _ in range(K):
        one_step(ring[step_no % RING])
    torch.cuda.synchronize()
    prof = {}
    for c in contexts:
        for name, (ms, cnt) in c.acc_profile_read().items():
            a = prof.get(name, (0.0, 0))
            prof[name] = (a[0] + ms, a[1] + cnt)
        c.acc_profile_enable(False)
    gpu_launches = sum(cnt for _, cnt in prof.values())  # the profiled pass repeats the timed pass launch for launch
    peak, peak_src = _peaks()
    units = W * table.n_matrix_params
    total_k_ms = sum(ms for ms, _ in prof.values())
    kernels = {}
    for name, (ms, cnt) in sorted(prof.items(), key=lambda kv: -kv[1][0]):
        alg = _kernel_alg_bytes(name, units)
        avg = ms / cnt
        kernels[name] = {"launches": cnt, "ms_total": round(ms, 4), "share": round(ms / total_k_ms, 4),
                         "avg_ms": round(avg, 5), "alg_gbs": round(alg / (avg * 1e-3) / 1e9, 1) if alg else None}
    dom = next(iter(kernels))
    dom_alg = _kernel_alg_bytes(dom, units)
    achieved = dom_alg / (prof[dom][0] / prof[dom][1] * 1e-3) / 1e9
    roofline = {"bound": "hbm", "kernel": dom, "achieved": round(achieved, 1), "peak": peak, "unit": "GB/s",
                "frac": round(achieved / peak, 4), "peak_source": peak_src,
                "traffic": (TRAFFIC_PER_UNIT[dom] * units if dom in TRAFFIC_PER_UNIT else None),
                "alg_bytes_per_launch": dom_alg}

    ke = max(1, min(args.e2e_steps, K))
    host = [torch.empty(W, table.stride, dtype=torch.float32).pin_memory() for _ in range(2)]
    for i in range(2):
        host[i].copy_(ring[i])
    stage = [torch.empty(W, table.stride, device=dev) for _ in range(2)]
    outs_host = [torch.empty(table.stride, dtype=torch.float32).pin_memory() for _ in engines]
    barrier()
    s2, e2 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    s2.record()
    for i in range(ke):
        stage[i & 1].copy_(host[i & 1], non_blocking=True)
        one_step(stage[i & 1])
        for oh, e in zip(outs_host, engines):
            oh.copy_(e.out, non_blocking=True)
    e2.record()
    barrier()
    e2e_ms = dist_util.max_over_ranks(s2.elapsed_time(e2), dev)
    e2e = {"value": dist_util.whole_job_throughput(grad_bytes_step, e2e_ms / ke, world) / 1e9, "unit": UNIT,
           "steps": ke, "ms_per_step": e2e_ms / ke, "h2d_bytes_per_step": int(4 * W * table.stride),
           "d2h_bytes_per_step": int(4 * table.stride * n_comp)}
    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": args.warmup,
                "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
                "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name + ", real workers", "workers_per_gpu": W, "workers_total": W * world,
                           "params": table.n_params, "compressors": list(w.compressors),
                           "gradient_bytes_per_step": grad_bytes_step,
                           "exchange_bytes_per_step_per_gpu": sum(e.bytes_exchanged_per_step() for e in engines),
                           "l2_policy": f"inputs larger than L2: {RING} gradient batches cycled, no flush",
                           "launch": "direct calls (collectives between the phases)",
                           "layer_groups": args.groups,
                           "multi_gpu": "NCCL all-reduce of the PowerSGD factors, all-gather of the packed TopK sets"},
                "clocks": clocks, "e2e": e2e, "gpu_launches": gpu_launches, "roofline": roofline,
                "cpu_baseline": None, "kernels": kernels}
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) per MATRIX parameter-worker, from the ncu captures
# summarised under profiles/; a launch's traffic is this figure times the units it processes (the kernels
# stream every element once, so traffic grows in proportion).
TRAFFIC_PER_UNIT = {"psgd_project_kernel": 13.15, "psgd_project_kernel/pipelined": 13.21, "topk_ef_hist1_kernel": 12.95}
# The same two counters per launch, taken on the benchmark configs themselves where a one-pass launch list could be
# (nothing is saved and restored around a single pass, so the full-size workloads are captured as they are);
# these come first, the per-unit figures serve the other cases (forced implementations, other worker counts).
TRAFFIC_PER_LAUNCH = {(5, "psgd_project_kernel/pipelined"): 5360.7e6, (5, "topk_ef_hist1_kernel"): 4850.1e6,
                      (4, "psgd_project_kernel"): 2165.8e6, (2, "psgd_project_kernel"): 614.1e6,
                      (3, "topk_ef_hist1_kernel"): 573.8e6}
TRAFFIC_SOURCE = {"psgd_project_kernel": "ncu capture of the direct kernel on config 4, scaled by units",
                  "psgd_project_kernel/pipelined": "ncu capture of the pipelined kernel on config 4, scaled by units",
                  "topk_ef_hist1_kernel": "ncu capture on config 3, scaled by units"}
# DRAM bytes of one whole steady-state step (all kernels; same counters, one-pass launch list) by (config, level)
STEP_TRAFFIC = {(5, "high"): 11467.8e6, (5, "low"): 12900.3e6, (4, "high"): 2280.9e6, (4, "low"): 2281.0e6,
                (3, "high"): 603.6e6, (3, "low"): 859.6e6, (2, "high"): 666.0e6, (2, "low"): 665.6e6}
PIPE_MIN_STAGES_PER_SM = 200  # the library's rule for choosing the pipelined first PowerSGD pass (acc_powersgd.cu)


def traffic_key(kernel, args, table, n_workers, sm_count):
    """The traffic figure that belongs to the implementation of the first PowerSGD pass this run used."""
    if kernel != "psgd_project_kernel":
        return kernel
    from paper_2010_16248_b200 import workloads as wl
    tiles = sum(-(-int(table.sizes[l]) // 8192) for l in range(table.n_layers) if table.kind[l] == wl.MATRIX)
    pipelined = args.pipeline == "always" or (args.pipeline == "auto" and
                                              tiles * n_workers // max(sm_count, 1) >= PIPE_MIN_STAGES_PER_SM)
    return kernel + "/pipelined" if pipelined else kernel

if __name__ == "__main__":
    main()
