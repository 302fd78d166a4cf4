#!/usr/bin/env python
"""Benchmark of the ARMOR per-layer optimisation on B200.

One "step" is one pass of the whole hot path over one synthetic layer: calibration Gram of all tokens,
initialisation, n_iters BCD iterations, proxy loss, and the factorised forward y = A S B x on a token batch.
Default workload: the Llama-7B-shaped attention projection (4096 x 4096, d_block 128, 262,144 calibration
tokens, 50 iterations).  Prints ONE JSON line (rank 0).

  python bench.py --gpus 1 --steps 3 --warmup 3
  python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N     (N independent replicas)
  python bench.py --impl reference      (the CPU oracle, timed on a bounded sample of the same workload)
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2510_05528_b200 import inputs  # noqa: E402

METRIC = "bcd_iterations_per_s"
UNIT = "iterations/s"
APPLY_TOKENS = 8192
# nominal dense tensor ratio tf32 : bf16 (1.1 : 2.25 PFLOP/s), used only if the tf32 yardstick cannot run
TF32_OVER_BF16 = 1.1 / 2.25
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM counters of the dominant kernel, one entry per precision mode, each naming the capture it comes from
TRAFFIC_FILE = os.path.join(ROOT, "profiles", "dram_traffic.json")


def gemm_traffic(precision):
    """DRAM bytes (read + write) of one dense 4096^3 launch of the tensor-core GEMM in the given mode, from the
    ncu capture recorded in profiles/dram_traffic.json; None when no capture of the current kernel is on file."""
    try:
        with open(TRAFFIC_FILE) as f:
            return json.load(f).get(precision, {}).get("dram_bytes_per_launch")
    except (OSError, ValueError):
        return None


def measure_tf32_yardstick(dev, seconds=2.0):
    """Measured tf32 rate of this GPU: a plain library matmul (fp32 storage, tf32 allowed) of 8192^3, best of 10
    launches (burst) and back to back for `seconds` (sustained, under the power cap).  A yardstick for the
    roofline only: nothing on the timed path calls it."""
    n = 8192
    old = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = True
    try:
        a = torch.randn(n, n, device=dev)
        b = torch.randn(n, n, device=dev)
        c = torch.empty(n, n, device=dev)
        for _ in range(3):
            torch.matmul(a, b, out=c)
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); torch.matmul(a, b, out=c); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        per = best * 1e-3
        reps = max(10, int(seconds / per))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            torch.matmul(a, b, out=c)
        e1.record(); torch.cuda.synchronize()
        flops = 2.0 * n ** 3
        return {"tf32_tflops": flops / per / 1e12, "tf32_tflops_sustained": flops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12,
                "how": f"torch.matmul fp32 8192^3 with tf32 allowed: best of 10 (burst), {reps} back to back (sustained)"}
    finally:
        torch.backends.cuda.matmul.allow_tf32 = old


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        for s in self.samples:
            f = [x.strip() for x in s.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(ms: float, device) -> float:
    """The slowest rank's time: what a job of independent replicas takes.  Works on any initialised process
    group (NCCL with a CUDA device, gloo with the CPU)."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(ms)
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(n_iters: int, world: int, ms_per_step: float) -> float:
    """Iterations per second of the whole job: every rank optimises its own layer (weak scaling)."""
    return world * n_iters / (ms_per_step / 1e3)


def dist_env():
    return int(os.environ.get("RANK", 0)), int(os.environ.get("LOCAL_RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))


# ------------------------------------------------------------------------------------- CPU oracle leg
def oracle_threads():
    try:
        from threadpoolctl import threadpool_info
        return int(max([p.get("num_threads", 1) for p in threadpool_info()] or [os.cpu_count()]))
    except Exception:
        return int(os.cpu_count() or 1)


def oracle_tiny_full():
    """The oracle (numpy fp64 on the host's threaded BLAS, as it stands) on the whole small configuration:
    Gram of all its tokens, initialisation, all its iterations.  A timing, not an extrapolation."""
    from oracle import armor_oracle as O
    cfg = inputs.CONFIGS["tiny"]
    W = inputs.make_weight(cfg).astype(np.float64)
    X = inputs.make_activations(cfg)
    t0 = time.perf_counter()
    H = O.gram(X)
    O.run(W, H, O.OracleConfig(cfg.d_block, seed=cfg.seed), cfg.n_iters, want_loss=False)
    dt = time.perf_counter() - t0
    return {"workload": f"tiny: W {cfg.d_out}x{cfg.d_in}, d_block {cfg.d_block}, {cfg.n_tokens} tokens, {cfg.n_iters} iterations",
            "seconds": dt, "iterations_per_s": cfg.n_iters / dt}


def oracle_sample(cfg, gram_tokens=8192):
    """Times the oracle, as it stands, on a bounded sample of the workload: the Gram of `gram_tokens` tokens and
    ONE full BCD iteration at the layer's full size.  The layer's time follows by scaling the Gram to all tokens
    and the iteration to all iterations (both are linear: profiles/ records one run of the whole workload that
    checks it)."""
    from oracle import armor_oracle as O
    W = inputs.make_weight(cfg).astype(np.float64)
    scales = torch.from_numpy(inputs.channel_scales(cfg))
    nchunk = max(1, min(inputs.n_chunks(cfg), (gram_tokens + cfg.chunk_rows - 1) // cfg.chunk_rows))
    X = np.concatenate([inputs.activation_chunk(cfg, i, scales).numpy() for i in range(nchunk)])[:gram_tokens]
    t_start = time.perf_counter()
    H = O.gram(X)
    t_gram = time.perf_counter() - t_start
    H *= cfg.n_tokens / X.shape[0]
    oc = O.OracleConfig(cfg.d_block, seed=cfg.seed, n_keep=cfg.n_keep, m_group=cfg.m_group)
    t0 = time.perf_counter()
    A, B, S, M = O.init(W, H, oc)
    t_init = time.perf_counter() - t0
    t0 = time.perf_counter()
    O.bcd_iteration(W, A, B, S, M, H, oc, 0, want_loss=False)
    t_iter = time.perf_counter() - t0
    t_sample = time.perf_counter() - t_start
    t_layer = t_gram * cfg.n_tokens / X.shape[0] + t_init + cfg.n_iters * t_iter
    return {"value": cfg.n_iters / t_layer, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"numpy fp64 on threaded BLAS: Gram of {X.shape[0]} of {cfg.n_tokens} tokens ({t_gram:.2f} s) + init "
                      f"({t_init:.2f} s) + 1 of {cfg.n_iters} BCD iterations at full {cfg.d_out}x{cfg.d_in} ({t_iter:.2f} s); "
                      f"the layer's time is these scaled to all tokens and all iterations",
            "sec_per_layer_scaled": t_layer, "sec_per_iteration": t_iter, "sample_seconds": t_sample}


def oracle_full(cfg):
    """The oracle on the WHOLE workload (every token chunk, every iteration): minutes of host time."""
    from oracle import armor_oracle as O
    W = inputs.make_weight(cfg).astype(np.float64)
    scales = torch.from_numpy(inputs.channel_scales(cfg))
    t_start = time.perf_counter()
    H = None
    t_gen = 0.0
    for i in range(inputs.n_chunks(cfg)):
        t0 = time.perf_counter()
        Xc = inputs.activation_chunk(cfg, i, scales).numpy()
        t_gen += time.perf_counter() - t0                  # drawing the synthetic tokens is not the method's work
        H = O.gram(Xc, H)
    t_gram = time.perf_counter() - t_start - t_gen
    oc = O.OracleConfig(cfg.d_block, seed=cfg.seed, n_keep=cfg.n_keep, m_group=cfg.m_group)
    t0 = time.perf_counter()
    (A, B, S, M), infos = O.run(W, H, oc, cfg.n_iters, want_loss=False)
    t_run = time.perf_counter() - t0
    loss = O.proxy_loss(W, A, B, S, H)
    t_layer = t_gram + t_run
    return {"value": cfg.n_iters / t_layer, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "sample": f"the whole workload: Gram of all {cfg.n_tokens} tokens ({t_gram:.1f} s) + init + all {cfg.n_iters} "
                      f"iterations ({t_run:.1f} s); final loss {loss:.6g}",
            "sec_per_layer": t_layer, "sec_per_iteration": t_run / cfg.n_iters}


def run_reference(args, cfg):
    """The reference arm: the CPU oracle on the host cores.  A step is a bounded sample of the workload (see
    oracle_sample); `ms_per_step` is the time the sample took, `value` the iterations per second of the whole
    workload that the sample implies.  --oracle-full times the whole workload instead (one step, minutes)."""
    rank, _, world = dist_env()
    if rank != 0:
        return
    vals = []
    for i in range((0 if args.oracle_full else args.warmup) + (1 if args.oracle_full else args.steps)):
        last = oracle_full(cfg) if args.oracle_full else oracle_sample(cfg, gram_tokens=4096)
        if args.oracle_full or i >= args.warmup:
            vals.append(last)
    key = "sec_per_layer" if args.oracle_full else "sec_per_layer_scaled"
    t_layer = float(np.mean([v[key] for v in vals]))
    t_step = t_layer if args.oracle_full else float(np.mean([v["sample_seconds"] for v in vals]))
    value = cfg.n_iters / t_layer
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": len(vals), "warmup": 0 if args.oracle_full else args.warmup, "ms_per_step": t_step * 1e3,
            "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": workload_config(cfg), "precision": "fp64 (numpy on threaded BLAS)",
            "sec_per_layer": t_layer,
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": last["cores"], "kind": "oracle", "sample": last["sample"]},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def kernel_table_rows(raw, peaks):
    """Per kernel class: launches, device time, algorithmic work per second and its fraction of the bound that
    applies (HBM copy bandwidth for the streaming classes, nothing for the classes of small kernels)."""
    rows = {}
    total = sum(ms for _, ms, _ in raw.values())
    for name, (n, ms, work) in raw.items():
        if n == 0:
            continue
        row = {"launches": n, "total_ms": ms, "avg_us": 1e3 * ms / n, "share": ms / total if total else None}
        if work > 0 and ms > 0:
            if name in ("gemm", "cholesky"):
                row["tflops"] = work / (ms * 1e-3) / 1e12
            else:
                row["gb_per_s"] = work / (ms * 1e-3) / 1e9
                row["frac_of_hbm_peak"] = row["gb_per_s"] / peaks["hbm_gbs"]
        rows[name] = row
    return rows


def workload_config(cfg):
    return {"workload": f"{cfg.name}: W {cfg.d_out}x{cfg.d_in} fp32, d_block {cfg.d_block}, {cfg.n_keep}:{cfg.m_group}, "
                        f"{cfg.n_tokens} calibration "
                        f"tokens, {cfg.n_iters} BCD iterations, h_mode FULL, apply on {APPLY_TOKENS} tokens",
            "l2": "inputs larger than L2 (X is %.2f GB, streamed every step)" % (cfg.n_tokens * cfg.d_in * 4 / 1e9),
            "step": "gram + init + bcd iterations + proxy loss + apply"}


# ------------------------------------------------------------------------------------- GPU arm
def run_ours(args, cfg):
    from paper_2510_05528_b200 import binding as Bd
    from paper_2510_05528_b200 import build as armor_build
    rank, local_rank, world = dist_env()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    armor_build.build()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    use_dist = world > 1
    if use_dist:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    prec = {"fp32x3": Bd.PREC_FP32X3, "tf32": Bd.PREC_TF32, "fp16x3": Bd.PREC_FP16X3}[args.precision]
    lcfg = cfg.with_(seed=cfg.seed + 1000 * rank)          # every rank optimises its own layer
    ctx = Bd.ArmorContext(lcfg.d_out, lcfg.d_in, lcfg.d_block, device=dev, precision=prec, seed=lcfg.seed,
                          n_keep=lcfg.n_keep, m_group=lcfg.m_group)
    if args.no_graphs:
        Bd.armor_use_graphs(ctx.ctx, False)

    # ---- synthetic inputs, generated on the host and staged in pinned memory
    W_h = torch.from_numpy(inputs.make_weight(lcfg)).pin_memory()
    X_h = torch.empty(lcfg.n_tokens, lcfg.d_in, dtype=torch.float32, pin_memory=True)
    scales = torch.from_numpy(inputs.channel_scales(lcfg))
    for i in range(inputs.n_chunks(lcfg)):
        lo = i * lcfg.chunk_rows
        inputs.activation_chunk(lcfg, i, scales, out=X_h[lo: lo + lcfg.chunk_rows])
    xt_h = torch.from_numpy(inputs.make_tokens(lcfg, APPLY_TOKENS)).pin_memory()
    X_d, W_d, xt_d = X_h.to(dev), W_h.to(dev), xt_h.to(dev)
    H = ctx.new_gram()
    loss_h = torch.zeros(1, dtype=torch.float64).pin_memory()

    def step_resident():
        H.zero_()
        ctx.gram(X_d, H)
        st = ctx.init(W_d, H)
        ctx.bcd_step(st, H, 0, lcfg.n_iters, want_stats=False)
        loss = ctx.proxy_loss(st, H)
        y = ctx.apply(st, xt_d)
        return st, loss, y

    e2e_chunk = 32768
    xbuf = [torch.empty(e2e_chunk, lcfg.d_in, dtype=torch.float32, device=dev) for _ in range(2)]
    copy_stream = torch.cuda.Stream(device=dev)
    out_h = {"A": torch.empty(lcfg.d_out // lcfg.d_block, lcfg.d_block, lcfg.d_block).pin_memory(),
             "B": torch.empty(lcfg.d_in // lcfg.d_block, lcfg.d_block, lcfg.d_block).pin_memory(),
             "S": torch.empty(lcfg.d_out, lcfg.d_in).pin_memory(),
             "M": torch.empty(lcfg.d_out, lcfg.d_in // lcfg.m_group, dtype=torch.uint8).pin_memory(),
             "y": torch.empty(APPLY_TOKENS, lcfg.d_out).pin_memory()}
    h2d = X_h.numel() * 4 + W_h.numel() * 4 + xt_h.numel() * 4
    d2h = sum(t.numel() * t.element_size() for t in out_h.values()) + 8

    def step_e2e():
        """Host buffers in, host buffers out: every copy is inside the timed region.  The token chunks are
        double-buffered so that the next host->device copy overlaps the Gram of the current chunk."""
        main = torch.cuda.current_stream()
        H.zero_()
        Wd = W_h.to(dev, non_blocking=True)
        n = lcfg.n_tokens
        evs = [None, None]
        for k, lo in enumerate(range(0, n, e2e_chunk)):
            b = k & 1
            rows = min(e2e_chunk, n - lo)
            with torch.cuda.stream(copy_stream):
                if evs[b] is not None:
                    copy_stream.wait_event(evs[b])          # the Gram that read this buffer has finished
                xbuf[b][:rows].copy_(X_h[lo: lo + rows], non_blocking=True)
                ready = torch.cuda.Event()
                ready.record(copy_stream)
            main.wait_event(ready)
            ctx.gram(xbuf[b][:rows], H)
            evs[b] = torch.cuda.Event()
            evs[b].record(main)
        st = ctx.init(Wd, H)
        ctx.bcd_step(st, H, 0, lcfg.n_iters, want_stats=False)
        loss = ctx.proxy_loss(st, H)
        y = ctx.apply(st, xt_h.to(dev, non_blocking=True))
        out_h["A"].copy_(st.A, non_blocking=True); out_h["B"].copy_(st.B, non_blocking=True)
        out_h["S"].copy_(st.S, non_blocking=True); out_h["M"].copy_(st.M, non_blocking=True)
        out_h["y"].copy_(y, non_blocking=True); loss_h.copy_(loss, non_blocking=True)
        return st

    def run_e2e_pipelined(n_steps, bufs):
        """The same step with the next step's tokens uploaded while the current step iterates (layers of a model are
        independent jobs: the upload of layer l+1 hides behind the BCD of layer l).  Every step's inputs still come
        from pinned host memory inside the timed region; the first step has nothing to hide behind and uploads chunk
        by chunk under its own Gram."""
        main = torch.cuda.current_stream()
        n = lcfg.n_tokens
        pre = None
        for i in range(n_steps):
            Xcur = bufs[i & 1]
            H.zero_()
            Wd = W_h.to(dev, non_blocking=True)
            if i == 0:
                for lo in range(0, n, e2e_chunk):
                    rows = min(e2e_chunk, n - lo)
                    with torch.cuda.stream(copy_stream):
                        Xcur[lo: lo + rows].copy_(X_h[lo: lo + rows], non_blocking=True)
                        ready = torch.cuda.Event()
                        ready.record(copy_stream)
                    main.wait_event(ready)
                    ctx.gram(Xcur[lo: lo + rows], H)
            else:
                main.wait_event(pre)
                for lo in range(0, n, e2e_chunk):
                    ctx.gram(Xcur[lo: min(lo + e2e_chunk, n)], H)
            if i + 1 < n_steps:
                # the other buffer was last read by the Gram of step i - 1, which precedes this point on the main stream
                free = torch.cuda.Event()
                free.record(main)
                with torch.cuda.stream(copy_stream):
                    copy_stream.wait_event(free)
                    bufs[(i + 1) & 1].copy_(X_h, non_blocking=True)
                    pre = torch.cuda.Event()
                    pre.record(copy_stream)
            st = ctx.init(Wd, H)
            ctx.bcd_step(st, H, 0, lcfg.n_iters, want_stats=False)
            loss = ctx.proxy_loss(st, H)
            y = ctx.apply(st, xt_h.to(dev, non_blocking=True))
            out_h["A"].copy_(st.A, non_blocking=True); out_h["B"].copy_(st.B, non_blocking=True)
            out_h["S"].copy_(st.S, non_blocking=True); out_h["M"].copy_(st.M, non_blocking=True)
            out_h["y"].copy_(y, non_blocking=True); loss_h.copy_(loss, non_blocking=True)

    def barrier():
        if use_dist:
            import torch.distributed as dist
            dist.barrier(device_ids=[local_rank])
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dev)

    for _ in range(args.warmup):
        step_resident()
    torch.cuda.synchronize()

    # ---- timed region (device-resident inputs)
    Bd.armor_gemm_timing_enable(ctx.ctx, True)
    Bd.armor_gemm_timing(ctx.ctx)
    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    l0 = ctx.launch_count()
    torch.cuda.nvtx.range_push("timed_steps")     # lets a profiler capture exactly the launches of the timed region
    ms_total = timed(step_resident, args.steps)
    torch.cuda.nvtx.range_pop()
    launches = ctx.launch_count() - l0
    clocks = sampler.stop() if rank == 0 else None
    n_gemm, gemm_ms, gemm_flops = Bd.armor_gemm_timing(ctx.ctx)
    Bd.armor_gemm_timing_enable(ctx.ctx, False)
    status = ctx.device_status()

    # ---- the same steps once more without the events around the GEMM launches: the library then replays each
    # repeated iteration of a call from ONE CUDA graph (the headline region above carries the events for the roofline,
    # so there the iteration is replayed in pieces, with the dense products launched directly between their events)
    for _ in range(2):
        step_resident()
    ms_graph = timed(step_resident, args.steps)

    # ---- per-phase breakdown (one extra step, not part of the headline)
    def t_phase(fn):
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); r = fn(); b.record(); torch.cuda.synchronize()
        return a.elapsed_time(b), r
    H.zero_()
    ms_gram, _ = t_phase(lambda: ctx.gram(X_d, H))
    ms_init, st = t_phase(lambda: ctx.init(W_d, H))
    ms_bcd, stats = t_phase(lambda: ctx.bcd_step(st, H, 0, lcfg.n_iters))
    ms_loss, loss = t_phase(lambda: ctx.proxy_loss(st, H))
    ms_apply, _ = t_phase(lambda: ctx.apply(st, xt_d))
    srec = ctx.read_stats(stats)

    # ---- every kernel class of one more step, each launch bracketed by events on its stream (the brackets cost
    # about a microsecond per launch, so this step is not part of the headline)
    kernel_table = None
    if args.kernel_table:
        Bd.armor_kernel_timing_enable(ctx.ctx, 2)
        Bd.armor_kernel_timing(ctx.ctx)
        step_resident()
        torch.cuda.synchronize()
        raw = Bd.armor_kernel_timing(ctx.ctx)
        Bd.armor_kernel_timing_enable(ctx.ctx, 0)
        kernel_table = kernel_table_rows(raw, load_peaks()[0])

    # ---- the one-pass tf32 mode on the same workload (context only; not the headline: its parity tolerance
    # is looser, see tests/helpers.py)
    tf32_mode = None
    if args.precision != "tf32" and not args.no_tf32:
        ctx32 = Bd.ArmorContext(lcfg.d_out, lcfg.d_in, lcfg.d_block, device=dev, precision=Bd.PREC_TF32, seed=lcfg.seed,
                                n_keep=lcfg.n_keep, m_group=lcfg.m_group)

        def step32():
            H.zero_()
            ctx32.gram(X_d, H)
            s32 = ctx32.init(W_d, H)
            ctx32.bcd_step(s32, H, 0, lcfg.n_iters, want_stats=False)
            l32 = ctx32.proxy_loss(s32, H)
            ctx32.apply(s32, xt_d)
            return l32
        for _ in range(3):
            step32()
        Bd.armor_gemm_timing_enable(ctx32.ctx, True)
        Bd.armor_gemm_timing(ctx32.ctx)
        ms32 = timed(step32, args.steps)
        n32, gms32, gfl32 = Bd.armor_gemm_timing(ctx32.ctx)
        Bd.armor_gemm_timing_enable(ctx32.ctx, False)
        l32 = step32()
        tf32_mode = {"ms_per_step": ms32 / args.steps, "iterations_per_s": world * lcfg.n_iters / (ms32 / args.steps / 1e3),
                     "final_loss": float(l32.item()),
                     "gemm_tflops": gfl32 / (gms32 * 1e-3) / 1e12 if gms32 > 0 else None,
                     "gemm_share_of_step": gms32 / ms32 if ms32 > 0 else None}
        del ctx32

    # ---- the paper's own operating point and two neighbours, on the same W and H (context only, rank-local):
    # diagonal weighting with the exact block solves; diagonal weighting with the joint Adam step (what the paper
    # runs, for 20,000 iterations per layer); full weighting with four sparse-core updates per iteration
    other_modes = None
    if args.other_modes:
        other_modes = {}
        H.zero_()
        ctx.gram(X_d, H)
        for name, kw, iters in (("diag_exact", dict(h_mode=Bd.H_DIAG), lcfg.n_iters),
                                ("diag_adam_lr1e-4", dict(h_mode=Bd.H_DIAG, ab_step=Bd.AB_ADAM), 10 * lcfg.n_iters),
                                ("full_adam_lr1e-4", dict(h_mode=Bd.H_FULL, ab_step=Bd.AB_ADAM), lcfg.n_iters),
                                ("full_exact_4_sweeps", dict(h_mode=Bd.H_FULL, mask_sweeps=4), lcfg.n_iters),
                                ("full_exact_4_groups", dict(h_mode=Bd.H_FULL, mask_groups=4), lcfg.n_iters),
                                ("diag_adam_lr1e-4_8_groups", dict(h_mode=Bd.H_DIAG, ab_step=Bd.AB_ADAM, mask_groups=8),
                                 10 * lcfg.n_iters)):
            cx = Bd.ArmorContext(lcfg.d_out, lcfg.d_in, lcfg.d_block, device=dev, precision=prec, seed=lcfg.seed,
                                 n_keep=lcfg.n_keep, m_group=lcfg.m_group, **kw)
            sx = cx.init(W_d, H)
            cx.bcd_step(sx, H, 0, 3, want_stats=False)          # warm-up
            sx = cx.init(W_d, H)
            l_init = float(cx.proxy_loss(sx, H).item())
            ms_x, _ = t_phase(lambda: cx.bcd_step(sx, H, 0, iters, want_stats=False))
            other_modes[name] = {"iterations": iters, "ms_per_iteration": ms_x / iters,
                                 "iterations_per_s": iters / (ms_x / 1e3),
                                 "loss_init": l_init, "loss_final": float(cx.proxy_loss(sx, H).item()),
                                 "device_status": cx.device_status()[:4]}
            if "adam" in name:
                other_modes[name]["s_per_20000_iterations"] = 20000 * ms_x / iters / 1e3
            del cx, sx

        # the deployment form on the same layer: fp32-grade, bf16 with the core dense, bf16 with the 2:4 core packed
        # for the sparse tensor cores (packed once, and packed on every call)
        cf = Bd.ArmorContext(lcfg.d_out, lcfg.d_in, lcfg.d_block, device=dev, precision=prec, seed=lcfg.seed,
                             n_keep=lcfg.n_keep, m_group=lcfg.m_group)
        sf = cf.init(W_d, H)
        cf.bcd_step(sf, H, 0, 2, want_stats=False)
        xb = xt_d.to(torch.bfloat16)
        y32 = cf.apply(sf, xt_d)
        fwd = {"tokens": APPLY_TOKENS}
        variants = [("fp32", lambda: cf.apply(sf, xt_d)), ("bf16_dense_core", lambda: cf.apply(sf, xb))]
        if lcfg.d_out % 128 == 0 and lcfg.d_in % 128 == 0 and lcfg.m_group == 4:
            packed = cf.pack_core(sf)
            variants += [("bf16_sparse_core_packed_once", lambda: cf.apply_packed(sf, packed, xb)),
                         ("bf16_sparse_core_packed_per_call", lambda: cf.apply(sf, xb, sparse=True))]
            if lcfg.d_block % 128 == 0:
                layer = cf.pack_layer(sf)
                variants += [("bf16_packed_layer", lambda: cf.apply_layer(layer, xb))]
        for name, fn in variants:
            for _ in range(3):
                yv = fn()
            torch.cuda.synchronize()
            Bd.armor_gemm_timing_enable(cf.ctx, True)
            Bd.armor_gemm_timing(cf.ctx)
            ms_f, _ = t_phase(lambda: [fn() for _ in range(10)])
            n_c, ms_c, fl_c = Bd.armor_gemm_timing(cf.ctx)
            Bd.armor_gemm_timing_enable(cf.ctx, False)
            fwd[name] = {"ms_per_forward": ms_f / 10, "core_product_ms": ms_c / 10,
                         "core_product_tflops_dense_equivalent": fl_c / (ms_c * 1e-3) / 1e12 if ms_c > 0 else None,
                         "rel_diff_to_fp32": float(((yv.float() - y32).norm() / y32.norm()).item())}
        fwd["device_status"] = cf.device_status()[:5]
        other_modes["forward"] = fwd
        del cf, sf

    # ---- end to end (host buffers)
    if args.no_e2e:
        ms_e2e = None
    else:
        for _ in range(min(args.warmup, 2)):
            step_e2e()
        ms_e2e = timed(step_e2e, args.steps)
    ms_e2e_pipe = None
    if not args.no_e2e and args.steps > 1:
        free_b, _ = torch.cuda.mem_get_info(dev)
        if free_b > 2 * X_h.numel() * 4:
            bufs = [X_d, torch.empty_like(X_d)]
            run_e2e_pipelined(2, bufs)
            ms_e2e_pipe = timed(lambda: run_e2e_pipelined(args.steps, bufs), 1)
            del bufs
    del X_d

    if rank != 0:
        if use_dist:
            import torch.distributed as dist
            dist.destroy_process_group()
        return
    peaks, peak_kind = load_peaks()
    yard = None
    if not args.no_yardstick:
        try:
            yard = measure_tf32_yardstick(dev)
        except RuntimeError:
            yard = None
    ms_step = ms_total / args.steps
    value = whole_job_value(lcfg.n_iters, world, ms_step)
    e2e_value = world * lcfg.n_iters / (ms_e2e / args.steps / 1e3) if ms_e2e else None
    f16_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])      # the kernel is timed inside a long step
    if yard:
        tf32_peak, tf32_kind = yard["tf32_tflops_sustained"], "measured in this run (" + yard["how"] + ")"
    else:
        tf32_peak, tf32_kind = f16_peak * TF32_OVER_BF16, f"{peak_kind} sustained bf16 x nominal tf32/bf16 ratio"
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    passes = 1 if args.precision == "tf32" else 3
    pipe = {"fp16x3": "kind::f16 (fp16 operands)", "fp32x3": "kind::tf32", "tf32": "kind::tf32"}[args.precision]
    pipe_peak = f16_peak if args.precision == "fp16x3" else tf32_peak
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic", "config": workload_config(lcfg), "precision": args.precision,
        "sec_per_layer": ms_step / 1e3,
        "bcd_only_iterations_per_s": lcfg.n_iters / (ms_bcd / 1e3),
        "phases_ms": {"gram": ms_gram, "init": ms_init, "bcd": ms_bcd, "bcd_per_iteration": ms_bcd / lcfg.n_iters,
                      "proxy_loss": ms_loss, "apply": ms_apply},
        "loss": {"init": float(srec["loss_start"][0]), "final": float(loss.item()),
                 "mask_steps_accepted": int(srec["mask_accepted"].sum()), "chol_failed": int(srec["chol_failed"].sum())},
        "device_status": status[:4],
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                "ms_per_step": ms_e2e / args.steps if ms_e2e else None,
                "pipelined_value": world * lcfg.n_iters / (ms_e2e_pipe / args.steps / 1e3) if ms_e2e_pipe else None,
                "pipelined_note": "same copies, but the tokens of step k+1 are uploaded while step k iterates; the first "
                                  "of the timed steps uploads its own under its Gram"},
        "gpu_launches": int(launches),
        "graph_replay": {"value": whole_job_value(lcfg.n_iters, world, ms_graph / args.steps), "unit": UNIT,
                         "ms_per_step": ms_graph / args.steps,
                         "note": "the same timed steps without events around the GEMM launches: armor_bcd_step then "
                                 "replays iterations 2..n of a call from one CUDA graph each (in the headline region "
                                 "from graph pieces between the directly launched, event-bracketed GEMMs)"},
        "kernel_table": kernel_table,
        "tf32_mode": tf32_mode,
        "other_modes": other_modes,
        "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": f"tc_gemm_kernel (tcgen05 {pipe}, Gram + dense .H contractions)",
                     "achieved": achieved, "peak": tf32_peak, "unit": "TFLOP/s", "frac": achieved / tf32_peak,
                     "traffic": gemm_traffic(args.precision),
                     "note": f"achieved = algorithmic flops (one fp32 product: 2 M N K, the Gram's lower triangle M (N + 128) K) "
                             f"of {n_gemm} launches / their CUDA-event time ({gemm_ms:.1f} ms of {ms_total:.1f} ms).  The "
                             f"operands are 32-bit, so the peak is the tf32 rate of this GPU, {tf32_kind}.  The "
                             f"{args.precision} mode issues {passes} tensor-core pass(es) per product on the {pipe} pipe: "
                             f"'pipe' gives the rate of issued flops against that pipe's own measured peak "
                             f"({peak_kind} sustained bf16 for kind::f16).  traffic = DRAM bytes of one dense 4096^3 launch",
                     "pipe": {"achieved": achieved * passes, "peak": pipe_peak, "frac": achieved * passes / pipe_peak,
                              "passes": passes},
                     "share_of_step": gemm_ms / ms_total},
        "tensor_yardstick": yard,
    }
    if world == 1 and not args.no_cpu_baseline:
        line["cpu_baseline"] = {k: v for k, v in oracle_sample(lcfg).items()
                                if k in ("value", "unit", "cores", "kind", "sample")}
        line["cpu_baseline"]["tiny_config_in_full"] = oracle_tiny_full()
    print(json.dumps(line), flush=True)
    if use_dist:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------------- long runs
def run_long(args, cfg):
    """Thousands of iterations in ONE armor_bcd_step call per mode (the regime of the paper's schedule): the
    loss the library tracks through the call against the loss evaluated afresh from the final state, which shows
    what the quantities carried from iteration to iteration (T H_w, the running loss) have drifted by."""
    from paper_2510_05528_b200 import binding as Bd
    from paper_2510_05528_b200 import build as armor_build
    armor_build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    prec = {"fp32x3": Bd.PREC_FP32X3, "tf32": Bd.PREC_TF32, "fp16x3": Bd.PREC_FP16X3}[args.precision]
    n = args.long_run
    W_d = torch.from_numpy(inputs.make_weight(cfg)).to(dev)
    base = Bd.ArmorContext(cfg.d_out, cfg.d_in, cfg.d_block, device=dev, precision=prec, seed=cfg.seed)
    H = base.new_gram()
    scales = torch.from_numpy(inputs.channel_scales(cfg))
    for i in range(inputs.n_chunks(cfg)):
        base.gram(inputs.activation_chunk(cfg, i, scales).to(dev), H)
    del base
    out = {}
    for name, kw in (("full_exact", dict(h_mode=Bd.H_FULL)),
                     ("diag_adam_lr1e-4", dict(h_mode=Bd.H_DIAG, ab_step=Bd.AB_ADAM))):
        ctx = Bd.ArmorContext(cfg.d_out, cfg.d_in, cfg.d_block, device=dev, precision=prec, seed=cfg.seed, **kw)
        st = ctx.init(W_d, H)
        l_init = float(ctx.proxy_loss(st, H).item())
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        stats = ctx.bcd_step(st, H, 0, n)
        e1.record()
        torch.cuda.synchronize()
        sr = ctx.read_stats(stats)
        fresh = float(ctx.proxy_loss(st, H).item())
        tracked = float(sr["loss_mask"][-1])
        seq = np.concatenate([[l_init], sr["loss_mask"]])
        Mb = st.M.cpu().numpy()
        out[name] = {"iterations": n, "ms_per_iteration": e0.elapsed_time(e1) / n, "seconds": e0.elapsed_time(e1) / 1e3,
                     "loss_init": l_init, "loss_after_100": float(sr["loss_mask"][min(99, n - 1)]),
                     "loss_tracked_final": tracked, "loss_evaluated_final": fresh,
                     "tracked_minus_evaluated_rel": (tracked - fresh) / fresh,
                     "largest_rise_between_iterations_rel": float(np.max(np.diff(seq) / seq[:-1])),
                     "mask_steps_accepted": int(sr["mask_accepted"].sum()), "groups_changed": int(sr["groups_changed"].sum()),
                     "chol_failed": int(sr["chol_failed"].sum()),
                     "valid_2_of_4": bool(np.all(np.unpackbits(Mb[:, :, None], axis=2)[:, :, 4:].sum(axis=2) == 2)),
                     "device_status": ctx.device_status()[:10]}
        del ctx, st
    print(json.dumps({"long_run": out, "config": workload_config(cfg), "precision": args.precision}), flush=True)


# ------------------------------------------------------------------------------------- whole layers
# Sets of matrices that share their calibration activations.  (matrix name, inputs.CONFIGS entry, seed offset of W)
LAYER_SETS = {
    # Qwen-shaped attention block with grouped-query attention: q, k, v and o on one shared X (262,144 x 5120)
    "qwen_layer": [("x_shared", [("q_proj", "qwen_q", 0), ("k_proj", "qwen_kv", 0), ("v_proj", "qwen_kv", 1),
                                 ("o_proj", "qwen_q", 1)])],
    # Llama-8B-shaped MLP: up and gate share the block's input, down has the gated activations
    "llama8b_mlp": [("x_mlp_in", [("up_proj", "llama8b_up", 0), ("gate_proj", "llama8b_up", 1)]),
                    ("x_gated", [("down_proj", "llama8b_down", 0)])],
    # 70B-scale MLP pair, d_block 256
    "mlp70b": [("x_mlp_in", [("up_like", "mlp70b_up", 0)]), ("x_gated", [("down_like", "mlp70b_down", 0)])],
}


def run_layer_set(args):
    """One timed region over a whole set of matrices: per group of matrices one Gram of the shared activations
    (resident in HBM when the region starts), then initialisation, all BCD iterations and the final loss of every
    matrix.  Prints one JSON line with seconds per layer and iterations per second over all matrices."""
    from paper_2510_05528_b200 import binding as Bd
    from paper_2510_05528_b200 import build as armor_build
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    armor_build.build()
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    prec = {"fp32x3": Bd.PREC_FP32X3, "tf32": Bd.PREC_TF32, "fp16x3": Bd.PREC_FP16X3}[args.precision]
    n_keep, m_group = (int(v) for v in args.nm.split(":"))
    groups = []
    for xname, mats in LAYER_SETS[args.config]:
        xcfg = inputs.CONFIGS[mats[0][1]]
        if args.tokens > 0:
            xcfg = xcfg.with_(n_tokens=args.tokens)
        X_d = torch.empty(xcfg.n_tokens, xcfg.d_in, dtype=torch.float32, device=dev)
        scales = torch.from_numpy(inputs.channel_scales(xcfg))
        for i in range(inputs.n_chunks(xcfg)):
            lo = i * xcfg.chunk_rows
            X_d[lo: lo + xcfg.chunk_rows].copy_(inputs.activation_chunk(xcfg, i, scales))
        entries = []
        for mname, cname, soff in mats:
            mcfg = inputs.CONFIGS[cname].with_(seed=inputs.CONFIGS[cname].seed + 100 * soff, n_keep=n_keep, m_group=m_group)
            if args.iters > 0:
                mcfg = mcfg.with_(n_iters=args.iters)
            ctx = Bd.ArmorContext(mcfg.d_out, mcfg.d_in, mcfg.d_block, device=dev, precision=prec, seed=mcfg.seed,
                                  n_keep=n_keep, m_group=m_group)
            entries.append((mname, mcfg, ctx, torch.from_numpy(inputs.make_weight(mcfg)).to(dev)))
        groups.append((xname, xcfg, X_d, entries, entries[0][2].new_gram()))

    results = {}

    def one_pass(record):
        for xname, xcfg, X_d, entries, H in groups:
            H.zero_()
            entries[0][2].gram(X_d, H)
            for mname, mcfg, ctx, W_d in entries:
                st = ctx.init(W_d, H)
                stats = ctx.bcd_step(st, H, 0, mcfg.n_iters, want_stats=record)
                loss = ctx.proxy_loss(st, H)
                if record:
                    sr = ctx.read_stats(stats)
                    results[mname] = {"shape": f"{mcfg.d_out}x{mcfg.d_in}", "iterations": mcfg.n_iters,
                                      "loss_init": float(sr["loss_start"][0]), "loss_final": float(loss.item()),
                                      "mask_steps_accepted": int(sr["mask_accepted"].sum()),
                                      "chol_failed": int(sr["chol_failed"].sum()), "device_status": ctx.device_status()[:4]}

    for _ in range(max(1, args.warmup // 3)):          # a whole layer per warm-up pass
        one_pass(False)
    torch.cuda.synchronize()
    ctxs = [e[2] for g in groups for e in g[3]]
    for c in ctxs:
        Bd.armor_gemm_timing_enable(c.ctx, True)
        Bd.armor_gemm_timing(c.ctx)
    sampler = ClockSampler(0)
    sampler.start()
    l0 = sum(c.launch_count() for c in ctxs)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        one_pass(False)
    e1.record()
    torch.cuda.synchronize()
    ms_total = e0.elapsed_time(e1)
    clocks = sampler.stop()
    launches = sum(c.launch_count() for c in ctxs) - l0
    n_gemm = gemm_ms = gemm_flops = 0
    for c in ctxs:
        n, ms, fl = Bd.armor_gemm_timing(c.ctx)
        Bd.armor_gemm_timing_enable(c.ctx, False)
        n_gemm += n; gemm_ms += ms; gemm_flops += fl

    # per-phase times of one more pass (not part of the headline)
    phases = {}
    for xname, xcfg, X_d, entries, H in groups:
        H.zero_()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(); entries[0][2].gram(X_d, H); b.record(); torch.cuda.synchronize()
        phases[f"gram_{xname}"] = a.elapsed_time(b)
        for mname, mcfg, ctx, W_d in entries:
            st = ctx.init(W_d, H)
            torch.cuda.synchronize()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(); ctx.bcd_step(st, H, 0, mcfg.n_iters, want_stats=False); b.record(); torch.cuda.synchronize()
            phases[f"bcd_{mname}"] = a.elapsed_time(b)
            phases[f"bcd_{mname}_per_iteration"] = a.elapsed_time(b) / mcfg.n_iters
    one_pass(True)
    torch.cuda.synchronize()

    peaks, peak_kind = load_peaks()
    yard = None if args.no_yardstick else measure_tf32_yardstick(dev)
    f16_peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    tf32_peak = yard["tf32_tflops_sustained"] if yard else f16_peak * TF32_OVER_BF16
    passes = 1 if args.precision == "tf32" else 3
    pipe_peak = f16_peak if args.precision == "fp16x3" else tf32_peak
    achieved = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    total_iters = sum(e[1].n_iters for g in groups for e in g[3])
    ms_step = ms_total / args.steps
    line = {
        "metric": METRIC, "value": total_iters / (ms_step / 1e3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(1, args.warmup // 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f32", "data": "synthetic", "precision": args.precision,
        "config": {"workload": f"{args.config}: " + "; ".join(
                       f"{xname} {xcfg.n_tokens}x{xcfg.d_in} shared by " + ", ".join(
                           f"{m} {c.d_out}x{c.d_in} ({c.n_iters} iterations)" for m, c, _, _ in entries)
                       for xname, xcfg, _, entries, _ in groups) + f"; d_block {groups[0][3][0][1].d_block}, {args.nm}",
                   "l2": "inputs larger than L2 (the activations are streamed by every Gram)",
                   "step": "per group of matrices: gram; per matrix: init + bcd iterations + proxy loss"},
        "sec_per_layer": ms_step / 1e3, "total_iterations": total_iters, "phases_ms": phases, "matrices": results,
        "e2e": None, "gpu_launches": int(launches / args.steps), "clocks": clocks,
        "roofline": {"bound": "tensor", "kernel": "tc_gemm_kernel (Gram + dense .H contractions)", "achieved": achieved,
                     "peak": tf32_peak, "unit": "TFLOP/s", "frac": achieved / tf32_peak, "traffic": None,
                     "pipe": {"achieved": achieved * passes, "peak": pipe_peak, "frac": achieved * passes / pipe_peak,
                              "passes": passes},
                     "share_of_step": gemm_ms / ms_total,
                     "note": f"{n_gemm} launches in {gemm_ms:.1f} ms of {ms_total:.1f} ms; peaks as in the single-matrix line"},
        "tensor_yardstick": yard,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="llama7b_attn", choices=sorted(inputs.CONFIGS) + sorted(LAYER_SETS),
                    help="one matrix (inputs.CONFIGS) or a whole set of matrices sharing activations: " + ", ".join(sorted(LAYER_SETS)))
    ap.add_argument("--nm", default="2:4", choices=["2:4", "4:8", "5:8", "6:8"], help="sparsity pattern of the core")
    ap.add_argument("--apply-tokens", type=int, default=0, help="token batch of the forward (default 8192)")
    ap.add_argument("--long-run", type=int, default=0,
                    help="instead of the benchmark: this many iterations in one call, with the full weighting and exact "
                         "solves and with the diagonal weighting and joint Adam; prints tracked and re-evaluated losses")
    ap.add_argument("--precision", default="fp16x3", choices=["fp16x3", "fp32x3", "tf32"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--tokens", type=int, default=0,
                    help="profiling aid: calibration tokens instead of the workload's (the line then says 'reduced')")
    ap.add_argument("--iters", type=int, default=0,
                    help="profiling aid: BCD iterations per step instead of the workload's")
    ap.add_argument("--no-e2e", action="store_true", help="profiling aid: skip the host-buffer leg")
    ap.add_argument("--no-tf32", action="store_true", help="skip the extra measurement of the one-pass tf32 mode")
    ap.add_argument("--no-yardstick", action="store_true", help="skip the library-matmul measurement of the tf32 peak")
    ap.add_argument("--no-graphs", action="store_true",
                    help="profiling aid: every iteration with direct launches (a profiler then sees one launch per kernel)")
    ap.add_argument("--oracle-full", action="store_true",
                    help="with --impl reference: time the oracle on the whole workload (minutes) instead of a sample")
    ap.add_argument("--kernel-table", action="store_true",
                    help="also run one step with every launch bracketed by events and report time, algorithmic "
                         "bytes per second and the fraction of the HBM roofline per kernel class")
    ap.add_argument("--other-modes", action="store_true",
                    help="also time the BCD loop with the diagonal weighting, the joint Adam step and several "
                         "sparse-core updates per iteration (a few seconds more)")
    args = ap.parse_args()
    if args.warmup < 3 and args.impl == "ours":
        args.warmup = 3
    if args.apply_tokens > 0:
        global APPLY_TOKENS
        APPLY_TOKENS = args.apply_tokens
    if args.config in LAYER_SETS:
        if args.impl == "reference":
            print(json.dumps({"impl": "reference", "unavailable": "layer sets are timed on the GPU arm only"}))
            return
        return run_layer_set(args)
    cfg = inputs.CONFIGS[args.config]
    n_keep, m_group = (int(v) for v in args.nm.split(":"))
    cfg = cfg.with_(n_keep=n_keep, m_group=m_group)
    if args.tokens > 0 or args.iters > 0:
        cfg = cfg.with_(name=cfg.name + " (reduced for profiling)", n_tokens=args.tokens or cfg.n_tokens,
                        n_iters=args.iters or cfg.n_iters)
    _, _, world = dist_env()
    if args.gpus > 1 and world == 1 and args.impl == "ours":
        # not launched by torchrun: start one process per GPU ourselves
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", "29511", os.path.abspath(__file__)] + sys.argv[1:]
        raise SystemExit(subprocess.call(cmd))
    if args.long_run > 0:
        run_long(args, cfg)
    elif args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
