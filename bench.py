#!/usr/bin/env python
"""Benchmark of the SFDA chunk-WY forward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference]

One "step" is one pass of the whole hot path (sfda_forward: cumulative phase-decay,
operand construction, Gram blocks, the WY triangular system, state-dependent
contractions, outputs, boundary-state scan) over one batch of synthetic input of the
headline configuration (B=8, T=8192, H=32, d_k=d_v=128, chunk=64, bf16 q/k/v, fp32
alpha/theta/beta/state, S0 ~ N(0, 0.02), o = Re + Im).  Prints ONE JSON line.

With N > 1 (launched by torch.distributed.run) every rank runs the same per-GPU
workload on its own batch (the path shards over (batch, head) with no collective):
weak scaling, value = all ranks' tokens / max-over-ranks time.

`--impl reference` times the CPU oracle (the deliberately plain per-token recurrence)
on a bounded sample of the same workload.
"""
import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

import workloads  # noqa: E402

METRIC = "SFDA chunk-WY forward tokens/sec at B=8,T=8192,H=32,d=128"
UNIT = "tokens/s"
HEADLINE = 2


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_tflops": float(p["bf16_tflops"]),
                "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


def algorithmic_bytes(cfg, want_im=True):
    """Compulsory HBM traffic of one forward: q, k, v, alpha, theta, beta read once, o (and o_im)
    written once, S0 read and S_T written once per (batch, head)."""
    eb = 2 if cfg.dtype == "bf16" else 4
    per_token_head = 2 * cfg.d_k * eb + cfg.d_v * eb + 2 * cfg.m * 4 + 4 + (2 if want_im else 1) * cfg.d_v * eb
    return cfg.B * cfg.T * cfg.H * per_token_head + cfg.B * cfg.H * 2 * cfg.d_k * cfg.d_v * 4


def algorithmic_flops(cfg, want_im=True):
    """F_chunk = 4 d_k C^2 + 12 C d_k d_v + 8 C^2 d_v real flops per chunk for Re + Im outputs
    (complex MAC = 8 flops, triangular products at their triangular size)."""
    C = cfg.chunk
    f = 4 * cfg.d_k * C * C + 12 * C * cfg.d_k * cfg.d_v + 8 * C * C * cfg.d_v
    if not want_im:
        f -= 2 * C * cfg.d_k * cfg.d_v + 2 * C * C * cfg.d_v
    return cfg.B * cfg.H * (-(-cfg.T // C)) * f


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons of one GPU while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.rows = []
        self._stop = threading.Event()
        self._thread = threading.Thread(target=self._run, daemon=True)

    def _run(self):
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.FIELDS,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=5)
                if out.returncode == 0 and out.stdout.strip():
                    self.rows.append([c.strip() for c in out.stdout.strip().splitlines()[0].split(",")])
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=10)

    def summary(self):
        sm, smax, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            try:
                sm.append(float(r[0]))
                smax.append(float(r[1]))
            except (ValueError, IndexError):
                continue
            for name, val in zip(names, r[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(smax) if smax else None,
                "reasons": sorted(reasons), "samples": len(sm),
                "sm_mhz_first": sm[0] if sm else None,
                "window": "timed region plus about a second of the same launches, longer until five samples are in "
                          "(the timed region alone is shorter than one nvidia-smi sample)"}


def cpu_oracle_throughput(cfg, n_pairs, T):
    """Time the oracle, as it stands, on n_pairs (batch, head) sequences of T tokens of the workload."""
    from oracle import recurrence
    sub = cfg.scaled(T=T)
    per_b = max(1, min(cfg.H, n_pairs))
    pairs = [(i // per_b, i % per_b) for i in range(n_pairs)]
    inp = workloads.forward_inputs(sub, batch=sorted({b for b, _ in pairs}))
    s = workloads.sequences(inp, pairs)
    recurrence.sfda_recurrence(s["q"][:, :64], s["k"][:, :64], s["v"][:, :64], s["alpha"][:, :64],
                               s["theta"][:, :64], s["beta"][:, :64], s["S0"])       # load + warm the library
    t0 = time.perf_counter()
    recurrence.sfda_recurrence(s["q"], s["k"], s["v"], s["alpha"], s["theta"], s["beta"], s["S0"])
    dt = time.perf_counter() - t0
    tokens = n_pairs * T / cfg.H          # a token carries all H heads
    return tokens / dt, dt, recurrence.num_threads()


def run_reference(args, rank):
    """--impl reference: the CPU oracle on a bounded sample; rank 0 only."""
    if rank != 0:
        return
    cfg = workloads.CONFIGS[HEADLINE]
    cores = len(os.sched_getaffinity(0))
    n_pairs, T = max(8, 2 * cores), 2048
    vals, times = [], []
    for i in range(args.warmup + args.steps):
        v, dt, threads = cpu_oracle_throughput(cfg, n_pairs, T)
        if i >= args.warmup:
            vals.append(v)
            times.append(dt)
    value = float(statistics.median(vals))
    sample = "%d (batch, head) sequences x first %d tokens of the headline workload per step" % (n_pairs, T)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * float(statistics.median(times)),
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "T": cfg.T, "H": cfg.H, "d_k": cfg.d_k, "d_v": cfg.d_v,
                   "chunk": cfg.chunk, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--re-only", action="store_true", help="write o = Re only (default: Re and Im)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-decode", action="store_true")
    ap.add_argument("--two-level", action="store_true",
                    help="sweeps only: time sfda_forward_two_level (slices chosen by the library) instead of sfda_forward")
    ap.add_argument("--no-long-context", action="store_true",
                    help="skip the leg that times configuration 3 with and without the two-level scan")
    ap.add_argument("--no-t-sweep", action="store_true",
                    help="skip the leg that times forward and backward at T = 4k, 16k, 64k, 128k")
    ap.add_argument("--no-variants", action="store_true", help="skip the leg that times the write-decoupled forward")
    ap.add_argument("--no-backward", action="store_true", help="skip the leg that times sfda_backward")
    ap.add_argument("--no-factors", action="store_true", help="skip the leg that times sfda_chunk_factors")
    ap.add_argument("--no-fused", action="store_true", help="skip the leg that times the forward on raw inputs")
    ap.add_argument("--seq-len", type=int, default=0,
                    help="sweeps only: run the headline shapes with this sequence length (use with --batch; the JSON "
                         "line then names the changed workload and is not a benchmark value)")
    ap.add_argument("--clock-load-s", type=float, default=1.0,
                    help="seconds of untimed continuation of the same launches under the clock sampler (0: none, "
                         "for profiler runs)")
    ap.add_argument("--batch", type=int, default=0,
                    help="profiling only: run the headline shapes with this batch size instead of 8 "
                         "(the JSON line then names the reduced workload and is not a benchmark value)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else max(args.warmup, 0)

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))

    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import torch.distributed as dist

    import paper_2607_11897_b200 as sfda
    from paper_2607_11897_b200 import dp

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    sfda.load()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    cfg = workloads.CONFIGS[HEADLINE]
    if args.batch > 0:
        cfg = cfg.scaled(name="%s_batch%d_profiling_only" % (cfg.name, args.batch), B=args.batch)
    if args.seq_len > 0:
        cfg = cfg.scaled(name="%s_T%d_sweep_only" % (cfg.name, args.seq_len), T=args.seq_len)
    want_im = not args.re_only
    # every rank draws its own batch: batch elements rank*B .. rank*B + B - 1 of the same recipe
    inp = workloads.forward_inputs(cfg, batch=dp.rank_batch_range(cfg.B, rank))
    host = {}
    for key, val in inp.items():
        t = torch.from_numpy(np.ascontiguousarray(val))
        if key in ("q", "k", "v"):
            t = t.to(torch.bfloat16)
        host[key] = t.pin_memory()
    d = {k: v.to(dev, non_blocking=True) for k, v in host.items()}
    o = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, device=dev, dtype=torch.bfloat16)
    o_im = torch.empty_like(o) if want_im else None
    S_T = torch.empty(cfg.B, cfg.H, cfg.d_k, cfg.d_v, device=dev)
    ws_bytes = sfda.sfda_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, 1)
    if args.two_level:
        ws_bytes = max(ws_bytes, sfda.sfda_forward_two_level_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v,
                                                                              cfg.chunk, 1, 0))
    ws = torch.empty(max(ws_bytes, 256), dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        if args.two_level:      # sweeps only: the library slices the time axis when that pays (few, long sequences)
            sfda.sfda_forward_two_level(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im,
                                        S_T, cfg.chunk, 0, ws, stream)
        else:
            sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, o_im, S_T,
                              cfg.chunk, ws, stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        step()
    launches_per_step = sfda.last_launch_count()
    barrier()
    events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with ClockSampler(local_rank) as clocks:
        barrier()
        start.record(stream)
        for e0, e1 in events:
            e0.record(stream)
            step()
            e1.record(stream)
        stop.record(stream)
        barrier()
        # The timed region lasts tens of milliseconds, too short for nvidia-smi to see: the same launches go on,
        # untimed, under the sampler until it has had about a second of this load.
        t_load = time.perf_counter()
        while args.clock_load_s > 0 and (time.perf_counter() - t_load < args.clock_load_s or
                                         (len(clocks.rows) < 5 and time.perf_counter() - t_load < 4.0)):
            for _ in range(20):
                step()
            torch.cuda.synchronize()
    total_ms = start.elapsed_time(stop)
    kernel_ms = [e0.elapsed_time(e1) for e0, e1 in events]      # one forward = one launch of the chunk kernel
    total_ms = dp.max_over_ranks(total_ms, dev)
    ms_per_step = total_ms / args.steps
    tokens_per_step = world * cfg.B * cfg.T
    value = dp.whole_job_throughput(cfg.B * cfg.T, world, ms_per_step * 1e-3)
    assert sfda.sfda_workspace_status(ws, stream) == 0      # no bounded device-side wait ran out

    # The other output mode beside the quoted one (Re + Im is the paper-literal o; Re only is what a real readout
    # uses).  By now the GPU has run for a second and sits at its power-capped clock, so both modes are timed again,
    # back to back, under the same conditions.
    other_mode = None
    if rank == 0:
        alt_im = None if want_im else torch.empty_like(o)

        def timed_mode(im):
            for _ in range(3):
                sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, im, S_T,
                                  cfg.chunk, ws, stream)
            a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a0.record(stream)
            for _ in range(max(args.steps, 10)):
                sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], o, im, S_T,
                                  cfg.chunk, ws, stream)
            a1.record(stream)
            torch.cuda.synchronize()
            return a0.elapsed_time(a1) / max(args.steps, 10)

        quoted_ms = timed_mode(o_im)
        alt_ms = timed_mode(alt_im)
        alt_bytes = algorithmic_bytes(cfg, not want_im)
        other_mode = {"outputs": "Re" if want_im else "Re+Im", "ms_per_step": alt_ms,
                      "tokens_per_s": cfg.B * cfg.T / (alt_ms * 1e-3), "algorithmic_bytes": alt_bytes,
                      "achieved_gbs": alt_bytes / (alt_ms * 1e-3) / 1e9,
                      "quoted_mode_ms_per_step_same_conditions": quoted_ms,
                      "note": "both modes timed back to back after about a second of load (power-capped clock)"}
        del alt_im

    # end to end through the host-buffer entry point: H2D of the inputs and D2H of the results inside the timing
    e2e = None
    if args.e2e_steps > 0:
        oh = torch.empty(cfg.B, cfg.T, cfg.H, cfg.d_v, dtype=torch.bfloat16).pin_memory()
        oh_im = torch.empty_like(oh).pin_memory() if want_im else None
        Sh = torch.empty(cfg.B, cfg.H, cfg.d_k, cfg.d_v).pin_memory()
        n = sfda.sfda_forward_host_arena_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, cfg.chunk, 1, want_im, True, True)
        arena = torch.empty(n, dtype=torch.uint8, device=dev)
        h2d = d2h = 0
        for i in range(1 + args.e2e_steps):
            if i == 1:
                barrier()
                t0 = time.perf_counter()
            h2d, d2h = sfda.sfda_forward_host(host["q"], host["k"], host["v"], host["alpha"], host["theta"],
                                              host["beta"], host["S0"], oh, oh_im, Sh, cfg.chunk, arena, stream)
            stream.synchronize()
        barrier()
        e2e_s = dp.max_over_ranks((time.perf_counter() - t0) / args.e2e_steps, dev)
        e2e = {"value": tokens_per_step / e2e_s, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": 1e3 * e2e_s}
        del arena

    # The forward on raw inputs (stable parameterisation fused into the operand preparation) beside the two-step
    # route it replaces: sfda_frontend writing alpha, theta, beta and the normalised key, then sfda_forward.
    fused = None
    if rank == 0 and not args.no_fused:
        raw = workloads.forward_raw_inputs(cfg)
        r = {}
        for key, val in raw.items():
            t = torch.from_numpy(np.ascontiguousarray(val))
            r[key] = (t.to(torch.bfloat16) if key in ("q", "k_raw", "v") else t).to(dev)
        del raw
        par = (0.0, 1.0, math.pi, 1e-6)
        al, th = torch.empty_like(r["a_raw"]), torch.empty_like(r["a_raw"])
        be, kn = torch.empty_like(r["c_raw"]), torch.empty_like(r["k_raw"])

        def timed(fn, n):
            for _ in range(3):
                fn()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0.record(stream)
            for _ in range(n):
                fn()
            t1.record(stream)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / n

        fused_ms = timed(lambda: sfda.sfda_forward_fused(r["q"], r["k_raw"], r["v"], r["a_raw"], r["b_raw"],
                                                         r["c_raw"], *par, r["S0"], o, o_im, S_T, cfg.chunk, ws,
                                                         stream), max(args.steps, 5))
        assert sfda.sfda_workspace_status(ws, stream) == 0
        front_ms = timed(lambda: sfda.sfda_frontend(r["a_raw"], r["b_raw"], r["c_raw"], r["k_raw"], *par, al, th, be,
                                                    kn, stream), max(args.steps, 5))
        two_ms = timed(lambda: (sfda.sfda_frontend(r["a_raw"], r["b_raw"], r["c_raw"], r["k_raw"], *par, al, th, be,
                                                   kn, stream),
                                sfda.sfda_forward(r["q"], kn, r["v"], al, th, be, r["S0"], o, o_im, S_T, cfg.chunk,
                                                  ws, stream)), max(args.steps, 5))
        # the derivative of the parameterisation (gradients in place: al, th, be, kn serve as incoming gradients)
        fb_ms = timed(lambda: sfda.sfda_frontend_backward(r["a_raw"], r["b_raw"], r["c_raw"], r["k_raw"], *par, al, th, be,
                                                          kn, al, th, be, kn, stream), max(args.steps, 5))
        rows = cfg.B * cfg.T * cfg.H
        fbytes = rows * 2 * (2 * cfg.m * 4 + 4 + cfg.d_k * 2)          # every array read once, written once
        fused = {"workload": cfg.name + " from raw a, b, c, k (alpha in [0,1], theta_max = pi, eps = 1e-6)",
                 "fused_ms_per_step": fused_ms, "fused_tokens_per_s": cfg.B * cfg.T / (fused_ms * 1e-3),
                 "frontend_kernel_ms": front_ms, "frontend_bytes": fbytes,
                 "frontend_achieved_gbs": fbytes / (front_ms * 1e-3) / 1e9,
                 "frontend_backward_kernel_ms": fb_ms, "frontend_backward_bytes": fbytes * 3 // 2,
                 "frontend_backward_achieved_gbs": fbytes * 1.5 / (fb_ms * 1e-3) / 1e9,
                 "two_step_ms_per_step": two_ms, "two_step_tokens_per_s": cfg.B * cfg.T / (two_ms * 1e-3)}
        del r, al, th, be, kn

    # few, long sequences (configuration 3: 16 sequences of 131072 tokens): the plain forward, one serial chain per
    # sequence, beside the two-level scan over time slices
    longctx = None
    if rank == 0 and not args.no_long_context:
        lcfg = workloads.CONFIGS[3]
        linp = workloads.forward_inputs(lcfg)
        ld = {}
        for key, val in linp.items():
            if val is None:
                ld[key] = None
                continue
            t = torch.from_numpy(np.ascontiguousarray(val))
            ld[key] = (t.to(torch.bfloat16) if key in ("q", "k", "v") else t).to(dev)
        del linp
        lo = torch.empty(lcfg.B, lcfg.T, lcfg.H, lcfg.d_v, device=dev, dtype=torch.bfloat16)
        lo_im = torch.empty_like(lo)
        lS = torch.empty(lcfg.B, lcfg.H, lcfg.d_k, lcfg.d_v, device=dev)
        lws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(lcfg.B, lcfg.T, lcfg.H, lcfg.d_k, lcfg.d_v,
                                                                      lcfg.chunk, 1, 0), dtype=torch.uint8, device=dev)

        def timed3(fn):
            fn()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0.record(stream)
            for _ in range(3):
                fn()
            t1.record(stream)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1) / 3

        plain_ms = timed3(lambda: sfda.sfda_forward(ld["q"], ld["k"], ld["v"], ld["alpha"], ld["theta"], ld["beta"],
                                                    ld["S0"], lo, lo_im, lS, lcfg.chunk, lws, stream))
        two_ms = timed3(lambda: sfda.sfda_forward_two_level(ld["q"], ld["k"], ld["v"], ld["alpha"], ld["theta"],
                                                            ld["beta"], ld["S0"], lo, lo_im, lS, lcfg.chunk, 0, lws,
                                                            stream))
        assert sfda.sfda_workspace_status(lws, stream) == 0
        two_launches = sfda.last_launch_count()
        # the backward pass on the same few sequences: the value columns are split over 4 CTAs per sequence
        lb_ms, lb_launches = None, None
        try:
            lg = [torch.empty_like(ld[key]) for key in ("q", "k", "v", "alpha", "theta", "beta")] + [torch.empty_like(lS)]
            lbws = torch.empty(sfda.sfda_backward_workspace_bytes(lcfg.B, lcfg.T, lcfg.H, lcfg.d_k, lcfg.d_v, 1),
                               dtype=torch.uint8, device=dev)

            def lbstep():
                sfda.sfda_backward(ld["q"], ld["k"], ld["v"], ld["alpha"], ld["theta"], ld["beta"], ld["S0"], lo, lo_im,
                                   lS, *lg, lbws, stream)

            lbstep()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0.record(stream)
            lbstep()
            t1.record(stream)
            torch.cuda.synchronize()
            lb_ms, lb_launches = t0.elapsed_time(t1), sfda.last_launch_count()
            del lg, lbws
        except torch.cuda.OutOfMemoryError:
            pass                                      # reported as null: not enough free device memory
        longctx = {"workload": lcfg.name + " (B=1, T=131072, H=16)", "plain_ms_per_step": plain_ms,
                   "plain_tokens_per_s": lcfg.B * lcfg.T / (plain_ms * 1e-3), "two_level_ms_per_step": two_ms,
                   "two_level_tokens_per_s": lcfg.B * lcfg.T / (two_ms * 1e-3),
                   "two_level_launches": two_launches, "workspace_bytes": int(lws.numel()),
                   "backward_ms_per_call": lb_ms, "backward_launches": lb_launches}
        del ld, lo, lo_im, lS, lws

    # sequence-length sweep of the kernel benchmark protocol (App. E): T = 4k, 16k, 64k, 128k at d_k = d_v = 128,
    # C = 64, H = 32, with B chosen for the headline's 65536 tokens per head (one sequence at 128k: twice that).
    # Inputs drawn on the device with the distributions of configuration 1.
    t_sweep = None
    if rank == 0 and not args.no_t_sweep and args.batch == 0 and args.seq_len == 0:
        t_sweep = []

        def sweep_point(Ts):
            Bs, Hs, dk, dv, ch = max(1, 65536 // Ts), cfg.H, cfg.d_k, cfg.d_v, cfg.chunk
            gs = torch.Generator(device=dev)
            gs.manual_seed(Ts)
            rn = lambda *shape: torch.randn(*shape, device=dev, generator=gs)
            sq, sv = rn(Bs, Ts, Hs, dk).to(torch.bfloat16), rn(Bs, Ts, Hs, dv).to(torch.bfloat16)
            sk = torch.nn.functional.normalize(rn(Bs, Ts, Hs, dk), dim=-1).to(torch.bfloat16)
            sal = torch.sigmoid(3.0 + rn(Bs, Ts, Hs, dk // 2))
            sth = (torch.rand(Bs, Ts, Hs, dk // 2, device=dev, generator=gs) * 2.0 - 1.0) * math.pi
            sbe = torch.sigmoid(rn(Bs, Ts, Hs))
            so, so_im = torch.empty_like(sv), torch.empty_like(sv)
            sS = torch.empty(Bs, Hs, dk, dv, device=dev)
            sws = torch.empty(sfda.sfda_forward_two_level_workspace_bytes(Bs, Ts, Hs, dk, dv, ch, 1, 0),
                              dtype=torch.uint8, device=dev)

            def timed(fn, reps):
                fn()
                t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                t0.record(stream)
                for _ in range(reps):
                    fn()
                t1.record(stream)
                torch.cuda.synchronize()
                return t0.elapsed_time(t1) / reps

            f_ms = timed(lambda: sfda.sfda_forward(sq, sk, sv, sal, sth, sbe, None, so, so_im, sS, ch, sws, stream), 3)
            assert sfda.sfda_workspace_status(sws, stream) == 0
            # slices chosen by the library: with enough sequences this is the same single launch
            f2_ms = timed(lambda: sfda.sfda_forward_two_level(sq, sk, sv, sal, sth, sbe, None, so, so_im, sS, ch, 0, sws,
                                                              stream), 3)
            f2_launches = sfda.last_launch_count()
            assert sfda.sfda_workspace_status(sws, stream) == 0
            sg = [torch.empty_like(x) for x in (sq, sk, sv, sal, sth, sbe)] + [torch.empty_like(sS)]
            sbws = torch.empty(sfda.sfda_backward_workspace_bytes(Bs, Ts, Hs, dk, dv, 1), dtype=torch.uint8, device=dev)
            b_ms = timed(lambda: sfda.sfda_backward(sq, sk, sv, sal, sth, sbe, None, so, so_im, sS, *sg, sbws, stream), 1)
            # the protocol's other chunk size (an exact superchunk of two 64-token tiles: same kernel, same launch)
            f128_ms = timed(lambda: sfda.sfda_forward(sq, sk, sv, sal, sth, sbe, None, so, so_im, sS, 128, sws, stream), 3)
            pcfg = cfg.scaled(B=Bs, T=Ts)
            best = min(f_ms, f2_ms)
            return {"T": Ts, "B": Bs, "H": Hs, "forward_ms": f_ms, "forward_two_level_auto_ms": f2_ms,
                    "forward_chunk128_ms": f128_ms,
                    "forward_tflops": algorithmic_flops(pcfg) / (best * 1e-3) / 1e12,
                    "forward_gbs": algorithmic_bytes(pcfg) / (best * 1e-3) / 1e9,
                    "forward_workspace_bytes": int(sws.numel()), "backward_workspace_bytes": int(sbws.numel()),
                    "two_level_launches": f2_launches, "backward_ms": b_ms,
                    "forward_tokens_per_s": Bs * Ts / (min(f_ms, f2_ms) * 1e-3),
                    "backward_tokens_per_s": Bs * Ts / (b_ms * 1e-3)}

        for Ts in (4096, 16384, 65536, 131072):      # (a point's buffers are released when its function returns)
            try:
                t_sweep.append(sweep_point(Ts))
            except torch.cuda.OutOfMemoryError:
                t_sweep.append({"T": Ts, "skipped": "not enough free device memory for this point"})
            torch.cuda.empty_cache()

    # backward pass (sfda_backward) on the headline inputs: token-level fp32 adjoint, a first correct path
    bwd = None
    if rank == 0 and not args.no_backward:
        g = torch.Generator(device=dev)
        g.manual_seed(1234)
        d_o = torch.randn(o.shape, device=dev, generator=g).to(torch.bfloat16)
        d_oi = torch.randn(o.shape, device=dev, generator=g).to(torch.bfloat16) if want_im else None
        dS_T = torch.randn(S_T.shape, device=dev, generator=g)
        dq, dk, dv_ = torch.empty_like(d["q"]), torch.empty_like(d["k"]), torch.empty_like(d["v"])
        dal, dth, dbe = torch.empty_like(d["alpha"]), torch.empty_like(d["theta"]), torch.empty_like(d["beta"])
        dS0 = torch.empty_like(S_T)
        bws = torch.empty(sfda.sfda_backward_workspace_bytes(cfg.B, cfg.T, cfg.H, cfg.d_k, cfg.d_v, 1),
                          dtype=torch.uint8, device=dev)

        def bstep():
            sfda.sfda_backward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"], d["S0"], d_o, d_oi, dS_T,
                               dq, dk, dv_, dal, dth, dbe, dS0, bws, stream)

        bstep()
        b0, b1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        b0.record(stream)
        for _ in range(2):
            bstep()
        b1.record(stream)
        torch.cuda.synchronize()
        b_ms = b0.elapsed_time(b1) / 2
        rows = cfg.B * cfg.T * cfg.H
        # inputs and cotangents read once, gradients written once (what an ideal backward moves)
        bb = rows * ((2 * cfg.d_k + cfg.d_v) * 2 + 2 * cfg.m * 4 + 4) * 2 + rows * cfg.d_v * 2 * (2 if want_im else 1) \
            + 3 * cfg.B * cfg.H * cfg.d_k * cfg.d_v * 4
        bwd = {"workload": cfg.name + " (gradients of all inputs)", "ms_per_call": b_ms,
               "tokens_per_s": cfg.B * cfg.T / (b_ms * 1e-3), "algorithmic_bytes": bb,
               "achieved_gbs": bb / (b_ms * 1e-3) / 1e9, "workspace_bytes": int(bws.numel()),
               "note": "token-level adjoint in fp32 on the CUDA cores, one CTA per (batch, head) pair"}
        del d_o, d_oi, dS_T, dq, dk, dv_, dal, dth, dbe, dS0, bws

    # forward of the write-decoupled variant (token-level fp32 reference path) on the headline inputs
    variant = None
    if rank == 0 and not args.no_variants:
        gv = torch.Generator(device=dev)
        gv.manual_seed(99)
        r_w = (0.1 * torch.randn(d["k"].shape, device=dev, generator=gv)).to(torch.bfloat16)
        eta_w = torch.rand(d["beta"].shape, device=dev, generator=gv)

        def vstep():
            sfda.sfda_forward_decoupled(d["q"], d["k"], r_w, d["v"], d["alpha"], d["theta"], eta_w, d["beta"], d["S0"],
                                        o, o_im, S_T, stream)

        vstep()
        v0, v1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        v0.record(stream)
        for _ in range(2):
            vstep()
        v1.record(stream)
        torch.cuda.synchronize()
        v_ms = v0.elapsed_time(v1) / 2
        # the same with 2 x 2 rotation / reflection control blocks and the real rank-one erase
        flip_w = (torch.rand(d["alpha"].shape, device=dev, generator=gv) < 0.3).to(torch.uint8)

        def bstep_():
            sfda.sfda_forward_blocks(d["q"], d["k"], r_w, d["v"], d["alpha"], d["theta"], flip_w, eta_w, d["beta"],
                                     d["S0"], o, o_im, S_T, sfda.ERASE_REAL, stream)

        bstep_()
        torch.cuda.synchronize()
        v0.record(stream)
        for _ in range(2):
            bstep_()
        v1.record(stream)
        torch.cuda.synchronize()
        vb_ms = v0.elapsed_time(v1) / 2
        variant = {"workload": cfg.name + " with a separate write direction r and erase strength eta",
                   "ms_per_step": v_ms, "tokens_per_s": cfg.B * cfg.T / (v_ms * 1e-3),
                   "reflection_blocks_real_erase_ms_per_step": vb_ms,
                   "note": "token-level fp32 reference path; the chunk kernels compute the tied model only"}
        del r_w, eta_w, flip_w

    # per-chunk factor export (sfda_chunk_factors) on the headline inputs: Gamma, Y, M, W and the phase turns
    factors = None
    if rank == 0 and not args.no_factors:
        NC = (cfg.T + cfg.chunk - 1) // cfg.chunk
        G = torch.empty(cfg.B, cfg.H, NC, cfg.m, 2, device=dev)
        Yf = torch.empty(cfg.B, cfg.H, NC, cfg.m, cfg.chunk, 2, device=dev)
        Wf = torch.empty_like(Yf)
        Mf = torch.empty(cfg.B, cfg.H, NC, cfg.chunk, cfg.chunk, 2, device=dev)
        turns = torch.empty(cfg.B, cfg.T, cfg.H, cfg.m, device=dev, dtype=torch.int32)

        def fstep():
            sfda.sfda_chunk_factors(d["k"], d["alpha"], d["theta"], d["beta"], G, Yf, Mf, Wf, turns, cfg.chunk, stream)

        for _ in range(2):
            fstep()
        nf = 3
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        f0.record(stream)
        for _ in range(nf):
            fstep()
        f1.record(stream)
        torch.cuda.synchronize()
        f_ms = f0.elapsed_time(f1) / nf
        rows = cfg.B * cfg.T * cfg.H
        fb = rows * (cfg.d_k * 2 + 2 * cfg.m * 4 + 4) + sum(t.numel() * 4 for t in (G, Yf, Wf, Mf, turns))
        factors = {"workload": cfg.name + " (k, alpha, theta, beta -> Gamma, Y, M, W, phase turns)",
                   "ms_per_call": f_ms, "chunks_per_s": cfg.B * cfg.H * NC / (f_ms * 1e-3),
                   "algorithmic_bytes": fb, "achieved_gbs": fb / (f_ms * 1e-3) / 1e9}
        del G, Yf, Wf, Mf
        # the kernel-benchmark protocol's other chunk size (App. E: C in {64, 128}): the forward runs a 128-token chunk as
        # an exact superchunk of two 64-token tiles (same launch, timed for the record), the factor export composes the
        # 128-token factors out of the tiles' (two launches)
        if cfg.T % 128 == 0:
            NC2 = cfg.T // 128
            G2 = torch.empty(cfg.B, cfg.H, NC2, cfg.m, 2, device=dev)
            Y2 = torch.empty(cfg.B, cfg.H, NC2, cfg.m, 128, 2, device=dev)
            W2 = torch.empty_like(Y2)
            M2 = torch.empty(cfg.B, cfg.H, NC2, 128, 128, 2, device=dev)

            def timed_n(fn, n):
                for _ in range(2):
                    fn()
                g0, g1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                torch.cuda.synchronize()
                g0.record(stream)
                for _ in range(n):
                    fn()
                g1.record(stream)
                torch.cuda.synchronize()
                return g0.elapsed_time(g1) / n

            f128_ms = timed_n(lambda: sfda.sfda_chunk_factors(d["k"], d["alpha"], d["theta"], d["beta"], G2, Y2, M2, W2,
                                                              turns, 128, stream), 3)
            fw128_ms = timed_n(lambda: sfda.sfda_forward(d["q"], d["k"], d["v"], d["alpha"], d["theta"], d["beta"],
                                                         d["S0"], o, o_im, S_T, 128, ws, stream), max(args.steps, 5))
            fb2 = rows * (cfg.d_k * 2 + 2 * cfg.m * 4 + 4) + sum(t.numel() * 4 for t in (G2, Y2, W2, M2, turns))
            factors["chunk_128"] = {"factors_ms_per_call": f128_ms, "factors_launches": 2,
                                    "factors_algorithmic_bytes": fb2,
                                    "factors_achieved_gbs": fb2 / (f128_ms * 1e-3) / 1e9,
                                    "forward_ms_per_step": fw128_ms,
                                    "forward_tokens_per_s": cfg.B * cfg.T / (fw128_ms * 1e-3),
                                    "note": "forward: exact superchunk of two 64-token tiles, the kernel and launch of "
                                            "chunk = 64; factors: tile kernel plus composition kernel"}
            del G2, Y2, W2, M2
            if cfg.T % 256 == 0:
                NC4 = cfg.T // 256
                G4 = torch.empty(cfg.B, cfg.H, NC4, cfg.m, 2, device=dev)
                Y4 = torch.empty(cfg.B, cfg.H, NC4, cfg.m, 256, 2, device=dev)
                W4 = torch.empty_like(Y4)
                M4 = torch.empty(cfg.B, cfg.H, NC4, 256, 256, 2, device=dev)
                f256_ms = timed_n(lambda: sfda.sfda_chunk_factors(d["k"], d["alpha"], d["theta"], d["beta"], G4, Y4, M4,
                                                                  W4, turns, 256, stream), 3)
                fb4 = rows * (cfg.d_k * 2 + 2 * cfg.m * 4 + 4) + sum(t.numel() * 4 for t in (G4, Y4, W4, M4, turns))
                factors["chunk_256"] = {"factors_ms_per_call": f256_ms, "factors_launches": 4,
                                        "factors_algorithmic_bytes": fb4,
                                        "factors_achieved_gbs": fb4 / (f256_ms * 1e-3) / 1e9}
                del G4, Y4, W4, M4
        del turns

    # one-token decode (sfda_step) on the decode configuration: HBM-bound, reported beside the headline
    decode = None
    if rank == 0 and not args.no_decode:
        del d, o, o_im
        torch.cuda.empty_cache()
        dcfg = workloads.CONFIGS[4]
        S = torch.from_numpy(workloads.decode_initial_state(dcfg)).to(dev)
        ring = []
        for st in range(8):                                  # eight distinct steps of inputs, cycled
            x = workloads.decode_step_inputs(dcfg, st)
            ring.append({k: (torch.from_numpy(v).to(dev).to(torch.bfloat16) if k in ("q", "k", "v")
                             else torch.from_numpy(v).to(dev)) for k, v in x.items()})
        od = torch.empty(dcfg.B, dcfg.H, dcfg.d_v, device=dev, dtype=torch.bfloat16)
        od_im = torch.empty_like(od)

        def dstep(i):
            x = ring[i % len(ring)]
            sfda.sfda_step(x["q"], x["k"], x["v"], x["alpha"], x["theta"], x["beta"], S, od, od_im, stream)

        for i in range(8):
            dstep(i)
        nd = 200
        d0, d1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        d0.record(stream)
        for i in range(nd):
            dstep(i)
        d1.record(stream)
        torch.cuda.synchronize()
        step_ms = d0.elapsed_time(d1) / nd
        dbytes = dcfg.B * dcfg.H * (2 * dcfg.d_k * dcfg.d_v * 4 + 2 * dcfg.d_k * 2 + dcfg.d_v * 2 + 2 * dcfg.m * 4 + 4
                                     + 2 * dcfg.d_v * 2)
        # the same step on raw inputs of the stable parameterisation (map applied inside the kernel)
        rawd = workloads.forward_raw_inputs(dcfg)
        rd = {k: torch.from_numpy(np.ascontiguousarray(v[:, 0])).to(dev) for k, v in rawd.items() if k != "S0"}
        for k in ("q", "k_raw", "v"):
            rd[k] = rd[k].to(torch.bfloat16)
        for _ in range(8):
            sfda.sfda_step_fused(rd["q"], rd["k_raw"], rd["v"], rd["a_raw"], rd["b_raw"], rd["c_raw"], 0.0, 1.0,
                                 math.pi, 1e-6, S, od, od_im, stream)
        torch.cuda.synchronize()
        d0.record(stream)
        for _ in range(nd):
            sfda.sfda_step_fused(rd["q"], rd["k_raw"], rd["v"], rd["a_raw"], rd["b_raw"], rd["c_raw"], 0.0, 1.0,
                                 math.pi, 1e-6, S, od, od_im, stream)
        d1.record(stream)
        torch.cuda.synchronize()
        fused_step_ms = d0.elapsed_time(d1) / nd
        # and one step of the write-decoupled variant (separate write direction r and erase strength eta)
        gd = torch.Generator(device=dev)
        gd.manual_seed(4321)
        r_dec = (0.1 * torch.randn(dcfg.B, dcfg.H, dcfg.d_k, device=dev, generator=gd)).to(torch.bfloat16)
        eta_dec = torch.rand(dcfg.B, dcfg.H, device=dev, generator=gd)
        x0 = ring[0]
        for _ in range(8):
            sfda.sfda_step_decoupled(x0["q"], x0["k"], r_dec, x0["v"], x0["alpha"], x0["theta"], eta_dec, x0["beta"], S,
                                     od, od_im, stream)
        torch.cuda.synchronize()
        d0.record(stream)
        for i in range(nd):
            x = ring[i % len(ring)]
            sfda.sfda_step_decoupled(x["q"], x["k"], r_dec, x["v"], x["alpha"], x["theta"], eta_dec, x["beta"], S, od,
                                     od_im, stream)
        d1.record(stream)
        torch.cuda.synchronize()
        dec_step_ms = d0.elapsed_time(d1) / nd
        # and with 2 x 2 rotation / reflection control blocks and the real rank-one erase
        flip_dec = (torch.rand(dcfg.B, dcfg.H, dcfg.d_k // 2, device=dev, generator=gd) < 0.3).to(torch.uint8)
        for _ in range(8):
            sfda.sfda_step_blocks(x0["q"], x0["k"], r_dec, x0["v"], x0["alpha"], x0["theta"], flip_dec, eta_dec,
                                  x0["beta"], S, od, od_im, sfda.ERASE_REAL, stream)
        torch.cuda.synchronize()
        d0.record(stream)
        for i in range(nd):
            x = ring[i % len(ring)]
            sfda.sfda_step_blocks(x["q"], x["k"], r_dec, x["v"], x["alpha"], x["theta"], flip_dec, eta_dec, x["beta"], S,
                                  od, od_im, sfda.ERASE_REAL, stream)
        d1.record(stream)
        torch.cuda.synchronize()
        blk_step_ms = d0.elapsed_time(d1) / nd
        decode = {"workload": dcfg.name, "ms_per_step": step_ms, "fused_raw_inputs_ms_per_step": fused_step_ms,
                  "write_decoupled_ms_per_step": dec_step_ms, "reflection_blocks_real_erase_ms_per_step": blk_step_ms,
                  "tokens_per_s": dcfg.B / (step_ms * 1e-3),
                  "algorithmic_bytes_per_step": dbytes, "achieved_gbs": dbytes / (step_ms * 1e-3) / 1e9,
                  "state_bytes": int(S.numel() * 4), "note": "state (537 MB) far larger than L2"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peaks = measured_peaks()
    abytes = algorithmic_bytes(cfg, want_im)
    aflops = algorithmic_flops(cfg, want_im)
    k_ms = float(statistics.mean(kernel_ms))
    achieved_gbs = abytes / (k_ms * 1e-3) / 1e9
    achieved_tf = aflops / (k_ms * 1e-3) / 1e12
    hbm_time = abytes / (peaks["hbm_gbs"] * 1e9)
    tensor_time = aflops / (peaks["bf16_tflops"] * 1e12)
    roofline = {
        "bound": "hbm", "achieved": achieved_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
        "frac": achieved_gbs / peaks["hbm_gbs"], "traffic": None, "peak_source": "of " + peaks["source"],
        "kernel": "sfda_forward chunk kernel (1 launch per step)", "kernel_ms": k_ms, "kernel_ms_median": float(statistics.median(kernel_ms)),
        "kernel_ms_best": float(min(kernel_ms)),
        "algorithmic_bytes": abytes, "algorithmic_flops": aflops, "achieved_tflops": achieved_tf,
        "tensor_frac": achieved_tf / peaks["bf16_tflops"],
        "roofline_ms": 1e3 * max(hbm_time, tensor_time),
    }
    if args.batch == 0 and args.seq_len == 0:
        # dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture of this kernel at B = 4 (1.867 GB,
        # profiles/sfda_forward_ws_kernel_batch4_ncu_full.md), scaled by the units processed (traffic grows with B)
        roofline["traffic"] = 1.867e9 * cfg.B / 4
        roofline["traffic_source"] = "ncu capture at B=4 scaled to B=%d; Re+Im outputs" % cfg.B

    if other_mode is not None:
        other_mode["frac"] = other_mode["achieved_gbs"] / peaks["hbm_gbs"]
    if bwd is not None:
        bwd["frac"] = bwd["achieved_gbs"] / peaks["hbm_gbs"]
        bwd["peak_source"] = "of " + peaks["source"]
    if factors is not None:
        factors["frac"] = factors["achieved_gbs"] / peaks["hbm_gbs"]
        factors["peak_source"] = "of " + peaks["source"]
    if fused is not None:
        fused["frontend_frac"] = fused["frontend_achieved_gbs"] / peaks["hbm_gbs"]
        fused["peak_source"] = "of " + peaks["source"]
    if decode is not None:
        decode["frac"] = decode["achieved_gbs"] / peaks["hbm_gbs"]
        decode["peak_source"] = "of " + peaks["source"]
    cpu = None
    if not args.no_cpu_baseline:
        cores = len(os.sched_getaffinity(0))
        n_pairs, T = max(8, 4 * cores), cfg.T
        v, dt, threads = cpu_oracle_throughput(cfg, n_pairs, T)
        cpu = {"value": v, "unit": UNIT, "cores": threads, "kind": "oracle", "seconds": dt,
               "sample": "%d of the %d (batch, head) sequences, all %d tokens" % (n_pairs, cfg.B * cfg.H, T)}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "bf16", "data": "synthetic",
        "config": {"workload": cfg.name, "B": cfg.B, "T": cfg.T, "H": cfg.H, "d_k": cfg.d_k, "d_v": cfg.d_v,
                   "chunk": cfg.chunk, "outputs": "Re+Im" if want_im else "Re", "state": "fp32", "S0": "N(0,0.02)",
                   "parallelism": "dp%d over (batch, head), no collective" % world,
                   "l2": "inputs+outputs %.2f GB per step, far larger than the 126 MB L2; no flush" % (abytes / 1e9)},
        "roofline": roofline, "cpu_baseline": cpu, "other_output_mode": other_mode, "e2e": e2e, "decode": decode, "fused_front_end": fused, "chunk_factors": factors, "backward": bwd, "write_decoupled_forward": variant, "long_context": longctx, "t_sweep": t_sweep,
        "gpu_launches": launches_per_step * args.steps, "clocks": clocks.summary(),
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
