#!/usr/bin/env python
"""Benchmark of the split-FFN hot path (FFSplit, arXiv 2401.04044) on B200.

Workload (N = 1): the BERT-base-shaped stack -- 12 GELU FFN layers, d = 768,
m = 3072, bf16, heavy k = 154, light rank r = 192, 4096 calibration tokens per
layer, prefill batch 32 x 128 = 4096 tokens.  One step is one pass of the whole
path over that batch: per layer score -> select -> pack, then the 12-layer split
forward.  `value` is forward tokens per second of that whole step; the phases
(forward only, dense comparator, calibration) are reported beside it.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Under torchrun every rank runs the same per-GPU workload (weak scaling, no
data-path collective: the path is token-parallel with replicated weights).
`--impl reference` times the CPU oracle (oracle/) on the host cores on a bounded
sample of the same workload.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

METRIC = "split-FFN tokens/s (prefill, decode) and % of roofline vs dense FFN"
UNIT = "tokens/s"
CFG_ID = 2


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return {"hbm_gbs": j["hbm_gbs"], "bf16_tflops": j["bf16_tflops"],
                "bf16_tflops_sustained": j.get("bf16_tflops_sustained"), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


# --------------------------------------------------------------------------------------
class ClockSampler:
    """nvidia-smi in the background during the timed region."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.tmp = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={gpu_index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=self.tmp, stderr=subprocess.DEVNULL)
        except OSError:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.tmp.flush()
        rows = [l.strip().split(", ") for l in open(self.tmp.name) if l.strip()]
        os.unlink(self.tmp.name)
        sm, reasons, mx = [], set(), None
        for r in rows:
            if len(r) < 9:
                continue
            try:
                sm.append(float(r[1]))
                mx = float(r[2])
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[5:9]):
                if v.strip().lower() == "active":
                    reasons.add(name)
        if sm:
            busy = [v for v in sm if v > 0.5 * max(sm)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=mx, reasons=sorted(reasons), samples=len(sm))
        return out


# --------------------------------------------------------------------------------------
class StackWorkload:
    """Device-resident synthetic stack plus everything one step touches."""

    def __init__(self, cfg, ctx, layers, T, device, cal_lanes=1):
        import torch
        from ffsplit_synth import make_layer
        from paper_2401_04044_b200 import make_shape
        from paper_2401_04044_b200.factors import light_factors
        self.cfg, self.ctx, self.T, self.n_layers = cfg, ctx, T, layers
        self.shape = make_shape(cfg.d, cfg.m, cfg.act, cfg.torch_dtype)
        ws = max(ctx.workspace_size(self.shape, T, cfg.t_cal, cfg.k, cfg.r),
                 ctx.workspace_size(self.shape, T, 0, cfg.m, 0))
        ctx.ensure_workspace(ws)
        # The calibrations of different layers do not depend on one another, and most of their kernels
        # (top-k in one CTA, the small preparation jobs) leave the GPU nearly idle: they are issued round
        # robin on `cal_lanes` streams, each with a library context (workspace, tickets) of its own.
        from paper_2401_04044_b200 import Context
        self.lanes = [(ctx, None)]   # lane 0: the calling stream (forward chain; everything when alone)
        for _ in range(cal_lanes if cal_lanes > 1 else 0):
            c = Context(ctx.device if hasattr(ctx, "device") else 0)
            c.ensure_workspace(c.workspace_size(self.shape, T, cfg.t_cal, cfg.k, cfg.r))
            self.lanes.append((c, torch.cuda.Stream(device=device)))
        self.layers = []
        padded, self.logical_bytes = ctx.pack_size(self.shape, cfg.k, cfg.r)
        padded_dense, self.logical_bytes_dense = ctx.pack_size(self.shape, cfg.m, 0)
        for l in range(layers):
            L = make_layer(cfg, l, device=device)
            e = {"L": L, "Xcal": L.tokens(cfg.t_cal)}
            e["energy"] = torch.empty(cfg.m, dtype=torch.float32, device=device)
            e["scores"] = torch.empty(cfg.m, dtype=torch.float32, device=device)
            e["heavy"] = torch.empty(cfg.k, dtype=torch.int32, device=device)
            e["light"] = torch.empty(cfg.m - cfg.k, dtype=torch.int32, device=device)
            e["blob"] = torch.empty(padded, dtype=torch.uint8, device=device)
            e["blob_dense"] = torch.empty(padded_dense, dtype=torch.uint8, device=device)
            e["Y"] = torch.empty(T, cfg.d, dtype=cfg.torch_dtype, device=device)
            self.layers.append(e)
        self.X = self.layers[0]["L"].tokens(T)
        # set-up (untimed): find each layer's heavy set once, factor its light slices (host-side
        # helper of the step between select and pack), build the dense comparator blobs
        for e in self.layers:
            self.calibrate_layer(e, pack=False)
        ctx.poll()
        all_idx = torch.arange(cfg.m, dtype=torch.int32, device=device)
        for e in self.layers:
            L = e["L"]
            e["heavy_setup"] = e["heavy"].clone()
            e["factors"] = light_factors(L.W1, L.W2, e["light"], cfg.r, L.W1u)
            ctx.pack(self.shape, L.W1, L.b1, L.W2, L.b2, all_idx, cfg.m, None, e["blob_dense"], W1u=L.W1u)
        ctx.poll()

    def calibrate_layer(self, e, pack=True, ctx=None):
        L, cfg, ctx = e["L"], self.cfg, ctx or self.ctx
        ctx.score(self.shape, L.W1, L.b1, L.W2, e["Xcal"], e["energy"], e["scores"], W1u=L.W1u)
        ctx.select(e["scores"], cfg.k, e["heavy"], e["light"])
        if pack:
            ctx.pack(self.shape, L.W1, L.b1, L.W2, L.b2, e["heavy"], cfg.k, e["factors"], e["blob"], W1u=L.W1u)

    def calibrate(self, events=None, before=None):
        """Score, select and pack every layer.  With several lanes the layers go round robin over the
        lanes' streams; `events`, if given, receives one event per layer, recorded behind its pack;
        `before(i)`, if given, is issued on the layer's stream ahead of its calibration (input copies)."""
        import torch
        if len(self.lanes) == 1:
            for i, e in enumerate(self.layers):
                if before is not None:
                    before(i)
                self.calibrate_layer(e)
            return
        main = torch.cuda.current_stream()
        fork = torch.cuda.Event()
        fork.record(main)
        side = self.lanes[1:]
        for _, s in side:
            s.wait_event(fork)
        for i, e in enumerate(self.layers):
            c, s = side[i % len(side)]
            with torch.cuda.stream(s):
                if before is not None:
                    before(i)
                self.calibrate_layer(e, ctx=c)
                if events is not None:
                    ev = torch.cuda.Event()
                    ev.record(s)
                    events.append(ev)
        if events is None:
            for _, s in side:
                join = torch.cuda.Event()
                join.record(s)
                main.wait_event(join)

    def launch_count(self):
        return sum(c.launch_count() for c, _ in self.lanes)

    def poll(self):
        for c, _ in self.lanes:
            c.poll()

    def forward(self, x=None, dense=False):
        x = self.X if x is None else x
        for e in self.layers:
            self.ctx.forward(e["blob_dense"] if dense else e["blob"], x, e["Y"])
            x = e["Y"]
        return x

    def step(self, x=None, before=None):
        """One pass of the whole path.  With several lanes, layer l's forward (on the calling stream) waits
        only for layer l's pack, so the forward chain runs under the calibrations of the later layers."""
        import torch
        if len(self.lanes) == 1:
            self.calibrate(before=before)
            return self.forward(x)
        events = []
        self.calibrate(events, before)
        main = torch.cuda.current_stream()
        x = self.X if x is None else x
        for e, ev in zip(self.layers, events):
            main.wait_event(ev)
            self.ctx.forward(e["blob"], x, e["Y"])
            x = e["Y"]
        return x

    def step_serial(self):
        """The same work on one stream and one context: what the per-kernel profile is taken on."""
        for e in self.layers:
            self.calibrate_layer(e)
        return self.forward()

    def check_selection_stable(self):
        import torch
        for e in self.layers:
            assert torch.equal(e["heavy"], e["heavy_setup"]), "selection changed between set-up and the timed steps"


# DRAM traffic of the tensor-core kernels (gemm_tc_kernel and fused_light_kernel: the launches the roofline
# object covers), average per launch over one step, from an ncu capture of
#   python bench.py --only step --steps 1 --warmup 1 --no-graph --no-cpu-baseline
# (dram__bytes_read.sum + dram__bytes_write.sum, last 48 launches; profiles/gemm_tc_and_fused_light__cfg2_traffic.md).
# Valid only for the kernel sources it was taken with: any change to them turns the field back to null.
TC_TRAFFIC_BYTES_PER_LAUNCH = 6352517
TC_TRAFFIC_SOURCES_SHA256 = "d68080571be2512e39f7db6b01648c105ff7a15b103e4e5d7da2691bfa15d806"
TC_SOURCES = ("gemm_tc.cu", "fused_light.cu", "ptx.cuh", "epilogue.cuh", "internal.h")


def tc_sources_sha256():
    import hashlib
    h = hashlib.sha256()
    for name in TC_SOURCES:
        with open(os.path.join(ROOT, "paper_2401_04044_b200", "csrc", name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()


def measured_traffic():
    if TC_TRAFFIC_BYTES_PER_LAUNCH is None or tc_sources_sha256() != TC_TRAFFIC_SOURCES_SHA256:
        return None
    return TC_TRAFFIC_BYTES_PER_LAUNCH


def time_region(fn, steps, warmup, flush, dist_barrier):
    """W untimed + K timed calls of fn, each timed with CUDA events on the current
    stream, L2 flushed (untimed) before every call.  Returns per-step milliseconds."""
    import torch
    for _ in range(warmup):
        flush()
        fn()
    torch.cuda.synchronize()
    dist_barrier()
    times = []
    for _ in range(steps):
        flush()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        fn()
        b.record()
        b.synchronize()
        times.append(a.elapsed_time(b))
    torch.cuda.synchronize()
    dist_barrier()
    return times


def max_over_ranks(ms: float, world: int, device) -> float:
    """The slowest rank's time for a timed region (every rank gets the same number back)."""
    if world <= 1:
        return ms
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_tokens_per_s(total_ms: float, tokens_per_rank_step: int, steps: int, world: int, device="cpu") -> float:
    """Weak scaling: every rank pushes its own batch through its own replica; the job's
    throughput is all ranks' tokens over the slowest rank's time."""
    slowest = max_over_ranks(total_ms, world, device)
    return world * tokens_per_rank_step * steps / (slowest * 1e-3)


def flops_per_token(cfg, dense=False):
    n_in = cfg.n_in
    if dense:
        return 2.0 * (n_in + 1) * cfg.d * cfg.m
    return 2.0 * (n_in + 1) * (cfg.d * cfg.k + cfg.r * (cfg.d + cfg.m - cfg.k))


def run_ours(args):
    import torch
    import torch.distributed as dist
    from ffsplit_synth import CONFIGS
    from paper_2401_04044_b200 import Context, build

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(f"cuda:{local_rank}"))
    if rank == 0:
        build.build()
    if world > 1:
        dist.barrier()
    torch.cuda.set_device(local_rank)
    device = f"cuda:{local_rank}"
    peaks = load_peaks()

    def barrier():
        if world > 1:
            dist.barrier()

    cfg = CONFIGS[CFG_ID]
    T = cfg.t_fwd[0]
    ctx = Context(local_rank)
    n_layers = args.layers or cfg.layers
    wl = StackWorkload(cfg, ctx, n_layers, T, device, cal_lanes=1 if args.only else args.cal_lanes)
    flush_buf = torch.empty(256 << 20, dtype=torch.uint8, device=device)

    def flush():
        flush_buf.add_(1)

    if args.only:
        # one phase alone, few launches: the form used under a profiler
        wl.calibrate()
        fn = {"step": wl.step, "forward": wl.forward, "dense": lambda: wl.forward(dense=True),
              "calibrate": wl.calibrate}[args.only]
        ms = time_region(fn, args.steps, args.warmup, flush, barrier)
        ctx.poll()
        if rank == 0:
            print(json.dumps({"only": args.only, "layers": n_layers, "tokens": T, "ms_per_call": ms}))
        return

    sampler = ClockSampler(local_rank) if rank == 0 else None
    # The step is launch-bound on the host (about a hundred launches of 5-50 us): capture it once in a
    # CUDA graph and time replays.  --no-graph times the plain stream launches instead.
    wl.step()
    wl.poll()
    n0 = wl.launch_count()
    wl.step()
    launches_per_step = wl.launch_count() - n0
    wl.poll()
    step_fn, launch_mode = wl.step, "stream"
    if not args.no_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                wl.step()
            step_fn, launch_mode = graph.replay, "cuda_graph"
        except Exception as exc:   # capture refused: fall back to stream launches, and say so
            launch_mode = f"stream (graph capture failed: {type(exc).__name__})"
            torch.cuda.synchronize()
    step_ms = time_region(step_fn, args.steps, args.warmup, flush, barrier)
    wl.poll()
    wl.check_selection_stable()
    total_ms = max_over_ranks(sum(step_ms), world, device)
    value = world * T * args.steps / (total_ms * 1e-3)

    # ---- phases, each timed the same way (kernel-only, inputs resident)
    k_ph, w_ph = max(3, min(args.steps, 10)), max(3, min(args.warmup, 3))
    fwd_ms = statistics.median(time_region(wl.forward, k_ph, w_ph, flush, lambda: None))
    dense_ms = statistics.median(time_region(lambda: wl.forward(dense=True), k_ph, w_ph, flush, lambda: None))
    cal_ms = statistics.median(time_region(wl.calibrate, k_ph, w_ph, flush, lambda: None))

    # ---- roofline of the dominant kernel (the tensor-core GEMM, all its launches in a step)
    ctx.profile_begin()
    for _ in range(3):
        flush()
        wl.step_serial()
    n_l, ms_l, flops_l = ctx.profile_end(0)
    achieved = flops_l / (ms_l * 1e-3) / 1e12 if ms_l > 0 else 0.0
    roofline = {"bound": "tensor", "kernel": "gemm_tc_kernel", "achieved": round(achieved, 2),
                "peak": peaks["bf16_tflops"], "unit": "TFLOP/s", "frac": round(achieved / peaks["bf16_tflops"], 4),
                "peak_source": f"{peaks['source']} (burst bf16; kernels of 5-40 us timed one by one)",
                "launches_per_step": n_l // 3, "avg_launch_us": round(1e3 * ms_l / max(n_l, 1), 2),
                "traffic": measured_traffic()}
    ctx.profile_begin()
    for _ in range(3):
        flush()
        wl.forward()
    n_f, ms_f, flops_f = ctx.profile_end(0)
    fwd_tflops = flops_f / (ms_f * 1e-3) / 1e12 if ms_f > 0 else 0.0

    # ---- end to end: host buffers, copies inside the timed region
    Xcal_host = [e["Xcal"].cpu().pin_memory() for e in wl.layers]
    X_host = wl.X.cpu().pin_memory()
    Y_host = torch.empty_like(X_host).pin_memory()
    x_dev = torch.empty_like(wl.X)

    def e2e_step():
        # every layer's calibration tokens are copied on the stream that calibrates that layer, so the
        # copy engine works under the kernels of the other streams
        x_dev.copy_(X_host, non_blocking=True)
        y = wl.step(x_dev, before=lambda i: wl.layers[i]["Xcal"].copy_(Xcal_host[i], non_blocking=True))
        Y_host.copy_(y, non_blocking=True)

    e2e_fn = e2e_step
    if not args.no_graph:
        # the copies are graph nodes like the kernels (pinned host buffers at fixed addresses)
        try:
            e2e_step()
            torch.cuda.synchronize()
            e2e_graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(e2e_graph):
                e2e_step()
            e2e_fn = e2e_graph.replay
        except Exception:
            torch.cuda.synchronize()
            e2e_fn = e2e_step
    e2e_ms = time_region(e2e_fn, k_ph, w_ph, flush, barrier)
    e2e_total = max_over_ranks(sum(e2e_ms), world, device)
    es = 2
    h2d = cfg.layers * cfg.t_cal * cfg.d * es + T * cfg.d * es
    d2h = T * cfg.d * es
    e2e = {"value": world * T * k_ph / (e2e_total * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h}

    # single layer through the host-buffer entry point of the C ABI
    e0 = wl.layers[0]
    host_ms = statistics.median(time_region(lambda: ctx.forward_host(e0["blob"], X_host, Y_host), k_ph, w_ph, flush,
                                            lambda: None))
    ctx.poll()
    clocks = sampler.stop() if sampler else None

    if rank == 0:
        roof_t = flops_per_token(cfg) * T / (peaks["bf16_tflops"] * 1e12) * 1e3          # ms per layer
        roof_t_dense = flops_per_token(cfg, True) * T / (peaks["bf16_tflops"] * 1e12) * 1e3
        out = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": "configs[1]: BERT-base-shaped stack, 12 GELU FFN layers, d=768 m=3072 k=154 r=192, "
                                   "4096 calibration tokens/layer, prefill 32x128=4096 tokens; step = score+select+pack "
                                   "per layer, then the 12-layer split forward",
                       "l2": "256 MiB buffer rewritten before every timed step (L2 flush)",
                       "launch": launch_mode, "calibration_streams": max(1, len(wl.lanes) - 1),
                       "tokens_per_step": T, "layers": cfg.layers},
            "roofline": roofline,
            "e2e": e2e,
            "gpu_launches": int(launches_per_step * args.steps),
            "gpu_launches_per_step": int(launches_per_step),
            "clocks": clocks,
            "phases": {
                "forward_split_ms_per_stack": fwd_ms, "forward_dense_ms_per_stack": dense_ms,
                "calibrate_ms_per_stack": cal_ms,
                "forward_split_tokens_per_s_per_stack": T / (fwd_ms * 1e-3),
                "forward_split_tokens_per_s_per_layer": T * cfg.layers / (fwd_ms * 1e-3),
                "forward_dense_tokens_per_s_per_stack": T / (dense_ms * 1e-3),
                "split_vs_dense_speedup": dense_ms / fwd_ms,
                "forward_split_roofline_frac": roof_t * cfg.layers / fwd_ms,
                "forward_dense_roofline_frac": roof_t_dense * cfg.layers / dense_ms,
                "forward_split_gemm_tflops": round(fwd_tflops, 2),
                "forward_host_one_layer_ms": host_ms,
                "model_bytes_split_per_layer": wl.logical_bytes, "model_bytes_dense_per_layer": wl.logical_bytes_dense,
            },
            "paper_context": "43.1% fewer parameters and 1.25-1.56x whole-model BERT-base speedup on V100 / Xeon "
                             "(Section 5.1); other hardware, not a target",
        }
        if world == 1 and not args.no_cpu_baseline:
            out["cpu_baseline"] = cpu_baseline_sample(cfg, T, layers_sample=cfg.layers, reps=2)
        print(json.dumps(out))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------
def oracle_layer_setup(cfg, layer):
    """Inputs of one layer for the oracle arm, as float64 numpy (exact up-casts), with
    the light factors it will use (set-up, untimed: the SVD is not on the hot path)."""
    import numpy as np
    from ffsplit_synth import make_layer
    from oracle import ffsplit_oracle as orc
    L = make_layer(cfg, layer)
    f = lambda t: None if t is None else t.double().numpy()
    W = {"W1": f(L.W1), "b1": f(L.b1), "W2": f(L.W2), "b2": f(L.b2)}
    Xcal = f(L.tokens(cfg.t_cal))
    sw = orc.split_weights(W["W1"], W["b1"], W["W2"], L.planted.numpy())
    fac = {}
    fac["A1"], fac["B1"] = orc.light_factors(sw["U2"], cfg.r)
    fac["A2"], fac["B2"] = orc.light_factors(sw["V2"], cfg.r)
    rnd = lambda a: np.asarray(__import__("torch").from_numpy(a).to(cfg.torch_dtype).double().numpy())
    fac = {k: rnd(v) for k, v in fac.items()}
    return W, Xcal, fac


def oracle_layer_step(cfg, W, Xcal, fac, X):
    from oracle import ffsplit_oracle as orc
    _, _, s = orc.neuron_scores(Xcal, W["W1"], W["b1"], W["W2"], cfg.act)
    heavy, _ = orc.select_heavy(s, cfg.k)
    return orc.split_ffn(X, W["W1"], W["b1"], W["W2"], W["b2"], heavy, fac, cfg.act)


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        return max(n) if n else (os.cpu_count() or 1)
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline_sample(cfg, T, layers_sample=12, reps=2):
    import numpy as np
    rng = np.random.default_rng(0)
    X = rng.standard_normal((T, cfg.d))
    layers_sample = min(layers_sample, cfg.layers)
    setups = [oracle_layer_setup(cfg, l) for l in range(layers_sample)]
    best = None
    for _ in range(reps):
        t0 = time.perf_counter()
        x = X
        for W, Xcal, fac in setups:
            x = oracle_layer_step(cfg, W, Xcal, fac, x)
        dt = time.perf_counter() - t0
        best = dt if best is None else min(best, dt)
    per_stack = best * cfg.layers / layers_sample
    return {"value": T / per_stack, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{layers_sample} of {cfg.layers} layers (score over {cfg.t_cal} calibration tokens + select + "
                      f"split forward of all {T} tokens, fp64 numpy), best of {reps} passes, time scaled by {cfg.layers}/{layers_sample}",
            "seconds_sampled": best * reps}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import numpy as np
    from ffsplit_synth import CONFIGS
    cfg = CONFIGS[CFG_ID]
    T = cfg.t_fwd[0]
    n_setups = 2
    setups = [oracle_layer_setup(cfg, l) for l in range(n_setups)]
    X = np.random.default_rng(0).standard_normal((T, cfg.d))
    times = []
    for i in range(args.warmup + args.steps):
        W, Xcal, fac = setups[i % n_setups]
        t0 = time.perf_counter()
        oracle_layer_step(cfg, W, Xcal, fac, X)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    per_step = sum(times) / len(times) * cfg.layers        # one sampled layer per step, scaled to the stack
    value = T / per_step
    sample = (f"each step = 1 of {cfg.layers} layers (score over {cfg.t_cal} calibration tokens + select + split "
              f"forward of all {T} tokens, fp64 numpy), time scaled by {cfg.layers}")
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": int(os.environ.get("WORLD_SIZE", "1")),
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_step * 1e3, "higher_is_better": True,
           "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
           "config": {"workload": "configs[1]: BERT-base-shaped stack, 12 GELU FFN layers, d=768 m=3072 k=154 r=192, "
                                  "4096 calibration tokens/layer, prefill 4096 tokens (CPU oracle, bounded sample)"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": sample},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="time plain stream launches instead of a CUDA-graph replay")
    ap.add_argument("--cal-lanes", type=int, default=3,
                    help="streams (each with its own library context) the per-layer calibrations are spread over")
    ap.add_argument("--only", default=None, choices=["step", "forward", "dense", "calibrate"],
                    help="run one phase alone and print its times (for profiler captures)")
    ap.add_argument("--layers", type=int, default=0, help="with --only: number of layers of the stack to build")
    args = ap.parse_args()
    if args.impl == "ours" and not args.only:
        args.warmup = max(args.warmup, 3)
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
