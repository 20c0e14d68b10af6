"""Throughput sweep over the synthetic configurations: split vs dense forward per
FFN layer (prefill and few-token sizes), scoring, and model size.

    python sweep.py --config 5 --tokens 1 32 4096 --out sweep_cfg5.jsonl

One JSON line per point: tokens/s per layer and per stack, achieved fraction of
the roofline (the slower of FLOPs at the bf16 tensor peak and bytes at the HBM
peak), split vs dense speed-up, logical model bytes.  Layers are timed on
distinct weight copies cycled so that consecutive calls do not find their
weights in L2.  Light factors for timing runs are random (their values do not
change the work); parity tests use true SVD factors.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import time
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from ffsplit_synth import CFG5_HEAVY_PERCENT, CFG5_RANKS, CONFIGS, cfg5_point, make_layer  # noqa: E402
from paper_2401_04044_b200 import Context, build, make_shape  # noqa: E402
from paper_2401_04044_b200.factors import light_factors  # noqa: E402


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        j = json.load(open(p))
        return j["hbm_gbs"], j["bf16_tflops"], "measured", j.get("bf16_tflops_sustained", j["bf16_tflops"])
    return 6650.0, 1590.0, "fallback", 1400.0


def random_factors(cfg, device, gen):
    d, ml, r, dt = cfg.d, cfg.m - cfg.k, cfg.r, cfg.torch_dtype
    mk = lambda *s: (torch.randn(*s, generator=gen, device=device, dtype=torch.float32) * 0.02).to(dt)
    f = {"A1": mk(d, r), "B1": mk(r, ml), "A2": mk(ml, r), "B2": mk(r, d)}
    if cfg.act == "swiglu":
        f["A1u"], f["B1u"] = mk(d, r), mk(r, ml)
    return f


def time_calls(fn, batch, reps, warmup, use_graph=True, settle=0.0):
    """Milliseconds per call of `fn`, one sample per timed batch of `batch` consecutive calls.

    A single few-token forward lasts tens of microseconds, less than the host needs to issue it, so
    the batch is recorded once into a CUDA graph and the replays are timed (device events around each
    replay); with use_graph=False, or if the capture fails, the batch is issued call by call."""
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    run = lambda: [fn() for _ in range(batch)]
    mode = "stream"
    if use_graph:
        try:
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph):
                run()
            run, mode = graph.replay, "cuda_graph"
        except Exception as exc:  # capture not possible: time the plain launches
            torch.cuda.synchronize()
            mode = f"stream (graph capture failed: {type(exc).__name__})"
    run()
    torch.cuda.synchronize()
    if settle > 0:
        # a long tensor-bound case leaves the SM clock power-capped for a while: let it recover, then warm up
        time.sleep(settle)
        run()
        torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        run()
        b.record()
        b.synchronize()
        ts.append(a.elapsed_time(b) / batch)
    return ts, mode


def run_point(ctx, cfg, tokens, copies, reps, svd, device="cuda", use_graph=True, which=("split", "dense"), settle=0.0):
    hbm, tf, src, tf_sus = peaks()
    shape = make_shape(cfg.d, cfg.m, cfg.act, cfg.torch_dtype)
    es = 2 if cfg.dtype == "bf16" else 4
    Tmax = max(tokens)
    ctx.ensure_workspace(max(ctx.workspace_size(shape, Tmax, 0, cfg.k, cfg.r), ctx.workspace_size(shape, Tmax, 0, cfg.m, 0)))
    padded, logical = ctx.pack_size(shape, cfg.k, cfg.r)
    padded_d, logical_d = ctx.pack_size(shape, cfg.m, 0)
    blobs, blobs_d = [], []
    gen = torch.Generator(device=device)
    gen.manual_seed(1234)
    all_idx = torch.arange(cfg.m, dtype=torch.int32, device=device)
    for c in range(copies):
        L = make_layer(cfg, c, device=device)
        heavy = L.planted.to(torch.int32)
        if svd:
            mask = torch.ones(cfg.m, dtype=torch.bool, device=device)
            mask[heavy.long()] = False
            fac = light_factors(L.W1, L.W2, torch.nonzero(mask).flatten(), cfg.r, L.W1u)
        else:
            fac = random_factors(cfg, device, gen)
        b = torch.empty(padded, dtype=torch.uint8, device=device)
        ctx.pack(shape, L.W1, L.b1, L.W2, L.b2, heavy, cfg.k, fac, b, W1u=L.W1u)
        bd = torch.empty(padded_d, dtype=torch.uint8, device=device)
        ctx.pack(shape, L.W1, L.b1, L.W2, L.b2, all_idx, cfg.m, None, bd, W1u=L.W1u)
        ctx.poll()
        blobs.append(b)
        blobs_d.append(bd)
        del L, fac
    out = []
    n_in = cfg.n_in
    for T in tokens:
        X = (torch.randn(T, cfg.d, generator=gen, device=device, dtype=torch.float32)).to(cfg.torch_dtype)
        Y = torch.empty_like(X)
        res = {"config": cfg.name, "d": cfg.d, "m": cfg.m, "k": cfg.k, "r": cfg.r, "act": cfg.act, "dtype": cfg.dtype,
               "tokens": T, "layers": cfg.layers, "weight_copies_cycled": copies, "peaks": src}
        for name, bl, params, lbytes in (("split", blobs, (n_in + 1) * (cfg.d * cfg.k + cfg.r * (cfg.d + cfg.m - cfg.k)), logical),
                                        ("dense", blobs_d, (n_in + 1) * cfg.d * cfg.m, logical_d)):
            if name not in which:
                continue
            state = {"i": 0}

            def call():
                ctx.forward(bl[state["i"] % copies], X, Y)
                state["i"] += 1

            # every batch walks all weight copies (more than L2 holds) the same number of times
            ts, mode = time_calls(call, copies * max(1, 16 // copies), reps, max(3, copies), use_graph, settle)
            ctx.poll()
            res["launch_mode"] = mode
            ms = statistics.median(ts)
            flops = 2.0 * params * T
            bytes_ = es * (params + cfg.m + cfg.d) + 2 * T * cfg.d * es
            roof_ms = max(flops / (tf * 1e12), bytes_ / (hbm * 1e9)) * 1e3
            res[name] = {"ms_per_layer": ms, "ms_best": min(ts), "tokens_per_s_per_layer": T / (ms * 1e-3),
                         "tokens_per_s_per_stack": T / (ms * 1e-3 * cfg.layers), "roofline_ms": roof_ms,
                         "roofline_frac": roof_ms / ms,
                         # the timed batches run back to back for tens of milliseconds: against the sustained peak
                         "roofline_frac_sustained": max(flops / (tf_sus * 1e12), bytes_ / (hbm * 1e9)) * 1e3 / ms, "bound": "tensor" if flops / (tf * 1e12) > bytes_ / (hbm * 1e9) else "hbm",
                         "tflops": flops / (ms * 1e-3) / 1e12, "gbs": bytes_ / (ms * 1e-3) / 1e9, "model_bytes_per_layer": lbytes}
        if "split" in res and "dense" in res:
            res["split_vs_dense_speedup"] = res["dense"]["ms_per_layer"] / res["split"]["ms_per_layer"]
        res["size_ratio"] = logical / logical_d
        out.append(res)
    return out


def run_quant(ctx, cfg, tokens, copies, reps, device="cuda", use_graph=True, settle=0.0):
    """The quantised split (Section 5.2: 8-bit heavy / 3-bit light, group 128) at few tokens: time per layer and
    fraction of the HBM roofline of the QUANTISED bytes, beside the bf16 dense layer's bytes."""
    hbm, tf, src, _ = peaks()
    shape = make_shape(cfg.d, cfg.m, cfg.act, cfg.torch_dtype)
    ctx.ensure_workspace(ctx.quant_workspace_size(shape, cfg.k))
    padded, logical = ctx.quant_pack_size(shape, cfg.k)
    _, logical_dense = ctx.pack_size(shape, cfg.m, 0)
    blobs = []
    for c in range(copies):
        L = make_layer(cfg, c, device=device)
        heavy = L.planted.to(torch.int32)
        mask = torch.ones(cfg.m, dtype=torch.bool, device=device)
        mask[heavy.long()] = False
        light = torch.nonzero(mask).flatten().to(torch.int32)
        b = torch.empty(padded, dtype=torch.uint8, device=device)
        ctx.quant_pack(shape, L.W1, L.b1, L.W2, L.b2, heavy, cfg.k, light, b, W1u=L.W1u)
        ctx.poll()
        blobs.append(b)
        del L
    out = []
    gen = torch.Generator(device=device)
    gen.manual_seed(4321)
    for T in tokens:
        X = (torch.randn(T, cfg.d, generator=gen, device=device, dtype=torch.float32)).to(cfg.torch_dtype)
        Y = torch.empty_like(X)
        state = {"i": 0}

        def call():
            ctx.quant_forward(blobs[state["i"] % copies], X, Y)
            state["i"] += 1

        ts, mode = time_calls(call, copies * max(1, 16 // copies), reps, max(3, copies), use_graph, settle)
        ctx.poll()
        ms = statistics.median(ts)
        bytes_ = logical + 2 * T * cfg.d * 2
        out.append({"config": cfg.name, "d": cfg.d, "m": cfg.m, "k": cfg.k, "act": cfg.act, "tokens": T, "launch_mode": mode,
                    "weight_copies_cycled": copies, "peaks": src,
                    "quant": {"ms_per_layer": ms, "ms_best": min(ts), "tokens_per_s_per_layer": T / (ms * 1e-3),
                              "tokens_per_s_per_stack": T / (ms * 1e-3 * cfg.layers), "model_bytes_per_layer": logical,
                              "roofline_ms": bytes_ / (hbm * 1e9) * 1e3, "roofline_frac": bytes_ / (hbm * 1e9) * 1e3 / ms,
                              "gbs": bytes_ / (ms * 1e-3) / 1e9, "bits_per_weight": 8.0 * (logical - 4 * (cfg.m + cfg.d)) / ((cfg.n_in + 1) * cfg.d * cfg.m)},
                    "size_ratio_vs_bf16_dense": logical / logical_dense})
    return out


def run_factor(ctx, cfg, iters, reps, device="cuda"):
    """On-device factors of one layer's light slices (Section 5.1.1): time per call, tensor-core rate of the block
    power iteration's products, and the Frobenius residual of U2 ~ A1 B1; the call without a round (gathers, one product, transposes) beside it."""
    hbm, tf, src, _ = peaks()
    shape = make_shape(cfg.d, cfg.m, cfg.act, cfg.torch_dtype)
    ctx.ensure_workspace(ctx.factor_workspace_size(shape, cfg.k, cfg.r))
    L = make_layer(cfg, 0, device=device)
    mask = torch.ones(cfg.m, dtype=torch.bool, device=device)
    mask[L.planted.long()] = False
    light = torch.nonzero(mask).flatten().to(torch.int32)
    n_mat = cfg.n_in + 1
    gen = torch.Generator(device=device)
    gen.manual_seed(99)
    start = torch.randn(n_mat, cfg.r, cfg.d, generator=gen, device=device, dtype=torch.float32).to(cfg.torch_dtype)
    ml = cfg.m - cfg.k
    U2 = L.W1[:, light.long()].float()
    out = {"config": cfg.name, "d": cfg.d, "m": cfg.m, "k": cfg.k, "r": cfg.r, "iters": iters, "peaks": src}
    for label, it in (("start_basis_only", 0), ("iterated", iters)):
        ts = []
        for i in range(reps + 1):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fac = ctx.factor_light(shape, L.W1, L.W2, light, cfg.k, cfg.r, it, start, W1u=L.W1u)
            b.record()
            b.synchronize()
            if i >= 1:
                ts.append(a.elapsed_time(b))
        ctx.poll()
        ms = statistics.median(ts)
        resid = torch.linalg.matrix_norm(U2 - fac["A1"].float() @ fac["B1"].float()).item()
        flops = n_mat * (it * 4.0 + 2.0) * cfg.r * cfg.d * ml
        out[label] = {"ms": ms, "product_tflops": flops / (ms * 1e-3) / 1e12}
        if it > 0:      # (without a round the start basis is not orthonormal and A1 B1 is no projection)
            out[label]["rel_residual_U2"] = resid / torch.linalg.matrix_norm(U2).item()
            if cfg.d <= 1024:
                # the optimum (Eckart-Young) from the singular values of the slice, in float64 on the device
                sv = torch.linalg.svdvals(U2.double())
                best = sv[cfg.r:].square().sum().sqrt().item()
                out[label]["residual_over_truncated_svd"] = resid / best
    return out


def run_encoder(ctx, cfg, batch, seq, layers, reps, device="cuda", use_graph=True, settle=0.0):
    """Whole transformer layers (attention, LayerNorms, FFN) of width cfg.d, `layers` distinct ones back to back as in
    a BERT-base encoder (Table 2's shape: batch 32, sequence 128): time per layer with the split FFN and with the
    dense FFN packed from the same weights, and the parts that are not the FFN."""
    hbm, tf, src, _ = peaks()
    d, heads = cfg.d, cfg.d // 64
    shape = make_shape(d, cfg.m, cfg.act, cfg.torch_dtype)
    T = batch * seq
    ctx.ensure_workspace(max(ctx.workspace_size(shape, T, 0, cfg.k, cfg.r), ctx.workspace_size(shape, T, 0, cfg.m, 0)))
    padded, _ = ctx.pack_size(shape, cfg.k, cfg.r)
    padded_d, _ = ctx.pack_size(shape, cfg.m, 0)
    gen = torch.Generator(device=device)
    gen.manual_seed(2024)
    rn = lambda *sz, std=1.0: torch.randn(*sz, generator=gen, device=device, dtype=torch.float32) * std
    all_idx = torch.arange(cfg.m, dtype=torch.int32, device=device)
    descs = {"split": [], "dense": []}
    keep = []
    for l in range(layers):
        L = make_layer(cfg, l, device=device)
        b = torch.empty(padded, dtype=torch.uint8, device=device)
        ctx.pack(shape, L.W1, L.b1, L.W2, L.b2, L.planted.to(torch.int32), cfg.k, random_factors(cfg, device, gen), b)
        bd = torch.empty(padded_d, dtype=torch.uint8, device=device)
        ctx.pack(shape, L.W1, L.b1, L.W2, L.b2, all_idx, cfg.m, None, bd)
        ctx.poll()
        w = (rn(3 * d, d, std=0.05).to(cfg.torch_dtype), rn(3 * d, std=0.02), rn(d, d, std=0.05).to(cfg.torch_dtype), rn(d, std=0.02),
             (1 + rn(d, std=0.1), rn(d, std=0.05)), (1 + rn(d, std=0.1), rn(d, std=0.05)))
        keep.append((w, b, bd))
        descs["split"].append(ctx.encoder_desc(batch, seq, heads, *w, 1e-12, b))
        descs["dense"].append(ctx.encoder_desc(batch, seq, heads, *w, 1e-12, bd))
        del L
    ctx.ensure_workspace(max(ctx.encoder_workspace_size(descs["split"][0]), ctx.encoder_workspace_size(descs["dense"][0])))
    X = rn(T, d).to(cfg.torch_dtype)
    bufs = [X, torch.empty_like(X), torch.empty_like(X)]
    out = {"config": cfg.name, "d": d, "m": cfg.m, "k": cfg.k, "r": cfg.r, "heads": heads, "batch": batch, "seq": seq,
           "layers": layers, "peaks": src}
    for name in ("split", "dense"):
        def stack():
            src_i = 0
            for l in range(layers):          # layer l reads layer l - 1's output
                dst_i = 1 + (l & 1)
                ctx.encoder_forward(descs[name][l], bufs[src_i], bufs[dst_i])
                src_i = dst_i
        ts, mode = time_calls(stack, 1, reps, 3, use_graph, settle)
        ctx.poll()
        ms = statistics.median(ts)
        out[name] = {"ms_per_stack": ms, "us_per_layer": 1e3 * ms / layers, "launch_mode": mode,
                     "sequences_per_s": batch / (ms * 1e-3)}
    # the FFN alone, same blobs, for the share of the layer it holds
    for name, idx in (("split", 1), ("dense", 2)):
        def ffn_only():
            for l in range(layers):
                ctx.forward(keep[l][idx], bufs[1], bufs[2])
        ts, _ = time_calls(ffn_only, 1, reps, 3, use_graph, settle)
        ctx.poll()
        out[name]["ffn_us_per_layer"] = 1e3 * statistics.median(ts) / layers
    out["split_vs_dense_speedup_whole_layer"] = out["dense"]["ms_per_stack"] / out["split"]["ms_per_stack"]
    out["split_vs_dense_speedup_ffn_only"] = out["dense"]["ffn_us_per_layer"] / out["split"]["ffn_us_per_layer"]
    return out


def run_scoring(ctx, cfg, reps, device="cuda", t_cal=None):
    """Scoring pass of one layer, both forms: from the calibration tokens (product + fused column energy)
    and from a stored activation matrix (one streaming read of H).  Events around each call, median."""
    hbm, tf, src, _ = peaks()
    shape = make_shape(cfg.d, cfg.m, cfg.act, cfg.torch_dtype)
    T = t_cal or cfg.t_cal
    es = 2 if cfg.dtype == "bf16" else 4
    ctx.ensure_workspace(ctx.workspace_size(shape, 0, T, 0, 0))
    L = make_layer(cfg, 0, device=device)
    X = L.tokens(T)
    H = torch.randn(T, cfg.m, device=device, dtype=torch.float32).mul_(0.5).to(cfg.torch_dtype)
    energy = torch.empty(cfg.m, dtype=torch.float32, device=device)
    scores = torch.empty(cfg.m, dtype=torch.float32, device=device)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=device)
    out = {"config": cfg.name, "d": cfg.d, "m": cfg.m, "T_cal": T, "dtype": cfg.dtype, "peaks": src}
    forms = (("fused", lambda: ctx.score(shape, L.W1, L.b1, L.W2, X, energy, scores, W1u=L.W1u)),
             ("stored", lambda: ctx.score_activations(shape, H, L.W2, energy, scores)))
    for name, fn in forms:
        ts = []
        for i in range(reps + 3):
            flush.add_(1)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            fn()
            b.record()
            b.synchronize()
            if i >= 3:
                ts.append(a.elapsed_time(b))
        ctx.poll()
        ms = statistics.median(ts)
        flops = 2.0 * cfg.n_in * T * cfg.d * cfg.m if name == "fused" else 0.0
        bytes_ = (es * (T * cfg.d + (cfg.n_in + 1) * cfg.d * cfg.m) if name == "fused"
                  else es * (T * cfg.m + cfg.m * cfg.d))
        roof_ms = max(flops / (tf * 1e12), bytes_ / (hbm * 1e9)) * 1e3
        out[name] = {"ms": ms, "roofline_ms": roof_ms, "roofline_frac": roof_ms / ms,
                     "bound": "tensor" if flops / (tf * 1e12) > bytes_ / (hbm * 1e9) else "hbm",
                     "tflops": flops / (ms * 1e-3) / 1e12, "gbs": bytes_ / (ms * 1e-3) / 1e9}
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--config", type=int, required=True)
    ap.add_argument("--tokens", type=int, nargs="*", default=None)
    ap.add_argument("--copies", type=int, default=0, help="distinct weight sets cycled (0: enough to exceed 2x L2)")
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--svd", action="store_true", help="true SVD factors instead of random ones")
    ap.add_argument("--sweep5", action="store_true", help="config 5: all heavy fractions x ranks")
    ap.add_argument("--point5", type=int, nargs=2, default=None, metavar=("HEAVY_PERCENT", "RANK"),
                    help="config 5: one point of the sweep")
    ap.add_argument("--out", default=None)
    ap.add_argument("--which", nargs="*", default=["split", "dense"], choices=["split", "dense"],
                    help="time the split layer, its dense counterpart, or both")
    ap.add_argument("--paper-point", action="store_true",
                    help="the paper's own hyper-parameters at BERT-base shape (Section 5.1.1): top 25 %% of the neurons "
                         "heavy (k = 768), light rank = 10 %% of full rank (r = 77); --config is ignored")
    ap.add_argument("--scoring", action="store_true", help="time the scoring pass (both forms) instead of the forward")
    ap.add_argument("--quant", action="store_true", help="time the quantised split (Section 5.2) at the given few-token counts")
    ap.add_argument("--encoder", action="store_true",
                    help="time whole transformer layers (attention + LayerNorms + FFN) of the config's width at batch 32 x "
                         "sequence 128, the config's layer count back to back, split FFN against dense FFN")
    ap.add_argument("--factor", type=int, default=-1, metavar="ITERS",
                    help="time the on-device factorisation of the light slices with this many rounds of block power iteration")
    ap.add_argument("--t-cal", type=int, default=0, help="with --scoring: calibration tokens (default: the config's)")
    ap.add_argument("--settle", type=float, default=1.0,
                    help="seconds of idle time before each timed case (the clocks recover from the case before)")
    ap.add_argument("--no-graph", action="store_true", help="issue the timed calls one by one instead of replaying a CUDA graph")
    args = ap.parse_args()
    build.build()
    ctx = Context(0)
    base = CONFIGS[args.config]
    if args.paper_point:
        from ffsplit_synth import custom_config
        import dataclasses
        base = dataclasses.replace(custom_config(768, 3072, 768, 77, act="gelu_erf", dtype="bf16", t_cal=4096),
                                   name="bert_base_paper_point_k768_r77", layers=12, t_fwd=(4096,))
    points = [base]
    if args.config == 5 and args.sweep5:
        points = [cfg5_point(h, r) for h in CFG5_HEAVY_PERCENT for r in CFG5_RANKS]
    if args.config == 5 and args.point5:
        points = [cfg5_point(*args.point5)]
    if args.scoring:
        print(json.dumps(run_scoring(ctx, base, args.reps, t_cal=args.t_cal or None)), flush=True)
        return
    if args.encoder:
        print(json.dumps(run_encoder(ctx, base, 32, 128, base.layers, args.reps, use_graph=not args.no_graph, settle=args.settle)), flush=True)
        return
    if args.factor >= 0:
        print(json.dumps(run_factor(ctx, base, args.factor, min(args.reps, 5))), flush=True)
        return
    tokens = args.tokens or list(base.t_fwd)
    lines = []
    if args.quant:
        qbytes = 0.45 * (base.n_in + 1) * base.d * base.m          # about 3.5 bits per weight
        copies = args.copies or max(2, min(24, int(-(-2 * 126 * (1 << 20) // qbytes))))
        for res in run_quant(ctx, base, [t for t in tokens if t <= 8] or [1], copies, args.reps, use_graph=not args.no_graph,
                             settle=args.settle):
            print(json.dumps(res), flush=True)
        return
    for cfg in points:
        es = 2 if cfg.dtype == "bf16" else 4
        split_bytes = es * (cfg.n_in + 1) * (cfg.d * cfg.k + cfg.r * (cfg.d + cfg.m - cfg.k))
        copies = args.copies or max(2, min(24, -(-2 * 126 * (1 << 20) // split_bytes)))
        for res in run_point(ctx, cfg, tokens, copies, args.reps, args.svd, use_graph=not args.no_graph, which=tuple(args.which), settle=args.settle):
            line = json.dumps(res)
            print(line, flush=True)
            lines.append(line)
        torch.cuda.empty_cache()
    if args.out:
        os.makedirs(os.path.dirname(os.path.abspath(args.out)), exist_ok=True)
        with open(args.out, "w") as f:
            f.write("\n".join(lines) + "\n")


if __name__ == "__main__":
    main()
