#!/usr/bin/env python
"""Benchmark of the MRP drafting step on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config 1] [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic input: mrp_draft (head
chain, shared LM head, softmax statistics), mrp_reveal_remask and, in static mode,
mrp_verify.  The metric is drafted tokens per second = K_chain * M per step.  Rank 0 prints
one JSON line.  With N > 1 (torchrun) every rank runs an independent replica of the same
workload on its own GPU (the path has no collective); the value is the sum over ranks
divided by the slowest rank's time.
"""
from __future__ import annotations

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

METRIC = "MRP draft tokens/s on 1 B200; % of LM-head roofline (HBM or bf16 TC)"
UNIT = "draft tokens/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the fused LM-head kernel,
# from the ncu captures summarised under profiles/ (bytes per launch; None = not captured).
NCU_TRAFFIC_BYTES = {"decode_1p7b": 628542208}   # profiles/sk_gemm_kernel_decode_1p7b.md


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=1000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="1",
                    help="0..3 = benchmark configuration, sweep:M:K = one roofline-sweep point, sweep = all 21 points")
    ap.add_argument("--flags", type=int, default=0, help="mrp_config.flags (MRP_FLAG_* bits) for A/B timing")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--from-hidden", action="store_true",
                    help="draft with mrp_draft_from_hidden: the base logits are computed in the LM-head pass "
                         "instead of being an input (no [rows, V] read or host copy)")
    return ap.parse_args()


def resolve_config(name):
    from paper_2605_18817_b200 import synth
    if name.startswith("sweep:"):
        _, M, K = name.split(":")
        return synth.sweep_config(int(M), int(K))
    return dict(synth.CONFIGS[int(name)])


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        try:
            d = json.load(open(p))
            return {k: float(d[k]) for k in FALLBACK_PEAKS}, "measured"
        except Exception:
            pass
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock / throttle-reason samples while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.samples = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), "--query-gpu=" + self.Q,
                 "--format=csv,noheader,nounits", "-lms", "100"],
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
                self.proc.kill()

    def summary(self, t0, t1):
        rows = [s for t, s in self.samples if t0 <= t <= t1 + 0.15] or [s for _, s in self.samples]
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm)}


def replica_throughput(dist, device, units_per_rank, seconds):
    """Whole-job throughput of independent replicas (the path has no collective): every rank
    processed ``units_per_rank`` units; the job's time is the slowest rank's.  Returns
    (units per second over all ranks, that time).  ``dist`` None = a single process."""
    import torch
    world = 1
    if dist is not None:
        t = torch.tensor([seconds], dtype=torch.float64, device=device)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        seconds = float(t.item())
        world = dist.get_world_size()
    return world * units_per_rank / seconds, seconds


def lm_head_roofline(cfg, M, lm_ms, peaks, peaks_kind, traffic, from_hidden=False):
    """Roofline of the fused LM-head kernel: algorithmic bytes 2Vd + 4MV + 2KMd (one read of
    the LM head, one read of l_0, the stacked residual rows), flops 2KMVd.  With the base
    logits computed in the pass: bytes 2Vd + 2(K+1)Md, flops 2(K+1)MVd."""
    V, d, K = cfg["V"], cfg["d"], cfg["K"]
    nbytes = 2.0 * V * d + 4.0 * M * V + 2.0 * K * M * d
    flops = 2.0 * K * M * V * d
    if from_hidden:
        nbytes = 2.0 * V * d + 2.0 * (K + 1) * M * d
        flops = 2.0 * (K + 1) * M * V * d
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12)
    sec = lm_ms * 1e-3
    if t_hbm >= t_tc:
        ach = nbytes / sec / 1e9
        return {"bound": "hbm", "achieved": ach, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                "frac": ach / peaks["hbm_gbs"], "traffic": traffic, "kernel": "fused LM head",
                "kernel_ms": lm_ms, "alg_bytes": nbytes, "alg_flops": flops,
                "peak_source": "MEASURED_PEAKS.json hbm_gbs" if peaks_kind == "measured"
                else "fallback 6650 GB/s"}
    ach = flops / sec / 1e12
    return {"bound": "tensor", "achieved": ach, "peak": peaks["bf16_tflops_sustained"],
            "unit": "TFLOP/s", "frac": ach / peaks["bf16_tflops_sustained"], "traffic": traffic,
            "kernel": "fused LM head", "kernel_ms": lm_ms, "alg_bytes": nbytes, "alg_flops": flops,
            "peak_source": "MEASURED_PEAKS.json bf16_tflops_sustained" if peaks_kind == "measured"
            else "fallback 1400 TFLOP/s sustained"}


def oracle_sample(cfg, w, inp, budget_s=12.0):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload's rows (whole
    blocks).  Returns (draft tokens/s, cores, description)."""
    import numpy as np
    import oracle
    K, L = cfg["K"], cfg["L"]
    M = len(inp.row_index)

    def run(rows):
        t = time.perf_counter()
        r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index[rows])
        blocks = np.unique(inp.row_index[rows] // L)
        remap = {b: i for i, b in enumerate(blocks)}
        ri = np.array([remap[x // L] * L + x % L for x in inp.row_index[rows]], np.int32)
        mode = oracle.STATIC if cfg["mode"] == "static" else oracle.DYNAMIC_REMASK
        s = oracle.select(r.conf.astype(np.float32), r.token, ri, len(blocks), L, mode, tau=cfg["tau"])
        if cfg["mode"] == "static":
            oracle.verify(s.draft_tok, s.draft_tok, s.draft_len)
        return time.perf_counter() - t

    first_block = np.flatnonzero(inp.row_index // L == inp.row_index[0] // L)
    t1 = run(first_block)
    per_row = t1 / len(first_block)
    n_rows = int(max(len(first_block), min(M, budget_s / max(per_row, 1e-9))))
    # whole blocks only
    order = np.argsort(inp.row_index // L, kind="stable")
    rows = np.sort(order[:n_rows])
    last_block = inp.row_index[rows[-1]] // L
    rows = np.flatnonzero(inp.row_index // L <= last_block)
    if len(rows) > n_rows * 1.5:
        rows = first_block
    reps = int(max(1, min(20, budget_s / max(per_row * len(rows), 1e-9))))
    t = min(run(rows) for _ in range(reps)) if reps > 1 else run(rows)
    desc = "%d of %d masked rows (whole blocks), all V columns, best of %d" % (len(rows), M, reps)
    return K * len(rows) / t, oracle.num_threads(), desc


def run_reference(args, cfg):
    """Reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only)."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import oracle
    from paper_2605_18817_b200 import synth
    oracle.build()
    w, inp = synth.make_config(cfg)
    M = len(inp.row_index)
    K, L = cfg["K"], cfg["L"]
    # bounded sample per step: the first rows of the workload, sized so that the whole run
    # (warm-up + timed steps) stays near two minutes; never fewer than one row
    t0 = time.perf_counter()
    oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index[:1])
    per_row = time.perf_counter() - t0
    total = args.steps + args.warmup
    n_rows = int(max(1, min(M, 120.0 / total / max(per_row, 1e-9))))
    rows = np.arange(n_rows)

    def step():
        r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index[rows])
        blocks = np.unique(inp.row_index[rows] // L)
        remap = {b: i for i, b in enumerate(blocks)}
        ri = np.array([remap[x // L] * L + x % L for x in inp.row_index[rows]], np.int32)
        mode = oracle.STATIC if cfg["mode"] == "static" else oracle.DYNAMIC_REMASK
        s = oracle.select(r.conf.astype(np.float32), r.token, ri, len(blocks), L, mode, tau=cfg["tau"])
        if cfg["mode"] == "static":
            oracle.verify(s.draft_tok, s.draft_tok, s.draft_len)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = K * len(rows) * args.steps / dt
    sample = "first %d of %d masked rows per step, all V columns" % (len(rows), M)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": cfg["name"], "rows": M, "chain": K, "d": cfg["d"], "d_ff": cfg["F"],
                   "vocab": cfg["V"], "seqs": cfg["B"], "block_len": L, "mode": cfg["mode"],
                   "l2": "host cores (oracle)", "parallelism": "rank 0 only"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def run_sweep(args):
    """Roofline sweep (configuration 4): d = 4096, V = 151936, masked rows M in {1 .. 4096} times
    chain length K in {1, 2, 4}, one weight set shared by all points.  Prints one JSON line per
    point: time per drafting pass, draft tokens/s, the fused LM-head kernel's time and its
    fraction of the roofline (slower of algorithmic bytes over HBM bandwidth and flops over the
    bf16 tensor peak), and the same fraction for the whole mrp_draft call."""
    import numpy as np
    import torch
    from paper_2605_18817_b200 import build as _build
    if not os.environ.get("MRP_B200_LIB"):
        _build.build()
    from paper_2605_18817_b200 import binding, harness, synth
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks, peaks_kind = load_peaks()
    w = synth.make_weights(4096, 8192, 151936, 4, "bf16", 4000)
    heads, w_lm = harness.upload_weights(w, dev)
    logits_fn = harness.device_logits_fn(w_lm)
    d, F, V = w.d, w.F, w.V
    for M in synth.SWEEP_ROWS:
        for K in synth.SWEEP_CHAIN:
            cfg = synth.sweep_config(M, K)
            _, inp = synth.make_config(cfg, w, logits_fn=logits_fn)
            ctx = binding.mrp_create(d, F, V, heads[:K], w_lm, max_rows=M, max_seqs=M, block_len=1,
                                     flags=args.flags)
            hid = harness.to_device(inp.hidden, w.dtype, dev)
            l0 = torch.from_numpy(inp.logits0).to(dev)
            ri = torch.from_numpy(inp.row_index).to(dev)
            out = harness.alloc_draft_out(M, K, V, d, dev, margin=False)
            for _ in range(3):
                harness.draft(ctx, hid, l0, ri, M, K, out)
            torch.cuda.synchronize()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            ev0.record()
            harness.draft(ctx, hid, l0, ri, M, K, out)
            ev1.record()
            torch.cuda.synchronize()
            n = int(max(5, min(200, 300.0 / max(ev0.elapsed_time(ev1), 1e-3))))
            ev0.record()
            for _ in range(n):
                harness.draft(ctx, hid, l0, ri, M, K, out)
            ev1.record()
            torch.cuda.synchronize()
            ms = ev0.elapsed_time(ev1) / n
            binding.mrp_profile_enable(ctx, True)
            for _ in range(n):
                harness.draft(ctx, hid, l0, ri, M, K, out)
            torch.cuda.synchronize()
            (ms_heads, ms_lm, ms_comb), nc = binding.mrp_profile_read(ctx)
            binding.mrp_profile_enable(ctx, False)
            roof = lm_head_roofline(cfg, M, ms_lm / nc, peaks, peaks_kind, None)
            call_bytes = 2.0 * V * d + K * (6.0 * d * F + 2 * d) + 4.0 * M * V + 2.0 * M * d + 12.0 * (K + 1) * M
            call_flops = 2.0 * K * M * V * d + 6.0 * K * M * d * F
            t_roof = max(call_bytes / (peaks["hbm_gbs"] * 1e9), call_flops / (peaks["bf16_tflops_sustained"] * 1e12))
            print(json.dumps({
                "workload": cfg["name"], "rows": M, "chain": K, "ms_per_draft": ms,
                "draft_tokens_per_s": K * M / (ms * 1e-3), "heads_ms": ms_heads / nc,
                "lm_head_ms": ms_lm / nc, "combine_ms": ms_comb / nc,
                "lm_head_roofline": {k: roof[k] for k in ("bound", "achieved", "peak", "unit", "frac")},
                "draft_call_roofline_frac": t_roof / (ms * 1e-3), "family": ctx.family,
                "peaks": peaks_kind}), flush=True)
            binding.mrp_destroy(ctx)
            del hid, l0, ri, out


def main():
    args = parse_args()
    if args.config == "sweep":
        run_sweep(args)
        return
    cfg = resolve_config(args.config)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    import numpy as np
    import torch
    from paper_2605_18817_b200 import build as _build
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if rank == 0 and not os.environ.get("MRP_B200_LIB"):
        _build.build()
    dist = None
    if world > 1:
        import torch.distributed as dist
        torch.cuda.set_device(local)
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
        dist.barrier()
    else:
        torch.cuda.set_device(local)
    from paper_2605_18817_b200 import binding, harness, synth
    dev = torch.device("cuda", local)

    w, inp = synth.make_config(cfg)
    K, B, L = cfg["K"], cfg["B"], cfg["L"]
    M = len(inp.row_index)
    static = cfg["mode"] == "static"
    ctx = harness.create_for(cfg, w, dev, flags=args.flags)
    hid = harness.to_device(inp.hidden, w.dtype, dev)
    l0 = torch.from_numpy(inp.logits0).to(dev)
    ri = torch.from_numpy(inp.row_index).to(dev)
    # hidden states and row index of a step share one device arena too: one host-to-device copy
    hid_bytes = (hid.numel() * hid.element_size() + 15) // 16 * 16
    in_arena = torch.zeros(hid_bytes + ri.numel() * 4, device=dev, dtype=torch.uint8)
    hid_v = in_arena[:hid.numel() * hid.element_size()].view(hid.dtype).view(hid.shape)
    ri_v = in_arena[hid_bytes:].view(torch.int32)
    hid_v.copy_(hid)
    ri_v.copy_(ri)
    hid, ri = hid_v, ri_v
    out = harness.alloc_draft_out(M, K, w.V, w.d, dev, margin=False)
    sel = harness.alloc_select_out(B, L, K, dev)
    alen = torch.empty(B, device=dev, dtype=torch.int32)
    # The results a caller reads back after a step live in one device arena (the library only
    # sees pointers), so the end-to-end leg returns them with a single device-to-host copy.
    res_names = [(out, "conf"), (out, "token"), (sel, "reveal_mask"), (sel, "remask_mask"),
                 (sel, "out_token"), (sel, "draft_len")]
    res_shapes = [(getattr(o, n).shape, getattr(o, n).dtype) for o, n in res_names] + [(alen.shape, alen.dtype)]
    offs, total = [], 0
    for shp, dt in res_shapes:
        offs.append(total)
        nbytes = int(np.prod(shp)) * torch.empty((), dtype=dt).element_size()
        total += (nbytes + 15) // 16 * 16
    arena = torch.zeros(total, device=dev, dtype=torch.uint8)
    views = []
    for (shp, dt), o in zip(res_shapes, offs):
        nbytes = int(np.prod(shp)) * torch.empty((), dtype=dt).element_size()
        views.append(arena[o:o + nbytes].view(dt).view(shp))
    for (o, n), v in zip(res_names, views[:-1]):
        setattr(o, n, v)
    alen = views[-1]
    mode = binding.MRP_SELECT_STATIC if static else binding.MRP_SELECT_DYNAMIC_REMASK
    launches = [0]

    def step():
        if args.from_hidden:
            harness.draft_from_hidden(ctx, hid, None, ri, M, K, out)
        else:
            harness.draft(ctx, hid, l0, ri, M, K, out)
        n = ctx.last_launch_count
        harness.select(ctx, out.conf, out.token, ri, M, K, B, L, mode, sel, tau=cfg["tau"])
        n += ctx.last_launch_count
        if static:
            binding.mrp_verify(ctx, sel.draft_tok, vt, sel.draft_len, B, K, False, alen, amask)
            n += ctx.last_launch_count
        launches[0] = n

    amask = torch.empty((B, K), device=dev, dtype=torch.int8)
    vt = torch.zeros((B, K), device=dev, dtype=torch.int32)
    step()
    torch.cuda.synchronize()
    if static:   # synthetic backbone verification tokens for the drafted tokens
        vt.copy_(torch.from_numpy(synth.make_verify_tokens(sel.draft_tok.cpu().numpy(), w.V,
                                                           cfg["seed"], 0.7)))

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    sampler = ClockSampler(local)
    sampler.start()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    ev0.record()
    for _ in range(args.steps):
        step()
    ev1.record()
    barrier()
    t_wall1 = time.time()
    ms_total = ev0.elapsed_time(ev1)
    # keep the GPU busy a little longer if the region was too short for a clock sample
    if t_wall1 - t_wall0 < 0.6:
        t_end = time.time() + 0.8
        while time.time() < t_end:
            for _ in range(50):
                step()
            torch.cuda.synchronize()
        t_wall1 = time.time()
    sampler.stop()
    clocks = sampler.summary(t_wall0, t_wall1)
    value, sec_total = replica_throughput(dist, dev, K * M * args.steps, ms_total * 1e-3)
    ms_total = sec_total * 1e3
    ms_step = ms_total / args.steps

    # per-phase kernel times, CUDA events on the launching stream, same number of steps
    binding.mrp_profile_enable(ctx, True)
    n_prof = min(args.steps, 1000)
    for _ in range(n_prof):
        step()
    torch.cuda.synchronize()
    (ms_heads, ms_lm, ms_comb), n_calls = binding.mrp_profile_read(ctx)
    binding.mrp_profile_enable(ctx, False)
    n_calls = max(n_calls, 1)
    peaks, peaks_kind = load_peaks()
    roofline = lm_head_roofline(cfg, M, ms_lm / n_calls, peaks, peaks_kind,
                                None if args.from_hidden else NCU_TRAFFIC_BYTES.get(cfg["name"]),
                                from_hidden=args.from_hidden)
    phases = {"heads_ms": ms_heads / n_calls, "lm_head_ms": ms_lm / n_calls,
              "combine_ms": ms_comb / n_calls, "family": ctx.family}

    # end to end through the public API with host buffers: H2D of the step's inputs from
    # pinned memory and D2H of its results inside the timed region
    e2e = None
    if not args.no_e2e:
        h_in = in_arena.cpu().pin_memory()
        h_l0 = l0.cpu().pin_memory()
        h_arena = torch.empty_like(arena, device="cpu").pin_memory()
        bi = hid.numel() * hid.element_size() + ri.numel() * 4
        if not args.from_hidden:
            bi += h_l0.numel() * 4
        bo = arena.numel()
        n_e2e = max(3, min(args.steps, 300))

        # The base logits are needed by the LM-head kernel only: their copy (the bulk of the input
        # bytes) runs on a second stream beside the head chain, and the library waits for it right
        # before the LM head (mrp_set_logits0_event).
        side = torch.cuda.Stream()
        l0_ready = torch.cuda.Event()
        if not args.from_hidden:
            l0_ready.record()
            binding.mrp_set_logits0_event(ctx, l0_ready)

        def e2e_body():
            if not args.from_hidden:
                cur = torch.cuda.current_stream()
                side.wait_stream(cur)
                with torch.cuda.stream(side):
                    l0.copy_(h_l0, non_blocking=True)
                    l0_ready.record(side)
            in_arena.copy_(h_in, non_blocking=True)
            step()
            h_arena.copy_(arena, non_blocking=True)

        # The library's calls are stream-ordered and allocate nothing, so a caller can record
        # the whole step (input copies, the three C-ABI calls, result copies) in a CUDA graph
        # and replay it: one launch per step instead of some twenty.  Falls back to eager calls.
        graph, e2e_mode = None, "eager calls"
        try:
            cap = torch.cuda.Stream()
            cap.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(cap):
                e2e_body()
            cap.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=cap):
                e2e_body()
            g.replay()
            torch.cuda.synchronize()
            graph, e2e_mode = g, "CUDA graph of the step (copies + kernels), one replay + sync per step"
        except Exception as ex:      # capture unsupported here: measure the eager path
            torch.cuda.synchronize()
            e2e_mode = "eager calls (graph capture failed: %s)" % type(ex).__name__

        def e2e_step():
            if graph is not None:
                graph.replay()
            else:
                e2e_body()
            torch.cuda.current_stream().synchronize()

        for _ in range(3):
            e2e_step()
        barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        barrier()
        dt = time.perf_counter() - t0
        e2e_value, dt = replica_throughput(dist, dev, K * M * n_e2e, dt)
        binding.mrp_set_logits0_event(ctx, None)
        e2e = {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": bi,
               "d2h_bytes_per_step": bo, "steps": n_e2e, "ms_per_step": dt / n_e2e * 1e3, "mode": e2e_mode}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        v, cores, desc = oracle_sample(cfg, w, inp)
        cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16" if cfg["dtype"] == "bf16" else "f32", "data": "synthetic",
            "config": {"workload": cfg["name"], "rows": M, "chain": K, "d": cfg["d"], "d_ff": cfg["F"],
                       "vocab": cfg["V"], "seqs": B, "block_len": L, "mode": cfg["mode"],
                       "entry": "mrp_draft_from_hidden" if args.from_hidden else "mrp_draft",
                       "l2": "weights streamed per step (%.0f MB) exceed the 126 MB L2; no flush"
                             % ((2.0 * cfg["V"] * cfg["d"] + K * 6.0 * cfg["d"] * cfg["F"]) / 1e6),
                       "parallelism": "replicas x%d" % world},
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches[0] * args.steps,
            "launches_per_step": launches[0], "roofline": roofline, "phases": phases,
            "cpu_baseline": cpu,
        }
        print(json.dumps(line), flush=True)
    binding.mrp_destroy(ctx)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
