#!/usr/bin/env python
"""Benchmark of the MRP drafting step on B200.

    python bench.py [--gpus N] [--steps S] [--warmup W] [--config all|0..3|module|module:2|module:L16|module:P1024|sweep:M:K|sweep]
                    [--impl ours|reference]

A step is one pass of the whole hot path over one batch of synthetic input: mrp_draft (row
gather, head chain, shared LM head with fused softmax statistics, combine), mrp_reveal_remask
and, in static mode, mrp_verify.  The metric is drafted tokens per second = K_chain * M per step.

With no --config the five benchmark configurations are measured in one process: the tiny fp32
instance, the 1.7B-class decode shape, the 8B-class speculative shape, the 8B-class remask
shape and four points of the roofline sweep.  Rank 0 prints ONE JSON line whose top-level
figures are those of the largest named single-GPU configuration (remask_8b); the list
``configs`` carries the same figures for every other workload.  Each workload is timed as
repeated batches of S steps (CUDA events around every batch) until at least --min-seconds of
GPU time have been spent; the reported time per step is the median batch divided by S.

With N > 1 (torchrun) every rank runs an independent replica of the same workloads on its own
GPU (the path has no collective); a value is the sum over ranks divided by the slowest rank's
time.
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
NOMINAL = {"hbm_gbs": 8000.0, "bf16_tflops": 2250.0}     # the figures the benchmark spec names
HEADLINE = "3"
DEFAULT_WORKLOADS = ("0", "1", "module", "2", "3", "sweep:1:1", "sweep:64:4", "sweep:256:1", "sweep:4096:4")
MODULE_LAYERS, MODULE_ATTN_HEADS = 3, 16      # the paper's depth D = 3 (Sec. 4.1); 128 features per attention head

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the fused LM-head kernel, from
# the ncu captures summarised under profiles/ (bytes per launch, and the summary they come from).
NCU_TRAFFIC = {
    "decode_1p7b": (628348416, "profiles/lm_head_dram_traffic.md"),
    "spec_8b": (1372888320, "profiles/lm_head_dram_traffic.md"),
    "remask_8b": (2638083328, "profiles/lm_head_dram_traffic.md"),
    "sweep_M64_K4": (1365900032, "profiles/lm_head_dram_traffic.md"),
    "sweep_M256_K1": (1486500096, "profiles/lm_head_dram_traffic.md"),
    "sweep_M4096_K4": (36579955712, "profiles/lm_head_dram_traffic.md"),
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20, help="steps per timed batch")
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="all",
                    help="all = the five configurations in one line (default); 0..3 = one configuration; "
                         "module / module:2 / module:L16 = the token-conditioned module at the decode shape, at "
                         "spec_8b's shape, at the decode shape with one block of 16 positions (:P<n> adds a clean prefix of n "
                         "positions to the module's attention); "
                         "sweep:M:K = one roofline-sweep point; sweep = all 21 points, one line each")
    ap.add_argument("--min-seconds", type=float, default=1.0,
                    help="GPU time per workload spent in timed batches of --steps steps")
    ap.add_argument("--flags", type=int, default=0, help="mrp_config.flags (MRP_FLAG_* bits) for A/B timing")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--fp8-lm", action="store_true",
                    help="decode-regime workloads: run the LM head on the 8-bit (e4m3, per-row scale) copy of W_lm "
                         "(MRP_FLAG_FP8_LM); the roofline then counts one byte per LM-head weight")
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


def config_dict(cfg, M, entry="mrp_draft"):
    """What names a workload; the reference arm prints the same dictionary."""
    K = cfg["K"]
    return {"workload": cfg["name"], "rows": int(M), "chain": K, "d": cfg["d"], "d_ff": cfg["F"],
            "vocab": cfg["V"], "seqs": cfg["B"], "block_len": cfg["L"], "mode": cfg["mode"], "entry": entry,
            "l2": "weights streamed per step (%.0f MB) %s the 126 MB L2; no flush between steps"
                  % ((cfg["V"] * cfg["d"] + K * 3.0 * cfg["d"] * cfg["F"]) * (4 if cfg["dtype"] == "f32" else 2) / 1e6,
                     "exceed" if cfg["V"] * cfg["d"] > 40e6 else "fit in (latency case)"),
            "parallelism": "independent replicas, no collective"}


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
        """Samples taken inside [t0, t1] (wall clock of the timed region)."""
        rows = [s for t, s in self.samples if t0 <= t <= t1]
        sm, mx, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                sm.append(float(f[0]))
                mx.append(float(f[1]))
                pw.append(float(f[2]))
            except (ValueError, IndexError):
                continue
            for n, v in zip(names, f[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        sm.sort()
        return {"sm_mhz": sm[len(sm) // 2], "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(pw), "sampled": "inside the timed region"}


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


def lm_head_roofline(cfg, M, lm_ms, peaks, peaks_kind, from_hidden=False, fp8=False):
    """Roofline of the fused LM-head kernel: algorithmic bytes 2Vd + 4MV + 2KMd (one read of
    the LM head, one read of l_0, the stacked residual rows), flops 2KMVd.  With the base
    logits computed in the pass: bytes 2Vd + 2(K+1)Md, flops 2(K+1)MVd.  The bound is the slower
    of bytes over the HBM copy bandwidth and flops over the bf16 tensor peak; ``frac`` is against
    the peaks measured on this machine (sustained bf16 figure: the kernel is timed inside a loop of a
    second or more), ``frac_nominal`` against 8 TB/s and 2250 TFLOP/s."""
    V, d, K = cfg["V"], cfg["d"], cfg["K"]
    esz = 4 if cfg["dtype"] == "f32" else 2
    wsz = 1 if fp8 else esz                       # bytes per LM-head weight (+ 4 bytes of scale per row)
    nbytes = float(wsz) * V * d + (4.0 * V if fp8 else 0.0) + 4.0 * M * V + float(esz) * K * M * d
    flops = 2.0 * K * M * V * d
    if from_hidden:
        nbytes = float(wsz) * V * d + (4.0 * V if fp8 else 0.0) + float(esz) * (K + 1) * M * d
        flops = 2.0 * (K + 1) * M * V * d
    t_hbm = nbytes / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops_sustained"] * 1e12)
    sec = lm_ms * 1e-3
    traffic = NCU_TRAFFIC.get(cfg["name"]) if not (from_hidden or fp8) else None
    common = {"traffic": traffic[0] if traffic else None, "traffic_source": traffic[1] if traffic else None,
              "kernel": "fused LM head", "kernel_ms": lm_ms, "alg_bytes": nbytes, "alg_flops": flops,
              "units_per_launch": K * M}
    if t_hbm >= t_tc:
        ach = nbytes / sec / 1e9
        return dict(common, bound="hbm", achieved=ach, peak=peaks["hbm_gbs"], unit="GB/s",
                    frac=ach / peaks["hbm_gbs"], frac_nominal=ach / NOMINAL["hbm_gbs"],
                    peak_source=("MEASURED_PEAKS.json hbm_gbs" if peaks_kind == "measured"
                                 else "fallback 6650 GB/s") + "; frac_nominal against 8000 GB/s")
    ach = flops / sec / 1e12
    return dict(common, bound="tensor", achieved=ach, peak=peaks["bf16_tflops_sustained"], unit="TFLOP/s",
                frac=ach / peaks["bf16_tflops_sustained"], frac_burst=ach / peaks["bf16_tflops"],
                frac_nominal=ach / NOMINAL["bf16_tflops"],
                peak_source=("MEASURED_PEAKS.json bf16_tflops_sustained" if peaks_kind == "measured"
                             else "fallback 1400 TFLOP/s sustained")
                + "; frac_burst against the burst figure, frac_nominal against 2250 TFLOP/s")


def call_roofline_seconds(cfg, M, peaks):
    """Roofline time of the whole mrp_draft call: every weight read once, l_0 read once."""
    V, d, F, K = cfg["V"], cfg["d"], cfg["F"], cfg["K"]
    esz = 4 if cfg["dtype"] == "f32" else 2
    nbytes = float(esz) * V * d + K * (3.0 * esz * d * F + esz * d) + 4.0 * M * V + float(esz) * M * d + 12.0 * (K + 1) * M
    flops = 2.0 * K * M * V * d + 6.0 * K * M * d * F
    return max(nbytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops_sustained"] * 1e12))


def oracle_step_fn(cfg, w, inp, rows):
    """One pass of the hot path by the CPU oracle over the masked rows ``rows`` (indices into
    inp.row_index; their blocks are renumbered densely)."""
    import numpy as np
    import oracle
    K, L = cfg["K"], cfg["L"]
    ri_rows = inp.row_index[rows]
    blocks = np.unique(ri_rows // L)
    remap = {b: i for i, b in enumerate(blocks)}
    ri = np.array([remap[x // L] * L + x % L for x in ri_rows], np.int32)
    mode = oracle.STATIC if cfg["mode"] == "static" else oracle.DYNAMIC_REMASK

    def step():
        r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=ri_rows)
        s = oracle.select(r.conf.astype(np.float32), r.token, ri, len(blocks), L, mode, tau=cfg["tau"])
        if cfg["mode"] == "static":
            oracle.verify(s.draft_tok, s.draft_tok, s.draft_len)
    return step


def oracle_sample(cfg, w, inp, budget_s):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload's rows (whole
    blocks).  Returns (draft tokens/s, cores, description)."""
    import numpy as np
    import oracle
    K, L = cfg["K"], cfg["L"]
    M = len(inp.row_index)
    blk = inp.row_index // L
    first_block = np.flatnonzero(blk == blk[0])
    step = oracle_step_fn(cfg, w, inp, first_block)
    t = time.perf_counter()
    step()
    per_row = (time.perf_counter() - t) / len(first_block)
    n_rows = int(max(len(first_block), min(M, budget_s / max(per_row, 1e-9))))
    order = np.argsort(blk, kind="stable")            # whole blocks only
    last_block = blk[np.sort(order[:n_rows])[-1]]
    rows = np.flatnonzero(blk <= last_block)
    if len(rows) > n_rows * 1.5:
        rows = first_block
    reps = int(max(1, min(20, budget_s / max(per_row * len(rows), 1e-9))))
    step = oracle_step_fn(cfg, w, inp, rows)
    best = None
    for _ in range(reps):
        t = time.perf_counter()
        step()
        dt = time.perf_counter() - t
        best = dt if best is None else min(best, dt)
    desc = "%d of %d masked rows (whole blocks), all V columns, best of %d%s" % (
        len(rows), M, reps, "" if len(rows) == M else "; per-row rate extrapolated to the workload")
    return K * len(rows) / best, oracle.num_threads(), desc


def run_reference(args):
    """Reference arm: the CPU oracle, as it stands, on the host cores (rank 0 only), on the
    headline workload (or the one --config names); each step is a bounded sample of its rows."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import numpy as np
    import oracle
    from paper_2605_18817_b200 import synth
    name = HEADLINE if args.config == "all" else args.config
    cfg = resolve_config(name)
    oracle.build()
    w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"],
                           4000 if name.startswith("sweep:") else cfg["seed"])
    # base logits only for the rows the sample can reach (input generation, not the method)
    inp = synth.make_inputs(w, cfg["B"], cfg["L"], cfg["seed"], cfg["s_lo"], cfg["s_hi"], cfg["mask_prob"],
                            logits_rows=256)
    M = len(inp.row_index)
    K = cfg["K"]
    step1 = oracle_step_fn(cfg, w, inp, np.arange(1))
    t0 = time.perf_counter()
    step1()
    per_row = time.perf_counter() - t0
    total = args.steps + args.warmup
    # bounded sample per step, sized so that warm-up + timed steps stay near two minutes
    n_rows = int(max(1, min(M, 256, 120.0 / total / max(per_row, 1e-9))))
    step = oracle_step_fn(cfg, w, inp, np.arange(n_rows))
    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = K * n_rows * args.steps / dt
    sample = "first %d of %d masked rows per step, all V columns" % (n_rows, M)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic", "config": config_dict(cfg, M),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(),
                         "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
        "note": "the oracle on the host cores; every step covers the sample named in cpu_baseline, not the "
                "whole workload; rank 0 only",
    }
    print(json.dumps(line), flush=True)


class Bench:
    """Process-wide state of the GPU arm: device, process group, peaks, cached weight sets."""

    def __init__(self, args):
        import torch
        from paper_2605_18817_b200 import build as _build
        self.args = args
        self.rank = int(os.environ.get("RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.local = int(os.environ.get("LOCAL_RANK", "0"))
        if self.local == 0 and not os.environ.get("MRP_B200_LIB"):
            _build.build()
        self.dist = None
        torch.cuda.set_device(self.local)
        if self.world > 1:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=torch.device("cuda", self.local))
            dist.barrier()
            self.dist = dist
        self.dev = torch.device("cuda", self.local)
        self.peaks, self.peaks_kind = load_peaks()
        self.weights = {}      # (d, F, V, n_heads, dtype, seed) -> (host weights, device heads, device w_lm)

    def barrier(self):
        import torch
        torch.cuda.synchronize()
        if self.dist is not None:
            self.dist.barrier()
            torch.cuda.synchronize()

    def weights_for(self, cfg, name):
        from paper_2605_18817_b200 import harness, synth
        seed = 4000 if name.startswith("sweep:") else cfg["seed"]
        n_heads = 4 if name.startswith("sweep:") else cfg["n_heads"]      # one weight set for all sweep points
        key = (cfg["d"], cfg["F"], cfg["V"], n_heads, cfg["dtype"], seed)
        if key not in self.weights:
            self.weights.clear()                                          # one large weight set on the device at a time
            import gc
            import torch
            gc.collect()
            torch.cuda.empty_cache()
            w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], n_heads, cfg["dtype"], seed)
            heads, w_lm = harness.upload_weights(w, self.dev)
            self.weights[key] = (w, heads, w_lm)
        return self.weights[key]

    def time_step(self, step, units_per_step, launches, ctx=None, cfg=None, M=None):
        """Warm-up, then batches of --steps steps (CUDA events around every batch) until --min-seconds of GPU
        time; the median batch gives the time per step; clocks sampled inside the region.  With cfg: the
        common keys of a workload's result."""
        import numpy as np
        import torch
        args, dev, dist = self.args, self.dev, self.dist
        S = max(args.steps, 1)
        warm = max(args.warmup, 3)
        for _ in range(warm):
            step()
        # one batch to size the run
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(S):
            step()
        e1.record()
        torch.cuda.synchronize()
        n_batches = int(max(1, min(5000, np.ceil(args.min_seconds * 1e3 / max(e0.elapsed_time(e1), 1e-3)))))
        evs = [torch.cuda.Event(enable_timing=True) for _ in range(n_batches + 1)]
        sampler = ClockSampler(self.local)
        sampler.start()
        t_w = time.time()                      # the sampler's first line (nvidia-smi can take a second to come up)
        while not sampler.samples and sampler.proc is not None and time.time() - t_w < 3.0:
            time.sleep(0.02)
        self.barrier()
        t_wall0 = time.time()
        evs[0].record()
        for b in range(n_batches):
            for _ in range(S):
                step()
            evs[b + 1].record()
        self.barrier()
        t_wall1 = time.time()
        sampler.stop()
        batch_ms = sorted(evs[b].elapsed_time(evs[b + 1]) for b in range(n_batches))
        med = batch_ms[len(batch_ms) // 2]
        clocks = sampler.summary(t_wall0, t_wall1)
        value, sec_batch = replica_throughput(dist, dev, units_per_step * S, med * 1e-3)
        ms_step = sec_batch * 1e3 / S

        out = {"value": value, "unit": UNIT, "ms_per_step": ms_step, "steps_per_batch": S, "batches": n_batches,
               "batch_ms_median": med, "batch_ms_min": batch_ms[0], "batch_ms_max": batch_ms[-1],
               "timed_gpu_seconds": sum(batch_ms) * 1e-3, "clocks": clocks,
               "gpu_launches": launches[0] * S * n_batches, "launches_per_step": launches[0]}
        if cfg is not None:
            out["dtype"] = "bf16" if cfg["dtype"] == "bf16" else "f32"
            out["config"] = config_dict(cfg, M, "mrp_module_step x %d" % cfg["K"])
        return out

    # -------------------------------------------------------------------------------------
    def run_workload(self, name, cpu_budget_s):
        import numpy as np
        import torch
        from paper_2605_18817_b200 import binding, harness, synth
        args, dev, dist = self.args, self.dev, self.dist
        cfg = resolve_config(name)
        w, heads, w_lm = self.weights_for(cfg, name)
        big = cfg["d"] >= 4096          # base logits of the synthetic backbone: fp32 product on the device
        _, inp = synth.make_config(cfg, w, logits_fn=harness.device_logits_fn(w_lm) if big else None)
        K, B, L = cfg["K"], cfg["B"], cfg["L"]
        M = len(inp.row_index)
        static = cfg["mode"] == "static"
        ctx = binding.mrp_create(w.d, w.F, w.V, heads[:cfg["n_heads"]], w_lm, max_rows=B * L, max_seqs=B,
                                 block_len=L, flags=args.flags | (binding.MRP_FLAG_FP8_LM if args.fp8_lm else 0))
        hid = harness.to_device(inp.hidden, w.dtype, dev)
        l0 = torch.from_numpy(inp.logits0).to(dev)
        ri = torch.from_numpy(inp.row_index).to(dev)
        # hidden states and row index of a step share one device arena: one host-to-device copy
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
        amask = torch.empty((B, K), device=dev, dtype=torch.int8)
        vt = torch.zeros((B, K), device=dev, dtype=torch.int32)

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

        step()
        torch.cuda.synchronize()
        if static:   # synthetic backbone verification tokens for the drafted tokens
            vt.copy_(torch.from_numpy(synth.make_verify_tokens(sel.draft_tok.cpu().numpy(), w.V, cfg["seed"], 0.7)))

        timed = self.time_step(step, K * M, launches)
        S, n_batches = timed["steps_per_batch"], timed["batches"]
        clocks, value, ms_step = timed["clocks"], timed["value"], timed["ms_per_step"]

        # per-phase kernel times (CUDA events on the launching stream inside mrp_draft)
        binding.mrp_profile_enable(ctx, True)
        n_prof = int(min(1000, max(S, S * n_batches // 2)))
        for _ in range(n_prof):
            step()
        torch.cuda.synchronize()
        (ms_heads, ms_lm, ms_comb), n_calls = binding.mrp_profile_read(ctx)
        binding.mrp_profile_enable(ctx, False)
        n_calls = max(n_calls, 1)
        roofline = lm_head_roofline(cfg, M, ms_lm / n_calls, self.peaks, self.peaks_kind, from_hidden=args.from_hidden,
                                    fp8=args.fp8_lm)
        if clocks.get("sm_mhz"):
            roofline["kernel_ms_x_sm_mhz"] = ms_lm / n_calls * clocks["sm_mhz"]
        if ctx.family == "simt" and launches[0] <= 3:
            # the whole drafting pass ran as one kernel (a few short rows on the CUDA cores): its phases are not
            # separate launches, the profile books all of it under the first phase, and the kernel the roofline
            # names is that one, against the bytes of the whole call
            t_call = call_roofline_seconds(cfg, M, self.peaks)
            k_ms = (ms_heads + ms_lm + ms_comb) / n_calls
            ach = t_call * self.peaks["hbm_gbs"] / max(k_ms * 1e-3, 1e-12)
            roofline = {"bound": "hbm", "achieved": ach, "peak": self.peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": ach / self.peaks["hbm_gbs"], "frac_nominal": ach / NOMINAL["hbm_gbs"], "traffic": None,
                        "traffic_source": None, "kernel": "one-kernel drafting pass (all steps)", "kernel_ms": k_ms,
                        "alg_bytes": t_call * self.peaks["hbm_gbs"] * 1e9, "units_per_launch": K * M,
                        "peak_source": roofline.get("peak_source")}
        if cfg["V"] * cfg["d"] <= 40e6:
            roofline["note"] = "all weights fit in L2 and a step is a handful of launches of a few microseconds: " \
                               "this workload measures launch latency (ms_per_step), not a roofline"

        phases = {"heads_ms": ms_heads / n_calls, "lm_head_ms": ms_lm / n_calls,
                  "combine_ms": ms_comb / n_calls, "family": ctx.family,
                  "draft_call_roofline_frac": call_roofline_seconds(cfg, M, self.peaks) /
                  max((ms_heads + ms_lm + ms_comb) / n_calls * 1e-3, 1e-12)}

        # end to end through the public API with host buffers: H2D of the step's inputs from
        # pinned memory and D2H of its results inside the timed region
        e2e = None
        if not args.no_e2e:
            e2e = self.run_e2e(ctx, cfg, step, in_arena, l0, arena, hid, ri, K, M, S)

        cpu = None
        if self.rank == 0 and self.world == 1 and not args.no_cpu_baseline:
            v, cores, desc = oracle_sample(cfg, w, inp, cpu_budget_s)
            cpu = {"value": v, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc}

        status = binding.mrp_fetch_status(ctx)
        binding.mrp_destroy(ctx)
        res = {
            "value": value, "unit": UNIT, "ms_per_step": ms_step,
            "batches": n_batches, "batch_ms_median": timed["batch_ms_median"], "batch_ms_min": timed["batch_ms_min"],
            "batch_ms_max": timed["batch_ms_max"], "timed_gpu_seconds": timed["timed_gpu_seconds"],
            "dtype": "bf16" if cfg["dtype"] == "bf16" else "f32",
            "config": config_dict(cfg, M, ("mrp_draft_from_hidden" if args.from_hidden else "mrp_draft") +
                                  (" on the 8-bit LM head" if args.fp8_lm else "")),
            "clocks": clocks, "e2e": e2e, "gpu_launches": launches[0] * S * n_batches,
            "launches_per_step": launches[0], "roofline": roofline, "phases": phases, "cpu_baseline": cpu,
            "device_status_word": status,
        }
        del hid, l0, ri, out, sel, arena, in_arena
        return res

    def run_e2e(self, ctx, cfg, step, in_arena, l0, arena, hid, ri, K, M, S):
        import torch
        from paper_2605_18817_b200 import binding
        args, dev, dist = self.args, self.dev, self.dist
        h_in = in_arena.cpu().pin_memory()
        h_l0 = l0.cpu().pin_memory()
        h_arena = torch.empty_like(arena, device="cpu").pin_memory()
        bi = hid.numel() * hid.element_size() + ri.numel() * 4
        if not args.from_hidden:
            bi += h_l0.numel() * 4
        bo = arena.numel()

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
        t0 = time.perf_counter()
        e2e_step()
        one = time.perf_counter() - t0
        n_e2e = int(max(3, min(2000, 0.5 * args.min_seconds / max(one, 1e-6)))) if args.min_seconds > 0 else max(3, S)
        self.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        self.barrier()
        dt = time.perf_counter() - t0
        e2e_value, dt = replica_throughput(dist, dev, K * M * n_e2e, dt)
        binding.mrp_set_logits0_event(ctx, None)
        return {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": bi, "d2h_bytes_per_step": bo,
                "steps": n_e2e, "ms_per_step": dt / n_e2e * 1e3, "mode": e2e_mode}


def run_module_workload(bench, cpu_budget_s, which=1, block_len=None, prefix=0):
    """The token-conditioned module at the shape of configuration `which` (1: the decode shape, one block of 4
    positions; 2: 32 blocks of 4, d = 4096): a step is the K = 3 MRP steps that follow one backbone forward in
    direct decoding (Algorithm 2), each = mrp_module_step (module forward + one LM-head pass) +
    mrp_reveal_remask + mrp_commit, the reveals of a step conditioning the next.  Drafted tokens per step:
    K * B (one reveal per block and MRP step).  prefix > 0: every sequence has a clean prefix of that many positions
    in the module's key / value cache (Fig. 1(c)), random values."""
    import numpy as np
    import torch
    import oracle
    from paper_2605_18817_b200 import binding, harness, synth
    args, dev, dist = bench.args, bench.dev, bench.dist
    base = synth.CONFIGS[which]
    if block_len:                                      # the paper's block length (Sec. 4.1) instead of the configuration's
        base = dict(base, L=block_len, name="%s_L%d" % (base["name"], block_len))
    cfg = dict(base, name="module_" + base["name"] + ("_P%d" % prefix if prefix else "") + ("_fp8lm" if args.fp8_lm else ""))
    w, heads, w_lm = bench.weights_for(base, str(which))
    big = base["d"] >= 4096
    _, inp = synth.make_config(base, w, logits_fn=harness.device_logits_fn(w_lm) if big else None)
    K, B, L, d, V, F = cfg["K"], cfg["B"], cfg["L"], cfg["d"], cfg["V"], cfg["F"]
    n = B * L
    n_attn = d // 128                                  # 128 features per attention head
    # (layer weights scaled so that the residual stays inside the accuracy range of the tensor-core LM head:
    # d * rms(h - h_0) <= MRP_RANGE_LIMIT, checked by the device status word below)
    mw = synth.make_module_weights(d, F, V, MODULE_LAYERS, n_attn, "bf16", 11, std=0.02 if d < 4096 else 0.01)
    ctx = binding.mrp_create(d, F, V, heads[:1], w_lm, max_rows=n, max_seqs=B, block_len=L,
                             flags=args.flags | (binding.MRP_FLAG_FP8_LM if args.fp8_lm else 0))
    up = lambda a: harness.to_device(a, "bf16", dev)
    binding.mrp_module_attach(ctx, up(mw.emb), up(mw.w_proj), [{k: up(v) for k, v in lay.items()} for lay in mw.layers],
                              n_attn, mw.mask_token)
    caches = None
    if prefix:
        g = torch.Generator().manual_seed(13)
        host_kv = [(torch.randn((B, prefix, d), generator=g).bfloat16(), torch.randn((B, prefix, d), generator=g).bfloat16())
                   for _ in range(MODULE_LAYERS)]
        caches = [(binding.prefix_to_head_major(k, n_attn).to(dev), binding.prefix_to_head_major(v, n_attn).to(dev))
                  for k, v in host_kv]
        plen = torch.full((B,), prefix, dtype=torch.int32, device=dev)
        binding.mrp_module_set_prefix(ctx, caches, plen)
    hid0 = harness.to_device(inp.hidden, "bf16", dev)
    l0 = torch.from_numpy(inp.logits0).to(dev)
    h_state = torch.empty((n, d), device=dev)
    # block state after the backbone's own reveal of one token (position 0 here: any would do for timing)
    tokens0 = np.full(n, -1, np.int32)
    tokens0[::L] = 17
    state = harness.alloc_block_state(B, L, dev)
    tok_init = torch.from_numpy(tokens0).to(dev)
    out = harness.alloc_draft_out(n, 1, V, d, dev, margin=False)
    sel = harness.alloc_select_out(B, L, 0, dev)
    launches = [0]
    conf_flat, token_flat = out.conf.view(-1), out.token.view(-1)
    ri = torch.from_numpy(np.flatnonzero(tokens0 < 0).astype(np.int32)).to(dev)

    def step():
        state.tokens.copy_(tok_init)
        m = n - B                                   # rows still masked: one fewer per block after every MRP step
        cnt = 1                                     # the tensor fill above
        for k in range(K):
            rows = ri[:m] if k == 0 else state.row_index[:m]
            # a call with m rows writes [2, m] step-major into the front of the [2, n] buffers
            binding.mrp_module_step(ctx, state.tokens, hid0, h_state, l0, rows, m, B, L, k == 0, out.conf, out.lse, out.token)
            cnt += ctx.last_launch_count
            harness.select(ctx, conf_flat[m:2 * m].view(1, m), token_flat[m:2 * m].view(1, m), rows, m, 0, B, L,
                           binding.MRP_SELECT_STATIC, sel, r_reveal=1)
            cnt += ctx.last_launch_count
            harness.commit(ctx, sel, state, B, L, 0)
            cnt += ctx.last_launch_count
            m -= B
        launches[0] = cnt

    step()
    torch.cuda.synchronize()
    res = bench.time_step(step, K * B, launches, ctx, cfg, n - B)
    res.pop("steps_per_batch")
    # roofline of the dominant kernel: the LM-head kernel, launched once per MRP step (K weight streams)
    binding.mrp_profile_enable(ctx, True)
    for _ in range(50):
        step()
    torch.cuda.synchronize()
    (ms_mod, ms_lm, ms_comb), n_calls = binding.mrp_profile_read(ctx)
    binding.mrp_profile_enable(ctx, False)
    one = dict(cfg, K=1)
    roofline = lm_head_roofline(one, n - 2 * B, ms_lm / max(n_calls, 1), bench.peaks, bench.peaks_kind, fp8=args.fp8_lm)
    roofline["kernel"] = "fused LM head, one launch per MRP step (K = %d weight streams per backbone forward)" % K
    roofline["units_per_launch"] = 1
    res["roofline"] = roofline
    res["phases"] = {"module_ms_per_mrp_step": ms_mod / max(n_calls, 1), "lm_head_ms_per_mrp_step": ms_lm / max(n_calls, 1),
                     "combine_ms_per_mrp_step": ms_comb / max(n_calls, 1), "family": ctx.family,
                     "module": "D = %d layers, %d attention heads, %s" % (
                         MODULE_LAYERS, n_attn, "one cooperative tcgen05 kernel per step" if n <= 64 else
                         "products on the row-major tcgen05 kernel"),
                     "prefix_positions": prefix}
    # end to end with host buffers: hidden states, base logits and the block's tokens in, the block state out
    e2e = None
    if not args.no_e2e:
        h_hid, h_l0, h_tok = hid0.cpu().pin_memory(), l0.cpu().pin_memory(), tok_init.cpu().pin_memory()
        h_out = torch.empty_like(state.tokens, device="cpu").pin_memory()

        def e2e_step():
            hid0.copy_(h_hid, non_blocking=True)
            l0.copy_(h_l0, non_blocking=True)
            tok_init.copy_(h_tok, non_blocking=True)
            step()
            h_out.copy_(state.tokens, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        for _ in range(3):
            e2e_step()
        n_e2e = 200 if args.min_seconds > 0 else 3
        bench.barrier()
        t0 = time.perf_counter()
        for _ in range(n_e2e):
            e2e_step()
        bench.barrier()
        dt = time.perf_counter() - t0
        v, dt = replica_throughput(dist, dev, K * B * n_e2e, dt)
        e2e = {"value": v, "unit": UNIT, "h2d_bytes_per_step": h_hid.numel() * 2 + h_l0.numel() * 4 + h_tok.numel() * 4,
               "d2h_bytes_per_step": h_out.numel() * 4, "steps": n_e2e, "ms_per_step": dt / n_e2e * 1e3, "mode": "eager calls"}
    res["e2e"] = e2e
    cpu = None
    if bench.rank == 0 and bench.world == 1 and not args.no_cpu_baseline:
        # a bounded sample: the first blocks only (blocks are independent), one application when the shape is large
        Bs = B if not big else 2
        ns = Bs * L
        ri_h = np.flatnonzero(tokens0[:ns] < 0).astype(np.int32)
        Ks = K if not big else 1
        pre = None
        if prefix:
            pre = ([k[:Bs].float().numpy() for k, _ in host_kv], [v[:Bs].float().numpy() for _, v in host_kv],
                   np.full(Bs, prefix, np.int32))
        t0 = time.perf_counter()
        reps = 0
        while time.perf_counter() - t0 < min(cpu_budget_s, 6.0) or reps == 0:
            for k in range(Ks):
                oracle.module(inp.hidden[:ns], tokens0[:ns], Bs, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, n_attn,
                              mw.mask_token, row_index=ri_h[:len(ri_h) - Bs * k], prefix=pre)
            reps += 1
        cpu = {"value": Ks * Bs * reps / (time.perf_counter() - t0), "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
               "sample": "the module oracle, %d application(s) on %d of %d blocks, %d repetitions" % (Ks, Bs, B, reps)}
    res["cpu_baseline"] = cpu
    res["device_status_word"] = binding.mrp_fetch_status(ctx)
    binding.mrp_destroy(ctx)
    return res


def run_sweep(args):
    """All 21 points of the roofline sweep (configuration 4), one JSON line per point."""
    bench = Bench(args)
    from paper_2605_18817_b200 import synth
    for M in synth.SWEEP_ROWS:
        for K in synth.SWEEP_CHAIN:
            r = bench.run_workload("sweep:%d:%d" % (M, K), 0.0)
            if bench.rank == 0:
                print(json.dumps({
                    "workload": r["config"]["workload"], "rows": M, "chain": K, "ms_per_draft_step": r["ms_per_step"],
                    "draft_tokens_per_s": r["value"], "heads_ms": r["phases"]["heads_ms"],
                    "lm_head_ms": r["phases"]["lm_head_ms"], "combine_ms": r["phases"]["combine_ms"],
                    "lm_head_roofline": {k: r["roofline"].get(k) for k in
                                         ("bound", "achieved", "peak", "unit", "frac", "frac_burst", "frac_nominal")},
                    "draft_call_roofline_frac": r["phases"]["draft_call_roofline_frac"],
                    "sm_mhz": r["clocks"].get("sm_mhz"), "reasons": r["clocks"].get("reasons"),
                    "family": r["phases"]["family"], "peaks": bench.peaks_kind}), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.config == "sweep":
        args.no_e2e = True
        args.no_cpu_baseline = True
        run_sweep(args)
        return
    bench = Bench(args)
    names = list(DEFAULT_WORKLOADS) if args.config == "all" else [args.config]
    head_name = HEADLINE if args.config == "all" else args.config
    results = {}
    for name in names:
        if name == "module" or name.startswith("module:"):
            # module[:1|:2][:L<block length>][:P<prefix positions>], e.g. module:L16 (decode shape, one block of 16), module:P1024
            parts = name.split(":")[1:]
            which = 2 if "2" in parts else 1
            blen = [int(x[1:]) for x in parts if x.startswith("L")]
            pre = [int(x[1:]) for x in parts if x.startswith("P")]
            results[name] = run_module_workload(bench, 5.0, which, blen[0] if blen else None, pre[0] if pre else 0)
        else:
            results[name] = bench.run_workload(name, 12.0 if name == head_name else 5.0)
    if bench.rank == 0:
        head = results[head_name]
        line = {
            "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": bench.world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": head["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic",
            "timing": "per workload: batches of `steps` steps, CUDA events around every batch, repeated until "
                      ">= %.2f s of GPU time; ms_per_step = median batch / steps (max over ranks)" % args.min_seconds,
        }
        for k in ("config", "clocks", "e2e", "gpu_launches", "launches_per_step", "roofline", "phases",
                  "cpu_baseline", "batches", "batch_ms_median", "batch_ms_min", "batch_ms_max",
                  "timed_gpu_seconds", "device_status_word"):
            line[k] = head[k]
        line["configs"] = [results[n] for n in names if n != head_name]
        print(json.dumps(line), flush=True)
    if bench.dist is not None:
        bench.dist.destroy_process_group()


if __name__ == "__main__":
    main()
