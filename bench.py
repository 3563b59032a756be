#!/usr/bin/env python
"""Benchmark of the HeatKV hot path on B200.

One "step" = one image (a cond/uncond pair, batch 2) through the attention + cache path of a 2B-class model:
32 layers of the single-layer workload (16 heads, d=128, 13 scales = 10 521 tokens, 20x KV compression), every
layer with seeded activations of its own.  A layer's sweep is, for every scale, the eviction before the scale,
the ragged attention over the retained keys plus the scale's own keys, and the append/compaction of the new
K/V.  The schedule comes from the library's own calibration kernel run once on seeded samples before timing
(the paper computes it offline, once per model and budget).  MLP, VAE and text encoder are not part of it.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every rank runs an independent replica
of the workload on its own GPU -- the path has no exchange step -- and the value is the sum of
images over the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import heatkv_workloads as W  # noqa: E402

B_BUDGET = 1.0 / 20.0
CALIB_SEEDS = (100, 101, 102, 103)
DATA_SEED = 0
METRIC = "images_per_sec_scale_step_attention_2b_class_20x"
N_LAYERS = 32            # layers of the 2B-class model: one step replays the layer sweep this many times
UNIT = "images/s"
# dram__bytes_read.sum + dram__bytes_write.sum of the dominant kernel's seven launches of one layer sweep, from
# the ncu capture summarised in profiles/attn_tc_kernel_config2.md, with the sources the captured kernel was
# built from (first 16 hex digits of their SHA-256); reported as null once either file has changed
TRAFFIC_CAPTURE = {"bytes_per_layer_sweep": 311.3e6,
                   "sources": {"attn_tc.cu": "ea1e2fd4850f5b71", "tc_common.cuh": "d2e60f2b58b21146"}}


def captured_traffic():
    import hashlib
    for name, want in TRAFFIC_CAPTURE["sources"].items():
        path = os.path.join(ROOT, "paper_2605_14877_b200", "csrc", name)
        try:
            got = hashlib.sha256(open(path, "rb").read()).hexdigest()[:16]
        except OSError:
            return None
        if got != want:
            return None
    return TRAFFIC_CAPTURE["bytes_per_layer_sweep"]


def oracle_threads():
    """Threads the oracle's numpy really computes with: those of the BLAS behind its matrix products."""
    try:
        import threadpoolctl
        n = [int(x["num_threads"]) for x in threadpoolctl.threadpool_info() if x.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return 1


def peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm_gbs": p["hbm_gbs"], "bf16_tflops": p["bf16_tflops"],
                "bf16_tflops_sustained": p.get("bf16_tflops_sustained", p["bf16_tflops"]), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    Q_OLD = Q.replace("clocks_event_reasons", "clocks_throttle_reasons")

    def __init__(self, index: int):
        self.index, self.proc, self.lines = index, None, []

    def start(self):
        try:
            query = self.Q
            probe = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={query}",
                                    "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=30)
            if probe.returncode != 0 or "not a valid" in (probe.stdout + probe.stderr).lower():
                query = self.Q_OLD
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={query}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
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
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for n, v in zip(names, parts[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def aggregate_replicas(total_ms, e2e_ms, steps, dist=None, device="cpu", images_per_replica_step=1):
    """Whole-job numbers of N independent replicas (the path has no exchange step): every rank times
    its own K sweeps; the job's time is the slowest rank's, the job's work the sum over ranks.
    Returns (ms_per_step, images/s, e2e images/s)."""
    world = 1
    if dist is not None:
        tt = torch.tensor([total_ms, e2e_ms], dtype=torch.float64, device=device)
        dist.all_reduce(tt, op=dist.ReduceOp.MAX)
        total_ms, e2e_ms = (float(x) for x in tt.cpu())
        world = dist.get_world_size()
    images = images_per_replica_step * world
    ms_per_step = total_ms / steps
    return ms_per_step, images / (ms_per_step * 1e-3), images / (e2e_ms * 1e-3)


def attention_flops(shape, am, n_seq):
    """Algorithmic flops of every (step) attention launch: 4*d*t_k*n_vis summed over (seq, head),
    n_vis = retained prior keys + the scale's own keys."""
    t = shape.t
    out = []
    for k in range(shape.K):
        tot = 0
        for l in range(shape.L):
            for h in range(shape.H):
                prior = sum(t[i] for i in range(k) if (int(am[k, l, h]) >> i) & 1)
                tot += 4 * shape.d * t[k] * (prior + t[k])
        out.append(tot * n_seq)
    return out


def attention_bytes(shape, am, n_seq):
    """Algorithmic bytes of every (step) attention launch: K and V of the visible keys plus Q and O, bf16,
    summed over (seq, head): 2*2*d*n_vis + 2*2*d*t_k."""
    t = shape.t
    out = []
    for k in range(shape.K):
        tot = 0
        for l in range(shape.L):
            for h in range(shape.H):
                prior = sum(t[i] for i in range(k) if (int(am[k, l, h]) >> i) & 1)
                tot += 4 * shape.d * (prior + t[k]) + 4 * shape.d * t[k]
        out.append(tot * n_seq)
    return out


def oracle_context(shape):
    """Inputs of the oracle timing: the oracle's own schedule from seeded scores, one sequence of
    the workload widened to fp64."""
    from oracle import heatkv_oracle as O
    scores = W.synthetic_scas(shape, 0)
    sch = O.heatkv_schedule(scores, B_BUDGET, shape.s, shape.sides)
    q, k, v = W.qkv_layer(shape, DATA_SEED, 0, n_seq=1)
    f = lambda x: O.bf16_bits_to_f64(W.bf16_bits(x))
    return {"O": O, "sch": sch, "q": f(q), "k": f(k), "v": f(v), "kb": W.bf16_bits(k), "vb": W.bf16_bits(v),
            "bias": W.seg_bias_current_scale(shape, DATA_SEED), "sm": 1.0 / math.sqrt(shape.d)}


def oracle_flops(shape, ctx, head, steps):
    """Algorithmic attention flops (4*d*t_k*n_vis) of the given 1-based steps for one head under the
    oracle's schedule."""
    O, sch = ctx["O"], ctx["sch"]
    tot = 0
    for step in steps:
        n_vis = sum(int(sch.t[i - 1]) for i in O.visible_scales(sch, step, 0, head)) + shape.t[step - 1]
        tot += 4 * shape.d * shape.t[step - 1] * n_vis
    return tot


def oracle_seconds(shape, ctx, head, steps):
    """Times the CPU oracle as it stands (attention + cache contents) on one (seq, head) unit for the
    given 1-based steps."""
    O, sch = ctx["O"], ctx["sch"]
    t0 = time.perf_counter()
    for step in steps:
        lo, hi = (shape.c[step - 2] if step > 1 else 0), shape.c[step - 1]
        brow = ctx["bias"][0, step - 1, head].astype(np.float64)
        O.scale_attention(ctx["q"][0, head, lo:hi], ctx["k"][0, head], ctx["v"][0, head], sch, step, 0, head,
                          ctx["sm"], brow)
        if step < shape.K:
            O.cache_after_layer(ctx["kb"][0, head], ctx["vb"][0, head], sch, step, 0, head)
    return time.perf_counter() - t0


def oracle_images_per_s(shape, ctx, samples):
    """samples: list of (head, steps).  Extrapolates to one image (N_LAYERS layers of n_seq * H units, all scales)
    by algorithmic flops.  Returns (images/s, seconds spent, flops covered / flops of one image)."""
    all_steps = list(range(1, shape.K + 1))
    image_flops = N_LAYERS * shape.n_seq * sum(oracle_flops(shape, ctx, h, all_steps) for h in range(shape.H))
    secs = sum(oracle_seconds(shape, ctx, h, st) for h, st in samples)
    done = sum(oracle_flops(shape, ctx, h, st) for h, st in samples)
    return done / secs / image_flops, secs, done / image_flops


def run_reference(args, rank):
    """Reference arm: the CPU oracle as it stands, timed on the host cores.  Every step times a
    bounded sample (one (seq, head) unit, all scales or a rotating subset of them when K is large)
    and the per-image rate is extrapolated by algorithmic flops."""
    if rank != 0:
        return
    shape = W.CFG2
    ctx = oracle_context(shape)
    all_steps = list(range(1, shape.K + 1))
    unit_s = oracle_seconds(shape, ctx, 0, all_steps)
    for _ in range(max(args.warmup - 1, 0)):
        oracle_seconds(shape, ctx, 0, all_steps[-2:])
    budget_s = 150.0
    stride = max(1, int(math.ceil(args.steps * unit_s / budget_s)))
    samples = [(i % shape.H, [st for st in all_steps if (st + i) % stride == 0] or [shape.K]) for i in range(args.steps)]
    value, secs, frac = oracle_images_per_s(shape, ctx, samples)
    threads = oracle_threads()
    sample = (f"per step one (layer, seq, head) unit of {N_LAYERS * shape.n_seq * shape.H}, every {stride}-th scale "
              f"(all 13 when 1); {secs:.1f} s of CPU work = {frac:.3g} images, extrapolated by flops")
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 / value,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": shape.name, "L": shape.L, "H": shape.H, "d": shape.d, "scales": shape.K,
                       "tokens": shape.n_tokens, "n_seq": shape.n_seq, "budget": B_BUDGET, "policy": "heatkv",
                       "s": shape.s, "layers": N_LAYERS},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def cache_update_numbers(reps, cases=("append_paged", "append_ragged", "compact_ragged", "append_fp8_paged"), first_scale=1):
    """Cache-update kernels at a saturating shape: the larger-model layer shape (32 heads, d=128, 16 sequences,
    one layer).  Appends are timed with every head storing (full budget, paged and ragged); the in-place
    compaction of the ragged layout under a 1/5 budget.  Bytes are algorithmic: 8*d*t_k per storing head (K and
    V, read + write), 8*d*moved tokens per move; the quantising append of the fp8 cache reads 4*d and writes 2*(d+1) bytes per
    token.  Rows for scales >= first_scale."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session
    sh = W.Shape("larger_layer", L=1, H=32, d=128, sides=W.SIDES_13, n_seq=16, s=3)
    pk = peaks()
    out = {"workload": "cache_update_saturating", "shape": {"H": sh.H, "d": sh.d, "n_seq": sh.n_seq, "scales": sh.K},
           "peak_gbs": pk["hbm_gbs"], "peak_source": pk["source"]}
    ks = [torch.randn(sh.n_seq, sh.H, sh.t[k], sh.d, device="cuda").to(torch.bfloat16) for k in range(sh.K)]
    vs = [torch.randn_like(x) for x in ks]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()
    for name, layout, b in (("append_paged", hk.LAYOUT_PAGED, 1.0), ("append_ragged", hk.LAYOUT_RAGGED, 1.0),
                            ("compact_ragged", hk.LAYOUT_RAGGED, 0.2), ("append_fp8_paged", hk.LAYOUT_PAGED, 1.0)):
        if name not in cases:
            continue
        fp8 = name == "append_fp8_paged"
        ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K) + 64, layout=layout,
                      cache_dtype=hk.CACHE_FP8_E4M3 if fp8 else hk.CACHE_BF16)
        sch = ses.schedule(scas=W.synthetic_scas(sh, 0), b=b)
        am, km, nk, _ = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
        plan = hk.heatkv_schedule_plan(sch, layout)
        ms = np.zeros(sh.K)
        for rep in range(reps + 1):
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            for step in range(sh.K - 1):
                flush.fill_(step)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                # compact_ragged: the eviction before the scale and the update after the layer (in-place
                # compaction of G_k \\ A_k, then the append) are timed together
                if name != "compact_ragged":
                    ses.pre_step(ids, step)
                e0.record(stream)
                if name == "compact_ragged":
                    ses.pre_step(ids, step)
                hk.heatkv_append_compact(ses.ctx, ids, 0, step, ks[step], vs[step], None)
                e1.record(stream)
                torch.cuda.synchronize()
                if rep > 0:
                    ms[step] += e0.elapsed_time(e1) / reps
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
        rows = []
        hdr = plan[:20]
        for step in range(first_scale - 1, sh.K - 1):
            storing = sum(1 for h in range(sh.H) if (int(km[step, 0, h]) >> step) & 1)
            nbytes = 8 * sh.d * sh.t[step] * storing * sh.n_seq
            if fp8:      # K and V: 2 d bytes read, d codes + 1 exponent byte written, per token
                nbytes = 2 * (2 * sh.d + sh.d + 1) * sh.t[step] * storing * sh.n_seq
            if name == "compact_ragged":
                # plus the tokens moved by both evictions of the step: the plan's move lists (src, dst, n, 0)
                off_move = int(hdr[10])
                moved = 0
                for off_b, off_c in ((int(hdr[11]), int(hdr[12])), (int(hdr[13]), int(hdr[14]))):
                    for h in range(sh.H):
                        u = (step * sh.L + 0) * sh.H + h
                        b0, cnt = int(plan[off_b + u]), int(plan[off_c + u])
                        for m in range(cnt):
                            moved += int(plan[off_move + 4 * (b0 + m) + 2])
                nbytes += 8 * sh.d * moved * sh.n_seq
            if nbytes and ms[step] > 0:
                rows.append({"scale": step + 1, "MB": round(nbytes / 1e6, 2), "us": round(ms[step] * 1e3, 2),
                             **({"moved_tokens_per_seq": moved} if name == "compact_ragged" else {}),
                             "GBs": round(nbytes / (ms[step] * 1e-3) / 1e9, 1),
                             "frac": round(nbytes / (ms[step] * 1e-3) / 1e9 / pk["hbm_gbs"], 3)})
        out[name] = rows
        st = hk.heatkv_kernel_launches(ses.ctx)
        out[name + "_kernels"] = {"append_kernel": int(st.append), "compact_kernel": int(st.compact)}
        hk.heatkv_schedule_free(sch)
        ses.close()
    del ks, vs, flush
    torch.cuda.empty_cache()
    return out


def run_cache_workload(args):
    torch.cuda.set_device(0)
    print(json.dumps(cache_update_numbers(max(3, min(args.steps, 10)))), flush=True)


def run_few_heads_workload(args):
    """Key-range splitting on launches that cannot fill the GPU with whole heads (not the headline line):
    one sequence, 2 or 8 heads, d=128, 13 scales, full or half budget.  Every sweep is timed call by call
    with the scratch region present (splitting allowed) and absent (whole heads only)."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session
    torch.cuda.set_device(0)
    rows = []
    for H, b in ((2, 1.0), (8, 0.5)):
        sh = W.Shape("few_heads", L=1, H=H, d=128, sides=W.SIDES_13, n_seq=1, s=3)
        scores = W.synthetic_scas(sh, 0)
        q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
        c = [0] + sh.c
        qs, ks, vs = ([x[:, :, c[i]:c[i + 1]].contiguous() for i in range(sh.K)] for x in (q, k, v))
        outs = [torch.zeros_like(x) for x in qs]
        flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
        res = {"H": H, "budget": b}
        for name, scratch in (("whole_heads_ms", 1024), ("split_ms", 1 << 27)):
            ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=2 * sh.H * (sh.c[-2] + 64 * sh.K), scratch_bytes=scratch)
            sch = ses.schedule(scas=scores, b=b)
            ms, reps = np.zeros(sh.K), max(3, min(args.steps, 20))
            for rep in range(reps + 2):
                ids = [hk.heatkv_seq_open(ses.ctx, sch)]
                if rep == 0 and scratch > 1024:
                    res["split_tiles_per_scale"] = [hk.heatkv_attention_split(ses.ctx, ids, 0, st)[0] for st in range(sh.K)]
                    res["ctas_per_scale"] = [hk.heatkv_attention_split(ses.ctx, ids, 0, st)[1] for st in range(sh.K)]
                for step in range(sh.K):
                    ses.pre_step(ids, step)
                    flush.fill_(1)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    hk.heatkv_scale_attention(ses.ctx, ids, 0, step, qs[step], ks[step], vs[step], None, None, outs[step])
                    e1.record()
                    hk.heatkv_append_compact(ses.ctx, ids, 0, step, ks[step], vs[step], None)
                    torch.cuda.synchronize()
                    if rep >= 2:
                        ms[step] += e0.elapsed_time(e1) / reps
                hk.heatkv_seq_close(ses.ctx, ids[0])
            res[name] = [round(float(x), 4) for x in ms]
            res[name.replace("_ms", "_sum_ms")] = round(float(ms.sum()), 4)
            assert hk.heatkv_device_status(ses.ctx) == 0
            hk.heatkv_schedule_free(sch)
            ses.close()
        rows.append(res)
    print(json.dumps({"workload": "few_heads_key_range_splitting", "runs": rows}), flush=True)


def run_head_dim_64_workload(args):
    """A layer of the same width as the headline's with heads of 64 instead of 128 dimensions (32 heads, 13
    scales, batch 2, budget 1/20; not the headline line): every sweep timed call by call on the tcgen05 kernel's
    head_dim-64 instantiation (kernel auto) and on the warp-level MMA kernel alone."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session
    torch.cuda.set_device(0)
    sh = W.Shape("width2048_d64", L=1, H=32, d=64, sides=W.SIDES_13, n_seq=2, s=3)
    scores = W.synthetic_scas(sh, 0)
    q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
    c = [0] + sh.c
    qs, ks, vs = ([x[:, :, c[i]:c[i + 1]].contiguous() for i in range(sh.K)] for x in (q, k, v))
    outs = [torch.zeros_like(x) for x in qs]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    res = {"workload": "head_dim_64_layer", "H": sh.H, "d": sh.d, "n_seq": sh.n_seq, "budget": B_BUDGET}
    for name, kernel in (("auto", hk.KERNEL_AUTO), ("generic", hk.KERNEL_GENERIC)):
        ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=2 * sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K), kernel=kernel)
        sch = ses.schedule(scas=scores, b=B_BUDGET)
        am, _, _, _ = hk.heatkv_schedule_masks(sch, sh.K, sh.L, sh.H)
        flops = attention_flops(sh, am, sh.n_seq)
        ms, reps = np.zeros(sh.K), max(3, min(args.steps, 20))
        for rep in range(reps + 2):
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            for step in range(sh.K):
                ses.pre_step(ids, step)
                flush.fill_(1)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                hk.heatkv_attention_append(ses.ctx, ids, 0, step, qs[step], ks[step], vs[step], None, None, outs[step])
                e1.record()
                torch.cuda.synchronize()
                if rep >= 2:
                    ms[step] += e0.elapsed_time(e1) / reps
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
        assert hk.heatkv_device_status(ses.ctx) == 0
        res[name + "_ms_per_scale"] = [round(float(x), 4) for x in ms]
        res[name + "_sum_ms"] = round(float(ms.sum()), 4)
        res[name + "_tflops_largest"] = round(flops[sh.K - 1] / (float(ms[sh.K - 1]) * 1e-3) / 1e12, 1)
        hk.heatkv_schedule_free(sch)
        ses.close()
    print(json.dumps(res), flush=True)


def run_fp8_cache_workload(args):
    """The single-layer workload (16 heads, d=128, 13 scales, batch 2, budget 1/20) with the bf16 cache and with
    the fp8 cache (not the headline line): layer sweeps timed call by call, heatkv_attention_append per step.
    With the fp8 cache a step is three kernels (expansion of the visible rows, attention, quantising append)
    instead of one; the cache at the end of the sweep takes (d + 1) / (2 d) of the bytes."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session
    torch.cuda.set_device(0)
    sh = W.CFG2
    scores = W.synthetic_scas(sh, 0)
    q, k, v = W.qkv_layer(sh, 0, 0, device="cuda")
    c = [0] + sh.c
    qs, ks, vs = ([x[:, :, c[i]:c[i + 1]].contiguous() for i in range(sh.K)] for x in (q, k, v))
    outs = [torch.zeros_like(x) for x in qs]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    res = {"workload": "fp8_cache_single_layer", "H": sh.H, "d": sh.d, "n_seq": sh.n_seq, "budget": B_BUDGET,
           "scores": "synthetic"}
    for name, dtype in (("bf16", hk.CACHE_BF16), ("fp8", hk.CACHE_FP8_E4M3)):
        ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=2 * sh.n_seq * sh.H * (sh.c[-2] + 64 * sh.K), cache_dtype=dtype)
        sch = ses.schedule(scas=scores, b=B_BUDGET)
        ms, reps = np.zeros(sh.K), max(3, min(args.steps, 20))
        n0 = hk.heatkv_launch_count(ses.ctx)
        for rep in range(reps + 2):
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            for step in range(sh.K):
                ses.pre_step(ids, step)
                flush.fill_(1)
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                e0.record()
                hk.heatkv_attention_append(ses.ctx, ids, 0, step, qs[step], ks[step], vs[step], None, None, outs[step])
                e1.record()
                torch.cuda.synchronize()
                if rep >= 2:
                    ms[step] += e0.elapsed_time(e1) / reps
            if rep == reps + 1:
                res[name + "_cache_bytes_per_sequence"] = int(hk.heatkv_cache_bytes(ses.ctx, ids[0])[0])
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
        assert hk.heatkv_device_status(ses.ctx) == 0
        res[name + "_ms_per_scale"] = [round(float(x), 4) for x in ms]
        res[name + "_sum_ms"] = round(float(ms.sum()), 4)
        res[name + "_launches_per_sweep"] = int((hk.heatkv_launch_count(ses.ctx) - n0) // (reps + 2))

        # the same sweep as one CUDA graph (what a generation loop would replay): launch gaps mostly gone
        def sweep_once():
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(sh.n_seq)]
            for step in range(sh.K):
                ses.pre_step(ids, step)
                hk.heatkv_attention_append(ses.ctx, ids, 0, step, qs[step], ks[step], vs[step], None, None, outs[step])
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            sweep_once()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            sweep_once()
        g.replay()
        torch.cuda.synchronize()
        gms = 0.0
        for rep in range(reps):
            flush.fill_(2)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            g.replay()
            e1.record()
            torch.cuda.synchronize()
            gms += e0.elapsed_time(e1) / reps
        assert hk.heatkv_device_status(ses.ctx) == 0
        res[name + "_graph_sweep_ms"] = round(gms, 4)
        del g
        hk.heatkv_schedule_free(sch)
        ses.close()
    print(json.dumps(res), flush=True)


def run_stability_workload(args):
    """Synthetic analogue of the paper's S-CAS stability study (not the headline line): the S-CAS head
    ordering is computed from 10 independently seeded calibration sets (4 sequences each) of a 4-layer x
    16-head model with per-head log-normal locality, and the spread of every head's rank position across
    the runs is reported per source scale, as the appendix does."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.analysis import scas_rank_dispersion
    from paper_2605_14877_b200.sweep import Session
    torch.cuda.set_device(0)
    sh = W.Shape("stability", L=4, H=16, d=128, sides=W.SIDES_13, n_seq=2, s=3)
    bias = torch.from_numpy(W.seg_bias_prior_lognormal(sh, 0)).cuda()
    ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=64)
    runs, n_runs, batches = [], 10, 2
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    calib_ms = 0.0
    for run in range(n_runs):
        beta = torch.zeros(sh.L, sh.H, sh.K, sh.K, dtype=torch.float32, device="cuda")
        for bt in range(batches):
            for l in range(sh.L):
                q, k, _ = W.qkv_layer(sh, 1000 + run * batches + bt, l, device="cuda")
                ev0.record()
                for step in range(sh.K):
                    lo, hi = ses.step_slices(step)
                    qs, ks = q[:, :, lo:hi], k[:, :, :hi]
                    hk.heatkv_calibrate_scores(ses.ctx, l, step, sh.n_seq, qs, ks, None, hk.Strides.of(qs, ks),
                                               bias[l, step], beta, None)
                ev1.record()
                torch.cuda.synchronize()
                calib_ms += ev0.elapsed_time(ev1)
        _, scas, _ = hk.heatkv_finalize_scores(ses.ctx, beta, batches * sh.n_seq, sh.L, sh.H, sh.K)
        runs.append(scas)
    assert hk.heatkv_device_status(ses.ctx) == 0
    ses.close()
    disp = scas_rank_dispersion(np.stack(runs), sh.s)
    T = sh.L * sh.H
    print(json.dumps({"workload": "scas_rank_stability", "heads": T, "runs": n_runs, "samples_per_run": batches * sh.n_seq,
                      "rank_std_per_source_scale": {str(k + 1): round(float(disp[k]), 3) for k in range(sh.s, sh.K - 1)},
                      "worst_fraction_of_ordering_range": round(float(disp.max()) / T, 4),
                      "calibration_ms_total": round(calib_ms, 2)}), flush=True)


def run_model_workload(args, which):
    print(json.dumps(model_workload(which, max(1, min(args.steps, 3)), args.launch == "graph")), flush=True)


def model_workload(which, reps, with_graph, only_budget=None):
    """Whole-model sweeps (not the headline metric).  `full`: 2B-class full model cache, 32 layers x 16
    heads, batch 8, budgets 1/5, 1/10, 1/20.  `larger`: 40 layers x 32 heads, batch 16, 1/20.  `serving`:
    64 concurrent images of the 2B shape, per-request budgets from {1/5, 1/10, 1/20, 1/40}, paged cache,
    four admission waves one scale apart.  All layers reuse one layer's seeded activations (the kernels see
    per-layer schedules, caches and biases); one heatkv_attention_append call per (step, layer) in generation order.
    Attention + cache path only: images/s excludes everything else a model does."""
    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session
    torch.cuda.set_device(0)
    sh = {"full": W.CFG3, "larger": W.CFG4, "serving": W.CFG5}[which]
    scores = W.synthetic_scas(sh, 0)
    bias_dev = torch.from_numpy(W.seg_bias_prior_lognormal(sh, 0)).cuda()
    data = W.qkv_layer(sh, 0, 0, device="cuda")
    out = torch.zeros_like(data[0])
    cfg0 = hk.Config.make(sh.L, sh.H, sh.d, sh.t, sh.s)
    results = []
    runs = {"full": [[b] * sh.n_seq for b in (1 / 5, 1 / 10, 1 / 20) if only_budget is None or abs(b - only_budget) < 1e-9],
            "larger": [[1 / 20] * sh.n_seq], "serving": [W.serving_budgets(sh.n_seq, 0)]}[which]
    n_waves = 4 if which == "serving" else 1
    wave = sh.n_seq // n_waves
    for budgets in runs:
        schs, rows = {}, {}
        for b in sorted(set(budgets)):
            schs[b] = hk.heatkv_build_schedule(cfg0, scas=scores, b=b)
            rows[b] = hk.heatkv_schedule_footprint(schs[b], hk.LAYOUT_PAGED)[1]
        pool_rows = sum(rows[b] for b in budgets) + 64
        ses = Session(sh.L, sh.H, sh.d, sh.t, sh.s, pool_rows=pool_rows, meta_bytes=256 << 20)
        stream = torch.cuda.current_stream()

        def generation(measure):
            ids = [None] * sh.n_seq
            peak_used, peak_reserved = 0, 0
            for tick in range(sh.K + n_waves - 1):
                for w in range(n_waves):
                    step = tick - w
                    if step < 0 or step >= sh.K:
                        continue
                    members = list(range(w * wave, (w + 1) * wave))
                    if step == 0:
                        for s_ in members:
                            ids[s_] = hk.heatkv_seq_open(ses.ctx, schs[budgets[s_]])
                    wid = [ids[s_] for s_ in members]
                    lo, hi = ses.step_slices(step)
                    q, k, v = (x[members[0]: members[-1] + 1, :, lo:hi] for x in data)
                    o = out[members[0]: members[-1] + 1, :, lo:hi]
                    st = hk.Strides.of(q, k, o)
                    ses.pre_step(wid, step)
                    for l in range(sh.L):
                        hk.heatkv_attention_append(ses.ctx, wid, l, step, q, k, v, st, bias_dev[l, step], o)
                if measure:
                    a = hk.heatkv_allocator_stats(ses.ctx)
                    peak_used, peak_reserved = max(peak_used, a.used_tokens), max(peak_reserved, a.reserved_rows)
            a = hk.heatkv_allocator_stats(ses.ctx)
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)
            return a, peak_used, peak_reserved

        generation(False)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0 = time.perf_counter()
        e0.record(stream)
        for _ in range(reps):
            a, peak_used, peak_reserved = generation(True)
        e1.record(stream)
        torch.cuda.synchronize()
        ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0)) / reps
        assert hk.heatkv_device_status(ses.ctx) == 0
        # the same generation as one CUDA graph (all launches of all layers and scales), replayed
        graph_ms = None
        if with_graph:
            side = torch.cuda.Stream()
            side.wait_stream(torch.cuda.current_stream())
            with torch.cuda.stream(side):
                generation(False)
            torch.cuda.current_stream().wait_stream(side)
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                generation(False)
            g.replay()
            torch.cuda.synchronize()
            e0.record(stream)
            for _ in range(reps):
                g.replay()
            e1.record(stream)
            torch.cuda.synchronize()
            graph_ms = e0.elapsed_time(e1) / reps
            assert hk.heatkv_device_status(ses.ctx) == 0
        n_images = sh.n_seq / (2 if which != "serving" else 1)      # cond/uncond pair = one image outside serving
        # algorithmic attention flops of the generation (4*d*t_k*n_vis over all sequences, layers, heads, scales)
        gen_flops = 0
        for b in sorted(set(budgets)):
            am_b = hk.heatkv_schedule_masks(schs[b], sh.K, sh.L, sh.H)[0]
            gen_flops += sum(attention_flops(sh, am_b, sum(1 for x in budgets if x == b)))
        best_ms = min(ms, graph_ms) if graph_ms is not None else ms
        full_bytes = sh.n_seq * sh.L * sh.H * sh.c[-2] * sh.d * 4
        results.append({"budgets": sorted(set(round(b, 4) for b in budgets)), "ms_per_generation": round(ms, 2),
                        "images_per_s": round(n_images / (ms * 1e-3), 2),
                        "graph_ms_per_generation": None if graph_ms is None else round(graph_ms, 2),
                        "graph_images_per_s": None if graph_ms is None else round(n_images / (graph_ms * 1e-3), 2),
                        "attention_tflops": round(gen_flops / (best_ms * 1e-3) / 1e12, 1),
                        "attention_frac_of_bf16_peak": round(gen_flops / (best_ms * 1e-3) / 1e12 / peaks()["bf16_tflops_sustained"], 3),
                        "cache_GB_end": round(a.used_tokens * sh.d * 4 / 1e9, 3),
                        "cache_GB_uncompressed": round(full_bytes / 1e9, 3),
                        "reserved_GB": round(a.reserved_rows * sh.d * 4 / 1e9, 3),
                        "occupancy_end": round(a.used_tokens / max(a.reserved_rows, 1), 3),
                        "peak_reserved_rows": int(peak_reserved), "pool_rows": int(a.pool_rows)})
        for sch in schs.values():
            hk.heatkv_schedule_free(sch)
        ses.close()
    del data, out
    torch.cuda.empty_cache()
    return ({"workload": sh.name, "L": sh.L, "H": sh.H, "n_seq": sh.n_seq, "launch": "calls issued from Python (ms_per_generation) and one CUDA graph replay (graph_*)",
                      "data": "synthetic, one layer's activations reused by all layers",
                      "peak": "attention_frac_of_bf16_peak is against the %s sustained bf16 figure (a generation lasts tens of milliseconds and more)" % peaks()["source"],
                      "runs": results})


def main():
    global N_LAYERS
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--layout", default="paged", choices=["paged", "ragged"])
    ap.add_argument("--kernel", default="auto", choices=["auto", "generic", "tcgen05"])
    ap.add_argument("--launch", default="graph", choices=["graph", "eager"],
                    help="timed steps replay one captured CUDA graph of the 32 x 13 launches, or issue every call")
    ap.add_argument("--calls", default="fused", choices=["fused", "separate"],
                    help="fused: heatkv_attention_append (one launch per step in the paged layout); separate: "
                         "heatkv_scale_attention followed by heatkv_append_compact")
    ap.add_argument("--workload", default="config2", choices=["config2", "cache", "full", "larger", "serving", "fewheads", "stability", "d64", "fp8"],
                    help="config2: the headline line; cache: append / compaction GB/s at a saturating shape; "
                         "full / larger / serving: whole-model sweeps of the other workloads; fewheads: key-range "
                         "splitting on launches with few (sequence, head) units; stability: S-CAS rank spread "
                         "over seeded calibration sets")
    ap.add_argument("--layers", type=int, default=N_LAYERS,
                    help="layers one step replays (default: the 2B-class model's 32; profiling runs use 1 to keep the "
                         "device footprint small -- such a line is not the headline metric and says so in config)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true", help="skip the host-buffer leg (profiling runs)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    N_LAYERS = max(1, args.layers)

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if args.impl == "reference":
        run_reference(args, rank)
        return
    if args.workload == "cache":
        if rank == 0:
            run_cache_workload(args)
        return
    if args.workload == "stability":
        if rank == 0:
            run_stability_workload(args)
        return
    if args.workload == "d64":
        run_head_dim_64_workload(args)
        return
    if args.workload == "fp8":
        if rank == 0:
            run_fp8_cache_workload(args)
        return
    if args.workload == "fewheads":
        if rank == 0:
            run_few_heads_workload(args)
        return
    if args.workload in ("full", "larger", "serving"):
        if rank == 0:
            run_model_workload(args, args.workload)
        return

    import paper_2605_14877_b200 as hk
    from paper_2605_14877_b200.sweep import Session

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    shape = W.CFG2
    layout = hk.LAYOUT_PAGED if args.layout == "paged" else hk.LAYOUT_RAGGED
    kernel = {"auto": hk.KERNEL_AUTO, "generic": hk.KERNEL_GENERIC, "tcgen05": hk.KERNEL_TCGEN05}[args.kernel]
    n_seq = shape.n_seq
    ses = Session(shape.L, shape.H, shape.d, shape.t, shape.s,
                  pool_rows=2 * n_seq * shape.L * shape.H * (shape.c[-2] + 64 * shape.K), layout=layout,
                  kernel=kernel, device=str(dev))
    bias_np = W.seg_bias_current_scale(shape, DATA_SEED)
    bias = torch.from_numpy(bias_np).to(dev)

    # ---- offline part (untimed): calibration on seeded samples -> S-CAS -> static schedule
    beta = torch.zeros(shape.L, shape.H, shape.K, shape.K, dtype=torch.float32, device=dev)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    calib_ms, calib_ms_step_calls = 0.0, 0.0
    for i, seed in enumerate([CALIB_SEEDS[0]] + list(CALIB_SEEDS)):
        # the first pass is a warm-up into a scratch accumulator (first launches load the kernels), not timed
        acc = torch.zeros_like(beta) if i == 0 else beta
        q, k, v = W.qkv_layer(shape, seed, 0, device=dev)
        # all 13 steps of the sample batch in one call (one tensor-memory launch over the large steps) ...
        ev0.record()
        hk.heatkv_calibrate_scores_steps(ses.ctx, 0, 0, shape.K, n_seq, q, k, hk.Strides.of(q, k), bias[0], acc)
        ev1.record()
        torch.cuda.synchronize()
        if i > 0:
            calib_ms += ev0.elapsed_time(ev1)
        # ... and step by step, as a calibration that rides on a real forward pass issues them (into a scratch copy)
        scratch_acc = torch.zeros_like(beta)
        ev0.record()
        for step in range(shape.K):
            lo, hi = ses.step_slices(step)
            qs, ks = q[:, :, lo:hi], k[:, :, :hi]
            hk.heatkv_calibrate_scores(ses.ctx, 0, step, n_seq, qs, ks, None, hk.Strides.of(qs, ks), bias[0, step],
                                       scratch_acc, None)
        ev1.record()
        torch.cuda.synchronize()
        if i > 0:
            calib_ms_step_calls += ev0.elapsed_time(ev1)
        del q, k, v, scratch_acc
    _, scas, _ = hk.heatkv_finalize_scores(ses.ctx, beta, len(CALIB_SEEDS) * n_seq, shape.L, shape.H, shape.K)
    sch = ses.schedule(scas=scas, b=B_BUDGET)
    am, km, nk, budget = hk.heatkv_schedule_masks(sch, shape.K, shape.L, shape.H)
    flops = attention_flops(shape, am, n_seq)
    by = attention_bytes(shape, am, n_seq)
    calib_flops = sum(2 * shape.d * shape.t[k] * shape.c[k] for k in range(shape.K)) * shape.H * n_seq * len(CALIB_SEEDS)
    tc_steps = [kk for kk in range(shape.K) if args.kernel != "generic" and (shape.t[kk] >= 256 or (shape.t[kk] >= 128 and n_seq * shape.H >= 64) or args.kernel == "tcgen05")]

    # ---- device-resident inputs of the timed workload: per layer, one [n_seq, H, t_k, d] block per scale
    # (N_LAYERS x 345 MB: every layer reads activations of its own, far more than the L2 holds)
    layer_bufs = []
    for layer in range(N_LAYERS):
        q, k, v = W.qkv_layer(shape, DATA_SEED, layer, device=dev)
        bq, bk, bv, bo = [], [], [], []
        for step in range(shape.K):
            lo, hi = ses.step_slices(step)
            bq.append(q[:, :, lo:hi].contiguous()); bk.append(k[:, :, lo:hi].contiguous())
            bv.append(v[:, :, lo:hi].contiguous()); bo.append(torch.zeros_like(bq[-1]))
        layer_bufs.append((bq, bk, bv, bo))
        del q, k, v
    qs_, ks_, vs_, os_ = layer_bufs[0]
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)

    def sweep(events=None, bufs=None):
        """One image pair through one layer: 13 x (pre-step eviction, attention, append/compaction)."""
        stream = torch.cuda.current_stream()
        bq, bk, bv, bo = bufs or (qs_, ks_, vs_, os_)
        ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(n_seq)]
        for step in range(shape.K):
            ses.pre_step(ids, step)
            if events is not None and step in events:
                events[step][0].record(stream)
            if args.calls == "fused":
                hk.heatkv_attention_append(ses.ctx, ids, 0, step, bq[step], bk[step], bv[step], None, bias[0, step], bo[step])
            else:
                hk.heatkv_scale_attention(ses.ctx, ids, 0, step, bq[step], bk[step], bv[step], None, bias[0, step], bo[step])
            if events is not None and step in events:
                events[step][1].record(stream)
            if args.calls != "fused":
                hk.heatkv_append_compact(ses.ctx, ids, 0, step, bk[step], bv[step], None)
        for i in ids:
            hk.heatkv_seq_close(ses.ctx, i)

    def image():
        """One step: the image pair through all N_LAYERS layers (the context is one layer wide, so every layer
        is a fresh pair of sequences on the same pool rows, with that layer's activations)."""
        for layer in range(N_LAYERS):
            sweep(bufs=layer_bufs[layer])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
            torch.cuda.synchronize()

    for _ in range(args.warmup):
        image()
    barrier()
    launches0, kern0 = hk.heatkv_launch_count(ses.ctx), hk.heatkv_kernel_launches(ses.ctx)
    image()
    launches_per_step = hk.heatkv_launch_count(ses.ctx) - launches0
    kern1 = hk.heatkv_kernel_launches(ses.ctx)
    per_step_kernels = {n: int(getattr(kern1, n) - getattr(kern0, n)) for n in
                        ("attention_tcgen05", "attention_generic", "append", "compact")}
    graph = None
    if args.launch == "graph":
        # the calls are plain launches on the current stream once the schedule's plan is resident, so the
        # whole sweep records into one graph; every replay issues the same kernels on the same buffers
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            image()
        torch.cuda.current_stream().wait_stream(side)
        barrier()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            image()
        for _ in range(args.warmup):
            graph.replay()
        barrier()

    # ---- timed region: exactly K steps (images), L2 flushed (untimed) before each
    stream = torch.cuda.current_stream()
    sampler = ClockSampler(local)
    sampler.start()
    step_events = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                   for _ in range(args.steps)]
    barrier()
    for it in range(args.steps):
        flush.fill_(it & 0xff)
        step_events[it][0].record(stream)
        if graph is not None:
            graph.replay()
        else:
            image()
        step_events[it][1].record(stream)
    barrier()
    total_ms = sum(a.elapsed_time(b) for a, b in step_events)

    # ---- kernel durations: layer sweeps issued call by call with events around every attention launch
    n_kern = max(N_LAYERS, min(args.steps, 64))
    kern_events = [{kk: (torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
                    for kk in range(shape.K)} for _ in range(n_kern)]
    for it in range(n_kern):
        flush.fill_(it & 0xff)
        sweep(kern_events[it], layer_bufs[it % N_LAYERS])
    barrier()
    clocks = sampler.stop()
    per_step_ms = np.array([[ke[kk][0].elapsed_time(ke[kk][1]) for kk in range(shape.K)] for ke in kern_events])
    assert hk.heatkv_device_status(ses.ctx) == 0
    # how the tensor-memory launches cut their work (host-side report of the library's choice)
    ids_ = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(n_seq)]
    cuts = [hk.heatkv_attention_split(ses.ctx, ids_, 0, kk) for kk in range(shape.K)]
    for i in ids_:
        hk.heatkv_seq_close(ses.ctx, i)

    # ---- end to end: the same step from pinned host buffers, copies inside the timed region.  Every layer's
    # Q/K/V go up and its output comes down (one pinned set serves all layers: the bytes moved are what counts).
    h2d = N_LAYERS * 3 * sum(x.numel() for x in qs_) * 2
    d2h = N_LAYERS * sum(x.numel() for x in qs_) * 2
    e2e_ms = float("nan")
    e2e_steps = max(3, min(args.steps, 5))
    if not args.no_e2e:
        hq, hkk, hv = ([x.cpu().pin_memory() for x in xs] for xs in (qs_, ks_, vs_))
        hout = [torch.empty_like(x).pin_memory() for x in hq]
        dq, dk, dv, do = ([torch.empty_like(x) for x in xs] for xs in (qs_, ks_, vs_, os_))

        # Three streams, as a caller that feeds the library from the host would do: uploads of the later
        # scales run while the earlier ones compute, and each scale's result goes back as soon as it is done.
        s_in, s_out = torch.cuda.Stream(), torch.cuda.Stream()

        def sweep_e2e():
            ids = [hk.heatkv_seq_open(ses.ctx, sch) for _ in range(n_seq)]
            s_in.wait_stream(stream)                 # the previous sweep has read its inputs
            ev_in = []
            with torch.cuda.stream(s_in):
                for step in range(shape.K):
                    for src, dst in ((hq, dq), (hkk, dk), (hv, dv)):
                        dst[step].copy_(src[step], non_blocking=True)
                    ev = torch.cuda.Event()
                    ev.record(s_in)
                    ev_in.append(ev)
            stream.wait_stream(s_out)                # the previous sweep's results have left the device
            for step in range(shape.K):
                stream.wait_event(ev_in[step])
                ses.pre_step(ids, step)
                if args.calls == "fused":
                    hk.heatkv_attention_append(ses.ctx, ids, 0, step, dq[step], dk[step], dv[step], None, bias[0, step], do[step])
                else:
                    hk.heatkv_scale_attention(ses.ctx, ids, 0, step, dq[step], dk[step], dv[step], None, bias[0, step], do[step])
                    hk.heatkv_append_compact(ses.ctx, ids, 0, step, dk[step], dv[step], None)
                ev = torch.cuda.Event()
                ev.record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev)
                    hout[step].copy_(do[step], non_blocking=True)
            stream.wait_stream(s_out)                # the sweep ends when its last result is on the host
            for i in ids:
                hk.heatkv_seq_close(ses.ctx, i)

        sweep_e2e()
        barrier()
        t0 = time.perf_counter()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(e2e_steps):
            for _layer in range(N_LAYERS):
                sweep_e2e()
        e1.record(stream)
        barrier()
        e2e_ms = max(e0.elapsed_time(e1), 1e3 * (time.perf_counter() - t0)) / e2e_steps

    # ---- aggregate over ranks (replicas): slowest rank's time
    ms_per_step, value, e2e_value = aggregate_replicas(total_ms, e2e_ms, args.steps, dist, dev)   # one image pair per replica

    # ---- which kernels ran (the library's own count), and the cache-update kernels at their saturating shape
    ks1 = hk.heatkv_kernel_launches(ses.ctx)
    if args.kernel != "generic":
        assert ks1.tcgen05_attention_ready == 1 and per_step_kernels["attention_tcgen05"] == N_LAYERS * len(tc_steps), per_step_kernels
    dominant = ("tc::attn_tc_kernel<%d> (tcgen05.mma, TMEM accumulators, TMA gathers)" % shape.d
                if per_step_kernels["attention_tcgen05"] else "attn_generic_kernel<%d> (mma.sync)" % shape.d)
    cache_update = None
    if rank == 0 and world == 1 and args.layout == "paged":
        cu = cache_update_numbers(5, cases=("append_paged", "compact_ragged", "append_fp8_paged"), first_scale=9)
        cache_update = {"shape": cu["shape"], "peak_gbs": cu["peak_gbs"], "peak_source": cu["peak_source"],
                        "append_kernel_paged": cu["append_paged"], "append_plus_compact_kernel_ragged_budget_1_5": cu["compact_ragged"],
                        "append_fp8_kernel_paged": cu["append_fp8_paged"],
                        "kernels_launched": {"append_paged": cu["append_paged_kernels"], "compact_ragged": cu["compact_ragged_kernels"]},
                        "bytes": "algorithmic: 8*d*t_k per storing head, 8*d per moved token; fp8 append: (4*d + 2*(d+1))*t_k per storing head"}

    # ---- roofline of the dominant kernel, all its launches of a layer sweep
    pk = peaks()
    attn_ms = per_step_ms.mean(axis=0)                            # [K] mean duration per launch
    dom_flops = sum(flops[kk] for kk in tc_steps)
    dom_ms = float(sum(attn_ms[kk] for kk in tc_steps))
    achieved = dom_flops / (dom_ms * 1e-3) / 1e12 if tc_steps else 0.0
    big = shape.K - 1
    uncompressed_kv_bytes = sum(2 * shape.c[kk] * shape.d * 2 for kk in range(shape.K)) * shape.H * n_seq
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": shape.name, "L": shape.L, "H": shape.H, "d": shape.d, "scales": shape.K,
                   "tokens": shape.n_tokens, "n_seq": n_seq, "budget": B_BUDGET, "policy": "heatkv", "s": shape.s,
                   "layout": args.layout, "kernel": args.kernel, "launch": args.launch, "calls": args.calls,
                   "layers": N_LAYERS,
                   "l2": "256 MB flush write between timed steps; every layer reads its own 345 MB of activations",
                   "one_image": "cond/uncond pair through the attention + cache path of 32 layers (the single-layer "
                                "workload replayed per layer with that layer's seeded activations); MLP/VAE/text not included",
                   "n_k": [int(x) for x in nk], "replicas": world},
        "ms_per_layer_sweep": ms_per_step / N_LAYERS,
        "image_pairs_per_s_one_layer": value * N_LAYERS,
        "effective_kv_tb_per_s": uncompressed_kv_bytes / (float(attn_ms.sum()) * 1e-3) / 1e12,
        "attention_ms_per_scale": [round(float(x), 5) for x in attn_ms],
        "work_items_per_scale": [int(c[1]) for c in cuts],
        "longest_piece_tiles_per_scale": [int(c[0]) for c in cuts],
        "attention_tflops_per_scale": [round(flops[kk] / (float(attn_ms[kk]) * 1e-3) / 1e12, 1) for kk in range(shape.K)],
        "attention_algorithmic_gb_per_s_per_scale": [round(by[kk] / (float(attn_ms[kk]) * 1e-3) / 1e9, 1) for kk in range(shape.K)],
        "attention_tflops_all_scales": sum(flops) / (float(attn_ms.sum()) * 1e-3) / 1e12,
        "calibration": {"ms_per_sample_batch": calib_ms / len(CALIB_SEEDS),
                        "tflops": calib_flops / (calib_ms * 1e-3) / 1e12, "samples": len(CALIB_SEEDS) * n_seq,
                        "call": "heatkv_calibrate_scores_steps (all 13 steps of a batch in one call)",
                        "ms_per_sample_batch_step_calls": calib_ms_step_calls / len(CALIB_SEEDS)},
        "kernels_per_step": per_step_kernels,
        "roofline": {"bound": "tensor", "kernel": f"{dominant}: its {len(tc_steps)} launches per layer sweep (scales with t_k >= 256), "
                                                  f"{per_step_kernels['attention_tcgen05']} per step",
                     "timing": "CUDA events around each launch, call by call, mean over layer sweeps",
                     "achieved": achieved, "peak": pk["bf16_tflops"], "unit": "TFLOP/s",
                     "frac": achieved / pk["bf16_tflops"], "peak_source": pk["source"] + " burst bf16",
                     "largest_launch": {"scale": big + 1, "tflops": flops[big] / (float(attn_ms[big]) * 1e-3) / 1e12,
                                        "frac": flops[big] / (float(attn_ms[big]) * 1e-3) / 1e12 / pk["bf16_tflops"]},
                     "traffic": captured_traffic(), "traffic_unit": "bytes per layer sweep (7 launches), ncu dram read + write"},
        "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps},
        "gpu_launches": int(launches_per_step * args.steps),
        "clocks": clocks,
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        ctx = oracle_context(shape)
        samples = [(h, list(range(1, shape.K + 1))) for h in (0, 3, 5, 7, 8, 11, 13, 15)] * 5
        v, secs, frac = oracle_images_per_s(shape, ctx, samples)
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
                                "sample": f"{len(samples)} (layer, seq, head) units of {N_LAYERS * shape.n_seq * shape.H}, all 13 scales "
                                          f"(attention + cache contents); {secs:.1f} s of CPU work = {frac:.3g} images, "
                                          "extrapolated by flops"}
    if cache_update is not None:
        line["cache_update"] = cache_update
    hk.heatkv_schedule_free(sch)
    ses.close()
    if rank == 0 and world == 1 and args.layout == "paged" and args.kernel == "auto" and N_LAYERS == 32:
        # the same model at the batch the paper's full-model workload has (8 sequences = 4 image pairs, 32 layers,
        # budget 1/20): launches large enough to fill the GPU; fraction against the sustained bf16 peak
        del layer_bufs, flush
        torch.cuda.empty_cache()
        line["full_model_batch8"] = model_workload("full", 2, True, only_budget=B_BUDGET)
    if dist is not None:
        dist.barrier()
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


if __name__ == "__main__":
    main()
