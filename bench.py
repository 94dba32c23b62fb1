"""Benchmark: batch-1 Speculative Thinking decode of the 1.5B + 32B pair on one B200.

A step is one whole generation of the workload (prompt prefill, small-model decode, handoffs with
catch-up prefill, target segments).  Prints one JSON line.
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

import numpy as np

from paper_2504_12329_b200 import workloads as W

METRIC = "tokens/s batch-1 1.5B+32B spec-thinking decode; % of HBM roofline"
UNIT = "tokens/s"


def measured_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def measured_tensor_peak():
    """Dense bf16 TFLOP/s of a long-running GEMM (the multi-row passes run for tens of milliseconds)."""
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d.get("bf16_tflops_sustained", d["bf16_tflops"])), "measured (sustained)"
    return 1400.0, "fallback (sustained)"


def paper_accounting(r, wl):
    """The paper's own figures for this run, as context: share of target tokens and its FLOP-model speed estimate
    (formulas as printed, capacity constant 3.12e10 FLOP/s -- accounting, not a measurement)."""
    from paper_2504_12329_b200 import accounting as A
    return {"modify_ratio": A.modify_ratio(r.source),
            "estimated_speed_tokens_per_s": A.estimated_speed(r, wl.prompt_len, wl.small.as_dict(), wl.large.as_dict() if wl.large else None),
            "note": "paper's FLOP model and capacity constant; context only"}


def time_multi_row_passes(torch, model, shape, ctx, row_counts, hbm_peak):
    """Catch-up / prefill passes of one model on their own: `rows` new tokens over `ctx` cached ones, timed with
    CUDA events on the launching stream.  Every pass streams the model's weights once (larger than L2)."""
    tensor_peak, tensor_kind = measured_tensor_peak()
    lm_head_bytes = 2 * shape.vocab * shape.hidden
    layer_params = (model.st_weight_bytes() - lm_head_bytes) / 2
    out = []
    for rows in row_counts:
        best = None
        for rep in range(3):
            slot = model.st_seq_alloc()
            i = 0
            while i < ctx:
                c = min(256, ctx - i)
                model.st_prefill(slot, W.prompt_ids(7 + i, c, shape.vocab))
                i += c
            toks = W.prompt_ids(99, rows, shape.vocab)
            torch.cuda.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            model.st_prefill(slot, toks)
            e1.record()
            torch.cuda.synchronize()
            t = e0.elapsed_time(e1) * 1e-3
            model.st_seq_free(slot)
            if rep > 0:
                best = t if best is None else min(best, t)
        flops = 2.0 * rows * layer_params + 2.0 * lm_head_bytes / 2 \
            + 4.0 * rows * (ctx + rows / 2) * shape.n_q_heads * shape.head_dim * shape.n_layers
        gbs = (model.st_weight_bytes() + model.st_kv_bytes_per_token() * (ctx + rows)) / best / 1e9
        useful = flops / best / 1e12
        hbm_time = (model.st_weight_bytes() / 1e9) / hbm_peak
        tensor_time = 2.0 * flops / 1e12 / tensor_peak      # hi and lo activation planes: two MMAs per product
        out.append({"model": shape.name, "rows": rows, "context": ctx, "ms": best * 1e3, "tokens_per_s": rows / best,
                    "hbm_gbs": gbs, "frac_hbm": gbs / hbm_peak, "tflops_useful": useful, "tflops_issued": 2 * useful,
                    "frac_tensor_useful": useful / tensor_peak, "frac_tensor_issued": 2 * useful / tensor_peak,
                    "bound": "hbm" if hbm_time >= tensor_time else "tensor", "tensor_peak": tensor_peak,
                    "tensor_peak_source": tensor_kind})
    return out


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([x.strip() for x in line.split(",")])

    def stop(self):
        if self.proc:
            self.proc.terminate()
            try:
                self.proc.wait(timeout=5)
            except Exception:
                pass
        rows = [r for r in self.rows if len(r) >= 6]
        sm = [float(r[0]) for r in rows if r[0].replace(".", "").isdigit()]
        mx = [float(r[1]) for r in rows if r[1].replace(".", "").isdigit()]
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        reasons = [n for i, n in enumerate(names) if any(r[2 + i].lower().startswith("active") for r in rows)]
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None, "reasons": reasons}


def cpu_oracle_sample(w: W.Workload, stats: dict | None):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: decode steps of the small
    model (all layers) and decode steps of the large model cut to two layers plus its LM head, scaled
    to the full depth; combined with the workload's pass mix into tokens/s."""
    import ctypes as C
    from oracle import oracle as O
    rng = np.random.default_rng(1)
    cores = os.cpu_count() or 1
    om = O.Model(O.Config(**w.small.as_dict()), w.weight_seed, 0)
    kv = O.KV(om, 64)
    kv.forward(rng.integers(0, w.small.vocab, 4))
    n_s = 6
    t0 = time.perf_counter()
    for _ in range(n_s):
        kv.forward(rng.integers(0, w.small.vocab, 1))
    t_small = (time.perf_counter() - t0) / n_s
    om.close()
    t_large = None
    sample = f"{n_s} decode steps of the {w.small.name} oracle"
    if w.large is not None:
        sh = w.large.as_dict()
        sh["n_layers"] = 2
        ol = O.Model(O.Config(**sh), w.weight_seed, 1)
        kv = O.KV(ol, 64)
        kv.forward(rng.integers(0, w.large.vocab, 2))
        n_l = 3
        t0 = time.perf_counter()
        for _ in range(n_l):
            kv.forward(rng.integers(0, w.large.vocab, 1))
        t_with_head = (time.perf_counter() - t0) / n_l
        t0 = time.perf_counter()
        for _ in range(n_l):   # the same steps without the LM head (no logits requested)
            tok = np.ascontiguousarray(rng.integers(0, w.large.vocab, 1), dtype=np.int32)
            O.lib().orc_forward(ol.h, kv.h, tok.ctypes.data_as(C.c_void_p), 1, 0, None)
        t_layers2 = (time.perf_counter() - t0) / n_l
        t_large = t_layers2 / 2 * w.large.n_layers + max(t_with_head - t_layers2, 0.0)
        ol.close()
        sample += (f" + {2 * n_l} decode steps of the {w.large.name} oracle cut to 2 layers (with and without LM head), "
                   f"scaled to {w.large.n_layers} layers")
    if stats:
        total = stats["steps_small"] * t_small + stats["steps_large"] * (t_large or 0.0)
        value = stats["n_tokens"] / total
        sample += (f"; combined with the run's pass mix ({stats['steps_small']} small, {stats['steps_large']} large passes; "
                   "a catch-up pass counted as one decode pass)")
    else:
        value = 1.0 / t_small
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
            "s_per_small_step": t_small, "s_per_large_step": t_large}


def schedule_stats(w: W.Workload):
    """Pass mix of the workload from its forcing schedule alone: a replay of the handoff rule on the
    forced tokens, unforced steps counted as ordinary tokens."""
    _, force = W.workload_inputs(w)
    active, remaining, gen, t, last = 0, 0, 0, 0, -1
    steps = [0, 0]
    while gen < w.max_new_tokens:
        tok = int(force[t]) if force is not None and t < len(force) and force[t] >= 0 else -2
        steps[active] += 1
        t += 1
        if w.large is not None and active == 0 and last == W.DELIMITER_ID and tok in W.KEYWORD_IDS:
            active, remaining = 1, W.N1
            continue
        last = tok
        gen += 1
        if active == 1:
            remaining -= 1
            if remaining == 0:
                active = 0
    return {"steps_small": steps[0], "steps_large": steps[1], "n_tokens": gen}


def aggregate_over_ranks(dev_s: float, e2e_s: float, n_tokens: float, dist_mod=None, device="cpu"):
    """Whole-job figures of a replicas-only run: time = the slowest rank, tokens = the sum over ranks."""
    if dist_mod is None or not dist_mod.is_initialized() or dist_mod.get_world_size() == 1:
        return dev_s, e2e_s, n_tokens
    import torch
    t = torch.tensor([dev_s, e2e_s], dtype=torch.float64, device=device)
    dist_mod.all_reduce(t, op=dist_mod.ReduceOp.MAX)
    n = torch.tensor([n_tokens], dtype=torch.float64, device=device)
    dist_mod.all_reduce(n, op=dist_mod.ReduceOp.SUM)
    return float(t[0]), float(t[1]), float(n[0])


def rank_workload(w: W.Workload, rank: int) -> W.Workload:
    """Each rank runs an independent replica of the workload with its own input seed."""
    return W.Workload(**{**w.__dict__, "input_seed": w.input_seed + 1000 * rank})


def run_reference(args, w):
    if int(os.environ.get("RANK", "0")) != 0:
        return
    stats = schedule_stats(w)
    vals, base = [], None
    for _ in range(args.warmup + args.steps):
        base = cpu_oracle_sample(w, stats)
        vals.append(base["value"])
    v = float(np.mean(vals[args.warmup:]))
    base["value"] = v
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": 1e3 * stats["n_tokens"] / v, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": w.name, "prompt_len": w.prompt_len, "max_new_tokens": w.max_new_tokens},
            "cpu_baseline": base,
            "e2e": {"value": v, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="qwen1p5b_32b", choices=sorted(W.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--max-new", type=int, default=0, help="shorten the generation (profiling runs only)")
    ap.add_argument("--mean-interval", type=float, default=0.0, help="delimiter spacing override (profiling runs only)")
    ap.add_argument("--layers", type=int, default=0, help="cut both models to this many layers (profiling runs only)")
    args = ap.parse_args()
    w = W.CONFIGS[args.workload]
    if args.max_new > 0 or args.mean_interval > 0:
        w = W.Workload(**{**w.__dict__, "name": w.name + "-short",
                          "max_new_tokens": args.max_new if args.max_new > 0 else w.max_new_tokens,
                          "mean_interval": args.mean_interval if args.mean_interval > 0 else w.mean_interval})
    if args.layers > 0:
        import dataclasses
        cut = lambda sh: None if sh is None else dataclasses.replace(sh, name=f"{sh.name}-{args.layers}L", n_layers=args.layers)
        w = W.Workload(**{**w.__dict__, "name": w.name + f"-{args.layers}L", "small": cut(w.small), "large": cut(w.large)})
    if args.impl == "reference":
        return run_reference(args, w)

    import torch
    import torch.distributed as dist
    from paper_2504_12329_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    # The generation is one dependent chain of tokens: it does not shard.  With N > 1 every rank runs
    # an independent replica of the workload (its own input seed); there is no data-path collective.
    wl = rank_workload(w, rank)
    prompt, force = W.workload_inputs(wl)
    cap = wl.prompt_len + wl.max_new_tokens + 64
    # room for the batched decode measurement at the end: BATCH more sequences of BATCH_CTX + 64 tokens on the large model
    BATCH, BATCH_CTX = 64, 512
    small = B.Model(wl.small.as_dict(), seed=wl.weight_seed, tag=0, max_tokens=cap)
    large = B.Model(wl.large.as_dict(), seed=wl.weight_seed, tag=1, max_seqs=BATCH + 1,
                    max_tokens=cap + BATCH * (BATCH_CTX + 64)) if wl.large else None
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1, max_new_tokens=wl.max_new_tokens, force=force)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(args.warmup):
        B.st_generate_spec(small, large, prompt, **kw)
    sampler = ClockSampler(local)
    launches0 = B.st_kernel_launches()
    barrier()
    sampler.start()
    dev_s, e2e_s, results = 0.0, 0.0, []
    t_region = time.perf_counter()
    for _ in range(args.steps):
        t0 = time.perf_counter()
        r = B.st_generate_spec(small, large, prompt, **kw)   # host buffers in, host buffers out
        e2e_s += time.perf_counter() - t0
        dev_s += r.seconds
        results.append(r)
    barrier()
    t_region = time.perf_counter() - t_region
    clocks = sampler.stop()
    launches = B.st_kernel_launches() - launches0

    r = results[-1]
    n_tokens = float(sum(len(x.tokens) for x in results))
    dev_s, e2e_s, n_tokens = aggregate_over_ranks(dev_s, e2e_s, n_tokens, dist if world > 1 else None, "cuda")
    value = n_tokens / dev_s
    e2e_value = n_tokens / e2e_s

    peak, peak_kind = measured_peaks()
    # Dominant kernel: the single-kernel decode step of the large model (it moves ~3/4 of the run's bytes).
    # Timed on its own after the run: back-to-back launches with CUDA events on the launching stream
    # (torch's current stream), at a mid-run context length; every launch streams all weights (>> L2).
    dom = large if large is not None else small
    shp = wl.large if wl.large else wl.small
    ctx = min(3000, cap - 64)
    slot = dom.st_seq_alloc()
    dom.st_prefill(slot, W.prompt_ids(7, ctx, shp.vocab))
    tok_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    amax_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(3):
        dom.st_decode_step([slot], tok_dev, None, amax_dev)
    n_k = 20
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n_k):
        dom.st_decode_step([slot], tok_dev, None, amax_dev)
    e1.record()
    torch.cuda.synchronize()
    kern_s = e0.elapsed_time(e1) * 1e-3 / n_k
    kern_bytes = dom.st_weight_bytes() + dom.st_kv_bytes_per_token() * (ctx + 3 + n_k // 2)
    achieved = kern_bytes / kern_s / 1e9
    dom.st_seq_free(slot)
    # multi-row passes (handoff catch-up and prompt prefill) of the same model, and the small model's decode step
    mean_catchup = int(np.mean([h[2] for h in r.handoffs])) if len(r.handoffs) else 128
    prefill = time_multi_row_passes(torch, dom, shp, max(0, min(1024, cap - 64 - 256)), [min(256, max(2, mean_catchup)), 256], peak)
    small_step = None
    if large is not None:
        sslot = small.st_seq_alloc()
        small.st_prefill(sslot, W.prompt_ids(7, ctx, wl.small.vocab))
        for _ in range(3):
            small.st_decode_step([sslot], tok_dev, None, amax_dev)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(n_k):
            small.st_decode_step([sslot], tok_dev, None, amax_dev)
        e1.record()
        torch.cuda.synchronize()
        s_s = e0.elapsed_time(e1) * 1e-3 / n_k
        s_bytes = small.st_weight_bytes() + small.st_kv_bytes_per_token() * (ctx + 3 + n_k // 2)
        small_step = {"kernel": f"decode_mega_kernel ({wl.small.name}, context {ctx})", "us_per_launch": s_s * 1e6,
                      "achieved": s_bytes / s_s / 1e9, "frac": s_bytes / s_s / 1e9 / peak, "unit": "GB/s"}
        small.st_seq_free(sslot)
    # batched decode of the same model (the 64-sequence workload's step): one pass over the weights for all rows
    batched = None
    if large is not None:
        bslots = [large.st_seq_alloc() for _ in range(BATCH)]
        for i, sl in enumerate(bslots):
            for j in range(0, BATCH_CTX, 256):
                large.st_prefill(sl, W.prompt_ids(50 + i, min(256, BATCH_CTX - j), shp.vocab))
        btok = torch.zeros(BATCH, dtype=torch.int32, device="cuda")
        bamax = torch.zeros(BATCH, dtype=torch.int32, device="cuda")
        for _ in range(3):
            large.st_decode_step(bslots, btok, None, bamax)
        torch.cuda.synchronize()
        n_b = 10
        e0.record()
        for _ in range(n_b):
            large.st_decode_step(bslots, btok, None, bamax)
        e1.record()
        torch.cuda.synchronize()
        b_s = e0.elapsed_time(e1) * 1e-3 / n_b
        b_bytes = large.st_weight_bytes() + large.st_kv_bytes_per_token() * BATCH * (BATCH_CTX + 3 + n_b // 2)
        batched = {"model": shp.name, "batch": BATCH, "context": BATCH_CTX, "ms_per_step": b_s * 1e3, "tokens_per_s": BATCH / b_s,
                   "hbm_gbs": b_bytes / b_s / 1e9, "frac_hbm": b_bytes / b_s / 1e9 / peak,
                   "note": "st_decode_step with 64 sequences: tcgen05 projections, per-sequence attention over paged K/V"}
        for sl in bslots:
            large.st_seq_free(sl)
    path_gbs = sum(x.bytes_algorithmic for x in results) / sum(x.seconds for x in results) / 1e9
    steps_small = int((r.emission_source == 0).sum())
    steps_large = int((r.emission_source == 1).sum())

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dev_s / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "small": wl.small.name, "large": wl.large.name if wl.large else None,
                       "prompt_len": wl.prompt_len, "max_new_tokens": wl.max_new_tokens, "n1": W.N1,
                       "handoffs": len(r.handoffs), "target_share": float(r.source.mean()),
                       "passes_small": steps_small, "passes_large": steps_large,
                       "arithmetic": "bf16 weights and KV, fp32 activations and accumulation",
                       "l2": "inputs larger than L2: every pass streams 3.1 GB (small) or 64 GB (large) of weights",
                       "multi_gpu": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": int(prompt.nbytes + (force.nbytes if force is not None else 0) + min(wl.small.vocab, shp.vocab)),
                    "d2h_bytes_per_step": int(5 * len(r.tokens) + 13 * r.n_steps + 12 * len(r.handoffs) + 80 * r.n_steps)},
            "gpu_launches": int(launches),
            "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                         # DRAM bytes per launch: ncu measured read+write = 1.013 x the algorithmic bytes on a 4-layer
                         # case of this kernel (profiles/decode_mega_kernel_4layer_pair.md); scaled to this launch
                         "traffic": int(1.013 * kern_bytes),
                         "traffic_source": "ncu dram__bytes_read+write on a 4-layer capture, scaled by streamed bytes",
                         "kernel": f"decode_mega_kernel ({shp.name}, one decode step per launch, context {ctx})",
                         "algorithmic_bytes_per_launch": int(kern_bytes),
                         "peak_source": f"{peak_kind} copy bandwidth", "us_per_launch": kern_s * 1e6},
            "path_roofline": {"achieved_gbs": path_gbs, "frac_of_measured_hbm": path_gbs / peak,
                              "frac_of_nominal_8tbs": path_gbs / 8000.0,
                              "note": "algorithmic bytes of every pass (weights + KV) / device time of the generation"},
            "paper_accounting": paper_accounting(r, wl),
            "prefill": prefill,
            "small_model_decode": small_step,
            "batched_decode": batched,
            "wall_s_timed_region": t_region,
        }
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_sample(wl, {"steps_small": steps_small, "steps_large": steps_large,
                                                          "n_tokens": len(r.tokens)})
        print(json.dumps(line), flush=True)
    small.close()
    if large:
        large.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
