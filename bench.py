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
    """Time the CPU oracle, as it stands, on a bounded sample of the workload.

    Small model: a teacher-forced window right after a short prompt (all layers, real per-token cost of the
    projections and the LM head).  Large model: the same on a two-layer cut plus its LM head, scaled to the full
    depth.  The oracle cannot afford to prefill the run's real contexts (its prefill costs seconds per token), so the
    attention cost at the contexts of the run's start, middle and end is timed with the oracle's own attention
    routine on vectors of those lengths and added per layer and head.  Combined with the workload's pass mix into
    tokens/s."""
    import ctypes as C
    from oracle import oracle as O
    rng = np.random.default_rng(1)
    cores = os.cpu_count() or 1
    contexts = [w.prompt_len, w.prompt_len + w.max_new_tokens // 2, w.prompt_len + w.max_new_tokens]

    def attend_seconds(shape, n_keys):   # one query head over n_keys cached keys
        d = shape.head_dim
        q, k, v = rng.standard_normal(d), rng.standard_normal((n_keys, d)), rng.standard_normal((n_keys, d))
        O.attend(q, k, v)
        reps = 3
        t0 = time.perf_counter()
        for _ in range(reps):
            O.attend(q, k, v)
        return (time.perf_counter() - t0) / reps

    def attention_extra(shape):   # mean over the window contexts of the attention time the short-context steps lack
        per_head = np.mean([attend_seconds(shape, c) for c in contexts])
        # the oracle spreads (row, head) pairs over its threads
        return per_head * shape.n_q_heads * shape.n_layers / max(1, min(cores, shape.n_q_heads))

    om = O.Model(O.Config(**w.small.as_dict()), w.weight_seed, 0)
    kv = O.KV(om, 64)
    kv.forward(rng.integers(0, w.small.vocab, 4))
    n_s = 6
    t0 = time.perf_counter()
    for _ in range(n_s):
        kv.forward(rng.integers(0, w.small.vocab, 1))
    t_small = (time.perf_counter() - t0) / n_s
    om.close()
    att_small = attention_extra(w.small)
    t_large = att_large = None
    sample = f"{n_s} decode steps of the {w.small.name} oracle at a short context"
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
        att_large = attention_extra(w.large)
        sample += (f" + {2 * n_l} decode steps of the {w.large.name} oracle cut to 2 layers (with and without LM head), "
                   f"scaled to {w.large.n_layers} layers")
    sample += f"; attention over the run's contexts {contexts} timed with the oracle's attention routine and added per layer and head"
    ts, tl = t_small + att_small, (t_large or 0.0) + (att_large or 0.0)
    if stats:
        total = stats["steps_small"] * ts + stats["steps_large"] * tl
        value = stats["n_tokens"] / total
        sample += (f"; combined with the run's pass mix ({stats['steps_small']} small, {stats['steps_large']} large passes; "
                   "a catch-up pass counted as one decode pass)")
    else:
        value = 1.0 / ts
    return {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
            "s_per_small_step": ts, "s_per_large_step": tl if w.large is not None else None,
            "s_attention_small": att_small, "s_attention_large": att_large}


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


def timed_decode_step(torch, model, shape, ctx, n_launches=20):
    """Back-to-back single-kernel decode steps of one model at a context of `ctx` tokens, timed with CUDA events on
    the launching stream (torch's current stream); every launch streams all weights (far larger than L2)."""
    slot = model.st_seq_alloc()
    for i in range(0, ctx, 256):
        model.st_prefill(slot, W.prompt_ids(7 + i, min(256, ctx - i), shape.vocab))
    tok_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    amax_dev = torch.zeros(1, dtype=torch.int32, device="cuda")
    for _ in range(3):
        model.st_decode_step([slot], tok_dev, None, amax_dev)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n_launches):
        model.st_decode_step([slot], tok_dev, None, amax_dev)
    e1.record()
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) * 1e-3 / n_launches
    nbytes = model.st_weight_bytes() + model.st_kv_bytes_per_token() * (ctx + 3 + n_launches // 2)
    model.st_seq_free(slot)
    return sec, nbytes


def timed_batched_step(torch, model, shape, batch, ctx, peak, n_launches=10):
    slots = [model.st_seq_alloc() for _ in range(batch)]
    for i, sl in enumerate(slots):
        for j in range(0, ctx, 256):
            model.st_prefill(sl, W.prompt_ids(50 + i, min(256, ctx - j), shape.vocab))
    btok = torch.zeros(batch, dtype=torch.int32, device="cuda")
    bamax = torch.zeros(batch, dtype=torch.int32, device="cuda")
    for _ in range(3):
        model.st_decode_step(slots, btok, None, bamax)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record()
    for _ in range(n_launches):
        model.st_decode_step(slots, btok, None, bamax)
    e1.record()
    torch.cuda.synchronize()
    sec = e0.elapsed_time(e1) * 1e-3 / n_launches
    nbytes = model.st_weight_bytes() + model.st_kv_bytes_per_token() * batch * (ctx + 3 + n_launches // 2)
    for sl in slots:
        model.st_seq_free(sl)
    return {"model": shape.name, "batch": batch, "context": ctx, "ms_per_step": sec * 1e3, "tokens_per_s": batch / sec,
            "hbm_gbs": nbytes / sec / 1e9, "frac_hbm": nbytes / sec / 1e9 / peak,
            "note": "st_decode_step with 64 sequences: tcgen05 projections, per-sequence attention over paged K/V"}


def timed_prompt_prefill(torch, model, shape, rows, peak):
    """A long prompt ingested from an empty cache (passes of 256 rows): tokens/s and the tensor fraction."""
    tensor_peak, tensor_kind = measured_tensor_peak()
    toks = W.prompt_ids(123, rows, shape.vocab)
    best = None
    for rep in range(2):
        slot = model.st_seq_alloc()
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        model.st_prefill(slot, toks)
        torch.cuda.synchronize()
        t = time.perf_counter() - t0
        model.st_seq_free(slot)
        best = t if best is None else min(best, t)
    lm_head_bytes = 2 * shape.vocab * shape.hidden
    layer_params = (model.st_weight_bytes() - lm_head_bytes) / 2
    flops = 2.0 * rows * layer_params + 4.0 * rows * (rows / 2) * shape.n_q_heads * shape.head_dim * shape.n_layers
    passes = (rows + 255) // 256
    return {"model": shape.name, "rows": rows, "passes": passes, "ms": best * 1e3, "tokens_per_s": rows / best,
            "tflops_useful": flops / best / 1e12, "frac_tensor_useful": flops / best / 1e12 / tensor_peak,
            "hbm_gbs": passes * model.st_weight_bytes() / best / 1e9, "tensor_peak": tensor_peak, "tensor_peak_source": tensor_kind,
            "timing": "host clock around st_prefill + synchronize (the call syncs between passes)"}


def pass_kind_times(r):
    """Device time per kind of pass (stamped by the router on the device): the run's own version of the paper's table
    of decode against prefix times."""
    out = {}
    for kind, (sec, n) in (r.phase_times or {}).items():
        out[kind] = {"passes": int(n), "seconds": float(sec), "ms_per_pass": 1e3 * float(sec) / n if n else None}
    return out


def generation_summary(r, peak):
    """Figures of one timed generation (device time from the call's own CUDA events)."""
    gbs = r.bytes_algorithmic / r.seconds / 1e9
    phases = pass_kind_times(r)
    return {"pass_kinds": phases, "tokens": int(len(r.tokens)), "seconds": r.seconds, "tokens_per_s": len(r.tokens) / r.seconds, "handoffs": len(r.handoffs),
            "passes": int(r.n_steps), "target_share": float(r.source.mean()) if len(r.source) else 0.0,
            "achieved_gbs": gbs, "frac_of_measured_hbm": gbs / peak}


def other_workloads(torch, B, small, large, peak, want_batch):
    """One timed generation of each of the other workloads (after the main loop; single GPU only).  Returns a dict
    keyed by workload name.  The 64-sequence workload needs most of the device memory for its KV pages, so the
    models of the main loop are closed before it runs (the caller passes them in and must not use them after)."""
    out = {}
    # tiny pair (config 0): the case the oracle checks token by token
    wl = W.CONFIGS["tiny_pair"]
    prompt, force = W.workload_inputs(wl)
    ts = B.Model(wl.small.as_dict(), seed=0, tag=0, max_tokens=512)
    tl = B.Model(wl.large.as_dict(), seed=0, tag=1, max_tokens=512)
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1, max_new_tokens=wl.max_new_tokens, force=force)
    B.st_generate_spec(ts, tl, prompt, **kw)
    out[wl.name] = generation_summary(B.st_generate_spec(ts, tl, prompt, **kw), peak)
    ts.close()
    tl.close()
    # the small model alone (config 1)
    wl = W.CONFIGS["qwen1p5b_alone"]
    prompt, force = W.workload_inputs(wl)
    kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1, max_new_tokens=wl.max_new_tokens, force=force)
    B.st_generate_spec(small, None, prompt, **dict(kw, max_new_tokens=64))
    out[wl.name] = generation_summary(B.st_generate_spec(small, None, prompt, **kw), peak)
    # 7B + 32B with a 4096-token prompt (config 3): the target model is the one of the main loop
    wl = W.CONFIGS["qwen7b_32b_long"]
    if large is not None:
        prompt, force = W.workload_inputs(wl)
        cap = wl.prompt_len + wl.max_new_tokens + 64
        mid = B.Model(wl.small.as_dict(), seed=wl.weight_seed, tag=0, max_tokens=cap)
        kw = dict(delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1, max_new_tokens=wl.max_new_tokens, force=force)
        out[wl.name] = generation_summary(B.st_generate_spec(mid, large, prompt, **kw), peak)
        mid.close()
    # 64 independent sequences on the 1.5B + 32B pair (config 4)
    if want_batch and large is not None:
        shape_s, shape_l = W.QWEN_1P5B, W.QWEN_32B
        small.close()
        large.close()
        torch.cuda.empty_cache()
        n = 64
        prompts, budgets, forces = W.batch_inputs(5, n, min(shape_s.vocab, shape_l.vocab))
        cap = sum(len(p) + b + 80 for p, b in zip(prompts, budgets))
        bs = B.Model(shape_s.as_dict(), seed=0, tag=0, max_seqs=n, max_tokens=cap)
        bl = B.Model(shape_l.as_dict(), seed=0, tag=1, max_seqs=n, max_tokens=cap)
        t0 = time.perf_counter()
        got = B.st_generate_spec_batch(bs, bl, prompts, delimiter_id=W.DELIMITER_ID, keyword_ids=W.KEYWORD_IDS, n1=W.N1,
                                       max_new_tokens=budgets, forces=forces)
        wall = time.perf_counter() - t0
        tok = sum(len(r.tokens) for r in got)
        sec = got[0].seconds
        # bytes the batch had to move: one pass over a model's weights per round and model is what batching saves, so the
        # roofline compares against the per-sequence algorithmic bytes (what 64 separate generations would move)
        alone = sum(r.bytes_algorithmic for r in got)
        out["batch64_1p5b_32b"] = {"sequences": n, "tokens": int(tok), "seconds": sec, "wall_seconds": wall, "tokens_per_s": tok / sec,
                                   "handoffs": int(sum(len(r.handoffs) for r in got)),
                                   "target_share": float(sum(int((r.source == 1).sum()) for r in got) / max(tok, 1)),
                                   "prompt_lens": [int(min(len(p) for p in prompts)), int(max(len(p) for p in prompts))],
                                   "budgets": [int(min(budgets)), int(max(budgets))],
                                   "bytes_if_run_one_by_one": int(alone), "speedup_bound_note":
                                   "tokens/s of the whole batch; sequences share each round's pass over the weights"}
        bs.close()
        bl.close()
    return out


# DRAM bytes per launch of the dominant kernel, as a ratio to its algorithmic bytes: ncu dram__bytes_read.sum +
# dram__bytes_write.sum of decode_mega_kernel<128, 5> (the 32B's instance) on a two-layer cut of the 32B's widths,
# three launches.  None until a capture of the current kernel exists.
DOMINANT_TRAFFIC_RATIO = 1.002
DOMINANT_TRAFFIC_SOURCE = ("ncu dram__bytes_read.sum + dram__bytes_write.sum of decode_mega_kernel<128, 5> on a two-layer cut of the 32B's widths "
                           "(3517.5 MB per launch against 3510.1 MB algorithmic), scaled to the full-depth launch by its algorithmic bytes")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=3)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="native", choices=["native", "reference"])
    ap.add_argument("--workload", default="qwen1p5b_32b", choices=sorted(W.CONFIGS))
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true", help="skip the per-kernel figures and the other workloads")
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
    extras = not args.no_extras and args.layers == 0 and args.max_new == 0
    main_is_headline = wl.name == "qwen1p5b_32b" or wl.name.startswith("qwen1p5b_32b")
    # room for the other measurements on the same models: the 7B + 32B workload's 12k-token sequence and the batched
    # decode step's BATCH sequences of BATCH_CTX + 64 tokens on the large model
    BATCH, BATCH_CTX = 64, 512
    cap = wl.prompt_len + wl.max_new_tokens + 64
    cap_small = max(cap, 4096 + 64)
    long_cap = W.CONFIGS["qwen7b_32b_long"].prompt_len + W.CONFIGS["qwen7b_32b_long"].max_new_tokens + 64
    small = B.Model(wl.small.as_dict(), seed=wl.weight_seed, tag=0, max_tokens=cap_small)
    large = B.Model(wl.large.as_dict(), seed=wl.weight_seed, tag=1, max_seqs=BATCH + 1,
                    max_tokens=max(cap, long_cap) + BATCH * (BATCH_CTX + 64)) if wl.large else None
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
    # the metric's own fraction: algorithmic bytes of every pass of the timed generations / their device time
    path_bytes = sum(x.bytes_algorithmic for x in results)
    path_gbs = path_bytes / sum(x.seconds for x in results) / 1e9
    steps_small = int((r.emission_source == 0).sum())
    steps_large = int((r.emission_source == 1).sum())
    dom = large if large is not None else small
    shp = wl.large if wl.large else wl.small

    dominant = small_step = prefill = prompt_prefill = batched = None
    if extras:
        # Dominant kernel by bytes: the single-kernel decode step of the large model, on its own, mid-run context
        ctx = min(3000, cap - 64)
        kern_s, kern_bytes = timed_decode_step(torch, dom, shp, ctx)
        dominant = {"kernel": f"decode_mega_kernel ({shp.name}, one decode step per launch, context {ctx})", "bound": "hbm",
                    "us_per_launch": kern_s * 1e6, "algorithmic_bytes_per_launch": int(kern_bytes), "achieved": kern_bytes / kern_s / 1e9,
                    "peak": peak, "unit": "GB/s", "frac": kern_bytes / kern_s / 1e9 / peak,
                    "traffic": int(DOMINANT_TRAFFIC_RATIO * kern_bytes) if DOMINANT_TRAFFIC_RATIO else None,
                    "traffic_source": DOMINANT_TRAFFIC_SOURCE}
        if large is not None:
            s_s, s_bytes = timed_decode_step(torch, small, wl.small, ctx)
            small_step = {"kernel": f"decode_mega_kernel ({wl.small.name}, context {ctx})", "us_per_launch": s_s * 1e6,
                          "achieved": s_bytes / s_s / 1e9, "frac": s_bytes / s_s / 1e9 / peak, "unit": "GB/s"}
        # multi-row passes (handoff catch-up and prompt prefill) of the large model
        mean_catchup = int(np.mean([h[2] for h in r.handoffs])) if len(r.handoffs) else 128
        prefill = time_multi_row_passes(torch, dom, shp, max(0, min(1024, cap - 64 - 256)), [min(256, max(2, mean_catchup)), 256], peak)
        if world == 1:
            prompt_prefill = timed_prompt_prefill(torch, dom, shp, 4096, peak)
        if large is not None:
            batched = timed_batched_step(torch, large, shp, BATCH, BATCH_CTX, peak)
    accounting = paper_accounting(r, wl)
    others = None
    if extras and world == 1 and main_is_headline:
        others = other_workloads(torch, B, small, large, peak, want_batch=True)
        small = large = None   # closed by other_workloads

    if rank == 0:
        line = {
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": 1e3 * dev_s / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "bf16", "data": "synthetic",
            "config": {"workload": wl.name, "small": wl.small.name, "large": wl.large.name if wl.large else None,
                       "prompt_len": wl.prompt_len, "max_new_tokens": wl.max_new_tokens, "n1": W.N1,
                       "handoffs": len(r.handoffs), "target_share": float(r.source.mean()),
                       "passes_small": steps_small, "passes_large": steps_large,
                       "arithmetic": "bf16 weights, fp16 KV cache, fp32 activations and accumulation",
                       "l2": "inputs larger than L2: every pass streams 3.1 GB (small) or 64 GB (large) of weights",
                       "multi_gpu": "replicas only" if world > 1 else "single GPU"},
            "clocks": clocks,
            "e2e": {"value": e2e_value, "unit": UNIT,
                    "h2d_bytes_per_step": int(prompt.nbytes + (force.nbytes if force is not None else 0) + min(wl.small.vocab, shp.vocab)),
                    "d2h_bytes_per_step": int(5 * len(r.tokens) + 13 * r.n_steps + 12 * len(r.handoffs) + 80 * r.n_steps)},
            "gpu_launches": int(launches),
            # the metric's fraction: the whole generation against the HBM roofline
            "roofline": {"bound": "hbm", "achieved": path_gbs, "peak": peak, "unit": "GB/s", "frac": path_gbs / peak,
                         "traffic": None, "kernel": "whole path: every pass of the timed generations",
                         "algorithmic_bytes_per_step": int(path_bytes / len(results)),
                         "frac_of_nominal_8tbs": path_gbs / 8000.0, "peak_source": f"{peak_kind} copy bandwidth",
                         "note": "algorithmic bytes of every pass (weights + KV) / device time; per-kernel figures under dominant_kernel, decode_small, prefill, batched_decode"},
            "pass_kinds": pass_kind_times(r),
            "dominant_kernel": dominant,
            "decode_small": small_step,
            "prefill": prefill,
            "prompt_prefill": prompt_prefill,
            "batched_decode": batched,
            "workloads": others,
            "paper_accounting": accounting,
            "wall_s_timed_region": t_region,
        }
        if not args.no_cpu_baseline:
            line["cpu_baseline"] = cpu_oracle_sample(wl, {"steps_small": steps_small, "steps_large": steps_large,
                                                          "n_tokens": len(r.tokens)})
        print(json.dumps(line), flush=True)
    if small is not None:
        small.close()
    if large is not None:
        large.close()
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
