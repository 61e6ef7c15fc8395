#!/usr/bin/env python
"""Benchmark of one EAGLE-3 speculative step (draft + verify) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload C2] [--impl ours|reference]

A "step" is one full pass of the hot path (fuse pending taps, D draft passes with tree expansion,
rerank, one tree-masked target forward, greedy acceptance, KV compaction) for every sequence of the
batch.  Metric: accepted tokens per second (sum of per-step counts / time); ms_per_step is the
`spec_step ms` of the same run.  The workload at N=1 is the 8B-shaped batch-1 configuration (32
layers, hidden 4096, 32/8 heads of 128, FFN 14336, vocab 128256 / 32000, prompt 512, depth 6,
top-k 10, 60 verified nodes) on seeded random-init weights and random prompt ids; with N>1 every rank
runs an independent replica (the path has no collective), so the value is the sum over ranks.

Prints ONE JSON line on rank 0.
"""
import argparse
import gc
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2503_01840_b200 import synth  # noqa: E402

METRIC = "spec_step accepted tok/s"
UNIT = "tok/s"

# DRAM traffic of the GEMM kernel relative to its weight bytes, from the ncu capture summarised in
# profiles/gemm_fused_kernel_C2_shapes_ncu_full.md: (dram__bytes_read.sum + dram__bytes_write.sum) of the four GEMMs
# of an 8B-shaped layer = 448.6 MB for 436.2 MB of weights.  The capture ran on the 2-layer truncation (same kernels,
# same shapes); a full step's traffic is that ratio times its weight bytes (traffic grows with the weight bytes).
# Valid for the 8B shapes at 60 rows only; None elsewhere.
NCU_TRAFFIC_RATIO = {"C2-8B-b1": 448.6 / 436.2}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return float(d["hbm_gbs"]), "measured"
    return 6650.0, "fallback"


def workload_cfg(name: str):
    base, _, mod = name.partition(":")
    cfg = synth.CONFIGS[base]
    if mod.startswith("L="):
        cfg = cfg.truncated(int(mod[2:]))
    return cfg


class ClockSampler:
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        self.p = None
        try:
            self.p = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100",
                                       "-i", str(gpu_index)], stdout=self.f, stderr=subprocess.DEVNULL)
        except Exception:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except Exception:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        for line in self.f.read().splitlines():
            c = [x.strip() for x in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1])); mx.append(float(c[2]))
            except ValueError:
                continue
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            busy = [s for s in sm if s > 0]
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm))
        return out


def weight_bytes_per_step(cfg) -> float:
    """Algorithmic weight bytes of one step: every weight once per pass (D draft passes + FC3 + L layers + LM head)."""
    e = 4 if cfg.dtype == "fp32" else 2
    k, qd, kvd, F = cfg.hidden, cfg.n_heads * cfg.head_dim, cfg.n_kv_heads * cfg.head_dim, cfg.ffn
    layer = (k * qd + 2 * k * kvd + qd * k + 3 * k * F) * e
    draft_pass = 2 * k * k * e + layer + cfg.draft_vocab * k * e
    return cfg.tree_depth * draft_pass + 3 * k * k * e + cfg.n_layers * layer + cfg.vocab * k * e


# ----------------------------------------------------------------------------------------------- CPU oracle legs
CPU_MAX_PROMPT = 512     # the oracle's prefill of longer prompts would take many minutes; longer contexts are cut here
CPU_FULL_DEPTH_MAX_LAYERS = 40   # deeper (70B-shaped) models are timed on truncations and extrapolated, labelled as such


def _oracle_for(cfg, layers, tw=None, dw=None):
    """(oracle, prompt): the CPU oracle on `layers` layers of cfg at full widths, batch 1, for the workload's first
    prompt (cut to CPU_MAX_PROMPT tokens).  tw/dw: the full model's weights, reused when given."""
    sys.path.insert(0, os.path.join(ROOT, "oracle"))
    import pyoracle as po
    prompt = synth.make_prompts(cfg)[0].numpy()[:CPU_MAX_PROMPT]
    c = cfg.replace(batch=1, prompt_len=len(prompt)) if layers == cfg.n_layers else cfg.truncated(layers, batch=1, prompt_len=len(prompt))
    cpu = lambda w: {k: ([cpu(x) for x in v] if isinstance(v, list) else v.to("cpu")) for k, v in w.items()}
    if tw is None or layers != cfg.n_layers:
        dev = "cuda" if torch.cuda.is_available() else "cpu"      # the seeded generator runs on either device
        tw, dw = synth.make_target_weights(c, device=dev), synth.make_draft_weights(c, device=dev)
    tw, dw = cpu(tw), cpu(dw)
    if torch.cuda.is_available():
        torch.cuda.empty_cache()
    return po.Oracle(c, tw, dw, len(prompt) + 8 * (cfg.tree_depth + 1) * 64 + 256), prompt


def _time_oracle_steps(o, n, warmup=0):
    ts, toks = [], 0
    for i in range(warmup + n):
        t0 = time.perf_counter()
        k = len(o.step())
        dt = time.perf_counter() - t0
        if i >= warmup:
            ts.append(dt)
            toks += k
    return ts, toks


def cpu_step_seconds(cfg, steps, warmup=0, tw=None, dw=None):
    """Wall time of `steps` oracle steps of one sequence of the workload.  Models of up to CPU_FULL_DEPTH_MAX_LAYERS layers
    are timed AS THEY ARE (full depth, the workload's context); deeper ones on 2- and 6-layer truncations, with the
    per-layer slope extended to the full depth.  Returns (list of per-step seconds, tokens, description)."""
    if cfg.n_layers <= CPU_FULL_DEPTH_MAX_LAYERS:
        o, prompt = _oracle_for(cfg, cfg.n_layers, tw, dw)
        t0 = time.perf_counter()
        o.prefill(prompt)
        t_pre = time.perf_counter() - t0
        ts, toks = _time_oracle_steps(o, steps, warmup)
        o.close()
        return ts, toks, (f"oracle spec_step of one sequence of {cfg.name} at full depth ({cfg.n_layers} layers) and a {len(prompt)}-token "
                          f"context, {steps} timed step(s) after {warmup} untimed: min {min(ts):.2f}s median {statistics.median(ts):.2f}s "
                          f"max {max(ts):.2f}s (oracle prefill {t_pre:.1f}s, not counted)")
    per = {}
    for L in (2, 6):
        o, prompt = _oracle_for(cfg, L)
        o.prefill(prompt)
        per[L], toks = _time_oracle_steps(o, max(3, min(steps, 5)), 0)
        o.close()
    m2, m6 = statistics.median(per[2]), statistics.median(per[6])
    slope = (m6 - m2) / 4.0
    full = m2 + (cfg.n_layers - 2) * slope
    return [full] * steps, steps, (f"oracle spec_step of one sequence of {cfg.name} on 2- and 6-layer truncations at full widths "
                                   f"({len(prompt)}-token context; medians {m2:.2f}s and {m6:.2f}s, {slope:.3f}s per layer), EXTRAPOLATED "
                                   f"linearly to {cfg.n_layers} layers = {full:.1f}s per step")


def cpu_baseline(cfg, tw=None, dw=None):
    """The oracle as it stands on the host cores, on a bounded sample: 3 steps of one sequence."""
    cores = os.cpu_count() or 1      # the oracle's OpenMP loops use every host core
    ts, toks, how = cpu_step_seconds(cfg, 3, 0, tw, dw)
    # the oracle decodes one sequence at a time: a batch costs the sum over its sequences
    return {"value": (toks / len(ts)) / statistics.median(ts), "unit": UNIT, "cores": cores, "kind": "oracle", "sample": how}


def run_reference(args, cfg):
    """`--impl reference`: the CPU oracle (there is no other implementation of the paper here).  Every timed step is a
    measured oracle step of one sequence of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cores = os.cpu_count() or 1
    ts, toks, how = cpu_step_seconds(cfg, args.steps, args.warmup)
    total = sum(ts)
    value = toks / total
    out = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup,
           "ms_per_step": 1e3 * total / len(ts), "higher_is_better": True, "scaling": "weak",
           "vs_baseline": None, "dtype": "f32", "data": "synthetic", "impl": "reference",
           "config": {"workload": cfg.name, "batch": cfg.batch, "tree": f"D{cfg.tree_depth} K{cfg.tree_topk} N{cfg.tree_nodes}",
                      "note": "one sequence at a time; a batch costs the sum over its sequences, so tok/s does not grow with the batch"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": how},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


# ----------------------------------------------------------------------------------------------- replicas
def aggregate_over_ranks(ms, toks, e2e_val, dist=None, device="cpu"):
    """The path has no exchange step, so N GPUs run N independent replicas: whole-job time is the slowest
    rank's device time (MAX), tokens and end-to-end throughput add up (SUM).  `dist` is an initialised
    torch.distributed module or None for a single process."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(ms), int(toks), float(e2e_val)
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    k = torch.tensor([toks, e2e_val], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(k, op=dist.ReduceOp.SUM)
    return float(t.item()), int(round(k[0].item())), float(k[1].item())


# ----------------------------------------------------------------------------------------------- the CUDA arm
def timed_steps(dec, n_steps, counts_dev):
    """n_steps x spec_step_async between two events on the decoder's stream; returns (ms, tokens)."""
    stream = dec.stream
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for i in range(n_steps):
        dec.step_async(None, counts_dev[i])
    e1.record(stream)
    e1.synchronize()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1), int(counts_dev[:n_steps].sum().item())


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="C2", help="C1..C8, optionally ':L=<layers>' for a truncation")
    ap.add_argument("--no-extras", action="store_true", help="skip plain-decode / structured-acceptance / CPU legs")
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--dump-stamps", default="", help="write the per-launch in-graph kernel stamps of one step to this text file")
    ap.add_argument("--nvtx", action="store_true", help="wrap the timed steps in an NVTX range 'timed_steps' (lets a profiler select them)")
    args = ap.parse_args()
    cfg = workload_cfg(args.workload)
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    args.warmup = max(args.warmup, 3)

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the speculative step has no CPU path")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    from paper_2503_01840_b200 import binding as sb

    B, D = cfg.batch, cfg.tree_depth
    prof_steps = 3
    total_steps = args.warmup + args.steps + prof_steps + 40
    reserve = total_steps * (D + 1) + 64
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    max_ctx = max(len(p) for p in prompts) + reserve + 192
    t0 = time.time()
    tw = synth.make_target_weights(cfg, device=dev)
    dw = synth.make_draft_weights(cfg, device=dev)
    torch.cuda.synchronize()
    t_gen = time.time() - t0
    dec = sb.SpecDecoder(cfg, tw, dw, batch=B, max_ctx=max_ctx, flags=args.flags, page_shuffle_seed=cfg.seed)
    t0 = time.time()
    dec.prefill(prompts, reserve)
    t_prefill = time.time() - t0
    prefill_launches = dec.launches_per_step()

    counts = torch.zeros(max(args.steps, args.warmup + 16, 16), B, dtype=torch.int32, device=dev)
    timed_steps(dec, args.warmup, counts)
    n_mid = dec.lengths().astype(np.float64)
    bytes_step = dec.step_bytes()
    if world > 1:
        dist.barrier()
    sampler = ClockSampler(local) if rank == 0 else None
    if args.nvtx:
        torch.cuda.nvtx.range_push("timed_steps")
    ms, toks = timed_steps(dec, args.steps, counts)
    if args.nvtx:
        torch.cuda.nvtx.range_pop()
    clocks = sampler.stop() if sampler else None
    launches = dec.launches_per_step()

    # ---- end to end through the host-buffer entry point (sync + device->host copy every step)
    e2e_steps = min(args.steps, 50)
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    e2e_toks = 0
    for _ in range(e2e_steps):
        e2e_toks += sum(len(o) for o in dec.step())
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    e2e_val = e2e_toks / e2e_s
    ms, toks, e2e_val = aggregate_over_ranks(ms, toks, e2e_val, dist if world > 1 else None, dev)
    ms_per_step = ms / args.steps
    value = toks / (ms * 1e-3)
    d2h = B * (D + 1) * 4 + B * 4 + 16 + B * 4

    # ---- dominant kernel (the tcgen05 weight GEMM).  Its time INSIDE the replayed graph comes from a second context
    # with kernel stamps: every GEMM and attention launch records when its inputs were ready (after its dependency
    # wait) and when its last CTA left; launch i is charged end_i - max(ready_i, end of the previous stamped launch),
    # so the charged intervals never overlap and sum to at most the step time.
    peak, peak_kind = peaks()
    breakdown = {}
    for _ in range(prof_steps):
        pr = dec.profile_step()
        for c, (m_, n_) in pr.items():
            a = breakdown.setdefault(c, [0.0, 0])
            a[0] += m_ / prof_steps
            a[1] = n_
    gemm_n = breakdown["gemm"][1]
    dec.close()
    decs = sb.SpecDecoder(cfg, tw, dw, batch=B, max_ctx=max_ctx, flags=args.flags | sb.FLAG_STAMPS, page_shuffle_seed=cfg.seed)
    decs.prefill(prompts, reserve)
    timed_steps(decs, args.warmup + min(args.steps, 30) // 2, counts)          # about the same context as the timed run
    st_ms, _ = timed_steps(decs, 10, counts)
    stamps, classes = decs.kernel_stamps()
    decs.close()
    charged = {"gemm": 0.0, "attention": 0.0}
    prev_end = None
    for (ready, end), cls in zip(stamps.astype(np.int64), classes):
        start = ready if prev_end is None else max(ready, prev_end)
        charged[cls] += max(0, end - start) * 1e-6
        prev_end = end if prev_end is None else max(prev_end, end)
    span_ms = float(stamps[:, 1].max() - stamps[:, 0].min()) * 1e-6 if len(stamps) else 0.0
    if args.dump_stamps and rank == 0 and len(stamps):
        t0s, prev = int(stamps[:, 0].min()), None
        with open(args.dump_stamps, "w") as fh:
            fh.write("# launch class ready_us end_us duration_us charged_us ready_minus_previous_end_us\n")
            for i, ((ready, end), cls) in enumerate(zip(stamps.astype(np.int64), classes)):
                start = ready if prev is None else max(ready, prev)
                gap = 0 if prev is None else ready - prev
                fh.write(f"{i} {cls} {(ready - t0s) / 1e3:.2f} {(end - t0s) / 1e3:.2f} {(end - ready) / 1e3:.2f} {max(0, end - start) / 1e3:.2f} {gap / 1e3:.2f}\n")
                prev = end if prev is None else max(prev, end)
    gemm_ms = charged["gemm"]
    timing = "in-graph kernel stamps (globaltimer) of one replayed step; non-overlapping charged intervals"
    if gemm_ms <= 0.0:           # the plain fp32 schedule has no stamped kernels: one event per launch instead
        gemm_ms = breakdown["gemm"][0]
        timing = "one CUDA event before every launch (no graph): the plain fp32 kernels carry no stamps"
    wbytes = weight_bytes_per_step(cfg)
    achieved = wbytes / (gemm_ms * 1e-3) / 1e9 if gemm_ms > 0 else 0.0
    ratio = NCU_TRAFFIC_RATIO.get(cfg.name)
    traffic = ratio * wbytes / max(1, gemm_n) if ratio else None
    ev_gemm_ms = breakdown["gemm"][0]
    roofline = {"bound": "hbm", "kernel": ("gemm_fused_kernel" if cfg.dtype == "bf16" else "gemm_ref_kernel") + " (all weight GEMMs of the step)", "achieved": achieved,
                "peak": peak, "peak_kind": peak_kind, "unit": "GB/s", "frac": achieved / peak,
                "bytes_per_launch": wbytes / max(1, gemm_n), "avg_launch_us": 1e3 * gemm_ms / max(1, gemm_n),
                "launches_per_step": gemm_n, "traffic": traffic,
                "timing": timing,
                "in_graph_ms": {"gemm": round(gemm_ms, 4), "attention": round(charged["attention"], 4),
                                "first_ready_to_last_exit": round(span_ms, 4), "step_with_stamps": round(st_ms / 10, 4),
                                "step": round(ms_per_step, 4)},
                "step": {"algorithmic_bytes": bytes_step, "achieved": bytes_step / (ms_per_step * 1e-3) / 1e9,
                         "frac_of_measured_copy": bytes_step / (ms_per_step * 1e-3) / 1e9 / peak,
                         "frac_of_8TBs": bytes_step / (ms_per_step * 1e-3) / 1e9 / 8000.0},
                "event_per_launch": {"note": "one CUDA event before every launch, no graph, no dependent-launch overlap: an upper bound "
                                             "per class that does not add up to the step time",
                                     "gemm_frac": (wbytes / (ev_gemm_ms * 1e-3) / 1e9 / peak) if ev_gemm_ms > 0 else None,
                                     "class_ms": {c: round(v[0], 4) for c, v in breakdown.items()}}}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": cfg.dtype, "data": "synthetic",
            "config": {"workload": cfg.name, "batch": B, "context_mid_run": float(n_mid.mean()),
                       "tree": f"D{D} K{cfg.tree_topk} N{cfg.tree_nodes}", "page_size": cfg.page_size,
                       "parallelism": "replicas" if world > 1 else "single GPU",
                       "l2": "inputs (weights + KV) far larger than L2, no flush", "tau": toks / (args.steps * B * world)},
            "clocks": clocks, "e2e": {"value": e2e_val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": d2h,
                                      "note": "spec_step with host outputs, synchronised every step; a step has no host input"},
            "gpu_launches": launches * args.steps, "roofline": roofline,
            "setup_s": {"weights": round(t_gen, 2), "prefill": round(t_prefill, 2)},
            "launches": {"per_step": launches, "prefill": prefill_launches}}

    if rank == 0 and world == 1 and not args.no_extras:
        extras = {}
        # plain greedy decoding on the same kernels (the paper's vanilla baseline), synchronised per token
        dec = sb.SpecDecoder(cfg, tw, dw, batch=B, max_ctx=max(len(p) for p in prompts) + 256, page_shuffle_seed=cfg.seed)
        dec.prefill(prompts, 64)
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        for _ in range(20):
            dec.plain_step()
        torch.cuda.synchronize()
        extras["plain_decode_tok_s"] = 20 * B / (time.perf_counter() - t0)
        # temperature 1: the same step ending in the stochastic acceptance kernel (host API, synchronised per step, uniforms
        # drawn on the host); after the plain tokens the draft cache is stale, so this leg runs on a fresh prefill
        dec.close()
        dec = sb.SpecDecoder(cfg, tw, dw, batch=B, max_ctx=max(len(p) for p in prompts) + 40 * (D + 1) + 256,
                             page_shuffle_seed=cfg.seed)
        dec.prefill(prompts, 40 * (D + 1))
        rng = np.random.default_rng(0)
        us = rng.random((25, B, 2 * cfg.tree_nodes), dtype=np.float32)
        for i in range(5):
            dec.step_sampled(1.0, us[i])
        torch.cuda.synchronize()
        t0 = time.perf_counter()
        toks_s = 0
        for i in range(5, 25):
            toks_s += sum(len(o) for o in dec.step_sampled(1.0, us[i]))
        dt = time.perf_counter() - t0
        extras["sampled_T1"] = {"ms_per_step": 1e3 * dt / 20, "accepted_tok_s": toks_s / dt,
                                "note": "spec_step_sampled, wall clock with host synchronisation every step"}
        dec.close()
        if cfg.n_layers <= CPU_FULL_DEPTH_MAX_LAYERS:
            line["cpu_baseline"] = cpu_baseline(cfg, tw, dw)          # reuses the weights that are already generated
        del dec, tw, dw                      # the 70B-shaped weights leave no room for a second model beside them
        gc.collect()
        torch.cuda.empty_cache()
        if cfg.batch == 1 and cfg.tree_depth >= 2:
            # designed draft/target agreement: same shapes and bytes, acceptance length near the paper's
            tw2, dw2, _, _ = synth.make_structured(cfg, 0.96, device=dev)
            pr = synth.structured_prompt(cfg, dw2["d2t"].cpu(), len(prompts[0])).numpy()
            dec2 = sb.SpecDecoder(cfg, tw2, dw2, batch=1, max_ctx=len(pr) + 60 * (D + 1) + 256, page_shuffle_seed=cfg.seed)
            dec2.prefill([pr], 60 * (D + 1))
            c2 = torch.zeros(40, 1, dtype=torch.int32, device=dev)
            timed_steps(dec2, 5, c2)
            ms2, tk2 = timed_steps(dec2, 40, c2)
            extras["structured_agreement"] = {"p_agree": 0.96, "tau": tk2 / 40, "ms_per_step": ms2 / 40,
                                              "accepted_tok_s": tk2 / (ms2 * 1e-3)}
            dec2.close()
            del dec2, tw2, dw2
        extras["projection_at_paper_tau"] = {"tau": 6.23, "tok_s": 6.23 * B / (ms_per_step * 1e-3),
                                            "note": "paper's mean acceptance length for the 8B target (Table 1) / measured step time"}
        line["extras"] = extras
        torch.cuda.empty_cache()
        if "cpu_baseline" not in line:
            line["cpu_baseline"] = cpu_baseline(cfg)
    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
