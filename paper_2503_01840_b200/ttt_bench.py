"""Times training-time-test attention (Section 3.2) on one GPU and prints one JSON line.

    python -m paper_2503_01840_b200.ttt_bench [--T 8192] [--heads 32] [--kv-heads 8] [--steps-simulated 3] [--iters 20]

The dense causal part is a contraction: algorithmic flops = 4 * head_dim * heads * T (T + 1) / 2 (Q K^T and P V over the
allowed keys only); the fraction is taken against the measured dense bf16 peak when a peaks file is given."""
import argparse
import json

import torch

from . import binding as sb


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--T", type=int, default=8192)
    ap.add_argument("--heads", type=int, default=32)
    ap.add_argument("--kv-heads", type=int, default=8)
    ap.add_argument("--steps-simulated", type=int, default=3)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--peak-tflops", type=float, default=0.0, help="measured dense bf16 peak for the fraction (0: omit)")
    a = ap.parse_args()
    T, H, G, J, hd, ps = a.T, a.heads, a.kv_heads, a.steps_simulated, 128, 16
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(1)
    q = torch.randn(T, H, hd, generator=g, device=dev).to(torch.bfloat16)
    pps = (T + ps - 1) // ps
    kp = torch.randn(pps, G, ps, hd, generator=g, device=dev).to(torch.bfloat16)
    vp = torch.randn(pps, G, ps, hd, generator=g, device=dev).to(torch.bfloat16)
    table = torch.randperm(pps, generator=g, device=dev).to(torch.int32)
    kd = torch.randn(J, T, G, hd, generator=g, device=dev).to(torch.bfloat16) if J else None
    vd = torch.randn(J, T, G, hd, generator=g, device=dev).to(torch.bfloat16) if J else None
    for _ in range(3):
        sb.ttt_attention(q, kp, vp, table, kd, vd)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        sb.ttt_attention(q, kp, vp, table, kd, vd)
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / a.iters
    flops = 4.0 * hd * H * T * (T + 1) / 2
    line = {"op": "ttt_attention", "T": T, "heads": H, "kv_heads": G, "simulated_steps": J, "ms": round(ms, 4),
            "tflops": round(flops / ms / 1e9, 2), "note": "includes the binding's padding copies and the merge kernel"}
    if a.peak_tflops > 0:
        line["frac_of_measured_bf16_peak"] = round(flops / ms / 1e9 / a.peak_tflops, 4)
    print(json.dumps(line))


if __name__ == "__main__":
    main()
