"""Writes tests/golden/c1_oracle_trajectory.json: the CPU oracle's own output on configuration 1 (tiny fp32 target,
prompt of 64 seeded ids, depth 3, top-k 4, 16 verified nodes, 32 generated tokens).

The paper prints no logits, trees or token ids, so there is no paper value to store; this fixture is a regression
anchor for the oracle (it calls nothing but `oracle/` and the seeded input generator) and the reference the GPU
smoke check can be compared with by eye.  Run from the repository root:

    python tests/golden/make_golden.py
"""
import json
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
for p in (ROOT, os.path.join(ROOT, "oracle")):
    sys.path.insert(0, p)

import pyoracle as po  # noqa: E402
from paper_2503_01840_b200 import synth  # noqa: E402


def trajectory():
    cfg = synth.C1
    tw, dw = synth.make_target_weights(cfg), synth.make_draft_weights(cfg)
    prompt = synth.make_prompts(cfg)[0].numpy()
    o = po.Oracle(cfg, tw, dw, 256)
    first = int(o.prefill(prompt))
    counts, tokens = [], [first]
    while len(tokens) < 1 + cfg.gen_tokens:
        out = o.step()
        counts.append(len(out))
        tokens += [int(t) for t in out]
    g = po.Oracle(cfg, tw, dw, 256)
    g.prefill(prompt)
    greedy = [first] + [int(t) for t in g.greedy(len(tokens) - 1)]
    # the same start at temperature 1 with stored uniforms (multiples of 2^-16, so the file holds them exactly): the
    # stochastic acceptance rule's own trajectory
    import numpy as np
    rng = np.random.default_rng(2503)
    s = po.Oracle(cfg, tw, dw, 256)
    s.prefill(prompt)
    sampled_u, sampled_tokens, sampled_counts = [], [first], []
    for _ in range(8):
        u = (rng.integers(0, 1 << 16, 2 * cfg.tree_nodes) / float(1 << 16)).astype(np.float32)
        out = s.step_sampled(1.0, u)
        sampled_u.append([float(x) for x in u])
        sampled_counts.append(len(out))
        sampled_tokens += [int(t) for t in out]
    return {"config": cfg.name, "prompt_head": [int(t) for t in prompt[:8]], "first_token": first, "tokens": tokens,
            "counts": counts, "greedy": greedy,
            "sampled_T1": {"uniforms": sampled_u, "tokens": sampled_tokens, "counts": sampled_counts}}


if __name__ == "__main__":
    out = os.path.join(os.path.dirname(os.path.abspath(__file__)), "c1_oracle_trajectory.json")
    with open(out, "w") as f:
        json.dump(trajectory(), f, indent=1)
    print("wrote", out)
