"""Seeded synthetic inputs for the EAGLE-3 speculative step.

This module only *generates inputs* (weights, prompts, draft->target id maps,
model shapes).  It contains none of the method's arithmetic and is the one piece
of code that both the CUDA path's tests and the CPU oracle's tests feed from.

Every value is a pure function of (seed, tensor id, flat index) through a
counter-based integer hash, evaluated with torch integer ops so the same code
runs on the CPU and on a CUDA device and yields bit-identical tensors:

    h   = lowbias32(idx_lo ^ lowbias32(idx_hi + key)),  key = lowbias32(seed * 0x9E3779B1 + tensor_id)
    u   = (h >> 8) * 2^-23 - 1 + 2^-24          (24 exact bits, uniform on (-1, 1))
    w   = u * sqrt(3) * std                     (one fp32 multiply; std as listed below)

    matrices            std 1/sqrt(fan_in);  W_o and W_down additionally 1/sqrt(2 L)
    embeddings          std 1
    LM heads            std 1/sqrt(k)
    norm gains          1 + 0.1 u

For bf16 models the fp32 value is rounded to bf16 (round-to-nearest-even); the
oracle widens those same bf16 values back to fp32, so both sides see equal weights.

The paper's evaluation prompts (chat, code, maths, summarisation sets) and its
trained weights are not available; random ids and random-init weights of the
stated shapes stand in for them.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional

import torch

_M32 = 0xFFFFFFFF


# ----------------------------------------------------------------------------- shapes
@dataclasses.dataclass(frozen=True)
class ModelCfg:
    name: str
    dtype: str                 # "fp32" | "bf16"
    n_layers: int
    hidden: int
    n_heads: int
    n_kv_heads: int
    head_dim: int
    ffn: int
    vocab: int
    draft_vocab: int
    fuse_layers: tuple
    rope_theta: float
    rms_eps: float = 1e-5
    # workload
    batch: int = 1
    prompt_len: int = 64       # for batch > 1: lengths ~ U{prompt_lo..prompt_hi}
    prompt_lo: int = 0
    prompt_hi: int = 0
    gen_tokens: int = 32
    page_size: int = 16
    tree_depth: int = 3
    tree_topk: int = 4
    tree_nodes: int = 16       # verified nodes including the root
    seed: int = 1

    def replace(self, **kw) -> "ModelCfg":
        return dataclasses.replace(self, **kw)

    def truncated(self, n_layers: int, **kw) -> "ModelCfg":
        """Same widths, fewer target layers; taps are clamped into range."""
        fl = tuple(min(f, n_layers - 1) for f in self.fuse_layers)
        return dataclasses.replace(self, name=f"{self.name}-L{n_layers}", n_layers=n_layers,
                                   fuse_layers=fl, **kw)

    @property
    def pool(self) -> int:
        return self.tree_topk + (self.tree_depth - 1) * self.tree_topk ** 2


C1 = ModelCfg("C1-tiny-fp32", "fp32", 2, 256, 4, 2, 64, 688, 4096, 1024, (0, 1, 1), 10000.0,
              batch=1, prompt_len=64, gen_tokens=32, tree_depth=3, tree_topk=4, tree_nodes=16, seed=1)
C2 = ModelCfg("C2-8B-b1", "bf16", 32, 4096, 32, 8, 128, 14336, 128256, 32000, (2, 16, 29), 5e5,
              batch=1, prompt_len=512, gen_tokens=256, tree_depth=6, tree_topk=10, tree_nodes=60, seed=2)
C3 = C2.replace(name="C3-8B-b64-chain", batch=64, prompt_lo=256, prompt_hi=2048, gen_tokens=128,
                tree_depth=3, tree_topk=1, tree_nodes=4, seed=3)
C4 = C2.replace(name="C4-8B-16k", prompt_len=16384, gen_tokens=1024, tree_depth=8, seed=4)
C5 = ModelCfg("C5-70B-b1", "bf16", 80, 8192, 64, 8, 128, 28672, 128256, 32000, (2, 40, 77), 5e5,
              batch=1, prompt_len=4096, gen_tokens=128, tree_depth=6, tree_topk=10, tree_nodes=60, seed=5)
# Further workloads of the paper's evaluation (Section 4, Appendix A): full trees at a small batch, a 13B-shaped
# multi-head-attention target (vocabulary 32000, 50 tree nodes, depth 8) and the serving study's chain of 2.
C6 = C2.replace(name="C6-8B-b4-tree", batch=4, prompt_lo=256, prompt_hi=2048, gen_tokens=128, seed=6)
C7 = ModelCfg("C7-13B-mha-b1", "bf16", 40, 5120, 40, 40, 128, 13824, 32000, 32000, (2, 20, 37), 1e4,
              batch=1, prompt_len=512, gen_tokens=256, tree_depth=8, tree_topk=10, tree_nodes=50, seed=7)
C8 = C2.replace(name="C8-8B-b56-chain2", batch=56, prompt_lo=256, prompt_hi=2048, gen_tokens=128,
                tree_depth=2, tree_topk=1, tree_nodes=3, seed=8)
CONFIGS = {"C1": C1, "C2": C2, "C3": C3, "C4": C4, "C5": C5, "C6": C6, "C7": C7, "C8": C8}


# ----------------------------------------------------------------------------- hash
def _lowbias32(x: torch.Tensor) -> torch.Tensor:
    """32-bit integer mixer (public-domain 'lowbias32' constants) on int64 lanes."""
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    return x ^ (x >> 16)


def _lowbias32_int(x: int) -> int:
    x &= _M32
    x = ((x ^ (x >> 16)) * 0x7FEB352D) & _M32
    x = ((x ^ (x >> 15)) * 0x846CA68B) & _M32
    return x ^ (x >> 16)


def uniform_pm1(seed: int, tensor_id: int, numel: int, device="cpu", chunk: int = 1 << 25) -> torch.Tensor:
    """fp32 tensor of `numel` values uniform on (-1, 1); element i depends only on (seed, tensor_id, i)."""
    key = _lowbias32_int(seed * 0x9E3779B1 + tensor_id)
    out = torch.empty(numel, dtype=torch.float32, device=device)
    for s in range(0, numel, chunk):
        e = min(numel, s + chunk)
        idx = torch.arange(s, e, dtype=torch.int64, device=device)
        hi = _lowbias32(((idx >> 32) + key) & _M32)
        h = _lowbias32((idx & _M32) ^ hi)
        out[s:e] = (h >> 8).to(torch.float32) * (2.0 ** -23) - (1.0 - 2.0 ** -24)
    return out


def _tensor(seed, tid, shape, std, dtype, device):
    n = 1
    for d in shape:
        n *= d
    w = uniform_pm1(seed, tid, n, device) * float(math.sqrt(3.0) * std)
    return w.view(*shape).to(dtype)


def _gain(seed, tid, k, dtype, device):
    return (1.0 + 0.1 * uniform_pm1(seed, tid, k, device)).to(dtype)


def torch_dtype(cfg: ModelCfg):
    return torch.float32 if cfg.dtype == "fp32" else torch.bfloat16


_LAYER_FIELDS = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")


def _layer(seed, base_tid, cfg: ModelCfg, n_layers_for_scale: int, dtype, device) -> Dict[str, torch.Tensor]:
    k, H, G, hd, F = cfg.hidden, cfg.n_heads, cfg.n_kv_heads, cfg.head_dim, cfg.ffn
    res = 1.0 / math.sqrt(2.0 * n_layers_for_scale)
    return {
        "attn_norm": _gain(seed, base_tid + 0, k, dtype, device),
        "wq": _tensor(seed, base_tid + 1, (H * hd, k), 1 / math.sqrt(k), dtype, device),
        "wk": _tensor(seed, base_tid + 2, (G * hd, k), 1 / math.sqrt(k), dtype, device),
        "wv": _tensor(seed, base_tid + 3, (G * hd, k), 1 / math.sqrt(k), dtype, device),
        "wo": _tensor(seed, base_tid + 4, (k, H * hd), res / math.sqrt(H * hd), dtype, device),
        "mlp_norm": _gain(seed, base_tid + 5, k, dtype, device),
        "w_gate": _tensor(seed, base_tid + 6, (F, k), 1 / math.sqrt(k), dtype, device),
        "w_up": _tensor(seed, base_tid + 7, (F, k), 1 / math.sqrt(k), dtype, device),
        "w_down": _tensor(seed, base_tid + 8, (k, F), res / math.sqrt(F), dtype, device),
    }


def make_d2t(cfg: ModelCfg, seed: Optional[int] = None) -> torch.Tensor:
    """Strictly increasing int32 [draft_vocab]: a seeded sample of target ids without replacement."""
    g = torch.Generator(device="cpu").manual_seed(1000 + (cfg.seed if seed is None else seed))
    perm = torch.randperm(cfg.vocab, generator=g)[: cfg.draft_vocab]
    return torch.sort(perm).values.to(torch.int32)


def make_target_weights(cfg: ModelCfg, device="cpu", seed: Optional[int] = None) -> Dict:
    seed = cfg.seed if seed is None else seed
    dt = torch_dtype(cfg)
    k, V = cfg.hidden, cfg.vocab
    w = {
        "embed": _tensor(seed, 1, (V, k), 1.0, dt, device),
        "final_norm": _gain(seed, 2, k, dt, device),
        "lm_head": _tensor(seed, 3, (V, k), 1 / math.sqrt(k), dt, device),
        "layers": [_layer(seed, 100 + 10 * l, cfg, cfg.n_layers, dt, device) for l in range(cfg.n_layers)],
    }
    return w


def make_draft_weights(cfg: ModelCfg, device="cpu", seed: Optional[int] = None) -> Dict:
    """Draft head weights; `seed` lets a test swap the draft while keeping the target."""
    seed = (cfg.seed if seed is None else seed) + 7777
    dt = torch_dtype(cfg)
    k, Vd = cfg.hidden, cfg.draft_vocab
    w = {
        "fc3": _tensor(seed, 50, (k, 3 * k), 1 / math.sqrt(3 * k), dt, device),
        "fc2": _tensor(seed, 51, (k, 2 * k), 1 / math.sqrt(2 * k), dt, device),
        "final_norm": _gain(seed, 52, k, dt, device),
        "lm_head": _tensor(seed, 53, (Vd, k), 1 / math.sqrt(k), dt, device),
        "d2t": make_d2t(cfg).to(device),
    }
    w.update(_layer(seed, 60, cfg, 1, dt, device))
    return w


def make_prompts(cfg: ModelCfg, seed: Optional[int] = None) -> List[torch.Tensor]:
    """One int32 id tensor per sequence (CPU). Batch 1: `prompt_len` ids from seed; batch B: lengths
    ~ U{prompt_lo..prompt_hi} from seed, ids of sequence s from seed + s."""
    seed = cfg.seed if seed is None else seed
    if cfg.batch == 1:
        g = torch.Generator(device="cpu").manual_seed(seed)
        return [torch.randint(0, cfg.vocab, (cfg.prompt_len,), generator=g, dtype=torch.int64).to(torch.int32)]
    g = torch.Generator(device="cpu").manual_seed(seed)
    lens = torch.randint(cfg.prompt_lo, cfg.prompt_hi + 1, (cfg.batch,), generator=g)
    out = []
    for s in range(cfg.batch):
        gs = torch.Generator(device="cpu").manual_seed(seed + s)
        out.append(torch.randint(0, cfg.vocab, (int(lens[s]),), generator=gs, dtype=torch.int64).to(torch.int32))
    return out


# ----------------------------------------------------------------------------- structured workload
def make_structured(cfg: ModelCfg, p_agree: float, device="cpu", residual_scale: float = 0.0,
                    seed: Optional[int] = None):
    """'Permutation' weights with a designed acceptance length.

    Let Dset be the image of d2t.  pi is one cycle over Dset; pi2 equals pi except on a random
    subset (fraction 1 - p_agree) of Dset whose images are rotated among themselves.  The target's
    W_o and W_down are scaled by `residual_scale` (0 => the residual stream stays E[tok]) and its
    LM-head row pi(v) is E[v]/sqrt(k); the draft's FC2 passes the embedding half through, its
    W_o/W_down are scaled the same way and its LM-head row for pi2(v) is E[v]/sqrt(k).
    With residual_scale == 0 the target emits the pi-orbit of the root and the draft proposes
    pi2 of each token, so the accepted run per step is known without running anything.

    Returns (target_weights, draft_weights, pi, pi2) with pi/pi2 int64 [vocab] (-1 outside Dset).
    """
    seed = cfg.seed if seed is None else seed
    tw = make_target_weights(cfg, device, seed)
    dw = make_draft_weights(cfg, device, seed)
    dt = torch_dtype(cfg)
    k, V, Vd = cfg.hidden, cfg.vocab, cfg.draft_vocab
    d2t = dw["d2t"].to("cpu").to(torch.int64)
    g = torch.Generator(device="cpu").manual_seed(4242 + seed)
    order = d2t[torch.randperm(Vd, generator=g)]               # cycle order over Dset
    pi = torch.full((V,), -1, dtype=torch.int64)
    pi[order] = torch.roll(order, -1)
    pi2 = pi.clone()
    n_dis = int(round((1.0 - p_agree) * Vd))
    if n_dis >= 2:
        S = order[torch.randperm(Vd, generator=g)[:n_dis]]
        pi2[S] = torch.roll(pi[S], 1)
    # target LM head: row pi(v) = E[v] / sqrt(k); rows outside Dset keep their small random values
    E = tw["embed"].to(torch.float32)
    inv = torch.empty(Vd, dtype=torch.int64)
    lm = tw["lm_head"].to(torch.float32) * 0.05
    src = order.to(device)
    lm[pi[order].to(device)] = E[src] / math.sqrt(k)
    tw["lm_head"] = lm.to(dt)
    # draft LM head: draft id i (target id d2t[i]) = pi2(v)  =>  row i = E[v] / sqrt(k)
    pos_of = torch.full((V,), -1, dtype=torch.int64)
    pos_of[d2t] = torch.arange(Vd)
    dl = torch.empty(Vd, k, dtype=torch.float32, device=device)
    dl[pos_of[pi2[order]].to(device)] = E[src] / math.sqrt(k)
    dw["lm_head"] = dl.to(dt)
    fc2 = dw["fc2"].to(torch.float32) * residual_scale
    fc2[:, k:] += torch.eye(k, device=device)
    dw["fc2"] = fc2.to(dt)
    for lw in tw["layers"] + [dw]:
        lw["wo"] = (lw["wo"].to(torch.float32) * residual_scale).to(dt)
        lw["w_down"] = (lw["w_down"].to(torch.float32) * residual_scale).to(dt)
    del inv
    return tw, dw, pi, pi2


def structured_prompt(cfg: ModelCfg, d2t: torch.Tensor, length: int, seed: int = 0) -> torch.Tensor:
    """Random ids whose last one lies in the image of d2t (so the orbit starts inside Dset)."""
    g = torch.Generator(device="cpu").manual_seed(99 + seed)
    ids = torch.randint(0, cfg.vocab, (length,), generator=g, dtype=torch.int64)
    ids[-1] = int(d2t[int(torch.randint(0, d2t.numel(), (1,), generator=g))])
    return ids.to(torch.int32)
