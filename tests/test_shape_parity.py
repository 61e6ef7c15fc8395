"""Whole speculative steps against the CPU oracle at the widths and launch shapes the benchmark times.

The small-model trajectories prove the algorithm; these prove the kernels at the shapes that matter: hidden 4096
and 8192, 32/8 and 64/8 heads of 128, FFN 14336 / 28672, vocabularies 128256 / 32000, 60-node trees of depth 6 and 8,
256-row batch passes, a context long enough for the tcgen05 attention kernel with key splits, RoPE positions in the
thousands, and the tap layers of a full-depth 32-layer model.  Every case runs `parity.run_trajectory`: draft logits,
draft features, verify logits, hidden states and taps element by element, integer decisions wherever their own oracle
margin allows, and the test asserts how much was actually compared."""
import numpy as np
import pytest
import torch

import parity
from paper_2503_01840_b200 import binding as sb
from paper_2503_01840_b200 import synth

pytestmark = pytest.mark.gpu


def _run(cfg, n_steps, **kw):
    tw = synth.make_target_weights(cfg, device="cuda")
    dw = synth.make_draft_weights(cfg, device="cuda")
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    tw_cpu, dw_cpu = parity.to_cpu(tw), parity.to_cpu(dw)
    del tw, dw
    torch.cuda.empty_cache()
    st, emitted = parity.run_trajectory(cfg, tw_cpu, dw_cpu, prompts, n_steps=n_steps, tol=2e-2, tap_tol=3e-2, **kw)
    print(cfg.name, st)
    return st, emitted, prompts


def _assert_everything_compared(st, cfg, sequences=1):
    """Every draft pass and every verify pass of every step of every sequence was compared element by element, every
    draft decision was checked, and the committed caches were read back."""
    D, K = cfg.tree_depth, cfg.tree_topk
    for name in ("draft_logits", "draft_a", "pool_score", "tree_score", "target_logits", "node_hidden", "node_taps",
                 "kv_target", "kv_draft"):
        assert name in st.max_err, f"{name} was never compared"
    units = st.steps * sequences
    assert st.passes == units * D, st
    assert st.verify_compared == units, st
    per_step = K + (D - 1) * K * K + max(D - 2, 0) * K + 1    # every rank of every top-k row and frontier, the pruned set
    assert st.decisions == units * per_step, st


def test_c5_shape_two_layer_steps_vs_oracle():
    """70B-shaped widths (hidden 8192, 64 query / 8 KV heads, FFN 28672, FC 24576 -> 8192, vocab 128256 / 32000),
    depth 6, top-k 10, 60 nodes, 2-layer truncation: two greedy steps and one step with stochastic acceptance."""
    cfg = synth.C5.truncated(2, prompt_len=96)
    st, _, _ = _run(cfg, 2)
    assert st.steps == 2
    _assert_everything_compared(st, cfg)
    assert st.decisions_forced >= 200 and st.argmax_forced >= 60 and st.accept_checked == 2, st
    st2, _, _ = _run(cfg, 1, sampling=(0.8, 31))
    assert st2.steps == 1 and st2.passes == cfg.tree_depth and st2.verify_compared == 1, st2


def test_c4_shape_two_layer_long_context_steps_vs_oracle():
    """8B widths at a 2304-token context with the long-reasoning tree (depth 8, top-k 10, 60 nodes; 70 draft tail keys,
    i.e. two-word ancestor masks), 2-layer truncation: the tree passes run the tcgen05 attention kernel with several key
    tiles per CTA, key splits and the split merge inside a step that is compared with the oracle; RoPE positions and the
    paged cache reach 2.3k."""
    cfg = synth.C4.truncated(2, prompt_len=2304)
    st, _, _ = _run(cfg, 2, greedy_check=False)
    assert st.steps == 2
    _assert_everything_compared(st, cfg)
    assert st.decisions_forced >= 200 and st.argmax_forced >= 60 and st.accept_checked == 2, st


def test_c3_shape_two_layer_batch64_steps_vs_oracle():
    """8B widths at batch 64 with chains of 3 (Section 4.3's serving setting), ragged prompts of 16..64 tokens, 2-layer
    truncation: 256-row verify passes (the widest GEMM tiles, the gate/up pair kernel), the key-parallel attention
    kernel at <= 4 rows per sequence and longest-first issue, against 64 oracles."""
    cfg = synth.C3.truncated(2, prompt_lo=16, prompt_hi=64)
    st, _, prompts = _run(cfg, 2, page_shuffle_seed=13, greedy_check=False)
    assert len(prompts) == 64 and st.steps == 2
    # a chain: every step has 3 draft passes of one row per sequence
    _assert_everything_compared(st, cfg, sequences=64)
    assert st.decisions_forced >= 64 * 4 and st.same_tree >= 100, st
    assert st.argmax_forced >= 64 * 4 and st.accept_checked == 128 and st.exact_out >= 64, st


def test_c2_full_depth_steps_vs_oracle():
    """The benchmarked 8B-shaped model at its full depth of 32 layers (taps after layers 2, 16 and 29), prompt 64,
    depth 6, top-k 10, 60 nodes: two whole steps against the oracle."""
    cfg = synth.C2.replace(name="C2-8B-b1-p64", prompt_len=64)
    st, _, _ = _run(cfg, 2, greedy_check=False)
    assert st.steps == 2
    _assert_everything_compared(st, cfg)
    assert st.decisions_forced >= 200 and st.argmax_forced >= 60 and st.accept_checked == 2, st


def test_c3_shape_with_split_k_cta_pairs_vs_oracle():
    """The same batch-64 steps with the 256-row split-K GEMMs (QKV with RoPE and KV write, O and down with residual and
    norm statistics) ALSO running as CTA pairs (an optional mode; the gate/up kernel runs as pairs by default): the whole
    step is compared with the 64 oracles exactly as above."""
    L = sb.lib()
    cfg = synth.C3.truncated(2, prompt_lo=16, prompt_hi=64)
    try:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 3) == 0
        st, _, prompts = _run(cfg, 2, page_shuffle_seed=13, greedy_check=False)
    finally:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 2) == 0      # the library's default
    assert len(prompts) == 64 and st.steps == 2
    _assert_everything_compared(st, cfg, sequences=64)
    assert st.decisions_forced >= 64 * 4 and st.argmax_forced >= 64 * 4 and st.accept_checked == 128, st
