"""GPU parity tests: the CUDA path (through the C ABI) against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

import parity
import pyoracle as po
from paper_2503_01840_b200 import binding as sb
from paper_2503_01840_b200 import synth

pytestmark = pytest.mark.gpu

C1 = synth.C1
# the tiny model in bf16: exercises the tcgen05 GEMM and bf16 caches at a size the oracle runs in ms
T1 = C1.replace(name="T1-tiny-bf16", dtype="bf16")
# a wider small bf16 model with head_dim 128 and 4 query heads per KV head, like the 8B shapes
T2 = synth.ModelCfg("T2-small-bf16", "bf16", 3, 512, 8, 2, 128, 1408, 8192, 2048, (0, 1, 2), 5e5,
                    prompt_len=150, tree_depth=4, tree_topk=5, tree_nodes=24, seed=11)


def _weights(cfg):
    return synth.make_target_weights(cfg), synth.make_draft_weights(cfg)


# ----------------------------------------------------------------------------- single kernels
@pytest.mark.parametrize("rows,O,I", [(1, 128, 64), (7, 256, 256), (10, 1000, 512), (16, 4096, 4096), (17, 384, 200),
                                      (60, 6144, 4096), (64, 128, 14336), (65, 640, 1024), (200, 512, 768),
                                      (256, 1024, 2048)])
def test_gemm_tcgen05_vs_oracle(rows, O, I):
    g = torch.Generator().manual_seed(rows * 1000 + O + I)
    x = (torch.randn(rows, I, generator=g)).to(torch.bfloat16)
    w = (torch.randn(O, I, generator=g) / I ** 0.5).to(torch.bfloat16)
    ref = po.linear(w, x.float().numpy())
    out = sb.gemm(x.cuda(), w.cuda(), impl=0).cpu().numpy()
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() < 2e-3, np.abs(out - ref).max()
    out_ref_kernel = sb.gemm(x.cuda(), w.cuda(), impl=1).cpu().numpy()
    assert np.abs(out_ref_kernel - ref).max() < 2e-3


@pytest.mark.parametrize("rows,O,I,split,stages", [(1, 128, 64, 0, 0), (7, 256, 256, 2, 0), (10, 1000, 512, 0, 0),
                                                    (16, 4096, 4096, 4, 8), (17, 384, 200, 0, 0), (60, 6144, 4096, 3, 0),
                                                    (64, 128, 14336, 8, 0), (65, 640, 1024, 0, 0), (200, 512, 768, 0, 3),
                                                    (256, 1024, 2048, 5, 0), (60, 4096, 4096, 0, 0), (10, 32000, 512, 0, 0)])
def test_gemm_cluster_split_k_vs_oracle(rows, O, I, split, stages):
    """The step's GEMM kernel (cluster split-K through distributed shared memory) with the plain fp32 epilogue."""
    g = torch.Generator().manual_seed(rows * 1000 + O + I)
    x = (torch.randn(rows, I, generator=g)).to(torch.bfloat16)
    w = (torch.randn(O, I, generator=g) / I ** 0.5).to(torch.bfloat16)
    ref = po.linear(w, x.float().numpy())
    out = sb.gemm_fused(x.cuda(), w.cuda(), split=split, stages=stages).cpu().numpy()
    assert np.isfinite(out).all()
    assert np.abs(out - ref).max() < 2e-3, np.abs(out - ref).max()
    again = sb.gemm_fused(x.cuda(), w.cuda(), split=split, stages=stages).cpu().numpy()
    assert np.array_equal(out, again), "the cluster reduction must be deterministic"


@pytest.mark.parametrize("rows,F,I", [(1, 768, 512), (7, 896, 704), (10, 1000, 1024), (16, 1024, 520), (33, 2048, 4096),
                                      (60, 14336, 4096), (64, 1408, 576), (5, 256, 4096), (100, 1024, 512), (130, 1000, 520),
                                      (200, 1408, 576), (256, 2048, 1024), (60, 28672, 512), (12, 20480, 256)])
def test_gemm_swiglu_vs_oracle(rows, F, I):
    """Gate/up projection with SiLU(gate) * up: one CTA holds the gate and the up tile of its 128 features (two
    accumulators); up to 128 rows the K slices of a tile pair form a cluster, wider tiles run without K split.  An odd
    number of k-blocks, a ragged last k-block, F not a multiple of 128, every row-tile width, and feature counts large
    enough that a tile pair gets a single K slice (no cluster)."""
    g = torch.Generator().manual_seed(rows * 1000 + F + I)
    x = (torch.randn(rows, I, generator=g)).to(torch.bfloat16)
    wg = (torch.randn(F, I, generator=g) / I ** 0.5).to(torch.bfloat16)
    wu = (torch.randn(F, I, generator=g) / I ** 0.5).to(torch.bfloat16)
    xf = x.float().numpy()
    ref = po.swiglu(po.linear(wg, xf), po.linear(wu, xf))
    out = sb.gemm_swiglu(x.cuda(), wg.cuda(), wu.cuda()).float().cpu().numpy()
    assert np.isfinite(out).all()
    err = np.abs(out - ref) - 2.0 ** -8 * np.abs(ref)          # one bf16 rounding of the result
    assert err.max() < 2e-3, err.max()
    again = sb.gemm_swiglu(x.cuda(), wg.cuda(), wu.cuda()).float().cpu().numpy()
    assert np.array_equal(out, again), "the cluster reduction must be deterministic"


def test_gemm_plain_fp32_vs_oracle():
    g = torch.Generator().manual_seed(5)
    x, w = torch.randn(33, 300, generator=g), torch.randn(77, 300, generator=g) / 17
    ref = po.linear(w, x.numpy())
    out = sb.gemm(x.cuda(), w.cuda(), impl=1).cpu().numpy()
    assert np.abs(out - ref).max() < 1e-4


def test_logsoftmax_topk_and_argmax_bit_exact():
    g = torch.Generator().manual_seed(6)
    z = torch.randn(12, 32000, generator=g) * 1.5
    z[3, 100] = z[3, 200] = z[3].max() + 1.0          # a tie at the top: lowest index first
    z[5, :] = 0.25                                     # all equal
    am = sb.argmax(z.cuda()).cpu().numpy()
    for two_stage in (True, False):
        idx, lp = sb.logsoftmax_topk(z.cuda(), 10, two_stage=two_stage)
        idx, lp = idx.cpu().numpy(), lp.cpu().numpy()
        _check_topk(z, idx, lp, am)
    big = torch.randn(3, 128256, generator=g)
    assert sb.argmax(big.cuda()).cpu().tolist() == big.argmax(1).tolist()
    bi, bl = sb.logsoftmax_topk(big.cuda(), 16)
    for r in range(3):
        oi, ov, _ = po.topk(po.log_softmax(big[r].numpy()), 16)
        assert bi[r].cpu().tolist() == oi.tolist() and np.abs(bl[r].cpu().numpy() - ov).max() < 1e-5


def _check_topk(z, idx, lp, am):
    for r in range(z.shape[0]):
        olp = po.log_softmax(z[r].numpy())
        oi, ov, _ = po.topk(olp, 10)
        gaps = np.diff(ov)
        if r in (3, 5) or (np.abs(gaps) > 1e-5).all():
            assert idx[r].tolist() == oi.tolist(), r
        assert np.abs(lp[r] - ov).max() < 1e-5
        assert am[r] == po.argmax(z[r].numpy())[0]
    assert idx[3, 0] == 100 and idx[3, 1] == 200 and idx[5].tolist() == list(range(10))


@pytest.mark.parametrize("dtype,impl", [(torch.float32, 1), (torch.bfloat16, 1), (torch.bfloat16, 0), (torch.bfloat16, 2)])
def test_attention_kernel_vs_oracle(dtype, impl):
    """Paged, tree-masked GQA attention against the oracle's per-head routine."""
    H, G, hd, ps = 8, 2, 128, 16
    if impl != 1 and not _fast_attn_available(hd, H // G):
        pytest.skip("tensor-core attention not built for this shape")
    g = torch.Generator().manual_seed(7)
    n_seq, pps = 2, 24
    ctx = [203, 77]
    tail_len = 40
    perm = torch.randperm(n_seq * pps, generator=g).to(torch.int32).reshape(n_seq, pps)
    kp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(dtype)
    vp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(dtype)
    rows = 24
    q = torch.randn(rows, H, hd, generator=g).to(dtype)
    seq = torch.tensor([r % 2 for r in range(rows)], dtype=torch.int32)
    seq[5] = -1
    rctx = torch.tensor([ctx[r % 2] for r in range(rows)], dtype=torch.int32)
    lo = torch.randint(0, 2 ** 40, (rows,), generator=g, dtype=torch.int64) | 1
    lo[3] = 1
    hi = torch.zeros(rows, dtype=torch.int64)
    out = sb.attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(), ps, seq.cuda(), rctx.cuda(), rctx.cuda(),
                       lo.cuda(), hi.cuda(), tail_len, G, 512, impl=impl).float().cpu().numpy()
    tol = 1e-4 if dtype == torch.float32 else 2e-2
    for r in range(rows):
        if seq[r] < 0:
            assert (out[r] == 0).all()
            continue
        s = int(seq[r])
        pos = list(range(ctx[s])) + [ctx[s] + t for t in range(tail_len) if (int(lo[r]) >> t) & 1]
        for h in range(H):
            gk = h // (H // G)
            K = np.stack([kp[perm[s, p // ps], gk, p % ps].float().numpy() for p in pos])
            V = np.stack([vp[perm[s, p // ps], gk, p % ps].float().numpy() for p in pos])
            ref = po.attend(q[r, h].float().numpy(), K, V)
            assert np.abs(out[r, h] - ref).max() < tol, (r, h)


@pytest.mark.parametrize("rows,H,G,ctx,tail_len", [(60, 32, 8, 517, 60), (5, 8, 2, 64, 5), (24, 8, 2, 1000, 24), (33, 16, 2, 130, 33),
                                                   (10, 32, 8, 0, 10), (60, 32, 8, 4033, 60)])
def test_attention_tcgen05_kernel_vs_oracle(rows, H, G, ctx, tail_len):
    """tcgen05 tree attention (S = Q K^T and O += P V on tcgen05.mma, head_dim 128): one sequence, 128-row tiles that are
    full, partly filled and spread over two CTAs, contexts that end inside a key tile, an empty context, key splits."""
    hd, ps = 128, 16
    g = torch.Generator().manual_seed(rows * 31 + ctx)
    pps = (ctx + tail_len) // ps + 2
    perm = torch.randperm(pps, generator=g).to(torch.int32).reshape(1, pps)
    kp = torch.randn(pps, G, ps, hd, generator=g).to(torch.bfloat16)
    vp = torch.randn(pps, G, ps, hd, generator=g).to(torch.bfloat16)
    q = torch.randn(rows, H, hd, generator=g).to(torch.bfloat16)
    seq = torch.zeros(rows, dtype=torch.int32)
    seq[rows // 2] = -1                                       # a padding row
    rctx = torch.full((rows,), ctx, dtype=torch.int32)
    lo = torch.randint(0, 2 ** min(tail_len, 62), (rows,), generator=g, dtype=torch.int64) | 1
    hi = torch.zeros(rows, dtype=torch.int64)
    out = sb.attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(), ps, seq.cuda(), rctx.cuda(), rctx.cuda(), lo.cuda(),
                       hi.cuda(), tail_len, G, ctx + 64, impl=3).float().cpu().numpy()
    assert np.isfinite(out).all()
    page_of = perm[0].numpy()
    heads = sorted(set([0, H - 1, H // 2, 1]))
    for r in range(rows):
        if seq[r] < 0:
            assert (out[r] == 0).all()
            continue
        pos = np.array(list(range(ctx)) + [ctx + t for t in range(tail_len) if (int(lo[r]) >> t) & 1], dtype=np.int64)
        for h in heads:
            gk = h // (H // G)
            K = kp[torch.from_numpy(page_of[pos // ps]).long(), gk, torch.from_numpy(pos % ps)].float().numpy()
            V = vp[torch.from_numpy(page_of[pos // ps]).long(), gk, torch.from_numpy(pos % ps)].float().numpy()
            ref = po.attend(q[r, h].float().numpy(), K, V)
            assert np.abs(out[r, h] - ref).max() < 2e-2, (r, h, np.abs(out[r, h] - ref).max())


def _fast_attn_available(hd, group):
    return sb.lib().spec_attn_scratch_bytes(64, 8, hd, 1024) > 0


# ----------------------------------------------------------------------------- whole step
@pytest.mark.parametrize("flags", [0, sb.FLAG_NO_GRAPH])
def test_c1_full_trajectory_fp32(flags):
    """Config 1 end to end: 64-token prompt, depth 3, top-k 4, 16 nodes, 32 generated tokens, fp32, 1e-4."""
    tw, dw = _weights(C1)
    prompts = [p.numpy() for p in synth.make_prompts(C1)]
    st, emitted = parity.run_trajectory(C1, tw, dw, prompts, n_steps=32, tol=1e-4, flags=flags)
    print("C1", st)
    assert st.tokens >= 32 and st.passes == 32 * 3 and st.verify_compared == 32 and st.accept_checked == 32, st
    assert st.decisions_forced >= 800 and st.same_tree >= 30 and st.exact_out >= 24 and st.band_total == 0, st


@pytest.mark.parametrize("flags", [0, sb.FLAG_NO_PDL | sb.FLAG_NO_GRAPH, sb.FLAG_STAMPS, sb.FLAG_REF_GEMM | sb.FLAG_REF_ATTN])
def test_tiny_bf16_trajectory(flags):
    tw, dw = _weights(T1)
    prompts = [p.numpy() for p in synth.make_prompts(T1)]
    st, _ = parity.run_trajectory(T1, tw, dw, prompts, n_steps=16, tol=2e-2, flags=flags, tap_tol=3e-2)
    print("T1", flags, st)
    assert st.passes == 16 * 3 and st.verify_compared == 16 and st.accept_checked == 16, st
    assert st.decisions_forced >= 40 and st.same_tree >= 4 and st.argmax_forced >= 150, st


@pytest.mark.parametrize("flags", [0, sb.FLAG_NO_TMA_ATTN])
def test_small_bf16_hd128_trajectory(flags):
    tw, dw = _weights(T2)
    prompts = [p.numpy() for p in synth.make_prompts(T2)]
    st, _ = parity.run_trajectory(T2, tw, dw, prompts, n_steps=10, tol=2e-2, tap_tol=3e-2, flags=flags)
    print("T2", st)
    assert st.passes == 10 * 4 and st.verify_compared == 10 and st.decisions_forced >= 20 and st.argmax_forced >= 150, st


@pytest.mark.parametrize("batch", [1, 3])
def test_small_bf16_hd128_trajectory_tcgen05_attention(batch):
    """The same model with the tree passes' attention on the tcgen05 kernel (draft levels of 5 nodes x 4 heads, verify
    passes of 24 x 4 query rows per KV head), one sequence and a batch of three with different lengths."""
    cfg = T2.replace(name="T2-b%d" % batch, batch=batch, prompt_lo=90, prompt_hi=170) if batch > 1 else T2
    tw, dw = _weights(cfg)
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    st, _ = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=6, tol=2e-2, tap_tol=3e-2,
                                  tune=[(sb.SpecDecoder.TUNE_ATTN_UMMA, 1, 2)])
    print("T2 tcgen05 attention", st)
    assert st.passes == 6 * 4 * batch and st.verify_compared == 6 * batch and st.argmax_forced >= 80 * batch, st


# multi-head attention (one KV head per query head), as in the Vicuna-13B-shaped targets of the paper's Table 1
T3_MHA = synth.ModelCfg("T3-small-bf16-mha", "bf16", 2, 512, 4, 4, 128, 1024, 4096, 1024, (0, 1, 1), 1e4,
                        prompt_len=90, tree_depth=5, tree_topk=8, tree_nodes=50, seed=21)


@pytest.mark.parametrize("batch", [1, 2])
def test_mha_model_trajectory(batch):
    """G = H (no grouping): 50-node trees, 8 x 4 = 32 draft rows per pass, also at batch 2 (trees at batch)."""
    cfg = T3_MHA if batch == 1 else T3_MHA.replace(name="T3-b2", batch=2, prompt_lo=40, prompt_hi=100)
    tw, dw = _weights(cfg)
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    st, _ = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=6, tol=2e-2, tap_tol=3e-2)
    print("T3 MHA", batch, st)
    assert st.steps == 6 and st.passes == 6 * 5 * batch and st.verify_compared == 6 * batch and st.decisions_forced >= 10, st


@pytest.mark.parametrize("base", [C1, T1], ids=["fp32", "bf16"])
def test_prefill_chunk_boundaries(base):
    """Prompts of 127, 128, 129, 255, 256, 257 and 513 tokens: the prefill runs 256-position passes made of two
    128-position blocks (rows of a block see each other through the two-word causal masks, the earlier block of the same
    pass is context); the first token, the first steps and the committed K/V must match the oracle."""
    for n in (127, 128, 129, 255, 256, 257, 513):
        cfg = base.replace(name=f"{base.name}-p{n}", prompt_len=n)
        tw, dw = _weights(cfg)
        prompts = [p.numpy() for p in synth.make_prompts(cfg)]
        assert len(prompts[0]) == n
        tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
        st, _ = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=2, tol=tol, tap_tol=None if cfg.dtype == "fp32" else 3e-2)
        dec = sb.SpecDecoder(cfg, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=n + 64)
        orc = po.Oracle(cfg, tw, dw, n + 64)
        assert dec.prefill(prompts, 8)[0] == orc.prefill(prompts[0])
        for pos in sorted(set([0, 63, 64, 126, min(128, n - 1), min(200, n - 1), n - 2, n - 1])):
            for layer in range(cfg.n_layers):
                gk, gv = dec.read_kv(0, layer, pos)
                ok, ov = orc.target_kv(layer, pos)
                assert np.abs(gk - ok).max() < 4 * tol and np.abs(gv - ov).max() < 4 * tol, (n, pos, layer)
        dec.close()


DEGENERATE = {
    "depth1": dict(tree_depth=1, tree_topk=4, tree_nodes=5),                 # one draft pass, the tree is a star
    "chain_b1": dict(tree_depth=3, tree_topk=1, tree_nodes=4),               # top-1 chain at batch 1
    "pool_smaller_than_tree": dict(tree_depth=2, tree_topk=3, tree_nodes=40),  # N - 1 > K + (D-1) K^2: every candidate kept, padding rows
    "two_word_masks": dict(tree_depth=8, tree_topk=10, tree_nodes=60),       # (D-1) K = 70 draft tail keys: bits beyond 64
    "two_nodes": dict(tree_depth=2, tree_topk=2, tree_nodes=2),              # the root and one candidate
    "short_prompt": dict(tree_depth=3, tree_topk=4, tree_nodes=16, prompt_len=2),
}


@pytest.mark.parametrize("base", [C1, T1], ids=["fp32", "bf16"])
@pytest.mark.parametrize("case", sorted(DEGENERATE))
def test_degenerate_tree_shapes_trajectory(base, case):
    """Edge shapes of the draft tree against the oracle: depth 1, a chain, a pool smaller than the node budget, more than
    64 tail keys (two-word ancestor masks), a two-node tree, a two-token prompt."""
    cfg = base.replace(name=base.name + "-" + case, **DEGENERATE[case])
    tw, dw = _weights(cfg)
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
    st, _ = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=5, tol=tol, tap_tol=None if cfg.dtype == "fp32" else 3e-2)
    print(case, st)
    assert st.steps == 5 and st.passes == 5 * cfg.tree_depth and st.verify_compared == 5 and st.accept_checked == 5, st


@pytest.mark.parametrize("temperature", [1.0, 0.3])
@pytest.mark.parametrize("base", [C1, T1, T2], ids=["fp32", "bf16", "bf16_hd128"])
def test_sampled_acceptance_trajectory(base, temperature):
    """Temperature > 0: the stochastic acceptance kernel against the oracle's rule with the same uniforms, step by step
    (every accept / reject and the drawn token allowed by the oracle's probabilities within the logit tolerance, identical
    where the oracle's margin exceeds it), on the fp32 model, the tiny bf16 model and a batch of the head_dim-128 model."""
    cfg = base if base is not T2 else T2.replace(name="T2-b2-sampled", batch=2, prompt_lo=60, prompt_hi=120)
    tw, dw = _weights(cfg)
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
    st, emitted = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=10, tol=tol, tap_tol=None if cfg.dtype == "fp32" else 3e-2,
                                        sampling=(temperature, 17))
    print("sampled", cfg.name, temperature, st)
    # same_tree counts sequence-steps whose tree equals the oracle's OWN choice (not merely a valid one); at bf16 on the
    # batch-2 head_dim-128 model near-ties leave few of them, so only its presence is required there
    assert st.steps == 10 and st.same_tree >= (3 if cfg.batch == 1 else 1) and st.verify_compared == 10 * cfg.batch and st.passes == 10 * cfg.batch * cfg.tree_depth, st
    if cfg.dtype == "fp32":
        assert st.resyncs <= 1          # float errors of ~4e-6: the outputs coincide with the oracle's


@pytest.mark.parametrize("cfg", [C1, T1], ids=["fp32", "bf16"])
def test_sampled_acceptance_with_structured_weights_accepts_drafts(cfg):
    """Designed draft/target agreement at temperature 1: accepted paths longer than one node, multi-entry commit and
    extend under the stochastic rule."""
    tw, dw, pi, pi2 = synth.make_structured(cfg, 0.85, residual_scale=0.05)
    prompt = synth.structured_prompt(cfg, dw["d2t"], 48).numpy()
    tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
    st, emitted = parity.run_trajectory(cfg, tw, dw, [prompt], n_steps=12, tol=tol, tap_tol=tol * 1.5, sampling=(1.0, 5))
    print("structured sampled", cfg.name, st)
    assert st.tokens > 12 + 6, "the structured workload must accept draft tokens"


def test_sampled_step_low_temperature_is_greedy():
    """T -> 0: the sampled step emits what the greedy step emits (same kernels, same state)."""
    tw, dw = _weights(T1)
    prompts = [p.numpy() for p in synth.make_prompts(T1)]
    outs = []
    for sampled in (False, True):
        dec = sb.SpecDecoder(T1, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=len(prompts[0]) + 200)
        dec.prefill(prompts, 100)
        rng = np.random.default_rng(3)
        acc = []
        for _ in range(8):
            u = rng.uniform(0.01, 0.99, (1, 2 * T1.tree_nodes)).astype(np.float32)
            acc += (dec.step_sampled(1e-4, u) if sampled else dec.step())[0].tolist()
        outs.append(acc)
        dec.close()
    n = min(len(outs[0]), len(outs[1]))
    assert outs[0][:n] == outs[1][:n]


@pytest.mark.parametrize("cfg", [C1, T1], ids=["fp32", "bf16"])
def test_structured_weights_accept_more_than_one(cfg):
    """Designed agreement between draft and target: counts > 1, KV compaction and multi-entry extend."""
    tw, dw, pi, pi2 = synth.make_structured(cfg, 0.85, residual_scale=0.05)
    prompt = synth.structured_prompt(cfg, dw["d2t"], 48).numpy()
    tol = 1e-4 if cfg.dtype == "fp32" else 2e-2
    st, emitted = parity.run_trajectory(cfg, tw, dw, [prompt], n_steps=12, tol=tol, tap_tol=tol * 1.5)
    print("structured", cfg.name, st)
    assert st.tokens > 12 + 6, "the structured workload must accept draft tokens"
    # committed KV equals the oracle's for the whole prefix (compaction moved the right rows)
    B = 1
    dec = sb.SpecDecoder(cfg, parity.to_dev(tw), parity.to_dev(dw), batch=B, max_ctx=256)
    orc = po.Oracle(cfg, tw, dw, 256)
    assert dec.prefill([prompt], 120)[0] == orc.prefill(prompt)
    for _ in range(6):
        g = dec.step()[0]
        o = orc.step()
        if not np.array_equal(g, o):
            orc.force_state(np.concatenate([orc.ids[: orc.n - len(o)], g]).astype(np.int32), orc.n - len(o) + len(g), len(g))
    n = int(dec.lengths()[0])
    assert n == orc.n
    for pos in list(range(0, n, 7)) + [n - 1, n - 2]:
        for layer in range(cfg.n_layers):
            gk, gv = dec.read_kv(0, layer, pos)
            ok, ov = orc.target_kv(layer, pos)
            assert np.abs(gk - ok).max() < 4 * tol and np.abs(gv - ov).max() < 4 * tol, (pos, layer)
    for pos in range(0, n - orc.pending, 5):
        gk, gv = dec.read_kv(0, -1, pos)
        ok, ov = orc.draft_kv(pos)
        assert np.abs(gk - ok).max() < 4 * tol and np.abs(gv - ov).max() < 4 * tol, pos
    dec.close()


def test_batch_chain_with_shuffled_pages():
    """Serving-style case (Section 4.3): several sequences of different lengths, chain drafts (top-k 1)."""
    cfg = T1.replace(name="T1-chain", batch=5, prompt_lo=20, prompt_hi=90, tree_depth=3, tree_topk=1, tree_nodes=4, seed=3)
    tw, dw = _weights(cfg)
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    st, _ = parity.run_trajectory(cfg, tw, dw, prompts, n_steps=8, tol=2e-2, tap_tol=3e-2, page_shuffle_seed=77)
    print("chain", st)
    assert st.passes == 8 * 5 * 3 and st.verify_compared == 40 and st.accept_checked == 40 and st.decisions_forced >= 100, st


def test_page_permutation_invariance():
    cfg = C1
    tw, dw = _weights(cfg)
    prompt = synth.make_prompts(cfg)[0].numpy()
    outs = []
    for seed in (0, 5, 9):
        dec = sb.SpecDecoder(cfg, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=256, num_pages=40,
                             page_shuffle_seed=seed)
        first = dec.prefill([prompt], 100)
        toks = [int(first[0])]
        for _ in range(8):
            toks += dec.step()[0].tolist()
        table = dec.debug(sb.DBG_PAGE_TABLE, 0)
        logits = dec.debug(sb.DBG_TARGET_LOGITS, 0)
        outs.append((toks, table, logits))
        dec.close()
    assert not np.array_equal(outs[0][1], outs[1][1])
    for o in outs[1:]:
        assert o[0] == outs[0][0]
        assert np.array_equal(o[2], outs[0][2])          # physical placement must not change a single bit


def test_capacity_error_leaves_state_unchanged():
    cfg = C1
    tw, dw = _weights(cfg)
    prompt = synth.make_prompts(cfg)[0].numpy()
    dec = sb.SpecDecoder(cfg, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=256)
    dec.prefill([prompt], 4)
    n_ok = 0
    with pytest.raises(sb.SpecError) as e:
        for _ in range(40):
            dec.step()
            n_ok += 1
    assert e.value.code == -4 and n_ok >= 1
    n = dec.lengths()
    with pytest.raises(sb.SpecError):
        dec.step()
    assert np.array_equal(dec.lengths(), n)
    with pytest.raises(sb.SpecError) as e2:
        sb.SpecDecoder(cfg, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=256, num_pages=2).prefill([prompt], 4)
    assert e2.value.code == -4
    dec.close()


def test_plain_decode_matches_oracle_greedy():
    tw, dw = _weights(C1)
    prompt = synth.make_prompts(C1)[0].numpy()
    dec = sb.SpecDecoder(C1, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=256)
    first = dec.prefill([prompt], 40)
    got = [int(dec.plain_step()[0]) for _ in range(12)]
    o = po.Oracle(C1, tw, dw, 256)
    assert o.prefill(prompt) == first[0]
    ref, mg = o.greedy_margins(12)
    for i in range(12):
        if got[i] != ref[i]:
            assert mg[i] < parity.MARGIN
            break
    with pytest.raises(sb.SpecError):
        dec.step()                     # the draft cache is stale after plain decoding
    dec.close()


@pytest.mark.parametrize("flags", [0])
def test_c2_two_layer_truncation_first_steps(flags):
    """8B-shaped widths (hidden 4096, 32/8 heads of 128, FFN 14336, vocab 128256 / 32000, depth 6, top-k 10,
    60 nodes) on a 2-layer truncation, first steps, bf16."""
    cfg = synth.C2.truncated(2, prompt_len=48)
    tw = synth.make_target_weights(cfg, device="cuda")
    dw = synth.make_draft_weights(cfg, device="cuda")
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    st, _ = parity.run_trajectory(cfg, parity.to_cpu(tw), parity.to_cpu(dw), prompts, n_steps=2, tol=2e-2, tap_tol=3e-2, flags=flags)
    print("C2-L2", st)
    assert st.passes == 12 and st.verify_compared == 2 and st.decisions == 2 * (10 + 500 + 40 + 1) and st.argmax_forced >= 60, st


def test_c2_two_layer_truncation_sampled_steps():
    """The same 8B-shaped truncation at temperature 0.7: softmax, residual and inverse CDF over the 128256-entry
    vocabulary of 60 verify nodes against the oracle's rule."""
    cfg = synth.C2.truncated(2, prompt_len=48)
    tw = synth.make_target_weights(cfg, device="cuda")
    dw = synth.make_draft_weights(cfg, device="cuda")
    prompts = [p.numpy() for p in synth.make_prompts(cfg)]
    st, _ = parity.run_trajectory(cfg, parity.to_cpu(tw), parity.to_cpu(dw), prompts, n_steps=2, tol=2e-2, tap_tol=3e-2,
                                  sampling=(0.7, 23))
    print("C2-L2 sampled", st)
    assert st.passes == 12 and st.verify_compared == 2, st


@pytest.mark.parametrize("H,G,hd,rps", [(32, 8, 128, 4), (8, 2, 128, 1), (4, 2, 64, 3)])
def test_attention_few_query_rows_key_parallel_kernel(H, G, hd, rps):
    """At most 16 query rows per (sequence, KV head) (chain drafts at batch, single-token decoding): the key-parallel
    TMA kernel, several sequences of different lengths, against the oracle's per-head routine."""
    ps, n_seq, tail = 16, 5, rps
    g = torch.Generator().manual_seed(70 + H + rps)
    ctxs = [37, 250, 64, 1, 513]
    pps = (max(ctxs) + tail + ps - 1) // ps + 1
    perm = torch.randperm(n_seq * pps, generator=g).to(torch.int32).reshape(n_seq, pps)
    kp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(torch.bfloat16)
    vp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(torch.bfloat16)
    rows = n_seq * rps
    q = torch.randn(rows, H, hd, generator=g).to(torch.bfloat16)
    seq = torch.tensor([r // rps for r in range(rows)], dtype=torch.int32)
    rctx = torch.tensor([ctxs[r // rps] for r in range(rows)], dtype=torch.int32)
    lo = torch.tensor([(1 << ((r % rps) + 1)) - 1 for r in range(rows)], dtype=torch.int64)      # causal chain
    hi = torch.zeros(rows, dtype=torch.int64)
    out = sb.attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(), ps, seq.cuda(), rctx.cuda(), rctx.cuda(), lo.cuda(), hi.cuda(),
                       tail, G, 1024, impl=2).float().cpu().numpy()
    for r in range(rows):
        s = int(seq[r])
        pos = list(range(ctxs[s])) + [ctxs[s] + t for t in range(tail) if (int(lo[r]) >> t) & 1]
        for h in range(0, H, max(1, H // 4)):
            gk = h // (H // G)
            K = np.stack([kp[perm[s, p // ps], gk, p % ps].float().numpy() for p in pos])
            V = np.stack([vp[perm[s, p // ps], gk, p % ps].float().numpy() for p in pos])
            ref = po.attend(q[r, h].float().numpy(), K, V)
            assert np.abs(out[r, h] - ref).max() < 2e-2, (r, h)


def test_bounded_device_wait_runs_out_and_is_reported():
    """Failure detection without a fault: one CTA of the verify pass's LM-head GEMM never receives its first activation
    tile (test hook), so its bounded wait runs out.  The CTA records the time-out, skips its arithmetic, waits for its
    loads in flight, frees its tensor memory and leaves; the step returns SPEC_ERR_DEVICE_STATUS with the site of the
    wait, the context stays usable, and a fresh context matches the oracle afterwards."""
    tw, dw = _weights(T1)
    prompts = [p.numpy() for p in synth.make_prompts(T1)]
    for flags in (0, sb.FLAG_NO_GRAPH):
        dec = sb.SpecDecoder(T1, parity.to_dev(tw), parity.to_dev(dw), batch=1, max_ctx=len(prompts[0]) + 200, flags=flags)
        dec.prefill(prompts, 100)
        dec.step()                                           # a healthy step first
        dec.tune(sb.SpecDecoder.TUNE_DEBUG_WAIT_RUNS_OUT, 2000)
        with pytest.raises(sb.SpecError) as e:
            dec.step()
        assert e.value.code == -7 and "site 201" in str(e.value), str(e.value)
        assert (dec.debug(sb.DBG_STATUS, 0) == 0).all()      # the status words were cleared when they were reported
        dec.tune(sb.SpecDecoder.TUNE_DEBUG_WAIT_RUNS_OUT, 0)
        n0 = int(dec.lengths()[0])
        out = dec.step()[0]                                  # the context still runs steps
        assert 1 <= len(out) <= T1.tree_depth + 1 and int(dec.lengths()[0]) == n0 + len(out)
        dec.close()
    st, _ = parity.run_trajectory(T1, tw, dw, prompts, n_steps=4, tol=2e-2, tap_tol=3e-2)
    assert st.steps == 4 and st.verify_compared == 4


@pytest.mark.parametrize("O,K", [(32000, 10), (32768, 9), (1000, 4), (4096, 15), (130, 1)])
def test_lm_head_topk_epilogue_and_merge_bit_exact(O, K):
    """The draft LM head whose epilogue leaves per-tile top-K candidates and softmax statistics, followed by the merge
    (the logits are never written): ids bit-exact against the oracle's log-softmax + top-k, ties included (lower id
    first), an all-equal row, a vocabulary that is not a multiple of the tile.  The logits are planted exactly through
    the GEMM: x is an identity, so logits[r][o] = w[o][r]."""
    rows, I = 12, 16
    g = torch.Generator().manual_seed(O + K)
    z = (torch.randn(rows, O, generator=g) * 1.5).to(torch.bfloat16).float()
    if O > 300:
        z[3, 100] = z[3, 200] = z[3].max() + 1.0           # a tie at the top: lowest index first
        z[7, O - 1] = z[7, 0] = z[7].max() + 0.5           # a tie across the first and the last tile
    z[5, :] = 0.25                                         # all equal: ids 0..K-1
    x = torch.zeros(rows, I, dtype=torch.bfloat16)
    x[torch.arange(rows), torch.arange(rows)] = 1.0
    w = torch.zeros(O, I, dtype=torch.bfloat16)
    w[:, :rows] = z.t().to(torch.bfloat16)
    idx, lp = sb.gemm_topk(x.cuda(), w.cuda(), K)
    idx, lp = idx.cpu().numpy(), lp.cpu().numpy()
    for r in range(rows):
        oi, ov, _ = po.topk(po.log_softmax(z[r].numpy()), K)
        assert idx[r].tolist() == oi.tolist(), (r, idx[r], oi)
        assert np.abs(lp[r] - ov).max() < 5e-5, r           # fp32 sums of up to 32768 exp terms in two different orders
    assert idx[5].tolist() == list(range(K))
    if O > 300:
        assert idx[3, 0] == 100 and (K < 2 or idx[3, 1] == 200) and idx[7, 0] == 0 and (K < 2 or idx[7, 1] == O - 1)
    with pytest.raises(sb.SpecError):
        sb.gemm_topk(x.cuda(), torch.zeros(40000, I, dtype=torch.bfloat16, device="cuda"), K)     # more than 256 tiles


@pytest.mark.parametrize("T,H,G,J", [(300, 8, 2, 3), (128, 4, 4, 0), (517, 32, 8, 1), (70, 8, 2, 8)])
def test_ttt_attention_vs_oracle(T, H, G, J):
    """Training-time-test attention (Section 3.2): dense causal part on the tensor-core tile kernel over 128-position
    blocks (several blocks and a ragged last one), diagonal entries of J simulated steps as dot products, shuffled pages;
    sampled positions (all block boundaries among them) x every head against the oracle's definition: outputs within the
    bf16 tolerance 2e-2, log-normalisers within 2e-2."""
    hd, ps = 128, 16
    g = torch.Generator().manual_seed(T * 7 + J)
    q = torch.randn(T, H, hd, generator=g).to(torch.bfloat16)
    k0 = torch.randn(T, G, hd, generator=g).to(torch.bfloat16)
    v0 = torch.randn(T, G, hd, generator=g).to(torch.bfloat16)
    kd = torch.randn(J, T, G, hd, generator=g).to(torch.bfloat16) if J else None
    vd = torch.randn(J, T, G, hd, generator=g).to(torch.bfloat16) if J else None
    pps = (T + ps - 1) // ps + 1
    perm = torch.randperm(pps + 3, generator=g)[:pps].to(torch.int32)
    kp = torch.zeros(pps + 3, G, ps, hd, dtype=torch.bfloat16)
    vp = torch.zeros(pps + 3, G, ps, hd, dtype=torch.bfloat16)
    for p_ in range(T):
        kp[perm[p_ // ps], :, p_ % ps] = k0[p_]
        vp[perm[p_ // ps], :, p_ % ps] = v0[p_]
    out, lse = sb.ttt_attention(q.cuda(), kp.cuda(), vp.cuda(), perm.cuda(), kd.cuda() if J else None,
                                vd.cuda() if J else None, want_lse=True)
    out, lse = out.float().cpu().numpy(), lse.cpu().numpy()
    assert out.shape == (T, H, hd) and lse.shape == (T, H) and np.isfinite(out).all()
    rows = sorted(set(range(0, T, 5)) | ({0, 1, 63, 64, 127, 128, 129, 255, 256, 257, T - 2, T - 1} & set(range(T))))
    zero = np.zeros((0, T, G, hd))
    o_out, o_lse = po.ttt_attention_rows(q.float().numpy(), k0.float().numpy(), v0.float().numpy(),
                                         kd.float().numpy() if J else zero, vd.float().numpy() if J else zero, rows)
    assert np.abs(out[rows] - o_out).max() < 2e-2, np.abs(out[rows] - o_out).max()
    assert np.abs(lse[rows] - o_lse).max() < 2e-2, np.abs(lse[rows] - o_lse).max()


@pytest.mark.parametrize("rows,O,I,split", [(256, 512, 512, 2), (200, 4096, 4096, 0), (129, 768, 1024, 1), (256, 1024, 4096, 4)])
def test_gemm_cta_pairs_bit_equal(rows, O, I, split):
    """256-row GEMM tiles as CTA pairs (one M = 256 MMA over two CTAs, each loading half of the activation rows) against
    the single-CTA kernel: the same products are added in the same order, so the results must be bit-identical; and
    against a float64 matmul within the bf16-input tolerance."""
    g = torch.Generator().manual_seed(rows + O + I)
    x = torch.randn(rows, I, generator=g).to(torch.bfloat16).cuda()
    w = (torch.randn(O, I, generator=g) / I ** 0.5).to(torch.bfloat16).cuda()
    L = sb.lib()
    try:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 3) == 0
        paired = sb.gemm_fused(x, w, split=split).clone()
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 0) == 0
        single = sb.gemm_fused(x, w, split=min(split, 4)).clone()
    finally:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 2) == 0     # the library's default
    if 1 <= split <= 4:                      # the same K split on both sides
        assert torch.equal(paired, single)
    ref = x.double() @ w.double().t()
    assert (paired.double() - ref).abs().max().item() < 1e-4 * I ** 0.5
    assert (single.double() - ref).abs().max().item() < 1e-4 * I ** 0.5


@pytest.mark.parametrize("rows,F,I", [(256, 512, 512), (200, 1024, 4096), (129, 1792, 1024), (256, 384, 1024)])
def test_gate_up_cta_pairs_bit_equal(rows, F, I):
    """The 256-row gate/up kernel as CTA pairs (the default) against single CTAs: bit-identical activations, and both
    within bf16 rounding of SiLU(x Wg^T) * (x Wu^T) computed in float64."""
    g = torch.Generator().manual_seed(rows + F + I)
    x = torch.randn(rows, I, generator=g).to(torch.bfloat16).cuda()
    wg = (torch.randn(F, I, generator=g) / I ** 0.5).to(torch.bfloat16).cuda()
    wu = (torch.randn(F, I, generator=g) / I ** 0.5).to(torch.bfloat16).cuda()
    L = sb.lib()
    try:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 2) == 0
        paired = sb.gemm_swiglu(x, wg, wu).clone()
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 0) == 0
        single = sb.gemm_swiglu(x, wg, wu).clone()
    finally:
        assert L.spec_tune(None, sb.SpecDecoder.TUNE_GEMM_PAIRS, 2) == 0
    assert torch.equal(paired, single)
    gd, ud = x.double() @ wg.double().t(), x.double() @ wu.double().t()
    ref = torch.nn.functional.silu(gd) * ud
    assert ((paired.double() - ref).abs() <= 2.0 ** -8 * ref.abs() + 1e-3).all()
