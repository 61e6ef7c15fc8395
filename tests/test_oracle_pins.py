"""Pins for the CPU oracle: each test checks it against something other than itself — a library
routine, an independent Llama implementation, brute force, a closed form, or an invariant the
paper fixes (Section 2.1 losslessness, Section 2.2 tree attention, metric definition of tau)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

import hf_ref
import pyoracle as po
from paper_2503_01840_b200 import synth

C1 = synth.C1
TOL = 2e-5


@pytest.fixture(scope="module")
def c1():
    tw = synth.make_target_weights(C1)
    dw = synth.make_draft_weights(C1)
    ids = synth.make_prompts(C1)[0].numpy()
    return tw, dw, ids


def _mk(cfg, tw, dw, max_ctx=256):
    return po.Oracle(cfg, tw, dw, max_ctx)


# ----------------------------------------------------------------------------- building blocks
def test_linear_vs_matmul_fp64():
    g = torch.Generator().manual_seed(0)
    W = torch.randn(37, 129, generator=g)
    x = torch.randn(5, 129, generator=g)
    ref = (x.double() @ W.double().T).numpy()
    assert np.abs(po.linear(W, x.numpy()) - ref).max() < 1e-4
    Wb = W.to(torch.bfloat16)
    refb = (x.double() @ Wb.double().T).numpy()
    assert np.abs(po.linear(Wb, x.numpy()) - refb).max() < 1e-4
    # a transposed operand or swapped index would not survive a non-square W
    assert po.linear(W, x.numpy()).shape == (5, 37)


def test_linear_rows_are_independent():
    g = torch.Generator().manual_seed(1)
    W = torch.randn(50, 300, generator=g)
    x = torch.randn(70, 300, generator=g).numpy()
    full = po.linear(W, x)
    for m in (0, 13, 69):
        assert np.array_equal(full[m], po.linear(W, x[m:m + 1])[0])


def test_rmsnorm_vs_torch():
    g = torch.Generator().manual_seed(2)
    x = torch.randn(4, 256, generator=g) * 3
    gain = 1 + 0.1 * torch.randn(256, generator=g)
    ref = F.rms_norm(x, (256,), gain, 1e-5).numpy()
    assert np.abs(po.rmsnorm(gain, x.numpy(), 1e-5) - ref).max() < TOL


def test_rope_vs_transformers():
    from transformers.models.llama.modeling_llama import LlamaRotaryEmbedding, apply_rotary_pos_emb
    cfg = hf_ref._cfg(C1, 1, 16)
    rot = LlamaRotaryEmbedding(cfg)
    g = torch.Generator().manual_seed(3)
    H, hd = 4, 64
    x = torch.randn(1, H, 3, hd, generator=g)
    pos = torch.tensor([[0, 17, 1234]])
    cos, sin = rot(x, pos)
    ref, _ = apply_rotary_pos_emb(x, x, cos, sin)
    for t, p in enumerate(pos[0].tolist()):
        mine = po.rope(x[0, :, t].reshape(-1).numpy(), H, hd, p, C1.rope_theta).reshape(H, hd)
        assert np.abs(mine - ref[0, :, t].numpy()).max() < (2e-4 if p > 1000 else 1e-5), p
    assert np.array_equal(po.rope(x[0, :, 0].reshape(-1).numpy(), H, hd, 0, 1e4), x[0, :, 0].reshape(-1).numpy())


def test_swiglu_vs_torch():
    g = torch.Generator().manual_seed(4)
    a, b = torch.randn(1000, generator=g) * 4, torch.randn(1000, generator=g)
    assert np.abs(po.swiglu(a.numpy(), b.numpy()) - (F.silu(a) * b).numpy()).max() < TOL


def test_attend_vs_sdpa():
    g = torch.Generator().manual_seed(5)
    q, K, V = torch.randn(64, generator=g), torch.randn(37, 64, generator=g), torch.randn(37, 64, generator=g)
    ref = F.scaled_dot_product_attention(q[None, None, None], K[None, None], V[None, None])[0, 0, 0].numpy()
    assert np.abs(po.attend(q.numpy(), K.numpy(), V.numpy()) - ref).max() < TOL
    # a single key returns its value exactly
    assert np.allclose(po.attend(q.numpy(), K[:1].numpy(), V[:1].numpy()), V[0].numpy())


def test_log_softmax_topk_argmax():
    g = torch.Generator().manual_seed(6)
    z = torch.randn(1024, generator=g) * 2
    lp = po.log_softmax(z.numpy())
    assert np.abs(lp - torch.log_softmax(z, 0).numpy()).max() < TOL
    assert abs(np.exp(lp.astype(np.float64)).sum() - 1) < 1e-5
    idx, val, nxt = po.topk(z.numpy(), 5)
    tv, ti = torch.topk(z, 6)
    assert idx.tolist() == ti[:5].tolist() and np.array_equal(val, tv[:5].numpy()) and nxt == tv[5].item()
    # ties: lowest index first
    t = np.array([1, 3, 3, 2, 3, 0], np.float32)
    assert po.topk(t, 3)[0].tolist() == [1, 2, 4]
    assert po.argmax(t) == (1, 0.0)
    assert po.argmax(np.array([0, 5, 2], np.float32)) == (1, 3.0)


# ----------------------------------------------------------------------------- the target model
def test_target_forward_vs_independent_llama(c1):
    tw, dw, ids = c1
    hf = hf_ref.target_model(C1, tw)
    logits, blocks = hf_ref.forward(hf, torch.from_numpy(ids))
    o = _mk(C1, tw, dw)
    first = o.prefill(ids)
    assert first == int(logits[-1].argmax())
    for pos in (0, 1, 31, 63):
        taps = o.taps(pos).reshape(3, C1.hidden)
        for s, layer in enumerate(C1.fuse_layers):
            assert np.abs(taps[s] - blocks[layer][pos].numpy()).max() < 1e-4, (pos, s)


def test_greedy_vs_independent_llama(c1):
    tw, dw, ids = c1
    hf = hf_ref.target_model(C1, tw)
    gen = hf.generate(torch.from_numpy(ids)[None].long(), do_sample=False, max_new_tokens=12,
                      pad_token_id=0, eos_token_id=None)[0, len(ids):].tolist()
    o = _mk(C1, tw, dw)
    first = o.prefill(ids)
    mine = [first] + o.greedy(11).tolist()
    assert mine == gen


def test_tree_forward_vs_independent_llama_with_4d_mask(c1):
    """Tree attention (Section 2.2): node i sees the context and its ancestors only."""
    tw, dw, ids = c1
    hf = hf_ref.target_model(C1, tw)
    o = _mk(C1, tw, dw)
    o.prefill(ids)
    o.step()
    o.step()
    # state before the last step: n0 committed; reconstruct it from the inspection arrays
    tok, depth, mask = o.get(po.TREE_TOK), o.get(po.TREE_DEPTH), o.get(po.TREE_MASK)
    nn = tok.size
    n0 = o.n - len(o.get(po.PATH))
    ctx = o.ids[:n0]
    allids = torch.from_numpy(np.concatenate([ctx, tok]).astype(np.int64))
    T = n0 + nn
    vis = torch.zeros(T, T, dtype=torch.bool)
    vis[:n0, :n0] = torch.tril(torch.ones(n0, n0, dtype=torch.bool))
    for i in range(nn):
        vis[n0 + i, :n0] = True
        for j in range(nn):
            if (int(mask[i]) >> j) & 1:
                vis[n0 + i, n0 + j] = True
    posid = torch.cat([torch.arange(n0), n0 + torch.from_numpy(depth.astype(np.int64))])
    logits, blocks = hf_ref.forward(hf, allids, position_ids=posid, mask_bool=vis)
    mine = o.get(po.TARGET_LOGITS).reshape(nn, C1.vocab)
    assert np.abs(mine - logits[n0:].numpy()).max() < 2e-4
    taps = o.get(po.NODE_TAPS).reshape(nn, 3, C1.hidden)
    for s, layer in enumerate(C1.fuse_layers):
        assert np.abs(taps[:, s] - blocks[layer][n0:].numpy()).max() < 1e-4


# ----------------------------------------------------------------------------- the draft head
def test_draft_passes_vs_independent_llama_layer(c1):
    """Section 3.1: g = FC3[l;m;h]; x = FC2[g or a ; e(tok)]; decoder layer -> a; LM head.  The
    decoder layer, norm and head come from the independent implementation; every processed tree
    node is re-run as an ordinary causal sequence over its own ancestor path."""
    tw, dw, ids = c1
    hfd = hf_ref.draft_model(C1, dw)
    o = _mk(C1, tw, dw)
    o.prefill(ids)
    o.step()
    n = o.n
    P = o.pending
    committed = o.ids                          # [n+1], last = root
    o.step()
    k, K, D, Vd = C1.hidden, C1.tree_topk, C1.tree_depth, C1.draft_vocab
    fc3, fc2, E = dw["fc3"].double(), dw["fc2"].double(), tw["embed"].double()
    o_taps = po.Oracle(C1, tw, dw, 256)        # fresh oracle just to read taps of the committed prefix
    o_taps.prefill(committed[:n])
    taps = torch.from_numpy(np.stack([o_taps.taps(p) for p in range(n)])).double()
    gfeat = taps @ fc3.T                                                # [n][k]
    gp = o.get(po.G_PENDING).reshape(P, k)
    assert np.abs(gp - gfeat[n - P:].numpy()).max() < 1e-4
    x_ctx = torch.cat([gfeat, E[torch.from_numpy(committed[1:n + 1].astype(np.int64))]], 1) @ fc2.T   # entries 0..n-1
    logits_ctx, blocks = hf_ref.forward(hfd, embeds=x_ctx.float())
    dl = o.get(po.DRAFT_LOGITS).reshape(D, K, Vd)
    da = o.get(po.DRAFT_A).reshape(D, K, k)
    assert np.abs(dl[0, 0] - logits_ctx[-1].numpy()).max() < 2e-4
    assert np.abs(da[0, 0] - blocks[0][-1].numpy()).max() < 2e-4
    # tree passes: node u at depth d-1 fed with (a of its parent, e(tok_u)) after the context
    front = o.get(po.FRONTIER).reshape(D, K)
    ptok, ppar = o.get(po.POOL_TOK), o.get(po.POOL_PARENT)
    a_of = {0: torch.from_numpy(da[0, 0]).double()}
    for d in range(1, D):
        for r in range(K):
            a_of[int(front[d, r])] = torch.from_numpy(da[d, r]).double()
    checked = 0
    for d in range(1, D):
        for r in range(K):
            u = int(front[d, r])
            chain = []
            v = u
            while v != 0:
                chain.append(v)
                v = int(ppar[v])
            chain.reverse()
            rows = [torch.cat([a_of[int(ppar[v])], E[int(ptok[v])]]) @ fc2.T for v in chain]
            x = torch.cat([x_ctx, torch.stack(rows)], 0)
            lg, bl = hf_ref.forward(hfd, embeds=x.float())
            assert np.abs(dl[d, r] - lg[-1].numpy()).max() < 3e-4, (d, r)
            assert np.abs(da[d, r] - bl[0][-1].numpy()).max() < 3e-4
            checked += 1
    assert checked == (D - 1) * K


# ----------------------------------------------------------------------------- tree construction
def _check_tree(o, cfg):
    K, D, N = cfg.tree_topk, cfg.tree_depth, cfg.tree_nodes
    tok, par, dep, mask = (o.get(w) for w in (po.TREE_TOK, po.TREE_PARENT, po.TREE_DEPTH, po.TREE_MASK))
    pidx, sc = o.get(po.TREE_POOLIDX), o.get(po.TREE_SCORE)
    pscore, ppar, ptok = o.get(po.POOL_SCORE), o.get(po.POOL_PARENT), o.get(po.POOL_TOK)
    pool = cfg.pool
    nn = tok.size
    assert nn == min(N - 1, pool) + 1
    # masks == brute-force ancestor sets
    for i in range(nn):
        anc, v = set(), i
        while v != -1:
            anc.add(v)
            v = int(par[v])
        assert int(mask[i]) == sum(1 << a for a in anc)
        assert bin(int(mask[i])).count("1") == dep[i] + 1
        assert int(mask[i]) < (1 << (i + 1)) and (int(mask[i]) >> i) & 1
        if i:
            assert par[i] < i and dep[i] == dep[par[i]] + 1
            assert sc[i] <= sc[par[i]]
    # selection == stable sort of the pool by (-score, index); ancestor-closed by construction of that order
    order = sorted(range(1, pool + 1), key=lambda i: (-float(pscore[i]), i))
    chosen = sorted(order[: nn - 1])
    assert pidx[1:].tolist() == chosen
    sel = set(chosen) | {0}
    assert all(int(ppar[i]) in sel for i in chosen)
    if 0 < nn - 1 < pool:
        assert min(float(pscore[i]) for i in chosen) >= max(float(pscore[i]) for i in range(1, pool + 1) if i not in sel)
    # siblings carry distinct tokens (d2t is injective), so the accepted path is unique
    for p in range(nn):
        kids = [int(tok[c]) for c in range(1, nn) if par[c] == p]
        assert len(kids) == len(set(kids))
    # frontier of pass d = K best children of level d (score desc, pool index asc), all children of the previous frontier
    front = o.get(po.FRONTIER).reshape(D, K)
    assert front[0, 0] == 0
    if D > 1:
        assert front[1].tolist() == list(range(1, K + 1))
    for d in range(2, D):
        base = K + (d - 2) * K * K
        kids = list(range(base + 1, base + K * K + 1))
        best = sorted(kids, key=lambda i: (-float(pscore[i]), i))[:K]
        assert front[d].tolist() == best
        assert all(int(ppar[i]) in set(front[d - 1].tolist()) for i in best)
    # pool layout: children of frontier rank r of pass d
    for d in range(2, D + 1):
        base = K + (d - 2) * K * K
        for r in range(K):
            u = int(front[d - 1, r])
            for c in range(K):
                ci = base + r * K + c + 1
                assert ppar[ci] == u
                if c:
                    assert pscore[ci] <= pscore[ci - 1]
    return nn


@pytest.mark.parametrize("K,D,N", [(4, 3, 16), (1, 3, 4), (2, 4, 9), (3, 2, 64), (4, 1, 16), (5, 3, 1)])
def test_tree_invariants_and_losslessness(c1, K, D, N):
    """Section 2.1 / 'Metrics': strict acceptance leaves the output unchanged, so at temperature 0
    the emitted tokens equal plain greedy decoding, whatever tree was drafted."""
    tw, dw, ids = c1
    cfg = C1.replace(tree_topk=K, tree_depth=D, tree_nodes=N)
    o = _mk(cfg, tw, dw)
    first = o.prefill(ids)
    out = []
    for _ in range(12):
        n_before = o.n
        r = o.step()
        assert 1 <= len(r) <= D + 1                       # tau counts the bonus token
        assert o.n == n_before + len(r) and o.pending == len(r)
        nn = _check_tree(o, cfg)
        if K == 1:
            assert nn == min(N, D + 1)
            assert o.get(po.TREE_PARENT).tolist() == list(range(-1, nn - 1))   # a chain
        out += r.tolist()
    ref = _mk(cfg, tw, dw)
    assert ref.prefill(ids) == first
    assert ref.greedy(len(out)).tolist() == out


def test_output_invariant_to_draft_weights(c1):
    tw, dw, ids = c1
    dw2 = synth.make_draft_weights(C1, seed=123)
    outs = []
    for d in (dw, dw2):
        o = _mk(C1, tw, d)
        o.prefill(ids)
        acc = []
        while len(acc) < 16:
            acc += o.step().tolist()
        outs.append(acc[:16])
    assert outs[0] == outs[1]


def test_tree_forward_equals_per_path_sequential_bitwise(c1):
    """Tree attention == running each root-to-node path as an ordinary causal sequence."""
    tw, dw, ids = c1
    o = _mk(C1, tw, dw)
    o.prefill(ids)
    o.step()
    base_ids, n0 = o.ids, o.n
    o.step()
    tok, par = o.get(po.TREE_TOK), o.get(po.TREE_PARENT)
    dep, y = o.get(po.TREE_DEPTH), o.get(po.Y)
    taps = o.get(po.NODE_TAPS).reshape(tok.size, -1)
    for i in range(tok.size):
        chain, v = [], i
        while v != -1:
            chain.append(int(tok[v]))
            v = int(par[v])
        chain.reverse()                                   # root .. node i
        seq = np.concatenate([base_ids[:n0], np.array(chain, np.int32)])
        s = _mk(C1, tw, dw)
        nxt = s.prefill(seq)
        assert nxt == y[i]
        assert np.array_equal(s.taps(n0 + dep[i]), taps[i])          # bit-identical


def test_verify_tree_on_a_given_tree_equals_sequential_decoding(c1):
    """orc_verify_tree (step 5 on a caller-given tree): a hand-built tree whose branches are arbitrary token runs must
    give, at every node, the logits, hidden state and taps of an ordinary causal run over prompt + that node's path
    (a fresh prefill, bit for bit), also when the committed state has already moved past n_ctx."""
    tw, dw, ids = c1
    o = _mk(C1, tw, dw)
    o.prefill(ids)
    n0 = o.n
    root = int(o.ids[n0])
    #       0
    #     / | \
    #    1  2  3
    #    |     |\
    #    4     5 6
    #    |
    #    7
    tok = np.array([root, 11, 22, 33, 44, 55, 66, 77], np.int32)
    par = [-1, 0, 0, 0, 1, 3, 3, 4]
    dep = np.array([0, 1, 1, 1, 2, 2, 2, 3], np.int32)
    mask = np.zeros(8, np.uint64)
    for i, p_ in enumerate(par):
        mask[i] = np.uint64((int(mask[p_]) if p_ >= 0 else 0) | (1 << i))
    base = o.ids[:n0].copy()
    for advance in (False, True):
        if advance:
            o.step()                                      # commits past n0; the call below still verifies at n0
        lg, hid, taps = o.verify_tree(n0, tok, dep, mask)
        for i in range(8):
            chain, v = [], i
            while v != -1:
                chain.append(int(tok[v]))
                v = par[v]
            chain.reverse()
            s = _mk(C1, tw, dw)
            nxt = s.prefill(np.concatenate([base, np.array(chain, np.int32)]))
            assert nxt == int(np.argmax(lg[i]))
            assert np.array_equal(s.taps(n0 + dep[i]), taps[i])
    # rejects masks that are not ancestor-or-self sets below the node
    bad = mask.copy(); bad[2] = np.uint64(1 << 5 | 1 << 2)
    with pytest.raises(RuntimeError):
        o.verify_tree(n0, tok, dep, bad)


def _own_decisions(o):
    return o.get(po.POOL_TOK), o.get(po.FRONTIER), o.get(po.TREE_POOLIDX)


def test_follow_mode_reproduces_own_step_and_rejects_invalid_choices(c1):
    """orc_step_follow: (1) fed the oracle's own decisions it is the ordinary step, bit for bit, with no decision
    reported as different; (2) a followed top-k row with two children exchanged is adopted when their log-probabilities
    lie within eps and the later stages then run on the exchanged order; (3) with eps = 0 the same exchange, a child
    replaced by a token outside the top-k, and a pruned set that drops a better candidate are all refused."""
    tw, dw, ids = c1
    a, b = _mk(C1, tw, dw), _mk(C1, tw, dw)
    a.prefill(ids); b.prefill(ids)
    out_a = a.step()
    dec_a = _own_decisions(a)
    out_b, cnt = b.step_follow(*dec_a, eps=0.0, require=1e-2, band_lo=1e-2)
    K, D = C1.tree_topk, C1.tree_depth
    assert cnt["invalid"] == 0 and cnt["differs"] == 0 and cnt["required_differs"] == 0
    assert cnt["checked"] == K + (D - 1) * K * K + (D - 2) * K + 1   # every rank of every top-k row and frontier, the pruned set
    assert np.array_equal(out_a, out_b)
    for what in (po.TREE_TOK, po.TREE_MASK, po.TARGET_LOGITS, po.DRAFT_LOGITS, po.DRAFT_A, po.NODE_TAPS, po.POOL_SCORE):
        assert np.array_equal(a.get(what), b.get(what)), what
    # (2) exchange children 2 and 3 of the root: valid within a generous eps, and the step follows it
    c = _mk(C1, tw, dw); c.prefill(ids)
    pool, front, sel = (x.copy() for x in dec_a)
    pool[[2, 3]] = pool[[3, 2]]
    out_c, cnt_c = c.step_follow(pool, front, sel, eps=10.0, require=1e9, band_lo=1e9)
    assert cnt_c["invalid"] == 0 and cnt_c["differs"] >= 1
    assert np.array_equal(c.get(po.POOL_TOK)[:K + 1], pool[:K + 1])
    sc_a, sc_c = a.get(po.POOL_SCORE), c.get(po.POOL_SCORE)
    assert sc_c[2] == sc_a[3] and sc_c[3] == sc_a[2]                  # the oracle's own values, in the followed order
    # (3) eps = 0: refused, the oracle's own choice is used and the step equals the ordinary one
    for mutate in ("swap", "outsider", "prune"):
        d = _mk(C1, tw, dw); d.prefill(ids)
        pool, front, sel = (x.copy() for x in dec_a)
        if mutate == "swap":
            pool[[2, 3]] = pool[[3, 2]]
        elif mutate == "outsider":
            inside = set(pool[1:K + 1].tolist())
            pool[K] = next(int(t) for t in dw["d2t"].tolist() if int(t) not in inside)
        else:
            unsel = [i for i in range(1, C1.pool + 1) if i not in set(sel.tolist())]
            worst_unsel = min(unsel, key=lambda i: sc_a[i])
            leaf = max(sel.tolist())                                  # the highest pool index kept is a leaf
            if sc_a[worst_unsel] >= sc_a[leaf]:
                continue
            sel = np.sort(np.array([i for i in sel.tolist() if i != leaf] + [worst_unsel], np.int32))
        out_d, cnt_d = d.step_follow(pool, front, sel, eps=0.0, require=1e-2, band_lo=1e-2)
        assert cnt_d["invalid"] >= 1, mutate
        if mutate != "prune":
            assert np.array_equal(d.get(po.POOL_TOK)[:K + 1], dec_a[0][:K + 1]), mutate


def test_commit_equals_fresh_prefill(c1):
    tw, dw, ids = c1
    tws, dws, pi, pi2 = synth.make_structured(C1, 0.8, residual_scale=0.05)
    prompt = synth.structured_prompt(C1, dws["d2t"], 40).numpy()
    for (t, d, p) in ((tw, dw, ids), (tws, dws, prompt)):
        o = _mk(C1, t, d)
        o.prefill(p)
        for _ in range(5):
            o.step()
        f = _mk(C1, t, d)
        f.prefill(o.ids[: o.n])
        assert f.ids[o.n] == o.ids[o.n]
        for pos in range(o.n):
            assert np.array_equal(o.taps(pos), f.taps(pos))
            for l in range(C1.n_layers):
                ka, va = o.target_kv(l, pos); kb, vb = f.target_kv(l, pos)
                assert np.array_equal(ka, kb) and np.array_equal(va, vb)
        for pos in range(o.n - o.pending):
            ka, va = o.draft_kv(pos); kb, vb = f.draft_kv(pos)
            assert np.array_equal(ka, kb) and np.array_equal(va, vb)


def test_force_state_matches_stepping(c1):
    tw, dw, ids = c1
    a = _mk(C1, tw, dw)
    a.prefill(ids)
    for _ in range(3):
        a.step()
    b = _mk(C1, tw, dw)
    b.prefill(ids[:20])
    b.step()
    b.force_state(a.ids, a.n, a.pending)
    assert a.step().tolist() == b.step().tolist()
    for w in (po.TREE_TOK, po.TREE_PARENT, po.TREE_MASK, po.TARGET_LOGITS, po.DRAFT_LOGITS):
        assert np.array_equal(a.get(w), b.get(w))


# ----------------------------------------------------------------------------- acceptance > 0, closed form
@pytest.mark.parametrize("p_agree", [1.0, 0.8, 0.5])
def test_structured_weights_closed_form_counts(p_agree):
    """With zero W_o / W_down the target emits the pi-orbit of the root and the draft proposes pi2
    of every token, so count = 1 + (run of pi == pi2 along the orbit, capped at D)."""
    cfg = C1
    tw, dw, pi, pi2 = synth.make_structured(cfg, p_agree, residual_scale=0.0)
    prompt = synth.structured_prompt(cfg, dw["d2t"], 24, seed=int(p_agree * 10)).numpy()
    o = _mk(cfg, tw, dw)
    root = o.prefill(prompt)
    assert root == int(pi[int(prompt[-1])])
    seen_multi = False
    for _ in range(10):
        cur, run = root, 0
        while run < cfg.tree_depth and int(pi[cur]) == int(pi2[cur]):
            cur = int(pi[cur]); run += 1
        expect, cur = [], root
        for _ in range(run + 1):
            cur = int(pi[cur]); expect.append(cur)
        got = o.step().tolist()
        assert got == expect
        seen_multi |= len(got) > 1
        root = got[-1]
    assert seen_multi


def test_accept_walk_unit():
    #        0
    #      1   2
    #     3 4   5
    tok = [7, 10, 11, 20, 21, 30]
    par = [-1, 0, 0, 1, 1, 2]
    cnt, path, out = po.accept(tok, par, [10, 21, 0, 0, 99, 0])
    assert (cnt, path.tolist(), out.tolist()) == (3, [0, 1, 4], [10, 21, 99])
    cnt, path, out = po.accept(tok, par, [12, 0, 0, 0, 0, 0])
    assert (cnt, path.tolist(), out.tolist()) == (1, [0], [12])
    cnt, path, out = po.accept(tok, par, [11, 0, 30, 0, 0, 5])
    assert (cnt, path.tolist(), out.tolist()) == (3, [0, 2, 5], [11, 30, 5])


# ----------------------------------------------------------------------------- stochastic acceptance (T > 0)
_ST_TOK = [7, 1, 2, 5, 3, 4, 0]
_ST_PAR = [-1, 0, 0, 0, 1, 1, 2]     # root -> {1, 2, 3}; node 1 -> {4, 5}; node 2 -> {6}


def _st_logits(V=8, seed=0):
    return np.random.default_rng(seed).normal(0.0, 1.5, size=(len(_ST_TOK), V)).astype(np.float32)


def test_sampled_acceptance_is_lossless_on_a_small_tree():
    """Section 2.1: speculative sampling leaves the output distribution unchanged.  Over many draws of the uniforms, the
    first emitted token is distributed as softmax(z_root / T), and, given that the first token was accepted child c, the
    second as softmax(z_c / T), whatever the tree offers (chi-square against the exact probabilities)."""
    V, T, n_draws = 8, 0.8, 60000
    z = _st_logits(V)
    p = lambda row: np.exp((row - row.max()) / T) / np.exp((row - row.max()) / T).sum()
    rng = np.random.default_rng(1)
    first = np.zeros(V)
    second = {1: np.zeros(V), 2: np.zeros(V), 3: np.zeros(V)}
    counts = np.zeros(4, int)
    for _ in range(n_draws):
        u = rng.random(2 * len(_ST_TOK), dtype=np.float32)
        cnt, path, out, _, _ = po.accept_sampled(_ST_TOK, _ST_PAR, z, T, u)
        assert 1 <= cnt <= 3 and path[0] == 0
        counts[cnt] += 1
        first[out[0]] += 1
        if cnt >= 2:
            second[int(path[1])][out[1]] += 1

    def chi2_ok(obs, prob):
        n = obs.sum()
        exp_ = n * prob
        stat = ((obs - exp_) ** 2 / exp_).sum()
        return stat < 30.0          # 7 degrees of freedom: P(chi2 > 30) ~ 1e-4

    assert chi2_ok(first, p(z[0].astype(np.float64)))
    for c in (1, 2, 3):
        assert second[c].sum() > 500
        assert chi2_ok(second[c], p(z[c].astype(np.float64)))
    assert counts[2] > 0 and counts[3] > 0


def test_sampled_acceptance_probabilities_and_edges():
    """The probability child c is tested against is p(tok c) under the residual left by its rejected elder siblings;
    u = 0 accepts every first child, u -> 1 rejects all and draws the last id with mass left; T -> 0 is the greedy rule."""
    V, T = 8, 1.0
    z = _st_logits(V, seed=3)
    pr = np.exp(z[0].astype(np.float64) - z[0].max()); pr /= pr.sum()
    u = np.full(2 * len(_ST_TOK), 0.999999, np.float32)
    cnt, path, out, acc_p, (lo, hi) = po.accept_sampled(_ST_TOK, _ST_PAR, z, T, u)
    assert cnt == 1 and path.tolist() == [0]
    # children 1, 2, 3 carry tokens 1, 2, 5: each tested against the mass its elder siblings left
    assert abs(acc_p[1] - pr[1]) < 1e-6
    assert abs(acc_p[2] - pr[2] / (1 - pr[1])) < 1e-6
    assert abs(acc_p[3] - pr[5] / (1 - pr[1] - pr[2])) < 1e-6
    assert acc_p[4] == -1 and acc_p[6] == -1
    assert out[0] == 7 and hi == pytest.approx(1.0)            # ids 1, 2, 5 are gone; 7 is the last id with mass
    rest = pr.copy(); rest[[1, 2, 5]] = 0
    assert lo == pytest.approx(1 - rest[7] / rest.sum(), abs=1e-9)
    u0 = np.zeros(2 * len(_ST_TOK), np.float32)
    cnt, path, out, _, _ = po.accept_sampled(_ST_TOK, _ST_PAR, z, T, u0)
    assert path.tolist() == [0, 1, 4] and out.tolist()[:2] == [1, 3] and cnt == 3
    # inverse CDF: u picks the id whose interval contains it
    cdf = np.cumsum(pr)
    for ub in (0.0, 0.3, 0.77, 0.9999):
        u = np.full(2 * len(_ST_TOK), 0.999999, np.float32)
        one = np.array([7], np.int32)                                  # a tree of the root alone
        u1 = np.array([0.5, ub], np.float32)
        cnt, _, out, _, (lo, hi) = po.accept_sampled(one, [-1], z[:1], T, u1)
        assert cnt == 1 and out[0] == int(np.searchsorted(cdf, ub * cdf[-1], side="right"))
        assert lo <= ub < hi + 1e-12
    # T -> 0: equals the greedy walk for any uniforms that are not exactly 0
    for seed in range(5):
        zz = _st_logits(V, seed=10 + seed)
        y = zz.argmax(axis=1).astype(np.int32)
        cg, pg, og = po.accept(_ST_TOK, _ST_PAR, y)
        u = np.random.default_rng(seed).uniform(0.01, 0.99, 2 * len(_ST_TOK)).astype(np.float32)
        top2 = np.sort(zz, axis=1)[:, -2:]
        assert (top2[:, 1] - top2[:, 0]).min() > 5e-4          # far above the temperature: no near ties
        cs, ps, os_, _, _ = po.accept_sampled(_ST_TOK, _ST_PAR, zz, 1e-5, u)
        assert (cs, ps.tolist(), os_.tolist()) == (cg, pg.tolist(), og.tolist())


def test_sampled_step_wiring_and_greedy_limit(c1):
    """The sampled step applies the rule to the step's own tree and target logits, commits like the greedy step (cache ==
    fresh prefill of the committed tokens), and at T -> 0 emits the greedy tokens."""
    tw, dw, ids = c1
    N = C1.tree_nodes
    o = _mk(C1, tw, dw)
    g = _mk(C1, tw, dw)
    assert o.prefill(ids) == g.prefill(ids)
    rng = np.random.default_rng(5)
    for _ in range(4):
        u = rng.uniform(0.01, 0.99, 2 * N).astype(np.float32)
        assert o.step_sampled(1e-5, u).tolist() == g.step().tolist()
    o = _mk(C1, tw, dw)
    o.prefill(ids)
    emitted = []
    for _ in range(6):
        u = rng.random(2 * N, dtype=np.float32)
        n0 = o.n
        out = o.step_sampled(1.0, u)
        nn = o.get(po.TREE_TOK).size
        logits = o.get(po.TARGET_LOGITS).reshape(nn, C1.vocab)
        cnt, path, ref, acc_p, iv = po.accept_sampled(o.get(po.TREE_TOK), o.get(po.TREE_PARENT), logits, 1.0, u, n_max=N)
        assert out.tolist() == ref.tolist() and o.get(po.PATH).tolist() == path.tolist()
        assert np.array_equal(o.get(po.ACC_P), acc_p) and o.get(po.BONUS_INTERVAL).tolist() == list(iv)
        assert o.n == n0 + len(out) and o.pending == len(out)
        emitted += out.tolist()
    fresh = _mk(C1, tw, dw)
    fresh.prefill(o.ids[: o.n])
    for pos in (0, o.n // 2, o.n - 1):
        for layer in range(C1.n_layers):
            k1, v1 = o.target_kv(layer, pos); k2, v2 = fresh.target_kv(layer, pos)
            assert np.abs(k1 - k2).max() < TOL and np.abs(v1 - v2).max() < TOL


def test_rerank_unit_ties_and_closure():
    # pool: 1,2 children of root; 3,4 children of 1; 5,6 children of 2; log-prob 0 children tie with parents
    score = np.array([0, -0.5, -1.0, -0.5, -2.0, -1.0, -1.0], np.float32)
    parent = np.array([-1, 0, 0, 1, 1, 2, 2], np.int32)
    tok = np.arange(100, 107, dtype=np.int32)
    depth = np.array([0, 1, 1, 2, 2, 2, 2], np.int32)
    r = po.rerank(score, parent, tok, depth, 5, 100)
    assert r["poolidx"].tolist() == [0, 1, 2, 3, 5]      # ties resolved toward the lower index (parent first)
    assert r["parent"].tolist() == [-1, 0, 0, 1, 2]
    assert r["mask"].tolist() == [1, 3, 5, 11, 21]
    assert r["cut_margin"] == 0.0
    r = po.rerank(score, parent, tok, depth, 64, 100)
    assert r["n"] == 7 and math.isinf(r["cut_margin"])


def test_golden_c1_trajectory_is_reproduced_and_lossless():
    """tests/golden/c1_oracle_trajectory.json (written by tests/golden/make_golden.py from the oracle alone)."""
    import json
    import os
    import sys
    here = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
    sys.path.insert(0, here)
    import make_golden
    stored = json.load(open(os.path.join(here, "c1_oracle_trajectory.json")))
    assert stored["tokens"] == stored["greedy"][: len(stored["tokens"])]          # Section 2.1: lossless at temperature 0
    assert all(1 <= c <= C1.tree_depth + 1 for c in stored["counts"]) and sum(stored["counts"]) == len(stored["tokens"]) - 1
    assert sum(stored["sampled_T1"]["counts"]) == len(stored["sampled_T1"]["tokens"]) - 1
    assert make_golden.trajectory() == stored


# ----------------------------------------------------------------------------- training-time-test attention
def _ttt_case(T, H, G, hd, J, seed):
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(T, H, hd, generator=g)
    k0, v0 = torch.randn(T, G, hd, generator=g), torch.randn(T, G, hd, generator=g)
    kd, vd = torch.randn(J, T, G, hd, generator=g), torch.randn(J, T, G, hd, generator=g)
    return q, k0, v0, kd, vd


def test_ttt_attention_oracle_against_masked_library_attention():
    """The oracle's training-time-test attention against torch's scaled_dot_product_attention over the concatenated key
    set [native step ; simulated step 1 ; ... ; simulated step J] with the mask of Section 3.2's figure built by brute
    force: lower-triangular on the native block, diagonal on every simulated block.  With J = 0 it must be plain causal
    attention; a dropped diagonal entry, a shifted causal boundary or a wrong KV-head group fails."""
    for (T, H, G, hd, J) in [(9, 4, 2, 16, 0), (7, 4, 2, 16, 1), (12, 6, 3, 8, 3), (5, 2, 2, 32, 2)]:
        q, k0, v0, kd, vd = _ttt_case(T, H, G, hd, J, 100 + T + J)
        out, lse = po.ttt_attention(q.numpy(), k0.numpy(), v0.numpy(), kd.numpy(), vd.numpy())
        keys = torch.cat([k0] + [kd[s] for s in range(J)], 0)            # [(1+J) T][G][hd]
        vals = torch.cat([v0] + [vd[s] for s in range(J)], 0)
        mask = torch.zeros(T, (1 + J) * T, dtype=torch.bool)
        for i in range(T):
            mask[i, : i + 1] = True
            for s in range(J):
                mask[i, (1 + s) * T + i] = True
        grp = H // G
        kk = keys.permute(1, 0, 2).repeat_interleave(grp, 0).double()   # [H][(1+J) T][hd]
        vv = vals.permute(1, 0, 2).repeat_interleave(grp, 0).double()
        ref = torch.nn.functional.scaled_dot_product_attention(q.permute(1, 0, 2).double(), kk, vv, attn_mask=mask)
        assert np.abs(out - ref.permute(1, 0, 2).numpy()).max() < 1e-9, (T, J)
        if J == 0:
            causal = torch.nn.functional.scaled_dot_product_attention(q.permute(1, 0, 2).double(), kk, vv, is_causal=True)
            assert np.abs(out - causal.permute(1, 0, 2).numpy()).max() < 1e-9
        # the log-normaliser against a direct log-sum-exp of the allowed scores
        sc = torch.einsum("thd,hkd->thk", q.double(), kk) / hd ** 0.5
        ref_lse = torch.logsumexp(sc.masked_fill(~mask[:, None, :], float("-inf")), -1)
        assert np.abs(lse - ref_lse.numpy()).max() < 1e-9


def test_ttt_attention_oracle_closed_form_single_position():
    """T = 1: the softmax runs over the native key and the J diagonal entries only; with equal keys the output is the
    plain mean of the 1 + J values."""
    q = np.ones((1, 1, 4)); k0 = np.ones((1, 1, 4)); v0 = np.full((1, 1, 4), 3.0)
    kd = np.ones((2, 1, 1, 4)); vd = np.stack([np.full((1, 1, 4), 6.0), np.full((1, 1, 4), 0.0)])
    out, lse = po.ttt_attention(q, k0, v0, kd, vd)
    assert np.allclose(out, 3.0) and np.allclose(lse, 4 / 2.0 + np.log(3.0))
