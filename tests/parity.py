"""Step-by-step comparison of the CUDA path with the CPU oracle on identical seeded inputs.

Rule: integer results (tree structure, argmax, accepted ids, counts) must be bit-exact wherever every
decision that led to them had an oracle margin above MARGIN; floating-point results (logits, hidden
states, taps) must agree within `tol` max-abs.  One flipped low-margin decision changes all later
state, so after every step the oracle is put into the CUDA path's committed state (resync)."""
import numpy as np
import torch

import pyoracle as po
from paper_2503_01840_b200 import binding as sb
from paper_2503_01840_b200 import synth

MARGIN = 1e-2          # the stated rule: an integer decision whose oracle margin exceeds this must be bit-exact


def decision_margin(tol):
    """Oracle margin above which an integer decision of the CUDA path is REQUIRED to be bit-exact.  The stated rule
    (1e-2) presumes float errors well below it.  The bf16 bound on a logit is 2e-2, and two competing logits may each be
    off by it, so for bf16 models the requirement starts at twice the tolerance; decisions whose margin lies in the band
    (1e-2, 2 tol] are still compared and counted (Stats.band_total / band_diff) so that a run reports how many of them
    actually differed."""
    return MARGIN if tol < 1e-3 else max(MARGIN, 2.0 * tol)


def to_dev(w, dev="cuda"):
    if isinstance(w, dict):
        return {k: to_dev(v, dev) for k, v in w.items()}
    if isinstance(w, list):
        return [to_dev(v, dev) for v in w]
    return w.to(dev).contiguous()


def to_cpu(w):
    return to_dev(w, "cpu")


class Stats:
    """What a trajectory actually compared.  Every test asserts minimums on these, so that a run which diverged early
    and compared nothing cannot pass."""
    COUNTERS = ("steps", "tokens", "resyncs",
                "passes",            # draft passes whose logits and features were compared element by element
                "decisions",         # draft-side integer decisions checked (top-k rows, frontiers, pruned sets): each valid within 2 tol
                "decisions_forced",  # ... of which the oracle's own margin required bit-equality (and it held)
                "decisions_differ",  # ... of which the CUDA path resolved a near-tie differently (valid, followed)
                "exact_tree",        # steps in which every draft decision was required to be bit-exact
                "same_tree",         # steps whose tree equals the one the oracle builds on its own
                "verify_compared",   # steps whose verify logits / hidden states / taps were compared element by element
                "argmax_forced",     # verify nodes (and first tokens) whose argmax had to match
                "accept_checked",    # steps whose accepted path and ids equal the oracle's walk over the same tree and argmax
                "exact_out",         # steps whose emitted ids had to equal the oracle's
                "band_total", "band_diff")   # decisions with oracle margin in (1e-2, threshold]: seen / differed

    def __init__(self):
        for n in self.COUNTERS:
            setattr(self, n, 0)
        self.max_err = {}

    def err(self, name, a, b):
        e = float(np.abs(np.asarray(a, np.float64) - np.asarray(b, np.float64)).max()) if np.size(a) else 0.0
        self.max_err[name] = max(self.max_err.get(name, 0.0), e)
        return e

    def decide(self, margin, threshold, same, what):
        """One integer decision with oracle margin `margin`: required to match above `threshold`, counted in the band
        between the stated 1e-2 and the threshold.  Returns True when it was required."""
        if margin > threshold:
            assert same, f"{what} differs although its oracle margin {margin:.4g} exceeds {threshold:.4g}"
            return True
        if margin > MARGIN:
            self.band_total += 1
            self.band_diff += int(not same)
        return False

    def __repr__(self):
        errs = ", ".join(f"{k}={v:.2e}" for k, v in sorted(self.max_err.items()))
        return " ".join(f"{n}={getattr(self, n)}" for n in self.COUNTERS) + " | " + errs


def step_and_compare(dec, orc, seq, cfg, tol, st, gpu_out, check_floats=True, tap_tol=None, sampled=None):
    """The CUDA path has just executed a step; `orc` is in the same state before it.  The oracle now runs the step
    FOLLOWING the CUDA path's integer decisions (the K children of every draft row, every frontier, the pruned set):
    each must be valid on the oracle's own values within 2 tol (order non-increasing, nothing better left out), and
    bit-equal to the oracle's own choice wherever that choice has margin above the threshold.  Both sides then hold
    the same tree, so every float of the step is compared: draft logits and features of all D passes, tree scores,
    verify logits, hidden states, taps; each verify argmax is gated on its own margin; the acceptance walk must equal
    the oracle's walk over the same tree and argmax.  Returns (oracle's emitted ids, True if the emitted ids were
    required to be identical).  sampled = (temperature, u) for a step with stochastic acceptance."""
    K, D, N, Vd, k, V = cfg.tree_topk, cfg.tree_depth, cfg.tree_nodes, cfg.draft_vocab, cfg.hidden, cfg.vocab
    tap_tol = tol if tap_tol is None else tap_tol
    thr = decision_margin(tol)
    g_pool = dec.debug(sb.DBG_POOL_TOK, seq)
    g_front = dec.debug(sb.DBG_FRONTIER, seq)
    g_sel = dec.debug(sb.DBG_TREE_POOLIDX, seq)
    o_out, cnt = orc.step_follow(g_pool, g_front, g_sel, eps=2.0 * tol, require=thr, band_lo=MARGIN,
                                 temperature=sampled[0] if sampled else 0.0, u=sampled[1] if sampled else None)
    assert cnt["invalid"] == 0, f"{cnt['invalid']} draft decision(s) of the CUDA path are not valid within {2 * tol} on the oracle's values: {cnt}"
    assert cnt["required_differs"] == 0, f"a draft decision differs although its oracle margin exceeds {thr}: {cnt}"
    st.decisions += cnt["checked"]
    st.decisions_forced += cnt["required"]
    st.decisions_differ += cnt["differs"]
    st.band_total += cnt["band_total"]
    st.band_diff += cnt["band_differs"]
    st.same_tree += int(cnt["differs"] == 0)
    st.exact_tree += int(cnt["required"] == cnt["checked"])
    # ---- draft passes: all of them
    assert np.array_equal(g_pool, orc.get(po.POOL_TOK)), "candidate pools differ after following"
    if check_floats:
        g_dl = dec.debug(sb.DBG_DRAFT_LOGITS, seq).reshape(D, K, Vd)
        g_da = dec.debug(sb.DBG_DRAFT_A, seq).reshape(D, K, k)
        o_dl = orc.get(po.DRAFT_LOGITS).reshape(D, K, Vd)
        o_da = orc.get(po.DRAFT_A).reshape(D, K, k)
        for d in range(D):
            rows = 1 if d == 0 else K
            assert st.err("draft_logits", g_dl[d, :rows], o_dl[d, :rows]) <= tol, (d, st.max_err)
            assert st.err("draft_a", g_da[d, :rows], o_da[d, :rows]) <= tol, (d, st.max_err)
            st.passes += 1
    assert st.err("pool_score", dec.debug(sb.DBG_POOL_SCORE, seq)[1:], orc.get(po.POOL_SCORE)[1:]) <= D * tol
    # ---- the tree: identical integers, valid structure
    ints = {n: (dec.debug(g, seq), orc.get(o)) for n, g, o in (
        ("tok", sb.DBG_TREE_TOK, po.TREE_TOK), ("parent", sb.DBG_TREE_PARENT, po.TREE_PARENT),
        ("depth", sb.DBG_TREE_DEPTH, po.TREE_DEPTH), ("mask", sb.DBG_TREE_MASK, po.TREE_MASK),
        ("poolidx", sb.DBG_TREE_POOLIDX, po.TREE_POOLIDX))}
    for n, (a, b) in ints.items():
        assert np.array_equal(a, b), f"tree {n} differs on identical decisions\n{a}\n{b}"
    g_tok, g_par, g_dep, g_mask = ints["tok"][0], ints["parent"][0], ints["depth"][0], ints["mask"][0]
    nn = g_tok.size
    assert 1 <= nn <= N
    for i in range(nn):
        if i == 0:
            assert g_par[0] == -1 and g_dep[0] == 0 and int(g_mask[0]) == 1
        else:
            p = int(g_par[i])
            assert 0 <= p < i and g_dep[i] == g_dep[p] + 1 and int(g_mask[i]) == (int(g_mask[p]) | (1 << i))
    assert st.err("tree_score", dec.debug(sb.DBG_TREE_SCORE, seq), orc.get(po.TREE_SCORE)) <= D * tol
    # ---- verify pass
    if check_floats:
        assert st.err("target_logits", dec.debug(sb.DBG_TARGET_LOGITS, seq), orc.get(po.TARGET_LOGITS)) <= tol, st.max_err
        assert st.err("node_hidden", dec.debug(sb.DBG_NODE_HIDDEN, seq), orc.get(po.NODE_HIDDEN)) <= tol, st.max_err
        assert st.err("node_taps", dec.debug(sb.DBG_NODE_TAPS, seq), orc.get(po.NODE_TAPS)) <= tap_tol, st.max_err
        st.verify_compared += 1
    gy, oy, ym = dec.debug(sb.DBG_Y, seq), orc.get(po.Y), orc.get(po.Y_MARGIN)
    for i in range(nn):
        if st.decide(float(ym[i]), thr, gy[i] == oy[i], f"argmax of verify node {i}"):
            st.argmax_forced += 1
    if sampled is not None:
        return o_out, check_sampled_decisions(dec, orc, seq, cfg, tol, gpu_out, *sampled)
    # the acceptance walk is integer work: on the CUDA path's own argmax it must equal the oracle's walk
    _, w_path, w_out = po.accept(g_tok, g_par, gy)
    g_path = dec.debug(sb.DBG_PATH, seq)
    assert np.array_equal(g_path, w_path) and np.array_equal(np.asarray(gpu_out), w_out), (g_path, w_path, gpu_out, w_out)
    st.accept_checked += 1
    o_path = orc.get(po.PATH)
    exact_out = bool((ym[o_path] > thr).all())
    if exact_out:
        assert np.array_equal(g_path, o_path), (g_path, o_path)
    return o_out, exact_out


def check_sampled_decisions(dec, orc, seq, cfg, tol, gpu_out, temperature, u, own_inputs=False):
    """Stochastic acceptance on the same tree: every decision of the CUDA path (accept / reject of each tried child, the
    drawn token) must be one the oracle's probabilities allow within the slack that the logit tolerance implies (a logit
    error of tol moves a probability ratio by exp(2 tol / T) - 1), and equal to the oracle's decision wherever the
    oracle's own margin exceeds that slack.  Returns True when the outputs had to be (and were) identical."""
    V, N = cfg.vocab, cfg.tree_nodes
    if own_inputs:
        # the trees differ (a low-margin draft decision): the acceptance kernel is still checked, as a function of its
        # own inputs (the CUDA path's tree and verify logits), with the slack of the summation order only
        tok, par = dec.debug(sb.DBG_TREE_TOK, seq), dec.debug(sb.DBG_TREE_PARENT, seq)
        nn = tok.size
        z = dec.debug(sb.DBG_TARGET_LOGITS, seq).reshape(nn, V).astype(np.float64)
        tol = 1e-5
    else:
        tok, par = orc.get(po.TREE_TOK), orc.get(po.TREE_PARENT)
        nn = tok.size
        z = orc.get(po.TARGET_LOGITS).reshape(nn, V).astype(np.float64)
    g_path = dec.debug(sb.DBG_PATH, seq)
    assert len(gpu_out) == len(g_path) and g_path[0] == 0
    delta = float(np.expm1(2.0 * tol / temperature)) + 1e-5
    cur, forced = 0, True
    for j in range(len(g_path)):
        e = np.exp((z[cur] - z[cur].max()) / temperature)
        mass = e.sum()
        nxt = int(g_path[j + 1]) if j + 1 < len(g_path) else -1
        accepted = False
        for c in range(cur + 1, nn):
            if par[c] != cur:
                continue
            pc = e[tok[c]] / mass
            uc = float(u[c])
            if abs(uc - pc) <= delta * pc + 1e-7:
                forced = False
            if c == nxt:
                assert uc < pc * (1 + delta) + 1e-7, f"node {c} accepted with u={uc} against p={pc}"
                assert gpu_out[j] == tok[c]
                accepted = True
                break
            assert uc >= pc * (1 - delta) - 1e-7, f"node {c} rejected with u={uc} against p={pc}"
            mass -= e[tok[c]]
            e[tok[c]] = 0.0
        if accepted:
            cur = nxt
            continue
        assert nxt == -1, "the path continues through a node that is not a child of the current one"
        bonus = int(gpu_out[j])
        assert 0 <= bonus < V and e[bonus] > 0.0, "the drawn token has no mass in the residual"
        cdf = np.cumsum(e) / e.sum()
        lo, hi = (cdf[bonus - 1] if bonus else 0.0), cdf[bonus]
        ub = float(u[N + cur])
        assert lo - delta - 1e-6 <= ub <= hi + delta + 1e-6, f"token {bonus} drawn with u={ub} outside [{lo}, {hi})"
        if min(ub - lo, hi - ub) <= delta + 1e-6:
            forced = False
    if own_inputs:
        if forced:      # the oracle's rule on the same inputs must give the same walk and token
            cnt, o_path, o_out, _, _ = po.accept_sampled(tok, par, z.astype(np.float32), temperature, u, n_max=N)
            assert np.array_equal(g_path, o_path) and np.array_equal(np.asarray(gpu_out), o_out), (g_path, o_path, gpu_out, o_out)
        return False
    if forced:
        o_path = orc.get(po.PATH)
        assert np.array_equal(g_path, o_path), (g_path, o_path)
    return forced


def run_trajectory(cfg, tw, dw, prompts, n_steps, tol, flags=0, max_ctx=None, check_floats=True, tap_tol=None,
                   page_shuffle_seed=0, num_pages=None, tune=(), sampling=None, greedy_check=True):
    """tw/dw: CPU weight dicts; tune: (knob, value, value to restore) triples applied to the decoder (process-wide knobs).
    sampling = (temperature, seed): every step uses the stochastic acceptance rule with uniforms drawn from that seed.
    Returns Stats; raises AssertionError on a parity violation."""
    B = len(prompts)
    reserve = n_steps * (cfg.tree_depth + 1) + 8
    if max_ctx is None:
        max_ctx = max(len(p) for p in prompts) + reserve + 2 * max(cfg.tree_nodes, (cfg.tree_depth - 1) * cfg.tree_topk) + 8
    if check_floats:
        flags |= sb.FLAG_CAPTURE
    dec = sb.SpecDecoder(cfg, to_dev(tw), to_dev(dw), batch=B, max_ctx=max_ctx, flags=flags,
                         page_shuffle_seed=page_shuffle_seed, num_pages=num_pages)
    for knob, value, _ in tune:
        dec.tune(knob, value)
    try:
        return _run_trajectory(dec, cfg, tw, dw, prompts, n_steps, tol, max_ctx, reserve, check_floats, tap_tol, sampling,
                               greedy_check)
    finally:
        for knob, _, restore in tune:
            dec.tune(knob, restore)
        dec.close()


def _run_trajectory(dec, cfg, tw, dw, prompts, n_steps, tol, max_ctx, reserve, check_floats, tap_tol, sampling=None,
                    greedy_check=True):
    B = len(prompts)
    rng = np.random.default_rng(sampling[1]) if sampling else None
    st = Stats()
    first = dec.prefill([np.asarray(p) for p in prompts], reserve)
    orcs = []
    for b in range(B):
        o = po.Oracle(cfg, tw, dw, max_ctx)
        f = o.prefill(np.asarray(prompts[b]))
        # the first token is an argmax like any other: it has to match where the oracle's top-1 margin allows
        n0 = len(prompts[b])
        lg, _, _ = o.verify_tree(n0 - 1, prompts[b][-1:], [0], [1])
        top2 = np.partition(lg[0], -2)[-2:]
        st.err("prefill_logit_top1", lg[0, f], top2[1])
        if st.decide(float(top2[1] - top2[0]), decision_margin(tol), f == first[b], f"first token of sequence {b} ({f} vs {first[b]})"):
            st.argmax_forced += 1
        if f != first[b]:
            st.resyncs += 1
            o.force_state(np.concatenate([prompts[b], [first[b]]]).astype(np.int32), n0, 1)
        orcs.append(o)
    emitted = [[] for _ in range(B)]
    for step in range(n_steps):
        u = rng.random((B, 2 * cfg.tree_nodes), dtype=np.float32) if sampling else None
        outs = dec.step_sampled(sampling[0], u) if sampling else dec.step()
        for b in range(B):
            o = orcs[b]
            ids_before, n_before = o.ids, o.n
            g_out = outs[b]
            assert 1 <= len(g_out) <= cfg.tree_depth + 1
            o_out, exact = step_and_compare(dec, o, b, cfg, tol, st, g_out, check_floats, tap_tol,
                                            sampled=(sampling[0], u[b]) if sampling else None)
            if exact:
                assert np.array_equal(g_out, o_out), (g_out, o_out)
                st.exact_out += 1
            emitted[b] += g_out.tolist()
            if not np.array_equal(g_out, o_out):
                st.resyncs += 1
                new_ids = np.concatenate([ids_before, g_out]).astype(np.int32)
                o.force_state(new_ids, n_before + len(g_out), len(g_out))
            st.tokens += len(g_out)
        st.steps += 1
        assert np.array_equal(dec.lengths(), [o.n for o in orcs])
    # committed caches: K/V of sampled positions in the first and last target layer and in the draft layer against the
    # oracle (which is in the CUDA path's committed state after every step)
    for b in sorted(set([0, B // 2, B - 1])):
        o = orcs[b]
        n = o.n
        for pos in sorted(set([0, n // 2, n - 2, n - 1])):
            for layer in sorted(set([0, cfg.n_layers - 1])):
                gk, gv = dec.read_kv(b, layer, pos)
                ok, ov = o.target_kv(layer, pos)
                assert st.err("kv_target", gk, ok) <= 4 * tol and st.err("kv_target", gv, ov) <= 4 * tol, (b, pos, layer)
            if pos < n - o.pending:
                gk, gv = dec.read_kv(b, -1, pos)
                ok, ov = o.draft_kv(pos)
                assert st.err("kv_draft", gk, ok) <= 4 * tol and st.err("kv_draft", gv, ov) <= 4 * tol, (b, pos)
    # losslessness against plain greedy decoding of the oracle, up to the first low-margin token
    for b in range(B if (greedy_check and not sampling) else 0):
        g = po.Oracle(cfg, tw, dw, max_ctx)
        g.prefill(np.asarray(prompts[b]))
        ref, mg = g.greedy_margins(len(emitted[b]))
        for i, (a, r) in enumerate(zip(emitted[b], ref)):
            if a != r:
                assert mg[i] <= decision_margin(tol), f"sequence {b}: token {i} differs from greedy decoding with margin {mg[i]}"
                break
    return st, emitted
