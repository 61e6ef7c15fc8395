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
                "topk_forced",       # top-k rows (own margin above the threshold) required to match, order included
                "topk_set_forced",   # rows whose K-th vs (K+1)-th gap alone is above the threshold: the SET had to match
                "frontier_forced",   # frontier selections required to match
                "exact_tree",        # steps whose whole tree (tokens, parents, depths, masks, pool indices) had to match
                "same_tree",         # steps whose tree did match the oracle's
                "verify_compared",   # steps whose verify logits / hidden states / taps were compared element by element
                "accept_checked",    # steps whose accepted path and ids equal the oracle's walk over the same tree and argmax
                "argmax_forced",     # verify nodes whose argmax had to match
                "exact_out",         # steps whose accepted path and emitted ids had to match
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


def compare_step(dec, orc, seq, cfg, tol, st, gpu_out, check_floats=True, tap_tol=None, sampled=None, n_ctx=None):
    """`orc` has just executed the same step from the same state.  Every integer decision is gated on its OWN oracle
    margin: a top-k row, a frontier selection, the final cut of the candidate pool, each verify node's argmax and the
    accepted path.  Returns True if the outputs were required to be (and were) identical.
    sampled = (temperature, u) for a step with stochastic acceptance.  n_ctx = committed length before the step: when
    the trees differ (a low-margin draft decision), the oracle runs its verify pass on the CUDA path's tree over that
    prefix, so that the verify floats, the argmax and the acceptance walk are compared in every step."""
    K, D, N, Vd, k, V = cfg.tree_topk, cfg.tree_depth, cfg.tree_nodes, cfg.draft_vocab, cfg.hidden, cfg.vocab
    tap_tol = tol if tap_tol is None else tap_tol
    thr = decision_margin(tol)
    o_front = orc.get(po.FRONTIER).reshape(D, K)
    g_front = dec.debug(sb.DBG_FRONTIER, seq).reshape(D, K)
    tk_m = orc.get(po.TOPK_MARGIN).reshape(D, K)
    fr_m = orc.get(po.FRONTIER_MARGIN)
    rr_m = float(orc.get(po.RERANK_MARGIN)[0])
    capture = check_floats
    o_dl = orc.get(po.DRAFT_LOGITS).reshape(D, K, Vd)
    if capture:
        g_dl = dec.debug(sb.DBG_DRAFT_LOGITS, seq).reshape(D, K, Vd)
        g_da = dec.debug(sb.DBG_DRAFT_A, seq).reshape(D, K, k)
        o_da = orc.get(po.DRAFT_A).reshape(D, K, k)
    o_ptok, g_ptok = orc.get(po.POOL_TOK), dec.debug(sb.DBG_POOL_TOK, seq)
    pool_same = True                 # every candidate drafted so far is the same on both sides
    front_required = True            # the frontier of the next pass has to match (all decisions behind it were required)
    for d in range(D):
        rows = 1 if d == 0 else K
        # same nodes in the same order, carrying the same tokens (a swapped near-tie inside one top-k
        # row keeps the pool indices but exchanges the tokens)
        same_front = d == 0 or (np.array_equal(o_front[d], g_front[d]) and
                                np.array_equal(o_ptok[o_front[d]], g_ptok[g_front[d]]))
        if d > 0 and front_required:
            assert same_front, f"frontier of pass {d} differs although every decision behind it had margin > {thr}: {o_front[d]} vs {g_front[d]}"
            st.frontier_forced += 1
        if not same_front:
            pool_same = False
            break
        if capture:
            assert st.err("draft_logits", g_dl[d, :rows], o_dl[d, :rows]) <= tol, (d, st.max_err)
            assert st.err("draft_a", g_da[d, :rows], o_da[d, :rows]) <= tol, (d, st.max_err)
            st.passes += 1
        # the K children of every row of this pass: pool entries base + r K + 1 .. base + r K + K
        base = 0 if d == 0 else K + (d - 1) * K * K
        rows_same = True
        for r in range(rows):
            lo = base + r * K + 1
            o_t, g_t = o_ptok[lo:lo + K], g_ptok[lo:lo + K]
            same = bool(np.array_equal(o_t, g_t))
            if st.decide(float(tk_m[d, r]), thr, same, f"top-{K} of pass {d} row {r}"):
                st.topk_forced += 1
            else:
                # membership alone: the K-th against the (K+1)-th log-probability of the oracle's row
                z = o_dl[d, r].astype(np.float64)
                top = np.sort(z)[::-1][:K + 1]
                set_margin = float(top[K - 1] - top[K]) if Vd > K else np.inf
                same_set = set(o_t.tolist()) == set(g_t.tolist())
                if st.decide(set_margin, thr, same_set, f"top-{K} set of pass {d} row {r}"):
                    st.topk_set_forced += 1
            rows_same = rows_same and same
        pool_same = pool_same and rows_same
        # the next frontier: level 1 is taken whole, later levels are the K best children of the level
        if d + 1 < D:
            front_required = rows_same and (d == 0 or float(fr_m[d]) > thr)
            if rows_same and d >= 1 and MARGIN < float(fr_m[d]) <= thr:
                st.band_total += 1
                st.band_diff += int(not (np.array_equal(o_front[d + 1], g_front[d + 1])))
    ints = {n: (dec.debug(g, seq), orc.get(o)) for n, g, o in (
        ("tok", sb.DBG_TREE_TOK, po.TREE_TOK), ("parent", sb.DBG_TREE_PARENT, po.TREE_PARENT),
        ("depth", sb.DBG_TREE_DEPTH, po.TREE_DEPTH), ("mask", sb.DBG_TREE_MASK, po.TREE_MASK),
        ("poolidx", sb.DBG_TREE_POOLIDX, po.TREE_POOLIDX))}
    same_tree = all(np.array_equal(a, b) for a, b in ints.values())
    st.same_tree += int(same_tree)
    # the cut of the pool: required when both sides ranked the same candidates and the oracle's cut has margin
    if pool_same and st.decide(rr_m, thr, same_tree, "pruned tree"):
        for n, (a, b) in ints.items():
            assert np.array_equal(a, b), f"tree {n} differs although the pool matches and the cut margin > {thr}\n{a}\n{b}"
        st.exact_tree += 1
    # GPU tree must be a valid tree whatever the margins
    g_par, g_dep, g_mask = ints["parent"][0], ints["depth"][0], ints["mask"][0]
    for i in range(g_par.size):
        if i == 0:
            assert g_par[0] == -1 and g_dep[0] == 0 and int(g_mask[0]) == 1
        else:
            p = int(g_par[i])
            assert 0 <= p < i and g_dep[i] == g_dep[p] + 1 and int(g_mask[i]) == (int(g_mask[p]) | (1 << i))
    exact_out = False
    if sampled is not None and not same_tree and check_floats:
        check_sampled_decisions(dec, orc, seq, cfg, tol, gpu_out, *sampled, own_inputs=True)
        st.max_err["sampled_own_inputs_checks"] = st.max_err.get("sampled_own_inputs_checks", 0.0) + 1
    g_tok, g_par = ints["tok"][0], ints["parent"][0]
    nn = g_tok.size
    gy = dec.debug(sb.DBG_Y, seq)
    if same_tree:
        assert st.err("tree_score", dec.debug(sb.DBG_TREE_SCORE, seq), orc.get(po.TREE_SCORE)) <= tol
        o_logits, o_hidden, o_taps = orc.get(po.TARGET_LOGITS), orc.get(po.NODE_HIDDEN), orc.get(po.NODE_TAPS)
        oy, ym = orc.get(po.Y), orc.get(po.Y_MARGIN)
    elif check_floats and n_ctx is not None:
        # the oracle's verify pass on the CUDA path's (valid) tree
        o_logits, o_hidden, o_taps = orc.verify_tree(n_ctx, g_tok, g_dep, g_mask)
        top2 = np.partition(o_logits, -2, axis=1)[:, -2:]
        oy, ym = np.argmax(o_logits, axis=1), top2[:, 1] - top2[:, 0]
    else:
        return False
    if check_floats:
        assert st.err("target_logits", dec.debug(sb.DBG_TARGET_LOGITS, seq), np.ravel(o_logits)) <= tol, st.max_err
        assert st.err("node_hidden", dec.debug(sb.DBG_NODE_HIDDEN, seq), np.ravel(o_hidden)) <= tol, st.max_err
        assert st.err("node_taps", dec.debug(sb.DBG_NODE_TAPS, seq), np.ravel(o_taps)) <= tap_tol, st.max_err
        st.verify_compared += 1
    for i in range(nn):
        if st.decide(float(ym[i]), thr, gy[i] == oy[i], f"argmax of verify node {i}"):
            st.argmax_forced += 1
    if sampled is not None:
        return check_sampled_decisions(dec, orc, seq, cfg, tol, gpu_out, *sampled) if same_tree else False
    # the acceptance walk is integer work: on the CUDA path's own tree and argmax it must equal the oracle's walk
    cnt, w_path, w_out = po.accept(g_tok, g_par, gy)
    g_path = dec.debug(sb.DBG_PATH, seq)
    assert np.array_equal(g_path, w_path) and np.array_equal(np.asarray(gpu_out), w_out), (g_path, w_path, gpu_out, w_out)
    st.accept_checked += 1
    if same_tree:
        o_path = orc.get(po.PATH)
        if (ym[o_path] > thr).all():
            assert np.array_equal(g_path, o_path), (g_path, o_path)
            exact_out = True
    return exact_out


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
                   page_shuffle_seed=0, num_pages=None, tune=(), sampling=None):
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
        return _run_trajectory(dec, cfg, tw, dw, prompts, n_steps, tol, max_ctx, reserve, check_floats, tap_tol, sampling)
    finally:
        for knob, _, restore in tune:
            dec.tune(knob, restore)
        dec.close()


def _run_trajectory(dec, cfg, tw, dw, prompts, n_steps, tol, max_ctx, reserve, check_floats, tap_tol, sampling=None):
    B = len(prompts)
    rng = np.random.default_rng(sampling[1]) if sampling else None
    st = Stats()
    first = dec.prefill([np.asarray(p) for p in prompts], reserve)
    orcs = []
    for b in range(B):
        o = po.Oracle(cfg, tw, dw, max_ctx)
        f = o.prefill(np.asarray(prompts[b]))
        assert f == first[b], f"first token differs for sequence {b}: {f} vs {first[b]}"
        orcs.append(o)
    emitted = [[] for _ in range(B)]
    for step in range(n_steps):
        u = rng.random((B, 2 * cfg.tree_nodes), dtype=np.float32) if sampling else None
        outs = dec.step_sampled(sampling[0], u) if sampling else dec.step()
        for b in range(B):
            o = orcs[b]
            ids_before, n_before = o.ids, o.n
            o_out = o.step_sampled(sampling[0], u[b]) if sampling else o.step()
            g_out = outs[b]
            assert 1 <= len(g_out) <= cfg.tree_depth + 1
            exact = compare_step(dec, o, b, cfg, tol, st, g_out, check_floats, tap_tol,
                                 sampled=(sampling[0], u[b]) if sampling else None, n_ctx=n_before)
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
    for b in range(B if not sampling else 0):
        g = po.Oracle(cfg, tw, dw, max_ctx)
        g.prefill(np.asarray(prompts[b]))
        ref, mg = g.greedy_margins(len(emitted[b]))
        for i, (a, r) in enumerate(zip(emitted[b], ref)):
            if a != r:
                assert mg[i] <= decision_margin(tol), f"sequence {b}: token {i} differs from greedy decoding with margin {mg[i]}"
                break
    return st, emitted
