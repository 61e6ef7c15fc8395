"""ctypes wrapper around the CPU oracle (TEST INFRASTRUCTURE ONLY).

Only tests, the smoke check and the benchmark's CPU-baseline leg import this.  It takes weights
as dicts of CPU torch tensors (float32, or bfloat16 which is handed over as raw bf16 bit
patterns) in the layout the synthetic-input module produces, and never touches the CUDA library.
"""
from __future__ import annotations

import ctypes as C
import os
import sys

import numpy as np
import torch

sys.path.insert(0, os.path.dirname(os.path.abspath(__file__)))
import build as _build  # noqa: E402

_lib = None

(TREE_TOK, TREE_PARENT, TREE_DEPTH, TREE_MASK, TREE_POOLIDX, TREE_SCORE, Y, Y_MARGIN, TARGET_LOGITS,
 NODE_TAPS, NODE_HIDDEN, DRAFT_LOGITS, DRAFT_A, POOL_TOK, POOL_SCORE, POOL_PARENT, FRONTIER,
 TOPK_MARGIN, FRONTIER_MARGIN, RERANK_MARGIN, PATH, G_PENDING, ACC_P, BONUS_INTERVAL) = range(1, 25)
_DTYPES = {TREE_TOK: np.int32, TREE_PARENT: np.int32, TREE_DEPTH: np.int32, TREE_MASK: np.uint64,
           TREE_POOLIDX: np.int32, TREE_SCORE: np.float32, Y: np.int32, Y_MARGIN: np.float32,
           TARGET_LOGITS: np.float32, NODE_TAPS: np.float32, NODE_HIDDEN: np.float32,
           DRAFT_LOGITS: np.float32, DRAFT_A: np.float32, POOL_TOK: np.int32, POOL_SCORE: np.float32,
           POOL_PARENT: np.int32, FRONTIER: np.int32, TOPK_MARGIN: np.float32,
           FRONTIER_MARGIN: np.float32, RERANK_MARGIN: np.float32, PATH: np.int32, G_PENDING: np.float32,
           ACC_P: np.float32, BONUS_INTERVAL: np.float64}


class _Cfg(C.Structure):
    _fields_ = [("wdtype", C.c_int32), ("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
                ("draft_vocab", C.c_int32), ("fuse_layers", C.c_int32 * 3), ("rope_theta", C.c_float),
                ("rms_eps", C.c_float), ("max_ctx", C.c_int32), ("tree_depth", C.c_int32),
                ("tree_topk", C.c_int32), ("tree_nodes", C.c_int32)]


_PP = C.POINTER(C.c_void_p)


class _Follow(C.Structure):
    _fields_ = [("pool_tok", C.c_void_p), ("frontier", C.c_void_p), ("sel_poolidx", C.c_void_p), ("nsel", C.c_int32),
                ("eps", C.c_float), ("require", C.c_float), ("band_lo", C.c_float)] + \
               [(n, C.c_int32) for n in ("checked", "differs", "invalid", "required", "required_differs", "band_total",
                                         "band_differs")]


class _TW(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, _PP) for n in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")]


class _DW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("fc3", "fc2", "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm",
                                           "w_gate", "w_up", "w_down", "final_norm", "lm_head", "d2t")]


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(_build.build())
        L.orc_create.restype = C.c_void_p
        L.orc_create.argtypes = [C.POINTER(_Cfg), C.POINTER(_TW), C.POINTER(_DW)]
        L.orc_destroy.argtypes = [C.c_void_p]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_step.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_step_sampled.argtypes = [C.c_void_p, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_greedy.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_greedy_margins.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.orc_force_state.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32]
        L.orc_step_follow.restype = C.c_int
        L.orc_step_follow.argtypes = [C.c_void_p, C.POINTER(_Follow), C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_verify_tree.restype = C.c_int
        L.orc_verify_tree.argtypes = [C.c_void_p, C.c_int32, C.c_int32] + [C.c_void_p] * 6
        L.orc_n.argtypes = [C.c_void_p]
        L.orc_pending.argtypes = [C.c_void_p]
        L.orc_ids.argtypes = [C.c_void_p]
        L.orc_ids.restype = C.POINTER(C.c_int32)
        L.orc_get.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int64)]
        L.orc_get.restype = C.c_void_p
        for f in (L.orc_read_target_kv, L.orc_read_draft_kv, L.orc_read_taps):
            f.restype = C.c_int
        L.orc_read_target_kv.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p]
        L.orc_read_draft_kv.argtypes = [C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        L.orc_read_taps.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_linear.argtypes = [C.c_int32, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_rmsnorm.argtypes = [C.c_int32, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_void_p]
        L.orc_rope.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float]
        L.orc_swiglu.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_void_p]
        L.orc_attend.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.orc_log_softmax.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_topk.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_argmax.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.orc_argmax.restype = C.c_int32
        L.orc_rerank.restype = C.c_int32
        L.orc_rerank.argtypes = [C.c_void_p] * 4 + [C.c_int32, C.c_int32, C.c_int32] + [C.c_void_p] * 7
        L.orc_accept.restype = C.c_int32
        L.orc_accept.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p]
        _lib = L
    return _lib


def _raw(t: torch.Tensor):
    """(wdtype, contiguous CPU tensor to keep alive, data pointer)."""
    t = t.detach().to("cpu").contiguous()
    if t.dtype == torch.bfloat16:
        return 1, t, t.data_ptr()
    if t.dtype == torch.float32:
        return 0, t, t.data_ptr()
    raise TypeError(t.dtype)


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.c_void_p)


# ------------------------------------------------------------------ building blocks
def linear(W: torch.Tensor, x: np.ndarray) -> np.ndarray:
    wd, keep, ptr = _raw(W)
    x = _np(x, np.float32)
    M, I = x.shape
    O = W.shape[0]
    out = np.empty((M, O), np.float32)
    lib().orc_linear(wd, ptr, O, I, _p(x), M, _p(out))
    return out


def rmsnorm(gain: torch.Tensor, x: np.ndarray, eps: float) -> np.ndarray:
    wd, keep, ptr = _raw(gain)
    x = _np(x, np.float32)
    out = np.empty_like(x)
    lib().orc_rmsnorm(wd, ptr, _p(x), x.shape[0], x.shape[1], eps, _p(out))
    return out


def rope(x: np.ndarray, n_heads: int, head_dim: int, pos: int, theta: float) -> np.ndarray:
    x = _np(x, np.float32).copy()
    lib().orc_rope(_p(x), n_heads, head_dim, pos, theta)
    return x


def swiglu(g: np.ndarray, u: np.ndarray) -> np.ndarray:
    g = _np(g, np.float32); u = _np(u, np.float32)
    out = np.empty_like(g)
    lib().orc_swiglu(_p(g), _p(u), g.size, _p(out))
    return out


def attend(q: np.ndarray, K: np.ndarray, V: np.ndarray) -> np.ndarray:
    """q [hd], K/V [n][hd] -> [hd]"""
    q = _np(q, np.float32); K = _np(K, np.float32); V = _np(V, np.float32)
    n, hd = K.shape
    kp = (C.c_void_p * n)(*[K.ctypes.data + i * hd * 4 for i in range(n)])
    vp = (C.c_void_p * n)(*[V.ctypes.data + i * hd * 4 for i in range(n)])
    out = np.empty(hd, np.float32)
    lib().orc_attend(_p(q), kp, vp, n, hd, _p(out))
    return out


def log_softmax(z: np.ndarray) -> np.ndarray:
    z = _np(z, np.float32)
    out = np.empty_like(z)
    lib().orc_log_softmax(_p(z), z.size, _p(out))
    return out


def topk(v: np.ndarray, K: int):
    v = _np(v, np.float32)
    idx = np.empty(K, np.int32); val = np.empty(K, np.float32); nxt = np.empty(1, np.float32)
    lib().orc_topk(_p(v), v.size, K, _p(idx), _p(val), _p(nxt))
    return idx, val, float(nxt[0])


def argmax(v: np.ndarray):
    v = _np(v, np.float32)
    m = np.empty(1, np.float32)
    i = lib().orc_argmax(_p(v), v.size, _p(m))
    return int(i), float(m[0])


def rerank(pool_score, pool_parent, pool_tok, pool_depth, n_nodes_max, root_tok):
    ps = _np(pool_score, np.float32); pp = _np(pool_parent, np.int32)
    pt = _np(pool_tok, np.int32); pd = _np(pool_depth, np.int32)
    pool = ps.size - 1
    tok = np.zeros(64, np.int32); par = np.zeros(64, np.int32); dep = np.zeros(64, np.int32)
    mask = np.zeros(64, np.uint64); pidx = np.zeros(64, np.int32); sc = np.zeros(64, np.float32)
    cut = np.zeros(1, np.float32)
    nn = lib().orc_rerank(_p(ps), _p(pp), _p(pt), _p(pd), pool, n_nodes_max, root_tok,
                          _p(tok), _p(par), _p(dep), _p(mask), _p(pidx), _p(sc), _p(cut))
    return dict(n=nn, tok=tok[:nn], parent=par[:nn], depth=dep[:nn], mask=mask[:nn], poolidx=pidx[:nn],
                score=sc[:nn], cut_margin=float(cut[0]))


def accept(tok, parent, y):
    tok = _np(tok, np.int32); parent = _np(parent, np.int32); y = _np(y, np.int32)
    path = np.zeros(64, np.int32); out = np.zeros(64, np.int32)
    cnt = lib().orc_accept(_p(tok), _p(parent), _p(y), tok.size, _p(path), _p(out))
    return cnt, path[:cnt].copy(), out[:cnt].copy()


def accept_sampled(tok, parent, logits, temperature, u, n_max=None):
    """The stochastic acceptance rule on a given tree: logits [nodes][V], u [2 * n_max].  Returns
    (count, path, out_ids, acc_p, (bonus_lo, bonus_hi))."""
    tok = _np(tok, np.int32); parent = _np(parent, np.int32)
    logits = _np(logits, np.float32)
    nn, V = logits.shape
    n_max = nn if n_max is None else n_max
    u = _np(u, np.float32)
    assert u.size == 2 * n_max and tok.size == nn
    path = np.zeros(64, np.int32); out = np.zeros(64, np.int32)
    acc_p = np.zeros(nn, np.float32)
    lo = C.c_double(0.0); hi = C.c_double(0.0)
    f = lib().orc_accept_sampled
    f.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_void_p, C.c_void_p,
                  C.c_void_p, C.c_void_p, C.POINTER(C.c_double), C.POINTER(C.c_double)]
    cnt = f(_p(tok), _p(parent), _p(logits), V, nn, n_max, float(temperature), _p(u), _p(path), _p(out), _p(acc_p),
            C.byref(lo), C.byref(hi))
    return cnt, path[:cnt].copy(), out[:cnt].copy(), acc_p, (lo.value, hi.value)


def ttt_attention_rows(q, k0, v0, kd, vd, rows):
    """Training-time-test attention of one simulated step for the positions in `rows`, written out from its definition
    (Section 3.2, the figure of the attention masks during training-time test) in float64: the query at position i sees
    the native step's keys 0..i and, of every simulated step s, only the entry at position i.  q [T][H][hd]; k0, v0
    [T][G][hd]; kd, vd [J][T][G][hd] (J may be 0).  Returns (out [len(rows)][H][hd], lse [len(rows)][H]) as float64."""
    q = np.asarray(q, np.float64); k0 = np.asarray(k0, np.float64); v0 = np.asarray(v0, np.float64)
    kd = np.asarray(kd, np.float64); vd = np.asarray(vd, np.float64)
    T, H, hd = q.shape
    G = k0.shape[1]
    J = kd.shape[0] if kd.size else 0
    out = np.zeros((len(rows), H, hd)); lse = np.zeros((len(rows), H))
    for n, i in enumerate(rows):
        for h in range(H):
            g = h // (H // G)
            keys = np.concatenate([k0[: i + 1, g]] + [kd[s, i, g][None] for s in range(J)], 0)
            vals = np.concatenate([v0[: i + 1, g]] + [vd[s, i, g][None] for s in range(J)], 0)
            sc = keys @ q[i, h] / np.sqrt(hd)
            m = sc.max()
            e = np.exp(sc - m)
            out[n, h] = (e[:, None] * vals).sum(0) / e.sum()
            lse[n, h] = m + np.log(e.sum())
    return out, lse


def ttt_attention(q, k0, v0, kd, vd):
    """The same for every position."""
    return ttt_attention_rows(q, k0, v0, kd, vd, list(range(np.asarray(q).shape[0])))


# ------------------------------------------------------------------ the model
class Oracle:
    """One sequence.  `cfg` is a synth.ModelCfg-like object; weights are the synth dicts."""

    def __init__(self, cfg, target_w, draft_w, max_ctx: int):
        L = lib()
        self.cfg = cfg
        self._keep = []
        wds = set()

        def reg(t):
            wd, keep, ptr = _raw(t)
            self._keep.append(keep)
            wds.add(wd)
            return ptr

        tw = _TW()
        tw.embed, tw.final_norm, tw.lm_head = reg(target_w["embed"]), reg(target_w["final_norm"]), reg(target_w["lm_head"])
        nL = len(target_w["layers"])
        assert nL == cfg.n_layers
        for name in ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down"):
            arr = (C.c_void_p * nL)(*[reg(l[name]) for l in target_w["layers"]])
            self._keep.append(arr)
            setattr(tw, name, C.cast(arr, _PP))
        dw = _DW()
        for name, _ in _DW._fields_:
            if name == "d2t":
                d = draft_w["d2t"].detach().to("cpu").to(torch.int32).contiguous()
                self._keep.append(d)
                dw.d2t = d.data_ptr()
            else:
                setattr(dw, name, reg(draft_w[name]))
        assert len(wds) == 1, "all weights must share one dtype"
        c = _Cfg()
        c.wdtype = wds.pop()
        for f in ("n_layers", "hidden", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab", "draft_vocab",
                  "tree_depth", "tree_topk", "tree_nodes"):
            setattr(c, f, getattr(cfg, f))
        c.fuse_layers = (C.c_int32 * 3)(*cfg.fuse_layers)
        c.rope_theta, c.rms_eps, c.max_ctx = cfg.rope_theta, cfg.rms_eps, max_ctx
        self._tw, self._dw, self._c = tw, dw, c
        self.h = L.orc_create(C.byref(c), C.byref(tw), C.byref(dw))
        if not self.h:
            raise ValueError("orc_create rejected the configuration")
        self.kvd = cfg.n_kv_heads * cfg.head_dim

    def close(self):
        if self.h:
            lib().orc_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def prefill(self, ids) -> int:
        ids = _np(ids, np.int32)
        first = np.zeros(1, np.int32)
        rc = lib().orc_prefill(self.h, _p(ids), ids.size, _p(first))
        if rc:
            raise RuntimeError("orc_prefill failed")
        return int(first[0])

    def step(self):
        out = np.zeros(self.cfg.tree_depth + 1, np.int32)
        cnt = np.zeros(1, np.int32)
        rc = lib().orc_step(self.h, _p(out), _p(cnt))
        if rc:
            raise RuntimeError("orc_step failed (capacity?)")
        return out[: int(cnt[0])].copy()

    def step_sampled(self, temperature: float, u) -> np.ndarray:
        """One step with the stochastic acceptance rule; u: 2 * tree_nodes uniforms in [0, 1) (see the header)."""
        u = _np(u, np.float32)
        assert u.size == 2 * self.cfg.tree_nodes
        out = np.zeros(self.cfg.tree_depth + 1, np.int32)
        cnt = np.zeros(1, np.int32)
        rc = lib().orc_step_sampled(self.h, float(temperature), _p(u), _p(out), _p(cnt))
        if rc:
            raise RuntimeError("orc_step_sampled failed (capacity, temperature?)")
        return out[: int(cnt[0])].copy()

    def step_follow(self, pool_tok, frontier, sel_poolidx, eps: float, require: float, band_lo: float,
                    temperature: float = 0.0, u=None):
        """One step that adopts another implementation's decisions wherever they are valid within eps on the oracle's own
        values (see the header).  Returns (out_ids, counters dict)."""
        pool_tok = _np(pool_tok, np.int32); frontier = _np(frontier, np.int32); sel = _np(sel_poolidx, np.int32)
        assert pool_tok.size == self.cfg.pool + 1 and frontier.size == self.cfg.tree_depth * self.cfg.tree_topk
        fw = _Follow()
        fw.pool_tok, fw.frontier, fw.sel_poolidx, fw.nsel = pool_tok.ctypes.data, frontier.ctypes.data, sel.ctypes.data, sel.size
        fw.eps, fw.require, fw.band_lo = eps, require, band_lo
        uu = _np(u, np.float32) if u is not None else None
        out = np.zeros(self.cfg.tree_depth + 1, np.int32)
        cnt = np.zeros(1, np.int32)
        rc = lib().orc_step_follow(self.h, C.byref(fw), float(temperature), _p(uu) if uu is not None else None, _p(out), _p(cnt))
        if rc:
            raise RuntimeError("orc_step_follow failed (capacity, arguments?)")
        names = ("checked", "differs", "invalid", "required", "required_differs", "band_total", "band_differs")
        return out[: int(cnt[0])].copy(), {n: int(getattr(fw, n)) for n in names}

    def greedy(self, gen: int) -> np.ndarray:
        out = np.zeros(gen, np.int32)
        if lib().orc_greedy(self.h, gen, _p(out)):
            raise RuntimeError("orc_greedy failed")
        return out

    def greedy_margins(self, gen: int):
        out = np.zeros(gen, np.int32)
        mg = np.zeros(gen, np.float32)
        if lib().orc_greedy_margins(self.h, gen, _p(out), _p(mg)):
            raise RuntimeError("orc_greedy failed")
        return out, mg

    def force_state(self, ids, n: int, P: int):
        ids = _np(ids, np.int32)
        assert ids.size >= n + 1
        if lib().orc_force_state(self.h, _p(ids), n, P):
            raise RuntimeError("orc_force_state failed")

    def verify_tree(self, n_ctx: int, tok, depth, mask):
        """The verify pass (step 5) on a given tree over the committed prefix [0, n_ctx): returns (logits [nn][V],
        hidden [nn][k], taps [nn][3k])."""
        tok = _np(tok, np.int32); depth = _np(depth, np.int32); mask = _np(mask, np.uint64)
        nn, k, V = tok.size, self.cfg.hidden, self.cfg.vocab
        logits = np.empty((nn, V), np.float32); hidden = np.empty((nn, k), np.float32); taps = np.empty((nn, 3 * k), np.float32)
        rc = lib().orc_verify_tree(self.h, n_ctx, nn, _p(tok), _p(depth), _p(mask), _p(logits), _p(hidden), _p(taps))
        if rc:
            raise RuntimeError("orc_verify_tree rejected the tree")
        return logits, hidden, taps

    @property
    def n(self) -> int:
        return lib().orc_n(self.h)

    @property
    def pending(self) -> int:
        return lib().orc_pending(self.h)

    @property
    def ids(self) -> np.ndarray:
        p = lib().orc_ids(self.h)
        return np.ctypeslib.as_array(p, shape=(self.n + 1,)).copy()

    def get(self, what: int) -> np.ndarray:
        cnt = C.c_int64(0)
        p = lib().orc_get(self.h, what, C.byref(cnt))
        dt = np.dtype(_DTYPES[what])
        if cnt.value == 0:
            return np.zeros(0, dt)
        buf = (C.c_char * (cnt.value * dt.itemsize)).from_address(p)
        return np.frombuffer(buf, dtype=dt).copy()

    def target_kv(self, layer: int, pos: int):
        k = np.empty(self.kvd, np.float32); v = np.empty(self.kvd, np.float32)
        assert lib().orc_read_target_kv(self.h, layer, pos, _p(k), _p(v)) == 0
        return k, v

    def draft_kv(self, pos: int):
        k = np.empty(self.kvd, np.float32); v = np.empty(self.kvd, np.float32)
        assert lib().orc_read_draft_kv(self.h, pos, _p(k), _p(v)) == 0
        return k, v

    def taps(self, pos: int):
        t = np.empty(3 * self.cfg.hidden, np.float32)
        assert lib().orc_read_taps(self.h, pos, _p(t)) == 0
        return t
