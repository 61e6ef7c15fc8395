"""ctypes binding of the C-ABI library (include/spec_b200.h): argument marshalling only.

Every step of the speculative step runs inside the library's CUDA kernels; this module only packs
pointers of torch CUDA tensors into the C structs, allocates the workspace with torch and copies
small results back.  There is no CPU or PyTorch fallback: if the compiled library is missing and
cannot be built, importing the symbols raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import numpy as np
import torch

from . import build as _build

_lib = None

F32, BF16 = 0, 1
FLAG_REF_GEMM, FLAG_REF_ATTN, FLAG_CAPTURE, FLAG_NO_GRAPH, FLAG_STAMPS, FLAG_NO_PDL, FLAG_NO_TMA_ATTN = 1, 2, 4, 8, 16, 32, 128

(DBG_TREE_TOK, DBG_TREE_PARENT, DBG_TREE_DEPTH, DBG_TREE_MASK, DBG_TREE_POOLIDX, DBG_TREE_SCORE, DBG_Y,
 DBG_TARGET_LOGITS, DBG_NODE_TAPS, DBG_NODE_HIDDEN, DBG_DRAFT_LOGITS, DBG_DRAFT_A, DBG_POOL_TOK, DBG_POOL_SCORE,
 DBG_POOL_PARENT, DBG_FRONTIER, DBG_PATH, DBG_STATUS, DBG_PAGE_TABLE) = range(1, 20)
DBG_RAW_X, DBG_RAW_H, DBG_RAW_Q, DBG_RAW_AO, DBG_RAW_ACT, DBG_RAW_CAT, DBG_RAW_SSQ, DBG_RAW_LOGITS = range(100, 108)
DBG_STAMPS, DBG_STAMP_CLASS = 120, 121
_DBG_DTYPE = {**{i: np.float32 for i in range(100, 108)}, DBG_STAMPS: np.uint64, DBG_STAMP_CLASS: np.int32, DBG_TREE_TOK: np.int32, DBG_TREE_PARENT: np.int32, DBG_TREE_DEPTH: np.int32, DBG_TREE_MASK: np.uint64,
              DBG_TREE_POOLIDX: np.int32, DBG_TREE_SCORE: np.float32, DBG_Y: np.int32, DBG_TARGET_LOGITS: np.float32,
              DBG_NODE_TAPS: np.float32, DBG_NODE_HIDDEN: np.float32, DBG_DRAFT_LOGITS: np.float32,
              DBG_DRAFT_A: np.float32, DBG_POOL_TOK: np.int32, DBG_POOL_SCORE: np.float32, DBG_POOL_PARENT: np.int32,
              DBG_FRONTIER: np.int32, DBG_PATH: np.int32, DBG_STATUS: np.int32, DBG_PAGE_TABLE: np.int32}

_PP = C.POINTER(C.c_void_p)
_LAYER_FIELDS = ("attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate", "w_up", "w_down")


class _TW(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p)] + \
               [(n, _PP) for n in _LAYER_FIELDS]


class _DW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("fc3", "fc2", "attn_norm", "wq", "wk", "wv", "wo", "mlp_norm", "w_gate",
                                           "w_up", "w_down", "final_norm", "lm_head", "d2t")]


class _Cfg(C.Structure):
    _fields_ = [("dtype", C.c_int32), ("n_layers", C.c_int32), ("hidden", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32), ("ffn", C.c_int32), ("vocab", C.c_int32),
                ("draft_vocab", C.c_int32), ("fuse_layers", C.c_int32 * 3), ("rope_theta", C.c_float),
                ("rms_eps", C.c_float), ("batch", C.c_int32), ("max_ctx", C.c_int32), ("page_size", C.c_int32),
                ("num_pages", C.c_int32), ("page_shuffle_seed", C.c_int32), ("tree_depth", C.c_int32),
                ("tree_topk", C.c_int32), ("tree_nodes", C.c_int32), ("flags", C.c_int32),
                ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t), ("stream", C.c_void_p)]


EXPORTS = ("spec_workspace_bytes", "spec_init", "spec_prefill", "spec_step", "spec_step_async", "spec_step_sampled", "spec_plain_step",
           "spec_lengths", "spec_profile_step", "spec_tune", "spec_launches_per_step", "spec_step_bytes", "spec_free", "spec_last_error",
           "spec_debug_read", "spec_debug_read_kv", "spec_gemm", "spec_gemm_fused", "spec_gemm_swiglu", "spec_gemm_topk_scratch_bytes", "spec_gemm_topk", "spec_ttt_attention_scratch_bytes", "spec_ttt_attention",
           "spec_topk_scratch_bytes", "spec_attn_scratch_bytes",
           "spec_attention", "spec_attention_static", "spec_attention_static_capacity", "spec_logsoftmax_topk", "spec_argmax")


def library_path() -> str:
    return _build.LIB


def lib():
    """Loads (building first if the .so is absent or stale) the CUDA library."""
    global _lib
    if _lib is not None:
        return _lib
    path = _build.build()
    L = C.CDLL(path)
    vp, i32, i64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_size_t
    L.spec_workspace_bytes.restype = sz
    L.spec_workspace_bytes.argtypes = [C.POINTER(_Cfg)]
    L.spec_init.argtypes = [C.POINTER(vp), C.POINTER(_TW), C.POINTER(_DW), C.POINTER(_Cfg)]
    L.spec_prefill.argtypes = [vp, vp, vp, i32, vp]
    L.spec_step.argtypes = [vp, vp, vp]
    L.spec_step_async.argtypes = [vp, vp, vp]
    L.spec_plain_step.argtypes = [vp, vp]
    L.spec_step_sampled.argtypes = [vp, C.c_float, vp, vp, vp]
    L.spec_lengths.argtypes = [vp, vp]
    L.spec_launches_per_step.argtypes = [vp]
    L.spec_tune.argtypes = [vp, i32, i32]
    L.spec_profile_step.argtypes = [vp, vp, vp]
    L.spec_step_bytes.argtypes = [vp, C.POINTER(C.c_double)]
    L.spec_free.argtypes = [vp]
    L.spec_last_error.argtypes = [vp]
    L.spec_last_error.restype = C.c_char_p
    L.spec_debug_read.argtypes = [vp, i32, i32, vp, sz]
    L.spec_debug_read.restype = i64
    L.spec_debug_read_kv.argtypes = [vp, i32, i32, i32, vp, vp]
    L.spec_gemm.argtypes = [i32, i32, vp, vp, vp, i32, i32, i32, i32, vp]
    L.spec_attn_scratch_bytes.argtypes = [i32, i32, i32, i32]
    L.spec_attn_scratch_bytes.restype = sz
    L.spec_attention.argtypes = [i32, i32, vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, i32, vp, i32, i32, i32, i32, i32,
                                 vp, vp]
    L.spec_attention_static_capacity.argtypes = []
    L.spec_attention_static_capacity.restype = sz
    L.spec_attention_static.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, i32, vp, i32, i32, i32, i32, i32, vp]
    L.spec_gemm_fused.argtypes = [vp, vp, vp, i32, i32, i32, i32, i32, i32, vp]
    L.spec_gemm_swiglu.argtypes = [vp, vp, vp, vp, i32, i32, i32, vp]
    L.spec_gemm_topk_scratch_bytes.argtypes = [i32, i32, i32]
    L.spec_gemm_topk_scratch_bytes.restype = sz
    L.spec_gemm_topk.argtypes = [vp, vp, i32, i32, i32, i32, vp, vp, vp, vp]
    L.spec_ttt_attention_scratch_bytes.argtypes = [i32, i32, i32, i32]
    L.spec_ttt_attention_scratch_bytes.restype = sz
    L.spec_ttt_attention.argtypes = [vp, vp, vp, vp, i32, i32, vp, vp, i32, vp, vp, i32, i32, i32, i32, vp, vp]
    L.spec_topk_scratch_bytes.argtypes = [i32, i32, i32]
    L.spec_topk_scratch_bytes.restype = sz
    L.spec_logsoftmax_topk.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp]
    L.spec_argmax.argtypes = [vp, i32, i32, vp, vp]
    _lib = L
    return L


class SpecError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"spec error {code}: {msg}")
        self.code = code


def _dt(t: torch.dtype) -> int:
    if t == torch.float32:
        return F32
    if t == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t}")


def _stream_ptr(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def make_cfg(m, batch: int, max_ctx: int, num_pages: int, flags: int = 0, page_shuffle_seed: int = 0) -> _Cfg:
    """Packs a model/workload description (any object with the fields of synth.ModelCfg) into spec_cfg."""
    c = _Cfg()
    c.dtype = F32 if m.dtype == "fp32" else BF16
    for f in ("n_layers", "hidden", "n_heads", "n_kv_heads", "head_dim", "ffn", "vocab", "draft_vocab", "page_size",
              "tree_depth", "tree_topk", "tree_nodes"):
        setattr(c, f, int(getattr(m, f)))
    c.fuse_layers = (C.c_int32 * 3)(*m.fuse_layers)
    c.rope_theta, c.rms_eps = float(m.rope_theta), float(m.rms_eps)
    c.batch, c.max_ctx, c.num_pages, c.flags, c.page_shuffle_seed = batch, max_ctx, num_pages, flags, page_shuffle_seed
    return c


class SpecDecoder:
    """Owns one spec_ctx.  `target_w` / `draft_w` are dicts of CUDA tensors in the layout of
    synth.make_target_weights / make_draft_weights; they must stay alive (kept here)."""

    def __init__(self, model_cfg, target_w: Dict, draft_w: Dict, batch: int = 1, max_ctx: int = 1024,
                 num_pages: Optional[int] = None, flags: int = 0, page_shuffle_seed: int = 0,
                 stream: Optional[torch.cuda.Stream] = None):
        L = lib()
        self.m = model_cfg
        self.batch = batch
        self.Pmax = model_cfg.tree_depth + 1
        self.tree_nodes = model_cfg.tree_nodes
        if num_pages is None:
            num_pages = batch * ((max_ctx + model_cfg.page_size - 1) // model_cfg.page_size)
        self._keep = [target_w, draft_w]
        dev = target_w["embed"].device
        assert dev.type == "cuda", "weights must live on the GPU"
        self.device = dev
        # a dedicated stream: the legacy default stream cannot be captured into a CUDA graph
        self.stream = stream if stream is not None else torch.cuda.Stream(device=dev)
        stream = self.stream
        torch.cuda.synchronize(dev)          # weights may still be in flight on torch's current stream
        cfg = make_cfg(model_cfg, batch, max_ctx, num_pages, flags, page_shuffle_seed)
        need = L.spec_workspace_bytes(C.byref(cfg))
        if need == 0:
            raise SpecError(-1, "invalid configuration (spec_workspace_bytes returned 0)")
        self.workspace = torch.empty(need + 256, dtype=torch.uint8, device=dev)
        base = (self.workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace, cfg.workspace_bytes, cfg.stream = base, need, _stream_ptr(stream)
        self.workspace_bytes = need
        tw = _TW()
        want = torch.float32 if model_cfg.dtype == "fp32" else torch.bfloat16

        def ptr(t):
            assert t.is_cuda and t.is_contiguous() and t.dtype == want, (t.dtype, want)
            return t.data_ptr()

        tw.embed, tw.final_norm, tw.lm_head = ptr(target_w["embed"]), ptr(target_w["final_norm"]), ptr(target_w["lm_head"])
        nL = len(target_w["layers"])
        assert nL == model_cfg.n_layers
        for name in _LAYER_FIELDS:
            arr = (C.c_void_p * nL)(*[ptr(l[name]) for l in target_w["layers"]])
            self._keep.append(arr)
            setattr(tw, name, C.cast(arr, _PP))
        dw = _DW()
        for name, _ in _DW._fields_:
            if name == "d2t":
                d = draft_w["d2t"]
                assert d.is_cuda and d.dtype == torch.int32 and d.is_contiguous()
                dw.d2t = d.data_ptr()
            else:
                setattr(dw, name, ptr(draft_w[name]))
        h = C.c_void_p()
        rc = L.spec_init(C.byref(h), C.byref(tw), C.byref(dw), C.byref(cfg))
        if rc:
            raise SpecError(rc, L.spec_last_error(None).decode())
        self.h = h
        self._cfg = cfg

    # -- lifecycle
    def close(self):
        if getattr(self, "h", None):
            lib().spec_free(self.h)
            self.h = None
        self._keep = []          # the weights and the workspace may be freed once the context is gone
        self.workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, rc: int):
        if rc:
            raise SpecError(rc, lib().spec_last_error(self.h).decode())

    # -- the path
    def prefill(self, prompts: Sequence, reserve_tokens: int) -> np.ndarray:
        lens = np.array([len(p) for p in prompts], np.int32)
        assert lens.size == self.batch
        ids = np.ascontiguousarray(np.concatenate([np.asarray(p, np.int32) for p in prompts]))
        first = np.zeros(self.batch, np.int32)
        self._check(lib().spec_prefill(self.h, ids.ctypes.data, lens.ctypes.data, int(reserve_tokens), first.ctypes.data))
        return first

    def step(self) -> List[np.ndarray]:
        ids = np.zeros((self.batch, self.Pmax), np.int32)
        cnt = np.zeros(self.batch, np.int32)
        self._check(lib().spec_step(self.h, ids.ctypes.data, cnt.ctypes.data))
        return [ids[b, : cnt[b]].copy() for b in range(self.batch)]

    def step_async(self, dev_ids: Optional[torch.Tensor] = None, dev_counts: Optional[torch.Tensor] = None):
        self._check(lib().spec_step_async(self.h, dev_ids.data_ptr() if dev_ids is not None else None,
                                          dev_counts.data_ptr() if dev_counts is not None else None))

    def step_sampled(self, temperature: float, u) -> List[np.ndarray]:
        """One step with the stochastic acceptance rule; u: float32 [batch][2 * tree_nodes] uniforms in [0, 1)."""
        u = np.ascontiguousarray(u, dtype=np.float32).reshape(self.batch, 2 * self.tree_nodes)
        ids = np.zeros((self.batch, self.Pmax), np.int32)
        cnt = np.zeros(self.batch, np.int32)
        self._check(lib().spec_step_sampled(self.h, float(temperature), u.ctypes.data, ids.ctypes.data, cnt.ctypes.data))
        return [ids[b, : cnt[b]].copy() for b in range(self.batch)]

    def plain_step(self) -> np.ndarray:
        out = np.zeros(self.batch, np.int32)
        self._check(lib().spec_plain_step(self.h, out.ctypes.data))
        return out

    def lengths(self) -> np.ndarray:
        out = np.zeros(self.batch, np.int32)
        self._check(lib().spec_lengths(self.h, out.ctypes.data))
        return out

    PROF_CLASSES = ("gemm", "attention", "add_norm", "rope_kv", "silu_mul", "misc", "topk", "tree", "argmax", "commit")

    def profile_step(self):
        """One step with an event before every launch: {class: (ms, launches)}."""
        ms = np.zeros(len(self.PROF_CLASSES), np.float32)
        n = np.zeros(len(self.PROF_CLASSES), np.int32)
        self._check(lib().spec_profile_step(self.h, ms.ctypes.data, n.ctypes.data))
        return {c: (float(ms[i]), int(n[i])) for i, c in enumerate(self.PROF_CLASSES)}

    def kernel_stamps(self):
        """FLAG_STAMPS: (uint64 [n][2] {inputs ready, last CTA left} in ns of the GPU timer, class names [n]) of the GEMM
        and attention launches of the last step, in launch order."""
        st = self.debug(DBG_STAMPS, 0).reshape(-1, 2)
        cls = self.debug(DBG_STAMP_CLASS, 0)
        return st, [self.PROF_CLASSES[c] for c in cls[: len(st)]]

    TUNE_GEMM_CTAS, TUNE_DEBUG_LAUNCH_BUDGET, TUNE_ATTN_CTAS, TUNE_DEBUG_WAIT_RUNS_OUT, TUNE_ATTN_UMMA = 2, 3, 4, 5, 6
    TUNE_GEMM_PAIRS = 7

    def tune(self, what: int, value: int):
        self._check(lib().spec_tune(self.h, what, value))

    def launches_per_step(self) -> int:
        return lib().spec_launches_per_step(self.h)

    def step_bytes(self) -> float:
        v = C.c_double(0)
        self._check(lib().spec_step_bytes(self.h, C.byref(v)))
        return v.value

    # -- inspection
    def debug(self, what: int, seq: int = 0) -> np.ndarray:
        L = lib()
        n = L.spec_debug_read(self.h, what, seq, None, 0)
        if n < 0:
            self._check(int(n))
        dt = np.dtype(_DBG_DTYPE[what])
        buf = np.zeros(n // dt.itemsize, dt)
        if n:
            got = L.spec_debug_read(self.h, what, seq, buf.ctypes.data, n)
            if got < 0:
                self._check(int(got))
        return buf

    def read_kv(self, seq: int, layer: int, pos: int):
        kvd = self.m.n_kv_heads * self.m.head_dim
        k = np.zeros(kvd, np.float32)
        v = np.zeros(kvd, np.float32)
        self._check(lib().spec_debug_read_kv(self.h, seq, layer, pos, k.ctypes.data, v.ctypes.data))
        return k, v


# ------------------------------------------------------------------ single kernels (tests, timing)
def gemm(x: torch.Tensor, w: torch.Tensor, impl: int = 0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out[r][o] = sum_i x[r][i] w[o][i] (fp32 out).  impl 0: tcgen05 kernel (bf16), 1: plain kernel."""
    rows, I = x.shape
    O = w.shape[0]
    assert w.shape[1] == I and x.is_contiguous() and w.is_contiguous() and x.dtype == w.dtype
    if out is None:
        out = torch.empty(rows, O, dtype=torch.float32, device=x.device)
    rc = lib().spec_gemm(_dt(x.dtype), impl, x.data_ptr(), w.data_ptr(), out.data_ptr(), rows, O, I, out.stride(0),
                         _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_gemm")
    return out


def attention(q, k_pool, v_pool, page_table, page_size, row_seq, row_ctx, row_tail_base, mask_lo, mask_hi, tail_len,
              n_kv_heads, max_ctx, impl: int = 0):
    rows, H, hd = q.shape
    out = torch.empty_like(q)
    nbytes = lib().spec_attn_scratch_bytes(rows, H, hd, max_ctx)
    scratch = torch.empty(max(64, nbytes), dtype=torch.uint8, device=q.device)
    rc = lib().spec_attention(_dt(q.dtype), impl, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), page_table.data_ptr(),
                              page_table.shape[1], page_size, row_seq.data_ptr(), row_ctx.data_ptr(),
                              row_tail_base.data_ptr(), mask_lo.data_ptr(), mask_hi.data_ptr(), tail_len, out.data_ptr(),
                              rows, H, n_kv_heads, hd, max_ctx, scratch.data_ptr(), _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_attention")
    return out


def attention_static(q, k_pool, v_pool, page_table, page_size, row_seq, row_ctx, row_tail_base, mask_lo, mask_hi,
                     tail_len, n_kv_heads, max_ctx, out: Optional[torch.Tensor] = None):
    """spec_attention_static: the tensor-core attention kernel with its split-KV scratch in the library's
    built-in device array, for callers that cannot allocate.  `out` may be passed in so that the call itself
    allocates nothing; raises SpecError(-3) when the shape needs more scratch than the array holds."""
    rows, H, hd = q.shape
    if out is None:
        out = torch.empty_like(q)
    rc = lib().spec_attention_static(q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), page_table.data_ptr(),
                                     page_table.shape[1], page_size, row_seq.data_ptr(), row_ctx.data_ptr(),
                                     row_tail_base.data_ptr(), mask_lo.data_ptr(), mask_hi.data_ptr(), tail_len,
                                     out.data_ptr(), rows, H, n_kv_heads, hd, max_ctx, _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_attention_static")
    return out


def gemm_fused(x: torch.Tensor, w: torch.Tensor, split: int = 0, stages: int = 0, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """out = x . w^T (fp32) on the cluster split-K tcgen05 kernel of the step; split/stages 0 = library's choice."""
    rows, I = x.shape
    O = w.shape[0]
    assert w.shape[1] == I and x.is_contiguous() and w.is_contiguous() and x.dtype == w.dtype == torch.bfloat16
    if out is None:
        out = torch.empty(rows, O, dtype=torch.float32, device=x.device)
    rc = lib().spec_gemm_fused(x.data_ptr(), w.data_ptr(), out.data_ptr(), rows, O, I, out.stride(0), split, stages,
                               _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_gemm_fused")
    return out


def gemm_topk(x: torch.Tensor, w: torch.Tensor, K: int):
    """Top-K ids and log-probabilities of softmax(x . w^T) per row without materialising the logits: (int32 [rows][K],
    float32 [rows][K])."""
    rows, I = x.shape
    O = w.shape[0]
    assert x.is_contiguous() and w.is_contiguous() and x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    idx = torch.empty(rows, K, dtype=torch.int32, device=x.device)
    lp = torch.empty(rows, K, dtype=torch.float32, device=x.device)
    scratch = torch.empty(max(64, lib().spec_gemm_topk_scratch_bytes(rows, O, K)), dtype=torch.uint8, device=x.device)
    rc = lib().spec_gemm_topk(x.data_ptr(), w.data_ptr(), rows, O, I, K, idx.data_ptr(), lp.data_ptr(), scratch.data_ptr(),
                              _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_gemm_topk")
    return idx, lp


def ttt_attention(q: torch.Tensor, k_pool: torch.Tensor, v_pool: torch.Tensor, page_table: torch.Tensor, k_diag, v_diag,
                  want_lse: bool = False):
    """Training-time-test attention of one simulated step.  q bf16 [T][H][128]; k_pool / v_pool the native step's paged
    keys / values [pages][G][page_size][128]; page_table int32 [pages_per_seq]; k_diag / v_diag bf16 [J][T][G][128] or None.
    Returns out bf16 [T][H][128] (and the float32 [T][H] log-normaliser when want_lse)."""
    T, H, hd = q.shape
    G, ps = k_pool.shape[1], k_pool.shape[2]
    rows = (T + 127) // 128 * 128
    qp = torch.zeros(rows, H, hd, dtype=torch.bfloat16, device=q.device)
    qp[:T] = q
    out = torch.zeros_like(qp)
    J = 0 if k_diag is None else k_diag.shape[0]
    lse = torch.empty(T, H, dtype=torch.float32, device=q.device) if want_lse else None
    scratch = torch.empty(max(64, lib().spec_ttt_attention_scratch_bytes(T, H, G, hd)), dtype=torch.uint8, device=q.device)
    rc = lib().spec_ttt_attention(qp.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), page_table.data_ptr(), page_table.numel(), ps,
                                  k_diag.data_ptr() if J else None, v_diag.data_ptr() if J else None, J, out.data_ptr(),
                                  lse.data_ptr() if want_lse else None, T, H, G, hd, scratch.data_ptr(), _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_ttt_attention")
    return (out[:T], lse) if want_lse else out[:T]


def gemm_swiglu(x: torch.Tensor, w_gate: torch.Tensor, w_up: torch.Tensor) -> torch.Tensor:
    """act = bf16(silu(x . w_gate^T) * (x . w_up^T)) on the step's gate/up kernel."""
    rows, I = x.shape
    F = w_gate.shape[0]
    assert w_gate.shape == w_up.shape == (F, I) and x.dtype == w_gate.dtype == w_up.dtype == torch.bfloat16
    assert x.is_contiguous() and w_gate.is_contiguous() and w_up.is_contiguous()
    act = torch.empty(rows, F, dtype=torch.bfloat16, device=x.device)
    rc = lib().spec_gemm_swiglu(x.data_ptr(), w_gate.data_ptr(), w_up.data_ptr(), act.data_ptr(), rows, F, I,
                                _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_gemm_swiglu")
    return act


def logsoftmax_topk(logits: torch.Tensor, K: int, two_stage: bool = True):
    rows, n = logits.shape
    idx = torch.empty(rows, K, dtype=torch.int32, device=logits.device)
    lp = torch.empty(rows, K, dtype=torch.float32, device=logits.device)
    scratch = None
    if two_stage:
        scratch = torch.empty(lib().spec_topk_scratch_bytes(rows, n, K), dtype=torch.uint8, device=logits.device)
    rc = lib().spec_logsoftmax_topk(logits.data_ptr(), rows, n, K, idx.data_ptr(), lp.data_ptr(),
                                    scratch.data_ptr() if scratch is not None else None, _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_logsoftmax_topk")
    return idx, lp


def argmax(logits: torch.Tensor) -> torch.Tensor:
    rows, n = logits.shape
    idx = torch.empty(rows, dtype=torch.int32, device=logits.device)
    rc = lib().spec_argmax(logits.data_ptr(), rows, n, idx.data_ptr(), _stream_ptr(None))
    if rc:
        raise SpecError(rc, "spec_argmax")
    return idx
