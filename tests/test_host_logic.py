"""Host-side checks that need no GPU: the CUDA library loads, exports every symbol the header declares,
rejects bad configurations before touching a device, and sizes its workspace sensibly."""
import ctypes as C
import os
import re

import pytest

from paper_2503_01840_b200 import binding as sb
from paper_2503_01840_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    hdr = open(os.path.join(ROOT, "include", "spec_b200.h")).read()
    declared = set(re.findall(r"\b(spec_[a-z_0-9]+)\s*\(", hdr))
    declared -= {"spec_ctx"}
    L = sb.lib()
    assert declared, "no declarations found"
    for name in sorted(declared):
        assert hasattr(L, name), f"{name} is declared in spec_b200.h but not exported"
    assert set(sb.EXPORTS) == declared


def test_workspace_bytes_and_cfg_validation():
    L = sb.lib()
    cfg = sb.make_cfg(synth.C1, batch=1, max_ctx=256, num_pages=16)
    n = L.spec_workspace_bytes(C.byref(cfg))
    assert n > 0 and n % 256 == 0
    cfg2 = sb.make_cfg(synth.C1, batch=1, max_ctx=256, num_pages=32)
    kv_page = synth.C1.n_kv_heads * synth.C1.page_size * synth.C1.head_dim * 4
    grow = L.spec_workspace_bytes(C.byref(cfg2)) - n
    assert grow == 16 * kv_page * 2 * (synth.C1.n_layers + 1)     # K and V pools of every layer + the draft layer
    for field, bad in (("tree_nodes", 65), ("tree_topk", 0), ("tree_depth", 0), ("head_dim", 60), ("page_size", 24),
                       ("dtype", 7), ("n_kv_heads", 3), ("batch", 0)):
        c = sb.make_cfg(synth.C1, batch=1, max_ctx=256, num_pages=16)
        setattr(c, field, bad)
        assert L.spec_workspace_bytes(C.byref(c)) == 0, field


def test_init_rejects_bad_arguments_without_a_device():
    L = sb.lib()
    h = C.c_void_p()
    assert L.spec_init(C.byref(h), None, None, None) == -2
    cfg = sb.make_cfg(synth.C1, batch=1, max_ctx=256, num_pages=16)
    tw, dw = sb._TW(), sb._DW()
    cfg.tree_nodes = 100
    assert L.spec_init(C.byref(h), C.byref(tw), C.byref(dw), C.byref(cfg)) == -1
    assert b"tree_nodes" in L.spec_last_error(None)
    cfg.tree_nodes = 16
    assert L.spec_init(C.byref(h), C.byref(tw), C.byref(dw), C.byref(cfg)) == -2      # workspace NULL
    cfg.workspace, cfg.workspace_bytes = 4096 + 8, 1 << 20
    assert L.spec_init(C.byref(h), C.byref(tw), C.byref(dw), C.byref(cfg)) == -3      # misaligned
    cfg.workspace = 4096
    assert L.spec_init(C.byref(h), C.byref(tw), C.byref(dw), C.byref(cfg)) == -2      # NULL weights
    assert not h.value


def test_paper_shaped_workspaces_fit_one_gpu():
    L = sb.lib()
    for name, reserve in (("C2", 256), ("C3", 128), ("C4", 1024), ("C5", 128)):
        m = synth.CONFIGS[name]
        plen = m.prompt_hi if m.batch > 1 else m.prompt_len
        max_ctx = plen + reserve + 160
        pages = m.batch * ((max_ctx + m.page_size - 1) // m.page_size)
        cfg = sb.make_cfg(m, batch=m.batch, max_ctx=max_ctx, num_pages=pages)
        n = L.spec_workspace_bytes(C.byref(cfg))
        assert 0 < n < 40e9, (name, n)


def test_single_kernel_entry_points_reject_null():
    L = sb.lib()
    assert L.spec_gemm(1, 0, None, None, None, 1, 1, 8, 1, None, None) == -2
    assert L.spec_argmax(None, 1, 1, None, None) == -2
    assert L.spec_logsoftmax_topk(None, 1, 1, 1, None, None, None, None) == -2
    assert L.spec_gemm_fused(None, None, None, 1, 1, 8, 1, 0, 0, None) == -2
    assert L.spec_gemm_swiglu(None, None, None, None, 1, 128, 8, None) == -2
    assert L.spec_step_sampled(None, 1.0, None, None, None) == -2
    assert L.spec_topk_scratch_bytes(10, 32000, 10) > 0


def _kernel_bodies():
    """(file, kernel name, body text) of every __global__ function of the CUDA sources."""
    csrc = os.path.join(ROOT, "paper_2503_01840_b200", "csrc")
    for fn in sorted(os.listdir(csrc)):
        if not fn.endswith(".cu"):
            continue
        s = open(os.path.join(csrc, fn)).read()
        for m in re.finditer(r"__global__\s+void\s+(?:__launch_bounds__\([^)]*\)\s*)?(\w+)\s*\(", s):
            i = s.index("{", m.end())
            depth, j = 0, i
            while True:
                depth += {"{": 1, "}": -1}.get(s[j], 0)
                if depth == 0:
                    break
                j += 1
            yield fn, m.group(1), s[i:j]


def test_every_step_kernel_orders_itself_behind_its_predecessor():
    """Kernels of a step are launched with programmatic dependent launch: a kernel may start before its predecessor
    has finished, and its successor waits only for IT.  A kernel without griddepcontrol.wait would let its successor
    overtake the kernel before it (the first QKV GEMM reading a RoPE table that is still being written), so every
    kernel the scheduler launches with the attribute must wait, and must do so before it touches global memory."""
    never_pdl = {"gemm_tcgen05_kernel", "reduce_slices_kernel"}      # launched without the attribute
    seen = 0
    for fn, name, body in _kernel_bodies():
        if name in never_pdl:
            continue
        seen += 1
        assert "pdl_wait()" in body, f"{fn}: {name} never calls pdl_wait()"
        assert "pdl_trigger()" in body, f"{fn}: {name} never calls pdl_trigger()"
    assert seen >= 25
    # the elementwise / tree kernels wait first thing: nothing but declarations may precede the wait
    for fn, name, body in _kernel_bodies():
        if fn in ("elementwise.cu", "tree.cu", "gemm_ref.cu", "attn_ref.cu") and name not in never_pdl:
            head = body[: body.index("pdl_wait()")]
            head = "\n".join(l for l in head.split("\n") if "__shared__" not in l)
            assert "[" not in head and "->" not in head, f"{fn}: {name} touches memory before pdl_wait()"
