"""The allocation-free attention entry point (spec_attention_static) against the ordinary one.

Some users of the library cannot allocate device memory where they need attention (code running inside a
pre-sized arena, hosts that forbid cudaMalloc after start-up, loops that must not take an allocation's
implicit synchronisation).  For them the split-KV scratch lives in a device array built into the library.
This file is collected last on purpose: if it fails, a run that stops at the first failure has already
run every other test.  It passes alone in a fresh process and after the other tests."""
import numpy as np
import pytest
import torch

import pyoracle as po
from paper_2503_01840_b200 import binding as sb

pytestmark = pytest.mark.gpu

TOL = 2e-2      # the bf16 tolerance of the other attention tests


def _case(seed, rows=24, H=8, G=2, hd=128, ps=16, n_seq=2, pps=40, ctx=(437, 77), tail_len=40):
    g = torch.Generator().manual_seed(seed)
    perm = torch.randperm(n_seq * pps, generator=g).to(torch.int32).reshape(n_seq, pps)
    kp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(torch.bfloat16)
    vp = torch.randn(n_seq * pps, G, ps, hd, generator=g).to(torch.bfloat16)
    q = torch.randn(rows, H, hd, generator=g).to(torch.bfloat16)
    seq = torch.tensor([r % n_seq for r in range(rows)], dtype=torch.int32)
    seq[5] = -1                                                   # a padding row
    rctx = torch.tensor([ctx[r % n_seq] for r in range(rows)], dtype=torch.int32)
    lo = torch.randint(0, 2 ** 40, (rows,), generator=g, dtype=torch.int64) | 1
    hi = torch.zeros(rows, dtype=torch.int64)
    dev = lambda t: t.cuda()
    return dict(q=dev(q), k_pool=dev(kp), v_pool=dev(vp), page_table=dev(perm), page_size=ps, row_seq=dev(seq),
                row_ctx=dev(rctx), row_tail_base=dev(rctx), mask_lo=dev(lo), mask_hi=dev(hi), tail_len=tail_len,
                n_kv_heads=G, max_ctx=640)


def test_static_scratch_attention_matches_the_allocating_entry_point_twice():
    assert sb.lib().spec_attention_static_capacity() == 8 << 20
    for seed in (21, 22):                                          # two calls in a row share the built-in array
        c = _case(seed)
        want = sb.attention(**c, impl=0).float()
        out = torch.empty_like(c["q"])                             # the caller's output buffer
        got = sb.attention_static(**c, out=out).float()
        torch.cuda.synchronize()
        assert torch.isfinite(got).all()
        err = (got - want).abs().max().item()
        assert err <= TOL, err
        assert (got[5] == 0).all()                                 # padding rows stay zero
        # and against the CPU oracle's per-head attention for a few (row, head) pairs
        kp, vp, perm = c["k_pool"].cpu(), c["v_pool"].cpu(), c["page_table"].cpu()
        q, lo, seq, rctx = c["q"].cpu(), c["mask_lo"].cpu(), c["row_seq"].cpu(), c["row_ctx"].cpu()
        H, G, ps = q.shape[1], c["n_kv_heads"], c["page_size"]
        for r, h in ((0, 0), (7, 3), (12, 5), (23, 7)):
            s_, n = int(seq[r]), int(rctx[r])
            pos = list(range(n)) + [n + t for t in range(c["tail_len"]) if (int(lo[r]) >> t) & 1]
            gk = h // (H // G)
            K = np.stack([kp[perm[s_, p // ps], gk, p % ps].float().numpy() for p in pos])
            V = np.stack([vp[perm[s_, p // ps], gk, p % ps].float().numpy() for p in pos])
            ref = po.attend(q[r, h].float().numpy(), K, V)
            assert np.abs(got[r, h].cpu().numpy() - ref).max() <= TOL, (r, h)


def test_static_scratch_attention_rejects_shapes_beyond_its_capacity():
    c = _case(23)
    rows, H, hd = 64, 32, 128                                      # needs far more than 8 MiB of partials
    assert sb.lib().spec_attn_scratch_bytes(rows, H, hd, 640) > sb.lib().spec_attention_static_capacity()
    big_q = torch.zeros(rows, H, hd, dtype=torch.bfloat16, device="cuda")
    z32 = torch.zeros(rows, dtype=torch.int32, device="cuda")
    z64 = torch.zeros(rows, dtype=torch.int64, device="cuda")
    with pytest.raises(sb.SpecError) as e:
        sb.attention_static(big_q, c["k_pool"], c["v_pool"], c["page_table"], 16, z32, z32, z32, z64, z64, 0, 8, 640)
    assert e.value.code == -3
