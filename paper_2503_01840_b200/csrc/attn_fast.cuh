// Tensor-core tree-masked paged GQA attention (bf16): host-side interface.
#pragma once
#include "common.cuh"

namespace spec {

bool attn_fast_supported(int head_dim, int group);
size_t attn_fast_scratch_bytes(int rows, int n_heads, int head_dim, int max_ctx);
// rows are grouped as rows/rps consecutive blocks of rps rows that belong to one sequence (rps = 1 when
// nothing is known); ctx_hint sizes the key split (any value is correct); scratch may be NULL (one
// split).  Returns the number of kernels launched.
int launch_attn_fast(const bf16 *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, bf16 *out, int rows, int H, int G,
                     int hd, int rps, int ctx_hint, void *scratch, cudaStream_t s, bool contiguous_tail = false,
                     int32_t *status = nullptr, const int32_t *order = nullptr, int order_len = 0,
                     unsigned long long *stamp = nullptr);
// contiguous_tail: every row's tail_base equals its ctx (the tail keys follow the context in the cache), which lets the
// TMA-staged kernel fetch whole pages; status: device status words for its bounded waits (may be NULL).
// order: a permutation of the rows / rps row blocks (device, order_len entries; used when order_len == rows / rps): the
// TMA-staged kernels give block order[i] to the i-th group of CTAs, e.g. longest sequence first.
// stamp: profiling aid, see KernelStamp (may be NULL).
// Drops the cached K/V tensor maps (pools of one-shot callers come and go).
void attn_fast_forget_maps();
// CTAs an attention launch aims at when it splits the keys (process-wide; default 148 = one wave)
void attn_fast_set_target_ctas(int n);
// tcgen05 kernel for passes with more than 16 query rows per (sequence, KV head) and head_dim 128 (process-wide):
// 0 never, 1 always, 2 (default) when every CTA gets several key tiles; and a per-thread override for single calls (-1: none)
void attn_fast_set_umma(int mode);
void attn_fast_override_umma(int v);

}  // namespace spec
