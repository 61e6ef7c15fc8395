// Tensor-core tree-masked paged GQA attention (bf16): host-side interface.
#pragma once
#include "common.cuh"

namespace spec {

bool attn_fast_supported(int head_dim, int group);
size_t attn_fast_scratch_bytes(int rows, int n_heads, int head_dim, int max_ctx);
// returns the number of kernels launched
int launch_attn_fast(const bf16 *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, bf16 *out, int rows, int H, int G,
                     int hd, int max_ctx, void *scratch, cudaStream_t s);

}  // namespace spec
