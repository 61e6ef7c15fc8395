// Tensor-core tree-masked paged GQA attention (bf16).
#include "attn_fast.cuh"

namespace spec {

bool attn_fast_supported(int head_dim, int group) { (void)head_dim; (void)group; return false; }
size_t attn_fast_scratch_bytes(int rows, int n_heads, int head_dim, int max_ctx) { return 0; }
int launch_attn_fast(const bf16 *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, bf16 *out, int rows, int H, int G,
                     int hd, int max_ctx, void *scratch, cudaStream_t s) {
  return 0;
}

}  // namespace spec
