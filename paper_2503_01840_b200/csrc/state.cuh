// Device-resident per-sequence state and tree buffers of a speculative-step context.
#pragma once
#include "common.cuh"

namespace spec {

struct SeqState {        // arrays of [batch]
  int32_t *n;            // committed length; the root token sits at position n
  int32_t *n_prev;       // n before the last commit
  int32_t *P;            // pending draft entries (positions n-P .. n-1)
  int32_t *root;         // token at position n (already emitted)
  int32_t *cap;          // positions this sequence has pages for
  int32_t *last_row;     // row of the last pending entry in the extend pass
  int32_t *active;       // 0: sequence skipped this step (capacity)
  int32_t *order;        // sequence indices by decreasing committed length: the order attention CTAs are issued in
};

struct TreeBufs {
  int32_t pool, K, D, N, Pmax;          // pool = K + (D-1) K^2 ; Pmax = D + 1
  int32_t *pool_tok, *pool_parent, *pool_depth;   // [B][pool+1]
  float *pool_score;
  int32_t *frontier;     // [B][D][K] pool indices processed by each pass
  int32_t *front_cur;    // [B][K]
  int32_t *feat_row;     // [B*K] row (of the previous pass's residual) holding the parent's output
  int32_t *tk_idx;       // [rows][K] top-k draft ids
  float *tk_lp;          // [rows][K]
  int32_t *tok, *parent, *depth, *poolidx;   // [B][N]
  float *score;
  uint64_t *mask;
  int32_t *nn;           // [B] nodes in the tree
  int32_t *y;            // [B*N] target argmax per node
  int32_t *path;         // [B][Pmax]
  int32_t *out_ids;      // [B][Pmax]
  int32_t *out_cnt;      // [B]
  int32_t *pend_tok;     // [B][Pmax] token following each pending position
};

void launch_prep_extend(SeqState st, TreeBufs tb, RowMeta m, int B, int need_positions, int32_t *status, cudaStream_t s);
void launch_expand(SeqState st, TreeBufs tb, RowMeta m, const int32_t *d2t, int pass, int B, cudaStream_t s);
// One launch between two draft passes (merge of the LM head's per-tile candidates, expansion, the next pass's row
// metadata, FC2 input and RoPE angles); returns -1 when the shape does not fit (tiles > 256, K > 15 or too many candidates).
size_t draft_tree_step_smem(int tiles, int K);
int draft_tree_cand_ld(int tiles);      // row pitch (in tiles) of the candidate arrays: tiles rounded up to a multiple of 4
int launch_draft_tree_step(SeqState st, TreeBufs tb, RowMeta m, const int32_t *d2t, int pass, const float *cand_val,
                           const int32_t *cand_idx, const float *cand_max, const float *cand_sum, int tiles, int ld, const float *x,
                           const bf16 *embed, bf16 *cat, int k, const double *inv_freq, float2 *cs, int half, int B, cudaStream_t s);
// the merge of per-tile candidates alone: idx / lp [rows][K]; -1 when the shape does not fit
int launch_merge_candidates(const float *cand_val, const int32_t *cand_idx, const float *cand_max, const float *cand_sum, int tiles,
                            int ld, int rows, int K, int32_t *idx, float *lp, cudaStream_t s);
void launch_rerank(SeqState st, TreeBufs tb, RowMeta m, int B, cudaStream_t s);
void launch_plain_tree(SeqState st, TreeBufs tb, RowMeta m, int B, cudaStream_t s);
void launch_accept(SeqState st, TreeBufs tb, int B, int rows_per_seq, cudaStream_t s);
// Stochastic acceptance: logits fp32 [B * rows_per_seq][V] of the verify pass; u = B x 2N uniforms followed by one float,
// 1 / temperature (all device memory).
void launch_accept_sampled(SeqState st, TreeBufs tb, const float *logits, int V, const float *u, int B, int rows_per_seq,
                           cudaStream_t s);
template <typename T>
void launch_commit(SeqState st, TreeBufs tb, const KvPool *pools /*device array [L]*/, PageMap pm, const T *node_taps,
                   T *pend_taps, int B, int L, int G, int hd, int k, int rows_per_seq, cudaStream_t s);

}  // namespace spec
