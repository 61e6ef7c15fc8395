/*
 * eagle3_oracle.h — CPU oracle for one EAGLE-3 speculative step.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-precision restatement of what the
 * speculative step computes, written from the EAGLE-3 paper (Section 2.1 speculative sampling,
 * Section 2.2 tree drafts / tree attention / dynamic tree, Section 3.1 inference pipeline,
 * Appendix A tree knobs).  It shares no code with the CUDA library; only tests, the smoke check
 * and the benchmark's CPU-baseline leg may call it.
 *
 * All arithmetic is fp32 in a fixed index order; no blocking, fusion or reordering.  A row's
 * result never depends on which other rows are processed in the same call, so a tree-masked
 * forward is bit-identical to decoding each root-to-leaf path as an ordinary sequence.
 *
 * Parity status: the emitted tokens, tree masks, tree-masked forward, building blocks and the
 * commit are pinned by tests (greedy-decode equality, brute-force ancestor sets, per-path
 * sequential runs, an independent Llama implementation, closed-form permutation weights).
 * The paper prints no logits, trees or ids, so agreement with the paper's own numbers
 * (acceptance lengths, speedups of Table 1) is "parity unpinned".
 */
#ifndef EAGLE3_ORACLE_H
#define EAGLE3_ORACLE_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ORC_MAX_NODES 64

typedef struct {
  int32_t wdtype;            /* weight storage: 0 = float32, 1 = bf16 bit patterns (widened exactly) */
  int32_t n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, draft_vocab;
  int32_t fuse_layers[3];    /* taps: residual stream after block i (0-based), low / mid / high  */
  float rope_theta, rms_eps;
  int32_t max_ctx;           /* positions the caches can hold                                  */
  int32_t tree_depth, tree_topk, tree_nodes;   /* D, K, N (N counts the root)                   */
} orc_cfg;

typedef struct {             /* row-major [out][in]; pointers are borrowed for the ctx lifetime */
  const void *embed, *final_norm, *lm_head;
  const void *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *mlp_norm, *const *w_gate, *const *w_up, *const *w_down;
} orc_target_weights;

typedef struct {
  const void *fc3, *fc2, *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down,
             *final_norm, *lm_head;
  const int32_t *d2t;
} orc_draft_weights;

typedef struct orc_ctx orc_ctx;

orc_ctx *orc_create(const orc_cfg *, const orc_target_weights *, const orc_draft_weights *);
void orc_destroy(orc_ctx *);

/* Section 3.1 "prefill phase": target forward over the prompt, taps everywhere, first token =
 * argmax at the last position; draft cache filled for entries 0..n-2; pending = {n-1}. */
int orc_prefill(orc_ctx *, const int32_t *ids, int32_t n, int32_t *first_id);

/* One draft + verify cycle.  out_ids gets `count` tokens (accepted drafts then the target's own
 * token), 1 <= count <= D+1. */
int orc_step(orc_ctx *, int32_t *out_ids, int32_t *count);

/* The same cycle at temperature T > 0 (Section 2.1's acceptance rule on the deterministic top-K tree of Section 2.2:
 * child c of the current node is accepted with probability p(tok[c]) under the residual of softmax(z / T), a rejected
 * token is removed from the residual, and when no child is left the token is drawn from the residual).  The random
 * numbers are inputs: u [2 * tree_nodes] in [0, 1); u[c] decides node c, u[tree_nodes + cur] draws the final token at
 * node cur (inverse CDF over increasing ids).  The emitted tokens are distributed exactly as plain sampling. */
int orc_step_sampled(orc_ctx *, float temperature, const float *u, int32_t *out_ids, int32_t *count);

/* The same cycle (greedy when temperature <= 0, else the stochastic rule with uniforms u) FOLLOWING another
 * implementation's integer decisions, so that a harness can compare every later stage after a near-tie the two sides
 * resolved differently.  Inputs: the other side's candidate tokens in pool layout (pool_tok [pool+1], target ids), its
 * frontier per pass (frontier [D][K], pool indices) and the pool indices of its pruned tree (sel_poolidx [nsel],
 * ascending, entry 0 = the root).  A followed choice of K items is adopted when it is valid on the oracle's own
 * values: order non-increasing within eps, nothing left out that beats the worst chosen item by more than eps (for the
 * pruned set also: parents kept).  An invalid choice is counted and the oracle's own is used.  Values (log-probs,
 * scores, logits) are always the oracle's own arithmetic.  A decision is one rank of a top-K choice (margin: the
 * smaller gap to its neighbours in the oracle's own order; last rank: to the best item left out) or the pruned set as
 * a whole (margin: the cut).  Outputs: decisions looked at, how many differed from the oracle's own choice, how many
 * choices were invalid; of those whose own margin exceeds `require`: how many, and how many
 * differed (must be 0 for a conforming implementation); the same two counts for margins in (band_lo, require]. */
typedef struct {
  const int32_t *pool_tok, *frontier, *sel_poolidx;
  int32_t nsel;
  float eps, require, band_lo;
  int32_t checked, differs, invalid, required, required_differs, band_total, band_differs;
} orc_follow;
int orc_step_follow(orc_ctx *, orc_follow *, float temperature, const float *u, int32_t *out_ids, int32_t *count);

/* Plain greedy autoregressive decoding of the target (the paper's "vanilla" baseline): continue the
 * current state by `gen` tokens, one target forward per token.  Needs a prefilled ctx. */
int orc_greedy(orc_ctx *, int32_t gen, int32_t *out_ids);
/* same, also reporting the top1 - top2 logit gap of every emitted token */
int orc_greedy_margins(orc_ctx *, int32_t gen, int32_t *out_ids, float *margins);

/* Step 5 alone (Section 2.2: one target forward over all tree nodes with tree attention) on a tree the caller
 * gives: node i holds tok[i] at RoPE position n_ctx + depth[i] and attends the committed positions [0, n_ctx) and
 * the nodes in mask[i] (ancestor-or-self bits, bit i set, none above i).  n_ctx <= committed length.  Outputs:
 * logits [nn][vocab], hidden [nn][hidden] (either may be NULL), taps [nn][3*hidden] (may be NULL).  Writes only the
 * step's tail scratch.  Lets a harness check a verify pass on a tree that differs from the oracle's own. */
int orc_verify_tree(orc_ctx *, int32_t n_ctx, int32_t nn, const int32_t *tok, const int32_t *depth, const uint64_t *mask,
                    float *logits, float *hidden, float *taps);

/* Put the ctx into the state "ids[0..n-1] committed, ids[n] is the root, P pending entries",
 * recomputing whatever the current caches do not already hold (common prefix is kept). */
int orc_force_state(orc_ctx *, const int32_t *ids, int32_t n, int32_t P);

int32_t orc_n(const orc_ctx *);          /* committed length          */
int32_t orc_pending(const orc_ctx *);    /* P                         */
const int32_t *orc_ids(const orc_ctx *); /* ids[0..n], ids[n] = root  */

/* Inspection of the last step (pointers stay valid until the next call on the ctx). */
enum {
  ORC_TREE_TOK = 1,      /* int32 [nodes]                         */
  ORC_TREE_PARENT,       /* int32 [nodes], node index, root: -1   */
  ORC_TREE_DEPTH,        /* int32 [nodes]                         */
  ORC_TREE_MASK,         /* uint64 [nodes] ancestor-or-self bits  */
  ORC_TREE_POOLIDX,      /* int32 [nodes] pool index (root 0)     */
  ORC_TREE_SCORE,        /* float [nodes]                         */
  ORC_Y,                 /* int32 [nodes] target argmax           */
  ORC_Y_MARGIN,          /* float [nodes] top1 - top2 logit       */
  ORC_TARGET_LOGITS,     /* float [nodes][V]                      */
  ORC_NODE_TAPS,         /* float [nodes][3k]                     */
  ORC_NODE_HIDDEN,       /* float [nodes][k] residual after last block */
  ORC_DRAFT_LOGITS,      /* float [D][K][Vd] (pass 0 uses row 0)  */
  ORC_DRAFT_A,           /* float [D][K][k]                       */
  ORC_POOL_TOK,          /* int32 [pool+1] target ids             */
  ORC_POOL_SCORE,        /* float [pool+1]                        */
  ORC_POOL_PARENT,       /* int32 [pool+1] pool index of parent   */
  ORC_FRONTIER,          /* int32 [D][K] pool indices processed by pass d (pass 0: root) */
  ORC_TOPK_MARGIN,       /* float [D][K] min gap between consecutive entries of the top K+1 */
  ORC_FRONTIER_MARGIN,   /* float [D] score gap at the frontier cut (inf if no cut) */
  ORC_RERANK_MARGIN,     /* float [1] score gap at the rerank cut (inf if no cut)   */
  ORC_PATH,              /* int32 [count] accepted node indices, root first */
  ORC_G_PENDING,         /* float [P_in][k] fused features of the step's pending entries */
  ORC_ACC_P,             /* float [nodes] sampled step: probability the node was tested against, -1 if not tried */
  ORC_BONUS_INTERVAL     /* double [2] sampled step: CDF interval (fractions of the residual mass) of the drawn token */
};
const void *orc_get(const orc_ctx *, int32_t what, int64_t *count);

/* cache reads for the commit pin: copies G*hd floats each */
int orc_read_target_kv(const orc_ctx *, int32_t layer, int32_t pos, float *k, float *v);
int orc_read_draft_kv(const orc_ctx *, int32_t pos, float *k, float *v);
int orc_read_taps(const orc_ctx *, int32_t pos, float *taps3k);

/* ---- building blocks, exported so tests can pin each against a library routine and so that
 * per-kernel parity tests can call exactly the arithmetic the step uses ---------------------- */
void orc_linear(int32_t wdtype, const void *W, int32_t O, int32_t I, const float *x, int32_t M, float *out);
void orc_rmsnorm(int32_t wdtype, const void *gain, const float *x, int32_t M, int32_t k, float eps, float *out);
void orc_rope(float *x, int32_t n_heads, int32_t head_dim, int32_t pos, float theta);
void orc_swiglu(const float *gate, const float *up, int64_t n, float *out);
/* one query head against keys/values given as arrays of row pointers, scale 1/sqrt(hd) */
void orc_attend(const float *q, const float *const *K, const float *const *V, int32_t n_keys,
                int32_t head_dim, float *out);
void orc_log_softmax(const float *z, int32_t n, float *lp);
/* top-K by (value desc, index asc); also writes the (K+1)-th value to next_val if non-null */
void orc_topk(const float *v, int32_t n, int32_t K, int32_t *idx, float *val, float *next_val);
int32_t orc_argmax(const float *v, int32_t n, float *margin);
/* tree assembly from a pool: select top-M by (score desc, pool index asc), order by pool index,
 * emit node arrays (node 0 = root).  pool arrays have pool_size+1 entries, entry 0 = root. */
int32_t orc_rerank(const float *pool_score, const int32_t *pool_parent, const int32_t *pool_tok,
                   const int32_t *pool_depth, int32_t pool_size, int32_t n_nodes_max,
                   int32_t root_tok, int32_t *tok, int32_t *parent, int32_t *depth, uint64_t *mask,
                   int32_t *poolidx, float *score, float *cut_margin);
/* greedy acceptance walk; returns count, writes path (node indices, root first) and ids */
int32_t orc_accept_sampled(const int32_t *tok, const int32_t *parent, const float *logits, int32_t V, int32_t n_nodes,
                           int32_t n_max, float temperature, const float *u, int32_t *path, int32_t *out_ids,
                           float *acc_p, double *bonus_lo, double *bonus_hi);
int32_t orc_accept(const int32_t *tok, const int32_t *parent, const int32_t *y, int32_t n_nodes,
                   int32_t *path, int32_t *out_ids);

#ifdef __cplusplus
}
#endif
#endif
