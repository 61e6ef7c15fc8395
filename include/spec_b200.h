/*
 * spec_b200.h — C ABI of the B200 (sm_100a) EAGLE-3 speculative-step library.
 *
 * One speculative step = drafting (feature fusion, draft decoder layer, reduced-vocabulary LM head,
 * dynamic draft tree) followed by verification (one tree-masked target forward, greedy acceptance,
 * KV-cache compaction).  The operations follow the EAGLE-3 paper: Section 2.1 (draft / verify
 * alternation and the acceptance rule), Section 2.2 (tree drafts, tree attention, the dynamic tree
 * with end-of-draft pruning), Section 3.1 (the inference pipeline: l/m/h fusion, g/a + embedding
 * through an FC layer into one decoder layer, LM head), Appendix A (tree depth, total draft tokens,
 * nodes per expansion).
 *
 * Conventions
 *   - Every function returns 0 on success and a negative spec_status otherwise; nothing aborts or
 *     throws.  spec_last_error() gives a static, human-readable string for the last failure of a ctx
 *     (or of spec_init when ctx is NULL).
 *   - "device" pointers are CUDA device memory of the current device, "host" pointers ordinary host
 *     memory.  All matrices are row-major [out][in]; dtype is cfg.dtype for weights and caches.
 *   - The caller owns weights, workspace and stream; they are borrowed from spec_init to spec_free.
 *     Weights are never written; the workspace is written only by this library while the ctx lives.
 *   - The library allocates no device memory except where a function says so.
 */
#ifndef SPEC_B200_H
#define SPEC_B200_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct spec_ctx spec_ctx;

enum spec_status {
  SPEC_OK = 0,
  SPEC_ERR_INVALID_CFG = -1,     /* a cfg field is out of range (message names it)                    */
  SPEC_ERR_NULL = -2,            /* a required pointer is NULL                                        */
  SPEC_ERR_WORKSPACE = -3,       /* workspace too small or misaligned (256 B)                         */
  SPEC_ERR_CAPACITY = -4,        /* a sequence would outgrow max_ctx / its pages; state is unchanged  */
  SPEC_ERR_STATE = -5,           /* call order: step before prefill, etc.                             */
  SPEC_ERR_CUDA = -6,            /* a CUDA runtime/driver call failed                                 */
  SPEC_ERR_DEVICE_STATUS = -7,   /* a kernel reported a bounded-wait timeout or a failed bounds check */
  SPEC_ERR_UNSUPPORTED = -8
};

enum spec_dtype { SPEC_F32 = 0, SPEC_BF16 = 1 };

/* cfg.flags */
enum {
  SPEC_FLAG_REF_GEMM = 1,        /* use the plain CUDA-core GEMM kernel also for bf16 (debugging aid)   */
  SPEC_FLAG_REF_ATTN = 2,        /* use the plain CUDA-core attention kernel also for bf16             */
  SPEC_FLAG_CAPTURE = 4,         /* keep per-pass draft logits / features for spec_debug_read          */
  SPEC_FLAG_NO_GRAPH = 8,        /* launch kernels one by one instead of replaying a CUDA graph        */
  SPEC_FLAG_STAMPS = 16,         /* profiling aid: every GEMM and attention launch of a step records when its
                                    inputs became ready and when its last CTA left (SPEC_DBG_STAMPS); costs two
                                    atomics per CTA, so timed runs leave it off                          */
  SPEC_FLAG_NO_PDL = 32,         /* no programmatic dependent launch between the kernels of a step    */
  SPEC_FLAG_NO_TMA_ATTN = 128    /* attention K/V tiles through cp.async instead of TMA page copies    */
};

/* Target model weights (Section 3.1: the frozen target whose layers are tapped).  Device pointers;
 * the per-layer members are HOST arrays of n_layers device pointers. */
typedef struct {
  const void *embed;        /* [vocab][hidden]                       */
  const void *final_norm;   /* [hidden]                              */
  const void *lm_head;      /* [vocab][hidden]                       */
  const void *const *attn_norm, *const *wq, *const *wk, *const *wv, *const *wo;
  const void *const *mlp_norm, *const *w_gate, *const *w_up, *const *w_down;
} spec_target_weights;

/* Draft head (Section 3.1): fc3 fuses [l;m;h] (3k -> k); fc2 maps [g or a ; e(token)] (2k -> k);
 * one decoder layer of the target's shape; final norm; LM head over the draft vocabulary;
 * d2t[i] = target id of draft id i, strictly increasing. */
typedef struct {
  const void *fc3, *fc2, *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down,
             *final_norm, *lm_head;
  const int32_t *d2t;       /* device, [draft_vocab] */
} spec_draft_weights;

typedef struct {
  int32_t dtype;            /* spec_dtype: storage type of weights, activations fed to GEMMs, KV cache */
  int32_t n_layers, hidden, n_heads, n_kv_heads, head_dim, ffn, vocab, draft_vocab;
  int32_t fuse_layers[3];   /* taps = residual stream after block i (0-based): low, mid, high          */
  float rope_theta, rms_eps;
  int32_t batch;            /* sequences advanced together by one spec_step                            */
  int32_t max_ctx;          /* largest committed length + tree any sequence may reach                  */
  int32_t page_size;        /* KV tokens per page (16 in the paper-shaped workloads)                   */
  int32_t num_pages;        /* pages in the pool shared by all sequences                               */
  int32_t page_shuffle_seed;/* 0: pages handed out in index order; else a seeded shuffle of the pool   */
  int32_t tree_depth;       /* D: draft passes per step (Appendix A: "depth")                          */
  int32_t tree_topk;        /* K: nodes kept per expansion                                            */
  int32_t tree_nodes;       /* N: verified nodes including the root, <= 64                             */
  int32_t flags;
  void *workspace;          /* device, 256-byte aligned, spec_workspace_bytes(cfg) bytes               */
  size_t workspace_bytes;
  void *stream;             /* cudaStream_t on which every kernel is launched                          */
} spec_cfg;

/* Bytes of device workspace the ctx needs for this cfg (0 if the cfg is invalid). Pure host code. */
size_t spec_workspace_bytes(const spec_cfg *cfg);

/* Validates cfg, carves the workspace (KV pages, page tables, draft cache, tree buffers, counters),
 * builds TMA descriptors.  Launches only small set-up kernels.  On failure *out is NULL. */
int spec_init(spec_ctx **out, const spec_target_weights *tw, const spec_draft_weights *dw, const spec_cfg *cfg);

/* Prefill (Section 3.1, "prefill phase"): target forward over each prompt, filling the paged KV cache
 * and the three tapped feature streams, the first generated token (argmax at the last position), and
 * the draft head's own cache for all but the last position.
 *   prompt_ids  host, all prompts concatenated; prompt_lens host [batch]; reserve_tokens: tokens each
 *   sequence may still generate (pages for prompt + reserve + tree are taken now);
 *   first_ids   host [batch], out: the root token of the first step.
 * Synchronises the stream before returning. */
int spec_prefill(spec_ctx *ctx, const int32_t *prompt_ids, const int32_t *prompt_lens, int32_t reserve_tokens,
                 int32_t *first_ids);

/* One speculative step for every sequence (Sections 2.1, 2.2, 3.1).
 *   out_ids    host [batch][tree_depth+1]: accepted draft tokens followed by the target's own token
 *   out_counts host [batch]: tokens emitted, 1..tree_depth+1 (the paper's per-cycle acceptance length)
 * Synchronises the stream.  SPEC_ERR_CAPACITY leaves every sequence unchanged. */
int spec_step(spec_ctx *ctx, int32_t *out_ids, int32_t *out_counts);

/* Same step without synchronisation: results go to DEVICE buffers dev_ids [batch][tree_depth+1] and
 * dev_counts [batch] (either may be NULL).  Capacity is checked against an upper bound of the
 * committed lengths (each async step may add tree_depth+1). */
int spec_step_async(spec_ctx *ctx, int32_t *dev_ids, int32_t *dev_counts);

/* One speculative step at temperature T > 0 (the non-greedy setting of Section 2.1 / Table 1): drafting and the
 * tree-masked target forward are those of spec_step; acceptance is stochastic.  Section 2.1 states the rule for a chain
 * whose tokens were sampled from the draft distribution; the tree of Section 2.2 is the draft's deterministic top-K, so a
 * tried child is a point-mass proposal: child c of the current node is accepted with probability p(tok[c]) under what
 * is left of softmax(logits / T) after its rejected elder siblings were removed, and when no child is left the token is
 * drawn from that residual (inverse CDF over increasing ids).  The emitted tokens are distributed as plain sampling
 * from the target.  The random numbers are inputs: u host float [batch][2 * tree_nodes] in [0, 1); u[b][c] decides
 * node c of sequence b, u[b][tree_nodes + cur] draws the final token at node cur.  out_ids / out_counts as spec_step.
 * 0 < temperature <= 1e4.  Synchronises. */
int spec_step_sampled(spec_ctx *ctx, float temperature, const float *u, int32_t *out_ids, int32_t *out_counts);

/* Plain greedy decoding of the target on the same kernels (the paper's "vanilla" baseline): one target
 * forward per token for every sequence, draft untouched.  out_ids host [batch]. Synchronises. */
int spec_plain_step(spec_ctx *ctx, int32_t *out_ids);

/* Committed length of every sequence (host [batch]); synchronises. */
int spec_lengths(spec_ctx *ctx, int32_t *lens);

/* One speculative step launched kernel by kernel with a CUDA event in front of every launch; reports,
 * per kernel class, the summed time to the next launch (ms) and the number of launches.  Arrays of
 * SPEC_PROF_CLASSES entries.  State advances exactly as in spec_step; synchronises.  Timing aid only. */
enum spec_prof_class {
  SPEC_PROF_GEMM = 0, SPEC_PROF_ATTN, SPEC_PROF_NORM, SPEC_PROF_ROPE_KV, SPEC_PROF_ACT, SPEC_PROF_MISC,
  SPEC_PROF_TOPK, SPEC_PROF_TREE, SPEC_PROF_ARGMAX, SPEC_PROF_COMMIT, SPEC_PROF_CLASSES
};
int spec_profile_step(spec_ctx *ctx, float *class_ms, int32_t *class_launches);

/* Performance knobs (the defaults are tuned for B200; results never depend on them).
 *   SPEC_TUNE_GEMM_CTAS   CTAs a weight-streaming GEMM launch aims at (process-wide) */
enum spec_tune_knob { SPEC_TUNE_GEMM_CTAS = 2,
                      SPEC_TUNE_DEBUG_LAUNCH_BUDGET = 3 /* debugging: run only the first n kernels of each step (-1: all) */,
                      SPEC_TUNE_ATTN_CTAS = 4 /* CTAs an attention launch aims at when splitting keys (process-wide) */,
                      SPEC_TUNE_DEBUG_WAIT_RUNS_OUT = 5 /* test hook for the bounded device waits: with a value n > 0 one CTA of the verify
                                                  pass's LM-head GEMM never receives its first activation tile and gives up after n
                                                  polls; the step then returns SPEC_ERR_DEVICE_STATUS (0 = off) */,
                      SPEC_TUNE_GEMM_PAIRS = 7 /* 256-row GEMM tiles of neighbouring feature tiles as CTA pairs (tcgen05 cta_group::2): bit 0 = the split-K
                                                  kernel (default off: measured no faster), bit 1 = the gate/up kernel (default on); process-wide;
                                                  the one knob that may be set with a NULL ctx */,
                      SPEC_TUNE_ATTN_UMMA = 6 /* tree passes (head_dim 128): 1 = tcgen05 attention kernel, 0 = mma.sync kernel, 2 (default) = tcgen05
                                                  when every CTA gets several key tiles, i.e. long contexts (process-wide) */ };
int spec_tune(spec_ctx *ctx, int32_t what, int32_t value);

/* Number of kernels one spec_step launches (for launch accounting). */
int spec_launches_per_step(const spec_ctx *ctx);

/* Algorithmic HBM bytes of one step at the current committed lengths: every weight once per pass,
 * target and draft KV once (Section 4.3's "memory accesses"); synchronises to read the lengths. */
int spec_step_bytes(spec_ctx *ctx, double *bytes);

int spec_free(spec_ctx *ctx);
const char *spec_last_error(const spec_ctx *ctx);

/* ---- inspection for parity tests (synchronises; copies to host) ----------------------------- */
enum spec_debug_what {
  SPEC_DBG_TREE_TOK = 1,     /* int32 [nodes]            */
  SPEC_DBG_TREE_PARENT,      /* int32 [nodes], root -1   */
  SPEC_DBG_TREE_DEPTH,       /* int32 [nodes]            */
  SPEC_DBG_TREE_MASK,        /* uint64 [nodes]           */
  SPEC_DBG_TREE_POOLIDX,     /* int32 [nodes]            */
  SPEC_DBG_TREE_SCORE,       /* float [nodes]            */
  SPEC_DBG_Y,                /* int32 [nodes]            */
  SPEC_DBG_TARGET_LOGITS,    /* float [nodes][vocab]; bf16 models keep them only with SPEC_FLAG_CAPTURE */
  SPEC_DBG_NODE_TAPS,        /* float [nodes][3*hidden] (widened from the storage dtype) */
  SPEC_DBG_NODE_HIDDEN,      /* float [nodes][hidden] residual stream after the last block */
  SPEC_DBG_DRAFT_LOGITS,     /* float [D][K][draft_vocab]; needs SPEC_FLAG_CAPTURE      */
  SPEC_DBG_DRAFT_A,          /* float [D][K][hidden];      needs SPEC_FLAG_CAPTURE      */
  SPEC_DBG_POOL_TOK,         /* int32 [pool+1]           */
  SPEC_DBG_POOL_SCORE,       /* float [pool+1]           */
  SPEC_DBG_POOL_PARENT,      /* int32 [pool+1]           */
  SPEC_DBG_FRONTIER,         /* int32 [D][K]             */
  SPEC_DBG_PATH,             /* int32 [count]            */
  SPEC_DBG_STATUS,           /* int32 [4] device status words */
  SPEC_DBG_PAGE_TABLE,       /* int32 [pages of seq]     */
  /* raw activation buffers of the last pass as floats, all allocated rows (debugging) */
  SPEC_DBG_RAW_X = 100, SPEC_DBG_RAW_H, SPEC_DBG_RAW_Q, SPEC_DBG_RAW_AO, SPEC_DBG_RAW_ACT, SPEC_DBG_RAW_CAT,
  SPEC_DBG_RAW_SSQ, SPEC_DBG_RAW_LOGITS,
  /* SPEC_FLAG_STAMPS: per stamped launch of the last step, in launch order, uint64 [n][2] = {earliest time a CTA of the
   * launch had its inputs ready (after its programmatic-dependent-launch wait), latest time a CTA left}, nanoseconds
   * of the GPU's global timer; and the launch's profile class, int32 [n] */
  SPEC_DBG_STAMPS = 120, SPEC_DBG_STAMP_CLASS
};
/* Copies up to `bytes` of item `what` of sequence `seq` (last step) to host_dst; returns bytes
 * available (>= 0) or a negative status. */
int64_t spec_debug_read(spec_ctx *ctx, int32_t what, int32_t seq, void *host_dst, size_t bytes);
/* K/V of a committed position as floats: k,v host [n_kv_heads*head_dim]; layer -1 = draft cache. */
int spec_debug_read_kv(spec_ctx *ctx, int32_t seq, int32_t layer, int32_t pos, float *k, float *v);

/* ---- single kernels on caller-provided DEVICE buffers, for per-kernel parity tests and timing ---
 * Each launches on `stream` and does not synchronise.  dtype as spec_dtype. */

/* out[r][o] = sum_i x[r][i] * w[o][i]; x [rows][in] dtype, w [out][in] dtype, out fp32 [rows][ldo]
 * (first `out` columns).  impl 0: the step's tcgen05/TMEM kernel with the library's own plan (bf16 only; the shape
 * limits of spec_gemm_fused), 1: plain CUDA-core kernel. */
int spec_gemm(int32_t dtype, int32_t impl, const void *x, const void *w, float *out_f32, int32_t rows, int32_t out,
              int32_t in, int32_t ldo, void *stream);

/* The same contraction on the kernel the step uses (Section 3.1's FC, projection and LM-head layers are
 * all of this form): bf16, tcgen05/TMEM, split-K reduced across a thread-block cluster through
 * distributed shared memory, no scratch.  rows <= 256, in % 8 == 0, 16-byte aligned x and w.
 * split: K slices (= cluster size, 1..8), stages: TMA pipeline depth; 0 lets the library choose. */
int spec_gemm_fused(const void *x, const void *w, float *out_f32, int32_t rows, int32_t out, int32_t in, int32_t ldo,
                    int32_t split, int32_t stages, void *stream);

/* The draft LM head followed by log-softmax and top-K (Section 2.2: the draft tree is expanded by the draft model's
 * confidence; Appendix A: nodes per expansion), on the kernels the step uses, without ever writing the logits: the
 * GEMM's epilogue leaves, per 128-logit tile and row, the tile maximum, the sum of exp relative to it and the tile's K
 * best logits, and a merge kernel turns them into each row's K best ids (value descending, lower id first on ties) and
 * their log-probabilities.  x [rows][in] bf16, w [out][in] bf16, out_idx int32 [rows][K], out_lp float [rows][K];
 * scratch: spec_gemm_topk_scratch_bytes(rows, out, K) bytes of device memory.  rows <= 256, in % 8 == 0, K <= 15,
 * out <= 32768 and out / 128 * K <= 3200 (SPEC_ERR_UNSUPPORTED otherwise). */
size_t spec_gemm_topk_scratch_bytes(int32_t rows, int32_t out, int32_t K);
int spec_gemm_topk(const void *x, const void *w, int32_t rows, int32_t out, int32_t in, int32_t K, int32_t *out_idx,
                   float *out_lp, void *scratch, void *stream);

/* Gate/up half of the decoder layer's MLP (the draft layer and every target layer are LLaMA-style decoder layers,
 * Section 3.1), on the kernel the step uses: act[r][f] = bf16(silu(g) * u), g = sum_i x[r][i] * w_gate[f][i], u likewise
 * with w_up, both accumulated in fp32 (a cluster holds the gate and the up tile of the same 128 features and their K
 * slices).  x [rows][in] bf16, w_gate / w_up [F][in] bf16, act [rows][F] bf16, all device pointers, 16-byte aligned;
 * rows <= 256, in % 8 == 0.  Returns SPEC_OK or a negative code; nothing is allocated. */
int spec_gemm_swiglu(const void *x, const void *w_gate, const void *w_up, void *act, int32_t rows, int32_t F, int32_t in,
                     void *stream);

/* Tree-masked paged GQA attention (Section 2.2 "tree attention") for `rows` query rows of one or
 * more sequences.  q [rows][H][hd] dtype; K/V pools [num_pages][G][page_size][hd] dtype;
 * page_table int32 [n_seq][pages_per_seq]; per row: seq, ctx_len (positions 0..ctx_len-1 all visible),
 * tail_base (first tail position), mask lo/hi (bit t: tail position tail_base+t visible);
 * out [rows][H][hd] dtype.  impl 0: tensor-core kernel (bf16), 1: plain kernel, 2: tensor-core kernel with
 * TMA-staged K/V pages (bf16; needs row_tail_base[r] == row_ctx[r] for every row and page_size 16, 32 or 64;
 * other shapes fall back to impl 0), 3: tcgen05 kernel (bf16, head_dim 128, the conditions of impl 2, and ALL rows
 * belong to one sequence: equal row_seq and row_ctx; S = Q K^T and O += P V on tcgen05.mma with TMEM accumulators;
 * other shapes fall back to impl 2).
 * scratch: spec_attn_scratch_bytes(...) bytes of device memory for split-KV partial results. */
size_t spec_attn_scratch_bytes(int32_t rows, int32_t n_heads, int32_t head_dim, int32_t max_ctx);
int spec_attention(int32_t dtype, int32_t impl, const void *q, const void *k_pool, const void *v_pool,
                   const int32_t *page_table, int32_t pages_per_seq, int32_t page_size, const int32_t *row_seq,
                   const int32_t *row_ctx, const int32_t *row_tail_base, const uint64_t *row_mask_lo,
                   const uint64_t *row_mask_hi, int32_t tail_len, void *out, int32_t rows, int32_t n_heads,
                   int32_t n_kv_heads, int32_t head_dim, int32_t max_ctx, void *scratch, void *stream);

/* spec_attention without any allocation (the paper has no counterpart: this is a packaging variant
 * of the tensor-core kernel, bf16 only).  It is meant for callers that cannot obtain device memory
 * at the point where they need attention - code living inside a pre-sized memory arena, plugins
 * whose host forbids cudaMalloc after start-up, loops that must not take the implicit device
 * synchronisation of an allocation.  The split-KV partial results go to an 8 MiB device array that
 * is part of the library image (every GPU that loads the library holds it until the process ends);
 * inputs and outputs are still the caller's, with the meaning and layout of spec_attention.
 *   - Limit: spec_attn_scratch_bytes(rows, n_heads, head_dim, max_ctx) must not exceed
 *     spec_attention_static_capacity(); larger calls return SPEC_ERR_WORKSPACE and print the sizes.
 *   - The first call on each device looks up the array's device address (that device must be
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array.  Nothing in it has to start at zero (every partial
 *     that is read was written by the same call), but two calls whose kernels overlap on the GPU
 *     (different streams) race on it: keep calls on one stream or order them yourself.
 *   - Calls no cudaMalloc/cudaFree and no allocating library routine; does not synchronise. */
size_t spec_attention_static_capacity(void);
int spec_attention_static(const void *q, const void *k_pool, const void *v_pool, const int32_t *page_table,
                          int32_t pages_per_seq, int32_t page_size, const int32_t *row_seq, const int32_t *row_ctx,
                          const int32_t *row_tail_base, const uint64_t *row_mask_lo, const uint64_t *row_mask_hi,
                          int32_t tail_len, void *out, int32_t rows, int32_t n_heads, int32_t n_kv_heads,
                          int32_t head_dim, int32_t max_ctx, void *stream);

/* Training-time-test attention, forward (Section 3.2 and its figure of the attention masks: while the draft model is
 * trained its own outputs are fed back for further simulated steps; a query then sees the original sequence through the
 * ordinary causal mask and, of every earlier simulated step, only the entry at its own position: the mask is lower
 * triangular over the native keys and diagonal over every simulated step's keys, so the diagonal part needs no matrix
 * product, only one dot product per step).  One call = the attention of one simulated step for one sequence:
 *   out[i][h] = softmax over { q[i][h].K0[p][g] : p <= i } U { q[i][h].Kd[s][i][g] : s < n_steps } (scale hd^-1/2) applied
 *   to the matching rows of V0 / Vd, with g = h / (n_heads / n_kv_heads).
 * q, out: bf16 [T rounded up to a multiple of 128][n_heads][128] (rows >= T are padding: read, never used; out rows >= T
 * are not written).  Pool positions T .. (T rounded up to 128) - 1 that fall in a mapped page are read with weight zero
 * and must hold finite values.  K0 / V0 (the native step's keys and values, RoPE already applied): a paged pool
 * [num_pages][n_kv_heads][page_size][128] bf16 with page_table int32 [pages_per_seq] (position p lives in page
 * page_table[p / page_size]); page_size 16, 32 or 64.  k_diag / v_diag: bf16 [n_steps][T][n_kv_heads][128], the keys and
 * values each simulated step produced at every position (may be NULL when n_steps is 0: plain causal attention);
 * n_steps <= 8.  lse: optional float [T * n_heads], the natural-log normaliser of every row (what a backward pass needs).
 * scratch: spec_ttt_attention_scratch_bytes(...) bytes of device memory.  head_dim must be 128 (SPEC_ERR_UNSUPPORTED
 * otherwise).  The dense causal part runs on the tcgen05 tile kernel of the tree attention; the backward pass is not
 * part of this library. */
size_t spec_ttt_attention_scratch_bytes(int32_t T, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim);
int spec_ttt_attention(const void *q, const void *k_pool, const void *v_pool, const int32_t *page_table, int32_t pages_per_seq,
                       int32_t page_size, const void *k_diag, const void *v_diag, int32_t n_steps, void *out, float *lse,
                       int32_t T, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void *scratch, void *stream);

/* Per-row log-softmax + top-K (value desc, index asc) over fp32 logits [rows][n]: the expansion
 * step of the dynamic tree (Section 2.2; Appendix A "nodes during the expansion phase").  K <= 16.
 * out_idx int32 [rows][K], out_lp float [rows][K].  scratch: device buffer of
 * spec_topk_scratch_bytes(rows, n, K) bytes for the two-stage kernel (chunk candidates, then a per-row merge; the step
 * itself takes its candidates from the draft LM head's epilogue, see spec_gemm_topk); NULL selects the plain
 * one-CTA-per-row kernel. */
size_t spec_topk_scratch_bytes(int32_t rows, int32_t n, int32_t K);
int spec_logsoftmax_topk(const float *logits, int32_t rows, int32_t n, int32_t K, int32_t *out_idx, float *out_lp,
                         void *scratch, void *stream);
/* Per-row argmax (lowest index on ties) over fp32 [rows][n]. */
int spec_argmax(const float *logits, int32_t rows, int32_t n, int32_t *out_idx, void *stream);

#ifdef __cplusplus
}
#endif
#endif
