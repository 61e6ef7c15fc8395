// C ABI of the speculative-step library: configuration checks, workspace carving, the kernel
// schedule of prefill / spec_step / plain decode, and the inspection entry points.
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>
#include <string>
#include <vector>

#include "../../include/spec_b200.h"
#include "tma_maps.cuh"
#include "gemm_fused.cuh"
#include "attn_fast.cuh"
#include "state.cuh"

using namespace spec;

namespace spec {
thread_local bool tl_pdl = false;
thread_local int tl_launch_budget = -1;

void launch_logsoftmax_topk_rows(const float *logits, const int32_t *src_row, int rows, int n, int K, int32_t *idx,
                                 float *lp, cudaStream_t s);

// dst row b*dst_stride_rows <- src row src_row[b] (fp32, `width` columns); rows with src_row < 0 are skipped
__global__ void gather_rows_kernel(const float *__restrict__ src, const int32_t *__restrict__ src_row,
                                   float *__restrict__ dst, int width, int dst_stride_rows) {
  pdl_wait();
  pdl_trigger();
  int b = blockIdx.x, sr = src_row[b];
  if (sr < 0) return;
  for (int i = threadIdx.x; i < width; i += blockDim.x)
    dst[(size_t)b * dst_stride_rows * width + i] = src[(size_t)sr * width + i];
}
static void launch_gather_rows(const float *src, const int32_t *src_row, float *dst, int B, int width, int dst_stride_rows,
                               cudaStream_t s) {
  launch_k(gather_rows_kernel, dim3(B), dim3(256), 0, s, src, src_row, dst, width, dst_stride_rows);
}
}

static char g_init_err[256] = "";

constexpr int MAX_STAMPS = 1024;   // stamped launches of one step (profiling aid)

struct LayerW {
  const void *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
};

// Bump allocator over the caller's workspace; with base == nullptr it only measures.
struct Carver {
  char *base;
  size_t off = 0;
  explicit Carver(void *b) : base((char *)b) {}
  template <typename U> U *take(size_t n) {
    off = (off + 255) & ~(size_t)255;
    U *p = base ? (U *)(base + off) : nullptr;
    off += n * sizeof(U);
    return p;
  }
  void *take_bytes(size_t n) { return take<char>(n); }
};

struct spec_ctx {
  spec_cfg cfg;
  cudaStream_t stream;
  int B, L, k, H, G, hd, F, V, Vd, D, K, N, Pmax, pool, esz;
  int Te, Td, Tv, R, Ralloc, pps, tail_tree, need_pos;
  std::vector<LayerW> tl;
  LayerW dl;
  const void *embed, *final_norm, *lm_head, *fc3, *fc2, *dfinal_norm, *dlm_head;
  const int32_t *d2t;
  // device buffers
  float *x, *proj, *qkv, *gu, *logits;
  void *h, *q, *ao, *act, *cat, *node_taps, *pend_taps;
  float2 *cs;
  double *inv_freq;
  RowMeta meta;
  std::vector<KvPool> pools;   // [L] target, [L] = draft
  KvPool *pools_dev;
  int32_t *page_table;
  SeqState st;
  TreeBufs tb;
  int32_t *status;
  float *cap_logits, *cap_a;   // capture buffers (SPEC_FLAG_CAPTURE)
  // fused bf16 path: GEMM epilogues do the norm / RoPE / activation / residual / argmax work
  bool fused = false;
  float *ssq = nullptr;        // [ceil(k/128)][Ralloc] per-tile sums of squares of the residual stream
  float *best_val = nullptr;   // [ceil(V/128)][Ralloc] per-tile argmax candidates of the target LM head
  int32_t *best_idx = nullptr;
  void *topk_scratch = nullptr;
  int ktiles = 0, vtiles = 0, dtiles = 0;
  // per-tile candidates of the draft LM head (fused path): [dtiles][Ralloc][K] values / indices, [dtiles][Ralloc] max / sum
  float *cand_val = nullptr, *cand_max = nullptr, *cand_sum = nullptr;
  int32_t *cand_idx = nullptr;
  bool tree_fused = false;     // one launch between two draft passes (merge + expansion + next pass's inputs)
  // profiling aid (SPEC_FLAG_STAMPS): per stamped launch {earliest "inputs ready" time, latest CTA exit} in globaltimer ns
  unsigned long long *stamps = nullptr;      // [MAX_STAMPS][2]
  std::vector<int> stamp_cls;                // class of each stamped launch of the last scheduled step
  int stamp_n = 0;
  int dbg_launch_budget = -1;   // debugging aid: kernels of the next step to run (-1: all)
  int dbg_withhold_spin = 0;    // test hook: > 0 makes one CTA of the verify LM-head GEMM run a bounded wait out after that many polls
  void *attn_scratch;
  size_t attn_scratch_bytes;
  // partial-sum bookkeeping of the plain (fp32 / debug) schedule: its GEMMs write one slice
  int np_proj = 1, np_qkv = 1, np_gu = 1;
  size_t ps_proj = 0, ps_qkv = 0, ps_gu = 0;
  // host mirrors
  std::vector<int32_t> n_upper, cap_host, n_pages_host;
  std::vector<int32_t> page_table_host;
  bool prefilled = false, draft_stale = false;
  cudaGraphExec_t graph = nullptr;
  cudaGraphExec_t graph_sampled = nullptr;   // the same step with the stochastic acceptance kernel
  int launches = 0, launches_graph = 0, launches_graph_sampled = 0;
  bool sampled = false;        // the step being scheduled ends with the stochastic acceptance
  float *u_dev = nullptr;      // [B][2N] uniforms of the sampled step, then 1 / temperature
  int32_t *prompt_dev = nullptr;   // [B * max_ctx] the prompts of the prefill being run, concatenated
  int sched_err = 0;
  int cur_rps = 1;             // rows per sequence of the pass being scheduled
  int ctx_hint = -1;           // prefill: context length of the pass being scheduled (sizes the key split); -1: from n_upper
  bool prof = false;
  std::vector<cudaEvent_t> prof_ev;
  std::vector<int> prof_cls;
  int prof_n = 0;
  TmaMaps *fg = nullptr;
  char err[256];
};

static int fail(spec_ctx *c, int code, const char *fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(c ? c->err : g_init_err, 256, fmt, ap);
  va_end(ap);
  return code;
}
#define CUDA_TRY(c, call)                                                                       \
  do {                                                                                          \
    cudaError_t e_ = (call);                                                                    \
    if (e_ != cudaSuccess) return fail(c, SPEC_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

static const char *check_cfg(const spec_cfg *c) {
  if (c->dtype != SPEC_F32 && c->dtype != SPEC_BF16) return "dtype must be 0 (fp32) or 1 (bf16)";
  if (c->n_layers < 1 || c->n_layers > 1024) return "n_layers out of range";
  if (c->hidden < 16 || c->hidden % 8) return "hidden must be a positive multiple of 8";
  if (c->n_heads < 1 || c->n_kv_heads < 1 || c->n_heads % c->n_kv_heads) return "n_heads must be a multiple of n_kv_heads";
  if (c->head_dim < 16 || c->head_dim > 256 || c->head_dim % 16) return "head_dim must be a multiple of 16 in [16,256]";
  if (c->ffn < 8 || c->ffn % 8) return "ffn must be a positive multiple of 8";
  if (c->vocab < 2 || c->draft_vocab < 1 || c->draft_vocab > c->vocab) return "vocab / draft_vocab out of range";
  for (int i = 0; i < 3; i++)
    if (c->fuse_layers[i] < 0 || c->fuse_layers[i] >= c->n_layers) return "fuse_layers must index target layers";
  if (!(c->rope_theta > 1.0f) || !(c->rms_eps > 0.0f)) return "rope_theta must exceed 1 and rms_eps must be positive";
  if (c->batch < 1 || c->batch > 4096) return "batch out of range";
  if (c->tree_depth < 1 || c->tree_depth > 16) return "tree_depth must be in [1,16]";
  if (c->tree_topk < 1 || c->tree_topk > 16 || c->tree_topk > c->draft_vocab) return "tree_topk must be in [1,16] and <= draft_vocab";
  if (c->tree_nodes < 1 || c->tree_nodes > 64) return "tree_nodes must be in [1,64]";
  if ((c->tree_depth - 1) * c->tree_topk > 128) return "(tree_depth-1)*tree_topk must be <= 128 (draft ancestor mask)";
  if (c->tree_topk + (c->tree_depth - 1) * c->tree_topk * c->tree_topk > 1023) return "candidate pool must be <= 1023";
  if (c->page_size < 1 || c->page_size > 256 || (c->page_size & (c->page_size - 1))) return "page_size must be a power of two <= 256";
  if (c->max_ctx < 2 || c->max_ctx > (1 << 22)) return "max_ctx out of range";
  if (c->num_pages < 1) return "num_pages must be positive";
  return nullptr;
}

// Prompt positions per prefill pass.  A pass holds PREFILL_CHUNK / PREFILL_BLOCK blocks of PREFILL_BLOCK positions: the
// rows of a block are each other's tail keys (causal through the two-word masks), and the blocks before it, whose K/V
// the same pass's QKV epilogue has already written, are plain context.  The widest GEMM tile (256 rows) streams every
// weight once per 256 prompt positions.
constexpr int PREFILL_CHUNK = 256;
constexpr int PREFILL_BLOCK = 128;

// Derives sizes and carves every buffer; with c->cfg.workspace == nullptr (measure mode) only sizes.
static size_t carve(spec_ctx *c, void *base) {
  const spec_cfg &g = c->cfg;
  c->B = g.batch; c->L = g.n_layers; c->k = g.hidden; c->H = g.n_heads; c->G = g.n_kv_heads; c->hd = g.head_dim;
  c->F = g.ffn; c->V = g.vocab; c->Vd = g.draft_vocab; c->D = g.tree_depth; c->K = g.tree_topk; c->N = g.tree_nodes;
  c->Pmax = c->D + 1;
  c->pool = c->K + (c->D - 1) * c->K * c->K;
  c->esz = g.dtype == SPEC_F32 ? 4 : 2;
  c->Te = c->B * c->Pmax; c->Td = c->B * c->K; c->Tv = c->B * c->N;
  c->R = std::max(std::max(c->Te, c->Td), std::max(c->Tv, PREFILL_CHUNK));
  c->Ralloc = (c->R + 63) / 64 * 64;
  c->pps = (g.max_ctx + g.page_size - 1) / g.page_size;
  c->tail_tree = std::max(1, (c->D - 1) * c->K);
  c->need_pos = std::max(c->N, c->tail_tree) + 1;
  int B = c->B, k = c->k, R = c->Ralloc, qd = c->H * c->hd, qkvd = (c->H + 2 * c->G) * c->hd;
  size_t e = c->esz;
  Carver cv(base);
  c->x = cv.take<float>((size_t)R * k);
  c->proj = cv.take<float>((size_t)R * k);
  c->qkv = cv.take<float>((size_t)R * qkvd);
  c->gu = cv.take<float>((size_t)R * 2 * c->F);
  c->logits = cv.take<float>((size_t)R * std::max(c->V, c->Vd));
  c->h = cv.take_bytes((size_t)R * k * e);
  c->q = cv.take_bytes((size_t)R * qd * e);
  c->ao = cv.take_bytes((size_t)R * qd * e);
  c->act = cv.take_bytes((size_t)R * c->F * e);
  c->cat = cv.take_bytes((size_t)R * 2 * k * e);
  c->node_taps = cv.take_bytes((size_t)R * 3 * k * e);
  c->pend_taps = cv.take_bytes((size_t)R * 3 * k * e);
  c->cs = cv.take<float2>((size_t)R * (c->hd / 2));
  c->inv_freq = cv.take<double>(c->hd / 2);
  c->meta.seq = cv.take<int32_t>(R); c->meta.pos = cv.take<int32_t>(R); c->meta.kvpos = cv.take<int32_t>(R);
  c->meta.ctx = cv.take<int32_t>(R); c->meta.tail_base = cv.take<int32_t>(R); c->meta.tok = cv.take<int32_t>(R);
  c->meta.mask_lo = cv.take<uint64_t>(R); c->meta.mask_hi = cv.take<uint64_t>(R);
  size_t pool_elems = (size_t)g.num_pages * c->G * g.page_size * c->hd;
  c->pools.resize(c->L + 1);
  for (int l = 0; l <= c->L; l++) {
    c->pools[l].k = cv.take_bytes(pool_elems * e);
    c->pools[l].v = cv.take_bytes(pool_elems * e);
  }
  c->pools_dev = cv.take<KvPool>(c->L + 1);
  c->page_table = cv.take<int32_t>((size_t)B * c->pps);
  c->st.n = cv.take<int32_t>(B); c->st.n_prev = cv.take<int32_t>(B); c->st.P = cv.take<int32_t>(B);
  c->st.root = cv.take<int32_t>(B); c->st.cap = cv.take<int32_t>(B); c->st.last_row = cv.take<int32_t>(B);
  c->st.active = cv.take<int32_t>(B);
  c->st.order = cv.take<int32_t>(B);
  TreeBufs &t = c->tb;
  t.pool = c->pool; t.K = c->K; t.D = c->D; t.N = c->N; t.Pmax = c->Pmax;
  size_t pe = (size_t)B * (c->pool + 1);
  t.pool_tok = cv.take<int32_t>(pe); t.pool_parent = cv.take<int32_t>(pe); t.pool_depth = cv.take<int32_t>(pe);
  t.pool_score = cv.take<float>(pe);
  t.frontier = cv.take<int32_t>((size_t)B * c->D * c->K);
  t.front_cur = cv.take<int32_t>((size_t)B * c->K);
  t.feat_row = cv.take<int32_t>(R);
  t.tk_idx = cv.take<int32_t>((size_t)R * c->K); t.tk_lp = cv.take<float>((size_t)R * c->K);
  size_t ne = (size_t)std::max(B * c->N, R);
  t.tok = cv.take<int32_t>(ne); t.parent = cv.take<int32_t>(ne); t.depth = cv.take<int32_t>(ne);
  t.poolidx = cv.take<int32_t>(ne); t.score = cv.take<float>(ne); t.mask = cv.take<uint64_t>(ne);
  t.nn = cv.take<int32_t>(B); t.y = cv.take<int32_t>(ne);
  t.path = cv.take<int32_t>((size_t)B * c->Pmax); t.out_ids = cv.take<int32_t>((size_t)B * c->Pmax);
  t.out_cnt = cv.take<int32_t>(B); t.pend_tok = cv.take<int32_t>((size_t)B * c->Pmax);
  c->u_dev = cv.take<float>((size_t)B * 2 * c->N + 1);
  c->prompt_dev = cv.take<int32_t>((size_t)B * g.max_ctx + 1);
  c->status = cv.take<int32_t>(8);
  if (g.flags & SPEC_FLAG_CAPTURE) {
    c->cap_logits = cv.take<float>((size_t)c->D * c->Td * c->Vd);
    c->cap_a = cv.take<float>((size_t)c->D * c->Td * k);
  } else {
    c->cap_logits = c->cap_a = nullptr;
  }
  c->ktiles = (k + 127) / 128; c->vtiles = (c->V + 127) / 128;
  c->ssq = cv.take<float>((size_t)c->ktiles * R);
  c->best_val = cv.take<float>((size_t)c->vtiles * R);
  c->best_idx = cv.take<int32_t>((size_t)c->vtiles * R);
  c->topk_scratch = cv.take_bytes(topk_scratch_bytes(R, c->Vd, c->K));
  c->dtiles = (c->Vd + 127) / 128;
  const size_t cld = (size_t)draft_tree_cand_ld(c->dtiles);
  c->cand_val = cv.take<float>(cld * R * c->K);
  c->cand_idx = cv.take<int32_t>(cld * R * c->K);
  c->cand_max = cv.take<float>(cld * R);
  c->cand_sum = cv.take<float>(cld * R);
  c->stamps = (g.flags & SPEC_FLAG_STAMPS) ? cv.take<unsigned long long>((size_t)MAX_STAMPS * 2) : nullptr;
  c->attn_scratch_bytes = attn_fast_scratch_bytes(R, c->H, c->hd, g.max_ctx);
  c->attn_scratch = cv.take_bytes(c->attn_scratch_bytes);
  return (cv.off + 255) & ~(size_t)255;
}

extern "C" size_t spec_workspace_bytes(const spec_cfg *cfg) {
  if (!cfg || check_cfg(cfg)) return 0;
  spec_ctx tmp;
  tmp.cfg = *cfg;
  return carve(&tmp, nullptr);
}

extern "C" const char *spec_last_error(const spec_ctx *ctx) { return ctx ? ctx->err : g_init_err; }

extern "C" int spec_init(spec_ctx **out, const spec_target_weights *tw, const spec_draft_weights *dw, const spec_cfg *cfg) {
  if (out) *out = nullptr;
  if (!out || !tw || !dw || !cfg) return fail(nullptr, SPEC_ERR_NULL, "spec_init: NULL argument");
  if (const char *why = check_cfg(cfg)) return fail(nullptr, SPEC_ERR_INVALID_CFG, "spec_init: %s", why);
  if (!cfg->workspace) return fail(nullptr, SPEC_ERR_NULL, "spec_init: workspace is NULL");
  if ((uintptr_t)cfg->workspace & 255) return fail(nullptr, SPEC_ERR_WORKSPACE, "spec_init: workspace must be 256-byte aligned");
  const void *req[] = {tw->embed, tw->final_norm, tw->lm_head, tw->attn_norm, tw->wq, tw->wk, tw->wv, tw->wo, tw->mlp_norm,
                       tw->w_gate, tw->w_up, tw->w_down, dw->fc3, dw->fc2, dw->attn_norm, dw->wq, dw->wk, dw->wv, dw->wo,
                       dw->mlp_norm, dw->w_gate, dw->w_up, dw->w_down, dw->final_norm, dw->lm_head, dw->d2t};
  for (const void *p : req)
    if (!p) return fail(nullptr, SPEC_ERR_NULL, "spec_init: a weight pointer is NULL");
  spec_ctx *c = new spec_ctx();
  c->cfg = *cfg;
  c->err[0] = 0;
  c->stream = (cudaStream_t)cfg->stream;
  size_t need = carve(c, cfg->workspace);
  if (need > cfg->workspace_bytes) {
    delete c;
    return fail(nullptr, SPEC_ERR_WORKSPACE, "spec_init: workspace has %zu bytes, %zu needed", cfg->workspace_bytes, need);
  }
  for (int l = 0; l < c->L; l++) {
    LayerW w = {tw->attn_norm[l], tw->wq[l], tw->wk[l], tw->wv[l], tw->wo[l], tw->mlp_norm[l], tw->w_gate[l], tw->w_up[l], tw->w_down[l]};
    const void *ps[] = {w.attn_norm, w.wq, w.wk, w.wv, w.wo, w.mlp_norm, w.w_gate, w.w_up, w.w_down};
    for (const void *p : ps)
      if (!p) { delete c; return fail(nullptr, SPEC_ERR_NULL, "spec_init: layer %d has a NULL weight", l); }
    c->tl.push_back(w);
  }
  c->dl = LayerW{dw->attn_norm, dw->wq, dw->wk, dw->wv, dw->wo, dw->mlp_norm, dw->w_gate, dw->w_up, dw->w_down};
  c->embed = tw->embed; c->final_norm = tw->final_norm; c->lm_head = tw->lm_head;
  c->fc3 = dw->fc3; c->fc2 = dw->fc2; c->dfinal_norm = dw->final_norm; c->dlm_head = dw->lm_head; c->d2t = dw->d2t;
  cudaStream_t s = c->stream;
  cudaError_t e = cudaMemsetAsync(cfg->workspace, 0, need, s);
  std::vector<double> inv(c->hd / 2);
  for (int i = 0; i < c->hd / 2; i++) inv[i] = pow((double)cfg->rope_theta, -2.0 * (double)i / (double)c->hd);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->inv_freq, inv.data(), inv.size() * 8, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->pools_dev, c->pools.data(), sizeof(KvPool) * (c->L + 1), cudaMemcpyHostToDevice, s);
  std::vector<int32_t> ident(c->B);
  for (int b = 0; b < c->B; b++) ident[b] = b;
  if (e == cudaSuccess) e = cudaMemcpyAsync(c->st.order, ident.data(), sizeof(int32_t) * c->B, cudaMemcpyHostToDevice, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) {
    int rc = fail(nullptr, SPEC_ERR_CUDA, "spec_init: %s", cudaGetErrorString(e));
    delete c;
    return rc;
  }
  c->n_upper.assign(c->B, 0); c->cap_host.assign(c->B, 0); c->n_pages_host.assign(c->B, 0);
  c->page_table_host.assign((size_t)c->B * c->pps, 0);
  if (cfg->dtype == SPEC_BF16 && !((cfg->flags & SPEC_FLAG_REF_GEMM))) {
    std::string why;
    c->fg = tma_maps_create(why);
    if (!c->fg) {
      int rc = fail(nullptr, SPEC_ERR_CUDA, "spec_init: tcgen05 GEMM set-up failed: %s", why.c_str());
      delete c;
      return rc;
    }
  }
  c->fused = c->fg != nullptr;
  c->tree_fused = c->fused && draft_tree_step_smem(c->dtiles, c->K) > 0;
  if (c->fg && !(c->hd <= 128 && (c->hd & (c->hd - 1)) == 0)) {
    int rc = fail(nullptr, SPEC_ERR_UNSUPPORTED, "spec_init: the bf16 tensor-core path takes a power-of-two head_dim <= 128 (got %d)", c->hd);
    tma_maps_destroy(c->fg);
    delete c;
    return rc;
  }
  if (c->fg && c->R > 256) {
    int rc = fail(nullptr, SPEC_ERR_UNSUPPORTED, "spec_init: %d rows per pass exceed the 256 the tensor-core GEMM takes", c->R);
    tma_maps_destroy(c->fg);
    delete c;
    return rc;
  }
  *out = c;
  return SPEC_OK;
}

extern "C" int spec_free(spec_ctx *c) {
  if (!c) return SPEC_OK;
  if (c->graph) cudaGraphExecDestroy(c->graph);
  if (c->graph_sampled) cudaGraphExecDestroy(c->graph_sampled);
  if (c->fg) tma_maps_destroy(c->fg);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  delete c;
  return SPEC_OK;
}

// ------------------------------------------------------------------------------------------ schedule
template <typename T> struct Sched {
  spec_ctx *c;
  cudaStream_t s;
  explicit Sched(spec_ctx *ctx) : c(ctx), s(ctx->stream) { tl_pdl = c->fused && !(c->cfg.flags & SPEC_FLAG_NO_PDL); }
  ~Sched() { tl_pdl = false; }
  Sched(const Sched &) = delete;
  void tick(int n = 1) { c->launches += n; }
  // profiling: one event at the start of every launch; the interval to the next event is charged to `cls`
  void mark(int cls) { prof_mark(cls); }
  // profiling aid: the next stamped launch's slot (nullptr when stamps are off or the step has more launches than slots)
  unsigned long long *next_stamp(int cls) {
    if (!c->stamps || c->stamp_n >= MAX_STAMPS) return nullptr;
    c->stamp_cls.push_back(cls);
    return c->stamps + 2 * (size_t)c->stamp_n++;
  }
  void prof_mark(int cls) {
    if (!c->prof) return;
    if (c->prof_n >= (int)c->prof_ev.size()) {
      cudaEvent_t e;
      cudaEventCreate(&e);
      c->prof_ev.push_back(e);
      c->prof_cls.push_back(0);
    }
    cudaEventRecord(c->prof_ev[c->prof_n], s);
    c->prof_cls[c->prof_n] = cls;
    c->prof_n++;
  }

  // number of split-K slices for a weight of shape [O][I] whose output buffer holds smax slices
  int pick(int, int, int) const { return 1; }
  size_t pstride(int ldo) const { return (size_t)c->Ralloc * ldo; }

  // S fp32 partial slices of x . w^T into columns [col0, col0+O) of `out` (row pitch ldo)
  void gemm(const void *x, const void *w, float *out, int rows, int O, int I, int ldo, int col0, int S) {
    mark(SPEC_PROF_GEMM);
    (void)S;
    launch_gemm_ref<T>((const T *)x, (const T *)w, out + col0, rows, O, I, ldo, s);
    tick();
  }

  // ---- fused bf16 path -----------------------------------------------------------------------
  FusedGemmArgs fargs(const void *x, int rows, int I) const {
    FusedGemmArgs a;
    a.x = (const bf16 *)x; a.rows = rows; a.I = I; a.status = c->status; a.pdl = tl_pdl;
    return a;
  }
  // the GEMM input is bf16(residual * gain): apply the RMSNorm factor of the residual as a row scale
  void with_norm_scale(FusedGemmArgs &a) const {
    a.ssq_in = c->ssq; a.ssq_in_tiles = c->ktiles; a.ssq_ld = c->Ralloc; a.k_in = c->k; a.eps = c->cfg.rms_eps;
  }
  void fgemm(FusedEpi epi, FusedGemmArgs a) {
    prof_mark(SPEC_PROF_GEMM);
    a.stamp = next_stamp(SPEC_PROF_GEMM);
    int rc = fused_gemm_launch(c->fg, epi, a, s);
    if (rc && !c->sched_err) c->sched_err = rc;
    tick();
  }
  // residual-producing GEMM: x (+)= in . w^T, h = bf16(x * gain), ssq, optional taps
  void fgemm_resid(const void *in, int I, const void *w, int rows, bool add, const void *gain, int tap_mask) {
    FusedGemmArgs a = fargs(in, rows, I);
    a.w[0] = (const bf16 *)w; a.O[0] = c->k; a.nw = 1;
    a.xres = c->x; a.gain = (const bf16 *)gain; a.hb = (bf16 *)c->h; a.ssq_out = c->ssq; a.ssq_ld = c->Ralloc;
    a.taps = (bf16 *)c->node_taps; a.tap_mask = tap_mask; a.resid_add = add ? 1 : 0;
    fgemm(EPI_RESID, a);
  }
  void block_fused(const LayerW &w, KvPool pool, int rows, int tail_len, const void *next_gain, int tap_mask) {
    int k = c->k, qd = c->H * c->hd, kvd = c->G * c->hd, F = c->F;
    FusedGemmArgs a = fargs(c->h, rows, k);
    a.w[0] = (const bf16 *)w.wq; a.w[1] = (const bf16 *)w.wk; a.w[2] = (const bf16 *)w.wv;
    a.O[0] = qd; a.O[1] = kvd; a.O[2] = kvd; a.nw = 3;
    with_norm_scale(a);
    a.cs = c->cs; a.m = c->meta; a.q = (bf16 *)c->q; a.pool = pool;
    a.pm = PageMap{c->page_table, c->pps, c->cfg.page_size, c->cfg.num_pages};
    a.H = c->H; a.G = c->G; a.hd = c->hd;
    fgemm(EPI_QKV, a);
    attention(pool, rows, tail_len);
    fgemm_resid(c->ao, qd, w.wo, rows, true, w.mlp_norm, 0);
    FusedGemmArgs g = fargs(c->h, rows, k);
    g.w[0] = (const bf16 *)w.w_gate; g.w[1] = (const bf16 *)w.w_up; g.O[0] = F; g.O[1] = F; g.nw = 2;
    with_norm_scale(g);
    g.act = (bf16 *)c->act;
    fgemm(EPI_SWIGLU, g);
    fgemm_resid(c->act, F, w.w_down, rows, true, next_gain, tap_mask);
  }
  void target_forward_fused(int rows, int tail_len, bool want_logits) {
    mark(SPEC_PROF_MISC); launch_rope_table(c->meta.pos, rows, c->hd / 2, c->inv_freq, c->cs, s); tick();
    mark(SPEC_PROF_MISC);
    launch_embed_norm((const bf16 *)c->embed, c->meta.tok, (const bf16 *)c->tl[0].attn_norm, c->x, (bf16 *)c->h, c->ssq, rows, c->k,
                      c->Ralloc, s);
    tick();
    for (int l = 0; l < c->L; l++)
      block_fused(c->tl[l], c->pools[l], rows, tail_len, l + 1 < c->L ? c->tl[l + 1].attn_norm : c->final_norm, tap_mask_of(l));
    if (want_logits) {
      FusedGemmArgs a = fargs(c->h, rows, c->k);
      a.w[0] = (const bf16 *)c->lm_head; a.O[0] = c->V; a.nw = 1;
      with_norm_scale(a);
      a.best_val = c->best_val; a.best_idx = c->best_idx; a.best_ld = c->Ralloc;
      if (c->cap_logits || c->sampled) { a.out_f32 = c->logits; a.ldo = c->V; }
      if (c->dbg_withhold_spin > 0) { a.withhold = true; a.spin_limit = (unsigned)c->dbg_withhold_spin; }
      fgemm(EPI_ARGMAX, a);
      mark(SPEC_PROF_ARGMAX); launch_argmax_merge(c->best_val, c->best_idx, c->vtiles, c->Ralloc, rows, c->tb.y, s); tick();
    }
  }
  void fuse_fused(const void *taps, int rows) {
    FusedGemmArgs a = fargs(taps, rows, 3 * c->k);
    a.w[0] = (const bf16 *)c->fc3; a.O[0] = c->k; a.nw = 1;
    a.out_f32 = c->proj; a.ldo = c->k;
    fgemm(EPI_F32, a);
    c->np_proj = 1; c->ps_proj = 0;
  }
  // prebuilt: the launch that closed the previous draft pass already wrote this pass's FC2 input and RoPE angles
  void draft_forward_fused(const float *feat, int nparts, size_t fstride, const int32_t *src_row, int rows, int tail_len,
                           bool prebuilt = false) {
    if (!prebuilt) {
      mark(SPEC_PROF_MISC); launch_rope_table(c->meta.pos, rows, c->hd / 2, c->inv_freq, c->cs, s); tick();
      mark(SPEC_PROF_MISC);
      launch_build_cat<bf16>(feat, nparts, fstride, src_row, (const bf16 *)c->embed, c->meta.tok, c->meta.seq, (bf16 *)c->cat, rows, c->k, s);
      tick();
    }
    fgemm_resid(c->cat, 2 * c->k, c->fc2, rows, false, c->dl.attn_norm, 0);
    block_fused(c->dl, c->pools[c->L], rows, tail_len, c->dfinal_norm, 0);
  }
  void draft_logits_fused(int rows) {
    FusedGemmArgs a = fargs(c->h, rows, c->k);
    a.w[0] = (const bf16 *)c->dlm_head; a.O[0] = c->Vd; a.nw = 1;
    with_norm_scale(a);
    a.out_f32 = c->logits; a.ldo = c->Vd;
    fgemm(EPI_F32, a);
  }
  // draft LM head whose epilogue leaves per-tile softmax statistics and top-K candidates (the logits themselves are
  // written only when they are captured for inspection)
  void draft_logits_topk(int rows, const int32_t *want_rows, int n_want) {
    FusedGemmArgs a = fargs(c->h, rows, c->k);
    a.w[0] = (const bf16 *)c->dlm_head; a.O[0] = c->Vd; a.nw = 1;
    with_norm_scale(a);
    if (c->cap_logits) { a.out_f32 = c->logits; a.ldo = c->Vd; }
    a.topk = c->K; a.cand_val = c->cand_val; a.cand_idx = c->cand_idx; a.cand_max = c->cand_max; a.cand_sum = c->cand_sum;
    a.cand_ld = draft_tree_cand_ld(c->dtiles); a.want_rows = want_rows; a.n_want = n_want;
    fgemm(EPI_TOPK, a);
  }
  void tree_step(int pass) {
    mark(SPEC_PROF_TREE);
    int rc = launch_draft_tree_step(c->st, c->tb, c->meta, c->d2t, pass, c->cand_val, c->cand_idx, c->cand_max, c->cand_sum, c->dtiles,
                                    draft_tree_cand_ld(c->dtiles), c->x, (const bf16 *)c->embed, (bf16 *)c->cat, c->k, c->inv_freq, c->cs, c->hd / 2, c->B, s);
    if (rc && !c->sched_err) c->sched_err = rc;
    tick();
  }
  void topk(const int32_t *src_row, int rows) {
    mark(SPEC_PROF_TOPK);
    if (c->fused) tick(launch_topk2(c->logits, src_row, rows, c->Vd, c->K, c->tb.tk_idx, c->tb.tk_lp, c->topk_scratch, s));
    else { launch_logsoftmax_topk_rows(c->logits, src_row, rows, c->Vd, c->K, c->tb.tk_idx, c->tb.tk_lp, s); tick(); }
  }

  void attention(KvPool pool, int rows, int tail_len) {
    mark(SPEC_PROF_ATTN);
    PageMap pm{c->page_table, c->pps, c->cfg.page_size, c->cfg.num_pages};
    bool fast = c->cfg.dtype == SPEC_BF16 && !(c->cfg.flags & SPEC_FLAG_REF_ATTN) && attn_fast_supported(c->hd, c->H / c->G);
    if (fast) {
      int hint = std::max(0, c->ctx_hint);
      if (c->ctx_hint < 0)
        for (int b = 0; b < c->B; b++) hint = std::max(hint, c->n_upper[b]);
      tick(launch_attn_fast((const bf16 *)c->q, pool, pm, c->meta, tail_len, (bf16 *)c->ao, rows, c->H, c->G, c->hd,
                            c->cur_rps, hint, c->attn_scratch, s, !(c->cfg.flags & SPEC_FLAG_NO_TMA_ATTN), c->status,
                            c->st.order, c->B, next_stamp(SPEC_PROF_ATTN)));
    } else {
      launch_attn_ref<T>((const T *)c->q, pool, pm, c->meta, tail_len, (T *)c->ao, rows, c->H, c->G, c->hd,
                         c->cfg.max_ctx + tail_len, s);
      tick();
    }
  }

  // One decoder block on `rows` rows described by c->meta.  first_mode: how the residual stream is
  // formed from the pending partial sums (0 keep, 1 set, 2 add); tap_mask: taps of the previous block.
  void block(const LayerW &w, KvPool pool, int rows, int tail_len, int first_mode, int tap_mask) {
    int k = c->k, qd = c->H * c->hd, kvd = c->G * c->hd, qkvd = qd + 2 * kvd, F = c->F;
    PageMap pm{c->page_table, c->pps, c->cfg.page_size, c->cfg.num_pages};
    mark(SPEC_PROF_NORM); launch_add_norm<T>(c->x, c->proj, c->np_proj, c->ps_proj, first_mode, (T *)c->node_taps, tap_mask, (const T *)w.attn_norm,
                       c->cfg.rms_eps, (T *)c->h, nullptr, rows, rows, k, s);
    tick();
    c->np_qkv = pick(qd, k, 1); c->ps_qkv = pstride(qkvd);
    gemm(c->h, w.wq, c->qkv, rows, qd, k, qkvd, 0, c->np_qkv);
    gemm(c->h, w.wk, c->qkv, rows, kvd, k, qkvd, qd, c->np_qkv);
    gemm(c->h, w.wv, c->qkv, rows, kvd, k, qkvd, qd + kvd, c->np_qkv);
    mark(SPEC_PROF_ROPE_KV); launch_rope_kv<T>(c->qkv, c->np_qkv, c->ps_qkv, c->cs, c->meta, (T *)c->q, pool, pm, rows, c->H, c->G, c->hd, c->status, s);
    tick();
    attention(pool, rows, tail_len);
    c->np_proj = pick(k, qd, 1); c->ps_proj = pstride(k);
    gemm(c->ao, w.wo, c->proj, rows, k, qd, k, 0, c->np_proj);
    mark(SPEC_PROF_NORM); launch_add_norm<T>(c->x, c->proj, c->np_proj, c->ps_proj, 2, (T *)nullptr, 0, (const T *)w.mlp_norm, c->cfg.rms_eps,
                       (T *)c->h, nullptr, rows, rows, k, s);
    tick();
    c->np_gu = pick(F, k, 1); c->ps_gu = pstride(2 * F);
    gemm(c->h, w.w_gate, c->gu, rows, F, k, 2 * F, 0, c->np_gu);
    gemm(c->h, w.w_up, c->gu, rows, F, k, 2 * F, F, c->np_gu);
    mark(SPEC_PROF_ACT); launch_silu_mul<T>(c->gu, c->np_gu, c->ps_gu, (T *)c->act, rows, F, s);
    tick();
    c->np_proj = pick(k, F, 1); c->ps_proj = pstride(k);
    gemm(c->act, w.w_down, c->proj, rows, k, F, k, 0, c->np_proj);
  }

  int tap_mask_of(int layer) const {
    int m = 0;
    for (int i = 0; i < 3; i++) m |= (c->cfg.fuse_layers[i] == layer) ? (1 << i) : 0;
    return m;
  }

  // target forward over the rows of c->meta: taps -> node_taps, argmax -> tb.y
  void target_forward(int rows, int tail_len, bool want_logits) {
    if (c->fused) return target_forward_fused(rows, tail_len, want_logits);
    mark(SPEC_PROF_MISC); launch_rope_table(c->meta.pos, rows, c->hd / 2, c->inv_freq, c->cs, s); tick();
    mark(SPEC_PROF_MISC); launch_embed<T>((const T *)c->embed, c->meta.tok, c->x, rows, c->k, s); tick();
    for (int l = 0; l < c->L; l++)
      block(c->tl[l], c->pools[l], rows, tail_len, l == 0 ? 0 : 2, l == 0 ? 0 : tap_mask_of(l - 1));
    mark(SPEC_PROF_NORM); launch_add_norm<T>(c->x, c->proj, c->np_proj, c->ps_proj, 2, (T *)c->node_taps, tap_mask_of(c->L - 1),
                       (const T *)c->final_norm, c->cfg.rms_eps, (T *)c->h, nullptr, rows, rows, c->k, s);
    tick();
    if (want_logits) {
      gemm(c->h, c->lm_head, c->logits, rows, c->V, c->k, c->V, 0, 1);
      mark(SPEC_PROF_ARGMAX); launch_argmax(c->logits, rows, c->V, c->tb.y, s); tick();
    }
  }

  // FC3 over `rows` rows of taps -> proj (Section 3.1: g = FC([l;m;h]))
  void fuse(const void *taps, int rows) {
    if (c->fused) return fuse_fused(taps, rows);
    c->np_proj = pick(c->k, 3 * c->k, 1); c->ps_proj = pstride(c->k);
    gemm(taps, c->fc3, c->proj, rows, c->k, 3 * c->k, c->k, 0, c->np_proj);
  }

  // draft head on the rows of c->meta: cat = [feat ; e(tok)], FC2, decoder block, final norm (-> h)
  void draft_forward(const float *feat, int nparts, size_t fstride, const int32_t *src_row, int rows, int tail_len,
                     bool prebuilt = false) {
    if (c->fused) return draft_forward_fused(feat, nparts, fstride, src_row, rows, tail_len, prebuilt);
    mark(SPEC_PROF_MISC); launch_rope_table(c->meta.pos, rows, c->hd / 2, c->inv_freq, c->cs, s); tick();
    mark(SPEC_PROF_MISC); launch_build_cat<T>(feat, nparts, fstride, src_row, (const T *)c->embed, c->meta.tok, c->meta.seq, (T *)c->cat, rows, c->k, s);
    tick();
    c->np_proj = pick(c->k, 2 * c->k, 1); c->ps_proj = pstride(c->k);
    gemm(c->cat, c->fc2, c->proj, rows, c->k, 2 * c->k, c->k, 0, c->np_proj);
    block(c->dl, c->pools[c->L], rows, tail_len, 1, 0);
    mark(SPEC_PROF_NORM); launch_add_norm<T>(c->x, c->proj, c->np_proj, c->ps_proj, 2, (T *)nullptr, 0, (const T *)c->dfinal_norm, c->cfg.rms_eps,
                       (T *)c->h, nullptr, rows, rows, c->k, s);
    tick();
  }

  void draft_logits(int rows) {
    if (c->fused) return draft_logits_fused(rows);
    gemm(c->h, c->dlm_head, c->logits, rows, c->Vd, c->k, c->Vd, 0, 1);
  }

  void capture(int pass, int rows, bool first) {
    if (!c->cap_logits) return;
    // pass 1: only the last pending row of each sequence matters; it lands in slot [0][b*K]
    size_t lo = (size_t)(pass - 1) * c->Td;
    mark(SPEC_PROF_MISC);
    if (first) {
      launch_gather_rows(c->logits, c->st.last_row, c->cap_logits + lo * c->Vd, c->B, c->Vd, c->K, s);
      launch_gather_rows(c->x, c->st.last_row, c->cap_a + lo * c->k, c->B, c->k, c->K, s);
    } else if (tl_launch_budget != 0) {
      cudaMemcpyAsync(c->cap_logits + lo * c->Vd, c->logits, (size_t)rows * c->Vd * 4, cudaMemcpyDeviceToDevice, s);
      cudaMemcpyAsync(c->cap_a + lo * c->k, c->x, (size_t)rows * c->k * 4, cudaMemcpyDeviceToDevice, s);
    }
    tick(2);
  }

  void step(bool plain) {
    int rows = plain ? c->B : c->Tv, rps = plain ? 1 : c->N;
    tl_launch_budget = c->dbg_launch_budget;
    c->stamp_n = 0;
    c->stamp_cls.clear();
    if (c->stamps) {             // both slots start from all ones (see KernelStamp)
      cudaMemsetAsync(c->stamps, 0xff, (size_t)MAX_STAMPS * 2 * sizeof(unsigned long long), s);
    }
    if (!plain) {
      mark(SPEC_PROF_TREE); launch_prep_extend(c->st, c->tb, c->meta, c->B, c->need_pos, c->status, s); tick();
      c->cur_rps = c->Pmax;
      fuse(c->pend_taps, c->Te);
      draft_forward(c->proj, c->np_proj, c->ps_proj, nullptr, c->Te, c->Pmax);
      if (c->tree_fused) {
        draft_logits_topk(c->Te, c->st.last_row, c->B);
        capture(1, c->Te, true);
        tree_step(1);
      } else {
        draft_logits(c->Te);
        topk(c->st.last_row, c->B);
        capture(1, c->Te, true);
        mark(SPEC_PROF_TREE); launch_expand(c->st, c->tb, c->meta, c->d2t, 1, c->B, s); tick();
      }
      for (int p = 2; p <= c->D; p++) {
        c->cur_rps = c->K;
        draft_forward(c->x, 1, 0, c->tb.feat_row, c->Td, c->tail_tree, c->tree_fused);
        if (c->tree_fused) {
          draft_logits_topk(c->Td, nullptr, 0);
          capture(p, c->Td, false);
          tree_step(p);
        } else {
          draft_logits(c->Td);
          topk(nullptr, c->Td);
          capture(p, c->Td, false);
          mark(SPEC_PROF_TREE); launch_expand(c->st, c->tb, c->meta, c->d2t, p, c->B, s); tick();
        }
      }
      mark(SPEC_PROF_TREE); launch_rerank(c->st, c->tb, c->meta, c->B, s); tick();
    } else {
      mark(SPEC_PROF_TREE); launch_plain_tree(c->st, c->tb, c->meta, c->B, s); tick();
    }
    c->cur_rps = rps;
    target_forward(rows, rps, true);
    mark(SPEC_PROF_TREE);
    if (c->sampled && !plain) launch_accept_sampled(c->st, c->tb, c->logits, c->V, c->u_dev, c->B, rps, s);
    else launch_accept(c->st, c->tb, c->B, rps, s);
    tick();
    PageMap pm{c->page_table, c->pps, c->cfg.page_size, c->cfg.num_pages};
    mark(SPEC_PROF_COMMIT); launch_commit<T>(c->st, c->tb, c->pools_dev, pm, (const T *)c->node_taps, (T *)c->pend_taps, c->B, c->L, c->G, c->hd,
                     c->k, rps, s);
    tick();
    mark(-1);
    tl_launch_budget = -1;
  }
};

// hazard note: draft_forward for tree passes reads c->x (previous pass) in build_cat before FC2 + the
// block's first add_norm overwrite it; everything is ordered on one stream.

static int read_status(spec_ctx *c) {
  int32_t st[4] = {0, 0, 0, 0};
  CUDA_TRY(c, cudaMemcpyAsync(st, c->status, sizeof st, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  if (st[0] != 0) {
    cudaMemsetAsync(c->status, 0, 16, c->stream);
    int code = st[0] == ST_CAPACITY ? SPEC_ERR_CAPACITY : SPEC_ERR_DEVICE_STATUS;
    return fail(c, code, "device status %d at site %d (detail %d, %d)", st[0], st[1], st[2], st[3]);
  }
  return SPEC_OK;
}

template <typename T> static int do_prefill(spec_ctx *c, const int32_t *ids, const int32_t *lens, int32_t reserve, int32_t *first) {
  const spec_cfg &g = c->cfg;
  cudaStream_t s = c->stream;
  int B = c->B, ps = g.page_size;
  // ---- pages: each sequence takes what prompt + reserve + one tree needs, from a (shuffled) free list
  std::vector<int32_t> order(g.num_pages);
  for (int i = 0; i < g.num_pages; i++) order[i] = i;
  if (g.page_shuffle_seed) {
    uint64_t z = (uint64_t)(uint32_t)g.page_shuffle_seed * 0x9E3779B97F4A7C15ull + 1;
    for (int i = g.num_pages - 1; i > 0; i--) {
      z = z * 6364136223846793005ull + 1442695040888963407ull;
      int j = (int)((z >> 33) % (uint64_t)(i + 1));
      std::swap(order[i], order[j]);
    }
  }
  size_t next = 0;
  std::vector<int32_t> cap(B);
  for (int b = 0; b < B; b++) {
    if (lens[b] < 1) return fail(c, SPEC_ERR_INVALID_CFG, "spec_prefill: prompt %d is empty", b);
    long long want = (long long)lens[b] + reserve + c->need_pos;
    if (want > g.max_ctx) return fail(c, SPEC_ERR_CAPACITY, "spec_prefill: sequence %d needs %lld positions, max_ctx is %d", b, want, g.max_ctx);
    int np = (int)((want + ps - 1) / ps);
    if (next + np > (size_t)g.num_pages) return fail(c, SPEC_ERR_CAPACITY, "spec_prefill: page pool exhausted at sequence %d", b);
    for (int p = 0; p < c->pps; p++) c->page_table_host[(size_t)b * c->pps + p] = p < np ? order[next + p] : -1;
    next += np;
    c->n_pages_host[b] = np;
    cap[b] = std::min(np * ps, g.max_ctx);
  }
  c->cap_host = cap;
  CUDA_TRY(c, cudaMemcpyAsync(c->page_table, c->page_table_host.data(), c->page_table_host.size() * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaMemcpyAsync(c->st.cap, cap.data(), B * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaStreamSynchronize(s));

  Sched<T> sc(c);
  const int CH = PREFILL_CHUNK;
  // the prompts go to the device once; each pass's row metadata is then built by a small kernel, so the host never
  // waits inside the loop over passes
  size_t total_ids = 0;
  for (int b = 0; b < B; b++) total_ids += (size_t)lens[b];
  CUDA_TRY(c, cudaMemcpyAsync(c->prompt_dev, ids, total_ids * 4, cudaMemcpyHostToDevice, s));
  auto upload_meta = [&](int nvalid, int b, int start, const int32_t *toks_dev) -> cudaError_t {
    launch_prefill_meta(c->meta, toks_dev, b, start, nvalid, CH, PREFILL_BLOCK, s);
    sc.tick();
    return cudaGetLastError();
  };
  size_t off = 0;
  std::vector<int32_t> n_host(B), P_host(B, 1), root_host(B);
  for (int b = 0; b < B; b++) {
    const int32_t *p = ids + off;
    int n = lens[b];
    for (int i = 0; i < n; i++)
      if (p[i] < 0 || p[i] >= g.vocab) return fail(c, SPEC_ERR_INVALID_CFG, "spec_prefill: token id out of range in prompt %d", b);
    for (int start = 0; start < n; start += CH) {
      int nv = std::min(CH, n - start);
      bool last = start + nv == n;
      CUDA_TRY(c, upload_meta(nv, b, start, c->prompt_dev + off + start));
      c->cur_rps = PREFILL_BLOCK;
      c->ctx_hint = start + CH - PREFILL_BLOCK;
      sc.target_forward(CH, PREFILL_BLOCK, last);
      if (last) {
        // the last position stays pending: its taps become pending entry 0
        CUDA_TRY(c, cudaMemcpyAsync((char *)c->pend_taps + (size_t)b * c->Pmax * 3 * c->k * c->esz,
                                    (char *)c->node_taps + (size_t)(nv - 1) * 3 * c->k * c->esz, (size_t)3 * c->k * c->esz,
                                    cudaMemcpyDeviceToDevice, s));
        CUDA_TRY(c, cudaMemcpyAsync(&root_host[b], c->tb.y + (nv - 1), 4, cudaMemcpyDeviceToHost, s));
      }
      int nd = last ? nv - 1 : nv;        // draft entries j use token j+1; the last position waits for the root
      if (nd > 0) {
        sc.fuse(c->node_taps, CH);
        CUDA_TRY(c, upload_meta(nd, b, start, c->prompt_dev + off + start + 1));
        sc.draft_forward(c->proj, c->np_proj, c->ps_proj, nullptr, CH, PREFILL_BLOCK);
      }
    }
    CUDA_TRY(c, cudaStreamSynchronize(s));
    c->ctx_hint = -1;
    n_host[b] = n;
    off += n;
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->st.n, n_host.data(), B * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaMemcpyAsync(c->st.n_prev, n_host.data(), B * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaMemcpyAsync(c->st.P, P_host.data(), B * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaMemcpyAsync(c->st.root, root_host.data(), B * 4, cudaMemcpyHostToDevice, s));
  std::vector<int32_t> pt((size_t)B * c->Pmax, 0);
  for (int b = 0; b < B; b++) pt[(size_t)b * c->Pmax] = root_host[b];
  CUDA_TRY(c, cudaMemcpyAsync(c->tb.pend_tok, pt.data(), pt.size() * 4, cudaMemcpyHostToDevice, s));
  CUDA_TRY(c, cudaStreamSynchronize(s));
  for (int b = 0; b < B; b++) { c->n_upper[b] = n_host[b]; first[b] = root_host[b]; }
  c->prefilled = true;
  c->draft_stale = false;
  if (c->graph) { cudaGraphExecDestroy(c->graph); c->graph = nullptr; }
  if (c->graph_sampled) { cudaGraphExecDestroy(c->graph_sampled); c->graph_sampled = nullptr; }
  return read_status(c);
}

extern "C" int spec_prefill(spec_ctx *c, const int32_t *ids, const int32_t *lens, int32_t reserve, int32_t *first) {
  if (!c) return SPEC_ERR_NULL;
  if (!ids || !lens || !first) return fail(c, SPEC_ERR_NULL, "spec_prefill: NULL argument");
  if (reserve < 0) return fail(c, SPEC_ERR_INVALID_CFG, "spec_prefill: reserve_tokens is negative");
  return c->cfg.dtype == SPEC_F32 ? do_prefill<float>(c, ids, lens, reserve, first) : do_prefill<bf16>(c, ids, lens, reserve, first);
}

static int launch_step(spec_ctx *c, bool plain) {
  bool use_graph = !(c->cfg.flags & SPEC_FLAG_NO_GRAPH) && !plain;
  c->launches = 0;
  if (!use_graph) {
    if (c->cfg.dtype == SPEC_F32) Sched<float>(c).step(plain); else Sched<bf16>(c).step(plain);
    CUDA_TRY(c, cudaGetLastError());
    if (c->sched_err) return fail(c, SPEC_ERR_CUDA, "a GEMM launch was rejected (code %d)", c->sched_err);
    return SPEC_OK;
  }
  cudaGraphExec_t &graph = c->sampled ? c->graph_sampled : c->graph;
  int &launches_graph = c->sampled ? c->launches_graph_sampled : c->launches_graph;
  if (!graph) {
    cudaGraph_t gr;
    CUDA_TRY(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal));
    if (c->cfg.dtype == SPEC_F32) Sched<float>(c).step(false); else Sched<bf16>(c).step(false);
    cudaError_t e = cudaStreamEndCapture(c->stream, &gr);
    if (e != cudaSuccess) return fail(c, SPEC_ERR_CUDA, "graph capture: %s", cudaGetErrorString(e));
    if (c->sched_err) { cudaGraphDestroy(gr); return fail(c, SPEC_ERR_CUDA, "a GEMM launch was rejected (code %d)", c->sched_err); }
    e = cudaGraphInstantiate(&graph, gr, 0);
    cudaGraphDestroy(gr);
    if (e != cudaSuccess) { graph = nullptr; return fail(c, SPEC_ERR_CUDA, "graph instantiate: %s", cudaGetErrorString(e)); }
    launches_graph = c->launches;
  }
  c->launches = launches_graph;
  CUDA_TRY(c, cudaGraphLaunch(graph, c->stream));
  return SPEC_OK;
}

static int check_capacity(spec_ctx *c, int grow, const char *who) {
  if (!c->prefilled) return fail(c, SPEC_ERR_STATE, "%s before spec_prefill", who);
  for (int b = 0; b < c->B; b++)
    if (c->n_upper[b] + c->need_pos > c->cap_host[b])
      return fail(c, SPEC_ERR_CAPACITY, "%s: sequence %d may reach %d positions (+%d for the tree) but has pages for %d", who, b,
                  c->n_upper[b], c->need_pos, c->cap_host[b]);
  (void)grow;
  return SPEC_OK;
}

extern "C" int spec_step_async(spec_ctx *c, int32_t *dev_ids, int32_t *dev_counts) {
  if (!c) return SPEC_ERR_NULL;
  if (c->draft_stale) return fail(c, SPEC_ERR_STATE, "spec_step after spec_plain_step: the draft cache is stale, prefill again");
  if (int rc = check_capacity(c, c->Pmax, "spec_step")) return rc;
  if (int rc = launch_step(c, false)) return rc;
  for (int b = 0; b < c->B; b++) c->n_upper[b] += c->Pmax;
  if (dev_ids) CUDA_TRY(c, cudaMemcpyAsync(dev_ids, c->tb.out_ids, (size_t)c->B * c->Pmax * 4, cudaMemcpyDeviceToDevice, c->stream));
  if (dev_counts) CUDA_TRY(c, cudaMemcpyAsync(dev_counts, c->tb.out_cnt, (size_t)c->B * 4, cudaMemcpyDeviceToDevice, c->stream));
  return SPEC_OK;
}

static int sync_lengths(spec_ctx *c) {
  std::vector<int32_t> n(c->B);
  CUDA_TRY(c, cudaMemcpyAsync(n.data(), c->st.n, c->B * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  c->n_upper = n;
  return SPEC_OK;
}

extern "C" int spec_step(spec_ctx *c, int32_t *out_ids, int32_t *out_counts) {
  if (!c) return SPEC_ERR_NULL;
  if (!out_ids || !out_counts) return fail(c, SPEC_ERR_NULL, "spec_step: NULL output");
  if (int rc = spec_step_async(c, nullptr, nullptr)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(out_ids, c->tb.out_ids, (size_t)c->B * c->Pmax * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(out_counts, c->tb.out_cnt, (size_t)c->B * 4, cudaMemcpyDeviceToHost, c->stream));
  if (int rc = read_status(c)) return rc;
  return sync_lengths(c);
}

extern "C" int spec_step_sampled(spec_ctx *c, float temperature, const float *u, int32_t *out_ids, int32_t *out_counts) {
  if (!c) return SPEC_ERR_NULL;
  if (!u || !out_ids || !out_counts) return fail(c, SPEC_ERR_NULL, "spec_step_sampled: NULL argument");
  if (!(temperature > 0.0f) || !(temperature <= 1e4f)) return fail(c, SPEC_ERR_INVALID_CFG, "spec_step_sampled: the temperature must be in (0, 1e4]");
  if (c->draft_stale) return fail(c, SPEC_ERR_STATE, "spec_step_sampled after spec_plain_step: the draft cache is stale, prefill again");
  if (int rc = check_capacity(c, c->Pmax, "spec_step_sampled")) return rc;
  const size_t nu = (size_t)c->B * 2 * c->N;
  const float inv_t = 1.0f / temperature;
  CUDA_TRY(c, cudaMemcpyAsync(c->u_dev, u, nu * sizeof(float), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(c->u_dev + nu, &inv_t, sizeof(float), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));           // inv_t lives on this stack frame
  c->sampled = true;
  int rc = launch_step(c, false);
  c->sampled = false;
  if (rc) return rc;
  for (int b = 0; b < c->B; b++) c->n_upper[b] += c->Pmax;
  CUDA_TRY(c, cudaMemcpyAsync(out_ids, c->tb.out_ids, (size_t)c->B * c->Pmax * 4, cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(out_counts, c->tb.out_cnt, (size_t)c->B * 4, cudaMemcpyDeviceToHost, c->stream));
  if (int rc2 = read_status(c)) return rc2;
  return sync_lengths(c);
}

extern "C" int spec_plain_step(spec_ctx *c, int32_t *out_ids) {
  if (!c) return SPEC_ERR_NULL;
  if (!out_ids) return fail(c, SPEC_ERR_NULL, "spec_plain_step: NULL output");
  if (int rc = check_capacity(c, 1, "spec_plain_step")) return rc;
  c->draft_stale = true;
  if (int rc = launch_step(c, true)) return rc;
  std::vector<int32_t> ids((size_t)c->B * c->Pmax);
  CUDA_TRY(c, cudaMemcpyAsync(ids.data(), c->tb.out_ids, ids.size() * 4, cudaMemcpyDeviceToHost, c->stream));
  if (int rc = read_status(c)) return rc;
  for (int b = 0; b < c->B; b++) out_ids[b] = ids[(size_t)b * c->Pmax];
  return sync_lengths(c);
}

extern "C" int spec_lengths(spec_ctx *c, int32_t *lens) {
  if (!c || !lens) return SPEC_ERR_NULL;
  if (int rc = sync_lengths(c)) return rc;
  for (int b = 0; b < c->B; b++) lens[b] = c->n_upper[b];
  return SPEC_OK;
}

extern "C" int spec_profile_step(spec_ctx *c, float *class_ms, int32_t *class_launches) {
  if (!c || !class_ms || !class_launches) return SPEC_ERR_NULL;
  if (c->draft_stale) return fail(c, SPEC_ERR_STATE, "spec_profile_step after spec_plain_step");
  if (int rc = check_capacity(c, c->Pmax, "spec_profile_step")) return rc;
  for (int i = 0; i < SPEC_PROF_CLASSES; i++) { class_ms[i] = 0.0f; class_launches[i] = 0; }
  c->prof = true;
  c->prof_n = 0;
  c->launches = 0;
  if (c->cfg.dtype == SPEC_F32) Sched<float>(c).step(false); else Sched<bf16>(c).step(false);
  c->prof = false;
  for (int b = 0; b < c->B; b++) c->n_upper[b] += c->Pmax;
  CUDA_TRY(c, cudaGetLastError());
  if (int rc = read_status(c)) return rc;
  for (int i = 0; i + 1 < c->prof_n; i++) {
    float ms = 0.0f;
    CUDA_TRY(c, cudaEventElapsedTime(&ms, c->prof_ev[i], c->prof_ev[i + 1]));
    int cls = c->prof_cls[i];
    if (cls >= 0 && cls < SPEC_PROF_CLASSES) { class_ms[cls] += ms; class_launches[cls] += 1; }
  }
  return sync_lengths(c);
}

extern "C" int spec_tune(spec_ctx *c, int32_t what, int32_t value) {
  if (!c) {   // the per-kernel entry points have no context: the pair switch alone may be set without one
    if (what != SPEC_TUNE_GEMM_PAIRS) return SPEC_ERR_NULL;
    if (value < 0 || value > 3) return SPEC_ERR_INVALID_CFG;
    fused_gemm_set_pairs(value);
    return SPEC_OK;
  }
  if (what == SPEC_TUNE_ATTN_CTAS) {
    if (value < 1 || value > 4096) return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: the attention CTA target must be 1..4096");
    attn_fast_set_target_ctas(value);
  } else if (what == SPEC_TUNE_ATTN_UMMA) {
    if (value < 0 || value > 2) return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: the tcgen05 attention mode must be 0, 1 or 2");
    attn_fast_set_umma(value);
  } else if (what == SPEC_TUNE_DEBUG_LAUNCH_BUDGET) {
    c->dbg_launch_budget = value;
  } else if (what == SPEC_TUNE_DEBUG_WAIT_RUNS_OUT) {
    if (value < 0 || value > (1 << 20)) return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: the poll count must be 0..2^20");
    c->dbg_withhold_spin = value;
  } else if (what == SPEC_TUNE_GEMM_PAIRS) {
    if (value < 0 || value > 3) return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: the CTA-pair switch must be 0..3");
    fused_gemm_set_pairs(value);
  } else if (what == SPEC_TUNE_GEMM_CTAS) {
    if (value < 32 || value > 2048) return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: the GEMM CTA target must be 32..2048");
    fused_gemm_set_target_ctas(value);
  } else {
    return fail(c, SPEC_ERR_INVALID_CFG, "spec_tune: unknown knob %d", what);
  }
  if (c->graph) { cudaStreamSynchronize(c->stream); cudaGraphExecDestroy(c->graph); c->graph = nullptr; }   // re-capture with the new plan
  if (c->graph_sampled) { cudaStreamSynchronize(c->stream); cudaGraphExecDestroy(c->graph_sampled); c->graph_sampled = nullptr; }
  return SPEC_OK;
}

extern "C" int spec_launches_per_step(const spec_ctx *c) { return c ? c->launches : 0; }

extern "C" int spec_step_bytes(spec_ctx *c, double *bytes) {
  if (!c || !bytes) return SPEC_ERR_NULL;
  if (int rc = sync_lengths(c)) return rc;
  double e = c->esz, k = c->k, qd = (double)c->H * c->hd, kvd = (double)c->G * c->hd, F = c->F;
  double layer = (k * qd + 2 * k * kvd + qd * k + 3 * k * F + 2 * k) * e;
  double draft_pass = (2 * k * k + k) * e + layer + (double)c->Vd * k * e;
  double w = c->D * draft_pass + 3 * k * k * e + c->L * layer + ((double)c->V * k + k) * e;
  double kv = 0;
  for (int b = 0; b < c->B; b++) kv += (double)c->n_upper[b] * 2 * kvd * e * (c->L + c->D);
  *bytes = w + kv;
  return SPEC_OK;
}

// ------------------------------------------------------------------------------------------ inspection
template <typename U> static int64_t copy_out(spec_ctx *c, const U *dev, size_t count, void *dst, size_t bytes) {
  size_t avail = count * sizeof(U);
  size_t n = std::min(avail, bytes);
  if (n && dst) {
    if (cudaMemcpyAsync(dst, dev, n, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
    if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
  }
  return (int64_t)avail;
}

// widen a [rows][width] block of the storage dtype to floats on the host
static int64_t copy_widen(spec_ctx *c, const void *dev, size_t count, void *dst, size_t bytes) {
  size_t avail = count * 4;
  if (!dst || !bytes) return (int64_t)avail;
  size_t n = std::min(count, bytes / 4);
  if (c->esz == 4) return copy_out(c, (const float *)dev, n, dst, n * 4) < 0 ? SPEC_ERR_CUDA : (int64_t)avail;
  std::vector<uint16_t> tmp(n);
  if (cudaMemcpyAsync(tmp.data(), dev, n * 2, cudaMemcpyDeviceToHost, c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
  float *f = (float *)dst;
  for (size_t i = 0; i < n; i++) { uint32_t u = (uint32_t)tmp[i] << 16; memcpy(&f[i], &u, 4); }
  return (int64_t)avail;
}

extern "C" int64_t spec_debug_read(spec_ctx *c, int32_t what, int32_t seq, void *dst, size_t bytes) {
  if (!c) return SPEC_ERR_NULL;
  if (seq < 0 || seq >= c->B) return fail(c, SPEC_ERR_INVALID_CFG, "spec_debug_read: sequence %d out of range", seq);
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
  int32_t nn = 0, cnt = 0;
  cudaMemcpy(&nn, c->tb.nn + seq, 4, cudaMemcpyDeviceToHost);
  cudaMemcpy(&cnt, c->tb.out_cnt + seq, 4, cudaMemcpyDeviceToHost);
  size_t t0 = (size_t)seq * c->N, p0 = (size_t)seq * (c->pool + 1);
  const TreeBufs &t = c->tb;
  switch (what) {
    case SPEC_DBG_TREE_TOK: return copy_out(c, t.tok + t0, nn, dst, bytes);
    case SPEC_DBG_TREE_PARENT: return copy_out(c, t.parent + t0, nn, dst, bytes);
    case SPEC_DBG_TREE_DEPTH: return copy_out(c, t.depth + t0, nn, dst, bytes);
    case SPEC_DBG_TREE_MASK: return copy_out(c, t.mask + t0, nn, dst, bytes);
    case SPEC_DBG_TREE_POOLIDX: return copy_out(c, t.poolidx + t0, nn, dst, bytes);
    case SPEC_DBG_TREE_SCORE: return copy_out(c, t.score + t0, nn, dst, bytes);
    case SPEC_DBG_Y: return copy_out(c, t.y + t0, nn, dst, bytes);
    case SPEC_DBG_TARGET_LOGITS:
      if (c->fused && !c->cap_logits) return fail(c, SPEC_ERR_STATE, "spec_debug_read: target logits need SPEC_FLAG_CAPTURE on the fused path");
      return copy_out(c, c->logits + t0 * c->V, (size_t)nn * c->V, dst, bytes);
    case SPEC_DBG_NODE_TAPS: return copy_widen(c, (const char *)c->node_taps + t0 * 3 * c->k * c->esz, (size_t)nn * 3 * c->k, dst, bytes);
    case SPEC_DBG_NODE_HIDDEN: return copy_out(c, c->x + t0 * c->k, (size_t)nn * c->k, dst, bytes);
    case SPEC_DBG_DRAFT_LOGITS:
    case SPEC_DBG_DRAFT_A: {
      if (!c->cap_logits) return fail(c, SPEC_ERR_STATE, "spec_debug_read: needs SPEC_FLAG_CAPTURE");
      size_t w = what == SPEC_DBG_DRAFT_LOGITS ? c->Vd : c->k;
      const float *src = what == SPEC_DBG_DRAFT_LOGITS ? c->cap_logits : c->cap_a;
      size_t per_pass = (size_t)c->K * w, avail = (size_t)c->D * per_pass * 4;
      if (!dst || !bytes) return (int64_t)avail;
      if (bytes < avail) return fail(c, SPEC_ERR_INVALID_CFG, "spec_debug_read: buffer too small");
      for (int d = 0; d < c->D; d++)
        if (cudaMemcpy((float *)dst + d * per_pass, src + ((size_t)d * c->Td + (size_t)seq * c->K) * w, per_pass * 4,
                       cudaMemcpyDeviceToHost) != cudaSuccess) return SPEC_ERR_CUDA;
      return (int64_t)avail;
    }
    case SPEC_DBG_POOL_TOK: return copy_out(c, t.pool_tok + p0, c->pool + 1, dst, bytes);
    case SPEC_DBG_POOL_SCORE: return copy_out(c, t.pool_score + p0, c->pool + 1, dst, bytes);
    case SPEC_DBG_POOL_PARENT: return copy_out(c, t.pool_parent + p0, c->pool + 1, dst, bytes);
    case SPEC_DBG_FRONTIER: return copy_out(c, t.frontier + (size_t)seq * c->D * c->K, (size_t)c->D * c->K, dst, bytes);
    case SPEC_DBG_PATH: return copy_out(c, t.path + (size_t)seq * c->Pmax, cnt, dst, bytes);
    case SPEC_DBG_STATUS: return copy_out(c, c->status, 4, dst, bytes);
    case SPEC_DBG_PAGE_TABLE: return copy_out(c, c->page_table + (size_t)seq * c->pps, c->n_pages_host[seq], dst, bytes);
    case SPEC_DBG_RAW_X: return copy_out(c, c->x, (size_t)c->Ralloc * c->k, dst, bytes);
    case SPEC_DBG_RAW_H: return copy_widen(c, c->h, (size_t)c->Ralloc * c->k, dst, bytes);
    case SPEC_DBG_RAW_Q: return copy_widen(c, c->q, (size_t)c->Ralloc * c->H * c->hd, dst, bytes);
    case SPEC_DBG_RAW_AO: return copy_widen(c, c->ao, (size_t)c->Ralloc * c->H * c->hd, dst, bytes);
    case SPEC_DBG_RAW_ACT: return copy_widen(c, c->act, (size_t)c->Ralloc * c->F, dst, bytes);
    case SPEC_DBG_RAW_CAT: return copy_widen(c, c->cat, (size_t)c->Ralloc * 2 * c->k, dst, bytes);
    case SPEC_DBG_RAW_SSQ: return copy_out(c, c->ssq, (size_t)c->ktiles * c->Ralloc, dst, bytes);
    case SPEC_DBG_STAMPS:
      if (!c->stamps) return fail(c, SPEC_ERR_STATE, "spec_debug_read: kernel stamps need SPEC_FLAG_STAMPS");
    {
      // the device keeps the exit time complemented (both slots are updated with atomicMin from all ones)
      size_t cnt = (size_t)c->stamp_n * 2, avail = cnt * sizeof(unsigned long long);
      if (!dst || !bytes) return (int64_t)avail;
      std::vector<unsigned long long> tmp(cnt);
      if (copy_out(c, c->stamps, cnt, tmp.data(), avail) < 0) return SPEC_ERR_CUDA;
      for (size_t i = 1; i < cnt; i += 2) tmp[i] = ~tmp[i];
      memcpy(dst, tmp.data(), std::min(avail, bytes));
      return (int64_t)avail;
    }
    case SPEC_DBG_STAMP_CLASS: {
      size_t avail = c->stamp_cls.size() * sizeof(int32_t);
      if (dst && bytes) memcpy(dst, c->stamp_cls.data(), std::min(avail, bytes));
      return (int64_t)avail;
    }
    case SPEC_DBG_RAW_LOGITS: return copy_out(c, c->logits, (size_t)c->Ralloc * c->Vd, dst, bytes);
    default: return fail(c, SPEC_ERR_INVALID_CFG, "spec_debug_read: unknown item %d", what);
  }
}

extern "C" int spec_debug_read_kv(spec_ctx *c, int32_t seq, int32_t layer, int32_t pos, float *k, float *v) {
  if (!c || !k || !v) return SPEC_ERR_NULL;
  if (seq < 0 || seq >= c->B || layer < -1 || layer >= c->L || pos < 0 || pos >= c->cap_host[seq])
    return fail(c, SPEC_ERR_INVALID_CFG, "spec_debug_read_kv: index out of range");
  int l = layer < 0 ? c->L : layer;
  int ps = c->cfg.page_size;
  int page = c->page_table_host[(size_t)seq * c->pps + pos / ps];
  if (cudaStreamSynchronize(c->stream) != cudaSuccess) return SPEC_ERR_CUDA;
  for (int g = 0; g < c->G; g++) {
    size_t off = (((size_t)page * c->G + g) * ps + pos % ps) * c->hd;
    if (copy_widen(c, (const char *)c->pools[l].k + off * c->esz, c->hd, k + (size_t)g * c->hd, (size_t)c->hd * 4) < 0) return SPEC_ERR_CUDA;
    if (copy_widen(c, (const char *)c->pools[l].v + off * c->esz, c->hd, v + (size_t)g * c->hd, (size_t)c->hd * 4) < 0) return SPEC_ERR_CUDA;
  }
  return SPEC_OK;
}

// ------------------------------------------------------------------------------------------ single kernels

extern "C" int spec_gemm(int32_t dtype, int32_t impl, const void *x, const void *w, float *out, int32_t rows, int32_t O,
                         int32_t I, int32_t ldo, void *stream) {
  if (!x || !w || !out) return SPEC_ERR_NULL;
  if (rows < 1 || O < 1 || I < 1 || ldo < O) return SPEC_ERR_INVALID_CFG;
  cudaStream_t s = (cudaStream_t)stream;
  if (impl == 1) {
    if (dtype == SPEC_F32) launch_gemm_ref<float>((const float *)x, (const float *)w, out, rows, O, I, ldo, s);
    else if (dtype == SPEC_BF16) launch_gemm_ref<bf16>((const bf16 *)x, (const bf16 *)w, out, rows, O, I, ldo, s);
    else return SPEC_ERR_INVALID_CFG;
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
  }
  if (dtype != SPEC_BF16) return SPEC_ERR_UNSUPPORTED;
  return spec_gemm_fused(x, w, out, rows, O, I, ldo, 0, 0, stream);
}

extern "C" int spec_gemm_fused(const void *x, const void *w, float *out, int32_t rows, int32_t O, int32_t I, int32_t ldo,
                               int32_t split, int32_t stages, void *stream) {
  if (!x || !w || !out) return SPEC_ERR_NULL;
  if (rows < 1 || O < 1 || I < 1 || ldo < O || split < 0 || stages < 0) return SPEC_ERR_INVALID_CFG;
  static TmaMaps *g = nullptr;
  if (!g) {
    std::string why;
    g = tma_maps_create(why);
    if (!g) return SPEC_ERR_CUDA;
  }
  FusedGemmArgs a;
  a.x = (const bf16 *)x; a.rows = rows; a.I = I; a.w[0] = (const bf16 *)w; a.O[0] = O; a.nw = 1;
  a.out_f32 = out; a.ldo = ldo; a.split = split; a.stages = stages;
  if (!fused_gemm_supported(EPI_F32, a)) return SPEC_ERR_UNSUPPORTED;
  int rc = fused_gemm_launch(g, EPI_F32, a, (cudaStream_t)stream);
  tma_maps_forget(g);   // test buffers come and go; do not keep descriptors of freed memory
  if (rc) return rc == -1 ? SPEC_ERR_INVALID_CFG : SPEC_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

extern "C" int spec_gemm_swiglu(const void *x, const void *w_gate, const void *w_up, void *act, int32_t rows, int32_t F, int32_t I,
                                void *stream) {
  if (!x || !w_gate || !w_up || !act) return SPEC_ERR_NULL;
  if (rows < 1 || F < 1 || I < 1) return SPEC_ERR_INVALID_CFG;
  static TmaMaps *g = nullptr;
  if (!g) {
    std::string why;
    g = tma_maps_create(why);
    if (!g) return SPEC_ERR_CUDA;
  }
  FusedGemmArgs a;
  a.x = (const bf16 *)x; a.rows = rows; a.I = I; a.nw = 2;
  a.w[0] = (const bf16 *)w_gate; a.w[1] = (const bf16 *)w_up; a.O[0] = a.O[1] = F;
  a.act = (bf16 *)act;
  if (!fused_gemm_supported(EPI_SWIGLU, a)) return SPEC_ERR_UNSUPPORTED;
  int rc = fused_gemm_launch(g, EPI_SWIGLU, a, (cudaStream_t)stream);
  tma_maps_forget(g);
  if (rc) return rc == -1 ? SPEC_ERR_INVALID_CFG : SPEC_ERR_CUDA;
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

extern "C" size_t spec_gemm_topk_scratch_bytes(int32_t rows, int32_t out, int32_t K) {
  if (rows < 1 || out < 1 || K < 1) return 0;
  const size_t tiles = ((size_t)out + 127) / 128;
  return (tiles + 3) * rows * ((size_t)K * 8 + 8) + 1024;
}

extern "C" int spec_gemm_topk(const void *x, const void *w, int32_t rows, int32_t O, int32_t I, int32_t K, int32_t *out_idx,
                              float *out_lp, void *scratch, void *stream) {
  if (!x || !w || !out_idx || !out_lp || !scratch) return SPEC_ERR_NULL;
  if (rows < 1 || O < 1 || I < 1 || K < 1 || K > O) return SPEC_ERR_INVALID_CFG;
  const int tiles = (O + 127) / 128;
  if (!draft_tree_step_smem(tiles, K)) return SPEC_ERR_UNSUPPORTED;
  static TmaMaps *g = nullptr;
  if (!g) {
    std::string why;
    g = tma_maps_create(why);
    if (!g) return SPEC_ERR_CUDA;
  }
  char *base = (char *)(((uintptr_t)scratch + 255) & ~(uintptr_t)255);
  FusedGemmArgs a;
  a.x = (const bf16 *)x; a.rows = rows; a.I = I; a.w[0] = (const bf16 *)w; a.O[0] = O; a.nw = 1;
  const size_t cld = (size_t)draft_tree_cand_ld(tiles);
  a.topk = K; a.cand_ld = (int)cld;
  a.cand_val = (float *)base;
  a.cand_idx = (int32_t *)(a.cand_val + cld * rows * K);
  a.cand_max = (float *)(a.cand_idx + cld * rows * K);
  a.cand_sum = a.cand_max + cld * rows;
  if (!fused_gemm_supported(EPI_TOPK, a)) return SPEC_ERR_UNSUPPORTED;
  int rc = fused_gemm_launch(g, EPI_TOPK, a, (cudaStream_t)stream);
  tma_maps_forget(g);
  if (rc) return rc == -1 ? SPEC_ERR_INVALID_CFG : SPEC_ERR_CUDA;
  if (launch_merge_candidates(a.cand_val, a.cand_idx, a.cand_max, a.cand_sum, tiles, (int)cld, rows, K, out_idx, out_lp, (cudaStream_t)stream))
    return SPEC_ERR_UNSUPPORTED;
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

extern "C" size_t spec_attn_scratch_bytes(int32_t rows, int32_t n_heads, int32_t head_dim, int32_t max_ctx) {
  return attn_fast_scratch_bytes(rows, n_heads, head_dim, max_ctx);
}

extern "C" int spec_attention(int32_t dtype, int32_t impl, const void *q, const void *k_pool, const void *v_pool,
                              const int32_t *page_table, int32_t pages_per_seq, int32_t page_size, const int32_t *row_seq,
                              const int32_t *row_ctx, const int32_t *row_tail_base, const uint64_t *row_mask_lo,
                              const uint64_t *row_mask_hi, int32_t tail_len, void *out, int32_t rows, int32_t H, int32_t G,
                              int32_t hd, int32_t max_ctx, void *scratch, void *stream) {
  if (!q || !k_pool || !v_pool || !page_table || !row_seq || !row_ctx || !row_tail_base || !row_mask_lo || !row_mask_hi || !out)
    return SPEC_ERR_NULL;
  if (rows < 1 || H < 1 || G < 1 || H % G || hd < 16 || hd % 16 || tail_len < 0 || tail_len > 128) return SPEC_ERR_INVALID_CFG;
  cudaStream_t s = (cudaStream_t)stream;
  RowMeta m{};
  m.seq = (int32_t *)row_seq; m.ctx = (int32_t *)row_ctx; m.tail_base = (int32_t *)row_tail_base;
  m.mask_lo = (uint64_t *)row_mask_lo; m.mask_hi = (uint64_t *)row_mask_hi;
  KvPool pool{(void *)k_pool, (void *)v_pool};
  PageMap pm{page_table, pages_per_seq, page_size, 1 << 30};
  if (impl < 0 || impl > 3) return SPEC_ERR_INVALID_CFG;
  if (impl == 1) {
    if (dtype == SPEC_F32) launch_attn_ref<float>((const float *)q, pool, pm, m, tail_len, (float *)out, rows, H, G, hd, max_ctx + tail_len, s);
    else if (dtype == SPEC_BF16) launch_attn_ref<bf16>((const bf16 *)q, pool, pm, m, tail_len, (bf16 *)out, rows, H, G, hd, max_ctx + tail_len, s);
    else return SPEC_ERR_INVALID_CFG;
    return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
  }
  if (dtype != SPEC_BF16 || !attn_fast_supported(hd, H / G)) return SPEC_ERR_UNSUPPORTED;
  // impl 3: the rows are one block of one sequence, which is what the tcgen05 kernel tiles over
  attn_fast_override_umma(impl == 3 ? 1 : 0);
  launch_attn_fast((const bf16 *)q, pool, pm, m, tail_len, (bf16 *)out, rows, H, G, hd, impl == 3 ? rows : 1, max_ctx, scratch, s, impl >= 2, nullptr);
  attn_fast_override_umma(-1);
  attn_fast_forget_maps();
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

extern "C" size_t spec_topk_scratch_bytes(int32_t rows, int32_t n, int32_t K) {
  if (rows < 1 || n < 1 || K < 1) return 0;
  return topk_scratch_bytes(rows, n, K);
}

extern "C" int spec_logsoftmax_topk(const float *logits, int32_t rows, int32_t n, int32_t K, int32_t *out_idx, float *out_lp,
                                    void *scratch, void *stream) {
  if (!logits || !out_idx || !out_lp) return SPEC_ERR_NULL;
  if (rows < 1 || n < 1 || K < 1 || K > n || K > 16) return SPEC_ERR_INVALID_CFG;
  if (scratch) launch_topk2(logits, nullptr, rows, n, K, out_idx, out_lp, scratch, (cudaStream_t)stream);
  else launch_logsoftmax_topk(logits, rows, n, K, out_idx, out_lp, (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}

extern "C" int spec_argmax(const float *logits, int32_t rows, int32_t n, int32_t *out_idx, void *stream) {
  if (!logits || !out_idx) return SPEC_ERR_NULL;
  if (rows < 1 || n < 1) return SPEC_ERR_INVALID_CFG;
  launch_argmax(logits, rows, n, out_idx, (cudaStream_t)stream);
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}
