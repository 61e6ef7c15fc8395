/*
 * eagle3_oracle.c — CPU oracle for one EAGLE-3 speculative step (see eagle3_oracle.h).
 *
 * TEST INFRASTRUCTURE ONLY: never linked into, imported by or called from the CUDA library.
 *
 * fp32 arithmetic in fixed index order.  Build: gcc -O2 -fopenmp -ffp-contract=off (no fused
 * multiply-add, no reassociation), so each output element is the same sequence of IEEE
 * operations however many rows are processed together.
 */
#include "eagle3_oracle.h"

#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ small helpers */
static inline float bf16_bits_to_f32(uint16_t b) {
  uint32_t u = (uint32_t)b << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}
static inline float wget(int wd, const void *W, size_t i) {
  return wd ? bf16_bits_to_f32(((const uint16_t *)W)[i]) : ((const float *)W)[i];
}
static void *xcalloc(size_t n, size_t sz) {
  void *p = calloc(n ? n : 1, sz);
  if (!p) { fprintf(stderr, "oracle: out of memory (%zu x %zu)\n", n, sz); abort(); }
  return p;
}

/* ------------------------------------------------------------------ building blocks */

/* out[m][o] = sum_i W[o][i] * x[m][i], i ascending.  The activations are transposed first so the
 * innermost loop runs over rows m (independent accumulators): same per-element operation order
 * for any M. */
#define LIN_MC 64
void orc_linear(int32_t wd, const void *W, int32_t O, int32_t I, const float *x, int32_t M, float *out) {
  float *xT = (float *)xcalloc((size_t)I * M, sizeof(float));
  for (int m = 0; m < M; m++)
    for (int i = 0; i < I; i++) xT[(size_t)i * M + m] = x[(size_t)m * I + i];
#pragma omp parallel for schedule(static)
  for (int o = 0; o < O; o++) {
    float acc[LIN_MC];
    for (int m0 = 0; m0 < M; m0 += LIN_MC) {
      int mc = M - m0 < LIN_MC ? M - m0 : LIN_MC;
      for (int mm = 0; mm < mc; mm++) acc[mm] = 0.0f;
      if (wd) {
        const uint16_t *w = (const uint16_t *)W + (size_t)o * I;
        for (int i = 0; i < I; i++) {
          float wv = bf16_bits_to_f32(w[i]);
          const float *xr = xT + (size_t)i * M + m0;
          for (int mm = 0; mm < mc; mm++) acc[mm] += wv * xr[mm];
        }
      } else {
        const float *w = (const float *)W + (size_t)o * I;
        for (int i = 0; i < I; i++) {
          float wv = w[i];
          const float *xr = xT + (size_t)i * M + m0;
          for (int mm = 0; mm < mc; mm++) acc[mm] += wv * xr[mm];
        }
      }
      for (int mm = 0; mm < mc; mm++) out[(size_t)(m0 + mm) * O + o] = acc[mm];
    }
  }
  free(xT);
}

/* y = x / sqrt(mean(x^2) + eps) * gain */
void orc_rmsnorm(int32_t wd, const void *gain, const float *x, int32_t M, int32_t k, float eps, float *out) {
  for (int m = 0; m < M; m++) {
    const float *xr = x + (size_t)m * k;
    float ss = 0.0f;
    for (int i = 0; i < k; i++) ss += xr[i] * xr[i];
    float inv = 1.0f / sqrtf(ss / (float)k + eps);
    for (int i = 0; i < k; i++) out[(size_t)m * k + i] = xr[i] * inv * wget(wd, gain, i);
  }
}

/* Rotary embedding, half-split pairing: (x[i], x[i+hd/2]) rotated by pos * theta^(-2i/hd).
 * Angles are formed in double and rounded once. */
void orc_rope(float *x, int32_t n_heads, int32_t hd, int32_t pos, float theta) {
  int half = hd / 2;
  for (int h = 0; h < n_heads; h++) {
    float *v = x + (size_t)h * hd;
    for (int i = 0; i < half; i++) {
      double ang = (double)pos * pow((double)theta, -2.0 * (double)i / (double)hd);
      float cs = (float)cos(ang), sn = (float)sin(ang);
      float a = v[i], b = v[i + half];
      v[i] = a * cs - b * sn;
      v[i + half] = b * cs + a * sn;
    }
  }
}

/* SwiGLU: silu(gate) * up, silu(x) = x / (1 + exp(-x)) */
void orc_swiglu(const float *gate, const float *up, int64_t n, float *out) {
  for (int64_t i = 0; i < n; i++) {
    float g = gate[i];
    out[i] = (g / (1.0f + expf(-g))) * up[i];
  }
}

/* softmax(q.K^T / sqrt(hd)) V for one head; keys in the order given */
void orc_attend(const float *q, const float *const *K, const float *const *V, int32_t nk, int32_t hd, float *out) {
  float *s = (float *)xcalloc((size_t)nk, sizeof(float));
  float scale = 1.0f / sqrtf((float)hd);
  float mx = -INFINITY;
  for (int j = 0; j < nk; j++) {
    float d = 0.0f;
    const float *kr = K[j];
    for (int i = 0; i < hd; i++) d += q[i] * kr[i];
    s[j] = d * scale;
    if (s[j] > mx) mx = s[j];
  }
  float sum = 0.0f;
  for (int j = 0; j < nk; j++) { s[j] = expf(s[j] - mx); sum += s[j]; }
  for (int i = 0; i < hd; i++) out[i] = 0.0f;
  for (int j = 0; j < nk; j++) {
    float p = s[j] / sum;
    const float *vr = V[j];
    for (int i = 0; i < hd; i++) out[i] += p * vr[i];
  }
  free(s);
}

void orc_log_softmax(const float *z, int32_t n, float *lp) {
  float mx = -INFINITY;
  for (int i = 0; i < n; i++) if (z[i] > mx) mx = z[i];
  float sum = 0.0f;
  for (int i = 0; i < n; i++) sum += expf(z[i] - mx);
  float lse = logf(sum);
  for (int i = 0; i < n; i++) lp[i] = (z[i] - mx) - lse;
}

/* K passes of "largest remaining, lowest index on ties" */
void orc_topk(const float *v, int32_t n, int32_t K, int32_t *idx, float *val, float *next_val) {
  char *used = (char *)xcalloc((size_t)n, 1);
  for (int r = 0; r <= K; r++) {
    int best = -1;
    for (int i = 0; i < n; i++)
      if (!used[i] && (best < 0 || v[i] > v[best])) best = i;
    if (r < K) {
      idx[r] = best;
      val[r] = best >= 0 ? v[best] : -INFINITY;
      if (best >= 0) used[best] = 1;
    } else if (next_val) {
      *next_val = best >= 0 ? v[best] : -INFINITY;
    }
  }
  free(used);
}

int32_t orc_argmax(const float *v, int32_t n, float *margin) {
  int best = 0;
  for (int i = 1; i < n; i++) if (v[i] > v[best]) best = i;
  if (margin) {
    float second = -INFINITY;
    for (int i = 0; i < n; i++) if (i != best && v[i] > second) second = v[i];
    *margin = v[best] - second;
  }
  return best;
}

/* Pruning at the end of drafting (Section 2.2): keep the M = min(N-1, pool) best-scored candidates,
 * (score desc, pool index asc); nodes are then numbered in pool-index order after the root. */
/* numbers the selected candidates in pool-index order after the root and fills the tree arrays */
static int32_t tree_from_selection(const char *sel, const float *pscore, const int32_t *pparent, const int32_t *ptok,
                                   const int32_t *pdepth, int32_t pool, int32_t root_tok, int32_t *tok, int32_t *parent,
                                   int32_t *depth, uint64_t *mask, int32_t *poolidx, float *score) {
  int32_t *node_of = (int32_t *)xcalloc((size_t)pool + 1, sizeof(int32_t));
  int nn = 1;
  tok[0] = root_tok; parent[0] = -1; depth[0] = 0; mask[0] = 1ull; poolidx[0] = 0; score[0] = 0.0f;
  node_of[0] = 0;
  for (int i = 1; i <= pool; i++) {
    if (!sel[i]) continue;
    node_of[i] = nn;
    tok[nn] = ptok[i];
    parent[nn] = node_of[pparent[i]];   /* parents have smaller pool indices and are selected */
    depth[nn] = pdepth[i];
    mask[nn] = mask[parent[nn]] | (1ull << nn);
    poolidx[nn] = i;
    score[nn] = pscore[i];
    nn++;
  }
  free(node_of);
  return nn;
}

/* the M best-scored candidates, (score desc, pool index asc); returns the last selected score and the best unselected */
static void rerank_select(const float *pscore, int32_t pool, int M, char *sel, float *last_out, float *next_out) {
  float last = INFINITY;
  for (int r = 0; r < M; r++) {
    int best = -1;
    for (int i = 1; i <= pool; i++)
      if (!sel[i] && (best < 0 || pscore[i] > pscore[best])) best = i;
    sel[best] = 1;
    last = pscore[best];
  }
  float nxt = -INFINITY;
  for (int i = 1; i <= pool; i++) if (!sel[i] && pscore[i] > nxt) nxt = pscore[i];
  *last_out = last; *next_out = nxt;
}

int32_t orc_rerank(const float *pscore, const int32_t *pparent, const int32_t *ptok, const int32_t *pdepth,
                   int32_t pool, int32_t nmax, int32_t root_tok, int32_t *tok, int32_t *parent,
                   int32_t *depth, uint64_t *mask, int32_t *poolidx, float *score, float *cut_margin) {
  int M = nmax - 1 < pool ? nmax - 1 : pool;
  char *sel = (char *)xcalloc((size_t)pool + 1, 1);
  float last, nxt;
  rerank_select(pscore, pool, M, sel, &last, &nxt);
  if (cut_margin) *cut_margin = (M < pool && M > 0) ? last - nxt : INFINITY;
  int nn = tree_from_selection(sel, pscore, pparent, ptok, pdepth, pool, root_tok, tok, parent, depth, mask, poolidx, score);
  free(sel);
  return nn;
}

/* Greedy acceptance (the temperature-0 limit of the acceptance rule of Section 2.1): a draft token
 * is kept iff it equals the target's argmax after its parent; the first mismatch is replaced by
 * that argmax and the rest of the draft is dropped. */
int32_t orc_accept(const int32_t *tok, const int32_t *parent, const int32_t *y, int32_t nn,
                   int32_t *path, int32_t *out_ids) {
  int cur = 0, a = 0;
  path[0] = 0;
  for (;;) {
    int nxt = -1;
    for (int c = 1; c < nn; c++)
      if (parent[c] == cur && tok[c] == y[cur]) { nxt = c; break; }
    if (nxt < 0) break;
    out_ids[a] = tok[nxt];
    cur = nxt;
    path[++a] = cur;
  }
  out_ids[a] = y[cur];
  return a + 1;
}

/* Stochastic acceptance at temperature T > 0 on the draft tree.  Section 2.1 gives the rule for a chain whose
 * tokens were sampled from the draft distribution p^: accept with probability min(1, p / p^), else resample from
 * norm(max(0, p - p^)).  The tree of Section 2.2 is not sampled: the children of a node are the draft's top-K, a
 * deterministic set, so the proposal that puts child c forward is the point mass on tok[c] (p^ = 1 there, 0
 * elsewhere).  The rule then reads: accept c with probability p(tok[c]); on rejection the residual
 * norm(max(0, p - p^)) is p with tok[c] removed and renormalised, and the next child is tried against it.  When no
 * child is left the token is drawn from the residual.  By sequential conditioning the emitted token has exactly
 * distribution p = softmax(z / T), whatever the tree.
 *
 * logits [nn][V]; u [2 * n_max]: u[c] decides node c (1 <= c < nn), u[n_max + cur] draws the final token at node
 * cur by inverse CDF over the ids in increasing order.  acc_p[c] = the probability c was tried against (-1: not
 * tried); *bonus_lo / *bonus_hi = the CDF interval of the drawn token as fractions of the residual mass. */
int32_t orc_accept_sampled(const int32_t *tok, const int32_t *parent, const float *logits, int32_t V, int32_t nn,
                           int32_t n_max, float temperature, const float *u, int32_t *path, int32_t *out_ids,
                           float *acc_p, double *bonus_lo, double *bonus_hi) {
  double *e = (double *)xcalloc((size_t)V, sizeof(double));
  int cur = 0, a = 0;
  path[0] = 0;
  for (int i = 0; i < nn; i++) acc_p[i] = -1.0f;
  for (;;) {
    const float *z = logits + (size_t)cur * V;
    float zmax = z[0];
    for (int v = 1; v < V; v++) if (z[v] > zmax) zmax = z[v];
    double mass = 0.0;
    for (int v = 0; v < V; v++) { e[v] = exp(((double)z[v] - (double)zmax) / (double)temperature); mass += e[v]; }
    int nxt = -1;
    for (int c = cur + 1; c < nn && nxt < 0; c++) {
      if (parent[c] != cur) continue;
      double pc = mass > 0.0 ? e[tok[c]] / mass : 0.0;
      acc_p[c] = (float)pc;
      if ((double)u[c] < pc) nxt = c;
      else { mass -= e[tok[c]]; e[tok[c]] = 0.0; }
    }
    if (nxt >= 0) {
      out_ids[a] = tok[nxt];
      cur = nxt;
      path[++a] = cur;
      continue;
    }
    /* inverse CDF over the residual, ids in increasing order */
    double total = 0.0;
    for (int v = 0; v < V; v++) total += e[v];
    double target = (double)u[n_max + cur] * total, cum = 0.0;
    int pick = -1, last = 0;
    double lo = 0.0;
    for (int v = 0; v < V; v++) {
      if (e[v] <= 0.0) continue;
      last = v;
      if (cum + e[v] > target) { pick = v; lo = cum; break; }
      cum += e[v];
    }
    if (pick < 0) { pick = last; lo = total - e[last]; }
    out_ids[a] = pick;
    if (bonus_lo) *bonus_lo = total > 0.0 ? lo / total : 0.0;
    if (bonus_hi) *bonus_hi = total > 0.0 ? (lo + e[pick]) / total : 1.0;
    break;
  }
  free(e);
  return a + 1;
}

/* ------------------------------------------------------------------ context */
typedef struct {
  const void *attn_norm, *wq, *wk, *wv, *wo, *mlp_norm, *w_gate, *w_up, *w_down;
} layer_w;

struct orc_ctx {
  orc_cfg cfg;
  const void *embed, *final_norm, *lm_head;
  layer_w *tl;                 /* [L] */
  orc_draft_weights dw;
  int n;                       /* committed length; ids[n] is the root */
  int dn;                      /* draft-cache length; pending P = n - dn */
  int32_t *ids;                /* [max_ctx + 1] */
  float *tk, *tv;              /* [L][max_ctx][G*hd] */
  float *taps;                 /* [max_ctx][3k] */
  float *dk, *dv;              /* [max_ctx][G*hd] */
  int pool;                    /* K + (D-1) K^2 */
  /* last-step inspection */
  int nn, count, P_in;
  int32_t tok[ORC_MAX_NODES], parent[ORC_MAX_NODES], depth[ORC_MAX_NODES], poolidx[ORC_MAX_NODES];
  int32_t y[ORC_MAX_NODES], path[ORC_MAX_NODES];
  uint64_t mask[ORC_MAX_NODES];
  float score[ORC_MAX_NODES], y_margin[ORC_MAX_NODES];
  float acc_p[ORC_MAX_NODES];   /* sampled acceptance: probability each tried node was tested against */
  double bonus_iv[2];           /* CDF interval of the drawn token */
  float *target_logits, *node_taps, *node_hidden;       /* [N][V], [N][3k], [N][k] */
  float *draft_logits, *draft_a;                        /* [D][K][Vd], [D][K][k] */
  int32_t *pool_tok, *pool_parent, *pool_depth;         /* [pool+1] */
  float *pool_score;
  int32_t *frontier;                                    /* [D][K] */
  float *topk_margin, *frontier_margin, rerank_margin;  /* [D][K], [D] */
  float *g_pending;                                     /* [max P][k] */
  float *a_store;                                       /* [pool+1][k]: layer output of each processed node */
  float *tree_dk, *tree_dv;                             /* [pool+1][G*hd]: draft K/V of processed tree nodes */
  float *tail_k, *tail_v;                               /* [L][N][G*hd]: target K/V of the tree nodes */
};

/* Which keys a row sees: cache positions 0..n_cache-1, then tail rows listed in extra[] (the
 * row itself last).  Rows write their own K/V either into the cache or into the tail first. */
typedef struct {
  float *Kc, *Vc, *Kt, *Vt;
  const int *cache_slot, *tail_slot, *n_cache, *extra, *n_extra;
  int extra_stride;
} attn_spec;

/* One Llama-style decoder block on M rows: RMSNorm, QKV, RoPE, attention, O, residual, RMSNorm,
 * SwiGLU MLP, residual. */
static void decoder_block(const orc_ctx *c, const layer_w *w, float *x, int M, const int *pos, const attn_spec *sp) {
  const orc_cfg *g = &c->cfg;
  int k = g->hidden, H = g->n_heads, G = g->n_kv_heads, hd = g->head_dim, F = g->ffn, wd = g->wdtype;
  int qd = H * hd, kvd = G * hd, grp = H / G;
  float *h = (float *)xcalloc((size_t)M * k, 4);
  float *q = (float *)xcalloc((size_t)M * qd, 4);
  float *kk = (float *)xcalloc((size_t)M * kvd, 4);
  float *vv = (float *)xcalloc((size_t)M * kvd, 4);
  float *o = (float *)xcalloc((size_t)M * qd, 4);
  orc_rmsnorm(wd, w->attn_norm, x, M, k, g->rms_eps, h);
  orc_linear(wd, w->wq, qd, k, h, M, q);
  orc_linear(wd, w->wk, kvd, k, h, M, kk);
  orc_linear(wd, w->wv, kvd, k, h, M, vv);
  for (int m = 0; m < M; m++) {
    orc_rope(q + (size_t)m * qd, H, hd, pos[m], g->rope_theta);
    orc_rope(kk + (size_t)m * kvd, G, hd, pos[m], g->rope_theta);
    float *kd, *vd;
    if (sp->cache_slot) { kd = sp->Kc + (size_t)sp->cache_slot[m] * kvd; vd = sp->Vc + (size_t)sp->cache_slot[m] * kvd; }
    else { kd = sp->Kt + (size_t)sp->tail_slot[m] * kvd; vd = sp->Vt + (size_t)sp->tail_slot[m] * kvd; }
    memcpy(kd, kk + (size_t)m * kvd, (size_t)kvd * 4);
    memcpy(vd, vv + (size_t)m * kvd, (size_t)kvd * 4);
  }
#pragma omp parallel for schedule(dynamic)
  for (int mh = 0; mh < M * H; mh++) {
    int m = mh / H, hh = mh % H, kvh = hh / grp;
    int nc = sp->n_cache[m], ne = sp->n_extra ? sp->n_extra[m] : 0, nk = nc + ne;
    const float **Kp = (const float **)xcalloc((size_t)nk, sizeof(float *));
    const float **Vp = (const float **)xcalloc((size_t)nk, sizeof(float *));
    for (int j = 0; j < nc; j++) { Kp[j] = sp->Kc + (size_t)j * kvd + kvh * hd; Vp[j] = sp->Vc + (size_t)j * kvd + kvh * hd; }
    for (int e = 0; e < ne; e++) {
      int t = sp->extra[(size_t)m * sp->extra_stride + e];
      Kp[nc + e] = sp->Kt + (size_t)t * kvd + kvh * hd;
      Vp[nc + e] = sp->Vt + (size_t)t * kvd + kvh * hd;
    }
    orc_attend(q + (size_t)m * qd + hh * hd, Kp, Vp, nk, hd, o + (size_t)m * qd + hh * hd);
    free(Kp); free(Vp);
  }
  float *t = (float *)xcalloc((size_t)M * k, 4);
  orc_linear(wd, w->wo, k, qd, o, M, t);
  for (size_t i = 0; i < (size_t)M * k; i++) x[i] += t[i];
  orc_rmsnorm(wd, w->mlp_norm, x, M, k, g->rms_eps, h);
  float *gt = (float *)xcalloc((size_t)M * F, 4);
  float *up = (float *)xcalloc((size_t)M * F, 4);
  orc_linear(wd, w->w_gate, F, k, h, M, gt);
  orc_linear(wd, w->w_up, F, k, h, M, up);
  orc_swiglu(gt, up, (int64_t)M * F, gt);
  orc_linear(wd, w->w_down, k, F, gt, M, t);
  for (size_t i = 0; i < (size_t)M * k; i++) x[i] += t[i];
  free(h); free(q); free(kk); free(vv); free(o); free(t); free(gt); free(up);
}

/* Target forward on M rows.  taps_out: [M][3k] (row m), hidden_out: [M][k] or NULL,
 * logits_out: rows logit_from..M-1 -> [M-logit_from][V] or NULL. */
static void target_forward(orc_ctx *c, int M, const int32_t *tok, const int *pos, attn_spec sp, int tail_rows,
                           float *taps_out, float *hidden_out, int logit_from, float *logits_out) {
  const orc_cfg *g = &c->cfg;
  int k = g->hidden, L = g->n_layers, kvd = g->n_kv_heads * g->head_dim, wd = g->wdtype;
  float *x = (float *)xcalloc((size_t)M * k, 4);
  for (int m = 0; m < M; m++)
    for (int i = 0; i < k; i++) x[(size_t)m * k + i] = wget(wd, c->embed, (size_t)tok[m] * k + i);
  for (int l = 0; l < L; l++) {
    sp.Kc = c->tk + (size_t)l * g->max_ctx * kvd;
    sp.Vc = c->tv + (size_t)l * g->max_ctx * kvd;
    sp.Kt = c->tail_k + (size_t)l * tail_rows * kvd;
    sp.Vt = c->tail_v + (size_t)l * tail_rows * kvd;
    decoder_block(c, &c->tl[l], x, M, pos, &sp);
    for (int s = 0; s < 3; s++)
      if (g->fuse_layers[s] == l && taps_out)
        for (int m = 0; m < M; m++)
          memcpy(taps_out + (size_t)m * 3 * k + (size_t)s * k, x + (size_t)m * k, (size_t)k * 4);
  }
  if (hidden_out) memcpy(hidden_out, x, (size_t)M * k * 4);
  if (logits_out && logit_from < M) {
    int R = M - logit_from;
    float *h = (float *)xcalloc((size_t)R * k, 4);
    orc_rmsnorm(wd, c->final_norm, x + (size_t)logit_from * k, R, k, g->rms_eps, h);
    orc_linear(wd, c->lm_head, g->vocab, k, h, R, logits_out);
    free(h);
  }
  free(x);
}

/* Causal target forward over positions from..to-1 (tokens ids[pos]); K/V and taps go to the caches.
 * Returns the argmax at position to-1 through *last_y (and its logits through last_logits if given). */
#define PREFILL_CHUNK 256
static void target_extend(orc_ctx *c, int from, int to, int32_t *last_y, float *last_logits) {
  int V = c->cfg.vocab;
  for (int s = from; s < to; s += PREFILL_CHUNK) {
    int e = s + PREFILL_CHUNK < to ? s + PREFILL_CHUNK : to, M = e - s;
    int *pos = (int *)xcalloc((size_t)M, sizeof(int)), *nc = (int *)xcalloc((size_t)M, sizeof(int));
    for (int m = 0; m < M; m++) { pos[m] = s + m; nc[m] = s + m + 1; }
    attn_spec sp; memset(&sp, 0, sizeof sp);
    sp.cache_slot = pos; sp.n_cache = nc;
    int want = (e == to) && (last_y || last_logits);
    float *lg = want ? (float *)xcalloc((size_t)V, 4) : NULL;
    target_forward(c, M, c->ids + s, pos, sp, 1, c->taps + (size_t)s * 3 * c->cfg.hidden, NULL, M - 1, lg);
    if (want) {
      if (last_y) *last_y = orc_argmax(lg, V, NULL);
      if (last_logits) memcpy(last_logits, lg, (size_t)V * 4);
      free(lg);
    }
    free(pos); free(nc);
  }
}

/* Draft head on M rows (Section 3.1): x = FC2 [f ; e(tok)], one decoder block -> a; logits of rows
 * logit_from.. = W_d RMSNorm(a).  a_out: [M][k]. */
static void draft_forward(orc_ctx *c, int M, const float *f, const int32_t *tok, const int *pos, attn_spec sp,
                          float *a_out, int logit_from, float *logits_out) {
  const orc_cfg *g = &c->cfg;
  int k = g->hidden, wd = g->wdtype;
  float *cat = (float *)xcalloc((size_t)M * 2 * k, 4);
  for (int m = 0; m < M; m++) {
    memcpy(cat + (size_t)m * 2 * k, f + (size_t)m * k, (size_t)k * 4);
    for (int i = 0; i < k; i++) cat[(size_t)m * 2 * k + k + i] = wget(wd, c->embed, (size_t)tok[m] * k + i);
  }
  orc_linear(wd, c->dw.fc2, k, 2 * k, cat, M, a_out);
  free(cat);
  layer_w w = { c->dw.attn_norm, c->dw.wq, c->dw.wk, c->dw.wv, c->dw.wo, c->dw.mlp_norm,
                c->dw.w_gate, c->dw.w_up, c->dw.w_down };
  sp.Kc = c->dk; sp.Vc = c->dv; sp.Kt = c->tree_dk; sp.Vt = c->tree_dv;
  decoder_block(c, &w, a_out, M, pos, &sp);
  if (logits_out && logit_from < M) {
    int R = M - logit_from;
    float *h = (float *)xcalloc((size_t)R * k, 4);
    orc_rmsnorm(wd, c->dw.final_norm, a_out + (size_t)logit_from * k, R, k, g->rms_eps, h);
    orc_linear(wd, c->dw.lm_head, g->draft_vocab, k, h, R, logits_out);
    free(h);
  }
}

/* Draft entries from..to-1: entry j = (g_j = FC3 [l;m;h]_j, token ids[j+1]) at position j, causal
 * over the draft cache.  g_out ([to-from][k]), a_last ([k]) and logits_last ([Vd]) are optional. */
static void draft_extend(orc_ctx *c, int from, int to, float *g_out, float *a_last, float *logits_last) {
  int k = c->cfg.hidden, wd = c->cfg.wdtype;
  for (int s = from; s < to; s += PREFILL_CHUNK) {
    int e = s + PREFILL_CHUNK < to ? s + PREFILL_CHUNK : to, M = e - s;
    float *gf = (float *)xcalloc((size_t)M * k, 4), *a = (float *)xcalloc((size_t)M * k, 4);
    orc_linear(wd, c->dw.fc3, k, 3 * k, c->taps + (size_t)s * 3 * k, M, gf);
    if (g_out) memcpy(g_out + (size_t)(s - from) * k, gf, (size_t)M * k * 4);
    int *pos = (int *)xcalloc((size_t)M, sizeof(int)), *nc = (int *)xcalloc((size_t)M, sizeof(int));
    for (int m = 0; m < M; m++) { pos[m] = s + m; nc[m] = s + m + 1; }
    attn_spec sp; memset(&sp, 0, sizeof sp);
    sp.cache_slot = pos; sp.n_cache = nc;
    int last = (e == to);
    draft_forward(c, M, gf, c->ids + s + 1, pos, sp, a, M - 1, last ? logits_last : NULL);
    if (last && a_last) memcpy(a_last, a + (size_t)(M - 1) * k, (size_t)k * 4);
    free(gf); free(a); free(pos); free(nc);
  }
}

/* ------------------------------------------------------------------ lifecycle */
orc_ctx *orc_create(const orc_cfg *cfg, const orc_target_weights *tw, const orc_draft_weights *dw) {
  if (!cfg || !tw || !dw) return NULL;
  if (cfg->tree_nodes > ORC_MAX_NODES || cfg->tree_nodes < 1 || cfg->tree_topk < 1 ||
      cfg->tree_topk > cfg->draft_vocab || cfg->tree_depth < 1 || cfg->n_heads % cfg->n_kv_heads ||
      cfg->head_dim % 2)
    return NULL;
  orc_ctx *c = (orc_ctx *)xcalloc(1, sizeof *c);
  c->cfg = *cfg;
  int L = cfg->n_layers, k = cfg->hidden, kvd = cfg->n_kv_heads * cfg->head_dim;
  int K = cfg->tree_topk, D = cfg->tree_depth, N = cfg->tree_nodes;
  c->embed = tw->embed; c->final_norm = tw->final_norm; c->lm_head = tw->lm_head;
  c->tl = (layer_w *)xcalloc((size_t)L, sizeof(layer_w));
  for (int l = 0; l < L; l++) {
    layer_w w = { tw->attn_norm[l], tw->wq[l], tw->wk[l], tw->wv[l], tw->wo[l], tw->mlp_norm[l],
                  tw->w_gate[l], tw->w_up[l], tw->w_down[l] };
    c->tl[l] = w;
  }
  c->dw = *dw;
  c->pool = K + (D - 1) * K * K;
  size_t mc = (size_t)cfg->max_ctx;
  c->ids = (int32_t *)xcalloc(mc + 1, 4);
  c->tk = (float *)xcalloc((size_t)L * mc * kvd, 4);
  c->tv = (float *)xcalloc((size_t)L * mc * kvd, 4);
  c->taps = (float *)xcalloc(mc * 3 * k, 4);
  c->dk = (float *)xcalloc(mc * kvd, 4);
  c->dv = (float *)xcalloc(mc * kvd, 4);
  c->target_logits = (float *)xcalloc((size_t)N * cfg->vocab, 4);
  c->node_taps = (float *)xcalloc((size_t)N * 3 * k, 4);
  c->node_hidden = (float *)xcalloc((size_t)N * k, 4);
  c->draft_logits = (float *)xcalloc((size_t)D * K * cfg->draft_vocab, 4);
  c->draft_a = (float *)xcalloc((size_t)D * K * k, 4);
  c->pool_tok = (int32_t *)xcalloc((size_t)c->pool + 1, 4);
  c->pool_parent = (int32_t *)xcalloc((size_t)c->pool + 1, 4);
  c->pool_depth = (int32_t *)xcalloc((size_t)c->pool + 1, 4);
  c->pool_score = (float *)xcalloc((size_t)c->pool + 1, 4);
  c->frontier = (int32_t *)xcalloc((size_t)D * K, 4);
  c->topk_margin = (float *)xcalloc((size_t)D * K, 4);
  c->frontier_margin = (float *)xcalloc((size_t)D, 4);
  c->g_pending = (float *)xcalloc(mc * k, 4);
  c->a_store = (float *)xcalloc(((size_t)c->pool + 1) * k, 4);
  c->tree_dk = (float *)xcalloc(((size_t)c->pool + 1) * kvd, 4);
  c->tree_dv = (float *)xcalloc(((size_t)c->pool + 1) * kvd, 4);
  c->tail_k = (float *)xcalloc((size_t)L * N * kvd, 4);
  c->tail_v = (float *)xcalloc((size_t)L * N * kvd, 4);
  return c;
}

void orc_destroy(orc_ctx *c) {
  if (!c) return;
  free(c->tl); free(c->ids); free(c->tk); free(c->tv); free(c->taps); free(c->dk); free(c->dv);
  free(c->target_logits); free(c->node_taps); free(c->node_hidden); free(c->draft_logits);
  free(c->draft_a); free(c->pool_tok); free(c->pool_parent); free(c->pool_depth); free(c->pool_score);
  free(c->frontier); free(c->topk_margin); free(c->frontier_margin); free(c->g_pending);
  free(c->a_store); free(c->tree_dk); free(c->tree_dv); free(c->tail_k); free(c->tail_v);
  free(c);
}

int32_t orc_n(const orc_ctx *c) { return c->n; }
int32_t orc_pending(const orc_ctx *c) { return c->n - c->dn; }
const int32_t *orc_ids(const orc_ctx *c) { return c->ids; }

int orc_prefill(orc_ctx *c, const int32_t *ids, int32_t n, int32_t *first_id) {
  if (n < 1 || n + c->cfg.tree_nodes > c->cfg.max_ctx) return -1;
  memcpy(c->ids, ids, (size_t)n * 4);
  int32_t y = 0;
  target_extend(c, 0, n, &y, NULL);
  c->ids[n] = y;
  c->n = n;
  draft_extend(c, 0, n - 1, NULL, NULL, NULL);
  c->dn = n - 1;
  if (first_id) *first_id = y;
  return 0;
}

int orc_greedy_margins(orc_ctx *c, int32_t gen, int32_t *out, float *margins) {
  if (c->n + gen + 1 > c->cfg.max_ctx) return -1;
  float *lg = (float *)xcalloc((size_t)c->cfg.vocab, 4);
  for (int i = 0; i < gen; i++) {
    float mg = 0.0f;
    target_extend(c, c->n, c->n + 1, NULL, lg);   /* forwards ids[n] at position n */
    int32_t y = orc_argmax(lg, c->cfg.vocab, &mg);
    c->n += 1;
    c->ids[c->n] = y;
    out[i] = y;
    if (margins) margins[i] = mg;
  }
  free(lg);
  return 0;
}
int orc_greedy(orc_ctx *c, int32_t gen, int32_t *out) { return orc_greedy_margins(c, gen, out, NULL); }

int orc_force_state(orc_ctx *c, const int32_t *ids, int32_t n, int32_t P) {
  if (n < 1 || P < 1 || P > n || n + c->cfg.tree_nodes > c->cfg.max_ctx) return -1;
  int keep = 0;
  while (keep < c->n && keep < n && c->ids[keep] == ids[keep]) keep++;
  /* draft entry j was built from the taps of position j and token ids[j+1]: it survives while
   * both are unchanged */
  int dmax = c->dn < n - P ? c->dn : n - P, dkeep = 0;
  while (dkeep < dmax && dkeep < keep && c->ids[dkeep + 1] == ids[dkeep + 1]) dkeep++;
  memcpy(c->ids, ids, ((size_t)n + 1) * 4);
  if (keep < n) target_extend(c, keep, n, NULL, NULL);
  c->n = n;
  if (dkeep < n - P) draft_extend(c, dkeep, n - P, NULL, NULL, NULL);
  c->dn = n - P;
  return 0;
}

/* ------------------------------------------------------------------ following another implementation's decisions
 * A harness that compares a second implementation with this one loses everything after the first near-tie that the
 * two resolve differently.  In follow mode the step takes the other side's integer decisions (the K children of every
 * row, every frontier, the pruned set) wherever they are VALID on this oracle's own values: a followed choice of K
 * items is valid when its order is non-increasing within eps and no item left out beats the worst chosen one by more
 * than eps.  All values (log-probabilities, scores) stay the oracle's own.  Each decision is also compared with the
 * oracle's own choice: above `require` of its own margin a difference is recorded as a violation. */
static void follow_note(orc_follow *fw, int same, float own_margin, int valid) {
  fw->checked++;
  if (!valid) { fw->invalid++; return; }
  if (!same) fw->differs++;
  if (own_margin > fw->require) { fw->required++; if (!same) fw->required_differs++; }
  else if (own_margin > fw->band_lo) { fw->band_total++; if (!same) fw->band_differs++; }
}

/* v[n]: the oracle's values; own[K] / own_val[K]: its own choice in rank order, next_val: its (K+1)-th value;
 * cand[K]: the followed choice (indices into v, -1 = unknown).  Every rank is one decision whose margin is the
 * smaller of the gaps to its neighbours in the oracle's own order (the last rank: to the best item left out).
 * Returns 1 and overwrites own / own_val with the followed choice when that is valid. */
static int follow_choice(orc_follow *fw, const float *v, int n, int K, int32_t *own, float *own_val, float next_val,
                         const int32_t *cand) {
  int valid = 1;
  for (int r = 0; r < K && valid; r++) {
    if (cand[r] < 0 || cand[r] >= n) valid = 0;
    for (int q = 0; q < r && valid; q++) if (cand[q] == cand[r]) valid = 0;
  }
  float worst = INFINITY;
  for (int r = 0; r < K && valid; r++) {
    if (r + 1 < K && v[cand[r]] < v[cand[r + 1]] - fw->eps) valid = 0;
    if (v[cand[r]] < worst) worst = v[cand[r]];
  }
  if (valid) {
    for (int i = 0; i < n && valid; i++) {
      if (v[i] <= worst + fw->eps) continue;
      int chosen = 0;
      for (int r = 0; r < K; r++) if (cand[r] == i) chosen = 1;
      if (!chosen) valid = 0;
    }
  }
  if (!valid) { fw->checked += K; fw->invalid++; return 0; }
  for (int r = 0; r < K; r++) {
    float below = own_val[r] - (r + 1 < K ? own_val[r + 1] : next_val);
    float above = r > 0 ? own_val[r - 1] - own_val[r] : INFINITY;
    follow_note(fw, cand[r] == own[r], below < above ? below : above, 1);
  }
  for (int r = 0; r < K; r++) { own[r] = cand[r]; own_val[r] = v[cand[r]]; }
  return 1;
}

/* draft id of a target token (d2t is strictly increasing), -1 if the draft cannot emit it */
static int32_t d2t_inverse(const orc_ctx *c, int32_t target_id) {
  int lo = 0, hi = c->cfg.draft_vocab - 1;
  while (lo <= hi) {
    int mid = (lo + hi) / 2;
    int32_t t = c->dw.d2t[mid];
    if (t == target_id) return mid;
    if (t < target_id) lo = mid + 1; else hi = mid - 1;
  }
  return -1;
}

/* ------------------------------------------------------------------ the speculative step */
static int step_impl(orc_ctx *c, int32_t *out_ids, int32_t *count, float temperature, const float *u, orc_follow *fw) {
  const orc_cfg *g = &c->cfg;
  int n = c->n, P = c->n - c->dn, K = g->tree_topk, D = g->tree_depth, N = g->tree_nodes;
  int k = g->hidden, Vd = g->draft_vocab, V = g->vocab, L = g->n_layers, kvd = g->n_kv_heads * g->head_dim;
  if (P < 1 || n + N > g->max_ctx) return -1;
  c->P_in = P;
  for (int i = 0; i < D * K; i++) { c->frontier[i] = -1; c->topk_margin[i] = INFINITY; }
  for (int i = 0; i < D; i++) c->frontier_margin[i] = INFINITY;
  float *lp = (float *)xcalloc((size_t)Vd, 4);
  int32_t *tid = (int32_t *)xcalloc((size_t)K, 4);
  float *tval = (float *)xcalloc((size_t)K + 1, 4);
  int32_t *cand = (int32_t *)xcalloc((size_t)K, 4);
  if (fw) fw->checked = fw->differs = fw->invalid = fw->required = fw->required_differs = fw->band_total = fw->band_differs = 0;

  /* 1+2. fuse the pending taps (FC 3k->k) and run the draft layer over the pending entries */
  draft_extend(c, n - P, n, c->g_pending, c->a_store, c->draft_logits);
  c->dn = n;   /* restored to n_old at commit time below (the cache keeps the entries) */
  memcpy(c->draft_a, c->a_store, (size_t)k * 4);
  c->pool_tok[0] = c->ids[n]; c->pool_parent[0] = -1; c->pool_depth[0] = 0; c->pool_score[0] = 0.0f;
  c->frontier[0] = 0;
  orc_log_softmax(c->draft_logits, Vd, lp);
  orc_topk(lp, Vd, K, tid, tval, &tval[K]);
  for (int r = 0; r < K; r++) {
    float gap = tval[r] - tval[r + 1];
    if (gap < c->topk_margin[0]) c->topk_margin[0] = gap;
  }
  if (fw) {
    for (int r = 0; r < K; r++) cand[r] = d2t_inverse(c, fw->pool_tok[1 + r]);
    follow_choice(fw, lp, Vd, K, tid, tval, tval[K], cand);
  }
  for (int r = 0; r < K; r++) {
    c->pool_tok[1 + r] = c->dw.d2t[tid[r]];
    c->pool_parent[1 + r] = 0; c->pool_depth[1 + r] = 1; c->pool_score[1 + r] = tval[r];
  }
  /* frontier after level 1: all K level-1 nodes in rank order */
  int32_t *front = (int32_t *)xcalloc((size_t)K, 4);
  for (int r = 0; r < K; r++) front[r] = 1 + r;

  /* 3. tree passes d = 2..D: the frontier (depth d-1) is fed back with the draft's own output a */
  for (int d = 2; d <= D; d++) {
    float *f = (float *)xcalloc((size_t)K * k, 4), *a = (float *)xcalloc((size_t)K * k, 4);
    int32_t *tk = (int32_t *)xcalloc((size_t)K, 4);
    int *pos = (int *)xcalloc((size_t)K, sizeof(int)), *nc = (int *)xcalloc((size_t)K, sizeof(int));
    int *ts = (int *)xcalloc((size_t)K, sizeof(int)), *ne = (int *)xcalloc((size_t)K, sizeof(int));
    int *ex = (int *)xcalloc((size_t)K * (D + 1), sizeof(int));
    for (int r = 0; r < K; r++) {
      int u = front[r];
      c->frontier[(size_t)(d - 1) * K + r] = u;
      memcpy(f + (size_t)r * k, c->a_store + (size_t)c->pool_parent[u] * k, (size_t)k * 4);
      tk[r] = c->pool_tok[u]; pos[r] = n + d - 2; nc[r] = n; ts[r] = u;
      /* ancestors below the root, root-side first, then the node itself */
      int chain[ORC_MAX_NODES], len = 0;
      for (int v = u; v != 0; v = c->pool_parent[v]) chain[len++] = v;
      for (int e = 0; e < len; e++) ex[(size_t)r * (D + 1) + e] = chain[len - 1 - e];
      ne[r] = len;
    }
    attn_spec sp; memset(&sp, 0, sizeof sp);
    sp.tail_slot = ts; sp.n_cache = nc; sp.extra = ex; sp.n_extra = ne; sp.extra_stride = D + 1;
    float *lg = c->draft_logits + (size_t)(d - 1) * K * Vd;
    draft_forward(c, K, f, tk, pos, sp, a, 0, lg);
    memcpy(c->draft_a + (size_t)(d - 1) * K * k, a, (size_t)K * k * 4);
    int base = K + (d - 2) * K * K;
    for (int r = 0; r < K; r++) {
      int u = front[r];
      memcpy(c->a_store + (size_t)u * k, a + (size_t)r * k, (size_t)k * 4);
      orc_log_softmax(lg + (size_t)r * Vd, Vd, lp);
      orc_topk(lp, Vd, K, tid, tval, &tval[K]);
      float mg = INFINITY;
      for (int cc = 0; cc < K; cc++) {
        float gap = tval[cc] - tval[cc + 1];
        if (gap < mg) mg = gap;
      }
      if (fw) {
        for (int cc = 0; cc < K; cc++) cand[cc] = d2t_inverse(c, fw->pool_tok[base + r * K + cc + 1]);
        follow_choice(fw, lp, Vd, K, tid, tval, tval[K], cand);
      }
      for (int cc = 0; cc < K; cc++) {
        int ci = base + r * K + cc + 1;
        c->pool_tok[ci] = c->dw.d2t[tid[cc]];
        c->pool_parent[ci] = u; c->pool_depth[ci] = d;
        c->pool_score[ci] = c->pool_score[u] + tval[cc];
      }
      c->topk_margin[(size_t)(d - 1) * K + r] = mg;
    }
    /* next frontier: the K best of this level's K*K children, (score desc, pool index asc) */
    if (d < D) {
      float *sc = c->pool_score + base + 1;
      float nxt = -INFINITY;
      orc_topk(sc, K * K, K, tid, tval, &nxt);
      if (K * K > K) {
        float mg = tval[K - 1] - nxt;
        for (int r = 0; r + 1 < K; r++) if (tval[r] - tval[r + 1] < mg) mg = tval[r] - tval[r + 1];
        c->frontier_margin[d - 1] = mg;
      }
      if (fw) {
        for (int r = 0; r < K; r++) cand[r] = fw->frontier[(size_t)d * K + r] - (base + 1);
        follow_choice(fw, sc, K * K, K, tid, tval, nxt, cand);
      }
      for (int r = 0; r < K; r++) front[r] = base + 1 + tid[r];
    }
    free(f); free(a); free(tk); free(pos); free(nc); free(ts); free(ne); free(ex);
  }

  /* 4. prune to the N-1 best candidates and number the nodes */
  int nn = orc_rerank(c->pool_score, c->pool_parent, c->pool_tok, c->pool_depth, c->pool, N, c->ids[n],
                      c->tok, c->parent, c->depth, c->mask, c->poolidx, c->score, &c->rerank_margin);
  if (fw) {
    /* the followed pruned set: as many candidates, none left out that beats the worst kept one by more than eps,
     * every kept candidate's parent kept */
    int M = N - 1 < c->pool ? N - 1 : c->pool, valid = fw->nsel == M + 1, same = valid && fw->nsel == nn;
    char *sel = (char *)xcalloc((size_t)c->pool + 1, 1);
    float worst = INFINITY;
    for (int i = 1; i < fw->nsel && valid; i++) {
      int pi = fw->sel_poolidx[i];
      if (pi < 1 || pi > c->pool || sel[pi] || (i > 1 && pi <= fw->sel_poolidx[i - 1])) { valid = 0; break; }
      sel[pi] = 1;
      if (c->pool_score[pi] < worst) worst = c->pool_score[pi];
      if (same && c->poolidx[i] != pi) same = 0;
    }
    for (int i = 1; i <= c->pool && valid; i++) {
      if (sel[i] && c->pool_parent[i] != 0 && !sel[c->pool_parent[i]]) valid = 0;
      if (!sel[i] && c->pool_score[i] > worst + fw->eps) valid = 0;
    }
    follow_note(fw, same, c->rerank_margin, valid);
    if (valid)
      nn = tree_from_selection(sel, c->pool_score, c->pool_parent, c->pool_tok, c->pool_depth, c->pool, c->ids[n],
                               c->tok, c->parent, c->depth, c->mask, c->poolidx, c->score);
    free(sel);
  }
  c->nn = nn;

  /* 5. one target forward over all nodes with tree attention */
  {
    int *pos = (int *)xcalloc((size_t)nn, sizeof(int)), *nc = (int *)xcalloc((size_t)nn, sizeof(int));
    int *ts = (int *)xcalloc((size_t)nn, sizeof(int)), *ne = (int *)xcalloc((size_t)nn, sizeof(int));
    int *ex = (int *)xcalloc((size_t)nn * ORC_MAX_NODES, sizeof(int));
    for (int i = 0; i < nn; i++) {
      pos[i] = n + c->depth[i]; nc[i] = n; ts[i] = i;
      int len = 0;
      for (int j = 0; j <= i; j++) if ((c->mask[i] >> j) & 1ull) ex[(size_t)i * ORC_MAX_NODES + len++] = j;
      ne[i] = len;
    }
    attn_spec sp; memset(&sp, 0, sizeof sp);
    sp.tail_slot = ts; sp.n_cache = nc; sp.extra = ex; sp.n_extra = ne; sp.extra_stride = ORC_MAX_NODES;
    target_forward(c, nn, c->tok, pos, sp, N, c->node_taps, c->node_hidden, 0, c->target_logits);
    for (int i = 0; i < nn; i++) c->y[i] = orc_argmax(c->target_logits + (size_t)i * V, V, &c->y_margin[i]);
    free(pos); free(nc); free(ts); free(ne); free(ex);
  }

  /* 6. acceptance: greedy, or the stochastic rule when a temperature and uniforms are given */
  int cnt = (temperature > 0.0f && u)
                ? orc_accept_sampled(c->tok, c->parent, c->target_logits, V, nn, N, temperature, u, c->path, out_ids, c->acc_p,
                                     &c->bonus_iv[0], &c->bonus_iv[1])
                : orc_accept(c->tok, c->parent, c->y, nn, c->path, out_ids);
  c->count = cnt;
  if (count) *count = cnt;

  /* 7. commit: accepted nodes' K/V and taps move to positions n..n+a; they become the pending
   * entries of the next step; the draft-tree K/V is dropped */
  for (int j = 0; j < cnt; j++) {
    int node = c->path[j];
    for (int l = 0; l < L; l++) {
      memcpy(c->tk + ((size_t)l * g->max_ctx + n + j) * kvd, c->tail_k + ((size_t)l * N + node) * kvd, (size_t)kvd * 4);
      memcpy(c->tv + ((size_t)l * g->max_ctx + n + j) * kvd, c->tail_v + ((size_t)l * N + node) * kvd, (size_t)kvd * 4);
    }
    memcpy(c->taps + (size_t)(n + j) * 3 * k, c->node_taps + (size_t)node * 3 * k, (size_t)3 * k * 4);
    c->ids[n + 1 + j] = out_ids[j];
  }
  c->n = n + cnt;
  c->dn = n;
  free(lp); free(tid); free(tval); free(front); free(cand);
  return 0;
}

int orc_step(orc_ctx *c, int32_t *out_ids, int32_t *count) { return step_impl(c, out_ids, count, 0.0f, NULL, NULL); }

int orc_step_follow(orc_ctx *c, orc_follow *fw, float temperature, const float *u, int32_t *out_ids, int32_t *count) {
  if (!fw || !fw->pool_tok || !fw->frontier || !fw->sel_poolidx || !(fw->eps >= 0.0f)) return -1;
  if (temperature > 0.0f && !u) return -1;
  return step_impl(c, out_ids, count, temperature > 0.0f ? temperature : 0.0f, temperature > 0.0f ? u : NULL, fw);
}

int orc_step_sampled(orc_ctx *c, float temperature, const float *u, int32_t *out_ids, int32_t *count) {
  if (!(temperature > 0.0f) || !u) return -1;
  return step_impl(c, out_ids, count, temperature, u, NULL);
}

/* Step 5 (Section 2.2, tree attention) on a caller-given tree: node i carries tok[i], sits at RoPE position
 * n_ctx + depth[i], and attends the committed positions [0, n_ctx) plus the nodes j with bit j of mask[i].  Only the
 * per-step tail scratch is written, the committed caches are read; n_ctx may be smaller than the committed length
 * (the state before the last step). */
int orc_verify_tree(orc_ctx *c, int32_t n_ctx, int32_t nn, const int32_t *tok, const int32_t *depth, const uint64_t *mask,
                    float *logits, float *hidden, float *taps) {
  const orc_cfg *g = &c->cfg;
  int N = g->tree_nodes;
  if (n_ctx < 0 || n_ctx > c->n || nn < 1 || nn > N || n_ctx + N > g->max_ctx) return -1;
  for (int i = 0; i < nn; i++)
    if (tok[i] < 0 || tok[i] >= g->vocab || depth[i] < 0 || !((mask[i] >> i) & 1ull) || (i + 1 < 64 && (mask[i] >> (i + 1)))) return -1;
  int *pos = (int *)xcalloc((size_t)nn, sizeof(int)), *nc = (int *)xcalloc((size_t)nn, sizeof(int));
  int *ts = (int *)xcalloc((size_t)nn, sizeof(int)), *ne = (int *)xcalloc((size_t)nn, sizeof(int));
  int *ex = (int *)xcalloc((size_t)nn * ORC_MAX_NODES, sizeof(int));
  for (int i = 0; i < nn; i++) {
    pos[i] = n_ctx + depth[i]; nc[i] = n_ctx; ts[i] = i;
    int len = 0;
    for (int j = 0; j <= i; j++) if ((mask[i] >> j) & 1ull) ex[(size_t)i * ORC_MAX_NODES + len++] = j;
    ne[i] = len;
  }
  attn_spec sp; memset(&sp, 0, sizeof sp);
  sp.tail_slot = ts; sp.n_cache = nc; sp.extra = ex; sp.n_extra = ne; sp.extra_stride = ORC_MAX_NODES;
  float *tp = taps ? taps : (float *)xcalloc((size_t)nn * 3 * g->hidden, 4);
  target_forward(c, nn, tok, pos, sp, N, tp, hidden, 0, logits);
  if (!taps) free(tp);
  free(pos); free(nc); free(ts); free(ne); free(ex);
  return 0;
}

const void *orc_get(const orc_ctx *c, int32_t what, int64_t *count) {
  const orc_cfg *g = &c->cfg;
  int64_t cn = 0; const void *p = NULL;
  int K = g->tree_topk, D = g->tree_depth;
  switch (what) {
    case ORC_TREE_TOK: p = c->tok; cn = c->nn; break;
    case ORC_TREE_PARENT: p = c->parent; cn = c->nn; break;
    case ORC_TREE_DEPTH: p = c->depth; cn = c->nn; break;
    case ORC_TREE_MASK: p = c->mask; cn = c->nn; break;
    case ORC_TREE_POOLIDX: p = c->poolidx; cn = c->nn; break;
    case ORC_TREE_SCORE: p = c->score; cn = c->nn; break;
    case ORC_Y: p = c->y; cn = c->nn; break;
    case ORC_Y_MARGIN: p = c->y_margin; cn = c->nn; break;
    case ORC_TARGET_LOGITS: p = c->target_logits; cn = (int64_t)c->nn * g->vocab; break;
    case ORC_NODE_TAPS: p = c->node_taps; cn = (int64_t)c->nn * 3 * g->hidden; break;
    case ORC_NODE_HIDDEN: p = c->node_hidden; cn = (int64_t)c->nn * g->hidden; break;
    case ORC_DRAFT_LOGITS: p = c->draft_logits; cn = (int64_t)D * K * g->draft_vocab; break;
    case ORC_DRAFT_A: p = c->draft_a; cn = (int64_t)D * K * g->hidden; break;
    case ORC_POOL_TOK: p = c->pool_tok; cn = c->pool + 1; break;
    case ORC_POOL_SCORE: p = c->pool_score; cn = c->pool + 1; break;
    case ORC_POOL_PARENT: p = c->pool_parent; cn = c->pool + 1; break;
    case ORC_FRONTIER: p = c->frontier; cn = (int64_t)D * K; break;
    case ORC_TOPK_MARGIN: p = c->topk_margin; cn = (int64_t)D * K; break;
    case ORC_FRONTIER_MARGIN: p = c->frontier_margin; cn = D; break;
    case ORC_RERANK_MARGIN: p = &c->rerank_margin; cn = 1; break;
    case ORC_PATH: p = c->path; cn = c->count; break;
    case ORC_G_PENDING: p = c->g_pending; cn = (int64_t)c->P_in * g->hidden; break;
    case ORC_ACC_P: p = c->acc_p; cn = c->nn; break;
    case ORC_BONUS_INTERVAL: p = c->bonus_iv; cn = 2; break;
    default: break;
  }
  if (count) *count = cn;
  return p;
}

int orc_read_target_kv(const orc_ctx *c, int32_t layer, int32_t pos, float *kk, float *vv) {
  int kvd = c->cfg.n_kv_heads * c->cfg.head_dim;
  if (layer < 0 || layer >= c->cfg.n_layers || pos < 0 || pos >= c->n) return -1;
  memcpy(kk, c->tk + ((size_t)layer * c->cfg.max_ctx + pos) * kvd, (size_t)kvd * 4);
  memcpy(vv, c->tv + ((size_t)layer * c->cfg.max_ctx + pos) * kvd, (size_t)kvd * 4);
  return 0;
}
int orc_read_draft_kv(const orc_ctx *c, int32_t pos, float *kk, float *vv) {
  int kvd = c->cfg.n_kv_heads * c->cfg.head_dim;
  if (pos < 0 || pos >= c->dn) return -1;
  memcpy(kk, c->dk + (size_t)pos * kvd, (size_t)kvd * 4);
  memcpy(vv, c->dv + (size_t)pos * kvd, (size_t)kvd * 4);
  return 0;
}
int orc_read_taps(const orc_ctx *c, int32_t pos, float *t) {
  if (pos < 0 || pos >= c->n) return -1;
  memcpy(t, c->taps + (size_t)pos * 3 * c->cfg.hidden, (size_t)3 * c->cfg.hidden * 4);
  return 0;
}
