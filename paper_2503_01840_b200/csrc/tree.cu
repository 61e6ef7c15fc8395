// Integer / fp32-compare kernels of the step: per-row log-softmax + top-k, dynamic-tree expansion
// (Section 2.2: expand by draft confidence, cumulative log-probability as the node value), the
// end-of-draft pruning ("rerank") that fixes the verified tree and its ancestor masks, per-node
// argmax, greedy acceptance (Section 2.1 at temperature 0) and KV-cache compaction.
#include "state.cuh"

namespace spec {

size_t draft_tree_step_smem(int tiles, int K);
int draft_tree_cand_ld(int tiles);

// ---------------------------------------------------------------- block argmax helpers
struct VI { float v; int i; };

__device__ __forceinline__ VI block_best(VI x, VI *sh) {
  for (int o = 16; o > 0; o >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, x.v, o);
    int oi = __shfl_xor_sync(0xffffffffu, x.i, o);
    if (oi >= 0 && (x.i < 0 || before(ov, oi, x.v, x.i))) { x.v = ov; x.i = oi; }
  }
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = blockDim.x >> 5;
  if (l == 0) sh[w] = x;
  __syncthreads();
  if (w == 0) {
    VI t = (l < nw) ? sh[l] : VI{0.0f, -1};
    for (int o = 16; o > 0; o >>= 1) {
      float ov = __shfl_xor_sync(0xffffffffu, t.v, o);
      int oi = __shfl_xor_sync(0xffffffffu, t.i, o);
      if (oi >= 0 && (t.i < 0 || before(ov, oi, t.v, t.i))) { t.v = ov; t.i = oi; }
    }
    if (l == 0) sh[0] = t;
  }
  __syncthreads();
  VI r = sh[0];
  __syncthreads();
  return r;
}

__global__ void __launch_bounds__(256) argmax_kernel(const float *__restrict__ logits, int n, int32_t *__restrict__ out) {
  pdl_wait();
  pdl_trigger();
  __shared__ VI sh[32];
  const float *z = logits + (size_t)blockIdx.x * n;
  VI b{0.0f, -1};
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    float v = z[i];
    if (b.i < 0 || before(v, i, b.v, b.i)) { b.v = v; b.i = i; }
  }
  b = block_best(b, sh);
  if (threadIdx.x == 0) out[blockIdx.x] = b.i;
}
void launch_argmax(const float *logits, int rows, int n, int32_t *idx, cudaStream_t s) {
  launch_k(argmax_kernel, dim3(rows), dim3(256), 0, s, logits, n, idx);
}

// log-softmax + top-K, (value desc, index asc).  Row r reads logits row src_row[r] when given.
__global__ void __launch_bounds__(256) logsoftmax_topk_kernel(const float *__restrict__ logits, const int32_t *src_row,
                                                              int n, int K, int32_t *__restrict__ idx,
                                                              float *__restrict__ lp) {
  pdl_wait();
  pdl_trigger();
  __shared__ VI sh[32];
  __shared__ float shf[32];
  int r = blockIdx.x;
  int sr = src_row ? src_row[r] : r;
  if (sr < 0) {
    for (int c = threadIdx.x; c < K; c += blockDim.x) { idx[(size_t)r * K + c] = 0; lp[(size_t)r * K + c] = 0.0f; }
    return;
  }
  const float *z = logits + (size_t)sr * n;
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < n; i += blockDim.x) mx = fmaxf(mx, z[i]);
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = shf[0];
  for (int w = 1; w < (int)(blockDim.x >> 5); w++) mx = fmaxf(mx, shf[w]);
  __syncthreads();
  float sum = 0.0f;
  for (int i = threadIdx.x; i < n; i += blockDim.x) sum += expf(z[i] - mx);
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = sum;
  __syncthreads();
  sum = 0.0f;
  for (int w = 0; w < (int)(blockDim.x >> 5); w++) sum += shf[w];
  float lse = logf(sum);
  __syncthreads();
  float pv = INFINITY;
  int pi = -1;
  for (int c = 0; c < K; c++) {
    VI b{0.0f, -1};
    for (int i = threadIdx.x; i < n; i += blockDim.x) {
      float v = (z[i] - mx) - lse;
      bool after_prev = (pi < 0) || before(pv, pi, v, i);
      if (after_prev && (b.i < 0 || before(v, i, b.v, b.i))) { b.v = v; b.i = i; }
    }
    b = block_best(b, sh);
    if (threadIdx.x == 0) { idx[(size_t)r * K + c] = b.i; lp[(size_t)r * K + c] = b.v; }
    pv = b.v; pi = b.i;
  }
}
void launch_logsoftmax_topk(const float *logits, int rows, int n, int K, int32_t *idx, float *lp, cudaStream_t s) {
  launch_k(logsoftmax_topk_kernel, dim3(rows), dim3(256), 0, s, logits, nullptr, n, K, idx, lp);
}
void launch_logsoftmax_topk_rows(const float *logits, const int32_t *src_row, int rows, int n, int K, int32_t *idx,
                                 float *lp, cudaStream_t s) {
  launch_k(logsoftmax_topk_kernel, dim3(rows), dim3(256), 0, s, logits, src_row, n, K, idx, lp);
}


// ---------------------------------------------------------------- two-stage log-softmax + top-K
// Stage 1: one CTA per (row, chunk of TOPK_CHUNK logits): chunk maximum, sum of exp relative to it, and
// the chunk's K best (value desc, index asc).  Stage 2: one CTA per row merges the chunks: log-sum-exp
// of the row and the K best of the chunk candidates, ranked by counting.
constexpr int TOPK_CHUNK = 1024;
constexpr int TOPK_MAXK = 16;

__global__ void __launch_bounds__(256) topk_partial_kernel(const float *__restrict__ logits, const int32_t *src_row, int n,
                                                           int K, int nch, float *__restrict__ pmax,
                                                           float *__restrict__ psum, float *__restrict__ cval,
                                                           int32_t *__restrict__ cidx) {
  pdl_wait();
  pdl_trigger();
  // Warp w owns the 128 consecutive logits base + 128 w ...: it finds its own K best with shuffles only (no block
  // barrier per round); the 8 x K warp candidates are then ranked against each other by counting.
  __shared__ float shf[8];
  __shared__ float wv[8 * TOPK_MAXK];
  __shared__ int32_t wi[8 * TOPK_MAXK];
  const int r = blockIdx.y, ch = blockIdx.x;
  const int sr = src_row ? src_row[r] : r;
  if (sr < 0) return;
  const float *z = logits + (size_t)sr * n;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int base = ch * TOPK_CHUNK + warp * 128;
  float v[4];
  int id[4];
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < 4; j++) {
    id[j] = base + j * 32 + lane;
    v[j] = id[j] < n ? z[id[j]] : -INFINITY;
    if (id[j] >= n) id[j] = -1;
    mx = fmaxf(mx, v[j]);
  }
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if (lane == 0) shf[warp] = mx;
  __syncthreads();
  mx = shf[0];
  for (int w = 1; w < 8; w++) mx = fmaxf(mx, shf[w]);
  __syncthreads();
  float sum = 0.0f;
#pragma unroll
  for (int j = 0; j < 4; j++) sum += id[j] >= 0 ? expf(v[j] - mx) : 0.0f;
  for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
  if (lane == 0) shf[warp] = sum;
  // ---- this warp's K best, best first
  for (int c = 0; c < K; c++) {
    float bv = 0.0f;
    int bi = -1;
#pragma unroll
    for (int j = 0; j < 4; j++)
      if (id[j] >= 0 && (bi < 0 || before(v[j], id[j], bv, bi))) { bv = v[j]; bi = id[j]; }
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (oi >= 0 && (bi < 0 || before(ov, oi, bv, bi))) { bv = ov; bi = oi; }
    }
#pragma unroll
    for (int j = 0; j < 4; j++)
      if (id[j] == bi) id[j] = -1;            // taken (bi is -1 only when the warp's range is exhausted)
    if (lane == 0) { wv[warp * K + c] = bv; wi[warp * K + c] = bi; }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.0f;
    for (int w = 0; w < 8; w++) t += shf[w];
    pmax[(size_t)r * nch + ch] = mx;
    psum[(size_t)r * nch + ch] = t;
  }
  // ---- the chunk's K best of the 8 K warp candidates, by rank (value desc, index asc)
  const int nc = 8 * K;
  int my = -1;
  float mv = 0.0f;
  if ((int)threadIdx.x < nc) { my = wi[threadIdx.x]; mv = wv[threadIdx.x]; }
  const int nvalid = __syncthreads_count(my >= 0);
  if (my >= 0) {
    int rank = 0;
    for (int j = 0; j < nc; j++) rank += (wi[j] >= 0 && before(wv[j], wi[j], mv, my)) ? 1 : 0;
    if (rank < K) {
      cval[((size_t)r * nch + ch) * K + rank] = mv;
      cidx[((size_t)r * nch + ch) * K + rank] = my;
    }
  }
  for (int c = nvalid + (int)threadIdx.x; c < K; c += blockDim.x) {      // fewer than K logits in the chunk
    cval[((size_t)r * nch + ch) * K + c] = 0.0f;
    cidx[((size_t)r * nch + ch) * K + c] = -1;
  }
}

__global__ void __launch_bounds__(256) topk_merge_kernel(const int32_t *src_row, int K, int nch, const float *__restrict__ pmax,
                                                         const float *__restrict__ psum, const float *__restrict__ cval,
                                                         const int32_t *__restrict__ cidx, int32_t *__restrict__ idx,
                                                         float *__restrict__ lp) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned char smraw[];
  __shared__ float shf[32];
  int r = blockIdx.x;
  int sr = src_row ? src_row[r] : r;
  if (sr < 0) {
    for (int c = threadIdx.x; c < K; c += blockDim.x) { idx[(size_t)r * K + c] = 0; lp[(size_t)r * K + c] = 0.0f; }
    return;
  }
  int nc = nch * K;
  float *cv = (float *)smraw;              // [nc]
  int32_t *ci = (int32_t *)(cv + nc);      // [nc]
  float *pm = (float *)(ci + nc);          // [nch]
  float *ps = pm + nch;                    // [nch]
  __shared__ float sv[TOPK_MAXK * TOPK_MAXK];      // candidates that can still be among the K best
  __shared__ int32_t si[TOPK_MAXK * TOPK_MAXK];
  __shared__ int nsurv, thr_i;
  __shared__ float thr_v;
  for (int i = threadIdx.x; i < nc; i += blockDim.x) { cv[i] = cval[(size_t)r * nc + i]; ci[i] = cidx[(size_t)r * nc + i]; }
  float mx = -INFINITY;
  for (int i = threadIdx.x; i < nch; i += blockDim.x) {
    float m = pmax[(size_t)r * nch + i];
    pm[i] = m; ps[i] = psum[(size_t)r * nch + i];
    mx = fmaxf(mx, m);
  }
  for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  if ((threadIdx.x & 31) == 0) shf[threadIdx.x >> 5] = mx;
  if (threadIdx.x == 0) { nsurv = 0; thr_i = -1; thr_v = 0.0f; }
  __syncthreads();
  mx = shf[0];
  for (int w = 1; w < 8; w++) mx = fmaxf(mx, shf[w]);
  __syncthreads();
  // chunk sums are combined in chunk order by one thread: the result does not depend on the launch shape
  if (threadIdx.x == 0) {
    float t = 0.0f;
    for (int i = 0; i < nch; i++) t += ps[i] * expf(pm[i] - mx);
    shf[0] = logf(t);
  }
  // A chunk's candidates are stored best first.  With t = the K-th best of the chunks' best candidates, K
  // candidates are at least as good as t, so a candidate after t cannot be among the K best of the row.
  for (int ch = (int)threadIdx.x - 32; ch < nch; ch += (int)blockDim.x - 32) {       // warp 0 is busy with the sum
    if (ch < 0) break;
    int c0 = ch * K, my = ci[c0];
    if (my < 0) continue;
    float v = cv[c0];
    int rank = 0;
    for (int j = 0; j < nch; j++) rank += (ci[j * K] >= 0 && before(cv[j * K], ci[j * K], v, my)) ? 1 : 0;
    if (rank == K - 1) { thr_v = v; thr_i = my; }
  }
  __syncthreads();
  float lse = shf[0];
  const float tv = thr_v;
  const int ti = thr_i;
  for (int i = threadIdx.x; i < nc; i += blockDim.x) {
    int my = ci[i];
    if (my < 0 || (ti >= 0 && before(tv, ti, cv[i], my))) continue;
    int pos = atomicAdd(&nsurv, 1);        // at most K chunks x K candidates survive; their order does not matter
    if (pos < TOPK_MAXK * TOPK_MAXK) { sv[pos] = cv[i]; si[pos] = my; }
  }
  __syncthreads();
  int ns = nsurv < TOPK_MAXK * TOPK_MAXK ? nsurv : TOPK_MAXK * TOPK_MAXK;
  for (int i = threadIdx.x; i < ns; i += blockDim.x) {
    int my = si[i];
    float v = sv[i];
    int rank = 0;
    for (int j = 0; j < ns; j++) rank += before(sv[j], si[j], v, my) ? 1 : 0;
    if (rank < K) { idx[(size_t)r * K + rank] = my; lp[(size_t)r * K + rank] = (v - mx) - lse; }
  }
}

size_t topk_scratch_bytes(int rows, int n, int K) {
  size_t nch = (size_t)(n + TOPK_CHUNK - 1) / TOPK_CHUNK;
  return (size_t)rows * nch * (2 + 2 * (size_t)K) * 4 + 256;
}

// scratch: topk_scratch_bytes(rows, n, K) bytes.  Returns the number of kernels launched.
int launch_topk2(const float *logits, const int32_t *src_row, int rows, int n, int K, int32_t *idx, float *lp, void *scratch,
                 cudaStream_t s) {
  int nch = (n + TOPK_CHUNK - 1) / TOPK_CHUNK;
  float *pmax = (float *)scratch;
  float *psum = pmax + (size_t)rows * nch;
  float *cval = psum + (size_t)rows * nch;
  int32_t *cidx = (int32_t *)(cval + (size_t)rows * nch * K);
  {
    // Launched without the programmatic-dependent-launch attribute: pre-launched under the LM-head GEMM, the
    // rows x nch small CTAs become resident wherever that kernel leaves room, packed onto a few SMs instead of spread
    // over all of them, and the pair ran 8 us slower per draft pass (measured on the 8B shapes).
    const bool pdl = tl_pdl;
    tl_pdl = false;
    launch_k(topk_partial_kernel, dim3(nch, rows), dim3(256), 0, s, logits, src_row, n, K, nch, pmax, psum, cval, cidx);
    tl_pdl = pdl;
  }
  size_t smem = (size_t)nch * K * 8 + (size_t)nch * 8;
  static SmemLimit limit;
  if (smem > 48 * 1024) limit.ensure(topk_merge_kernel, (int)smem);
  launch_k(topk_merge_kernel, dim3(rows), dim3(256), smem, s, src_row, K, nch, pmax, psum, cval, cidx, idx, lp);
  return 2;
}

// ---------------------------------------------------------------- argmax over per-tile candidates
// y[r] = index of the best (value desc, index asc) of best_val/best_idx[t][r], t < tiles.
__global__ void __launch_bounds__(256) argmax_merge_kernel(const float *__restrict__ best_val, const int32_t *__restrict__ best_idx,
                                                           int tiles, int ld, int32_t *__restrict__ out) {
  pdl_wait();
  pdl_trigger();
  __shared__ VI sh[32];
  int r = blockIdx.x;
  VI b{0.0f, -1};
  for (int t = threadIdx.x; t < tiles; t += blockDim.x) {
    float v = best_val[(size_t)t * ld + r];
    int i = best_idx[(size_t)t * ld + r];
    if (i >= 0 && (b.i < 0 || before(v, i, b.v, b.i))) { b.v = v; b.i = i; }
  }
  b = block_best(b, sh);
  if (threadIdx.x == 0) out[r] = b.i;
}
void launch_argmax_merge(const float *best_val, const int32_t *best_idx, int tiles, int ld, int rows, int32_t *out, cudaStream_t s) {
  launch_k(argmax_merge_kernel, dim3(rows), dim3(256), 0, s, best_val, best_idx, tiles, ld, out);
}

__device__ __forceinline__ int block_sum_int(int v) {
  __shared__ int acc;
  if (threadIdx.x == 0) acc = 0;
  __syncthreads();
  if (v) atomicAdd(&acc, v);
  __syncthreads();
  return acc;
}

// ---------------------------------------------------------------- step set-up: rows of the extend pass
// Row b*Pmax + j is pending entry j of sequence b: position n-P+j, causal among the pending rows.
__global__ void prep_extend_kernel(SeqState st, TreeBufs tb, RowMeta m, int need_positions, int32_t *status) {
  pdl_wait();
  pdl_trigger();
  int b = blockIdx.x, j = threadIdx.x;
  int n = st.n[b], P = st.P[b];
  bool ok = (n + need_positions <= st.cap[b]) && P >= 1 && P <= tb.Pmax;
  // rank of this sequence by (length desc, index asc): longest sequences get their attention CTAs first, which
  // packs CTAs of unequal length into fewer waves
  int longer = 0;
  for (int o = j; o < (int)gridDim.x; o += blockDim.x) {
    int no = st.n[o];
    longer += (no > n || (no == n && o < b)) ? 1 : 0;
  }
  longer = block_sum_int(longer);
  if (j == 0) {
    st.order[longer] = b;
    st.active[b] = ok ? 1 : 0;
    st.last_row[b] = ok ? b * tb.Pmax + P - 1 : -1;
    if (!ok) set_status(status, ST_CAPACITY, 10, b, n);
    tb.frontier[(size_t)b * tb.D * tb.K] = 0;
    tb.pool_tok[(size_t)b * (tb.pool + 1)] = st.root[b];
    tb.pool_parent[(size_t)b * (tb.pool + 1)] = -1;
    tb.pool_depth[(size_t)b * (tb.pool + 1)] = 0;
    tb.pool_score[(size_t)b * (tb.pool + 1)] = 0.0f;
  }
  if (j >= tb.Pmax) return;
  int r = b * tb.Pmax + j;
  bool valid = ok && j < P;
  m.seq[r] = valid ? b : -1;
  m.pos[r] = valid ? n - P + j : 0;
  m.kvpos[r] = valid ? n - P + j : 0;
  m.ctx[r] = valid ? n - P : 0;
  m.tail_base[r] = valid ? n - P : 0;
  m.mask_lo[r] = valid ? ((j >= 63) ? ~0ull : ((1ull << (j + 1)) - 1ull)) : 0ull;
  m.mask_hi[r] = 0ull;
  m.tok[r] = valid ? tb.pend_tok[b * tb.Pmax + j] : 0;
}
void launch_prep_extend(SeqState st, TreeBufs tb, RowMeta m, int B, int need_positions, int32_t *status, cudaStream_t s) {
  int threads = ((tb.Pmax + 31) / 32) * 32;
  launch_k(prep_extend_kernel, dim3(B), dim3(threads), 0, s, st, tb, m, need_positions, status);
}

// ---------------------------------------------------------------- dynamic-tree expansion after draft pass `pass` (1-based)
// Adds this pass's children to the pool (cumulative log-prob scores), picks the next frontier (the K
// best of the level) and writes the row metadata of the next draft pass.
__global__ void __launch_bounds__(256) expand_kernel(SeqState st, TreeBufs tb, RowMeta m, const int32_t *__restrict__ d2t,
                                                     int pass) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned char smraw[];
  int K = tb.K, D = tb.D, b = blockIdx.x;
  int nch = (pass == 1) ? K : K * K;        // children created by this pass
  float *cs = (float *)smraw;               // [nch] child scores
  uint64_t *pm_lo = (uint64_t *)(cs + ((nch + 1) & ~1));   // [K] parent masks
  uint64_t *pm_hi = pm_lo + K;
  int32_t *newf = (int32_t *)(pm_hi + K);   // [K] local child index of the new frontier
  int32_t *ctok = newf + K;                 // [nch] child tokens (target ids)
  // every load that does not depend on another is issued up front: the kernel is a chain of L2 round trips otherwise
  const int active = st.active[b], n = st.n[b], last_row = st.last_row[b];
  if (!active) {   // skipped sequence: its rows of the next pass are padding
    for (int rr = threadIdx.x; rr < K; rr += blockDim.x) { m.seq[b * K + rr] = -1; m.tok[b * K + rr] = 0; m.pos[b * K + rr] = 0; }
    return;
  }
  size_t pb = (size_t)b * (tb.pool + 1);
  int base = (pass == 1) ? 0 : K + (pass - 2) * K * K;     // pool index of child 0 is base + 1
  for (int r = threadIdx.x; r < K; r += blockDim.x) {
    pm_lo[r] = (pass == 1) ? 0ull : m.mask_lo[b * K + r];
    pm_hi[r] = (pass == 1) ? 0ull : m.mask_hi[b * K + r];
  }
  for (int c = threadIdx.x; c < nch; c += blockDim.x) {
    int r = (pass == 1) ? 0 : c / K, cc = (pass == 1) ? c : c % K;
    int row = (pass == 1) ? b : b * K + r;                  // row of the top-k output
    int u = (pass == 1) ? 0 : tb.front_cur[b * K + r];
    const float lp = tb.tk_lp[(size_t)row * K + cc];
    const int tokid = d2t[tb.tk_idx[(size_t)row * K + cc]];
    float sc = tb.pool_score[pb + u] + lp;
    int ci = base + c + 1;
    tb.pool_tok[pb + ci] = tokid;
    ctok[c] = tokid;
    tb.pool_parent[pb + ci] = u;
    tb.pool_depth[pb + ci] = pass;
    tb.pool_score[pb + ci] = sc;
    cs[c] = sc;
  }
  __syncthreads();
  if (pass >= D) return;
  // next frontier: rank by (score desc, pool index asc)
  for (int c = threadIdx.x; c < nch; c += blockDim.x) {
    float s = cs[c];
    int rank = 0;
    for (int j = 0; j < nch; j++) rank += (cs[j] > s || (cs[j] == s && j < c)) ? 1 : 0;
    if (rank < K) newf[rank] = c;
  }
  __syncthreads();
  for (int rr = threadIdx.x; rr < K; rr += blockDim.x) {
    int c = newf[rr];
    int ci = base + c + 1;
    int pr = (pass == 1) ? 0 : c / K;                       // parent's rank in the current pass
    int row = b * K + rr;
    int slot = (pass - 1) * K + rr;
    tb.front_cur[b * K + rr] = ci;
    tb.frontier[((size_t)b * D + pass) * K + rr] = ci;
    tb.feat_row[row] = (pass == 1) ? last_row : b * K + pr;
    uint64_t lo = pm_lo[pr], hi = pm_hi[pr];
    if (slot < 64) lo |= 1ull << slot; else hi |= 1ull << (slot - 64);
    m.seq[row] = b;
    m.pos[row] = n + pass - 1;
    m.kvpos[row] = n + slot;
    m.ctx[row] = n;
    m.tail_base[row] = n;
    m.mask_lo[row] = lo;
    m.mask_hi[row] = hi;
    m.tok[row] = ctok[c];
  }
}
void launch_expand(SeqState st, TreeBufs tb, RowMeta m, const int32_t *d2t, int pass, int B, cudaStream_t s) {
  int K = tb.K, nch = K * K;
  size_t smem = (size_t)((nch + 1) & ~1) * 4 + (size_t)K * 16 + (size_t)K * 4 + (size_t)nch * 4 + 16;
  launch_k(expand_kernel, dim3(B), dim3(256), smem, s, st, tb, m, d2t, pass);
}

// One warp merges the per-tile candidates of one row (the draft LM head's epilogue left, per 128-logit tile, the tile
// maximum, the sum of exp relative to it and the tile's K best logits, best first): the row's log-sum-exp and its K best
// (value desc, index asc) as log-probabilities.  Layout: candidates [row][ld][K], statistics [row][ld], ld a multiple of
// 4 and the arrays 16-byte aligned, so a row is fetched with 16-byte asynchronous copies that are all in flight at once.
// stage_v / stage_i: ld * K floats / ints of 16-byte aligned scratch owned by the warp; tiles <= 256, K <= 15.
__device__ __forceinline__ void merge_tile_candidates(const float *__restrict__ cand_val, const int32_t *__restrict__ cand_idx,
                                                      const float *__restrict__ cand_max, const float *__restrict__ cand_sum,
                                                      int tiles, int ld, int row, int K, float *stage_v, int32_t *stage_i,
                                                      int32_t *out_id, float *out_lp) {
  const int lane = threadIdx.x & 31;
  const int nvec = ld * K / 4;                           // ld % 4 == 0
  const float4 *gv = (const float4 *)(cand_val + (size_t)row * ld * K);
  const int4 *gi = (const int4 *)(cand_idx + (size_t)row * ld * K);
  for (int e = lane; e < nvec; e += 32) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(stage_v + 4 * e)), "l"(gv + e) : "memory");
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(stage_i + 4 * e)), "l"(gi + e) : "memory");
  }
  asm volatile("cp.async.commit_group;" ::: "memory");
  // the tile statistics meanwhile: at most 8 tiles per lane, all loads issued before the first use
  float pm[8], ps[8];
#pragma unroll
  for (int j = 0; j < 8; j++) {
    const int t = lane + 32 * j;
    pm[j] = t < tiles ? cand_max[(size_t)row * ld + t] : -INFINITY;
    ps[j] = t < tiles ? cand_sum[(size_t)row * ld + t] : 0.0f;
  }
  float mx = -INFINITY;
#pragma unroll
  for (int j = 0; j < 8; j++) mx = fmaxf(mx, pm[j]);
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  float sum = 0.0f;                                      // lane l adds its tiles in tile order, then a fixed shuffle tree
#pragma unroll
  for (int j = 0; j < 8; j++) sum += (lane + 32 * j < tiles) ? ps[j] * expf(pm[j] - mx) : 0.0f;
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  const float lse = logf(sum);
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncwarp();
  // a tile's candidates are stored best first: only its current head can be the next winner.  hp = head position of
  // each of this lane's (at most 8) tiles, four bits each.
  unsigned hp = 0;
  for (int c = 0; c < K; c++) {
    float bv = 0.0f;
    int bi = -1, bj = 0;
#pragma unroll
    for (int j = 0; j < 8; j++) {
      const int t = lane + 32 * j, h = (hp >> (4 * j)) & 15;
      if (t < tiles && h < K) {
        const int ci = stage_i[t * K + h];
        const float cv = stage_v[t * K + h];
        if (ci >= 0 && (bi < 0 || before(cv, ci, bv, bi))) { bv = cv; bi = ci; bj = j; }
      }
    }
    unsigned wk;
    const int wi = warp_best(ordered_key(bv), bi, &wk);  // two redux instructions instead of a shuffle tree
    if (wi >= 0 && wi == bi) hp += 1u << (4 * bj);       // indices are unique: exactly one lane owns the winner
    if (lane == 0) { out_id[c] = wi < 0 ? 0 : wi; out_lp[c] = wi < 0 ? 0.0f : (key_value(wk) - mx) - lse; }
  }
  __syncwarp();
}

// The merge alone, one warp per row (per-kernel parity tests of the LM-head epilogue + merge).
__global__ void __launch_bounds__(256) merge_candidates_kernel(const float *cand_val, const int32_t *cand_idx, const float *cand_max,
                                                               const float *cand_sum, int tiles, int ld, int rows, int K,
                                                               int32_t *__restrict__ idx, float *__restrict__ lp) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(16) unsigned char smraw[];
  const int warp = threadIdx.x >> 5, row = blockIdx.x * 8 + warp;
  if (row >= rows) return;
  float *stage_v = (float *)smraw + (size_t)warp * 2 * ld * K;
  merge_tile_candidates(cand_val, cand_idx, cand_max, cand_sum, tiles, ld, row, K, stage_v, (int32_t *)(stage_v + ld * K),
                        idx + (size_t)row * K, lp + (size_t)row * K);
}
int launch_merge_candidates(const float *cand_val, const int32_t *cand_idx, const float *cand_max, const float *cand_sum, int tiles,
                            int ld, int rows, int K, int32_t *idx, float *lp, cudaStream_t s) {
  const size_t smem = draft_tree_step_smem(tiles, K);
  if (!smem || ld != draft_tree_cand_ld(tiles)) return -1;
  static SmemLimit limit;
  if (smem > 48 * 1024 && !limit.ensure(merge_candidates_kernel, (int)smem)) return -6;
  launch_k(merge_candidates_kernel, dim3((rows + 7) / 8), dim3(256), smem, s, cand_val, cand_idx, cand_max, cand_sum, tiles, ld, rows, K, idx, lp);
  return 0;
}

// ---------------------------------------------------------------- one launch between two draft passes
// After the draft LM head of pass `pass` (whose epilogue left, per 128-logit tile and row, the tile maximum, the sum of
// exp relative to it and the tile's K best logits): merges the tiles into each row's log-softmax top-K, adds the children
// to the candidate pool with cumulative log-probability scores, picks the next frontier, writes the next pass's row
// metadata, and builds that pass's inputs (the FC2 input [feature ; embedding] of every frontier node and its RoPE
// angles).  Section 2.2 (dynamic draft tree: expansion by the draft's confidence), Section 3.1 (the draft's own output
// is the feature of the next step), Appendix A (nodes per expansion).
//
// grid (B, Z): the Z CTAs of a sequence each redo the small merge + expansion (same inputs, same order of operations,
// hence identical results) and then take one Z-th of the elements of the next pass's inputs; only CTA z = 0 writes the
// tree state.  Nothing a CTA reads is written by another CTA of the launch.
struct TreeStepArgs {
  SeqState st; TreeBufs tb; RowMeta m;
  const int32_t *d2t;
  int pass;                       // 1-based draft pass that just ran
  const float *cand_val, *cand_max, *cand_sum; const int32_t *cand_idx; int tiles, ld;   // [rows][ld][K], [rows][ld]
  const float *x; const bf16 *embed; bf16 *cat; int k;                                    // next pass's FC2 input
  const double *inv_freq; float2 *cs; int half;                                           // next pass's RoPE angles
};

constexpr int TREE_WARPS = 10;   // one warp per row of a top-10 level
__global__ void __launch_bounds__(TREE_WARPS * 32) draft_tree_step_kernel(const TreeStepArgs a) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ __align__(16) unsigned char smraw[];
  const TreeBufs &tb = a.tb;
  const int K = tb.K, D = tb.D, b = blockIdx.x, pass = a.pass;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nrows = (pass == 1) ? 1 : K;                 // rows of this sequence in the pass that just ran
  const int nchild = nrows * K;
  // shared memory: per-warp candidate staging, then the expansion's small arrays
  const int ncand = a.ld * K;
  float *stage_v = (float *)smraw + (size_t)warp * 2 * ncand;      // [ld][K] values, then indices
  int32_t *stage_i = (int32_t *)(stage_v + ncand);
  unsigned char *tail = smraw + (size_t)TREE_WARPS * 2 * ncand * 4;
  float *tk_lp = (float *)tail;                          // [nrows][K]
  int32_t *tk_id = (int32_t *)(tk_lp + K * K);           // [nrows][K] draft ids
  float *cscore = (float *)(tk_id + K * K);              // [nchild]
  int32_t *ctok = (int32_t *)(cscore + K * K);           // [nchild] target ids
  int32_t *newf = ctok + K * K;                          // [K] child index (within the level) of the new frontier
  int32_t *par_u = newf + K;                             // [K] pool index of the node each row of this pass processed
  float *par_sc = (float *)(par_u + K);                  // [K] its score
  const int active = a.st.active[b], n = a.st.n[b], last_row = a.st.last_row[b];
  const size_t pb = (size_t)b * (tb.pool + 1);
  const int base = (pass == 1) ? 0 : K + (pass - 2) * K * K;       // pool index of child 0 is base + 1
  const bool writer = blockIdx.y == 0;
  if (!active) {   // skipped sequence: its rows of the next pass are padding
    if (pass < D) {
      if (writer)
        for (int rr = threadIdx.x; rr < K; rr += blockDim.x) { a.m.seq[b * K + rr] = -1; a.m.tok[b * K + rr] = 0; a.m.pos[b * K + rr] = 0; }
      const size_t total = (size_t)K * 2 * a.k;
      for (size_t e = (size_t)blockIdx.y * blockDim.x + threadIdx.x; e < total; e += (size_t)gridDim.y * blockDim.x)
        a.cat[(size_t)b * K * 2 * a.k + e] = __float2bfloat16_rn(0.0f);
    }
    return;
  }
  // the parents of this pass's rows (two dependent loads) are fetched while the candidates are on their way
  if ((int)threadIdx.x < nrows) {
    const int u = (pass == 1) ? 0 : tb.frontier[((size_t)b * D + pass - 1) * K + threadIdx.x];
    par_u[threadIdx.x] = u;
    par_sc[threadIdx.x] = tb.pool_score[pb + u];
  }
  // ---- 1. per row: log-sum-exp over the tiles and the K best of the tiles' candidates (value desc, index asc)
  for (int r = warp; r < nrows; r += TREE_WARPS) {
    const int row = (pass == 1) ? last_row : b * K + r;
    merge_tile_candidates(a.cand_val, a.cand_idx, a.cand_max, a.cand_sum, a.tiles, a.ld, row, K, stage_v, stage_i, tk_id + r * K,
                          tk_lp + r * K);
  }
  __syncthreads();
  if (writer) {   // kept for inspection: the top-K of this pass in the layout of the per-row kernels
    for (int i = threadIdx.x; i < nchild; i += blockDim.x) {
      const int row = (pass == 1) ? b : b * K + i / K;
      tb.tk_idx[(size_t)row * K + i % K] = tk_id[i];
      tb.tk_lp[(size_t)row * K + i % K] = tk_lp[i];
    }
  }
  // ---- 2. children join the pool with cumulative scores
  for (int c = threadIdx.x; c < nchild; c += blockDim.x) {
    const int r = c / K;
    const int u = par_u[r];                                // the node row r processed
    const float sc = par_sc[r] + tk_lp[c];
    const int tokid = a.d2t[tk_id[c]];
    cscore[c] = sc;
    ctok[c] = tokid;
    if (writer) {
      const int ci = base + c + 1;
      tb.pool_tok[pb + ci] = tokid;
      tb.pool_parent[pb + ci] = u;
      tb.pool_depth[pb + ci] = pass;
      tb.pool_score[pb + ci] = sc;
    }
  }
  __syncthreads();
  if (pass >= D) return;
  // ---- 3. next frontier: the K best children of the level, (score desc, pool index asc)
  for (int c = threadIdx.x; c < nchild; c += blockDim.x) {
    const float s = cscore[c];
    int rank = 0;
    for (int j = 0; j < nchild; j++) rank += (cscore[j] > s || (cscore[j] == s && j < c)) ? 1 : 0;
    if (rank < K) newf[rank] = c;
  }
  __syncthreads();
  {
    // the parents' masks are read by every writing thread before any row of the next pass is written
    const int rr = threadIdx.x;
    const bool mine = writer && rr < K;
    const int c = mine ? newf[rr] : 0;
    const int pr = c / K;                                  // parent's row in the pass that just ran (0 in pass 1)
    uint64_t lo = 0ull, hi = 0ull;
    if (mine && pass > 1) { lo = a.m.mask_lo[b * K + pr]; hi = a.m.mask_hi[b * K + pr]; }
    __syncthreads();
    if (mine) {
      const int ci = base + c + 1;
      const int row = b * K + rr;
      const int slot = (pass - 1) * K + rr;
      if (slot < 64) lo |= 1ull << slot; else hi |= 1ull << (slot - 64);
      tb.front_cur[b * K + rr] = ci;
      tb.frontier[((size_t)b * D + pass) * K + rr] = ci;
      tb.feat_row[row] = (pass == 1) ? last_row : b * K + pr;
      a.m.seq[row] = b;
      a.m.pos[row] = n + pass - 1;
      a.m.kvpos[row] = n + slot;
      a.m.ctx[row] = n;
      a.m.tail_base[row] = n;
      a.m.mask_lo[row] = lo;
      a.m.mask_hi[row] = hi;
      a.m.tok[row] = ctok[c];
    }
  }
  // ---- 4. inputs of the next pass: FC2 input [bf16(feature of the parent's row) ; embedding of the node's token] and
  // the RoPE angles of its position (double precision, rounded once), split over the CTAs of the sequence
  const int k = a.k, vpr = 2 * k / 8;                      // 8-element vectors per row (hidden % 8 == 0)
  for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < K * vpr; e += gridDim.y * blockDim.x) {
    const int rr = e / vpr, i = (e % vpr) * 8;
    const int c = newf[rr];
    uint4 out;
    if (i < k) {
      const int fr = (pass == 1) ? last_row : b * K + c / K;
      const float4 lo = *(const float4 *)(a.x + (size_t)fr * k + i), hi = *(const float4 *)(a.x + (size_t)fr * k + i + 4);
      __nv_bfloat162 p0 = __floats2bfloat162_rn(lo.x, lo.y), p1 = __floats2bfloat162_rn(lo.z, lo.w);
      __nv_bfloat162 p2 = __floats2bfloat162_rn(hi.x, hi.y), p3 = __floats2bfloat162_rn(hi.z, hi.w);
      out = make_uint4(*(uint32_t *)&p0, *(uint32_t *)&p1, *(uint32_t *)&p2, *(uint32_t *)&p3);
    } else {
      out = *(const uint4 *)(a.embed + (size_t)ctok[c] * k + (i - k));
    }
    *(uint4 *)(a.cat + ((size_t)(b * K + rr)) * 2 * k + i) = out;
  }
  const int nang = K * a.half;
  for (int e = blockIdx.y * blockDim.x + threadIdx.x; e < nang; e += gridDim.y * blockDim.x) {
    const int rr = e / a.half, i = e % a.half;
    double sn, cs_;
    sincos((double)(n + pass - 1) * a.inv_freq[i], &sn, &cs_);
    a.cs[(size_t)(b * K + rr) * a.half + i] = make_float2((float)cs_, (float)sn);
  }
}

// shared memory the launch needs; 0 when the shape does not fit the kernel (the caller then uses the separate kernels)
int draft_tree_cand_ld(int tiles) { return (tiles + 3) & ~3; }
size_t draft_tree_step_smem(int tiles, int K) {
  if (tiles > 256 || K > 15) return 0;
  const size_t need = (size_t)TREE_WARPS * 2 * draft_tree_cand_ld(tiles) * K * 4 + (size_t)K * K * 16 + (size_t)K * 12 + 64;
  return need <= 220 * 1024 ? need : 0;
}
int launch_draft_tree_step(SeqState st, TreeBufs tb, RowMeta m, const int32_t *d2t, int pass, const float *cand_val,
                           const int32_t *cand_idx, const float *cand_max, const float *cand_sum, int tiles, int ld, const float *x,
                           const bf16 *embed, bf16 *cat, int k, const double *inv_freq, float2 *cs, int half, int B, cudaStream_t s) {
  const size_t smem = draft_tree_step_smem(tiles, tb.K);
  if (!smem || ld != draft_tree_cand_ld(tiles) || (k % 8)) return -1;
  static SmemLimit limit;
  if (smem > 48 * 1024 && !limit.ensure(draft_tree_step_kernel, (int)smem)) return -6;
  TreeStepArgs a{st, tb, m, d2t, pass, cand_val, cand_max, cand_sum, cand_idx, tiles, ld, x, embed, cat, k, inv_freq, cs, half};
  const int Z = B >= 16 ? 1 : 8;        // CTAs per sequence that share the next pass's input assembly
  launch_k(draft_tree_step_kernel, dim3(B, Z), dim3(TREE_WARPS * 32), smem, s, a);
  return 0;
}

// ---------------------------------------------------------------- pruning + tree assembly
// Keeps the M = min(N-1, pool) best candidates (score desc, pool index asc), numbers them in pool
// order after the root and emits parents, depths, ancestor-or-self bit masks and the verify rows.
__global__ void __launch_bounds__(256) rerank_kernel(SeqState st, TreeBufs tb, RowMeta m) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ unsigned char smraw[];
  int b = blockIdx.x, pool = tb.pool, N = tb.N;
  float *sc = (float *)smraw;                       // [pool+1]
  int32_t *node_of = (int32_t *)(sc + pool + 1);    // [pool+1], -1 = dropped
  int32_t *par = node_of + pool + 1;                // [pool+1]
  int M = (N - 1 < pool) ? N - 1 : pool;
  size_t pb = (size_t)b * (pool + 1);
  int n = st.n[b];
  bool act = st.active[b] != 0;
  for (int i = threadIdx.x; i <= pool; i += blockDim.x) { sc[i] = tb.pool_score[pb + i]; par[i] = tb.pool_parent[pb + i]; }
  __syncthreads();
  for (int i = threadIdx.x; i <= pool; i += blockDim.x) {
    if (i == 0) { node_of[0] = 0; continue; }
    float s = sc[i];
    int rank = 0;
    for (int j = 1; j <= pool; j++) rank += (sc[j] > s || (sc[j] == s && j < i)) ? 1 : 0;
    node_of[i] = (rank < M) ? 1 : -1;
  }
  __syncthreads();
  // number the kept candidates in pool order
  int mine[4];   // pool <= 1024 with 256 threads -> up to 4 candidates each (checked on the host)
  int cnt = 0;
  for (int i = threadIdx.x; i <= pool; i += blockDim.x) {
    int idx = -1;
    if (i == 0) idx = 0;
    else if (node_of[i] > 0) {
      idx = 1;
      for (int j = 1; j < i; j++) idx += (node_of[j] > 0) ? 1 : 0;
    }
    mine[cnt++] = idx;
  }
  __syncthreads();
  cnt = 0;
  for (int i = threadIdx.x; i <= pool; i += blockDim.x) node_of[i] = mine[cnt++];
  __syncthreads();
  if (threadIdx.x == 0) tb.nn[b] = act ? M + 1 : 0;
  for (int i = threadIdx.x; i <= pool; i += blockDim.x) {
    int ni = node_of[i];
    if (ni < 0) continue;
    uint64_t mask = 0;
    for (int v = i, it = 0; v >= 0 && v <= pool && it < 64; v = par[v], it++) mask |= 1ull << (node_of[v] & 63);
    size_t t = (size_t)b * N + ni;
    int depth = tb.pool_depth[pb + i];
    tb.tok[t] = tb.pool_tok[pb + i];
    tb.parent[t] = (i == 0) ? -1 : node_of[par[i]];
    tb.depth[t] = depth;
    tb.poolidx[t] = i;
    tb.score[t] = sc[i];
    tb.mask[t] = mask;
    m.seq[t] = act ? b : -1;
    m.pos[t] = act ? n + depth : 0;
    m.kvpos[t] = act ? n + ni : 0;
    m.ctx[t] = act ? n : 0;
    m.tail_base[t] = act ? n : 0;
    m.mask_lo[t] = mask;
    m.mask_hi[t] = 0ull;
    m.tok[t] = act ? tb.pool_tok[pb + i] : 0;
  }
  // rows beyond the tree (only when pool < N-1) are padding
  for (int i = M + 1 + threadIdx.x; i < N; i += blockDim.x) {
    size_t t = (size_t)b * N + i;
    m.seq[t] = -1; m.pos[t] = 0; m.kvpos[t] = 0; m.ctx[t] = 0; m.tail_base[t] = 0;
    m.mask_lo[t] = 0; m.mask_hi[t] = 0; m.tok[t] = 0;
  }
}
void launch_rerank(SeqState st, TreeBufs tb, RowMeta m, int B, cudaStream_t s) {
  size_t smem = (size_t)(tb.pool + 1) * 12 + 16;
  launch_k(rerank_kernel, dim3(B), dim3(256), smem, s, st, tb, m);
}

// Tree of the root alone (plain autoregressive decoding on the same kernels): one row per sequence.
__global__ void plain_tree_kernel(SeqState st, TreeBufs tb, RowMeta m, int B) {
  pdl_wait();
  pdl_trigger();
  int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  int n = st.n[b];
  bool act = n + 1 <= st.cap[b];
  st.active[b] = act ? 1 : 0;
  tb.nn[b] = act ? 1 : 0;
  tb.tok[b] = st.root[b]; tb.parent[b] = -1; tb.depth[b] = 0; tb.poolidx[b] = 0; tb.score[b] = 0.0f; tb.mask[b] = 1ull;
  m.seq[b] = act ? b : -1; m.pos[b] = n; m.kvpos[b] = n; m.ctx[b] = n; m.tail_base[b] = n;
  m.mask_lo[b] = 1ull; m.mask_hi[b] = 0ull; m.tok[b] = act ? st.root[b] : 0;
}
void launch_plain_tree(SeqState st, TreeBufs tb, RowMeta m, int B, cudaStream_t s) {
  launch_k(plain_tree_kernel, dim3((B + 63) / 64), dim3(64), 0, s, st, tb, m, B);
}

// ---------------------------------------------------------------- greedy acceptance
// Follow, from the root, the child whose token equals the target's argmax at the current node.
__global__ void accept_kernel(SeqState st, TreeBufs tb, int rows_per_seq) {
  pdl_wait();
  pdl_trigger();
  int b = blockIdx.x;
  int Pmax = tb.Pmax;
  int nn = tb.nn[b];
  // the walk is serial: the tree goes to shared memory first, so that no iteration waits for a global load
  __shared__ int32_t tok[64], par[64], y[64];
  for (int i = threadIdx.x; i < nn && i < 64; i += blockDim.x) {
    tok[i] = tb.tok[(size_t)b * rows_per_seq + i];
    par[i] = tb.parent[(size_t)b * rows_per_seq + i];
    y[i] = tb.y[(size_t)b * rows_per_seq + i];
  }
  __syncthreads();
  if (threadIdx.x != 0) return;
  if (!st.active[b] || nn < 1) { tb.out_cnt[b] = 0; return; }
  int cur = 0, a = 0;
  tb.path[b * Pmax] = 0;
  while (a + 1 < Pmax) {
    int nxt = -1;
    for (int c = cur + 1; c < nn; c++)
      if (par[c] == cur && tok[c] == y[cur]) { nxt = c; break; }
    if (nxt < 0) break;
    tb.out_ids[b * Pmax + a] = tok[nxt];
    tb.pend_tok[b * Pmax + a] = tok[nxt];
    cur = nxt;
    tb.path[b * Pmax + (++a)] = cur;
  }
  tb.out_ids[b * Pmax + a] = y[cur];
  tb.pend_tok[b * Pmax + a] = y[cur];
  for (int j = a + 1; j < Pmax; j++) tb.out_ids[b * Pmax + j] = -1;
  tb.out_cnt[b] = a + 1;
  int n = st.n[b];
  st.n_prev[b] = n;
  st.n[b] = n + a + 1;
  st.P[b] = a + 1;
  st.root[b] = y[cur];
}
void launch_accept(SeqState st, TreeBufs tb, int B, int rows_per_seq, cudaStream_t s) {
  launch_k(accept_kernel, dim3(B), dim3(32), 0, s, st, tb, rows_per_seq);
}

// ---------------------------------------------------------------- stochastic acceptance (temperature > 0)
// Section 2.1's rule on the deterministic top-K tree: child c of the current node is accepted with probability
// p(tok[c]) under what is left of softmax(z / T) after its rejected elder siblings were removed; when no child is
// left the token is drawn from the residual by inverse CDF over increasing ids.  The uniforms are inputs:
// u[b][c] decides node c, u[b][N + cur] draws the final token at node cur.  One CTA per sequence; every reduction
// has a fixed order, so a step is reproducible on this kernel.
constexpr int ACC_THREADS = 1024;
constexpr int ACC_MAX_REJ = 64;

__device__ __forceinline__ float block_reduce_max(float v, float *sh) {
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = sh[0];
  for (int w = 1; w < ACC_THREADS / 32; w++) r = fmaxf(r, sh[w]);
  __syncthreads();
  return r;
}
__device__ __forceinline__ float block_reduce_sum(float v, float *sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = v;
  __syncthreads();
  float r = 0.0f;
  for (int w = 0; w < ACC_THREADS / 32; w++) r += sh[w];      // every thread adds the 32 warp sums in the same order
  __syncthreads();
  return r;
}

// exp on the special-function unit (ex2.approx): every term of a row goes through the same routine, so the
// probabilities stay consistent; its relative error (~1e-6 near the maximum) is far inside the parity slack
__device__ __forceinline__ float acc_exp(float x) { return __expf(x); }

__global__ void __launch_bounds__(ACC_THREADS) accept_sampled_kernel(SeqState st, TreeBufs tb, const float *__restrict__ logits,
                                                                     int V, const float *__restrict__ u, int rows_per_seq) {
  pdl_wait();
  pdl_trigger();
  __shared__ float red[ACC_THREADS / 32];
  __shared__ float part[ACC_THREADS / 32];
  extern __shared__ float seg[];                           // [ceil(V / 32)] residual terms of the range that holds the drawn token
  __shared__ int32_t rej[ACC_MAX_REJ];
  __shared__ int s_next, s_nrej, s_pick, s_owner;
  __shared__ float s_target;
  const int b = blockIdx.x, tid = threadIdx.x;
  const int Pmax = tb.Pmax, N = tb.N;
  const int nn = tb.nn[b];
  if (!st.active[b] || nn < 1) {
    if (tid == 0) tb.out_cnt[b] = 0;
    return;
  }
  // the tree and the uniforms go to shared memory once: the walk below is serial, and a global load per node would
  // put an L2 round trip into every iteration
  __shared__ int32_t tok[64], par[64];
  __shared__ float ub[128];
  if (tid < nn && tid < 64) { tok[tid] = tb.tok[(size_t)b * rows_per_seq + tid]; par[tid] = tb.parent[(size_t)b * rows_per_seq + tid]; }
  if (tid < 2 * N && tid < 128) ub[tid] = u[(size_t)b * 2 * N + tid];
  const float inv_T = u[(size_t)gridDim.x * 2 * N];          // 1 / temperature follows the uniforms
  __syncthreads();
  int cur = 0, a = 0;
  if (tid == 0) tb.path[b * Pmax] = 0;
  for (;;) {
    const float *z = logits + ((size_t)b * rows_per_seq + cur) * V;
    // one SM reads the row from L2: wide, unrolled loads keep enough requests in flight
    const bool vec = (V & 3) == 0;                       // rows are then 16-byte aligned
    const float4 *z4 = (const float4 *)z;
    float m = -INFINITY;
    if (vec) {
#pragma unroll 4
      for (int i = tid; i < V / 4; i += ACC_THREADS) {
        const float4 q = z4[i];
        m = fmaxf(m, fmaxf(fmaxf(q.x, q.y), fmaxf(q.z, q.w)));
      }
    } else {
#pragma unroll 8
      for (int v = tid; v < V; v += ACC_THREADS) m = fmaxf(m, z[v]);
    }
    const float zmax = block_reduce_max(m, red);
    float sum = 0.0f;
    if (vec) {
#pragma unroll 4
      for (int i = tid; i < V / 4; i += ACC_THREADS) {
        const float4 q = z4[i];
        sum += (acc_exp((q.x - zmax) * inv_T) + acc_exp((q.y - zmax) * inv_T)) + (acc_exp((q.z - zmax) * inv_T) + acc_exp((q.w - zmax) * inv_T));
      }
    } else {
#pragma unroll 8
      for (int v = tid; v < V; v += ACC_THREADS) sum += acc_exp((z[v] - zmax) * inv_T);
    }
    float mass = block_reduce_sum(sum, red);
    // ---- the children of cur in node order, tried by one thread
    if (tid == 0) {
      int nxt = -1, nrej = 0;
      if (a + 1 < Pmax) {
        for (int c = cur + 1; c < nn && nxt < 0; c++) {
          if (par[c] != cur) continue;
          const float e = acc_exp((z[tok[c]] - zmax) * inv_T);
          const float pc = mass > 0.0f ? e / mass : 0.0f;
          if (ub[c] < pc) nxt = c;
          else { mass -= e; if (nrej < ACC_MAX_REJ) rej[nrej++] = tok[c]; }
        }
      }
      s_next = nxt; s_nrej = nrej;
    }
    __syncthreads();
    const int nxt = s_next, nrej = s_nrej;
    if (nxt >= 0) {
      if (tid == 0) {
        tb.out_ids[b * Pmax + a] = tok[nxt];
        tb.pend_tok[b * Pmax + a] = tok[nxt];
        tb.path[b * Pmax + a + 1] = nxt;
      }
      cur = nxt;
      a++;
      __syncthreads();
      continue;
    }
    // ---- the final token: inverse CDF over the residual, in two levels.  Warp w owns the ids [w * CW, (w + 1) * CW):
    // its lanes read them coalesced and the warp sum goes to part[w]; one thread finds the warp whose range holds the
    // target; that warp then walks its range 32 ids at a time with a warp prefix sum.
    const int NWARP = ACC_THREADS / 32, wid = tid >> 5, ln = tid & 31;
    const int CW = (V + NWARP - 1) / NWARP;
    const int w0 = wid * CW, w1 = (w0 + CW < V) ? w0 + CW : V;
    float loc = 0.0f;
#pragma unroll 8
    for (int v = w0 + ln; v < w1; v += 32) loc += acc_exp((z[v] - zmax) * inv_T);
    for (int o = 16; o > 0; o >>= 1) loc += __shfl_xor_sync(0xffffffffu, loc, o);
    if (ln == 0) part[wid] = loc;
    __syncthreads();
    if (tid == 0) {
      for (int r = 0; r < nrej; r++) {                   // the rejected tokens leave the residual
        const float e = acc_exp((z[rej[r]] - zmax) * inv_T);
        const int w = rej[r] / CW;
        part[w] = fmaxf(part[w] - e, 0.0f);
      }
      float total = 0.0f;
      for (int w = 0; w < NWARP; w++) total += part[w];
      const float target = ub[N + cur] * total;
      float cum = 0.0f;
      int owner = -1;
      for (int w = 0; w < NWARP; w++) {
        if (part[w] > 0.0f && cum + part[w] > target) { owner = w; break; }
        cum += part[w];
      }
      if (owner < 0) {                                   // rounding at the upper end: the last warp with mass
        cum = total;
        for (int w = NWARP - 1; w >= 0; w--)
          if (part[w] > 0.0f) { owner = w; cum = total - part[w]; break; }
      }
      s_owner = owner; s_target = target - cum; s_pick = 0;
    }
    __syncthreads();
    // the owning warp's range goes to shared memory with every thread's help (one parallel, coalesced pass), so the
    // ordered walk below reads no global memory
    {
      const int o0 = s_owner * CW, o1 = (o0 + CW < V) ? o0 + CW : V;
      for (int v = o0 + tid; v < o1; v += ACC_THREADS) {
        float e = acc_exp((z[v] - zmax) * inv_T);
        for (int r = 0; r < nrej; r++) if (rej[r] == v) e = 0.0f;
        seg[v - o0] = e;
      }
    }
    __syncthreads();
    if (wid == s_owner) {
      const float target = s_target;
      float cum = 0.0f;
      int pick = -1, last = -1;
      for (int base = w0; base < w1 && pick < 0; base += 32) {
        const int v = base + ln;
        const float e = v < w1 ? seg[v - w0] : 0.0f;
        float inc = e;                                   // inclusive prefix sum over the 32 lanes
        for (int o = 1; o < 32; o <<= 1) {
          const float t = __shfl_up_sync(0xffffffffu, inc, o);
          if (ln >= o) inc += t;
        }
        const bool hit = e > 0.0f && cum + inc > target;
        const unsigned hits = __ballot_sync(0xffffffffu, hit), alive = __ballot_sync(0xffffffffu, e > 0.0f);
        if (alive) last = base + 31 - __clz(alive);
        if (hits) pick = base + __ffs(hits) - 1;
        cum += __shfl_sync(0xffffffffu, inc, 31);
      }
      if (ln == 0) s_pick = pick >= 0 ? pick : (last >= 0 ? last : w0);
    }
    __syncthreads();
    if (tid == 0) {
      const int bonus = s_pick;
      tb.out_ids[b * Pmax + a] = bonus;
      tb.pend_tok[b * Pmax + a] = bonus;
      for (int j = a + 1; j < Pmax; j++) tb.out_ids[b * Pmax + j] = -1;
      tb.out_cnt[b] = a + 1;
      const int n = st.n[b];
      st.n_prev[b] = n;
      st.n[b] = n + a + 1;
      st.P[b] = a + 1;
      st.root[b] = bonus;
    }
    break;
  }
}
void launch_accept_sampled(SeqState st, TreeBufs tb, const float *logits, int V, const float *u, int B, int rows_per_seq, cudaStream_t s) {
  const size_t smem = (size_t)((V + ACC_THREADS / 32 - 1) / (ACC_THREADS / 32)) * sizeof(float);
  static SmemLimit limit;
  if (smem > 40 * 1024) limit.ensure(accept_sampled_kernel, (int)smem);
  launch_k(accept_sampled_kernel, dim3(B), dim3(ACC_THREADS), smem, s, st, tb, logits, V, u, rows_per_seq);
}

// ---------------------------------------------------------------- commit: KV compaction + tap gather
// Accepted node path[j] (K/V at cache position n+path[j]) moves to position n+j in every layer; its
// taps become pending entry j.  path[j] >= j and is increasing, and a thread copies the same element
// offsets for every j, so the in-place move in increasing j never reads an overwritten slot.
template <typename T>
__global__ void __launch_bounds__(256) commit_kernel(SeqState st, TreeBufs tb, const KvPool *__restrict__ pools,
                                                     PageMap pm, const T *__restrict__ node_taps,
                                                     T *__restrict__ pend_taps, int L, int G, int hd, int k,
                                                     int rows_per_seq) {
  pdl_wait();
  pdl_trigger();
  int b = blockIdx.x, l = blockIdx.y;
  int cnt = tb.out_cnt[b];
  if (cnt <= 0) return;
  int n0 = st.n_prev[b], Pmax = tb.Pmax;
  constexpr int VEC = 16 / (int)sizeof(T);           // elements per 16-byte vector (head_dim is a multiple of 16)
  constexpr int JB = 8;                              // accepted nodes moved per batch
  __shared__ int32_t path_s[64];
  for (int j = threadIdx.x; j < cnt && j < 64; j += blockDim.x) path_s[j] = tb.path[b * Pmax + j];
  __syncthreads();
  if (l < L) {
    // A thread owns the same 16-byte vectors of every position.  Per batch of JB accepted nodes it issues all its loads
    // before its first store: a destination slot j can only be the source of an earlier node (path[j'] >= j'), never
    // of a later batch, and within a batch every load has been issued before any store.
    T *Kp = (T *)pools[l].k, *Vp = (T *)pools[l].v;
    const int nvec = G * hd / VEC;
    for (int t = threadIdx.x; t < nvec; t += blockDim.x) {
      const int g = (t * VEC) / hd, i = (t * VEC) % hd;
      for (int j0 = 0; j0 < cnt; j0 += JB) {
        uint4 kv[JB], vv[JB];
        size_t dof[JB];
        bool mv[JB];
#pragma unroll
        for (int jj = 0; jj < JB; jj++) {
          const int j = j0 + jj;
          mv[jj] = false;
          if (j < cnt) {
            const int src = n0 + path_s[j], dst = n0 + j;
            mv[jj] = src != dst;
            if (mv[jj]) {
              const size_t so = kv_offset(pm, b, src, g, G, hd) + i;
              dof[jj] = kv_offset(pm, b, dst, g, G, hd) + i;
              kv[jj] = *(const uint4 *)(Kp + so);
              vv[jj] = *(const uint4 *)(Vp + so);
            }
          }
        }
#pragma unroll
        for (int jj = 0; jj < JB; jj++)
          if (mv[jj]) { *(uint4 *)(Kp + dof[jj]) = kv[jj]; *(uint4 *)(Vp + dof[jj]) = vv[jj]; }
      }
    }
  } else {
    // taps of the accepted nodes -> pending entries (different buffers: no ordering needed)
    const int nvec = 3 * k / VEC;
    for (int j = 0; j < cnt; j++) {
      const uint4 *src = (const uint4 *)(node_taps + ((size_t)b * rows_per_seq + path_s[j]) * 3 * k);
      uint4 *dst = (uint4 *)(pend_taps + ((size_t)b * Pmax + j) * 3 * k);
      for (int e = threadIdx.x; e < nvec; e += blockDim.x) dst[e] = src[e];
    }
  }
}
template <typename T>
void launch_commit(SeqState st, TreeBufs tb, const KvPool *pools, PageMap pm, const T *node_taps, T *pend_taps, int B,
                   int L, int G, int hd, int k, int rows_per_seq, cudaStream_t s) {
  launch_k(commit_kernel<T>, dim3(B, L + 1), dim3(256), 0, s, st, tb, pools, pm, node_taps, pend_taps, L, G, hd, k, rows_per_seq);
}
template void launch_commit<float>(SeqState, TreeBufs, const KvPool *, PageMap, const float *, float *, int, int, int,
                                   int, int, int, cudaStream_t);
template void launch_commit<bf16>(SeqState, TreeBufs, const KvPool *, PageMap, const bf16 *, bf16 *, int, int, int, int,
                                  int, int, cudaStream_t);

}  // namespace spec
