// Weight-streaming bf16 GEMM with fused epilogues (tcgen05.mma, TMEM accumulators, TMA-staged
// operands, split-K reduced across a thread-block cluster through distributed shared memory):
// host-side interface.
#pragma once
#include "tma_maps.cuh"

namespace spec {

enum FusedEpi {
  EPI_F32 = 0,      // out_f32[r][o] = scale[r] * acc
  EPI_RESID = 1,    // x[r][o] (+)= acc; hb = bf16(x * gain[o]); per-tile sum of squares; optional taps
  EPI_QKV = 2,      // scale, rotate q and k by the row's position, store q, write K/V into the paged cache
  EPI_SWIGLU = 3,   // two weights (gate, up): act = bf16(silu(scale*g) * scale*u)
  EPI_ARGMAX = 4,   // per (feature tile, row) best (value, index); optional fp32 logits
  EPI_TOPK = 5      // per (feature tile, wanted row): tile maximum, sum of exp relative to it, the tile's K best (value,
                    // index) best first: what a log-softmax + top-K over all features needs; optional fp32 logits
};

struct FusedGemmArgs {
  // ---- operands: out[r][o] = sum_i x[r][i] * w[o][i]
  const bf16 *x = nullptr;      // [rows][I]
  int rows = 0, I = 0;
  const bf16 *w[3] = {nullptr, nullptr, nullptr};   // [O[j]][I]; several weights share one launch (q,k,v / gate,up)
  int O[3] = {0, 0, 0};
  int nw = 1;
  // ---- per-row scale of the input (RMSNorm statistic of the tensor x was derived from):
  // scale[r] = rsqrt(sum_t ssq_in[t * ssq_ld + r] / k_in + eps); nullptr: scale 1
  const float *ssq_in = nullptr;
  int ssq_in_tiles = 0, ssq_ld = 0, k_in = 1;
  float eps = 0.0f;
  // ---- EPI_F32 (and the optional logits of EPI_ARGMAX)
  float *out_f32 = nullptr;
  int ldo = 0;
  // ---- EPI_RESID (O[0] = width of the residual stream)
  float *xres = nullptr;        // [rows][O]
  const bf16 *gain = nullptr;   // [O] gain of the norm that consumes the new residual
  bf16 *hb = nullptr;           // [rows][O] = bf16(x * gain)
  float *ssq_out = nullptr;     // [ceil(O/128)][ssq_ld]
  bf16 *taps = nullptr;         // [rows][3*O], slot s written when bit s of tap_mask is set
  int tap_mask = 0;
  int resid_add = 1;            // 1: x += acc, 0: x = acc
  // ---- EPI_QKV (w = {wq, wk, wv})
  const float2 *cs = nullptr;   // [rows][hd/2] (cos, sin)
  RowMeta m = {};
  bf16 *q = nullptr;            // [rows][H][hd]
  KvPool pool = {nullptr, nullptr};
  PageMap pm = {nullptr, 0, 0, 0};
  int H = 0, G = 0, hd = 0;
  // ---- EPI_SWIGLU (w = {gate, up})
  bf16 *act = nullptr;          // [rows][O[0]]
  // ---- EPI_ARGMAX
  float *best_val = nullptr;    // [tiles][best_ld]
  int32_t *best_idx = nullptr;
  int best_ld = 0;
  // ---- EPI_TOPK: candidates [rows][cand_ld][topk], tile statistics [rows][cand_ld]; cand_ld >= tiles (a multiple of 4
  // keeps every row 16-byte aligned for the merge)
  int topk = 0;                 // K (1..16)
  float *cand_val = nullptr, *cand_max = nullptr, *cand_sum = nullptr;
  int32_t *cand_idx = nullptr;  // -1: the tile has fewer than K features
  int cand_ld = 0;
  const int32_t *want_rows = nullptr;   // device list of the rows that need candidates (entries < 0 ignored); nullptr: all rows
  int n_want = 0;
  // ---- launch
  int32_t *status = nullptr;    // device status words
  int split = 0, stages = 0;    // 0 = chosen by the library
  bool pdl = false;             // programmatic dependent launch (weights are prefetched before the wait)
  // ---- test hook for the bounded waits: polls before a wait gives up (0 = the library's limit), and, when `withhold`
  // is set, CTA 0 leaves out the activation load of its first k-block, so that its first wait runs out: the CTA records
  // ST_TIMEOUT in the status words, skips its arithmetic, keeps its cluster barriers, waits for its loads in flight,
  // frees its tensor memory and exits
  unsigned spin_limit = 0;
  bool withhold = false;
  // ---- profiling aid: stamp[0] = earliest time (globaltimer ns) a CTA saw its inputs ready, stamp[1] = complement of the latest CTA exit (both start from all ones)
  unsigned long long *stamp = nullptr;
};

// true when the shapes fit the fused kernels (rows <= 256, I % 8 == 0, 16-byte aligned pointers, and for
// EPI_QKV a power-of-two head_dim <= 128)
bool fused_gemm_supported(FusedEpi epi, const FusedGemmArgs &a);
// number of 128-feature tiles of the launch (EPI_ARGMAX: rows of best_val / best_idx needed)
int fused_gemm_tiles(FusedEpi epi, const FusedGemmArgs &a);
// CTAs a launch aims at (K slices are chosen to come close to it); process-wide.
void fused_gemm_set_target_ctas(int n);
void fused_gemm_set_pairs(int on);   // 256-row tiles as CTA pairs (cta_group::2); process-wide
// Returns 0 or a negative code.
int fused_gemm_launch(TmaMaps *g, FusedEpi epi, const FusedGemmArgs &a, cudaStream_t s);

}  // namespace spec
