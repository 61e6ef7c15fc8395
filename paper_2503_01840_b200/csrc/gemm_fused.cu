// Weight-streaming bf16 GEMM with fused epilogues for sm_100a.
//
//   out[r][o] = sum_i x[r][i] * w[o][i],  rows <= 256 token rows, weights far larger than the L2.
//
// The contraction is HBM-bound (every weight byte is read once per launch), so the kernel is built
// around keeping many weight bytes in flight per SM and wasting no extra pass over the result:
//
//  * swap-AB mapping: the weight tile (128 output features x 64 k, K-major, 128-byte swizzle) is the
//    UMMA M side, the token rows the N side (NT = 16/64/128/256), the fp32 accumulator sits in TMEM;
//  * warp 0 streams tiles with TMA through a ring of shared-memory stages, warp 1 issues tcgen05.mma; both walk their
//    loops as converged warps and one lane chosen by elect.sync issues (the issuing warp, not shared memory or HBM,
//    is what limits a single CTA: see ubench/issue_loop.cu);
//  * split-K: the S slices of one feature tile form a thread-block cluster.  Each CTA parks its
//    accumulator in its own shared memory and every CTA reduces a share of the rows by reading its
//    peers' copies through distributed shared memory, in slice order (deterministic, no atomics, no
//    round trip of partial sums through global memory);
//  * the epilogue that follows the reduction is the consumer's work: residual add + bf16 copy scaled
//    by the next norm's gain + RMSNorm statistics (+ feature taps); RoPE + q store + paged K/V write;
//    SiLU(gate)*up (the gate and up tiles of a feature range are two members of the same cluster);
//    per-tile argmax.  RMSNorm of the input is applied as a per-row scale in the
//    epilogue (the normalisation factor is a row constant, so it commutes with the contraction);
//  * programmatic dependent launch: the producer prefetches the first weight tiles (which never depend
//    on the previous kernel) before griddepcontrol.wait, so the pipeline is full when the activations
//    become valid.
//
// Every mbarrier wait is bounded; on timeout the CTA records it, skips its arithmetic, still takes part
// in the cluster barriers (so its peers are not left waiting), frees its TMEM and exits.
#include <cuda.h>
#include <stdio.h>

#include <algorithm>

#include "gemm_fused.cuh"
#include "tcgen05_ptx.cuh"

namespace spec {

namespace {

using namespace tc;

constexpr int MAX_STAGES = 16;
constexpr int CHUNK = 64;                       // rows reduced per epilogue round (tiles of up to 64 rows)
constexpr int MAX_CHUNK = 256;                  // wider tiles take as many rows per round as the free ring holds
constexpr int A_BYTES = TILE_M * TILE_K * 2;    // one weight tile of a stage

struct alignas(64) FusedParams {
  CUtensorMap map_w[3];
  CUtensorMap map_x;
  int tiles0, tiles1;          // tile index ranges of the weights: [0,tiles0) w0, [tiles0,tiles1) w1, rest w2
  int O[3];
  int rows, KB, S, Sk, stages, ctrl_off;   // S = cluster size, Sk = K slices (S = 2 Sk for EPI_SWIGLU)
  int chunk;                               // rows per epilogue round
  const float *ssq_in; int ssq_in_tiles, ssq_ld; float inv_k_in, eps;
  float *out_f32; int ldo;
  float *xres; const bf16 *gain; bf16 *hb; float *ssq_out; bf16 *taps; int tap_mask, resid_add;
  const float2 *cs; RowMeta m; bf16 *q; KvPool pool; PageMap pm; int H, G, hd;
  bf16 *act;
  float *best_val; int32_t *best_idx; int best_ld;
  int topk; float *cand_val, *cand_max, *cand_sum; int32_t *cand_idx; int cand_ld; const int32_t *want_rows; int n_want;
  int32_t *status;
  unsigned long long *stamp;
  unsigned spin;               // polls before a wait gives up
  int withhold;                // test hook: CTA 0 leaves out the activation load of its first k-block
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_peer(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

__device__ __forceinline__ uint32_t ld_peer_u32(uint32_t local_addr, uint32_t rank) {
  uint32_t ra, v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(v) : "r"(ra) : "memory");
  return v;
}

// 16-byte load from the same shared-memory offset in cluster member `rank`.  Deliberately without a
// "memory" clobber: consecutive loads stay in program order (volatile) but do not wait for one another,
// so a thread keeps several remote requests in flight.
__device__ __forceinline__ float4 ld_peer4(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  float4 v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(ra));
  return v;
}
// sum over cluster members [s0, s0+n) (n <= 16) of the float4 at local_addr, added in member order
__device__ __forceinline__ float4 sum_peers4(uint32_t local_addr, int s0, int n, int stride = 1) {
  float4 acc = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
#pragma unroll
  for (int b = 0; b < 16; b += 8) {
    if (b >= n) break;
    float4 v[8];
#pragma unroll
    for (int s = 0; s < 8; s++)
      if (b + s < n) v[s] = ld_peer4(local_addr, (uint32_t)(s0 + (b + s) * stride));
#pragma unroll
    for (int s = 0; s < 8; s++)
      if (b + s < n) { acc.x += v[s].x; acc.y += v[s].y; acc.z += v[s].z; acc.w += v[s].w; }
  }
  return acc;
}

// PAIR (EPI_SWIGLU only): the CTA streams the gate tile AND the up tile of its 128 features for its K slice, both
// MMAs of a k-block share one activation tile (half the activation fill traffic of the form in which gate and up are
// separate cluster members), the two accumulators sit side by side in tensor memory, and the cluster holds only the
// Sk K slices.
//
// DUO (256-row tiles; EPI_F32 / EPI_RESID / EPI_QKV): two neighbouring feature tiles run as a CTA pair (cta_group::2).
// Each CTA streams its own weight tile but only HALF of the activation k-block (128 of the 256 rows); the even CTA issues
// one M = 256 MMA per k-step that reads both CTAs' shared memory, and each CTA's tensor memory receives the accumulator
// of its own tile.  At 256 rows the activation k-block (32 KB) is twice a weight tile, so the shared-memory fill traffic
// per weight byte drops from 3 x to 2 x, which is what bounds the loop at this width.  The cluster is (2, S): x = the
// pair, y = the K slices; the reduction runs over the members with the same x.
// Threads per CTA: 128 (thread = output feature in the epilogue); the 256-row tiles with a row-wise epilogue run 256, so
// that two threads share a feature and split the tile's columns / rows between them (the epilogue of a 256-row tile is
// as long as its main loop).
constexpr int fused_threads(int nt, int epi) { return (nt == 256 && (epi == EPI_F32 || epi == EPI_RESID || epi == EPI_QKV)) ? 256 : 128; }

template <int NT, int EPI, bool PAIR = false, bool DUO = false>
__global__ void __launch_bounds__(fused_threads(NT, EPI)) gemm_fused_kernel(const __grid_constant__ FusedParams p) {
  constexpr int THREADS = fused_threads(NT, EPI), NH = THREADS / 128;
  static_assert(!PAIR || EPI == EPI_SWIGLU, "two weight tiles per CTA exist for the gate/up epilogue only");
  static_assert(!DUO || (NT == 256 && !PAIR && (EPI == EPI_F32 || EPI == EPI_RESID || EPI == EPI_QKV)), "CTA pairs serve the 256-row tiles");
  constexpr int A_TILES = PAIR ? 2 : 1;
  constexpr int B_BYTES = (DUO ? NT / 2 : NT) * TILE_K * 2;
  constexpr int STAGE = A_TILES * A_BYTES + B_BYTES;
  constexpr int TMEM_COLS = (A_TILES * NT < 32) ? 32 : A_TILES * NT;
  static_assert(TMEM_COLS <= 512, "accumulators must fit the tensor memory");

  extern __shared__ unsigned char smem_raw[];
  unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char *ctrl = tiles + p.ctrl_off;
  uint64_t *full = (uint64_t *)ctrl;
  uint64_t *empty = full + MAX_STAGES;
  uint64_t *acc_bar = empty + MAX_STAGES;
  uint32_t *tmem_slot = (uint32_t *)(acc_bar + 1);
  volatile uint32_t *abort_flag = tmem_slot + 1;
  volatile int *n_issued = (volatile int *)(tmem_slot + 2), *n_consumed = (volatile int *)(tmem_slot + 3);   // stage loads issued / seen complete
  float *inv_s = (float *)(ctrl + 512);          // [256] per-row input scale
  float *wpart = inv_s + 256;                    // [4][MAX_CHUNK] per-warp partial sums / argmax exchange

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stages = p.stages, S = p.S, Sk = p.Sk;
  const uint32_t crank = (S > 1 || DUO) ? cluster_rank() : 0u;
  const int xr = DUO ? (int)(crank & 1u) : 0;                 // DUO: position in the CTA pair (0 issues the MMAs)
  const int slice = DUO ? (int)(crank >> 1) : (int)crank;     // K slice = rank among the CTAs that share this feature tile
  const int ksl = (EPI == EPI_SWIGLU && !PAIR) ? slice % Sk : slice;   // K slice
  const int kb0 = (int)(((long long)ksl * p.KB) / Sk), kb1 = (int)(((long long)(ksl + 1) * p.KB) / Sk);
  const int nkb = kb1 - kb0;
  int mi = 0, tm = blockIdx.x;                   // weight index and tile within that weight
  if (EPI == EPI_SWIGLU) {
    mi = PAIR ? 0 : slice / Sk;                  // ranks [0,Sk) stream the gate tile, [Sk,2Sk) the up tile
  } else {
    if (tm >= p.tiles1) { mi = 2; tm -= p.tiles1; }
    else if (tm >= p.tiles0) { mi = 1; tm -= p.tiles0; }
  }

  if (threadIdx.x == 0) {
    for (int i = 0; i < stages; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_bar, 1);
    *abort_flag = 0;
    *n_issued = 0; *n_consumed = 0;
    // pairs rely on cluster ranks running x first (rank = x + 2 y): checked, never assumed
    if (DUO && ((crank & 1u) != (blockIdx.x & 1u) || (int)(crank >> 1) != (int)(blockIdx.y % (unsigned)S))) {
      *abort_flag = 1;
      set_status(p.status, ST_TIMEOUT, 234, blockIdx.x, (int)crank);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation is a whole-warp operation (pairs: the same warp of both CTAs, same slot offset)
    if (DUO) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (DUO) cluster_sync_all(); else __syncthreads();   // pairs: the partner's barriers must exist before anything signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();

  if (DUO && *abort_flag) {
    pdl_wait();            // wrong cluster layout: nothing is loaded or issued; the epilogue below writes nothing
  } else if (DUO && warp == 0) {
    // ---- producer of a CTA pair: own weight tile + own half of the activation rows; every byte of both CTAs is counted
    // on the even CTA's full barrier (it alone announces the byte count: one arrival per phase).
    const CUtensorMap *mw0 = &p.map_w[mi];
    const uint64_t pol = l2_policy_evict_first();
    const uint32_t lead = crank & ~1u;
    const int npre = nkb < stages ? nkb : stages;
    if (elect_one())
      for (int i = 0; i < npre; i++) {
        if (xr == 0) mbar_expect_tx(&full[i], 2 * STAGE);
        tma_load_2d_pair_hint(tiles + i * STAGE, mw0, (kb0 + i) * TILE_K, tm * TILE_M, mapa_u32(smem_u32(&full[i]), lead), pol);
      }
    __syncwarp();
    pdl_wait();
    if (elect_one()) {
      if (p.stamp) atomicMin(p.stamp, global_ns());
      for (int i = 0; i < npre; i++)
        tma_load_2d_pair(tiles + i * STAGE + A_BYTES, &p.map_x, (kb0 + i) * TILE_K, xr * (NT / 2), mapa_u32(smem_u32(&full[i]), lead));
    }
    __syncwarp();
    // steady state: stage and phase advance by increments (no divisions), nothing but the wait and the copies per k-block
    int i = npre, st = 0;
    uint32_t ph = 0;
    for (; i < nkb; i++) {
      if (!mbar_wait_warp(&empty[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 230, blockIdx.x, i); break; }
      if (elect_one()) {
        unsigned char *a = tiles + st * STAGE;
        const uint32_t fb = mapa_u32(smem_u32(&full[st]), lead);
        if (xr == 0) mbar_expect_tx(&full[st], 2 * STAGE);
        tma_load_2d_pair_hint(a, mw0, (kb0 + i) * TILE_K, tm * TILE_M, fb, pol);
        tma_load_2d_pair(a + A_BYTES, &p.map_x, (kb0 + i) * TILE_K, xr * (NT / 2), fb);
      }
      __syncwarp();
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
    if (lane == 0) *n_issued = i;
  } else if (!DUO && warp == 0) {
    // ---- producer warp (all lanes walk the loop, the elected lane issues).  Weight tiles do not depend on the previous
    // kernel: fill the ring with them first.
    const CUtensorMap *mw0 = &p.map_w[mi];
    const uint64_t pol = l2_policy_evict_first();
    const int npre = nkb < stages ? nkb : stages;
    if (elect_one())
      for (int i = 0; i < npre; i++) {
        unsigned char *a = tiles + i * STAGE;
        mbar_expect_tx(&full[i], STAGE);
        tma_load_2d_hint(a, mw0, (kb0 + i) * TILE_K, tm * TILE_M, &full[i], pol);
        if (PAIR) tma_load_2d_hint(a + A_BYTES, &p.map_w[1], (kb0 + i) * TILE_K, tm * TILE_M, &full[i], pol);
      }
    __syncwarp();
    pdl_wait();
    if (elect_one()) {
      if (p.stamp) atomicMin(p.stamp, global_ns());
      const bool hold = p.withhold && blockIdx.x == 0 && blockIdx.y == 0;     // test hook: the first stage never completes
      for (int i = hold ? 1 : 0; i < npre; i++) tma_load_2d(tiles + i * STAGE + A_TILES * A_BYTES, &p.map_x, (kb0 + i) * TILE_K, 0, &full[i]);
    }
    __syncwarp();
    int i = npre, st = 0;             // the loop runs only when the prefill used every stage: it restarts at stage 0
    uint32_t ph = 0;
    for (; i < nkb; i++) {
      if (!mbar_wait_warp(&empty[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 200, blockIdx.x, i); break; }
      if (elect_one()) {
        unsigned char *a = tiles + st * STAGE;
        mbar_expect_tx(&full[st], STAGE);
        tma_load_2d_hint(a, mw0, (kb0 + i) * TILE_K, tm * TILE_M, &full[st], pol);
        if (PAIR) tma_load_2d_hint(a + A_BYTES, &p.map_w[1], (kb0 + i) * TILE_K, tm * TILE_M, &full[st], pol);
        tma_load_2d(a + A_TILES * A_BYTES, &p.map_x, (kb0 + i) * TILE_K, 0, &full[st]);
      }
      __syncwarp();
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
    if (lane == 0) *n_issued = i;
  } else {
    pdl_wait();
    if (DUO && warp == 1) {
      // ---- MMA issuer of a CTA pair (even CTA only): M = 256 over both CTAs' weight tiles, N = both activation halves
      if (xr == 0) {
        constexpr uint32_t idesc = umma_idesc_m(NT, 2 * TILE_M);
        const uint32_t pair_lead = crank;                        // this (even) CTA and its partner crank + 1
        const uint32_t partner_base = ld_peer_u32(smem_u32(tmem_slot), crank | 1u);
        if (partner_base != tmem_base) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 233, blockIdx.x, (int)partner_base); }
        const uint64_t desc0 = umma_desc_sw128(smem_u32(tiles));
        int i = 0, st = 0;
        uint32_t ph = 0, ready = 0;
        if (!*abort_flag)
          for (; i < nkb; i++) {
            if (!ready && !mbar_wait_warp(&full[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 231, blockIdx.x, i); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t da = desc0 + (uint64_t)((st * STAGE) >> 4);
            int nst = st + 1;
            uint32_t nph = ph;
            if (nst == stages) { nst = 0; nph ^= 1u; }
            if (elect_one()) {
#pragma unroll
              for (int j = 0; j < TILE_K / UMMA_K; j++) umma_bf16_pair(tmem_base, da + 2 * j, da + (A_BYTES >> 4) + 2 * j, idesc, (i | j) ? 1u : 0u);
              umma_commit_pair(&empty[st], pair_lead);      // frees the stage in both CTAs
            }
            __syncwarp();
            ready = mbar_test_warp(&full[nst], nph) ? 1u : 0u;
            st = nst; ph = nph;
          }
        if (lane == 0) *n_consumed = i;
        __syncwarp();
        if (!*abort_flag && elect_one()) umma_commit_pair(acc_bar, pair_lead);   // both accumulators complete
      }
    } else if (!DUO && warp == 1) {
      // ---- MMA issuer warp (all lanes walk the loop, the elected lane issues)
      // The issuing warp is what limits a CTA's streaming rate, so the loop is kept to a non-blocking look at the
      // barrier (the blocking wait only when the stage is not full yet), one fence, four MMAs and the commit.
      constexpr uint32_t idesc = umma_idesc(NT);
      const uint64_t desc0 = umma_desc_sw128(smem_u32(tiles));
      int i = 0, st = 0;
      uint32_t ph = 0, ready = 0;
      for (; i < nkb; i++) {
        if (!ready && !mbar_wait_warp(&full[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 201, blockIdx.x, i); break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t da = desc0 + (uint64_t)((st * STAGE) >> 4), db = da + (uint64_t)((A_TILES * A_BYTES) >> 4);
        int nst = st + 1;
        uint32_t nph = ph;
        if (nst == stages) { nst = 0; nph ^= 1u; }
        if (elect_one()) {
#pragma unroll
          for (int j = 0; j < TILE_K / UMMA_K; j++) {      // a K = 16 step advances the descriptors by 32 bytes = 2 units
            umma_bf16(tmem_base, da + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);
            if (PAIR) umma_bf16(tmem_base + NT, da + (A_BYTES >> 4) + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);   // the up accumulator
          }
          umma_commit(&empty[st]);      // frees the stage once these MMAs have read it
        }
        __syncwarp();
        ready = mbar_test_warp(&full[nst], nph) ? 1u : 0u;      // a cheap look at the next stage: mostly spares the wait
        st = nst; ph = nph;
      }
      if (lane == 0) *n_consumed = i;
      if (elect_one()) umma_commit(acc_bar);           // accumulator complete
    } else if (warp >= 2) {
      // ---- per-row scale of the input: rsqrt(mean square + eps) from the producer kernel's per-tile sums
      for (int r = threadIdx.x - 64; r < p.rows; r += THREADS - 64) {
        float sc = 1.0f;
        if (p.ssq_in) {
          float ss = 0.0f;
          for (int t = 0; t < p.ssq_in_tiles; t++) ss += p.ssq_in[(size_t)t * p.ssq_ld + r];
          sc = 1.0f / sqrtf(ss * p.inv_k_in + p.eps);
        }
        inv_s[r] = sc;
      }
    }
  }
  __syncthreads();

  // ---- wait for the accumulator (one bounded wait per warp)
  int good = 0;
  if (lane == 0) {
    bool ok = *abort_flag ? false : mbar_wait(acc_bar, 0, p.spin);    // after an abort the accumulator never completes
    if (!ok && !*abort_flag) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 202, blockIdx.x, slice); }
    good = (ok && !*abort_flag) ? 1 : 0;
  }
  good = __shfl_sync(0xffffffffu, good, 0);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // ---- epilogue, CH rows at a time.  The stage ring is free now (every load landed, every MMA that
  // read it completed) and is reused: red = this CTA's accumulator, sumb = this CTA's rows after the cluster sum.
  const int CH = (NT <= CHUNK || EPI == EPI_ARGMAX) ? CHUNK : p.chunk;   // a constant for the narrow tiles
  float *red = (float *)tiles;                       // [CH][128]
  float *red_u = red + CH * TILE_M;                  // PAIR: the up accumulator, [CH][128]
  float *sumb = red + A_TILES * CH * TILE_M;         // [rows of this CTA][128] (EPI_SWIGLU: gate rows, then up rows at CH/2)
  const int f = threadIdx.x & (TILE_M - 1);          // feature of the tile = tensor-memory lane (a warp reads lanes 32 (warp % 4) ..)
  const int hw = threadIdx.x >> 7;                   // 0, or with 256 threads which half of the columns / rows
  const int o = tm * TILE_M + f;                     // output feature within weight mi
  for (int c0 = 0; c0 < p.rows; c0 += CH) {
    const int nrow = (p.rows - c0 < CH) ? p.rows - c0 : CH;
    if (good) {
#pragma unroll 1
      for (int cc = hw * (CH / NH); cc < (hw + 1) * (CH / NH) && c0 + cc < NT; cc += 16) {
        if (cc >= nrow) break;
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(c0 + cc), v);
#pragma unroll
        for (int j = 0; j < 16; j++) red[(cc + j) * TILE_M + f] = __uint_as_float(v[j]);
        if (PAIR) {
          tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(NT + c0 + cc), v);
#pragma unroll
          for (int j = 0; j < 16; j++) red_u[(cc + j) * TILE_M + f] = __uint_as_float(v[j]);
        }
      }
    }
    if (S > 1) cluster_sync_all(); else __syncthreads();
    const int per = (nrow + S - 1) / S;
    const int r0 = (slice * per < nrow) ? slice * per : nrow, r1 = (r0 + per < nrow) ? r0 + per : nrow;   // r0 <= r1

    // ---- phase A (clusters): this CTA's rows, summed over the K slices, land in its own sumb.  Each thread
    // takes (row, 4 features) items and keeps all its remote loads in flight before adding them up.
    const float *src = red + r0 * TILE_M;              // S == 1: the accumulator dump is the sum
    const float *src_u = red_u + r0 * TILE_M;          // EPI_SWIGLU: the up values of the same rows
    if (S > 1) {
      const int nitems = (r1 - r0) * 32;
      for (int item = threadIdx.x; item < nitems; item += THREADS) {
        const int i = item >> 5, qd = item & 31;
        const uint32_t la = smem_u32(&red[(r0 + i) * TILE_M + qd * 4]);
        *(float4 *)&sumb[i * TILE_M + qd * 4] = DUO ? sum_peers4(la, xr, Sk, 2) : sum_peers4(la, 0, Sk);
        if (EPI == EPI_SWIGLU) {
          if (PAIR) *(float4 *)&sumb[(CH / 2 + i) * TILE_M + qd * 4] = sum_peers4(smem_u32(&red_u[(r0 + i) * TILE_M + qd * 4]), 0, Sk);
          else *(float4 *)&sumb[(CH / 2 + i) * TILE_M + qd * 4] = sum_peers4(la, Sk, Sk);
        }
      }
      __syncthreads();
      src = sumb;
      src_u = sumb + (CH / 2) * TILE_M;
      // this CTA has everything it needs from its peers: announce it now and wait only at the end of the round, so
      // that the per-feature epilogue below runs while the slower members are still summing
      asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    // ---- phase B: per-feature epilogue from local shared memory (thread = feature f of the tile).  Rows go
    // in batches of RB: all global loads of a batch are issued before its first store, so the loop is not
    // a chain of dependent L2 round trips.
    constexpr int RB = 8;
    if (EPI == EPI_F32) {
      for (int r = r0 + hw; r < r1; r += NH)
        if (good && o < p.O[0]) p.out_f32[(size_t)(c0 + r) * p.ldo + o] = src[(r - r0) * TILE_M + f] * inv_s[c0 + r];
    } else if (EPI == EPI_RESID) {
      const bool act_o = good && o < p.O[0];
      const float gn = act_o ? __bfloat162float(p.gain[o]) : 0.0f;
      for (int rb = r0 + hw * RB; rb < r1; rb += NH * RB) {
        float xin[RB];
#pragma unroll
        for (int j = 0; j < RB; j++)
          xin[j] = (act_o && p.resid_add && rb + j < r1) ? p.xres[(size_t)(c0 + rb + j) * p.O[0] + o] : 0.0f;
#pragma unroll
        for (int j = 0; j < RB; j++) {
          const int r = rb + j;
          if (r < r1) {              // uniform over the CTA
            const int row = c0 + r;
            float xo = 0.0f;
            if (act_o) {
              size_t xi = (size_t)row * p.O[0] + o;
              xo = xin[j] + src[(r - r0) * TILE_M + f];
              p.xres[xi] = xo;
              p.hb[xi] = __float2bfloat16_rn(xo * gn);
              if (p.tap_mask) {
#pragma unroll
                for (int s = 0; s < 3; s++)
                  if ((p.tap_mask >> s) & 1) p.taps[(size_t)row * 3 * p.O[0] + (size_t)s * p.O[0] + o] = __float2bfloat16_rn(xo);
              }
            }
            float sq = xo * xo;
            for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
            if (lane == 0) wpart[(warp & 3) * CH + (r - r0)] = sq;
          }
        }
      }
      __syncthreads();
      if (good)
        for (int t = threadIdx.x; t < r1 - r0; t += THREADS)
          p.ssq_out[(size_t)tm * p.ssq_ld + c0 + r0 + t] = ((wpart[t] + wpart[CH + t]) + wpart[2 * CH + t]) + wpart[3 * CH + t];
    } else if (EPI == EPI_QKV) {
      const int hd = p.hd, half = hd >> 1;
      const int head = o / hd, i = o % hd;
      const bool valid_o = (o < p.O[mi]) && good;
      bf16 *Kp = (bf16 *)p.pool.k, *Vp = (bf16 *)p.pool.v;
      // per-row cache slot of this CTA's rows: one thread per row resolves sequence -> position -> page
      int32_t *slot_s = (int32_t *)wpart;              // [CH] element offset / hd of the row's K/V slot, -1: none
      int32_t *seq_s = slot_s + CH;                    // [CH]
      for (int t = threadIdx.x; t < r1 - r0; t += THREADS) {
        const int row = c0 + r0 + t;
        const int seq = p.m.seq[row];
        int slot = -1;
        if (seq >= 0 && mi > 0) {
          const int kvpos = p.m.kvpos[row];
          if (kvpos < 0 || kvpos / p.pm.page_size >= p.pm.pages_per_seq) {
            set_status(p.status, ST_BOUNDS, 1, row, kvpos);
          } else {
            const int page = p.pm.table[(size_t)seq * p.pm.pages_per_seq + kvpos / p.pm.page_size];
            if (page < 0 || page >= p.pm.num_pages) set_status(p.status, ST_BOUNDS, 2, row, page);
            else slot = (page * p.G) * p.pm.page_size + (kvpos % p.pm.page_size);   // + head * page_size below
          }
        }
        slot_s[t] = slot;
        seq_s[t] = seq;
      }
      __syncthreads();
      for (int rb = r0 + hw * RB; rb < r1; rb += NH * RB) {
        float2 cs[RB];
#pragma unroll
        for (int j = 0; j < RB; j++)
          cs[j] = (valid_o && mi < 2 && rb + j < r1) ? p.cs[(size_t)(c0 + rb + j) * half + (i & (half - 1))] : make_float2(1.0f, 0.0f);
#pragma unroll
        for (int j = 0; j < RB; j++) {
          const int r = rb + j;
          if (r >= r1 || !valid_o) continue;
          const int row = c0 + r;
          const float sc = inv_s[row];
          float v = src[(r - r0) * TILE_M + f] * sc;
          if (mi < 2) {                             // rotate-half RoPE: partner feature is f ^ half
            float w = src[(r - r0) * TILE_M + (f ^ half)] * sc;
            v = (i < half) ? v * cs[j].x - w * cs[j].y : v * cs[j].x + w * cs[j].y;
          }
          if (mi == 0) {
            p.q[((size_t)row * p.H + head) * hd + i] = __float2bfloat16_rn(seq_s[r - r0] < 0 ? 0.0f : v);
          } else if (slot_s[r - r0] >= 0) {
            size_t off = ((size_t)slot_s[r - r0] + (size_t)head * p.pm.page_size) * hd + i;
            (mi == 1 ? Kp : Vp)[off] = __float2bfloat16_rn(v);
          }
        }
      }
    } else if (EPI == EPI_SWIGLU) {
      for (int r = r0; r < r1; r++) {
        const int row = c0 + r;
        const float sc = inv_s[row];
        const float g = src[(r - r0) * TILE_M + f] * sc, u = src_u[(r - r0) * TILE_M + f] * sc;
        if (good && o < p.O[0]) p.act[(size_t)row * p.O[0] + o] = __float2bfloat16_rn((g / (1.0f + expf(-g))) * u);
      }
    } else if (EPI == EPI_TOPK) {
      // which rows need candidates (a list made by an earlier kernel: read after the dependency wait, i.e. here)
      unsigned char *want = (unsigned char *)wpart;                // [256]
      for (int t = threadIdx.x; t < 256; t += 128) want[t] = p.want_rows ? 0 : 1;
      __syncthreads();
      if (p.want_rows)
        for (int t = threadIdx.x; t < p.n_want; t += 128) { const int wr = p.want_rows[t]; if (wr >= 0 && wr < 256) want[wr] = 1; }
      __syncthreads();
      if (good && p.out_f32 && o < p.O[0])
        for (int r = r0; r < r1; r++) p.out_f32[(size_t)(c0 + r) * p.ldo + o] = src[(r - r0) * TILE_M + f] * inv_s[c0 + r];
      // One warp takes four rows at a time: their selection rounds are four independent dependency chains, written
      // without branches so that they interleave (a CTA has only four warps, nothing else hides the latencies).
      // Lane l holds features l, l+32, l+64, l+96 of the tile as order-preserving keys; id < 0 = nothing there.
      const int K = p.topk;
      for (int rb = r0 + warp; rb < r1; rb += 16) {
        unsigned key[4][4];
        int id[4][4];
        bool act[4];
        size_t slot[4];
#pragma unroll
        for (int q = 0; q < 4; q++) {
          const int r = rb + 4 * q, row = c0 + r;
          const int rs = r < r1 ? r : r0;                                  // a row that exists (results are masked)
          act[q] = good && r < r1 && want[row < 256 ? row : 255];          // uniform over the warp
          slot[q] = (size_t)row * p.cand_ld * K + (size_t)blockIdx.x * K;
          const float sc = inv_s[c0 + rs];
          float v[4];
          float mx = -INFINITY;
#pragma unroll
          for (int j2 = 0; j2 < 4; j2++) {
            const int ff = lane + 32 * j2, oo = tm * TILE_M + ff;
            id[q][j2] = (act[q] && oo < p.O[0]) ? oo : -1;
            v[j2] = id[q][j2] >= 0 ? src[(rs - r0) * TILE_M + ff] * sc : -INFINITY;
            key[q][j2] = ordered_key(v[j2]);
            mx = fmaxf(mx, v[j2]);
          }
          for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
          float sum = 0.0f;
#pragma unroll
          for (int j2 = 0; j2 < 4; j2++) sum += id[q][j2] >= 0 ? expf(v[j2] - mx) : 0.0f;
          for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
          // row-major: all candidates / statistics of a row are contiguous, so that the merge fetches a row in one go
          if (act[q] && lane == 0) { p.cand_max[(size_t)row * p.cand_ld + blockIdx.x] = mx; p.cand_sum[(size_t)row * p.cand_ld + blockIdx.x] = sum; }
        }
        for (int c = 0; c < K; c++) {
#pragma unroll
          for (int q = 0; q < 4; q++) {
            unsigned bk = 0u;
            int bi = -1;
#pragma unroll
            for (int j2 = 0; j2 < 4; j2++) {
              const bool better = id[q][j2] >= 0 && (bi < 0 || key[q][j2] > bk || (key[q][j2] == bk && id[q][j2] < bi));
              bk = better ? key[q][j2] : bk;
              bi = better ? id[q][j2] : bi;
            }
            unsigned wk;
            const int wi = warp_best(bk, bi, &wk);
#pragma unroll
            for (int j2 = 0; j2 < 4; j2++) id[q][j2] = (id[q][j2] == wi) ? -1 : id[q][j2];   // taken (wi = -1: tile exhausted)
            if (act[q] && lane == 0) { p.cand_val[slot[q] + c] = wi < 0 ? 0.0f : key_value(wk); p.cand_idx[slot[q] + c] = wi; }
          }
        }
      }
    } else {   // EPI_ARGMAX
      if (good && p.out_f32 && o < p.O[0])
        for (int r = r0; r < r1; r++) p.out_f32[(size_t)(c0 + r) * p.ldo + o] = red[r * TILE_M + f] * inv_s[c0 + r];
      // thread t scans half of the tile's features for row t % 64, starting at a row-dependent feature
      // so that the 32 rows of a warp touch 32 different banks
      const int row = threadIdx.x & (CHUNK - 1), hf = threadIdx.x >> 6;
      float bv = 0.0f;
      int bi = -1;
      if (row < nrow) {
        for (int j = 0; j < 64; j++) {
          int ff = hf * 64 + ((j + row) & 63), oo = tm * TILE_M + ff;
          float v = red[row * TILE_M + ff];
          if (oo < p.O[0] && (bi < 0 || v > bv || (v == bv && oo < bi))) { bv = v; bi = oo; }
        }
      }
      if (hf == 1) { wpart[row] = bv; wpart[CHUNK + row] = __int_as_float(bi); }
      __syncthreads();
      if (hf == 0 && row < nrow && good) {
        float ov = wpart[row];
        int oi = __float_as_int(wpart[CHUNK + row]);
        if (oi >= 0 && (bi < 0 || ov > bv || (ov == bv && oi < bi))) { bv = ov; bi = oi; }
        p.best_val[(size_t)blockIdx.x * p.best_ld + c0 + row] = bv;
        p.best_idx[(size_t)blockIdx.x * p.best_ld + c0 + row] = bi;
      }
    }
    // peers may still be reading this CTA's red; nobody overwrites or leaves before all are done
    if (S > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); else __syncthreads();
  }
  if (*abort_flag && threadIdx.x == 0 && xr == 0) {
    // gave up on a wait: no bulk copy may still be landing in this CTA's shared memory when it exits.  Every stage
    // load that was issued and not seen complete is waited for (bounded; a load that was never issued runs the wait out).
    // (Pairs: the even CTA's barriers count both CTAs' bytes, and the odd CTA leaves only after the barrier below.)
    for (int i = *n_consumed; i < *n_issued; i++) mbar_wait(&full[i % stages], (i / stages) & 1, p.spin);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (DUO) cluster_sync_all(); else __syncthreads();   // pairs: neither CTA frees tensor memory the other's MMAs may still use
  if (warp == 1) {
    if (DUO) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (p.stamp && threadIdx.x == 0) atomicMin(p.stamp + 1, ~global_ns());
}

// ----------------------------------------------------------------------------------------------
// Gate/up GEMM with SiLU(gate) * up for wide row tiles (129..256 token rows).  At this width the k-block of activations
// (32 KB) is twice a weight tile, and re-reading it from L2 for every weight tile is what bounds the loop.  Here ONE CTA
// owns the gate tile AND the up tile of the same 128 features: both MMAs of a k-block share one activation tile
// (64 KB per stage instead of 96), the two accumulators fill the tensor memory (2 x 256 columns), and since a thread
// then holds gate and up of its feature for every row the activation is applied straight from the accumulators:
// no cluster, no shared-memory round trip.
// DUO: two neighbouring feature tiles as a CTA pair (cta_group::2, cluster of 2): each CTA streams its own gate and up
// tile and HALF of the activation rows, the even CTA issues one M = 256 MMA per accumulator and k-step (fill bytes per
// k-block 48 KB instead of 64 KB per CTA, four stages instead of three).
// PAIR_THREADS threads: several threads share a feature (tensor-memory lane) and split the rows in the epilogue, which
// converts 2 x 256 accumulator columns per feature (with 128 threads it took a quarter of the launch).
constexpr int PAIR_THREADS = 512, PAIR_GROUPS = PAIR_THREADS / 128;
template <int NT, bool DUO = false>
__global__ void __launch_bounds__(PAIR_THREADS) gemm_swiglu_pair_kernel(const __grid_constant__ FusedParams p) {
  constexpr int B_BYTES = (DUO ? NT / 2 : NT) * TILE_K * 2;
  constexpr int STAGE = 2 * A_BYTES + B_BYTES;
  constexpr int TMEM_COLS = 2 * NT;
  static_assert(TMEM_COLS <= 512, "two accumulators must fit the tensor memory");
  extern __shared__ unsigned char smem_raw[];
  unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char *ctrl = tiles + p.ctrl_off;
  uint64_t *full = (uint64_t *)ctrl;
  uint64_t *empty = full + MAX_STAGES;
  uint64_t *acc_bar = empty + MAX_STAGES;
  uint32_t *tmem_slot = (uint32_t *)(acc_bar + 1);
  volatile uint32_t *abort_flag = tmem_slot + 1;
  volatile int *n_issued = (volatile int *)(tmem_slot + 2), *n_consumed = (volatile int *)(tmem_slot + 3);
  float *inv_s = (float *)(ctrl + 512);          // [256] per-row input scale

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int stages = p.stages, KB = p.KB;
  const int tm = blockIdx.x;                     // feature tile (of gate and of up)
  const uint32_t crank = DUO ? cluster_rank() : 0u;
  const int xr = (int)(crank & 1u);              // DUO: position in the pair (0 issues the MMAs)

  if (threadIdx.x == 0) {
    for (int i = 0; i < stages; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_bar, 1);
    *abort_flag = 0;
    *n_issued = 0; *n_consumed = 0;
    if (DUO && crank != (blockIdx.x & 1u)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 224, blockIdx.x, (int)crank); }   // pairs = (even, odd) tile
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    if (DUO) {
      asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
    } else {
      asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                   : "memory");
      asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (DUO) cluster_sync_all(); else __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  pdl_trigger();

  if (DUO && *abort_flag) {
    pdl_wait();
  } else if (DUO && warp == 0) {
    // ---- producer warp of a CTA pair: every byte of both CTAs is counted on the even CTA's full barrier
    const uint64_t pol = l2_policy_evict_first();
    const int npre = KB < stages ? KB : stages;
    if (elect_one())
      for (int i = 0; i < npre; i++) {
        unsigned char *a = tiles + i * STAGE;
        const uint32_t fb = mapa_u32(smem_u32(&full[i]), 0u);
        if (xr == 0) mbar_expect_tx(&full[i], 2 * STAGE);
        tma_load_2d_pair_hint(a, &p.map_w[0], i * TILE_K, tm * TILE_M, fb, pol);
        tma_load_2d_pair_hint(a + A_BYTES, &p.map_w[1], i * TILE_K, tm * TILE_M, fb, pol);
      }
    __syncwarp();
    pdl_wait();
    if (elect_one()) {
      if (p.stamp) atomicMin(p.stamp, global_ns());
      for (int i = 0; i < npre; i++)
        tma_load_2d_pair(tiles + i * STAGE + 2 * A_BYTES, &p.map_x, i * TILE_K, xr * (NT / 2), mapa_u32(smem_u32(&full[i]), 0u));
    }
    __syncwarp();
    int i = npre, st = 0;
    uint32_t ph = 0;
    for (; i < KB; i++) {
      if (!mbar_wait_warp(&empty[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 225, blockIdx.x, i); break; }
      if (elect_one()) {
        unsigned char *a = tiles + st * STAGE;
        const uint32_t fb = mapa_u32(smem_u32(&full[st]), 0u);
        if (xr == 0) mbar_expect_tx(&full[st], 2 * STAGE);
        tma_load_2d_pair_hint(a, &p.map_w[0], i * TILE_K, tm * TILE_M, fb, pol);
        tma_load_2d_pair_hint(a + A_BYTES, &p.map_w[1], i * TILE_K, tm * TILE_M, fb, pol);
        tma_load_2d_pair(a + 2 * A_BYTES, &p.map_x, i * TILE_K, xr * (NT / 2), fb);
      }
      __syncwarp();
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
    if (lane == 0) *n_issued = i;
  } else if (!DUO && warp == 0) {
    // ---- producer warp (the elected lane issues): the weight tiles do not depend on the previous kernel
    const uint64_t pol = l2_policy_evict_first();
    const int npre = KB < stages ? KB : stages;
    if (elect_one())
      for (int i = 0; i < npre; i++) {
        unsigned char *a = tiles + i * STAGE;
        mbar_expect_tx(&full[i], STAGE);
        tma_load_2d_hint(a, &p.map_w[0], i * TILE_K, tm * TILE_M, &full[i], pol);
        tma_load_2d_hint(a + A_BYTES, &p.map_w[1], i * TILE_K, tm * TILE_M, &full[i], pol);
      }
    __syncwarp();
    pdl_wait();
    if (elect_one()) {
      if (p.stamp) atomicMin(p.stamp, global_ns());
      for (int i = 0; i < npre; i++) tma_load_2d(tiles + i * STAGE + 2 * A_BYTES, &p.map_x, i * TILE_K, 0, &full[i]);
    }
    __syncwarp();
    int i = npre, st = 0;
    uint32_t ph = 0;
    for (; i < KB; i++) {
      if (!mbar_wait_warp(&empty[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 220, blockIdx.x, i); break; }
      if (elect_one()) {
        unsigned char *a = tiles + st * STAGE;
        mbar_expect_tx(&full[st], STAGE);
        tma_load_2d_hint(a, &p.map_w[0], i * TILE_K, tm * TILE_M, &full[st], pol);
        tma_load_2d_hint(a + A_BYTES, &p.map_w[1], i * TILE_K, tm * TILE_M, &full[st], pol);
        tma_load_2d(a + 2 * A_BYTES, &p.map_x, i * TILE_K, 0, &full[st]);
      }
      __syncwarp();
      if (++st == stages) { st = 0; ph ^= 1u; }
    }
    if (lane == 0) *n_issued = i;
  } else {
    pdl_wait();
    if (DUO && warp == 1) {
      // ---- MMA issuer warp of a CTA pair (even CTA only): M = 256 over both CTAs' gate tiles, then both up tiles
      if (xr == 0) {
        constexpr uint32_t idesc = umma_idesc_m(NT, 2 * TILE_M);
        const uint32_t partner_base = ld_peer_u32(smem_u32(tmem_slot), 1u);
        if (partner_base != tmem_base) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 226, blockIdx.x, (int)partner_base); }
        const uint64_t desc0 = umma_desc_sw128(smem_u32(tiles));
        int i = 0, st = 0;
        uint32_t ph = 0, ready = 0;
        if (!*abort_flag)
          for (; i < KB; i++) {
            if (!ready && !mbar_wait_warp(&full[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 227, blockIdx.x, i); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t dg = desc0 + (uint64_t)((st * STAGE) >> 4), du = dg + (A_BYTES >> 4), db = dg + ((2 * A_BYTES) >> 4);
            int nst = st + 1;
            uint32_t nph = ph;
            if (nst == stages) { nst = 0; nph ^= 1u; }
            if (elect_one()) {
#pragma unroll
              for (int j = 0; j < TILE_K / UMMA_K; j++) {
                umma_bf16_pair(tmem_base, dg + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);
                umma_bf16_pair(tmem_base + NT, du + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);
              }
              umma_commit_pair(&empty[st], 0u);
            }
            __syncwarp();
            ready = mbar_test_warp(&full[nst], nph) ? 1u : 0u;
            st = nst; ph = nph;
          }
        if (lane == 0) *n_consumed = i;
        __syncwarp();
        if (!*abort_flag && elect_one()) umma_commit_pair(acc_bar, 0u);
      }
    } else if (!DUO && warp == 1) {
      // ---- MMA issuer warp (the elected lane issues): gate accumulator at column 0, up accumulator at column NT
      constexpr uint32_t idesc = umma_idesc(NT);
      const uint64_t desc0 = umma_desc_sw128(smem_u32(tiles));
      int i = 0, st = 0;
      uint32_t ph = 0, ready = 0;
      for (; i < KB; i++) {
        if (!ready && !mbar_wait_warp(&full[st], ph, p.spin)) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 221, blockIdx.x, i); break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t dg = desc0 + (uint64_t)((st * STAGE) >> 4), du = dg + (A_BYTES >> 4), db = dg + ((2 * A_BYTES) >> 4);
        int nst = st + 1;
        uint32_t nph = ph;
        if (nst == stages) { nst = 0; nph ^= 1u; }
        if (elect_one()) {
#pragma unroll
          for (int j = 0; j < TILE_K / UMMA_K; j++) {
            umma_bf16(tmem_base, dg + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);
            umma_bf16(tmem_base + NT, du + 2 * j, db + 2 * j, idesc, (i | j) ? 1u : 0u);
          }
          umma_commit(&empty[st]);
        }
        __syncwarp();
        ready = mbar_test_warp(&full[nst], nph) ? 1u : 0u;
        st = nst; ph = nph;
      }
      if (lane == 0) *n_consumed = i;
      __syncwarp();
      if (elect_one()) umma_commit(acc_bar);
    } else if (warp >= 2) {
      for (int r = threadIdx.x - 64; r < p.rows; r += PAIR_THREADS - 64) {
        float sc = 1.0f;
        if (p.ssq_in) {
          float ss = 0.0f;
          for (int t = 0; t < p.ssq_in_tiles; t++) ss += p.ssq_in[(size_t)t * p.ssq_ld + r];
          sc = 1.0f / sqrtf(ss * p.inv_k_in + p.eps);
        }
        inv_s[r] = sc;
      }
    }
  }
  __syncthreads();

  int good = 0;
  if (lane == 0) {
    bool ok = *abort_flag ? false : mbar_wait(acc_bar, 0, p.spin);
    if (!ok && !*abort_flag) { *abort_flag = 1; set_status(p.status, ST_TIMEOUT, 222, blockIdx.x, 0); }
    good = (ok && !*abort_flag) ? 1 : 0;
  }
  good = __shfl_sync(0xffffffffu, good, 0);
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

  // ---- epilogue: thread = feature f (tensor-memory lane), 16 rows (columns) of both accumulators at a time
  const int o = tm * TILE_M + (threadIdx.x & (TILE_M - 1));
  const int hw = threadIdx.x >> 7;               // which share of the rows (accumulator columns) this thread converts
  if (good) {
#pragma unroll 1
    for (int cc = hw * (NT / PAIR_GROUPS); cc < p.rows && cc < (hw + 1) * (NT / PAIR_GROUPS); cc += 16) {
      uint32_t g[16], u[16];
      tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)cc, g);
      tmem_ld16(tmem_base + ((uint32_t)((warp & 3) * 32) << 16) + (uint32_t)(NT + cc), u);
      if (o < p.O[0]) {
#pragma unroll
        for (int j = 0; j < 16; j++) {
          const int row = cc + j;
          if (row < p.rows) {
            const float sc = inv_s[row];
            const float gv = __uint_as_float(g[j]) * sc, uv = __uint_as_float(u[j]) * sc;
            p.act[(size_t)row * p.O[0] + o] = __float2bfloat16_rn((gv / (1.0f + expf(-gv))) * uv);
          }
        }
      }
    }
  }
  if (*abort_flag && threadIdx.x == 0 && xr == 0) {      // no bulk copy may still be landing when the CTA exits
    for (int i = *n_consumed; i < *n_issued; i++) mbar_wait(&full[i % stages], (i / stages) & 1, p.spin);
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  if (DUO) cluster_sync_all(); else __syncthreads();   // pairs: neither CTA frees tensor memory the other's MMAs may still use
  if (warp == 1) {
    if (DUO) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
    else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
  if (p.stamp && threadIdx.x == 0) atomicMin(p.stamp + 1, ~global_ns());
}

// ---------------------------------------------------------------------------------------------- host side
int pick_nt(int rows) { return rows <= 16 ? 16 : rows <= 64 ? 64 : rows <= 128 ? 128 : 256; }

constexpr int NUM_SMS = 148;
constexpr int SMEM_ONE = 200 * 1024;      // ring budget with one CTA per SM
constexpr int SMEM_TWO = 104 * 1024;      // ring budget that lets two CTAs share an SM

struct Plan { int nt, tiles, S, Sk, stages, smem, ctrl_off, KB, chunk; bool pair, duo; };

// K slices per feature tile.  An SM streams at a capped rate whether one or two CTAs feed it, so the time
// of a launch goes with (CTAs on the busiest SM) x (k-blocks per CTA + a fixed cost per CTA); two CTAs per SM
// are needed to hide one CTA's MMA and epilogue time behind the other's loads.
int g_target_ctas = 222;   // measured best on the 8B shapes (1.5 CTAs per SM)
constexpr int MAX_CLUSTER = 8;    // portable cluster sizes only: size 9 (non-portable) measured 20 % slower per step

// force_two: plan a wide tile (whose full ring takes the SM) as two CTAs per SM with two-stage rings
constexpr int NUM_GPCS = 8;
constexpr int MAX_BUMPED_CTAS = 266;   // 90 % of the 296 CTA slots: fuller grids fail to place all their clusters
// duo: neighbouring feature tiles as CTA pairs (clusters of 2 x Sk members; the stage holds half of the activation rows)
Plan make_plan(FusedEpi epi, const FusedGemmArgs &a, bool force_two = false, bool duo = false) {
  Plan pl;
  pl.duo = duo;
  pl.nt = pick_nt(a.rows);
  pl.KB = (a.I + TILE_K - 1) / TILE_K;
  pl.tiles = fused_gemm_tiles(epi, a);
  // gate/up below 256 rows: gate and up tile in ONE CTA (256 rows: the pair kernel without K split)
  pl.pair = epi == EPI_SWIGLU && pl.nt <= 128;
  const int stage = (pl.pair ? 2 : 1) * A_BYTES + (duo ? pl.nt / 2 : pl.nt) * TILE_K * 2;
  const int wmul = (epi == EPI_SWIGLU && !pl.pair) ? 2 : 1;   // cluster members per K slice
  const int smax = MAX_CLUSTER / (duo ? 2 : wmul);
  const bool wide = duo || SMEM_TWO / stage < (pl.pair ? 2 : 3);     // 256-row tiles: the ring of one CTA takes the SM
  const bool one_per_sm = wide && !force_two;
  const int target = one_per_sm ? NUM_SMS : g_target_ctas;   // one wave
  int Sk = 1;
  if (epi != EPI_ARGMAX) {
    Sk = one_per_sm ? target / std::max(1, pl.tiles * wmul)  // never more CTAs than SMs
                    : (target + pl.tiles * wmul / 2) / std::max(1, pl.tiles * wmul);   // nearest to the target CTA count
    Sk = std::max(1, std::min(Sk, smax));
    Sk = std::max(1, std::min(Sk, pl.KB / 4));
  }
  // One more K slice when that shortens the longest per-SM queue (CTAs per SM x k-blocks per CTA: with 64 tiles
  // of the 70B shapes, 4 slices make 256 CTAs of 112 k-blocks against 192 of 150) and every cluster can still be
  // placed in the first wave: a cluster lives inside one GPC, and with two CTAs per SM a GPC of at least 16 SMs holds 32 / S clusters of S CTAs.  (The
  // occupancy query counts one CTA per SM for these launches, so the bound is spelled out here.)
  if (!one_per_sm && epi != EPI_ARGMAX && a.split == 0) {
    auto queue = [&](int sk) { return ((pl.tiles * wmul * sk + NUM_SMS - 1) / NUM_SMS) * ((pl.KB + sk - 1) / sk); };
    const int up = Sk + 1, s_up = up * wmul;
    // only up to clusters of 4: with 7 -> 8 slices on the 8B shapes the longer reduction and the fuller grid (less
    // room for the next launch's early CTAs) cost more than the shorter queue saves (+2.6 % per step, measured)
    if (s_up <= 4 && up <= smax && up <= pl.KB / 4 && pl.tiles * s_up <= MAX_BUMPED_CTAS && pl.tiles <= NUM_GPCS * (32 / s_up) &&
        queue(up) < queue(Sk)) {
      Sk = up;
    }
  }
  if (a.split > 0) Sk = std::max(1, std::min(std::min(a.split, smax), pl.KB));
  pl.Sk = Sk;
  pl.S = Sk * wmul;
  // more tiles than SMs and a ring that fills the SM: two CTAs with two stages each beat two waves of one
  const int budget = !wide ? SMEM_TWO : ((force_two || pl.tiles * wmul * Sk > NUM_SMS) ? 2 * stage : SMEM_ONE);
  int stages = std::max(2, std::min(MAX_STAGES, budget / stage));
  if (a.stages > 0) stages = std::max(2, std::min(std::min(a.stages, MAX_STAGES), (220 * 1024) / stage));
  int per_slice = (pl.KB + Sk - 1) / Sk;
  stages = std::max(2, std::min(stages, per_slice));
  pl.stages = stages;
  // rows per epilogue round: accumulator dump [chunk][128] + this CTA's reduced rows; wide tiles take the most rows
  // the stage ring (free by then) holds, which saves cluster barriers
  auto epi_bytes = [&](int ch) {
    const int mine = pl.S > 1 ? (ch + pl.S - 1) / pl.S : 0;
    const int sum_rows = pl.S > 1 ? (epi == EPI_SWIGLU ? ch / 2 + mine : mine) : 0;
    return ((pl.pair ? 2 : 1) * ch + sum_rows) * TILE_M * 4;
  };
  pl.chunk = CHUNK;
  if (epi != EPI_ARGMAX)
    for (int ch = MAX_CHUNK; ch > CHUNK; ch >>= 1)
      if (ch <= pl.nt && epi_bytes(ch) <= std::max(stages * stage, 2 * CHUNK * TILE_M * 4)) { pl.chunk = ch; break; }
  pl.ctrl_off = (std::max(stages * stage, std::max(epi_bytes(pl.chunk), 2 * CHUNK * TILE_M * 4)) + 1023) & ~1023;
  pl.smem = pl.ctrl_off + 512 + 256 * 4 + 4 * MAX_CHUNK * 4 + 1024 /*alignment slack*/;
  return pl;
}

template <int NT, int EPI, bool PAIR = false, bool DUO = false>
int launch_inst(const FusedParams &p, const Plan &pl, bool pdl, cudaStream_t s) {
  static SmemLimit limit;
  if (!limit.ensure(gemm_fused_kernel<NT, EPI, PAIR, DUO>, pl.smem)) return -6;
  if (pl.S * (DUO ? 2 : 1) > 8 || (DUO && (pl.tiles & 1))) return -1;   // portable cluster sizes only; pairs need an even tile count
  if (!launch_allowed()) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.tiles, pl.S, 1);
  cfg.blockDim = dim3(fused_threads(NT, EPI), 1, 1);
  cfg.dynamicSmemBytes = pl.smem;
  cfg.stream = s;
  cudaLaunchAttribute at[2];
  int na = 0;
  if (pl.S > 1 || DUO) {
    at[na].id = cudaLaunchAttributeClusterDimension;
    at[na].val.clusterDim.x = DUO ? 2 : 1; at[na].val.clusterDim.y = pl.S; at[na].val.clusterDim.z = 1;
    na++;
  }
  if (pdl) {
    at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[na].val.programmaticStreamSerializationAllowed = 1;
    na++;
  }
  cfg.attrs = at;
  cfg.numAttrs = na;
  return cudaLaunchKernelEx(&cfg, gemm_fused_kernel<NT, EPI, PAIR, DUO>, p) == cudaSuccess ? 0 : -6;
}

// clusters of the plan's shape that can be resident at once (0: unknown)
template <int NT, int EPI>
int resident_clusters_inst(const Plan &pl) {
  static int cached_smem = -1, cached_S = -1, cached_n = 0;
  if (cached_smem == pl.smem && cached_S == pl.S) return cached_n;
  if (cudaFuncSetAttribute(gemm_fused_kernel<NT, EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, pl.smem) != cudaSuccess) return 0;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(pl.tiles, pl.S, 1);
  cfg.blockDim = dim3(fused_threads(NT, EPI), 1, 1);
  cfg.dynamicSmemBytes = pl.smem;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = pl.S; at[0].val.clusterDim.z = 1;
  cfg.attrs = at;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, gemm_fused_kernel<NT, EPI>, &cfg) != cudaSuccess) { cudaGetLastError(); n = 0; }
  cached_smem = pl.smem; cached_S = pl.S; cached_n = n;
  return n;
}
int resident_clusters_wide(FusedEpi epi, const Plan &pl) {
  if (pl.nt != 256) return 0;
  switch (epi) {
    case EPI_F32: return resident_clusters_inst<256, EPI_F32>(pl);
    case EPI_RESID: return resident_clusters_inst<256, EPI_RESID>(pl);
    case EPI_QKV: return resident_clusters_inst<256, EPI_QKV>(pl);
    case EPI_SWIGLU: return resident_clusters_inst<256, EPI_SWIGLU>(pl);
    default: return 0;
  }
}

template <int EPI>
int launch_epi(const FusedParams &p, const Plan &pl, bool pdl, cudaStream_t s) {
  switch (pl.nt) {
    case 16: return launch_inst<16, EPI>(p, pl, pdl, s);
    case 64: return launch_inst<64, EPI>(p, pl, pdl, s);
    case 128: return launch_inst<128, EPI>(p, pl, pdl, s);
    default: return launch_inst<256, EPI>(p, pl, pdl, s);
  }
}
int launch_swiglu_pair(const FusedParams &p, const Plan &pl, bool pdl, cudaStream_t s) {
  switch (pl.nt) {
    case 16: return launch_inst<16, EPI_SWIGLU, true>(p, pl, pdl, s);
    case 64: return launch_inst<64, EPI_SWIGLU, true>(p, pl, pdl, s);
    default: return launch_inst<128, EPI_SWIGLU, true>(p, pl, pdl, s);
  }
}

}  // namespace

void fused_gemm_set_target_ctas(int n) { g_target_ctas = n; }
// 256-row tiles of neighbouring feature tiles as CTA pairs.  Bit 0: the split-K kernel (measured no faster: off); bit 1: the
// gate/up kernel (gate/up launch -1 %, C3 step -0.6 %: on)
namespace { int g_pairs = 0, g_pairs_swiglu = 1; }
void fused_gemm_set_pairs(int on) { g_pairs = on & 1; g_pairs_swiglu = (on >> 1) & 1; }

int fused_gemm_tiles(FusedEpi epi, const FusedGemmArgs &a) {
  if (epi == EPI_SWIGLU) return (a.O[0] + TILE_M - 1) / TILE_M;
  int t = 0;
  for (int j = 0; j < a.nw; j++) t += (a.O[j] + TILE_M - 1) / TILE_M;
  return t;
}

bool fused_gemm_supported(FusedEpi epi, const FusedGemmArgs &a) {
  if (a.rows < 1 || a.rows > 256 || a.I < 8 || (a.I % 8) != 0 || ((uintptr_t)a.x & 15)) return false;
  int need = epi == EPI_QKV ? 3 : epi == EPI_SWIGLU ? 2 : 1;
  if (a.nw != need) return false;
  for (int j = 0; j < a.nw; j++)
    if (!a.w[j] || ((uintptr_t)a.w[j] & 15) || a.O[j] < 1) return false;
  if (epi == EPI_SWIGLU && a.O[0] != a.O[1]) return false;
  if (epi == EPI_TOPK && (a.topk < 1 || a.topk > 16 || !a.cand_val || !a.cand_idx || !a.cand_max || !a.cand_sum || a.cand_ld < (a.O[0] + TILE_M - 1) / TILE_M)) return false;
  if (epi == EPI_QKV) {
    if (a.hd < 2 || a.hd > TILE_M || (a.hd & (a.hd - 1))) return false;
    if (a.O[0] != a.H * a.hd || a.O[1] != a.G * a.hd || a.O[2] != a.G * a.hd) return false;
  }
  return true;
}

int fused_gemm_launch(TmaMaps *g, FusedEpi epi, const FusedGemmArgs &a, cudaStream_t s) {
  if (!g || !fused_gemm_supported(epi, a)) return -1;
  Plan pl = make_plan(epi, a);
  // 256 rows: CTA pairs when every weight's tile count is even (pairs never straddle two weights)
  bool duo = g_pairs && pl.nt == 256 && (epi == EPI_F32 || epi == EPI_RESID || epi == EPI_QKV);
  for (int j = 0; j < a.nw; j++) duo = duo && (a.O[j] % (2 * TILE_M)) == 0;
  if (duo) pl = make_plan(epi, a, false, true);
  if (!duo && pl.nt == 256 && pl.S > 1 && a.split == 0 && a.stages == 0 && pl.tiles * pl.S <= NUM_SMS) {
    // clusters are placed inside one GPC: a grid that counts fewer CTAs than SMs can still need a second wave
    const int fit = resident_clusters_wide(epi, pl);
    if (fit > 0 && pl.tiles > fit) pl = make_plan(epi, a, true);
  }
  FusedParams p;
  memset(&p, 0, sizeof p);
  for (int j = 0; j < a.nw; j++) {
    const CUtensorMap *mw = tma_maps_get(g, a.w[j], a.O[j], a.I, TILE_M);
    if (!mw) return -6;
    p.map_w[j] = *mw;
    p.O[j] = a.O[j];
  }
  const CUtensorMap *mx = tma_maps_get(g, a.x, a.rows, a.I, duo ? pl.nt / 2 : pl.nt);   // pairs: each CTA loads half of the rows
  if (!mx) return -6;
  p.map_x = *mx;
  p.tiles0 = (a.O[0] + TILE_M - 1) / TILE_M;
  p.tiles1 = p.tiles0 + (a.nw > 1 ? (a.O[1] + TILE_M - 1) / TILE_M : 0);
  p.rows = a.rows; p.KB = pl.KB; p.S = pl.S; p.Sk = pl.Sk; p.stages = pl.stages; p.ctrl_off = pl.ctrl_off; p.chunk = pl.chunk;
  p.ssq_in = a.ssq_in; p.ssq_in_tiles = a.ssq_in_tiles; p.ssq_ld = a.ssq_ld; p.inv_k_in = 1.0f / (float)a.k_in; p.eps = a.eps;
  p.out_f32 = a.out_f32; p.ldo = a.ldo;
  p.xres = a.xres; p.gain = a.gain; p.hb = a.hb; p.ssq_out = a.ssq_out; p.taps = a.tap_mask ? a.taps : nullptr;
  p.tap_mask = a.taps ? a.tap_mask : 0; p.resid_add = a.resid_add;
  p.cs = a.cs; p.m = a.m; p.q = a.q; p.pool = a.pool; p.pm = a.pm; p.H = a.H; p.G = a.G; p.hd = a.hd;
  p.act = a.act;
  p.best_val = a.best_val; p.best_idx = a.best_idx; p.best_ld = a.best_ld;
  p.topk = a.topk; p.cand_val = a.cand_val; p.cand_max = a.cand_max; p.cand_sum = a.cand_sum; p.cand_idx = a.cand_idx;
  p.cand_ld = a.cand_ld; p.want_rows = a.want_rows; p.n_want = a.n_want;
  p.status = a.status;
  p.stamp = a.stamp;
  p.spin = a.spin_limit ? a.spin_limit : SPIN_LIMIT;
  p.withhold = a.withhold ? 1 : 0;
  if (epi == EPI_SWIGLU && pl.nt == 256 && a.split == 0 && a.stages == 0) {
    // wide rows: one CTA per (gate tile, up tile) pair sharing the activation tiles; optionally two such CTAs as a
    // CTA pair that also share the activation k-block (each loads half of the rows)
    const bool duo2 = g_pairs_swiglu && (p.tiles0 % 2) == 0;
    const int stage2 = 2 * A_BYTES + (duo2 ? 128 : 256) * TILE_K * 2;
    if (duo2) {
      const CUtensorMap *mxh = tma_maps_get(g, a.x, a.rows, a.I, 128);
      if (!mxh) return -6;
      p.map_x = *mxh;
    }
    p.stages = std::max(2, std::min(SMEM_ONE / stage2, pl.KB));
    p.S = 1; p.Sk = 1;
    p.ctrl_off = (p.stages * stage2 + 1023) & ~1023;
    const int smem = p.ctrl_off + 512 + 256 * 4 + 1024;
    static SmemLimit limit, limit_duo;
    if (!(duo2 ? limit_duo.ensure(gemm_swiglu_pair_kernel<256, true>, smem) : limit.ensure(gemm_swiglu_pair_kernel<256>, smem))) return -6;
    if (!launch_allowed()) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(p.tiles0, 1, 1);
    cfg.blockDim = dim3(PAIR_THREADS, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[2];
    int na = 0;
    if (duo2) {
      at[na].id = cudaLaunchAttributeClusterDimension;
      at[na].val.clusterDim.x = 2; at[na].val.clusterDim.y = 1; at[na].val.clusterDim.z = 1;
      na++;
    }
    if (a.pdl) {
      at[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
      at[na].val.programmaticStreamSerializationAllowed = 1;
      na++;
    }
    cfg.attrs = at;
    cfg.numAttrs = na;
    if (duo2) return cudaLaunchKernelEx(&cfg, gemm_swiglu_pair_kernel<256, true>, p) == cudaSuccess ? 0 : -6;
    return cudaLaunchKernelEx(&cfg, gemm_swiglu_pair_kernel<256>, p) == cudaSuccess ? 0 : -6;
  }
  if (duo) {
    switch (epi) {
      case EPI_F32: return launch_inst<256, EPI_F32, false, true>(p, pl, a.pdl, s);
      case EPI_RESID: return launch_inst<256, EPI_RESID, false, true>(p, pl, a.pdl, s);
      default: return launch_inst<256, EPI_QKV, false, true>(p, pl, a.pdl, s);
    }
  }
  switch (epi) {
    case EPI_F32: return launch_epi<EPI_F32>(p, pl, a.pdl, s);
    case EPI_RESID: return launch_epi<EPI_RESID>(p, pl, a.pdl, s);
    case EPI_QKV: return launch_epi<EPI_QKV>(p, pl, a.pdl, s);
    case EPI_SWIGLU: return pl.pair ? launch_swiglu_pair(p, pl, a.pdl, s) : launch_epi<EPI_SWIGLU>(p, pl, a.pdl, s);
    case EPI_TOPK: return launch_epi<EPI_TOPK>(p, pl, a.pdl, s);
    default: return launch_epi<EPI_ARGMAX>(p, pl, a.pdl, s);
  }
}

}  // namespace spec
