// Tree-masked paged GQA attention on tensor cores (Section 2.2 "tree attention"), bf16.
//
// One CTA owns up to 128 query rows of one (sequence, KV head): the rows are (tree node, query head of
// the GQA group) pairs, so every K/V tile fetched from the paged cache is shared by all nodes and all
// heads of the group.  Keys are split across CTAs (flash-decoding style); each CTA streams 64-key
// tiles through a two-stage cp.async pipeline, computes S = Q K^T and O += P V with mma.sync
// m16n8k16, keeps the softmax statistics in registers (quad shuffles), applies the bit-packed
// ancestor mask to the tail keys, and writes either the final output (one split) or an unnormalised
// partial (several splits) that a small combine kernel merges.
#include <stdio.h>

#include <mutex>

#include <cuda.h>

#include <map>
#include <tuple>

#include "../../include/spec_b200.h"
#include "attn_fast.cuh"
#include "tcgen05_ptx.cuh"

namespace spec {

namespace {

constexpr int KT = 64;          // keys per tile
constexpr int MT = 128;         // query rows per CTA (8 warps x 16)
constexpr int MAX_SPLITS = 32;

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void *src, bool valid) {
  int sz = valid ? 16 : 0;
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sz) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *(uint32_t *)&v;
}

// 2^x on the special-function unit (ex2.approx: -inf -> +0; relative error 2^-22, far below the bf16 rounding of P)
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// Tail masks as one word per 64-key tile.  clip_tail drops mask bits at and past tail_len; tile_allow returns the word
// whose bit j says whether key k0 + j may be attended: every context key (k0 + j < ctx), and tail key
// tt = k0 + j - ctx by bit tt of the row's two-word mask.
__device__ __forceinline__ void clip_tail(uint64_t &lo, uint64_t &hi, int tail_len) {
  if (tail_len < 64) { lo &= (tail_len <= 0) ? 0ull : (~0ull >> (64 - tail_len)); hi = 0ull; }
  else if (tail_len < 128) hi &= (tail_len == 64) ? 0ull : (~0ull >> (128 - tail_len));
}
__device__ __forceinline__ uint64_t tile_allow(uint64_t lo, uint64_t hi, int ctx, int k0) {
  const int sft = k0 - ctx;                     // tail index of the tile's first key (negative: context keys first)
  if (sft <= -64) return ~0ull;
  if (sft < 0) return (~0ull >> (64 + sft)) | (lo << (-sft));
  if (sft == 0) return lo;
  if (sft < 64) return (lo >> sft) | (hi << (64 - sft));
  if (sft == 64) return hi;
  if (sft < 128) return hi >> (sft - 64);
  return 0ull;
}
// byte offset of 16-byte chunk `c` of row `row` in a tile with ROWB bytes per row, XOR-swizzled
template <int ROWB> __device__ __forceinline__ uint32_t swz(int row, int c) { return (uint32_t)(row * ROWB + ((c ^ (row & 7)) << 4)); }

struct AttnParams {
  const bf16 *q;
  const bf16 *kpool, *vpool;
  PageMap pm;
  RowMeta m;
  int tail_len, rows, H, G, rps, nsplit;
  bf16 *out;
  float *part_o;    // [nsplit][rows*H][hd]
  float *part_ml;   // [nsplit][rows*H][2]
  const int32_t *order;   // row block handled by the i-th CTA group (nullptr: i)
  unsigned long long *stamp;   // profiling aid (see KernelStamp), may be null
  int keep_partial;            // 1: write unnormalised partial results and statistics even with a single key split
};

template <int HD>
__global__ void __launch_bounds__(256) attn_mma_kernel(AttnParams p) {
  pdl_wait();
  pdl_trigger();
  KernelStamp stamp_guard(p.stamp);
  constexpr int ROWB = HD * 2, CPR = HD / 8;          // bytes / 16-byte chunks per row
  constexpr int NKS = HD / 16;                        // k-steps of Q K^T
  extern __shared__ __align__(128) unsigned char sm[];
  unsigned char *sK[2] = {sm, sm + 2 * KT * ROWB};
  unsigned char *sV[2] = {sm + KT * ROWB, sm + 3 * KT * ROWB};
  unsigned char *sQ = sm;                              // the Q tile borrows the stage memory before the main loop
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = p.H / p.G;
  const int b = blockIdx.z / p.G, g = blockIdx.z % p.G;
  const int M = p.rps * grp;                           // query rows of this (sequence, KV head)
  const int m0 = blockIdx.x * MT;
  const int row0 = b * p.rps;
  // sequence-level quantities from the first row of the sequence (all rows of a sequence share them)
  int seq = -1, ctx = 0, tb = 0;
  for (int i = 0; i < p.rps; i++) {
    int s = p.m.seq[row0 + i];
    if (s >= 0) { seq = s; ctx = p.m.ctx[row0 + i]; tb = p.m.tail_base[row0 + i]; break; }
  }
  const int nkeys = (seq >= 0) ? ctx + p.tail_len : 0;
  const int ntiles = (nkeys + KT - 1) / KT;
  const int t_begin = (int)(((long long)blockIdx.y * ntiles) / p.nsplit);
  const int t_end = (int)(((long long)(blockIdx.y + 1) * ntiles) / p.nsplit);

  // ---- Q tile -> shared (swizzled) -> A fragments
  for (int id = threadIdx.x; id < MT * CPR; id += 256) {
    int lr = id / CPR, c = id % CPR, mrow = m0 + lr;
    bool v = mrow < M;
    int i = v ? mrow / grp : 0, hq = v ? mrow % grp : 0;
    v = v && p.m.seq[row0 + i] >= 0;
    const bf16 *src = p.q + ((size_t)(row0 + i) * p.H + g * grp + hq) * HD + c * 8;
    cp_async16(smem_u32(sQ + swz<ROWB>(lr, c)), src, v);
  }
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();
  uint32_t qf[NKS][4];
#pragma unroll
  for (int ks = 0; ks < NKS; ks++) {
    int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
    ldsm_x4(smem_u32(sQ + swz<ROWB>(r, c)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
  }
  __syncthreads();

  // rows owned by this thread: rA = quad row, rB = rA + 8 (within the warp's 16 rows)
  const int mA = m0 + warp * 16 + (lane >> 2), mB = mA + 8;
  uint64_t loA = 0, hiA = 0, loB = 0, hiB = 0;
  bool vA = false, vB = false;
  if (mA < M) { int r = row0 + mA / grp; vA = p.m.seq[r] >= 0; if (vA) { loA = p.m.mask_lo[r]; hiA = p.m.mask_hi[r]; } }
  if (mB < M) { int r = row0 + mB / grp; vB = p.m.seq[r] >= 0; if (vB) { loB = p.m.mask_lo[r]; hiB = p.m.mask_hi[r]; } }

  float o[HD / 8][4];
#pragma unroll
  for (int n = 0; n < HD / 8; n++) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.0f; }
  float mxA = -INFINITY, mxB = -INFINITY, lA = 0.0f, lB = 0.0f;
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;    // softmax scale folded into exp2

  auto load_tile = [&](int t, int st) {
    int k0 = t * KT;
    for (int id = threadIdx.x; id < KT * CPR; id += 256) {
      int kr = id / CPR, c = id % CPR, key = k0 + kr;
      bool v = key < nkeys;
      int pos = key < ctx ? key : tb + (key - ctx);
      size_t off = 0;
      if (v) {
        int pidx = pos / p.pm.page_size;
        v = pidx < p.pm.pages_per_seq;
        if (v) {
          int page = p.pm.table[(size_t)seq * p.pm.pages_per_seq + pidx];
          v = page >= 0 && page < p.pm.num_pages;
          off = (((size_t)page * p.G + g) * p.pm.page_size + (pos % p.pm.page_size)) * HD + c * 8;
        }
      }
      if (!v) off = 0;
      cp_async16(smem_u32(sK[st] + swz<ROWB>(kr, c)), p.kpool + off, v);
      cp_async16(smem_u32(sV[st] + swz<ROWB>(kr, c)), p.vpool + off, v);
    }
    cp_async_commit();
  };

  if (t_begin < t_end) load_tile(t_begin, 0);
  for (int t = t_begin; t < t_end; t++) {
    int st = (t - t_begin) & 1;
    if (t + 1 < t_end) { load_tile(t + 1, st ^ 1); cp_async_wait<1>(); } else { cp_async_wait<0>(); }
    __syncthreads();
    // ---- S = Q K^T for 64 keys: 8 n-tiles of 8 keys
    float s[KT / 8][4];
#pragma unroll
    for (int n = 0; n < KT / 8; n++) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.0f; }
#pragma unroll
    for (int ks = 0; ks < NKS; ks++) {
#pragma unroll
      for (int n2 = 0; n2 < KT / 16; n2++) {
        uint32_t b0, b1, b2, b3;
        int kr = n2 * 16 + (lane & 7) + (lane >> 4) * 8, c = ks * 2 + ((lane >> 3) & 1);
        ldsm_x4(smem_u32(sK[st] + swz<ROWB>(kr, c)), b0, b1, b2, b3);
        mma_bf16(s[2 * n2], qf[ks], b0, b1);
        mma_bf16(s[2 * n2 + 1], qf[ks], b2, b3);
      }
    }
    // ---- mask + online softmax (two rows per thread, reductions across the quad)
    float tmA = -INFINITY, tmB = -INFINITY;
#pragma unroll
    for (int n = 0; n < KT / 8; n++) {
#pragma unroll
      for (int e = 0; e < 2; e++) {
        int key = t * KT + n * 8 + (lane & 3) * 2 + e;
        bool in_ctx = key < ctx;
        int tt = key - ctx;
        bool in_tail = !in_ctx && tt < p.tail_len;
        bool okA = vA && (in_ctx || (in_tail && ((tt < 64 ? (loA >> tt) : (hiA >> (tt - 64))) & 1ull)));
        bool okB = vB && (in_ctx || (in_tail && ((tt < 64 ? (loB >> tt) : (hiB >> (tt - 64))) & 1ull)));
        s[n][e] = okA ? s[n][e] : -INFINITY;
        s[n][2 + e] = okB ? s[n][2 + e] : -INFINITY;
        tmA = fmaxf(tmA, s[n][e]);
        tmB = fmaxf(tmB, s[n][2 + e]);
      }
    }
    tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 1)); tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 2));
    tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 1)); tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 2));
    float nmA = fmaxf(mxA, tmA), nmB = fmaxf(mxB, tmB);
    float fA = (nmA == -INFINITY) ? 1.0f : exp2f((mxA - nmA) * sc), fB = (nmB == -INFINITY) ? 1.0f : exp2f((mxB - nmB) * sc);
    float baseA = (nmA == -INFINITY) ? 0.0f : nmA, baseB = (nmB == -INFINITY) ? 0.0f : nmB;
    float rsA = 0.0f, rsB = 0.0f;
    uint32_t pf[KT / 16][4];
#pragma unroll
    for (int n = 0; n < KT / 8; n++) {
      float p0 = exp2f((s[n][0] - baseA) * sc), p1 = exp2f((s[n][1] - baseA) * sc);
      float p2 = exp2f((s[n][2] - baseB) * sc), p3 = exp2f((s[n][3] - baseB) * sc);
      rsA += p0 + p1; rsB += p2 + p3;
      pf[n >> 1][(n & 1) * 2] = pack_bf16(p0, p1);
      pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    rsA += __shfl_xor_sync(0xffffffffu, rsA, 1); rsA += __shfl_xor_sync(0xffffffffu, rsA, 2);
    rsB += __shfl_xor_sync(0xffffffffu, rsB, 1); rsB += __shfl_xor_sync(0xffffffffu, rsB, 2);
    lA = lA * fA + rsA; lB = lB * fB + rsB;
    mxA = nmA; mxB = nmB;
#pragma unroll
    for (int n = 0; n < HD / 8; n++) { o[n][0] *= fA; o[n][1] *= fA; o[n][2] *= fB; o[n][3] *= fB; }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < KT / 16; kk++) {
#pragma unroll
      for (int d2 = 0; d2 < HD / 16; d2++) {
        uint32_t b0, b1, b2, b3;
        int kr = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = d2 * 2 + (lane >> 4);
        ldsm_x4_t(smem_u32(sV[st] + swz<ROWB>(kr, c)), b0, b1, b2, b3);
        mma_bf16(o[2 * d2], pf[kk], b0, b1);
        mma_bf16(o[2 * d2 + 1], pf[kk], b2, b3);
      }
    }
    __syncthreads();      // all warps done with this stage before it is refilled
  }

  // ---- write: final (one split) or partial
  const int qcol = (lane & 3) * 2;
#pragma unroll
  for (int half = 0; half < 2; half++) {
    int mrow = half ? mB : mA;
    if (mrow >= M) continue;
    int r = row0 + mrow / grp, h = g * grp + mrow % grp;
    float l = half ? lB : lA, mx = half ? mxB : mxA;
    if (p.nsplit == 1) {
      float inv = l > 0.0f ? 1.0f / l : 0.0f;
      bf16 *dst = p.out + ((size_t)r * p.H + h) * HD;
#pragma unroll
      for (int n = 0; n < HD / 8; n++)
        *(uint32_t *)(dst + n * 8 + qcol) = pack_bf16(o[n][half * 2] * inv, o[n][half * 2 + 1] * inv);
    } else {
      size_t idx = (size_t)blockIdx.y * p.rows * p.H + (size_t)r * p.H + h;
      float *dst = p.part_o + idx * HD;
#pragma unroll
      for (int n = 0; n < HD / 8; n++) *(float2 *)(dst + n * 8 + qcol) = make_float2(o[n][half * 2], o[n][half * 2 + 1]);
      if ((lane & 3) == 0) { p.part_ml[idx * 2] = mx; p.part_ml[idx * 2 + 1] = l; }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// TMA-staged variant.  One page of one KV head ([page_size][hd], contiguous) is fetched by ONE tensor copy
// (cp.async.bulk.tensor, 128-byte swizzle) per K and per V; a producer warp keeps STAGES 64-key tiles in flight
// through full/empty mbarriers, eight consumer warps run the tensor-core math of the kernel above.  Needs the
// tail keys to follow the context directly (tail_base == ctx, true for every pass of a speculative step) and a
// page size of 16, 32 or 64 keys.  Waits are bounded; a timeout is recorded in the status words.
constexpr uint32_t ATT_SPIN_LIMIT = 1u << 20;
__device__ __forceinline__ void mbar_init(uint64_t *bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t *bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// One lane of a fully converged warp: the producer and issuer warps walk their loops whole and let this lane issue the
// copies / MMAs (the same instructions issued from a branch on the lane id cost the warp about 1.5 x the cycles).
__device__ __forceinline__ bool elect_one() {
  uint32_t pred = 0;
  asm volatile("{\n\t.reg .pred p;\n\telect.sync _|p, 0xffffffff;\n\t@p mov.u32 %0, 1;\n\t}" : "+r"(pred));
  return pred != 0;
}
__device__ __forceinline__ bool mbar_wait(uint64_t *bar, uint32_t parity) {
  uint32_t addr = smem_u32(bar);
  {   // non-blocking test first: a phase that is already complete costs a tenth of a try_wait
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(addr), "r"(parity) : "memory");
    if (ok) return true;
  }
  for (uint32_t it = 0; it < ATT_SPIN_LIMIT; it++) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(addr), "r"(parity)
        : "memory");
    if (ok) return true;
  }
  return false;
}
// the same for a converged warp (all 32 lanes call it): one lane's sight of the completed phase counts for all, so that
// no lane leaves its loop alone and strands the warp's next elect.sync
__device__ __forceinline__ bool mbar_wait_warp(uint64_t *bar, uint32_t parity) {
  const bool ok = mbar_wait(bar, parity);
  const bool any = __any_sync(0xffffffffu, ok);
  if (any && !ok) mbar_wait(bar, parity);      // completed: returns at its first test, with this lane's own acquire
  return any;
}
__device__ __forceinline__ void tma_load_3d(void *smem_dst, const CUtensorMap *map, int c0, int c1, int c2, uint64_t *bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];" ::"r"(
          smem_u32(smem_dst)),
      "l"(map), "r"(smem_u32(bar)), "r"(c0), "r"(c1), "r"(c2)
      : "memory");
}

// Page ids of the (at most four) pages of key tile t, as the producer thread needs them: every load is issued
// before any is used, and the caller asks for tile t + 1 before it starts on tile t, so the table look-ups
// (dependent global loads) are never on the producer's critical path.
__device__ __forceinline__ void tile_pages(int (&pg)[4], const int32_t *tbl, int pages_per_seq, int t, int ps) {
  const int ppt = KT / ps, first = (t * KT) / ps;
#pragma unroll
  for (int j = 0; j < 4; j++) pg[j] = (j < ppt && first + j < pages_per_seq) ? tbl[first + j] : -1;
}

template <int HD, int STAGES>
__global__ void __launch_bounds__(288) attn_tma_kernel(const __grid_constant__ CUtensorMap map_k,
                                                       const __grid_constant__ CUtensorMap map_v, AttnParams p, int32_t *status) {
  pdl_trigger();   // the next kernel may start staging its weights; it still waits for this grid to complete
  pdl_wait();
  KernelStamp stamp_guard(p.stamp);
  constexpr int ROWB = HD * 2, CPR = HD / 8;
  constexpr int NKS = HD / 16;
  constexpr int TILEB = KT * ROWB;                     // bytes of one K (or V) tile
  extern __shared__ __align__(1024) unsigned char sm[];
  unsigned char *sQ = sm + (STAGES - 1) * 2 * TILEB;   // the Q tile borrows the last stage until its fragments are in registers
  uint64_t *full = (uint64_t *)(sm + STAGES * 2 * TILEB);
  uint64_t *empty = full + STAGES;
  uint64_t *q_bar = empty + STAGES;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = p.H / p.G;
  const int zb = blockIdx.z / p.G, g = blockIdx.z % p.G;
  const unsigned nblk = gridDim.z / (unsigned)p.G;
  int b = (p.order && nblk > 1) ? p.order[zb] : zb;    // row block (sequence) of this CTA
  if ((unsigned)b >= nblk) b = zb;
  const int M = p.rps * grp;
  const int m0 = blockIdx.x * MT;
  const int row0 = b * p.rps;
  const int ps = p.pm.page_size;                       // keys per page = rows per tensor copy
  int seq = -1, ctx = 0;
  for (int i = 0; i < p.rps; i++) {
    const int s = p.m.seq[row0 + i], cx = p.m.ctx[row0 + i];   // both loads in flight together
    if (s >= 0) { seq = s; ctx = cx; break; }
  }
  const int nkeys = (seq >= 0) ? ctx + p.tail_len : 0;
  const int ntiles = (nkeys + KT - 1) / KT;
  const int t_begin = (int)(((long long)blockIdx.y * ntiles) / p.nsplit);
  const int t_end = (int)(((long long)(blockIdx.y + 1) * ntiles) / p.nsplit);

  // consumer warps that own at least one query row; the others leave after the Q phase
  const int nactive = (M - m0 >= MT) ? 8 : (M - m0 + 15) / 16;
  // The producer warp sets up the barriers and starts the first K/V copies while the consumer warps fetch Q: the
  // page-table look-up and the copies overlap the Q round trip.  Named barrier 1 (288 threads): the producer only
  // arrives, the consumers wait there for the barrier set-up and for each other's part of the Q tile.
  if (warp < 8) {
    for (int id = threadIdx.x; id < MT * CPR; id += 256) {
      int lr = id / CPR, c = id % CPR, mrow = m0 + lr;
      bool v = mrow < M;
      int i = v ? mrow / grp : 0, hq = v ? mrow % grp : 0;
      v = v && p.m.seq[row0 + i] >= 0;
      const bf16 *src = p.q + ((size_t)(row0 + i) * p.H + g * grp + hq) * HD + c * 8;
      cp_async16(smem_u32(sQ + swz<ROWB>(lr, c)), src, v);
    }
    cp_async_commit();
    cp_async_wait<0>();
    asm volatile("bar.sync 1, 288;" ::: "memory");
  } else {
    // ================================================================ producer
    if (lane == 0) {
      for (int i = 0; i < STAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], nactive); }
      mbar_init(q_bar, nactive);
      asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
      __threadfence_block();
    }
    __syncwarp();
    asm volatile("bar.arrive 1, 288;" ::: "memory");
    if (seq >= 0) {     // the whole warp walks the loop (same page ids in every lane), the elected lane issues the copies
      const int32_t *tbl = p.pm.table + (size_t)seq * p.pm.pages_per_seq;
      const int fallback = tbl[0];                     // keys past the last page are masked; they still need a valid source
      const int ppt = KT / ps;                         // pages per tile
      int cur[4], nxt[4] = {-1, -1, -1, -1};
      if (t_begin < t_end) tile_pages(cur, tbl, p.pm.pages_per_seq, t_begin, ps);
      for (int t = t_begin; t < t_end; t++) {
        const int i = t - t_begin, st = i % STAGES;
        if (t + 1 < t_end) tile_pages(nxt, tbl, p.pm.pages_per_seq, t + 1, ps);
        if (i == STAGES - 1 && !mbar_wait_warp(q_bar, 0)) { if (status) set_status(status, ST_TIMEOUT, 400, blockIdx.z, t); break; }
        if (i >= STAGES && !mbar_wait_warp(&empty[st], (uint32_t)(((i / STAGES) - 1) & 1))) { if (status) set_status(status, ST_TIMEOUT, 401, blockIdx.z, t); break; }
        if (elect_one()) {
          unsigned char *kb = sm + st * 2 * TILEB, *vb = kb + TILEB;
          mbar_expect_tx(&full[st], 2 * TILEB);
#pragma unroll
          for (int pg = 0; pg < 4; pg++) {
            if (pg >= ppt) break;
            int page = cur[pg];
            if (page < 0 || page >= p.pm.num_pages) page = fallback;
            const int row = (page * p.G + g) * ps;
            tma_load_3d(kb + pg * ps * ROWB, &map_k, 0, row, 0, &full[st]);
            tma_load_3d(vb + pg * ps * ROWB, &map_v, 0, row, 0, &full[st]);
          }
        }
        __syncwarp();
#pragma unroll
        for (int pg = 0; pg < 4; pg++) cur[pg] = nxt[pg];
      }
    }
    return;
  }

  // ================================================================== consumers (8 warps x 16 query rows)
  if (warp >= nactive) return;
  uint32_t qf[NKS][4];
#pragma unroll
  for (int ks = 0; ks < NKS; ks++) {
    int r = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
    ldsm_x4(smem_u32(sQ + swz<ROWB>(r, c)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
  }
  __syncwarp();
  if (lane == 0) mbar_arrive(q_bar);
  // byte offset of 16-byte chunk c of key kr inside a tile: [page][half of hd][key in page][128 B], chunks XOR-swizzled
  const int psb = ps * ROWB, psh = __ffs(ps) - 1;      // the page size is a power of two
  auto koff = [&](int kr, int c) -> uint32_t {
    return (uint32_t)((kr >> psh) * psb + (c >> 3) * (ps * 128) + (kr & (ps - 1)) * 128 + (((c & 7) ^ (kr & 7)) << 4));
  };
  const int tb = ctx;                                   // tail keys follow the context
  (void)tb;
  // rows owned by this thread: rA = quad row, rB = rA + 8 (within the warp's 16 rows)
  const int mA = m0 + warp * 16 + (lane >> 2), mB = mA + 8;
  uint64_t loA = 0, hiA = 0, loB = 0, hiB = 0;
  bool vA = false, vB = false;
  if (mA < M) { int r = row0 + mA / grp; vA = p.m.seq[r] >= 0; if (vA) { loA = p.m.mask_lo[r]; hiA = p.m.mask_hi[r]; } }
  if (mB < M) { int r = row0 + mB / grp; vB = p.m.seq[r] >= 0; if (vB) { loB = p.m.mask_lo[r]; hiB = p.m.mask_hi[r]; } }
  clip_tail(loA, hiA, p.tail_len);
  clip_tail(loB, hiB, p.tail_len);

  float o[HD / 8][4];
#pragma unroll
  for (int n = 0; n < HD / 8; n++) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.0f; }
  float mxA = -INFINITY, mxB = -INFINITY, lA = 0.0f, lB = 0.0f;
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;    // softmax scale folded into exp2


  bool alive = true;
  for (int t = t_begin; t < t_end && alive; t++) {
    const int i = t - t_begin, st = i % STAGES;
    if (!mbar_wait(&full[st], (uint32_t)((i / STAGES) & 1))) { if (lane == 0) if (status) set_status(status, ST_TIMEOUT, 402, blockIdx.z, t); alive = false; break; }
    const unsigned char *kbase = sm + st * 2 * TILEB, *vbase = kbase + TILEB;
    // ---- S = Q K^T for 64 keys: 8 n-tiles of 8 keys
    float s[KT / 8][4];
#pragma unroll
    for (int n = 0; n < KT / 8; n++) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.0f; }
#pragma unroll
    for (int ks = 0; ks < NKS; ks++) {
#pragma unroll
      for (int n2 = 0; n2 < KT / 16; n2++) {
        uint32_t b0, b1, b2, b3;
        int kr = n2 * 16 + (lane & 7) + (lane >> 4) * 8, c = ks * 2 + ((lane >> 3) & 1);
        ldsm_x4(smem_u32(kbase + koff(kr, c)), b0, b1, b2, b3);
        mma_bf16(s[2 * n2], qf[ks], b0, b1);
        mma_bf16(s[2 * n2 + 1], qf[ks], b2, b3);
      }
    }
    // ---- mask + online softmax (two rows per thread, reductions across the quad)
    float tmA = -INFINITY, tmB = -INFINITY;
    if (t * KT + KT <= ctx && vA && vB) {
      // every key of the tile is context and both rows are real: nothing to mask
#pragma unroll
      for (int n = 0; n < KT / 8; n++) {
        tmA = fmaxf(tmA, fmaxf(s[n][0], s[n][1]));
        tmB = fmaxf(tmB, fmaxf(s[n][2], s[n][3]));
      }
    } else {
      // one allow word per row for the tile, shifted so that this lane's keys sit at bits 8 n + e
      const uint64_t wA = (vA ? tile_allow(loA, hiA, ctx, t * KT) : 0ull) >> ((lane & 3) * 2);
      const uint64_t wB = (vB ? tile_allow(loB, hiB, ctx, t * KT) : 0ull) >> ((lane & 3) * 2);
      const uint32_t wA0 = (uint32_t)wA, wA1 = (uint32_t)(wA >> 32), wB0 = (uint32_t)wB, wB1 = (uint32_t)(wB >> 32);
#pragma unroll
      for (int n = 0; n < KT / 8; n++) {
#pragma unroll
        for (int e = 0; e < 2; e++) {
          const uint32_t bit = 1u << ((n & 3) * 8 + e);
          const bool okA = ((n < 4 ? wA0 : wA1) & bit) != 0u, okB = ((n < 4 ? wB0 : wB1) & bit) != 0u;
          s[n][e] = okA ? s[n][e] : -INFINITY;
          s[n][2 + e] = okB ? s[n][2 + e] : -INFINITY;
          tmA = fmaxf(tmA, s[n][e]);
          tmB = fmaxf(tmB, s[n][2 + e]);
        }
      }
    }
    tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 1)); tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 2));
    tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 1)); tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 2));
    float nmA = fmaxf(mxA, tmA), nmB = fmaxf(mxB, tmB);
    float fA = (nmA == -INFINITY) ? 1.0f : ex2_approx((mxA - nmA) * sc), fB = (nmB == -INFINITY) ? 1.0f : ex2_approx((mxB - nmB) * sc);
    float baseA = (nmA == -INFINITY) ? 0.0f : nmA, baseB = (nmB == -INFINITY) ? 0.0f : nmB;
    float rsA = 0.0f, rsB = 0.0f;
    uint32_t pf[KT / 16][4];
#pragma unroll
    for (int n = 0; n < KT / 8; n++) {
      float p0 = ex2_approx((s[n][0] - baseA) * sc), p1 = ex2_approx((s[n][1] - baseA) * sc);
      float p2 = ex2_approx((s[n][2] - baseB) * sc), p3 = ex2_approx((s[n][3] - baseB) * sc);
      rsA += p0 + p1; rsB += p2 + p3;
      pf[n >> 1][(n & 1) * 2] = pack_bf16(p0, p1);
      pf[n >> 1][(n & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    rsA += __shfl_xor_sync(0xffffffffu, rsA, 1); rsA += __shfl_xor_sync(0xffffffffu, rsA, 2);
    rsB += __shfl_xor_sync(0xffffffffu, rsB, 1); rsB += __shfl_xor_sync(0xffffffffu, rsB, 2);
    lA = lA * fA + rsA; lB = lB * fB + rsB;
    mxA = nmA; mxB = nmB;
#pragma unroll
    for (int n = 0; n < HD / 8; n++) { o[n][0] *= fA; o[n][1] *= fA; o[n][2] *= fB; o[n][3] *= fB; }
    // ---- O += P V
#pragma unroll
    for (int kk = 0; kk < KT / 16; kk++) {
#pragma unroll
      for (int d2 = 0; d2 < HD / 16; d2++) {
        uint32_t b0, b1, b2, b3;
        int kr = kk * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, c = d2 * 2 + (lane >> 4);
        ldsm_x4_t(smem_u32(vbase + koff(kr, c)), b0, b1, b2, b3);
        mma_bf16(o[2 * d2], pf[kk], b0, b1);
        mma_bf16(o[2 * d2 + 1], pf[kk], b2, b3);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty[st]);              // this warp is done with the stage
  }

  // ---- write: final (one split) or partial
  const int qcol = (lane & 3) * 2;
#pragma unroll
  for (int half = 0; half < 2; half++) {
    int mrow = half ? mB : mA;
    if (mrow >= M) continue;
    int r = row0 + mrow / grp, h = g * grp + mrow % grp;
    float l = half ? lB : lA, mx = half ? mxB : mxA;
    if (p.nsplit == 1 && !p.keep_partial) {
      float inv = l > 0.0f ? 1.0f / l : 0.0f;
      bf16 *dst = p.out + ((size_t)r * p.H + h) * HD;
#pragma unroll
      for (int n = 0; n < HD / 8; n++)
        *(uint32_t *)(dst + n * 8 + qcol) = pack_bf16(o[n][half * 2] * inv, o[n][half * 2 + 1] * inv);
    } else {
      size_t idx = (size_t)blockIdx.y * p.rows * p.H + (size_t)r * p.H + h;
      float *dst = p.part_o + idx * HD;
#pragma unroll
      for (int n = 0; n < HD / 8; n++) *(float2 *)(dst + n * 8 + qcol) = make_float2(o[n][half * 2], o[n][half * 2 + 1]);
      if ((lane & 3) == 0) { p.part_ml[idx * 2] = mx; p.part_ml[idx * 2 + 1] = l; }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// tcgen05 variant for head_dim 128 and more than 16 query rows per (sequence, KV head): the tree passes (verify,
// wide draft levels).  With a long context this pass is bound by the two contractions, not by the cache reads, so
// they run on the fifth-generation tensor cores:
//   S = Q K^T : A = the CTA's 128 query rows (K-major, 128-byte swizzle, written once), B = a 64-key K tile as it lands
//               from TMA ([hd half][key][128 B]), accumulator = 64 columns of tensor memory;
//   O += P V  : A = P (bf16, written to shared memory by the softmax threads), B = the V tile read MN-major (the keys
//               are the contraction dimension and the slow axis of the tile), accumulator = 128 columns that stay in
//               tensor memory for the whole key range.
// Thread r of the four softmax warps owns query row r = tensor-memory lane r: its row maximum and row sum need no
// shuffles.  When a row maximum grows, the warp rescales its 32 rows of O in tensor memory (rare once the maximum has
// settled).  Warp 4 is the TMA producer, warp 5 issues the MMAs.  Same masks, statistics and partial-result format as
// the kernels above.  Every wait is bounded; a timeout is recorded in the status words and the CTA winds down.
constexpr int UM_STAGES = 4;
constexpr int UM_HD = 128;
constexpr int UM_TILE = KT * UM_HD * 2;            // 16 KB: the K (or the V) tile of 64 keys
constexpr int UM_HALF = KT * 128;                  // 8 KB: one 64-element half of head_dim for 64 keys
constexpr int UM_Q_BYTES = MT * UM_HD * 2;         // 32 KB
constexpr int UM_P_BYTES = MT * KT * 2;            // 16 KB
constexpr int UM_XCHG_BYTES = 2 * MT * 4;          // row statistics handed from softmax warpgroup 1 to warpgroup 0
constexpr int UM_SMEM = UM_Q_BYTES + 2 * UM_P_BYTES + UM_STAGES * 2 * UM_TILE + 128 + UM_XCHG_BYTES;
constexpr int UM_THREADS = 320;                    // two softmax warpgroups, the TMA producer warp, the MMA warp
constexpr uint32_t UM_TMEM_COLS = 512;             // S of the two warpgroups: columns 0..127, their O: columns 128..383

// MN-major operand tile with 128-byte swizzle: rows (contraction index) of 128 bytes = 64 elements of the MN
// dimension, 8-row groups 1024 bytes apart, the next 64 MN elements lbo bytes further on.
__device__ __forceinline__ uint64_t umma_desc_sw128_mn(uint32_t saddr, uint32_t lbo) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFF) >> 4);
  d |= (uint64_t)(lbo >> 4) << 16;
  d |= (uint64_t)(1024 >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// 64 consecutive columns of this thread's tensor-memory lane in one instruction
__device__ __forceinline__ void tmem_ld64(uint32_t taddr, float (&v)[64]) {
  uint32_t *u = (uint32_t *)v;
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x64.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, "
      "%32, %33, %34, %35, %36, %37, %38, %39, %40, %41, %42, %43, %44, %45, %46, %47, %48, %49, %50, %51, %52, %53, %54, %55, %56, %57, %58, %59, %60, %61, %62, %63}, [%64];"
      : "=r"(u[0]), "=r"(u[1]), "=r"(u[2]), "=r"(u[3]), "=r"(u[4]), "=r"(u[5]), "=r"(u[6]), "=r"(u[7]), "=r"(u[8]), "=r"(u[9]), "=r"(u[10]),
        "=r"(u[11]), "=r"(u[12]), "=r"(u[13]), "=r"(u[14]), "=r"(u[15]), "=r"(u[16]), "=r"(u[17]), "=r"(u[18]), "=r"(u[19]), "=r"(u[20]),
        "=r"(u[21]), "=r"(u[22]), "=r"(u[23]), "=r"(u[24]), "=r"(u[25]), "=r"(u[26]), "=r"(u[27]), "=r"(u[28]), "=r"(u[29]), "=r"(u[30]),
        "=r"(u[31]), "=r"(u[32]), "=r"(u[33]), "=r"(u[34]), "=r"(u[35]), "=r"(u[36]), "=r"(u[37]), "=r"(u[38]), "=r"(u[39]), "=r"(u[40]),
        "=r"(u[41]), "=r"(u[42]), "=r"(u[43]), "=r"(u[44]), "=r"(u[45]), "=r"(u[46]), "=r"(u[47]), "=r"(u[48]), "=r"(u[49]), "=r"(u[50]),
        "=r"(u[51]), "=r"(u[52]), "=r"(u[53]), "=r"(u[54]), "=r"(u[55]), "=r"(u[56]), "=r"(u[57]), "=r"(u[58]), "=r"(u[59]), "=r"(u[60]),
        "=r"(u[61]), "=r"(u[62]), "=r"(u[63])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&v)[16]) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]), "r"(v[10]),
      "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15])
      : "memory");
}

__global__ void __launch_bounds__(UM_THREADS, 1) attn_umma_kernel(const __grid_constant__ CUtensorMap map_k,
                                                        const __grid_constant__ CUtensorMap map_v, AttnParams p, int32_t *status) {
  pdl_trigger();   // the next kernel may start staging its weights; it still waits for this grid to complete
  pdl_wait();
  KernelStamp stamp_guard(p.stamp);
  constexpr int HD = UM_HD;
  extern __shared__ __align__(1024) unsigned char sm[];
  unsigned char *sQ = sm;                                   // [2 halves][128 rows][128 B]
  unsigned char *sP = sm + UM_Q_BYTES;                      // one [128 rows][128 B] tile (64 keys) per softmax warpgroup
  unsigned char *ring = sP + 2 * UM_P_BYTES;                    // stage: K [2 halves][64 keys][128 B], then V likewise
  uint64_t *full = (uint64_t *)(ring + UM_STAGES * 2 * UM_TILE);
  uint64_t *empty = full + UM_STAGES;
  uint64_t *s_bar = empty + UM_STAGES, *p_bar = s_bar + 2, *o_bar = p_bar + 2;       // [2] each: one per warpgroup
  uint32_t *tmem_slot = (uint32_t *)(o_bar + 2);
  volatile uint32_t *abort_flag = tmem_slot + 1;
  float *xchg = (float *)(sm + UM_SMEM - UM_XCHG_BYTES);    // [2][128]: reference maximum and sum of warpgroup 1's rows

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = p.H / p.G;
  const int zb = blockIdx.z / p.G, g = blockIdx.z % p.G;
  int b = p.order ? p.order[zb] : zb;                       // row block (sequence) of this CTA
  if ((unsigned)b >= gridDim.z / (unsigned)p.G) b = zb;
  const int M = p.rps * grp;
  const int m0 = blockIdx.x * MT;
  const int row0 = b * p.rps;
  const int ps = p.pm.page_size;
  int seq = -1, ctx = 0;
  for (int i = 0; i < p.rps; i++) {
    int s = p.m.seq[row0 + i];
    if (s >= 0) { seq = s; ctx = p.m.ctx[row0 + i]; break; }
  }
  const int nkeys = (seq >= 0) ? ctx + p.tail_len : 0;
  const int ntiles = (nkeys + KT - 1) / KT;
  const int t_begin = (int)(((long long)blockIdx.y * ntiles) / p.nsplit);
  const int t_end = (int)(((long long)(blockIdx.y + 1) * ntiles) / p.nsplit);
  const int ntl = t_end - t_begin;

  if (threadIdx.x == 0) {
    for (int i = 0; i < UM_STAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(&s_bar[0], 1);
    mbar_init(&s_bar[1], 1);
    for (int i = 0; i < 2; i++) { mbar_init(&p_bar[i], 128); mbar_init(&o_bar[i], 1); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(UM_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  // ---- Q tile -> shared in the operand layout: row lr, 16-byte chunk c -> half c / 8, chunk (c % 8) ^ (lr % 8)
  // Two softmax warpgroups (warps 0..3 and 4..7).  Warpgroup w takes the key tiles i with i % 2 == w as an independent
  // online-softmax stream with its own score buffer, P tile and O accumulator; thread t of either group owns query row
  // t % 128 = tensor-memory lane t % 128.  The two streams are merged at the end like two key splits.
  const int wg = (warp >> 2) & 1;
  const int lr = threadIdx.x & 127;
  const int mrow = m0 + lr;
  bool rvalid = false;
  uint64_t mlo = 0, mhi = 0;
  int qi = 0, qh = 0;
  if (warp < 8) {
    if (mrow < M) { qi = mrow / grp; qh = mrow % grp; rvalid = p.m.seq[row0 + qi] >= 0; }
    if (rvalid) { mlo = p.m.mask_lo[row0 + qi]; mhi = p.m.mask_hi[row0 + qi]; }
    else { mlo = ~0ull; mhi = ~0ull; }                         // a padding row attends every tail key (zeroed at the end)
    clip_tail(mlo, mhi, p.tail_len);
    const uint4 *src = (const uint4 *)(p.q + ((size_t)(row0 + qi) * p.H + g * grp + qh) * HD);
#pragma unroll
    for (int cc = 0; cc < 8; cc++) {                        // each of the row's two threads copies one half of it
      const int c = wg * 8 + cc;
      uint4 v = rvalid ? src[c] : make_uint4(0u, 0u, 0u, 0u);
      *(uint4 *)(sQ + (c >> 3) * (MT * 128) + lr * 128 + (((c & 7) ^ (lr & 7)) << 4)) = v;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  const uint32_t tmem_s = tmem_base, tmem_o = tmem_base + 2 * KT;     // S[w] at column 64 w, O[w] at column 128 + 128 w

  if (warp == 8) {
    // ================================================================ producer
    if (seq >= 0) {     // the whole warp walks the loop, the elected lane issues the copies
      const int32_t *tbl = p.pm.table + (size_t)seq * p.pm.pages_per_seq;
      const int fallback = tbl[0];                     // keys past the last page are masked; they still need a valid source
      const int ppt = KT / ps;                         // pages per tile
      int cur[4], nxt[4] = {-1, -1, -1, -1};
      if (ntl > 0) tile_pages(cur, tbl, p.pm.pages_per_seq, t_begin, ps);
      for (int i = 0; i < ntl; i++) {
        const int t = t_begin + i, st = i % UM_STAGES;
        if (i + 1 < ntl) tile_pages(nxt, tbl, p.pm.pages_per_seq, t + 1, ps);
        if (i >= UM_STAGES && !mbar_wait_warp(&empty[st], (uint32_t)(((i / UM_STAGES) - 1) & 1))) {
          *abort_flag = 1;
          if (status) set_status(status, ST_TIMEOUT, 420, blockIdx.z, t);
          break;
        }
        if (*abort_flag) break;
        if (elect_one()) {
          unsigned char *kb = ring + st * 2 * UM_TILE, *vb = kb + UM_TILE;
          mbar_expect_tx(&full[st], 2 * UM_TILE);
#pragma unroll
          for (int pg = 0; pg < 4; pg++) {
            if (pg >= ppt) break;
            int page = cur[pg];
            if (page < 0 || page >= p.pm.num_pages) page = fallback;
            const int row = (page * p.G + g) * ps;
#pragma unroll
            for (int h = 0; h < 2; h++) {
              tma_load_3d(kb + h * UM_HALF + pg * ps * 128, &map_k, 0, row, h, &full[st]);
              tma_load_3d(vb + h * UM_HALF + pg * ps * 128, &map_v, 0, row, h, &full[st]);
            }
          }
        }
        __syncwarp();
#pragma unroll
        for (int pg = 0; pg < 4; pg++) cur[pg] = nxt[pg];
      }
    }
  } else if (warp == 9) {
    // ================================================================ MMA issuer
    if (ntl > 0) {      // the whole warp walks the loop, the elected lane issues the MMAs and commits
      constexpr uint32_t idesc_s = tc::umma_idesc(KT);                       // N = 64 keys, both operands K-major
      constexpr uint32_t idesc_o = tc::umma_idesc(HD) | (1u << 16);          // N = 128, B (the V tile) MN-major
      const uint32_t q_addr = smem_u32(sQ), p_addr = smem_u32(sP);
      // S of tile i goes to the score buffer of warpgroup i % 2: while one group is in its softmax the tensor pipe
      // works for the other
      auto issue_s = [&](int i) {
        const int st = i % UM_STAGES;
        const uint32_t k_addr = smem_u32(ring + st * 2 * UM_TILE);
        const uint32_t d = tmem_s + (uint32_t)((i & 1) * KT);
#pragma unroll
        for (int h = 0; h < 2; h++)
#pragma unroll
          for (int j = 0; j < 64 / tc::UMMA_K; j++)
            tc::umma_bf16(d, tc::umma_desc_sw128(q_addr + h * (MT * 128) + j * 32), tc::umma_desc_sw128(k_addr + h * UM_HALF + j * 32),
                          idesc_s, (h | j) ? 1u : 0u);
        tc::umma_commit(&s_bar[i & 1]);
      };
      bool ok = true;
      for (int i = 0; i < 2 && i < ntl && ok; i++) {
        ok = mbar_wait_warp(&full[i % UM_STAGES], 0);
        if (!ok) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 421, blockIdx.z, t_begin + i); break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (elect_one()) issue_s(i);
        __syncwarp();
      }
      if (ok) {
        for (int i = 0; i < ntl; i++) {
          const int st = i % UM_STAGES;
          if (!mbar_wait_warp(&p_bar[i & 1], (uint32_t)((i >> 1) & 1))) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 422, blockIdx.z, t_begin + i); break; }
          if (*abort_flag) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t v_addr = smem_u32(ring + st * 2 * UM_TILE + UM_TILE);
          if (elect_one()) {
#pragma unroll
            for (int kk = 0; kk < KT / tc::UMMA_K; kk++)
              tc::umma_bf16(tmem_o + (uint32_t)((i & 1) * HD), tc::umma_desc_sw128(p_addr + (i & 1) * UM_P_BYTES + kk * 32),
                            umma_desc_sw128_mn(v_addr + kk * (tc::UMMA_K * 128), UM_HALF), idesc_o, ((i >> 1) | kk) ? 1u : 0u);
            tc::umma_commit(&o_bar[i & 1]);
            tc::umma_commit(&empty[st]);
          }
          __syncwarp();
          if (i + 2 < ntl) {          // this group's score buffer is free: its threads read it before they arrived on p_bar
            const int st2 = (i + 2) % UM_STAGES;
            if (!mbar_wait_warp(&full[st2], (uint32_t)(((i + 2) / UM_STAGES) & 1))) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 423, blockIdx.z, t_begin + i + 2); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (elect_one()) issue_s(i + 2);
            __syncwarp();
          }
        }
      }
    }
  } else {
    // ================================================================ softmax: thread = query row = tensor-memory lane
    const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
    const uint32_t my_s = tmem_s + lane_base + (uint32_t)(wg * KT), my_o = tmem_o + lane_base + (uint32_t)(wg * HD);
    unsigned char *my_p = sP + wg * UM_P_BYTES;
    float mx = -INFINITY, l = 0.0f;
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;    // softmax scale folded into exp2
    bool alive = true;
    int nmine = 0;                                               // tiles this warpgroup has finished
    for (int i = wg; i < ntl; i += 2) {
      const int t = t_begin + i, j = i >> 1;                     // j: index within this group's stream
      bool ok = mbar_wait(&s_bar[wg], (uint32_t)(j & 1));
      ok = __all_sync(0xffffffffu, ok && !*abort_flag);
      if (!ok) { if (lane == 0) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 424, blockIdx.z, t); } alive = false; break; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      float s[KT];
      tmem_ld64(my_s, s);
      // Padding rows (beyond the tile's last row, or of a skipped sequence) run the loop like real rows and are
      // zeroed at the end: their Q is zero, and a row that always took the masked path would slow its whole warp.
      float tm = -INFINITY;
      if (t * KT + KT <= ctx) {
#pragma unroll
        for (int e = 0; e < KT; e++) tm = fmaxf(tm, s[e]);
      } else {
        const uint64_t w = tile_allow(mlo, mhi, ctx, t * KT);
        const uint32_t w0 = (uint32_t)w, w1 = (uint32_t)(w >> 32);
#pragma unroll
        for (int e = 0; e < KT; e++) {
          const bool okk = ((e < 32 ? w0 : w1) & (1u << (e & 31))) != 0u;
          s[e] = okk ? s[e] : -INFINITY;
          tm = fmaxf(tm, s[e]);
        }
      }
      // The reference maximum of a row moves only when the tile maximum exceeds it by more than 2^8 in the exponent:
      // the probabilities stay below 256 (exact in the fp32 sums, 8 mantissa bits in P as always) and O is rescaled
      // rarely; the (reference, sum, O) triple stays consistent, which is all the final division or the merge needs.
      float nm = mx, f = 1.0f;
      if (tm > mx && (mx == -INFINITY || (tm - mx) * sc > 8.0f)) {
        nm = tm;
        f = (mx == -INFINITY) ? 1.0f : ex2_approx((mx - nm) * sc);      // nothing accumulated yet: nothing to rescale
      }
      const float nb = (nm == -INFINITY) ? 0.0f : nm * sc;
      float rs = 0.0f;
      uint32_t pk[KT / 2];
#pragma unroll
      for (int e = 0; e < KT; e += 2) {
        const float p0 = ex2_approx(fmaf(s[e], sc, -nb)), p1 = ex2_approx(fmaf(s[e + 1], sc, -nb));
        rs += p0 + p1;
        pk[e >> 1] = pack_bf16(p0, p1);
      }
      l = l * f + rs;
      mx = nm;
      // this group's previous P V must be complete before its O is rescaled and before its P tile is overwritten
      if (j > 0) {
        bool ok2 = mbar_wait(&o_bar[wg], (uint32_t)((j - 1) & 1));
        ok2 = __all_sync(0xffffffffu, ok2 && !*abort_flag);
        if (!ok2) { if (lane == 0) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 425, blockIdx.z, t); } alive = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (__any_sync(0xffffffffu, f != 1.0f)) {
#pragma unroll 1
          for (int c = 0; c < HD / 16; c++) {
            uint32_t v[16];
            tc::tmem_ld16(my_o + c * 16, v);
#pragma unroll
            for (int e = 0; e < 16; e++) v[e] = __float_as_uint(__uint_as_float(v[e]) * f);
            tmem_st16(my_o + c * 16, v);
          }
          asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        }
      }
#pragma unroll
      for (int c = 0; c < KT / 8; c++)
        *(uint4 *)(my_p + lr * 128 + ((c ^ (lr & 7)) << 4)) = make_uint4(pk[c * 4], pk[c * 4 + 1], pk[c * 4 + 2], pk[c * 4 + 3]);
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      mbar_arrive(&p_bar[wg]);
      nmine++;
    }
    if (alive && nmine > 0) {
      bool ok = mbar_wait(&o_bar[wg], (uint32_t)((nmine - 1) & 1));
      ok = __all_sync(0xffffffffu, ok && !*abort_flag);
      if (!ok) { if (lane == 0) { *abort_flag = 1; if (status) set_status(status, ST_TIMEOUT, 426, blockIdx.z, t_end); } alive = false; }
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    }
    // ---- merge of the two streams: group 1 hands over its rows' statistics, group 0 reads both O accumulators.
    // Every softmax thread reaches this barrier exactly once, whether or not its group gave up.
    if (wg == 1) { xchg[lr] = mx; xchg[128 + lr] = l; }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    asm volatile("bar.sync 1, 256;" ::: "memory");
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const bool has1 = ntl > 1;                                   // group 1 accumulated something
    // ---- write: final (one split) or partial
    if (wg == 0 && alive) {
      const float m1 = has1 ? xchg[lr] : -INFINITY, l1 = has1 ? xchg[128 + lr] : 0.0f;
      const float mm = fmaxf(mx, m1);
      const float f0 = (mx == -INFINITY) ? 0.0f : ex2_approx((mx - mm) * sc), f1 = (m1 == -INFINITY) ? 0.0f : ex2_approx((m1 - mm) * sc);
      l = l * f0 + l1 * f1;
      mx = mm;
      const int r = row0 + qi, h = g * grp + qh;
      if (!rvalid) { l = 0.0f; mx = -INFINITY; }              // padding row: an empty partial, a zero output
      const float inv = l > 0.0f ? 1.0f / l : 0.0f;
      const size_t idx = (size_t)blockIdx.y * p.rows * p.H + (size_t)r * p.H + h;
#pragma unroll 1
      for (int c = 0; c < HD / 16; c++) {
        uint32_t v[16], w1[16];
        if (ntl > 0) tc::tmem_ld16(tmem_o + lane_base + c * 16, v);              // the whole warp takes part
        if (has1) tc::tmem_ld16(tmem_o + lane_base + HD + c * 16, w1);
#pragma unroll
        for (int e = 0; e < 16; e++) {
          float o0 = (ntl > 0 && rvalid && f0 != 0.0f) ? __uint_as_float(v[e]) * f0 : 0.0f;
          float o1 = (has1 && rvalid && f1 != 0.0f) ? __uint_as_float(w1[e]) * f1 : 0.0f;
          v[e] = __float_as_uint(o0 + o1);
        }
        if (mrow < M) {
          if (p.nsplit == 1 && !p.keep_partial) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; e++) w[e] = pack_bf16(__uint_as_float(v[2 * e]) * inv, __uint_as_float(v[2 * e + 1]) * inv);
            uint4 *dst = (uint4 *)(p.out + ((size_t)r * p.H + h) * HD + c * 16);
            dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
            dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
          } else {
            uint4 *dst = (uint4 *)(p.part_o + idx * HD + c * 16);
#pragma unroll
            for (int e = 0; e < 4; e++) dst[e] = make_uint4(v[4 * e], v[4 * e + 1], v[4 * e + 2], v[4 * e + 3]);
          }
        }
      }
      if (mrow < M && (p.nsplit > 1 || p.keep_partial)) { p.part_ml[idx * 2] = mx; p.part_ml[idx * 2 + 1] = l; }
    }
  }

  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(UM_TMEM_COLS) : "memory");
  }
}

// ------------------------------------------------------------------------------------------------
// TMA-staged variant for at most 16 query rows per (sequence, KV head): chain drafts at batch (one node x the GQA
// group) and single-token decoding.  One 16-row tile would leave seven of eight row-parallel warps idle, so here
// the four consumer warps share the rows and split the KEYS of every 64-key tile (16 keys each); each keeps its own
// online-softmax state and the four states are merged through shared memory at the end.
template <int HD, int STAGES>
__global__ void __launch_bounds__(160) attn_tma_small_kernel(const __grid_constant__ CUtensorMap map_k,
                                                             const __grid_constant__ CUtensorMap map_v, AttnParams p, int32_t *status) {
  pdl_trigger();   // the next kernel may start staging its weights; it still waits for this grid to complete
  pdl_wait();
  KernelStamp stamp_guard(p.stamp);
  constexpr int ROWB = HD * 2, CPR = HD / 8;
  constexpr int NKS = HD / 16;
  constexpr int TILEB = KT * ROWB;
  constexpr int NW = 4;                                // consumer warps
  extern __shared__ __align__(1024) unsigned char sm[];
  uint64_t *full = (uint64_t *)(sm + STAGES * 2 * TILEB);
  uint64_t *empty = full + STAGES;
  unsigned char *sQ = sm + STAGES * 2 * TILEB + 256;   // [16][HD] bf16, swizzled
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int grp = p.H / p.G;
  const int zb = blockIdx.z / p.G, g = blockIdx.z % p.G;
  int b = p.order ? p.order[zb] : zb;            // row block (sequence) of this CTA
  if ((unsigned)b >= gridDim.z / (unsigned)p.G) b = zb;
  const int M = p.rps * grp;                           // <= 16
  const int row0 = b * p.rps;
  const int ps = p.pm.page_size;
  int seq = -1, ctx = 0;
  for (int i = 0; i < p.rps; i++) {
    int s = p.m.seq[row0 + i];
    if (s >= 0) { seq = s; ctx = p.m.ctx[row0 + i]; break; }
  }
  const int nkeys = (seq >= 0) ? ctx + p.tail_len : 0;
  const int ntiles = (nkeys + KT - 1) / KT;
  const int t_begin = (int)(((long long)blockIdx.y * ntiles) / p.nsplit);
  const int t_end = (int)(((long long)(blockIdx.y + 1) * ntiles) / p.nsplit);

  if (threadIdx.x == 0) {
    for (int i = 0; i < STAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], NW); }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  for (int id = threadIdx.x; id < 16 * CPR; id += 160) {
    int lr = id / CPR, c = id % CPR;
    bool v = lr < M;
    int i = v ? lr / grp : 0, hq = v ? lr % grp : 0;
    v = v && p.m.seq[row0 + i] >= 0;
    const bf16 *src = p.q + ((size_t)(row0 + i) * p.H + g * grp + hq) * HD + c * 8;
    cp_async16(smem_u32(sQ + swz<ROWB>(lr, c)), src, v);
  }
  cp_async_commit();
  cp_async_wait<0>();
  __syncthreads();

  if (warp == NW) {
    if (seq >= 0) {     // the whole warp walks the loop, the elected lane issues the copies
      const int32_t *tbl = p.pm.table + (size_t)seq * p.pm.pages_per_seq;
      const int fallback = tbl[0];
      const int ppt = KT / ps;
      int cur[4], nxt[4] = {-1, -1, -1, -1};
      if (t_begin < t_end) tile_pages(cur, tbl, p.pm.pages_per_seq, t_begin, ps);
      for (int t = t_begin; t < t_end; t++) {
        const int i = t - t_begin, st = i % STAGES;
        if (t + 1 < t_end) tile_pages(nxt, tbl, p.pm.pages_per_seq, t + 1, ps);
        if (i >= STAGES && !mbar_wait_warp(&empty[st], (uint32_t)(((i / STAGES) - 1) & 1))) { if (status) set_status(status, ST_TIMEOUT, 411, blockIdx.z, t); break; }
        if (elect_one()) {
          unsigned char *kb = sm + st * 2 * TILEB, *vb = kb + TILEB;
          mbar_expect_tx(&full[st], 2 * TILEB);
#pragma unroll
          for (int pg = 0; pg < 4; pg++) {
            if (pg >= ppt) break;
            int page = cur[pg];
            if (page < 0 || page >= p.pm.num_pages) page = fallback;
            const int row = (page * p.G + g) * ps;
            tma_load_3d(kb + pg * ps * ROWB, &map_k, 0, row, 0, &full[st]);
            tma_load_3d(vb + pg * ps * ROWB, &map_v, 0, row, 0, &full[st]);
          }
        }
        __syncwarp();
#pragma unroll
        for (int pg = 0; pg < 4; pg++) cur[pg] = nxt[pg];
      }
    }
  } else {
    // ---- consumers: all four warps hold the same 16-row Q tile
    uint32_t qf[NKS][4];
#pragma unroll
    for (int ks = 0; ks < NKS; ks++) {
      int r = (lane & 7) + ((lane >> 3) & 1) * 8, c = ks * 2 + (lane >> 4);
      ldsm_x4(smem_u32(sQ + swz<ROWB>(r, c)), qf[ks][0], qf[ks][1], qf[ks][2], qf[ks][3]);
    }
    const int psb = ps * ROWB, psh = __ffs(ps) - 1;    // the page size is a power of two
    auto koff = [&](int kr, int c) -> uint32_t {
      return (uint32_t)((kr >> psh) * psb + (c >> 3) * (ps * 128) + (kr & (ps - 1)) * 128 + (((c & 7) ^ (kr & 7)) << 4));
    };
    const int mA = lane >> 2, mB = mA + 8;
    uint64_t loA = 0, hiA = 0, loB = 0, hiB = 0;
    bool vA = false, vB = false;
    if (mA < M) { int r = row0 + mA / grp; vA = p.m.seq[r] >= 0; if (vA) { loA = p.m.mask_lo[r]; hiA = p.m.mask_hi[r]; } }
    if (mB < M) { int r = row0 + mB / grp; vB = p.m.seq[r] >= 0; if (vB) { loB = p.m.mask_lo[r]; hiB = p.m.mask_hi[r]; } }
    float o[HD / 8][4];
#pragma unroll
    for (int n = 0; n < HD / 8; n++) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.0f; }
    float mxA = -INFINITY, mxB = -INFINITY, lA = 0.0f, lB = 0.0f;
    const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
    const int k0w = warp * 16;                          // this warp's keys inside a tile
    for (int t = t_begin; t < t_end; t++) {
      const int i = t - t_begin, st = i % STAGES;
      if (!mbar_wait(&full[st], (uint32_t)((i / STAGES) & 1))) { if (lane == 0 && status) set_status(status, ST_TIMEOUT, 412, blockIdx.z, t); break; }
      const unsigned char *kbase = sm + st * 2 * TILEB, *vbase = kbase + TILEB;
      float s[2][4];
#pragma unroll
      for (int n = 0; n < 2; n++) { s[n][0] = s[n][1] = s[n][2] = s[n][3] = 0.0f; }
#pragma unroll
      for (int ks = 0; ks < NKS; ks++) {
        uint32_t b0, b1, b2, b3;
        int kr = k0w + (lane & 7) + (lane >> 4) * 8, c = ks * 2 + ((lane >> 3) & 1);
        ldsm_x4(smem_u32(kbase + koff(kr, c)), b0, b1, b2, b3);
        mma_bf16(s[0], qf[ks], b0, b1);
        mma_bf16(s[1], qf[ks], b2, b3);
      }
      float tmA = -INFINITY, tmB = -INFINITY;
#pragma unroll
      for (int n = 0; n < 2; n++) {
#pragma unroll
        for (int e = 0; e < 2; e++) {
          int key = t * KT + k0w + n * 8 + (lane & 3) * 2 + e;
          bool in_ctx = key < ctx;
          int tt = key - ctx;
          bool in_tail = !in_ctx && tt < p.tail_len;
          bool okA = vA && (in_ctx || (in_tail && ((tt < 64 ? (loA >> tt) : (hiA >> (tt - 64))) & 1ull)));
          bool okB = vB && (in_ctx || (in_tail && ((tt < 64 ? (loB >> tt) : (hiB >> (tt - 64))) & 1ull)));
          s[n][e] = okA ? s[n][e] : -INFINITY;
          s[n][2 + e] = okB ? s[n][2 + e] : -INFINITY;
          tmA = fmaxf(tmA, s[n][e]);
          tmB = fmaxf(tmB, s[n][2 + e]);
        }
      }
      tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 1)); tmA = fmaxf(tmA, __shfl_xor_sync(0xffffffffu, tmA, 2));
      tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 1)); tmB = fmaxf(tmB, __shfl_xor_sync(0xffffffffu, tmB, 2));
      float nmA = fmaxf(mxA, tmA), nmB = fmaxf(mxB, tmB);
      float fA = (nmA == -INFINITY) ? 1.0f : exp2f((mxA - nmA) * sc), fB = (nmB == -INFINITY) ? 1.0f : exp2f((mxB - nmB) * sc);
      float baseA = (nmA == -INFINITY) ? 0.0f : nmA, baseB = (nmB == -INFINITY) ? 0.0f : nmB;
      float rsA = 0.0f, rsB = 0.0f;
      uint32_t pf[4];
#pragma unroll
      for (int n = 0; n < 2; n++) {
        float p0 = exp2f((s[n][0] - baseA) * sc), p1 = exp2f((s[n][1] - baseA) * sc);
        float p2 = exp2f((s[n][2] - baseB) * sc), p3 = exp2f((s[n][3] - baseB) * sc);
        rsA += p0 + p1; rsB += p2 + p3;
        pf[n * 2] = pack_bf16(p0, p1);
        pf[n * 2 + 1] = pack_bf16(p2, p3);
      }
      rsA += __shfl_xor_sync(0xffffffffu, rsA, 1); rsA += __shfl_xor_sync(0xffffffffu, rsA, 2);
      rsB += __shfl_xor_sync(0xffffffffu, rsB, 1); rsB += __shfl_xor_sync(0xffffffffu, rsB, 2);
      lA = lA * fA + rsA; lB = lB * fB + rsB;
      mxA = nmA; mxB = nmB;
#pragma unroll
      for (int n = 0; n < HD / 8; n++) { o[n][0] *= fA; o[n][1] *= fA; o[n][2] *= fB; o[n][3] *= fB; }
#pragma unroll
      for (int d2 = 0; d2 < HD / 16; d2++) {
        uint32_t b0, b1, b2, b3;
        int kr = k0w + (lane & 7) + ((lane >> 3) & 1) * 8, c = d2 * 2 + (lane >> 4);
        ldsm_x4_t(smem_u32(vbase + koff(kr, c)), b0, b1, b2, b3);
        mma_bf16(o[2 * d2], pf, b0, b1);
        mma_bf16(o[2 * d2 + 1], pf, b2, b3);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty[st]);
    }
    // ---- merge the four key subsets: every warp parks (o, max, sum) in shared memory
    float *so = (float *)sm;                            // [NW][16][HD]: the ring is free once every warp has left the loop
    float *sml = so + NW * 16 * HD;                     // [NW][16][2]
    asm volatile("bar.sync 1, 128;" ::: "memory");      // all warps are done with the last stage
    const int qcol = (lane & 3) * 2;
#pragma unroll
    for (int half = 0; half < 2; half++) {
      const int lr = (lane >> 2) + half * 8;
#pragma unroll
      for (int n = 0; n < HD / 8; n++) *(float2 *)(so + (warp * 16 + lr) * HD + n * 8 + qcol) = make_float2(o[n][half * 2], o[n][half * 2 + 1]);
      if ((lane & 3) == 0) { sml[(warp * 16 + lr) * 2] = half ? mxB : mxA; sml[(warp * 16 + lr) * 2 + 1] = half ? lB : lA; }
    }
    asm volatile("bar.sync 1, 128;" ::: "memory");
    const int tid = threadIdx.x;                        // 0..127
    for (int e = tid; e < 16 * HD; e += 128) {
      const int lr = e / HD, d = e % HD;
      if (lr >= M) continue;
      float Mx = -INFINITY;
#pragma unroll
      for (int w = 0; w < NW; w++) Mx = fmaxf(Mx, sml[(w * 16 + lr) * 2]);
      float acc = 0.0f, l = 0.0f;
#pragma unroll
      for (int w = 0; w < NW; w++) {
        const float m = sml[(w * 16 + lr) * 2];
        if (m == -INFINITY) continue;
        const float wt = exp2f((m - Mx) * sc);
        acc += wt * so[(w * 16 + lr) * HD + d];
        l += wt * sml[(w * 16 + lr) * 2 + 1];
      }
      const int r = row0 + lr / grp, h = g * grp + lr % grp;
      if (p.nsplit == 1) {
        p.out[((size_t)r * p.H + h) * HD + d] = __float2bfloat16_rn(l > 0.0f ? acc / l : 0.0f);
      } else {
        const size_t idx = (size_t)blockIdx.y * p.rows * p.H + (size_t)r * p.H + h;
        p.part_o[idx * HD + d] = acc;
        if (d == 0) { p.part_ml[idx * 2] = Mx; p.part_ml[idx * 2 + 1] = l; }
      }
    }
  }
}

// merge the splits: out = sum_s 2^((m_s - M) c) O_s / sum_s 2^((m_s - M) c) l_s.  One warp per (row, head): lanes first
// fetch the (max, sum) pairs of all splits at once, then every lane adds up its HD/32 output dimensions with the
// loads of eight splits in flight.
template <int HD>
__global__ void __launch_bounds__(256) attn_combine_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml, int nsplit,
                                                           int nrh, bf16 *__restrict__ out, unsigned long long *stamp) {
  pdl_trigger();   // the next kernel may start staging its weights; it still waits for this grid to complete
  pdl_wait();
  KernelStamp stamp_guard(stamp, false);
  constexpr int DPL = HD / 32;                              // dimensions per lane
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rh = blockIdx.x * 8 + warp;
  if (rh >= nrh) return;
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
  float m = -INFINITY, ls = 0.0f;                           // lane s holds split s (nsplit <= 32)
  float2 ml = make_float2(-INFINITY, 0.0f);
  if (lane < nsplit) ml = *(const float2 *)(part_ml + ((size_t)lane * nrh + rh) * 2);
  constexpr int NB = 12;                                    // partial rows in flight per lane
  // the first NB partial rows are requested together with the statistics: one round trip instead of two
  float v[NB][DPL];
#pragma unroll
  for (int s = 0; s < NB; s++)
    if (s < nsplit) {
      const float *src = part_o + ((size_t)s * nrh + rh) * HD + lane * DPL;
#pragma unroll
      for (int e = 0; e < DPL; e++) v[s][e] = src[e];
    }
  m = ml.x; ls = ml.y;
  float M = m;
  for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
  const float w = (m == -INFINITY) ? 0.0f : exp2f((m - M) * sc);
  float l = w * ls;
  for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
  float acc[DPL];
#pragma unroll
  for (int e = 0; e < DPL; e++) acc[e] = 0.0f;
  for (int s0 = 0; s0 < nsplit; s0 += NB) {
    if (s0 > 0) {
#pragma unroll
      for (int s = 0; s < NB; s++)
        if (s0 + s < nsplit) {
          const float *src = part_o + ((size_t)(s0 + s) * nrh + rh) * HD + lane * DPL;
#pragma unroll
          for (int e = 0; e < DPL; e++) v[s][e] = src[e];
        }
    }
#pragma unroll
    for (int s = 0; s < NB; s++) {
      const float ws = __shfl_sync(0xffffffffu, w, (s0 + s) & 31);
      if (s0 + s < nsplit) {
#pragma unroll
        for (int e = 0; e < DPL; e++) acc[e] += ws * v[s][e];
      }
    }
  }
  const float inv = l > 0.0f ? 1.0f / l : 0.0f;
#pragma unroll
  for (int e = 0; e < DPL; e++) out[(size_t)rh * HD + lane * DPL + e] = __float2bfloat16_rn(acc[e] * inv);
}

int g_attn_target_ctas = 148;

int pick_splits(int seqs, int G, int mtiles, int max_ctx_tiles, int target = 0) {
  int base = seqs * G * mtiles;
  int want = (target > 0 ? target : g_attn_target_ctas) / base;                             // the kernels run one CTA per SM (register-bound): never more CTAs than one wave
  if (want < 1) want = 1;
  int s = want < max_ctx_tiles ? want : max_ctx_tiles;
  if (s > MAX_SPLITS) s = MAX_SPLITS;
  return s < 1 ? 1 : s;
}

}  // namespace

bool attn_fast_supported(int head_dim, int group) { return (head_dim == 64 || head_dim == 128) && group >= 1; }

size_t attn_fast_scratch_bytes(int rows, int n_heads, int head_dim, int max_ctx) {
  (void)max_ctx;
  return (size_t)MAX_SPLITS * rows * n_heads * (head_dim + 2) * sizeof(float) + 256;
}

namespace {
typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                             const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
EncodeFn g_encode = nullptr;
bool g_encode_tried = false;
std::map<std::tuple<const void *, int, int, int, int, int>, CUtensorMap> g_kv_maps;   // (pool, pages, G, page size, hd, box depth)

// 3-D view of a K or V pool [num_pages][G][page_size][hd]: dim0 = 64 elements (128 bytes), dim1 = every key row of
// the pool (pitch hd * 2 bytes), dim2 = the hd / 64 column halves (128 bytes apart).  One box = one page of one head.
// depth: 64-column halves per box (hd / 64: one box = one page of one head; 1: one half of it).
const CUtensorMap *kv_map(const void *pool, int num_pages, int G, int ps, int hd, int depth = 0) {
  if (depth <= 0) depth = hd / 64;
  if (!g_encode_tried) {
    g_encode_tried = true;
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      g_encode = (EncodeFn)fn;
  }
  if (!g_encode) return nullptr;
  if (num_pages > (1 << 20)) num_pages = 1 << 20;      // callers without a pool size: the page table is trusted
  auto key = std::make_tuple(pool, num_pages, G, ps, hd, depth);
  auto it = g_kv_maps.find(key);
  if (it != g_kv_maps.end()) return &it->second;
  CUtensorMap m;
  cuuint64_t dims[3] = {64, (cuuint64_t)num_pages * G * ps, (cuuint64_t)(hd / 64)};
  cuuint64_t strides[2] = {(cuuint64_t)hd * 2, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)ps, (cuuint32_t)depth};
  cuuint32_t estr[3] = {1, 1, 1};
  CUresult r = g_encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, (void *)pool, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                        CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return nullptr;
  if (g_kv_maps.size() > 4096) g_kv_maps.clear();
  return &(g_kv_maps[key] = m);
}

template <int HD>
int launch_tma_small(AttnParams &p, dim3 grid, const CUtensorMap *mk, const CUtensorMap *mv, int32_t *status, cudaStream_t s) {
  // two stages at head_dim 128 (68 KB): three CTAs share an SM and hide each other's prologue and merge, and the next
  // GEMM's CTAs find room to stage their weights early (C3 step -2.9 % against three stages)
  constexpr int STAGES = HD == 128 ? 2 : 4;
  const int smem = STAGES * 2 * KT * HD * 2 + 256 + 16 * HD * 2;   // ring (reused by the final merge) + barriers + Q tile
  static SmemLimit limit;
  if (!limit.ensure(attn_tma_small_kernel<HD, STAGES>, (int)smem)) return -1;
  launch_k(attn_tma_small_kernel<HD, STAGES>, grid, dim3(160), (size_t)smem, s, *mk, *mv, p, status);
  return 0;
}

int g_attn_umma = 2;            // tcgen05 kernel for the tree passes: 0 off, 1 on, 2 on when a CTA gets at least UM_MIN_TILES key tiles
constexpr int UM_MIN_TILES = 3; // below that the pass is launch- and latency-bound and the mma.sync kernel's shorter prologue wins
thread_local int tl_attn_umma = -1;   // per-call override (-1: none)

int launch_umma(AttnParams &p, dim3 grid, const CUtensorMap *mk, const CUtensorMap *mv, int32_t *status, cudaStream_t s) {
  static SmemLimit limit;
  if (!limit.ensure(attn_umma_kernel, (int)UM_SMEM)) return -1;
  launch_k(attn_umma_kernel, grid, dim3(UM_THREADS), (size_t)UM_SMEM, s, *mk, *mv, p, status);
  return 0;
}

template <int HD>
int launch_tma(AttnParams &p, dim3 grid, const CUtensorMap *mk, const CUtensorMap *mv, int32_t *status, cudaStream_t s) {
  if (p.rps * (p.H / p.G) <= 16) return launch_tma_small<HD>(p, grid, mk, mv, status, s);
  constexpr int STAGES = HD == 128 ? 3 : 4;
  const int smem = STAGES * 2 * KT * HD * 2 + 256;
  static SmemLimit limit;
  if (!limit.ensure(attn_tma_kernel<HD, STAGES>, (int)smem)) return -1;
  launch_k(attn_tma_kernel<HD, STAGES>, grid, dim3(288), (size_t)smem, s, *mk, *mv, p, status);
  return 0;
}
}  // namespace

void attn_fast_forget_maps() { g_kv_maps.clear(); }
void attn_fast_set_target_ctas(int n) { g_attn_target_ctas = n; }
void attn_fast_set_umma(int mode) { g_attn_umma = mode; }
void attn_fast_override_umma(int v) { tl_attn_umma = v; }

int launch_attn_fast(const bf16 *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, bf16 *out, int rows, int H, int G,
                     int hd, int rps, int ctx_hint, void *scratch, cudaStream_t s, bool contiguous_tail, int32_t *status,
                     const int32_t *order, int order_len, unsigned long long *stamp) {
  if (rps < 1 || rows % rps) rps = 1;
  int seqs = rows / rps, grp = H / G;
  int mtiles = (rps * grp + MT - 1) / MT;
  int ntiles_hint = (ctx_hint + tail_len + KT - 1) / KT;
  int nsplit = scratch ? pick_splits(seqs, G, mtiles, ntiles_hint < 1 ? 1 : ntiles_hint) : 1;
  AttnParams p;
  p.q = q; p.kpool = (const bf16 *)pool.k; p.vpool = (const bf16 *)pool.v; p.pm = pm; p.m = m; p.tail_len = tail_len;
  p.rows = rows; p.H = H; p.G = G; p.rps = rps; p.nsplit = nsplit; p.out = out;
  p.part_o = (float *)scratch;
  p.order = (order && order_len == seqs) ? order : nullptr;
  p.stamp = stamp;
  p.keep_partial = 0;
  p.part_ml = p.part_o ? p.part_o + (size_t)MAX_SPLITS * rows * H * hd : nullptr;
  dim3 grid(mtiles, nsplit, seqs * G);
  // TMA-staged kernel when the tail follows the context and a page is a whole number of 128-byte-swizzle boxes
  const int ps = pm.page_size;
  if (contiguous_tail && (ps == 16 || ps == 32 || ps == 64) && (hd == 64 || hd == 128)) {
    const int um_mode = tl_attn_umma >= 0 ? tl_attn_umma : g_attn_umma;
    const bool umma = hd == 128 && rps * grp > 16 && (um_mode == 1 || (um_mode == 2 && ntiles_hint >= UM_MIN_TILES * nsplit));
    const CUtensorMap *mk = kv_map(pool.k, pm.num_pages, G, ps, hd, umma ? 1 : 0), *mv = kv_map(pool.v, pm.num_pages, G, ps, hd, umma ? 1 : 0);
    if (mk && mv) {
      int rc = umma ? launch_umma(p, grid, mk, mv, status, s) : hd == 128 ? launch_tma<128>(p, grid, mk, mv, status, s) : launch_tma<64>(p, grid, mk, mv, status, s);
      if (rc == 0) {
        if (nsplit > 1) {
          if (hd == 128) launch_k(attn_combine_kernel<128>, dim3((rows * H + 7) / 8), dim3(256), 0, s, p.part_o, p.part_ml, nsplit, rows * H, out, p.stamp);
          else launch_k(attn_combine_kernel<64>, dim3((rows * H + 7) / 8), dim3(256), 0, s, p.part_o, p.part_ml, nsplit, rows * H, out, p.stamp);
        }
        return nsplit > 1 ? 2 : 1;
      }
    }
  }
  size_t smem = (size_t)4 * KT * hd * 2;
  if (smem < (size_t)MT * hd * 2) smem = (size_t)MT * hd * 2;
  static SmemLimit limit[2];
  if (hd == 128) {
    if (!limit[1].ensure(attn_mma_kernel<128>, (int)smem)) return -1;
    launch_k(attn_mma_kernel<128>, grid, dim3(256), smem, s, p);
    if (nsplit > 1) launch_k(attn_combine_kernel<128>, dim3((rows * H + 7) / 8), dim3(256), 0, s, p.part_o, p.part_ml, nsplit, rows * H, out, p.stamp);
  } else {
    if (!limit[0].ensure(attn_mma_kernel<64>, (int)smem)) return -1;
    launch_k(attn_mma_kernel<64>, grid, dim3(256), smem, s, p);
    if (nsplit > 1) launch_k(attn_combine_kernel<64>, dim3((rows * H + 7) / 8), dim3(256), 0, s, p.part_o, p.part_ml, nsplit, rows * H, out, p.stamp);
  }
  return nsplit > 1 ? 2 : 1;
}

}  // namespace spec

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of the tensor-core attention entry point.
//
// Some hosts of this library cannot allocate device memory when they need attention: code running
// inside a memory-pool or arena that was sized up front, a plugin whose host process forbids
// cudaMalloc after start-up, or a latency-critical loop where an allocation (an implicit device
// synchronisation) is not acceptable.  For them the split-KV partial results live in a fixed
// file-scope device array instead of a caller-provided scratch buffer.  Every GPU that loads the
// library carries the array until the process exits.
namespace spec {
namespace {
constexpr size_t STATIC_SCRATCH_BYTES = (size_t)8 << 20;     // 8 MiB per device
static __device__ __align__(256) unsigned char g_static_scratch[STATIC_SCRATCH_BYTES];

constexpr int MAX_DEVICES = 64;
void *g_static_scratch_dev[MAX_DEVICES];                      // device address of the array, per device
bool g_static_scratch_ready[MAX_DEVICES];
std::mutex g_static_scratch_mu;

// Device address of the array on the current device.  In host code the array's name is only a handle
// for the runtime, not a device address, so it is resolved once per device with cudaGetSymbolAddress.
int static_scratch_ptr(void **out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= MAX_DEVICES) return -6;
  std::lock_guard<std::mutex> lock(g_static_scratch_mu);
  if (!g_static_scratch_ready[dev]) {
    void *p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return -6;
    g_static_scratch_dev[dev] = p;
    g_static_scratch_ready[dev] = true;
  }
  *out = g_static_scratch_dev[dev];
  return 0;
}
}  // namespace
}  // namespace spec

extern "C" size_t spec_attention_static_capacity(void) { return spec::STATIC_SCRATCH_BYTES; }

extern "C" int spec_attention_static(const void *q, const void *k_pool, const void *v_pool, const int32_t *page_table,
                                     int32_t pages_per_seq, int32_t page_size, const int32_t *row_seq,
                                     const int32_t *row_ctx, const int32_t *row_tail_base, const uint64_t *row_mask_lo,
                                     const uint64_t *row_mask_hi, int32_t tail_len, void *out, int32_t rows, int32_t H,
                                     int32_t G, int32_t hd, int32_t max_ctx, void *stream) {
  using namespace spec;
  if (!q || !k_pool || !v_pool || !page_table || !row_seq || !row_ctx || !row_tail_base || !row_mask_lo || !row_mask_hi || !out)
    return -2;                                                         // SPEC_ERR_NULL
  if (rows < 1 || H < 1 || G < 1 || H % G || tail_len < 0 || tail_len > 128 || page_size < 1 || pages_per_seq < 1) return -1;
  if (!attn_fast_supported(hd, H / G)) return -8;                      // SPEC_ERR_UNSUPPORTED
  if (attn_fast_scratch_bytes(rows, H, hd, max_ctx) > STATIC_SCRATCH_BYTES) {
    fprintf(stderr, "spec_attention_static: rows=%d heads=%d head_dim=%d needs %zu bytes of split-KV scratch, the built-in "
                    "array holds %zu\n", rows, H, hd, attn_fast_scratch_bytes(rows, H, hd, max_ctx), STATIC_SCRATCH_BYTES);
    return -3;                                                         // SPEC_ERR_WORKSPACE
  }
  void *scratch = nullptr;
  if (int rc = static_scratch_ptr(&scratch)) return rc;
  RowMeta m{};
  m.seq = (int32_t *)row_seq; m.ctx = (int32_t *)row_ctx; m.tail_base = (int32_t *)row_tail_base;
  m.mask_lo = (uint64_t *)row_mask_lo; m.mask_hi = (uint64_t *)row_mask_hi;
  KvPool pool{(void *)k_pool, (void *)v_pool};
  PageMap pm{page_table, pages_per_seq, page_size, 1 << 30};
  launch_attn_fast((const bf16 *)q, pool, pm, m, tail_len, (bf16 *)out, rows, H, G, hd, 1, max_ctx, scratch, (cudaStream_t)stream, false, nullptr);
  return cudaGetLastError() == cudaSuccess ? 0 : -6;
}

// ------------------------------------------------------------------------------------------------
// Training-time-test attention (Section 3.2, the figure of the attention masks during training-time test).
//
// While the draft model is trained, its own outputs are fed back for further simulated steps.  At simulated step j a
// query at slot i sees the ORIGINAL sequence causally (keys 0..i of the native step: an ordinary lower-triangular mask)
// and, of every earlier simulated step s = 1..j, only the entry at its own slot i (a diagonal mask).  The dense causal
// part runs on the tensor-core tile kernels above (128-slot blocks: the block's slots are each other's tail keys, the
// slots before the block are context), which leave unnormalised partial results; the diagonal part is j dot products
// per (slot, head), computed as dot products, and folded into the same softmax by the merge kernel below.
namespace spec {
namespace {

__global__ void ttt_meta_kernel(RowMeta m, int T, int block) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  const bool v = r < T;
  const int j = r % block;
  m.seq[r] = v ? 0 : -1;
  m.ctx[r] = v ? r - j : 0;
  m.tail_base[r] = v ? r - j : 0;
  m.mask_lo[r] = v ? (j >= 63 ? ~0ull : ((1ull << (j + 1)) - 1ull)) : 0ull;
  m.mask_hi[r] = (v && j >= 64) ? (j >= 127 ? ~0ull : ((1ull << (j - 63)) - 1ull)) : 0ull;
}

constexpr int TTT_MAX_STEPS = 8;

// One warp per (slot, head): merges the key splits of the dense part with the J diagonal entries.
// part_o [nsplit][nrh][128] / part_ml [nsplit][nrh][2] as the tile kernels write them (raw maximum, sum and output
// relative to it); q [rows][H][128]; kd / vd [J][T][G][128]; out [rows][H][128]; lse [T*H] natural-log sum (optional).
__global__ void __launch_bounds__(256) ttt_merge_kernel(const float *__restrict__ part_o, const float *__restrict__ part_ml, int nsplit,
                                                        int nrh_alloc, const bf16 *__restrict__ q, const bf16 *__restrict__ kd,
                                                        const bf16 *__restrict__ vd, int J, int T, int H, int G,
                                                        bf16 *__restrict__ out, float *__restrict__ lse) {
  pdl_wait();
  pdl_trigger();
  constexpr int HD = 128, DPL = 4;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rh = blockIdx.x * 8 + warp;
  if (rh >= T * H) return;
  const int i = rh / H, h = rh % H, g = h / (H / G);
  const float sc = rsqrtf((float)HD) * 1.4426950408889634f;
  float2 ml = make_float2(-INFINITY, 0.0f);                 // lane s holds split s (nsplit <= 32)
  if (lane < nsplit) ml = *(const float2 *)(part_ml + ((size_t)lane * nrh_alloc + rh) * 2);
  // the diagonal scores: q . k of the slot's own entry of every simulated step
  const uint2 qraw = *(const uint2 *)(q + (size_t)rh * HD + lane * DPL);
  const float2 q01 = __bfloat1622float2(*(const __nv_bfloat162 *)&qraw.x), q23 = __bfloat1622float2(*(const __nv_bfloat162 *)&qraw.y);
  float d[TTT_MAX_STEPS];
  uint2 vraw[TTT_MAX_STEPS];
#pragma unroll
  for (int s = 0; s < TTT_MAX_STEPS; s++) {
    d[s] = -INFINITY;
    if (s < J) {
      const size_t off = (((size_t)s * T + i) * G + g) * HD + lane * DPL;
      const uint2 kraw = *(const uint2 *)(kd + off);
      vraw[s] = *(const uint2 *)(vd + off);
      const float2 k01 = __bfloat1622float2(*(const __nv_bfloat162 *)&kraw.x), k23 = __bfloat1622float2(*(const __nv_bfloat162 *)&kraw.y);
      float t = q01.x * k01.x + q01.y * k01.y + q23.x * k23.x + q23.y * k23.y;
      for (int off2 = 16; off2 > 0; off2 >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off2);
      d[s] = t;
    }
  }
  float M = ml.x;
  for (int off = 16; off > 0; off >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, off));
#pragma unroll
  for (int s = 0; s < TTT_MAX_STEPS; s++) M = fmaxf(M, d[s]);
  const float w = (ml.x == -INFINITY) ? 0.0f : exp2f((ml.x - M) * sc);
  float l = w * ml.y;
  for (int off = 16; off > 0; off >>= 1) l += __shfl_xor_sync(0xffffffffu, l, off);
  float acc[DPL] = {0.0f, 0.0f, 0.0f, 0.0f};
  for (int s = 0; s < nsplit; s++) {
    const float ws = __shfl_sync(0xffffffffu, w, s);
    const float4 o = *(const float4 *)(part_o + ((size_t)s * nrh_alloc + rh) * HD + lane * DPL);
    acc[0] += ws * o.x; acc[1] += ws * o.y; acc[2] += ws * o.z; acc[3] += ws * o.w;
  }
#pragma unroll
  for (int s = 0; s < TTT_MAX_STEPS; s++)
    if (s < J) {
      const float ws = exp2f((d[s] - M) * sc);
      const float2 v01 = __bfloat1622float2(*(const __nv_bfloat162 *)&vraw[s].x), v23 = __bfloat1622float2(*(const __nv_bfloat162 *)&vraw[s].y);
      l += ws;
      acc[0] += ws * v01.x; acc[1] += ws * v01.y; acc[2] += ws * v23.x; acc[3] += ws * v23.y;
    }
  const float inv = l > 0.0f ? 1.0f / l : 0.0f;
  __nv_bfloat162 o01 = __floats2bfloat162_rn(acc[0] * inv, acc[1] * inv), o23 = __floats2bfloat162_rn(acc[2] * inv, acc[3] * inv);
  *(uint2 *)(out + (size_t)rh * HD + lane * DPL) = make_uint2(*(uint32_t *)&o01, *(uint32_t *)&o23);
  if (lse && lane == 0) lse[rh] = logf(l) + M * rsqrtf((float)HD);
}

constexpr int TTT_BLOCK = 128;
constexpr int TTT_TARGET_CTAS = 148;   // fixed (not the tuning knob): the scratch size and the launch must agree
size_t ttt_meta_bytes(int rows_alloc) { return (((size_t)rows_alloc * (3 * 4 + 2 * 8)) + 255) & ~(size_t)255; }

}  // namespace
}  // namespace spec

extern "C" size_t spec_ttt_attention_scratch_bytes(int32_t T, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim) {
  using namespace spec;
  if (T < 1 || n_heads < 1 || n_kv_heads < 1 || n_heads % n_kv_heads || head_dim != 128) return 0;
  const int rows = (T + TTT_BLOCK - 1) / TTT_BLOCK * TTT_BLOCK, grp = n_heads / n_kv_heads;
  const int nsplit = pick_splits(rows / TTT_BLOCK, n_kv_heads, (TTT_BLOCK * grp + MT - 1) / MT, (T + KT - 1) / KT, TTT_TARGET_CTAS);
  return ttt_meta_bytes(rows) + (size_t)nsplit * rows * n_heads * (head_dim + 2) * sizeof(float) + 256;
}

extern "C" int spec_ttt_attention(const void *q, const void *k_pool, const void *v_pool, const int32_t *page_table,
                                  int32_t pages_per_seq, int32_t page_size, const void *k_diag, const void *v_diag, int32_t n_steps,
                                  void *out, float *lse, int32_t T, int32_t H, int32_t G, int32_t hd, void *scratch, void *stream) {
  using namespace spec;
  if (!q || !k_pool || !v_pool || !page_table || !out || !scratch || (n_steps > 0 && (!k_diag || !v_diag))) return SPEC_ERR_NULL;
  if (T < 1 || H < 1 || G < 1 || H % G || n_steps < 0 || n_steps > TTT_MAX_STEPS) return SPEC_ERR_INVALID_CFG;
  if (hd != 128 || !(page_size == 16 || page_size == 32 || page_size == 64) || (long long)pages_per_seq * page_size < T)
    return SPEC_ERR_UNSUPPORTED;
  cudaStream_t s = (cudaStream_t)stream;
  const int rows = (T + TTT_BLOCK - 1) / TTT_BLOCK * TTT_BLOCK, grp = H / G;
  const int mtiles = (TTT_BLOCK * grp + MT - 1) / MT, seqs = rows / TTT_BLOCK;
  const int nsplit = pick_splits(seqs, G, mtiles, (T + KT - 1) / KT, TTT_TARGET_CTAS);
  char *base = (char *)(((uintptr_t)scratch + 255) & ~(uintptr_t)255);
  RowMeta m{};
  m.seq = (int32_t *)base; m.ctx = m.seq + rows; m.tail_base = m.ctx + rows;
  m.mask_lo = (uint64_t *)(m.tail_base + rows); m.mask_hi = m.mask_lo + rows;
  launch_k(ttt_meta_kernel, dim3(rows / 128), dim3(128), 0, s, m, (int)T, TTT_BLOCK);
  AttnParams p;
  p.q = (const bf16 *)q; p.kpool = (const bf16 *)k_pool; p.vpool = (const bf16 *)v_pool;
  p.pm = PageMap{page_table, pages_per_seq, page_size, 1 << 20};
  p.m = m; p.tail_len = TTT_BLOCK; p.rows = rows; p.H = H; p.G = G; p.rps = TTT_BLOCK; p.nsplit = nsplit; p.out = (bf16 *)out;
  p.part_o = (float *)(base + ttt_meta_bytes(rows));
  p.part_ml = p.part_o + (size_t)nsplit * rows * H * hd;
  p.order = nullptr; p.stamp = nullptr; p.keep_partial = 1;
  const CUtensorMap *mk = kv_map(k_pool, p.pm.num_pages, G, page_size, hd, 1), *mv = kv_map(v_pool, p.pm.num_pages, G, page_size, hd, 1);
  if (!mk || !mv) return SPEC_ERR_CUDA;
  dim3 grid(mtiles, nsplit, seqs * G);
  if (launch_umma(p, grid, mk, mv, nullptr, s)) return SPEC_ERR_CUDA;
  launch_k(ttt_merge_kernel, dim3((T * H + 7) / 8), dim3(256), 0, s, p.part_o, p.part_ml, nsplit, rows * H, (const bf16 *)q,
           (const bf16 *)k_diag, (const bf16 *)v_diag, (int)n_steps, (int)T, (int)H, (int)G, (bf16 *)out, lse);
  attn_fast_forget_maps();
  return cudaGetLastError() == cudaSuccess ? SPEC_OK : SPEC_ERR_CUDA;
}
