// Persistent chain of weight-streaming bf16 GEMMs for sm_100a.
//
// A decoder layer at batch 1 is a chain of small dependent GEMMs (tens of MB of weights each).  Launched one
// by one, each pays a start-up (first tiles in flight) and a tail (reduction, epilogue) during which HBM idles.
// Here the GEMMs of a chain run inside one kernel:
//
//  * P persistent CTAs (two per SM).  Every GEMM ("op") is cut into (feature tile, k-block) units laid out
//    tile-major; CTA c owns the contiguous unit range [c U/P, (c+1) U/P), i.e. every SM streams the same
//    number of weight bytes of every op, whatever the op's shape;
//  * warp 4 is the TMA producer.  It walks the whole chain ahead of the math: weight tiles never depend on
//    earlier ops, so while an op's results are still being reduced the ring fills with the next op's weights;
//    only the activation tiles of op j wait for op j-1 (a counter in global memory);
//  * warp 5 issues tcgen05.mma into one of two TMEM accumulators (ping-pong over the tile fragments);
//  * warps 0-3 drain the accumulators: fragment partial sums go to an fp32 scratch in global memory (L2
//    resident), a grid-wide counter says when an op's partials are complete, then every warp reduces its
//    share of (tile, row) items in slice order and applies the op's epilogue (residual + next norm's input
//    and statistics, RoPE + q/K/V stores, SiLU(gate)*up, plain fp32), one warp per item, four features per
//    lane, so the epilogue needs no block-level synchronisation;
//  * a second counter per op says when its outputs are complete; the producer waits on it before loading
//    the next op's activation tiles.
//
// All waits (mbarriers, counters) are bounded; a timeout is recorded in the status words and in an abort word
// that makes every CTA leave its loops.  Counters belong to one launch and are zeroed by the host beforehand.
#include <cuda.h>
#include <stdio.h>
#include <string.h>

#include <algorithm>

#include "gemm_chain.cuh"
#include "tcgen05_ptx.cuh"

namespace spec {

namespace {

using namespace tc;

constexpr int MAX_STAGES = 16;
constexpr int A_BYTES = TILE_M * TILE_K * 2;
constexpr int NUM_SMS = 148;
constexpr int ABORT_WORD = CHAIN_COUNTERS - 1;       // counters[ABORT_WORD] != 0: every CTA gives up
constexpr uint32_t GRID_SPIN_LIMIT = 1u << 22;

struct ChainOp {
  CUtensorMap map_w[3];
  CUtensorMap map_x;
  int epi, tiles0, tiles1, ntiles, etiles, KB, maxslots;
  int O[3];
  unsigned U;                  // ntiles * KB (U * P < 2^31, checked on the host, so all unit arithmetic is 32-bit)
  int Pj;                      // CTAs that take units of this op: min(P, U), so that every one of them has work
  const float *ssq_in; int ssq_in_tiles; float inv_k_in, eps;
  float *out_f32; int ldo;
  float *xres; const bf16 *gain; bf16 *hb; float *ssq_out; bf16 *taps; int tap_mask, resid_add;
  const float2 *cs; bf16 *q; KvPool pool; int H, G, hd;
  bf16 *act;
};

struct alignas(64) ChainParams {
  ChainOp op[MAX_CHAIN_OPS];
  RowMeta m;
  PageMap pm;
  int ssq_ld, nops, rows, stages, ctrl_off;
  float *part;
  int32_t *ctr;
  int32_t *status;
  long long *timing;           // optional [P][MAX_CHAIN_OPS][8] globaltimer stamps (profiling aid)
};

__device__ __forceinline__ long long global_ns() {
  long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// stamps per (CTA, op): 0 producer: activations of the op available, 1 producer: last load of the op issued,
// 2 MMA: last MMA of the op issued, 3 drain: first accumulator ready, 4 drain: partials written,
// 5 drain: all partials of the grid present, 6 drain: epilogue share done, 7 kernel entry
#define CSTAMP(j, i) do { if (p.timing) p.timing[((size_t)blockIdx.x * MAX_CHAIN_OPS + (j)) * 16 + (i)] = global_ns(); } while (0)

__device__ __forceinline__ int ld_acquire(const int32_t *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
__device__ __forceinline__ void mbar_arrive(uint64_t *bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void bar_epi() { asm volatile("bar.sync 1, 128;" ::: "memory"); }
// CTA that owns unit u when U units are split over P CTAs as [c U / P, (c + 1) U / P)
__device__ __forceinline__ int owner_of(unsigned u, unsigned U, int P) { return (int)(((u + 1u) * (unsigned)P - 1u) / U); }

constexpr int FLAG_BASE = 2 * MAX_CHAIN_OPS;   // ctr[FLAG_BASE + b] != 0: all CTAs arrived at barrier b
// counts this CTA in at barrier b; the last CTA to arrive publishes the barrier's flag, which is what waiters poll
// (a word nobody does atomics on)
__device__ __forceinline__ void arrive_and_publish(int32_t *ctr, int b, int P) {
  __threadfence();
  if (atomicAdd(ctr + b, 1) == P - 1) {
    __threadfence();
    asm volatile("st.release.gpu.global.s32 [%0], %1;" ::"l"(ctr + FLAG_BASE + b), "r"(1) : "memory");
  }
}
// waits until counter >= target; false on timeout or abort
__device__ __forceinline__ bool wait_counter(const int32_t *ctr, int target, const int32_t *abort_word) {
  for (uint32_t it = 0; it < GRID_SPIN_LIMIT; it++) {
    if (ld_acquire(ctr) >= target) return true;
    if ((it & 63) == 63 && ld_acquire(abort_word) != 0) return false;
    __nanosleep(20);
  }
  return false;
}


__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c2, float d) {
  __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c2, d);
  return make_uint2(*(uint32_t *)&lo, *(uint32_t *)&hi);
}

// One warp's share of an op's (tile, row) items.  RB items are handled together and every global load of the
// group (slice partial sums, norm statistics, residual, gain, RoPE angles) is issued before the first use, so a
// group costs about one L2 round trip.  CAP = slices of one tile loaded per round.  Lane l owns features 4l..4l+3.
template <int RB, int CAP, int NTI>
__device__ __forceinline__ void epilogue_items(const ChainParams &p, const ChainOp &op, int P, int c, int warp, int lane,
                                               const int32_t *slot_s, const int32_t *seq_s, long long *tm_out) {
  const int rows = p.rows;
  long long t_idx = 0, t_wait = 0, t_rest = 0, n_groups = 0;
  const unsigned N = (unsigned)op.etiles * (unsigned)rows;
  const unsigned i0 = (unsigned)c * N / (unsigned)P, i1 = (unsigned)(c + 1) * N / (unsigned)P;
  const size_t sstride = (size_t)rows * TILE_M;              // floats between two slices of a tile
  for (unsigned it0 = i0 + warp; it0 < i1; it0 += 4 * RB) {
    int et[RB], row[RB], ns[RB][NTI];
    const float *base[RB][NTI];
    bool valid[RB];
    float4 acc[RB][NTI];
    float ss[RB];
    float4 xin[RB];
    uint2 gn[RB];
    float4 csv[RB][2];
    long long ta = global_ns();
    // ---- loads
#pragma unroll
    for (int b = 0; b < RB; b++) {
      const unsigned it = it0 + 4 * b;
      valid[b] = it < i1;
      et[b] = valid[b] ? (int)(it / (unsigned)rows) : 0;
      row[b] = valid[b] ? (int)(it - (unsigned)et[b] * (unsigned)rows) : 0;
      ss[b] = 0.0f;
      xin[b] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
      gn[b] = make_uint2(0u, 0u);
      csv[b][0] = csv[b][1] = make_float4(1.0f, 0.0f, 1.0f, 0.0f);
#pragma unroll
      for (int w2 = 0; w2 < NTI; w2++) {
        acc[b][w2] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
        ns[b][w2] = 0;
        base[b][w2] = p.part;
        if (!valid[b]) continue;
        const int T = et[b] + w2 * op.etiles;
        const int cf = owner_of((unsigned)T * (unsigned)op.KB, op.U, op.Pj), cl = owner_of((unsigned)(T + 1) * (unsigned)op.KB - 1u, op.U, op.Pj);
        ns[b][w2] = cl - cf + 1;
        base[b][w2] = p.part + (((size_t)T * op.maxslots) * rows + row[b]) * TILE_M + lane * 4;
      }
    }
    long long tb = global_ns();
    float4 v[RB][NTI][CAP];
#pragma unroll
    for (int b = 0; b < RB; b++)
#pragma unroll
      for (int w2 = 0; w2 < NTI; w2++)
#pragma unroll
        for (int s2 = 0; s2 < CAP; s2++)
          if (s2 < ns[b][w2]) v[b][w2][s2] = __ldcg((const float4 *)(base[b][w2] + (size_t)s2 * sstride));
#pragma unroll
    for (int b = 0; b < RB; b++) {
      if (!valid[b]) continue;
      if (op.ssq_in)
        for (int tt = lane; tt < op.ssq_in_tiles; tt += 32) ss[b] += __ldcg(op.ssq_in + (size_t)tt * p.ssq_ld + row[b]);
      const int o = (op.epi == EPI_QKV ? 0 : et[b] * TILE_M) + lane * 4;
      if (op.epi == EPI_RESID && o < op.O[0]) {
        if (op.resid_add) xin[b] = __ldcg((const float4 *)(op.xres + (size_t)row[b] * op.O[0] + o));
        gn[b] = *(const uint2 *)(op.gain + o);
      } else if (op.epi == EPI_QKV && et[b] < op.tiles1) {          // q and k tiles are rotated
        int tm = et[b] >= op.tiles0 ? et[b] - op.tiles0 : et[b];
        const int half = op.hd >> 1, i = (tm * TILE_M + lane * 4) % op.hd;
        const float4 *cp = (const float4 *)(op.cs + (size_t)row[b] * half + (i & (half - 1)));
        csv[b][0] = cp[0];
        csv[b][1] = cp[1];
      }
    }
    // ---- slice sums in slice order (further rounds only for tiles cut into more than CAP slices)
#pragma unroll
    for (int b = 0; b < RB; b++)
#pragma unroll
      for (int w2 = 0; w2 < NTI; w2++) {
#pragma unroll
        for (int s2 = 0; s2 < CAP; s2++)
          if (s2 < ns[b][w2]) { acc[b][w2].x += v[b][w2][s2].x; acc[b][w2].y += v[b][w2][s2].y; acc[b][w2].z += v[b][w2][s2].z; acc[b][w2].w += v[b][w2][s2].w; }
        for (int s2 = CAP; s2 < ns[b][w2]; s2++) {
          float4 t4 = __ldcg((const float4 *)(base[b][w2] + (size_t)s2 * sstride));
          acc[b][w2].x += t4.x; acc[b][w2].y += t4.y; acc[b][w2].z += t4.z; acc[b][w2].w += t4.w;
        }
      }
    long long tc = global_ns();
    // ---- epilogue
#pragma unroll
    for (int b = 0; b < RB; b++) {
      float sc = 1.0f;
      if (op.ssq_in) {                                            // all lanes take part in the shuffles
        float t = ss[b];
        for (int off = 16; off > 0; off >>= 1) t += __shfl_xor_sync(0xffffffffu, t, off);
        sc = 1.0f / sqrtf(t * op.inv_k_in + op.eps);
      }
      float v4[4] = {acc[b][0].x * sc, acc[b][0].y * sc, acc[b][0].z * sc, acc[b][0].w * sc};
      const int r = row[b];
      if (NTI == 1 && op.epi == EPI_F32) {
        const int o = et[b] * TILE_M + lane * 4;
        if (valid[b] && o < op.O[0]) *(float4 *)(op.out_f32 + (size_t)r * op.ldo + o) = make_float4(v4[0], v4[1], v4[2], v4[3]);
      } else if (NTI == 1 && op.epi == EPI_RESID) {
        const int o = et[b] * TILE_M + lane * 4;
        float sq = 0.0f;
        if (valid[b] && o < op.O[0]) {
          const size_t xi = (size_t)r * op.O[0] + o;
          const float x0 = xin[b].x + v4[0], x1 = xin[b].y + v4[1], x2 = xin[b].z + v4[2], x3 = xin[b].w + v4[3];
          *(float4 *)(op.xres + xi) = make_float4(x0, x1, x2, x3);
          const __nv_bfloat162 g01 = *(const __nv_bfloat162 *)&gn[b].x, g23 = *(const __nv_bfloat162 *)&gn[b].y;
          *(uint2 *)(op.hb + xi) = pack4_bf16(x0 * __low2float(g01), x1 * __high2float(g01), x2 * __low2float(g23), x3 * __high2float(g23));
          if (op.tap_mask) {
            const uint2 tp = pack4_bf16(x0, x1, x2, x3);
#pragma unroll
            for (int s2 = 0; s2 < 3; s2++)
              if ((op.tap_mask >> s2) & 1) *(uint2 *)(op.taps + (size_t)r * 3 * op.O[0] + (size_t)s2 * op.O[0] + o) = tp;
          }
          sq = x0 * x0 + x1 * x1 + x2 * x2 + x3 * x3;
        }
        for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
        if (valid[b] && lane == 0) op.ssq_out[(size_t)et[b] * p.ssq_ld + r] = sq;
      } else if (NTI == 2) {
        const int o = et[b] * TILE_M + lane * 4;
        const float u4[4] = {acc[b][NTI - 1].x * sc, acc[b][NTI - 1].y * sc, acc[b][NTI - 1].z * sc, acc[b][NTI - 1].w * sc};
        if (valid[b] && o < op.O[0]) {
          float a4[4];
#pragma unroll
          for (int e = 0; e < 4; e++) a4[e] = (v4[e] / (1.0f + expf(-v4[e]))) * u4[e];
          *(uint2 *)(op.act + (size_t)r * op.O[0] + o) = pack4_bf16(a4[0], a4[1], a4[2], a4[3]);
        }
      } else if (NTI == 1 && op.epi == EPI_QKV) {
        int mi = 0, tm = et[b];
        if (tm >= op.tiles1) { mi = 2; tm -= op.tiles1; }
        else if (tm >= op.tiles0) { mi = 1; tm -= op.tiles0; }
        const int hd = op.hd, half = hd >> 1;
        const int o = tm * TILE_M + lane * 4;                  // feature within weight mi; 4 features stay in one half
        const int head = o / hd, i = o % hd;
        float w4[4];
#pragma unroll
        for (int e = 0; e < 4; e++) w4[e] = __shfl_xor_sync(0xffffffffu, v4[e], half >> 2);   // rotate-half partner
        if (valid[b] && o < op.O[mi]) {
          if (mi < 2) {
            const float cc[4] = {csv[b][0].x, csv[b][0].z, csv[b][1].x, csv[b][1].z}, sn[4] = {csv[b][0].y, csv[b][0].w, csv[b][1].y, csv[b][1].w};
#pragma unroll
            for (int e = 0; e < 4; e++) v4[e] = (i < half) ? v4[e] * cc[e] - w4[e] * sn[e] : v4[e] * cc[e] + w4[e] * sn[e];
          }
          const int seq = seq_s[r];
          if (mi == 0) {
            const bool z = seq < 0;
            *(uint2 *)(op.q + ((size_t)r * op.H + head) * hd + i) = pack4_bf16(z ? 0.0f : v4[0], z ? 0.0f : v4[1], z ? 0.0f : v4[2], z ? 0.0f : v4[3]);
          } else if (slot_s[r] >= 0) {
            const int kvpos = p.m.kvpos[r];
            const size_t off = (((size_t)slot_s[r] * op.G + head) * p.pm.page_size + (kvpos % p.pm.page_size)) * hd + i;
            *(uint2 *)((bf16 *)(mi == 1 ? op.pool.k : op.pool.v) + off) = pack4_bf16(v4[0], v4[1], v4[2], v4[3]);
          }
        }
      }
    }
    long long td = global_ns();
    t_idx += tb - ta; t_wait += tc - tb; t_rest += td - tc; n_groups++;
  }
  if (tm_out && warp == 0 && lane == 0) { tm_out[8] = t_idx; tm_out[9] = t_wait; tm_out[10] = t_rest; tm_out[11] = n_groups; }
}

template <int NT>
__global__ void __launch_bounds__(192, 2) chain_kernel(const __grid_constant__ ChainParams p) {
  constexpr int B_BYTES = NT * TILE_K * 2;
  constexpr int STAGE = A_BYTES + B_BYTES;
  constexpr int TMEM_COLS = (2 * NT < 32) ? 32 : 2 * NT;

  extern __shared__ unsigned char smem_raw[];
  unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  unsigned char *ctrl = tiles + p.ctrl_off;
  uint64_t *full = (uint64_t *)ctrl;
  uint64_t *empty = full + MAX_STAGES;
  uint64_t *acc_full = empty + MAX_STAGES;       // [2]
  uint64_t *acc_empty = acc_full + 2;            // [2]
  uint32_t *tmem_slot = (uint32_t *)(acc_empty + 2);
  volatile uint32_t *abort_flag = tmem_slot + 1;
  int32_t *slot_s = (int32_t *)(ctrl + 512);     // [64] K/V cache slot of each row (-1: none)
  int32_t *seq_s = slot_s + 64;                  // [64]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int c = blockIdx.x, P = gridDim.x;
  const int stages = p.stages, rows = p.rows;
  const int32_t *abort_word = p.ctr + ABORT_WORD;

  if (threadIdx.x == 0) {
    for (int i = 0; i < stages; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    for (int i = 0; i < 2; i++) { mbar_init(&acc_full[i], 1); mbar_init(&acc_empty[i], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;
  if (threadIdx.x == 0) CSTAMP(0, 7);

  if (warp == 4) {
    // ================================================================== producer
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();
      int kbs[MAX_STAGES];                       // k-block held by each stage (for deferred activation loads)
      const CUtensorMap *xmap[MAX_STAGES];
      unsigned g = 0;                            // stage items issued so far (all ops)
      bool dead = false;
      for (int j = 0; j < p.nops && !dead; j++) {
        const ChainOp &op = p.op[j];
        const unsigned u0 = c < op.Pj ? (unsigned)c * op.U / (unsigned)op.Pj : op.U, u1 = c < op.Pj ? (unsigned)(c + 1) * op.U / (unsigned)op.Pj : op.U;
        bool dep_ok = false;
        unsigned pend_lo = g;                    // first item of this op whose activation tile is not issued yet
        auto dep_ready = [&]() -> bool { return j > 0 && ld_acquire(p.ctr + FLAG_BASE + 2 * (j - 1) + 1) != 0; };
        auto dep_wait = [&]() -> bool {
          if (j == 0) { pdl_wait(); return true; }
          return wait_counter(p.ctr + FLAG_BASE + 2 * (j - 1) + 1, 1, abort_word);
        };
        auto flush_b = [&]() {
          asm volatile("fence.proxy.async;" ::: "memory");   // other CTAs' generic-proxy stores -> this CTA's TMA reads
          for (unsigned gi = pend_lo; gi < g; gi++) {
            int st = (int)(gi % (unsigned)stages);
            tma_load_2d(tiles + st * STAGE + A_BYTES, xmap[st], kbs[st] * TILE_K, 0, &full[st]);
          }
          pend_lo = g;
          CSTAMP(j, 0);
        };
        int t = (int)(u0 / (unsigned)op.KB), kb = (int)(u0 - (unsigned)t * (unsigned)op.KB);
        for (unsigned u = u0; u < u1 && !dead; u++) {
          const int st = (int)(g % (unsigned)stages);
          if (g >= (unsigned)stages) {
            const uint32_t par = ((g / (unsigned)stages) - 1u) & 1u;
            if (!dep_ok && g - (unsigned)stages >= pend_lo) {
              // the stage still holds an item of this op that waits for its activations: resolve the dependency first
              if (!dep_wait()) { dead = true; break; }
              dep_ok = true;
              flush_b();
            }
            uint32_t it = 0;
            while (!mbar_test(&empty[st], par)) {
              if (!dep_ok && dep_ready()) { dep_ok = true; flush_b(); }
              if (++it > SPIN_LIMIT || *abort_flag) { dead = true; break; }
            }
            if (dead) { set_status(p.status, ST_TIMEOUT, 300, c, j); break; }
          }
          int mi = 0, tm = t;
          if (tm >= op.tiles1) { mi = 2; tm -= op.tiles1; }
          else if (tm >= op.tiles0) { mi = 1; tm -= op.tiles0; }
          mbar_expect_tx(&full[st], STAGE);
          tma_load_2d_hint(tiles + st * STAGE, &op.map_w[mi], kb * TILE_K, tm * TILE_M, &full[st], pol);
          kbs[st] = kb;
          xmap[st] = &op.map_x;
          g++;
          if (!dep_ok && dep_ready()) { dep_ok = true; flush_b(); }
          else if (dep_ok) { tma_load_2d(tiles + st * STAGE + A_BYTES, &op.map_x, kb * TILE_K, 0, &full[st]); pend_lo = g; }
          if (++kb == op.KB) { kb = 0; t++; }
        }
        CSTAMP(j, 1);
        if (!dead && !dep_ok) {
          if (!dep_wait()) { dead = true; set_status(p.status, ST_TIMEOUT, 301, c, j); }
          else { dep_ok = true; flush_b(); }
        }
      }
      if (dead) { *abort_flag = 1; atomicExch(p.ctr + ABORT_WORD, 1); }
    }
  } else if (warp == 5) {
    // ================================================================== MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc(NT);
      unsigned g = 0;
      int pc = 0;                                // tile fragments processed so far
      bool dead = false;
      for (int j = 0; j < p.nops && !dead; j++) {
        const ChainOp &op = p.op[j];
        const unsigned u0 = c < op.Pj ? (unsigned)c * op.U / (unsigned)op.Pj : op.U, u1 = c < op.Pj ? (unsigned)(c + 1) * op.U / (unsigned)op.Pj : op.U;
        unsigned u = u0;
        int kb_lo = (int)(u0 % (unsigned)op.KB);
        while (u < u1 && !dead) {
          const int kb_hi = (int)min((unsigned)op.KB, (unsigned)kb_lo + (u1 - u));
          const int buf = pc & 1;
          if (pc >= 2 && !mbar_wait(&acc_empty[buf], (uint32_t)(((pc >> 1) - 1) & 1))) { dead = true; set_status(p.status, ST_TIMEOUT, 310, c, j); break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          for (int kb = kb_lo; kb < kb_hi; kb++) {
            const int st = (int)(g % (unsigned)stages);
            if (!mbar_wait(&full[st], ((g / (unsigned)stages) & 1u)) || *abort_flag) { dead = true; set_status(p.status, ST_TIMEOUT, 311, c, j); break; }
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a = smem_u32(tiles + st * STAGE), b = a + A_BYTES;
#pragma unroll
            for (int q4 = 0; q4 < TILE_K / UMMA_K; q4++)
              umma_bf16(tmem_base + buf * NT, umma_desc_sw128(a + q4 * UMMA_K * 2), umma_desc_sw128(b + q4 * UMMA_K * 2), idesc,
                        (kb > kb_lo || q4) ? 1u : 0u);
            umma_commit(&empty[st]);
            g++;
          }
          if (dead) break;
          umma_commit(&acc_full[buf]);
          pc++;
          u += kb_hi - kb_lo;
          kb_lo = 0;
        }
        CSTAMP(j, 2);
      }
      if (dead) { *abort_flag = 1; atomicExch(p.ctr + ABORT_WORD, 1); }
    }
  } else {
    // ================================================================== accumulator drain + epilogue (warps 0-3)
    pdl_wait();                                  // row metadata comes from the kernels before this one
    if ((int)threadIdx.x < rows) {
      // cache slot of every row's K/V (for EPI_QKV ops): sequence -> position -> page, resolved once
      const int row = threadIdx.x;
      const int seq = p.m.seq ? p.m.seq[row] : -1;
      int slot = -1;
      if (seq >= 0 && p.pm.table) {
        const int kvpos = p.m.kvpos[row];
        if (kvpos < 0 || kvpos / p.pm.page_size >= p.pm.pages_per_seq) {
          set_status(p.status, ST_BOUNDS, 1, row, kvpos);
        } else {
          const int page = p.pm.table[(size_t)seq * p.pm.pages_per_seq + kvpos / p.pm.page_size];
          if (page < 0 || page >= p.pm.num_pages) set_status(p.status, ST_BOUNDS, 2, row, page);
          else slot = page;                      // page index; the element offset is formed per KV head below
        }
      }
      slot_s[row] = slot;
      seq_s[row] = seq;
    }
    bar_epi();
    int pc = 0;
    bool dead = false;
    for (int j = 0; j < p.nops; j++) {
      const ChainOp &op = p.op[j];
      const unsigned u0 = c < op.Pj ? (unsigned)c * op.U / (unsigned)op.Pj : op.U, u1 = c < op.Pj ? (unsigned)(c + 1) * op.U / (unsigned)op.Pj : op.U;
      // ---- 1. fragment partial sums -> scratch
      {
        unsigned u = u0;
        int t = (int)(u0 / (unsigned)op.KB), kb_lo = (int)(u0 - (unsigned)t * (unsigned)op.KB);
        while (u < u1 && !dead) {
          const int kb_hi = (int)min((unsigned)op.KB, (unsigned)kb_lo + (u1 - u));
          const int buf = pc & 1;
          if (!mbar_wait(&acc_full[buf], (uint32_t)((pc >> 1) & 1)) || *abort_flag) { dead = true; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          if (threadIdx.x == 0 && u == u0) CSTAMP(j, 3);
          const int slot = c - owner_of((unsigned)t * (unsigned)op.KB, op.U, op.Pj);
          float *dst = p.part + (((size_t)t * op.maxslots + slot) * rows) * TILE_M + threadIdx.x;
#pragma unroll 1
          for (int cc = 0; cc < rows; cc += 16) {
            uint32_t v[16];
            tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + (uint32_t)(buf * NT + cc), v);
#pragma unroll
            for (int r = 0; r < 16; r++)
              if (cc + r < rows) dst[(size_t)(cc + r) * TILE_M] = __uint_as_float(v[r]);
          }
          asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
          __syncwarp();
          if (lane == 0) mbar_arrive(&acc_empty[buf]);
          pc++;
          u += kb_hi - kb_lo;
          kb_lo = 0;
          t++;
        }
      }
      // ---- 2. all partial sums of the op are in memory (grid-wide)
      __threadfence();
      bar_epi();
      if (threadIdx.x == 0) {
        arrive_and_publish(p.ctr, 2 * j, P);
        CSTAMP(j, 4);
        if (!wait_counter(p.ctr + FLAG_BASE + 2 * j, 1, abort_word)) *abort_flag = 1;
      }
      bar_epi();
      dead = dead || *abort_flag != 0;
      if (threadIdx.x == 0) CSTAMP(j, 5);
      // ---- 3. this warp's share of the (tile, row) items: reduce in slice order + epilogue
      if (!dead) {
        if (op.epi == EPI_SWIGLU) {
          if (op.maxslots <= 3) epilogue_items<2, 3, 2>(p, op, P, c, warp, lane, slot_s, seq_s, p.timing ? p.timing + ((size_t)blockIdx.x * MAX_CHAIN_OPS + j) * 16 : nullptr);
          else epilogue_items<1, 6, 2>(p, op, P, c, warp, lane, slot_s, seq_s, p.timing ? p.timing + ((size_t)blockIdx.x * MAX_CHAIN_OPS + j) * 16 : nullptr);
        } else {
          if (op.maxslots <= 6) epilogue_items<2, 6, 1>(p, op, P, c, warp, lane, slot_s, seq_s, p.timing ? p.timing + ((size_t)blockIdx.x * MAX_CHAIN_OPS + j) * 16 : nullptr);
          else epilogue_items<1, 12, 1>(p, op, P, c, warp, lane, slot_s, seq_s, p.timing ? p.timing + ((size_t)blockIdx.x * MAX_CHAIN_OPS + j) * 16 : nullptr);
        }
      }
      // ---- 4. outputs of the op are complete (grid-wide): the producers may load the next op's activations
      asm volatile("fence.proxy.async;" ::: "memory");
      __threadfence();
      bar_epi();
      if (threadIdx.x == 0) { arrive_and_publish(p.ctr, 2 * j + 1, P); CSTAMP(j, 6); }
    }
    if (dead && lane == 0) { *abort_flag = 1; atomicExch(p.ctr + ABORT_WORD, 1); set_status(p.status, ST_TIMEOUT, 320, c, 0); }
  }
  pdl_trigger();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(TMEM_COLS) : "memory");
  }
}

int host_owner(long long u, long long U, int P) { return (int)(((u + 1) * P - 1) / U); }

int ntiles_of(FusedEpi epi, const FusedGemmArgs &a) {
  int t = 0;
  for (int j = 0; j < a.nw; j++) t += (a.O[j] + TILE_M - 1) / TILE_M;
  (void)epi;
  return t;
}

int g_chain_ctas = 2 * NUM_SMS;

int pick_P() { return g_chain_ctas; }

int max_slots(int ntiles, int KB, int P) {
  long long U = (long long)ntiles * KB;
  int m = 1;
  for (int t = 0; t < ntiles; t++) m = std::max(m, host_owner((long long)(t + 1) * KB - 1, U, P) - host_owner((long long)t * KB, U, P) + 1);
  return m;
}

}  // namespace

int chain_ctas() { return pick_P(); }

bool chain_supported(const FusedEpi *epi, const FusedGemmArgs *ops, int nops) {
  if (nops < 1 || nops > MAX_CHAIN_OPS) return false;
  for (int j = 0; j < nops; j++) {
    if (epi[j] == EPI_ARGMAX || !fused_gemm_supported(epi[j], ops[j])) return false;
    if (ops[j].rows != ops[0].rows || ops[j].rows > 64) return false;
    if (epi[j] == EPI_QKV && (ops[j].hd < 16)) return false;
    if (epi[j] == EPI_F32 && (ops[j].ldo % 4)) return false;
    for (int w = 0; w < ops[j].nw; w++)
      if (ops[j].O[w] % 4) return false;                       // a lane's four features are stored as one vector
    long long U = (long long)ntiles_of(epi[j], ops[j]) * ((ops[j].I + TILE_K - 1) / TILE_K);
    if ((U + 1) * pick_P() >= (1ll << 31) || (long long)ntiles_of(epi[j], ops[j]) * 64 * pick_P() >= (1ll << 31)) return false;
  }
  return true;
}

size_t chain_scratch_bytes(const FusedEpi *epi, const FusedGemmArgs *ops, int nops) {
  size_t need = 0;
  const int P = pick_P();
  for (int j = 0; j < nops; j++) {
    int nt = ntiles_of(epi[j], ops[j]), KB = (ops[j].I + TILE_K - 1) / TILE_K;
    int Pj = (int)std::min<long long>(P, (long long)nt * KB);
    need = std::max(need, (size_t)nt * max_slots(nt, KB, Pj) * ops[j].rows * TILE_M * sizeof(float));
  }
  return need;
}

int chain_launch(FastGemm *g, const FusedEpi *epi, const FusedGemmArgs *ops, int nops, float *scratch, size_t scratch_bytes,
                 int32_t *counters, int32_t *status, bool pdl, cudaStream_t s, long long *timing) {
  if (!g || !chain_supported(epi, ops, nops) || !scratch || !counters) return -1;
  if (chain_scratch_bytes(epi, ops, nops) > scratch_bytes) return -3;
  static ChainParams p;                          // ~5 KB: kept off the stack; launches are issued by one host thread at a time
  memset(&p, 0, sizeof p);
  const int P = pick_P();
  const int rows = ops[0].rows, nt = rows <= 16 ? 16 : 64;
  for (int j = 0; j < nops; j++) {
    const FusedGemmArgs &a = ops[j];
    ChainOp &o = p.op[j];
    for (int w = 0; w < a.nw; w++) {
      const CUtensorMap *mw = fast_gemm_map(g, a.w[w], a.O[w], a.I, TILE_M);
      if (!mw) return -6;
      o.map_w[w] = *mw;
      o.O[w] = a.O[w];
    }
    const CUtensorMap *mx = fast_gemm_map(g, a.x, a.rows, a.I, nt);
    if (!mx) return -6;
    o.map_x = *mx;
    o.epi = epi[j];
    o.tiles0 = (a.O[0] + TILE_M - 1) / TILE_M;
    o.tiles1 = o.tiles0 + (a.nw > 1 ? (a.O[1] + TILE_M - 1) / TILE_M : 0);
    o.ntiles = ntiles_of(epi[j], a);
    o.etiles = epi[j] == EPI_SWIGLU ? o.tiles0 : o.ntiles;
    o.KB = (a.I + TILE_K - 1) / TILE_K;
    o.U = (unsigned)o.ntiles * (unsigned)o.KB;
    o.Pj = (int)std::min<long long>(P, (long long)o.U);
    o.maxslots = max_slots(o.ntiles, o.KB, o.Pj);
    o.ssq_in = a.ssq_in; o.ssq_in_tiles = a.ssq_in_tiles; o.inv_k_in = 1.0f / (float)a.k_in; o.eps = a.eps;
    o.out_f32 = a.out_f32; o.ldo = a.ldo;
    o.xres = a.xres; o.gain = a.gain; o.hb = a.hb; o.ssq_out = a.ssq_out; o.taps = a.tap_mask ? a.taps : nullptr;
    o.tap_mask = a.taps ? a.tap_mask : 0; o.resid_add = a.resid_add;
    o.cs = a.cs; o.q = a.q; o.pool = a.pool; o.H = a.H; o.G = a.G; o.hd = a.hd;
    o.act = a.act;
    if (a.ssq_ld) p.ssq_ld = a.ssq_ld;
    if (epi[j] == EPI_QKV) { p.m = a.m; p.pm = a.pm; }
  }
  const int stage = A_BYTES + nt * TILE_K * 2;
  p.stages = std::max(2, std::min(MAX_STAGES, (100 * 1024) / stage));
  p.ctrl_off = (p.stages * stage + 1023) & ~1023;
  const int smem = p.ctrl_off + 512 + 2 * 64 * 4 + 1024;
  p.nops = nops; p.rows = rows; p.part = scratch; p.ctr = counters; p.status = status; p.timing = timing;
  static int configured_nt[2] = {0, 0};          // the two instantiations have the same function type: one slot each
  auto launch = [&](auto kern) -> int {
    int &configured = configured_nt[nt == 16 ? 0 : 1];
    if (smem > configured) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
      if (e != cudaSuccess) { fprintf(stderr, "chain_launch: set attribute: %s\n", cudaGetErrorString(e)); return -6; }
      configured = smem;
    }
    if (!launch_allowed()) return 0;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(P); cfg.blockDim = dim3(192); cfg.dynamicSmemBytes = smem; cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at; cfg.numAttrs = pdl ? 1 : 0;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kern, p);
    if (e != cudaSuccess) fprintf(stderr, "chain_launch: %s (params %zu bytes, smem %d, grid %d)\n", cudaGetErrorString(e), sizeof(p), smem, P);
    return e == cudaSuccess ? 0 : -6;
  };
  return nt == 16 ? launch(chain_kernel<16>) : launch(chain_kernel<64>);
}

}  // namespace spec
