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
  long long U;                 // ntiles * KB
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
};

__device__ __forceinline__ int ld_acquire(const int32_t *p) {
  int v;
  asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
  return v;
}
__device__ __forceinline__ bool mbar_test(uint64_t *bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
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
__device__ __forceinline__ int owner_of(long long u, long long U, int P) { return (int)(((u + 1) * P - 1) / U); }

// waits until counter >= target; false on timeout or abort
__device__ __forceinline__ bool wait_counter(const int32_t *ctr, int target, const int32_t *abort_word) {
  for (uint32_t it = 0; it < GRID_SPIN_LIMIT; it++) {
    if (ld_acquire(ctr) >= target) return true;
    if ((it & 63) == 63 && ld_acquire(abort_word) != 0) return false;
    __nanosleep(20);
  }
  return false;
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

  if (warp == 4) {
    // ================================================================== producer
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();
      int kbs[MAX_STAGES];                       // k-block held by each stage (for deferred activation loads)
      const CUtensorMap *xmap[MAX_STAGES];
      long long g = 0;                           // stage items issued so far (all ops)
      bool dead = false;
      for (int j = 0; j < p.nops && !dead; j++) {
        const ChainOp &op = p.op[j];
        const long long u0 = c < op.Pj ? (long long)c * op.U / op.Pj : op.U, u1 = c < op.Pj ? (long long)(c + 1) * op.U / op.Pj : op.U;
        bool dep_ok = false;
        long long pend_lo = g;                   // first item of this op whose activation tile is not issued yet
        auto dep_ready = [&]() -> bool { return j > 0 && ld_acquire(p.ctr + 2 * (j - 1) + 1) >= P; };
        auto dep_wait = [&]() -> bool {
          if (j == 0) { pdl_wait(); return true; }
          return wait_counter(p.ctr + 2 * (j - 1) + 1, P, abort_word);
        };
        auto flush_b = [&]() {
          asm volatile("fence.proxy.async;" ::: "memory");   // other CTAs' generic-proxy stores -> this CTA's TMA reads
          for (long long gi = pend_lo; gi < g; gi++) {
            int st = (int)(gi % stages);
            tma_load_2d(tiles + st * STAGE + A_BYTES, xmap[st], kbs[st] * TILE_K, 0, &full[st]);
          }
          pend_lo = g;
        };
        int t = (int)(u0 / op.KB), kb = (int)(u0 - (long long)t * op.KB);
        for (long long u = u0; u < u1 && !dead; u++) {
          const int st = (int)(g % stages);
          if (g >= stages) {
            const uint32_t par = (uint32_t)(((g / stages) - 1) & 1);
            if (!dep_ok && g - stages >= pend_lo) {
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
      long long g = 0;
      int pc = 0;                                // tile fragments processed so far
      bool dead = false;
      for (int j = 0; j < p.nops && !dead; j++) {
        const ChainOp &op = p.op[j];
        const long long u0 = c < op.Pj ? (long long)c * op.U / op.Pj : op.U, u1 = c < op.Pj ? (long long)(c + 1) * op.U / op.Pj : op.U;
        long long u = u0;
        int kb_lo = (int)(u0 % op.KB);
        while (u < u1 && !dead) {
          const int kb_hi = (int)std::min<long long>(op.KB, kb_lo + (u1 - u));
          const int buf = pc & 1;
          if (pc >= 2 && !mbar_wait(&acc_empty[buf], (uint32_t)(((pc >> 1) - 1) & 1))) { dead = true; set_status(p.status, ST_TIMEOUT, 310, c, j); break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          for (int kb = kb_lo; kb < kb_hi; kb++) {
            const int st = (int)(g % stages);
            if (!mbar_wait(&full[st], (uint32_t)((g / stages) & 1)) || *abort_flag) { dead = true; set_status(p.status, ST_TIMEOUT, 311, c, j); break; }
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
      const long long u0 = c < op.Pj ? (long long)c * op.U / op.Pj : op.U, u1 = c < op.Pj ? (long long)(c + 1) * op.U / op.Pj : op.U;
      // ---- 1. fragment partial sums -> scratch
      {
        long long u = u0;
        int t = (int)(u0 / op.KB), kb_lo = (int)(u0 - (long long)t * op.KB);
        while (u < u1 && !dead) {
          const int kb_hi = (int)std::min<long long>(op.KB, kb_lo + (u1 - u));
          const int buf = pc & 1;
          if (!mbar_wait(&acc_full[buf], (uint32_t)((pc >> 1) & 1)) || *abort_flag) { dead = true; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const int slot = c - owner_of((long long)t * op.KB, op.U, op.Pj);
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
      if (threadIdx.x == 0) atomicAdd(p.ctr + 2 * j, 1);
      if (!dead && lane == 0) dead = !wait_counter(p.ctr + 2 * j, P, abort_word);
      dead = __shfl_sync(0xffffffffu, dead ? 1 : 0, 0) != 0;
      // ---- 3. this warp's share of the (tile, row) items: reduce in slice order + epilogue
      if (!dead) {
        const long long N = (long long)op.etiles * rows;
        const long long i0 = (long long)c * N / P, i1 = (long long)(c + 1) * N / P;
        const size_t sstride = (size_t)rows * TILE_M;              // floats between two slices of a tile
        for (long long it = i0 + warp; it < i1; it += 4) {
          const int et = (int)(it / rows), row = (int)(it - (long long)et * rows);
          // slices of the tile(s) of this item
          float4 acc[2];
          const int nt_item = op.epi == EPI_SWIGLU ? 2 : 1;
#pragma unroll
          for (int w2 = 0; w2 < 2; w2++) {
            acc[w2] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            if (w2 >= nt_item) continue;
            const int T = et + w2 * op.etiles;
            const int cf = owner_of((long long)T * op.KB, op.U, op.Pj), cl = owner_of((long long)(T + 1) * op.KB - 1, op.U, op.Pj);
            const int ns = cl - cf + 1;
            const float *base = p.part + (((size_t)T * op.maxslots) * rows + row) * TILE_M + lane * 4;
            for (int s0 = 0; s0 < ns; s0 += 8) {
              float4 v[8];
#pragma unroll
              for (int s = 0; s < 8; s++)
                if (s0 + s < ns) v[s] = __ldcg((const float4 *)(base + (size_t)(s0 + s) * sstride));
#pragma unroll
              for (int s = 0; s < 8; s++)
                if (s0 + s < ns) { acc[w2].x += v[s].x; acc[w2].y += v[s].y; acc[w2].z += v[s].z; acc[w2].w += v[s].w; }
            }
          }
          // per-row scale of the input (RMSNorm factor), every lane gets the total
          float sc = 1.0f;
          if (op.ssq_in) {
            float ss = 0.0f;
            for (int tt = lane; tt < op.ssq_in_tiles; tt += 32) ss += __ldcg(op.ssq_in + (size_t)tt * p.ssq_ld + row);
            for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            sc = 1.0f / sqrtf(ss * op.inv_k_in + op.eps);
          }
          float v4[4] = {acc[0].x * sc, acc[0].y * sc, acc[0].z * sc, acc[0].w * sc};
          if (op.epi == EPI_F32) {
            const int o = et * TILE_M + lane * 4;
#pragma unroll
            for (int e = 0; e < 4; e++)
              if (o + e < op.O[0]) op.out_f32[(size_t)row * op.ldo + o + e] = v4[e];
          } else if (op.epi == EPI_RESID) {
            const int o = et * TILE_M + lane * 4;
            float sq = 0.0f;
#pragma unroll
            for (int e = 0; e < 4; e++) {
              if (o + e < op.O[0]) {
                const size_t xi = (size_t)row * op.O[0] + o + e;
                const float xo = (op.resid_add ? __ldcg(op.xres + xi) : 0.0f) + v4[e];
                op.xres[xi] = xo;
                op.hb[xi] = __float2bfloat16_rn(xo * __bfloat162float(op.gain[o + e]));
                if (op.tap_mask) {
#pragma unroll
                  for (int s = 0; s < 3; s++)
                    if ((op.tap_mask >> s) & 1) op.taps[(size_t)row * 3 * op.O[0] + (size_t)s * op.O[0] + o + e] = __float2bfloat16_rn(xo);
                }
                sq += xo * xo;
              }
            }
            for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
            if (lane == 0) op.ssq_out[(size_t)et * p.ssq_ld + row] = sq;
          } else if (op.epi == EPI_SWIGLU) {
            const int o = et * TILE_M + lane * 4;
            const float u4[4] = {acc[1].x * sc, acc[1].y * sc, acc[1].z * sc, acc[1].w * sc};
#pragma unroll
            for (int e = 0; e < 4; e++)
              if (o + e < op.O[0]) op.act[(size_t)row * op.O[0] + o + e] = __float2bfloat16_rn((v4[e] / (1.0f + expf(-v4[e]))) * u4[e]);
          } else if (op.epi == EPI_QKV) {
            int mi = 0, tm = et;
            if (tm >= op.tiles1) { mi = 2; tm -= op.tiles1; }
            else if (tm >= op.tiles0) { mi = 1; tm -= op.tiles0; }
            const int hd = op.hd, half = hd >> 1;
            const int o = tm * TILE_M + lane * 4;                  // feature within weight mi; 4 features stay in one half
            const int head = o / hd, i = o % hd;
            if (mi < 2) {                                          // rotate-half RoPE: partner features sit half/4 lanes away
              float w4[4];
#pragma unroll
              for (int e = 0; e < 4; e++) w4[e] = __shfl_xor_sync(0xffffffffu, v4[e], half >> 2);
              if (o < op.O[mi]) {
#pragma unroll
                for (int e = 0; e < 4; e++) {
                  const float2 cs = op.cs[(size_t)row * half + ((i + e) & (half - 1))];
                  v4[e] = (i < half) ? v4[e] * cs.x - w4[e] * cs.y : v4[e] * cs.x + w4[e] * cs.y;
                }
              }
            }
            if (o < op.O[mi]) {
              const int seq = seq_s[row];
              if (mi == 0) {
#pragma unroll
                for (int e = 0; e < 4; e++) op.q[((size_t)row * op.H + head) * hd + i + e] = __float2bfloat16_rn(seq < 0 ? 0.0f : v4[e]);
              } else if (slot_s[row] >= 0) {
                const int kvpos = p.m.kvpos[row];
                const size_t off = (((size_t)slot_s[row] * op.G + head) * p.pm.page_size + (kvpos % p.pm.page_size)) * hd + i;
                bf16 *dst = (bf16 *)(mi == 1 ? op.pool.k : op.pool.v) + off;
#pragma unroll
                for (int e = 0; e < 4; e++) dst[e] = __float2bfloat16_rn(v4[e]);
              }
            }
          }
        }
      }
      // ---- 4. outputs of the op are complete (grid-wide): the producers may load the next op's activations
      asm volatile("fence.proxy.async;" ::: "memory");
      __threadfence();
      bar_epi();
      if (threadIdx.x == 0) atomicAdd(p.ctr + 2 * j + 1, 1);
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

bool chain_supported(const FusedEpi *epi, const FusedGemmArgs *ops, int nops) {
  if (nops < 1 || nops > MAX_CHAIN_OPS) return false;
  for (int j = 0; j < nops; j++) {
    if (epi[j] == EPI_ARGMAX || !fused_gemm_supported(epi[j], ops[j])) return false;
    if (ops[j].rows != ops[0].rows || ops[j].rows > 64) return false;
    if (epi[j] == EPI_QKV && (ops[j].hd < 16)) return false;
    if (epi[j] == EPI_F32 && (ops[j].ldo % 4)) return false;
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
                 int32_t *counters, int32_t *status, bool pdl, cudaStream_t s) {
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
    o.U = (long long)o.ntiles * o.KB;
    o.Pj = (int)std::min<long long>(P, o.U);
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
  p.nops = nops; p.rows = rows; p.part = scratch; p.ctr = counters; p.status = status;
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
