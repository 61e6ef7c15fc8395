// bf16 weight-streaming GEMM for sm_100a: out[r][o] = sum_i x[r][i] * w[o][i] with few rows
// (a speculative step has 4..256 token rows) and large weights, i.e. an HBM-bound contraction.
//
// Mapping ("swap-AB"): the weight tile is the MMA's M side (128 output features x 64 k-elements,
// K-major, 128-byte swizzle), the token rows are the N side (NT = 16..256 rows x 64 k-elements),
// the fp32 accumulator [128 x NT] lives in TMEM.  One CTA = one (feature tile, K slice); slices
// write fp32 partial sums that the consumer kernel adds up (deterministic, no atomics).
// Warp 0 streams tiles with TMA into a ring of shared-memory stages, warp 1 issues tcgen05.mma,
// all four warps drain TMEM in the epilogue.  Every wait is bounded: on timeout the CTA records
// it in the status words, releases its TMEM and exits.
#include <cuda.h>
#include <stdio.h>

#include <map>
#include <string>
#include <tuple>

#include "gemm_fast.cuh"
#include "tcgen05_ptx.cuh"

namespace spec {

namespace {

using namespace tc;

template <int NT> struct Cfg {
  static constexpr int A_BYTES = TILE_M * TILE_K * 2;
  static constexpr int B_BYTES = NT * TILE_K * 2;
  static constexpr int STAGE = A_BYTES + B_BYTES;
  static constexpr int STAGES = NT <= 64 ? 4 : (NT == 128 ? 4 : 3);
  static constexpr int TMEM_COLS = NT < 32 ? 32 : NT;
  static constexpr int SMEM = STAGES * STAGE + 1024 /*alignment slack*/ + 256 /*barriers*/;
};

template <int NT>
__global__ void __launch_bounds__(128) gemm_tcgen05_kernel(const __grid_constant__ CUtensorMap map_w,
                                                           const __grid_constant__ CUtensorMap map_x, float *__restrict__ out,
                                                           int rows, int O, int KB, int S, int ldo, size_t pstride,
                                                           int32_t *status) {
  using C = Cfg<NT>;
  extern __shared__ unsigned char smem_raw[];
  unsigned char *tiles = (unsigned char *)(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  uint64_t *full = (uint64_t *)(tiles + C::STAGES * C::STAGE);
  uint64_t *empty = full + C::STAGES;
  uint64_t *acc_bar = empty + C::STAGES;
  uint32_t *tmem_slot = (uint32_t *)(acc_bar + 1);
  volatile uint32_t *abort_flag = tmem_slot + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tile = blockIdx.x, s = blockIdx.y;
  const int kb0 = (int)(((long long)s * KB) / S), kb1 = (int)(((long long)(s + 1) * KB) / S);
  const int nkb = kb1 - kb0;

  if (threadIdx.x == 0) {
    for (int i = 0; i < C::STAGES; i++) { mbar_init(&full[i], 1); mbar_init(&empty[i], 1); }
    mbar_init(acc_bar, 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // TMEM allocation is a whole-warp operation
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(C::TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0 && lane == 0) {
    // ---- producer: stream weight and activation tiles
    for (int i = 0; i < nkb; i++) {
      int st = i % C::STAGES;
      if (i >= C::STAGES && !mbar_wait(&empty[st], ((i / C::STAGES) - 1) & 1)) {
        *abort_flag = 1; set_status(status, ST_TIMEOUT, 100, tile, i); break;
      }
      if (*abort_flag) break;
      unsigned char *a = tiles + st * C::STAGE, *b = a + C::A_BYTES;
      mbar_expect_tx(&full[st], C::STAGE);
      tma_load_2d(a, &map_w, (kb0 + i) * TILE_K, tile * TILE_M, &full[st]);
      tma_load_2d(b, &map_x, (kb0 + i) * TILE_K, 0, &full[st]);
    }
  } else if (warp == 1 && lane == 0) {
    // ---- MMA issuer
    constexpr uint32_t idesc = umma_idesc(NT);
    for (int i = 0; i < nkb; i++) {
      int st = i % C::STAGES;
      if (!mbar_wait(&full[st], (i / C::STAGES) & 1)) { *abort_flag = 1; set_status(status, ST_TIMEOUT, 101, tile, i); break; }
      if (*abort_flag) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      uint32_t a = smem_u32(tiles + st * C::STAGE), b = a + C::A_BYTES;
#pragma unroll
      for (int j = 0; j < TILE_K / UMMA_K; j++)
        umma_bf16(tmem_base, umma_desc_sw128(a + j * UMMA_K * 2), umma_desc_sw128(b + j * UMMA_K * 2), idesc, (i | j) ? 1u : 0u);
      umma_commit(&empty[st]);      // frees the stage once these MMAs have read it
    }
    umma_commit(acc_bar);           // accumulator complete
  }
  // ---- epilogue: all four warps; warp w owns TMEM lanes 32w..32w+31 (= output features)
  bool ok = true;
  if (lane == 0) ok = mbar_wait(acc_bar, 0);
  ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
  if (!ok && lane == 0) { *abort_flag = 1; set_status(status, ST_TIMEOUT, 102, tile, s); }
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  int go = (lane == 0) ? ((ok && !*abort_flag) ? 1 : 0) : 0;      // one decision per warp: tcgen05.ld is warp-wide
  go = __shfl_sync(0xffffffffu, go, 0);
  if (go && nkb > 0) {
    const int o = tile * TILE_M + warp * 32 + lane;
    float *dst = out + (size_t)s * pstride + o;
#pragma unroll 1
    for (int c0 = 0; c0 < NT; c0 += 16) {
      if (c0 >= rows) break;
      uint32_t v[16];
      tmem_ld16(tmem_base + ((uint32_t)(warp * 32) << 16) + c0, v);
      if (o < O) {
#pragma unroll
        for (int j = 0; j < 16; j++)
          if (c0 + j < rows) dst[(size_t)(c0 + j) * ldo] = __uint_as_float(v[j]);
      }
    }
  } else if (nkb <= 0) {
    const int o = tile * TILE_M + warp * 32 + lane;
    if (o < O)
      for (int r = 0; r < rows; r++) out[(size_t)s * pstride + (size_t)r * ldo + o] = 0.0f;
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(C::TMEM_COLS) : "memory");
  }
}

// sum of S slices -> out (one-shot entry point)
__global__ void reduce_slices_kernel(const float *__restrict__ parts, int S, size_t pstride, float *__restrict__ out, int rows,
                                     int O, int ldo) {
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)rows * O) return;
  size_t r = idx / O, o = idx % O;
  float v = 0.0f;
  for (int p = 0; p < S; p++) v += parts[(size_t)p * pstride + r * O + o];
  out[r * ldo + o] = v;
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                             const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

struct FastGemm {
  EncodeFn encode = nullptr;
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> cache;   // (ptr, outer, inner, box_outer)
  bool attr_done[5] = {false, false, false, false, false};
};

static EncodeFn get_encode(std::string &why) {
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
    why = std::string("cuTensorMapEncodeTiled not available: ") + cudaGetErrorString(e);
    return nullptr;
  }
  return (EncodeFn)fn;
}

FastGemm *fast_gemm_create(std::string &why) {
  EncodeFn f = get_encode(why);
  if (!f) return nullptr;
  FastGemm *g = new FastGemm();
  g->encode = f;
  return g;
}
void fast_gemm_destroy(FastGemm *g) { delete g; }

// 2D bf16 tensor [outer][inner] (row pitch inner), box [box_outer][64], 128-byte swizzle
static const CUtensorMap *get_map(FastGemm *g, const void *ptr, int outer, int inner, int box_outer) {
  auto key = std::make_tuple(ptr, outer, inner, box_outer);
  auto it = g->cache.find(key);
  if (it != g->cache.end()) return &it->second;
  CUtensorMap m;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)outer};
  cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, (cuuint32_t)box_outer};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = g->encode(&m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, (void *)ptr, dims, strides, box, estr,
                         CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return nullptr;
  return &(g->cache[key] = m);
}

const CUtensorMap *fast_gemm_map(FastGemm *g, const void *ptr, int outer, int inner, int box_outer) {
  return get_map(g, ptr, outer, inner, box_outer);
}

void fast_gemm_forget(FastGemm *g) { g->cache.clear(); }

int fast_gemm_pick_split(int O, int I, int smax) {
  int tiles = (O + TILE_M - 1) / TILE_M, KB = (I + TILE_K - 1) / TILE_K;
  int want = (2 * 148 + tiles - 1) / tiles;          // aim at two resident CTAs per SM
  int S = std::min(want, std::max(1, KB / 4));       // keep at least 4 k-blocks per slice
  S = std::min(S, smax);
  return std::max(1, std::min(S, KB));
}

static int pick_nt(int rows) { return rows <= 16 ? 16 : rows <= 32 ? 32 : rows <= 64 ? 64 : rows <= 128 ? 128 : 256; }

template <int NT>
static int launch_nt(FastGemm *g, int slot, const CUtensorMap *mw, const CUtensorMap *mx, float *out, int rows, int O, int KB,
                     int S, int ldo, size_t pstride, int32_t *status, cudaStream_t s) {
  if (!g->attr_done[slot]) {
    if (cudaFuncSetAttribute(gemm_tcgen05_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, Cfg<NT>::SMEM) != cudaSuccess)
      return -6;
    g->attr_done[slot] = true;
  }
  dim3 grid((O + TILE_M - 1) / TILE_M, S);
  gemm_tcgen05_kernel<NT><<<grid, 128, Cfg<NT>::SMEM, s>>>(*mw, *mx, out, rows, O, KB, S, ldo, pstride, status);
  return 0;
}

int fast_gemm_run(FastGemm *g, const bf16 *x, const bf16 *w, float *out, int rows, int O, int I, int ldo, size_t pstride, int S,
                  int32_t *status, cudaStream_t s) {
  if (rows < 1 || rows > 256 || (I % 8) != 0 || ((uintptr_t)x & 15) || ((uintptr_t)w & 15)) return -1;
  int nt = pick_nt(rows), KB = (I + TILE_K - 1) / TILE_K;
  if (S < 1 || S > KB) return -1;
  const CUtensorMap *mw = get_map(g, w, O, I, TILE_M);
  const CUtensorMap *mx = get_map(g, x, rows, I, nt);
  if (!mw || !mx) return -6;
  switch (nt) {
    case 16: return launch_nt<16>(g, 0, mw, mx, out, rows, O, KB, S, ldo, pstride, status, s);
    case 32: return launch_nt<32>(g, 1, mw, mx, out, rows, O, KB, S, ldo, pstride, status, s);
    case 64: return launch_nt<64>(g, 2, mw, mx, out, rows, O, KB, S, ldo, pstride, status, s);
    case 128: return launch_nt<128>(g, 3, mw, mx, out, rows, O, KB, S, ldo, pstride, status, s);
    default: return launch_nt<256>(g, 4, mw, mx, out, rows, O, KB, S, ldo, pstride, status, s);
  }
}

size_t fast_gemm_scratch_bytes(int rows, int O, int I) {
  int S = fast_gemm_pick_split(O, I, 16);
  return S > 1 ? (size_t)S * rows * O * sizeof(float) + 64 : 64;
}

int fast_gemm_oneshot(const bf16 *x, const bf16 *w, float *out, int rows, int O, int I, int ldo, void *scratch, cudaStream_t s) {
  static FastGemm *g = nullptr;
  if (!g) {
    std::string why;
    g = fast_gemm_create(why);
    if (!g) return -6;
  }
  if (!scratch) return -2;
  int S = fast_gemm_pick_split(O, I, 16);
  int32_t *status = (int32_t *)scratch;              // first 64 bytes: status words
  float *parts = (float *)((char *)scratch + 64);
  cudaMemsetAsync(status, 0, 64, s);
  int rc;
  if (S == 1) {
    rc = fast_gemm_run(g, x, w, out, rows, O, I, ldo, 0, 1, status, s);
  } else {
    rc = fast_gemm_run(g, x, w, parts, rows, O, I, O, (size_t)rows * O, S, status, s);
    if (rc == 0) {
      size_t n = (size_t)rows * O;
      reduce_slices_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(parts, S, (size_t)rows * O, out, rows, O, ldo);
    }
  }
  g->cache.clear();   // test buffers come and go; do not keep descriptors of freed memory
  if (rc) return rc;
  return cudaGetLastError() == cudaSuccess ? 0 : -6;
}

}  // namespace spec
