// Shared declarations of the speculative-step library: dtype helpers, per-row metadata, the
// device-side state block and the launchers each .cu file exports to the step scheduler.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace spec {

typedef __nv_bfloat16 bf16;

__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// Device status words: [0] error code (0 = fine), [1] where, [2..3] detail.
enum { ST_OK = 0, ST_CAPACITY = 1, ST_BOUNDS = 2, ST_TIMEOUT = 3 };
__device__ __forceinline__ void set_status(int32_t *st, int code, int where, int a = 0, int b = 0) {
  if (atomicCAS(st, 0, code) == 0) { st[1] = where; st[2] = a; st[3] = b; }
}

// "a before b" in (value desc, index asc) order: the tie-break of every argmax / top-k of the step
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) { return va > vb || (va == vb && ia < ib); }

// Order-preserving map of a float to an unsigned key (larger float = larger key; -0 is folded into +0 first, so equal
// floats give equal keys) and back: lets a warp pick its best (value desc, index asc) entry with two redux instructions
// instead of a five-step shuffle tree.
__device__ __forceinline__ unsigned ordered_key(float v) {
  const unsigned u = __float_as_uint(v + 0.0f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_value(unsigned k) { return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k); }
// Best (key desc, index asc) over the warp; idx < 0 marks a lane without an entry.  Returns the winning index (-1: none)
// and its key through *key.
__device__ __forceinline__ int warp_best(unsigned key_in, int idx, unsigned *key) {
  const unsigned k = idx >= 0 ? key_in : 0u;             // real keys are >= 1 (the key of -inf is 0x007fffff)
  const unsigned m = __reduce_max_sync(0xffffffffu, k);
  const unsigned cand = (idx >= 0 && k == m) ? (unsigned)idx : 0xffffffffu;
  const unsigned w = __reduce_min_sync(0xffffffffu, cand);
  *key = m;
  return w == 0xffffffffu ? -1 : (int)w;
}

// Programmatic dependent launch: a kernel launched with the attribute may start while its predecessor
// on the stream is still running; everything it reads that the predecessor wrote must come after
// pdl_wait().  Both instructions do nothing in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Profiling aid: the GPU's global nanosecond timer, and a guard that records into stamp[0] the earliest time a CTA
// of the launch got past its dependency wait and into stamp[1] the bitwise complement of the latest time a warp of
// the launch left the kernel (early returns included), so that both slots start from all ones and are updated with
// atomicMin.  A null pointer switches it off.
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
struct KernelStamp {
  unsigned long long *p;
  __device__ __forceinline__ KernelStamp(unsigned long long *stamp, bool start = true) : p(stamp) {
    if (p && start && threadIdx.x == 0) atomicMin(p, global_ns());
  }
  __device__ __forceinline__ ~KernelStamp() {
    if (p && (threadIdx.x & 31) == 0) atomicMin(p + 1, ~global_ns());
  }
};

// When set (per host thread, by the step scheduler), launch_k adds the programmatic-dependent-launch
// attribute to every launch.
extern thread_local bool tl_pdl;
// Debugging aid: when >= 0, the number of kernel launches still allowed on this host thread; further
// launches are dropped (lets a test look at intermediate buffers after the n-th kernel of a step).
extern thread_local int tl_launch_budget;
inline bool launch_allowed() {
  if (tl_launch_budget < 0) return true;
  if (tl_launch_budget == 0) return false;
  tl_launch_budget--;
  return true;
}

template <typename... KArgs, typename... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
  if (!launch_allowed()) return cudaSuccess;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = tl_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// Kernel function attributes belong to one device: remembers, per device ordinal, the largest dynamic
// shared-memory size a kernel has been configured with, and raises the limit on the current device when needed.
struct SmemLimit {
  int have[64] = {};
  template <typename F> bool ensure(F kern, int smem) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64 && smem <= have[dev]) return true;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess) return false;
    if (dev >= 0 && dev < 64) have[dev] = smem;
    return true;
  }
};

// Per-row description of one forward pass (draft extend, draft tree pass, target verify).  A row
// attends cache positions [0, ctx) unmasked, then "tail" positions tail_base + t for every set bit t
// of (mask_lo, mask_hi); it writes its own K/V at cache position kvpos and is rotated by pos.
struct RowMeta {
  int32_t *seq;        // sequence id, -1 = padding row
  int32_t *pos;        // RoPE position
  int32_t *kvpos;      // cache position of this row's K/V
  int32_t *ctx;        // unmasked context length
  int32_t *tail_base;
  uint64_t *mask_lo, *mask_hi;
  int32_t *tok;        // token id whose embedding this row consumes
};

// Paged KV pool of one layer: [num_pages][G][page_size][hd]
struct KvPool {
  void *k, *v;
};

struct PageMap {
  const int32_t *table;    // [batch][pages_per_seq]
  int32_t pages_per_seq, page_size, num_pages;
};

__device__ __forceinline__ size_t kv_offset(const PageMap &pm, int seq, int pos, int g, int G, int hd) {
  int page = pm.table[(size_t)seq * pm.pages_per_seq + pos / pm.page_size];
  return (((size_t)page * G + g) * pm.page_size + (pos % pm.page_size)) * hd;
}

// ---------------------------------------------------------------- launchers (elementwise.cu)
template <typename T>
void launch_embed(const T *embed, const int32_t *tok, float *x, int rows, int k, cudaStream_t s);

// fused-path embedding: x = E[tok], hb = bf16(x * gain), ssq[tile][row] = per-128-feature sums of x^2
void launch_embed_norm(const bf16 *embed, const int32_t *tok, const bf16 *gain, float *x, bf16 *hb, float *ssq, int rows,
                       int k, int ssq_ld, cudaStream_t s);

// x (+)= sum of `nparts` partial slices [nparts][rows][k]; optional taps (T, [rows][3k], slots by bitmask);
// optional h[r] = rmsnorm(x[src_row ? src_row[r] : r]) * gain.  mode: 0 keep x, 1 x = parts, 2 x += parts.
template <typename T>
void launch_add_norm(float *x, const float *parts, int nparts, size_t part_stride, int mode, T *taps, int tap_mask,
                     const T *gain, float eps, T *h, const int32_t *src_row, int rows_x, int rows_h, int k,
                     cudaStream_t s);

// row metadata of one prefill pass of `rows` rows (a multiple of 64): nvalid prompt positions from `start` of sequence b,
// tokens toks[0..nvalid) (device), causal blocks of `block` positions
void launch_prefill_meta(RowMeta m, const int32_t *toks, int b, int start, int nvalid, int rows, int block, cudaStream_t s);

void launch_rope_table(const int32_t *pos, int rows, int half, const double *inv_freq, float2 *cs, cudaStream_t s);

// qkv partial sums [nparts][rows][(H+2G)hd] fp32 -> q (T, [rows][H][hd], rotated) and K/V written into the
// paged pool at kvpos (K rotated).
template <typename T>
void launch_rope_kv(const float *qkv, int nparts, size_t part_stride, const float2 *cs, RowMeta m, T *q, KvPool pool,
                    PageMap pm, int rows, int H, int G, int hd, int32_t *status, cudaStream_t s);

template <typename T>
void launch_silu_mul(const float *gu, int nparts, size_t part_stride, T *act, int rows, int F, cudaStream_t s);

// cat[r] = [ T(feat[src_row[r]]) ; embed[tok[r]] ], feat = sum of partial slices (fp32)
template <typename T>
void launch_build_cat(const float *feat, int nparts, size_t part_stride, const int32_t *src_row, const T *embed,
                      const int32_t *tok, const int32_t *seq, T *cat, int rows, int k, cudaStream_t s);

// ---------------------------------------------------------------- launchers (gemm_ref.cu)
template <typename T>
void launch_gemm_ref(const T *x, const T *w, float *out, int rows, int O, int I, int ldo, cudaStream_t s);

// ---------------------------------------------------------------- launchers (attn_ref.cu)
template <typename T>
void launch_attn_ref(const T *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, T *out, int rows, int H, int G,
                     int hd, int max_keys, cudaStream_t s);
size_t attn_ref_smem_bytes(int max_keys, int hd);

// ---------------------------------------------------------------- launchers (tree.cu)
void launch_logsoftmax_topk(const float *logits, int rows, int n, int K, int32_t *idx, float *lp, cudaStream_t s);
void launch_argmax(const float *logits, int rows, int n, int32_t *idx, cudaStream_t s);
// two-stage log-softmax + top-K (chunk candidates, then a per-row merge); scratch of topk_scratch_bytes
size_t topk_scratch_bytes(int rows, int n, int K);
int launch_topk2(const float *logits, const int32_t *src_row, int rows, int n, int K, int32_t *idx, float *lp, void *scratch,
                 cudaStream_t s);
// y[r] = best index over per-tile (value, index) candidates [tiles][ld]
void launch_argmax_merge(const float *best_val, const int32_t *best_idx, int tiles, int ld, int rows, int32_t *out,
                         cudaStream_t s);

}  // namespace spec
