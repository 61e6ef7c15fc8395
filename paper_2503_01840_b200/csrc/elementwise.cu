// Elementwise / per-row kernels between the GEMMs: embedding gather, split-K reduction fused with
// residual add + RMSNorm (+ feature taps), RoPE + paged K/V write, SiLU*up, FC2 input assembly.
// All statistics and the residual stream are fp32; T is the storage type (fp32 or bf16).
#include "common.cuh"

namespace spec {

__device__ __forceinline__ float block_sum(float v, float *sh) {
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  int w = threadIdx.x >> 5, l = threadIdx.x & 31, nw = (blockDim.x + 31) >> 5;
  if (l == 0) sh[w] = v;
  __syncthreads();
  float t = (threadIdx.x < nw) ? sh[threadIdx.x] : 0.0f;
  if (w == 0) {
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    if (l == 0) sh[0] = t;
  }
  __syncthreads();
  t = sh[0];
  __syncthreads();
  return t;
}

// ---------------------------------------------------------------- embedding gather
template <typename T>
__global__ void embed_kernel(const T *__restrict__ embed, const int32_t *__restrict__ tok, float *__restrict__ x, int k) {
  pdl_wait();
  pdl_trigger();
  int r = blockIdx.x;
  const T *e = embed + (size_t)tok[r] * k;
  for (int i = threadIdx.x; i < k; i += blockDim.x) x[(size_t)r * k + i] = to_f32(e[i]);
}
template <typename T>
void launch_embed(const T *embed, const int32_t *tok, float *x, int rows, int k, cudaStream_t s) {
  launch_k(embed_kernel<T>, dim3(rows), dim3(256), 0, s, embed, tok, x, k);
}
template void launch_embed<float>(const float *, const int32_t *, float *, int, int, cudaStream_t);
template void launch_embed<bf16>(const bf16 *, const int32_t *, float *, int, int, cudaStream_t);

// ---------------------------------------------------------------- embedding gather feeding the fused GEMM path
// x = E[tok] (fp32 residual stream), hb = bf16(x * gain) (input of the first QKV GEMM, which applies
// the RMSNorm factor as a row scale), ssq[tile][row] = sum of x^2 over the tile's 128 features.
__global__ void embed_norm_kernel(const bf16 *__restrict__ embed, const int32_t *__restrict__ tok,
                                  const bf16 *__restrict__ gain, float *__restrict__ x, bf16 *__restrict__ hb,
                                  float *__restrict__ ssq, int k, int ssq_ld) {
  // The wait also orders this kernel's successors after its predecessor: the first QKV GEMM waits only for this
  // kernel and reads the RoPE table the kernel before it wrote.
  pdl_wait();
  pdl_trigger();
  __shared__ float sh[4];
  int r = blockIdx.x, tile = blockIdx.y, o = tile * 128 + threadIdx.x;
  float v = 0.0f;
  if (o < k) {
    v = __bfloat162float(embed[(size_t)tok[r] * k + o]);
    x[(size_t)r * k + o] = v;
    hb[(size_t)r * k + o] = __float2bfloat16_rn(v * __bfloat162float(gain[o]));
  }
  float sq = v * v;
  for (int off = 16; off > 0; off >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, off);
  if ((threadIdx.x & 31) == 0) sh[threadIdx.x >> 5] = sq;
  __syncthreads();
  if (threadIdx.x == 0) ssq[(size_t)tile * ssq_ld + r] = ((sh[0] + sh[1]) + sh[2]) + sh[3];
}
void launch_embed_norm(const bf16 *embed, const int32_t *tok, const bf16 *gain, float *x, bf16 *hb, float *ssq, int rows,
                       int k, int ssq_ld, cudaStream_t s) {
  launch_k(embed_norm_kernel, dim3(rows, (k + 127) / 128), dim3(128), 0, s, embed, tok, gain, x, hb, ssq, k, ssq_ld);
}

// ---------------------------------------------------------------- partial-sum reduce + residual + RMSNorm (+ taps)
template <typename T>
__global__ void add_norm_kernel(float *__restrict__ x, const float *__restrict__ parts, int nparts, size_t part_stride,
                                int mode, T *__restrict__ taps, int tap_mask, const T *__restrict__ gain, float eps,
                                T *__restrict__ h, int k) {
  pdl_wait();
  pdl_trigger();
  __shared__ float sh[32];
  int r = blockIdx.x;
  float *xr = x + (size_t)r * k;
  float ss = 0.0f;
  for (int i = threadIdx.x; i < k; i += blockDim.x) {
    float v = (mode == 1) ? 0.0f : xr[i];
    if (mode != 0)
      for (int p = 0; p < nparts; p++) v += parts[(size_t)p * part_stride + (size_t)r * k + i];
    if (mode != 0) xr[i] = v;
    if (taps) {
#pragma unroll
      for (int s = 0; s < 3; s++)
        if ((tap_mask >> s) & 1) taps[(size_t)r * 3 * k + (size_t)s * k + i] = from_f32<T>(v);
    }
    ss += v * v;
  }
  if (!gain) return;
  ss = block_sum(ss, sh);
  float inv = 1.0f / sqrtf(ss / (float)k + eps);
  for (int i = threadIdx.x; i < k; i += blockDim.x)
    h[(size_t)r * k + i] = from_f32<T>(xr[i] * inv * to_f32(gain[i]));
}
template <typename T>
void launch_add_norm(float *x, const float *parts, int nparts, size_t part_stride, int mode, T *taps, int tap_mask,
                     const T *gain, float eps, T *h, const int32_t *src_row, int rows_x, int rows_h, int k,
                     cudaStream_t s) {
  (void)src_row; (void)rows_h;
  launch_k(add_norm_kernel<T>, dim3(rows_x), dim3(256), 0, s, x, parts, nparts, part_stride, mode, tap_mask ? taps : nullptr, tap_mask,
                                           gain, eps, h, k);
}
template void launch_add_norm<float>(float *, const float *, int, size_t, int, float *, int, const float *, float,
                                     float *, const int32_t *, int, int, int, cudaStream_t);
template void launch_add_norm<bf16>(float *, const float *, int, size_t, int, bf16 *, int, const bf16 *, float, bf16 *,
                                    const int32_t *, int, int, int, cudaStream_t);

// ---------------------------------------------------------------- RoPE angles (double, rounded once)
__global__ void rope_table_kernel(const int32_t *__restrict__ pos, int rows, int half, const double *__restrict__ inv_freq,
                                  float2 *__restrict__ cs) {
  pdl_wait();
  pdl_trigger();
  int idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= rows * half) return;
  int r = idx / half, i = idx % half;
  double ang = (double)pos[r] * inv_freq[i];
  double sn, c;
  sincos(ang, &sn, &c);
  cs[idx] = make_float2((float)c, (float)sn);
}
void launch_rope_table(const int32_t *pos, int rows, int half, const double *inv_freq, float2 *cs, cudaStream_t s) {
  int n = rows * half;
  launch_k(rope_table_kernel, dim3((n + 255) / 256), dim3(256), 0, s, pos, rows, half, inv_freq, cs);
}

// ---------------------------------------------------------------- row metadata of one prefill pass
// Row r < nvalid is prompt position start + r of sequence b, fed with toks[r]; a pass is made of blocks of `block`
// positions: the rows of a block are each other's tail keys (causal through the two-word masks), everything before the
// block is context.  Rows >= nvalid are padding.
__global__ void prefill_meta_kernel(RowMeta m, const int32_t *__restrict__ toks, int b, int start, int nvalid, int block) {
  pdl_wait();
  pdl_trigger();
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  const bool v = r < nvalid;
  const int j = r % block;                           // position inside the block
  m.seq[r] = v ? b : -1;
  m.pos[r] = v ? start + r : 0;
  m.kvpos[r] = v ? start + r : 0;
  m.ctx[r] = v ? start + r - j : 0;
  m.tail_base[r] = v ? start + r - j : 0;
  m.tok[r] = v ? toks[r] : 0;
  m.mask_lo[r] = v ? (j >= 63 ? ~0ull : ((1ull << (j + 1)) - 1ull)) : 0ull;
  m.mask_hi[r] = (v && j >= 64) ? (j >= 127 ? ~0ull : ((1ull << (j - 63)) - 1ull)) : 0ull;
}
void launch_prefill_meta(RowMeta m, const int32_t *toks, int b, int start, int nvalid, int rows, int block, cudaStream_t s) {
  launch_k(prefill_meta_kernel, dim3(rows / 64), dim3(64), 0, s, m, toks, b, start, nvalid, block);
}

// ---------------------------------------------------------------- RoPE + q store + paged K/V write
template <typename T>
__global__ void rope_kv_kernel(const float *__restrict__ qkv, int nparts, size_t part_stride,
                               const float2 *__restrict__ cs, RowMeta m, T *__restrict__ q, KvPool pool, PageMap pm,
                               int H, int G, int hd, int32_t *status) {
  pdl_wait();
  pdl_trigger();
  int r = blockIdx.x;
  int seq = m.seq[r];
  int half = hd / 2, ld = (H + 2 * G) * hd;
  T *Kp = (T *)pool.k, *Vp = (T *)pool.v;
  if (seq < 0) {
    for (int i = threadIdx.x; i < H * hd; i += blockDim.x) q[(size_t)r * H * hd + i] = from_f32<T>(0.0f);
    return;
  }
  int kvpos = m.kvpos[r];
  if (kvpos < 0 || kvpos / pm.page_size >= pm.pages_per_seq) {
    if (threadIdx.x == 0) set_status(status, ST_BOUNDS, 1, r, kvpos);
    return;
  }
  int page = pm.table[(size_t)seq * pm.pages_per_seq + kvpos / pm.page_size];
  if (page < 0 || page >= pm.num_pages) {
    if (threadIdx.x == 0) set_status(status, ST_BOUNDS, 2, r, page);
    return;
  }
  const float *row = qkv + (size_t)r * ld;
  // rotated heads: H query heads then G key heads
  for (int idx = threadIdx.x; idx < (H + G) * half; idx += blockDim.x) {
    int hh = idx / half, i = idx % half;
    float a = 0.0f, b = 0.0f;
    for (int p = 0; p < nparts; p++) {
      a += row[(size_t)p * part_stride + hh * hd + i];
      b += row[(size_t)p * part_stride + hh * hd + i + half];
    }
    float2 c = cs[(size_t)r * half + i];
    float ra = a * c.x - b * c.y, rb = b * c.x + a * c.y;
    if (hh < H) {
      q[((size_t)r * H + hh) * hd + i] = from_f32<T>(ra);
      q[((size_t)r * H + hh) * hd + i + half] = from_f32<T>(rb);
    } else {
      size_t o = kv_offset(pm, seq, kvpos, hh - H, G, hd);
      Kp[o + i] = from_f32<T>(ra);
      Kp[o + i + half] = from_f32<T>(rb);
    }
  }
  for (int idx = threadIdx.x; idx < G * hd; idx += blockDim.x) {
    int g = idx / hd, i = idx % hd;
    float v = 0.0f;
    for (int p = 0; p < nparts; p++) v += row[(size_t)p * part_stride + (H + G) * hd + idx];
    Vp[kv_offset(pm, seq, kvpos, g, G, hd) + i] = from_f32<T>(v);
  }
}
template <typename T>
void launch_rope_kv(const float *qkv, int nparts, size_t part_stride, const float2 *cs, RowMeta m, T *q, KvPool pool,
                    PageMap pm, int rows, int H, int G, int hd, int32_t *status, cudaStream_t s) {
  launch_k(rope_kv_kernel<T>, dim3(rows), dim3(256), 0, s, qkv, nparts, part_stride, cs, m, q, pool, pm, H, G, hd, status);
}
template void launch_rope_kv<float>(const float *, int, size_t, const float2 *, RowMeta, float *, KvPool, PageMap, int,
                                    int, int, int, int32_t *, cudaStream_t);
template void launch_rope_kv<bf16>(const float *, int, size_t, const float2 *, RowMeta, bf16 *, KvPool, PageMap, int, int,
                                   int, int, int32_t *, cudaStream_t);

// ---------------------------------------------------------------- SwiGLU activation
template <typename T>
__global__ void silu_mul_kernel(const float *__restrict__ gu, int nparts, size_t part_stride, T *__restrict__ act,
                                int rows, int F) {
  pdl_wait();
  pdl_trigger();
  size_t idx = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (size_t)rows * F) return;
  size_t r = idx / F, f = idx % F;
  float g = 0.0f, u = 0.0f;
  for (int p = 0; p < nparts; p++) {
    g += gu[(size_t)p * part_stride + r * 2 * F + f];
    u += gu[(size_t)p * part_stride + r * 2 * F + F + f];
  }
  act[idx] = from_f32<T>((g / (1.0f + expf(-g))) * u);
}
template <typename T>
void launch_silu_mul(const float *gu, int nparts, size_t part_stride, T *act, int rows, int F, cudaStream_t s) {
  size_t n = (size_t)rows * F;
  launch_k(silu_mul_kernel<T>, dim3((unsigned)((n + 255) / 256)), dim3(256), 0, s, gu, nparts, part_stride, act, rows, F);
}
template void launch_silu_mul<float>(const float *, int, size_t, float *, int, int, cudaStream_t);
template void launch_silu_mul<bf16>(const float *, int, size_t, bf16 *, int, int, cudaStream_t);

// ---------------------------------------------------------------- FC2 input: [feature ; embedding]
template <typename T>
__global__ void build_cat_kernel(const float *__restrict__ feat, int nparts, size_t part_stride,
                                 const int32_t *__restrict__ src_row, const T *__restrict__ embed,
                                 const int32_t *__restrict__ tok, const int32_t *__restrict__ seq, T *__restrict__ cat,
                                 int k) {
  pdl_wait();
  pdl_trigger();
  // one element per thread (grid.y slices of the row): every load of the launch is in flight at once
  int r = blockIdx.x;
  int i = blockIdx.y * blockDim.x + threadIdx.x;
  if (i >= k) return;
  T *c = cat + (size_t)r * 2 * k;
  if (seq[r] < 0) {
    c[i] = from_f32<T>(0.0f);
    c[k + i] = from_f32<T>(0.0f);
    return;
  }
  int sr = src_row ? src_row[r] : r;
  T e = embed[(size_t)tok[r] * k + i];
  float v = 0.0f;
  for (int p = 0; p < nparts; p++) v += feat[(size_t)p * part_stride + (size_t)sr * k + i];
  c[i] = from_f32<T>(v);
  c[k + i] = e;
}
template <typename T>
void launch_build_cat(const float *feat, int nparts, size_t part_stride, const int32_t *src_row, const T *embed,
                      const int32_t *tok, const int32_t *seq, T *cat, int rows, int k, cudaStream_t s) {
  launch_k(build_cat_kernel<T>, dim3(rows, (k + 255) / 256), dim3(256), 0, s, feat, nparts, part_stride, src_row, embed, tok, seq, cat, k);
}
template void launch_build_cat<float>(const float *, int, size_t, const int32_t *, const float *, const int32_t *,
                                      const int32_t *, float *, int, int, cudaStream_t);
template void launch_build_cat<bf16>(const float *, int, size_t, const int32_t *, const bf16 *, const int32_t *,
                                     const int32_t *, bf16 *, int, int, cudaStream_t);

}  // namespace spec
