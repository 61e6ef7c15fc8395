// Plain tree-masked paged GQA attention (Section 2.2 "tree attention"): one CTA per (row, query head),
// two-pass softmax with the scores in shared memory.  Used by the fp32 model and as a debugging
// stand-in for the tensor-core kernel on bf16 models.
#include "common.cuh"

namespace spec {

template <typename T>
__global__ void __launch_bounds__(128) attn_ref_kernel(const T *__restrict__ q, KvPool pool, PageMap pm, RowMeta m,
                                                       int tail_len, T *__restrict__ out, int H, int G, int hd) {
  pdl_wait();
  pdl_trigger();
  extern __shared__ float smem[];
  float *qs = smem;            // [hd]
  float *sc = smem + hd;       // [ctx + tail_len]
  __shared__ float red[4];
  int r = blockIdx.x, h = blockIdx.y, g = h / (H / G);
  int seq = m.seq[r];
  T *o = out + ((size_t)r * H + h) * hd;
  if (seq < 0) {
    for (int i = threadIdx.x; i < hd; i += blockDim.x) o[i] = from_f32<T>(0.0f);
    return;
  }
  int ctx = m.ctx[r], tb = m.tail_base[r];
  uint64_t mlo = m.mask_lo[r], mhi = m.mask_hi[r];
  int nk = ctx + tail_len;
  const T *Kp = (const T *)pool.k, *Vp = (const T *)pool.v;
  for (int i = threadIdx.x; i < hd; i += blockDim.x) qs[i] = to_f32(q[((size_t)r * H + h) * hd + i]);
  __syncthreads();
  float scale = 1.0f / sqrtf((float)hd);
  float mx = -INFINITY;
  for (int j = threadIdx.x; j < nk; j += blockDim.x) {
    int pos;
    bool vis = true;
    if (j < ctx) pos = j;
    else {
      int t = j - ctx;
      vis = t < 64 ? ((mlo >> t) & 1ull) : ((mhi >> (t - 64)) & 1ull);
      pos = tb + t;
    }
    float s = -INFINITY;
    if (vis) {
      const T *kr = Kp + kv_offset(pm, seq, pos, g, G, hd);
      float d = 0.0f;
      for (int i = 0; i < hd; i++) d = fmaf(qs[i], to_f32(kr[i]), d);
      s = d * scale;
    }
    sc[j] = s;
    mx = fmaxf(mx, s);
  }
  for (int off = 16; off > 0; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
  __syncthreads();
  float sum = 0.0f;
  for (int j = threadIdx.x; j < nk; j += blockDim.x) {
    float e = (sc[j] == -INFINITY) ? 0.0f : expf(sc[j] - mx);
    sc[j] = e;
    sum += e;
  }
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = sum;
  __syncthreads();
  sum = red[0] + red[1] + red[2] + red[3];
  float inv = 1.0f / sum;
  for (int i = threadIdx.x; i < hd; i += blockDim.x) {
    float acc = 0.0f;
    for (int j = 0; j < nk; j++) {
      float p = sc[j];
      if (p == 0.0f) continue;
      int pos = j < ctx ? j : tb + (j - ctx);
      acc = fmaf(p, to_f32(Vp[kv_offset(pm, seq, pos, g, G, hd) + i]), acc);
    }
    o[i] = from_f32<T>(acc * inv);
  }
}

size_t attn_ref_smem_bytes(int max_keys, int hd) { return ((size_t)max_keys + hd) * sizeof(float); }

template <typename T>
void launch_attn_ref(const T *q, KvPool pool, PageMap pm, RowMeta m, int tail_len, T *out, int rows, int H, int G,
                     int hd, int max_keys, cudaStream_t s) {
  size_t smem = attn_ref_smem_bytes(max_keys, hd);
  static size_t configured[2] = {0, 0};
  int which = sizeof(T) == 4 ? 0 : 1;
  if (smem > 48 * 1024 && smem > configured[which]) {
    cudaFuncSetAttribute(attn_ref_kernel<T>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    configured[which] = smem;
  }
  launch_k(attn_ref_kernel<T>, dim3(rows, H), dim3(128), smem, s, q, pool, pm, m, tail_len, out, H, G, hd);
}
template void launch_attn_ref<float>(const float *, KvPool, PageMap, RowMeta, int, float *, int, int, int, int, int,
                                     cudaStream_t);
template void launch_attn_ref<bf16>(const bf16 *, KvPool, PageMap, RowMeta, int, bf16 *, int, int, int, int, int,
                                    cudaStream_t);

}  // namespace spec
