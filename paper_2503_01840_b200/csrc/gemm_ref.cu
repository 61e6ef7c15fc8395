// Plain CUDA-core GEMM: out[r][o] = sum_i x[r][i] * w[o][i], fp32 accumulation with FMA.
// This is the fp32 model's GEMM (tensor-core tf32 would not hold a 1e-4 bound) and a debugging
// stand-in for the tcgen05 kernel on bf16 models.
#include "common.cuh"

namespace spec {

template <typename T>
__global__ void __launch_bounds__(256) gemm_ref_kernel(const T *__restrict__ x, const T *__restrict__ w,
                                                       float *__restrict__ out, int rows, int O, int I, int ldo) {
  pdl_wait();
  pdl_trigger();
  constexpr int BM = 64, BN = 64, BK = 16;
  __shared__ float xs[BK][BM + 1];
  __shared__ float ws[BK][BN + 1];
  int r0 = blockIdx.y * BM, o0 = blockIdx.x * BN;
  int tx = threadIdx.x % 16, ty = threadIdx.x / 16;   // tx -> o, ty -> r
  float acc[4][4];
#pragma unroll
  for (int a = 0; a < 4; a++)
#pragma unroll
    for (int b = 0; b < 4; b++) acc[a][b] = 0.0f;
  for (int i0 = 0; i0 < I; i0 += BK) {
    for (int e = threadIdx.x; e < BM * BK; e += 256) {
      int rr = e / BK, kk = e % BK;
      int r = r0 + rr, i = i0 + kk;
      xs[kk][rr] = (r < rows && i < I) ? to_f32(x[(size_t)r * I + i]) : 0.0f;
      int o = o0 + rr;
      ws[kk][rr] = (o < O && i < I) ? to_f32(w[(size_t)o * I + i]) : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; kk++) {
      float xv[4], wv[4];
#pragma unroll
      for (int a = 0; a < 4; a++) xv[a] = xs[kk][ty * 4 + a];
#pragma unroll
      for (int b = 0; b < 4; b++) wv[b] = ws[kk][tx * 4 + b];
#pragma unroll
      for (int a = 0; a < 4; a++)
#pragma unroll
        for (int b = 0; b < 4; b++) acc[a][b] = fmaf(xv[a], wv[b], acc[a][b]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int a = 0; a < 4; a++) {
    int r = r0 + ty * 4 + a;
    if (r >= rows) continue;
#pragma unroll
    for (int b = 0; b < 4; b++) {
      int o = o0 + tx * 4 + b;
      if (o < O) out[(size_t)r * ldo + o] = acc[a][b];
    }
  }
}

template <typename T>
void launch_gemm_ref(const T *x, const T *w, float *out, int rows, int O, int I, int ldo, cudaStream_t s) {
  dim3 grid((O + 63) / 64, (rows + 63) / 64);
  launch_k(gemm_ref_kernel<T>, dim3(grid), dim3(256), 0, s, x, w, out, rows, O, I, ldo);
}
template void launch_gemm_ref<float>(const float *, const float *, float *, int, int, int, int, cudaStream_t);
template void launch_gemm_ref<bf16>(const bf16 *, const bf16 *, float *, int, int, int, int, cudaStream_t);

}  // namespace spec
