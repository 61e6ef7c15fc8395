// bf16 weight-streaming GEMM on the 5th-generation tensor cores (tcgen05.mma, TMEM accumulators,
// TMA-staged operands): host-side interface.
#pragma once
#include <cuda.h>

#include <string>
#include "common.cuh"

namespace spec {

struct FastGemm;   // caches TMA descriptors; one per context

FastGemm *fast_gemm_create(std::string &why);
void fast_gemm_destroy(FastGemm *);

// Cached TMA descriptor of a bf16 matrix [outer][inner] (row pitch inner) with box [box_outer][64] and
// 128-byte swizzle; nullptr if the driver rejects it.
const CUtensorMap *fast_gemm_map(FastGemm *, const void *ptr, int outer, int inner, int box_outer);

// drops every cached descriptor (buffers of one-shot callers come and go)
void fast_gemm_forget(FastGemm *);

// number of split-K slices for a [O][I] weight when at most smax slices fit the output buffer
int fast_gemm_pick_split(int O, int I, int smax);

// out[s][r][o] (fp32, slice stride pstride, row stride ldo) = partial sums over the s-th K range of
// x[r][:] . w[o][:].  x: [rows][I] bf16 (row pitch I), w: [O][I] bf16.  Returns 0 or a negative code.
int fast_gemm_run(FastGemm *, const bf16 *x, const bf16 *w, float *out, int rows, int O, int I, int ldo, size_t pstride,
                  int S, int32_t *status, cudaStream_t s);

// One-shot variant for tests: picks the split itself, reduces the slices into out (needs scratch of
// fast_gemm_scratch_bytes when more than one slice is used).
size_t fast_gemm_scratch_bytes(int rows, int O, int I);
int fast_gemm_oneshot(const bf16 *x, const bf16 *w, float *out, int rows, int O, int I, int ldo, void *scratch,
                      cudaStream_t s);

}  // namespace spec
