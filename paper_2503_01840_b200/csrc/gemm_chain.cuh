// Persistent chain of weight-streaming GEMMs: consecutive dependent GEMMs of a decoder layer (for example
// O-projection -> gate/up -> down -> next layer's QKV) run inside ONE kernel whose CTAs stay resident and
// keep streaming the next GEMM's weights while the current GEMM's results are being reduced: host-side interface.
#pragma once
#include "gemm_fused.cuh"

namespace spec {

constexpr int MAX_CHAIN_OPS = 4;   // keeps the kernel parameter block under 4 KB (the limit for launches captured into a CUDA graph)
constexpr int CHAIN_COUNTERS = 16;      // int32 words of grid-barrier counters one launch uses

// true when the chain kernel can run these ops (rows <= 64, every op supported by the fused GEMM, no argmax epilogue)
bool chain_supported(const FusedEpi *epi, const FusedGemmArgs *ops, int nops);
// bytes of fp32 scratch the launch needs for its split-K partial sums
size_t chain_scratch_bytes(const FusedEpi *epi, const FusedGemmArgs *ops, int nops);
// counters: CHAIN_COUNTERS zeroed int32 words owned by this launch (zeroed by the caller before the launch runs).
// meta / pm: row metadata and page map shared by the ops with an EPI_QKV epilogue.  Returns 0 or a negative code.
int chain_launch(FastGemm *g, const FusedEpi *epi, const FusedGemmArgs *ops, int nops, float *scratch, size_t scratch_bytes,
                 int32_t *counters, int32_t *status, bool pdl, cudaStream_t s, long long *timing = nullptr);
// CTAs of a chain launch
int chain_ctas();

}  // namespace spec
