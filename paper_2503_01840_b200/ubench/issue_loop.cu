// Cycle cost of the instructions of the GEMM main loop (barrier tests and waits, elect, commit, MMA issue at three tile
// widths, from an elected lane and from a lane-id branch), one warp of one CTA, zero operands in shared memory.  It is how
// the issue loop of gemm_fused.cu was sized; run it with  python -m paper_2503_01840_b200.ubench_issue
#include <cstdio>
#include <cstdint>
#include <cuda_runtime.h>
#include "../csrc/tcgen05_ptx.cuh"
using namespace spec::tc;
constexpr int IT = 64;
__global__ void __launch_bounds__(128) k(long long *out, int nt) {
  extern __shared__ __align__(1024) unsigned char sm[];
  unsigned char *tiles = (unsigned char *)(((uintptr_t)sm + 1023) & ~(uintptr_t)1023);
  uint64_t *bars = (uint64_t *)(tiles + 96 * 1024);
  uint32_t *slot = (uint32_t *)(bars + 8);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int i = threadIdx.x; i < 96 * 1024 / 4; i += 128) ((uint32_t *)tiles)[i] = 0;
  if (threadIdx.x == 0) { for (int i = 0; i < 8; i++) mbar_init(&bars[i], 1); asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(slot)), "r"(512) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tm = *slot;
  if (threadIdx.x == 0) { uint64_t st; asm volatile("mbarrier.arrive.shared::cta.b64 %0, [%1];" : "=l"(st) : "r"(smem_u32(&bars[0])) : "memory"); }   // bars[0]: phase 0 complete
  __syncthreads();
  if (warp == 1) {
    const uint64_t da = umma_desc_sw128(smem_u32(tiles)), db = umma_desc_sw128(smem_u32(tiles) + 16384);
    const uint32_t idesc = umma_idesc(nt);
    long long t[16];
    int n = 0;
    uint32_t acc = 0;
#define T0 { __syncwarp(); t[n] = clock64(); }
#define T1 { __syncwarp(); t[n] = clock64() - t[n]; n++; }
    T0 for (int i = 0; i < IT; i++) { acc += elect_one(); } T1                                  // 0 elect
    T0 for (int i = 0; i < IT; i++) { acc += __reduce_or_sync(0xffffffffu, acc + i); } T1       // 1 redux
    T0 for (int i = 0; i < IT; i++) { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); } T1   // 2 fence
    T0 for (int i = 0; i < IT; i++) { acc += mbar_wait(&bars[0], 0, 4) ? 1 : 0; } T1            // 3 try_wait (complete), all lanes
    T0 for (int i = 0; i < IT; i++) { uint32_t ok; asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}" : "=r"(ok) : "r"(smem_u32(&bars[0])), "r"(0) : "memory"); acc += ok; } T1   // 4 test_wait
    T0 for (int i = 0; i < IT; i++) { if (elect_one()) umma_commit(&bars[1 + (i & 3)]); } T1   // 5 commit (elected), nothing outstanding
    T0 for (int i = 0; i < IT; i++) { if (elect_one()) umma_bf16(tm, da, db, idesc, 1u); } T1   // 6 one MMA (elected)
    T0 for (int i = 0; i < IT; i++) { if (elect_one()) { umma_bf16(tm, da, db, idesc, 1u); umma_bf16(tm, da + 2, db + 2, idesc, 1u); umma_bf16(tm, da + 4, db + 4, idesc, 1u); umma_bf16(tm, da + 6, db + 6, idesc, 1u); } } T1   // 7 four MMAs
    T0 for (int i = 0; i < IT; i++) { if (elect_one()) { umma_bf16(tm, da, db, idesc, 1u); umma_bf16(tm, da + 2, db + 2, idesc, 1u); umma_bf16(tm, da + 4, db + 4, idesc, 1u); umma_bf16(tm, da + 6, db + 6, idesc, 1u); umma_commit(&bars[1 + (i & 3)]); } } T1   // 8 four MMAs + commit
    T0 for (int i = 0; i < IT; i++) { if (lane == 0) { umma_bf16(tm, da, db, idesc, 1u); umma_bf16(tm, da + 2, db + 2, idesc, 1u); umma_bf16(tm, da + 4, db + 4, idesc, 1u); umma_bf16(tm, da + 6, db + 6, idesc, 1u); umma_commit(&bars[1 + (i & 3)]); } } T1   // 9 the same from lane 0
    {   // two accumulators side by side (gate and up of one feature tile), alternating: 8 MMAs + commit per k-block
      T0 for (int i = 0; i < IT; i++) { if (elect_one()) { for (int j = 0; j < 4; j++) { umma_bf16(tm, da + 2 * j, db + 2 * j, idesc, 1u); umma_bf16(tm + nt, da + 2 * j + 512, db + 2 * j, idesc, 1u); } umma_commit(&bars[1 + (i & 3)]); } } T1
    }
    T0 for (int i = 0; i < IT; i++) { if (elect_one()) mbar_expect_tx(&bars[5], 0); } T1       // 10 arrive.expect_tx
    // wait until every MMA has completed before freeing tensor memory
    if (elect_one()) umma_commit(&bars[6]);
    __syncwarp();
    bool ok = mbar_wait(&bars[6], 0, 1u << 22);
    if (lane == 0) { for (int i = 0; i < n; i++) out[i] = t[i]; out[15] = acc + ok; }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tm), "r"(512) : "memory");
}
int main() {
  long long *d, h[16];
  cudaMalloc(&d, sizeof h);
  cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
  const char *names[] = {"elect", "redux", "tcgen05.fence", "bounded wait(done)", "test_wait(done)", "commit", "1 mma", "4 mma", "4 mma+commit", "same, lane 0 branch", "8 mma, two accumulators + commit", "arrive.expect_tx"};
  for (int nt : {16, 64, 256}) {
    for (int rep = 0; rep < 2; rep++) {
      cudaMemset(d, 0, sizeof h);
      k<<<1, 128, 100 * 1024>>>(d, nt);
      cudaError_t e = cudaDeviceSynchronize();
      if (e != cudaSuccess) { printf("error %s\n", cudaGetErrorString(e)); return 1; }
    }
    cudaMemcpy(h, d, sizeof h, cudaMemcpyDeviceToHost);
    printf("N=%d:", nt);
    for (int i = 0; i < 12; i++) printf("  %s %.0f", names[i], (double)h[i] / IT);
    printf("\n");
  }
  return 0;
}
