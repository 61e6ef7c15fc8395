// Cache of TMA descriptors for the bf16 operands of the tensor-core GEMMs: 2-D tensors [outer][inner] read in boxes of
// [box_outer][64 elements] with the 128-byte swizzle that the tcgen05 shared-memory descriptors expect.
#include <cuda.h>

#include <map>
#include <string>
#include <tuple>

#include "tma_maps.cuh"
#include "tcgen05_ptx.cuh"

namespace spec {

using namespace tc;

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                             const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                             CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct TmaMaps {
  EncodeFn encode = nullptr;
  std::map<std::tuple<const void *, int, int, int>, CUtensorMap> cache;   // (ptr, outer, inner, box_outer)
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

TmaMaps *tma_maps_create(std::string &why) {
  EncodeFn f = get_encode(why);
  if (!f) return nullptr;
  TmaMaps *g = new TmaMaps();
  g->encode = f;
  return g;
}
void tma_maps_destroy(TmaMaps *g) { delete g; }

// 2D bf16 tensor [outer][inner] (row pitch inner), box [box_outer][64], 128-byte swizzle
static const CUtensorMap *get_map(TmaMaps *g, const void *ptr, int outer, int inner, int box_outer) {
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

const CUtensorMap *tma_maps_get(TmaMaps *g, const void *ptr, int outer, int inner, int box_outer) {
  return get_map(g, ptr, outer, inner, box_outer);
}

void tma_maps_forget(TmaMaps *g) { g->cache.clear(); }

}  // namespace spec
