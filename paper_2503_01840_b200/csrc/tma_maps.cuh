// Cache of TMA descriptors (CUtensorMap) for the bf16 operands of the tensor-core GEMMs: host-side interface.
#pragma once
#include <cuda.h>

#include <string>
#include "common.cuh"

namespace spec {

struct TmaMaps;   // one per context

TmaMaps *tma_maps_create(std::string &why);
void tma_maps_destroy(TmaMaps *);

// Cached descriptor of a bf16 matrix [outer][inner] (row pitch inner) with box [box_outer][64] and
// 128-byte swizzle; nullptr if the driver rejects it.
const CUtensorMap *tma_maps_get(TmaMaps *, const void *ptr, int outer, int inner, int box_outer);

// drops every cached descriptor (buffers of one-shot callers come and go)
void tma_maps_forget(TmaMaps *);

}  // namespace spec
