// Tensor maps (TMA descriptors) of the pool slab and of caller tensors, encoded through the driver entry
// point so that the library links against the runtime only.
#pragma once
#include <cuda.h>
#include <stdint.h>
#include "pool.cuh"

namespace tmap {

// A bf16 tensor of `rank` dimensions (innermost first), `strides_bytes` for dimensions 1 .. rank-1, box in
// elements; 128-byte swizzle (the innermost box extent is at most 64 elements).  Returns FL_OK or FL_ECUDA.
int encode_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box);

// The slab as [block][K|V x kv head][token][128] with a box of one 16-token page of one plane (4 KiB), laid out in
// shared memory as [8-token group][64-value half][8 tokens][64 values] (cached in the pool, keyed by the KV head count).
int kv_pages(fl_pool* p, int n_kv, const CUtensorMap** out);

}  // namespace tmap
