// Tensor-map encoding shared by the TMA-fed kernels.
#include <stdlib.h>
#include "tmap.cuh"

namespace tmap {
namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

struct KvCache {
  int n_kv;
  CUtensorMap kv;
};

}  // namespace

int encode_bf16(CUtensorMap* out, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                const uint32_t* box) {
  EncodeTiledFn enc = encode_fn();
  if (!enc || rank < 1 || rank > 5) return FL_ECUDA;
  cuuint64_t d[5], s[4];
  cuuint32_t b[5], es[5];
  for (int i = 0; i < rank; ++i) {
    d[i] = dims[i];
    b[i] = box[i];
    es[i] = 1;
    if (i + 1 < rank) s[i] = strides_bytes[i];
  }
  if (enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), d, s, b, es,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return FL_ECUDA;
  return FL_OK;
}

int kv_pages(fl_pool* p, int n_kv, const CUtensorMap** out) {
  KvCache* tc = reinterpret_cast<KvCache*>(p->tmap_cache);
  if (!tc || tc->n_kv != n_kv) {
    if (!tc) {
      if (posix_memalign(reinterpret_cast<void**>(&tc), 64, sizeof(KvCache)) != 0) return FL_ENOMEM;
      tc->n_kv = -1;
      p->tmap_cache = tc;
    }
    // One box = K (or V) of one head of one block, 16 tokens x 128 values = 4 KiB, written to shared memory as
    // [8-token group][64-value half][token][64 values]: coordinates {value, token in group, half, 2 KiB chunk of the
    // block, block}; a chunk is one 8-token group of one (K|V, head) plane.
    const uint64_t dims[5] = {64, 8, 2, (uint64_t)(4 * n_kv), (uint64_t)p->n_blocks};
    const uint64_t strides[4] = {(uint64_t)FL_HEAD_DIM * 2, 128, (uint64_t)8 * FL_HEAD_DIM * 2, (uint64_t)p->block_bytes};
    const uint32_t box[5] = {64, 8, 2, 2, 1};
    tc->n_kv = -1;
    if (encode_bf16(&tc->kv, p->slab, 5, dims, strides, box) != FL_OK) return FL_ECUDA;
    tc->n_kv = n_kv;
  }
  *out = &tc->kv;
  return FL_OK;
}

}  // namespace tmap
