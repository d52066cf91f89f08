// The per-batch plan shared by the tensor-core kernels that add the LoRA term tile by tile: for every tile of 128
// consecutive tokens, the LoRA stages it needs, one per 32 ranks of every segment that overlaps the tile and carries
// a registered adapter.  A tile needs no alignment with the segments.
#pragma once
#include "pool.cuh"

namespace lora_plan {

constexpr int BM = 128;               // tokens per tile
constexpr int ER = 32;                // ranks per LoRA stage
constexpr int EXT_CAP = 2 * BM;       // LoRA stages a tile can need: every token another adapter of rank 64

struct PlanArgs {
  PoolView pv;
  const int32_t* seg_indptr;
  const int32_t* lora_ids;
  int n_seg, n_tokens, m_tiles;
  int n_mats;
  int mat_index[FL_MAX_MATS];
};

inline size_t plan_bytes(int n_tokens) {   // ext_count [m_tiles] + ext_list [m_tiles][EXT_CAP], both 256-byte aligned
  const size_t m_tiles = (size_t)(n_tokens + BM - 1) / BM;
  return ((sizeof(int) * m_tiles + 255) & ~(size_t)255) + ((sizeof(int) * m_tiles * EXT_CAP + 255) & ~(size_t)255);
}
inline int* plan_count(void* base) { return reinterpret_cast<int*>(base); }
inline int* plan_list(void* base, int n_tokens) {
  const size_t m_tiles = (size_t)(n_tokens + BM - 1) / BM;
  return reinterpret_cast<int*>(reinterpret_cast<unsigned char*>(base) + ((sizeof(int) * m_tiles + 255) & ~(size_t)255));
}

#ifdef __CUDACC__
// ext_list[m][e] = segment << 1 | which half of the ranks.
static __global__ void __launch_bounds__(128) plan_kernel(const PlanArgs a, int* __restrict__ ext_count, int* __restrict__ ext_list) {
  pdl_wait();
  pdl_launch_dependents();
  const int m = blockIdx.x * 128 + threadIdx.x;
  if (m >= a.m_tiles) return;
  const int tok0 = m * BM, tok1 = min(a.n_tokens, tok0 + BM);
  int lo = 0, hi = a.n_seg;          // first segment that ends behind tok0
  while (lo < hi) {
    const int mid = (lo + hi) >> 1;
    if (a.seg_indptr[mid + 1] > tok0) hi = mid; else lo = mid + 1;
  }
  int c = 0;
  for (int s = lo; s < a.n_seg && c + 2 <= EXT_CAP; ++s) {
    const int s0 = a.seg_indptr[s], s1 = a.seg_indptr[s + 1];
    if (s0 >= tok1) break;
    if (s1 <= s0 || s1 <= tok0) continue;
    const int lid = a.lora_ids[s];
    if (lid < 0) continue;
    bool ok = (uint32_t)lid < a.pv.dir_cap && a.pv.dir[lid].rank > 0;
    for (int j = 0; ok && j < a.n_mats; ++j) ok = a.mat_index[j] < a.pv.dir[lid].n_mats;
    if (!ok) {
      atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
      continue;
    }
    ext_list[(size_t)m * EXT_CAP + c++] = s << 1;
    if (a.pv.dir[lid].rank > ER) ext_list[(size_t)m * EXT_CAP + c++] = s << 1 | 1;
  }
  ext_count[m] = c;
}

inline cudaError_t launch_plan(const PlanArgs& a, int* ext_count, int* ext_list, cudaStream_t st) {
  return launch_pdl(plan_kernel, dim3((a.m_tiles + 127) / 128), dim3(128), 0, st, a, ext_count, ext_list);
}
#endif

}  // namespace lora_plan
