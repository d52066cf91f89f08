// The shrink half of the segmented LoRA projection, for kernels that consume its partial sums themselves.
#pragma once
#include "pool.cuh"

namespace sgmv {

struct ShrinkInfo {
  int ksplit;   // slices of d_in whose partial sums have to be added
  int rmax;     // row pitch of the partial sums (16, 32 or 64: the pool's highest rank rounded up)
};

// v = x A_i per segment for the listed projections (which share x), unscaled fp32 partial sums written to
// workspace as [projection][slice][token][rmax]; workspace sized by fl_lora_sgmv_workspace(n_tokens, n_mats).
// Rows of segments without an adapter are left untouched.
int shrink(fl_pool* p, const fl_bf16* x, const int* mat_indices, int n_mats, const int32_t* seg_indptr,
           const int32_t* lora_ids, int n_seg, int n_tokens, void* workspace, size_t workspace_bytes, fl_stream stream,
           ShrinkInfo* info);


#ifdef __CUDACC__
// Token tile `tile` (tiles of TM tokens, counted over segments that carry an adapter, or over all segments) -> segment and
// token range.  Every warp evaluates it redundantly with a warp scan over 32 segments at a time.
template <int TM>
__device__ __forceinline__ bool find_tile(const int32_t* __restrict__ seg_indptr, const int32_t* __restrict__ lora_ids,
                                          int n_seg, int tile, int& seg, int& tok0, int& tok1, bool all_segments = false) {
  const int lane = threadIdx.x & 31;
  int base = 0;
  for (int s0 = 0; s0 < n_seg; s0 += 32) {
    const int s = s0 + lane;
    int lo = 0, hi = 0, nt = 0;
    if (s < n_seg) {
      lo = seg_indptr[s];
      hi = seg_indptr[s + 1];
      if ((all_segments || lora_ids[s] >= 0) && hi > lo) nt = (hi - lo + TM - 1) / TM;
    }
    int incl = nt;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int o = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += o;
    }
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    if (tile < base + total) {
      const int first = base + incl - nt;
      const bool mine = nt > 0 && tile >= first && tile < first + nt;
      const int src = __ffs(__ballot_sync(0xffffffffu, mine)) - 1;
      const int k = tile - __shfl_sync(0xffffffffu, first, src);
      seg = s0 + src;
      tok0 = __shfl_sync(0xffffffffu, lo, src) + k * TM;
      tok1 = min(tok0 + TM, __shfl_sync(0xffffffffu, hi, src));
      return true;
    }
    base += total;
  }
  return false;
}

// Start of rank-row `row` of a stream (class table entry tab, first row row0, rows per block rpb, row width).
__device__ __forceinline__ const unsigned char* lora_row(const PoolView& pv, uint32_t table_off, uint32_t tab,
                                                         uint32_t row0, uint32_t rpb, int width, int row, bool& ok) {
  const uint32_t g = row0 + (uint32_t)row;
  const uint32_t blk = pv.tables[table_off + tab + g / rpb];
  if (blk >= pv.n_blocks) {
    atomicOr(pv.flags, (uint32_t)FLAG_BAD_BLOCK);
    ok = false;
    return pv.slab;
  }
  ok = true;
  return pv.slab + (size_t)blk * pv.block_bytes + (size_t)(g % rpb) * 2 * (size_t)width;
}

#endif

// The same shrink on the 5th-generation tensor cores for long segments (tiles of 128 tokens, x by TMA, adapter rows
// by cp.async, accumulator in TMEM); same scratch layout.  Returns FL_EINVAL when it does not cover the case
// (the caller then takes the mma.sync kernels).
struct TcShrinkArgs {
  PoolView pv;
  float* v;
  int ksplit, n_mats;
  int mat_index[3];
  const int32_t* seg_indptr;
  const int32_t* lora_ids;
  int n_seg, n_tokens, d_in;
};
int shrink_tc(fl_pool* p, const TcShrinkArgs& a, const void* x, int rmax, cudaStream_t st);

}  // namespace sgmv
