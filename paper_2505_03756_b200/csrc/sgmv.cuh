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

}  // namespace sgmv
