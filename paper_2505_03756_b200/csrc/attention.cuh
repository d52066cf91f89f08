// Declarations shared by the attention translation units.
#pragma once
#include "pool.cuh"

namespace attn {

constexpr int D = FL_HEAD_DIM;
constexpr int BT = 16;                 // tokens per block these kernels cover
constexpr int PAGE_BYTES = BT * D * 2;   // one (block, kv head, K or V) piece
constexpr int QT_MMA = 64;             // query rows per prefill tile, mma.sync kernel
constexpr int KT = 64;                 // keys per prefill iteration
constexpr int ATT_THREADS = 128;
constexpr int DEC_ROWS = 16;

struct PlanHdr {
  int n_prefill, n_decode, chunk;
  int next_unit;   // work counter of the persistent prefill kernel, zeroed by the plan kernel
};

struct AttnArgs {
  PoolView pv;
  __nv_bfloat16* out;
  const __nv_bfloat16* q;
  const int32_t* req_indptr;
  const int32_t* tbl_indptr;
  const uint32_t* tbl;
  const int32_t* prefix_lens;
  const int32_t* new_lens;
  int n_req, n_q, n_kv;
  float scale_log2;
  // workspace
  PlanHdr* hdr;
  int2* prefill_list;   // (request, first query token of the tile inside the request), longest requests first
  int2* decode_list;    // (request, chunk)
  int4* req_info;       // (first partial slot, chunks, decode?, 0)
  float* part_o;        // [slot][kv head][16 rows][128]
  float2* part_ml;      // [slot][kv head][16 rows] (running max in log2 units, sum)
  int max_prefill, max_decode;
};


// Launches the two-tiles-per-CTA kernel; the plan's tiles are tc2_tile_tokens(n_q, n_kv) tokens long.
int launch_prefill_tc2(fl_pool* p, const AttnArgs& a, int n_tokens, int max_items, cudaStream_t st);
inline int tc2_tile_tokens(int n_q, int n_kv) { return (n_q / n_kv) % 2 == 0 ? 128 : 256; }

}  // namespace attn
