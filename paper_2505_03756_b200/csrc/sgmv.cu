// Segmented LoRA projection y += scale * (x A_i) B_i over adapter rank-rows stored in pool blocks
// (Eq. 1, Eq. 2; the segmented batching of Section 2.1).
//
// Two kernels.  shrink: v = x A_i for a tile of tokens of one segment and a slice of d_in, adapter
// rows fetched through the adapter's block table with 16-byte cp.async, bf16 mma.sync with fp32
// accumulation, partial sums written to scratch [mat][k-slice][token][RMAX].  expand: sums the
// partials, scales, rounds v to bf16, multiplies by the B rows of a column range (fp32 accumulation),
// rounds that LoRA term to bf16 into a tile of its own and adds it to the staged y rows with packed
// bf16 adds while the rows go out as coalesced 16-byte stores: y_out = rn(y + rn(term)).  The term is a
// small correction of y, so its own 2^-9 roundings stay far below y's final rounding.  Both kernels are
// bound by memory traffic (x and y rows for long segments, adapter rows for decode-sized segments) and by
// the instructions spent per byte, not by the contraction.
#include <algorithm>
#include "mma_utils.cuh"
#include "pool.cuh"
#include "sgmv.cuh"

namespace {

using sgmv::find_tile;
using sgmv::lora_row;

constexpr int SG_THREADS = 128;
constexpr int KS = 64;            // d_in elements per shrink pipeline stage (128-byte rows)
constexpr int SH_STAGES = 4;
constexpr int NSUB = 128;         // y columns per expand sub-tile (256-byte rows)
constexpr int EXPAND_COLS_MIN = 512, EXPAND_COLS_MAX = 2048;   // y columns per expand CTA: picked per call
constexpr int KSPLIT_MAX = 8;

struct SgmvArgs {
  PoolView pv;
  const __nv_bfloat16* x;
  __nv_bfloat16* y[FL_MAX_MATS];
  int mat_index[FL_MAX_MATS];
  int n_mats;
  const int32_t* seg_indptr;
  const int32_t* lora_ids;
  int n_seg, n_tokens;
  float scale;
  float* v;        // [n_mats][ksplit][n_tokens][RMAX]
  int ksplit;
  int tc_ksplit;     // slices of d_in for the tcgen05 shrink of long segments (0 = not applicable)
  int expand_cols;   // y columns one expand CTA covers
  int d_out[FL_MAX_MATS];
  // K / V projections whose result goes straight into the requests' pool blocks instead of back into y
  // (kv_side[j] = 0: K, 1: V, -1: y updated in place); then segments without an adapter are tiled too
  int kv_side[FL_MAX_MATS];
  int all_segments;
  const int32_t* req_indptr;
  const int32_t* tbl_indptr;
  const uint32_t* tbl;
  const int32_t* prefix_lens;
  int n_req, n_kv, bt;
};

// Eight bf16 sums (round to nearest even each) of two 16-byte chunks.
__device__ __forceinline__ uint4 add_bf16x8(uint4 a, uint4 b) {
  uint4 r;
  const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
  const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
  __nv_bfloat162* pr = reinterpret_cast<__nv_bfloat162*>(&r);
#pragma unroll
  for (int i = 0; i < 4; ++i) pr[i] = __hadd2(pa[i], pb[i]);
  return r;
}

template <int TM, int RMAX>
__global__ void __launch_bounds__(SG_THREADS) sgmv_shrink_kernel(const SgmvArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  pdl_wait();                 // x may come from the kernel right before this one
  pdl_launch_dependents();    // the expand may start its look-ups and first loads while this grid drains
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int j = blockIdx.x % a.n_mats;
  const int tile = blockIdx.x / a.n_mats;
  const int split = blockIdx.y;
  int seg, tok0, tok1;
  if (!find_tile<TM>(a.seg_indptr, a.lora_ids, a.n_seg, tile, seg, tok0, tok1, a.all_segments != 0)) return;
  const int lid = a.lora_ids[seg];
  if (lid < 0) return;
  if ((uint32_t)lid >= a.pv.dir_cap || a.pv.dir[lid].rank <= 0 || a.mat_index[j] >= a.pv.dir[lid].n_mats) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
    return;
  }
  const LoraEntry* e = a.pv.dir + lid;
  const LoraMat lm = e->mats[a.mat_index[j]];
  const int rank = min(e->rank, RMAX);
  // an adapter of a higher rank than this instantiation covers (registered after the launch was recorded
  // into a graph): its extra rank-rows are left out, and the status word says so
  if (e->rank > RMAX && tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
  const uint32_t table_off = e->table_off;
  const int d_in = lm.d_in;
  const int kchunk = ((d_in + a.ksplit * KS - 1) / (a.ksplit * KS)) * KS;
  const int kb = split * kchunk, ke = min(d_in, kb + kchunk);
  const int n_it = ke > kb ? (ke - kb + KS - 1) / KS : 0;

  constexpr int XR = TM / 16;      // x rows per thread per stage
  constexpr int AR = RMAX / 16;    // adapter rows per thread per stage
  constexpr int STAGE_BYTES = (TM + RMAX) * 128;
  const int crow = tid >> 3, cchunk = tid & 7;
  const __nv_bfloat16* xrow[XR];
  bool xok[XR];
#pragma unroll
  for (int i = 0; i < XR; ++i) {
    const int t = tok0 + crow + 16 * i;
    xok[i] = t < tok1;
    xrow[i] = a.x + (size_t)(xok[i] ? t : tok0) * d_in;
  }
  const __nv_bfloat16* arow[AR];
  bool aok[AR];
#pragma unroll
  for (int i = 0; i < AR; ++i) {
    const int r = crow + 16 * i;
    aok[i] = false;
    arow[i] = reinterpret_cast<const __nv_bfloat16*>(a.pv.slab);
    if (r < rank)
      arow[i] = reinterpret_cast<const __nv_bfloat16*>(
          lora_row(a.pv, table_off, lm.a_tab, lm.a_row0, lm.a_rpb, d_in, r, aok[i]));
  }
  const uint32_t sbase = smem_u32(smem);
  auto load_stage = [&](int it, int st) {
    const int kk = kb + it * KS + cchunk * 8;
    const bool kok = kk < ke;
    const uint32_t xs = sbase + st * STAGE_BYTES, as = xs + TM * 128;
#pragma unroll
    for (int i = 0; i < XR; ++i) cp_async16(xs + swz(crow + 16 * i, cchunk, 8), xrow[i] + kk, xok[i] && kok);
#pragma unroll
    for (int i = 0; i < AR; ++i) cp_async16(as + swz(crow + 16 * i, cchunk, 8), arow[i] + kk, aok[i] && kok);
  };

  float acc[RMAX / 8][4];
#pragma unroll
  for (int n = 0; n < RMAX / 8; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;

#pragma unroll
  for (int s = 0; s < SH_STAGES - 1; ++s) {
    if (s < n_it) load_stage(s, s);
    cp_async_commit();
  }
  const int mrow = (TM == 64 ? warp * 16 : 0) + (lane & 7) + 8 * ((lane >> 3) & 1);
  for (int it = 0; it < n_it; ++it) {
    cp_async_wait<SH_STAGES - 2>();
    __syncthreads();
    if (it + SH_STAGES - 1 < n_it) load_stage(it + SH_STAGES - 1, (it + SH_STAGES - 1) % SH_STAGES);
    cp_async_commit();
    const uint32_t xs = sbase + (it % SH_STAGES) * STAGE_BYTES, as = xs + TM * 128;
#pragma unroll
    for (int ks = 0; ks < KS / 16; ++ks) {
      if (TM == 16 && ks != warp) continue;   // short tiles: the four warps split each stage along k
      uint32_t af[4];
      ldmatrix_x4(af, xs + swz(mrow, 2 * ks + (lane >> 4), 8));
#pragma unroll
      for (int p = 0; p < RMAX / 16; ++p) {
        if (16 * p < rank) {
          uint32_t bf[4];
          ldmatrix_x4(bf, as + swz(16 * p + (lane & 7) + 8 * (lane >> 4), 2 * ks + ((lane >> 3) & 1), 8));
          mma_bf16(acc[2 * p], af, bf[0], bf[1]);
          mma_bf16(acc[2 * p + 1], af, bf[2], bf[3]);
        }
      }
    }
  }
  float* vout = a.v + ((size_t)(j * a.ksplit + split) * a.n_tokens) * RMAX;
  const int g = lane >> 2, t4 = lane & 3;
  if (TM == 64) {
#pragma unroll
    for (int n = 0; n < RMAX / 8; ++n) {
      const int r0 = tok0 + warp * 16 + g;
      if (r0 < tok1) *reinterpret_cast<float2*>(vout + (size_t)r0 * RMAX + 8 * n + 2 * t4) = make_float2(acc[n][0], acc[n][1]);
      if (r0 + 8 < tok1) *reinterpret_cast<float2*>(vout + (size_t)(r0 + 8) * RMAX + 8 * n + 2 * t4) = make_float2(acc[n][2], acc[n][3]);
    }
  } else {
    cp_async_wait<0>();
    __syncthreads();
    float* red = reinterpret_cast<float*>(smem);   // [4 warps][16 rows][RMAX]
#pragma unroll
    for (int n = 0; n < RMAX / 8; ++n) {
      float* r = red + (warp * 16 + g) * RMAX + 8 * n + 2 * t4;
      r[0] = acc[n][0]; r[1] = acc[n][1];
      r[8 * RMAX] = acc[n][2]; r[8 * RMAX + 1] = acc[n][3];
    }
    __syncthreads();
    for (int i = tid; i < 16 * RMAX; i += SG_THREADS) {
      const int row = i / RMAX;
      if (tok0 + row < tok1)
        vout[(size_t)(tok0 + row) * RMAX + (i % RMAX)] =
            red[i] + red[16 * RMAX + i] + red[32 * RMAX + i] + red[48 * RMAX + i];
    }
  }
}

// The shrink of three projections that share x (q, k, v) for long segments and ranks up to 16: one CTA stages each x tile once and
// multiplies it by the three adapters' rank-rows, instead of three CTAs reading the same x rows.  With long
// segments the shrink is bound by the traffic from L2 into shared memory, and x is most of it.
template <int RMAX>
__global__ void __launch_bounds__(SG_THREADS) sgmv_shrink3_kernel(const SgmvArgs a) {
  constexpr int TM = 64, NM = 3;
  constexpr int STAGES = RMAX == 64 ? 3 : 4;
  extern __shared__ __align__(128) unsigned char smem[];
  pdl_wait();                 // x may come from the kernel right before this one
  pdl_launch_dependents();    // the expand may start its look-ups and first loads while this grid drains
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int tile = blockIdx.x, split = blockIdx.y;
  int seg, tok0, tok1;
  if (!find_tile<TM>(a.seg_indptr, a.lora_ids, a.n_seg, tile, seg, tok0, tok1, a.all_segments != 0)) return;
  const int lid = a.lora_ids[seg];
  if (lid < 0) return;
  if ((uint32_t)lid >= a.pv.dir_cap || a.pv.dir[lid].rank <= 0) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
    return;
  }
  const LoraEntry* e = a.pv.dir + lid;
  for (int m = 0; m < NM; ++m) {
    if (a.mat_index[m] >= e->n_mats) {
      if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
      return;
    }
  }
  const int rank = min(e->rank, RMAX);
  // an adapter of a higher rank than this instantiation covers (registered after the launch was recorded
  // into a graph): its extra rank-rows are left out, and the status word says so
  if (e->rank > RMAX && tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
  const uint32_t table_off = e->table_off;
  const int d_in = e->mats[a.mat_index[0]].d_in;
  const int kchunk = ((d_in + a.ksplit * KS - 1) / (a.ksplit * KS)) * KS;
  const int kb = split * kchunk, ke = min(d_in, kb + kchunk);
  const int n_it = ke > kb ? (ke - kb + KS - 1) / KS : 0;

  constexpr int XR = TM / 16, AR = RMAX / 16;
  constexpr int STAGE_BYTES = (TM + NM * RMAX) * 128;
  const int crow = tid >> 3, cchunk = tid & 7;
  const __nv_bfloat16* xrow[XR];
  bool xok[XR];
#pragma unroll
  for (int i = 0; i < XR; ++i) {
    const int t = tok0 + crow + 16 * i;
    xok[i] = t < tok1;
    xrow[i] = a.x + (size_t)(xok[i] ? t : tok0) * d_in;
  }
  const __nv_bfloat16* arow[NM][AR];
  bool aok[NM][AR];
#pragma unroll
  for (int m = 0; m < NM; ++m) {
    const LoraMat lm = e->mats[a.mat_index[m]];
#pragma unroll
    for (int i = 0; i < AR; ++i) {
      const int r = crow + 16 * i;
      aok[m][i] = false;
      arow[m][i] = reinterpret_cast<const __nv_bfloat16*>(a.pv.slab);
      if (r < rank)
        arow[m][i] = reinterpret_cast<const __nv_bfloat16*>(
            lora_row(a.pv, table_off, lm.a_tab, lm.a_row0, lm.a_rpb, d_in, r, aok[m][i]));
    }
  }
  const uint32_t sbase = smem_u32(smem);
  auto load_stage = [&](int it, int st) {
    const int kk = kb + it * KS + cchunk * 8;
    const bool kok = kk < ke;
    const uint32_t xs = sbase + st * STAGE_BYTES;
#pragma unroll
    for (int i = 0; i < XR; ++i) cp_async16(xs + swz(crow + 16 * i, cchunk, 8), xrow[i] + kk, xok[i] && kok);
#pragma unroll
    for (int m = 0; m < NM; ++m) {
      const uint32_t as = xs + (TM + m * RMAX) * 128;
#pragma unroll
      for (int i = 0; i < AR; ++i) cp_async16(as + swz(crow + 16 * i, cchunk, 8), arow[m][i] + kk, aok[m][i] && kok);
    }
  };

  float acc[NM][RMAX / 8][4];
#pragma unroll
  for (int m = 0; m < NM; ++m)
#pragma unroll
    for (int n = 0; n < RMAX / 8; ++n) acc[m][n][0] = acc[m][n][1] = acc[m][n][2] = acc[m][n][3] = 0.f;

#pragma unroll
  for (int s = 0; s < STAGES - 1; ++s) {
    if (s < n_it) load_stage(s, s);
    cp_async_commit();
  }
  const int mrow = warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1);
  for (int it = 0; it < n_it; ++it) {
    cp_async_wait<STAGES - 2>();
    __syncthreads();
    if (it + STAGES - 1 < n_it) load_stage(it + STAGES - 1, (it + STAGES - 1) % STAGES);
    cp_async_commit();
    const uint32_t xs = sbase + (it % STAGES) * STAGE_BYTES;
#pragma unroll
    for (int ks = 0; ks < KS / 16; ++ks) {
      uint32_t af[4];
      ldmatrix_x4(af, xs + swz(mrow, 2 * ks + (lane >> 4), 8));
#pragma unroll
      for (int m = 0; m < NM; ++m) {
        const uint32_t as = xs + (TM + m * RMAX) * 128;
#pragma unroll
        for (int p = 0; p < RMAX / 16; ++p) {
          if (16 * p < rank) {
            uint32_t bf[4];
            ldmatrix_x4(bf, as + swz(16 * p + (lane & 7) + 8 * (lane >> 4), 2 * ks + ((lane >> 3) & 1), 8));
            mma_bf16(acc[m][2 * p], af, bf[0], bf[1]);
            mma_bf16(acc[m][2 * p + 1], af, bf[2], bf[3]);
          }
        }
      }
    }
  }
  const int g = lane >> 2, t4 = lane & 3;
  const int r0 = tok0 + warp * 16 + g;
#pragma unroll
  for (int m = 0; m < NM; ++m) {
    float* vout = a.v + ((size_t)(m * a.ksplit + split) * a.n_tokens) * RMAX;
#pragma unroll
    for (int n = 0; n < RMAX / 8; ++n) {
      if (r0 < tok1) *reinterpret_cast<float2*>(vout + (size_t)r0 * RMAX + 8 * n + 2 * t4) = make_float2(acc[m][n][0], acc[m][n][1]);
      if (r0 + 8 < tok1) *reinterpret_cast<float2*>(vout + (size_t)(r0 + 8) * RMAX + 8 * n + 2 * t4) = make_float2(acc[m][n][2], acc[m][n][3]);
    }
  }
}

// KV: some projections of the call write their result rows into pool blocks (SgmvArgs::kv_side).
// CTAs per SM the register budget is sized for (the kernel is bound by memory latency: occupancy matters more
// than a few spilled values)
constexpr int expand_min_ctas(int tm, int rmax, bool) { return tm == 16 ? 5 : (rmax == 16 ? 4 : 3); }

// whether the LoRA-term tile reuses the adapter-row buffer of the stage (it has to fit there)
__host__ __device__ constexpr bool expand_alias(int tm, int rmax) { return rmax >= 64 && rmax >= tm; }
constexpr int expand_smem_bytes(int tm, int rmax) { return 2 * (tm + rmax) * 256 + (expand_alias(tm, rmax) ? 0 : tm * 256); }

template <int TM, int RMAX, bool KV>
__global__ void __launch_bounds__(SG_THREADS, expand_min_ctas(TM, RMAX, KV)) sgmv_expand_kernel(const SgmvArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int j = blockIdx.x % a.n_mats;
  const int tile = blockIdx.x / a.n_mats;
  int seg, tok0, tok1;
  if (!find_tile<TM>(a.seg_indptr, a.lora_ids, a.n_seg, tile, seg, tok0, tok1, a.all_segments != 0)) return;
  const int lid = a.lora_ids[seg];
  const int side = KV ? a.kv_side[j] : -1;   // >= 0: the result rows go into the requests' pool blocks
  int rank = 0;
  uint32_t table_off = 0;
  LoraMat lm = {};
  if (lid >= 0) {
    if ((uint32_t)lid >= a.pv.dir_cap || a.pv.dir[lid].rank <= 0 || a.mat_index[j] >= a.pv.dir[lid].n_mats) return;
    const LoraEntry* e = a.pv.dir + lid;
    lm = e->mats[a.mat_index[j]];
    rank = min(e->rank, RMAX);
    table_off = e->table_off;
  } else if (side < 0) {
    return;                                // no adapter and y stays where it is: nothing to do
  }
  const int d_out = a.d_out[j];
  const int c0 = blockIdx.y * a.expand_cols;
  if (c0 >= d_out) return;
  const int c1 = min(d_out, c0 + a.expand_cols);
  const int n_sub = (c1 - c0 + NSUB - 1) / NSUB;

  constexpr int WM = TM / 16, WN = 4 / WM;     // warps along tokens / along columns
  constexpr int NTW = 16 / WN;                 // 8-column tiles per warp inside a sub-tile
  const int warp_m = warp % WM, warp_n = warp / WM;
  const int g = lane >> 2, t4 = lane & 3;

  constexpr int YR = TM / 8;       // y rows per thread per sub-tile
  constexpr int BR = RMAX / 8;     // adapter rows per thread per sub-tile
  constexpr int STAGE_BYTES = (TM + RMAX) * 256;
  const int crow = tid >> 4, cchunk = tid & 15;
  __nv_bfloat16* yrow[YR];
  bool yok[YR];
#pragma unroll
  for (int i = 0; i < YR; ++i) {
    const int t = tok0 + crow + 8 * i;
    yok[i] = t < tok1;
    yrow[i] = a.y[j] + (size_t)(yok[i] ? t : tok0) * d_out;
  }
  // K / V rows: where each of this thread's token rows lives in the pool (block and slot of its position),
  // and how many slots behind it have to be cleared (V of a request's last token)
  uint32_t kvloc[KV ? YR : 1];      // block << 8 | slot << 1 | "last token of its request" (slot < 128, block < 2^24)
  if (KV && side >= 0) {
    int r = 0;
    {
      int lo = 0, hi = a.n_req;
      const int t0 = tok0 + crow;
      while (hi - lo > 1) {
        const int mid = (lo + hi) >> 1;
        if (a.req_indptr[mid] <= t0) lo = mid; else hi = mid;
      }
      r = lo;
    }
#pragma unroll
    for (int i = 0; i < YR; ++i) {
      kvloc[i] = 0;
      const int t = tok0 + crow + 8 * i;
      if (!yok[i]) continue;
      while (r + 1 < a.n_req && t >= a.req_indptr[r + 1]) ++r;
      const int pos = a.prefix_lens[r] + (t - a.req_indptr[r]);
      const int entry = pos / a.bt, slot = pos - entry * a.bt;
      if (pos < 0 || t < a.req_indptr[r] || t >= a.req_indptr[r + 1] || entry >= a.tbl_indptr[r + 1] - a.tbl_indptr[r]) {
        atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
        yok[i] = false;
        continue;
      }
      const uint32_t blk = a.tbl[a.tbl_indptr[r] + entry];
      if (blk >= a.pv.n_blocks || blk >= (1u << 24)) {
        atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_BLOCK);
        yok[i] = false;
        continue;
      }
      kvloc[i] = blk << 8 | (uint32_t)slot << 1 | (t == a.req_indptr[r + 1] - 1 ? 1u : 0u);
    }
  }
  const __nv_bfloat16* brow[BR];
  bool bok[BR];
#pragma unroll
  for (int i = 0; i < BR; ++i) {
    const int r = crow + 8 * i;
    bok[i] = false;
    brow[i] = reinterpret_cast<const __nv_bfloat16*>(a.pv.slab);
    if (r < rank)
      brow[i] = reinterpret_cast<const __nv_bfloat16*>(
          lora_row(a.pv, table_off, lm.b_tab, lm.b_row0, lm.b_rpb, d_out, r, bok[i]));
  }
  const uint32_t sbase = smem_u32(smem);
  auto load_sub = [&](int sub, int st) {
    const int col = c0 + sub * NSUB + cchunk * 8;
    const bool cok = col < c1;
    const uint32_t ys = sbase + st * STAGE_BYTES, bs = ys + TM * 256;
#pragma unroll
    for (int i = 0; i < YR; ++i) cp_async16(ys + swz(crow + 8 * i, cchunk, 16), yrow[i] + col, yok[i] && cok);
#pragma unroll
    for (int i = 0; i < BR; ++i) cp_async16(bs + swz(crow + 8 * i, cchunk, 16), brow[i] + col, bok[i] && cok);
  };

  load_sub(0, 0);
  cp_async_commit();
  // v fragments: sum of the k-slices, scaled, rounded to bf16.  Everything above reads only what was in memory
  // before the shrink started; v is the shrink's output, so this is where a programmatic dependent launch waits.
  pdl_wait();
  uint32_t av[RMAX / 16][4];
  {
    const int r0 = tok0 + warp_m * 16 + g, r1 = r0 + 8;
#pragma unroll
    for (int ks = 0; ks < RMAX / 16; ++ks) {
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        const int row = (q & 1) ? r1 : r0;
        const int col = 16 * ks + 2 * t4 + ((q & 2) ? 8 : 0);
        float2 s = make_float2(0.f, 0.f);
        if (row < tok1 && col < rank) {
          for (int sp = 0; sp < a.ksplit; ++sp) {
            const float2 p = *reinterpret_cast<const float2*>(
                a.v + ((size_t)(j * a.ksplit + sp) * a.n_tokens + row) * RMAX + col);
            s.x += p.x; s.y += p.y;
          }
        }
        s.x *= a.scale; s.y *= a.scale;
        av[ks][q] = pack_bf16(s.x, s.y);
      }
    }
  }

  for (int sub = 0; sub < n_sub; ++sub) {
    const int st = sub & 1;
    if (sub + 1 < n_sub) load_sub(sub + 1, st ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    unsigned char* ysm = smem + st * STAGE_BYTES;
    const uint32_t bs = sbase + st * STAGE_BYTES + TM * 256;
    float acc[NTW][4];
#pragma unroll
    for (int n = 0; n < NTW; ++n) acc[n][0] = acc[n][1] = acc[n][2] = acc[n][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < RMAX / 16; ++ks) {
      if (16 * ks < rank) {
#pragma unroll
        for (int p = 0; p < NTW / 2; ++p) {
          uint32_t bf[4];
          ldmatrix_x4_trans(bf, bs + swz(16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1),
                                         warp_n * NTW + 2 * p + (lane >> 4), 16));
          mma_bf16(acc[2 * p], av[ks], bf[0], bf[1]);
          mma_bf16(acc[2 * p + 1], av[ks], bf[2], bf[3]);
        }
      }
    }
    // the LoRA term of this sub-tile as bf16 pairs into a tile of its own (each element is owned by exactly one
    // thread); at rank 64 that tile takes the place of the adapter rows the MMAs have just consumed, which brings
    // the CTA to 64 KB and a third CTA onto the SM
    constexpr bool ALIAS = expand_alias(TM, RMAX);
    unsigned char* dsm = ALIAS ? smem + st * STAGE_BYTES + TM * 256 : smem + 2 * STAGE_BYTES;
    if (ALIAS) __syncthreads();
#pragma unroll
    for (int n = 0; n < NTW; ++n) {
      const int chunk = warp_n * NTW + n;
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int row = warp_m * 16 + g + 8 * h;
        *reinterpret_cast<uint32_t*>(dsm + swz(row, chunk, 16) + 4 * t4) = pack_bf16(acc[n][2 * h], acc[n][2 * h + 1]);
      }
    }
    __syncthreads();
    {
      const int col = c0 + sub * NSUB + cchunk * 8;
      if (col < c1) {
        if (!KV || side < 0) {
#pragma unroll
          for (int i = 0; i < YR; ++i)
            if (yok[i])
              *reinterpret_cast<uint4*>(yrow[i] + col) = add_bf16x8(*reinterpret_cast<const uint4*>(ysm + swz(crow + 8 * i, cchunk, 16)),
                                                                    *reinterpret_cast<const uint4*>(dsm + swz(crow + 8 * i, cchunk, 16)));
        } else if (KV) {
          // a sub-tile is one KV head: [K|V][head][slot][128] inside the block
          static_assert(NSUB == FL_HEAD_DIM, "a sub-tile must be one head");
          const size_t head_off = ((size_t)side * a.n_kv + (c0 + sub * NSUB) / FL_HEAD_DIM) * a.bt * (FL_HEAD_DIM * 2) + cchunk * 16;
#pragma unroll
          for (int i = 0; i < YR; ++i) {
            if (yok[i]) {
              const uint32_t loc = kvloc[KV ? i : 0];
              const int slot = (loc >> 1) & 127;
              unsigned char* dst = a.pv.slab + (size_t)(loc >> 8) * a.pv.block_bytes + head_off + slot * (FL_HEAD_DIM * 2);
              *reinterpret_cast<uint4*>(dst) = add_bf16x8(*reinterpret_cast<const uint4*>(ysm + swz(crow + 8 * i, cchunk, 16)),
                                                          *reinterpret_cast<const uint4*>(dsm + swz(crow + 8 * i, cchunk, 16)));
              if (side == 1 && (loc & 1u))     // V of a request's last token: clear the slots behind it
                for (int z = slot + 1; z < a.bt; ++z)
                  *reinterpret_cast<uint4*>(dst + (z - slot) * (FL_HEAD_DIM * 2)) = make_uint4(0u, 0u, 0u, 0u);
            }
          }
        }
      }
    }
    __syncthreads();
  }
}

int pick_ksplit(int n_tokens) {
  // decode-sized batches have few token tiles: slice d_in so that enough CTAs stream adapter rows
  const int tiles = n_tokens / 16 + 1;
  int ks = 592 / tiles;
  if (ks < 1) ks = 1;
  if (ks > KSPLIT_MAX) ks = KSPLIT_MAX;
  return ks;
}

// Columns per expand CTA.  Every CTA pays a prologue of dependent look-ups (its tile, the adapter's directory
// entry and row tables, the v fragments, the K/V destinations) that wider CTAs spread over more sub-tiles; the
// widest slice that still leaves about ten CTAs per SM in the grid wins.
int pick_expand_cols(const SgmvArgs& a, int tiles) {
  int cols = EXPAND_COLS_MAX;
  for (; cols > EXPAND_COLS_MIN; cols /= 2) {
    long ctas = 0;
    for (int j = 0; j < a.n_mats; ++j) ctas += (long)tiles * ((a.d_out[j] + cols - 1) / cols);
    if (ctas >= 1480) break;
  }
  return cols;
}

template <int TM, int RMAX>
int launch_pair(fl_pool* p, SgmvArgs& a, int tiles, int d_out_max, cudaStream_t st, bool shrink_only) {
  a.expand_cols = pick_expand_cols(a, tiles);
  static bool configured[16] = {};
  const int shrink_smem = SH_STAGES * (TM + RMAX) * 128;
  const int expand_smem = expand_smem_bytes(TM, RMAX);     // two stages of (y, B) + the LoRA-term tile
  if (!configured[p->device & 15]) {
    FL_CUDA(p, cudaFuncSetAttribute(sgmv_shrink_kernel<TM, RMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, shrink_smem));
    FL_CUDA(p, cudaFuncSetAttribute(sgmv_expand_kernel<TM, RMAX, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, expand_smem));
    FL_CUDA(p, cudaFuncSetAttribute(sgmv_expand_kernel<TM, RMAX, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, expand_smem));
    configured[p->device & 15] = true;
  }
  if (TM == 64 && p->sgmv_shrink_kind == 0 && a.n_mats <= 3 && a.tc_ksplit > 0) {
    // long segments: the shrink on tcgen05 tensor cores, tiles of 128 tokens, its own number of d_in slices
    a.ksplit = a.tc_ksplit;
    sgmv::TcShrinkArgs t;
    t.pv = a.pv;
    t.v = a.v;
    t.ksplit = a.ksplit;
    t.n_mats = a.n_mats;
    for (int j = 0; j < 3; ++j) t.mat_index[j] = a.mat_index[j < a.n_mats ? j : 0];
    t.seg_indptr = a.seg_indptr;
    t.lora_ids = a.lora_ids;
    t.n_seg = a.n_seg;
    t.n_tokens = a.n_tokens;
    t.d_in = p->mats[a.mat_index[0]].d_in;
    const int rc = sgmv::shrink_tc(p, t, a.x, RMAX, st);
    if (rc != FL_OK) return rc;
  } else if (TM == 64 && RMAX == 16 && a.n_mats == 3) {      // at higher ranks the three accumulators cost too many registers
    static bool configured3[16] = {};
    const int smem3 = (RMAX == 64 ? 3 : 4) * (64 + 3 * RMAX) * 128;
    if (!configured3[p->device & 15]) {
      FL_CUDA(p, cudaFuncSetAttribute(sgmv_shrink3_kernel<RMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem3));
      configured3[p->device & 15] = true;
    }
    FL_CUDA(p, launch_pdl(sgmv_shrink3_kernel<RMAX>, dim3(tiles, a.ksplit), dim3(SG_THREADS), smem3, st, a));
  } else {
    FL_CUDA(p, launch_pdl(sgmv_shrink_kernel<TM, RMAX>, dim3(tiles * a.n_mats, a.ksplit), dim3(SG_THREADS), shrink_smem, st, a));
  }
  if (shrink_only) return FL_OK;       // the caller consumes the partial sums itself
  const dim3 egrid(tiles * a.n_mats, (d_out_max + a.expand_cols - 1) / a.expand_cols);
  // the expand may start while the shrink drains (it waits for the shrink's output inside the kernel)
  FL_CUDA(p, cudaGetLastError());
  if (a.all_segments) FL_CUDA(p, launch_pdl(sgmv_expand_kernel<TM, RMAX, true>, egrid, dim3(SG_THREADS), expand_smem, st, a));
  else FL_CUDA(p, launch_pdl(sgmv_expand_kernel<TM, RMAX, false>, egrid, dim3(SG_THREADS), expand_smem, st, a));
  return FL_OK;
}

int rmax_of(const fl_pool* p) { return p->max_rank <= 16 ? 16 : (p->max_rank <= 32 ? 32 : 64); }

}  // namespace

extern "C" {

size_t fl_lora_sgmv_workspace(int n_tokens, int n_mats) {
  if (n_tokens <= 0 || n_mats <= 0) return 256;
  return (size_t)n_mats * pick_ksplit(n_tokens) * (size_t)n_tokens * FL_MAX_RANK * sizeof(float) + 256;
}

}  // extern "C"

namespace {

struct KvDest {      // where K and V results go when they are appended to the pool by the projection itself
  int k_slot, v_slot;           // positions of the K and V projections in the call's list
  const int32_t* req_indptr;
  const int32_t* tbl_indptr;
  const uint32_t* tbl;
  const int32_t* prefix_lens;
  int n_req, n_kv;
};

int sgmv_common(fl_pool* p, fl_bf16* const* ys, const fl_bf16* x, const int* mat_indices, int n_mats,
                const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                float scale, void* workspace, size_t workspace_bytes, fl_stream stream, const KvDest* kv,
                sgmv::ShrinkInfo* shrink_only = nullptr) {
  if (!p || n_mats < 1 || n_mats > FL_MAX_MATS || n_seg < 0 || n_tokens < 0 || !ys || !mat_indices) return FL_EINVAL;
  if (n_seg == 0 || n_tokens == 0) return FL_OK;
  if (!x || !seg_indptr || !lora_ids || !workspace) return FL_EINVAL;
  if (p->n_mats == 0) return FL_EBADID;   // no adapter registered
  SgmvArgs a;
  a.pv = p->view();
  a.x = reinterpret_cast<const __nv_bfloat16*>(x);
  int d_out_max = 0;
  for (int j = 0; j < n_mats; ++j) {
    const int mi = mat_indices[j];
    if (mi < 0 || mi >= p->n_mats || (!ys[j] && !shrink_only)) return FL_EINVAL;
    if (p->mats[mi].d_in != p->mats[mat_indices[0]].d_in) return FL_EINVAL;   // the projections share x
    a.y[j] = reinterpret_cast<__nv_bfloat16*>(ys[j]);
    a.mat_index[j] = mi;
    d_out_max = d_out_max > p->mats[mi].d_out ? d_out_max : p->mats[mi].d_out;
  }
  for (int j = 0; j < FL_MAX_MATS; ++j) {
    a.kv_side[j] = -1;
    a.d_out[j] = j < n_mats ? p->mats[mat_indices[j]].d_out : 0;
  }
  a.all_segments = 0;
  a.req_indptr = a.tbl_indptr = a.prefix_lens = nullptr;
  a.tbl = nullptr;
  a.n_req = a.n_kv = a.bt = 0;
  if (kv) {
    const size_t per_tok = (size_t)2 * kv->n_kv * FL_HEAD_DIM * 2;
    if (kv->n_kv < 1 || kv->n_req < 1 || p->block_bytes % per_tok != 0 || kv->k_slot == kv->v_slot) return FL_EINVAL;
    if (!kv->req_indptr || !kv->tbl_indptr || !kv->tbl || !kv->prefix_lens) return FL_EINVAL;
    for (int side = 0; side < 2; ++side) {
      const int slot = side ? kv->v_slot : kv->k_slot;
      if (slot < 0 || slot >= n_mats || a.d_out[slot] != kv->n_kv * FL_HEAD_DIM) return FL_EINVAL;
      a.kv_side[slot] = side;
    }
    a.all_segments = 1;
    a.req_indptr = kv->req_indptr;
    a.tbl_indptr = kv->tbl_indptr;
    a.tbl = kv->tbl;
    a.prefix_lens = kv->prefix_lens;
    a.n_req = kv->n_req;
    a.n_kv = kv->n_kv;
    a.bt = (int)(p->block_bytes / per_tok);
    // the expand packs a token's destination into one word: 7 bits of slot, 24 bits of block id
    if (a.bt > 128 || p->n_blocks > (1u << 24)) return FL_EINVAL;
  }
  a.n_mats = n_mats;
  a.seg_indptr = seg_indptr;
  a.lora_ids = lora_ids;
  a.n_seg = n_seg;
  a.n_tokens = n_tokens;
  a.scale = scale;
  a.v = reinterpret_cast<float*>(workspace);
  a.ksplit = pick_ksplit(n_tokens);
  if (workspace_bytes < fl_lora_sgmv_workspace(n_tokens, n_mats)) return FL_ENOMEM;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != p->device) cudaSetDevice(p->device);
  const bool small = n_tokens <= 16 * n_seg;   // average segment of at most 16 tokens: decode-like
  const int rmax = rmax_of(p);
  const cudaStream_t st = (cudaStream_t)stream;
  if (!small && rmax == 16 && a.ksplit == 1) {
    // A long-segment batch of a few thousand tokens gives the shrink about two CTAs per SM (eight warps), too few to
    // keep the loads of a rank-16 shrink in flight: two slices of d_in double them.  The scratch is sized for rank 64,
    // so at rank 16 two slices fit in what the caller already brought.
    const long shrink_ctas = (long)(n_seg + n_tokens / 64) * (n_mats == 3 ? 1 : n_mats);
    const size_t need = (size_t)n_mats * 2 * (size_t)n_tokens * rmax * sizeof(float) + 256;
    if (shrink_ctas < 592 && need <= workspace_bytes) a.ksplit = 2;
  }
  a.tc_ksplit = 0;
  if (!small && n_mats <= 3 && rmax >= 32) {     // at rank 16 the mma.sync shrink is the faster one
    // units of (128-token tile, slice of d_in) for the tcgen05 shrink: about four per SM when the scratch the caller
    // brought has room for the slices, every slice at least 512 values deep
    const int d_in = p->mats[mat_indices[0]].d_in;
    const long tiles = (long)n_seg + n_tokens / 128;
    int ks = (int)std::min<long>(8, std::max<long>(1, (4L * p->sm_count + tiles - 1) / tiles));
    ks = std::min(ks, std::max(1, d_in / 512));
    // (measured against the size every caller has to bring, not against what this caller brought: the number of
    // slices fixes the order of the sums, and equal calls should give equal bits)
    const size_t room = fl_lora_sgmv_workspace(n_tokens, n_mats);
    while (ks > 1 && (size_t)n_mats * ks * (size_t)n_tokens * rmax * sizeof(float) + 256 > room) --ks;
    if ((size_t)n_mats * ks * (size_t)n_tokens * rmax * sizeof(float) + 256 <= room) a.tc_ksplit = ks;
  }
  int rc;
  const bool so = shrink_only != nullptr;
  if (so) {
    shrink_only->ksplit = (!small && p->sgmv_shrink_kind == 0 && a.tc_ksplit > 0) ? a.tc_ksplit : a.ksplit;
    shrink_only->rmax = rmax;
  }
  if (small) {
    const int tiles = n_seg + n_tokens / 16;
    rc = rmax == 16 ? launch_pair<16, 16>(p, a, tiles, d_out_max, st, so)
       : rmax == 32 ? launch_pair<16, 32>(p, a, tiles, d_out_max, st, so)
                    : launch_pair<16, 64>(p, a, tiles, d_out_max, st, so);
  } else {
    const int tiles = n_seg + n_tokens / 64;
    rc = rmax == 16 ? launch_pair<64, 16>(p, a, tiles, d_out_max, st, so)
       : rmax == 32 ? launch_pair<64, 32>(p, a, tiles, d_out_max, st, so)
                    : launch_pair<64, 64>(p, a, tiles, d_out_max, st, so);
  }
  if (prev != p->device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

}  // namespace

namespace sgmv {
int shrink(fl_pool* p, const fl_bf16* x, const int* mat_indices, int n_mats, const int32_t* seg_indptr,
           const int32_t* lora_ids, int n_seg, int n_tokens, void* workspace, size_t workspace_bytes, fl_stream stream,
           ShrinkInfo* info) {
  fl_bf16* none[FL_MAX_MATS] = {};
  return sgmv_common(p, none, x, mat_indices, n_mats, seg_indptr, lora_ids, n_seg, n_tokens, 1.f, workspace,
                     workspace_bytes, stream, nullptr, info);
}
}  // namespace sgmv

extern "C" {

int fl_lora_sgmv_multi(fl_pool* p, fl_bf16* const* ys, const fl_bf16* x, const int* mat_indices, int n_mats,
                       const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                       float scale, void* workspace, size_t workspace_bytes, fl_stream stream) {
  return sgmv_common(p, ys, x, mat_indices, n_mats, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace,
                     workspace_bytes, stream, nullptr);
}

int fl_lora_sgmv_qkv_append(fl_pool* p, fl_bf16* y_q, const fl_bf16* y_k, const fl_bf16* y_v, const fl_bf16* x,
                            int mat_q, int mat_k, int mat_v, const int32_t* seg_indptr, const int32_t* lora_ids,
                            int n_seg, int n_tokens, float scale, const int32_t* req_indptr,
                            const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                            int n_req, int n_kv_heads, void* workspace, size_t workspace_bytes, fl_stream stream) {
  fl_bf16* ys[3] = {y_q, const_cast<fl_bf16*>(y_k), const_cast<fl_bf16*>(y_v)};
  const int mi[3] = {mat_q, mat_k, mat_v};
  const KvDest kv = {1, 2, req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_kv_heads};
  return sgmv_common(p, ys, x, mi, 3, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace, workspace_bytes, stream, &kv);
}

int fl_lora_sgmv(fl_pool* p, fl_bf16* y, const fl_bf16* x, int mat_index,
                 const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                 float scale, void* workspace, size_t workspace_bytes, fl_stream stream) {
  fl_bf16* ys[1] = {y};
  const int mi[1] = {mat_index};
  return fl_lora_sgmv_multi(p, ys, x, mi, 1, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace,
                            workspace_bytes, stream);
}

// ---------------------------------------------------------------- fl_lora_sgmv_static: no allocation anywhere
// The scratch that fl_lora_sgmv takes from its caller lives here instead, inside the library image.
// Every GPU that loads the library holds these FL_SGMV_STATIC_BYTES until the process exits.
}  // extern "C"

static __device__ __align__(256) unsigned char g_sgmv_static_scratch[FL_SGMV_STATIC_BYTES];

namespace {
constexpr int STATIC_MAX_DEVICES = 64;
void* g_static_scratch_addr[STATIC_MAX_DEVICES] = {};   // device address of the array, per device; one copy per process
}  // namespace

extern "C" {

int fl_lora_sgmv_static(fl_pool* p, fl_bf16* y, const fl_bf16* x, int mat_index,
                        const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                        float scale, fl_stream stream) {
  if (!p || n_seg < 0 || n_tokens < 0) return FL_EINVAL;
  if (p->device < 0 || p->device >= STATIC_MAX_DEVICES) return FL_EINVAL;
  if (n_seg == 0 || n_tokens == 0) return FL_OK;      // nothing to do, as in fl_lora_sgmv
  if (fl_lora_sgmv_workspace(n_tokens, 1) > (size_t)FL_SGMV_STATIC_BYTES) return FL_ENOMEM;   // batch too large for the built-in scratch
  void* scratch = g_static_scratch_addr[p->device];
  if (!scratch) {
    // First call on this device: in host code the array's name is only a handle, so ask the runtime
    // for the array's address on the pool's device (which must be current for the query).
    int prev = -1;
    cudaGetDevice(&prev);
    if (prev != p->device) cudaSetDevice(p->device);
    const cudaError_t e = cudaGetSymbolAddress(&scratch, g_sgmv_static_scratch);
    if (prev != p->device && prev >= 0) cudaSetDevice(prev);
    if (e != cudaSuccess || !scratch) {
      p->last_cuda = (int)e;
      return FL_ECUDA;
    }
    g_static_scratch_addr[p->device] = scratch;
  }
  // Nothing in the scratch has to start at zero: the shrink kernel writes every partial sum that the
  // expand kernel reads, so whatever the previous call left behind is overwritten before use.
  return fl_lora_sgmv(p, y, x, mat_index, seg_indptr, lora_ids, n_seg, n_tokens, scale, scratch,
                      (size_t)FL_SGMV_STATIC_BYTES, stream);
}

}  // extern "C"
