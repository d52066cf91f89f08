// Paged attention over [cached prefix || new tokens] read from pool blocks (Section 2.1, Section 4.2).
//
// A plan kernel sorts the requests of a batch into two work lists: requests with at most 16 query
// rows per KV head (decode steps) are cut into chunks of keys that independent CTAs reduce
// (split-KV, merged afterwards); the others (prefill) are cut into tiles of 64 query rows per head.
// Both kernels stage KV pages (one 4 KiB contiguous piece per block, KV head and K/V side) into
// shared memory with 16-byte cp.async through the block table and run QK^T and PV on bf16 tensor
// cores with an fp32 online softmax.
#include <math.h>
#include <algorithm>
#include "mma_utils.cuh"
#include "attention.cuh"
#include "pool.cuh"

using namespace attn;

namespace {

constexpr int QT = QT_MMA;

__device__ __forceinline__ int block_excl_scan(int val, int* sh, int& total) {
  // exclusive scan over the 256 threads of the plan CTA
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int incl = val;
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    const int o = __shfl_up_sync(0xffffffffu, incl, d);
    if (lane >= d) incl += o;
  }
  if (lane == 31) sh[warp] = incl;
  __syncthreads();
  int wbase = 0, tot = 0;
  for (int w = 0; w < 8; ++w) {
    if (w < warp) wbase += sh[w];
    tot += sh[w];
  }
  __syncthreads();
  total = tot;
  return wbase + incl - val;
}

__global__ void __launch_bounds__(256) attn_plan_kernel(const AttnArgs a, int chunk, int qt) {
  __shared__ int sh[8];
  __shared__ int hist[64], cursor[64];
  pdl_wait();                 // the lists may still be read, and the request arrays written, by the kernel before
  pdl_launch_dependents();    // the prefill kernel sets itself up (barriers, TMEM) while this single CTA plans
  const int group = a.n_q / a.n_kv;
  if (threadIdx.x < 64) hist[threadIdx.x] = 0;
  __syncthreads();
  // Prefill requests are ordered by context length (in 128-key steps), longest first, so that the CTAs that take work
  // from the list finish together; the tiles of one request stay next to each other (its later tiles first), so the
  // units that read the same K/V pages run at about the same time and the second reader finds them in L2.
  auto key_of = [&](int i) { return min(63, (a.prefix_lens[i] + a.new_lens[i] + 127) / 128); };
  int base_p = 0, base_d = 0;
  for (int i0 = 0; i0 < a.n_req; i0 += 256) {
    const int i = i0 + threadIdx.x;
    int n = 0, ctx = 0, tiles = 0, chunks = 0;
    bool dec = false;
    if (i < a.n_req) {
      n = a.new_lens[i];
      ctx = a.prefix_lens[i] + n;
      if (n > 0) {
        dec = n * group <= DEC_ROWS;
        if (dec) chunks = (ctx + chunk - 1) / chunk; else tiles = (n + qt - 1) / qt;
      }
    }
    int tot_p, tot_d;
    block_excl_scan(tiles, sh, tot_p);
    const int off_d = base_d + block_excl_scan(chunks, sh, tot_d);
    if (i < a.n_req) {
      // a request whose chunks do not all fit in the list (contexts longer than the caller's n_tbl covers) gets no
      // output: the chunks that did fit only write partial slots inside the workspace, and the merge, which would
      // read all of them, skips the request (the overflow raises FLAG_BAD_POS below)
      a.req_info[i] = make_int4(off_d, off_d + chunks > a.max_decode ? 0 : chunks, dec ? 1 : 0, 0);
      if (tiles > 0) atomicAdd(&hist[key_of(i)], tiles);
      for (int c = 0; c < chunks; ++c)
        if (off_d + c < a.max_decode) a.decode_list[off_d + c] = make_int2(i, c);
    }
    base_p += tot_p;
    base_d += tot_d;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int start = 0;
    for (int b = 63; b >= 0; --b) {
      cursor[b] = start;
      start += hist[b];
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < a.n_req; i += 256) {
    const int n = a.new_lens[i];
    if (n <= 0 || n * group <= DEC_ROWS) continue;
    const int tiles = (n + qt - 1) / qt;
    const int first = atomicAdd(&cursor[key_of(i)], tiles);
    // An item of 256 tokens is two 128-row tiles that share one K/V stream and costs as many key tiles as its later
    // tile needs.  With an odd number of 128-row tiles the request's FIRST tile (shortest context) goes alone and the
    // pairs start at token 128, instead of the last tile (longest context) going alone: one key tile less per pair.
    const bool lone_first = qt == 256 && (((n + 127) / 128) & 1);
    for (int t = 0; t < tiles; ++t) {
      const int u = tiles - 1 - t;      // item number in token order
      const int q0 = lone_first ? (u == 0 ? 0 : 128 + (u - 1) * 256) : u * qt;
      if (first + t < a.max_prefill) a.prefill_list[first + t] = make_int2(i, q0);
    }
  }
  if (threadIdx.x == 0) {
    if (base_p > a.max_prefill || base_d > a.max_decode) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
    a.hdr->n_prefill = min(base_p, a.max_prefill);
    a.hdr->n_decode = min(base_d, a.max_decode);
    a.hdr->chunk = chunk;
    a.hdr->next_unit = 0;
  }
}

// Online-softmax update for one warp: S holds NT 8-key tiles of raw scores for rows g and g+8.
// Key index of S[n][c] is u0 + 8n + 2*(lane&3) + (c&1); row g sees keys <= lim0, row g+8 keys <= lim1.
template <int NT>
__device__ __forceinline__ void softmax_step(float (&S)[NT][4], float (&O)[16][4], float (&m)[2], float (&l)[2],
                                             int u0, int lim0, int lim1, float scale_log2, uint32_t (&P)[NT / 2][4]) {
  const int t4 = threadIdx.x & 3;
  float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    const int u = u0 + 8 * n + 2 * t4;
    S[n][0] = u <= lim0 ? S[n][0] * scale_log2 : -INFINITY;
    S[n][1] = u + 1 <= lim0 ? S[n][1] * scale_log2 : -INFINITY;
    S[n][2] = u <= lim1 ? S[n][2] * scale_log2 : -INFINITY;
    S[n][3] = u + 1 <= lim1 ? S[n][3] * scale_log2 : -INFINITY;
    mx0 = fmaxf(mx0, fmaxf(S[n][0], S[n][1]));
    mx1 = fmaxf(mx1, fmaxf(S[n][2], S[n][3]));
  }
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
  mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
  mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
  const float mn0 = fmaxf(m[0], mx0), mn1 = fmaxf(m[1], mx1);
  // a row that has seen no key yet keeps max = -inf; use 0 as the reference so nothing becomes NaN
  const float r0 = mn0 == -INFINITY ? 0.f : mn0, r1 = mn1 == -INFINITY ? 0.f : mn1;
  const float a0 = exp2f(m[0] - r0), a1 = exp2f(m[1] - r1);
  m[0] = mn0; m[1] = mn1;
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int n = 0; n < NT; ++n) {
    S[n][0] = exp2f(S[n][0] - r0); S[n][1] = exp2f(S[n][1] - r0);
    S[n][2] = exp2f(S[n][2] - r1); S[n][3] = exp2f(S[n][3] - r1);
    s0 += S[n][0] + S[n][1];
    s1 += S[n][2] + S[n][3];
  }
  l[0] = l[0] * a0 + s0;
  l[1] = l[1] * a1 + s1;
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    O[n][0] *= a0; O[n][1] *= a0; O[n][2] *= a1; O[n][3] *= a1;
  }
#pragma unroll
  for (int k = 0; k < NT / 2; ++k) {
    P[k][0] = pack_bf16(S[2 * k][0], S[2 * k][1]);
    P[k][1] = pack_bf16(S[2 * k][2], S[2 * k][3]);
    P[k][2] = pack_bf16(S[2 * k + 1][0], S[2 * k + 1][1]);
    P[k][3] = pack_bf16(S[2 * k + 1][2], S[2 * k + 1][3]);
  }
}

// S[NT] += Q(16 x 128) K^T for NT*8 keys staged as [key][128] rows (swizzled, 16 chunks per row).
template <int NT>
__device__ __forceinline__ void qk_tile(float (&S)[NT][4], const uint32_t (&qf)[8][4], uint32_t ksm) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int ks = 0; ks < 8; ++ks) {
#pragma unroll
    for (int p = 0; p < NT / 2; ++p) {
      uint32_t bf[4];
      ldmatrix_x4(bf, ksm + swz(16 * p + (lane & 7) + 8 * (lane >> 4), 2 * ks + ((lane >> 3) & 1), 16));
      mma_bf16(S[2 * p], qf[ks], bf[0], bf[1]);
      mma_bf16(S[2 * p + 1], qf[ks], bf[2], bf[3]);
    }
  }
}

// O += P(16 x NT*8 keys) V for values staged as [key][128] rows.
template <int NT>
__device__ __forceinline__ void pv_tile(float (&O)[16][4], const uint32_t (&P)[NT / 2][4], uint32_t vsm) {
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int ks = 0; ks < NT / 2; ++ks) {
#pragma unroll
    for (int p = 0; p < 8; ++p) {
      uint32_t bf[4];
      ldmatrix_x4_trans(bf, vsm + swz(16 * ks + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * p + (lane >> 4), 16));
      mma_bf16(O[2 * p], P[ks], bf[0], bf[1]);
      mma_bf16(O[2 * p + 1], P[ks], bf[2], bf[3]);
    }
  }
}

__device__ __forceinline__ const unsigned char* page_ptr(const PoolView& pv, uint32_t blk, int side_head, bool& ok) {
  if (blk >= pv.n_blocks) {
    atomicOr(pv.flags, (uint32_t)FLAG_BAD_BLOCK);
    ok = false;
    return pv.slab;
  }
  ok = true;
  return pv.slab + (size_t)blk * pv.block_bytes + (size_t)side_head * PAGE_BYTES;
}

// ------------------------------------------------------------------ decode (split-KV)
// One CTA per (request, chunk of keys, KV head).  Rows = new tokens x query heads of the group
// (at most 16).  The four warps take pages round-robin, each with its own double buffer, and merge
// their partial (max, sum, O) through shared memory at the end.
__global__ void __launch_bounds__(ATT_THREADS) attn_decode_kernel(const AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  pdl_wait();
  const int item = blockIdx.x / a.n_kv, h = blockIdx.x % a.n_kv;
  if (item >= a.hdr->n_decode) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int2 it = a.decode_list[item];
  const int i = it.x, c = it.y;
  const int chunk = a.hdr->chunk;
  const int n_new = a.new_lens[i], prefix = a.prefix_lens[i], ctx = prefix + n_new;
  const int group = a.n_q / a.n_kv;
  const int rows = n_new * group;
  const int tok0 = a.req_indptr[i];
  const int u_begin = c * chunk, u_end = min(ctx, u_begin + chunk);
  const int n_pages = (u_end - u_begin + BT - 1) / BT;
  const int tbl0 = a.tbl_indptr[i], tbl_n = a.tbl_indptr[i + 1] - tbl0;
  const int pg0 = u_begin / BT;
  if (pg0 + n_pages > tbl_n) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
    return;
  }
  // query fragments: row r -> (new token r / group, query head h*group + r % group)
  uint32_t qf[8][4];
  int lim[2];
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    const int r = g + 8 * hh;
    const bool ok = r < rows;
    const int j = ok ? r / group : 0;
    lim[hh] = ok ? prefix + j : -1;
    const __nv_bfloat16* qp = a.q + ((size_t)(tok0 + j) * a.n_q + (h * group + (ok ? r % group : 0))) * D;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      qf[ks][hh] = ok ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 2 * t4) : 0u;
      qf[ks][hh + 2] = ok ? *reinterpret_cast<const uint32_t*>(qp + 16 * ks + 2 * t4 + 8) : 0u;
    }
  }
  float O[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) O[n][0] = O[n][1] = O[n][2] = O[n][3] = 0.f;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};

  const uint32_t wbase = smem_u32(smem) + warp * (4 * PAGE_BYTES);   // per warp: 2 stages x (K page, V page)
  auto load_page = [&](int pg, int st) {
    const uint32_t blk = a.tbl[tbl0 + pg0 + pg];
    bool ok;
    const unsigned char* kp = page_ptr(a.pv, blk, h, ok);
    const unsigned char* vp = kp + (size_t)a.n_kv * PAGE_BYTES;
    const uint32_t ks = wbase + st * 2 * PAGE_BYTES, vs = ks + PAGE_BYTES;
    // slots behind the last stored token may hold anything: their V rows are zero-filled so that a
    // zero weight times a stale non-finite value cannot reach the output
    const int valid = u_end - (u_begin + pg * BT);
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int cidx = lane + 32 * q;          // 256 chunks per page: row = cidx / 16
      const int row = cidx >> 4, ch = cidx & 15;
      cp_async16(ks + swz(row, ch, 16), kp + cidx * 16, ok);
      cp_async16(vs + swz(row, ch, 16), vp + cidx * 16, ok && row < valid);
    }
  };
  if (warp < n_pages) load_page(warp, 0);
  cp_async_commit();
  int st = 0;
  for (int pg = warp; pg < n_pages; pg += 4, st ^= 1) {
    if (pg + 4 < n_pages) load_page(pg + 4, st ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncwarp();
    const uint32_t ks = wbase + st * 2 * PAGE_BYTES, vs = ks + PAGE_BYTES;
    float S[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    qk_tile<2>(S, qf, ks);
    uint32_t P[1][4];
    softmax_step<2>(S, O, m, l, u_begin + pg * BT, lim[0], lim[1], a.scale_log2, P);
    pv_tile<2>(O, P, vs);
    __syncwarp();
  }
  cp_async_wait<0>();
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 1);
    l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 2);
  }
  __syncthreads();
  // merge the four warps: red_o [warp][16][128], red_ml [warp][16]
  float* red_o = reinterpret_cast<float*>(smem);
  float2* red_ml = reinterpret_cast<float2*>(smem + 4 * DEC_ROWS * D * 4);
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    float* p = red_o + (warp * DEC_ROWS + g) * D + 8 * n + 2 * t4;
    p[0] = O[n][0]; p[1] = O[n][1];
    p[8 * D] = O[n][2]; p[8 * D + 1] = O[n][3];
  }
  if (t4 == 0) {
    red_ml[warp * DEC_ROWS + g] = make_float2(m[0], l[0]);
    red_ml[warp * DEC_ROWS + g + 8] = make_float2(m[1], l[1]);
  }
  __syncthreads();
  const int4 info = a.req_info[i];
  for (int e = tid; e < rows * D; e += ATT_THREADS) {
    const int r = e / D, col = e % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < 4; ++w) M = fmaxf(M, red_ml[w * DEC_ROWS + r].x);
    const float ref = M == -INFINITY ? 0.f : M;
    float L = 0.f, o = 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) {
      const float2 ml = red_ml[w * DEC_ROWS + r];
      const float sc = exp2f(ml.x - ref);
      L += ml.y * sc;
      o += red_o[(w * DEC_ROWS + r) * D + col] * sc;
    }
    if (info.y == 1) {
      const int j = r / group, hq = h * group + r % group;
      a.out[((size_t)(tok0 + j) * a.n_q + hq) * D + col] = __float2bfloat16_rn(L > 0.f ? o / L : 0.f);
    } else {
      const size_t slot = ((size_t)(info.x + c) * a.n_kv + h) * DEC_ROWS + r;
      a.part_o[slot * D + col] = o;
      if (col == 0) a.part_ml[slot] = make_float2(M, L);
    }
  }
}

// Combines the chunk partials of one (request, KV head): grid = n_req * n_kv.
__global__ void __launch_bounds__(ATT_THREADS) attn_merge_kernel(const AttnArgs a) {
  pdl_wait();
  const int i = blockIdx.x / a.n_kv, h = blockIdx.x % a.n_kv;
  const int4 info = a.req_info[i];
  if (!info.z || info.y <= 1) return;
  const int group = a.n_q / a.n_kv;
  const int rows = a.new_lens[i] * group;
  const int tok0 = a.req_indptr[i];
  for (int e = threadIdx.x; e < rows * D; e += ATT_THREADS) {
    const int r = e / D, col = e % D;
    float M = -INFINITY;
    for (int c = 0; c < info.y; ++c)
      M = fmaxf(M, a.part_ml[((size_t)(info.x + c) * a.n_kv + h) * DEC_ROWS + r].x);
    const float ref = M == -INFINITY ? 0.f : M;
    float L = 0.f, o = 0.f;
    for (int c = 0; c < info.y; ++c) {
      const size_t slot = ((size_t)(info.x + c) * a.n_kv + h) * DEC_ROWS + r;
      const float2 ml = a.part_ml[slot];
      const float sc = exp2f(ml.x - ref);
      L += ml.y * sc;
      o += a.part_o[slot * D + col] * sc;
    }
    const int j = r / group, hq = h * group + r % group;
    a.out[((size_t)(tok0 + j) * a.n_q + hq) * D + col] = __float2bfloat16_rn(L > 0.f ? o / L : 0.f);
  }
}

// ------------------------------------------------------------------ prefill (tensor-core tiles, mma.sync)
// One CTA per (request, tile of 64 new tokens, query head); warp w owns rows 16w..16w+15.
__global__ void __launch_bounds__(ATT_THREADS) attn_prefill_kernel(const AttnArgs a) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int item = blockIdx.x / a.n_q, hq = blockIdx.x % a.n_q;
  if (item >= a.hdr->n_prefill) return;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = lane >> 2, t4 = lane & 3;
  const int2 it = a.prefill_list[item];
  const int i = it.x, q0 = it.y;
  const int n_new = a.new_lens[i], prefix = a.prefix_lens[i], ctx = prefix + n_new;
  const int h = hq / (a.n_q / a.n_kv);
  const int tok0 = a.req_indptr[i] + q0;
  const int q_rows = min(QT, n_new - q0);
  const int kv_end = min(ctx, prefix + q0 + QT);
  const int n_kt = (kv_end + KT - 1) / KT;
  const int tbl0 = a.tbl_indptr[i], tbl_n = a.tbl_indptr[i + 1] - tbl0;
  if ((kv_end + BT - 1) / BT > tbl_n) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
    return;
  }
  constexpr int TILE_BYTES = KT * D * 2;     // 16 KiB
  const uint32_t qs = smem_u32(smem);        // Q tile, later the output tile
  const uint32_t kv0 = qs + QT * D * 2;      // 2 stages x (K tile, V tile)
  const int crow = tid >> 4, cch = tid & 15;
  // Q tile
#pragma unroll
  for (int r = 0; r < QT / 8; ++r) {
    const int row = crow + 8 * r;
    const bool ok = row < q_rows;
    cp_async16(qs + swz(row, cch, 16), a.q + ((size_t)(tok0 + (ok ? row : 0)) * a.n_q + hq) * D + cch * 8, ok);
  }
  auto load_kv = [&](int kt, int st) {
    const uint32_t ks = kv0 + st * 2 * TILE_BYTES, vs = ks + TILE_BYTES;
#pragma unroll
    for (int r = 0; r < KT / 8; ++r) {
      const int row = crow + 8 * r;
      const int u = kt * KT + row;
      bool ok = u < kv_end;
      const unsigned char* kp = a.pv.slab;
      if (ok) kp = page_ptr(a.pv, a.tbl[tbl0 + u / BT], h, ok);
      const unsigned char* vp = kp + (size_t)a.n_kv * PAGE_BYTES;
      const int off = (u % BT) * (D * 2) + cch * 16;
      cp_async16(ks + swz(row, cch, 16), kp + off, ok);
      cp_async16(vs + swz(row, cch, 16), vp + off, ok);
    }
  };
  load_kv(0, 0);
  cp_async_commit();

  float O[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) O[n][0] = O[n][1] = O[n][2] = O[n][3] = 0.f;
  float m[2] = {-INFINITY, -INFINITY}, l[2] = {0.f, 0.f};
  const int row0 = warp * 16 + g;
  const int lim0 = row0 < q_rows ? prefix + q0 + row0 : -1;
  const int lim1 = row0 + 8 < q_rows ? prefix + q0 + row0 + 8 : -1;
  uint32_t qf[8][4];

  for (int kt = 0; kt < n_kt; ++kt) {
    const int st = kt & 1;
    if (kt + 1 < n_kt) load_kv(kt + 1, st ^ 1);
    cp_async_commit();
    cp_async_wait<1>();
    __syncthreads();
    if (kt == 0) {
#pragma unroll
      for (int ks = 0; ks < 8; ++ks)
        ldmatrix_x4(qf[ks], qs + swz(warp * 16 + (lane & 7) + 8 * ((lane >> 3) & 1), 2 * ks + (lane >> 4), 16));
    }
    const uint32_t ks = kv0 + st * 2 * TILE_BYTES, vs = ks + TILE_BYTES;
    // keys beyond every row of this warp contribute nothing: skip the tile for this warp
    if (kt * KT <= prefix + q0 + warp * 16 + 15) {
      float S[8][4];
#pragma unroll
      for (int n = 0; n < 8; ++n) S[n][0] = S[n][1] = S[n][2] = S[n][3] = 0.f;
      qk_tile<8>(S, qf, ks);
      uint32_t P[4][4];
      softmax_step<8>(S, O, m, l, kt * KT, lim0, lim1, a.scale_log2, P);
      pv_tile<8>(O, P, vs);
    }
    __syncthreads();
  }
  cp_async_wait<0>();
#pragma unroll
  for (int hh = 0; hh < 2; ++hh) {
    l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 1);
    l[hh] += __shfl_xor_sync(0xffffffffu, l[hh], 2);
  }
  const float inv0 = l[0] > 0.f ? 1.f / l[0] : 0.f, inv1 = l[1] > 0.f ? 1.f / l[1] : 0.f;
  // stage the output tile in the Q buffer (each warp only touches its own 16 rows), then 16-byte stores
#pragma unroll
  for (int n = 0; n < 16; ++n) {
    *reinterpret_cast<uint32_t*>(smem + swz(row0, n, 16) + 4 * t4) = pack_bf16(O[n][0] * inv0, O[n][1] * inv0);
    *reinterpret_cast<uint32_t*>(smem + swz(row0 + 8, n, 16) + 4 * t4) = pack_bf16(O[n][2] * inv1, O[n][3] * inv1);
  }
  __syncthreads();
#pragma unroll
  for (int r = 0; r < QT / 8; ++r) {
    const int row = crow + 8 * r;
    if (row < q_rows)
      *reinterpret_cast<uint4*>(a.out + ((size_t)(tok0 + row) * a.n_q + hq) * D + cch * 8) =
          *reinterpret_cast<const uint4*>(smem + swz(row, cch, 16));
  }
}

int pick_chunk(int n_tbl, int n_kv) {
  // enough (chunk, head) items to fill the GPU several times over, chunks of 64..1024 keys
  long long c = ((long long)n_tbl * BT * n_kv + 1183) / 1184;
  c = (c + 63) / 64 * 64;
  if (c < 64) c = 64;
  if (c > 1024) c = 1024;
  return (int)c;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct WsLayout {
  size_t hdr, prefill_list, decode_list, req_info, part_o, part_ml, total;
  int max_prefill, max_decode, chunk;
};

WsLayout ws_layout(int n_req, int n_tokens, int n_tbl, int n_kv) {
  WsLayout w;
  w.chunk = pick_chunk(n_tbl, n_kv);
  w.max_prefill = n_tokens / QT + n_req;
  w.max_decode = (int)(((long long)n_tbl * BT) / w.chunk) + n_req;
  size_t off = 0;
  w.hdr = off; off = align256(off + sizeof(PlanHdr));
  w.prefill_list = off; off = align256(off + sizeof(int2) * (size_t)w.max_prefill);
  w.decode_list = off; off = align256(off + sizeof(int2) * (size_t)w.max_decode);
  w.req_info = off; off = align256(off + sizeof(int4) * (size_t)n_req);
  w.part_o = off; off = align256(off + sizeof(float) * (size_t)w.max_decode * n_kv * DEC_ROWS * D);
  w.part_ml = off; off = align256(off + sizeof(float2) * (size_t)w.max_decode * n_kv * DEC_ROWS);
  w.total = off;
  return w;
}

}  // namespace

extern "C" {

size_t fl_paged_attention_workspace(int n_req, int n_tokens, int n_tbl, int n_q_heads, int n_kv_heads) {
  (void)n_q_heads;
  if (n_req <= 0 || n_tokens < 0 || n_tbl < 0 || n_kv_heads <= 0) return 256;
  return ws_layout(n_req, n_tokens, n_tbl, n_kv_heads).total;
}

int fl_paged_attention(fl_pool* p, fl_bf16* out, const fl_bf16* q, const int32_t* req_indptr,
                       const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                       const int32_t* new_lens, int n_req, int n_tokens, int n_tbl,
                       int n_q_heads, int n_kv_heads, float sm_scale,
                       void* workspace, size_t workspace_bytes, fl_stream stream) {
  if (!p || n_req < 0 || n_tokens < 0 || n_tbl < 0 || n_q_heads < 1 || n_kv_heads < 1 || n_q_heads % n_kv_heads != 0)
    return FL_EINVAL;
  if (p->block_bytes != (size_t)2 * n_kv_heads * PAGE_BYTES) return FL_EINVAL;   // needs 16-token blocks
  if (n_req == 0 || n_tokens == 0) return FL_OK;
  if (!out || !q || !req_indptr || !kv_tbl_indptr || !kv_tbl || !prefix_lens || !new_lens || !workspace) return FL_EINVAL;
  const WsLayout w = ws_layout(n_req, n_tokens, n_tbl, n_kv_heads);
  if (workspace_bytes < w.total) return FL_ENOMEM;
  unsigned char* ws = reinterpret_cast<unsigned char*>(workspace);
  AttnArgs a;
  a.pv = p->view();
  a.out = reinterpret_cast<__nv_bfloat16*>(out);
  a.q = reinterpret_cast<const __nv_bfloat16*>(q);
  a.req_indptr = req_indptr;
  a.tbl_indptr = kv_tbl_indptr;
  a.tbl = kv_tbl;
  a.prefix_lens = prefix_lens;
  a.new_lens = new_lens;
  a.n_req = n_req;
  a.n_q = n_q_heads;
  a.n_kv = n_kv_heads;
  a.scale_log2 = sm_scale * 1.4426950408889634f;
  a.hdr = reinterpret_cast<PlanHdr*>(ws + w.hdr);
  a.prefill_list = reinterpret_cast<int2*>(ws + w.prefill_list);
  a.decode_list = reinterpret_cast<int2*>(ws + w.decode_list);
  a.req_info = reinterpret_cast<int4*>(ws + w.req_info);
  a.part_o = reinterpret_cast<float*>(ws + w.part_o);
  a.part_ml = reinterpret_cast<float2*>(ws + w.part_ml);
  a.max_prefill = w.max_prefill;
  a.max_decode = w.max_decode;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != p->device) cudaSetDevice(p->device);
  const cudaStream_t st = (cudaStream_t)stream;
  constexpr int DEC_SMEM = 4 * 4 * PAGE_BYTES;                 // 64 KiB
  constexpr int PRE_SMEM = QT * D * 2 + 2 * 2 * KT * D * 2;    // 80 KiB
  static bool configured[16] = {};
  int rc = FL_OK;
  do {
    if (!configured[p->device & 15]) {
      if (cudaFuncSetAttribute(attn_decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DEC_SMEM) != cudaSuccess ||
          cudaFuncSetAttribute(attn_prefill_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PRE_SMEM) != cudaSuccess) {
        p->last_cuda = (int)cudaGetLastError();
        rc = FL_ECUDA;
        break;
      }
      configured[p->device & 15] = true;
    }
    // the tensor-core kernels fold sm_scale into the exponent and take row maxima of raw scores: they need sm_scale > 0
    const int kind = sm_scale > 0.f ? p->prefill_kernel : 1;
    // every kernel of the call is a programmatic dependent launch: it may start while the one before it drains
    // and waits inside for that kernel's results
    if (launch_pdl(attn_plan_kernel, dim3(1), dim3(256), 0, st, a, w.chunk,
                   kind == 0 ? tc2_tile_tokens(n_q_heads, n_kv_heads) : QT_MMA) != cudaSuccess) {
      p->last_cuda = (int)cudaGetLastError();
      rc = FL_ECUDA;
      break;
    }
    if (kind == 0) {
      // upper bound of the plan's tile count: full tiles plus one ragged tile per prefill request, and a
      // request is a prefill only with more than DEC_ROWS / group new tokens
      const int group = n_q_heads / n_kv_heads;
      const int max_req = std::min(n_req, n_tokens / (DEC_ROWS / group + 1));
      const int max_items = std::min(w.max_prefill, n_tokens / tc2_tile_tokens(n_q_heads, n_kv_heads) + max_req);
      rc = launch_prefill_tc2(p, a, n_tokens, max_items, st);
      if (rc != FL_OK) break;
    } else {
      attn_prefill_kernel<<<(unsigned)w.max_prefill * n_q_heads, ATT_THREADS, PRE_SMEM, st>>>(a);
    }
    cudaError_t e = launch_pdl(attn_decode_kernel, dim3((unsigned)w.max_decode * n_kv_heads), dim3(ATT_THREADS), DEC_SMEM, st, a);
    if (e == cudaSuccess) e = launch_pdl(attn_merge_kernel, dim3((unsigned)n_req * n_kv_heads), dim3(ATT_THREADS), 0, st, a);
    if (e == cudaSuccess) e = cudaGetLastError();
    if (e != cudaSuccess) {
      p->last_cuda = (int)e;
      rc = FL_ECUDA;
    }
  } while (0);
  if (prev != p->device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

}  // extern "C"
