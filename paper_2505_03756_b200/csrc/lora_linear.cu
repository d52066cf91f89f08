// Base projection with the LoRA branch folded in: y = x W + scale * (x A_i) B_i per segment (Eq. 1: W' = W + A B;
// Eq. 2: the same branch on the K/V projections), written once, never read back.
//
// A persistent tcgen05 GEMM.  One CTA per SM walks tiles of 128 tokens x BN output columns; the accumulator of a
// tile lives in TMEM (two buffers, so the epilogue of one tile overlaps the MMAs of the next).  The LoRA branch is a
// few extra k-steps into the same accumulator: for every segment that overlaps the tile, the shrink result
// v = x A_i of the tile's tokens (rows outside the segment zeroed, scaled, rounded to bf16) times the adapter's B
// rank-rows of the tile's columns, fetched through the adapter's block table out of the pool blocks.  A tile thus
// needs no alignment with the segments, and a decode batch whose every token uses another adapter is the same
// code path (one extra 16..64-deep k-block per token's adapter).
//   warp 0      TMA producer: x tile [128 x 64] (K-major) and W tile [64 x BN] (N contiguous, as stored) per stage
//   warp 1      MMA issuer: per tile first the LoRA stages, then the d_in / 64 main stages, 128 x BN x 16 MMAs
//   warps 2-5   LoRA stage filler (v rows and B rows into a ring slot, by hand, in the swizzled operand layout),
//               then epilogue of the tile: TMEM -> bf16 -> y
// Main stages and LoRA stages (32 ranks each) have rings of their own, each with one producer and one consumer, so a
// parity wait never has to tell phases two apart; a plan kernel lists, per 128-token tile, the LoRA stages it needs.
// Every mbarrier wait is bounded; a wait that gives up raises a sticky flag, the CTA drains its copies and frees
// its TMEM.  No cluster launch, no multicast.
#include <cuda.h>
#include <string.h>
#include <algorithm>
#include "lora_plan.cuh"
#include "mma_utils.cuh"
#include "pool.cuh"
#include "sgmv.cuh"
#include "tc_ptx.cuh"
#include "tmap.cuh"

namespace {

using namespace tc;

using lora_plan::BM;
using lora_plan::ER;
using lora_plan::EXT_CAP;

constexpr int LT_THREADS = 192;
constexpr int BK = 64;
constexpr int MAX_LIN = 3;                       // projections per launch (q, k, v share x)
constexpr uint32_t A_BYTES = BM * BK * 2;        // x tile, K-major: 128 rows of 128 bytes
constexpr uint32_t B_GROUP = BK * 128;           // one 64-column group of a W tile: 64 k-rows of 128 bytes

template <int BN>
struct Cfg {
  static constexpr uint32_t B_BYTES = (BN / 64) * B_GROUP;
  static constexpr uint32_t STAGE = A_BYTES + B_BYTES;
  static constexpr int NS = BN == 256 ? 4 : BN == 128 ? 5 : 6;
  // a LoRA stage: v tile [128 x 32 ranks] in 128-byte rows (half of each row used) + B rows [32 x BN]
  static constexpr uint32_t EB_GROUP = ER * 128;
  static constexpr uint32_t EXT = A_BYTES + (BN / 64) * EB_GROUP;
  static constexpr int NE = BN == 256 ? 1 : BN == 128 ? 2 : 4;
  static constexpr uint32_t OFF_EXT = NS * STAGE;
  static constexpr uint32_t OFF_BAR = OFF_EXT + NE * EXT;
  static constexpr uint32_t SMEM = OFF_BAR + 256 + 1024;      // barriers and bookkeeping; slack for 1024-byte alignment
  static constexpr uint32_t TMEM_COLS = 2 * BN;               // two accumulators
  static_assert(TMEM_COLS == 512 || TMEM_COLS == 256 || TMEM_COLS == 128, "TMEM allocations are powers of two");
  static_assert(SMEM <= 227 * 1024, "shared memory");
  static_assert(EXT % 1024 == 0 && STAGE % 1024 == 0, "operand tiles start on 1024-byte boundaries");
};

struct LinArgs {
  PoolView pv;
  const float* v;              // shrink partial sums [projection][slice][token][rmax]
  int ksplit, rmax;
  float scale;
  const int32_t* seg_indptr;
  const int32_t* lora_ids;
  int n_seg, n_tokens, d_in;
  int n_mats;
  __nv_bfloat16* y[MAX_LIN];
  int d_out[MAX_LIN], mat_index[MAX_LIN], n_tiles_n[MAX_LIN], tile_base[MAX_LIN + 1];
  int m_tiles;
  const int* ext_count;        // per 128-token tile: LoRA stages (32 ranks of one overlapping segment's adapter)
  const int* ext_list;         // [m_tiles][EXT_CAP]: segment << 1 | which half of the ranks
  // K / V projections whose rows go straight into the requests' pool blocks (kv_side: -1 = rows go to y, 0 = K, 1 = V)
  int kv_side[MAX_LIN];
  const int32_t* req_indptr;
  const int32_t* tbl_indptr;
  const uint32_t* tbl;
  const int32_t* prefix_lens;
  int n_req, n_kv, bt;
};

struct LinMaps {
  CUtensorMap x;
  CUtensorMap w[MAX_LIN];
};

struct Tile {
  int j, m, n;       // projection, token tile, column tile
};
__device__ __forceinline__ Tile decode_tile(const LinArgs& a, int idx) {
  Tile t;
  t.j = 0;
  while (t.j + 1 < a.n_mats && idx >= a.tile_base[t.j + 1]) ++t.j;
  const int local = idx - a.tile_base[t.j];
  t.m = local / a.n_tiles_n[t.j];
  t.n = local - t.m * a.n_tiles_n[t.j];
  return t;
}

template <int BN, int RMAX>
__global__ void __launch_bounds__(LT_THREADS, 1) lora_linear_kernel(const LinArgs a, const __grid_constant__ LinMaps maps) {
  using C = Cfg<BN>;
  constexpr int NS = C::NS;
  extern __shared__ unsigned char smem_raw[];
  // the swizzled operand tiles need 1024-byte alignment
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  constexpr int NE = C::NE;
  enum { B_FULL = 0, B_EMPTY = NS, B_ACC_FULL = 2 * NS, B_ACC_EMPTY = 2 * NS + 2, B_EFULL = 2 * NS + 4,
         B_EEMPTY = B_EFULL + NE, B_COUNT = B_EEMPTY + NE };
  const uint32_t bar0 = sbase + C::OFF_BAR;
  auto bar = [&](int k) { return bar0 + 8u * k; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_BAR + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * B_COUNT + 4);
  volatile int* ext_ksteps = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * B_COUNT + 8);   // [NE]
  static_assert(8 * B_COUNT + 8 + 4 * NE <= 256, "bookkeeping area too small");

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(bar(B_FULL + s), 1);
      mbar_init(bar(B_EMPTY + s), 1);
    }
    for (int e = 0; e < NE; ++e) {
      mbar_init(bar(B_EFULL + e), 1);
      mbar_init(bar(B_EEMPTY + e), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(B_ACC_FULL + b), 1);
      mbar_init(bar(B_ACC_EMPTY + b), 4);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(C::TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  pdl_wait();     // x, the shrink's partial sums and the plan are the work of the kernels before this one

  const int total = a.tile_base[a.n_mats];
  const int nk = (a.d_in + BK - 1) / BK;

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (one lane)
    if (lane == 0) {
      long long f = 0;       // main stages so far
      bool ok = true;
      for (int idx = blockIdx.x; ok && idx < total; idx += gridDim.x) {
        const Tile t = decode_tile(a, idx);
        const CUtensorMap* wm = &maps.w[t.j];
        for (int ks = 0; ks < nk; ++ks, ++f) {
          const int s = (int)(f % NS);
          const long long use = f / NS;
          if (use > 0) ok = mbar_wait(bar(B_EMPTY + s), (uint32_t)((use - 1) & 1), abort_flag);
          if (!ok) break;
          mbar_expect_tx(bar(B_FULL + s), C::STAGE);
          const uint32_t dst = sbase + s * C::STAGE;
          tma_load_2d(dst, &maps.x, bar(B_FULL + s), ks * BK, t.m * BM);
#pragma unroll
          for (int g = 0; g < BN / 64; ++g)
            tma_load_2d(dst + A_BYTES + g * B_GROUP, wm, bar(B_FULL + s), t.n * BN + g * 64, ks * BK);
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer (one lane)
    if (lane == 0) {
      constexpr uint32_t IDESC = instr_desc(BN, true);     // A (x, v) K-major, B (W, adapter rows) N-contiguous
      long long f = 0, g = 0;      // main stages and LoRA stages so far
      bool ok = true;
      int k = 0;             // tiles of this CTA so far
      for (int idx = blockIdx.x; ok && idx < total; idx += gridDim.x, ++k) {
        const Tile t = decode_tile(a, idx);
        const int n_ext = a.ext_count[t.m];
        const int buf = k & 1;
        if (k >= 2) ok = mbar_wait(bar(B_ACC_EMPTY + buf), (uint32_t)(((k >> 1) - 1) & 1), abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem + buf * BN;
        uint32_t acc = 0;
        for (int e = 0; e < n_ext; ++e, ++g) {
          const int s = (int)(g % NE);
          ok = mbar_wait(bar(B_EFULL + s), (uint32_t)((g / NE) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          const int steps = min(ext_ksteps[s], ER / 16);
          const uint32_t ab = sbase + C::OFF_EXT + s * C::EXT, bb = ab + A_BYTES;
          for (int ks = 0; ks < steps; ++ks) {
            umma_bf16(d_tmem, smem_desc(ab + ks * 32, 16, 1024), smem_desc(bb + ks * (16 * 128), C::EB_GROUP, 1024), IDESC, acc);
            acc = 1;
          }
          umma_commit(bar(B_EEMPTY + s));
        }
        if (!ok) break;
        for (int st = 0; st < nk; ++st, ++f) {
          const int s = (int)(f % NS);
          ok = mbar_wait(bar(B_FULL + s), (uint32_t)((f / NS) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t ab = sbase + s * C::STAGE, bb = ab + A_BYTES;
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks) {
            umma_bf16(d_tmem, smem_desc(ab + ks * 32, 16, 1024), smem_desc(bb + ks * (16 * 128), B_GROUP, 1024), IDESC, acc);
            acc = 1;
          }
          umma_commit(bar(B_EMPTY + s));
        }
        if (ok) umma_commit(bar(B_ACC_FULL + buf));
      }
    }
  } else {
    // ------------------------------------------------ LoRA stage filler + epilogue (128 threads; thread = token row = TMEM lane)
    const int et = tid - 64;                 // 0..127
    const int quarter = warp & 3;            // the TMEM lanes this warp may touch
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    long long g = 0;                         // LoRA stages so far
    bool ok = true;
    int k = 0;
    // fills the LoRA stages of tile `idx`
    auto fill_ext = [&](int idx) {
      const Tile t = decode_tile(a, idx);
      const int n_ext = a.ext_count[t.m];
      const int tok = t.m * BM + row;
      const int n0 = t.n * BN;
      const int d_out = a.d_out[t.j];
      for (int e = 0; ok && e < n_ext; ++e, ++g) {
        const int entry = a.ext_list[(size_t)t.m * EXT_CAP + e];
        const int sg = entry >> 1, r0 = (entry & 1) * ER;
        const int lid = a.lora_ids[sg];
        const LoraEntry* en = a.pv.dir + lid;
        const int rank = min(en->rank, RMAX);
        const int nr = max(0, min(ER, rank - r0));       // ranks of this stage
        const int steps = (nr + 15) >> 4;
        const LoraMat lm = en->mats[a.mat_index[t.j]];
        const uint32_t table_off = en->table_off;
        const bool mine = tok >= a.seg_indptr[sg] && tok < a.seg_indptr[sg + 1] && tok < a.n_tokens;
        // this row of v (ranks r0 ..): slices summed; everything is in registers before the slot is waited for
        constexpr int VR = RMAX < ER ? RMAX : ER;
        float vr[VR];
#pragma unroll
        for (int c = 0; c < VR; ++c) vr[c] = 0.f;
        if (mine) {
          for (int sp = 0; sp < a.ksplit; ++sp) {
            const float4* src = reinterpret_cast<const float4*>(
                a.v + ((size_t)(t.j * a.ksplit + sp) * a.n_tokens + tok) * RMAX + r0);
#pragma unroll
            for (int c = 0; c < VR / 4; ++c) {
              if (4 * c < 16 * steps) {
                const float4 p4 = src[c];
                vr[4 * c] += p4.x; vr[4 * c + 1] += p4.y; vr[4 * c + 2] += p4.z; vr[4 * c + 3] += p4.w;
              }
            }
          }
        }
        // the adapter's B rows r0 .. of this tile's columns: 16-byte chunk c of the [32 x BN] tile, c = et + 128 i
        constexpr int BCH = ER * BN / 8 / 128;      // chunks per thread
        constexpr int CPR = BN / 8;                 // chunks per row
        uint4 bq[BCH];
#pragma unroll
        for (int i = 0; i < BCH; ++i) {
          const int c = et + 128 * i;
          const int r = c / CPR, cc = c % CPR;
          bq[i] = make_uint4(0u, 0u, 0u, 0u);
          if (r < nr && n0 + cc * 8 < d_out) {
            const uint32_t gr = lm.b_row0 + (uint32_t)(r0 + r);
            const uint32_t blk = a.pv.tables[table_off + lm.b_tab + gr / lm.b_rpb];
            if (blk >= a.pv.n_blocks) {
              atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_BLOCK);
            } else {
              const unsigned char* rp = a.pv.slab + (size_t)blk * a.pv.block_bytes + (size_t)(gr % lm.b_rpb) * 2 * (size_t)d_out;
              bq[i] = __ldg(reinterpret_cast<const uint4*>(rp + (size_t)(n0 + cc * 8) * 2));
            }
          }
        }
        const int s = (int)(g % NE);
        const long long use = g / NE;
        // the 128 threads decide together (a wait that gave up in one of them ends the loop for all: they meet at a
        // named barrier further down)
        if (use > 0) ok = group_and(mbar_wait(bar(B_EEMPTY + s), (uint32_t)((use - 1) & 1), abort_flag), 1, 128);
        if (!ok) break;
        unsigned char* as = smem + C::OFF_EXT + s * C::EXT;
        unsigned char* bs = as + A_BYTES;
#pragma unroll
        for (int c8 = 0; c8 < VR / 8; ++c8) {
          if (c8 < 2 * steps) {
            uint4 q;
            q.x = pack_bf16(vr[8 * c8] * a.scale, vr[8 * c8 + 1] * a.scale);
            q.y = pack_bf16(vr[8 * c8 + 2] * a.scale, vr[8 * c8 + 3] * a.scale);
            q.z = pack_bf16(vr[8 * c8 + 4] * a.scale, vr[8 * c8 + 5] * a.scale);
            q.w = pack_bf16(vr[8 * c8 + 6] * a.scale, vr[8 * c8 + 7] * a.scale);
            *reinterpret_cast<uint4*>(as + row * 128 + ((c8 ^ (row & 7)) << 4)) = q;
          }
        }
#pragma unroll
        for (int i = 0; i < BCH; ++i) {
          const int c = et + 128 * i;
          const int r = c / CPR, cc = c % CPR;
          if (r < 16 * steps)
            *reinterpret_cast<uint4*>(bs + (cc >> 3) * C::EB_GROUP + r * 128 + (((cc & 7) ^ (r & 7)) << 4)) = bq[i];
        }
        fence_async_smem();                            // the tensor core reads shared memory through the async proxy
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (et == 0) {
          ext_ksteps[s] = steps;
          mbar_arrive(bar(B_EFULL + s));
        }
      }
    };
    int idx = blockIdx.x;
    if (idx < total) fill_ext(idx);
    for (; ok && idx < total; idx += gridDim.x, ++k) {
      const Tile t = decode_tile(a, idx);
      // the next tile's LoRA stages go in before this tile's epilogue: the issuer needs them the moment this
      // tile's last MMA is out
      if (idx + (int)gridDim.x < total) fill_ext(idx + gridDim.x);
      if (!ok) break;
      const int buf = k & 1;
      const int tok = t.m * BM + row;
      const int d_out = a.d_out[t.j];
      const int n0 = t.n * BN;
      const int side = a.kv_side[t.j];
      // a K / V row belongs in its token's pool block: block and slot of the token's position, found while the
      // tile's MMAs are still running
      uint32_t kv_blk = 0;
      int kv_slot = -1, kv_last = 0;
      if (side >= 0 && tok < a.n_tokens) {
        int lo = 0, hi = a.n_req;
        while (hi - lo > 1) {
          const int mid = (lo + hi) >> 1;
          if (a.req_indptr[mid] <= tok) lo = mid; else hi = mid;
        }
        const int pos = a.prefix_lens[lo] + (tok - a.req_indptr[lo]);
        const int entry = pos / a.bt, slot = pos - entry * a.bt;
        if (pos < 0 || tok < a.req_indptr[lo] || tok >= a.req_indptr[lo + 1] || entry >= a.tbl_indptr[lo + 1] - a.tbl_indptr[lo]) {
          atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
        } else {
          const uint32_t blk = a.tbl[a.tbl_indptr[lo] + entry];
          if (blk >= a.pv.n_blocks) {
            atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_BLOCK);
          } else {
            kv_blk = blk;
            kv_slot = slot;
            kv_last = tok == a.req_indptr[lo + 1] - 1;
          }
        }
      }
      ok = group_and(mbar_wait(bar(B_ACC_FULL + buf), (uint32_t)((k >> 1) & 1), abort_flag), 1, 128);
      if (!ok) break;
      tc_fence_after();
      __nv_bfloat16* yrow = side < 0 ? a.y[t.j] + (size_t)tok * d_out + n0 : nullptr;
#pragma unroll 2
      for (int cb = 0; cb < BN; cb += 32) {
        uint32_t o[32];
        tmem_ld32(lane_addr + buf * BN + cb, o);
        tmem_wait_ld();
        if (tok < a.n_tokens) {
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            if (n0 + cb + 8 * c < d_out) {
              uint4 q;
              q.x = pack_bf16(__uint_as_float(o[8 * c + 0]), __uint_as_float(o[8 * c + 1]));
              q.y = pack_bf16(__uint_as_float(o[8 * c + 2]), __uint_as_float(o[8 * c + 3]));
              q.z = pack_bf16(__uint_as_float(o[8 * c + 4]), __uint_as_float(o[8 * c + 5]));
              q.w = pack_bf16(__uint_as_float(o[8 * c + 6]), __uint_as_float(o[8 * c + 7]));
              if (side < 0) {
                *reinterpret_cast<uint4*>(yrow + cb + 8 * c) = q;
              } else if (kv_slot >= 0) {
                // [K|V][kv head][slot][128] inside the block
                const int colg = n0 + cb + 8 * c;
                unsigned char* dst = a.pv.slab + (size_t)kv_blk * a.pv.block_bytes +
                                     ((size_t)(side * a.n_kv + colg / FL_HEAD_DIM) * a.bt + kv_slot) * (FL_HEAD_DIM * 2) +
                                     (colg % FL_HEAD_DIM) * 2;
                *reinterpret_cast<uint4*>(dst) = q;
                if (side == 1 && kv_last)       // V of a request's last token: clear the slots behind it
                  for (int z = kv_slot + 1; z < a.bt; ++z)
                    *reinterpret_cast<uint4*>(dst + (z - kv_slot) * (FL_HEAD_DIM * 2)) = make_uint4(0u, 0u, 0u, 0u);
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_ACC_EMPTY + buf));
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    // copies still in flight target this CTA's shared memory: give every armed barrier a bounded chance to complete
    if (warp == 0 && lane == 0) {
      for (int s = 0; s < NS; ++s)
        for (uint32_t i = 0; i < (1u << 16); ++i)
          if (mbar_try(bar(B_FULL + s), 0) || mbar_try(bar(B_FULL + s), 1)) break;   // (an idle barrier answers at once)
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
  }
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

struct LinWs {
  size_t v, ext_count, ext_list, total;
  int m_tiles;
};
LinWs lin_ws(int n_tokens, int n_mats) {
  LinWs w;
  w.m_tiles = (n_tokens + BM - 1) / BM;
  size_t off = 0;
  w.v = off; off = align256(off + fl_lora_sgmv_workspace(n_tokens, n_mats));
  w.ext_count = off; off = align256(off + sizeof(int) * (size_t)w.m_tiles);
  w.ext_list = off; off = align256(off + sizeof(int) * (size_t)w.m_tiles * EXT_CAP);
  w.total = off;
  return w;
}

template <int BN, int RMAX>
int launch_linear(fl_pool* p, const LinArgs& a, const LinMaps& maps, cudaStream_t st) {
  using C = Cfg<BN>;
  static bool configured[16] = {};
  if (!configured[p->device & 15]) {
    FL_CUDA(p, cudaFuncSetAttribute(lora_linear_kernel<BN, RMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM));
    configured[p->device & 15] = true;
  }
  const int total = a.tile_base[a.n_mats];
  const unsigned grid = (unsigned)std::min(total, p->sm_count);
  FL_CUDA(p, launch_pdl(lora_linear_kernel<BN, RMAX>, dim3(grid), dim3(LT_THREADS), C::SMEM, st, a, maps));
  FL_CUDA(p, cudaGetLastError());
  return FL_OK;
}

int launch_width(fl_pool* p, const LinArgs& a, const LinMaps& maps, cudaStream_t st, int bn, int rmax) {
  if (bn == 256)
    return rmax == 16 ? launch_linear<256, 16>(p, a, maps, st)
         : rmax == 32 ? launch_linear<256, 32>(p, a, maps, st) : launch_linear<256, 64>(p, a, maps, st);
  if (bn == 128)
    return rmax == 16 ? launch_linear<128, 16>(p, a, maps, st)
         : rmax == 32 ? launch_linear<128, 32>(p, a, maps, st) : launch_linear<128, 64>(p, a, maps, st);
  return rmax == 16 ? launch_linear<64, 16>(p, a, maps, st)
       : rmax == 32 ? launch_linear<64, 32>(p, a, maps, st) : launch_linear<64, 64>(p, a, maps, st);
}

}  // namespace

extern "C" {

size_t fl_lora_linear_workspace(int n_tokens, int n_mats) {
  if (n_tokens <= 0 || n_mats <= 0) return 256;
  return lin_ws(n_tokens, n_mats).total;
}

}  // extern "C"

namespace {

struct LinKv {        // K and V projections of the call whose rows go into pool blocks
  int k_slot, v_slot;
  const int32_t* req_indptr;
  const int32_t* tbl_indptr;
  const uint32_t* tbl;
  const int32_t* prefix_lens;
  int n_req, n_kv;
  fl_bf16* tmp_k;     // [n_tokens, n_kv * 128] each: needed by batches of short segments only
  fl_bf16* tmp_v;
};

int linear_common(fl_pool* p, fl_bf16* const* ys_in, const fl_bf16* x, const fl_bf16* const* ws, const int* mat_indices,
                  int n_mats, const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                  float scale, void* workspace, size_t workspace_bytes, fl_stream stream, const LinKv* kv) {
  if (!p || n_mats < 1 || n_mats > MAX_LIN || n_seg < 0 || n_tokens < 0 || !ys_in || !ws || !mat_indices) return FL_EINVAL;
  fl_bf16* ys[MAX_LIN] = {};
  for (int j = 0; j < n_mats; ++j) ys[j] = ys_in[j];
  if (n_tokens == 0) return FL_OK;
  if (!x || !workspace || (n_seg > 0 && (!seg_indptr || !lora_ids))) return FL_EINVAL;
  if (p->n_mats == 0) return FL_EBADID;           // the projection shapes come with the first registered adapter
  const LinWs lw = lin_ws(n_tokens, n_mats);
  if (workspace_bytes < lw.total) return FL_ENOMEM;
  LinArgs a;
  memset(&a, 0, sizeof(a));
  a.pv = p->view();
  int d_out_min = 1 << 30;
  for (int j = 0; j < n_mats; ++j) {
    const int mi = mat_indices[j];
    const bool to_pool = kv && (j == kv->k_slot || j == kv->v_slot);
    if (mi < 0 || mi >= p->n_mats || (!ys[j] && !to_pool) || !ws[j]) return FL_EINVAL;
    if (p->mats[mi].d_in != p->mats[mat_indices[0]].d_in) return FL_EINVAL;   // the projections share x
    a.y[j] = reinterpret_cast<__nv_bfloat16*>(ys[j]);
    a.mat_index[j] = mi;
    a.d_out[j] = p->mats[mi].d_out;
    d_out_min = std::min(d_out_min, a.d_out[j]);
  }
  a.d_in = p->mats[mat_indices[0]].d_in;
  a.n_mats = n_mats;
  a.seg_indptr = seg_indptr;
  a.lora_ids = lora_ids;
  a.n_seg = n_seg;
  a.n_tokens = n_tokens;
  a.scale = scale;
  unsigned char* wsb = reinterpret_cast<unsigned char*>(workspace);
  a.v = reinterpret_cast<const float*>(wsb + lw.v);
  int* ext_count = reinterpret_cast<int*>(wsb + lw.ext_count);
  int* ext_list = reinterpret_cast<int*>(wsb + lw.ext_list);
  a.ext_count = ext_count;
  a.ext_list = ext_list;
  a.m_tiles = lw.m_tiles;
  // Segments of a few tokens each (a decode batch): a 128-token tile would take one LoRA stage per segment, each
  // for a handful of rows, and y is small next to W.  Then the GEMM computes x W alone (no LoRA stages in the plan)
  // and the segmented projection adds the LoRA term to y afterwards.
  const bool hybrid = n_seg > 0 && n_tokens <= 16 * n_seg;
  if (hybrid) a.n_seg = 0;
  for (int j = 0; j < MAX_LIN; ++j) a.kv_side[j] = -1;
  if (kv) {
    const size_t per_tok = (size_t)2 * kv->n_kv * FL_HEAD_DIM * 2;
    if (kv->n_kv < 1 || kv->n_req < 1 || p->block_bytes % per_tok != 0 || kv->k_slot == kv->v_slot) return FL_EINVAL;
    if (!kv->req_indptr || !kv->tbl_indptr || !kv->tbl || !kv->prefix_lens) return FL_EINVAL;
    for (int side = 0; side < 2; ++side) {
      const int slot = side ? kv->v_slot : kv->k_slot;
      if (slot < 0 || slot >= n_mats || a.d_out[slot] != kv->n_kv * FL_HEAD_DIM) return FL_EINVAL;
      if (hybrid) {      // x W goes to a scratch row first; the segmented projection then stores base + LoRA term in the pool
        fl_bf16* tmp = side ? kv->tmp_v : kv->tmp_k;
        if (!tmp) return FL_EINVAL;
        ys[slot] = tmp;
        a.y[slot] = reinterpret_cast<__nv_bfloat16*>(tmp);
      } else {
        a.kv_side[slot] = side;
      }
    }
    a.req_indptr = kv->req_indptr;
    a.tbl_indptr = kv->tbl_indptr;
    a.tbl = kv->tbl;
    a.prefix_lens = kv->prefix_lens;
    a.n_req = kv->n_req;
    a.n_kv = kv->n_kv;
    a.bt = (int)(p->block_bytes / per_tok);
  }
  // few token tiles: narrower column tiles, so that every SM streams a slice of W.  Among 256, 128 and 64 columns the
  // width with the least bytes through the busiest SM wins: rounds of tiles over the SMs times what a tile pulls per
  // k-stage (its W slice and its x rows).
  int bn = 256;
  {
    auto tiles = [&](int w) {
      long t = 0;
      for (int j = 0; j < n_mats; ++j) t += (long)lw.m_tiles * ((a.d_out[j] + w - 1) / w);
      return t;
    };
    if (tiles(256) < p->sm_count || hybrid) {
      long best = -1;
      for (int w = 256; w >= 64; w /= 2) {
        const long cost = ((tiles(w) + p->sm_count - 1) / p->sm_count) * (w + BM);
        if (best < 0 || cost < best) { best = cost; bn = w; }
      }
    }
  }
  a.tile_base[0] = 0;
  for (int j = 0; j < n_mats; ++j) {
    a.n_tiles_n[j] = (a.d_out[j] + bn - 1) / bn;
    a.tile_base[j + 1] = a.tile_base[j] + lw.m_tiles * a.n_tiles_n[j];
  }
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != p->device) cudaSetDevice(p->device);
  const cudaStream_t st = (cudaStream_t)stream;
  int rc = FL_OK;
  do {
    alignas(64) LinMaps maps;
    {
      const uint64_t dims[2] = {(uint64_t)a.d_in, (uint64_t)n_tokens};
      const uint64_t strides[1] = {(uint64_t)a.d_in * 2};
      const uint32_t box[2] = {BK, BM};
      rc = tmap::encode_bf16(&maps.x, x, 2, dims, strides, box);
      if (rc != FL_OK) break;
    }
    for (int j = 0; j < n_mats && rc == FL_OK; ++j) {
      const uint64_t dims[2] = {(uint64_t)a.d_out[j], (uint64_t)a.d_in};
      const uint64_t strides[1] = {(uint64_t)a.d_out[j] * 2};
      const uint32_t box[2] = {64, BK};
      rc = tmap::encode_bf16(&maps.w[j], ws[j], 2, dims, strides, box);
    }
    for (int j = n_mats; j < MAX_LIN; ++j) maps.w[j] = maps.w[0];
    if (rc != FL_OK) break;
    lora_plan::PlanArgs pa;
    pa.pv = a.pv;
    pa.seg_indptr = a.seg_indptr;
    pa.lora_ids = a.lora_ids;
    pa.n_seg = a.n_seg;
    pa.n_tokens = n_tokens;
    pa.m_tiles = lw.m_tiles;
    pa.n_mats = n_mats;
    for (int j = 0; j < FL_MAX_MATS; ++j) pa.mat_index[j] = j < n_mats ? a.mat_index[j] : 0;
    if (lora_plan::launch_plan(pa, ext_count, ext_list, st) != cudaSuccess) {
      p->last_cuda = (int)cudaGetLastError();
      rc = FL_ECUDA;
      break;
    }
    sgmv::ShrinkInfo info = {1, p->max_rank <= 16 ? 16 : (p->max_rank <= 32 ? 32 : 64)};
    if (hybrid) {
      // y = x W from the GEMM alone, then the segmented projection adds the LoRA term to it
      a.ksplit = 1;
      a.rmax = info.rmax;
      rc = launch_width(p, a, maps, st, bn, info.rmax);
      if (rc != FL_OK) break;
      if (kv && n_mats == 3 && kv->k_slot == 1 && kv->v_slot == 2)
        rc = fl_lora_sgmv_qkv_append(p, ys[0], ys[1], ys[2], x, mat_indices[0], mat_indices[1], mat_indices[2], seg_indptr,
                                     lora_ids, n_seg, n_tokens, scale, kv->req_indptr, kv->tbl_indptr, kv->tbl,
                                     kv->prefix_lens, kv->n_req, kv->n_kv, wsb + lw.v,
                                     fl_lora_sgmv_workspace(n_tokens, n_mats), stream);
      else if (kv)
        rc = FL_EINVAL;
      else
        rc = fl_lora_sgmv_multi(p, ys, x, mat_indices, n_mats, seg_indptr, lora_ids, n_seg, n_tokens, scale, wsb + lw.v,
                                fl_lora_sgmv_workspace(n_tokens, n_mats), stream);
      break;
    }
    if (n_seg > 0) {
      rc = sgmv::shrink(p, x, mat_indices, n_mats, seg_indptr, lora_ids, n_seg, n_tokens, wsb + lw.v,
                        fl_lora_sgmv_workspace(n_tokens, n_mats), stream, &info);
      if (rc != FL_OK) break;
    }
    a.ksplit = info.ksplit;
    a.rmax = info.rmax;
    rc = launch_width(p, a, maps, st, bn, info.rmax);
  } while (0);
  if (prev != p->device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

}  // namespace

extern "C" {

int fl_lora_linear_multi(fl_pool* p, fl_bf16* const* ys, const fl_bf16* x, const fl_bf16* const* ws, const int* mat_indices,
                         int n_mats, const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                         float scale, void* workspace, size_t workspace_bytes, fl_stream stream) {
  return linear_common(p, ys, x, ws, mat_indices, n_mats, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace,
                       workspace_bytes, stream, nullptr);
}

int fl_lora_linear_qkv_append(fl_pool* p, fl_bf16* y_q, const fl_bf16* x, const fl_bf16* w_q, const fl_bf16* w_k,
                              const fl_bf16* w_v, int mat_q, int mat_k, int mat_v, const int32_t* seg_indptr,
                              const int32_t* lora_ids, int n_seg, int n_tokens, float scale, const int32_t* req_indptr,
                              const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens, int n_req,
                              int n_kv_heads, fl_bf16* scratch_k, fl_bf16* scratch_v, void* workspace,
                              size_t workspace_bytes, fl_stream stream) {
  fl_bf16* ys[3] = {y_q, nullptr, nullptr};
  const fl_bf16* ws[3] = {w_q, w_k, w_v};
  const int mi[3] = {mat_q, mat_k, mat_v};
  const LinKv kv = {1, 2, req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_kv_heads, scratch_k, scratch_v};
  return linear_common(p, ys, x, ws, mi, 3, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace, workspace_bytes,
                       stream, &kv);
}

int fl_lora_linear(fl_pool* p, fl_bf16* y, const fl_bf16* x, const fl_bf16* w, int mat_index,
                   const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                   float scale, void* workspace, size_t workspace_bytes, fl_stream stream) {
  fl_bf16* ys[1] = {y};
  const fl_bf16* ws[1] = {w};
  const int mi[1] = {mat_index};
  return fl_lora_linear_multi(p, ys, x, ws, mi, 1, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace,
                              workspace_bytes, stream);
}

}  // extern "C"
