// Prefill attention, two query tiles per CTA sharing one K/V stream, persistent CTAs (Section 2.1 / 4.2:
// attention over the reused prefix KV plus the new tokens, read in place from pool blocks).
//
// One CTA per SM.  A work unit is 2 x 128 query rows of one (request, KV head): with grouped heads the two
// tiles are two query heads over the same 128 new tokens, otherwise two consecutive 128-token tiles of
// one head.  Both tiles read the same K/V tiles, so every pool page is staged into shared memory once
// for 256 query rows.  CTAs take units from a counter in device memory until none is left; the loads of
// the next unit start while the current one is still in its last tiles and its epilogue.
//   warps 0-3   softmax of tile A (thread = query row = TMEM lane)      warp 8   TMA producer, unit fetch
//   warps 4-7   softmax of tile B                                        warp 9   MMA issuer, TMEM owner
//   (warps 10, 11 only complete the third warpgroup, whose registers go to the softmax warpgroups)
//   K_j / V_j (128 keys = 8 pool pages each, one 4 KiB TMA box per page) -> ring of 32 KiB slots, 128-byte swizzle;
//   a page lands as [8-key group][64-value half][8 keys][64 values], so a tile's 8-key groups are 2 KiB apart
//   S_X = Q_X K_j^T     tcgen05.mma 128x128x16 (x8) into TMEM columns of tile X
//   P_X = exp2(S_X - m) -> bf16 pairs written back over the first half of S_X in TMEM
//   O_X += P_X V_j      tcgen05.mma with the A operand read from TMEM, V MN-major as stored
// The issuer alternates the tiles (PV_A, S_A, PV_B, S_B): while one tile's softmax runs, the tensor pipe
// works for the other.  MMAs of one thread execute in issue order, so S_X(j+1) may overwrite P_X(j)
// without a barrier, "S_X(j+1) complete" implies "PV_X(j) complete", and the first PV of a unit cannot
// start before every softmax warp has finished the previous unit's epilogue (it waits for their P).
// O is rescaled only when a row maximum grew by more than 2^8.  Every mbarrier wait is bounded; a wait
// that gives up raises a sticky flag, the CTA drains its copies and frees its TMEM.
#include <cuda.h>
#include <math.h>
#include <string.h>
#include <algorithm>
#include "attention.cuh"
#include "mma_utils.cuh"
#include "tc_ptx.cuh"
#include "tmap.cuh"

namespace attn {
namespace {

using namespace tc;

constexpr int T2_THREADS = 384;                        // three warpgroups: softmax A, softmax B, {TMA, MMA, 2 idle warps}
constexpr int KT2 = 128;                               // keys per tile
constexpr int NSLOT = 5;                               // ring slots; fills go K_0, V_0, K_1, V_1, ... across units
constexpr uint32_t HALF_BYTES = 128 * 128;             // [128 rows][64 bf16], swizzled
constexpr uint32_t TILE_BYTES = 2 * HALF_BYTES;        // a Q, K or V tile
constexpr uint32_t PAGE_BYTES = BT * 128 * 2;          // K or V of one head of one block: [2 groups][2 halves][8 tokens][64 bf16]
constexpr uint32_t GROUP_BYTES = PAGE_BYTES / 2;       // stride between 8-key groups of a K/V tile
constexpr uint32_t OFF_Q2 = 0;                         // Q_A, Q_B
constexpr uint32_t OFF_RING = 2 * TILE_BYTES;
constexpr uint32_t OFF_BAR2 = OFF_RING + NSLOT * TILE_BYTES;
constexpr uint32_t T2_SMEM = OFF_BAR2 + 512;           // barriers, TMEM address, abort flag, two unit descriptors
constexpr uint32_t T2_TMEM_COLS = 512;                 // S_A | S_B | O_A | O_B, 128 columns each
constexpr float RESCALE_LOG2 = 8.f;

enum { C_QFULL = 0, C_QEMPTY = 1, C_FULL = 2, C_EMPTY = C_FULL + NSLOT, C_SFULL = C_EMPTY + NSLOT, C_PFULL = C_SFULL + 2,
       C_ODONE = C_PFULL + 2, C_UFULL = C_ODONE + 2, C_UEMPTY = C_UFULL + 2, C_COUNT = C_UEMPTY + 2 };
constexpr int UNIT_READERS = 9;                        // MMA issuer + 8 softmax warps

// 32 bytes to a 32-byte aligned global address in one instruction.
__device__ __forceinline__ void st_global_v8(void* dst, const uint32_t* r) {
  asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]),
               "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]) : "memory");
}

struct Unit {           // what a CTA works on at one time
  int tok0[2];          // first token row (in the packed q / out tensors) of each tile
  int hq[2];            // query head of each tile
  int rows[2];          // valid query rows (0 = tile unused)
  int lim0[2];          // last visible key of row 0 of each tile
  int n_kt[2];          // K/V tiles each tile takes part in
  int n_kt_max, n_pages, tbl0, h;
  int valid;            // 0: the unit's table is too short for its keys (skipped by every role)
  int index;            // -1 = no more work
};

// Unit u = (plan tile u / heads_per_item, head slot u % heads_per_item), decoded once by the producer and handed
// to the other roles through shared memory.
__device__ __forceinline__ Unit decode_unit(const AttnArgs& a, int u, int heads_per_item) {
  Unit t;
  const int item = u / heads_per_item, hslot = u % heads_per_item;
  const int2 it = a.prefill_list[item];
  const int i = it.x, q0 = it.y;
  const int n_new = a.new_lens[i], prefix = a.prefix_lens[i], ctx = prefix + n_new;
  const int group = a.n_q / a.n_kv;
  if (group % 2 == 0) {
    t.hq[0] = 2 * hslot; t.hq[1] = 2 * hslot + 1;
    t.h = t.hq[0] / group;
    t.tok0[0] = t.tok0[1] = a.req_indptr[i] + q0;
    t.rows[0] = t.rows[1] = min(128, n_new - q0);
    t.lim0[0] = t.lim0[1] = prefix + q0;
  } else {
    t.hq[0] = t.hq[1] = hslot;
    t.h = hslot / group;
    t.tok0[0] = a.req_indptr[i] + q0; t.tok0[1] = t.tok0[0] + 128;
    // a request with an odd number of 128-row tiles has its first tile alone (the plan starts its pairs at token 128)
    const bool lone = q0 == 0 && (((n_new + 127) / 128) & 1);
    t.rows[0] = min(128, n_new - q0); t.rows[1] = lone ? 0 : max(0, min(128, n_new - q0 - 128));
    t.lim0[0] = prefix + q0; t.lim0[1] = prefix + q0 + 128;
  }
#pragma unroll
  for (int x = 0; x < 2; ++x) t.n_kt[x] = t.rows[x] > 0 ? (t.lim0[x] + t.rows[x] + KT2 - 1) / KT2 : 0;
  t.n_kt_max = max(t.n_kt[0], t.n_kt[1]);
  const int kv_end = min(ctx, t.n_kt_max * KT2);
  t.tbl0 = a.tbl_indptr[i];
  t.n_pages = (kv_end + BT - 1) / BT;
  t.valid = t.rows[0] >= 1 && t.n_pages >= 1 && t.n_pages <= a.tbl_indptr[i + 1] - t.tbl0;
  t.index = u;
  return t;
}

__global__ void __launch_bounds__(T2_THREADS, 1)
attn_prefill_tc2_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ CUtensorMap q_map,
                        int heads_per_item, int wide_out) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {   // the swizzled operand tiles need 1024-byte alignment
    if (threadIdx.x == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t bar0 = sbase + OFF_BAR2;
  auto bar = [&](int k) { return bar0 + 8u * k; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR2 + 8 * C_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR2 + 8 * C_COUNT + 4);
  Unit* unit_slot = reinterpret_cast<Unit*>(smem + OFF_BAR2 + 8 * C_COUNT + 8);   // [2]
  static_assert(8 * C_COUNT + 8 + 2 * sizeof(Unit) <= 512, "barrier area too small");

  if (tid == 0) {
    mbar_init(bar(C_QFULL), 1);
    mbar_init(bar(C_QEMPTY), 1);
    for (int s = 0; s < NSLOT; ++s) {
      mbar_init(bar(C_FULL + s), 1);
      mbar_init(bar(C_EMPTY + s), 1);
    }
    for (int x = 0; x < 2; ++x) {
      mbar_init(bar(C_SFULL + x), 1);
      mbar_init(bar(C_PFULL + x), 4);
      mbar_init(bar(C_ODONE + x), 1);
      mbar_init(bar(C_UFULL + x), 1);
      mbar_init(bar(C_UEMPTY + x), UNIT_READERS);
    }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(T2_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  // everything above touched only this CTA's shared memory and TMEM; the plan (and q, K, V) are the work of the
  // kernels before this one
  pdl_wait();
  const int n_units = a.hdr->n_prefill * heads_per_item;   // a CTA beyond the last unit finds no work and tears down

  // Readers take the k-th unit of this CTA from slot k & 1 (index -1 = no more work) and release the slot.

  // the softmax warpgroups keep 128 scores per thread in registers: they take the registers the third
  // warpgroup does not need
  if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 72;");
    if (warp == 8) {
      // ------------------------------------------------ unit fetch + TMA producer
      // The whole warp runs the loop; lane 0 fetches units and does the waiting, lanes 0-7 each own one of a tile's eight
      // pages (their block-id loads and their TMA issues run side by side).
      int fill = 0;                    // ring fills so far, over all units
      int n_valid = 0;                 // units whose Q tiles were loaded so far
      bool ok = true;
      for (int k = 0; ok; ++k) {
        if (lane == 0) {
          Unit t;
          t.index = -1;
          t.valid = 0;
          if (k < 2 || mbar_wait(bar(C_UEMPTY + (k & 1)), ((k >> 1) - 1) & 1, abort_flag)) {
            const int u = k == 0 ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(&a.hdr->next_unit, 1);
            if (u < n_units) t = decode_unit(a, u, heads_per_item);
          }
          unit_slot[k & 1] = t;
          mbar_arrive(bar(C_UFULL + (k & 1)));
        }
        __syncwarp();
        const Unit* up = unit_slot + (k & 1);
        if (up->index < 0) break;
        if (!up->valid) {
          if (lane == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
          continue;
        }
        const int n_kt_max = up->n_kt_max, n_pages = up->n_pages, tbl0 = up->tbl0, h = up->h;
        const int rows_b = up->rows[1];
        // Q buffers are free once the previous unit's last S MMA has completed
        if (lane == 0) {
          if (n_valid > 0) ok = mbar_wait(bar(C_QEMPTY), (n_valid - 1) & 1, abort_flag);
          if (ok) mbar_expect_tx(bar(C_QFULL), rows_b > 0 ? 2 * TILE_BYTES : TILE_BYTES);
        }
        ++n_valid;
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
        if (lane < 4 && (lane < 2 || rows_b > 0)) {          // lane = 2 * tile + half
          const int x = lane >> 1, half = lane & 1;
          tma_load_3d(sbase + OFF_Q2 + x * TILE_BYTES + half * HALF_BYTES, &q_map, bar(C_QFULL), 64 * half, up->hq[x], up->tok0[x]);
        }
        for (int j = 0; ok && j < n_kt_max; ++j) {
          // this lane's page of the tile (pages behind the last needed key are masked anyway: re-read the last
          // valid page); K_j and V_j come from the same blocks
          // lane = page: eight lanes issue one 4 KiB box each
          uint32_t blk = 0;
          if (lane < KT2 / BT) {
            blk = a.tbl[tbl0 + min(j * (KT2 / BT) + lane, n_pages - 1)];
            if (blk >= a.pv.n_blocks) {
              atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_BLOCK);
              blk = 0;
            }
          }
#pragma unroll
          for (int side = 0; side < 2; ++side, ++fill) {
            const int s = fill % NSLOT, use = fill / NSLOT;
            if (lane == 0) {
              if (use > 0) ok = mbar_wait(bar(C_EMPTY + s), (use - 1) & 1, abort_flag);
              if (ok) mbar_expect_tx(bar(C_FULL + s), TILE_BYTES);
            }
            ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;     // the transaction count is armed before any copy is issued
            if (!ok) break;
            if (lane < KT2 / BT)
              tma_load_5d(sbase + OFF_RING + s * TILE_BYTES + lane * PAGE_BYTES, &kv_map, bar(C_FULL + s), 0, 0, 0,
                          2 * (side * a.n_kv + h), (int)blk);
          }
        }
      }
    } else if (warp == 9) {
      // ------------------------------------------------ MMA issuer
      // The issuer's own instruction stream is on the critical path of every hand-off (it shares its scheduler with two
      // softmax warps, and the tensor pipe's queue is an instruction or two deep), so the loop is kept lean: the whole warp
      // runs it converged and an elected lane issues a tile's eight MMAs and their commit as one block, descriptors are a
      // fixed high word and a low word that steps by constants, ring slot and phase are running counters, and a barrier is
      // tested once before the bounded wait loop is entered.
      constexpr uint32_t IDESC = instr_desc(128, false);        // S: both operands K-major
      constexpr uint32_t IDESC_PV = instr_desc(D, true);        // O: V is MN-major
      constexpr uint32_t HI_Q = desc_hi(1024), HI_KV = desc_hi(GROUP_BYTES);
      const uint32_t q_lo[2] = {desc_lo(sbase + OFF_Q2, 16), desc_lo(sbase + OFF_Q2 + TILE_BYTES, 16)};
      const uint32_t ring_k_lo = desc_lo(sbase + OFF_RING, 16), ring_v_lo = desc_lo(sbase + OFF_RING, 1024);
      struct Cur {                     // a position in the K/V ring: slot and the parity of its current use
        int s;
        uint32_t ph;
        __device__ Cur next() const { return s + 1 == NSLOT ? Cur{0, ph ^ 1u} : Cur{s + 1, ph}; }
      };
      Cur cur{0, 0};                   // K_0 of the next unit
      uint32_t ph_p[2] = {0, 0};       // parity of the next P tile per tile (C_PFULL)
      uint32_t ph_q = 0;               // parity of the next unit's Q (C_QFULL)
      auto wait_all = [&](uint32_t b, uint32_t parity) {
        if (__all_sync(0xffffffffu, mbar_try(b, parity))) return true;       // the common case: one test
        return __all_sync(0xffffffffu, mbar_wait(b, parity, abort_flag)) != 0;
      };
      auto wait_full = [&](Cur c) { return wait_all(bar(C_FULL + c.s), c.ph); };
      auto issue_s = [&](int x, Cur c) {
        umma_s_tile_elect(tmem + x * 128, q_lo[x], ring_k_lo + (uint32_t)c.s * (TILE_BYTES >> 4), HI_Q, HI_KV, IDESC, bar(C_SFULL + x));
      };
      auto issue_pv = [&](int x, Cur c, bool first, bool last) {
        umma_pv_tile_elect(tmem + 256 + x * 128, tmem + x * 128, ring_v_lo + (uint32_t)c.s * (TILE_BYTES >> 4), HI_KV, IDESC_PV,
                           first ? 0u : 1u);
        if (last) umma_commit_elect(bar(C_ODONE + x));
      };
      bool ok = true;
      for (int k = 0; ok; ++k) {
        if (!wait_all(bar(C_UFULL + (k & 1)), (k >> 1) & 1)) break;
        const int u_index = unit_slot[k & 1].index, u_valid = unit_slot[k & 1].valid;
        const int n_kt = unit_slot[k & 1].n_kt_max, nA = unit_slot[k & 1].n_kt[0], nB = unit_slot[k & 1].n_kt[1];
        __syncwarp();
        if (lane == 0 && u_index >= 0) mbar_arrive(bar(C_UEMPTY + (k & 1)));
        if (u_index < 0) break;
        if (!u_valid) continue;
        Cur ck = cur;                  // K_j; V_j and K_(j+1) follow it in the ring
        ok = wait_all(bar(C_QFULL), ph_q) && wait_full(ck);
        if (!ok) break;
        ph_q ^= 1u;
        tc_fence_after();
        if (nA > 0) issue_s(0, ck);
        if (nB > 0) issue_s(1, ck);
        umma_commit_elect(bar(C_EMPTY + ck.s));
        if (n_kt == 1) umma_commit_elect(bar(C_QEMPTY));
        for (int j = 0; ok && j < n_kt; ++j) {
          const bool more = j + 1 < n_kt;
          const Cur cv = ck.next(), cn = cv.next();
          // V_j and K_(j+1) landed long ago as a rule: both tests go first, where the tensor pipe still works on S_B or waits
          // for tile A's softmax anyway, and not between tile A's two MMA groups
          ok = wait_full(cv) && (!more || wait_full(cn));
          if (ok && j < nA) {
            ok = wait_all(bar(C_PFULL + 0), ph_p[0]);
            ph_p[0] ^= 1u;
            if (ok) { tc_fence_after(); issue_pv(0, cv, j == 0, j == nA - 1); }
          }
          if (!ok) break;
          if (j + 1 < nA) issue_s(0, cn);
          if (j < nB) {
            ok = wait_all(bar(C_PFULL + 1), ph_p[1]);
            ph_p[1] ^= 1u;
            if (!ok) break;
            tc_fence_after();
            issue_pv(1, cv, j == 0, j == nB - 1);
          }
          umma_commit_elect(bar(C_EMPTY + cv.s));
          if (j + 1 < nB) issue_s(1, cn);
          if (more) umma_commit_elect(bar(C_EMPTY + cn.s));
          if (j + 2 == n_kt) umma_commit_elect(bar(C_QEMPTY));     // the unit's last S MMAs are in the pipe: Q is free after them
          ck = cn;
        }
        cur = ck;                      // behind V of the last key tile: K_0 of the next unit
      }
    }
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 216;");
    // ------------------------------------------------ softmax of tile x: thread = query row = TMEM lane
    const int x = warp >> 2, row = tid & 127;
    const uint32_t lane_addr = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const uint32_t s_addr = lane_addr + x * 128, o_addr = lane_addr + 256 + x * 128;
    const float sl2 = a.scale_log2;
    int steps = 0;      // S tiles of this tile taken so far (phase of C_SFULL)
    int epis = 0;       // epilogues so far (phase of C_ODONE)
    for (int k = 0;; ++k) {
      // this tile's few fields straight from the published descriptor
      if (!mbar_wait(bar(C_UFULL + (k & 1)), (k >> 1) & 1, abort_flag)) break;
      const Unit* up = unit_slot + (k & 1);
      const int u_index = up->index, u_valid = up->valid;
      const int rows = up->rows[x], nk = up->n_kt[x], lim0 = up->lim0[x], out_tok0 = up->tok0[x], out_hq = up->hq[x];
      __syncwarp();
      if (lane == 0 && u_index >= 0) mbar_arrive(bar(C_UEMPTY + (k & 1)));
      if (u_index < 0) break;
      if (!u_valid || nk == 0) continue;
      const int lim = row < rows ? lim0 + row : -1;
      float m_used = 0.f, m_run = -INFINITY, l = 0.f;
      bool ok = true;
      for (int j = 0; j < nk; ++j) {
        ok = mbar_wait(bar(C_SFULL + x), steps++ & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        uint32_t s[4][32];
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_ld32(s_addr + 32 * c, s[c]);
        tmem_wait_ld();
        const int u0 = j * KT2;
        if (u0 + KT2 - 1 > lim) {     // a tile that reaches past this row's last visible key
#pragma unroll
          for (int c = 0; c < 4; ++c)
#pragma unroll
            for (int e = 0; e < 32; ++e)
              if (u0 + 32 * c + e > lim) s[c][e] = 0xff800000u;   // -inf
        }
        float mx[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int c = 0; c < 4; ++c)
#pragma unroll
          for (int e = 0; e < 32; e += 2)
            mx[(e >> 1) & 3] = max3(mx[(e >> 1) & 3], __uint_as_float(s[c][e]), __uint_as_float(s[c][e + 1]));
        m_run = fmaxf(m_run, fmaxf(fmaxf(mx[0], mx[1]), fmaxf(mx[2], mx[3])));
        bool rescale = false;
        float alpha = 1.f;
        if (j == 0) {
          m_used = m_run == -INFINITY ? 0.f : m_run;
        } else if ((m_run - m_used) * sl2 > RESCALE_LOG2) {
          rescale = true;
          alpha = ex2_approx((m_used - m_run) * sl2);
          m_used = m_run;
        }
        // S_X(j) complete implies PV_X(j-1) complete: O may be touched here
        if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
          for (int cb = 0; cb < D; cb += 32) {
            uint32_t o[32];
            tmem_ld32(o_addr + cb, o);
            tmem_wait_ld();
#pragma unroll
            for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
            tmem_st32(o_addr + cb, o);
          }
          l *= alpha;
        }
        const float2 sc2 = make_float2(sl2, sl2);
        const float nm = -m_used * sl2;
        const float2 nm2 = make_float2(nm, nm);
        float2 sum[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int c = 0; c < 4; ++c) {      // 32 keys -> 16 bf16 pairs -> TMEM columns 16c .. 16c+15 of this tile
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float2 arg = __ffma2_rn(make_float2(__uint_as_float(s[c][2 * e]), __uint_as_float(s[c][2 * e + 1])), sc2, nm2);
            const float2 p = make_float2(ex2_approx(arg.x), ex2_approx(arg.y));
            sum[e & 1] = __fadd2_rn(sum[e & 1], p);
            pk[e] = pack_bf16(p.x, p.y);
          }
          tmem_st16(s_addr + 16 * c, pk);
        }
        l += (sum[0].x + sum[0].y) + (sum[1].x + sum[1].y);
        tmem_wait_st();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(bar(C_PFULL + x));
      }
      // ---- epilogue: O / l -> bf16, each thread stores its own row (8 x 32 bytes, contiguous)
      if (ok) ok = mbar_wait(bar(C_ODONE + x), epis++ & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      uint4* orow = reinterpret_cast<uint4*>(a.out + ((size_t)(out_tok0 + row) * a.n_q + out_hq) * D);
#pragma unroll
      for (int cb = 0; cb < D; cb += 32) {
        uint32_t o[32];
        tmem_ld32(o_addr + cb, o);
        tmem_wait_ld();
        if (row < rows) {
          uint32_t pk[16];
#pragma unroll
          for (int c = 0; c < 16; ++c) pk[c] = pack_bf16(__uint_as_float(o[2 * c]) * inv, __uint_as_float(o[2 * c + 1]) * inv);
          if (wide_out) {                              // 32 bytes per lane: half as many store instructions per row
            st_global_v8(orow + (cb >> 3), pk);
            st_global_v8(orow + (cb >> 3) + 2, pk + 8);
          } else {
#pragma unroll
            for (int c = 0; c < 4; ++c) orow[(cb >> 3) + c] = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
          }
        }
      }
      tc_fence_before();
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    // copies still in flight target this CTA's shared memory: give every armed barrier a bounded
    // chance to complete before the CTA exits
    if (warp == 8 && lane == 0) {
      for (int s = 0; s < NSLOT; ++s)
        for (uint32_t k = 0; k < (1u << 16); ++k)
          if (mbar_try(bar(C_FULL + s), 0) || mbar_try(bar(C_FULL + s), 1)) break;
      for (uint32_t k = 0; k < (1u << 16); ++k)
        if (mbar_try(bar(C_QFULL), 0) || mbar_try(bar(C_QFULL), 1)) break;
    }
    __syncthreads();
  }
  if (warp == 9) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(T2_TMEM_COLS) : "memory");
  }
}

}  // namespace

int launch_prefill_tc2(fl_pool* p, const AttnArgs& a, int n_tokens, int max_items, cudaStream_t st) {
  const CUtensorMap* kv = nullptr;
  alignas(64) CUtensorMap qmap;
  int rc = tmap::kv_pages(p, a.n_kv, &kv);
  if (rc != FL_OK) return rc;
  {   // q as [token][head][128]: box = 64 elements x 128 tokens of one head
    const uint64_t dims[3] = {(uint64_t)D, (uint64_t)a.n_q, (uint64_t)n_tokens};
    const uint64_t strides[2] = {(uint64_t)D * 2, (uint64_t)a.n_q * D * 2};
    const uint32_t box[3] = {64, 1, 128};
    rc = tmap::encode_bf16(&qmap, a.q, 3, dims, strides, box);
    if (rc != FL_OK) return rc;
  }
  static bool configured[16] = {};
  if (!configured[p->device & 15]) {
    FL_CUDA(p, cudaFuncSetAttribute(attn_prefill_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)T2_SMEM));
    configured[p->device & 15] = true;
  }
  const int group = a.n_q / a.n_kv;
  const int heads_per_item = group % 2 == 0 ? a.n_q / 2 : a.n_q;
  // one CTA per SM (shared memory and TMEM allow no more); a CTA beyond the plan's unit count finds no work and tears down
  const long long units = (long long)max_items * heads_per_item;
  const unsigned grid = (unsigned)std::min<long long>(units, p->sm_count);
  if (grid == 0) return FL_OK;
  FL_CUDA(p, launch_pdl(attn_prefill_tc2_kernel, dim3(grid), dim3(T2_THREADS), T2_SMEM, st, a, *kv, qmap, heads_per_item,
                     (reinterpret_cast<uintptr_t>(a.out) & 31) == 0 ? 1 : 0));   // 32-byte stores where the output allows them
  FL_CUDA(p, cudaGetLastError());
  return FL_OK;
}

}  // namespace attn
