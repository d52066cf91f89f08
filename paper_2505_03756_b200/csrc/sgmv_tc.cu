// The shrink v = x A_i of the segmented LoRA projection (Eq. 1, Eq. 2; Section 2.1) for long segments, on the
// 5th-generation tensor cores.
//
// At rank 32-64 and three projections per call the mma.sync shrink is bound by the legacy tensor path and by the
// ldmatrix traffic, not by reading x.  Here a CTA takes a tile of 128 tokens of one segment and a slice of d_in:
//   warp 0      TMA producer: x tile [128 tokens x 64] per stage (K-major, 128-byte swizzle)
//   warp 1      MMA issuer: D[128 x (projections * RMAX)] += x tile * adapter rows^T, tcgen05.mma 128 x N x 16
//   warps 2-5   adapter rows (row p of A is d_in contiguous values in a pool block, found through the adapter's block
//               table) by 16-byte cp.async into the stage, in the operand's swizzled layout, a few stages in flight
//   warps 6-9   epilogue: TMEM -> fp32 partial sums [projection][slice][token][RMAX], rows of the segment only
// The accumulator is double buffered in TMEM, so a unit's epilogue overlaps the next unit's stages.  Units go to
// the CTAs round robin.  Every mbarrier wait is bounded; a wait that gives up raises a sticky flag and the CTA
// tears down (its copies drained, its TMEM freed).  No cluster launch, no multicast.
#include <cuda.h>
#include <algorithm>
#include "mma_utils.cuh"
#include "pool.cuh"
#include "sgmv.cuh"
#include "tc_ptx.cuh"
#include "tmap.cuh"

namespace {

using namespace tc;

constexpr int ST_THREADS = 320;
constexpr int TM = 128, BK = 64;
constexpr uint32_t X_BYTES = TM * BK * 2;
constexpr int PF = 4;                 // adapter-row stages a copy thread keeps in flight

template <int N>
struct Cfg {
  static constexpr uint32_t B_BYTES = N * 128;
  static constexpr uint32_t STAGE = X_BYTES + ((B_BYTES + 1023) / 1024) * 1024;
  static constexpr int NS = (220 * 1024) / STAGE < 8 ? (220 * 1024) / STAGE : 8;      // ring slots: what fits, at most 8
  static constexpr uint32_t OFF_BAR = NS * STAGE;
  static constexpr uint32_t SMEM = OFF_BAR + 256 + 1024;
  static constexpr uint32_t TMEM_COLS = 2 * N <= 32 ? 32 : 2 * N <= 64 ? 64 : 2 * N <= 128 ? 128 : 2 * N <= 256 ? 256 : 512;
  static_assert(2 * N <= 512, "two accumulators must fit in TMEM");
  static_assert(SMEM <= 227 * 1024, "shared memory");
};

struct Unit {
  int seg, tok0, tok1, lid, kb, n_it, split;
  bool ok;
};

// Unit u -> token tile and slice of d_in; the whole warp takes part (the tile search is a warp scan).
__device__ __forceinline__ Unit decode_unit(const sgmv::TcShrinkArgs& a, int u) {
  Unit t;
  const int tile = u / a.ksplit;
  t.split = u - tile * a.ksplit;
  t.ok = sgmv::find_tile<TM>(a.seg_indptr, a.lora_ids, a.n_seg, tile, t.seg, t.tok0, t.tok1);
  t.lid = -1;
  t.kb = t.n_it = 0;
  if (!t.ok) return t;
  t.lid = a.lora_ids[t.seg];
  bool good = t.lid >= 0 && (uint32_t)t.lid < a.pv.dir_cap && a.pv.dir[t.lid].rank > 0;
  for (int j = 0; good && j < a.n_mats; ++j) good = a.mat_index[j] < a.pv.dir[t.lid].n_mats;
  if (!good) {
    if ((threadIdx.x & 31) == 0 && t.lid >= 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
    t.ok = false;
    return t;
  }
  const int kchunk = ((a.d_in + a.ksplit * BK - 1) / (a.ksplit * BK)) * BK;
  t.kb = t.split * kchunk;
  const int ke = min(a.d_in, t.kb + kchunk);
  t.n_it = ke > t.kb ? (ke - t.kb + BK - 1) / BK : 0;
  return t;
}

template <int RMAX, int NM>
__global__ void __launch_bounds__(ST_THREADS, 1) sgmv_shrink_tc_kernel(const sgmv::TcShrinkArgs a, const __grid_constant__ CUtensorMap xmap,
                                                                       int n_units) {
  constexpr int N = RMAX * NM;
  using C = Cfg<N>;
  constexpr int NS = C::NS;
  static_assert(NS > PF, "the ring must hold more stages than a copy thread keeps in flight");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  enum { B_FULL = 0, B_EMPTY = NS, B_ACC_FULL = 2 * NS, B_ACC_EMPTY = 2 * NS + 2, B_COUNT = 2 * NS + 4 };
  const uint32_t bar0 = sbase + C::OFF_BAR;
  auto bar = [&](int k) { return bar0 + 8u * k; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + C::OFF_BAR + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + C::OFF_BAR + 8 * B_COUNT + 4);
  static_assert(8 * B_COUNT + 8 <= 256, "bookkeeping area too small");

  if (tid == 0) {
    for (int s = 0; s < NS; ++s) {
      mbar_init(bar(B_FULL + s), 1 + 128);     // the TMA producer's arrive (with the byte count) + the 128 copy threads
      mbar_init(bar(B_EMPTY + s), 1);
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
  pdl_wait();                 // x may come from the kernel right before this one
  pdl_launch_dependents();    // the kernel that consumes the partial sums may set itself up while this grid runs

  if (warp == 0) {
    // ------------------------------------------------ TMA producer (lane 0 issues; the warp decodes units together)
    long long f = 0;
    bool ok = true;
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
      const Unit t = decode_unit(a, u);
      if (!t.ok) continue;
      for (int it = 0; it < t.n_it; ++it, ++f) {
        if (lane == 0) {
          const int s = (int)(f % NS);
          const long long use = f / NS;
          if (use > 0) ok = mbar_wait(bar(B_EMPTY + s), (uint32_t)((use - 1) & 1), abort_flag);
          if (ok) {
            mbar_expect_tx(bar(B_FULL + s), X_BYTES);
            tma_load_2d(sbase + s * C::STAGE, &xmap, bar(B_FULL + s), t.kb + it * BK, t.tok0);
          }
        }
        ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
        if (!ok) break;
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------ MMA issuer
    constexpr uint32_t IDESC = instr_desc(N, false);     // both operands K-major
    long long f = 0;
    bool ok = true;
    int k = 0;       // units with work so far
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
      const Unit t = decode_unit(a, u);
      if (!t.ok || t.n_it == 0) continue;
      const int buf = k & 1;
      if (lane == 0) {
        if (k >= 2) ok = mbar_wait(bar(B_ACC_EMPTY + buf), (uint32_t)(((k >> 1) - 1) & 1), abort_flag);
        tc_fence_after();
        const uint32_t d_tmem = tmem + buf * N;
        for (int it = 0; ok && it < t.n_it; ++it) {
          const long long ff = f + it;
          const int s = (int)(ff % NS);
          ok = mbar_wait(bar(B_FULL + s), (uint32_t)((ff / NS) & 1), abort_flag);
          if (!ok) break;
          tc_fence_after();
          const uint32_t ab = sbase + s * C::STAGE, bb = ab + X_BYTES;
#pragma unroll
          for (int ks = 0; ks < BK / 16; ++ks)
            umma_bf16(d_tmem, smem_desc(ab + ks * 32, 16, 1024), smem_desc(bb + ks * 32, 16, 1024), IDESC, (it > 0 || ks > 0) ? 1u : 0u);
          umma_commit(bar(B_EMPTY + s));
        }
        if (ok) umma_commit(bar(B_ACC_FULL + buf));
      }
      ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
      f += t.n_it;
      ++k;
    }
  } else if (warp < 6) {
    // ------------------------------------------------ adapter rows: row n = projection * RMAX + rank row, 8 chunks of 16 bytes
    const int ct = tid - 64;                      // 0..127
    constexpr int RPT = N / 16;                   // rows per thread: n = ct / 8 + 16 i
    const int cc = ct & 7;
    long long f = 0, arrived = 0;                 // stages issued / stages this thread has signalled
    bool ok = true;
    auto signal = [&](long long upto) {           // the copies of stages < upto have landed: make them visible, arrive
      fence_async_smem();
      for (; arrived < upto; ++arrived) mbar_arrive(bar(B_FULL + (int)(arrived % NS)));
    };
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
      const Unit t = decode_unit(a, u);
      if (!t.ok) continue;
      const LoraEntry* e = a.pv.dir + t.lid;
      const int rank = min(e->rank, RMAX);
      if (e->rank > RMAX && ct == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_LORA);
      const uint32_t table_off = e->table_off;
      const unsigned char* rowp[RPT];
      bool rok[RPT];
#pragma unroll
      for (int i = 0; i < RPT; ++i) {
        const int n = (ct >> 3) + 16 * i;
        const int m = n / RMAX, r = n % RMAX;
        rok[i] = false;
        rowp[i] = a.pv.slab;
        if (m < a.n_mats && r < rank) {
          const LoraMat& lm = e->mats[a.mat_index[m]];
          rowp[i] = sgmv::lora_row(a.pv, table_off, lm.a_tab, lm.a_row0, lm.a_rpb, a.d_in, r, rok[i]);
        }
      }
      const int ke = min(a.d_in, t.kb + ((a.d_in + a.ksplit * BK - 1) / (a.ksplit * BK)) * BK);
      for (int it = 0; it < t.n_it; ++it, ++f) {
        const int s = (int)(f % NS);
        const long long use = f / NS;
        if (use > 0) ok = mbar_wait(bar(B_EMPTY + s), (uint32_t)((use - 1) & 1), abort_flag);
        if (!ok) break;
        const int kk = t.kb + it * BK + cc * 8;
        const uint32_t bs = sbase + s * C::STAGE + X_BYTES;
#pragma unroll
        for (int i = 0; i < RPT; ++i) {
          const int n = (ct >> 3) + 16 * i;
          cp_async16(bs + n * 128 + ((cc ^ (n & 7)) << 4), rowp[i] + (size_t)kk * 2, rok[i] && kk < ke);
        }
        cp_async_commit();
        if (f + 1 >= PF) {                         // once at most PF - 1 groups are pending, the stages before them have landed
          cp_async_wait<PF - 1>();
          signal(f + 2 - PF);
        }
      }
      // the unit's last stages: the issuer should not wait for them until this thread has found its next unit
      cp_async_wait<0>();
      if (ok) signal(f);
    }
    cp_async_wait<0>();
  } else {
    // ------------------------------------------------ epilogue: thread = token row = TMEM lane
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_addr = tmem + ((uint32_t)(quarter * 32) << 16);
    bool ok = true;
    int k = 0;
    for (int u = blockIdx.x; ok && u < n_units; u += gridDim.x) {
      const Unit t = decode_unit(a, u);
      if (!t.ok) continue;
      const int tok = t.tok0 + row;
      const bool mine = tok < t.tok1;
      if (t.n_it == 0) {          // an empty slice of d_in still owes its zeros to the sum over slices
        if (mine)
          for (int j = 0; j < a.n_mats; ++j) {
            float4* dst = reinterpret_cast<float4*>(a.v + ((size_t)(j * a.ksplit + t.split) * a.n_tokens + tok) * RMAX);
            for (int c = 0; c < RMAX / 4; ++c) dst[c] = make_float4(0.f, 0.f, 0.f, 0.f);
          }
        continue;
      }
      const int buf = k & 1;
      ok = mbar_wait(bar(B_ACC_FULL + buf), (uint32_t)((k >> 1) & 1), abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      tc_fence_after();
#pragma unroll
      for (int c0 = 0; c0 < N; c0 += 16) {
        uint32_t o[16];
        tmem_ld16(lane_addr + buf * N + c0, o);
        tmem_wait_ld();
        const int j = c0 / RMAX, col = c0 % RMAX;
        if (mine && j < a.n_mats) {
          float4* dst = reinterpret_cast<float4*>(a.v + ((size_t)(j * a.ksplit + t.split) * a.n_tokens + tok) * RMAX + col);
#pragma unroll
          for (int c = 0; c < 4; ++c)
            dst[c] = make_float4(__uint_as_float(o[4 * c]), __uint_as_float(o[4 * c + 1]), __uint_as_float(o[4 * c + 2]),
                                 __uint_as_float(o[4 * c + 3]));
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_ACC_EMPTY + buf));
      ++k;
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    // x copies still in flight target this CTA's shared memory: give every armed barrier a bounded chance to complete
    // (the adapter-row copies were waited for by their own threads above)
    if (warp == 0 && lane == 0) {
      for (int s = 0; s < NS; ++s)
        for (uint32_t i = 0; i < (1u << 16); ++i)
          if (mbar_try(bar(B_FULL + s), 0) || mbar_try(bar(B_FULL + s), 1)) break;
    }
    __syncthreads();
  }
  if (warp == 1) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::TMEM_COLS) : "memory");
  }
}

template <int RMAX, int NM>
int launch(fl_pool* p, const sgmv::TcShrinkArgs& a, const CUtensorMap& xmap, int n_units, cudaStream_t st) {
  using C = Cfg<RMAX * NM>;
  static bool configured[16] = {};
  if (!configured[p->device & 15]) {
    FL_CUDA(p, cudaFuncSetAttribute(sgmv_shrink_tc_kernel<RMAX, NM>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM));
    configured[p->device & 15] = true;
  }
  const unsigned grid = (unsigned)std::min(n_units, p->sm_count);
  FL_CUDA(p, launch_pdl(sgmv_shrink_tc_kernel<RMAX, NM>, dim3(grid), dim3(ST_THREADS), C::SMEM, st, a, xmap, n_units));
  FL_CUDA(p, cudaGetLastError());
  return FL_OK;
}

}  // namespace

namespace sgmv {

int shrink_tc(fl_pool* p, const TcShrinkArgs& a, const void* x, int rmax, cudaStream_t st) {
  if (a.n_mats < 1 || a.n_mats > 3 || a.d_in % 8 != 0 || a.ksplit < 1) return FL_EINVAL;
  if ((long long)(a.ksplit - 1) * BK >= a.d_in) return FL_EINVAL;      // every slice of d_in must hold something
  alignas(64) CUtensorMap xmap;
  const uint64_t dims[2] = {(uint64_t)a.d_in, (uint64_t)a.n_tokens};
  const uint64_t strides[1] = {(uint64_t)a.d_in * 2};
  const uint32_t box[2] = {BK, TM};
  int rc = tmap::encode_bf16(&xmap, x, 2, dims, strides, box);
  if (rc != FL_OK) return rc;
  const int n_units = (a.n_seg + a.n_tokens / TM) * a.ksplit;     // upper bound of the tile count, times the slices
  const int nm = a.n_mats;
  if (rmax == 16) return nm == 1 ? launch<16, 1>(p, a, xmap, n_units, st) : nm == 2 ? launch<16, 2>(p, a, xmap, n_units, st) : launch<16, 3>(p, a, xmap, n_units, st);
  if (rmax == 32) return nm == 1 ? launch<32, 1>(p, a, xmap, n_units, st) : nm == 2 ? launch<32, 2>(p, a, xmap, n_units, st) : launch<32, 3>(p, a, xmap, n_units, st);
  if (rmax == 64) return nm == 1 ? launch<64, 1>(p, a, xmap, n_units, st) : nm == 2 ? launch<64, 2>(p, a, xmap, n_units, st) : launch<64, 3>(p, a, xmap, n_units, st);
  return FL_EINVAL;
}

}  // namespace sgmv
