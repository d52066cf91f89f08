// Prefill attention on the 5th-generation tensor cores: tcgen05.mma with TMEM accumulators,
// operands staged by TMA straight out of pool blocks (Section 2.1 / 4.2: attention over the reused
// prefix KV plus the new tokens).
//
// One CTA = 128 query rows (new tokens) of one (request, query head); two CTAs share an SM so that
// one CTA's softmax overlaps the other's MMAs.  Warps 0-3: softmax, one thread per query row (= TMEM
// lane).  Warp 4: TMA producer.  Warp 5: MMA issuer and TMEM owner.
//   K/V tile j (64 keys = 4 pool pages) -> shared memory, 128-byte swizzle, 2 stages
//   S_j = Q K_j^T      tcgen05.mma 128x64x16 (x8), accumulator in TMEM, double buffered
//   P_j = exp2(S_j - m) rows -> bf16 -> shared memory (K-major, swizzled); row sum in registers
//   O  += P_j V_j      tcgen05.mma 128x128x16 (x4), V read MN-major as stored ([key][d])
// O stays in TMEM for the whole tile; it is rescaled only when a row maximum grows by more than 2^8
// (the stale maximum keeps exp2 arguments <= 8, exact in fp32/bf16 range), so the rescale is rare.
// Every wait on an mbarrier is bounded; a wait that gives up raises a sticky flag, the CTA drains
// and frees its TMEM.
#include <cuda.h>
#include <math.h>
#include <string.h>
#include "attention.cuh"
#include "mma_utils.cuh"
#include "tc_ptx.cuh"

namespace attn {
namespace {

using namespace tc;

constexpr int TC_THREADS = 192;
constexpr int KT_TC = 64;
constexpr int STAGES = 2;
constexpr uint32_t Q_HALF = QT_TC * 128;          // bytes of one 64-wide half of the Q tile
constexpr uint32_t KV_HALF = KT_TC * 128;         // bytes of one half of a K or V tile
constexpr uint32_t OFF_Q = 0;
constexpr uint32_t OFF_KV = 2 * Q_HALF;                               // stage s: K (2 halves), V (2 halves)
constexpr uint32_t STAGE_BYTES = 4 * KV_HALF;
constexpr uint32_t OFF_P = OFF_KV + STAGES * STAGE_BYTES;             // [128 rows][64 keys] bf16
constexpr uint32_t OFF_BAR = OFF_P + QT_TC * KT_TC * 2;
constexpr uint32_t TC_SMEM = OFF_BAR + 128;
constexpr uint32_t TMEM_COLS = 256;               // S0 | S1 (64 each) | O (128)
constexpr uint32_t TM_S = 0, TM_O = 128;
constexpr float RESCALE_STEP = 8.f;

enum { B_QFULL = 0, B_KVFULL = 1, B_KVEMPTY = 3, B_SFULL = 5, B_SFREE = 7, B_PFULL = 9, B_PVDONE = 10, B_COUNT = 11 };

__global__ void __launch_bounds__(TC_THREADS, 2)
attn_prefill_tc_kernel(const AttnArgs a, const __grid_constant__ CUtensorMap kv_map, const __grid_constant__ CUtensorMap q_map) {
  extern __shared__ __align__(1024) unsigned char smem[];
  const int item = blockIdx.x / a.n_q, hq = blockIdx.x % a.n_q;
  if (item >= a.hdr->n_prefill) return;
  const uint32_t sbase = smem_u32(smem);
  if (sbase & 1023u) {   // the swizzled operand tiles need 1024-byte alignment
    if (threadIdx.x == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    return;
  }
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int2 it = a.prefill_list[item];
  const int i = it.x, q0 = it.y;
  const int n_new = a.new_lens[i], prefix = a.prefix_lens[i], ctx = prefix + n_new;
  const int h = hq / (a.n_q / a.n_kv);
  const int tok0 = a.req_indptr[i] + q0;
  const int q_rows = min(QT_TC, n_new - q0);
  const int kv_end = min(ctx, prefix + q0 + QT_TC);
  const int n_kt = (kv_end + KT_TC - 1) / KT_TC;
  const int tbl0 = a.tbl_indptr[i], tbl_n = a.tbl_indptr[i + 1] - tbl0;
  const int n_pages = (kv_end + BT - 1) / BT;
  if (n_pages > tbl_n || n_pages < 1) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_POS);
    return;
  }
  const uint32_t bar0 = sbase + OFF_BAR;
  auto bar = [&](int k) { return bar0 + 8u * k; };
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_BAR + 8 * B_COUNT);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * B_COUNT + 4);

  if (tid == 0) {
    mbar_init(bar(B_QFULL), 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(bar(B_KVFULL + s), 1);
      mbar_init(bar(B_KVEMPTY + s), 1);
      mbar_init(bar(B_SFULL + s), 1);
      mbar_init(bar(B_SFREE + s), 4);
    }
    mbar_init(bar(B_PFULL), 4);
    mbar_init(bar(B_PVDONE), 1);
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {   // TMEM: 256 columns for this CTA (two CTAs per SM use all 512)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)tmem_slot)), "r"(TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  if (warp == 4) {
    // ------------------------------------------------ TMA producer
    if (lane == 0) {
      mbar_expect_tx(bar(B_QFULL), 2 * Q_HALF);
      tma_load_3d(sbase + OFF_Q, &q_map, bar(B_QFULL), 0, hq, tok0);
      tma_load_3d(sbase + OFF_Q + Q_HALF, &q_map, bar(B_QFULL), 64, hq, tok0);
      for (int j = 0; j < n_kt; ++j) {
        const int s = j % STAGES, use = j / STAGES;
        if (use > 0 && !mbar_wait(bar(B_KVEMPTY + s), (use - 1) & 1, abort_flag)) break;
        mbar_expect_tx(bar(B_KVFULL + s), STAGE_BYTES);
        const uint32_t kbase = sbase + OFF_KV + s * STAGE_BYTES, vbase = kbase + 2 * KV_HALF;
#pragma unroll
        for (int pg = 0; pg < KT_TC / BT; ++pg) {
          // pages behind the last needed key are masked anyway: re-read the last valid page
          const int page = min(j * (KT_TC / BT) + pg, n_pages - 1);
          uint32_t blk = a.tbl[tbl0 + page];
          if (blk >= a.pv.n_blocks) {
            atomicOr(a.pv.flags, (uint32_t)FLAG_BAD_BLOCK);
            blk = 0;
          }
          const uint32_t off = pg * (BT * 128);
          tma_load_4d(kbase + off, &kv_map, bar(B_KVFULL + s), 0, 0, h, (int)blk);
          tma_load_4d(kbase + KV_HALF + off, &kv_map, bar(B_KVFULL + s), 64, 0, h, (int)blk);
          tma_load_4d(vbase + off, &kv_map, bar(B_KVFULL + s), 0, 0, a.n_kv + h, (int)blk);
          tma_load_4d(vbase + KV_HALF + off, &kv_map, bar(B_KVFULL + s), 64, 0, a.n_kv + h, (int)blk);
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t IDESC_S = instr_desc(KT_TC, false);
      constexpr uint32_t IDESC_O = instr_desc(D, true);
      auto issue_s = [&](int j) {   // S_j = Q K_j^T into TMEM buffer j & 1
        const uint32_t kbase = sbase + OFF_KV + (j % STAGES) * STAGE_BYTES;
#pragma unroll
        for (int ks = 0; ks < D / 16; ++ks) {
          const uint32_t koff = (ks >> 2) * Q_HALF + (ks & 3) * 32, boff = (ks >> 2) * KV_HALF + (ks & 3) * 32;
          umma_bf16(tmem + TM_S + (j & 1) * KT_TC, smem_desc(sbase + OFF_Q + koff, 16, 1024),
                    smem_desc(kbase + boff, 16, 1024), IDESC_S, ks > 0);
        }
        umma_commit(bar(B_SFULL + (j & 1)));
      };
      bool ok = mbar_wait(bar(B_QFULL), 0, abort_flag) && mbar_wait(bar(B_KVFULL + 0), 0, abort_flag);
      if (ok) {
        tc_fence_after();
        issue_s(0);
      }
      for (int j = 0; ok && j < n_kt; ++j) {
        if (j + 1 < n_kt) {
          const int s1 = (j + 1) % STAGES, use1 = (j + 1) / STAGES;
          ok = mbar_wait(bar(B_KVFULL + s1), use1 & 1, abort_flag);
          if (ok && j + 1 >= 2) ok = mbar_wait(bar(B_SFREE + ((j + 1) & 1)), (((j + 1) >> 1) - 1) & 1, abort_flag);
          if (!ok) break;
          tc_fence_after();
          issue_s(j + 1);
        }
        ok = mbar_wait(bar(B_PFULL), j & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
        const uint32_t vbase = sbase + OFF_KV + (j % STAGES) * STAGE_BYTES + 2 * KV_HALF;
#pragma unroll
        for (int ks = 0; ks < KT_TC / 16; ++ks)
          umma_bf16(tmem + TM_O, smem_desc(sbase + OFF_P + ks * 32, 16, 1024),
                    smem_desc(vbase + ks * (16 * 128), KV_HALF, 1024), IDESC_O, (j > 0 || ks > 0));
        umma_commit(bar(B_PVDONE));
        umma_commit(bar(B_KVEMPTY + (j % STAGES)));
      }
    }
  } else {
    // ------------------------------------------------ softmax: thread = query row = TMEM lane
    const int row = tid;
    const int lim = row < q_rows ? prefix + q0 + row : -1;
    const uint32_t lane_addr = tmem + ((uint32_t)(warp * 32) << 16);
    float m_used = 0.f, m_run = -INFINITY, l = 0.f;
    bool ok = true;
    for (int j = 0; j < n_kt; ++j) {
      ok = mbar_wait(bar(B_SFULL + (j & 1)), (j >> 1) & 1, abort_flag);
      if (!ok) break;
      tc_fence_after();
      uint32_t sr[64];
      {
        uint32_t lo[32], hi[32];
        tmem_ld32(lane_addr + TM_S + (j & 1) * KT_TC, lo);
        tmem_ld32(lane_addr + TM_S + (j & 1) * KT_TC + 32, hi);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 32; ++c) { sr[c] = lo[c]; sr[32 + c] = hi[c]; }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_SFREE + (j & 1)));     // S buffer is in registers now
      const int u0 = j * KT_TC;
      float mx = -INFINITY;
      float sc[64];
      if (u0 + KT_TC - 1 > lim) {
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          sc[c] = (u0 + c <= lim) ? __uint_as_float(sr[c]) * a.scale_log2 : -INFINITY;
          mx = fmaxf(mx, sc[c]);
        }
      } else {
#pragma unroll
        for (int c = 0; c < 64; ++c) {
          sc[c] = __uint_as_float(sr[c]) * a.scale_log2;
          mx = fmaxf(mx, sc[c]);
        }
      }
      m_run = fmaxf(m_run, mx);
      bool rescale = false;
      float alpha = 1.f;
      if (j == 0) {
        m_used = m_run == -INFINITY ? 0.f : m_run;
      } else if (m_run > m_used + RESCALE_STEP) {
        rescale = true;
        alpha = exp2f(m_used - m_run);
        m_used = m_run;
      }
      float sum = 0.f;
      uint32_t pk[32];
#pragma unroll
      for (int c = 0; c < 64; c += 2) {
        const float p0 = exp2f(sc[c] - m_used), p1 = exp2f(sc[c + 1] - m_used);
        sum += p0 + p1;
        pk[c >> 1] = pack_bf16(p0, p1);
      }
      l = l * alpha + sum;
      if (j > 0) {   // P buffer and O are free once PV_{j-1} has completed
        ok = mbar_wait(bar(B_PVDONE), (j - 1) & 1, abort_flag);
        if (!ok) break;
        tc_fence_after();
      }
      if (__any_sync(0xffffffffu, rescale)) {
#pragma unroll
        for (int cb = 0; cb < D; cb += 32) {
          uint32_t o[32];
          tmem_ld32(lane_addr + TM_O + cb, o);
          tmem_wait_ld();
#pragma unroll
          for (int c = 0; c < 32; ++c) o[c] = __float_as_uint(__uint_as_float(o[c]) * alpha);
          tmem_st32(lane_addr + TM_O + cb, o);
        }
        tmem_wait_st();
      }
      unsigned char* prow = smem + OFF_P + row * 128;
#pragma unroll
      for (int c = 0; c < 8; ++c)
        *reinterpret_cast<uint4*>(prow + ((c ^ (row & 7)) << 4)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
      fence_async_smem();
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(bar(B_PFULL));
    }
    // ---- epilogue: O / l -> bf16 -> staged in the Q buffer -> coalesced 16-byte stores
    if (ok) ok = mbar_wait(bar(B_PVDONE), (n_kt - 1) & 1, abort_flag);
    if (ok) {
      tc_fence_after();
      const float inv = l > 0.f ? 1.f / l : 0.f;
      unsigned char* orow = smem + OFF_Q + row * 256;
#pragma unroll
      for (int cb = 0; cb < D; cb += 32) {
        uint32_t o[32];
        tmem_ld32(lane_addr + TM_O + cb, o);
        tmem_wait_ld();
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          uint4 v;
          v.x = pack_bf16(__uint_as_float(o[8 * c + 0]) * inv, __uint_as_float(o[8 * c + 1]) * inv);
          v.y = pack_bf16(__uint_as_float(o[8 * c + 2]) * inv, __uint_as_float(o[8 * c + 3]) * inv);
          v.z = pack_bf16(__uint_as_float(o[8 * c + 4]) * inv, __uint_as_float(o[8 * c + 5]) * inv);
          v.w = pack_bf16(__uint_as_float(o[8 * c + 6]) * inv, __uint_as_float(o[8 * c + 7]) * inv);
          const int chunk = (cb >> 3) + c;
          *reinterpret_cast<uint4*>(orow + ((chunk ^ (row & 7)) << 4)) = v;
        }
      }
      tc_fence_before();
    }
    // the four softmax warps exchange rows through shared memory: named barrier over 128 threads
    asm volatile("bar.sync 1, 128;" ::: "memory");
    if (ok && !*abort_flag) {
      const int cch = tid & 15;
#pragma unroll
      for (int r = 0; r < QT_TC / 8; ++r) {
        const int orow_i = (tid >> 4) + 8 * r;
        if (orow_i < q_rows)
          *reinterpret_cast<uint4*>(a.out + ((size_t)(tok0 + orow_i) * a.n_q + hq) * D + cch * 8) =
              *reinterpret_cast<const uint4*>(smem + OFF_Q + orow_i * 256 + ((cch ^ (orow_i & 7)) << 4));
    }
    }
  }
  // ------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (*abort_flag) {
    if (tid == 0) atomicOr(a.pv.flags, (uint32_t)FLAG_WAIT_GAVE_UP);
    // copies still in flight target this CTA's shared memory: give every armed barrier a bounded
    // chance to complete before the CTA exits
    if (warp == 4 && lane == 0) {
      for (int s = 0; s < STAGES; ++s)
        for (uint32_t k = 0; k < (1u << 16); ++k)
          if (mbar_try(bar(B_KVFULL + s), 0) || mbar_try(bar(B_KVFULL + s), 1)) break;
    }
    __syncthreads();
  }
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
  }
}

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

struct TmapCache {
  int n_kv;
  CUtensorMap kv;
};

}  // namespace

int prefill_tensor_maps(fl_pool* p, const AttnArgs& a, int n_tokens, const CUtensorMap** kv_out, CUtensorMap* qmap) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return FL_ECUDA;
  TmapCache* tc = reinterpret_cast<TmapCache*>(p->tmap_cache);
  if (!tc || tc->n_kv != a.n_kv) {
    if (!tc) {
      if (posix_memalign(reinterpret_cast<void**>(&tc), 64, sizeof(TmapCache)) != 0) return FL_ENOMEM;
      p->tmap_cache = tc;
    }
    // the slab as [block][K|V x kv head][token][128]: box = 64 elements x 16 tokens of one (block, slot)
    const cuuint64_t dims[4] = {(cuuint64_t)D, (cuuint64_t)BT, (cuuint64_t)(2 * a.n_kv), (cuuint64_t)p->n_blocks};
    const cuuint64_t strides[3] = {(cuuint64_t)D * 2, (cuuint64_t)PAGE_BYTES, (cuuint64_t)p->block_bytes};
    const cuuint32_t box[4] = {64, (cuuint32_t)BT, 1, 1};
    const cuuint32_t es[4] = {1, 1, 1, 1};
    if (enc(&tc->kv, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, p->slab, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS) {
      tc->n_kv = -1;
      return FL_ECUDA;
    }
    tc->n_kv = a.n_kv;
  }
  // q as [token][head][128]: box = 64 elements x 128 tokens of one head
  const cuuint64_t dims[3] = {(cuuint64_t)D, (cuuint64_t)a.n_q, (cuuint64_t)n_tokens};
  const cuuint64_t strides[2] = {(cuuint64_t)D * 2, (cuuint64_t)a.n_q * D * 2};
  const cuuint32_t box[3] = {64, 1, (cuuint32_t)QT_TC};
  const cuuint32_t es[3] = {1, 1, 1};
  if (enc(qmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(a.q), dims, strides, box, es,
          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
    return FL_ECUDA;
  *kv_out = &tc->kv;
  return FL_OK;
}

int launch_prefill_tc(fl_pool* p, const AttnArgs& a, int n_tokens, cudaStream_t st) {
  const CUtensorMap* kv = nullptr;
  alignas(64) CUtensorMap qmap;
  int rc = prefill_tensor_maps(p, a, n_tokens, &kv, &qmap);
  if (rc != FL_OK) return rc;
  static bool configured[16] = {};
  if (!configured[p->device & 15]) {
    FL_CUDA(p, cudaFuncSetAttribute(attn_prefill_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)TC_SMEM));
    configured[p->device & 15] = true;
  }
  // tiles of 128 rows: at most n_tokens / 128 + n_req of them
  const unsigned tiles = (unsigned)(n_tokens / QT_TC + a.n_req);
  attn_prefill_tc_kernel<<<tiles * a.n_q, TC_THREADS, TC_SMEM, st>>>(a, *kv, qmap);
  FL_CUDA(p, cudaGetLastError());
  return FL_OK;
}

}  // namespace attn
