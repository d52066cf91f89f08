// Block swap between the pinned host slab and the device slab, on a side stream (copy engines),
// and the KV store kernel that writes new tokens' K,V into pool blocks.
#include <chrono>
#include <thread>
#include "pool.cuh"

namespace {

int swap_blocks(fl_pool* p, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side, bool in) {
  if (!p || (n && (!dev_ids || !host_ids))) return FL_EINVAL;
  for (uint32_t k = 0; k < n; ++k) {
    if (dev_ids[k] >= p->n_blocks || !p->dev.used[dev_ids[k]]) return FL_EBADID;
    if (host_ids[k] >= p->n_host_blocks || !p->host.used[host_ids[k]]) return FL_EBADID;
  }
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != p->device) cudaSetDevice(p->device);
  int rc = FL_OK;
  // one DMA per run of pairs that are consecutive in both memories
  for (uint32_t k = 0; k < n;) {
    uint32_t run = 1;
    while (k + run < n && dev_ids[k + run] == dev_ids[k] + run && host_ids[k + run] == host_ids[k] + run) ++run;
    unsigned char* d = p->slab + (size_t)dev_ids[k] * p->block_bytes;
    unsigned char* h = p->host_slab + (size_t)host_ids[k] * p->block_bytes;
    cudaError_t e = in ? cudaMemcpyAsync(d, h, run * p->block_bytes, cudaMemcpyHostToDevice, (cudaStream_t)side)
                       : cudaMemcpyAsync(h, d, run * p->block_bytes, cudaMemcpyDeviceToHost, (cudaStream_t)side);
    if (e != cudaSuccess) {
      p->last_cuda = (int)e;
      rc = FL_ECUDA;
      break;
    }
    (in ? p->bytes_in : p->bytes_out) += (uint64_t)run * p->block_bytes;
    k += run;
  }
  if (prev != p->device && prev >= 0) cudaSetDevice(prev);
  return rc;
}

// One CTA per new token: copies its K and V rows (n_kv * 128 bf16 each) into the token's slot.
__global__ void kv_append_kernel(PoolView pv, const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                                 const int32_t* __restrict__ req_indptr, const int32_t* __restrict__ tbl_indptr,
                                 const uint32_t* __restrict__ tbl, const int32_t* __restrict__ prefix_lens,
                                 int n_req, int n_tokens, int n_kv, int bt) {
  const int t = blockIdx.x;
  if (t >= n_tokens) return;
  // request of token t: last i with req_indptr[i] <= t
  int lo = 0, hi = n_req;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (req_indptr[mid] <= t) lo = mid; else hi = mid;
  }
  const int i = lo;
  if (t < req_indptr[i] || t >= req_indptr[i + 1]) return;   // token not owned by any request
  const int pos = prefix_lens[i] + (t - req_indptr[i]);
  const int entry = pos / bt, slot = pos % bt;
  if (pos < 0 || entry >= tbl_indptr[i + 1] - tbl_indptr[i]) {
    if (threadIdx.x == 0) atomicOr(pv.flags, (uint32_t)FLAG_BAD_POS);
    return;
  }
  const uint32_t blk = tbl[tbl_indptr[i] + entry];
  if (blk >= pv.n_blocks) {
    if (threadIdx.x == 0) atomicOr(pv.flags, (uint32_t)FLAG_BAD_BLOCK);
    return;
  }
  constexpr int CH = FL_HEAD_DIM * 2 / 16;                     // 16-byte chunks per (head, token) row
  uint4* dst = reinterpret_cast<uint4*>(pv.slab + (size_t)blk * pv.block_bytes);
  const int per_side = n_kv * CH;
  for (int c = threadIdx.x; c < 2 * per_side; c += blockDim.x) {
    const int w = c / per_side, r = c - w * per_side;
    const int h = r / CH, e = r - h * CH;
    const uint4 val = (w ? v_new : k_new)[(size_t)t * per_side + r];
    dst[((size_t)(w * n_kv + h) * bt + slot) * CH + e] = val;
  }
  // The request's last token also clears the V slots behind it in its block, so that attention can
  // multiply those slots by a zero weight without meeting stale non-finite bit patterns.
  if (t == req_indptr[i + 1] - 1 && slot + 1 < bt) {
    const int rest = (bt - 1 - slot) * CH;
    for (int c = threadIdx.x; c < n_kv * rest; c += blockDim.x) {
      const int h = c / rest, r = c - h * rest;
      dst[((size_t)(n_kv + h) * bt + slot + 1) * CH + r] = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

}  // namespace

extern "C" {

int fl_swap_out(fl_pool* p, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side) {
  return swap_blocks(p, dev_ids, host_ids, n, side, false);
}
int fl_swap_in(fl_pool* p, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side) {
  return swap_blocks(p, dev_ids, host_ids, n, side, true);
}
int fl_swap_record(fl_pool* p, fl_event ev, fl_stream side) {
  if (!p || !ev) return FL_EINVAL;
  FL_CUDA(p, cudaEventRecord((cudaEvent_t)ev, (cudaStream_t)side));
  return FL_OK;
}
int fl_swap_wait(fl_pool* p, fl_event ev, int timeout_ms) {
  if (!p || !ev) return FL_EINVAL;
  const auto deadline = std::chrono::steady_clock::now() + std::chrono::milliseconds(timeout_ms);
  for (;;) {
    cudaError_t e = cudaEventQuery((cudaEvent_t)ev);
    if (e == cudaSuccess) return FL_OK;
    if (e != cudaErrorNotReady) {
      p->last_cuda = (int)e;
      return FL_ECUDA;
    }
    if (std::chrono::steady_clock::now() >= deadline) return FL_ETIMEOUT;
    std::this_thread::sleep_for(std::chrono::microseconds(50));
  }
}

int fl_kv_append(fl_pool* p, const fl_bf16* k_new, const fl_bf16* v_new, const int32_t* req_indptr,
                 const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                 int n_req, int n_tokens, int n_kv_heads, fl_stream stream) {
  if (!p || n_req < 0 || n_tokens < 0 || n_kv_heads < 1) return FL_EINVAL;
  const size_t per_tok = (size_t)2 * n_kv_heads * FL_HEAD_DIM * 2;
  if (p->block_bytes % per_tok != 0) return FL_EINVAL;
  if (n_req == 0 || n_tokens == 0) return FL_OK;
  if (!k_new || !v_new || !req_indptr || !kv_tbl_indptr || !kv_tbl || !prefix_lens) return FL_EINVAL;
  const int bt = (int)(p->block_bytes / per_tok);
  kv_append_kernel<<<n_tokens, 256, 0, (cudaStream_t)stream>>>(
      p->view(), reinterpret_cast<const uint4*>(k_new), reinterpret_cast<const uint4*>(v_new), req_indptr,
      kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_tokens, n_kv_heads, bt);
  FL_CUDA(p, cudaGetLastError());
  return FL_OK;
}

}  // extern "C"
