// Block swap between the pinned host slab and the device slab, on a side stream (copy engines),
// and the KV store kernel that writes new tokens' K,V into pool blocks.
#include <algorithm>
#include <chrono>
#include <thread>
#include <vector>
#include "pool.cuh"

namespace {

constexpr uint32_t STAGE_CHUNK = 512;            // block ids per gather/scatter launch (passed by value)
struct IdChunk { uint32_t ids[STAGE_CHUNK]; };

// Copies whole pool blocks between the slab and a contiguous staging area: block ch.ids[k] <-> stage
// block k.  blockIdx.x = k * parts + part; every CTA moves one slice of one block with 16-byte accesses.
__global__ void __launch_bounds__(256) block_stage_kernel(unsigned char* __restrict__ slab, unsigned char* __restrict__ stage,
                                                          const __grid_constant__ IdChunk ch, uint32_t u4_per_block,
                                                          uint32_t parts, uint32_t n_pool_blocks, int to_stage,
                                                          uint32_t* __restrict__ flags) {
  const uint32_t k = blockIdx.x / parts, part = blockIdx.x % parts;
  const uint32_t blk = ch.ids[k];
  if (blk >= n_pool_blocks) {
    if (threadIdx.x == 0) atomicOr(flags, (uint32_t)FLAG_BAD_BLOCK);
    return;
  }
  const uint32_t per = (u4_per_block + parts - 1) / parts;
  const uint32_t lo = part * per, hi = min(u4_per_block, lo + per);
  uint4* pool_blk = reinterpret_cast<uint4*>(slab) + (size_t)blk * u4_per_block;
  uint4* stage_blk = reinterpret_cast<uint4*>(stage) + (size_t)k * u4_per_block;
  const uint4* src = to_stage ? pool_blk : stage_blk;
  uint4* dst = to_stage ? stage_blk : pool_blk;
  uint32_t i = lo + threadIdx.x;
  for (; i + 3 * 256 < hi; i += 4 * 256) {       // four independent 16-byte loads in flight per thread
    const uint4 a = src[i], b = src[i + 256], c = src[i + 512], d = src[i + 768];
    dst[i] = a; dst[i + 256] = b; dst[i + 512] = c; dst[i + 768] = d;
  }
  for (; i < hi; i += 256) dst[i] = src[i];
}

// Swap of the listed (device block, host block) pairs on stream `side`.  Runs of consecutive host blocks
// whose device blocks are scattered over the pool go through a contiguous staging area in device memory:
// one gather kernel + one DMA per run (swap-out), or one DMA + one scatter kernel (swap-in), so the copy
// engine moves a few large pieces instead of one small piece per block.  Everything else is one DMA per
// run of pairs consecutive in both memories.
int swap_blocks(fl_pool* p, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side, bool in) {
  if (!p || (n && (!dev_ids || !host_ids))) return FL_EINVAL;
  // validate everything before the first copy: range, allocated, no block listed twice
  int bad = FL_OK;
  uint32_t marked = 0;
  for (; marked < n; ++marked) {
    const uint32_t d = dev_ids[marked], h = host_ids[marked];
    if (d >= p->n_blocks || h >= p->n_host_blocks || !p->dev.used[d] || !p->host.used[h]) { bad = FL_EBADID; break; }
    if (p->dev.used[d] == 2 || p->host.used[h] == 2) { bad = FL_EINVAL; break; }
    p->dev.used[d] = 2;
    p->host.used[h] = 2;
  }
  for (uint32_t k = 0; k < marked; ++k) p->dev.used[dev_ids[k]] = p->host.used[host_ids[k]] = 1;
  if (bad != FL_OK) return bad;
  if (n == 0) return FL_OK;
  int prev = -1;
  cudaGetDevice(&prev);
  if (prev != p->device) cudaSetDevice(p->device);
  const cudaStream_t st = (cudaStream_t)side;
  const size_t bb = p->block_bytes;
  std::vector<uint32_t> order(n);
  for (uint32_t k = 0; k < n; ++k) order[k] = k;
  std::sort(order.begin(), order.end(), [&](uint32_t a, uint32_t b) { return host_ids[a] < host_ids[b]; });
  const int dir = in ? 1 : 0;
  const uint32_t u4 = (uint32_t)(bb / 16);
  const uint32_t parts = std::max(1u, std::min(32u, u4 / 1024));
  bool staged_any = false;
  cudaError_t e = cudaSuccess;
  for (uint32_t k = 0; k < n && e == cudaSuccess;) {
    uint32_t run = 1, both = 1;
    while (k + run < n && host_ids[order[k + run]] == host_ids[order[k]] + run) {
      if (both == run && dev_ids[order[k + run]] == dev_ids[order[k]] + run) ++both;
      ++run;
    }
    unsigned char* h = p->host_slab + (size_t)host_ids[order[k]] * bb;
    if (both > 1 || run == 1 || !p->stage[dir]) {
      // pairs consecutive in both memories (or a lone block): one DMA
      const uint32_t len = both;
      unsigned char* d = p->slab + (size_t)dev_ids[order[k]] * bb;
      e = in ? cudaMemcpyAsync(d, h, len * bb, cudaMemcpyHostToDevice, st) : cudaMemcpyAsync(h, d, len * bb, cudaMemcpyDeviceToHost, st);
      k += len;
      continue;
    }
    // scattered device blocks, consecutive host blocks: through the staging area, STAGE_CHUNK blocks at most per piece
    const uint32_t len = std::min(run, std::min(p->stage_blocks, STAGE_CHUNK));
    if (!staged_any) {
      e = cudaStreamWaitEvent(st, p->stage_done[dir], 0);   // the staging area may still be in use on another stream
      if (e != cudaSuccess) break;
      staged_any = true;
    }
    IdChunk ch;
    for (uint32_t i = 0; i < len; ++i) ch.ids[i] = dev_ids[order[k + i]];
    if (in) {
      e = cudaMemcpyAsync(p->stage[dir], h, len * bb, cudaMemcpyHostToDevice, st);
      if (e == cudaSuccess) {
        block_stage_kernel<<<len * parts, 256, 0, st>>>(p->slab, p->stage[dir], ch, u4, parts, p->n_blocks, 0, p->d_flags);
        e = cudaGetLastError();
      }
    } else {
      block_stage_kernel<<<len * parts, 256, 0, st>>>(p->slab, p->stage[dir], ch, u4, parts, p->n_blocks, 1, p->d_flags);
      e = cudaGetLastError();
      if (e == cudaSuccess) e = cudaMemcpyAsync(h, p->stage[dir], len * bb, cudaMemcpyDeviceToHost, st);
    }
    k += len;
  }
  if (staged_any && e == cudaSuccess) e = cudaEventRecord(p->stage_done[dir], st);
  int rc = FL_OK;
  if (e != cudaSuccess) {
    p->last_cuda = (int)e;
    rc = FL_ECUDA;
  } else {
    (in ? p->bytes_in : p->bytes_out) += (uint64_t)n * bb;
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
  // four independent 16-byte loads in flight per thread before the first store
  for (int c0 = threadIdx.x; c0 < 2 * per_side; c0 += 4 * blockDim.x) {
    uint4 val[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + u * blockDim.x;
      if (c < 2 * per_side) {
        const int w = c / per_side, r = c - w * per_side;
        val[u] = (w ? v_new : k_new)[(size_t)t * per_side + r];
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int c = c0 + u * blockDim.x;
      if (c < 2 * per_side) {
        const int w = c / per_side, r = c - w * per_side;
        const int h = r / CH, e = r - h * CH;
        dst[((size_t)(w * n_kv + h) * bt + slot) * CH + e] = val[u];
      }
    }
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

// ---- which requests may run while swap-ins are in flight (Section 4.3)
namespace {
// Polls the events of the live tickets; a finished ticket releases its blocks lazily (when they are looked at).
int poll_tickets(fl_pool* p) {
  for (auto& t : p->tickets) {
    if (t.n_blocks == 0 || t.done) continue;
    const cudaError_t e = cudaEventQuery(t.ev);
    if (e == cudaSuccess) {
      t.done = true;
    } else if (e != cudaErrorNotReady) {
      p->last_cuda = (int)e;
      return FL_ECUDA;
    }
  }
  return FL_OK;
}
// True while block b waits for a copy; clears the mark of a block whose ticket has finished.
bool block_in_flight(fl_pool* p, uint32_t b) {
  const uint32_t m = p->inflight[b];
  if (m == 0) return false;
  fl_pool::Ticket& t = p->tickets[m - 1];
  if (!t.done) return true;
  p->inflight[b] = 0;
  if (--t.n_blocks == 0) { t.ev = nullptr; t.done = false; }
  return false;
}
}  // namespace

int fl_inflight_mark(fl_pool* p, const uint32_t* dev_ids, uint32_t n, fl_event ev) {
  if (!p || !ev || (n && !dev_ids)) return FL_EINVAL;
  for (uint32_t k = 0; k < n; ++k)
    if (dev_ids[k] >= p->n_blocks) return FL_EBADID;
  if (n == 0) return FL_OK;
  if (p->inflight.empty()) p->inflight.assign(p->n_blocks, 0u);
  uint32_t slot = 0;
  while (slot < p->tickets.size() && p->tickets[slot].n_blocks != 0) ++slot;
  if (slot == p->tickets.size()) p->tickets.emplace_back();
  fl_pool::Ticket& t = p->tickets[slot];
  t.ev = (cudaEvent_t)ev;
  t.done = false;
  t.n_blocks = 0;
  for (uint32_t k = 0; k < n; ++k) {
    const uint32_t b = dev_ids[k];
    const uint32_t old = p->inflight[b];
    if (old == slot + 1) continue;                    // listed twice in this call
    if (old != 0) {                                   // a newer copy supersedes the older mark
      fl_pool::Ticket& o = p->tickets[old - 1];
      if (--o.n_blocks == 0) { o.ev = nullptr; o.done = false; }
    }
    p->inflight[b] = slot + 1;
    ++t.n_blocks;
  }
  return FL_OK;
}

int fl_requests_ready(fl_pool* p, const int32_t* blk_indptr, const uint32_t* blks, int n_req, uint8_t* ready,
                      int* n_ready) {
  if (!p || n_req < 0 || (n_req && (!blk_indptr || !ready))) return FL_EINVAL;
  for (int r = 0; r < n_req; ++r) {
    if (blk_indptr[r + 1] < blk_indptr[r] || blk_indptr[r] < 0) return FL_EINVAL;
    if (blk_indptr[r + 1] > blk_indptr[r] && !blks) return FL_EINVAL;
    for (int k = blk_indptr[r]; k < blk_indptr[r + 1]; ++k)
      if (blks[k] >= p->n_blocks) return FL_EBADID;
  }
  const int rc = poll_tickets(p);
  if (rc != FL_OK) return rc;
  int count = 0;
  for (int r = 0; r < n_req; ++r) {
    bool ok = true;
    if (!p->inflight.empty())
      for (int k = blk_indptr[r]; k < blk_indptr[r + 1]; ++k)
        if (block_in_flight(p, blks[k])) ok = false;   // no early exit: every finished mark it meets is cleared
    ready[r] = ok ? 1 : 0;
    count += ok ? 1 : 0;
  }
  if (n_ready) *n_ready = count;
  return FL_OK;
}

int fl_inflight_count(fl_pool* p, uint32_t* n_blocks) {
  if (!p || !n_blocks) return FL_EINVAL;
  const int rc = poll_tickets(p);
  if (rc != FL_OK) return rc;
  uint32_t c = 0;
  for (const auto& t : p->tickets)
    if (t.n_blocks != 0 && !t.done) c += t.n_blocks;
  *n_blocks = c;
  return FL_OK;
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
