// Unified block pool: slabs, LIFO block allocators, device-side adapter directory, status.
#include <string.h>
#include <algorithm>
#include <new>
#include "pool.cuh"

namespace {

struct DeviceGuard {
  int prev = -1;
  explicit DeviceGuard(int dev) { cudaGetDevice(&prev); if (prev != dev) cudaSetDevice(dev); else prev = -1; }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

int stack_alloc(BlockStack& s, uint32_t n, uint32_t* ids) {
  if (n > s.free.size()) return FL_ENOMEM;
  for (uint32_t i = 0; i < n; ++i) {
    ids[i] = s.free.back();
    s.free.pop_back();
    s.used[ids[i]] = 1;
  }
  return FL_OK;
}

int stack_free(BlockStack& s, uint32_t n, const uint32_t* ids) {
  // validate everything first (range, allocated, no duplicate inside the list), then release
  for (uint32_t i = 0; i < n; ++i) {
    if (ids[i] >= s.used.size() || s.used[ids[i]] != 1) {
      for (uint32_t j = 0; j < i; ++j) s.used[ids[j]] = 1;
      return FL_EBADID;
    }
    s.used[ids[i]] = 2;   // marks "seen in this call"
  }
  for (uint32_t i = 0; i < n; ++i) {
    s.used[ids[i]] = 0;
    s.free.push_back(ids[i]);
  }
  return FL_OK;
}

uint32_t arena_take(fl_pool* p, uint32_t len) {
  for (auto it = p->arena_free.begin(); it != p->arena_free.end(); ++it) {
    if (it->second >= len) {
      uint32_t off = it->first, rest = it->second - len;
      p->arena_free.erase(it);
      if (rest) p->arena_free[off + len] = rest;
      return off;
    }
  }
  return UINT32_MAX;
}

void arena_give(fl_pool* p, uint32_t off, uint32_t len) {
  if (!len) return;
  auto next = p->arena_free.lower_bound(off);
  if (next != p->arena_free.begin()) {
    auto prev = std::prev(next);
    if (prev->first + prev->second == off) {
      off = prev->first;
      len += prev->second;
      p->arena_free.erase(prev);
    }
  }
  if (next != p->arena_free.end() && off + len == next->first) {
    len += next->second;
    p->arena_free.erase(next);
  }
  p->arena_free[off] = len;
}

}  // namespace

int fl_layout_adapter(size_t block_bytes, int32_t rank, const fl_lora_shape* mats, int n_mats,
                      LoraMat* out, uint32_t* n_table) {
  if (!mats || n_mats < 1 || n_mats > FL_MAX_MATS || rank < 1 || rank > FL_MAX_RANK) return FL_EINVAL;
  struct Cls { int32_t width; uint32_t rows, base, rpb; };
  Cls cls[2 * FL_MAX_MATS];
  int n_cls = 0;
  int cls_of[FL_MAX_MATS][2];
  uint32_t row0[FL_MAX_MATS][2];
  for (int m = 0; m < n_mats; ++m) {
    const int32_t w[2] = {mats[m].d_in, mats[m].d_out};
    for (int side = 0; side < 2; ++side) {
      if (w[side] <= 0 || w[side] % 8 != 0 || (size_t)w[side] * 2 > block_bytes) return FL_EINVAL;
      int c = 0;
      while (c < n_cls && cls[c].width != w[side]) ++c;
      if (c == n_cls) cls[n_cls++] = Cls{w[side], 0, 0, 0};
      cls_of[m][side] = c;
      row0[m][side] = cls[c].rows;
      cls[c].rows += (uint32_t)rank;
    }
  }
  uint32_t base = 0;
  for (int c = 0; c < n_cls; ++c) {
    cls[c].rpb = (uint32_t)(block_bytes / (2 * (size_t)cls[c].width));
    cls[c].base = base;
    base += (cls[c].rows + cls[c].rpb - 1) / cls[c].rpb;
  }
  if (out) {
    for (int m = 0; m < n_mats; ++m) {
      const Cls& a = cls[cls_of[m][0]];
      const Cls& b = cls[cls_of[m][1]];
      out[m] = LoraMat{a.base, row0[m][0], a.rpb, b.base, row0[m][1], b.rpb, mats[m].d_in, mats[m].d_out};
    }
  }
  if (n_table) *n_table = base;
  return FL_OK;
}

extern "C" {

int fl_pool_create(fl_pool** out, size_t block_bytes, uint32_t n_blocks, uint32_t n_host_blocks, int device) {
  if (!out || block_bytes == 0 || block_bytes % 512 != 0 || n_blocks == 0) return FL_EINVAL;
  fl_pool* p = new (std::nothrow) fl_pool();
  if (!p) return FL_ENOMEM;
  p->device = device;
  p->block_bytes = block_bytes;
  p->n_blocks = n_blocks;
  p->n_host_blocks = n_host_blocks;
  cudaError_t e = cudaSetDevice(device);
  if (e == cudaSuccess) e = cudaMalloc(&p->slab, (size_t)n_blocks * block_bytes);
  if (e == cudaSuccess && n_host_blocks)
    e = cudaHostAlloc(&p->host_slab, (size_t)n_host_blocks * block_bytes, cudaHostAllocDefault);
  p->dir_cap = 4096;
  p->tables_cap = n_blocks;
  if (e == cudaSuccess) e = cudaMalloc(&p->d_dir, sizeof(LoraEntry) * p->dir_cap);
  if (e == cudaSuccess) e = cudaMemset(p->d_dir, 0, sizeof(LoraEntry) * p->dir_cap);
  if (e == cudaSuccess) e = cudaMalloc(&p->d_tables, sizeof(uint32_t) * (size_t)p->tables_cap);
  if (e == cudaSuccess) e = cudaMalloc(&p->d_flags, 64);
  if (e == cudaSuccess) e = cudaMemset(p->d_flags, 0, 64);
  if (e == cudaSuccess && n_host_blocks > 1) {
    // staging areas of the swap path: up to 256 blocks per direction
    p->stage_blocks = std::min(256u, std::min(n_blocks, n_host_blocks));
    for (int d = 0; d < 2 && e == cudaSuccess; ++d) {
      e = cudaMalloc(&p->stage[d], (size_t)p->stage_blocks * block_bytes);
      if (e == cudaSuccess) e = cudaEventCreateWithFlags(&p->stage_done[d], cudaEventDisableTiming);
    }
  }
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&p->sm_count, cudaDevAttrMultiProcessorCount, device);
  if (e != cudaSuccess) {
    cudaGetLastError();
    fl_pool_destroy(p);
    return FL_ECUDA;
  }
  p->dev.init(n_blocks);
  p->host.init(n_host_blocks);
  p->arena_free[0] = p->tables_cap;
  *out = p;
  return FL_OK;
}

int fl_pool_destroy(fl_pool* p) {
  if (!p) return FL_EINVAL;
  cudaSetDevice(p->device);
  cudaDeviceSynchronize();
  if (p->slab) cudaFree(p->slab);
  if (p->host_slab) cudaFreeHost(p->host_slab);
  if (p->d_dir) cudaFree(p->d_dir);
  if (p->d_tables) cudaFree(p->d_tables);
  if (p->d_flags) cudaFree(p->d_flags);
  for (int d = 0; d < 2; ++d) {
    if (p->stage[d]) cudaFree(p->stage[d]);
    if (p->stage_done[d]) cudaEventDestroy(p->stage_done[d]);
  }
  if (p->tmap_cache) free(p->tmap_cache);
  delete p;
  return FL_OK;
}

int fl_block_alloc(fl_pool* p, uint32_t n, uint32_t* ids) {
  if (!p || (n && !ids)) return FL_EINVAL;
  return stack_alloc(p->dev, n, ids);
}
int fl_block_free(fl_pool* p, uint32_t n, const uint32_t* ids) {
  if (!p || (n && !ids)) return FL_EINVAL;
  const int rc = stack_free(p->dev, n, ids);
  if (rc == FL_OK && p->poison_freed) {
    // debugging aid: a freed block is filled with bf16 NaN patterns (0xFFFF), behind everything already enqueued
    // on the device, so that a table that still names it shows up as NaN in whatever reads it
    DeviceGuard g(p->device);
    FL_CUDA(p, cudaDeviceSynchronize());
    for (uint32_t i = 0; i < n; ++i)
      FL_CUDA(p, cudaMemset(p->slab + (size_t)ids[i] * p->block_bytes, 0xFF, p->block_bytes));
  }
  return rc;
}
int fl_host_block_alloc(fl_pool* p, uint32_t n, uint32_t* ids) {
  if (!p || (n && !ids)) return FL_EINVAL;
  return stack_alloc(p->host, n, ids);
}
int fl_host_block_free(fl_pool* p, uint32_t n, const uint32_t* ids) {
  if (!p || (n && !ids)) return FL_EINVAL;
  return stack_free(p->host, n, ids);
}

void* fl_pool_device_base(fl_pool* p) { return p ? p->slab : nullptr; }
void* fl_pool_host_base(fl_pool* p) { return p ? p->host_slab : nullptr; }

int fl_block_read(fl_pool* p, uint32_t id, void* dst) {
  if (!p || !dst) return FL_EINVAL;
  if (id >= p->n_blocks) return FL_EBADID;
  DeviceGuard g(p->device);
  FL_CUDA(p, cudaDeviceSynchronize());
  FL_CUDA(p, cudaMemcpy(dst, p->slab + (size_t)id * p->block_bytes, p->block_bytes, cudaMemcpyDeviceToHost));
  return FL_OK;
}
int fl_block_write(fl_pool* p, uint32_t id, const void* src) {
  if (!p || !src) return FL_EINVAL;
  if (id >= p->n_blocks) return FL_EBADID;
  DeviceGuard g(p->device);
  FL_CUDA(p, cudaMemcpy(p->slab + (size_t)id * p->block_bytes, src, p->block_bytes, cudaMemcpyHostToDevice));
  return FL_OK;
}

int fl_pool_snapshot(fl_pool* p, int host, uint32_t* free_ids, uint32_t cap, uint32_t* n_free) {
  if (!p || !n_free) return FL_EINVAL;
  const std::vector<uint32_t>& f = host ? p->host.free : p->dev.free;
  *n_free = (uint32_t)f.size();
  if (free_ids) {
    if (cap < f.size()) return FL_EINVAL;
    if (!f.empty()) memcpy(free_ids, f.data(), f.size() * sizeof(uint32_t));
  }
  return FL_OK;
}

int fl_pool_status(fl_pool* p, fl_status* out, int clear) {
  if (!p || !out) return FL_EINVAL;
  DeviceGuard g(p->device);
  uint32_t flags = 0;
  FL_CUDA(p, cudaDeviceSynchronize());
  FL_CUDA(p, cudaMemcpy(&flags, p->d_flags, sizeof(flags), cudaMemcpyDeviceToHost));
  if (clear) FL_CUDA(p, cudaMemset(p->d_flags, 0, sizeof(flags)));
  out->device_flags = flags;
  out->blocks_free = (uint32_t)p->dev.free.size();
  out->blocks_used = p->n_blocks - out->blocks_free;
  out->host_blocks_free = (uint32_t)p->host.free.size();
  out->host_blocks_used = p->n_host_blocks - out->host_blocks_free;
  out->lora_blocks = p->lora_blocks;
  out->bytes_swapped_in = p->bytes_in;
  out->bytes_swapped_out = p->bytes_out;
  out->staging_bytes = (uint64_t)2 * p->stage_blocks * p->block_bytes;
  return FL_OK;
}

int fl_last_cuda_error(fl_pool* p) { return p ? p->last_cuda : 0; }

int fl_pool_set_option(fl_pool* p, int key, int value) {
  if (!p) return FL_EINVAL;
  if (key == FL_OPT_PREFILL_KERNEL && value >= 0 && value <= 1) {
    p->prefill_kernel = value;
    return FL_OK;
  }
  if (key == FL_OPT_SGMV_SHRINK && (value == 0 || value == 1)) {
    p->sgmv_shrink_kind = value;
    return FL_OK;
  }
  if (key == FL_OPT_POISON_FREED && (value == 0 || value == 1)) {
    p->poison_freed = value;
    return FL_OK;
  }
  return FL_EINVAL;
}

int fl_lora_blocks(size_t block_bytes, int32_t rank, const fl_lora_shape* mats, int n_mats, uint32_t* n_table) {
  if (!n_table || block_bytes == 0) return FL_EINVAL;
  return fl_layout_adapter(block_bytes, rank, mats, n_mats, nullptr, n_table);
}

int fl_lora_pack_host(fl_pool* p, int32_t rank, const fl_lora_shape* mats, int n_mats,
                      const fl_bf16* const* A, const fl_bf16* const* B,
                      const uint32_t* host_blocks, uint32_t n_table) {
  if (!p || !A || !B || !host_blocks) return FL_EINVAL;
  LoraMat lay[FL_MAX_MATS];
  uint32_t need = 0;
  int rc = fl_layout_adapter(p->block_bytes, rank, mats, n_mats, lay, &need);
  if (rc != FL_OK) return rc;
  if (need != n_table) return FL_EINVAL;
  for (uint32_t i = 0; i < n_table; ++i)
    if (host_blocks[i] >= p->n_host_blocks || !p->host.used[host_blocks[i]]) return FL_EBADID;
  for (int m = 0; m < n_mats; ++m) {
    if (!A[m] || !B[m]) return FL_EINVAL;
    const int32_t d_in = lay[m].d_in, d_out = lay[m].d_out;
    for (int32_t r = 0; r < rank; ++r) {
      // row r of A = column r of the [d_in, rank] matrix
      uint32_t g = lay[m].a_row0 + (uint32_t)r;
      fl_bf16* dst = (fl_bf16*)(p->host_slab + (size_t)host_blocks[lay[m].a_tab + g / lay[m].a_rpb] * p->block_bytes) +
                     (size_t)(g % lay[m].a_rpb) * d_in;
      for (int32_t k = 0; k < d_in; ++k) dst[k] = A[m][(size_t)k * rank + r];
      g = lay[m].b_row0 + (uint32_t)r;
      dst = (fl_bf16*)(p->host_slab + (size_t)host_blocks[lay[m].b_tab + g / lay[m].b_rpb] * p->block_bytes) +
            (size_t)(g % lay[m].b_rpb) * d_out;
      memcpy(dst, B[m] + (size_t)r * d_out, (size_t)d_out * sizeof(fl_bf16));
    }
  }
  return FL_OK;
}

int fl_lora_snapshot(fl_pool* p, int32_t lora_id, fl_lora_placement* out, uint32_t* table, uint32_t cap, uint32_t* n_table) {
  if (!p || !out || lora_id < 0) return FL_EINVAL;
  if ((uint32_t)lora_id >= p->dir_cap) return FL_EBADID;
  DeviceGuard g(p->device);
  LoraEntry e;
  FL_CUDA(p, cudaDeviceSynchronize());
  FL_CUDA(p, cudaMemcpy(&e, p->d_dir + lora_id, sizeof(e), cudaMemcpyDeviceToHost));
  if (e.rank <= 0) return FL_EBADID;
  if (e.n_mats < 0 || e.n_mats > FL_MAX_MATS || (size_t)e.table_off + e.n_table > p->tables_cap) return FL_EINVAL;
  out->rank = e.rank;
  out->n_mats = e.n_mats;
  out->table_off = e.table_off;
  out->n_table = e.n_table;
  for (int m = 0; m < FL_MAX_MATS; ++m) {
    const LoraMat& lm = e.mats[m];
    out->mats[m] = fl_lora_mat_placement{lm.a_tab, lm.a_row0, lm.a_rpb, lm.b_tab, lm.b_row0, lm.b_rpb, lm.d_in, lm.d_out};
  }
  if (n_table) *n_table = e.n_table;
  if (table) {
    if (cap < e.n_table) return FL_EINVAL;
    if (e.n_table)
      FL_CUDA(p, cudaMemcpy(table, p->d_tables + e.table_off, sizeof(uint32_t) * e.n_table, cudaMemcpyDeviceToHost));
  }
  return FL_OK;
}

int fl_lora_unregister(fl_pool* p, int32_t lora_id) {
  if (!p) return FL_EINVAL;
  auto it = p->registered.find(lora_id);
  if (it == p->registered.end()) return FL_EBADID;
  DeviceGuard g(p->device);
  // kernels on any stream may still be reading the entry and its table range, which is reused right away
  FL_CUDA(p, cudaDeviceSynchronize());
  FL_CUDA(p, cudaMemset(p->d_dir + lora_id, 0, sizeof(LoraEntry)));
  arena_give(p, it->second.table_off, it->second.n_table);
  p->lora_blocks -= it->second.n_table;
  p->registered.erase(it);
  return FL_OK;
}

int fl_lora_register(fl_pool* p, int32_t lora_id, int32_t rank, const fl_lora_shape* mats, int n_mats,
                     const uint32_t* block_table, uint32_t n_table) {
  if (!p || !block_table || lora_id < 0 || lora_id >= FL_MAX_LORA_ID) return FL_EINVAL;
  LoraEntry e;
  memset(&e, 0, sizeof(e));
  uint32_t need = 0;
  int rc = fl_layout_adapter(p->block_bytes, rank, mats, n_mats, e.mats, &need);
  if (rc != FL_OK) return rc;
  if (need != n_table) return FL_EINVAL;
  if (p->n_mats) {
    if (n_mats != p->n_mats) return FL_EINVAL;
    for (int m = 0; m < n_mats; ++m)
      if (mats[m].d_in != p->mats[m].d_in || mats[m].d_out != p->mats[m].d_out) return FL_EINVAL;
  }
  for (uint32_t i = 0; i < n_table; ++i)
    if (block_table[i] >= p->n_blocks || !p->dev.used[block_table[i]]) return FL_EBADID;
  DeviceGuard g(p->device);
  FL_CUDA(p, cudaDeviceSynchronize());   // no kernel may be reading the directory while it changes
  if (p->registered.count(lora_id)) {
    rc = fl_lora_unregister(p, lora_id);
    if (rc != FL_OK) return rc;
  }
  if ((uint32_t)lora_id >= p->dir_cap) {   // grow the directory
    uint32_t cap = p->dir_cap;
    while (cap <= (uint32_t)lora_id) cap *= 2;
    LoraEntry* nd = nullptr;
    FL_CUDA(p, cudaMalloc(&nd, sizeof(LoraEntry) * cap));
    FL_CUDA(p, cudaMemset(nd, 0, sizeof(LoraEntry) * cap));
    FL_CUDA(p, cudaMemcpy(nd, p->d_dir, sizeof(LoraEntry) * p->dir_cap, cudaMemcpyDeviceToDevice));
    cudaFree(p->d_dir);
    p->d_dir = nd;
    p->dir_cap = cap;
  }
  uint32_t off = arena_take(p, n_table);
  if (off == UINT32_MAX) return FL_ENOMEM;
  e.rank = rank;
  e.n_mats = n_mats;
  e.table_off = off;
  e.n_table = n_table;
  cudaError_t ce = cudaMemcpy(p->d_tables + off, block_table, sizeof(uint32_t) * n_table, cudaMemcpyHostToDevice);
  if (ce == cudaSuccess) ce = cudaMemcpy(p->d_dir + lora_id, &e, sizeof(e), cudaMemcpyHostToDevice);
  if (ce != cudaSuccess) {
    arena_give(p, off, n_table);
    p->last_cuda = (int)ce;
    return FL_ECUDA;
  }
  if (!p->n_mats) {
    p->n_mats = n_mats;
    memcpy(p->mats, mats, sizeof(fl_lora_shape) * n_mats);
  }
  p->registered[lora_id] = e;
  p->lora_blocks += n_table;
  p->max_rank = std::max(p->max_rank, rank);
  return FL_OK;
}

}  // extern "C"
