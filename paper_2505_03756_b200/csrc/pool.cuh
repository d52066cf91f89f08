// Internal definitions shared by the translation units of libfastpool.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <map>
#include <vector>
#include "fastpool.h"

// Placement of one projection's rank-row streams inside its adapter's block table.
struct LoraMat {
  uint32_t a_tab, a_row0, a_rpb;   // table entry of the class, first row inside the class, rows per block
  uint32_t b_tab, b_row0, b_rpb;
  int32_t d_in, d_out;
};
// Device-side adapter directory entry, indexed by lora id.
struct LoraEntry {
  int32_t rank;        // 0 = not registered
  int32_t n_mats;
  uint32_t table_off;  // first entry of this adapter's table inside the table arena
  uint32_t n_table;
  LoraMat mats[FL_MAX_MATS];
};

// What kernels need to address the pool.
struct PoolView {
  unsigned char* slab;
  size_t block_bytes;
  uint32_t n_blocks;
  const LoraEntry* dir;
  uint32_t dir_cap;
  const uint32_t* tables;
  uint32_t* flags;     // sticky status word
};

enum { FLAG_BAD_BLOCK = 1, FLAG_BAD_POS = 2, FLAG_BAD_LORA = 4, FLAG_WAIT_GAVE_UP = 8 };

struct BlockStack {
  std::vector<uint32_t> free;   // top = back
  std::vector<uint8_t> used;
  void init(uint32_t n) {
    free.resize(n);
    for (uint32_t i = 0; i < n; ++i) free[i] = n - 1 - i;
    used.assign(n, 0);
  }
};

struct fl_pool {
  int device = 0;
  size_t block_bytes = 0;
  uint32_t n_blocks = 0, n_host_blocks = 0;
  unsigned char* slab = nullptr;
  unsigned char* host_slab = nullptr;
  BlockStack dev, host;
  // adapter directory
  LoraEntry* d_dir = nullptr;
  uint32_t dir_cap = 0;
  uint32_t* d_tables = nullptr;
  uint32_t tables_cap = 0;
  std::map<uint32_t, uint32_t> arena_free;        // offset -> length of free table-arena ranges
  std::map<int32_t, LoraEntry> registered;        // host mirror
  int n_mats = 0;
  fl_lora_shape mats[FL_MAX_MATS];
  int max_rank = 0;
  uint32_t lora_blocks = 0;
  uint32_t* d_flags = nullptr;
  uint64_t bytes_in = 0, bytes_out = 0;
  int last_cuda = 0;
  int sm_count = 148;
  int prefill_kernel = 0;                           // 0: tcgen05 two-tile kernel, 1: mma.sync kernel
  int sgmv_shrink_kind = 0;                         // 0: tcgen05 shrink for long segments, 1: mma.sync shrink everywhere
  int poison_freed = 0;                             // debugging aid: freed device blocks are filled with NaN patterns
  unsigned char* stage[2] = {nullptr, nullptr};     // contiguous staging areas of the swap path (out, in)
  uint32_t stage_blocks = 0;
  cudaEvent_t stage_done[2] = {nullptr, nullptr};   // last use of each staging area
  void* tmap_cache = nullptr;                      // tensor maps of the slab, keyed by KV head count
  // blocks that copies in flight are still filling: inflight[b] = 1 + index into tickets, 0 = none
  struct Ticket { cudaEvent_t ev = nullptr; uint32_t n_blocks = 0; bool done = false; };
  std::vector<uint32_t> inflight;
  std::vector<Ticket> tickets;
  PoolView view() const { return PoolView{slab, block_bytes, n_blocks, d_dir, dir_cap, d_tables, d_flags}; }
};

// Programmatic dependent launch.  A kernel launched through launch_pdl may start while the kernel before it on
// the stream is still running; it calls pdl_wait() before it touches anything that kernel may have written (or
// may still read), which waits for that whole grid and its memory operations.  A kernel that calls
// pdl_launch_dependents() lets the next one start once all its CTAs are past that point.  Both instructions do
// nothing in a kernel launched the ordinary way.
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

#define FL_CUDA(pool, call)                                  \
  do {                                                       \
    cudaError_t e__ = (call);                                \
    if (e__ != cudaSuccess) {                                \
      if (pool) (pool)->last_cuda = (int)e__;                \
      return FL_ECUDA;                                       \
    }                                                        \
  } while (0)

// Layout arithmetic of an adapter (host side).
int fl_layout_adapter(size_t block_bytes, int32_t rank, const fl_lora_shape* mats, int n_mats,
                      LoraMat* out, uint32_t* n_table);
