/*
 * fastpool - C ABI of the multi-LoRA forward step over one unified LoRA/KV block pool (sm_100a).
 *
 * The paper (Section 4.3, "Unified Caching Pool for LoRAs and KVs") cuts HBM and main memory into
 * blocks of one size, keeps LoRA adapters (partitioned block-wise along the rank dimension) and KV
 * caches in the same blocks, addresses them through block tables, and swaps whole blocks between
 * the two memories on a side stream.  This library is that pool plus the three computations that
 * run over it: the segmented LoRA projection (Eq. 1, Eq. 2, Section 2.1), paged prefill/decode
 * attention over [cached prefix || new tokens] (Section 2.1, Section 4.2), and the block swap
 * (Section 4.3 "Asynchronous Swapping-in/out").
 *
 * Conventions
 *  - Every function returns an int status: FL_OK or a negative FL_E* code.  Nothing throws or aborts.
 *  - "device pointer" = memory of the pool's GPU, owned by the caller, at least 16-byte aligned;
 *    "host pointer" = ordinary host memory.  The library never frees caller memory.
 *  - bf16 values are passed as raw 16-bit patterns (fl_bf16).  Head dimension is 128.
 *  - Kernel launches are asynchronous on the given stream; a status of FL_OK means "enqueued".  After one
 *    ordinary call of each kind (which configures its kernels), fl_lora_sgmv, fl_lora_sgmv_multi, fl_kv_append
 *    and fl_paged_attention only launch kernels on that stream and can be recorded into a CUDA graph.
 *    Kernels never trap: a block id or token position outside the pool makes the thread skip the
 *    access and set a sticky flag that fl_pool_status reports.
 *  - A pool belongs to one device; calls on one pool from several host threads must be serialised
 *    by the caller.
 */
#ifndef FASTPOOL_H
#define FASTPOOL_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct fl_pool fl_pool;
typedef uint16_t fl_bf16;
typedef struct CUstream_st* fl_stream;   /* a cudaStream_t; NULL = the default stream */
typedef struct CUevent_st* fl_event;     /* a cudaEvent_t */

enum {
  FL_OK = 0,
  FL_EINVAL = -1,   /* bad argument (null pointer, misaligned size, shape the kernels do not cover) */
  FL_ENOMEM = -2,   /* not enough free blocks (the paper's "HBM is full"), or workspace too small */
  FL_EBADID = -3,   /* block id out of range / not allocated / freed twice; unknown adapter id */
  FL_EBUSY = -4,    /* reserved */
  FL_ECUDA = -5,    /* a CUDA call failed; fl_last_cuda_error gives the cudaError_t */
  FL_ETIMEOUT = -6  /* fl_swap_wait: the copies did not finish before the deadline */
};

#define FL_HEAD_DIM 128
#define FL_MAX_MATS 8
#define FL_MAX_RANK 64
#define FL_MAX_LORA_ID (1 << 20)

/* Shape of one LoRA-carrying projection: A is [d_in, rank], B is [rank, d_out]. */
typedef struct { int32_t d_in, d_out; } fl_lora_shape;

/* Sticky device-side flags and counters, see fl_pool_status. */
typedef struct {
  uint32_t device_flags;        /* bit 0: block id out of range seen by a kernel; bit 1: token position
                                   beyond its block table; bit 2: adapter id not registered;
                                   bit 3: a bounded wait inside a kernel gave up */
  uint32_t blocks_used, blocks_free, host_blocks_used, host_blocks_free;
  uint32_t lora_blocks;         /* device blocks referenced by registered adapters */
  uint64_t bytes_swapped_in, bytes_swapped_out;
  uint64_t staging_bytes;       /* device memory the pool holds outside the slab for the swap path's two staging
                                   areas (see fl_swap_out); 0 when the pool has fewer than two host blocks */
} fl_status;

/* ---------------------------------------------------------------- pool (Section 4.3)
 * Allocates one device slab of n_blocks * block_bytes on `device` and one pinned host slab of
 * n_host_blocks * block_bytes ("both HBM and main memory are partitioned into memory blocks of the
 * same size").  block_bytes must be a multiple of 512.  The pool owns both slabs until
 * fl_pool_destroy.  FL_ECUDA if an allocation fails. */
int fl_pool_create(fl_pool** out, size_t block_bytes, uint32_t n_blocks, uint32_t n_host_blocks, int device);
int fl_pool_destroy(fl_pool* pool);

/* Block allocator.  The paper only says freed blocks are recycled for future allocations; the order
 * used here: each memory has a LIFO stack, a fresh pool hands out 0, 1, 2, ..., fl_block_free pushes
 * ids in list order.  Both calls are all-or-nothing: FL_ENOMEM (alloc) or FL_EBADID (free of an id
 * that is out of range, not allocated, or listed twice) leave the pool unchanged.  ids: host pointer. */
int fl_block_alloc(fl_pool* pool, uint32_t n, uint32_t* ids);
int fl_block_free(fl_pool* pool, uint32_t n, const uint32_t* ids);
int fl_host_block_alloc(fl_pool* pool, uint32_t n, uint32_t* ids);
int fl_host_block_free(fl_pool* pool, uint32_t n, const uint32_t* ids);

/* Base addresses of the two slabs (block i starts at base + i * block_bytes). */
void* fl_pool_device_base(fl_pool* pool);
void* fl_pool_host_base(fl_pool* pool);

/* Synchronous copy of one DEVICE block to / from ordinary host memory (block_bytes bytes); for
 * inspection and tests, not part of the hot path.  FL_EBADID if id >= n_blocks. */
int fl_block_read(fl_pool* pool, uint32_t id, void* dst_host);
int fl_block_write(fl_pool* pool, uint32_t id, const void* src_host);

/* Copies the free stack (bottom first; the last entry is handed out next) into `free_ids` (host pointer,
 * capacity `cap`) and writes its length to *n_free.  host != 0 selects the host memory's stack.
 * Used to compare allocator state bit for bit. */
int fl_pool_snapshot(fl_pool* pool, int host, uint32_t* free_ids, uint32_t cap, uint32_t* n_free);
/* Reads the sticky device flags (synchronises the device) and the counters.  clear != 0 resets the flags. */
int fl_pool_status(fl_pool* pool, fl_status* out, int clear);
int fl_last_cuda_error(fl_pool* pool);
/* Switches.  FL_OPT_PREFILL_KERNEL: 0 (default) = prefill attention on tcgen05 tensor cores with
 * TMEM accumulators and TMA-staged pages, two query tiles per CTA sharing the K/V stream; 1 = the
 * mma.sync kernel.  Same results within rounding.  The tcgen05 kernel needs sm_scale > 0; other values are
 * served by the mma.sync kernel.
 * FL_OPT_POISON_FREED: 1 = debugging aid that stands in for a memory checker: fl_block_free waits for the
 * device and fills every freed DEVICE block with 0xFF bytes (bf16 NaN patterns), so a block table that still
 * names a freed block turns the output of whatever reads it into NaN instead of plausible numbers.  0 (default)
 * = freed blocks keep their contents and fl_block_free touches no device memory. */
#define FL_OPT_PREFILL_KERNEL 1
#define FL_OPT_POISON_FREED 2
/* FL_OPT_SGMV_SHRINK: 0 (default) = batches of long segments run the shrink x A_i on tcgen05 tensor cores (tiles of
 * 128 tokens, x staged by TMA, adapter rows by cp.async, accumulator in TMEM); 1 = the mma.sync shrink for every
 * batch.  Same results within rounding (both accumulate in fp32; the order of the sums differs). */
#define FL_OPT_SGMV_SHRINK 3
int fl_pool_set_option(fl_pool* pool, int key, int value);

/* ---------------------------------------------------------------- adapters (Section 4.3)
 * "We perform block-wise partitioning of LoRAs along the rank dimension": an adapter is stored as
 * rank-rows.  Row p of A_m is A_m[:, p] (d_in values), row p of B_m is B_m[p, :] (d_out values); rows
 * are taken in the order A_0, B_0, A_1, B_1, ...; rows of equal width form one class (classes in order
 * of first appearance); a class is a packed sequence of rows that never straddle a block, with
 * rows_per_block = block_bytes / (2 * width); class c starts at the table entry after the blocks of
 * the classes before it.  Row g of a class is in table[class_base + g / rows_per_block] at byte
 * (g % rows_per_block) * 2 * width.  Every width must be a multiple of 8 and fit in one block.
 *
 * fl_lora_blocks: number of table entries (= blocks) such an adapter needs -> *n_table. */
int fl_lora_blocks(size_t block_bytes, int32_t rank, const fl_lora_shape* mats, int n_mats, uint32_t* n_table);
/* Writes the adapter into HOST pool blocks in that layout; weights reach HBM only through fl_swap_in
 * (the paper loads adapters from main memory).  A[m]: host pointer, [d_in, rank] row-major;
 * B[m]: host pointer, [rank, d_out] row-major; host_blocks: n_table allocated host block ids. */
int fl_lora_pack_host(fl_pool* pool, int32_t rank, const fl_lora_shape* mats, int n_mats,
                      const fl_bf16* const* A, const fl_bf16* const* B,
                      const uint32_t* host_blocks, uint32_t n_table);
/* Registers adapter `lora_id` (0 <= id < FL_MAX_LORA_ID, 1 <= rank <= FL_MAX_RANK, n_mats <= FL_MAX_MATS)
 * whose rows live in the DEVICE blocks block_table[0..n_table) (host pointer; copied into the device-side
 * adapter directory; the blocks stay allocated by the caller).  All adapters of a pool share the
 * projection shapes `mats` (ranks may differ): the first registration fixes them, a later mismatch
 * is FL_EINVAL.  Re-registering an id replaces it.  Synchronous with respect to the device. */
int fl_lora_register(fl_pool* pool, int32_t lora_id, int32_t rank, const fl_lora_shape* mats, int n_mats,
                     const uint32_t* block_table, uint32_t n_table);
int fl_lora_unregister(fl_pool* pool, int32_t lora_id);
/* Both calls wait for the device before they change the directory (kernels of any stream may be reading it).
 * A CUDA graph recorded from the compute calls keeps the directory's address and the rank its kernels were
 * built for: record it again after a registration that raises the pool's highest rank past 16 or 32, or whose
 * id is 4096 or more above every id registered before (the directory grows by doubling).  A kernel that meets
 * an adapter of a higher rank than it was built for leaves out the extra rank-rows and sets bit 2 of
 * device_flags. */

/* Read-back of what the DEVICE holds for adapter `lora_id` (Section 4.3: block tables record where each block
 * is): its directory entry and its block table, copied from device memory.  For every projection m: class table
 * entry, first row inside the class and rows per block of the A rows (a_*) and of the B rows (b_*), as defined
 * above.  table (host pointer, capacity cap; may be NULL) receives the n_table block ids, *n_table (may be
 * NULL) their count; table_off is the adapter's first entry inside the pool's table arena.  Synchronises the
 * device.  FL_EBADID: no such adapter. */
typedef struct {
  uint32_t a_tab, a_row0, a_rpb, b_tab, b_row0, b_rpb;
  int32_t d_in, d_out;
} fl_lora_mat_placement;
typedef struct {
  int32_t rank, n_mats;
  uint32_t table_off, n_table;
  fl_lora_mat_placement mats[FL_MAX_MATS];
} fl_lora_placement;
int fl_lora_snapshot(fl_pool* pool, int32_t lora_id, fl_lora_placement* out, uint32_t* table, uint32_t cap,
                     uint32_t* n_table);

/* ---------------------------------------------------------------- LoRA projection (Eq. 1, Eq. 2; Section 2.1 SGMV)
 * For every segment s (tokens seg_indptr[s] .. seg_indptr[s+1]) with adapter i = lora_ids[s]:
 *     y[t, :] += scale * (x[t, :] A_i) B_i        (A_i, B_i = projection `mat_index` of adapter i)
 * y already holds the base projection x W; lora_ids[s] < 0 leaves the segment untouched.
 * x: device [n_tokens, d_in] bf16 row-major; y: device [n_tokens, d_out] bf16 row-major, updated in place
 * (fp32 accumulation, one bf16 rounding of the sum).  seg_indptr [n_seg+1], lora_ids [n_seg]: device int32.
 * workspace: device scratch of at least fl_lora_sgmv_workspace(n_tokens, n_mats) bytes, contents
 * irrelevant before and after; calls that share a workspace must be ordered on one stream.
 * The _multi form applies n_mats projections that share x (q, k, v) in one pass: ys[j] and
 * mat_indices[j] are HOST arrays of device pointers / indices. */
size_t fl_lora_sgmv_workspace(int n_tokens, int n_mats);
int fl_lora_sgmv(fl_pool* pool, fl_bf16* y, const fl_bf16* x, int mat_index,
                 const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                 float scale, void* workspace, size_t workspace_bytes, fl_stream stream);
int fl_lora_sgmv_multi(fl_pool* pool, fl_bf16* const* ys, const fl_bf16* x, const int* mat_indices, int n_mats,
                       const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                       float scale, void* workspace, size_t workspace_bytes, fl_stream stream);

/* The q, k, v projections of a layer with the KV store folded in (Eq. 2 and Section 4.3 in one pass: the K/V a
 * query generates "is directly retained in the HBM" blocks).  q is updated in place like fl_lora_sgmv.  For k
 * and v the base projections are READ from y_k, y_v and the results (base + LoRA term) are WRITTEN only into
 * the requests' pool blocks, at the positions and in the layout fl_kv_append uses (including the cleared V slots
 * behind a request's last token); y_k and y_v are left as they were.  The result in the pool is bit for bit
 * what fl_lora_sgmv_multi followed by fl_kv_append gives, without writing k, v out and reading them back.
 * Segments with lora_ids[s] < 0 get their base k, v copied into the pool.  mat_k and mat_v must have
 * d_out = n_kv_heads * 128 and the three projections share x; req_indptr .. prefix_lens as in fl_kv_append;
 * workspace as in fl_lora_sgmv_multi with n_mats = 3. */
/* Blocks of up to 128 tokens and pools of up to 2^24 blocks (FL_EINVAL beyond). */
int fl_lora_sgmv_qkv_append(fl_pool* pool, fl_bf16* y_q, const fl_bf16* y_k, const fl_bf16* y_v, const fl_bf16* x,
                            int mat_q, int mat_k, int mat_v, const int32_t* seg_indptr, const int32_t* lora_ids,
                            int n_seg, int n_tokens, float scale, const int32_t* req_indptr,
                            const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                            int n_req, int n_kv_heads, void* workspace, size_t workspace_bytes, fl_stream stream);

/* fl_lora_sgmv without a workspace argument, for callers that cannot allocate device memory.  (The
 * paper has no counterpart; this is a convenience of the library.)  A serving engine that follows the
 * paper hands all of its HBM to the block pool at start-up; once it is serving, a cudaMalloc may fail
 * for lack of memory, and even when it succeeds it stalls the whole device, so the step loop of such
 * an engine (and any plug-in that is not allowed to touch the engine's memory budget) has nowhere to
 * get the scratch that fl_lora_sgmv asks for.  This entry point brings its own: a fixed array of
 * FL_SGMV_STATIC_BYTES that is part of the library image, so every GPU that loads the library holds
 * that much memory until the process exits.  Neither this call nor anything it calls allocates or
 * frees device or pinned memory.
 *  - Same arguments, results and status codes as fl_lora_sgmv (one projection per call).
 *  - Limit: FL_ENOMEM, with nothing launched, when fl_lora_sgmv_workspace(n_tokens, 1) exceeds
 *    FL_SGMV_STATIC_BYTES; the 8 MiB cover every batch of up to 32767 tokens.
 *  - The first call on a device looks up the array's device address (one runtime query, remembered
 *    per device); make that first call outside any stream capture.
 *  - All calls on one device, from every pool and every thread of the process, share the array (its address
 *    is remembered per process, not per pool), and it keeps whatever the last call left in it.  The
 *    kernels overwrite every value they later read, so nothing has to be cleared between calls, but two
 *    calls whose kernels may overlap on the GPU (different streams without an ordering between them)
 *    race on it: keep such calls on one stream or order them with events. */
#define FL_SGMV_STATIC_BYTES (8u << 20)
int fl_lora_sgmv_static(fl_pool* pool, fl_bf16* y, const fl_bf16* x, int mat_index,
                        const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                        float scale, fl_stream stream);

/* ---------------------------------------------------------------- base projection with the LoRA branch folded in
 * Eq. 1 (W' = W + A B) and Eq. 2 (W q + A B q) evaluated in one pass over the output: for every token t,
 *     y[t, :] = x[t, :] W + scale * (x[t, :] A_i) B_i        (i = adapter of t's segment; none: y = x W)
 * computed by one tensor-core GEMM whose accumulator also takes the low-rank term before it is stored, so y is
 * written once and never read (fl_lora_sgmv reads and rewrites a y that another kernel produced).
 * w: device [d_in, d_out] bf16 row-major, the base weight of projection `mat_index` (shapes as registered with the
 * adapters: at least one adapter must be registered, FL_EBADID otherwise); x, seg_indptr, lora_ids as in
 * fl_lora_sgmv; y: device [n_tokens, d_out] bf16, overwritten.  fp32 accumulation over d_in and the rank, the
 * shrink result x A_i is rounded to bf16 before it meets B_i, one bf16 rounding of the result.
 * n_seg = 0 is allowed (plain y = x W).  The _multi form runs up to 3 projections that share x (q, k, v) as one
 * launch: ys, ws and mat_indices are HOST arrays.  workspace: device scratch of at least
 * fl_lora_linear_workspace(n_tokens, n_mats) bytes, same sharing rule as fl_lora_sgmv.  After one ordinary call
 * the call only launches kernels on `stream`. */
size_t fl_lora_linear_workspace(int n_tokens, int n_mats);
int fl_lora_linear(fl_pool* pool, fl_bf16* y, const fl_bf16* x, const fl_bf16* w, int mat_index,
                   const int32_t* seg_indptr, const int32_t* lora_ids, int n_seg, int n_tokens,
                   float scale, void* workspace, size_t workspace_bytes, fl_stream stream);
int fl_lora_linear_multi(fl_pool* pool, fl_bf16* const* ys, const fl_bf16* x, const fl_bf16* const* ws,
                         const int* mat_indices, int n_mats, const int32_t* seg_indptr, const int32_t* lora_ids,
                         int n_seg, int n_tokens, float scale, void* workspace, size_t workspace_bytes,
                         fl_stream stream);

/* The q, k, v projections of a layer from x and the base weights, with the KV store folded in (Eq. 2 and Section 4.3
 * in one pass): q = x W_q + LoRA term goes to y_q; the k and v rows are never written anywhere but into the requests'
 * pool blocks, at the positions and in the layout of fl_kv_append (cleared V slots behind a request's last token
 * included).  Bit for bit what fl_lora_linear_multi followed by fl_kv_append stores.  mat_k and mat_v must have
 * d_out = n_kv_heads * 128.  scratch_k, scratch_v: device [n_tokens, n_kv_heads * 128] bf16 each, needed only by
 * batches of short segments (n_tokens <= 16 * n_seg, e.g. a decode step), where x W is formed first and the segmented
 * projection then stores base + LoRA term; may be NULL otherwise (FL_EINVAL if such a batch comes without them).
 * workspace as fl_lora_linear_workspace(n_tokens, 3). */
int fl_lora_linear_qkv_append(fl_pool* pool, fl_bf16* y_q, const fl_bf16* x, const fl_bf16* w_q, const fl_bf16* w_k,
                              const fl_bf16* w_v, int mat_q, int mat_k, int mat_v, const int32_t* seg_indptr,
                              const int32_t* lora_ids, int n_seg, int n_tokens, float scale, const int32_t* req_indptr,
                              const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens, int n_req,
                              int n_kv_heads, fl_bf16* scratch_k, fl_bf16* scratch_v, void* workspace,
                              size_t workspace_bytes, fl_stream stream);

/* ---------------------------------------------------------------- KV store (Section 4.3: new KV stays in HBM blocks)
 * Writes the new tokens' K and V into the pool.  Request i owns tokens req_indptr[i] .. req_indptr[i+1]
 * of k_new / v_new (device, [n_tokens, n_kv_heads, 128] bf16); its token j goes to logical position
 * prefix_lens[i] + j, i.e. block kv_tbl[kv_tbl_indptr[i] + pos / bt], slot pos % bt, where
 * bt = block_bytes / (2 * n_kv_heads * 128 * 2).  In-block layout: [K|V][kv_head][token][128] bf16.
 * req_indptr, kv_tbl_indptr [n_req+1], prefix_lens [n_req]: device int32; kv_tbl: device uint32.
 * The tables must already cover prefix_len + new tokens.  The V slots behind a request's last token in
 * its last block are set to zero (attention reads whole blocks; K/V stored by other means must keep
 * unused slots finite). */
int fl_kv_append(fl_pool* pool, const fl_bf16* k_new, const fl_bf16* v_new, const int32_t* req_indptr,
                 const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                 int n_req, int n_tokens, int n_kv_heads, fl_stream stream);

/* ---------------------------------------------------------------- paged attention (Section 2.1, Section 4.2)
 * For request i, query head h (KV head h / (n_q_heads / n_kv_heads)) and new token j:
 *     out = softmax_{u <= prefix_lens[i] + j}(sm_scale * <q, k_u>) . v_u
 * over the request's keys/values read from pool blocks through its table: the cached prefix is
 * reused as stored, the new tokens (already appended) are causal.  Prefill, decode (new_len 1) and
 * mixed batches go through the same call.  q, out: device [n_tokens, n_q_heads, 128] bf16 packed by
 * request (req_indptr); new_lens[i] = req_indptr[i+1] - req_indptr[i].  n_tbl = total number of
 * table entries.  Needs block tokens bt = 16.  out on a 32-byte boundary lets the prefill kernel store 32 bytes per
 * instruction (16-byte alignment, the general rule, is enough; the result is the same).  workspace: device scratch of at
 * least fl_paged_attention_workspace(...) bytes; same sharing rule as above. */
size_t fl_paged_attention_workspace(int n_req, int n_tokens, int n_tbl, int n_q_heads, int n_kv_heads);
int fl_paged_attention(fl_pool* pool, fl_bf16* out, const fl_bf16* q, const int32_t* req_indptr,
                       const int32_t* kv_tbl_indptr, const uint32_t* kv_tbl, const int32_t* prefix_lens,
                       const int32_t* new_lens, int n_req, int n_tokens, int n_tbl,
                       int n_q_heads, int n_kv_heads, float sm_scale,
                       void* workspace, size_t workspace_bytes, fl_stream stream);

/* ---------------------------------------------------------------- swap (Section 4.3 "Asynchronous Swapping-in/out")
 * Copies whole blocks between the device slab and the pinned host slab, pair k = (dev_ids[k],
 * host_ids[k]) (host pointers), asynchronously on `side`, so that it overlaps kernels running on other
 * streams.  Every listed block must be allocated (FL_EBADID) and no block may be listed twice in one
 * call (FL_EINVAL); on either error nothing is copied.  The transfers run on the copy engines: pairs
 * that are consecutive in both memories go as one DMA; a run of consecutive host blocks whose device
 * blocks are scattered goes through a staging area (one small gather or scatter kernel on `side` plus one
 * DMA for up to 256 blocks), which is what a fragmented pool needs to keep the host link busy.  The two
 * staging areas are device memory that fl_pool_create allocates OUTSIDE the slab: min(256, n_blocks,
 * n_host_blocks) blocks each (128 MiB in all at 256 KiB blocks), none when the pool has fewer than two host
 * blocks; fl_pool_status reports the total as staging_bytes.  Swap-out and swap-in have separate staging areas, so the two directions overlap when they
 * are given different streams; calls in one direction are ordered among themselves by the library even
 * across streams.  The caller guarantees that no kernel in flight touches the listed device blocks
 * (the paper evicts only nodes no running query uses, and a query whose blocks are in flight waits).
 * fl_swap_record records `ev` on the side stream; fl_swap_wait polls it on the host until done or
 * timeout_ms elapsed (FL_ETIMEOUT) - no device-side waiting. */
int fl_swap_out(fl_pool* pool, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side);
int fl_swap_in(fl_pool* pool, const uint32_t* dev_ids, const uint32_t* host_ids, uint32_t n, fl_stream side);
int fl_swap_record(fl_pool* pool, fl_event ev, fl_stream side);
int fl_swap_wait(fl_pool* pool, fl_event ev, int timeout_ms);

/* ---------------------------------------------------------------- readiness while blocks are in flight
 * Section 4.3 "Asynchronous Swapping-in/out": a query whose adapter or cached KV is still being swapped in
 * waits, and the queries that are ready run meanwhile.  Host code; all pointers are host pointers.
 * fl_inflight_mark: the listed device blocks are the targets of copies already enqueued on a side stream;
 * they count as in flight until `ev` - recorded behind those copies with fl_swap_record - has completed.  The
 * caller keeps `ev` alive until then.  A block marked again moves to the newer event.  FL_EBADID: id out of range.
 * fl_requests_ready: request r touches the device blocks blks[blk_indptr[r] .. blk_indptr[r+1]) (its adapter's
 * blocks and its KV blocks); ready[r] = 1 when none of them is in flight, else 0.  Events are polled first
 * (cudaEventQuery, no waiting) and finished ones release their blocks.  *n_ready (may be NULL) = how many are
 * ready.  fl_inflight_count: blocks still waiting for their copies after the same poll. */
int fl_inflight_mark(fl_pool* pool, const uint32_t* dev_ids, uint32_t n, fl_event ev);
int fl_requests_ready(fl_pool* pool, const int32_t* blk_indptr, const uint32_t* blks, int n_req, uint8_t* ready,
                      int* n_ready);
int fl_inflight_count(fl_pool* pool, uint32_t* n_blocks);

/* ---------------------------------------------------------------- cache swapper (Section 5; host code, no GPU work)
 * Decides WHICH nodes (LoRA adapters, KV caches) move between HBM and host memory; the block lists of
 * the chosen nodes then go to fl_swap_out / fl_swap_in.  A node is described by what the usage
 * dependency tree records for it (Section 4.3): kind, where it lives, size, visit count, last use. */
enum { FL_NODE_LORA = 0, FL_NODE_KV = 1 };
typedef struct {
  int32_t kind;         /* FL_NODE_LORA or FL_NODE_KV */
  int32_t in_hbm;       /* non-zero: resident in HBM; zero: in host memory */
  int32_t candidate;    /* non-zero: the tree offers this node (an HBM leaf for swap-out, the root of a
                           host-resident path for swap-in, Section 4.2) */
  uint32_t n_blocks;    /* size in pool blocks */
  double visits;        /* visit count of the node */
  double last_use_s;    /* time of its last use, seconds */
} fl_node_stat;
typedef struct {
  double now_s;             /* current time, seconds (t_i = now_s - last_use_s) */
  double total_visits;      /* prob_i = visits_i / total_visits */
  double low_lora;          /* Eq. 3, see fl_expected_lora_demand */
  int32_t now_lora;         /* adapters resident in HBM now */
  size_t block_bytes;
  double link_bytes_per_s;  /* host link bandwidth: cost_i = node bytes / bandwidth (Section 5.2) */
  double upper, lower;      /* HBM usage thresholds of the monitor tick (the paper uses 0.95 and 0.70) */
} fl_swap_params;
/* Eq. 3: expected number of distinct adapters a batch of `batch_size` queries needs,
 * sum_i (1 - (1 - prob_i)^batch_size).  prob: host pointer, n values in [0, 1]. */
int fl_expected_lora_demand(const double* prob, int n, int batch_size, double* low_lora);
/* Eq. 4 - Eq. 6 for every node: eval[i] = LoRA_Eval_i * cost_i * prob_i * (1 - sigmoid(t_i)), with
 * LoRA_Eval_i = max(1, low_lora / now_lora) for LoRA nodes and 1 for KV nodes (the coefficient rewards
 * loading adapters while fewer are resident than the batch is expected to need).  A higher value means
 * more benefit from keeping the node in HBM.  eval: host pointer, n doubles. */
int fl_swap_eval(const fl_node_stat* nodes, int n, const fl_swap_params* prm, double* eval);
/* One monitor tick (Section 5.3).  usage = blocks_used / blocks_total.  usage > upper: swap-out, candidates
 * resident in HBM in ascending eval, one by one until usage <= upper (*direction = -1).  usage < lower:
 * swap-in, candidates in host memory in descending eval, one by one until usage >= lower, skipping a node
 * that would push usage above upper (*direction = +1).  Otherwise nothing (*direction = 0, *n_order = 0).
 * Equal evals keep the lower node index first.  order: host pointer with room for n indices. */
int fl_swapper_decide(const fl_node_stat* nodes, int n, const fl_swap_params* prm, uint32_t blocks_used,
                      uint32_t blocks_total, int32_t* order, int* n_order, int* direction);

/* The ablations of Section 6 ("Effectiveness of the Cache Swapper", "Effectiveness of the Enough LoRAs"): the same
 * tick with parts of the cost model switched off.  FL_POLICY_LRU: candidates are ordered by last use alone (the
 * node used longest ago leaves first, the node used last enters first) instead of Eq. 6.  FL_POLICY_NO_LORA_REWARD:
 * the coefficient of Eq. 4 is 1 for every node.  policy = 0 is fl_swapper_decide.  Unlike fl_swapper_decide,
 * blocks_used may exceed blocks_total: a caller that needs room for blocks it has not allocated yet adds them to
 * blocks_used, and the swap-out list then frees enough for usage to fall back to `upper`.
 * FL_POLICY_ONLY_LORA / FL_POLICY_ONLY_KV: only nodes of that kind are offered; with blocks_used and blocks_total
 * those of one partition this is the tick of a statically partitioned HBM (Section 2.2: a fixed share for LoRAs,
 * the rest for KV caches, the setting the unified pool replaces). */
enum { FL_POLICY_LRU = 1, FL_POLICY_NO_LORA_REWARD = 2, FL_POLICY_ONLY_LORA = 4, FL_POLICY_ONLY_KV = 8 };
int fl_swapper_decide_policy(const fl_node_stat* nodes, int n, const fl_swap_params* prm, uint32_t blocks_used,
                             uint32_t blocks_total, uint32_t policy, int32_t* order, int* n_order, int* direction);

/* ---------------------------------------------------------------- usage dependency tree (Section 4; host code)
 * Virtual root -> LoRA nodes (second layer) -> KV nodes, one per pool block of block_tokens tokens, labelled
 * by those tokens; conversations with a common prefix share its nodes.  The tree only records block ids
 * ("without altering the physical allocation", Section 4.3); the caller allocates, frees and swaps blocks.
 * Node ids are dense, starting at 0, in creation order; fl_tree_stats index i describes node i, so the order
 * fl_swapper_decide returns is a list of node ids. */
typedef struct fl_tree fl_tree;
int fl_tree_create(fl_tree** out, int block_tokens);
int fl_tree_destroy(fl_tree* tree);
/* Adds the node of adapter lora_id with its block table (device blocks if in_hbm, else host blocks).
 * FL_EBADID if the adapter has a node already.  *node (may be NULL) receives the node id. */
int fl_tree_add_lora(fl_tree* tree, int32_t lora_id, const uint32_t* blocks, uint32_t n_blocks, int in_hbm,
                     double now_s, int32_t* node);
/* Matching of an arriving query (Section 4.2): its LoRA node, then KV nodes depth first, one per whole block
 * of `tokens`, until no child carries the next block_tokens tokens.  kv_nodes[0..*n_kv_nodes) is the matched
 * path (cap entries available, FL_ENOMEM if too few), *matched_tokens = *n_kv_nodes * block_tokens.  Every
 * matched node (the LoRA node included) gets one visit and last use = now_s.  Nodes that live in host memory
 * are still matched: the caller swaps them in (root first) before the query runs.  FL_EBADID: unknown adapter. */
int fl_tree_match(fl_tree* tree, int32_t lora_id, const int32_t* tokens, int n_tokens, double now_s,
                  int32_t* lora_node, int32_t* kv_nodes, int cap, int* n_kv_nodes, int* matched_tokens);
/* Inserts n_new_blocks KV nodes as a chain below `parent` (the last matched node, or the LoRA node): node k is
 * labelled tokens[k * block_tokens ..) and records device block block_ids[k].  New KV is generated in HBM, so
 * the parent must be in HBM (FL_EBUSY).  FL_EBADID if such a child exists already.  new_nodes may be NULL. */
int fl_tree_insert(fl_tree* tree, int32_t parent, const int32_t* tokens, int n_new_blocks, const uint32_t* block_ids,
                   double now_s, int32_t* new_nodes);
int fl_tree_size(fl_tree* tree);
int fl_tree_node_blocks(fl_tree* tree, int32_t node, uint32_t* blocks, uint32_t cap, uint32_t* n_blocks);
/* What the cache swapper needs (Section 5.3): one fl_node_stat per node, with `candidate` set for HBM nodes
 * without a child in HBM (the only nodes that may be swapped out) and for host nodes whose parent is in HBM or
 * is the virtual root (the only nodes that may be swapped in); the visit total (prob_i = visits_i / total) and
 * the number of adapters in HBM.  out may be NULL to query *n_nodes only. */
int fl_tree_stats(fl_tree* tree, fl_node_stat* out, int cap, int* n_nodes, double* total_visits, int32_t* now_lora);
/* Records a finished swap of `node` with its new block ids.  FL_EBUSY if the move would break the rule of
 * Section 4.2 (a node with a child in HBM may not leave; a node whose parent is in host memory may not enter). */
int fl_tree_set_location(fl_tree* tree, int32_t node, int in_hbm, const uint32_t* blocks, uint32_t n_blocks);
/* FL_TREE_OPT_DEPENDENCY (default 1).  0 = the ablation of Section 6 "Effectiveness of the Cache Manager": usage
 * dependencies are ignored, fl_tree_stats offers every node as a candidate and fl_tree_set_location refuses no
 * move, so KV nodes can stay in HBM below a node that has left ("invalid KV caches").  2 = adapters and KV caches
 * managed apart (the static partition of Section 2.2): LoRA nodes are always offered and never refused, KV nodes keep
 * the leaf / root rules among themselves, a KV node right below its adapter's node counting as a root.
 * fl_tree_invalid counts them: *hbm_kv = KV nodes in HBM, *invalid_kv = those with an ancestor (their adapter
 * included) outside HBM. */
enum { FL_TREE_OPT_DEPENDENCY = 0 };
int fl_tree_set_option(fl_tree* tree, int option, int value);
int fl_tree_invalid(fl_tree* tree, uint32_t* invalid_kv, uint32_t* hbm_kv);
/* Verifies that every node in HBM has its parent in HBM ("all KV caches that reside in the HBM are valid").
 * FL_EBADID and *first_bad (may be NULL) on a violation. */
int fl_tree_check(fl_tree* tree, int32_t* first_bad);

/* ---------------------------------------------------------------- trace replay (Sections 4.2, 5.3, 6; host code)
 * Replays a trace of queries through the dependency tree and the cache swapper with HBM reduced to `capacity`
 * blocks, and counts what the policy achieves.  Per query: match (Section 4.2); count the matched blocks that are
 * usable (adapter and whole prefix in HBM) or an adapter cold start; swap in what the query needs, root first, asking
 * the swapper for room with the query's own nodes held back (Section 5.3); insert the new KV below the matched
 * prefix; every tick_every queries one monitor tick and a sample of the share of KV nodes in HBM that an absent
 * ancestor makes unusable.  Query k arrives at t0 + k * dt seconds.  Adapters are nodes of lora_blocks blocks that
 * start in host memory.  variant: the full policy, or one of the ablations of Section 6 (FL_REPLAY_WOS: LRU instead
 * of Eq. 6; FL_REPLAY_WOL: Eq. 4 = 1; FL_REPLAY_WOM: dependencies ignored), or FL_REPLAY_STATIC: HBM cut into a
 * LoRA partition of floor(lora_share * capacity) blocks and a KV partition of the rest, each run by LRU on demand,
 * no tick moves (Section 2.2; the paper quotes a LoRA share of 0.2).
 * Query k uses adapter event_lora[k] and the tokens tokens[event_indptr[k] .. event_indptr[k+1]) (host pointers).
 * FL_ENOMEM: a query does not fit the pool even after everything offered has left. */
enum { FL_REPLAY_FULL = 0, FL_REPLAY_WOS = 1, FL_REPLAY_WOL = 2, FL_REPLAY_WOM = 3, FL_REPLAY_STATIC = 4 };
typedef struct {
  int32_t variant;
  uint32_t capacity;          /* HBM blocks */
  int32_t block_tokens;
  uint32_t lora_blocks;       /* size of every adapter */
  int32_t tick_every;
  int32_t batch_size;         /* BS of Eq. 3 */
  size_t block_bytes;
  double link_bytes_per_s, upper, lower, t0, dt;
  double lora_share;          /* FL_REPLAY_STATIC only */
} fl_replay_config;
typedef struct {
  uint64_t asked_blocks, hit_blocks, lora_cold, swapped_in, swapped_out, used_blocks, n_nodes;
  uint32_t n_samples;         /* monitor ticks taken; invalid_samples[0 .. min(n_samples, cap)) were written */
} fl_replay_result;
int fl_cache_replay(const fl_replay_config* cfg, int n_lora, const int32_t* event_lora, const int32_t* event_indptr,
                    const int32_t* tokens, int n_events, fl_replay_result* out, double* invalid_samples, uint32_t cap);

#ifdef __cplusplus
}
#endif
#endif /* FASTPOOL_H */
