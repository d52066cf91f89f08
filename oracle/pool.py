"""O3/O4/O5 - byte-level model of the unified caching pool (Section 4.3 of the paper).

The paper cuts HBM and main memory into blocks of one size, stores LoRA adapters (partitioned
block-wise along the rank dimension) and KV caches in the same blocks, recycles freed blocks, keeps
newly generated KV in HBM, addresses blocks through tables that never move the data, and swaps
whole blocks between the two memories.  The paper fixes no byte layout or allocation order; the
readings used here (and, independently, by the CUDA library) are:

  allocator   LIFO stack per memory; a fresh pool hands out 0, 1, 2, ...; free(ids) pushes ids in list
              order; both calls are all-or-nothing.
  KV block    [K|V][kv_head][token][d] bf16: byte offset (((w*n_kv + h)*bt + t)*d + e)*2,
              bt = block_bytes / (2 * n_kv * d * 2).
  adapter     rank-rows: row p of A is A[:, p] (d_in values), row p of B is B[p, :] (d_out values).
              Rows are taken in the order A_0, B_0, A_1, B_1, ...; rows of equal width form one class
              (classes ordered by first appearance), a class is a packed stream of rows that never
              straddle a block: rows_per_block = block_bytes // (2*width); class c starts at table
              entry sum of the block counts of the classes before it; row g of the class lives in
              table[class_base + g // rows_per_block] at byte (g % rows_per_block) * 2 * width.

Pins: paged gather == contiguous storage and results do not depend on which physical blocks are
used; allocator replayed against brute-force set bookkeeping (no id handed out twice, used + free
= n_blocks, a failed call changes nothing, LIFO order on a hand-written trace); swap-out followed
by swap-in elsewhere returns identical bytes and touches no other block; adapter block counts for
the paper-shaped layers (2 blocks for a 7B rank-8 adapter, 16 for the 13B rank-32 adapter with MLP,
100 for the 34B rank-64 adapter); table entry and byte offset of single adapter elements of the 34B
rank-64 adapter worked out by hand (both width classes, first and last value of a block).
"""
import numpy as np

OK, EINVAL, ENOMEM, EBADID = 0, -1, -2, -3


class PoolError(Exception):
    def __init__(self, code, msg=""):
        super().__init__(f"pool error {code} {msg}")
        self.code = code


def bf16_bits_to_f64(bits):
    b = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return b.view(np.float32).astype(np.float64)


def f64_to_bf16_bits(x):
    """Round to nearest even into bf16 storage (via float32, then the top 16 bits)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    return ((u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)).astype(np.uint16)


class _Stack:
    """LIFO block allocator of one memory."""

    def __init__(self, n):
        self.n = n
        self.free = list(range(n - 1, -1, -1))   # top of stack = end of list -> pops 0, 1, 2, ...
        self.used = [False] * n

    def alloc(self, n):
        if n > len(self.free):
            raise PoolError(ENOMEM)
        ids = [self.free.pop() for _ in range(n)]
        for i in ids:
            self.used[i] = True
        return ids

    def release(self, ids):
        seen = set()
        for i in ids:
            if i < 0 or i >= self.n or not self.used[i] or i in seen:
                raise PoolError(EBADID, str(i))
            seen.add(i)
        for i in ids:
            self.used[i] = False
            self.free.append(i)


def lora_layout(block_bytes, rank, mats):
    """Placement of every rank-row stream of an adapter.  mats = [(d_in, d_out), ...].

    Returns (n_table_entries, {(m, 'A'|'B'): (class_base, first_row, rows_per_block, width)}).
    """
    classes = []                      # [width, n_rows] in order of first appearance
    where = {}
    for m, (d_in, d_out) in enumerate(mats):
        for side, width in (("A", d_in), ("B", d_out)):
            for c in classes:
                if c[0] == width:
                    break
            else:
                c = [width, 0]
                classes.append(c)
            where[(m, side)] = (width, c[1])
            c[1] += rank
    base, bases = 0, {}
    for width, rows in classes:
        rpb = block_bytes // (2 * width)
        if rpb == 0:
            raise PoolError(EINVAL, "row wider than a block")
        bases[width] = (base, rpb)
        base += -(-rows // rpb)
    out = {key: (bases[w][0], first, bases[w][1], w) for key, (w, first) in where.items()}
    return base, out


class PoolModel:
    def __init__(self, block_bytes, n_blocks, n_host_blocks):
        self.block_bytes = block_bytes
        self.dev_alloc = _Stack(n_blocks)
        self.host_alloc = _Stack(n_host_blocks)
        self._mem = ({}, {})          # sparse block contents: (device, host)

    # ---- memory
    def block(self, bid, host=False):
        mem = self._mem[1 if host else 0]
        if bid not in mem:
            mem[bid] = np.zeros(self.block_bytes, dtype=np.uint8)
        return mem[bid]

    # ---- O4 allocator
    def alloc(self, n, host=False):
        return (self.host_alloc if host else self.dev_alloc).alloc(n)

    def free(self, ids, host=False):
        (self.host_alloc if host else self.dev_alloc).release(list(ids))

    def free_list(self, host=False):
        """Free stack, bottom first (the last entry is handed out next)."""
        return list((self.host_alloc if host else self.dev_alloc).free)

    # ---- O5 swap (whole blocks, list order)
    def _check_pair(self, d, h):
        if not (0 <= d < self.dev_alloc.n and self.dev_alloc.used[d]):
            raise PoolError(EBADID, f"device block {d}")
        if not (0 <= h < self.host_alloc.n and self.host_alloc.used[h]):
            raise PoolError(EBADID, f"host block {h}")

    def swap_out(self, dev_ids, host_ids):
        for d, h in zip(dev_ids, host_ids):
            self._check_pair(d, h)
        for d, h in zip(dev_ids, host_ids):
            self.block(h, host=True)[:] = self.block(d)

    def swap_in(self, dev_ids, host_ids):
        for d, h in zip(dev_ids, host_ids):
            self._check_pair(d, h)
        for d, h in zip(dev_ids, host_ids):
            self.block(d)[:] = self.block(h, host=True)

    # ---- adapters
    def pack_lora(self, table, rank, mats, A_bits, B_bits, host=True):
        """Write adapter rows (bf16 bit patterns; A_bits[m] is [d_in, r], B_bits[m] is [r, d_out])."""
        n_tab, where = lora_layout(self.block_bytes, rank, mats)
        if len(table) != n_tab:
            raise PoolError(EINVAL, "table length")
        for m in range(len(mats)):
            for side, rows in (("A", np.asarray(A_bits[m]).T), ("B", np.asarray(B_bits[m]))):
                base, first, rpb, width = where[(m, side)]
                for p in range(rank):
                    g = first + p
                    blk = self.block(int(table[base + g // rpb]), host=host).view(np.uint16)
                    off = (g % rpb) * width
                    blk[off:off + width] = rows[p]

    def read_lora(self, table, rank, mats, m, host=False):
        """Gather adapter matrix m back through its block table: (A [d_in, r], B [r, d_out]) float64."""
        _, where = lora_layout(self.block_bytes, rank, mats)
        res = []
        for side in ("A", "B"):
            base, first, rpb, width = where[(m, side)]
            rows = np.empty((rank, width), dtype=np.uint16)
            for p in range(rank):
                g = first + p
                blk = self.block(int(table[base + g // rpb]), host=host).view(np.uint16)
                off = (g % rpb) * width
                rows[p] = blk[off:off + width]
            res.append(bf16_bits_to_f64(rows))
        return res[0].T.copy(), res[1]

    # ---- KV
    def block_tokens(self, n_kv, d):
        return self.block_bytes // (2 * n_kv * d * 2)

    def kv_append(self, k_bits, v_bits, req_indptr, tables, prefix_lens, n_kv, d):
        """Store new tokens' K,V (bit patterns [T, n_kv, d]) at logical positions prefix_len_i + j."""
        bt = self.block_tokens(n_kv, d)
        for i, table in enumerate(tables):
            for j in range(int(req_indptr[i + 1]) - int(req_indptr[i])):
                t = int(req_indptr[i]) + j
                pos = int(prefix_lens[i]) + j
                blk = self.block(int(table[pos // bt])).view(np.uint16).reshape(2, n_kv, bt, d)
                blk[0, :, pos % bt, :] = k_bits[t]
                blk[1, :, pos % bt, :] = v_bits[t]

    def gather_kv(self, table, length, n_kv, d):
        """Contiguous (K, V) float64 [length, n_kv, d] of one request, read through its block table."""
        bt = self.block_tokens(n_kv, d)
        k = np.empty((length, n_kv, d), dtype=np.uint16)
        v = np.empty((length, n_kv, d), dtype=np.uint16)
        for pos in range(length):
            blk = self.block(int(table[pos // bt])).view(np.uint16).reshape(2, n_kv, bt, d)
            k[pos] = blk[0, :, pos % bt, :]
            v[pos] = blk[1, :, pos % bt, :]
        return bf16_bits_to_f64(k), bf16_bits_to_f64(v)
