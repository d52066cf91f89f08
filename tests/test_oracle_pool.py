"""Pins for oracle/pool.py (O3 storage, O4 allocator, O5 swap) and oracle/layer.py."""
import os

import numpy as np
import pytest

from oracle import pool as op
from oracle.attention import attend_request
from oracle.layer import attention_layer_step
from oracle.lora import lora_project
from paper_2505_03756_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_allocator_hand_trace():
    p = op.PoolModel(64, 6, 2)
    assert p.alloc(3) == [0, 1, 2]                 # fresh pool hands out 0, 1, 2, ...
    p.free([0, 2])                                 # pushed in list order -> 2 is on top
    assert p.alloc(3) == [2, 0, 3]
    with pytest.raises(op.PoolError) as e:
        p.alloc(3)                                 # only 4, 5 left: all-or-nothing
    assert e.value.code == op.ENOMEM
    assert p.alloc(2) == [4, 5]
    for bad in ([1, 1], [9], [-1]):
        with pytest.raises(op.PoolError) as e:
            p.free(bad)
        assert e.value.code == op.EBADID
    p.free([1])
    with pytest.raises(op.PoolError):
        p.free([3, 1])                             # 1 is already free: nothing is released
    assert p.alloc(1) == [1]
    assert p.alloc(2, host=True) == [0, 1]         # the host memory has its own stack


def test_allocator_random_trace_invariants():
    rs = synth.Stream(3, "alloc")
    p = op.PoolModel(16, 16, 0)
    held = []
    for step in range(400):
        u = rs.uniform(2)
        if u[0] < 0.55:
            n = int(u[1] * 6)
            before = p.free_list()
            try:
                ids = p.alloc(n)
            except op.PoolError as e:
                assert e.code == op.ENOMEM and n > 16 - len(held) and p.free_list() == before
                continue
            assert ids == before[::-1][:n]                         # LIFO
            assert not set(ids) & set(held) and len(set(ids)) == n  # never handed out twice
            held += ids
        elif held:
            k = 1 + int(u[1] * len(held)) % len(held)
            order = rs.permutation(len(held))[:k]
            ids = [held[i] for i in order]
            p.free(ids)
            held = [h for h in held if h not in ids]
            assert p.free_list()[-k:] == ids
        assert len(held) + len(p.free_list()) == 16 and set(held).isdisjoint(p.free_list())


def test_lora_block_counts_match_hand_arithmetic():
    for line in open(os.path.join(GOLD, "lora_blocks.txt")):
        if line.startswith("#") or not line.strip():
            continue
        _, hidden, n_q, n_kv, inter, rank, blocks = line.split()
        shp = synth.LayerShape(int(hidden), int(n_q), int(n_kv), inter=int(inter))
        n_tab, where = op.lora_layout(shp.block_bytes, int(rank), [(i, o) for _, i, o in shp.mats])
        assert n_tab == int(blocks), line
        # rows never straddle a block and no two rows overlap
        spans = set()
        for (m, side), (base, first, rpb, width) in where.items():
            assert rpb * 2 * width <= shp.block_bytes
            for r in range(int(rank)):
                g = first + r
                key = (base + g // rpb, (g % rpb) * 2 * width)
                assert key not in spans
                spans.add(key)


def test_adapter_bytes_by_hand_on_the_gqa_rank64_shape():
    """Placement of single adapter elements worked out by hand (Section 4.3: adapters are cut along the rank
    dimension into rows that share blocks with KV).  34B-class layer: hidden 8192, 64 query / 8 KV heads,
    rank 64, blocks of 64 KiB = 32768 bf16 values.  Row order A_q B_q A_k B_k A_v B_v A_o B_o; row p of A is
    A[:, p], row p of B is B[p, :].
      width 8192 (4 rows per block):  A_q rows 0..63, B_q 64..127, A_k 128..191, A_v 192..255, A_o 256..319,
                                      B_o 320..383  -> 96 blocks, table entries 0..95
      width 1024 (32 rows per block): B_k rows 0..63, B_v 64..127 -> 4 blocks, table entries 96..99
      A_k[5, 3]    = row 128 + 3 = 131  -> entry 131 // 4 = 32,     value index (131 % 4) * 8192 + 5    = 24581
      B_o[7, 100]  = row 320 + 7 = 327  -> entry 327 // 4 = 81,     value index (327 % 4) * 8192 + 100  = 24676
      B_v[9, 1000] = row 64 + 9 = 73    -> entry 96 + 73 // 32 = 98, value index (73 % 32) * 1024 + 1000 = 10216
      A_q[8191, 63] = row 63            -> entry 15,                value index 3 * 8192 + 8191 = 32767 (last of its block)
      B_k[0, 0]    = row 0 of its class -> entry 96,                value index 0"""
    shp = synth.LayerShape(8192, 64, 8)
    assert shp.block_bytes == 65536
    mats = [(i, o) for _, i, o in shp.mats]
    rank = 64
    rs = synth.Stream(12, "pin")
    A = [synth.bf16_bits(rs.normal((i, rank), 0.5)) for i, _ in mats]
    B = [synth.bf16_bits(rs.normal((rank, o), 0.5)) for _, o in mats]
    pool = op.PoolModel(shp.block_bytes, 8, 128)
    table = pool.alloc(100, host=True)[::-1]          # entry e -> host block 99 - e
    pool.pack_lora(table, rank, mats, A, B, host=True)
    q, k, v, o = 0, 1, 2, 3
    by_hand = [(32, 24581, A[k][5, 3]), (81, 24676, B[o][7, 100]), (98, 10216, B[v][9, 1000]),
               (15, 32767, A[q][8191, 63]), (96, 0, B[k][0, 0])]
    for entry, idx, want in by_hand:
        assert pool.block(99 - entry, host=True).view(np.uint16)[idx] == want, (entry, idx)
    # a whole row, so that a rotation inside the row would show as well: row 2 of B_q = entry (64 + 2) // 4, slot 2
    got = pool.block(99 - 16, host=True).view(np.uint16)[2 * 8192:3 * 8192]
    assert np.array_equal(got, B[q][2, :])
    # and the read side on its own: the gather returns A_k, not its transpose or another matrix
    a_k, b_k = pool.read_lora(table, rank, mats, k, host=True)
    assert a_k.shape == (8192, 64) and b_k.shape == (64, 1024)
    assert a_k[5, 3] == synth.bf16_to_f32(A[k][5:6, 3])[0] and b_k[9, 1000] == synth.bf16_to_f32(B[k][9:10, 1000])[0]


def _small_pool(n_blocks=40, n_kv=2, d=8, bt=4):
    return op.PoolModel(bt * 2 * n_kv * d * 2, n_blocks, 16), n_kv, d, bt


def test_paged_kv_equals_contiguous_and_ignores_block_choice():
    pool, n_kv, d, bt = _small_pool()
    rs = synth.Stream(4, "kv")
    lens = [9, 4, 13]
    k = [synth.bf16_bits(rs.normal((L, n_kv, d))) for L in lens]
    v = [synth.bf16_bits(rs.normal((L, n_kv, d))) for L in lens]
    ids = pool.alloc(20)
    pool.free([ids[i] for i in rs.permutation(20)])            # scramble the free stack
    tables = [pool.alloc(-(-L // bt)) for L in lens]
    indptr = np.concatenate([[0], np.cumsum(lens)])
    # store in two steps: a prefix first, then the rest behind it
    cut = [5, 0, 8]
    pool.kv_append(np.concatenate([a[:c] for a, c in zip(k, cut)]), np.concatenate([a[:c] for a, c in zip(v, cut)]),
                   np.concatenate([[0], np.cumsum(cut)]), tables, [0, 0, 0], n_kv, d)
    rest = [L - c for L, c in zip(lens, cut)]
    pool.kv_append(np.concatenate([a[c:] for a, c in zip(k, cut)]), np.concatenate([a[c:] for a, c in zip(v, cut)]),
                   np.concatenate([[0], np.cumsum(rest)]), tables, cut, n_kv, d)
    for i, L in enumerate(lens):
        gk, gv = pool.gather_kv(tables[i], L, n_kv, d)
        assert np.array_equal(gk, synth.bf16_to_f32(k[i]).astype(np.float64))
        assert np.array_equal(gv, synth.bf16_to_f32(v[i]).astype(np.float64))
    # byte placement of one element, by hand: request 0, position 6 -> table entry 1, slot 2
    blk = pool.block(tables[0][1]).view(np.uint16)
    assert blk[((0 * n_kv + 1) * bt + 2) * d + 3] == k[0][6, 1, 3]
    assert blk[((1 * n_kv + 0) * bt + 2) * d + 7] == v[0][6, 0, 7]
    assert indptr[-1] == 26


def test_lora_pack_gather_roundtrip_and_projection_through_pool():
    shp = synth.LayerShape(32, 2, 1, head_dim=8, inter=48, block_tokens=4)   # widths 32, 16, 8, 48
    pool = op.PoolModel(shp.block_bytes * 4, 64, 64)                        # 512-byte blocks
    mats = [(i, o) for _, i, o in shp.mats]
    rank = 3
    rs = synth.Stream(6, "lora")
    A = [synth.bf16_bits(rs.normal((i, rank), 0.5)) for i, _ in mats]
    B = [synth.bf16_bits(rs.normal((rank, o), 0.5)) for _, o in mats]
    n_tab, _ = op.lora_layout(pool.block_bytes, rank, mats)
    junk = pool.alloc(7, host=True)
    host_tab = pool.alloc(n_tab, host=True)[::-1]
    pool.pack_lora(host_tab, rank, mats, A, B, host=True)
    pool.alloc(5)
    dev_tab = pool.alloc(n_tab)
    pool.swap_in(dev_tab, host_tab)
    x = synth.round_bf16(rs.normal((5, 48)))
    for m, (d_in, d_out) in enumerate(mats):
        a, b = pool.read_lora(dev_tab, rank, mats, m)
        assert np.array_equal(a, synth.bf16_to_f32(A[m]).astype(np.float64))
        assert np.array_equal(b, synth.bf16_to_f32(B[m]).astype(np.float64))
    a, b = pool.read_lora(dev_tab, rank, mats, 5)                          # 'down': 48 -> 32
    y_pool = lora_project(np.zeros((5, 32)), x, [0, 5], [0], {0: (a, b)}, 2.0)
    y_flat = lora_project(np.zeros((5, 32)), x, [0, 5], [0],
                          {0: (synth.bf16_to_f32(A[5]), synth.bf16_to_f32(B[5]))}, 2.0)
    assert np.array_equal(y_pool, y_flat)
    assert junk == list(range(7))


def test_swap_roundtrip_is_identity_and_touches_nothing_else():
    pool = op.PoolModel(128, 12, 12)
    rs = synth.Stream(8, "swap")
    dev = pool.alloc(8)
    host = pool.alloc(6, host=True)
    for b in dev:
        pool.block(b)[:] = (rs.bits(128) & np.uint64(0xFF)).astype(np.uint8)
    before = {b: pool.block(b).copy() for b in dev}
    pool.swap_out([dev[1], dev[4], dev[6]], [host[5], host[0], host[2]])
    assert np.array_equal(pool.block(host[0], host=True), before[dev[4]])
    pool.swap_in([dev[0], dev[7], dev[3]], [host[5], host[0], host[2]])     # back into other blocks
    assert np.array_equal(pool.block(dev[0]), before[dev[1]])
    assert np.array_equal(pool.block(dev[7]), before[dev[4]])
    assert np.array_equal(pool.block(dev[3]), before[dev[6]])
    for b in (dev[1], dev[2], dev[4], dev[5], dev[6]):
        assert np.array_equal(pool.block(b), before[b])
    with pytest.raises(op.PoolError) as e:
        pool.swap_out([dev[0], 11], [host[0], host[1]])                     # 11 was never allocated
    assert e.value.code == op.EBADID
    assert np.array_equal(pool.block(host[0], host=True), before[dev[4]])   # and nothing was copied


def test_bf16_storage_rounding():
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: nearest even keeps 1.0; 1 + 3*2^-8 rounds up to 1 + 2^-6
    x = np.array([1.0, 1.0 + 2.0**-8, 1.0 + 3 * 2.0**-8, -2.5, 3.140625])
    bits = op.f64_to_bf16_bits(x)
    assert bits.tolist() == [0x3F80, 0x3F80, 0x3F82, 0xC020, 0x4049]
    assert op.bf16_bits_to_f64(bits).tolist() == [1.0, 1.0, 1.015625, -2.5, 3.140625]
    assert np.array_equal(bits, synth.bf16_bits(x.astype(np.float32)))


def test_layer_step_reduces_to_plain_attention_without_lora():
    wl = synth.make_workload("tiny", n_req=2, len_range=(0, 6),
                             shape=synth.LayerShape(16, 2, 2, head_dim=8, block_tokens=4), rank=2)
    s = wl.shape
    pool = op.PoolModel(s.block_bytes, 16, 0)
    tables = [pool.alloc(2), pool.alloc(2)]
    seg, ids = wl.segments()
    yb = {m: wl.y_base(m) for m in "qkvo"}
    zero = {m: {a: (wl.adapter(a, m)[0], 0 * wl.adapter(a, m)[1]) for a in (0, 1)} for m in "qkvo"}
    res = attention_layer_step(pool, wl.x(), yb, zero, seg, ids, wl.req_indptr, tables, wl.prefix_lens,
                               wl.new_lens, 2, 2, 8, 2.0, 0.35)
    for i in range(2):
        rows = slice(6 * i, 6 * i + 6)
        want = attend_request(yb["q"][rows].reshape(6, 2, 8), yb["k"][rows].reshape(6, 2, 8),
                              yb["v"][rows].reshape(6, 2, 8), 0, 0.35)
        np.testing.assert_allclose(res["attn"][rows], want, rtol=0, atol=2.0**-7 * np.abs(want).max())
    assert np.array_equal(res["o"], yb["o"].astype(np.float64))
