"""The seeded generator: determinism, bf16 representability, popularity sampling against Eq. 3."""
import os

import numpy as np

from oracle.demand import expected_distinct
from paper_2505_03756_b200 import synth

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def test_eq3_closed_forms():
    assert expected_distinct([0.2, 0.3, 0.5], 1) == 1.0
    n, bs = 16, 16
    assert abs(expected_distinct(np.full(n, 1 / n), bs) - n * (1 - (1 - 1 / n) ** bs)) < 1e-12
    assert abs(expected_distinct([1.0, 0.0], 5) - 1.0) < 1e-15


def test_eq3_golden_values_and_sampler():
    for line in open(os.path.join(GOLD, "eq3_expected_distinct.txt")):
        if line.startswith("#") or not line.strip():
            continue
        name, n, alpha, bs, want = line.split()
        p = synth.zipf_probs(int(n), float(alpha))
        assert abs(expected_distinct(p, int(bs)) - float(want)) < 0.006, line
        rs = synth.Stream(11, name)
        draws = rs.choice_p(p, int(bs) * 400).reshape(400, int(bs))
        mean = np.mean([len(set(r)) for r in draws])
        assert abs(mean - float(want)) < 0.05 * float(want), (line, mean)


def test_streams_are_deterministic_and_normal():
    a = synth.Stream(5, "x").normal((1000, 33))
    b = synth.Stream(5, "x").normal((1000, 33))
    assert np.array_equal(a, b)
    assert not np.array_equal(a, synth.Stream(6, "x").normal((1000, 33)))
    assert abs(a.mean()) < 0.02 and abs(a.std() - 1.0) < 0.02
    r = synth.round_bf16(a)
    assert np.array_equal(synth.bf16_to_f32(synth.bf16_bits(r)), r)
    assert np.max(np.abs(r - a) / np.abs(a)) <= 2.0**-8


def test_workload_shapes():
    wl = synth.make_workload("prefill7b")
    assert wl.n_req == 64 and wl.shape.block_bytes == 256 * 1024
    L = wl.prefix_lens + wl.new_lens
    assert L.min() >= 128 and L.max() <= 1024 and np.all(wl.prefix_lens % 16 == 0)
    assert np.all(wl.prefix_lens == (L // 2 // 16) * 16)
    assert np.all(np.diff(wl.lora_of_req) >= 0)
    seg, ids = wl.segments()
    assert seg[0] == 0 and seg[-1] == wl.n_tokens and len(set(ids.tolist())) == len(ids)
    wl = synth.make_workload("decode13b")
    assert wl.n_req == 256 and wl.n_tokens == 256 and wl.shape.block_bytes == 320 * 1024
    assert wl.prefix_lens.min() >= 512 and wl.prefix_lens.max() <= 4096
    wl = synth.make_workload("gqa34b")
    assert wl.pool_blocks == 915527 and wl.shape.block_bytes == 65536 and wl.n_tokens == 16384
    wl = synth.make_workload("swapstress")
    assert len(wl.ranks) == 1000 and set(wl.ranks.tolist()) == {8, 16, 32, 64}
    assert (wl.new_lens == 1).sum() == 32
    wl = synth.make_workload("tiny")
    assert wl.lora_of_req.tolist() == [0, 1, 2, 3] and wl.n_tokens == 128 and wl.shape.block_bytes == 65536
    k, v = wl.kv_prefix(2)
    assert k.shape == (32, 8, 128) and not np.array_equal(k, v)
