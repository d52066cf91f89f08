"""The C-ABI library loads and exports every symbol the header declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2505_03756_b200 import build
    lib = ctypes.CDLL(build.build())
    header = open(os.path.join(ROOT, "include", "fastpool.h")).read()
    declared = set(re.findall(r"\b(fl_[a-z_0-9]+)\s*\(", header))
    assert len(declared) >= 20
    for name in sorted(declared):
        assert hasattr(lib, name), name
    from paper_2505_03756_b200 import binding
    assert set(binding.EXPORTS) == declared


def test_layout_arithmetic_matches_hand_counts():
    # fl_lora_blocks is pure host arithmetic: callable without a GPU
    from paper_2505_03756_b200 import binding as fl, synth
    gold = os.path.join(ROOT, "tests", "golden", "lora_blocks.txt")
    for line in open(gold):
        if line.startswith("#") or not line.strip():
            continue
        _, hidden, n_q, n_kv, inter, rank, blocks = line.split()
        shp = synth.LayerShape(int(hidden), int(n_q), int(n_kv), inter=int(inter))
        assert fl.fl_lora_blocks(shp.block_bytes, int(rank), [(i, o) for _, i, o in shp.mats]) == int(blocks)
    assert fl.fl_lora_sgmv_workspace(256, 3) >= 3 * 256 * 64 * 4
    assert fl.fl_paged_attention_workspace(4, 128, 16, 8, 8) > 0
