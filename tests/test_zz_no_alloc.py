"""fl_lora_sgmv_static: the LoRA projection for callers that cannot allocate device memory.

An engine that has handed all of its HBM to the block pool (or a plug-in that may not touch the engine's
memory budget) has no scratch buffer to give fl_lora_sgmv.  fl_lora_sgmv_static uses a fixed array inside
the library instead.  This test calls it through the C ABI twice in a row, with different inputs, and
compares each result with the CPU oracle and, bit for bit, with what fl_lora_sgmv gives on a caller-provided
workspace (both run the same kernels).  The second call runs on whatever the first left in the shared scratch,
so a result that depended on stale contents would show.  Free device memory is read before and after: the calls
must not change it.
The file sorts last so that a run that stops at the first failure has already run every other test.
"""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from paper_2505_03756_b200 import synth

from oracle.lora import lora_project

from _util import assert_close, oracle_adapters


def test_static_scratch_matches_workspace_variant_twice():
    assert torch.cuda.is_available(), "this test needs a GPU"
    from paper_2505_03756_b200 import binding as fl, harness as H
    cases = [synth.make_workload("prefill7b", n_req=7, len_range=(40, 330)),                  # long segments
             synth.make_workload("decode13b", n_req=24, len_range=(30, 700), n_adapters=12)]  # one token each
    for wl in cases:
        s = H.Session(wl)
        try:
            s.load_adapters()
            s.build_batch()
            T = wl.n_tokens
            ws = s.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, 1))
            seg, ids = wl.segments()
            bufs = {}
            for mat in ("q", "o"):                     # every buffer exists before free memory is first read
                y = H.f32_to_dev(wl.y_base(mat), s.dev)
                bufs[mat] = (H.f32_to_dev(wl.x(mat), s.dev), y, y.clone())
            fl.fl_lora_sgmv_static(s.pool, bufs["q"][2].clone(), bufs["q"][0], s.mat_index["q"], s.t_seg_indptr,
                                   s.t_seg_lora, s.n_seg, T, 0.0)      # the first call on a device looks up the array
            torch.cuda.synchronize()
            free_before = torch.cuda.mem_get_info()[0]
            for call, (mat, scale) in enumerate([("q", wl.scale), ("o", -0.75)]):      # two calls in a row
                tx, y_ref, y_new = bufs[mat]
                fl.fl_lora_sgmv(s.pool, y_ref, tx, s.mat_index[mat], s.t_seg_indptr, s.t_seg_lora, s.n_seg, T,
                                scale, ws)
                fl.fl_lora_sgmv_static(s.pool, y_new, tx, s.mat_index[mat], s.t_seg_indptr, s.t_seg_lora, s.n_seg,
                                       T, scale)
            torch.cuda.synchronize()
            assert torch.cuda.mem_get_info()[0] == free_before, "the calls changed the amount of free device memory"
            for call, (mat, scale) in enumerate([("q", wl.scale), ("o", -0.75)]):
                tx, y_ref, y_new = bufs[mat]
                ref, got = H.dev_to_f32(y_ref), H.dev_to_f32(y_new)
                assert not np.array_equal(ref, wl.y_base(mat)), "the projection changed nothing"
                assert np.array_equal(got, ref), f"{wl.name} call {call}: differs from fl_lora_sgmv"
                want = lora_project(wl.y_base(mat), wl.x(mat), seg, ids, oracle_adapters(wl, mat), scale)
                assert_close(got, want, f"{wl.name} static call {call}")
            assert s.status()["device_flags"] == 0
        finally:
            s.close()


def test_static_scratch_rejects_oversized_batches():
    assert torch.cuda.is_available(), "this test needs a GPU"
    from paper_2505_03756_b200 import binding as fl
    pool = fl.fl_pool_create(4096, 4, 1, 0)
    try:
        too_many = 32768                     # needs more than FL_SGMV_STATIC_BYTES of scratch
        assert fl.fl_lora_sgmv_workspace(too_many, 1) > fl.FL_SGMV_STATIC_BYTES
        assert fl.fl_lora_sgmv_workspace(too_many - 1, 1) <= fl.FL_SGMV_STATIC_BYTES
        dummy = torch.zeros(16, dtype=torch.int32, device="cuda")
        with pytest.raises(fl.FlError) as e:
            fl.fl_lora_sgmv_static(pool, dummy, dummy, 0, dummy, dummy, 1, too_many, 1.0)
        assert e.value.code == fl.FL_ENOMEM
        # an empty batch is a no-op whatever its other arguments say, as in fl_lora_sgmv
        fl.fl_lora_sgmv_static(pool, dummy, dummy, 0, dummy, dummy, 0, too_many, 1.0)
    finally:
        fl.fl_pool_destroy(pool)
