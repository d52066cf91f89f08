"""Asynchronous swap-in (Section 4.3): queries whose blocks are still in flight wait while the ready ones run.
Two of four requests have their KV blocks in host memory; the swap-in is enqueued on a side stream behind a
bounded delay, the library reports exactly the other two as ready (same answer as the oracle's model), their
attention runs and matches the oracle while the copies are still pending, and after the event the whole batch
runs and matches."""
import math

import numpy as np
import pytest

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu

from oracle.attention import attend_request
from oracle.ready import InFlight
from paper_2505_03756_b200 import synth

from _util import assert_close, oracle_context


def test_ready_requests_run_while_the_others_wait_for_their_blocks():
    assert torch.cuda.is_available(), "this test needs a GPU"
    from paper_2505_03756_b200 import binding as fl, harness as H
    wl = synth.make_workload("tiny")
    s = H.Session(wl, adapters=[], extra_host_blocks=64)
    try:
        sh = s.shape
        s.build_batch()
        s.fill_prefix_kv()
        k_new, v_new = wl.kv_new()
        q = wl.q()
        s.kv_append(H.f32_to_dev(k_new, s.dev), H.f32_to_dev(v_new, s.dev))
        torch.cuda.synchronize()
        scale = 1.0 / math.sqrt(128)
        want = []
        for i in range(wl.n_req):
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            k, v = oracle_context(wl, i, k_new, v_new)
            want.append(attend_request(q[lo:hi], k, v, int(wl.prefix_lens[i]), scale))

        t_q = H.f32_to_dev(q, s.dev)
        warm = torch.zeros(q.shape, dtype=torch.bfloat16, device=s.dev)
        s.attention(warm, t_q)                     # first call: one-time set-up stays out of the timed window below
        torch.cuda.synchronize()

        n_run = wl.n_req // 2                      # requests [0, n_run) stay resident, the rest go to host memory
        assert 0 < n_run < wl.n_req
        waiting = np.concatenate([s.kv_tables[i] for i in range(n_run, wl.n_req)]).astype(np.uint32)
        assert len(waiting) > 0
        host = s.alloc(len(waiting), host=True)
        side = torch.cuda.Stream()
        ev = torch.cuda.Event()
        fl.fl_swap_out(s.pool, waiting, host, side)
        fl.fl_swap_record(s.pool, ev, side)
        assert fl.fl_swap_wait(s.pool, ev, 20000) == fl.FL_OK
        for b in waiting:                           # the device copies are gone: NaN patterns in their place
            fl.fl_block_write(s.pool, int(b), np.full(s.block_bytes, 0xFF, dtype=np.uint8))

        model = InFlight()
        lists = [list(map(int, t)) for t in s.kv_tables]
        assert fl.fl_requests_ready(s.pool, lists).tolist() == model.ready(lists) == [True] * wl.n_req

        # swap-in behind a bounded delay (about a second of spinning on the side stream)
        khz = getattr(torch.cuda.get_device_properties(0), "clock_rate", 1_900_000)
        with torch.cuda.stream(side):
            torch.cuda._sleep(int(1.0 * khz * 1000))
        fl.fl_swap_in(s.pool, waiting, host, side)
        ev2 = torch.cuda.Event()
        fl.fl_swap_record(s.pool, ev2, side)
        fl.fl_inflight_mark(s.pool, waiting, ev2)
        model.mark(waiting, "swap-in")
        ready = fl.fl_requests_ready(s.pool, lists)
        assert ready.tolist() == model.ready(lists) == [i < n_run for i in range(wl.n_req)]
        assert fl.fl_inflight_count(s.pool) == model.count() == len(set(map(int, waiting)))

        # the ready requests run now, on the main stream
        n_tok = int(wl.req_indptr[n_run])
        n_tbl = int(s.t_tbl_indptr[n_run].item())
        out = torch.zeros((n_tok,) + tuple(q.shape[1:]), dtype=torch.bfloat16, device=s.dev)
        ws = s.workspace("attn", fl.fl_paged_attention_workspace(wl.n_req, wl.n_tokens, s.n_tbl, sh.n_q_heads, sh.n_kv_heads))
        fl.fl_paged_attention(s.pool, out, t_q[:n_tok].contiguous(), s.t_req_indptr[:n_run + 1].contiguous(),
                              s.t_tbl_indptr[:n_run + 1].contiguous(), s.t_tbl, s.t_prefix[:n_run].contiguous(),
                              s.t_new[:n_run].contiguous(), n_run, n_tok, n_tbl, sh.n_q_heads, sh.n_kv_heads, scale, ws)
        torch.cuda.current_stream().synchronize()
        still_pending = not ev2.query()
        got = H.dev_to_f32(out)
        for i in range(n_run):
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            assert_close(got[lo:hi], want[i], f"ready request {i}")
        assert still_pending, "the ready requests were meant to finish while the swap-in was still in flight"

        # the copies land: everybody is ready, and the whole batch matches the oracle
        assert fl.fl_swap_wait(s.pool, ev2, 20000) == fl.FL_OK
        model.complete("swap-in")
        assert fl.fl_requests_ready(s.pool, lists).tolist() == model.ready(lists) == [True] * wl.n_req
        assert fl.fl_inflight_count(s.pool) == model.count() == 0
        out_all = torch.zeros(q.shape, dtype=torch.bfloat16, device=s.dev)
        s.attention(out_all, t_q)
        torch.cuda.synchronize()
        got = H.dev_to_f32(out_all)
        for i in range(wl.n_req):
            lo, hi = int(wl.req_indptr[i]), int(wl.req_indptr[i + 1])
            assert_close(got[lo:hi], want[i], f"request {i} after its blocks arrived")
        assert s.status()["device_flags"] == 0

        # argument checks
        with pytest.raises(Exception):
            fl.fl_inflight_mark(s.pool, [wl.pool_blocks + 5], ev2)
        with pytest.raises(Exception):
            fl.fl_requests_ready(s.pool, [[wl.pool_blocks + 5]])
    finally:
        s.close()
