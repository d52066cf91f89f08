"""Host-side logic of the multi-GPU benchmark run on CPU: two gloo ranks draw their own batches of one
shape and combine their timings as the maximum over ranks and their tokens as the sum (there is no
exchange on the data path: replicas only)."""
import os
import sys

import numpy as np
import pytest

torch = pytest.importorskip("torch")
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2505_03756_b200 import synth
    base = synth.make_workload("prefill7b", n_req=6)
    wl = bench.rank_workload("prefill7b", base.seed, rank, n_req=6)
    times, tokens = bench.reduce_over_ranks([10.0 + rank, 3.0 - rank], wl.n_tokens, world, torch.device("cpu"))
    out.put((rank, times, tokens, wl.n_tokens, wl.shape.hidden, wl.n_req, int(wl.new_lens.sum()), wl.lora_of_req.tolist()))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_reduce_and_draw_independent_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, t0, n0, own0, h0, q0, _, l0), (r1, t1, n1, own1, h1, q1, _, l1) = res
    assert t0 == t1 == [11.0, 3.0]                 # maximum over ranks of each time
    assert n0 == n1 == own0 + own1                 # tokens of the whole job
    assert (h0, q0) == (h1, q1)                    # same layer shape and request count on every rank
    assert own0 != own1 or l0 != l1                # but each rank drew its own batch
