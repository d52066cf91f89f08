#!/usr/bin/env python
"""Benchmark of the multi-LoRA layer step over the unified block pool.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload all|prefill7b|...] [--impl ours|reference]

One step = one pass of the whole hot path over one synthetic batch: block alloc/free for the batch's
new-token blocks, LoRA q/k/v projection (SGMV) with the new K, V written into their pool blocks (one fused call,
or projection and KV append as two calls with --separate-append), paged attention over [cached prefix ||
new tokens], LoRA o projection (plus up/down when the layer has them), and a block swap-out/swap-in
on a side stream that overlaps the kernels.  By default the four full-size workloads run one after the other in
one invocation; the JSON line (rank 0) carries the headline workload's numbers at the top level and one record per
workload under "workloads".  Each record also times the layer with the base projections on the path
(fl_lora_linear: y = x W + s (x A) B in one GEMM), which is what the end-to-end leg runs: x goes up, the layer's
output comes back.
"""
import argparse
import json
import math
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "multi-LoRA layer tokens/s (prefill, decode) on 1 B200; % of HBM/tensor roofline"
WORKLOAD_TEXT = {
    "tiny": "configs[0] tiny reference layer",
    "prefill7b": "configs[1] Llama-2-7B-shaped prefill: 64 requests, 32 adapters rank 16 Zipf(1.0), lengths U{128..1024}, half cached",
    "decode13b": "configs[2] Llama-2-13B-shaped decode: 256 requests x 1 token, 128 adapters rank 32 Zipf(0.8), contexts U{512..4096}",
    "gqa34b": "configs[3] 34B-class GQA prefill: 16 requests x (3072 cached + 1024 new), 64q/8kv heads, rank 64, 60 GB pool",
    "swapstress": "configs[4] swap-stress mixed step: 1000 adapters ranks {8..64}, 64 mixed requests Zipf(1.2), 256 blocks swapped each way per step",
}


def source_digest():
    """sha256 over the CUDA sources: the ncu figures under profiles/ only describe the kernels they were taken from."""
    import hashlib
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2505_03756_b200", "csrc")
    for f in sorted(os.listdir(csrc)):
        if f.endswith((".cu", ".cuh")):
            h.update(f.encode())
            h.update(open(os.path.join(csrc, f), "rb").read())
    return h.hexdigest()[:16]


def ncu_traffic(workload, call):
    """dram__bytes_read.sum + dram__bytes_write.sum per launch of a call's kernels, from the ncu capture summarised in
    profiles/ncu_traffic.json (bytes), or None when there is no capture or the sources have changed since."""
    p = os.path.join(ROOT, "profiles", "ncu_traffic.json")
    if not os.path.exists(p):
        return None
    d = json.load(open(p))
    e = d.get("captures", {}).get(f"{workload}/{call}")
    if not e or e.get("source_digest") != source_digest():
        return None
    return e["dram_bytes_per_launch"]


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return {"hbm": d["hbm_gbs"], "tensor": d["bf16_tflops"], "tensor_sustained": d.get("bf16_tflops_sustained"),
                "src": "measured"}
    return {"hbm": 6650.0, "tensor": 1590.0, "tensor_sustained": 1400.0, "src": "fallback"}


# ------------------------------------------------------------------ algorithmic work of each call
def work_model(wl):
    s = wl.shape
    T = wl.n_tokens
    d = s.head_dim
    distinct = wl.used_adapters()
    dims = {n: (i, o) for n, i, o in s.mats}

    def sgmv_bytes(mats):
        b = 2 * T * dims[mats[0]][0]                                    # x read once
        for m in mats:
            b += 4 * T * dims[m][1]                                     # y read + write
            b += sum(2 * int(wl.ranks[a]) * (dims[m][0] + dims[m][1]) for a in distinct)
        return b

    n, p = wl.new_lens.astype(np.float64), wl.prefix_lens.astype(np.float64)
    attn_flops = 4.0 * d * s.n_q_heads * float(np.sum(n * p + n * (n + 1) / 2))
    attn_bytes = 2 * (2 * T * s.n_q_heads * d) + float(np.sum(p + n)) * 2 * s.n_kv_heads * d * 2
    w = {
        "sgmv_qkv": {"bytes": sgmv_bytes(["q", "k", "v"]), "bound": "hbm"},
        # k, v: base rows read from y, result rows written into pool blocks: the same byte count as updating y in place
        "sgmv_qkv_append": {"bytes": sgmv_bytes(["q", "k", "v"]), "bound": "hbm"},
        "kv_append": {"bytes": 2 * 2 * T * s.n_kv_heads * d * 2, "bound": "hbm"},
        "attention": {"bytes": attn_bytes, "flops": attn_flops,
                      "bound": "tensor" if attn_flops / attn_bytes > 200 else "hbm"},
        "sgmv_o": {"bytes": sgmv_bytes(["o"]), "bound": "hbm"},
    }
    if s.inter:
        w["sgmv_up"] = {"bytes": sgmv_bytes(["up"]), "bound": "hbm"}
        w["sgmv_down"] = {"bytes": sgmv_bytes(["down"]), "bound": "hbm"}
    return w


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs."""

    def __init__(self, index):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.stop_flag, self.max_mhz = index, [], set(), False, None
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def run(self):
        if self.nv is None:
            return
        nv = self.nv
        names = {nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap", nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
                 nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
                 nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown"}
        while not self.stop_flag:
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for bit, name in names.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.01)

    def result(self):
        self.stop_flag = True
        if self.nv is not None and not self.samples:      # a timed region shorter than one sampling period
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            except Exception:
                pass
        if self.nv is None or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "note": "NVML unavailable"}
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------ the oracle leg (host cores)
def oracle_step_sample(wl, n_req_sample):
    """Runs the oracle's layer step on the first n_req_sample requests of the batch; returns (seconds, tokens)."""
    from oracle.attention import attend_request
    from oracle.lora import lora_project
    s = wl.shape
    rq = wl.req_indptr
    T = int(rq[n_req_sample])
    seg, ids = wl.segments()
    keep = [k for k in range(len(ids)) if seg[k] < T]
    seg_s = np.array([min(int(seg[k]), T) for k in keep] + [T], dtype=np.int32)
    ids_s = ids[keep]
    x = wl.x("q")[:T]
    groups = [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if s.inter else [])
    yb = {m: wl.y_base(m)[:T] for g in groups for m in g}
    ad = {m: {a: wl.adapter(a, m) for a in set(int(i) for i in ids_s)} for g in groups for m in g}
    ctx = [wl.kv_prefix(i) for i in range(n_req_sample)]
    q = wl.q()[:T]
    kn, vn = wl.kv_new()
    xin = {m: (x if m in ("q", "k", "v", "up") else wl.x(m)[:T]) for g in groups for m in g}
    t0 = time.perf_counter()
    for g in groups:
        for m in g:
            lora_project(yb[m], xin[m], seg_s, ids_s, ad[m], wl.scale)
    for i in range(n_req_sample):
        lo, hi = int(rq[i]), int(rq[i + 1])
        k = np.concatenate([ctx[i][0], kn[lo:hi]])
        v = np.concatenate([ctx[i][1], vn[lo:hi]])
        attend_request(q[lo:hi], k, v, int(wl.prefix_lens[i]), 1.0 / math.sqrt(s.head_dim))
    return time.perf_counter() - t0, T


def oracle_baseline(wl, budget_s=12.0):
    try:
        from threadpoolctl import threadpool_info
        cores = max([i.get("num_threads", 1) for i in threadpool_info()] + [1])
    except Exception:
        cores = os.cpu_count()
    n = min(2, wl.n_req)
    dt, tok = oracle_step_sample(wl, n)
    per_req = dt / n
    n2 = int(max(n, min(wl.n_req, budget_s / max(per_req, 1e-6))))
    if n2 > n:
        dt, tok = oracle_step_sample(wl, n2)
        n = n2
    return {"value": tok / dt, "unit": "tokens/s", "cores": int(cores), "kind": "oracle",
            "sample": f"first {n} of {wl.n_req} requests ({tok} of {wl.n_tokens} new tokens), whole layer step in "
                      f"fp64 numpy, {dt:.2f} s"}, dt, tok


def run_reference(args, wl, name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    vals = []
    for _ in range(args.warmup + args.steps):
        cb, dt, tok = oracle_baseline(wl, budget_s=max(1.0, 60.0 / max(1, args.warmup + args.steps)))
        vals.append((dt, tok, cb))
    timed = vals[args.warmup:]
    tot_t = sum(v[0] for v in timed)
    tot_tok = sum(v[1] for v in timed)
    value = tot_tok / tot_t
    cb = dict(timed[-1][2])
    cb["value"] = value
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": "tokens/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * tot_t / len(timed), "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_TEXT[name], "note": "CPU oracle on host cores, bounded sample per step"},
        "cpu_baseline": cb,
        "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))


def rank_workload(name, base_seed, rank, n_req=0):
    """Requests are independent, so rank r runs its own batch of the same shape, drawn from its own seed."""
    from paper_2505_03756_b200 import synth
    kw = {"n_req": n_req} if n_req else {}
    if rank == 0:
        return synth.make_workload(name, **kw)
    return synth.make_workload(name, seed=base_seed + 7919 * rank, **kw)


def reduce_over_ranks(times_ms, tokens, world, device):
    """Job-level numbers from per-rank ones: every time is the maximum over ranks, tokens are summed."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(times_ms), dtype=torch.float64, device=device)
    n = torch.tensor([tokens], dtype=torch.int64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return [float(v) for v in t], int(n[0])


# ------------------------------------------------------------------ the CUDA leg
FULL_SET = ["prefill7b", "decode13b", "gqa34b", "swapstress"]


def bench_workload(args, name, world, rank, local, oracle_budget_s):
    """All measurements of one workload on this rank's GPU; returns its record (rank 0) after reducing over ranks."""
    import torch
    import torch.distributed as dist
    from paper_2505_03756_b200 import binding as fl, harness as H, synth

    base = synth.make_workload(name, n_req=args.n_req) if args.n_req else synth.make_workload(name)
    wl = rank_workload(name, base.seed, rank, args.n_req)   # no exchange between ranks
    s = wl.shape
    T = wl.n_tokens
    n_swap = args.swap_blocks if args.swap_blocks >= 0 else (256 if name == "swapstress" else 32)
    sess = H.Session(wl, device=local, extra_host_blocks=2 * n_swap, register_all=(name == "swapstress"))
    if args.prefill_kernel >= 0:
        fl.fl_pool_set_option(sess.pool, fl.FL_OPT_PREFILL_KERNEL, args.prefill_kernel)
    sess.load_adapters()
    # the new-token blocks are taken and returned every step (allocator on the path); tables stay put
    sess.build_batch()
    sess.fill_prefix_kv()
    dev = sess.dev
    groups = [["q", "k", "v"], ["o"]] + ([["up"], ["down"]] if s.inter else [])
    names = [m for g in groups for m in g]
    dims = {n: (i, o) for n, i, o in s.mats}
    # host (pinned) copies of the step's inputs, device buffers
    h_x = torch.from_numpy(synth.bf16_bits(wl.x("q")).view(np.int16)).pin_memory()
    d_x = h_x.to(dev).view(torch.bfloat16)
    d_y = {m: H.f32_to_dev(wl.y_base(m), dev) for m in names}
    d_attn = torch.empty(T, s.n_q_heads, s.head_dim, dtype=torch.bfloat16, device=dev)
    h_out = torch.empty(T, s.hidden, dtype=torch.int16).pin_memory()
    # base weights of the layer (resident, drawn on the device), for the step with the projections on the path
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.seed % (1 << 31))
    d_w = {m: (torch.randn(dims[m][0], dims[m][1], generator=gen, device=dev, dtype=torch.float32) *
               dims[m][0] ** -0.5).to(torch.bfloat16) for m in names}
    d_z = {m: torch.empty(T, dims[m][1], dtype=torch.bfloat16, device=dev) for m in names}   # outputs of that step
    # swap sets: victims and targets disjoint from the batch's blocks
    swap_dev_out = sess.alloc(n_swap) if n_swap else np.zeros(0, np.uint32)
    swap_dev_in = sess.alloc(n_swap) if n_swap else np.zeros(0, np.uint32)
    swap_host_out = sess.alloc(n_swap, host=True) if n_swap else np.zeros(0, np.uint32)
    swap_host_in = sess.alloc(n_swap, host=True) if n_swap else np.zeros(0, np.uint32)
    spare = int(np.sum((wl.new_lens + s.block_tokens - 1) // s.block_tokens))
    spare = min(spare, fl.fl_pool_status(sess.pool)["blocks_free"])
    main = torch.cuda.Stream()
    side, side_in = torch.cuda.Stream(), torch.cuda.Stream()      # swap-out and swap-in overlap each other too
    ev_side, ev_side_in = torch.cuda.Event(), torch.cuda.Event()
    calls = (["sgmv_qkv", "kv_append"] if args.separate_append else ["sgmv_qkv_append"]) + ["attention", "sgmv_o"] + \
        (["sgmv_up", "sgmv_down"] if s.inter else [])
    # shrink + expand per SGMV call, KV append, plan + prefill + decode + merge, swap gather + scatter
    launches_per_step = 2 + (1 if args.separate_append else 0) + 4 + 2 + (4 if s.inter else 0) + \
        (2 * -(-n_swap // 256) if n_swap > 1 else 0)

    def compute(k, evs=None):
        """The kernels of one step, in order, on the compute stream."""
        sign = wl.scale if k % 2 == 0 else -wl.scale     # y += s*delta, then y -= s*delta: values stay bounded
        mark = (lambda: None) if evs is None else (lambda: evs.append(_rec(torch, main)))
        mark()
        if args.separate_append:
            sess.sgmv([d_y["q"], d_y["k"], d_y["v"]], d_x, ["q", "k", "v"], scale=sign, stream=main)
            mark()
            sess.kv_append(d_y["k"], d_y["v"], stream=main)
        else:       # a4 inside a3: the k, v projections write their rows straight into the pool blocks
            sess.sgmv_qkv_append(d_y["q"], d_y["k"], d_y["v"], d_x, scale=sign, stream=main)
        mark()
        sess.attention(d_attn, d_y["q"], stream=main)
        mark()
        sess.sgmv([d_y["o"]], d_attn.view(T, -1), ["o"], scale=sign, stream=main)
        mark()
        if s.inter:
            sess.sgmv([d_y["up"]], d_y["o"], ["up"], scale=sign, stream=main)
            mark()
            sess.sgmv([d_y["down"]], d_y["up"], ["down"], scale=sign, stream=main)
            mark()

    # the same layer with its base projections on the path: every projection is one GEMM that also takes the LoRA term
    fused_calls = ["linear_qkv_append", "attention", "linear_o"] + (["linear_up", "linear_down"] if s.inter else [])

    def fused_call(c):
        if c == "linear_qkv_append":      # q to d_z["q"], k and v straight into the requests' pool blocks
            sess.lora_linear_qkv_append(d_z["q"], d_x, d_w["q"], d_w["k"], d_w["v"], stream=main)
        elif c == "attention":
            sess.attention(d_attn, d_z["q"], stream=main)
        elif c == "linear_o":
            sess.lora_linear([d_z["o"]], d_attn.view(T, -1), [d_w["o"]], ["o"], stream=main)
        elif c == "linear_up":
            sess.lora_linear([d_z["up"]], d_z["o"], [d_w["up"]], ["up"], stream=main)
        elif c == "linear_down":
            sess.lora_linear([d_z["down"]], d_z["up"], [d_w["down"]], ["down"], stream=main)

    def fused_compute(evs=None):
        for c in fused_calls:
            if evs is not None:
                evs.append(_rec(torch, main))
            fused_call(c)
        if evs is not None:
            evs.append(_rec(torch, main))

    graphs = []          # the step's kernels captured once per sign; replayed when graph launches are on
    fused_graph = []

    def step(k, evs=None, swap=True, use_graph=False, fused=False):
        ids = fl.fl_block_alloc(sess.pool, spare)        # a1: the allocator runs every step
        fl.fl_block_free(sess.pool, ids[::-1])
        swap = swap and n_swap > 0
        if swap:                                          # a7: side streams, overlapped
            fl.fl_swap_out(sess.pool, swap_dev_out, swap_host_out, side)
            fl.fl_swap_in(sess.pool, swap_dev_in, swap_host_in, side_in)
        if fused:
            if use_graph and fused_graph:
                fused_graph[0].replay()
            else:
                fused_compute(evs)
        elif use_graph and graphs:
            graphs[k % 2].replay()
        else:
            compute(k, evs)
        if swap:
            ev_side.record(side)
            ev_side_in.record(side_in)
            main.wait_event(ev_side)
            main.wait_event(ev_side_in)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, n):
        barrier()
        t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t0.record(main)
        for k in range(n):
            fn(k)
        t1.record(main)
        barrier()
        return t0.elapsed_time(t1) / n

    with torch.cuda.stream(main):
        for k in range(args.warmup):
            step(k)
        barrier()
        launch_mode = "eager"
        if not args.no_graph:
            # the step's kernel launches go into CUDA graphs (one per sign): a step then costs one graph launch on
            # the host instead of one call into the library per kernel group
            try:
                for parity in range(2):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=main):
                        compute(parity)
                    graphs.append(g)
                for k in range(2):
                    step(k, use_graph=True)
                barrier()
                launch_mode = "cuda_graph"
            except Exception as exc:      # capture refused: time the eager launches and say so
                graphs.clear()
                launch_mode = "eager (graph capture failed: %s)" % type(exc).__name__
        sampler = ClockSampler(local)
        sampler.start()
        ms_step = timed(lambda k: step(k, use_graph=True), args.steps)
        clocks = sampler.result()
        # per-call device time: the same steps launched eagerly with an event between the calls
        def per_call(call_names, fused):
            evs = []
            barrier()
            for k in range(args.steps):
                step(k, evs, fused=fused)
            barrier()
            per = len(call_names) + 1
            out = {c: 0.0 for c in call_names}
            for k in range(args.steps):
                for j, c in enumerate(call_names):
                    out[c] += evs[k * per + j].elapsed_time(evs[k * per + j + 1])
            return {c: v / args.steps for c, v in out.items()}
        call_ms = per_call(calls, False)
        # every call by itself, ten launches back to back: its device time with the launch queue kept full (in
        # the step above a call of a few tens of microseconds is partly waiting for the host to issue it)
        def call_fn(c, k):
            sign = wl.scale if k % 2 == 0 else -wl.scale
            if c == "sgmv_qkv":
                sess.sgmv([d_y["q"], d_y["k"], d_y["v"]], d_x, ["q", "k", "v"], scale=sign, stream=main)
            elif c == "sgmv_qkv_append":
                sess.sgmv_qkv_append(d_y["q"], d_y["k"], d_y["v"], d_x, scale=sign, stream=main)
            elif c == "kv_append":
                sess.kv_append(d_y["k"], d_y["v"], stream=main)
            elif c == "attention":
                sess.attention(d_attn, d_y["q"], stream=main)
            elif c == "sgmv_o":
                sess.sgmv([d_y["o"]], d_attn.view(T, -1), ["o"], scale=sign, stream=main)
            elif c == "sgmv_up":
                sess.sgmv([d_y["up"]], d_y["o"], ["up"], scale=sign, stream=main)
            elif c == "sgmv_down":
                sess.sgmv([d_y["down"]], d_y["up"], ["down"], scale=sign, stream=main)
            else:
                fused_call(c)
        b2b_ms = {}
        for c in calls:
            for k in range(2):
                call_fn(c, k)
            b2b_ms[c] = timed(lambda k: call_fn(c, k), 10)
        # the same steps without the concurrent swap: how much of the swap the kernels hide
        overlap = None
        if n_swap:
            overlap = {"ms_per_step_without_swap": timed(lambda k: step(k, swap=False, use_graph=True), args.steps)}
        # the swap alone (both directions at once), and the host link's own peak for the same byte count
        swap = None
        if n_swap:
            def swap_once(_k):
                fl.fl_swap_out(sess.pool, swap_dev_out, swap_host_out, side)
                fl.fl_swap_in(sess.pool, swap_dev_in, swap_host_in, side_in)
                ev_side.record(side)
                ev_side_in.record(side_in)
                main.wait_event(ev_side)
                main.wait_event(ev_side_in)
            nbytes = n_swap * s.block_bytes
            lbytes = max(nbytes, 256 << 20)       # the link's peak is taken on copies large enough to reach it
            hp = torch.empty(2 * lbytes, dtype=torch.uint8).pin_memory()
            dp = torch.empty(2 * lbytes, dtype=torch.uint8, device=dev)

            def link_once(_k):
                with torch.cuda.stream(side):
                    hp[:lbytes].copy_(dp[:lbytes], non_blocking=True)
                with torch.cuda.stream(side_in):
                    dp[lbytes:].copy_(hp[lbytes:], non_blocking=True)
                ev_side.record(side)
                ev_side_in.record(side_in)
                main.wait_event(ev_side)
                main.wait_event(ev_side_in)
            res = {}
            for nm, fn in (("swap", swap_once), ("link", link_once)):
                fn(0)
                res[nm] = timed(fn, 5)
            del hp, dp
            gbs, peak = nbytes / res["swap"] / 1e6, lbytes / res["link"] / 1e6
            swap = {"ms": round(res["swap"], 4), "bytes_each_way": nbytes, "bound": "host link",
                    "gbs_each_way": round(gbs, 2), "link_peak_gbs_each_way": round(peak, 2), "frac_link": round(gbs / peak, 4),
                    "note": "both directions at once; peak = two contiguous pinned copies of %d MiB each, one per direction, "
                            "at once, measured here" % (lbytes >> 20)}
        # ---- the layer with its base projections on the path (after everything above: the GEMMs draw the most power,
        # and the numbers above should not inherit their clocks)
        for k in range(max(2, args.warmup // 2)):
            step(k, fused=True)
        barrier()
        if graphs:
            try:
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=main):
                    fused_compute()
                fused_graph.append(g)
                step(0, use_graph=True, fused=True)
                barrier()
            except Exception:
                fused_graph.clear()
        ms_fused = timed(lambda k: step(k, use_graph=True, fused=True), args.steps)
        fused_ms = per_call(fused_calls, True)
        for c in fused_calls:
            if c.startswith("linear"):
                b2b_ms[c] = timed(lambda k: fused_call(c), 10)

        # end to end: x starts in pinned host memory, the layer runs with its base projections, the output is read back
        def e2e_step(k):
            d_x.view(torch.int16).copy_(h_x, non_blocking=True)
            step(0, use_graph=True, fused=True)
            h_out.copy_(d_z["down" if s.inter else "o"].view(torch.int16), non_blocking=True)
        for k in range(2):
            e2e_step(k)
        ms_e2e_serial = timed(e2e_step, max(3, min(args.steps, 20)))

        # the same with consecutive steps pipelined, as a server would run them: while step k computes, the x of step k + 1
        # is on its way up and the output of step k - 1 on its way down (two staging buffers each way, three streams)
        up, down = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        out_t = d_z["down" if s.inter else "o"]
        st_in = [torch.empty_like(d_x) for _ in range(2)]
        st_out = [torch.empty_like(out_t) for _ in range(2)]
        pev = {n: [torch.cuda.Event() for _ in range(2)] for n in ("up", "in_free", "comp", "down")}

        def e2e_pipelined(k):
            b = k & 1
            if k >= 2:
                up.wait_event(pev["in_free"][b])
            with torch.cuda.stream(up):
                st_in[b].view(torch.int16).copy_(h_x, non_blocking=True)
                pev["up"][b].record(up)
            main.wait_event(pev["up"][b])
            d_x.copy_(st_in[b], non_blocking=True)
            pev["in_free"][b].record(main)
            step(0, use_graph=True, fused=True)
            if k >= 2:
                main.wait_event(pev["down"][b])
            st_out[b].copy_(out_t, non_blocking=True)
            pev["comp"][b].record(main)
            down.wait_event(pev["comp"][b])
            with torch.cuda.stream(down):
                h_out.copy_(st_out[b].view(torch.int16), non_blocking=True)
                pev["down"][b].record(down)

        def timed_pipeline(n):
            barrier()
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(main)
            for k in range(n):
                e2e_pipelined(k)
            for b in range(min(n, 2)):          # the last read-backs end the timed region
                main.wait_event(pev["down"][b])
            t1.record(main)
            barrier()
            return t0.elapsed_time(t1) / n
        timed_pipeline(3)
        ms_e2e = timed_pipeline(max(6, min(args.steps, 20)))
        del st_in, st_out
    st = sess.status()
    flags = st["device_flags"]
    (ms_step, ms_fused, ms_e2e, ms_e2e_serial), tokens_all = reduce_over_ranks([ms_step, ms_fused, ms_e2e, ms_e2e_serial], T, world, dev)
    rec = None
    if rank == 0:
        pk = peaks()
        wm = work_model(wl)
        kernels = {}
        for c in calls:
            w = wm[c]
            sec = call_ms[c] * 1e-3
            k = {"ms": round(call_ms[c], 4), "bound": w["bound"], "gbs": round(w["bytes"] / sec / 1e9, 1),
                 "frac_hbm": round(w["bytes"] / sec / 1e9 / pk["hbm"], 4)}
            k["ms_back_to_back"] = round(b2b_ms[c], 4)
            k["frac_hbm_back_to_back"] = round(w["bytes"] / (b2b_ms[c] * 1e-3) / 1e9 / pk["hbm"], 4)
            if "flops" in w:
                k["tflops"] = round(w["flops"] / sec / 1e12, 1)
                k["frac_tensor"] = round(w["flops"] / sec / 1e12 / pk["tensor"], 4)
                k["frac_tensor_back_to_back"] = round(w["flops"] / (b2b_ms[c] * 1e-3) / 1e12 / pk["tensor"], 4)
            k["algorithmic_bytes"] = int(w["bytes"])
            k["traffic"] = ncu_traffic(name, c) if not args.n_req else None
            kernels[c] = k
        if swap:
            kernels["swap"] = swap
            # 1 = the step with the swap costs no more than the longer of (step without swap, swap alone)
            overlap["ms_per_step_with_swap"] = ms_step
            overlap["efficiency"] = round(max(overlap["ms_per_step_without_swap"], swap["ms"]) / ms_step, 4)
            overlap["ms_per_step_without_swap"] = round(overlap["ms_per_step_without_swap"], 4)
        top = max(calls, key=lambda c: call_ms[c])
        w, sec = wm[top], call_ms[top] * 1e-3
        if w["bound"] == "tensor":
            ach, peak, unit = w["flops"] / sec / 1e12, pk["tensor"], "TFLOP/s"
        else:
            ach, peak, unit = w["bytes"] / sec / 1e9, pk["hbm"], "GB/s"
        roof = {"kernel": top, "bound": w["bound"], "achieved": round(ach, 2), "peak": peak, "unit": unit,
                "frac": round(ach / peak, 4), "traffic": kernels[top]["traffic"],
                "algorithmic_bytes": int(w["bytes"]), "peak_source": pk["src"] + " (burst)",
                "ms_per_launch": round(call_ms[top], 4)}
        # the layer with its base projections: GEMM flops against the sustained bf16 peak (a step runs for milliseconds)
        fused = {"ms_per_step": round(ms_fused, 4), "tokens_per_s": tokens_all / (ms_fused * 1e-3), "calls": {}}
        sustained = pk["tensor_sustained"] or pk["tensor"]
        for c in fused_calls:
            e = {"ms": round(fused_ms[c], 4)}
            if c.startswith("linear"):
                mats = {"linear_qkv_append": ["q", "k", "v"], "linear_o": ["o"], "linear_up": ["up"], "linear_down": ["down"]}[c]
                fl_ = sum(2.0 * T * dims[m][0] * dims[m][1] for m in mats)
                by = 2 * T * dims[mats[0]][0] + sum(2 * T * dims[m][1] + 2 * dims[m][0] * dims[m][1] for m in mats)
                e.update({"ms_back_to_back": round(b2b_ms[c], 4), "gemm_flops": fl_,
                          "tflops": round(fl_ / (fused_ms[c] * 1e-3) / 1e12, 1),
                          "frac_tensor_sustained": round(fl_ / (fused_ms[c] * 1e-3) / 1e12 / sustained, 4),
                          "frac_tensor_sustained_back_to_back": round(fl_ / (b2b_ms[c] * 1e-3) / 1e12 / sustained, 4),
                          "algorithmic_bytes": int(by), "frac_hbm": round(by / (fused_ms[c] * 1e-3) / 1e9 / pk["hbm"], 4),
                          "bound": "tensor" if fl_ / by > 250 else "hbm"})
            fused["calls"][c] = e
        fused["note"] = "x W + s (x A) B per projection in one tcgen05 GEMM (y written once, no read-modify-write; K and V " \
                        "rows go from the accumulator straight into the pool blocks), attention; weights resident in HBM"
        cb, _, _ = oracle_baseline(wl, budget_s=oracle_budget_s)
        rec = {
            "value": tokens_all / (ms_step * 1e-3), "unit": "tokens/s", "ms_per_step": ms_step,
            "config": {"workload": WORKLOAD_TEXT[name], "new_tokens_per_step": T, "requests": wl.n_req,
                       "distinct_adapters": len(wl.used_adapters()), "pool_blocks": wl.pool_blocks,
                       "block_bytes": s.block_bytes, "swap_blocks_each_way": n_swap,
                       "staging_bytes_outside_the_slab": int(st["staging_bytes"]),
                       "l2": "inputs larger than L2 (x, y and KV exceed 126 MB); no flush between steps",
                       "parallelism": "independent batch per GPU, no collective"},
            "roofline": roof, "kernels": kernels, "swap_overlap": overlap, "with_base_projections": fused,
            "cpu_baseline": cb,
            "e2e": {"value": tokens_all / (ms_e2e * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": int(h_x.numel() * 2),
                    "d2h_bytes_per_step": int(h_out.numel() * 2), "ms_per_step": ms_e2e,
                    "ms_per_step_one_at_a_time": ms_e2e_serial,
                    "step": "layer with base projections (fl_lora_linear), x uploaded from pinned host memory, the layer's "
                            "output read back, every step; consecutive steps pipelined (upload of the next and read-back "
                            "of the previous overlap the kernels); one_at_a_time = upload, kernels, read-back in sequence"},
            "gpu_launches": launches_per_step * args.steps, "launch_mode": launch_mode, "clocks": clocks, "device_flags": flags,
        }
    sess.close()
    del d_w, d_z, d_y, d_x, d_attn
    torch.cuda.empty_cache()
    return rec


def run_ours(args):
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    names = FULL_SET if args.workload == "all" else [args.workload]
    head = args.headline if args.headline in names else names[0]
    recs = {}
    for name in names:
        recs[name] = bench_workload(args, name, world, rank, local, 12.0 if name == head else 5.0)
    if rank == 0:
        h = recs[head]
        out = {"metric": METRIC, "value": h["value"], "unit": "tokens/s", "n_gpus": world, "steps": args.steps,
               "warmup": args.warmup, "ms_per_step": h["ms_per_step"], "higher_is_better": True, "scaling": "weak",
               "vs_baseline": None, "dtype": "bf16", "data": "synthetic"}
        for k in ("config", "roofline", "kernels", "swap_overlap", "with_base_projections", "cpu_baseline", "e2e",
                  "gpu_launches", "launch_mode", "clocks", "device_flags"):
            out[k] = h[k]
        out["headline_workload"] = head
        out["headline_note"] = "configs[1], the configuration the throughput metric is quoted on; the other full-size " \
                               "workloads of the same run are under 'workloads' with the same fields"
        if len(names) > 1:
            out["workloads"] = {n: r for n, r in recs.items() if n != head}
            out["targets"] = {
                "decode_attention_frac_hbm": recs["decode13b"]["kernels"]["attention"]["frac_hbm"] if "decode13b" in recs else None,
                "prefill_attention_frac_tensor_gqa34b": recs["gqa34b"]["kernels"]["attention"].get("frac_tensor") if "gqa34b" in recs else None,
                "sgmv_frac_hbm_back_to_back": {n: {c: k["frac_hbm_back_to_back"] for c, k in r["kernels"].items() if c.startswith("sgmv")}
                                               for n, r in recs.items()},
                "swap_frac_link": {n: r["kernels"]["swap"]["frac_link"] for n, r in recs.items() if "swap" in r["kernels"]},
            }
        print(json.dumps(out))
    if world > 1:
        dist.destroy_process_group()


def _rec(torch, stream):
    e = torch.cuda.Event(enable_timing=True)
    e.record(stream)
    return e


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all", choices=["all"] + list(WORKLOAD_TEXT),
                    help="all = the four full-size workloads one after the other (the default), or one of them")
    ap.add_argument("--headline", default="prefill7b", choices=list(WORKLOAD_TEXT),
                    help="the workload whose numbers go to the top level of the JSON line")
    ap.add_argument("--swap-blocks", type=int, default=-1)
    ap.add_argument("--prefill-kernel", type=int, default=-1, help="FL_OPT_PREFILL_KERNEL value (default: the library's)")
    ap.add_argument("--separate-append", action="store_true", help="q/k/v projection and KV append as two calls "
                    "(default: one call whose k, v results go straight into the pool blocks)")
    ap.add_argument("--no-graph", action="store_true", help="launch every step eagerly instead of replaying CUDA graphs")
    ap.add_argument("--n-req", type=int, default=0, help="reduced copy of the workload with this many requests "
                    "(small pool; for profiler captures, not a bench line)")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.n_req:
        for k in WORKLOAD_TEXT:
            WORKLOAD_TEXT[k] += f" -- REDUCED to {args.n_req} requests"
    if args.impl == "reference":
        from paper_2505_03756_b200 import synth
        name = args.headline if args.workload == "all" else args.workload
        wl = synth.make_workload(name, n_req=args.n_req) if args.n_req else synth.make_workload(name)
        run_reference(args, wl, name)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
