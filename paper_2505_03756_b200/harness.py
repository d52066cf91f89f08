"""Drives libfastpool for one synthetic workload: builds the pool, loads adapters from host blocks,
lays out the batch's KV block tables and runs the calls of one layer step.

Everything that computes runs inside the library (binding.py); this module only allocates device
memory with torch, uploads index arrays and sequences the calls.  Every allocator call is recorded
in `trace` so that a test can replay it on an independent allocator model.
"""
from __future__ import annotations

import math

import numpy as np
import torch

from . import binding as fl
from . import synth


def bits_to_dev(bits: np.ndarray, device) -> torch.Tensor:
    """uint16 bf16 bit patterns -> torch.bfloat16 CUDA tensor of the same shape."""
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).to(device)
    return t.view(torch.bfloat16)


def f32_to_dev(x: np.ndarray, device) -> torch.Tensor:
    """float32 array of bf16-representable values -> torch.bfloat16 CUDA tensor."""
    return bits_to_dev(synth.bf16_bits(x), device)


def dev_to_f32(t: torch.Tensor) -> np.ndarray:
    return t.detach().float().cpu().numpy()


class Session:
    def __init__(self, wl: synth.Workload, device: int = 0, scramble: bool = True, extra_host_blocks: int = 0,
                 adapters=None, register_all: bool = False):
        """adapters: ids to load (default: the ones the batch uses).  register_all: every adapter of the
        workload is packed, swapped in and registered; those the batch never touches get filler weights
        (one shared noise pattern), since drawing a thousand adapters value by value takes minutes."""
        self.wl = wl
        self.shape = wl.shape
        self.dev = torch.device("cuda", device)
        torch.cuda.set_device(self.dev)
        self.mats = [(i, o) for _, i, o in wl.shape.mats]
        self.mat_index = {n: k for k, (n, _, _) in enumerate(wl.shape.mats)}
        self.block_bytes = wl.shape.block_bytes
        self.bt = wl.shape.block_tokens
        self.adapter_ids = wl.used_adapters() if adapters is None else list(adapters)
        self.filler_ids = set()
        if register_all:
            self.filler_ids = set(range(len(wl.ranks))) - set(self.adapter_ids)
            self.adapter_ids = list(range(len(wl.ranks)))
        self.n_table = {a: fl.fl_lora_blocks(self.block_bytes, int(wl.ranks[a]), self.mats) for a in self.adapter_ids}
        self.n_host_blocks = sum(self.n_table.values()) + extra_host_blocks
        self.pool = fl.fl_pool_create(self.block_bytes, wl.pool_blocks, max(1, self.n_host_blocks), device)
        self.trace = []
        if scramble:
            # fragment the pool: take every block, give them back in a seeded random order
            ids = self.alloc(wl.pool_blocks)
            perm = synth.Stream(wl.seed, "scramble").permutation(wl.pool_blocks)
            self.free(ids[perm])
        self.lora_tables = {}
        self.lora_host_tables = {}
        self.kv_tables = None
        self._ws = {}

    # ---- allocator calls, recorded
    def alloc(self, n, host=False):
        ids = (fl.fl_host_block_alloc if host else fl.fl_block_alloc)(self.pool, n)
        self.trace.append(("alloc", host, n, ids.copy()))
        return ids

    def free(self, ids, host=False):
        (fl.fl_host_block_free if host else fl.fl_block_free)(self.pool, ids)
        self.trace.append(("free", host, len(ids), np.array(ids, dtype=np.uint32)))

    def close(self):
        if self.pool is not None:
            torch.cuda.synchronize()
            fl.fl_pool_destroy(self.pool)
            self.pool = None

    # ---- adapters: pack into host blocks, swap in, register
    def load_adapters(self, stream=None):
        side = stream or torch.cuda.Stream()
        for a in self.adapter_ids:
            rank = int(self.wl.ranks[a])
            A, B = [], []
            for name, d_in, d_out in self.shape.mats:
                if a in self.filler_ids:
                    A.append(self._filler(d_in * rank).reshape(d_in, rank))
                    B.append(self._filler(rank * d_out).reshape(rank, d_out))
                    continue
                am, bm = self.wl.adapter(a, name)
                A.append(synth.bf16_bits(am))
                B.append(synth.bf16_bits(bm))
            host_tab = self.alloc(self.n_table[a], host=True)
            fl.fl_lora_pack_host(self.pool, rank, self.mats, A, B, host_tab)
            dev_tab = self.alloc(self.n_table[a])
            fl.fl_swap_in(self.pool, dev_tab, host_tab, side)
            self.lora_tables[a] = dev_tab
            self.lora_host_tables[a] = host_tab
        side.synchronize()
        for a in self.adapter_ids:
            fl.fl_lora_register(self.pool, a, int(self.wl.ranks[a]), self.mats, self.lora_tables[a])

    def _filler(self, n):
        if getattr(self, "_filler_bits", None) is None or len(self._filler_bits) < n:
            self._filler_bits = synth.bf16_bits(synth.Stream(self.wl.seed, "filler").normal((max(n, 1 << 20),), self.wl.weight_std))
        return self._filler_bits[:n]

    # ---- batch index arrays and KV tables
    def build_batch(self):
        wl = self.wl
        self.kv_tables = [self.alloc(int(-(-(int(p) + int(n)) // self.bt))) for p, n in zip(wl.prefix_lens, wl.new_lens)]
        tbl_indptr = np.concatenate([[0], np.cumsum([len(t) for t in self.kv_tables])]).astype(np.int32)
        tbl = np.concatenate(self.kv_tables).astype(np.uint32) if self.kv_tables else np.zeros(0, np.uint32)
        seg_indptr, seg_lora = wl.segments()
        d = self.dev
        self.n_tbl = int(tbl_indptr[-1])
        self.t_tbl_indptr = torch.from_numpy(tbl_indptr).to(d)
        self.t_tbl = torch.from_numpy(tbl.view(np.int32)).to(d)
        self.t_req_indptr = torch.from_numpy(wl.req_indptr).to(d)
        self.t_prefix = torch.from_numpy(wl.prefix_lens.astype(np.int32)).to(d)
        self.t_new = torch.from_numpy(wl.new_lens.astype(np.int32)).to(d)
        self.t_seg_indptr = torch.from_numpy(seg_indptr).to(d)
        self.t_seg_lora = torch.from_numpy(seg_lora).to(d)
        self.n_seg = len(seg_lora)

    def fill_prefix_kv(self):
        """Writes every request's cached prefix K,V (rows of the noise bank) into its blocks."""
        wl, s = self.wl, self.shape
        total = int(wl.prefix_lens.sum())
        if total == 0:
            return
        req = np.repeat(np.arange(wl.n_req, dtype=np.int64), wl.prefix_lens)
        pos = np.concatenate([np.arange(int(p), dtype=np.int64) for p in wl.prefix_lens])
        bank = f32_to_dev(synth.kv_bank(wl.seed, s), self.dev)
        ik = torch.from_numpy(synth.kv_bank_index(req, pos, 0)).to(self.dev)
        iv = torch.from_numpy(synth.kv_bank_index(req, pos, 1)).to(self.dev)
        indptr = torch.from_numpy(np.concatenate([[0], np.cumsum(wl.prefix_lens)]).astype(np.int32)).to(self.dev)
        zeros = torch.zeros(wl.n_req, dtype=torch.int32, device=self.dev)
        step = 1 << 17          # tokens per call, bounds the temporaries
        # one call per slice of whole requests
        r0 = 0
        cum = np.concatenate([[0], np.cumsum(wl.prefix_lens)])
        while r0 < wl.n_req:
            r1 = r0 + 1
            while r1 < wl.n_req and cum[r1 + 1] - cum[r0] <= step:
                r1 += 1
            lo, hi = int(cum[r0]), int(cum[r1])
            k = bank[ik[lo:hi]].contiguous()
            v = bank[iv[lo:hi]].contiguous()
            ind = (indptr[r0:r1 + 1] - lo).contiguous()
            fl.fl_kv_append(self.pool, k, v, ind, self.t_tbl_indptr[r0:r1 + 1].contiguous(), self.t_tbl,
                            zeros[r0:r1], r1 - r0, hi - lo, s.n_kv_heads)
            torch.cuda.synchronize()
            del k, v
            r0 = r1

    # ---- the calls of a layer step
    def workspace(self, key, nbytes):
        t = self._ws.get(key)
        if t is None or t.numel() < nbytes:
            t = torch.empty(int(nbytes), dtype=torch.uint8, device=self.dev)
            self._ws[key] = t
        return t

    def sgmv(self, ys, x, mats, scale=None, stream=None):
        """ys[j] += scale * (x A) B for projections `mats` (names) sharing x."""
        T = self.wl.n_tokens
        ws = self.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, len(mats)))
        scale = self.wl.scale if scale is None else scale
        if len(mats) == 1:
            fl.fl_lora_sgmv(self.pool, ys[0], x, self.mat_index[mats[0]], self.t_seg_indptr, self.t_seg_lora,
                            self.n_seg, T, scale, ws, stream)
        else:
            fl.fl_lora_sgmv_multi(self.pool, ys, x, [self.mat_index[m] for m in mats], self.t_seg_indptr,
                                  self.t_seg_lora, self.n_seg, T, scale, ws, stream)

    def lora_linear(self, ys, x, ws, mats, scale=None, stream=None):
        """ys[j] = x ws[j] + scale * (x A) B for projections `mats` (names) sharing x; ys are overwritten."""
        T = self.wl.n_tokens
        wsp = self.workspace("linear", fl.fl_lora_linear_workspace(T, len(mats)))
        scale = self.wl.scale if scale is None else scale
        fl.fl_lora_linear_multi(self.pool, ys, x, ws, [self.mat_index[m] for m in mats], self.t_seg_indptr,
                                self.t_seg_lora, self.n_seg, T, scale, wsp, stream)

    def lora_linear_qkv_append(self, y_q, x, w_q, w_k, w_v, scale=None, stream=None):
        """q = x W_q + LoRA term into y_q; k, v = x W + LoRA term straight into the batch's pool blocks."""
        T, s = self.wl.n_tokens, self.shape
        wsp = self.workspace("linear", fl.fl_lora_linear_workspace(T, 3))
        scale = self.wl.scale if scale is None else scale
        tmp_k = tmp_v = None
        if T <= 16 * self.n_seg:           # short segments: the library forms x W in scratch rows first
            tmp = self.workspace("linear_kv", 2 * T * s.n_kv_heads * s.head_dim * 2)
            half = T * s.n_kv_heads * s.head_dim * 2
            tmp_k, tmp_v = tmp[:half], tmp[half:2 * half]
        fl.fl_lora_linear_qkv_append(self.pool, y_q, x, w_q, w_k, w_v, self.mat_index["q"], self.mat_index["k"],
                                     self.mat_index["v"], self.t_seg_indptr, self.t_seg_lora, self.n_seg, T, scale,
                                     self.t_req_indptr, self.t_tbl_indptr, self.t_tbl, self.t_prefix, self.wl.n_req,
                                     s.n_kv_heads, tmp_k, tmp_v, wsp, stream)

    def sgmv_qkv_append(self, y_q, y_k, y_v, x, scale=None, stream=None):
        """q += LoRA term in place; base k, v + LoRA term written straight into the batch's pool blocks."""
        T = self.wl.n_tokens
        ws = self.workspace("sgmv", fl.fl_lora_sgmv_workspace(T, 3))
        scale = self.wl.scale if scale is None else scale
        fl.fl_lora_sgmv_qkv_append(self.pool, y_q, y_k, y_v, x, self.mat_index["q"], self.mat_index["k"],
                                   self.mat_index["v"], self.t_seg_indptr, self.t_seg_lora, self.n_seg, T, scale,
                                   self.t_req_indptr, self.t_tbl_indptr, self.t_tbl, self.t_prefix, self.wl.n_req,
                                   self.shape.n_kv_heads, ws, stream)

    def kv_append(self, k_new, v_new, stream=None):
        fl.fl_kv_append(self.pool, k_new, v_new, self.t_req_indptr, self.t_tbl_indptr, self.t_tbl, self.t_prefix,
                        self.wl.n_req, self.wl.n_tokens, self.shape.n_kv_heads, stream)

    def attention(self, out, q, sm_scale=None, stream=None):
        s, wl = self.shape, self.wl
        ws = self.workspace("attn", fl.fl_paged_attention_workspace(wl.n_req, wl.n_tokens, self.n_tbl, s.n_q_heads,
                                                                    s.n_kv_heads))
        sm_scale = 1.0 / math.sqrt(s.head_dim) if sm_scale is None else sm_scale
        fl.fl_paged_attention(self.pool, out, q, self.t_req_indptr, self.t_tbl_indptr, self.t_tbl, self.t_prefix,
                              self.t_new, wl.n_req, wl.n_tokens, self.n_tbl, s.n_q_heads, s.n_kv_heads, sm_scale, ws,
                              stream)

    def status(self, clear=False):
        return fl.fl_pool_status(self.pool, clear)
