"""Seeded synthetic inputs for the multi-LoRA hot path.

This module only *draws inputs*: counter-based random numbers, bf16 rounding of the drawn
values, adapter popularity sampling and the batch shapes of the five workloads.  It holds none
of the method's arithmetic (no projection, no attention, no block layout, no allocator) and is
the one module that both the CPU oracle's tests and the CUDA path's tests may import.

Workload shapes follow the paper's evaluation setting: Llama-7B/13B/34B-shaped layers, adapters
with normally distributed weights and ranks up to 64 (Section 6.1), skewed adapter popularity
(Section 6.2, Section 6.6 "Skewed-x") and multi-turn prompts whose leading tokens hit cached
prefix KV (Section 2.1).  They stand in for the paper's datasets, which are not available.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np

BASE_SEED = 0x250503756000

_M64 = (1 << 64) - 1
_GOLD = np.uint64(0x9E3779B97F4A7C15)
_MIX1 = np.uint64(0xBF58476D1CE4E5B9)
_MIX2 = np.uint64(0x94D049BB133111EB)


def splitmix64(ctr: np.ndarray) -> np.ndarray:
    """splitmix64 finaliser applied to the counters `ctr` (uint64 array), value i = mix(ctr_i)."""
    with np.errstate(over="ignore"):
        z = ctr.astype(np.uint64) * _GOLD
        z = (z ^ (z >> np.uint64(30))) * _MIX1
        z = (z ^ (z >> np.uint64(27))) * _MIX2
        return z ^ (z >> np.uint64(31))


def _key(seed: int, name: str) -> int:
    k = seed & _M64
    for b in name.encode():
        k = int(splitmix64(np.array([(k ^ b) & _M64], dtype=np.uint64))[0])
    return k


class Stream:
    """A named, seeded, counter-based random stream (value i depends only on seed, name, i)."""

    def __init__(self, seed: int, name: str):
        self.key = _key(seed, name)
        self.pos = 0

    def bits(self, n: int) -> np.ndarray:
        ctr = (np.arange(self.pos, self.pos + n, dtype=np.uint64) + np.uint64(self.key))
        self.pos += n
        return splitmix64(ctr)

    def uniform(self, n: int) -> np.ndarray:
        """n doubles in (0, 1)."""
        return ((self.bits(n) >> np.uint64(11)).astype(np.float64) + 0.5) * (1.0 / (1 << 53))

    def normal(self, shape, std: float = 1.0) -> np.ndarray:
        """float32 normal draws (Box-Muller on pairs of uniforms)."""
        n = int(np.prod(shape))
        m = (n + 1) // 2
        out = np.empty(2 * m, dtype=np.float32)
        step = 1 << 22
        for s in range(0, m, step):
            e = min(m, s + step)
            u = self.uniform(2 * (e - s))
            r = np.sqrt(-2.0 * np.log(u[0::2]))
            t = (2.0 * np.pi) * u[1::2]
            out[2 * s:2 * e:2] = (r * np.cos(t) * std).astype(np.float32)
            out[2 * s + 1:2 * e:2] = (r * np.sin(t) * std).astype(np.float32)
        return out[:n].reshape(shape)

    def integers(self, lo: int, hi: int, n: int) -> np.ndarray:
        """n integers uniform in [lo, hi] inclusive."""
        return (lo + np.floor(self.uniform(n) * (hi - lo + 1))).astype(np.int64)

    def permutation(self, n: int) -> np.ndarray:
        return np.argsort(self.bits(n), kind="stable").astype(np.int64)

    def choice_p(self, p: np.ndarray, n: int) -> np.ndarray:
        """n indices drawn with probabilities p (inverse CDF)."""
        cdf = np.cumsum(p) / np.sum(p)
        return np.minimum(np.searchsorted(cdf, self.uniform(n), side="left"), len(p) - 1)


# ---------------------------------------------------------------- bf16 storage format helpers
def bf16_bits(f: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(f, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def round_bf16(f: np.ndarray) -> np.ndarray:
    """float32 values rounded to the nearest bf16-representable float32."""
    return bf16_to_f32(bf16_bits(f))


def zipf_probs(n: int, alpha: float) -> np.ndarray:
    """Popularity of adapter k (1-based) proportional to k**-alpha; alpha = 0 is uniform."""
    p = np.arange(1, n + 1, dtype=np.float64) ** (-alpha)
    return p / p.sum()


# ---------------------------------------------------------------- layer shapes
@dataclass(frozen=True)
class LayerShape:
    hidden: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int = 128
    inter: int = 0          # MLP intermediate size; 0 = LoRA on attention projections only
    block_tokens: int = 16

    @property
    def mats(self) -> Tuple[Tuple[str, int, int], ...]:
        """(name, d_in, d_out) of every projection that carries a LoRA branch, in fixed order."""
        h, dq, dkv = self.hidden, self.n_q_heads * self.head_dim, self.n_kv_heads * self.head_dim
        m = [("q", h, dq), ("k", h, dkv), ("v", h, dkv), ("o", dq, h)]
        if self.inter:
            m += [("up", h, self.inter), ("down", self.inter, h)]
        return tuple(m)

    @property
    def block_bytes(self) -> int:
        """One pool block = K and V of `block_tokens` tokens of one layer, bf16."""
        return self.block_tokens * 2 * self.n_kv_heads * self.head_dim * 2


@dataclass
class Workload:
    """One batch: which adapter each request uses and how many cached / new tokens it has.

    Requests are sorted by adapter so that each adapter's tokens form one contiguous segment.
    """
    name: str
    seed: int
    shape: LayerShape
    ranks: np.ndarray            # rank of every registered adapter
    scale: float
    lora_of_req: np.ndarray      # adapter id per request (ascending)
    prefix_lens: np.ndarray      # cached tokens per request
    new_lens: np.ndarray         # new tokens per request
    pool_blocks: int             # device pool size in blocks
    host_blocks: int = 0
    popularity: Optional[np.ndarray] = None
    weight_std: float = 0.02
    _cache: Dict = field(default_factory=dict, repr=False)

    # ---- derived index arrays
    @property
    def n_req(self) -> int:
        return len(self.lora_of_req)

    @property
    def n_tokens(self) -> int:
        return int(self.new_lens.sum())

    @property
    def req_indptr(self) -> np.ndarray:
        """Token offsets of each request inside the packed [T, ...] tensors."""
        return np.concatenate([[0], np.cumsum(self.new_lens)]).astype(np.int32)

    def segments(self) -> Tuple[np.ndarray, np.ndarray]:
        """(seg_indptr over tokens, lora id per segment): one segment per run of equal adapter."""
        ids, starts = [], []
        rp = self.req_indptr
        for i, a in enumerate(self.lora_of_req):
            if i == 0 or a != self.lora_of_req[i - 1]:
                ids.append(int(a))
                starts.append(int(rp[i]))
        return (np.array(starts + [int(rp[-1])], dtype=np.int32), np.array(ids, dtype=np.int32))

    def used_adapters(self) -> List[int]:
        return sorted(set(int(a) for a in self.lora_of_req if a >= 0))

    # ---- tensors (float32 arrays holding bf16-representable values)
    def _normal(self, tag: str, shape, std: float) -> np.ndarray:
        key = (tag, tuple(shape), std)
        if key not in self._cache:
            self._cache[key] = round_bf16(Stream(self.seed, tag).normal(shape, std))
        return self._cache[key]

    def x(self, mat: str = "q") -> np.ndarray:
        """Layer input rows [T, d_in] for projection `mat` (q, k, v share one x)."""
        d_in = dict((n, i) for n, i, _ in self.shape.mats)[mat]
        tag = "x" if mat in ("q", "k", "v", "up") else "x_" + mat
        return self._normal(tag, (self.n_tokens, d_in), 1.0)

    def y_base(self, mat: str) -> np.ndarray:
        """Stand-in for the base projection output x W of projection `mat`, [T, d_out]."""
        d_out = dict((n, o) for n, _, o in self.shape.mats)[mat]
        return self._normal("ybase_" + mat, (self.n_tokens, d_out), 1.0)

    def weight(self, mat: str) -> np.ndarray:
        """Base weight W [d_in, d_out] of projection `mat`, N(0, 1/d_in) so that x W has unit variance.  Values are
        taken from a seeded bank of 2^20 normal draws by a multiplicative hash of the element index (drawing the
        67 million values of an 8192 x 8192 matrix one by one takes longer than everything else in a test)."""
        key = ("W", mat)
        if key not in self._cache:
            d_in, d_out = dict((n, (i, o)) for n, i, o in self.shape.mats)[mat]
            bank = round_bf16(Stream(self.seed, "W_" + mat).normal((1 << 20,), 1.0 / np.sqrt(d_in)))
            k = np.arange(d_in * d_out, dtype=np.uint64)
            with np.errstate(over="ignore"):
                k = (k * np.uint64(0x9E3779B97F4A7C15)) >> np.uint64(44)
            self._cache[key] = bank[k.astype(np.int64)].reshape(d_in, d_out)
        return self._cache[key]

    def adapter(self, lora_id: int, mat: str) -> Tuple[np.ndarray, np.ndarray]:
        """(A [d_in, r], B [r, d_out]) of one adapter's projection, N(0, weight_std^2)."""
        d_in, d_out = dict((n, (i, o)) for n, i, o in self.shape.mats)[mat]
        r = int(self.ranks[lora_id])
        a = self._normal(f"A_{lora_id}_{mat}", (d_in, r), self.weight_std)
        b = self._normal(f"B_{lora_id}_{mat}", (r, d_out), self.weight_std)
        return a, b

    def q(self) -> np.ndarray:
        s = self.shape
        return self._normal("q", (self.n_tokens, s.n_q_heads, s.head_dim), 1.0)

    def kv_new(self) -> Tuple[np.ndarray, np.ndarray]:
        s = self.shape
        shp = (self.n_tokens, s.n_kv_heads, s.head_dim)
        return self._normal("k_new", shp, 1.0), self._normal("v_new", shp, 1.0)

    def kv_prefix(self, req: int) -> Tuple[np.ndarray, np.ndarray]:
        """Cached K, V of request `req`: [prefix_len, n_kv, d] each, rows taken from a noise bank."""
        return kv_bank_rows(self.seed, self.shape, req, np.arange(int(self.prefix_lens[req])))


# The cached KV of the large workloads (12 GB in the 13B decode case) is too much to draw value by
# value, so cached rows are looked up in a fixed bank of N(0,1) rows by a hash of (request, position).
BANK_ROWS = 4093


def kv_bank(seed: int, shape: LayerShape) -> np.ndarray:
    """[BANK_ROWS, n_kv * d] float32 bank of bf16-representable N(0,1) values."""
    return round_bf16(Stream(seed, "kv_bank").normal((BANK_ROWS, shape.n_kv_heads * shape.head_dim), 1.0))


def kv_bank_index(req, pos, which: int):
    """Bank row used for K (which=0) or V (which=1) of token `pos` of request `req` (array-friendly)."""
    return (req * 7919 + pos * 104729 + which * 1543 + 17) % BANK_ROWS


_bank_cache: Dict = {}


def kv_bank_rows(seed: int, shape: LayerShape, req: int, pos: np.ndarray):
    key = (seed, shape)
    if key not in _bank_cache:
        _bank_cache.clear()
        _bank_cache[key] = kv_bank(seed, shape)
    bank = _bank_cache[key]
    pos = np.asarray(pos, dtype=np.int64)
    k = bank[kv_bank_index(req, pos, 0)].reshape(len(pos), shape.n_kv_heads, shape.head_dim)
    v = bank[kv_bank_index(req, pos, 1)].reshape(len(pos), shape.n_kv_heads, shape.head_dim)
    return k, v


# ---------------------------------------------------------------- the five workloads
SHAPES = {
    "tiny": LayerShape(1024, 8, 8),
    "prefill7b": LayerShape(4096, 32, 32),
    "decode13b": LayerShape(5120, 40, 40, inter=13824),
    "gqa34b": LayerShape(8192, 64, 8),
    "swapstress": LayerShape(4096, 32, 32),
}
CONFIG_INDEX = {"tiny": 0, "prefill7b": 1, "decode13b": 2, "gqa34b": 3, "swapstress": 4}


def _sorted_by_adapter(lora, prefix, new):
    order = np.argsort(lora, kind="stable")
    return lora[order].astype(np.int32), prefix[order].astype(np.int32), new[order].astype(np.int32)


def make_workload(name: str, *, n_req: Optional[int] = None, len_range: Optional[Tuple[int, int]] = None,
                  n_adapters: Optional[int] = None, seed: Optional[int] = None,
                  shape: Optional[LayerShape] = None, rank: Optional[int] = None) -> Workload:
    """Build workload `name` at its full size, or a reduced copy when the keyword sizes are given.

    tiny        4 requests x (32 cached + 32 new), 4 adapters of rank 8, request i uses adapter i
    prefill7b   64 prefill requests, lengths U{128..1024}, half of each prompt cached (whole blocks),
                32 adapters of rank 16 with Zipf(1.0) popularity
    decode13b   256 requests x 1 new token, contexts U{512..4096}, 128 adapters rank 32, Zipf(0.8),
                LoRA also on MLP up/down
    gqa34b      16 requests x (3072 cached + 1024 new), 64 query / 8 KV heads, 16 adapters rank 64,
                request i uses adapter i
    swapstress  64 requests, first half decode (contexts U{512..4096}) and second half prefill as in
                prefill7b, 1000 adapters with ranks uniform in {8,16,32,64}, Zipf(1.2)
    """
    seed = BASE_SEED + CONFIG_INDEX[name] if seed is None else seed
    shp = shape or SHAPES[name]
    bt = shp.block_tokens
    rs = Stream(seed, "batch")
    pop = None
    if name == "tiny":
        n = n_req or 4
        na = n_adapters or 4
        ranks = np.full(na, rank or 8, dtype=np.int32)
        lora = np.arange(n) % na
        plen = len_range[0] if len_range else 32
        nlen = len_range[1] if len_range else 32
        prefix = np.full(n, plen)
        new = np.full(n, nlen)
        pool_blocks = 256
    elif name == "prefill7b":
        n = n_req or 64
        na = n_adapters or 32
        ranks = np.full(na, rank or 16, dtype=np.int32)
        pop = zipf_probs(na, 1.0)
        lora = rs.choice_p(pop, n)
        lo, hi = len_range or (128, 1024)
        L = rs.integers(lo, hi, n)
        prefix = (L // 2 // bt) * bt
        new = L - prefix
        pool_blocks = int(np.sum((L + bt - 1) // bt)) + 6 * na + 64
    elif name == "decode13b":
        n = n_req or 256
        na = n_adapters or 128
        ranks = np.full(na, rank or 32, dtype=np.int32)
        pop = zipf_probs(na, 0.8)
        lora = rs.choice_p(pop, n)
        lo, hi = len_range or (512, 4096)
        prefix = rs.integers(lo, hi, n)
        new = np.ones(n, dtype=np.int64)
        pool_blocks = int(np.sum((prefix + 1 + bt - 1) // bt)) + 18 * na + 64
    elif name == "gqa34b":
        n = n_req or 16
        na = n_adapters or 16
        ranks = np.full(na, rank or 64, dtype=np.int32)
        lora = np.arange(n) % na
        plen, nlen = len_range or (3072, 1024)
        prefix = np.full(n, plen)
        new = np.full(n, nlen)
        # full size: a 60e9-byte pool of 64 KiB blocks; reduced copies get a pool that just fits
        pool_blocks = (60 * 10**9) // shp.block_bytes if (n_req is None and len_range is None) \
            else int(n * ((plen + nlen + bt - 1) // bt)) + 110 * na + 64
    elif name == "swapstress":
        n = n_req or 64
        na = n_adapters or 1000
        ranks = np.array([8, 16, 32, 64], dtype=np.int32)[Stream(seed, "ranks").integers(0, 3, na)]
        pop = zipf_probs(na, 1.2)
        lora = rs.choice_p(pop, n)
        lo, hi = len_range or (512, 4096)
        nd = n // 2
        ctx = rs.integers(lo, hi, nd)
        plo, phi = (128, 1024) if len_range is None else (max(2 * bt, lo // 4), max(4 * bt, hi // 4))
        L = rs.integers(plo, phi, n - nd)
        pprefix = (L // 2 // bt) * bt
        prefix = np.concatenate([ctx, pprefix])
        new = np.concatenate([np.ones(nd, dtype=np.int64), L - pprefix])
        kv_blocks = int(np.sum((prefix + new + bt - 1) // bt))
        pool_blocks = kv_blocks + int(np.sum(ranks // 4)) + 1024
    else:
        raise KeyError(name)
    lora, prefix, new = _sorted_by_adapter(np.asarray(lora), np.asarray(prefix), np.asarray(new))
    return Workload(name=name, seed=seed, shape=shp, ranks=ranks, scale=2.0, lora_of_req=lora,
                    prefix_lens=prefix, new_lens=new, pool_blocks=pool_blocks,
                    host_blocks=0, popularity=pop)


# ---------------------------------------------------------------------------------------------------------------
# Multi-turn conversation traces for the cache manager / swapper (no arithmetic of the method here).
def conversation_trace(seed: int, n_lora: int, n_conv: int, n_turns: int, popularity: str = "uniform",
                       block_tokens: int = 16, system_blocks: int = 2, turn_tokens=(8, 72)):
    """Events (lora_id, tokens) of multi-turn chats: every turn repeats its conversation so far and adds new
    tokens; all conversations of an adapter start with that adapter's system prompt.  How conversations pick
    their adapter follows the paper's large-LoRA-count study (Section 6): "uniform" (equal probability),
    "distinct" (adapters taken in turn) or "skewed-x" (a Gaussian over the adapter index with standard
    deviation x, centred on the middle adapter)."""
    rs = Stream(seed, "conversation-trace/" + popularity)
    if popularity == "uniform":
        owner = rs.integers(0, n_lora - 1, n_conv)
    elif popularity == "distinct":
        owner = np.arange(n_conv, dtype=np.int64) % n_lora
    elif popularity.startswith("skewed-"):
        std = float(popularity.split("-", 1)[1])
        owner = np.clip(np.rint(n_lora / 2 + rs.normal((n_conv,), std)), 0, n_lora - 1).astype(np.int64)
    else:
        raise ValueError(popularity)
    system = {a: [int(v) for v in rs.integers(1, 999, system_blocks * block_tokens)] for a in range(n_lora)}
    convs = [dict(lora=int(owner[c]), tokens=[]) for c in range(n_conv)]
    events = []
    for _ in range(n_turns):
        for ci in rs.permutation(n_conv):
            c = convs[int(ci)]
            if not c["tokens"]:
                c["tokens"] = list(system[c["lora"]])
            n_new = int(rs.integers(turn_tokens[0], turn_tokens[1], 1)[0])
            c["tokens"] = c["tokens"] + [int(v) for v in rs.integers(1000, 30000, n_new)]
            events.append((c["lora"], list(c["tokens"])))
    return events
