"""One multi-LoRA attention-layer step over the pool model, chaining O1 -> KV store -> O2 -> O1.

Order of the step (Section 3.2 step 6 and Section 4.3 of the paper: the adapter and the prefix KV
are resident, the query runs, the KV it generates stays in HBM blocks):
  q, k, v = base projection + LoRA branch (Eq. 1, Eq. 2);  new K, V written into the request's
  blocks behind its cached prefix;  causal attention over [prefix || new];  o-projection + LoRA.
Values cross a stage boundary in bf16, because the path stores q, K, V and the attention output
in bf16 (pool blocks and activations); inside a stage everything is float64.

Pins: built only from the pinned functions of lora.py, attention.py and pool.py; with all B = 0 and
no prefix it reduces to plain causal attention of the base projections.
"""
import numpy as np

from .attention import attend_request
from .lora import lora_project
from .pool import bf16_bits_to_f64, f64_to_bf16_bits


def _store(x):
    return bf16_bits_to_f64(f64_to_bf16_bits(x))


def attention_layer_step(pool, x, y_base, adapters, seg_indptr, seg_lora, req_indptr, tables,
                         prefix_lens, new_lens, n_q, n_kv, d, scale, sm_scale):
    """y_base, adapters: dicts keyed 'q','k','v','o' (adapters[m] = {lora id: (A, B)}).

    Returns dict with bf16-stored q, k, v, attention output and the final o-projection output.
    """
    T = x.shape[0]
    proj = {m: _store(lora_project(y_base[m], x, seg_indptr, seg_lora, adapters[m], scale))
            for m in ("q", "k", "v")}
    k_new = proj["k"].reshape(T, n_kv, d)
    v_new = proj["v"].reshape(T, n_kv, d)
    pool.kv_append(f64_to_bf16_bits(k_new).reshape(T, n_kv, d), f64_to_bf16_bits(v_new).reshape(T, n_kv, d),
                   req_indptr, tables, prefix_lens, n_kv, d)
    q = proj["q"].reshape(T, n_q, d)
    attn = np.zeros((T, n_q, d))
    for i in range(len(new_lens)):
        lo, hi = int(req_indptr[i]), int(req_indptr[i + 1])
        k_ctx, v_ctx = pool.gather_kv(tables[i], int(prefix_lens[i]) + hi - lo, n_kv, d)
        attn[lo:hi] = attend_request(q[lo:hi], k_ctx, v_ctx, int(prefix_lens[i]), sm_scale)
    attn = _store(attn)
    out = lora_project(y_base["o"], attn.reshape(T, n_q * d), seg_indptr, seg_lora, adapters["o"], scale)
    return {"q": proj["q"], "k": proj["k"], "v": proj["v"], "attn": attn, "o": out}
