"""O2 - causal attention over [cached prefix || new tokens] (Section 2.1 "KV Caches for
Multi-LoRAs", Section 4.2: a matched prefix's stored KV is reused instead of recomputed).

For request i with p cached tokens and n new tokens, query head h reads KV head h // (n_q/n_kv).
New token j (0-based) sees keys 0 .. p + j: the whole prefix plus the new tokens up to itself.

    s_u = sm_scale * <q_j, k_u>,   w = softmax_u(s),   o_j = sum_u w_u v_u .

Reusing prefix KV must give what recomputing the whole sequence gives: that is the definition
written out here, on contiguous K and V.

Pins: prefix reuse == rows p.. of a full recompute with prefix 0; equal V rows -> that row; equal
keys -> mean of the visible V; one visible key -> its V; a two-key case with weights 1/4, 3/4;
grouped KV heads == replicated KV heads.
"""
import numpy as np


def attend_request(q, k, v, prefix_len, sm_scale):
    """q [n, n_q, d]; k, v [prefix_len + n, n_kv, d] (contiguous context). Returns [n, n_q, d] float64."""
    q = np.asarray(q, dtype=np.float64)
    k = np.asarray(k, dtype=np.float64)
    v = np.asarray(v, dtype=np.float64)
    n, n_q, d = q.shape
    n_kv = k.shape[1]
    group = n_q // n_kv
    out = np.zeros((n, n_q, d), dtype=np.float64)
    if n == 0:
        return out
    pos = np.arange(k.shape[0])
    visible = pos[None, :] <= (prefix_len + np.arange(n))[:, None]   # [n, L]
    for h in range(n_q):
        kh, vh = k[:, h // group, :], v[:, h // group, :]
        s = sm_scale * (q[:, h, :] @ kh.T)
        s = np.where(visible, s, -np.inf)
        s = s - s.max(axis=1, keepdims=True)
        w = np.exp(s)
        w = w / w.sum(axis=1, keepdims=True)
        out[:, h, :] = w @ vh
    return out


def attend_rows(q_rows, row_pos, k, v, sm_scale):
    """Same definition for a sample of rows: q_rows [m, n_q, d], row_pos[m] = last visible key index."""
    q_rows = np.asarray(q_rows, dtype=np.float64)
    out = np.zeros_like(q_rows)
    for r in range(q_rows.shape[0]):
        last = int(row_pos[r])
        out[r] = attend_request(q_rows[r:r + 1], k[:last + 1], v[:last + 1], last, sm_scale)[0]
    return out


def attend_batch(q, k_ctx, v_ctx, prefix_lens, new_lens, sm_scale):
    """Batch form: q [T, n_q, d] packed by request; k_ctx[i], v_ctx[i] the contiguous context of request i."""
    outs, t = [], 0
    for i, n in enumerate(new_lens):
        n = int(n)
        outs.append(attend_request(q[t:t + n], k_ctx[i], v_ctx[i], int(prefix_lens[i]), sm_scale))
        t += n
    if not outs:
        return np.zeros((0,) + tuple(np.shape(q)[1:]), dtype=np.float64)
    return np.concatenate(outs, axis=0)
