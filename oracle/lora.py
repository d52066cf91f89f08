"""O1 - heterogeneous-batch LoRA projection (Eq. 1 and Eq. 2 of the paper, Section 2.1).

Eq. 1 updates a weight as W' = W + A B; Eq. 2 applies the same low-rank branch to the K/V
projections.  In row-vector form with a LoRA scale s, a token row x that uses adapter i gets

    y = x W + s (x A_i) B_i ,   A_i: [d_in, r] (shrink),  B_i: [r, d_out] (expand).

Tokens of one batch are grouped into segments, one adapter per segment (the "segmented gather"
batching the paper cites in Section 2.1).  The base term x W arrives precomputed as y_base.

lora_linear is the same formula with the base term written out: y = x W + s (x A_i) B_i.

Pins: B = 0, scale = 0 or lora id -1 return y_base bit for bit; one adapter over the whole batch
equals the dense product x (W + s A B) (Eq. 1); linear in s; permuting segments permutes rows; a
hand-worked integer example.
"""
import numpy as np


def lora_project(y_base, x, seg_indptr, lora_ids, adapters, scale):
    """y[t] = y_base[t] + scale * (x[t] A_i) B_i for every token t of a segment that uses adapter i.

    y_base [T, d_out], x [T, d_in]; seg_indptr [n_seg+1] token offsets; lora_ids [n_seg], -1 means
    "no adapter" (row keeps y_base); adapters: {id: (A [d_in, r], B [r, d_out])}.  Returns float64.
    """
    y = np.array(y_base, dtype=np.float64, copy=True)
    x = np.asarray(x, dtype=np.float64)
    for s, lid in enumerate(lora_ids):
        lo, hi = int(seg_indptr[s]), int(seg_indptr[s + 1])
        if lid < 0 or hi <= lo:
            continue
        A, B = adapters[int(lid)]
        v = x[lo:hi] @ np.asarray(A, dtype=np.float64)          # shrink  [n, r]
        y[lo:hi] += scale * (v @ np.asarray(B, dtype=np.float64))  # expand  [n, d_out]
    return y


def lora_linear(x, W, seg_indptr, lora_ids, adapters, scale):
    """y[t] = x[t] W + scale * (x[t] A_i) B_i (Eq. 1 applied to a row vector); W [d_in, d_out].  Returns float64."""
    x = np.asarray(x, dtype=np.float64)
    return lora_project(x @ np.asarray(W, dtype=np.float64), x, seg_indptr, lora_ids, adapters, scale)
