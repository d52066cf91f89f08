"""Shared helpers of the GPU parity tests: tolerance, and the oracle-side mirror of a Session."""
import numpy as np

from oracle import pool as op
from paper_2505_03756_b200 import synth

REL = 1e-2   # spec bound: bf16 inputs, fp32 accumulation, bf16 output


def assert_close(got, ref, what=""):
    """Three checks per tensor, all tied to the benchmark spec's bound of 1e-2 (bf16 inputs, fp32 accumulation):
      max|d| <= 1e-2 max|ref|;   rms(d) <= 5e-3 rms(ref);   |d| <= 1e-2 |ref| + 4e-2 rms(ref) element-wise.
    The element-wise slack covers what bf16 storage itself costs: an attention weight kept as bf16 carries
    a relative error of 2^-9, so one dominant key moves an output by up to 2^-9 |v| (|v| up to ~4 rms)."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    if ref.size == 0:
        return
    assert np.all(np.isfinite(got)), what
    d = np.abs(got - ref)
    scale = np.abs(ref).max()
    rms = np.sqrt(np.mean(ref * ref))
    assert d.max() <= REL * max(scale, 1e-30), (what, "max", d.max(), scale)
    assert np.sqrt(np.mean(d * d)) <= 0.5 * REL * max(rms, 1e-30), (what, "rms", np.sqrt(np.mean(d * d)), rms)
    bad = d > REL * np.abs(ref) + 4 * REL * rms
    assert not bad.any(), (what, "elementwise", int(bad.sum()), d.max(), rms)


def replay_trace(sess):
    """Replays the session's allocator calls on the oracle's model; ids must match bit for bit."""
    model = op.PoolModel(sess.block_bytes, sess.wl.pool_blocks, max(1, sess.n_host_blocks))
    for kind, host, n, ids in sess.trace:
        if kind == "alloc":
            got = model.alloc(n, host=host)
            assert np.array_equal(np.array(got, dtype=np.uint32), ids), "allocator ids differ"
        else:
            model.free([int(i) for i in ids], host=host)
    return model


def oracle_adapters(wl, mat):
    return {a: tuple(m.astype(np.float64) for m in wl.adapter(a, mat)) for a in wl.used_adapters()}


def oracle_context(wl, req, k_new=None, v_new=None):
    """Contiguous float64 (K, V) of request `req`: cached prefix rows, then its new tokens' rows."""
    kp, vp = wl.kv_prefix(req)
    if k_new is None:
        return kp.astype(np.float64), vp.astype(np.float64)
    lo, hi = int(wl.req_indptr[req]), int(wl.req_indptr[req + 1])
    return (np.concatenate([kp, k_new[lo:hi]]).astype(np.float64),
            np.concatenate([vp, v_new[lo:hi]]).astype(np.float64))
