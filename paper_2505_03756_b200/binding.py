"""ctypes binding of libfastpool.so: argument marshalling only, one Python function per C call,
same names.  Device arguments are torch CUDA tensors (or raw integer addresses), host id lists are
numpy arrays.  Every step of the path runs inside the library; there is no Python or CPU fallback:
if the library has not been built, importing this module raises.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libfastpool.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2505_03756_b200.build` "
                      "(there is no fallback path)")
lib = C.CDLL(LIB_PATH)

FL_OK, FL_EINVAL, FL_ENOMEM, FL_EBADID, FL_EBUSY, FL_ECUDA, FL_ETIMEOUT = 0, -1, -2, -3, -4, -5, -6
_NAMES = {0: "FL_OK", -1: "FL_EINVAL", -2: "FL_ENOMEM", -3: "FL_EBADID", -4: "FL_EBUSY", -5: "FL_ECUDA",
          -6: "FL_ETIMEOUT"}


class FlError(RuntimeError):
    def __init__(self, code, where):
        super().__init__(f"{where}: {_NAMES.get(code, code)}")
        self.code = code


class fl_lora_shape(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("d_out", C.c_int32)]


class fl_node_stat(C.Structure):
    _fields_ = [("kind", C.c_int32), ("in_hbm", C.c_int32), ("candidate", C.c_int32), ("n_blocks", C.c_uint32),
                ("visits", C.c_double), ("last_use_s", C.c_double)]


class fl_swap_params(C.Structure):
    _fields_ = [("now_s", C.c_double), ("total_visits", C.c_double), ("low_lora", C.c_double), ("now_lora", C.c_int32),
                ("block_bytes", C.c_size_t), ("link_bytes_per_s", C.c_double), ("upper", C.c_double), ("lower", C.c_double)]


class fl_replay_config(C.Structure):
    _fields_ = [("variant", C.c_int32), ("capacity", C.c_uint32), ("block_tokens", C.c_int32), ("lora_blocks", C.c_uint32),
                ("tick_every", C.c_int32), ("batch_size", C.c_int32), ("block_bytes", C.c_size_t),
                ("link_bytes_per_s", C.c_double), ("upper", C.c_double), ("lower", C.c_double), ("t0", C.c_double),
                ("dt", C.c_double), ("lora_share", C.c_double)]


class fl_replay_result(C.Structure):
    _fields_ = [("asked_blocks", C.c_uint64), ("hit_blocks", C.c_uint64), ("lora_cold", C.c_uint64),
                ("swapped_in", C.c_uint64), ("swapped_out", C.c_uint64), ("used_blocks", C.c_uint64),
                ("n_nodes", C.c_uint64), ("n_samples", C.c_uint32)]


class fl_status(C.Structure):
    _fields_ = [("device_flags", C.c_uint32), ("blocks_used", C.c_uint32), ("blocks_free", C.c_uint32),
                ("host_blocks_used", C.c_uint32), ("host_blocks_free", C.c_uint32), ("lora_blocks", C.c_uint32),
                ("bytes_swapped_in", C.c_uint64), ("bytes_swapped_out", C.c_uint64), ("staging_bytes", C.c_uint64)]


class fl_lora_mat_placement(C.Structure):
    _fields_ = [("a_tab", C.c_uint32), ("a_row0", C.c_uint32), ("a_rpb", C.c_uint32), ("b_tab", C.c_uint32),
                ("b_row0", C.c_uint32), ("b_rpb", C.c_uint32), ("d_in", C.c_int32), ("d_out", C.c_int32)]


class fl_lora_placement(C.Structure):
    _fields_ = [("rank", C.c_int32), ("n_mats", C.c_int32), ("table_off", C.c_uint32), ("n_table", C.c_uint32),
                ("mats", fl_lora_mat_placement * 8)]


_vp, _u32p, _i32p = C.c_void_p, C.POINTER(C.c_uint32), C.POINTER(C.c_int32)
_SIGS = {
    "fl_pool_create": (C.c_int, [C.POINTER(_vp), C.c_size_t, C.c_uint32, C.c_uint32, C.c_int]),
    "fl_pool_destroy": (C.c_int, [_vp]),
    "fl_block_alloc": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_block_free": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_host_block_alloc": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_host_block_free": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_pool_device_base": (_vp, [_vp]),
    "fl_pool_host_base": (_vp, [_vp]),
    "fl_block_read": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_block_write": (C.c_int, [_vp, C.c_uint32, _vp]),
    "fl_pool_snapshot": (C.c_int, [_vp, C.c_int, _vp, C.c_uint32, _u32p]),
    "fl_pool_status": (C.c_int, [_vp, C.POINTER(fl_status), C.c_int]),
    "fl_last_cuda_error": (C.c_int, [_vp]),
    "fl_pool_set_option": (C.c_int, [_vp, C.c_int, C.c_int]),
    "fl_lora_blocks": (C.c_int, [C.c_size_t, C.c_int32, C.POINTER(fl_lora_shape), C.c_int, _u32p]),
    "fl_lora_pack_host": (C.c_int, [_vp, C.c_int32, C.POINTER(fl_lora_shape), C.c_int, C.POINTER(_vp),
                                    C.POINTER(_vp), _vp, C.c_uint32]),
    "fl_lora_register": (C.c_int, [_vp, C.c_int32, C.c_int32, C.POINTER(fl_lora_shape), C.c_int, _vp, C.c_uint32]),
    "fl_lora_unregister": (C.c_int, [_vp, C.c_int32]),
    "fl_lora_snapshot": (C.c_int, [_vp, C.c_int32, C.POINTER(fl_lora_placement), _vp, C.c_uint32, _u32p]),
    "fl_lora_sgmv_workspace": (C.c_size_t, [C.c_int, C.c_int]),
    "fl_lora_sgmv": (C.c_int, [_vp, _vp, _vp, C.c_int, _vp, _vp, C.c_int, C.c_int, C.c_float, _vp, C.c_size_t, _vp]),
    "fl_lora_sgmv_static": (C.c_int, [_vp, _vp, _vp, C.c_int, _vp, _vp, C.c_int, C.c_int, C.c_float, _vp]),
    "fl_lora_sgmv_multi": (C.c_int, [_vp, C.POINTER(_vp), _vp, _i32p, C.c_int, _vp, _vp, C.c_int, C.c_int,
                                     C.c_float, _vp, C.c_size_t, _vp]),
    "fl_lora_sgmv_qkv_append": (C.c_int, [_vp, _vp, _vp, _vp, _vp, C.c_int, C.c_int, C.c_int, _vp, _vp, C.c_int, C.c_int,
                                          C.c_float, _vp, _vp, _vp, _vp, C.c_int, C.c_int, _vp, C.c_size_t, _vp]),
    "fl_lora_linear_workspace": (C.c_size_t, [C.c_int, C.c_int]),
    "fl_lora_linear": (C.c_int, [_vp, _vp, _vp, _vp, C.c_int, _vp, _vp, C.c_int, C.c_int, C.c_float, _vp, C.c_size_t, _vp]),
    "fl_lora_linear_multi": (C.c_int, [_vp, C.POINTER(_vp), _vp, C.POINTER(_vp), _i32p, C.c_int, _vp, _vp, C.c_int,
                                       C.c_int, C.c_float, _vp, C.c_size_t, _vp]),
    "fl_lora_linear_qkv_append": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, C.c_int, C.c_int, C.c_int, _vp, _vp, C.c_int,
                                            C.c_int, C.c_float, _vp, _vp, _vp, _vp, C.c_int, C.c_int, _vp, _vp, _vp,
                                            C.c_size_t, _vp]),
    "fl_kv_append": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_int, C.c_int, C.c_int, _vp]),
    "fl_paged_attention_workspace": (C.c_size_t, [C.c_int, C.c_int, C.c_int, C.c_int, C.c_int]),
    "fl_paged_attention": (C.c_int, [_vp, _vp, _vp, _vp, _vp, _vp, _vp, _vp, C.c_int, C.c_int, C.c_int, C.c_int,
                                     C.c_int, C.c_float, _vp, C.c_size_t, _vp]),
    "fl_swap_out": (C.c_int, [_vp, _vp, _vp, C.c_uint32, _vp]),
    "fl_swap_in": (C.c_int, [_vp, _vp, _vp, C.c_uint32, _vp]),
    "fl_swap_record": (C.c_int, [_vp, _vp, _vp]),
    "fl_swap_wait": (C.c_int, [_vp, _vp, C.c_int]),
    "fl_inflight_mark": (C.c_int, [_vp, _vp, C.c_uint32, _vp]),
    "fl_requests_ready": (C.c_int, [_vp, _vp, _vp, C.c_int, _vp, C.POINTER(C.c_int)]),
    "fl_inflight_count": (C.c_int, [_vp, _u32p]),
    "fl_tree_create": (C.c_int, [C.POINTER(_vp), C.c_int]),
    "fl_tree_destroy": (C.c_int, [_vp]),
    "fl_tree_add_lora": (C.c_int, [_vp, C.c_int32, _vp, C.c_uint32, C.c_int, C.c_double, _i32p]),
    "fl_tree_match": (C.c_int, [_vp, C.c_int32, _vp, C.c_int, C.c_double, _i32p, _vp, C.c_int, C.POINTER(C.c_int),
                                C.POINTER(C.c_int)]),
    "fl_tree_insert": (C.c_int, [_vp, C.c_int32, _vp, C.c_int, _vp, C.c_double, _vp]),
    "fl_tree_size": (C.c_int, [_vp]),
    "fl_tree_node_blocks": (C.c_int, [_vp, C.c_int32, _vp, C.c_uint32, _u32p]),
    "fl_tree_stats": (C.c_int, [_vp, C.POINTER(fl_node_stat), C.c_int, C.POINTER(C.c_int), C.POINTER(C.c_double), _i32p]),
    "fl_tree_set_location": (C.c_int, [_vp, C.c_int32, C.c_int, _vp, C.c_uint32]),
    "fl_tree_check": (C.c_int, [_vp, _i32p]),
    "fl_tree_set_option": (C.c_int, [_vp, C.c_int, C.c_int]),
    "fl_tree_invalid": (C.c_int, [_vp, _u32p, _u32p]),
    "fl_cache_replay": (C.c_int, [C.POINTER(fl_replay_config), C.c_int, _vp, _vp, _vp, C.c_int,
                                  C.POINTER(fl_replay_result), _vp, C.c_uint32]),
    "fl_swapper_decide_policy": (C.c_int, [C.POINTER(fl_node_stat), C.c_int, C.POINTER(fl_swap_params), C.c_uint32,
                                           C.c_uint32, C.c_uint32, _vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
    "fl_expected_lora_demand": (C.c_int, [_vp, C.c_int, C.c_int, C.POINTER(C.c_double)]),
    "fl_swap_eval": (C.c_int, [C.POINTER(fl_node_stat), C.c_int, C.POINTER(fl_swap_params), _vp]),
    "fl_swapper_decide": (C.c_int, [C.POINTER(fl_node_stat), C.c_int, C.POINTER(fl_swap_params), C.c_uint32, C.c_uint32,
                                    _vp, C.POINTER(C.c_int), C.POINTER(C.c_int)]),
}
for _n, (_r, _a) in _SIGS.items():
    getattr(lib, _n).restype = _r
    getattr(lib, _n).argtypes = _a
EXPORTS = tuple(_SIGS)


def _check(code, where):
    if code != FL_OK:
        raise FlError(code, where)


def _dev(t):
    """Device address of a torch tensor (or pass an int / None through)."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    assert t.is_cuda and t.is_contiguous()
    return t.data_ptr()


def _ids(a):
    a = np.ascontiguousarray(a, dtype=np.uint32)
    return a, a.ctypes.data


def _stream(s):
    if s is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return s if isinstance(s, int) else s.cuda_stream


def _shapes(mats):
    arr = (fl_lora_shape * len(mats))()
    for i, (d_in, d_out) in enumerate(mats):
        arr[i].d_in, arr[i].d_out = int(d_in), int(d_out)
    return arr


# ------------------------------------------------------------------ one function per C call
def fl_pool_create(block_bytes, n_blocks, n_host_blocks, device=0):
    h = _vp()
    _check(lib.fl_pool_create(C.byref(h), block_bytes, n_blocks, n_host_blocks, device), "fl_pool_create")
    return h


def fl_pool_destroy(pool):
    _check(lib.fl_pool_destroy(pool), "fl_pool_destroy")


def _alloc(fn, name, pool, n):
    ids = np.empty(n, dtype=np.uint32)
    _check(fn(pool, n, ids.ctypes.data), name)
    return ids


def fl_block_alloc(pool, n):
    return _alloc(lib.fl_block_alloc, "fl_block_alloc", pool, n)


def fl_host_block_alloc(pool, n):
    return _alloc(lib.fl_host_block_alloc, "fl_host_block_alloc", pool, n)


def fl_block_free(pool, ids):
    a, p = _ids(ids)
    _check(lib.fl_block_free(pool, len(a), p), "fl_block_free")


def fl_host_block_free(pool, ids):
    a, p = _ids(ids)
    _check(lib.fl_host_block_free(pool, len(a), p), "fl_host_block_free")


def fl_pool_device_base(pool):
    return lib.fl_pool_device_base(pool)


def fl_pool_host_base(pool):
    return lib.fl_pool_host_base(pool)


def fl_block_read(pool, block_id, block_bytes):
    out = np.empty(block_bytes, dtype=np.uint8)
    _check(lib.fl_block_read(pool, int(block_id), out.ctypes.data), "fl_block_read")
    return out


def fl_block_write(pool, block_id, data):
    data = np.ascontiguousarray(data, dtype=np.uint8)
    _check(lib.fl_block_write(pool, int(block_id), data.ctypes.data), "fl_block_write")


def fl_pool_snapshot(pool, host=False):
    n = C.c_uint32()
    _check(lib.fl_pool_snapshot(pool, int(host), None, 0, C.byref(n)), "fl_pool_snapshot")
    ids = np.empty(n.value, dtype=np.uint32)
    _check(lib.fl_pool_snapshot(pool, int(host), ids.ctypes.data, n.value, C.byref(n)), "fl_pool_snapshot")
    return ids


def fl_pool_status(pool, clear=False):
    st = fl_status()
    _check(lib.fl_pool_status(pool, C.byref(st), int(clear)), "fl_pool_status")
    return {k: getattr(st, k) for k, _ in fl_status._fields_}


def fl_last_cuda_error(pool):
    return lib.fl_last_cuda_error(pool)


FL_OPT_PREFILL_KERNEL = 1
FL_OPT_POISON_FREED = 2
FL_OPT_SGMV_SHRINK = 3


def fl_pool_set_option(pool, key, value):
    _check(lib.fl_pool_set_option(pool, key, value), "fl_pool_set_option")


def fl_lora_blocks(block_bytes, rank, mats):
    n = C.c_uint32()
    _check(lib.fl_lora_blocks(block_bytes, rank, _shapes(mats), len(mats), C.byref(n)), "fl_lora_blocks")
    return n.value


def fl_lora_pack_host(pool, rank, mats, A_bits, B_bits, host_blocks):
    """A_bits[m]: numpy uint16 [d_in, rank]; B_bits[m]: numpy uint16 [rank, d_out] (bf16 bit patterns)."""
    A = [np.ascontiguousarray(a, dtype=np.uint16) for a in A_bits]
    B = [np.ascontiguousarray(b, dtype=np.uint16) for b in B_bits]
    pa = (_vp * len(A))(*[a.ctypes.data for a in A])
    pb = (_vp * len(B))(*[b.ctypes.data for b in B])
    ids, p = _ids(host_blocks)
    _check(lib.fl_lora_pack_host(pool, rank, _shapes(mats), len(mats), pa, pb, p, len(ids)), "fl_lora_pack_host")


def fl_lora_register(pool, lora_id, rank, mats, block_table):
    ids, p = _ids(block_table)
    _check(lib.fl_lora_register(pool, lora_id, rank, _shapes(mats), len(mats), p, len(ids)), "fl_lora_register")


def fl_lora_unregister(pool, lora_id):
    _check(lib.fl_lora_unregister(pool, lora_id), "fl_lora_unregister")


def fl_lora_snapshot(pool, lora_id):
    """What the device holds for the adapter: ({rank, n_mats, table_off, n_table, mats: [dict per projection]}, block table)."""
    pl = fl_lora_placement()
    n = C.c_uint32()
    _check(lib.fl_lora_snapshot(pool, lora_id, C.byref(pl), None, 0, C.byref(n)), "fl_lora_snapshot")
    table = np.empty(n.value, dtype=np.uint32)
    _check(lib.fl_lora_snapshot(pool, lora_id, C.byref(pl), table.ctypes.data, n.value, C.byref(n)), "fl_lora_snapshot")
    mats = [{k: getattr(pl.mats[m], k) for k, _ in fl_lora_mat_placement._fields_} for m in range(pl.n_mats)]
    return dict(rank=pl.rank, n_mats=pl.n_mats, table_off=pl.table_off, n_table=pl.n_table, mats=mats), table


def fl_lora_sgmv_workspace(n_tokens, n_mats=1):
    return lib.fl_lora_sgmv_workspace(n_tokens, n_mats)


def fl_lora_sgmv(pool, y, x, mat_index, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace, stream=None):
    _check(lib.fl_lora_sgmv(pool, _dev(y), _dev(x), mat_index, _dev(seg_indptr), _dev(lora_ids), n_seg, n_tokens,
                            scale, _dev(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "fl_lora_sgmv")


FL_SGMV_STATIC_BYTES = 8 << 20


def fl_lora_sgmv_static(pool, y, x, mat_index, seg_indptr, lora_ids, n_seg, n_tokens, scale, stream=None):
    """fl_lora_sgmv on the library's built-in scratch: the caller passes no workspace and nothing is allocated."""
    _check(lib.fl_lora_sgmv_static(pool, _dev(y), _dev(x), mat_index, _dev(seg_indptr), _dev(lora_ids), n_seg,
                                   n_tokens, scale, _stream(stream)), "fl_lora_sgmv_static")


def fl_lora_sgmv_multi(pool, ys, x, mat_indices, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace, stream=None):
    py = (_vp * len(ys))(*[_dev(y) for y in ys])
    mi = (C.c_int32 * len(ys))(*[int(m) for m in mat_indices])
    _check(lib.fl_lora_sgmv_multi(pool, py, _dev(x), mi, len(ys), _dev(seg_indptr), _dev(lora_ids), n_seg, n_tokens,
                                  scale, _dev(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "fl_lora_sgmv_multi")


def fl_lora_sgmv_qkv_append(pool, y_q, y_k, y_v, x, mat_q, mat_k, mat_v, seg_indptr, lora_ids, n_seg, n_tokens, scale,
                            req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_kv_heads, workspace, stream=None):
    _check(lib.fl_lora_sgmv_qkv_append(pool, _dev(y_q), _dev(y_k), _dev(y_v), _dev(x), mat_q, mat_k, mat_v,
                                       _dev(seg_indptr), _dev(lora_ids), n_seg, n_tokens, scale, _dev(req_indptr),
                                       _dev(kv_tbl_indptr), _dev(kv_tbl), _dev(prefix_lens), n_req, n_kv_heads,
                                       _dev(workspace), workspace.numel() * workspace.element_size(), _stream(stream)),
           "fl_lora_sgmv_qkv_append")


def fl_lora_linear_workspace(n_tokens, n_mats=1):
    return lib.fl_lora_linear_workspace(n_tokens, n_mats)


def fl_lora_linear(pool, y, x, w, mat_index, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace, stream=None):
    _check(lib.fl_lora_linear(pool, _dev(y), _dev(x), _dev(w), mat_index, _dev(seg_indptr), _dev(lora_ids), n_seg,
                              n_tokens, scale, _dev(workspace), workspace.numel() * workspace.element_size(),
                              _stream(stream)), "fl_lora_linear")


def fl_lora_linear_multi(pool, ys, x, ws, mat_indices, seg_indptr, lora_ids, n_seg, n_tokens, scale, workspace,
                         stream=None):
    py = (_vp * len(ys))(*[_dev(y) for y in ys])
    pw = (_vp * len(ws))(*[_dev(w) for w in ws])
    mi = (C.c_int32 * len(ys))(*[int(m) for m in mat_indices])
    _check(lib.fl_lora_linear_multi(pool, py, _dev(x), pw, mi, len(ys), _dev(seg_indptr), _dev(lora_ids), n_seg,
                                    n_tokens, scale, _dev(workspace), workspace.numel() * workspace.element_size(),
                                    _stream(stream)), "fl_lora_linear_multi")


def fl_lora_linear_qkv_append(pool, y_q, x, w_q, w_k, w_v, mat_q, mat_k, mat_v, seg_indptr, lora_ids, n_seg, n_tokens,
                              scale, req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_kv_heads, scratch_k,
                              scratch_v, workspace, stream=None):
    _check(lib.fl_lora_linear_qkv_append(pool, _dev(y_q), _dev(x), _dev(w_q), _dev(w_k), _dev(w_v), mat_q, mat_k, mat_v,
                                         _dev(seg_indptr), _dev(lora_ids), n_seg, n_tokens, scale, _dev(req_indptr),
                                         _dev(kv_tbl_indptr), _dev(kv_tbl), _dev(prefix_lens), n_req, n_kv_heads,
                                         _dev(scratch_k), _dev(scratch_v), _dev(workspace),
                                         workspace.numel() * workspace.element_size(), _stream(stream)),
           "fl_lora_linear_qkv_append")


def fl_kv_append(pool, k_new, v_new, req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, n_req, n_tokens, n_kv_heads,
                 stream=None):
    _check(lib.fl_kv_append(pool, _dev(k_new), _dev(v_new), _dev(req_indptr), _dev(kv_tbl_indptr), _dev(kv_tbl),
                            _dev(prefix_lens), n_req, n_tokens, n_kv_heads, _stream(stream)), "fl_kv_append")


def fl_paged_attention_workspace(n_req, n_tokens, n_tbl, n_q_heads, n_kv_heads):
    return lib.fl_paged_attention_workspace(n_req, n_tokens, n_tbl, n_q_heads, n_kv_heads)


def fl_paged_attention(pool, out, q, req_indptr, kv_tbl_indptr, kv_tbl, prefix_lens, new_lens, n_req, n_tokens, n_tbl,
                       n_q_heads, n_kv_heads, sm_scale, workspace, stream=None):
    _check(lib.fl_paged_attention(pool, _dev(out), _dev(q), _dev(req_indptr), _dev(kv_tbl_indptr), _dev(kv_tbl),
                                  _dev(prefix_lens), _dev(new_lens), n_req, n_tokens, n_tbl, n_q_heads, n_kv_heads,
                                  sm_scale, _dev(workspace), workspace.numel() * workspace.element_size(),
                                  _stream(stream)), "fl_paged_attention")


def fl_swap_out(pool, dev_ids, host_ids, side_stream):
    d, pd = _ids(dev_ids)
    h, ph = _ids(host_ids)
    assert len(d) == len(h)
    _check(lib.fl_swap_out(pool, pd, ph, len(d), _stream(side_stream)), "fl_swap_out")


def fl_swap_in(pool, dev_ids, host_ids, side_stream):
    d, pd = _ids(dev_ids)
    h, ph = _ids(host_ids)
    assert len(d) == len(h)
    _check(lib.fl_swap_in(pool, pd, ph, len(d), _stream(side_stream)), "fl_swap_in")


def fl_swap_record(pool, event, side_stream):
    if not event.cuda_event:          # torch creates the CUDA event lazily, on its first record
        event.record(side_stream if not isinstance(side_stream, int) else None)
    _check(lib.fl_swap_record(pool, event.cuda_event, _stream(side_stream)), "fl_swap_record")


def fl_swap_wait(pool, event, timeout_ms):
    return lib.fl_swap_wait(pool, event.cuda_event, timeout_ms)


def fl_inflight_mark(pool, dev_ids, event):
    """The listed device blocks wait for copies that finish when `event` (already recorded) completes."""
    d, pd = _ids(dev_ids)
    _check(lib.fl_inflight_mark(pool, pd, len(d), event.cuda_event), "fl_inflight_mark")


def fl_requests_ready(pool, block_lists):
    """block_lists[r] = device blocks request r touches; returns a bool array (True = may run now)."""
    n = len(block_lists)
    indptr = np.zeros(n + 1, dtype=np.int32)
    for r, b in enumerate(block_lists):
        indptr[r + 1] = indptr[r] + len(b)
    flat = np.ascontiguousarray(np.concatenate([np.asarray(b, dtype=np.uint32) for b in block_lists])
                                if indptr[-1] else np.zeros(0, dtype=np.uint32), dtype=np.uint32)
    ready = np.zeros(max(n, 1), dtype=np.uint8)
    n_ready = C.c_int(0)
    _check(lib.fl_requests_ready(pool, indptr.ctypes.data, flat.ctypes.data if flat.size else None, n,
                                 ready.ctypes.data, C.byref(n_ready)), "fl_requests_ready")
    out = ready[:n].astype(bool)
    assert int(out.sum()) == n_ready.value
    return out


def fl_inflight_count(pool):
    c = C.c_uint32(0)
    _check(lib.fl_inflight_count(pool, C.byref(c)), "fl_inflight_count")
    return int(c.value)


# ------------------------------------------------------------------ cache swapper (host side)
FL_NODE_LORA, FL_NODE_KV = 0, 1


def _nodes(nodes):
    arr = (fl_node_stat * len(nodes))()
    for k, nd in enumerate(nodes):
        arr[k].kind, arr[k].in_hbm, arr[k].candidate = int(nd["kind"]), int(nd["in_hbm"]), int(nd["candidate"])
        arr[k].n_blocks, arr[k].visits, arr[k].last_use_s = int(nd["n_blocks"]), float(nd["visits"]), float(nd["last_use_s"])
    return arr


def _params(prm):
    p = fl_swap_params()
    for name, _ in fl_swap_params._fields_:
        setattr(p, name, prm[name])
    return p


def fl_expected_lora_demand(prob, batch_size):
    prob = np.ascontiguousarray(prob, dtype=np.float64)
    out = C.c_double()
    _check(lib.fl_expected_lora_demand(prob.ctypes.data, len(prob), batch_size, C.byref(out)), "fl_expected_lora_demand")
    return out.value


def fl_swap_eval(nodes, prm):
    arr = nodes if isinstance(nodes, C.Array) else _nodes(nodes)
    out = np.empty(len(arr), dtype=np.float64)
    _check(lib.fl_swap_eval(arr, len(arr), C.byref(_params(prm)), out.ctypes.data), "fl_swap_eval")
    return out


def fl_swapper_decide(nodes, prm, blocks_used, blocks_total):
    """Returns (direction, ordered node indices): -1 swap-out, +1 swap-in, 0 nothing."""
    arr = nodes if isinstance(nodes, C.Array) else _nodes(nodes)
    order = np.empty(len(arr), dtype=np.int32)
    n, d = C.c_int(), C.c_int()
    _check(lib.fl_swapper_decide(arr, len(arr), C.byref(_params(prm)), blocks_used, blocks_total, order.ctypes.data,
                                 C.byref(n), C.byref(d)), "fl_swapper_decide")
    return d.value, order[:n.value].tolist()


FL_POLICY_LRU, FL_POLICY_NO_LORA_REWARD, FL_POLICY_ONLY_LORA, FL_POLICY_ONLY_KV = 1, 2, 4, 8
FL_TREE_OPT_DEPENDENCY = 0
FL_REPLAY_FULL, FL_REPLAY_WOS, FL_REPLAY_WOL, FL_REPLAY_WOM, FL_REPLAY_STATIC = 0, 1, 2, 3, 4


def fl_cache_replay(events, n_lora, variant, capacity, bt=16, lora_blocks=2, tick_every=8, batch_size=8,
                    block_bytes=65536, link_bytes_per_s=50e9, upper=0.95, lower=0.70, t0=1.0, dt=0.05, lora_share=0.2):
    """events: [(lora_id, tokens), ...].  Returns the counters of fl_replay_result plus the invalid-KV samples."""
    cfg = fl_replay_config(variant, capacity, bt, lora_blocks, tick_every, batch_size, block_bytes, link_bytes_per_s,
                           upper, lower, t0, dt, lora_share)
    lora = np.ascontiguousarray([e[0] for e in events], dtype=np.int32)
    indptr = np.zeros(len(events) + 1, dtype=np.int32)
    for k, e in enumerate(events):
        indptr[k + 1] = indptr[k] + len(e[1])
    tok = np.ascontiguousarray(np.concatenate([np.asarray(e[1], dtype=np.int32) for e in events])
                               if len(events) else np.zeros(0, np.int32), dtype=np.int32)
    res = fl_replay_result()
    cap = len(events) // max(1, tick_every) + 1
    samples = np.zeros(cap, dtype=np.float64)
    _check(lib.fl_cache_replay(C.byref(cfg), n_lora, lora.ctypes.data, indptr.ctypes.data, tok.ctypes.data, len(events),
                               C.byref(res), samples.ctypes.data, cap), "fl_cache_replay")
    out = {k: int(getattr(res, k)) for k, _ in fl_replay_result._fields_ if k != "n_samples"}
    out["invalid_samples"] = samples[:res.n_samples].tolist()
    return out


def fl_swapper_decide_policy(nodes, prm, blocks_used, blocks_total, policy):
    """fl_swapper_decide with parts of the cost model switched off (policy flags); blocks_used may exceed the total."""
    arr = nodes if isinstance(nodes, C.Array) else _nodes(nodes)
    order = np.empty(max(len(arr), 1), dtype=np.int32)
    n, d = C.c_int(), C.c_int()
    _check(lib.fl_swapper_decide_policy(arr, len(arr), C.byref(_params(prm)), blocks_used, blocks_total, policy,
                                        order.ctypes.data, C.byref(n), C.byref(d)), "fl_swapper_decide_policy")
    return d.value, order[:n.value].tolist()


# ------------------------------------------------------------------ usage dependency tree (host side)
def fl_tree_create(block_tokens):
    h = _vp()
    _check(lib.fl_tree_create(C.byref(h), block_tokens), "fl_tree_create")
    return h


def fl_tree_destroy(tree):
    _check(lib.fl_tree_destroy(tree), "fl_tree_destroy")


def fl_tree_add_lora(tree, lora_id, blocks, in_hbm, now_s):
    ids, p = _ids(blocks)
    node = C.c_int32()
    _check(lib.fl_tree_add_lora(tree, lora_id, p, len(ids), int(in_hbm), now_s, C.byref(node)), "fl_tree_add_lora")
    return node.value


def fl_tree_match(tree, lora_id, tokens, now_s):
    """Returns (LoRA node, [matched KV nodes in path order], matched token count)."""
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    cap = len(tok) + 1
    path = np.empty(cap, dtype=np.int32)
    ln, n, m = C.c_int32(), C.c_int(), C.c_int()
    _check(lib.fl_tree_match(tree, lora_id, tok.ctypes.data, len(tok), now_s, C.byref(ln), path.ctypes.data, cap,
                             C.byref(n), C.byref(m)), "fl_tree_match")
    return ln.value, path[:n.value].tolist(), m.value


def fl_tree_insert(tree, parent, tokens, block_ids, now_s):
    tok = np.ascontiguousarray(tokens, dtype=np.int32)
    ids, p = _ids(block_ids)
    new = np.empty(len(ids), dtype=np.int32)
    _check(lib.fl_tree_insert(tree, parent, tok.ctypes.data, len(ids), p, now_s, new.ctypes.data), "fl_tree_insert")
    return new.tolist()


def fl_tree_size(tree):
    return lib.fl_tree_size(tree)


def fl_tree_node_blocks(tree, node):
    n = C.c_uint32()
    _check(lib.fl_tree_node_blocks(tree, node, None, 0, C.byref(n)), "fl_tree_node_blocks")
    out = np.empty(n.value, dtype=np.uint32)
    _check(lib.fl_tree_node_blocks(tree, node, out.ctypes.data, n.value, C.byref(n)), "fl_tree_node_blocks")
    return out.tolist()


def fl_tree_stats(tree, raw=False):
    """Returns (per-node stats, total visits, adapters in HBM); raw=True keeps the ctypes array for fl_swapper_decide."""
    n = C.c_int()
    _check(lib.fl_tree_stats(tree, None, 0, C.byref(n), None, None), "fl_tree_stats")
    arr = (fl_node_stat * max(1, n.value))()
    tot, nl = C.c_double(), C.c_int32()
    _check(lib.fl_tree_stats(tree, arr, n.value, C.byref(n), C.byref(tot), C.byref(nl)), "fl_tree_stats")
    if raw:
        return arr, n.value, tot.value, nl.value
    stats = [{k: getattr(arr[i], k) for k, _ in fl_node_stat._fields_} for i in range(n.value)]
    return stats, tot.value, nl.value


def fl_tree_set_location(tree, node, in_hbm, blocks):
    ids, p = _ids(blocks)
    _check(lib.fl_tree_set_location(tree, node, int(in_hbm), p, len(ids)), "fl_tree_set_location")


def fl_tree_check(tree):
    bad = C.c_int32(-1)
    return lib.fl_tree_check(tree, C.byref(bad)), bad.value


def fl_tree_set_option(tree, option, value):
    _check(lib.fl_tree_set_option(tree, option, value), "fl_tree_set_option")


def fl_tree_invalid(tree):
    """(KV nodes in HBM with an ancestor outside HBM, KV nodes in HBM)."""
    bad, total = C.c_uint32(0), C.c_uint32(0)
    _check(lib.fl_tree_invalid(tree, C.byref(bad), C.byref(total)), "fl_tree_invalid")
    return int(bad.value), int(total.value)


# ------------------------------------------------------------------ views of the two slabs (for tests and tools)
def device_block_bytes(pool, block_bytes, ids):
    """Copies the listed device blocks to host: uint8 [len(ids), block_bytes]."""
    out = np.empty((len(ids), block_bytes), dtype=np.uint8)
    for k, b in enumerate(ids):
        out[k] = fl_block_read(pool, b, block_bytes)
    return out


def host_slab(pool, block_bytes, n_host_blocks):
    """numpy uint8 view [n_host_blocks, block_bytes] of the pinned host slab."""
    base = fl_pool_host_base(pool)
    buf = (C.c_uint8 * (block_bytes * n_host_blocks)).from_address(base)
    return np.frombuffer(buf, dtype=np.uint8).reshape(n_host_blocks, block_bytes)
