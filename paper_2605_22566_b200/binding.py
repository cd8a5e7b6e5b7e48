"""ctypes binding of the C-ABI library (include/gf.h).  Argument marshalling only.

Every function takes plain integers / device pointers (`tensor.data_ptr()`) and forwards them;
all of the path runs in the CUDA kernels of libgfpath.so.  There is no CPU fallback: importing
this module without the built library raises.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libgfpath.so")
GEN_PATH = os.path.join(_HERE, "libgfgen.so")

GF_OK = 0
GF_ERR_INVALID_ARG, GF_ERR_INVALID_GRAPH, GF_ERR_INVALID_PATH, GF_ERR_CAPACITY = 1, 2, 3, 4
GF_ERR_NOT_WRITTEN, GF_ERR_NOT_BUILT, GF_ERR_CUDA, GF_ERR_TIMEOUT, GF_ERR_BOUNDS = 5, 6, 7, 8, 9
GF_MODE_DECODE, GF_MODE_EXTEND = 0, 1
GF_MODE_DEFERRED = 0x100
GF_TILE_TOKENS = 64
GF_STATIC_SCRATCH_BYTES = 32 << 20

EXPORTS = [
    "gf_status_string", "gf_pool_bytes_per_tile", "gf_workspace_bytes", "gf_wgraph_create",
    "gf_wgraph_destroy", "gf_node_kv_write", "gf_node_kv_read", "gf_node_kv_reconstruct", "gf_residual_encode", "gf_transition_counts", "gf_select_transitions", "gf_build_path_tables", "gf_tables_info",
    "gf_tables_bad_request", "gf_tables_export", "gf_path_attention_decode",
    "gf_path_attention_extend", "gf_path_attention_decode_static", "gf_last_status", "gf_launch_count", "gf_profile_enable", "gf_profile_read",
    "gf_debug_counters", "gf_debug_wait_probe", "gf_node_kv_reserve", "gf_node_kv_release", "gf_pool_info",
    "gf_path_attention_extend_append", "gf_node_extent", "gf_debug_bounds_enabled", "gf_debug_bounds_site",
    "gf_node_kv_attach_residual", "gf_edge_scores", "gf_edge_scores_scratch_bytes",
]


class GfError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: status {status} ({status_string(status)})")


class WGraphDesc(C.Structure):
    _fields_ = [("num_nodes", C.c_int32), ("num_shared_nodes", C.c_int32), ("num_edges", C.c_int32),
                ("edge_src_host", C.c_void_p), ("edge_dst_host", C.c_void_p),
                ("num_layers", C.c_int32), ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32),
                ("head_dim", C.c_int32), ("softmax_scale", C.c_float),
                ("kv_pool_dev", C.c_void_p), ("kv_pool_bytes", C.c_uint64),
                ("workspace_dev", C.c_void_p), ("workspace_bytes", C.c_uint64), ("max_residual_nodes", C.c_int32)]


class Residual(C.Structure):
    _fields_ = [("bitmap_dev", C.c_void_p), ("values_dev", C.c_void_p), ("row_ptr_dev", C.c_void_p),
                ("nnz", C.c_int64)]


class ResidualBuf(C.Structure):
    _fields_ = [("bitmap_dev", C.c_void_p), ("values_dev", C.c_void_p), ("row_ptr_dev", C.c_void_p),
                ("capacity", C.c_int64), ("nnz_dev", C.c_void_p)]


class Policy(C.Structure):
    _fields_ = [("chunk_tokens", C.c_int32), ("group_tile", C.c_int32), ("group_unit", C.c_int32),
                ("max_chunk_mult", C.c_int32)]


_TABLE_FIELDS = ["seg_node", "seg_len", "seg_off", "grp_ptr", "grp_req", "req_len", "req_nseg", "items",
                 "mrg_ptr", "mrg_slot", "pseg_ptr", "pseg", "q_ptr", "self_seg"]


class TablesHost(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _TABLE_FIELDS]


class TablesInfo(C.Structure):
    _fields_ = [("num_requests", C.c_int32), ("num_segments", C.c_int32), ("num_pairs", C.c_int32),
                ("num_items", C.c_int32), ("num_slots", C.c_int32), ("mode", C.c_int32),
                ("resident_tokens", C.c_int64), ("materialised_tokens", C.c_int64),
                ("num_q_rows", C.c_int64)]


class Profile(C.Structure):
    _fields_ = [("tables_ms", C.c_double), ("decode_ms", C.c_double), ("merge_ms", C.c_double),
                ("extend_ms", C.c_double), ("tables_launches", C.c_uint64), ("decode_launches", C.c_uint64),
                ("merge_launches", C.c_uint64), ("extend_launches", C.c_uint64)]


class Scorer(C.Structure):
    _fields_ = [("d_in", C.c_int32), ("d_hidden", C.c_int32), ("d_mlp", C.c_int32),
                ("w_gcn1_dev", C.c_void_p), ("w_gcn2_dev", C.c_void_p), ("w_mlp1_dev", C.c_void_p),
                ("b_mlp1_dev", C.c_void_p), ("w_mlp2_dev", C.c_void_p), ("b_mlp2_dev", C.c_void_p),
                ("w_mlp3_dev", C.c_void_p), ("b_mlp3", C.c_float)]


class PoolInfo(C.Structure):
    _fields_ = [("capacity_tiles", C.c_uint32), ("tiles_in_use", C.c_uint32), ("high_water_tiles", C.c_uint32)]


_lib = None
_gen = None


def lib():
    """The loaded library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2605_22566_b200.build` "
                               "(the path has no CPU fallback)")
        L = C.CDLL(LIB_PATH)
        L.gf_status_string.restype = C.c_char_p
        L.gf_status_string.argtypes = [C.c_int]
        L.gf_pool_bytes_per_tile.restype = C.c_uint64
        L.gf_pool_bytes_per_tile.argtypes = [C.c_int32]
        L.gf_workspace_bytes.restype = C.c_uint64
        L.gf_workspace_bytes.argtypes = [C.c_int32] * 8
        L.gf_wgraph_create.argtypes = [C.POINTER(WGraphDesc), C.POINTER(C.c_void_p)]
        L.gf_wgraph_destroy.argtypes = [C.c_void_p]
        L.gf_node_kv_write.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                       C.c_int32, C.c_void_p]
        L.gf_node_kv_read.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.gf_node_kv_reconstruct.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.POINTER(Residual),
                                             C.POINTER(Residual), C.c_void_p]
        L.gf_node_kv_attach_residual.argtypes = L.gf_node_kv_reconstruct.argtypes
        L.gf_residual_encode.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_float,
                                         C.POINTER(ResidualBuf), C.POINTER(ResidualBuf), C.c_void_p]
        L.gf_transition_counts.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p,
                                           C.c_void_p, C.c_void_p]
        L.gf_select_transitions.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
        L.gf_build_path_tables.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p, C.c_void_p,
                                           C.c_int32, C.POINTER(Policy), C.POINTER(C.c_void_p), C.c_void_p]
        L.gf_tables_info.argtypes = [C.c_void_p, C.POINTER(TablesInfo)]
        L.gf_tables_bad_request.restype = C.c_int32
        L.gf_tables_bad_request.argtypes = [C.c_void_p]
        L.gf_tables_export.argtypes = [C.c_void_p, C.POINTER(TablesHost)]
        L.gf_path_attention_decode.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                               C.c_void_p, C.c_void_p]
        L.gf_path_attention_extend.argtypes = L.gf_path_attention_decode.argtypes
        L.gf_path_attention_decode_static.argtypes = L.gf_path_attention_decode.argtypes
        L.gf_last_status.argtypes = [C.c_void_p, C.c_void_p]
        L.gf_profile_enable.argtypes = [C.c_void_p, C.c_int32]
        L.gf_profile_read.argtypes = [C.c_void_p, C.POINTER(Profile)]
        L.gf_launch_count.restype = C.c_uint64
        L.gf_launch_count.argtypes = [C.c_void_p]
        L.gf_node_kv_reserve.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_void_p]
        L.gf_node_kv_release.argtypes = [C.c_void_p, C.c_int32, C.c_void_p]
        L.gf_node_extent.argtypes = [C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_int32)]
        L.gf_pool_info.argtypes = [C.c_void_p, C.POINTER(PoolInfo)]
        L.gf_path_attention_extend_append.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                                      C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.gf_edge_scores_scratch_bytes.restype = C.c_uint64
        L.gf_edge_scores_scratch_bytes.argtypes = [C.c_void_p, C.POINTER(Scorer), C.c_int32, C.c_int32]
        L.gf_edge_scores.argtypes = [C.c_void_p, C.POINTER(Scorer), C.c_void_p, C.c_int32, C.c_void_p, C.c_void_p,
                                     C.c_void_p, C.c_uint64, C.c_void_p]
        L.gf_debug_bounds_enabled.restype = C.c_int32
        L.gf_debug_bounds_site.restype = C.c_int32
        L.gf_debug_bounds_site.argtypes = [C.c_void_p]
        L.gf_debug_counters.argtypes = [C.c_void_p, C.POINTER(C.c_uint64), C.c_void_p]
        L.gf_debug_wait_probe.argtypes = [C.c_void_p, C.c_int64, C.POINTER(C.c_int32), C.c_void_p]
        _lib = L
    return _lib


def gen_lib():
    global _gen
    if _gen is None:
        if not os.path.exists(GEN_PATH):
            raise RuntimeError(f"{GEN_PATH} is missing: run `python -m paper_2605_22566_b200.build`")
        G = C.CDLL(GEN_PATH)
        G.gfgen_fill_bf16.argtypes = [C.c_void_p, C.c_uint64, C.c_uint64, C.c_uint64, C.c_void_p, C.c_void_p]
        _gen = G
    return _gen


def status_string(s: int) -> str:
    return lib().gf_status_string(int(s)).decode()


def gf_pool_bytes_per_tile(head_dim: int) -> int:
    return int(lib().gf_pool_bytes_per_tile(head_dim))


def gf_workspace_bytes(num_nodes, num_edges, max_requests, max_pairs, max_items, max_slots,
                       num_q_heads, head_dim) -> int:
    return int(lib().gf_workspace_bytes(num_nodes, num_edges, max_requests, max_pairs, max_items,
                                        max_slots, num_q_heads, head_dim))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(a, dtype=np.int32)


def gf_wgraph_create(*, num_nodes, num_shared_nodes, edge_src, edge_dst, num_layers, num_q_heads,
                     num_kv_heads, head_dim, kv_pool_ptr, kv_pool_bytes, workspace_ptr,
                     workspace_bytes, softmax_scale=0.0, max_residual_nodes=0):
    """Returns (status, handle).  edge_src/edge_dst are host integer sequences."""
    src, dst = _i32(edge_src), _i32(edge_dst)
    d = WGraphDesc(num_nodes, num_shared_nodes, len(src),
                   src.ctypes.data if len(src) else None, dst.ctypes.data if len(dst) else None,
                   num_layers, num_q_heads, num_kv_heads, head_dim, softmax_scale,
                   kv_pool_ptr, kv_pool_bytes, workspace_ptr, workspace_bytes, max_residual_nodes)
    h = C.c_void_p()
    st = lib().gf_wgraph_create(C.byref(d), C.byref(h))
    return st, h.value


def gf_wgraph_destroy(g) -> int:
    return lib().gf_wgraph_destroy(g)


def gf_node_kv_write(g, node, layer, k_ptr, v_ptr, n_tokens, stream=0) -> int:
    return lib().gf_node_kv_write(g, node, layer, k_ptr, v_ptr, n_tokens, stream)


def gf_node_kv_read(g, node, layer, k_out_ptr, v_out_ptr, stream=0) -> int:
    return lib().gf_node_kv_read(g, node, layer, k_out_ptr, v_out_ptr, stream)


def gf_node_kv_reconstruct(g, node, layer, base_node, k_res: Optional[tuple], v_res: Optional[tuple], stream=0) -> int:
    """k_res / v_res = (bitmap_ptr, values_ptr, row_ptr_ptr, nnz) device pointers, or None."""
    rk = C.byref(Residual(*k_res)) if k_res is not None else None
    rv = C.byref(Residual(*v_res)) if v_res is not None else None
    return lib().gf_node_kv_reconstruct(g, node, layer, base_node, rk, rv, stream)


def gf_node_kv_attach_residual(g, node, layer, base_node, k_res: Optional[tuple], v_res: Optional[tuple], stream=0) -> int:
    """Like gf_node_kv_reconstruct, but nothing is materialised: decode applies the residual to the base
    node's tiles in shared memory.  The residual arrays must stay alive while the node exists."""
    rk = C.byref(Residual(*k_res)) if k_res is not None else None
    rv = C.byref(Residual(*v_res)) if v_res is not None else None
    return lib().gf_node_kv_attach_residual(g, node, layer, base_node, rk, rv, stream)


def gf_residual_encode(g, base_node, layer, k_full_ptr, v_full_ptr, threshold, k_out: Optional[tuple],
                       v_out: Optional[tuple], stream=0) -> int:
    """k_out / v_out = (bitmap_ptr, values_ptr, row_ptr_ptr, capacity, nnz_ptr) device pointers, or None."""
    bk = C.byref(ResidualBuf(*k_out)) if k_out is not None else None
    bv = C.byref(ResidualBuf(*v_out)) if v_out is not None else None
    return lib().gf_residual_encode(g, base_node, layer, k_full_ptr, v_full_ptr, threshold, bk, bv, stream)


def gf_transition_counts(g, num_requests, num_path_nodes, path_ptr_dev, path_node_dev, counts_dev, misses_dev,
                         stream=0) -> int:
    return lib().gf_transition_counts(g, num_requests, num_path_nodes, path_ptr_dev, path_node_dev, counts_dev,
                                      misses_dev, stream)


def gf_select_transitions(g, counts_dev, min_count, keep_dev, totals_dev, stream=0) -> int:
    return lib().gf_select_transitions(g, counts_dev, min_count, keep_dev, totals_dev, stream)


def gf_build_path_tables(g, num_requests, num_path_nodes, path_ptr_dev, path_node_dev, mode,
                         policy: Optional[tuple] = None, stream=0):
    """Returns (status, tables handle or None).  policy = (chunk_tokens, group_tile, group_unit,
    max_chunk_mult) or None for the default."""
    t = C.c_void_p()
    pol = C.byref(Policy(*policy)) if policy is not None else None
    st = lib().gf_build_path_tables(g, num_requests, num_path_nodes, path_ptr_dev, path_node_dev,
                                    mode, pol, C.byref(t), stream)
    return st, t.value


def gf_tables_info(t) -> TablesInfo:
    info = TablesInfo()
    st = lib().gf_tables_info(t, C.byref(info))
    if st != GF_OK:
        raise GfError(st, "gf_tables_info")
    return info


def gf_tables_bad_request(t) -> int:
    return lib().gf_tables_bad_request(t)


def gf_tables_export(t) -> dict:
    """Host copies of T1..T7 as numpy int32 arrays (plus the info fields)."""
    info = gf_tables_info(t)
    sizes = {"seg_node": info.num_segments, "seg_len": info.num_segments, "seg_off": info.num_segments,
             "grp_ptr": info.num_segments + 1, "grp_req": info.num_pairs, "req_len": info.num_requests,
             "req_nseg": info.num_requests, "items": info.num_items * 6, "mrg_ptr": info.num_requests + 1,
             "mrg_slot": info.num_slots, "pseg_ptr": info.num_requests + 1, "pseg": info.num_pairs,
             "q_ptr": info.num_requests + 1, "self_seg": info.num_requests}
    arrs = {k: np.zeros(max(n, 1), dtype=np.int32) for k, n in sizes.items()}
    th = TablesHost(**{k: arrs[k].ctypes.data for k in _TABLE_FIELDS})
    st = lib().gf_tables_export(t, C.byref(th))
    if st != GF_OK:
        raise GfError(st, "gf_tables_export")
    out = {k: arrs[k][:sizes[k]] for k in _TABLE_FIELDS}
    out["items"] = out["items"].reshape(-1, 6)
    if info.mode != GF_MODE_EXTEND:
        del out["q_ptr"], out["self_seg"]
    out.update(num_slots=info.num_slots, resident_tokens=info.resident_tokens,
               materialised_tokens=info.materialised_tokens, num_q_rows=info.num_q_rows, bad_req=-1)
    return out


def gf_path_attention_decode(g, t, layer, q_ptr, out_ptr, lse_ptr=None, stream=0) -> int:
    return lib().gf_path_attention_decode(g, t, layer, q_ptr, out_ptr, lse_ptr, stream)


def gf_path_attention_decode_static(g, t, layer, q_ptr, out_ptr, lse_ptr=None, stream=0) -> int:
    """Decode with the partials in the library's resident array instead of the workspace, for
    callers that cannot hand over scratch memory; status GF_ERR_CAPACITY beyond 32 MiB."""
    return lib().gf_path_attention_decode_static(g, t, layer, q_ptr, out_ptr, lse_ptr, stream)


def gf_path_attention_extend(g, t, layer, q_ptr, out_ptr, lse_ptr=None, stream=0) -> int:
    return lib().gf_path_attention_extend(g, t, layer, q_ptr, out_ptr, lse_ptr, stream)


def gf_path_attention_extend_append(g, t, layer, q_ptr, k_new_ptr, v_new_ptr, out_ptr, lse_ptr=None, stream=0) -> int:
    return lib().gf_path_attention_extend_append(g, t, layer, q_ptr, k_new_ptr, v_new_ptr, out_ptr, lse_ptr, stream)


def gf_node_kv_reserve(g, node, n_tokens, stream=0) -> int:
    return lib().gf_node_kv_reserve(g, node, n_tokens, stream)


def gf_node_kv_release(g, node, stream=0) -> int:
    return lib().gf_node_kv_release(g, node, stream)


def gf_node_extent(g, node):
    """(status, n_tokens, token_offset) of a node's extent."""
    n, off = C.c_int32(-1), C.c_int32(-1)
    st = lib().gf_node_extent(g, node, C.byref(n), C.byref(off))
    return st, int(n.value), int(off.value)


def gf_pool_info(g) -> PoolInfo:
    info = PoolInfo()
    st = lib().gf_pool_info(g, C.byref(info))
    if st != GF_OK:
        raise GfError(st, "gf_pool_info")
    return info


def gf_edge_scores_scratch_bytes(g, scorer: Scorer, num_tasks: int, tasks_per_pass: int) -> int:
    return int(lib().gf_edge_scores_scratch_bytes(g, C.byref(scorer), num_tasks, tasks_per_pass))


def gf_edge_scores(g, scorer: Scorer, x_op_ptr, num_tasks, x_task_ptr, scores_ptr, scratch_ptr, scratch_bytes, stream=0) -> int:
    return lib().gf_edge_scores(g, C.byref(scorer), x_op_ptr, num_tasks, x_task_ptr, scores_ptr, scratch_ptr,
                                scratch_bytes, stream)


def gf_last_status(g, stream=0) -> int:
    return lib().gf_last_status(g, stream)


def gf_profile_enable(g, on: bool) -> int:
    return lib().gf_profile_enable(g, 1 if on else 0)


def gf_profile_read(g) -> Profile:
    p = Profile()
    st = lib().gf_profile_read(g, C.byref(p))
    if st != GF_OK:
        raise GfError(st, "gf_profile_read")
    return p


def gf_launch_count(g) -> int:
    return int(lib().gf_launch_count(g))


def gf_debug_bounds_enabled() -> bool:
    return bool(lib().gf_debug_bounds_enabled())


def gf_debug_bounds_site(g) -> int:
    return int(lib().gf_debug_bounds_site(g))


def gf_debug_counters(g, stream=0) -> dict:
    v = (C.c_uint64 * 2)(0, 0)
    st = lib().gf_debug_counters(g, v, stream)
    if st != GF_OK:
        raise GfError(st, "gf_debug_counters")
    return {"softmax_reference_moves": int(v[0]), "exact_reruns": int(v[1])}


def gf_debug_wait_probe(g, limit_cycles: int, stream=0):
    """(status, gave_up): runs one bounded wait on a barrier nothing completes."""
    gave_up = C.c_int32(0)
    st = lib().gf_debug_wait_probe(g, int(limit_cycles), C.byref(gave_up), stream)
    return st, int(gave_up.value)


def gfgen_fill_bf16(tab_ptr, key, start, count, out_ptr, stream=0) -> int:
    return gen_lib().gfgen_fill_bf16(tab_ptr, key, start, count, out_ptr, stream)


def check(status: int, what: str) -> None:
    if status != GF_OK:
        raise GfError(status, what)
