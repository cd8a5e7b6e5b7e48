"""The C-ABI library builds, loads, exports every symbol the header declares, and rejects bad
arguments on the host before touching the device.  No GPU needed."""
import ctypes as C
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    from paper_2605_22566_b200 import build
    build.build()
    from paper_2605_22566_b200 import binding
    binding.lib()
    return binding


def test_every_declared_symbol_is_exported(B):
    hdr = open(os.path.join(ROOT, "include", "gf.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    declared = set(re.findall(r"\b(gf_[a-z_0-9]+)\s*\(", hdr))
    assert declared >= {"gf_wgraph_create", "gf_node_kv_write", "gf_build_path_tables",
                        "gf_path_attention_decode", "gf_path_attention_extend"}
    for name in declared:
        assert hasattr(B.lib(), name), name
    assert declared == set(B.EXPORTS)
    assert hasattr(B.gen_lib(), "gfgen_fill_bf16")


def test_host_side_argument_errors(B):
    L = B.lib()
    assert B.status_string(B.GF_OK) == "ok" and "path" in B.status_string(B.GF_ERR_INVALID_PATH)
    assert B.gf_pool_bytes_per_tile(128) == 32768 and B.gf_pool_bytes_per_tile(64) == 16384
    assert B.gf_workspace_bytes(100, 10, 8, 64, 64, 64, 32, 128) > 64 * 32 * 130 * 4
    h = C.c_void_p()
    assert L.gf_wgraph_create(None, C.byref(h)) == B.GF_ERR_INVALID_ARG
    good = dict(num_nodes=4, num_shared_nodes=3, edge_src=[0, 1], edge_dst=[1, 2], num_layers=1,
                num_q_heads=4, num_kv_heads=2, head_dim=64, kv_pool_ptr=1 << 20, kv_pool_bytes=1 << 20,
                workspace_ptr=1 << 21, workspace_bytes=1 << 20)

    def create(**over):
        st, hnd = B.gf_wgraph_create(**{**good, **over})
        assert hnd is None
        return st

    assert create(head_dim=96) == B.GF_ERR_INVALID_ARG
    assert create(num_q_heads=5) == B.GF_ERR_INVALID_ARG
    assert create(num_shared_nodes=5) == B.GF_ERR_INVALID_ARG
    assert create(kv_pool_ptr=(1 << 20) + 16) == B.GF_ERR_INVALID_ARG
    assert create(workspace_ptr=0) == B.GF_ERR_INVALID_ARG
    assert create(softmax_scale=-1.0) == B.GF_ERR_INVALID_ARG
    assert create(edge_src=[0, 1, 2], edge_dst=[1, 2, 0]) == B.GF_ERR_INVALID_GRAPH   # cycle
    assert create(edge_src=[0, 1], edge_dst=[1, 3]) == B.GF_ERR_INVALID_GRAPH         # private endpoint
    assert create(edge_src=[1], edge_dst=[1]) == B.GF_ERR_INVALID_GRAPH               # self loop
    assert create(kv_pool_bytes=1024) == B.GF_ERR_CAPACITY
    # null handles
    assert B.gf_node_kv_write(None, 0, 0, None, None, 0) == B.GF_ERR_INVALID_ARG
    st, t = B.gf_build_path_tables(None, 1, 1, 16, 16, 0)
    assert st == B.GF_ERR_INVALID_ARG and t is None
    assert B.gf_path_attention_decode(None, None, 0, 16, 16) == B.GF_ERR_INVALID_ARG
    assert B.gf_path_attention_extend(None, None, 0, 16, 16) == B.GF_ERR_INVALID_ARG
    assert B.gf_last_status(None) == B.GF_ERR_INVALID_ARG
    assert B.gf_tables_bad_request(None) == -1 and B.gf_launch_count(None) == 0
