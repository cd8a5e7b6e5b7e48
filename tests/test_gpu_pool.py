"""The evictable pool and the on-the-fly branch (Sec. 5.2): extents that are released and reused, and
an extend that appends the new segments' K/V while it attends."""
import json
import os

import numpy as np
import pytest
import torch

from helpers import OracleView, assert_close, assert_tables_equal
from oracle import tables as OT
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "pool_release_sequence.json")


def _small_handle(capacity_tiles, num_nodes=16, hq=4, hkv=2, d=64, layers=2):
    from paper_2605_22566_b200 import binding as B
    pool_bytes = capacity_tiles * B.gf_pool_bytes_per_tile(d) * hkv * layers
    raw = torch.empty(pool_bytes + 1024, dtype=torch.uint8, device="cuda:0")
    skew = (-raw.data_ptr()) % 1024
    ws_bytes = B.gf_workspace_bytes(num_nodes, 0, 4, 16, 64, 64, hq, d)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device="cuda:0")
    st, g = B.gf_wgraph_create(num_nodes=num_nodes, num_shared_nodes=0, edge_src=np.zeros(0, np.int32),
                               edge_dst=np.zeros(0, np.int32), num_layers=layers, num_q_heads=hq, num_kv_heads=hkv,
                               head_dim=d, kv_pool_ptr=raw.data_ptr() + skew, kv_pool_bytes=pool_bytes,
                               workspace_ptr=ws.data_ptr(), workspace_bytes=ws_bytes)
    B.check(st, "gf_wgraph_create")
    return g, (raw, ws)


def test_hand_worked_release_sequence_through_the_abi():
    from paper_2605_22566_b200 import binding as B
    gold = json.load(open(GOLDEN))
    g, keep = _small_handle(gold["capacity_tiles"])
    model = OT.PoolModel(gold["capacity_tiles"])
    for step in gold["steps"]:
        if step["op"] == "reserve":
            st = B.gf_node_kv_reserve(g, step["node"], step["tokens"])
            assert model.reserve(step["node"], step["tokens"]) == step["offset"]
            if step["offset"] is None:
                assert st == B.GF_ERR_CAPACITY, step
                assert B.gf_node_extent(g, step["node"])[0] == B.GF_ERR_NOT_WRITTEN
            else:
                assert st == B.GF_OK, step
                assert B.gf_node_extent(g, step["node"]) == (B.GF_OK, step["tokens"], step["offset"]), step
        else:
            assert B.gf_node_kv_release(g, step["node"]) == B.GF_OK
            model.release(step["node"])
            assert B.gf_node_extent(g, step["node"])[0] == B.GF_ERR_NOT_WRITTEN
        info = B.gf_pool_info(g)
        assert (info.tiles_in_use, info.high_water_tiles) == (model.tiles_in_use(), model.high_water()), step
    assert B.gf_pool_info(g).tiles_in_use == gold["final_tiles_in_use"]
    assert B.gf_node_kv_release(g, 1) == B.GF_ERR_NOT_WRITTEN       # released long ago
    assert B.gf_node_kv_release(g, 99) == B.GF_ERR_INVALID_ARG
    torch.cuda.synchronize()
    B.gf_wgraph_destroy(g)


def test_random_reserve_release_matches_the_model():
    from paper_2605_22566_b200 import binding as B
    rng = np.random.default_rng(21)
    cap, nodes = 40, 64
    g, keep = _small_handle(cap, num_nodes=nodes)
    model = OT.PoolModel(cap)
    live = set()
    for _ in range(400):
        if live and rng.random() < 0.45:
            v = int(rng.choice(sorted(live)))
            assert B.gf_node_kv_release(g, v) == B.GF_OK
            model.release(v)
            live.remove(v)
        else:
            free = [v for v in range(nodes) if v not in live]
            if not free:
                continue
            v, n = int(rng.choice(free)), int(rng.integers(0, 7 * 64))
            want = model.reserve(v, n)
            st = B.gf_node_kv_reserve(g, v, n)
            if want is None:
                assert st == B.GF_ERR_CAPACITY
            else:
                assert B.gf_node_extent(g, v) == (B.GF_OK, n, want)
                live.add(v)
        info = B.gf_pool_info(g)
        assert (info.tiles_in_use, info.high_water_tiles) == (model.tiles_in_use(), model.high_water())
    torch.cuda.synchronize()
    B.gf_wgraph_destroy(g)


def test_released_tiles_are_reused_and_the_new_occupant_is_what_attention_sees():
    """Write every node, release some shared ones, write others of different lengths into the holes:
    the tables (offsets included) match the oracle built from the pool model, and decode over the new
    layout matches the oracle's attention."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(1, n_requests=40, n_nodes=64, root_len=333, len_lo=1, len_hi=200, suffix_max=70)
    pa = PathAttention(w, layers=1, extra_tiles=200)  # room for the fragmentation first fit leaves
    used = w.used_nodes().tolist()
    model = OT.PoolModel(B.gf_pool_info(pa.g).capacity_tiles)
    pa.write_nodes("device")
    for v in used:
        model.reserve(v, int(w.node_len[v]))
    # drop every third used node, then give them back in reverse order (different holes for most)
    victims = used[1::3]
    for v in victims:
        assert B.gf_node_kv_release(pa.g, v, pa.stream) == B.GF_OK
        model.release(v)
    with pytest.raises(B.GfError):  # the tables were stale anyway; and a released node on a path is an empty one
        pa.decode(0, pa.make_q(0))
    per_tok = w.num_kv_heads * w.head_dim
    for v in reversed(victims):
        kb, vb = w.node_kv_bits(0, v)
        kt = torch.from_numpy(kb.view(np.int16)).to(pa.dev).view(torch.bfloat16)
        vt = torch.from_numpy(vb.view(np.int16)).to(pa.dev).view(torch.bfloat16)
        B.check(B.gf_node_kv_write(pa.g, v, 0, kt.data_ptr(), vt.data_ptr(), int(w.node_len[v]), pa.stream), "rewrite")
        torch.cuda.synchronize()
        assert model.reserve(v, int(w.node_len[v])) is not None
    for v in used:
        assert B.gf_node_extent(pa.g, v) == (B.GF_OK, int(w.node_len[v]), model.extent[v][0] * 64)
    pa.build()
    off = np.full(w.num_nodes, -1, dtype=np.int64)
    for v in used:
        off[v] = model.extent[v][0] * 64
    ref = OT.build_tables(w.num_nodes, w.num_shared_nodes, w.edge_src, w.edge_dst, w.node_len, off, w.path_ptr,
                          w.path_node, OT.Policy(), OT.MODE_DECODE)
    assert_tables_equal(B.gf_tables_export(pa.tables), ref)
    out = tensor_to_f64(pa.decode(0, pa.make_q(0)))
    assert pa.status() == 0
    ref_o, _ = OracleView(w).decode()
    assert_close(out, ref_o, "decode after release and reuse")
    pa.close()


def _append_case(peaked):
    w = W.make_config(2, n_requests=6, new_len=200, root_len=300, len_lo=150, len_hi=400, prefix_lo=600,
                      prefix_hi=1500, group_lo=2, group_hi=3)
    if peaked:
        w.q_scale_log2, w.v_scale_log2 = 3, -2
        qp = w.q_row_ptr()
        w.planted = tuple((int(qp[r]) + 180, (5 * r + 2) % w.num_q_heads, int(w.path(r)[-1]), 140, 0)
                          for r in range(w.num_requests))
    return w


@pytest.mark.parametrize("peaked", [False, True])
def test_extend_append_matches_the_oracle_and_leaves_the_segments_in_the_pool(peaked):
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = _append_case(peaked)
    pa = PathAttention(w, layers=1)
    pa.write_prefix_nodes("device")     # the new segments are reserved, not written
    pa.build()
    q = pa.make_q(0)
    k_new, v_new = pa.new_kv(0)
    lse = torch.empty(q.shape[:2], dtype=torch.float32, device=pa.dev)
    out = pa.extend_append(0, q, k_new, v_new, lse=lse)
    assert pa.status() == 0
    ref_o, ref_l = OracleView(w).extend()
    assert_close(tensor_to_f64(out), ref_o, "extend with append")
    assert np.abs(tensor_to_f64(lse) - ref_l).max() < 2e-3 + 2e-6 * np.abs(ref_l).max()
    # afterwards the nodes hold exactly the appended K/V, and a plain extend over them agrees bit for bit
    for v in pa.new_nodes():
        kb, vb = w.node_kv_bits(0, v)
        got_k, got_v = pa.read_node(v, 0)
        assert np.array_equal(got_k, kb) and np.array_equal(got_v, vb)
    again = pa.extend(0, q)
    assert pa.status() == 0
    assert torch.equal(again.view(torch.int16), out.view(torch.int16))
    # a second append (same launch shape, counters re-armed) gives the same result
    out2 = pa.extend_append(0, q, k_new, v_new)
    assert pa.status() == 0
    assert torch.equal(out2.view(torch.int16), out.view(torch.int16))
    pa.close()


def test_extend_append_ragged_new_segments_and_config2_shape_sampled():
    """New segments of different lengths (1..150 tokens: partial tiles, writer jobs without work), then
    the benchmark's shape with sampled rows."""
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(2, n_requests=7, new_len=150, root_len=200, len_lo=20, len_hi=120, prefix_lo=300,
                      prefix_hi=900, group_lo=2, group_hi=3, hq=8, hkv=2, d=64)
    w.node_len = w.node_len.copy()
    for r, n in enumerate([1, 150, 64, 65, 7, 128, 100]):
        w.node_len[int(w.path(r)[-1])] = n
    pa = PathAttention(w, layers=1)
    pa.write_prefix_nodes("device")
    pa.build()
    q = pa.make_q(0)
    out = pa.extend_append(0, q, *pa.new_kv(0))
    assert pa.status() == 0
    ref_o, _ = OracleView(w).extend()
    assert_close(tensor_to_f64(out), ref_o, "append, ragged new segments")
    pa.close()

    w = W.make_config(2)
    pa = PathAttention(w, layers=1)
    pa.write_prefix_nodes("device")
    pa.build()
    q = pa.make_q(0)
    out = tensor_to_f64(pa.extend_append(0, q, *pa.new_kv(0)))
    assert pa.status() == 0
    rows = sorted(set(np.random.default_rng(6).choice(int(w.q_row_ptr()[-1]), size=16, replace=False).tolist()) | {0, 511})
    ref_o, _ = OracleView(w).extend(rows=rows)
    assert_close(out[rows], ref_o[rows], "append, config 2 sampled rows")
    assert np.all(np.isfinite(out))
    pa.close()
