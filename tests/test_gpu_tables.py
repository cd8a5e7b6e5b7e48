"""K1 parity: the device-built tables equal the oracle's bit for bit."""
import numpy as np
import pytest
import torch

from helpers import assert_tables_equal, oracle_tables
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu

CASES = [
    (0, {}),
    (1, {}),
    (1, dict(n_requests=48, n_nodes=96)),
    (2, {}),
    (2, dict(n_requests=12, new_len=40, root_len=200, prefix_lo=200, prefix_hi=1500, group_lo=2, group_hi=5)),
    (3, {}),
    (4, dict(layers=1)),
]
POLICIES = [None, (64, 2, 1, 3), (128, 5, 3, 1), (512, 16, 4, 8)]


def _pa(w, policy=None, size_for=(64, 1, 1, 1)):
    """A handle whose workspace is sized for the smallest chunk length any policy here uses (the
    slot bound grows as the chunks shrink), so that every policy is built and compared."""
    from paper_2605_22566_b200.runtime import PathAttention
    pa = PathAttention(w, layers=1, policy=size_for)
    pa.policy = policy
    return pa


def _register_lengths(pa):
    """Reserve every used node's extent without moving KV data: write from a scratch buffer."""
    from paper_2605_22566_b200 import binding as B
    w = pa.w
    used = w.used_nodes()
    nmax = int(w.node_len[used].max())
    buf = torch.zeros(nmax * w.num_kv_heads * w.head_dim, dtype=torch.bfloat16, device=pa.dev)
    for v in used.tolist():
        B.check(B.gf_node_kv_write(pa.g, v, 0, buf.data_ptr(), buf.data_ptr(), int(w.node_len[v]), pa.stream),
                "gf_node_kv_write")


@pytest.mark.parametrize("cfg,over", CASES)
def test_tables_bit_exact(cfg, over):
    from paper_2605_22566_b200 import binding as B
    w = W.make_config(cfg, **over)
    pa = _pa(w)
    _register_lengths(pa)
    for policy in POLICIES:
        pa.policy = policy
        info = pa.build()
        got = B.gf_tables_export(pa.tables)
        ref = oracle_tables(w, policy)
        assert_tables_equal(got, ref)
        assert info.num_items == len(ref["items"]) and info.num_pairs == len(ref["grp_req"])
    pa.close()


def test_tables_are_deterministic_run_to_run():
    from paper_2605_22566_b200 import binding as B
    w = W.make_config(3)
    pa = _pa(w)
    _register_lengths(pa)
    pa.build()
    first = B.gf_tables_export(pa.tables)
    for _ in range(9):
        pa.build()
        again = B.gf_tables_export(pa.tables)
        assert_tables_equal(again, {k: v for k, v in first.items()})
    pa.close()


def test_invalid_paths_are_reported_not_run():
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(0)
    base_ptr, base_nodes = w.path_ptr.copy(), w.path_node.copy()
    edges = set(zip(w.edge_src.tolist(), w.edge_dst.tolist()))

    def run(nodes, ptr=None, mode=B.GF_MODE_DECODE):
        pa = PathAttention(W.make_config(0), layers=1)
        _register_lengths(pa)
        pn = torch.tensor(nodes, dtype=torch.int32, device=pa.dev)
        pp = torch.tensor(base_ptr.tolist() if ptr is None else ptr, dtype=torch.int32, device=pa.dev)
        st, t = B.gf_build_path_tables(pa.g, len(pp) - 1, len(nodes), pp.data_ptr(), pn.data_ptr(),
                                       mode, None, pa.stream)
        bad = B.gf_tables_bad_request(t)
        q = torch.zeros((8, 4, 64), dtype=torch.bfloat16, device=pa.dev)
        o = torch.zeros_like(q)
        st2 = B.gf_path_attention_decode(pa.g, t, 0, q.data_ptr(), o.data_ptr(), None, pa.stream)
        torch.cuda.synchronize()
        pa.close()
        return st, bad, st2

    assert run(base_nodes.tolist()) == (B.GF_OK, -1, B.GF_OK)
    # a hop that is not a wGraph edge in request 2
    bad = base_nodes.copy()
    b2 = base_ptr[2]
    wrong = next(v for v in range(1, 16) if (int(bad[b2]), v) not in edges)
    bad[b2 + 1] = wrong
    assert run(bad.tolist()) == (B.GF_ERR_INVALID_PATH, 2, B.GF_ERR_NOT_BUILT)
    # repeated node in request 5, out-of-range id in request 6: smallest index wins
    bad = base_nodes.copy()
    bad[base_ptr[5] + 1] = bad[base_ptr[5]]
    bad[base_ptr[6]] = 9999
    assert run(bad.tolist())[:2] == (B.GF_ERR_INVALID_PATH, 5)
    bad = base_nodes.copy()
    bad[base_ptr[7]] = -3
    assert run(bad.tolist())[:2] == (B.GF_ERR_INVALID_PATH, 7)
    # an empty path (request 3)
    ptr = base_ptr.copy()
    n3 = ptr[4] - ptr[3]
    nodes = np.concatenate([base_nodes[:ptr[3]], base_nodes[ptr[4]:]])
    ptr[4:] -= n3
    assert run(nodes.tolist(), ptr.tolist())[:2] == (B.GF_ERR_INVALID_PATH, 3)


def test_zero_length_and_unwritten_nodes_are_dropped():
    from paper_2605_22566_b200 import binding as B
    w = W.make_config(4, layers=1, n_requests=200, n_nodes=400, token_budget=20000)
    assert (w.node_len[:400] == 0).sum() > 50  # control-only operations
    pa = _pa(w)
    _register_lengths(pa)
    # explicit empty write for one zero-length node; the others stay unwritten
    zero = int(np.nonzero(w.node_len[:400] == 0)[0][0])
    B.check(B.gf_node_kv_write(pa.g, zero, 0, None, None, 0, pa.stream), "empty write")
    pa.build()
    assert_tables_equal(B.gf_tables_export(pa.tables), oracle_tables(w))
    pa.close()


def test_deferred_build_matches_and_reports_late():
    """GF_MODE_DEFERRED: same tables, same decode output, errors surface at the first read-back."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(1, n_requests=40, n_nodes=64, root_len=333, len_lo=1, len_hi=200, suffix_max=70)
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    q = pa.make_q(0)
    pa.build()
    ref_tables = B.gf_tables_export(pa.tables)
    ref_out = tensor_to_f64(pa.decode(0, q))
    assert pa.build(deferred=True) is None
    out = tensor_to_f64(pa.decode(0, q))          # enqueued before anything was read back
    assert pa.status() == 0
    assert np.array_equal(out, ref_out)
    assert_tables_equal(B.gf_tables_export(pa.tables), ref_tables)
    # an invalid path: the deferred build itself says OK, decode leaves `out` alone, status reports
    bad = w.path_node.copy()
    bad[w.path_ptr[3]] = w.num_nodes + 5
    pa.path_node.copy_(torch.from_numpy(bad.astype(np.int32)))
    assert pa.build(deferred=True) is None
    canary = torch.full_like(q, 7.0)
    pa.decode(0, q, out=canary)
    assert pa.status() == B.GF_ERR_INVALID_PATH
    assert B.gf_tables_bad_request(pa.tables) == 3
    assert torch.all(canary == 7.0)
    with pytest.raises(B.GfError):
        pa.info()
    pa.close()


def _private_only_workload(n_requests, per_request, root_len=64, hq=4, hkv=4, d=64, seed=77):
    """One shared root plus `per_request` private nodes per request (ids above the shared range are not
    edge-checked): many segments without an edge list the oracle would have to search."""
    rng = np.random.default_rng(seed)
    n_nodes = 1 + n_requests * per_request
    node_len = np.zeros(n_nodes, dtype=np.int32)
    node_len[0] = root_len
    node_len[1:] = rng.integers(1, 9, size=n_nodes - 1)
    ptr, nodes = [0], []
    for r in range(n_requests):
        nodes.extend([0] + list(range(1 + r * per_request, 1 + (r + 1) * per_request)))
        ptr.append(len(nodes))
    return W.Workload(name="private-only", config_id=-2, seed=seed, mode="decode", num_layers=1, num_q_heads=hq,
                      num_kv_heads=hkv, head_dim=d, num_shared_nodes=1, num_nodes=n_nodes,
                      edge_src=np.zeros(0, np.int32), edge_dst=np.zeros(0, np.int32), node_len=node_len,
                      path_ptr=np.array(ptr, dtype=np.int32), path_node=np.array(nodes, dtype=np.int32))


def test_more_segments_than_the_item_search_caches():
    """4801 segments: the item builder searches the segments' item starts in global memory."""
    from helpers import OracleView, assert_close
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import tensor_to_f64
    w = _private_only_workload(600, 8)
    pa = _pa(w)
    pa.write_nodes("device")
    info = pa.build()
    assert info.num_segments == 4801
    assert_tables_equal(B.gf_tables_export(pa.tables), oracle_tables(w))
    out = tensor_to_f64(pa.decode(0, pa.make_q(0)))
    assert pa.status() == 0
    reqs = [0, 1, 299, 599]
    ref, _ = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref, "4801 segments")
    pa.close()


def test_more_requests_than_the_group_sort_bitmap_holds():
    """66 000 requests on one root: the group's members are sorted by rank counting, not through the
    shared-memory bitmap (which holds request ids below 65 536)."""
    from helpers import OracleView, assert_close
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import tensor_to_f64
    w = _private_only_workload(66000, 0, root_len=100)
    pa = _pa(w, size_for=None)
    pa.write_nodes("device")
    info = pa.build()
    assert info.num_segments == 1 and info.num_pairs == 66000
    assert_tables_equal(B.gf_tables_export(pa.tables), oracle_tables(w))
    out = tensor_to_f64(pa.decode(0, pa.make_q(0)))
    assert pa.status() == 0
    reqs = [0, 31, 32768, 65535, 65536, 65999]
    ref, _ = OracleView(w).decode(reqs)
    assert_close(out[reqs], ref, "66000 requests")
    assert np.all(np.isfinite(out))
    pa.close()


def test_extend_mode_rejects_more_requests_than_a_grid_dimension():
    from paper_2605_22566_b200 import binding as B
    w = W.make_config(0)
    pa = _pa(w)
    ptr = torch.zeros(65537 + 1, dtype=torch.int32, device=pa.dev)
    nodes = torch.zeros(65537, dtype=torch.int32, device=pa.dev)
    st, t = B.gf_build_path_tables(pa.g, 65537, 65537, ptr.data_ptr(), nodes.data_ptr(), B.GF_MODE_EXTEND, None,
                                   pa.stream)
    assert st == B.GF_ERR_INVALID_ARG and t is None
    pa.close()
