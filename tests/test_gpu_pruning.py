"""Effective path pruning (Sec. 5.2) through the C ABI: transition counts and the kept set, bit-exact."""
import numpy as np
import pytest
import torch

from oracle import pruning as OP
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run(w, path_ptr, path_node, min_counts):
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    pa = PathAttention(w, layers=1)
    dev = pa.dev
    E = len(w.edge_src)
    ptr = torch.from_numpy(np.asarray(path_ptr, dtype=np.int32)).to(dev)
    node = torch.from_numpy(np.asarray(path_node, dtype=np.int32)).to(dev)
    counts = torch.full((max(E, 1),), -7, dtype=torch.int32, device=dev)
    misses = torch.full((1,), -1, dtype=torch.int64, device=dev)
    B.check(B.gf_transition_counts(pa.g, len(path_ptr) - 1, len(path_node), ptr.data_ptr(), node.data_ptr(),
                                   counts.data_ptr(), misses.data_ptr(), pa.stream), "gf_transition_counts")
    sel = {}
    for m in min_counts:
        keep = torch.full((max(E, 1),), 9, dtype=torch.uint8, device=dev)
        totals = torch.full((3,), -1, dtype=torch.int64, device=dev)
        B.check(B.gf_select_transitions(pa.g, counts.data_ptr(), m, keep.data_ptr(), totals.data_ptr(), pa.stream),
                "gf_select_transitions")
        torch.cuda.synchronize()
        sel[m] = (keep[:E].cpu().numpy().astype(bool), [int(x) for x in totals.cpu().numpy()])
    torch.cuda.synchronize()
    assert pa.status() == 0
    res = counts[:E].cpu().numpy().astype(np.int64), int(misses.item()), sel
    pa.close()
    return res


def _check(w, path_ptr, path_node, min_counts=(0, 1, 2, 5, 1000)):
    counts, misses, sel = _run(w, path_ptr, path_node, min_counts)
    ref_c, ref_m = OP.transition_counts(w.num_shared_nodes, w.edge_src, w.edge_dst, path_ptr, path_node)
    assert np.array_equal(counts, ref_c) and misses == ref_m
    for m in min_counts:
        keep, kept, covered, total = OP.select_transitions(ref_c, m)
        assert np.array_equal(sel[m][0], keep) and sel[m][1] == [kept, covered, total]
    return counts


@pytest.mark.parametrize("cfg", [dict(config_id=0),
                                 dict(config_id=1, n_requests=60, n_nodes=64, root_len=100, len_lo=1, len_hi=50, suffix_max=20),
                                 dict(config_id=3)])
def test_counts_and_selection_match_the_oracle(cfg):
    w = W.make_config(**cfg)
    c = _check(w, w.path_ptr, w.path_node)
    assert c.sum() > 0


def test_more_edges_than_private_bins_and_a_repeated_trace():
    # config 4's graph has more edges than a CTA's private histogram has bins: both kinds of bin are used;
    # the trace is the batch three times over (counts triple)
    w = W.make_config(4)
    assert len(w.edge_src) > 8192
    reps = 3
    node = np.tile(w.path_node, reps)
    lens = np.diff(w.path_ptr)
    ptr = np.concatenate([[0], np.cumsum(np.tile(lens, reps))]).astype(np.int32)
    c3 = _check(w, ptr, node, min_counts=(1, 4, 50))
    c1, _ = OP.transition_counts(w.num_shared_nodes, w.edge_src, w.edge_dst, w.path_ptr, w.path_node)
    assert np.array_equal(c3, 3 * c1)


def test_misses_private_hops_and_empty_input():
    w = W.make_config(0)
    pairs = OP.sorted_edges(w.edge_src, w.edge_dst)
    u, v = pairs[0]
    non_edge = next((a, b) for a in range(w.num_shared_nodes) for b in range(w.num_shared_nodes)
                    if a != b and (a, b) not in set(pairs))
    priv = w.num_shared_nodes  # a private id
    paths = [[u, v], [non_edge[0], non_edge[1]], [u, priv, v], [v]]
    ptr = np.cumsum([0] + [len(p) for p in paths]).astype(np.int32)
    node = np.array([x for p in paths for x in p], dtype=np.int32)
    c = _check(w, ptr, node, min_counts=(1,))
    assert c.sum() == 1
    _check(w, np.zeros(1, np.int32), np.zeros(0, np.int32), min_counts=(0, 1))
