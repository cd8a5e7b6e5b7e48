"""Pins of the path-pruning oracle (Sec. 5.2) against things other than itself."""
import json
import os

import numpy as np

from oracle import pruning as OP
from paper_2605_22566_b200 import workloads as W


def _second_count(w):
    """Counts by another route: encode every hop between shared nodes as u * N + v and use numpy.unique."""
    N = w.num_nodes
    hops = []
    for r in range(w.num_requests):
        p = w.path(r).astype(np.int64)
        u, v = p[:-1], p[1:]
        m = (u < w.num_shared_nodes) & (v < w.num_shared_nodes)
        hops.append(u[m] * N + v[m])
    hops = np.concatenate(hops) if hops else np.zeros(0, np.int64)
    codes, cnt = np.unique(hops, return_counts=True)
    return dict(zip(codes.tolist(), cnt.tolist())), len(hops)


def test_counts_match_a_second_route_and_conserve_hops():
    for cfg in (dict(config_id=0), dict(config_id=1, n_requests=60, n_nodes=64, root_len=100, len_lo=1, len_hi=50, suffix_max=20)):
        w = W.make_config(**cfg)
        counts, misses = OP.transition_counts(w.num_shared_nodes, w.edge_src, w.edge_dst, w.path_ptr, w.path_node)
        ref, n_hops = _second_count(w)
        pairs = OP.sorted_edges(w.edge_src, w.edge_dst)
        assert misses == 0  # the generator only walks along edges
        assert int(counts.sum()) == n_hops
        for (u, v), c in zip(pairs, counts.tolist()):
            assert ref.get(u * w.num_nodes + v, 0) == c
        assert pairs == sorted(pairs) and len(pairs) == len(w.edge_src)


def test_paper_example_workflow_counted_by_hand():
    # the five-operation example workflow: edges 01->02, 01->03, 02->04, 03->04, 04->05 (ids 0..4 here)
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "paper_workflow_example.json")))
    src = [e[0] for e in g["edges"]]
    dst = [e[1] for e in g["edges"]]
    # three executions: twice through 02, once through 03, and one that stops at 04
    paths = [[0, 1, 3, 4], [0, 1, 3, 4], [0, 2, 3, 4], [0, 2, 3]]
    ptr = np.cumsum([0] + [len(p) for p in paths]).astype(np.int32)
    node = np.array([v for p in paths for v in p], dtype=np.int32)
    counts, misses = OP.transition_counts(g["nodes"], src, dst, ptr, node)
    pairs = OP.sorted_edges(src, dst)
    by_edge = dict(zip(pairs, counts.tolist()))
    assert by_edge == {(0, 1): 2, (0, 2): 2, (1, 3): 2, (2, 3): 2, (3, 4): 3} and misses == 0
    keep, kept, covered, total = OP.select_transitions(counts, 3)
    assert keep.tolist() == [False, False, False, False, True] and (kept, covered, total) == (1, 3, 11)
    # a hop that is not an edge is a miss; hops through a private node (id >= 5) are not transitions
    counts2, misses2 = OP.transition_counts(g["nodes"], src, dst, np.array([0, 3, 6]), np.array([0, 3, 4, 1, 7, 2]))
    assert misses2 == 1 and by_edge_sum(counts2) == 1


def by_edge_sum(c):
    return int(np.asarray(c).sum())


def test_selection_is_monotone_and_min_count_one_keeps_the_edges_taken():
    w = W.make_config(1, n_requests=80, n_nodes=96, root_len=64, len_lo=1, len_hi=32, suffix_max=8)
    counts, _ = OP.transition_counts(w.num_shared_nodes, w.edge_src, w.edge_dst, w.path_ptr, w.path_node)
    prev = None
    for m in (0, 1, 2, 5, 20, 10 ** 9):
        keep, kept, covered, total = OP.select_transitions(counts, m)
        assert kept == int(keep.sum()) and covered <= total == int(counts.sum())
        if prev is not None:
            assert not np.any(keep & ~prev)  # a larger threshold never adds an edge
        prev = keep
    keep1, *_ = OP.select_transitions(counts, 1)
    assert np.array_equal(keep1, counts > 0)
    assert OP.select_transitions(counts, 0)[1] == len(counts) and OP.select_transitions(counts, 10 ** 9)[1] == 0
