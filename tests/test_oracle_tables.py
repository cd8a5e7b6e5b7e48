"""Pins for the table oracle: the paper's example workflow worked by hand, brute-force
set semantics, counting / coverage invariants, closed-form memory ratios, validation."""
import json
import os

import numpy as np
import pytest

from oracle import tables as OT
from paper_2605_22566_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_workflow_example.json")


def _build(w, policy=OT.Policy(), mode=None, write_order=None):
    order = list(range(w.num_nodes)) if write_order is None else write_order
    off, _ = OT.pool_offsets([v for v in order if w.node_len[v] > 0], w.node_len, w.num_nodes)
    mode = (OT.MODE_EXTEND if w.mode == "extend" else OT.MODE_DECODE) if mode is None else mode
    return OT.build_tables(w.num_nodes, w.num_shared_nodes, w.edge_src, w.edge_dst, w.node_len, off,
                           w.path_ptr, w.path_node, policy, mode)


def test_paper_example_workflow_by_hand():
    g = json.load(open(GOLDEN))
    src = [e[0] for e in g["edges"]]
    dst = [e[1] for e in g["edges"]]
    ptr, nodes = [0], []
    for p in g["paths"]:
        nodes += p
        ptr.append(len(nodes))
    for case in g["cases"]:
        node_len = np.array(case["node_len"], dtype=np.int32)
        off, _ = OT.pool_offsets(range(g["nodes"]), node_len, g["nodes"])
        t = OT.build_tables(g["nodes"], g["nodes"], src, dst, node_len, off, np.array(ptr), np.array(nodes),
                            OT.Policy(**case["policy"]), OT.MODE_DECODE)
        assert t["bad_req"] == -1
        for key in ["seg_node", "seg_len", "seg_off", "grp_ptr", "grp_req", "req_len", "req_nseg",
                    "mrg_ptr", "mrg_slot", "pseg_ptr", "pseg"]:
            assert t[key].tolist() == case[key], (case["name"], key)
        assert t["items"].tolist() == case["items"], case["name"]
        for key in ["resident_tokens", "materialised_tokens", "num_slots"]:
            assert t[key] == case[key], (case["name"], key)
        # materialised / resident = 8/5 when all five segments have equal length
        if len(set(case["node_len"])) == 1:
            assert t["materialised_tokens"] * 5 == t["resident_tokens"] * 8


@pytest.mark.parametrize("cfg,over", [(0, {}), (1, dict(n_requests=48, n_nodes=96)),
                                      (3, dict(n_requests=64, n_nodes=128, root_len=700)),
                                      (4, dict(n_requests=80, n_nodes=300, token_budget=30000, layers=2)),
                                      (2, dict(n_requests=12, new_len=40, root_len=200, prefix_lo=200,
                                               prefix_hi=1500, group_lo=2, group_hi=5))])
@pytest.mark.parametrize("policy", [OT.Policy(), OT.Policy(64, 2, 1, 3), OT.Policy(128, 5, 3, 1)])
def test_invariants_on_configs(cfg, over, policy):
    w = W.make_config(cfg, **over)
    t = _build(w, policy)
    assert t["bad_req"] == -1
    R = w.num_requests
    S = len(t["seg_node"])
    # T1 against a second route, plain loops: a flag per node id, raised by every path that names it
    on_a_path = [False] * w.num_nodes
    for v in w.path_node.tolist():
        on_a_path[v] = True
    expect_nodes = [v for v in range(w.num_nodes) if on_a_path[v] and int(w.node_len[v]) > 0]
    assert t["seg_node"].tolist() == expect_nodes
    assert np.all(np.diff(t["seg_node"]) > 0)
    assert np.all(t["seg_off"] % 64 == 0)
    # extents must not overlap
    order = np.argsort(t["seg_off"])
    ends = t["seg_off"][order] + t["seg_len"][order]
    assert np.all(ends[:-1] <= t["seg_off"][order][1:])
    # T2 brute force: membership matrix
    member = np.zeros((S, R), dtype=bool)
    for r in range(R):
        for v in w.path(r):
            if w.node_len[v] > 0:
                member[np.searchsorted(t["seg_node"], v), r] = True
    for s in range(S):
        grp = t["grp_req"][t["grp_ptr"][s]:t["grp_ptr"][s + 1]]
        assert grp.tolist() == np.nonzero(member[s])[0].tolist()
    # counting invariant: sum_r L_r = sum_s len_s * |group_s|
    gsz = np.diff(t["grp_ptr"]).astype(np.int64)
    assert t["materialised_tokens"] == int((t["seg_len"].astype(np.int64) * gsz).sum())
    # totals by plain loops over the paths (what per-request caching would hold) and over the used nodes
    expect_req_len = []
    for r in range(R):
        total = 0
        for v in w.path_node[w.path_ptr[r]:w.path_ptr[r + 1]].tolist():
            total += int(w.node_len[v])
        expect_req_len.append(total)
    assert t["req_len"].tolist() == expect_req_len
    assert t["materialised_tokens"] == sum(expect_req_len)
    assert t["resident_tokens"] == sum(int(w.node_len[v]) for v in expect_nodes)
    # coverage: items tile every (segment token range x group) exactly once
    cover = {}
    part = 0
    prev_key = None
    for (s, tb, tc, gb, gc, pb) in t["items"].tolist():
        assert pb == part
        part += gc
        assert tc > 0 and gc > 0 and gc <= policy.group_tile
        assert tb % 64 == 0
        key = (s, tb, gb)
        assert prev_key is None or key > prev_key
        prev_key = key
        assert t["grp_ptr"][s] <= gb and gb + gc <= t["grp_ptr"][s + 1]
        for gi in range(gb, gb + gc):
            c = cover.setdefault((s, gi), np.zeros(t["seg_len"][s], dtype=np.int32))
            assert tb + tc <= len(c)
            c[tb:tb + tc] += 1
    assert part == t["num_slots"]
    assert len(cover) == len(t["grp_req"])
    assert all(np.all(c == 1) for c in cover.values())
    # merge map: request r's slots are exactly the (item, position) pairs that hold r
    owner = np.full(t["num_slots"], -1)
    tokens_in_slot = np.zeros(t["num_slots"], dtype=np.int64)
    for (s, tb, tc, gb, gc, pb) in t["items"].tolist():
        owner[pb:pb + gc] = t["grp_req"][gb:gb + gc]
        tokens_in_slot[pb:pb + gc] = tc
    for r in range(R):
        sl = t["mrg_slot"][t["mrg_ptr"][r]:t["mrg_ptr"][r + 1]]
        assert np.all(np.diff(sl) > 0)
        assert sl.tolist() == np.nonzero(owner == r)[0].tolist()
        assert tokens_in_slot[sl].sum() == t["req_len"][r]
    # T7
    for r in range(R):
        ps = t["pseg"][t["pseg_ptr"][r]:t["pseg_ptr"][r + 1]]
        assert t["seg_node"][ps].tolist() == [v for v in w.path(r) if w.node_len[v] > 0]
        assert len(ps) == t["req_nseg"][r]
    if w.mode == "extend":
        assert t["q_ptr"].tolist() == w.q_row_ptr().tolist()
        assert t["seg_node"][t["self_seg"]].tolist() == [int(w.path(r)[-1]) for r in range(R)]


def test_memory_ratio_closed_forms():
    # no sharing: every request has its own nodes -> materialised == resident
    R, d = 5, 3
    n = R * d
    node_len = np.arange(10, 10 + n, dtype=np.int32)
    ptr = np.arange(0, n + 1, d)
    nodes = np.arange(n)
    off, _ = OT.pool_offsets(range(n), node_len, n)
    t = OT.build_tables(n, 0, [], [], node_len, off, ptr, nodes)
    assert t["bad_req"] == -1 and t["materialised_tokens"] == t["resident_tokens"] == int(node_len.sum())
    # all paths identical: ratio = R
    src, dst = [0, 1], [1, 2]
    node_len = np.array([70, 33, 129], dtype=np.int32)
    off, _ = OT.pool_offsets(range(3), node_len, 3)
    t = OT.build_tables(3, 3, src, dst, node_len, off, np.arange(0, 3 * R + 1, 3), np.tile([0, 1, 2], R))
    assert t["materialised_tokens"] == R * t["resident_tokens"]
    assert np.diff(t["grp_ptr"]).tolist() == [R, R, R]


def test_zero_length_nodes_are_dropped():
    node_len = np.array([64, 0, 40, 0], dtype=np.int32)
    off, total = OT.pool_offsets([0, 2], node_len, 4)
    assert total == 128 and off.tolist() == [0, -1, 64, -1]
    t = OT.build_tables(4, 3, [0, 1], [1, 2], node_len, off, np.array([0, 3, 5]), np.array([0, 1, 2, 0, 3]))
    assert t["bad_req"] == -1
    assert t["seg_node"].tolist() == [0, 2]
    assert t["req_len"].tolist() == [104, 64] and t["req_nseg"].tolist() == [2, 1]
    assert t["pseg"].tolist() == [0, 1, 0]


def test_validation_reports_smallest_bad_request():
    src, dst = [0, 0, 1], [1, 2, 3]
    node_len = np.array([10, 10, 10, 10, 5, 0], dtype=np.int32)
    off, _ = OT.pool_offsets(range(6), node_len, 6)

    def bad(paths, mode=OT.MODE_DECODE):
        ptr, nodes = [0], []
        for p in paths:
            nodes += p
            ptr.append(len(nodes))
        return OT.build_tables(6, 4, src, dst, node_len, off, np.array(ptr), np.array(nodes, dtype=np.int64),
                               OT.Policy(), mode)["bad_req"]

    assert bad([[0, 1, 3], [0, 2], [0, 1, 4]]) == -1          # hop into private node 4 is exempt
    assert bad([[0, 1, 3], [0, 3]]) == 1                      # 0->3 is not an edge
    assert bad([[0, 1], [1, 0]]) == 1                         # reversed edge
    assert bad([[0, 1, 0]]) == 0                              # repeated node
    assert bad([[0, 1], [0, 6]]) == 1                         # id out of range
    assert bad([[0, 1], [0, -1]]) == 1
    assert bad([[0, 2], []]) == 1                             # empty path
    assert bad([[0, 7], [0, 3]]) == 0                         # smallest index wins
    assert bad([[0, 1, 4]], OT.MODE_EXTEND) == -1
    assert bad([[0, 1, 5]], OT.MODE_EXTEND) == 0              # new node has no tokens
