"""gf_edge_scores (Sec. 4.2: graph convolutional encoder + perceptron over the task-conditioned graph)
against the fp64 oracle.  Everything on the device is fp32 with sums of up to 768 terms of O(1/sqrt(n))
size, so embeddings agree to about 1e-5 relative and the scores, which lie in (0, 1), to 1e-4 absolute."""
import json
import os

import numpy as np
import pytest

from oracle import scoring as OS
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu
TOL = 1e-4


def _oracle(w, inp):
    return OS.edge_scores(inp["x_op"], inp["x_task"], w.edge_src, w.edge_dst, inp["w_gcn1"], inp["w_gcn2"], inp["w1"],
                          inp["b1"], inp["w2"], inp["b2"], inp["w3"], float(inp["b3"]))


def _check_edge_order(w):
    # scores come in ascending (source, destination) order, which is how the workloads list their edges
    key = w.edge_src.astype(np.int64) * (1 << 32) + w.edge_dst
    assert np.all(np.diff(key) > 0)


@pytest.mark.parametrize("cfg,over,dims,tasks,per_pass", [
    (0, {}, (384, 256, 128), 5, None),
    (1, dict(n_requests=8, n_nodes=70), (48, 40, 32), 7, 3),
    (3, dict(n_requests=8, n_nodes=150), (384, 256, 128), 3, 2),
    (0, {}, (17, 9, 64), 1, None),
])
def test_edge_scores_match_the_oracle(cfg, over, dims, tasks, per_pass):
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(cfg, **over)
    _check_edge_order(w)
    inp = W.scoring_inputs(w.seed, w.num_shared_nodes, tasks, *dims)
    pa = PathAttention(w, layers=1)
    got = pa.edge_scores(inp, per_pass).cpu().numpy().astype(np.float64)
    assert pa.status() == 0
    ref = _oracle(w, inp)
    assert got.shape == ref.shape and np.all(np.isfinite(got))
    assert np.abs(got - ref).max() < TOL, float(np.abs(got - ref).max())
    assert ref.std() > 1e-3   # the scores are not all alike: the comparison says something
    pa.close()


def test_hand_worked_path_graph_on_the_device():
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    g = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "scoring_path_graph.json")))
    w = W.make_config(0)
    w.num_shared_nodes, w.num_nodes = 3, 3 + w.num_requests
    w.edge_src = np.array([e[0] for e in g["edges"]], dtype=np.int32)
    w.edge_dst = np.array([e[1] for e in g["edges"]], dtype=np.int32)
    w.node_len = np.concatenate([[8, 8, 8], np.zeros(w.num_requests, np.int32)]).astype(np.int32)
    w.path_ptr = np.arange(w.num_requests + 1, dtype=np.int32)
    w.path_node = np.zeros(w.num_requests, dtype=np.int32)
    m = g["mlp"]
    # one feature and one hidden unit, padded to the perceptron width the kernel supports (32): the
    # extra units have zero weights and biases and change nothing
    dm = 32
    w1 = np.zeros((3, dm), np.float32); w1[:, 0] = np.array(m["w1"])[:, 0]
    b1 = np.zeros(dm, np.float32); b1[0] = m["b1"][0]
    w2 = np.zeros((dm, dm), np.float32); w2[0, 0] = m["w2"][0][0]
    b2 = np.zeros(dm, np.float32); b2[0] = m["b2"][0]
    w3 = np.zeros(dm, np.float32); w3[0] = m["w3"][0]
    inp = {"x_op": np.array(g["x_op"], np.float32), "x_task": np.array(g["x_task"], np.float32),
           "w_gcn1": np.array(g["w_gcn1"], np.float32), "w_gcn2": np.array(g["w_gcn2"], np.float32),
           "w1": w1, "b1": b1, "w2": w2, "b2": b2, "w3": w3, "b3": np.float32(m["b3"])}
    pa = PathAttention(w, layers=1)
    got = pa.edge_scores(inp).cpu().numpy().astype(np.float64)
    ref = OS.edge_scores(g["x_op"], g["x_task"], w.edge_src, w.edge_dst, g["w_gcn1"], g["w_gcn2"], np.array(m["w1"]),
                         np.array(m["b1"]), np.array(m["w2"]), np.array(m["b2"]), np.array(m["w3"]), m["b3"])
    assert np.abs(got - ref).max() < 1e-6
    bad = B.Scorer(1, 1, 48, 1, 1, 1, 1, 1, 1, 1, 0.0)   # a perceptron width the kernel does not take
    assert B.gf_edge_scores(pa.g, bad, 16, 1, 16, 16, 16, 1 << 20, pa.stream) == B.GF_ERR_INVALID_ARG
    pa.close()
