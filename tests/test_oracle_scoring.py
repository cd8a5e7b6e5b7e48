"""Pins for the edge-scoring oracle (graph convolutional encoder + perceptron, Sec. 4.2)."""
import json
import os

import numpy as np
import torch

from oracle import scoring as OS

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "scoring_path_graph.json")


def _random_model(rng, d_in, d_h, d_m):
    return dict(w_gcn1=rng.normal(size=(d_in, d_h)) / np.sqrt(d_in), w_gcn2=rng.normal(size=(d_h, d_h)) / np.sqrt(d_h),
                w1=rng.normal(size=(3 * d_h, d_m)) / np.sqrt(3 * d_h), b1=0.1 * rng.normal(size=d_m),
                w2=rng.normal(size=(d_m, d_m)) / np.sqrt(d_m), b2=0.1 * rng.normal(size=d_m),
                w3=rng.normal(size=d_m) / np.sqrt(d_m), b3=0.05)


def test_hand_worked_path_graph():
    g = json.load(open(GOLDEN))
    src = [e[0] for e in g["edges"]]
    dst = [e[1] for e in g["edges"]]
    nb = OS.neighbourhoods(g["ops"], src, dst)
    assert [sorted(s) for s in nb] == [[1, 3], [0, 2, 3], [1, 3], [0, 1, 2]]
    H0 = np.array(g["x_op"] + g["x_task"], dtype=np.float64)
    H1 = OS.gcn_layer(H0, nb, np.array(g["w_gcn1"]))
    assert np.allclose(H1[:, 0], g["layer1"]["values"], rtol=0, atol=1e-14)
    r12 = np.sqrt(12.0)   # the same numbers from the hand-written sums
    assert np.allclose(H1[:, 0], [1 / 3 + 6 / r12, 1.5 + 4 / r12, 1 + 6 / r12, 1.5 + 4 / r12], rtol=0, atol=1e-14)
    H2 = OS.gcn_layer(H1, nb, np.array(g["w_gcn2"]))
    m = g["mlp"]
    got = OS.edge_scores(g["x_op"], g["x_task"], src, dst, g["w_gcn1"], g["w_gcn2"], np.array(m["w1"]), np.array(m["b1"]),
                         np.array(m["w2"]), np.array(m["b2"]), np.array(m["w3"]), m["b3"])
    for e, (i, j) in enumerate(g["edges"]):
        inner = max(H2[i, 0] - H2[j, 0] + 0.5 * H2[3, 0] + 0.25, 0.0)
        logit = 0.5 * max(2.0 * inner - 1.0, 0.0) - 0.125
        assert abs(got[0, e] - 1.0 / (1.0 + np.exp(-logit))) < 1e-14


def test_dense_normalised_adjacency_route():
    """Second route: the encoder as ReLU(D^-1/2 (A + I) D^-1/2 H W) with a dense symmetric adjacency
    matrix of the task-conditioned graph, and the perceptron through torch's linear layers."""
    rng = np.random.default_rng(3)
    N, B, d_in, d_h, d_m = 9, 3, 6, 5, 4
    src, dst = [], []
    for a in range(N):
        for b in range(a + 1, N):
            if rng.random() < 0.3:
                src.append(a)
                dst.append(b)
    model = _random_model(rng, d_in, d_h, d_m)
    x_op, x_task = rng.normal(size=(N, d_in)), rng.normal(size=(B, d_in))
    got = OS.edge_scores(x_op, x_task, src, dst, **model)
    A = np.zeros((N + 1, N + 1))
    for a, b in zip(src, dst):
        A[a, b] = A[b, a] = 1.0
    A[:N, N] = A[N, :N] = 1.0
    A_hat = A + np.eye(N + 1)
    dinv = 1.0 / np.sqrt(A_hat.sum(axis=1))
    norm = dinv[:, None] * A_hat * dinv[None, :]
    lin = torch.nn.functional.linear
    t = lambda a: torch.tensor(np.asarray(a), dtype=torch.float64)
    for b in range(B):
        H = np.concatenate([x_op, x_task[b:b + 1]])
        H = np.maximum(norm @ H @ model["w_gcn1"], 0)
        H = np.maximum(norm @ H @ model["w_gcn2"], 0)
        z = torch.cat([t(H[src]), t(H[dst]), t(H[N]).expand(len(src), -1)], dim=1)
        a1 = torch.relu(lin(z, t(model["w1"]).T, t(model["b1"])))
        a2 = torch.relu(lin(a1, t(model["w2"]).T, t(model["b2"])))
        s = torch.sigmoid(a2 @ t(model["w3"]) + model["b3"]).numpy()
        assert np.abs(got[b] - s).max() < 1e-12


def test_special_cases():
    rng = np.random.default_rng(5)
    N, d_in, d_h, d_m = 6, 4, 3, 3
    src, dst = [0, 1, 2, 0], [1, 2, 3, 4]
    model = _random_model(rng, d_in, d_h, d_m)
    x_op, x_task = rng.normal(size=(N, d_in)), rng.normal(size=(2, d_in))
    # a last layer of zeros: every score is the sigmoid of the bias
    z = dict(model, w3=np.zeros(d_m), b3=0.0)
    assert np.all(OS.edge_scores(x_op, x_task, src, dst, **z) == 0.5)
    # scores lie strictly between 0 and 1; the edge order is the order given; tasks are independent
    s = OS.edge_scores(x_op, x_task, src, dst, **model)
    assert np.all((s > 0) & (s < 1))
    perm = [2, 0, 3, 1]
    s2 = OS.edge_scores(x_op, x_task, [src[i] for i in perm], [dst[i] for i in perm], **model)
    assert np.allclose(s2, s[:, perm], atol=1e-15)
    s3 = OS.edge_scores(x_op, x_task[1:], src, dst, **model)
    assert np.allclose(s3[0], s[1], atol=1e-15)
    # an operation without any operation edge still hears the task node (its embedding is not zero)
    nb = OS.neighbourhoods(N, src, dst)
    assert nb[5] == {N}
    # a negated source -> target pair is a different edge: direction matters to the perceptron
    s4 = OS.edge_scores(x_op, x_task, dst, src, **model)
    assert not np.allclose(s4, s)
