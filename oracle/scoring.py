"""fp64 definition of the workflow-construction model's edge scores (Sec. 4.1, 4.2; Appendix
"Network Architecture Details").

TEST INFRASTRUCTURE ONLY (see the package docstring).

The wGraph is extended by a virtual task node joined to every operation node in both directions
(Sec. 4.1).  A 2-layer graph convolutional encoder gives every node an embedding (Eq. 5; layer rule
in the appendix: h_i' = ReLU(sum over j in N(i) and i itself of h_j W / sqrt(deg(i) deg(j)))), and a
3-layer perceptron scores every edge (v_i, v_j) of the wGraph from the concatenation
[h_i, h_j, h_task] (Eq. 6), Linear-ReLU-Linear-ReLU-Linear followed by a sigmoid.

Readings the paper leaves open:
  * message passing treats the operation edges as undirected (the layer rule sums over a
    neighbourhood and normalises symmetrically, as in the graph convolution it cites);
  * deg(i) counts the node itself, i.e. it is the size of N(i) plus one (the sum runs over N(i) and i);
  * the encoder's layers have no bias (the layer rule shows none); the perceptron's layers do;
  * the second encoder layer ends in ReLU like the first (the rule is stated for every layer).
Weights are inputs: the trained parameters are not available, any values serve.
"""
from __future__ import annotations

import numpy as np


def neighbourhoods(num_ops: int, edge_src, edge_dst):
    """Neighbour sets of the task-conditioned graph: nodes 0..num_ops-1 are operations, node num_ops
    is the virtual task node.  Operation edges count in both directions; duplicates collapse."""
    nb = [set() for _ in range(num_ops + 1)]
    for a, b in zip(edge_src, edge_dst):
        a, b = int(a), int(b)
        if a != b:
            nb[a].add(b)
            nb[b].add(a)
    for v in range(num_ops):
        nb[v].add(num_ops)
        nb[num_ops].add(v)
    return nb


def gcn_layer(H, nb, W):
    """One layer of the appendix's rule on every node.  H: [n, d_in] fp64, W: [d_in, d_out]."""
    n = H.shape[0]
    deg = [len(nb[i]) + 1 for i in range(n)]
    HW = H @ W
    out = np.zeros((n, W.shape[1]), dtype=np.float64)
    for i in range(n):
        acc = HW[i] / np.sqrt(deg[i] * deg[i])
        for j in sorted(nb[i]):
            acc = acc + HW[j] / np.sqrt(deg[i] * deg[j])
        out[i] = np.maximum(acc, 0.0)
    return out


def edge_scores(x_op, x_task, edge_src, edge_dst, w_gcn1, w_gcn2, w1, b1, w2, b2, w3, b3):
    """Scores s[b, e] in (0, 1) of every wGraph edge e = (edge_src[e], edge_dst[e]) for every task b.

    x_op: [N, d_in] operation features; x_task: [B, d_in] task features; w_gcn1: [d_in, d_h];
    w_gcn2: [d_h, d_h]; w1: [3 d_h, d_m], b1: [d_m]; w2: [d_m, d_m], b2: [d_m]; w3: [d_m], b3: scalar.
    """
    x_op = np.asarray(x_op, dtype=np.float64)
    x_task = np.asarray(x_task, dtype=np.float64)
    N, B, E = x_op.shape[0], x_task.shape[0], len(edge_src)
    nb = neighbourhoods(N, edge_src, edge_dst)
    out = np.zeros((B, E), dtype=np.float64)
    for b in range(B):
        H = np.concatenate([x_op, x_task[b:b + 1]], axis=0)
        H = gcn_layer(H, nb, np.asarray(w_gcn1, dtype=np.float64))
        H = gcn_layer(H, nb, np.asarray(w_gcn2, dtype=np.float64))
        for e in range(E):
            z = np.concatenate([H[int(edge_src[e])], H[int(edge_dst[e])], H[N]])
            a = np.maximum(z @ w1 + b1, 0.0)
            a = np.maximum(a @ w2 + b2, 0.0)
            out[b, e] = 1.0 / (1.0 + np.exp(-(a @ w3 + b3)))
    return out
