"""fp64 definition of attention over a path of wGraph node KV segments.

TEST INFRASTRUCTURE ONLY (see the package docstring).

A request's context is the concatenation, in path order, of the KV segments of
the nodes on its workflow path (Sec. 5: the KV caches a workflow needs are
assembled from its operation nodes; the "stateful" alternative stores exactly
this concatenation once per prefix).  The method's sharing, per-segment
splitting and merging are exact reorganisations of softmax attention over that
concatenation, so the oracle is the plain definition: it copies the path's K/V
into one array per request and applies max-subtracted softmax attention.

Readings the paper leaves open (it prints no attention formula):
  * scaled dot-product attention, scale = 1/sqrt(head_dim) unless given;
  * grouped-query attention: query head h reads KV head h // (Hq // Hkv);
  * K and Q arrive already position-encoded (opaque vectors);
  * extend: the last node of the path is new; its query token i sees every
    token of the earlier nodes and tokens 0..i of the new node.
"""
from __future__ import annotations

import numpy as np


def attend(q, K, V, scale):
    """One query vector against explicit keys/values.

    q: [D], K: [L, D], V: [L, D] (fp64).  Returns (o[D], lse) with
    o = softmax(scale * K q)^T V and lse = log sum_j exp(scale * <q, K_j>).
    An empty context gives o = 0 and lse = -inf.
    """
    if K.shape[0] == 0:
        return np.zeros(V.shape[1], dtype=np.float64), -np.inf
    s = (K @ q) * scale
    m = s.max()
    p = np.exp(s - m)
    denom = p.sum()
    return (p @ V) / denom, m + np.log(denom)


def materialise(path, node_kv, kv_head):
    """Concatenate, in path order, the K and V of one KV head of every node on the path."""
    ks, vs = [], []
    for node in path:
        K, V = node_kv(int(node))
        ks.append(K[:, kv_head, :])
        vs.append(V[:, kv_head, :])
    return np.concatenate(ks, axis=0), np.concatenate(vs, axis=0)


def _scale(head_dim, scale):
    return 1.0 / np.sqrt(float(head_dim)) if scale is None else float(scale)


def decode(paths, node_kv, q, num_kv_heads, scale=None):
    """One query token per request.

    paths: list of node-id sequences; node_kv(node) -> (K, V) fp64 [len, Hkv, D];
    q: fp64 [R, Hq, D].  Returns (out [R, Hq, D], lse [R, Hq]).
    """
    R, Hq, D = q.shape
    g = Hq // num_kv_heads
    sc = _scale(D, scale)
    out = np.zeros((R, Hq, D), dtype=np.float64)
    lse = np.full((R, Hq), -np.inf, dtype=np.float64)
    for r in range(R):
        for kvh in range(num_kv_heads):
            Kc, Vc = materialise(paths[r], node_kv, kvh)
            for h in range(kvh * g, (kvh + 1) * g):
                out[r, h], lse[r, h] = attend(q[r, h], Kc, Vc, sc)
    return out, lse


def extend(paths, node_kv, q, num_kv_heads, scale=None, rows=None):
    """Every request appends its last path node; that node's tokens are the queries.

    q: fp64 [sum_r T_r, Hq, D], request-major, T_r = length of request r's last node.
    rows: optional list of global query-row indices to compute (others stay 0 / -inf).
    Returns (out [sum T_r, Hq, D], lse [sum T_r, Hq]).
    """
    n_rows, Hq, D = q.shape
    g = Hq // num_kv_heads
    sc = _scale(D, scale)
    out = np.zeros((n_rows, Hq, D), dtype=np.float64)
    lse = np.full((n_rows, Hq), -np.inf, dtype=np.float64)
    want = None if rows is None else set(int(x) for x in rows)
    row0 = 0
    for path in paths:
        T = node_kv(int(path[-1]))[0].shape[0]
        mine = [i for i in range(T) if want is None or (row0 + i) in want]
        if mine:
            for kvh in range(num_kv_heads):
                Kc, Vc = materialise(path, node_kv, kvh)
                prefix = Kc.shape[0] - T
                for i in mine:
                    visible = prefix + i + 1
                    for h in range(kvh * g, (kvh + 1) * g):
                        out[row0 + i, h], lse[row0 + i, h] = attend(
                            q[row0 + i, h], Kc[:visible], Vc[:visible], sc)
        row0 += T
    assert row0 == n_rows
    return out, lse


def lse_merge(outs, lses):
    """Combine attention results computed over disjoint parts of one context.

    outs: [P, D] partial outputs (each already normalised over its own part),
    lses: [P] their log-sum-exps.  Softmax over the union weights part i by
    exp(lse_i - logsumexp(lses)).  Parts with lse = -inf (empty) carry no weight.
    """
    outs = np.asarray(outs, dtype=np.float64)
    lses = np.asarray(lses, dtype=np.float64)
    M = lses.max()
    if not np.isfinite(M):
        return np.zeros(outs.shape[1], dtype=np.float64), -np.inf
    w = np.exp(lses - M)
    total = w.sum()
    return (w[:, None] * outs).sum(axis=0) / total, M + np.log(total)
