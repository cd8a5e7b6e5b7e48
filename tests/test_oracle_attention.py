"""Pins for the attention oracle.  Each test would fail on a plausible slip
(dropped scale, wrong head map, transposed operand, off-by-one causal mask,
wrong concatenation order in extend, un-normalised merge)."""
import math

import numpy as np
import pytest
import torch

from oracle import attention as OA
from paper_2605_22566_b200 import workloads as W


def _rand_nodes(rng, lens, Hkv, D):
    kv = {v: (rng.standard_normal((n, Hkv, D)), rng.standard_normal((n, Hkv, D))) for v, n in enumerate(lens)}
    return lambda v: kv[v]


def _brute(q, K, V, scale):
    """Two-pass softmax attention in pure Python floats with exact summation."""
    s = [scale * math.fsum(float(a) * float(b) for a, b in zip(q, row)) for row in K]
    m = max(s)
    e = [math.exp(x - m) for x in s]
    z = math.fsum(e)
    o = [math.fsum(e[j] * float(V[j][d]) for j in range(len(e))) / z for d in range(len(V[0]))]
    return o, m + math.log(z)


def test_brute_force_tiny():
    rng = np.random.default_rng(1)
    Hq, Hkv, D = 4, 2, 8
    lens = [5, 3, 7, 2]
    node_kv = _rand_nodes(rng, lens, Hkv, D)
    paths = [[0, 2], [1, 0, 3], [3]]
    q = rng.standard_normal((3, Hq, D))
    out, lse = OA.decode(paths, node_kv, q, Hkv)
    for r, p in enumerate(paths):
        for h in range(Hq):
            kvh = h // (Hq // Hkv)
            K = [row for v in p for row in node_kv(v)[0][:, kvh, :].tolist()]
            V = [row for v in p for row in node_kv(v)[1][:, kvh, :].tolist()]
            o, l = _brute(q[r, h].tolist(), K, V, 1.0 / math.sqrt(D))
            assert np.allclose(out[r, h], o, rtol=0, atol=1e-12)
            assert abs(lse[r, h] - l) < 1e-12


def test_brute_force_extend_tiny():
    rng = np.random.default_rng(2)
    Hq, Hkv, D = 2, 1, 4
    lens = [4, 3, 5]
    node_kv = _rand_nodes(rng, lens, Hkv, D)
    paths = [[0, 1], [0, 2]]  # new nodes: 1 (3 tokens), 2 (5 tokens)
    q = rng.standard_normal((8, Hq, D))
    out, lse = OA.extend(paths, node_kv, q, Hkv, scale=0.37)
    row = 0
    for p in paths:
        T = lens[p[-1]]
        for i in range(T):
            for h in range(Hq):
                K = node_kv(p[0])[0][:, 0, :].tolist() + node_kv(p[1])[0][: i + 1, 0, :].tolist()
                V = node_kv(p[0])[1][:, 0, :].tolist() + node_kv(p[1])[1][: i + 1, 0, :].tolist()
                o, l = _brute(q[row, h].tolist(), K, V, 0.37)
                assert np.allclose(out[row, h], o, rtol=0, atol=1e-12)
                assert abs(lse[row, h] - l) < 1e-12
            row += 1


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (8, 2)])
def test_single_node_equals_library_sdpa(Hq, Hkv):
    rng = np.random.default_rng(3)
    D, n, R = 16, 37, 3
    node_kv = _rand_nodes(rng, [n], Hkv, D)
    q = rng.standard_normal((R, Hq, D))
    out, _ = OA.decode([[0]] * R, node_kv, q, Hkv)
    K, V = node_kv(0)
    g = Hq // Hkv
    Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(g, dim=0)  # [Hq, n, D]
    Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(g, dim=0)
    for r in range(R):
        ref = torch.nn.functional.scaled_dot_product_attention(
            torch.from_numpy(q[r])[:, None, :], Kt, Vt)  # [Hq, 1, D]
        assert np.allclose(out[r], ref[:, 0, :].numpy(), rtol=0, atol=1e-12)


def test_single_node_extend_equals_library_causal_sdpa():
    rng = np.random.default_rng(4)
    Hq, Hkv, D, T = 4, 2, 16, 23
    node_kv = _rand_nodes(rng, [T], Hkv, D)
    q = rng.standard_normal((T, Hq, D))
    out, _ = OA.extend([[0]], node_kv, q, Hkv)
    K, V = node_kv(0)
    Kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(2, dim=0)
    Vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(2, dim=0)
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q).permute(1, 0, 2), Kt, Vt, is_causal=True)  # [Hq, T, D]
    assert np.allclose(out, ref.permute(1, 0, 2).numpy(), rtol=0, atol=1e-12)


def test_closed_forms():
    rng = np.random.default_rng(5)
    Hq, Hkv, D = 4, 2, 8
    lens = [6, 9]
    # identical keys -> uniform weights -> mean of V over the visible tokens
    kvec = rng.standard_normal((Hkv, D))
    kv = {v: (np.broadcast_to(kvec, (n, Hkv, D)).copy(), rng.standard_normal((n, Hkv, D)))
          for v, n in enumerate(lens)}
    q = rng.standard_normal((1, Hq, D))
    out, lse = OA.decode([[0, 1]], lambda v: kv[v], q, Hkv)
    Vall = np.concatenate([kv[0][1], kv[1][1]], axis=0)
    for h in range(Hq):
        assert np.allclose(out[0, h], Vall[:, h // 2, :].mean(axis=0), rtol=0, atol=1e-14)
        assert abs(lse[0, h] - (q[0, h] @ kvec[h // 2] / math.sqrt(D) + math.log(15))) < 1e-12
    # extend with identical keys: token i's output is the running mean over prefix + 0..i
    qe = rng.standard_normal((lens[1], Hq, D))
    oute, _ = OA.extend([[0, 1]], lambda v: kv[v], qe, Hkv)
    for i in range(lens[1]):
        assert np.allclose(oute[i, 1], Vall[: lens[0] + i + 1, 0, :].mean(axis=0), rtol=0, atol=1e-14)
    # constant V -> that constant; linearity in V
    node_kv = _rand_nodes(rng, lens, Hkv, D)
    c = rng.standard_normal(D)
    const = lambda v: (node_kv(v)[0], np.broadcast_to(c, node_kv(v)[1].shape))
    out, _ = OA.decode([[1, 0]], const, q, Hkv)
    assert np.allclose(out[0], np.broadcast_to(c, (Hq, D)), rtol=0, atol=1e-14)
    other = _rand_nodes(rng, lens, Hkv, D)
    comb = lambda v: (node_kv(v)[0], 2.0 * node_kv(v)[1] - 3.0 * other(v)[1])
    o1, _ = OA.decode([[0, 1]], node_kv, q, Hkv)
    o2, _ = OA.decode([[0, 1]], lambda v: (node_kv(v)[0], other(v)[1]), q, Hkv)
    o3, _ = OA.decode([[0, 1]], comb, q, Hkv)
    assert np.allclose(o3, 2.0 * o1 - 3.0 * o2, rtol=0, atol=1e-13)
    # one dominant key -> its value row
    K, V = node_kv(0)
    Kd = K.copy()
    Kd[3, 0, :] = 200.0 * q[0, 0] / np.linalg.norm(q[0, 0])
    out, _ = OA.decode([[0]], lambda v: (Kd, V), q, Hkv)
    assert np.allclose(out[0, 0], V[3, 0], rtol=0, atol=1e-10)
    # empty context
    o, l = OA.attend(q[0, 0], np.zeros((0, D)), np.zeros((0, D)), 1.0)
    assert np.all(o == 0) and l == -np.inf


def _cfg0_f64(w):
    cache = {}

    def node_kv(v):
        if v not in cache:
            k, vv = w.node_kv_bits(0, v)
            cache[v] = (W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv))
        return cache[v]
    return node_kv, W.bf16_bits_to_f64(w.q_bits(0))


def test_path_invariances_on_config0():
    w = W.make_config(0)
    node_kv, q = _cfg0_f64(w)
    paths = [w.path(r).tolist() for r in range(w.num_requests)]
    out, lse = OA.decode(paths, node_kv, q, w.num_kv_heads)
    # request-order invariance
    perm = np.random.default_rng(6).permutation(len(paths))
    outp, lsep = OA.decode([paths[i] for i in perm], node_kv, q[perm], w.num_kv_heads)
    assert np.array_equal(outp, out[perm]) and np.array_equal(lsep, lse[perm])
    # segment-order invariance (decode only)
    outr, lser = OA.decode([p[::-1] for p in paths], node_kv, q, w.num_kv_heads)
    assert np.allclose(outr, out, rtol=0, atol=1e-12) and np.allclose(lser, lse, rtol=0, atol=1e-12)
    # segment-split invariance: cut every node into two nodes holding consecutive halves
    N = w.num_nodes

    def split_kv(v):
        base, second = (v, False) if v < N else (v - N, True)
        K, V = node_kv(base)
        h = K.shape[0] // 2
        return (K[h:], V[h:]) if second else (K[:h], V[:h])
    outs, lses = OA.decode([[x for v in p for x in (v, v + N)] for p in paths], split_kv, q, w.num_kv_heads)
    assert np.allclose(outs, out, rtol=0, atol=1e-12) and np.allclose(lses, lse, rtol=0, atol=1e-12)
    # a shared path equals one private node that holds the concatenation
    for r in (0, 3):
        cat = (np.concatenate([node_kv(v)[0] for v in paths[r]]), np.concatenate([node_kv(v)[1] for v in paths[r]]))
        o1, l1 = OA.decode([[0]], lambda v: cat, q[r:r + 1], w.num_kv_heads)
        assert np.allclose(o1[0], out[r], rtol=0, atol=1e-12)


def test_lse_merge_identity():
    w = W.make_config(0)
    node_kv, q = _cfg0_f64(w)
    paths = [w.path(r).tolist() for r in range(w.num_requests)]
    out, lse = OA.decode(paths, node_kv, q, w.num_kv_heads)
    for r, p in enumerate(paths):
        parts = [OA.decode([[v]], node_kv, q[r:r + 1], w.num_kv_heads) for v in p]
        for h in range(w.num_q_heads):
            outs = [po[0, h] for po, _ in parts]
            lses = [pl[0, h] for _, pl in parts]
            o, l = OA.lse_merge(outs, lses)
            assert np.allclose(o, out[r, h], rtol=0, atol=1e-12) and abs(l - lse[r, h]) < 1e-12
            # lse(path) = logsumexp of the per-segment lse (library routine)
            assert abs(torch.logsumexp(torch.tensor(lses, dtype=torch.float64), 0).item() - lse[r, h]) < 1e-12
            # permutation of the partials and a single partial
            o2, l2 = OA.lse_merge(outs[::-1], lses[::-1])
            assert np.allclose(o2, o, rtol=0, atol=1e-13) and abs(l2 - l) < 1e-13
            o1, l1 = OA.lse_merge(outs[:1], lses[:1])
            assert np.array_equal(o1, outs[0]) and l1 == lses[0]
            # an empty part carries no weight
            o3, l3 = OA.lse_merge(outs + [np.zeros_like(outs[0])], lses + [-np.inf])
            assert np.allclose(o3, o, rtol=0, atol=1e-13) and abs(l3 - l) < 1e-13


def test_causal_extend_equals_decode_over_truncated_node():
    w = W.make_config(2, n_requests=4, new_len=9, root_len=40, len_lo=8, len_hi=20, prefix_lo=40,
                      prefix_hi=90, group_lo=2, group_hi=2, hq=4, hkv=2, d=16)
    cache = {}

    def node_kv(v):
        if v not in cache:
            k, vv = w.node_kv_bits(0, v)
            cache[v] = (W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv))
        return cache[v]
    q = W.bf16_bits_to_f64(w.q_bits(0))
    paths = [w.path(r).tolist() for r in range(w.num_requests)]
    out, lse = OA.extend(paths, node_kv, q, w.num_kv_heads)
    qp = w.q_row_ptr()
    for r, p in enumerate(paths):
        for i in range(9):
            def trunc(v, i=i, last=p[-1]):
                K, V = node_kv(v)
                return (K[: i + 1], V[: i + 1]) if v == last else (K, V)
            o, l = OA.decode([p], trunc, q[qp[r] + i: qp[r] + i + 1], w.num_kv_heads)
            assert np.allclose(o[0], out[qp[r] + i], rtol=0, atol=1e-12)
            assert np.allclose(l[0], lse[qp[r] + i], rtol=0, atol=1e-12)
    # `rows` computes the same values for the sampled rows only
    rows = [0, 10, 35]
    o2, l2 = OA.extend(paths, node_kv, q, w.num_kv_heads, rows=rows)
    assert np.array_equal(o2[rows], out[rows]) and np.all(o2[[1, 2, 34]] == 0)
