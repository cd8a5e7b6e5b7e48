"""Differential KV (Sec. 5.1, Eq. 7) through the C ABI: reconstruction bit for bit against the oracle,
and attention over paths that name reconstructed, prefix-conditioned nodes."""
import dataclasses

import numpy as np
import pytest
import torch

from helpers import assert_close
from oracle import attention as OA
from oracle import residual as OR
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _with_variants(w, bases):
    """The workload plus one private node per entry of `bases`, of the base node's length."""
    n0 = w.num_nodes
    node_len = np.concatenate([w.node_len, w.node_len[np.array(bases)]]).astype(w.node_len.dtype)
    return dataclasses.replace(w, num_nodes=n0 + len(bases), node_len=node_len), list(range(n0, n0 + len(bases)))


def _upload(res, dev):
    bitmap, vals, row_ptr = res
    t = (torch.from_numpy(bitmap.view(np.int32).copy()).to(dev),
         torch.from_numpy(np.concatenate([vals, np.zeros(8, np.uint16)]).view(np.int16).copy()).to(dev),
         torch.from_numpy(row_ptr.copy()).to(dev))
    return t, (t[0].data_ptr(), t[1].data_ptr(), t[2].data_ptr(), int(row_ptr[-1]))


def _read_node(pa, node, layer=0):
    from paper_2605_22566_b200 import binding as B
    w = pa.w
    n = int(w.node_len[node])
    k = torch.empty((n, w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device=pa.dev)
    v = torch.empty_like(k)
    B.check(B.gf_node_kv_read(pa.g, node, layer, k.data_ptr(), v.data_ptr(), pa.stream), "gf_node_kv_read")
    torch.cuda.synchronize()
    as_bits = lambda t: t.view(torch.int16).cpu().numpy().view(np.uint16)
    return as_bits(k), as_bits(v)


def _setup(cfg_kwargs, n_var, seed=3):
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(**cfg_kwargs)
    used = w.used_nodes()
    rng = np.random.default_rng(seed)
    bases = sorted(rng.choice(used[w.node_len[used] > 0], size=n_var, replace=False).tolist())
    w2, variants = _with_variants(w, bases)
    extra = int(((w2.node_len[np.array(variants)].astype(np.int64) + 63) // 64).sum())
    pa = PathAttention(w2, layers=1, extra_tiles=extra)
    pa.write_nodes("device")
    return w2, pa, bases, variants


@pytest.mark.parametrize("cfg", [dict(config_id=0), dict(config_id=1, n_requests=24, n_nodes=48, root_len=333, len_lo=1, len_hi=150, suffix_max=40)])
def test_read_back_returns_what_was_written(cfg):
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(**cfg)
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    for v in w.used_nodes().tolist()[:6]:
        k, vv = _read_node(pa, v)
        kb, vb = w.node_kv_bits(0, v)
        assert np.array_equal(k, kb) and np.array_equal(vv, vb)
    pa.close()


@pytest.mark.parametrize("cfg,dk,dv", [
    (dict(config_id=0), 0.25, 0.30),
    (dict(config_id=1, n_requests=24, n_nodes=48, root_len=333, len_lo=1, len_hi=150, suffix_max=40), 0.25, 0.30),
    (dict(config_id=1, n_requests=24, n_nodes=48, root_len=200, len_lo=1, len_hi=90, suffix_max=40), 0.0, 1.0),
])
def test_reconstruct_bit_exact(cfg, dk, dv):
    from paper_2605_22566_b200 import binding as B
    w, pa, bases, variants = _setup(cfg, n_var=5)
    rows_of = lambda v: int(w.node_len[v]) * w.num_kv_heads
    keep = []
    for i, (b, v) in enumerate(zip(bases, variants)):
        rk = W.residual_stream(w.seed, W.KIND_DK, 0, b, i + 1, rows_of(b), w.head_dim, dk)
        rv = W.residual_stream(w.seed, W.KIND_DV, 0, b, i + 1, rows_of(b), w.head_dim, dv)
        tk, pk = _upload(rk, pa.dev)
        tv, pv = _upload(rv, pa.dev)
        keep += [tk, tv]
        only_v = (i == 1)  # one variant leaves K without a residual
        B.check(B.gf_node_kv_reconstruct(pa.g, v, 0, b, None if only_v else pk, pv, pa.stream), "gf_node_kv_reconstruct")
        kb, vb = w.node_kv_bits(0, b)
        want_k = kb if only_v else OR.reconstruct(kb.reshape(-1, w.head_dim), *rk).reshape(kb.shape)
        want_v = OR.reconstruct(vb.reshape(-1, w.head_dim), *rv).reshape(vb.shape)
        got_k, got_v = _read_node(pa, v)
        assert np.array_equal(got_k, want_k), f"K of variant {i}"
        assert np.array_equal(got_v, want_v), f"V of variant {i}"
        base_k, base_v = _read_node(pa, b)  # the base is left as it was
        assert np.array_equal(base_k, kb) and np.array_equal(base_v, vb)
    assert pa.status() == 0
    pa.close()


def test_reconstruct_rejects_bad_arguments_and_reports_a_short_value_array():
    from paper_2605_22566_b200 import binding as B
    w, pa, bases, variants = _setup(dict(config_id=0), n_var=2)
    b, v = bases[0], variants[0]
    rows = int(w.node_len[b]) * w.num_kv_heads
    rk = W.residual_stream(w.seed, W.KIND_DK, 0, b, 1, rows, w.head_dim, 0.25)
    tk, pk = _upload(rk, pa.dev)
    assert B.gf_node_kv_reconstruct(pa.g, b, 0, b, pk, None, pa.stream) == B.GF_ERR_INVALID_ARG      # onto itself
    assert B.gf_node_kv_reconstruct(pa.g, v, 0, variants[1], pk, None, pa.stream) == B.GF_ERR_NOT_WRITTEN  # base never written
    assert B.gf_node_kv_reconstruct(pa.g, v, 7, b, pk, None, pa.stream) == B.GF_ERR_INVALID_ARG      # no such layer
    # nnz understated: the kernel reads no value at or beyond it, keeps the base there and says so
    short = (pk[0], pk[1], pk[2], pk[3] // 2)
    B.check(B.gf_node_kv_reconstruct(pa.g, v, 0, b, short, None, pa.stream), "gf_node_kv_reconstruct")
    torch.cuda.synchronize()
    assert pa.status() == B.GF_ERR_INVALID_ARG
    assert pa.status() == 0  # reading the status clears it
    pa.close()


def test_attention_over_paths_through_reconstructed_nodes():
    """Requests whose paths name the prefix-conditioned variant attend over base + residual."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import tensor_to_f64
    cfg = dict(config_id=1, n_requests=32, n_nodes=48, root_len=300, len_lo=1, len_hi=150, suffix_max=40)
    w, pa, bases, variants = _setup(cfg, n_var=4, seed=9)
    state, keep = {}, []
    for i, (b, v) in enumerate(zip(bases, variants)):
        rows = int(w.node_len[b]) * w.num_kv_heads
        rk = W.residual_stream(w.seed, W.KIND_DK, 0, b, 1, rows, w.head_dim, 0.25)
        rv = W.residual_stream(w.seed, W.KIND_DV, 0, b, 1, rows, w.head_dim, 0.30)
        tk, pk = _upload(rk, pa.dev)
        tv, pv = _upload(rv, pa.dev)
        keep += [tk, tv]
        B.check(B.gf_node_kv_reconstruct(pa.g, v, 0, b, pk, pv, pa.stream), "gf_node_kv_reconstruct")
        kb, vb = w.node_kv_bits(0, b)
        state[v] = (OR.bf16_to_f64(OR.reconstruct(kb.reshape(-1, w.head_dim), *rk)).reshape(kb.shape),
                    OR.bf16_to_f64(OR.reconstruct(vb.reshape(-1, w.head_dim), *rv)).reshape(vb.shape))
    # every second request that passes through a base node takes the variant instead (variants have
    # private ids, at or above num_shared_nodes, so no edge is required around them); requests that
    # swap the same node share the reconstructed segment like any other
    path_node = w.path_node.copy()
    swapped = 0
    for r in range(0, w.num_requests, 2):
        for i in range(w.path_ptr[r], w.path_ptr[r + 1]):
            if int(path_node[i]) in bases:
                path_node[i] = variants[bases.index(int(path_node[i]))]
                swapped += 1
    assert swapped >= 2
    pa.path_node = torch.from_numpy(path_node.astype(np.int32)).to(pa.dev)
    pa.build()
    q = pa.make_q(0)
    out = tensor_to_f64(pa.decode(0, q))
    assert pa.status() == 0

    def node_kv(v):
        if v in state:
            return state[v]
        k, vv = w.node_kv_bits(0, v)
        return W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv)

    paths = [[int(x) for x in path_node[w.path_ptr[r]:w.path_ptr[r + 1]] if w.node_len[x] > 0] for r in range(w.num_requests)]
    ref, _ = OA.decode(paths, node_kv, W.bf16_bits_to_f64(w.q_bits(0)), w.num_kv_heads)
    assert_close(out, ref, "decode over reconstructed nodes")
    pa.close()


def test_reconstruct_at_bench_size_sampled_rows():
    """The launch `bench.py --residual` times (a 32 768-token node, Llama-3-8B heads): sampled rows, the
    first and last rows and the rows around every tile boundary of the sample, bit for bit."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.residual_workload(n_base=1)
    T, H, D = int(w.node_len[0]), w.num_kv_heads, w.head_dim
    pa = PathAttention(w, layers=1, extra_tiles=(T + 63) // 64)
    pa.write_nodes("device")
    rows = T * H
    rk = W.residual_stream(w.seed, W.KIND_DK, 0, 0, 1, rows, D, 0.25)
    rv = W.residual_stream(w.seed, W.KIND_DV, 0, 0, 1, rows, D, 0.30)
    tk, pk = _upload(rk, pa.dev)
    tv, pv = _upload(rv, pa.dev)
    B.check(B.gf_node_kv_reconstruct(pa.g, 1, 0, 0, pk, pv, pa.stream), "gf_node_kv_reconstruct")
    got_k, got_v = _read_node(pa, 1)
    assert pa.status() == 0
    rng = np.random.default_rng(5)
    pick = np.unique(np.concatenate([rng.choice(rows, size=3000, replace=False), np.arange(0, 4 * H), np.arange(rows - 4 * H, rows),
                                     np.arange(63 * H, 66 * H)]))
    kb, vb = w.node_kv_bits(0, 0)
    for got, base, (bm, vals, rp) in ((got_k, kb, rk), (got_v, vb, rv)):
        base2, got2 = base.reshape(rows, D), got.reshape(rows, D)
        for r in pick.tolist():
            a, b = int(rp[r]), int(rp[r + 1])
            want = OR.reconstruct(base2[r:r + 1], bm[r:r + 1], vals[a:b], np.array([0, b - a], dtype=np.int32))
            assert np.array_equal(got2[r], want[0]), r
    # and as a whole: entries without a residual are the base, entries with one differ from it
    # (a value is never zero and never below half an ulp of a unit-scale base)
    has, _ = OR.densify(rk[0][:4096], rk[1][:int(rk[2][4096])], rk[2][:4097], D)
    g, b0 = got_k.reshape(rows, D)[:4096], kb.reshape(rows, D)[:4096]
    assert np.array_equal(g[~has], b0[~has])
    pa.close()


def test_reconstruct_of_an_empty_node_and_without_any_residual():
    """Degenerate cases: a base of zero tokens gives a variant of zero tokens; no residual at all is a copy."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(0)
    empty = np.nonzero(w.node_len == 0)[0].tolist()
    full = [v for v in w.used_nodes().tolist() if w.node_len[v] > 0][0]
    assert empty, "config 0 has a node of zero tokens"
    w2, (va, vb_) = _with_variants(w, [empty[0], full])
    pa = PathAttention(w2, layers=1, extra_tiles=(int(w.node_len[full]) + 63) // 64)
    pa.write_nodes("device")
    B.check(B.gf_node_kv_write(pa.g, empty[0], 0, 0, 0, 0, pa.stream), "gf_node_kv_write")   # records the empty node
    B.check(B.gf_node_kv_reconstruct(pa.g, va, 0, empty[0], None, None, pa.stream), "gf_node_kv_reconstruct")
    B.check(B.gf_node_kv_read(pa.g, va, 0, 0, 0, pa.stream), "gf_node_kv_read")          # nothing to copy
    B.check(B.gf_node_kv_reconstruct(pa.g, vb_, 0, full, None, None, pa.stream), "gf_node_kv_reconstruct")
    k, v = _read_node(pa, vb_)
    kb, vb = w.node_kv_bits(0, full)
    assert np.array_equal(k, kb) and np.array_equal(v, vb) and pa.status() == 0
    pa.close()
