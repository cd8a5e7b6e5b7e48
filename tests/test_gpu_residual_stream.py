"""Differential KV inside the segment stream (Sec. 5.1, Eq. 7): a prefix-conditioned state declared as
base + sparse residual (gf_node_kv_attach_residual) takes no tiles of its own; decode streams the
base node's tiles and completes them in shared memory.  Held to the oracle (attention over the
oracle's own reconstruction) and, bit for bit, to decode over the materialised variant."""
import dataclasses

import numpy as np
import pytest
import torch

from helpers import assert_close
from oracle import attention as OA
from oracle import residual as OR
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _upload(res, dev):
    bitmap, vals, row_ptr = res
    t = (torch.from_numpy(bitmap.view(np.int32).copy()).to(dev),
         torch.from_numpy(np.concatenate([vals, np.zeros(8, np.uint16)]).view(np.int16).copy()).to(dev),
         torch.from_numpy(row_ptr.copy()).to(dev))
    return t, (t[0].data_ptr(), t[1].data_ptr(), t[2].data_ptr(), int(row_ptr[-1]))


def _case(cfg, n_var, swap_every, seed=9, min_len=1):
    """Workload plus n_var variant nodes (private ids) of seeded base nodes; every swap_every-th request
    that passes through a base takes the variant instead.  Returns (w, bases, variants, path_node)."""
    w = W.make_config(**cfg)
    used = w.used_nodes()
    rng = np.random.default_rng(seed)
    cand = used[(w.node_len[used] >= min_len) & (used < w.num_shared_nodes)]
    bases = sorted(rng.choice(cand, size=n_var, replace=False).tolist())
    n0 = w.num_nodes
    node_len = np.concatenate([w.node_len, w.node_len[np.array(bases)]]).astype(w.node_len.dtype)
    w2 = dataclasses.replace(w, num_nodes=n0 + n_var, node_len=node_len)
    variants = list(range(n0, n0 + n_var))
    path_node = w.path_node.copy()
    swapped = 0
    for r in range(0, w.num_requests, swap_every):
        for i in range(w.path_ptr[r], w.path_ptr[r + 1]):
            if int(path_node[i]) in bases:
                path_node[i] = variants[bases.index(int(path_node[i]))]
                swapped += 1
    assert swapped >= 2
    return w2, bases, variants, path_node


def _residuals(w, bases, dev, dk=0.25, dv=0.30):
    out, keep = [], []
    for b in bases:
        rows = int(w.node_len[b]) * w.num_kv_heads
        rk = W.residual_stream(w.seed, W.KIND_DK, 0, b, 1, rows, w.head_dim, dk)
        rv = W.residual_stream(w.seed, W.KIND_DV, 0, b, 1, rows, w.head_dim, dv)
        tk, pk = _upload(rk, dev)
        tv, pv = _upload(rv, dev)
        keep += [tk, tv]
        out.append((rk, rv, pk, pv))
    return out, keep


def _oracle(w, bases, variants, res, path_node):
    state = {}
    for b, v, (rk, rv, _, _) in zip(bases, variants, res):
        kb, vb = w.node_kv_bits(0, b)
        state[v] = (OR.bf16_to_f64(OR.reconstruct(kb.reshape(-1, w.head_dim), *rk)).reshape(kb.shape),
                    OR.bf16_to_f64(OR.reconstruct(vb.reshape(-1, w.head_dim), *rv)).reshape(vb.shape))

    def node_kv(v):
        if v in state:
            return state[v]
        k, vv = w.node_kv_bits(0, v)
        return W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv)
    paths = [[int(x) for x in path_node[w.path_ptr[r]:w.path_ptr[r + 1]] if w.node_len[x] > 0]
             for r in range(w.num_requests)]
    return OA.decode(paths, node_kv, W.bf16_bits_to_f64(w.q_bits(0)), w.num_kv_heads)


def _decode(w, bases, variants, path_node, how, dk=0.25, dv=0.30):
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    extra = int(((w.node_len[np.array(variants)].astype(np.int64) + 63) // 64).sum()) if how == "reconstruct" else 0
    pa = PathAttention(w, layers=1, extra_tiles=extra, max_residual_nodes=len(variants))
    pa.write_nodes("device", skip=set(variants))
    in_use = B.gf_pool_info(pa.g).tiles_in_use
    res, keep = _residuals(w, bases, pa.dev, dk, dv)
    fn = B.gf_node_kv_reconstruct if how == "reconstruct" else B.gf_node_kv_attach_residual
    for b, v, (_, _, pk, pv) in zip(bases, variants, res):
        B.check(fn(pa.g, v, 0, b, pk, pv, pa.stream), how)
    if how == "attach":
        assert B.gf_pool_info(pa.g).tiles_in_use == in_use      # no tile was taken
        for b, v in zip(bases, variants):
            assert B.gf_node_extent(pa.g, v)[1:] == B.gf_node_extent(pa.g, b)[1:]  # same length, the base's tiles
    pa.path_node = torch.from_numpy(path_node.astype(np.int32)).to(pa.dev)
    pa.build()
    lse = pa.guarded(w.num_requests * w.num_q_heads * 4, "lse").view(torch.float32).view(w.num_requests, w.num_q_heads)
    out = pa.decode(0, pa.make_q(0), lse=lse)
    assert pa.status() == 0
    bits = out.view(torch.int16).cpu().numpy().copy()
    return pa, bits, out, lse, res, keep


@pytest.mark.parametrize("cfg,n_var", [
    (dict(config_id=1, n_requests=32, n_nodes=48, root_len=300, len_lo=1, len_hi=150, suffix_max=40), 4),
    (dict(config_id=0, hq=8, hkv=2, d=64, n_requests=19, root_len=77, len_lo=1, len_hi=90), 3),
    (dict(config_id=1, n_requests=40, n_nodes=24, root_len=900, len_lo=100, len_hi=700, suffix_max=30), 5),
])
def test_decode_over_attached_residuals_matches_oracle_and_the_materialised_variant(cfg, n_var):
    from paper_2605_22566_b200.runtime import tensor_to_f64
    w, bases, variants, path_node = _case(cfg, n_var, swap_every=2)
    pa, bits_a, out, lse, res, keep = _decode(w, bases, variants, path_node, "attach")
    ref_o, ref_l = _oracle(w, bases, variants, res, path_node)
    assert_close(tensor_to_f64(out), ref_o, "decode with the residual applied in the stream")
    assert np.abs(tensor_to_f64(lse) - ref_l).max() < 2e-3
    pa.close()
    pb, bits_r, _, _, _, keep2 = _decode(w, bases, variants, path_node, "reconstruct")
    pb.close()
    assert np.array_equal(bits_a, bits_r)   # the same tile bits reach the MMAs either way


def test_root_variant_shared_by_many_requests_and_release_rules():
    """A variant of the root taken by every second of 200 requests (its segment stays with the warp
    kernel although it is widely shared); a base cannot be released while a variant hangs on it, a
    variant can, and its row of the residual table is reused."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import tensor_to_f64
    cfg = dict(config_id=1, n_requests=200, n_nodes=12, root_len=500, len_lo=65, len_hi=300, depth_lo=3, depth_hi=4,
               suffix_max=30)
    w = W.make_config(**cfg)
    n0 = w.num_nodes
    w2 = dataclasses.replace(w, num_nodes=n0 + 1, node_len=np.append(w.node_len, w.node_len[0]))
    path_node = w.path_node.copy()
    for r in range(0, w.num_requests, 2):
        path_node[w.path_ptr[r]] = n0       # the root's variant
    pa, bits, out, lse, res, keep = _decode(w2, [0], [n0], path_node, "attach")
    reqs = list(range(0, 200, 7))
    ref_o, _ = _oracle(w2, [0], [n0], res, path_node)
    assert_close(tensor_to_f64(out)[reqs], ref_o[reqs], "variant of the root")
    assert B.gf_node_kv_release(pa.g, 0, pa.stream) == B.GF_ERR_INVALID_ARG      # the variant needs its tiles
    assert B.gf_node_kv_write(pa.g, n0, 0, 16, 16, int(w2.node_len[n0]), pa.stream) == B.GF_ERR_INVALID_ARG
    assert B.gf_node_kv_attach_residual(pa.g, 5, 0, n0, None, None, pa.stream) == B.GF_ERR_INVALID_ARG  # variant of a variant
    assert B.gf_node_kv_release(pa.g, n0, pa.stream) == B.GF_OK
    assert B.gf_node_extent(pa.g, n0)[0] == B.GF_ERR_NOT_WRITTEN
    _, _, pk, pv = res[0]
    assert B.gf_node_kv_attach_residual(pa.g, n0, 0, 0, pk, pv, pa.stream) == B.GF_OK   # the single row is free again
    assert B.gf_node_kv_attach_residual(pa.g, n0 - 1, 0, 0, pk, pv, pa.stream) in (B.GF_ERR_CAPACITY, B.GF_ERR_INVALID_ARG)
    pa.build()
    again = pa.decode(0, pa.make_q(0))
    assert pa.status() == 0
    assert np.array_equal(again.view(torch.int16).cpu().numpy(), bits)
    pa.close()


def test_extend_rejects_paths_through_attached_nodes():
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    w = W.make_config(2, n_requests=4, new_len=40, root_len=200, len_lo=16, len_hi=64, prefix_lo=200, prefix_hi=400,
                      group_lo=2, group_hi=2)
    n0 = w.num_nodes
    w2 = dataclasses.replace(w, num_nodes=n0 + 1, node_len=np.append(w.node_len, w.node_len[0]))
    pa = PathAttention(w2, layers=1, max_residual_nodes=1)
    pa.write_nodes("device", skip={n0})
    B.check(B.gf_node_kv_attach_residual(pa.g, n0, 0, 0, None, None, pa.stream), "attach")
    path_node = w.path_node.copy()
    path_node[w.path_ptr[2]] = n0
    pa.path_node = torch.from_numpy(path_node.astype(np.int32)).to(pa.dev)
    with pytest.raises(B.GfError) as e:
        pa.build()
    assert e.value.status == B.GF_ERR_INVALID_PATH and B.gf_tables_bad_request(pa.tables) == 2
    pa.close()
