"""Differential KV, the encoding side (Sec. 5.1): gf_residual_encode bit for bit against the oracle, and
the round trip encode -> reconstruct through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import residual as OR
from paper_2605_22566_b200 import workloads as W
from test_gpu_residual import _read_node, _setup

pytestmark = pytest.mark.gpu


def _full_state(w, base_node, kind_big, kind_tiny):
    """A prefix-conditioned state of the node: its base plus a sparse large change plus a dense tiny one."""
    rows = int(w.node_len[base_node]) * w.num_kv_heads
    k, v = w.node_kv_bits(0, base_node)
    out = []
    for bits, salt in ((k, 1), (v, 2)):
        b = bits.reshape(rows, w.head_dim)
        big = W.residual_stream(w.seed + salt, kind_big, 0, base_node, 1, rows, w.head_dim, 0.25, sigma=0.25)
        tiny = W.residual_stream(w.seed + salt, kind_tiny, 0, base_node, 2, rows, w.head_dim, 0.6, sigma=2.0 ** -12)
        out.append((b, OR.reconstruct(OR.reconstruct(b, *big), *tiny)))
    return out  # [(k_base, k_full), (v_base, v_full)], each uint16[rows, D]


def _bufs(rows, D, capacity, dev):
    t = dict(bitmap=torch.full((rows * (D // 32),), -1, dtype=torch.int32, device=dev),
             values=torch.full((max(capacity, 1),), -1, dtype=torch.int16, device=dev),
             row_ptr=torch.full((rows + 1,), -1, dtype=torch.int32, device=dev),
             nnz=torch.full((1,), -1, dtype=torch.int64, device=dev))
    return t, (t["bitmap"].data_ptr(), t["values"].data_ptr(), t["row_ptr"].data_ptr(), capacity, t["nnz"].data_ptr())


def _as_host(t, rows, D):
    nnz = int(t["nnz"].item())
    return (t["bitmap"].cpu().numpy().view(np.uint32).reshape(rows, D // 32),
            t["values"].cpu().numpy().view(np.uint16)[:nnz], t["row_ptr"].cpu().numpy(), nnz)


@pytest.mark.parametrize("cfg,tau", [
    (dict(config_id=0), 2.0 ** -8),
    (dict(config_id=1, n_requests=24, n_nodes=48, root_len=333, len_lo=1, len_hi=150, suffix_max=40), 2.0 ** -8),
    (dict(config_id=1, n_requests=24, n_nodes=48, root_len=200, len_lo=1, len_hi=90, suffix_max=40), 0.0),
])
def test_encode_bit_exact_and_round_trip(cfg, tau):
    from paper_2605_22566_b200 import binding as B
    w, pa, bases, variants = _setup(cfg, n_var=3)
    D = w.head_dim
    for b, v in zip(bases, variants):
        (kb, kf), (vb, vf) = _full_state(w, b, W.KIND_DK, W.KIND_DV)
        rows = kb.shape[0]
        d_kf = torch.from_numpy(kf.view(np.int16).copy()).to(pa.dev)
        d_vf = torch.from_numpy(vf.view(np.int16).copy()).to(pa.dev)
        tk, pk = _bufs(rows, D, rows * D, pa.dev)
        tv, pv = _bufs(rows, D, rows * D, pa.dev)
        B.check(B.gf_residual_encode(pa.g, b, 0, d_kf.data_ptr(), d_vf.data_ptr(), tau, pk, pv, pa.stream), "gf_residual_encode")
        torch.cuda.synchronize()
        assert pa.status() == 0
        for t, base, full in ((tk, kb, kf), (tv, vb, vf)):
            bm, vals, rp, nnz = _as_host(t, rows, D)
            rbm, rvals, rrp = OR.encode(base, full, tau)
            assert np.array_equal(bm, rbm) and np.array_equal(rp, rrp) and nnz == int(rrp[-1])
            assert np.array_equal(vals, rvals)
        # the round trip on the device: what was encoded, applied to the base, is the oracle's round trip
        rk = (tk["bitmap"].data_ptr(), tk["values"].data_ptr(), tk["row_ptr"].data_ptr(), int(tk["nnz"].item()))
        rv = (tv["bitmap"].data_ptr(), tv["values"].data_ptr(), tv["row_ptr"].data_ptr(), int(tv["nnz"].item()))
        B.check(B.gf_node_kv_reconstruct(pa.g, v, 0, b, rk, rv, pa.stream), "gf_node_kv_reconstruct")
        got_k, got_v = _read_node(pa, v)
        want_k = OR.reconstruct(kb, *OR.encode(kb, kf, tau))
        want_v = OR.reconstruct(vb, *OR.encode(vb, vf, tau))
        assert np.array_equal(got_k.reshape(rows, D), want_k) and np.array_equal(got_v.reshape(rows, D), want_v)
        err = np.abs(OR.bf16_to_f64(want_k) - OR.bf16_to_f64(kf)).max()
        assert err <= tau * 1.01 + 2.0 ** -6  # dropped entries change the state by at most the threshold
    pa.close()


def test_encode_reports_a_value_array_that_is_too_small_and_rejects_bad_arguments():
    from paper_2605_22566_b200 import binding as B
    w, pa, bases, variants = _setup(dict(config_id=0), n_var=1)
    b = bases[0]
    (kb, kf), _ = _full_state(w, b, W.KIND_DK, W.KIND_DV)
    rows, D = kb.shape
    d_kf = torch.from_numpy(kf.view(np.int16).copy()).to(pa.dev)
    need = int(OR.encode(kb, kf, 0.0)[2][-1])
    tk, pk = _bufs(rows, D, need // 2, pa.dev)
    B.check(B.gf_residual_encode(pa.g, b, 0, d_kf.data_ptr(), 0, 0.0, pk, None, pa.stream), "gf_residual_encode")
    torch.cuda.synchronize()
    assert pa.status() == B.GF_ERR_CAPACITY
    assert int(tk["nnz"].item()) == need                       # the number needed is still reported
    assert B.gf_residual_encode(pa.g, variants[0], 0, d_kf.data_ptr(), 0, 0.0, pk, None, pa.stream) == B.GF_ERR_NOT_WRITTEN  # never written
    assert B.gf_residual_encode(pa.g, b, 0, 0, 0, 0.0, pk, None, pa.stream) == B.GF_ERR_INVALID_ARG   # no state given
    assert B.gf_residual_encode(pa.g, b, 0, d_kf.data_ptr(), 0, -1.0, pk, None, pa.stream) == B.GF_ERR_INVALID_ARG
    pa.close()
