"""K3 parity: extend / prefill through the C ABI against the fp64 oracle."""
import numpy as np
import pytest
import torch

from helpers import OracleView, assert_close
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _run_extend(w, source="device"):
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    pa = PathAttention(w, layers=1)
    pa.write_nodes(source)
    info = pa.build()
    q = pa.make_q(0, source)
    assert info.num_q_rows == q.shape[0]
    lse = pa.guarded(q.shape[0] * q.shape[1] * 4, "lse").view(torch.float32).view(q.shape[0], q.shape[1])
    out = pa.extend(0, q, lse=lse)
    assert pa.status() == 0
    res = tensor_to_f64(out), tensor_to_f64(lse)
    pa.close()
    return res


@pytest.mark.parametrize("hq,hkv,d,new_len", [(4, 4, 64, 37), (8, 2, 64, 64), (32, 8, 128, 50), (8, 1, 128, 9)])
def test_small_extend_all_rows(hq, hkv, d, new_len):
    w = W.make_config(2, n_requests=6, new_len=new_len, root_len=150, len_lo=10, len_hi=90, prefix_lo=150,
                      prefix_hi=500, group_lo=2, group_hi=3, hq=hq, hkv=hkv, d=d)
    out, lse = _run_extend(w)
    ref_o, ref_l = OracleView(w).extend()
    assert_close(out, ref_o, f"extend {hq}/{hkv}/{d}")
    assert np.abs(lse - ref_l).max() < 2e-3


def test_single_node_extend_is_causal_self_attention():
    w = W.make_config(2, n_requests=2, new_len=130, root_len=64, len_lo=10, len_hi=20, prefix_lo=64,
                      prefix_hi=64, group_lo=1, group_hi=1, hq=8, hkv=2, d=128)
    # drop the prefix: each path is just its new node
    R = w.num_requests
    w.path_node = w.path_node[w.path_ptr[1:] - 1].copy()
    w.path_ptr = np.arange(R + 1, dtype=np.int32)
    out, _ = _run_extend(w, source="host")
    ref_o, _ = OracleView(w).extend()
    assert_close(out, ref_o, "single-node extend")
    # first token of each request sees only itself: output equals its own V row (GQA head map)
    qp = w.q_row_ptr()
    for r in range(R):
        _, v = w.node_kv_bits(0, int(w.path_node[r]))
        v0 = W.bf16_bits_to_f64(v)[0]
        for h in range(8):
            assert np.array_equal(out[qp[r], h], v0[h // 4])


def test_config2_full_size_sampled_rows():
    w = W.make_config(2)
    out, lse = _run_extend(w)
    rng = np.random.default_rng(5)
    total = int(w.q_row_ptr()[-1])
    rows = sorted(set(rng.choice(total, size=44, replace=False).tolist()) | {0, 511, 512, total - 1})
    ref_o, ref_l = OracleView(w).extend(rows=rows)
    assert_close(out[rows], ref_o[rows], "cfg2 sampled rows")
    assert np.abs(lse[rows] - ref_l[rows]).max() < 2e-3
    assert np.all(np.isfinite(out))
