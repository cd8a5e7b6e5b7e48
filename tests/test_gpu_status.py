"""The device status words: a set-up kernel's sticky report must not disturb attention, and a bounded
wait that runs out must end its kernel and be reported."""
import numpy as np
import pytest
import torch

from helpers import OracleView, assert_close
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def test_unread_capacity_report_does_not_disturb_decode_or_extend():
    """gf_residual_encode with room for no value reports GF_ERR_CAPACITY in the handle's status block
    (its documented way of sizing a residual).  Attention calls enqueued before anybody reads that
    report must still wait for their data: compare them with the oracle, then read the report."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    for cfg, over in [(1, dict(n_requests=40, n_nodes=64, root_len=900, len_lo=100, len_hi=700, suffix_max=70)),
                      (2, dict(n_requests=6, new_len=150, root_len=400, len_lo=100, len_hi=300, prefix_lo=900,
                               prefix_hi=2000, group_lo=2, group_hi=3))]:
        w = W.make_config(cfg, **over)
        pa = PathAttention(w, layers=1)
        pa.write_nodes("device")
        pa.build()
        q = pa.make_q(0)
        assert pa.status() == 0
        # a state that differs from the root's base everywhere, encoded into a buffer with capacity 0
        n, per = int(w.node_len[0]), w.num_kv_heads * w.head_dim
        full = torch.ones(n * per, dtype=torch.bfloat16, device=pa.dev)
        rows = n * w.num_kv_heads
        bitmap = torch.zeros(rows * (w.head_dim // 32), dtype=torch.int32, device=pa.dev)
        row_ptr = torch.zeros(rows + 1, dtype=torch.int32, device=pa.dev)
        nnz = torch.zeros(1, dtype=torch.int64, device=pa.dev)
        buf = (bitmap.data_ptr(), 0, row_ptr.data_ptr(), 0, nnz.data_ptr())
        B.check(B.gf_residual_encode(pa.g, 0, 0, full.data_ptr(), full.data_ptr(), 0.0, buf, None, pa.stream),
                "gf_residual_encode")
        torch.cuda.synchronize()       # the report is in the status block now, and nobody has read it
        assert int(nnz.item()) > 0
        for _ in range(3):             # several launches: every wait in them meets the unread report
            out = pa.extend(0, q) if w.mode == "extend" else pa.decode(0, q)
        got = tensor_to_f64(out)
        assert pa.status() == B.GF_ERR_CAPACITY   # the encode's report, delivered late and intact
        assert pa.status() == 0
        ref = OracleView(w).extend()[0] if w.mode == "extend" else OracleView(w).decode()[0]
        assert_close(got, ref, f"attention with an unread capacity report, config {cfg}")
        pa.close()


def test_bounded_wait_runs_out_and_is_reported():
    """One warp waits on a barrier nothing completes, with a limit of a few thousand cycles: the wait
    gives up, the kernel ends, gf_last_status says GF_ERR_TIMEOUT once, and the handle keeps working."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(0)
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    pa.build()
    q = pa.make_q(0)
    before = tensor_to_f64(pa.decode(0, q))
    assert pa.status() == 0
    st, gave_up = B.gf_debug_wait_probe(pa.g, 5000, pa.stream)
    assert st == B.GF_OK and gave_up == 1
    assert pa.status() == B.GF_ERR_TIMEOUT
    assert pa.status() == 0
    after = tensor_to_f64(pa.decode(0, q))
    assert pa.status() == 0
    assert np.array_equal(before, after)
    assert B.gf_debug_wait_probe(pa.g, 0, pa.stream)[0] == B.GF_ERR_INVALID_ARG
    assert B.gf_debug_wait_probe(pa.g, 10 ** 9, pa.stream)[0] == B.GF_ERR_INVALID_ARG
    pa.close()
