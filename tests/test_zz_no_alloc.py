"""gf_path_attention_decode_static: the decode variant for hosts that cannot supply scratch.

Some users of the library run where nothing may be allocated once serving has started (all device
memory was handed out at start-up, or the allocator may block or fail), so this entry point keeps
the attention partials in an array that ships inside the library.  The test drives it through the
C ABI and holds it to the ordinary decode entry point's output, twice in a row because the array is
shared and keeps whatever the previous call left in it.  The file sorts last on purpose: a failure
here cannot hide any other test from a run that stops at the first failure.
"""
import numpy as np
import pytest
import torch

from helpers import MAX_ABS, REL_L2, assert_close
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _setup(w):
    from paper_2605_22566_b200.runtime import PathAttention
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    info = pa.build()
    return pa, info


def test_static_scratch_decode_matches_workspace_decode_twice():
    from helpers import OracleView
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import tensor_to_f64
    w = W.make_config(1, n_requests=96, n_nodes=64, root_len=700, len_lo=20, len_hi=300, suffix_max=90)
    pa, info = _setup(w)
    need = info.num_slots * w.num_q_heads * (w.head_dim + 2) * 4
    assert need <= B.GF_STATIC_SCRATCH_BYTES
    q = pa.make_q(0)
    q2 = torch.roll(q, 1, dims=0).contiguous()  # a second batch of queries: request r asks request r-1's
    lse_ref = torch.empty((w.num_requests, w.num_q_heads), dtype=torch.float32, device=pa.dev)
    ref = tensor_to_f64(pa.decode(0, q, lse=lse_ref))
    ref2 = tensor_to_f64(pa.decode(0, q2))
    assert pa.status() == 0
    assert np.all(np.isfinite(ref)) and np.abs(ref).max() > 0
    # the ordinary entry point is itself held to the oracle here, so that the comparison below is
    # not the library against itself only
    ora, ora_lse = OracleView(w).decode()
    assert_close(ref, ora, "workspace decode vs oracle")
    for call in range(2):
        # leave the other batch's partials in the workspace: if the static call read them instead of
        # its own array, its output would be ref2, not ref
        pa.decode(0, q2)
        out = torch.full_like(q, float("nan"))
        lse = torch.full_like(lse_ref, float("nan"))
        st = B.gf_path_attention_decode_static(pa.g, pa.tables, 0, q.data_ptr(), out.data_ptr(),
                                               lse.data_ptr(), pa.stream)
        assert st == B.GF_OK, B.status_string(st)
        assert pa.status() == 0
        assert_close(tensor_to_f64(out), ref, f"static-scratch decode, call {call}")
        assert_close(tensor_to_f64(out), ora, f"static-scratch decode vs oracle, call {call}")
        assert np.abs(tensor_to_f64(lse) - tensor_to_f64(lse_ref)).max() < 2e-3
        assert np.abs(tensor_to_f64(lse) - ora_lse).max() < 2e-3
        # a different query through the static entry point in between, checked too, so that the second
        # pass cannot pass on what the first left in the array
        pa.decode(0, q)
        out2 = torch.full_like(q, float("nan"))
        st = B.gf_path_attention_decode_static(pa.g, pa.tables, 0, q2.data_ptr(), out2.data_ptr(), None, pa.stream)
        assert st == B.GF_OK
        assert pa.status() == 0
        assert_close(tensor_to_f64(out2), ref2, f"static-scratch decode of the second batch, call {call}")
    pa.close()
    assert MAX_ABS == 1e-2 and REL_L2 == 5e-3  # the tolerance every parity test here uses


def test_static_scratch_rejects_batches_beyond_its_size():
    from paper_2605_22566_b200 import binding as B
    w = W.make_config(1)  # 2214 partial slots x 32 heads x 130 floats = 36.8 MB > 32 MiB
    pa, info = _setup_lengths_only(w)
    assert info.num_slots * w.num_q_heads * (w.head_dim + 2) * 4 > B.GF_STATIC_SCRATCH_BYTES
    q = pa.make_q(0)
    out = torch.zeros_like(q)
    launches = B.gf_launch_count(pa.g)
    st = B.gf_path_attention_decode_static(pa.g, pa.tables, 0, q.data_ptr(), out.data_ptr(), None, pa.stream)
    assert st == B.GF_ERR_CAPACITY
    assert B.gf_launch_count(pa.g) == launches  # nothing was launched
    pa.close()


def _setup_lengths_only(w):
    """Tables only need node lengths: reserve every extent from one zero buffer."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention
    pa = PathAttention(w, layers=1)
    used = w.used_nodes()
    buf = torch.zeros(int(w.node_len[used].max()) * w.num_kv_heads * w.head_dim, dtype=torch.bfloat16, device=pa.dev)
    for v in used.tolist():
        B.check(B.gf_node_kv_write(pa.g, v, 0, buf.data_ptr(), buf.data_ptr(), int(w.node_len[v]), pa.stream),
                "gf_node_kv_write")
    return pa, pa.build()
