"""Parity on inputs with a large dynamic range of scores (peaked softmax), for all three attention
kernels: queries scaled by a power of two and, for chosen query rows, a key aligned with the query
planted in a late stage of a late segment, so that the running maximum jumps by tens to hundreds of
log2 units in the middle of a walk.  Outputs are O(1) here, so the absolute gate is a 1 % gate.
Values are scaled by 1/4 so that |out| stays below 2, where a bf16 output can be within 1e-2 at all
(half a bf16 ulp is 0.0156 above 4)."""
import numpy as np
import pytest
import torch

from helpers import OracleView, assert_close
from paper_2605_22566_b200 import workloads as W

pytestmark = pytest.mark.gpu


def _lse_close(got, ref):
    assert np.all(np.abs(got - ref) <= 2e-3 + 2e-6 * np.abs(ref)), float(np.abs(got - ref).max())


def _peaked_extend(qs, ps):
    w = W.make_config(2, n_requests=6, new_len=200, root_len=300, len_lo=150, len_hi=400, prefix_lo=600,
                      prefix_hi=1500, group_lo=2, group_hi=3)
    w.q_scale_log2, w.v_scale_log2 = qs, -2
    qp = w.q_row_ptr()
    rng = np.random.default_rng(5)
    pl = []
    for r in range(w.num_requests):
        path = w.path(r)
        node = int(path[-2])  # the last shared node: a late token of it, for query row 150 of the request
        pl.append((int(qp[r]) + 150, int(rng.integers(0, w.num_q_heads)), node, int(w.node_len[node]) - 3, ps))
        # and inside the new (causal) segment: key 140 aligned with query row 180
        pl.append((int(qp[r]) + 180, int(rng.integers(0, w.num_q_heads)), int(path[-1]), 140, ps))
    w.planted = tuple(pl)
    return w


@pytest.mark.parametrize("qs,ps", [(3, -1), (3, 0), (5, 1)])
def test_extend_peaked_all_rows(qs, ps):
    """(3, -1): jumps of some tens of log2 units; (3, 0): about a hundred; (5, 1): a planted score near
    820 nats, more than 2^1000 above the scores before it."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = _peaked_extend(qs, ps)
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    pa.build()
    q = pa.make_q(0)
    lse = torch.empty(q.shape[:2], dtype=torch.float32, device=pa.dev)
    B.gf_debug_counters(pa.g, pa.stream)
    out = pa.extend(0, q, lse=lse)
    assert pa.status() == 0
    counters = B.gf_debug_counters(pa.g, pa.stream)
    assert counters["softmax_reference_moves"] > 0, "no tile moved its softmax reference after its first stage"
    if (qs, ps) == (5, 1):  # far beyond what the walk against a lagging maximum may keep: walked again, exactly
        assert counters["exact_reruns"] > 0
    ref_o, ref_l = OracleView(w).extend()
    assert np.abs(ref_o).max() > 0.5  # peaked: outputs are single value rows, not means
    assert_close(tensor_to_f64(out), ref_o, f"peaked extend q*2^{qs}, planted*2^{ps}")
    _lse_close(tensor_to_f64(lse), ref_l)
    pa.close()


def test_extend_flat_inputs_are_walked_once():
    """Scores of ordinary range never send a CTA into its second, exact walk."""
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = _peaked_extend(0, 0)
    w.planted = ()
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    pa.build()
    B.gf_debug_counters(pa.g, pa.stream)
    out = pa.extend(0, pa.make_q(0))
    assert pa.status() == 0
    assert B.gf_debug_counters(pa.g, pa.stream)["exact_reruns"] == 0
    ref_o, _ = OracleView(w).extend()
    assert_close(tensor_to_f64(out), ref_o, "extend, flat inputs")
    pa.close()


def test_extend_host_written_inputs_match_device_written():
    """The planted rows and scalings reach the pool identically from the host and the device generator."""
    from paper_2605_22566_b200.runtime import PathAttention
    w = _peaked_extend(3, 0)
    outs = []
    for source in ("device", "host"):
        pa = PathAttention(w, layers=1)
        pa.write_nodes(source)
        pa.build()
        outs.append(pa.extend(0, pa.make_q(0, source)).view(torch.int16).cpu().numpy())
        assert pa.status() == 0
        pa.close()
    assert np.array_equal(outs[0], outs[1])


def test_extend_path_longer_than_the_cached_geometry():
    """A path of more than 48 segments: the walk reads the geometry of the later ones from global memory."""
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    w = W.make_config(2, n_requests=3, new_len=70, root_len=20, len_lo=5, len_hi=30, prefix_lo=1200,
                      prefix_hi=1200, group_lo=3, group_hi=3, hq=8, hkv=2, d=128)
    assert int(np.diff(w.path_ptr).max()) > 50
    w.q_scale_log2, w.v_scale_log2 = 2, -2
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    info = pa.build()
    q = pa.make_q(0)
    out = pa.extend(0, q)
    assert pa.status() == 0
    ref_o, _ = OracleView(w).extend()
    assert_close(tensor_to_f64(out), ref_o, "extend over 60+ segments")
    pa.close()


def _decode(w, check_moves=False):
    from paper_2605_22566_b200 import binding as B
    from paper_2605_22566_b200.runtime import PathAttention, tensor_to_f64
    pa = PathAttention(w, layers=1)
    pa.write_nodes("device")
    pa.build()
    q = pa.make_q(0)
    lse = torch.empty((w.num_requests, w.num_q_heads), dtype=torch.float32, device=pa.dev)
    B.gf_debug_counters(pa.g, pa.stream)
    out = pa.decode(0, q, lse=lse)
    assert pa.status() == 0
    counters = B.gf_debug_counters(pa.g, pa.stream)
    pa.close()
    _decode.last_counters = counters
    return tensor_to_f64(out), tensor_to_f64(lse), counters["softmax_reference_moves"]


@pytest.mark.parametrize("qs,ps", [(3, 0), (5, 1)])
def test_decode_wide_chunks_peaked(qs, ps):
    """Segments shared by 65..420 requests (the tensor-memory decode kernel), keys planted in the last
    stage of the root's single 700-token chunk and of a second-level node."""
    w = W.make_config(1, n_requests=420, n_nodes=12, root_len=700, len_lo=65, len_hi=400, depth_lo=3, depth_hi=4,
                      suffix_max=30)
    w.q_scale_log2, w.v_scale_log2 = qs, -2
    reqs = np.random.default_rng(29).choice(w.num_requests, size=24, replace=False).tolist()
    pl = []
    for i, r in enumerate(reqs[:12]):
        node = 0 if i % 2 == 0 else int(w.path(r)[1])
        pl.append((r, (5 * i + 3) % w.num_q_heads, node, int(w.node_len[node]) - 1 - i, ps))
    w.planted = tuple(pl)
    out, lse, moves = _decode(w)
    assert moves > 0
    if (qs, ps) == (5, 1):  # beyond what the lagging reference may keep: the exact kernel redid the launch
        assert _decode.last_counters["exact_reruns"] > 0
    ref_o, ref_l = OracleView(w).decode(reqs)
    assert np.abs(ref_o).max() > 0.5
    assert_close(out[reqs], ref_o, "peaked wide decode")
    _lse_close(lse[reqs], ref_l)
    assert np.all(np.isfinite(out))


@pytest.mark.parametrize("qs,ps", [(3, 0), (5, 1)])
def test_decode_warp_kernel_peaked(qs, ps):
    """Lightly shared segments (the warp kernel, exact running maximum), all requests."""
    w = W.make_config(1, n_requests=40, n_nodes=64, root_len=333, len_lo=1, len_hi=200, suffix_max=70)
    w.q_scale_log2, w.v_scale_log2 = qs, -2
    pl = []
    for r in range(0, w.num_requests, 3):
        path = [int(v) for v in w.path(r) if w.node_len[v] > 0]
        node = path[-1] if r % 2 else path[len(path) // 2]
        pl.append((r, (7 * r + 1) % w.num_q_heads, node, int(w.node_len[node]) - 1, ps))
    w.planted = tuple(pl)
    out, lse, _ = _decode(w)
    ref_o, ref_l = OracleView(w).decode()
    assert np.abs(ref_o).max() > 0.5
    assert_close(out, ref_o, "peaked warp-kernel decode")
    _lse_close(lse, ref_l)
