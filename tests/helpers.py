"""Shared test helpers: oracle-side views of a workload and the parity gate."""
import numpy as np

from oracle import attention as OA
from oracle import tables as OT
from paper_2605_22566_b200 import workloads as W

MAX_ABS = 1e-2   # tolerance for bf16 inputs with fp32 accumulation (bf16 output rounding, bf16 P, ex2.approx)
REL_L2 = 5e-3


class OracleView:
    """fp64 node KV / queries of a workload, converted exactly from the bf16 bit patterns."""

    def __init__(self, w, layer=0):
        self.w, self.layer, self._cache = w, layer, {}

    def node_kv(self, v):
        if v not in self._cache:
            k, vv = self.w.node_kv_bits(self.layer, v)
            self._cache[v] = (W.bf16_bits_to_f64(k), W.bf16_bits_to_f64(vv))
        return self._cache[v]

    def q(self):
        return W.bf16_bits_to_f64(self.w.q_bits(self.layer))

    def paths(self, reqs=None):
        reqs = range(self.w.num_requests) if reqs is None else reqs
        return [[v for v in self.w.path(r).tolist() if self.w.node_len[v] > 0] for r in reqs]

    def decode(self, reqs=None):
        reqs = list(range(self.w.num_requests)) if reqs is None else list(reqs)
        return OA.decode(self.paths(reqs), self.node_kv, self.q()[reqs], self.w.num_kv_heads)

    def extend(self, rows=None):
        return OA.extend(self.paths(), self.node_kv, self.q(), self.w.num_kv_heads, rows=rows)


def oracle_tables(w, policy=None, mode=None):
    pol = OT.Policy() if policy is None else OT.Policy(*policy)
    order = [v for v in w.used_nodes().tolist()]
    off, _ = OT.pool_offsets(order, w.node_len, w.num_nodes)
    mode = (OT.MODE_EXTEND if w.mode == "extend" else OT.MODE_DECODE) if mode is None else mode
    return OT.build_tables(w.num_nodes, w.num_shared_nodes, w.edge_src, w.edge_dst, w.node_len, off,
                           w.path_ptr, w.path_node, pol, mode)


def assert_tables_equal(got: dict, ref: dict):
    for key, val in ref.items():
        if isinstance(val, np.ndarray):
            assert key in got, key
            assert got[key].shape == val.shape, (key, got[key].shape, val.shape)
            assert np.array_equal(got[key], val), key
        else:
            assert int(got[key]) == int(val), (key, got[key], val)


def assert_close(got, ref, what=""):
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    assert np.all(np.isfinite(got)), f"{what}: non-finite output"
    max_abs = float(np.abs(got - ref).max())
    rel = float(np.linalg.norm((got - ref).ravel()) / max(np.linalg.norm(ref.ravel()), 1e-300))
    assert max_abs <= MAX_ABS and rel <= REL_L2, f"{what}: max_abs={max_abs:.3e} rel_l2={rel:.3e}"
    return max_abs, rel
