"""Device-memory plumbing around the C-ABI calls: allocates the KV pool / workspace with torch,
uploads a workload's wGraph, node KV and paths, and forwards to the library.  No attention or
table arithmetic lives here; PyTorch only supplies memory and streams."""
from __future__ import annotations

import weakref
from typing import Optional

import numpy as np
import torch

from . import binding as B
from . import workloads as W

GUARD_BYTES = 4096   # canary band on either side of every buffer the library is given
GUARD_VALUE = 0xA5
_live = weakref.WeakSet()


def verify_all_guards() -> None:
    """Checks the canary bands of every live PathAttention (an out-of-bounds write by a kernel lands
    there first); raises AssertionError naming the buffer."""
    for pa in list(_live):
        pa.verify_guards()


def _bits_to_tensor(bits: np.ndarray, device) -> torch.Tensor:
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def tensor_to_f64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to(torch.float64).cpu().numpy()


class PathAttention:
    """One wGraph handle with its pool and workspace, fed from a `workloads.Workload`."""

    def __init__(self, w: W.Workload, device: str = "cuda:0", layers: Optional[int] = None,
                 policy: Optional[tuple] = None, extra_tiles: int = 0, max_residual_nodes: int = 0):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required (the path has no CPU fallback)")
        self.w = w
        self.dev = torch.device(device)
        torch.cuda.set_device(self.dev)
        self.layers = w.num_layers if layers is None else layers
        self.policy = policy
        chunk = policy[0] if policy is not None else 256
        used = w.used_nodes()
        tiles = int(((w.node_len[used].astype(np.int64) + B.GF_TILE_TOKENS - 1) // B.GF_TILE_TOKENS).sum())
        tiles = max(tiles + extra_tiles, 1)
        self.pool_bytes = tiles * B.gf_pool_bytes_per_tile(w.head_dim) * w.num_kv_heads * self.layers
        self._guards = []
        # the pool must start on a 1024-byte boundary; the caching allocator only promises 512
        self.pool = self.guarded(self.pool_bytes, "kv pool", align=1024)
        pair_len = w.node_len[w.path_node].astype(np.int64)
        max_slots = int(((pair_len + chunk - 1) // chunk).sum()) + 1
        max_items = max_slots
        self.ws_bytes = B.gf_workspace_bytes(w.num_nodes, len(w.edge_src), w.num_requests,
                                             len(w.path_node), max_items, max_slots, w.num_q_heads,
                                             w.head_dim) + 64 * max_residual_nodes * self.layers + 256
        self.ws = self.guarded(self.ws_bytes, "workspace", align=256)
        st, self.g = B.gf_wgraph_create(
            num_nodes=w.num_nodes, num_shared_nodes=w.num_shared_nodes, edge_src=w.edge_src,
            edge_dst=w.edge_dst, num_layers=self.layers, num_q_heads=w.num_q_heads,
            num_kv_heads=w.num_kv_heads, head_dim=w.head_dim, kv_pool_ptr=self.pool.data_ptr(),
            kv_pool_bytes=self.pool_bytes, workspace_ptr=self.ws.data_ptr(), workspace_bytes=self.ws_bytes,
            max_residual_nodes=max_residual_nodes)
        B.check(st, "gf_wgraph_create")
        self.path_ptr = torch.from_numpy(w.path_ptr.astype(np.int32)).to(self.dev)
        self.path_node = torch.from_numpy(w.path_node.astype(np.int32)).to(self.dev)
        self.tables = None
        self._qtab = None
        _live.add(self)

    def guarded(self, nbytes: int, name: str, align: int = 256) -> torch.Tensor:
        """A uint8 device buffer of nbytes with a canary band before and after it."""
        raw = torch.empty(nbytes + 2 * GUARD_BYTES + align, dtype=torch.uint8, device=self.dev)
        lo = GUARD_BYTES + (-(raw.data_ptr() + GUARD_BYTES)) % align
        raw[lo - GUARD_BYTES:lo].fill_(GUARD_VALUE)
        raw[lo + nbytes:lo + nbytes + GUARD_BYTES].fill_(GUARD_VALUE)
        self._guards.append((name, raw, lo, nbytes))
        return raw[lo:lo + nbytes]

    def guarded_like(self, t: torch.Tensor, name: str) -> torch.Tensor:
        return self.guarded(t.numel() * t.element_size(), name).view(t.dtype).view(t.shape)

    def verify_guards(self) -> None:
        if not self._guards:
            return
        torch.cuda.synchronize(self.dev)
        for name, raw, lo, nbytes in self._guards:
            before = raw[lo - GUARD_BYTES:lo]
            after = raw[lo + nbytes:lo + nbytes + GUARD_BYTES]
            assert bool((before == GUARD_VALUE).all()), f"canary before the {name} was overwritten"
            assert bool((after == GUARD_VALUE).all()), f"canary after the {name} was overwritten"

    def close(self):
        if self.g is not None:
            self.verify_guards()
            B.gf_wgraph_destroy(self.g)
            self.g = None
            self._guards = []

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def stream(self) -> int:
        return torch.cuda.current_stream(self.dev).cuda_stream

    # ---- inputs -------------------------------------------------------------------------
    def _fill(self, key: int, count: int, out: torch.Tensor, start: int = 0):
        if self._qtab is None:
            self._qtab = torch.from_numpy(W.quantile_table().view(np.int16)).to(self.dev)
        if B.gfgen_fill_bf16(self._qtab.data_ptr(), key, start, count, out.data_ptr(), self.stream) != 0:
            raise RuntimeError("input fill kernel failed to launch")

    def write_nodes(self, source: str = "device", skip=(), only=None):
        """gf_node_kv_write for every used node (except those in `skip`; or exactly the nodes in `only`)
        and every materialised layer.  source="device" generates the bits with the fill kernel, "host"
        with numpy (identical bits)."""
        w = self.w
        used = w.used_nodes() if only is None else np.asarray(sorted(only), dtype=np.int64)
        if len(skip):
            used = used[~np.isin(used, list(skip))]
        if len(used) == 0:
            return
        per_tok = w.num_kv_heads * w.head_dim
        nmax = int(w.node_len[used].max())
        kbuf = torch.empty(nmax * per_tok, dtype=torch.bfloat16, device=self.dev)
        vbuf = torch.empty(nmax * per_tok, dtype=torch.bfloat16, device=self.dev)
        for layer in range(self.layers):
            for v in used.tolist():
                n = int(w.node_len[v])
                if source == "device":
                    self._fill(W.stream_key(w.seed, W.KIND_K, layer, v), n * per_tok, kbuf)
                    self._fill(W.stream_key(w.seed, W.KIND_V, layer, v), n * per_tok, vbuf)
                    if w.v_scale_log2:
                        vbuf[:n * per_tok].mul_(2.0 ** w.v_scale_log2)  # a power of two: exact in bf16
                    for token, kvh, row in w.planted_rows(layer, v):  # inputs with planted key rows
                        at = (token * w.num_kv_heads + kvh) * w.head_dim
                        kbuf[at:at + w.head_dim].copy_(_bits_to_tensor(row, self.dev))
                    kp, vp = kbuf.data_ptr(), vbuf.data_ptr()
                else:
                    kb, vb = w.node_kv_bits(layer, v)
                    kt, vt = _bits_to_tensor(kb, self.dev), _bits_to_tensor(vb, self.dev)
                    kp, vp = kt.data_ptr(), vt.data_ptr()
                B.check(B.gf_node_kv_write(self.g, v, layer, kp, vp, n, self.stream), "gf_node_kv_write")
                if source != "device":
                    torch.cuda.current_stream(self.dev).synchronize()  # kt/vt are freed next turn
        torch.cuda.current_stream(self.dev).synchronize()

    def new_nodes(self):
        """The last node of every path: in an extend batch, the request's new segment."""
        w = self.w
        return [int(w.path_node[w.path_ptr[r + 1] - 1]) for r in range(w.num_requests)]

    def write_prefix_nodes(self, source: str = "device"):
        """Like write_nodes, but the requests' new segments are only reserved (their K/V arrive with
        gf_path_attention_extend_append)."""
        w = self.w
        new = set(self.new_nodes())
        self.write_nodes(source, skip=new)
        for v in sorted(new):
            B.check(B.gf_node_kv_reserve(self.g, v, int(w.node_len[v]), self.stream), "gf_node_kv_reserve")

    def new_kv(self, layer: int):
        """K and V of the new segments, request-major rows in the order of the queries: two tensors
        [num_q_rows, Hkv, D] (generated on the host, identical bits to what write_nodes stores)."""
        w = self.w
        ks, vs = [], []
        for v in self.new_nodes():
            kb, vb = w.node_kv_bits(layer, v)
            ks.append(kb)
            vs.append(vb)
        return (_bits_to_tensor(np.concatenate(ks, axis=0), self.dev), _bits_to_tensor(np.concatenate(vs, axis=0), self.dev))

    def make_q(self, layer: int, source: str = "device") -> torch.Tensor:
        w = self.w
        rows = int(w.q_row_ptr()[-1])
        if source == "device":
            q = torch.empty((rows, w.num_q_heads, w.head_dim), dtype=torch.bfloat16, device=self.dev)
            self._fill(W.stream_key(w.seed, W.KIND_Q, layer, 0), q.numel(), q)
            if w.q_scale_log2:
                q.mul_(2.0 ** w.q_scale_log2)  # a power of two: exact in bf16
            return q
        return _bits_to_tensor(w.q_bits(layer), self.dev)

    # ---- the path ---------------------------------------------------------------------------
    def build(self, mode: Optional[int] = None, deferred: bool = False):
        """gf_build_path_tables.  deferred=True (decode only) enqueues the build without waiting and
        returns None; sizes and errors are then reported by info() / status()."""
        w = self.w
        if mode is None:
            mode = B.GF_MODE_EXTEND if w.mode == "extend" else B.GF_MODE_DECODE
        if deferred:
            mode |= B.GF_MODE_DEFERRED
        st, t = B.gf_build_path_tables(self.g, w.num_requests, len(w.path_node), self.path_ptr.data_ptr(),
                                       self.path_node.data_ptr(), mode, self.policy, self.stream)
        self.tables = t
        B.check(st, "gf_build_path_tables")
        return None if deferred else B.gf_tables_info(t)

    def info(self):
        return B.gf_tables_info(self.tables)

    def decode(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None):
        if out is None:
            out = self.guarded_like(q, "decode output")
        B.check(B.gf_path_attention_decode(self.g, self.tables, layer, q.data_ptr(), out.data_ptr(),
                                           None if lse is None else lse.data_ptr(), self.stream),
                "gf_path_attention_decode")
        return out

    def extend(self, layer: int, q: torch.Tensor, out: Optional[torch.Tensor] = None,
               lse: Optional[torch.Tensor] = None):
        if out is None:
            out = self.guarded_like(q, "extend output")
        B.check(B.gf_path_attention_extend(self.g, self.tables, layer, q.data_ptr(), out.data_ptr(),
                                           None if lse is None else lse.data_ptr(), self.stream),
                "gf_path_attention_extend")
        return out

    def extend_append(self, layer: int, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor,
                      out: Optional[torch.Tensor] = None, lse: Optional[torch.Tensor] = None):
        if out is None:
            out = self.guarded_like(q, "extend output")
        B.check(B.gf_path_attention_extend_append(self.g, self.tables, layer, q.data_ptr(), k_new.data_ptr(),
                                                  v_new.data_ptr(), out.data_ptr(),
                                                  None if lse is None else lse.data_ptr(), self.stream),
                "gf_path_attention_extend_append")
        return out

    def read_node(self, node: int, layer: int):
        """gf_node_kv_read: (K, V) uint16 bit patterns [len, Hkv, D] of a node's layer."""
        w = self.w
        st, n, _ = B.gf_node_extent(self.g, node)
        B.check(st, "gf_node_extent")
        k = torch.empty((max(n, 1), w.num_kv_heads, w.head_dim), dtype=torch.bfloat16, device=self.dev)
        v = torch.empty_like(k)
        B.check(B.gf_node_kv_read(self.g, node, layer, k.data_ptr(), v.data_ptr(), self.stream), "gf_node_kv_read")
        torch.cuda.current_stream(self.dev).synchronize()
        return (k[:n].view(torch.int16).cpu().numpy().view(np.uint16), v[:n].view(torch.int16).cpu().numpy().view(np.uint16))

    def edge_scores(self, inputs: dict, tasks_per_pass: Optional[int] = None) -> torch.Tensor:
        """gf_edge_scores over `inputs` (see workloads.scoring_inputs): fp32 [num_tasks, num_edges]."""
        t = {k: torch.from_numpy(np.ascontiguousarray(v)).to(self.dev) for k, v in inputs.items() if k != "b3"}
        sc = B.Scorer(inputs["w_gcn1"].shape[0], inputs["w_gcn1"].shape[1], inputs["w2"].shape[0],
                      t["w_gcn1"].data_ptr(), t["w_gcn2"].data_ptr(), t["w1"].data_ptr(), t["b1"].data_ptr(),
                      t["w2"].data_ptr(), t["b2"].data_ptr(), t["w3"].data_ptr(), float(inputs["b3"]))
        nt = inputs["x_task"].shape[0]
        nbytes = B.gf_edge_scores_scratch_bytes(self.g, sc, nt, nt if tasks_per_pass is None else tasks_per_pass)
        scratch = self.guarded(nbytes, "scoring scratch")
        scores = self.guarded(nt * len(self.w.edge_src) * 4, "edge scores").view(torch.float32).view(nt, len(self.w.edge_src))
        B.check(B.gf_edge_scores(self.g, sc, t["x_op"].data_ptr(), nt, t["x_task"].data_ptr(), scores.data_ptr(),
                                 scratch.data_ptr(), nbytes, self.stream), "gf_edge_scores")
        torch.cuda.current_stream(self.dev).synchronize()   # the inputs in `t` are freed on return
        return scores

    def status(self) -> int:
        return B.gf_last_status(self.g, self.stream)
