"""Seeded synthetic inputs: wGraphs, request paths, and K/V/Q bit patterns.

This module produces *inputs only*.  It holds none of the method's arithmetic
(no attention, no table building) and is the one module that both the CPU
oracle's tests and the CUDA path's tests/bench draw their data from.

The paper's workloads are agent workflows instantiated from a shared operation
DAG (Sec. 3: wGraph = DAG of atomic operations; Sec. 5: one KV state per
operation node, assembled along the workflow).  The datasets behind them are
not available, so the five benchmark configurations are synthetic stand-ins
with the stated shapes: a layered random DAG, root-anchored paths, a private
suffix per request, N(0,1) values rounded to bf16.

Values are counter based: element `i` of stream `key` is
    QTAB[ splitmix64(key + (i+1)*GOLDEN) & 0xFFFF ]
where QTAB holds the 65 536 standard-normal quantiles at (j+0.5)/65536 rounded
to bf16 (round-to-nearest-even).  Any element of any tensor is therefore
reproducible on demand, on the host (numpy, here) or on the device (a fill
kernel that receives the same table as data), bit for bit.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Optional

import numpy as np

MASK64 = (1 << 64) - 1
GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

KIND_K, KIND_V, KIND_Q = 1, 2, 3
KIND_DK, KIND_DV, KIND_MASK = 4, 5, 6  # residual values of K / V, and which entries carry one

TILE_TOKENS = 64  # pool extents are reserved in multiples of this many tokens


# --------------------------------------------------------------------------
# counter-based value generator
# --------------------------------------------------------------------------
def mix64_int(z: int) -> int:
    """SplitMix64 output function on a Python int (public-domain algorithm)."""
    z &= MASK64
    z = ((z ^ (z >> 30)) * _C1) & MASK64
    z = ((z ^ (z >> 27)) * _C2) & MASK64
    return z ^ (z >> 31)


def mix64(z: np.ndarray) -> np.ndarray:
    """Vectorised SplitMix64 output function on uint64 arrays (wraps mod 2^64)."""
    z = z.astype(np.uint64, copy=True)
    z ^= z >> np.uint64(30)
    z *= np.uint64(_C1)
    z ^= z >> np.uint64(27)
    z *= np.uint64(_C2)
    z ^= z >> np.uint64(31)
    return z


def stream_key(seed: int, kind: int, layer: int, node: int) -> int:
    """64-bit key of one tensor stream (kind = K/V/Q, layer, node id)."""
    tag = ((kind & 0xFF) << 56) | ((layer & 0xFFFF) << 40) | (node & 0xFFFFFFFFFF)
    return mix64_int(mix64_int(seed) ^ tag)


_QTAB: Optional[np.ndarray] = None


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round-to-nearest-even (finite inputs)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (b + np.uint32(0x7FFF) + ((b >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to fp64."""
    return bf16_bits_to_f32(bits).astype(np.float64)


def quantile_table() -> np.ndarray:
    """uint16[65536]: bf16 bits of the N(0,1) quantiles at (j+0.5)/65536."""
    global _QTAB
    if _QTAB is None:
        from scipy.special import ndtri

        p = (np.arange(65536, dtype=np.float64) + 0.5) / 65536.0
        _QTAB = f32_to_bf16_bits(ndtri(p).astype(np.float32))
    return _QTAB


def scale_bits_pow2(bits: np.ndarray, k: int) -> np.ndarray:
    """bf16 bit patterns of the values times 2**k, exact: k is added to the exponent field (the
    inputs are non-zero normal numbers, as every table value is, and the result stays normal)."""
    if k == 0:
        return bits
    e = ((bits >> np.uint16(7)) & np.uint16(0xFF)).astype(np.int32)
    assert np.all(e > 0) and np.all(e + k > 0) and np.all(e + k < 255)
    return (bits.astype(np.int32) + (k << 7)).astype(np.uint16)


def fill_bits(key: int, start: int, count: int) -> np.ndarray:
    """bf16 bit patterns of elements [start, start+count) of stream `key`."""
    idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
    z = idx * np.uint64(GOLDEN) + np.uint64(key)
    return quantile_table()[(mix64(z) & np.uint64(0xFFFF)).astype(np.int64)]


def residual_stream(seed: int, kind: int, layer: int, node: int, prefix: int, rows: int, head_dim: int,
                    density: float, sigma: float = 0.125):
    """Seeded sparse residual of one tensor (K or V) of one node under one prefix, in the bitmap format.

    The logical tensor is [rows, head_dim] with rows = tokens x KV heads (token-major, the caller
    layout of a node write).  Entry (row, d) carries a value when the low 16 bits of its hash are
    below density * 65536; the value is sigma times a standard-normal quantile, rounded to bf16
    (zeros are replaced by the smallest table magnitude so that every listed entry is non-zero).
    Returns (bitmap uint32[rows, head_dim // 32], values uint16[nnz], row_ptr int32[rows + 1]):
    bit j of word w of a row marks entry d = 32 * w + j; values follow in (row, d) order; row_ptr is
    the exclusive prefix sum of the rows' counts.  Inputs only: no arithmetic of the method is here.
    """
    assert head_dim % 32 == 0
    n = rows * head_dim
    idx = np.arange(1, n + 1, dtype=np.uint64)
    mkey = stream_key(seed ^ (prefix * 0x632BE59BD9B4E019 & MASK64), KIND_MASK + 8 * kind, layer, node)
    vkey = stream_key(seed ^ (prefix * 0x632BE59BD9B4E019 & MASK64), kind, layer, node)
    hit = (mix64(idx * np.uint64(GOLDEN) + np.uint64(mkey)) & np.uint64(0xFFFF)) < np.uint64(int(density * 65536))
    q = bf16_bits_to_f32(quantile_table()[(mix64(idx * np.uint64(GOLDEN) + np.uint64(vkey)) & np.uint64(0xFFFF)).astype(np.int64)])
    vals = f32_to_bf16_bits((q * np.float32(sigma)).astype(np.float32))
    vals = np.where((vals & 0x7FFF) == 0, np.uint16(0x0080), vals).astype(np.uint16)  # never a zero value
    hit2 = hit.reshape(rows, head_dim)
    weights = (np.uint64(1) << np.arange(32, dtype=np.uint64))
    bitmap = (hit2.reshape(rows, head_dim // 32, 32).astype(np.uint64) * weights).sum(axis=2).astype(np.uint32)
    row_ptr = np.concatenate([[0], np.cumsum(hit2.sum(axis=1))]).astype(np.int32)
    return bitmap, vals[hit], row_ptr


# --------------------------------------------------------------------------
# workload container
# --------------------------------------------------------------------------
@dataclass
class Workload:
    name: str
    config_id: int
    seed: int
    mode: str  # "decode": one query token per request; "extend": last path node is new, causal
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    num_shared_nodes: int  # ids below this are wGraph operation nodes; the rest are private
    num_nodes: int
    edge_src: np.ndarray
    edge_dst: np.ndarray
    node_len: np.ndarray  # int32[num_nodes], tokens in each node's KV segment
    path_ptr: np.ndarray  # int32[R+1]
    path_node: np.ndarray  # int32[path_ptr[R]]
    notes: dict = field(default_factory=dict)
    # Inputs with a large dynamic range of scores (peaked softmax).  Queries are the table values times
    # 2**q_scale_log2 (values: 2**v_scale_log2).  Every entry (q_row, query_head, node, token, scale_log2) of `planted` replaces
    # one key row: K[node][token][KV head of query_head] becomes the table values of query row q_row,
    # head query_head, times 2**scale_log2, i.e. a key aligned with that query, so that its score
    # stands far above the others'.  Input construction only: nothing of the method is computed here.
    q_scale_log2: int = 0
    v_scale_log2: int = 0  # values are the table values times 2**v_scale_log2 (keeps peaked outputs below 4)
    planted: tuple = ()

    @property
    def num_requests(self) -> int:
        return len(self.path_ptr) - 1

    def path(self, r: int) -> np.ndarray:
        return self.path_node[self.path_ptr[r]:self.path_ptr[r + 1]]

    def used_nodes(self) -> np.ndarray:
        """Ascending ids of nodes with a non-empty segment on at least one path."""
        u = np.unique(self.path_node)
        return u[self.node_len[u] > 0]

    def q_rows_per_request(self) -> np.ndarray:
        if self.mode == "decode":
            return np.ones(self.num_requests, dtype=np.int64)
        last = self.path_node[self.path_ptr[1:] - 1]
        return self.node_len[last].astype(np.int64)

    def q_row_ptr(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(self.q_rows_per_request())]).astype(np.int64)

    def node_kv_bits(self, layer: int, node: int):
        """(K, V) bf16 bit patterns, each uint16[len, Hkv, D] (the caller layout)."""
        n = int(self.node_len[node])
        shape = (n, self.num_kv_heads, self.head_dim)
        cnt = n * self.num_kv_heads * self.head_dim
        k = fill_bits(stream_key(self.seed, KIND_K, layer, node), 0, cnt).reshape(shape)
        v = scale_bits_pow2(fill_bits(stream_key(self.seed, KIND_V, layer, node), 0, cnt), self.v_scale_log2).reshape(shape)
        for token, kvh, row in self.planted_rows(layer, node):
            k = k.copy() if not k.flags.writeable else k
            k[token, kvh, :] = row
        return k, v

    def planted_rows(self, layer: int, node: int):
        """(token, kv_head, bf16 bits [D]) of the key rows `planted` replaces in this node."""
        out = []
        g = self.num_q_heads // self.num_kv_heads
        for q_row, head, v, token, sl in self.planted:
            if v != node:
                continue
            base = fill_bits(stream_key(self.seed, KIND_Q, layer, 0),
                             (q_row * self.num_q_heads + head) * self.head_dim, self.head_dim)
            out.append((int(token), head // g, scale_bits_pow2(base, sl)))
        return out

    def q_bits(self, layer: int, row_begin: int = 0, row_count: Optional[int] = None) -> np.ndarray:
        """Query bf16 bit patterns uint16[rows, Hq, D] (request-major rows)."""
        total = int(self.q_row_ptr()[-1])
        if row_count is None:
            row_count = total - row_begin
        per = self.num_q_heads * self.head_dim
        b = fill_bits(stream_key(self.seed, KIND_Q, layer, 0), row_begin * per, row_count * per)
        return scale_bits_pow2(b, self.q_scale_log2).reshape(row_count, self.num_q_heads, self.head_dim)

    def request_len(self) -> np.ndarray:
        return np.array([int(self.node_len[self.path(r)].sum()) for r in range(self.num_requests)],
                        dtype=np.int64)

    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2

    def resident_tokens(self) -> int:
        return int(self.node_len[self.used_nodes()].sum())

    def materialised_tokens(self) -> int:
        return int(self.request_len().sum())


# --------------------------------------------------------------------------
# DAG and path generators
# --------------------------------------------------------------------------
def geometric_level_sizes(n_nonroot: int, n_levels: int, ratio: float) -> list:
    """Split n_nonroot nodes over n_levels levels with widths ~ ratio**level (each >= 1)."""
    w = np.array([ratio ** i for i in range(n_levels)], dtype=np.float64)
    sizes = np.maximum(1, np.floor(w / w.sum() * n_nonroot)).astype(np.int64)
    i = n_levels - 1
    while sizes.sum() < n_nonroot:
        sizes[i] += 1
        i = (i - 1) % n_levels
    i = n_levels - 1
    while sizes.sum() > n_nonroot:
        if sizes[i] > 1:
            sizes[i] -= 1
        i = (i - 1) % n_levels
    return [int(s) for s in sizes]


def layered_dag(rng: np.random.Generator, level_sizes: list, max_parents: int = 3):
    """Root (node 0) plus levels; each non-root node draws 1..max_parents parents
    from the previous level, and every node of a non-final level gets >= 1 child.
    Node ids ascend level by level (a topological order).  Returns
    (edge_src, edge_dst, level_of_node, children list per node)."""
    levels = [[0]]
    nxt = 1
    for s in level_sizes:
        levels.append(list(range(nxt, nxt + s)))
        nxt += s
    edges = set()
    for li in range(1, len(levels)):
        prev = levels[li - 1]
        for v in levels[li]:
            k = int(rng.integers(1, max_parents + 1))
            k = min(k, len(prev))
            for p in rng.choice(len(prev), size=k, replace=False):
                edges.add((prev[int(p)], v))
        has_child = {e[0] for e in edges}
        for p in prev:
            if p not in has_child:
                edges.add((p, levels[li][int(rng.integers(0, len(levels[li])))]))
    e = sorted(edges)
    src = np.array([a for a, _ in e], dtype=np.int32)
    dst = np.array([b for _, b in e], dtype=np.int32)
    level_of = np.zeros(nxt, dtype=np.int32)
    for li, lv in enumerate(levels):
        level_of[lv] = li
    children = [[] for _ in range(nxt)]
    for a, b in e:
        children[a].append(b)
    return src, dst, level_of, children


def _walk(rng, children, depth, policy, pop_weight=None):
    """Root-anchored path with `depth` nodes (counting the root)."""
    path = [0]
    v = 0
    while len(path) < depth and children[v]:
        ch = children[v]
        if policy == "uniform":
            v = ch[int(rng.integers(0, len(ch)))]
        elif policy == "popularity":
            w = pop_weight[ch]
            v = ch[int(rng.choice(len(ch), p=w / w.sum()))]
        elif policy == "zipf_sibling":
            w = 1.0 / np.arange(1, len(ch) + 1, dtype=np.float64)
            v = ch[int(rng.choice(len(ch), p=w / w.sum()))]
        else:
            raise ValueError(policy)
        path.append(v)
    return path


def decode_workload(name, config_id, seed, *, layers, hq, hkv, d, n_nodes, n_requests,
                    root_len, len_lo, len_hi, len_dist="uniform", depth_lo, depth_hi,
                    suffix_max, child_policy="uniform", zipf_s=1.1, level_ratio=1.5,
                    token_budget=None) -> Workload:
    """Decode batch: R root-anchored paths over a layered DAG + private suffix nodes."""
    rng = np.random.default_rng(seed)
    n_levels = depth_hi - 1
    sizes = geometric_level_sizes(n_nodes - 1, n_levels, level_ratio)
    src, dst, level_of, children = layered_dag(rng, sizes)
    node_len = np.zeros(n_nodes + n_requests, dtype=np.int32)
    if len_dist == "uniform":
        node_len[:n_nodes] = rng.integers(len_lo, len_hi + 1, size=n_nodes)
    elif len_dist == "loguniform":
        node_len[:n_nodes] = np.floor(np.exp(rng.uniform(np.log(len_lo), np.log(len_hi + 1),
                                                         size=n_nodes))).astype(np.int32)
        node_len[:n_nodes] = np.clip(node_len[:n_nodes], len_lo, len_hi)
    else:
        raise ValueError(len_dist)
    node_len[0] = root_len
    if token_budget is not None:
        # Spend a fixed token budget over the nodes in a seeded order; nodes drawn
        # after the budget is spent keep an empty segment (control-only operations).
        order = np.concatenate([[0], 1 + rng.permutation(n_nodes - 1)])
        left = token_budget
        for v in order:
            take = min(int(node_len[v]), left)
            node_len[v] = take
            left -= take
    pop = None
    if child_policy == "popularity":
        rank = np.empty(n_nodes, dtype=np.float64)
        rank[rng.permutation(n_nodes)] = np.arange(1, n_nodes + 1)
        pop = rank ** (-zipf_s)
    ptr = [0]
    nodes = []
    for r in range(n_requests):
        depth = int(rng.integers(depth_lo, depth_hi + 1))
        p = _walk(rng, children, depth, child_policy, pop)
        sfx = int(rng.integers(0, suffix_max + 1))
        if sfx > 0:
            node_len[n_nodes + r] = sfx
            p.append(n_nodes + r)
        nodes.extend(p)
        ptr.append(len(nodes))
    return Workload(name=name, config_id=config_id, seed=seed, mode="decode", num_layers=layers,
                    num_q_heads=hq, num_kv_heads=hkv, head_dim=d, num_shared_nodes=n_nodes,
                    num_nodes=n_nodes + n_requests, edge_src=src, edge_dst=dst, node_len=node_len,
                    path_ptr=np.array(ptr, dtype=np.int32), path_node=np.array(nodes, dtype=np.int32),
                    notes={"level_sizes": sizes, "child_policy": child_policy})


def extend_workload(name, config_id, seed, *, layers, hq, hkv, d, n_requests, new_len,
                    root_len, len_lo, len_hi, prefix_lo, prefix_hi, group_lo, group_hi) -> Workload:
    """Extend batch: requests in sharing groups; each group owns a chain of nodes below a
    common root; every request appends a private new node of `new_len` tokens (causal)."""
    rng = np.random.default_rng(seed)
    groups = []
    left = n_requests
    while left > 0:
        g = int(rng.integers(group_lo, group_hi + 1))
        g = min(g, left)
        if g < group_lo and groups:
            groups[-1] += g
        else:
            groups.append(g)
        left -= g
    lens = [root_len]
    edges = []
    chains = []
    for _ in groups:
        target = int(rng.integers(prefix_lo, prefix_hi + 1))
        total = root_len
        chain = []
        prev = 0
        while total < target:
            ln = int(rng.integers(len_lo, len_hi + 1))
            ln = min(ln, target - total)
            v = len(lens)
            lens.append(ln)
            edges.append((prev, v))
            chain.append(v)
            prev = v
            total += ln
        chains.append(chain)
    n_shared = len(lens)
    node_len = np.array(lens + [new_len] * n_requests, dtype=np.int32)
    ptr = [0]
    nodes = []
    r = 0
    for g, chain in zip(groups, chains):
        for _ in range(g):
            nodes.extend([0] + chain + [n_shared + r])
            ptr.append(len(nodes))
            r += 1
    edges.sort()
    return Workload(name=name, config_id=config_id, seed=seed, mode="extend", num_layers=layers,
                    num_q_heads=hq, num_kv_heads=hkv, head_dim=d, num_shared_nodes=n_shared,
                    num_nodes=n_shared + n_requests,
                    edge_src=np.array([a for a, _ in edges], dtype=np.int32),
                    edge_dst=np.array([b for _, b in edges], dtype=np.int32),
                    node_len=node_len, path_ptr=np.array(ptr, dtype=np.int32),
                    path_node=np.array(nodes, dtype=np.int32), notes={"groups": groups})


KIND_FEATURE, KIND_WEIGHT = 7, 8


def scoring_inputs(seed: int, num_ops: int, num_tasks: int, d_in: int = 384, d_hidden: int = 256, d_mlp: int = 128) -> dict:
    """Seeded inputs of the workflow construction model (Sec. 4.2; the paper's sizes by default):
    operation and task features ~ N(0, 1), weights ~ N(0, 1 / fan_in), small biases, all fp32 (table
    values, exact in fp32).  The trained parameters and the sentence-encoder features are not available;
    these stand in for them.  Inputs only."""
    def normal(tag, shape, scale=1.0):
        n = int(np.prod(shape))
        bits = fill_bits(stream_key(seed, KIND_FEATURE if tag < 4 else KIND_WEIGHT, tag, 0), 0, n)
        return (bf16_bits_to_f32(bits) * np.float32(scale)).reshape(shape).astype(np.float32)
    return {"x_op": normal(1, (num_ops, d_in)), "x_task": normal(2, (num_tasks, d_in)),
            "w_gcn1": normal(4, (d_in, d_hidden), 1 / np.sqrt(d_in)), "w_gcn2": normal(5, (d_hidden, d_hidden), 1 / np.sqrt(d_hidden)),
            "w1": normal(6, (3 * d_hidden, d_mlp), 1 / np.sqrt(3 * d_hidden)), "b1": normal(7, (d_mlp,), 0.1),
            "w2": normal(8, (d_mlp, d_mlp), 1 / np.sqrt(d_mlp)), "b2": normal(9, (d_mlp,), 0.1),
            "w3": normal(10, (d_mlp,), 1 / np.sqrt(d_mlp)), "b3": np.float32(0.05)}


BASE_SEED = 0x6F10


def residual_workload(n_base: int = 4, n_tokens: int = 32768, *, hq: int = 32, hkv: int = 8, d: int = 128,
                      seed: int = 28433) -> Workload:
    """Nodes for timing the differential-KV reconstruction (Sec. 5.1): n_base base nodes of n_tokens
    tokens each (ids 0 .. n_base-1, no edges) and one prefix-conditioned variant per base (ids
    n_base .. 2*n_base-1, private), Llama-3-8B-shaped heads.  One single-node path per base, so that
    the pool is sized for the bases; the variants' extents are extra."""
    n = 2 * n_base
    return Workload(name="residual-reconstruct", config_id=-1, seed=seed, mode="decode", num_layers=1,
                    num_q_heads=hq, num_kv_heads=hkv, head_dim=d, num_shared_nodes=n_base, num_nodes=n,
                    edge_src=np.zeros(0, np.int32), edge_dst=np.zeros(0, np.int32),
                    node_len=np.full(n, n_tokens, np.int32), path_ptr=np.arange(n_base + 1, dtype=np.int32),
                    path_node=np.arange(n_base, dtype=np.int32),
                    notes={"what": "base nodes plus one variant each; residual density 25 % (K) / 30 % (V)"})


def make_config(config_id: int, seed: Optional[int] = None, **over) -> Workload:
    """The five benchmark configurations (keyword overrides shrink them for tests)."""
    seed = BASE_SEED + config_id if seed is None else seed
    if config_id == 0:
        kw = dict(layers=1, hq=4, hkv=4, d=64, n_nodes=16, n_requests=8, root_len=64, len_lo=16,
                  len_hi=64, depth_lo=3, depth_hi=5, suffix_max=16, level_ratio=1.0)
        kw.update(over)
        return decode_workload("cfg0-tiny", 0, seed, **kw)
    if config_id == 1:
        kw = dict(layers=1, hq=32, hkv=8, d=128, n_nodes=256, n_requests=256, root_len=2048,
                  len_lo=128, len_hi=1024, depth_lo=4, depth_hi=8, suffix_max=512)
        kw.update(over)
        return decode_workload("cfg1-llama8b-decode", 1, seed, **kw)
    if config_id == 2:
        kw = dict(layers=1, hq=32, hkv=8, d=128, n_requests=64, new_len=512, root_len=2048,
                  len_lo=128, len_hi=1024, prefix_lo=2048, prefix_hi=12288, group_lo=4, group_hi=16)
        kw.update(over)
        return extend_workload("cfg2-extend", 2, seed, **kw)
    if config_id == 3:
        kw = dict(layers=1, hq=32, hkv=8, d=128, n_nodes=1024, n_requests=1024, root_len=8192,
                  len_lo=64, len_hi=512, depth_lo=6, depth_hi=6, suffix_max=256,
                  child_policy="popularity", zipf_s=1.1, level_ratio=1.0)
        kw.update(over)
        return decode_workload("cfg3-high-sharing", 3, seed, **kw)
    if config_id == 4:
        kw = dict(layers=32, hq=32, hkv=8, d=128, n_nodes=4096, n_requests=2048, root_len=2048,
                  len_lo=32, len_hi=2048, len_dist="loguniform", depth_lo=3, depth_hi=10,
                  suffix_max=1024, child_policy="zipf_sibling", token_budget=524288,
                  level_ratio=1.6)
        kw.update(over)
        return decode_workload("cfg4-full-depth", 4, seed, **kw)
    raise ValueError(f"unknown config {config_id}")
