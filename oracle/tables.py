"""Exact-integer definition of the path -> block tables.

TEST INFRASTRUCTURE ONLY (see the package docstring).

Requests are workflow paths over the wGraph (Sec. 3: a DAG whose edges are the
valid dependencies between operations); every node owns one KV segment that all
requests through it share (Sec. 5).  The tables say which segments a batch
touches, who shares each, and how the attention work is cut into items.  The
paper fixes none of these formats; the definitions below are this library's
contract, written here by plain set / sort / loop semantics.

Tables (all int32 except the two int64 token totals):
  T1  seg_node/seg_len/seg_off : nodes with a non-empty segment on >= 1 path,
      ascending node id; seg_off = the node's token offset in the KV pool.
  T2  grp_ptr/grp_req          : CSR; group s = ascending ids of the requests
      whose path contains seg_node[s].
  T3  req_len/req_nseg         : context tokens / non-empty segments per request.
  T4  resident_tokens = sum seg_len; materialised_tokens = sum req_len.
  T5  items (seg, tok_begin, tok_count, grp_begin, grp_count, part_base),
      ordered by (segment, chunk, group tile); part_base is the running sum of
      grp_count.  Chunking policy (integers T, GT, GU, CM), per segment with
      length l and group size G:
          mult   = min(CM, max(1, ceil(G / GU)))
          n0     = ceil(l / (T * mult))
          chunk  = 64 * ceil(ceil(l / n0) / 64)
          chunks = ceil(l / chunk);  tiles = ceil(G / GT)
  T6  mrg_ptr/mrg_slot         : CSR by request of its partial slots, in item order
      (slot = part_base + index of the request inside the item's group tile).
  T7  pseg_ptr/pseg            : CSR by request of segment indices in path order
      (empty nodes dropped).  Extend mode adds q_ptr (query-row offsets; request r
      owns len(last node) rows) and self_seg (segment index of the last node).
  bad_req : smallest request index whose path is empty, names a node id outside
      [0, num_nodes), repeats a node, or hops between two wGraph nodes that are
      not joined by an edge (hops into or out of private nodes, ids >=
      num_shared_nodes, are exempt); in extend mode also a last node with an
      empty segment.  -1 when every path is valid.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

TILE_TOKENS = 64
MODE_DECODE = 0
MODE_EXTEND = 1


@dataclass(frozen=True)
class Policy:
    chunk_tokens: int = 256   # T  (multiple of 64)
    group_tile: int = 16      # GT (requests per item)
    group_unit: int = 2       # GU (requests per unit of chunk growth)
    max_chunk_mult: int = 16  # CM (1 = fixed-length chunks)


def ceil_div(a: int, b: int) -> int:
    return -(-a // b)


def pool_offsets(write_order, node_len, num_nodes):
    """Token offset of every node's extent: extents are reserved in first-write
    order, each rounded up to a whole number of 64-token tiles.  Unwritten nodes
    get offset -1."""
    off = np.full(num_nodes, -1, dtype=np.int64)
    cur = 0
    for v in write_order:
        if off[v] >= 0:
            continue
        off[v] = cur
        cur += ceil_div(int(node_len[v]), TILE_TOKENS) * TILE_TOKENS
    return off, cur


def validate(num_nodes, num_shared_nodes, edge_src, edge_dst, node_len, paths, mode):
    edges = list(zip([int(a) for a in edge_src], [int(b) for b in edge_dst]))
    for r, path in enumerate(paths):
        path = [int(v) for v in path]
        bad = len(path) == 0
        for v in path:
            if v < 0 or v >= num_nodes:
                bad = True
        if not bad:
            for i in range(len(path)):
                for j in range(i + 1, len(path)):
                    if path[i] == path[j]:
                        bad = True
            for a, b in zip(path[:-1], path[1:]):
                if a < num_shared_nodes and b < num_shared_nodes:
                    found = False
                    for e in edges:  # deliberately a linear search of the edge list
                        if e == (a, b):
                            found = True
                    if not found:
                        bad = True
            if mode == MODE_EXTEND and int(node_len[path[-1]]) <= 0:
                bad = True
        if bad:
            return r
    return -1


def build_tables(num_nodes, num_shared_nodes, edge_src, edge_dst, node_len, node_off,
                 path_ptr, path_node, policy: Policy = Policy(), mode: int = MODE_DECODE):
    R = len(path_ptr) - 1
    paths = [[int(v) for v in path_node[path_ptr[r]:path_ptr[r + 1]]] for r in range(R)]
    out = {"bad_req": validate(num_nodes, num_shared_nodes, edge_src, edge_dst, node_len, paths, mode)}
    if out["bad_req"] >= 0:
        return out

    # T1: the set of non-empty nodes on any path, ascending.
    used = sorted({v for p in paths for v in p if int(node_len[v]) > 0})
    seg_of = {v: s for s, v in enumerate(used)}
    out["seg_node"] = np.array(used, dtype=np.int32)
    out["seg_len"] = np.array([int(node_len[v]) for v in used], dtype=np.int32)
    out["seg_off"] = np.array([int(node_off[v]) for v in used], dtype=np.int32)

    # T2: who shares each segment.
    groups = [sorted(r for r in range(R) if v in paths[r]) for v in used]
    grp_ptr = [0]
    for g in groups:
        grp_ptr.append(grp_ptr[-1] + len(g))
    out["grp_ptr"] = np.array(grp_ptr, dtype=np.int32)
    out["grp_req"] = np.array([r for g in groups for r in g], dtype=np.int32)

    # T3 / T4.
    out["req_len"] = np.array([sum(int(node_len[v]) for v in p) for p in paths], dtype=np.int32)
    out["req_nseg"] = np.array([sum(1 for v in p if int(node_len[v]) > 0) for p in paths], dtype=np.int32)
    out["resident_tokens"] = int(sum(int(x) for x in out["seg_len"]))
    out["materialised_tokens"] = int(sum(int(x) for x in out["req_len"]))

    # T5: items in (segment, chunk, group tile) order.
    items = []
    slots_of_req = [[] for _ in range(R)]
    part = 0
    for s, v in enumerate(used):
        l = int(node_len[v])
        G = len(groups[s])
        mult = min(policy.max_chunk_mult, max(1, ceil_div(G, policy.group_unit)))
        n0 = ceil_div(l, policy.chunk_tokens * mult)
        chunk = TILE_TOKENS * ceil_div(ceil_div(l, n0), TILE_TOKENS)
        for c in range(ceil_div(l, chunk)):
            for t in range(ceil_div(G, policy.group_tile)):
                g0 = t * policy.group_tile
                gc = min(policy.group_tile, G - g0)
                items.append((s, c * chunk, min(chunk, l - c * chunk), grp_ptr[s] + g0, gc, part))
                for i in range(gc):
                    slots_of_req[groups[s][g0 + i]].append(part + i)
                part += gc
    out["items"] = np.array(items, dtype=np.int32).reshape(-1, 6)
    out["num_slots"] = part

    # T6: every request's slots, in item order.
    mrg_ptr = [0]
    for sl in slots_of_req:
        mrg_ptr.append(mrg_ptr[-1] + len(sl))
    out["mrg_ptr"] = np.array(mrg_ptr, dtype=np.int32)
    out["mrg_slot"] = np.array([x for sl in slots_of_req for x in sl], dtype=np.int32)

    # T7: per-request segment lists in path order.
    pseg = [[seg_of[v] for v in p if int(node_len[v]) > 0] for p in paths]
    pp = [0]
    for x in pseg:
        pp.append(pp[-1] + len(x))
    out["pseg_ptr"] = np.array(pp, dtype=np.int32)
    out["pseg"] = np.array([x for y in pseg for x in y], dtype=np.int32)
    if mode == MODE_EXTEND:
        qp = [0]
        for p in paths:
            qp.append(qp[-1] + int(node_len[p[-1]]))
        out["q_ptr"] = np.array(qp, dtype=np.int32)
        out["self_seg"] = np.array([seg_of[p[-1]] for p in paths], dtype=np.int32)
    return out


class PoolModel:
    """Bookkeeping of node extents in the KV pool when nodes can be released again.

    Sec. 5.2: only the states of frequent transitions stay materialised; a rare one is computed on
    the fly and need not stay.  The paper gives no allocator; this is the library's contract,
    written as plainly as possible.  The pool is a row of `capacity` tiles of 64 tokens.  A node's
    extent is a run of ceil(len / 64) consecutive tiles.  reserve() scans the tiles from the start
    and takes the first run of free tiles that is long enough (first fit); release() marks the
    node's tiles free again.  The state is one flag per tile, so neighbouring free runs are one run
    by construction.  Offsets are in tokens, as in seg_off.
    """

    def __init__(self, capacity_tiles: int):
        self.used = [False] * int(capacity_tiles)
        self.extent = {}  # node -> (first tile, tiles, tokens)

    def reserve(self, node: int, n_tokens: int):
        """Token offset of the node's new extent, or None when no free run is long enough.
        A node of zero tokens takes no tile; its offset is that of the first free tile."""
        assert node not in self.extent
        need = ceil_div(int(n_tokens), TILE_TOKENS)
        run = 0
        for i in range(len(self.used) + 1):
            if run >= need:
                first = i - run if need > 0 else self._first_free()
                for j in range(first, first + need):
                    self.used[j] = True
                self.extent[node] = (first, need, int(n_tokens))
                return first * TILE_TOKENS
            if i == len(self.used):
                break
            run = 0 if self.used[i] else run + 1
        return None

    def _first_free(self):
        for i, u in enumerate(self.used):
            if not u:
                return i
        return len(self.used)

    def release(self, node: int):
        first, need, _ = self.extent.pop(node)
        for j in range(first, first + need):
            assert self.used[j]
            self.used[j] = False

    def tiles_in_use(self) -> int:
        return sum(1 for u in self.used if u)

    def high_water(self) -> int:
        """One past the last tile in use."""
        last = 0
        for i, u in enumerate(self.used):
            if u:
                last = i + 1
        return last
