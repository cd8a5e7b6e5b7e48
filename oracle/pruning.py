"""Effective path pruning: transition statistics and the choice of transitions whose residuals are kept.

TEST INFRASTRUCTURE ONLY (see the package docstring).

Sec. 5.2: from execution statistics the high-frequency transitions are identified and only their
residual KV states are materialised; a workflow that takes a rare transition falls back to computing
KV on the fly.  The statistic is a count per wGraph edge over the executed workflows' paths; the
choice is a threshold on it.

Readings the paper leaves open:
  * what is counted: for every edge (u, v) of E_op, the number of (workflow, hop) pairs whose hop is
    u -> v; hops that touch a private node (id >= num_shared_nodes) are not transitions of the
    wGraph and are not counted; a hop between two shared nodes that is not an edge is reported as a
    miss and counted nowhere;
  * "high-frequency" (no threshold is given): an edge is kept when its count is at least min_count;
  * order of the result: edges ascending by (source, destination), the order of the graph's CSR.

Pins (tests/test_oracle_pruning.py): a second count by a different route (numpy unique over encoded
pairs), hand-counted paths of the paper's example workflow, conservation (counts + misses = hops
between shared nodes), monotonicity of the kept set in min_count, min_count = 1 keeps exactly the
edges that were taken.
"""
from __future__ import annotations

import numpy as np


def sorted_edges(edge_src, edge_dst):
    """The edge list ascending by (source, destination): the order counts are reported in."""
    pairs = sorted(zip((int(x) for x in edge_src), (int(x) for x in edge_dst)))
    return pairs


def transition_counts(num_shared_nodes, edge_src, edge_dst, path_ptr, path_node):
    """(counts int64[num_edges] in sorted_edges order, misses).  One pass over every hop of every path."""
    pairs = sorted_edges(edge_src, edge_dst)
    index = {p: i for i, p in enumerate(pairs)}
    counts = np.zeros(len(pairs), dtype=np.int64)
    misses = 0
    for r in range(len(path_ptr) - 1):
        b, e = int(path_ptr[r]), int(path_ptr[r + 1])
        for i in range(b, e - 1):
            u, v = int(path_node[i]), int(path_node[i + 1])
            if u >= num_shared_nodes or v >= num_shared_nodes:
                continue
            j = index.get((u, v))
            if j is None:
                misses += 1
            else:
                counts[j] += 1
    return counts, misses


def select_transitions(counts, min_count):
    """(keep bool[num_edges], kept edges, traversals covered by kept edges, traversals in total)."""
    counts = np.asarray(counts, dtype=np.int64)
    keep = counts >= int(min_count)
    return keep, int(keep.sum()), int(counts[keep].sum()), int(counts.sum())
