"""B200-native path attention over wGraph node KV segments (GraphFlow, Sec. 5).

Sub-modules:
  workloads  seeded synthetic wGraphs / paths / K,V,Q bits (no attention arithmetic)
  binding    ctypes binding of the C-ABI library (gf_* entry points)

Nothing is imported eagerly: `workloads` is pure numpy and usable without a GPU,
`binding` loads the CUDA library and fails loudly when it is missing.
"""

__all__ = ["workloads", "binding"]
