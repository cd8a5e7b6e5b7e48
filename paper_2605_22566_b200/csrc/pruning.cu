// Effective path pruning (Sec. 5.2): execution statistics over the wGraph's transitions and the choice
// of the transitions whose residual KV states are kept.
//
// A hop u -> v of an executed workflow between two operation nodes is a transition; its edge index is
// found by binary search in the graph's CSR row of u (destinations ascending), so counts come out in
// (source, destination) order.  Counting is a histogram over at most num_edges bins that millions of
// hops fall into, most of them on a few popular edges: every CTA counts into a private copy in shared
// memory (as many bins as fit; the rest go to global atomics) and adds its non-zero bins to the result
// once.  Integer adds: the result does not depend on the order.
#include "gf_internal.h"

namespace gf {
namespace {

constexpr int kStatThreads = 256;
constexpr int kStatBins = 8192;  // bins of a CTA's private histogram (32 KB)

__global__ void __launch_bounds__(kStatThreads) k_transition_counts(GraphDev g, int num_edges, int num_requests,
                                                                    int num_path_nodes,
                                                                    const int32_t* __restrict__ path_ptr,
                                                                    const int32_t* __restrict__ path_node,
                                                                    int32_t* counts, unsigned long long* misses) {
  __shared__ int32_t bins[kStatBins];
  const int local_bins = num_edges < kStatBins ? num_edges : kStatBins;
  for (int i = threadIdx.x; i < local_bins; i += kStatThreads) bins[i] = 0;
  __syncthreads();
  // One thread per request at a time: workflows are a handful of hops long, so lanes over the hops of
  // one request would mostly idle; neighbouring threads read neighbouring stretches of path_node.
  const int first = blockIdx.x * kStatThreads + threadIdx.x, stride = gridDim.x * kStatThreads;
  unsigned long long miss = 0;
  for (int r = first; r < num_requests; r += stride) {
    int b = path_ptr[r], e = path_ptr[r + 1];
    if (b < 0) b = 0;
    if (e > num_path_nodes) e = num_path_nodes;
    if (e - b < 2) continue;
    // the path is read eight nodes at a time, all eight loads in flight together
    int u = path_node[b];
    for (int i0 = b + 1; i0 < e; i0 += 8) {
      int nodes[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) nodes[k] = (i0 + k < e) ? path_node[i0 + k] : -1;
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        if (i0 + k >= e) break;
        const int v = nodes[k];
        const int from = u;
        u = v;
        if (from < 0 || v < 0 || from >= g.num_shared_nodes || v >= g.num_shared_nodes) continue;  // not a wGraph transition
        int lo = g.adj_ptr[from], hi = g.adj_ptr[from + 1];
        const int end = hi;
        while (lo < hi) {
          const int mid = (lo + hi) >> 1;
          if (g.adj_dst[mid] < v) lo = mid + 1; else hi = mid;
        }
        if (lo >= end || g.adj_dst[lo] != v) { ++miss; continue; }
        if (lo < local_bins) atomicAdd(&bins[lo], 1);
        else atomicAdd(&counts[lo], 1);
      }
    }
  }
  __syncthreads();
  for (int i = threadIdx.x; i < local_bins; i += kStatThreads) {
    const int c = bins[i];
    if (c != 0) atomicAdd(&counts[i], c);
  }
  if (miss != 0) atomicAdd(misses, miss);
}

// keep[e] = counts[e] >= min_count; totals: kept edges, traversals on kept edges, all traversals.
__global__ void __launch_bounds__(kStatThreads) k_select_transitions(const int32_t* __restrict__ counts, int num_edges,
                                                                     int min_count, uint8_t* keep,
                                                                     unsigned long long* totals) {
  unsigned long long kept = 0, covered = 0, total = 0;
  for (int i = blockIdx.x * kStatThreads + threadIdx.x; i < num_edges; i += gridDim.x * kStatThreads) {
    const int c = counts[i];
    const bool k = c >= min_count;
    keep[i] = k ? 1 : 0;
    kept += k ? 1u : 0u;
    covered += k ? (unsigned long long)c : 0ull;
    total += (unsigned long long)c;
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    kept += __shfl_xor_sync(0xffffffffu, kept, d);
    covered += __shfl_xor_sync(0xffffffffu, covered, d);
    total += __shfl_xor_sync(0xffffffffu, total, d);
  }
  if ((threadIdx.x & 31) == 0 && total + kept != 0) {
    atomicAdd(&totals[0], kept);
    atomicAdd(&totals[1], covered);
    atomicAdd(&totals[2], total);
  }
}

}  // namespace

int launch_transition_counts(const GraphDev& g, int num_edges, int num_requests, int num_path_nodes,
                             const int32_t* path_ptr, const int32_t* path_node, int32_t* counts,
                             unsigned long long* misses, cudaStream_t st) {
  if (cudaMemsetAsync(counts, 0, (size_t)(num_edges > 0 ? num_edges : 0) * 4, st) != cudaSuccess) return -1;
  if (cudaMemsetAsync(misses, 0, 8, st) != cudaSuccess) return -1;
  if (num_requests <= 0) return 0;
  long long blocks = ((long long)num_requests + kStatThreads - 1) / kStatThreads;
  if (blocks > 148 * 6) blocks = 148 * 6;
  k_transition_counts<<<(unsigned)blocks, kStatThreads, 0, st>>>(g, num_edges, num_requests, num_path_nodes, path_ptr,
                                                                 path_node, counts, misses);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_select_transitions(const int32_t* counts, int num_edges, int min_count, uint8_t* keep,
                              unsigned long long* totals, cudaStream_t st) {
  if (cudaMemsetAsync(totals, 0, 24, st) != cudaSuccess) return -1;
  if (num_edges <= 0) return 0;
  int blocks = (num_edges + kStatThreads - 1) / kStatThreads;
  if (blocks > 148 * 4) blocks = 148 * 4;
  k_select_transitions<<<blocks, kStatThreads, 0, st>>>(counts, num_edges, min_count, keep, totals);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
