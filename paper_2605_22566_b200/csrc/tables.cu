// K1: path -> block tables, on the device, bit-exact and order-deterministic.
//
// Requests are workflow paths over the wGraph (Sec. 3); every node's KV segment is shared by the
// requests through it (Sec. 5).  These kernels turn the batch's paths into: the ascending list of
// non-empty segments in use (T1), who shares each (T2), per-request totals (T3/T4), the work list
// under the integer chunking policy (T5), the merge map (T6) and per-request segment lists (T7).
//
// Determinism: atomics are used only where the result does not depend on their order (integer
// counts, sums, a minimum) or where the unordered result is sorted afterwards (group members).
#include <limits.h>

#include "gf_internal.h"

namespace gf {
namespace {

constexpr int kScanThreads = 1024;

__device__ __forceinline__ int ceil_div(int a, int b) { return (a + b - 1) / b; }

// Three exclusive scans of in*[0..n) into out*[0..n] in one pass, out*[n] = total (also returned in
// tot[3]).  One CTA; an input may alias its output.
__device__ void block_exclusive_scan3(const int32_t* in0, int32_t* out0, const int32_t* in1, int32_t* out1,
                                      const int32_t* in2, int32_t* out2, int n, int (&tot)[3]) {
  __shared__ int warp_tot3[3][32];
  __shared__ int carry3[3];
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  if (tid < 3) carry3[tid] = 0;
  __syncthreads();
  for (int base = 0; base < n; base += blockDim.x) {
    const int i = base + tid;
    int x[3] = {0, 0, 0}, incl[3];
    if (i < n) { x[0] = in0[i]; x[1] = in1[i]; x[2] = in2[i]; }
#pragma unroll
    for (int k = 0; k < 3; ++k) {
      incl[k] = x[k];
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl[k], d);
        if (lane >= d) incl[k] += y;
      }
      if (lane == 31) warp_tot3[k][wid] = incl[k];
    }
    __syncthreads();
    if (wid < 3) {
      int w = (lane < nw) ? warp_tot3[wid][lane] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, w, d);
        if (lane >= d) w += y;
      }
      warp_tot3[wid][lane] = w;  // inclusive totals of warps
    }
    __syncthreads();
    if (i < n) {
      out0[i] = carry3[0] + ((wid == 0) ? 0 : warp_tot3[0][wid - 1]) + incl[0] - x[0];
      out1[i] = carry3[1] + ((wid == 0) ? 0 : warp_tot3[1][wid - 1]) + incl[1] - x[1];
      out2[i] = carry3[2] + ((wid == 0) ? 0 : warp_tot3[2][wid - 1]) + incl[2] - x[2];
    }
    __syncthreads();
    if (tid < 3) carry3[tid] += warp_tot3[tid][nw - 1];
    __syncthreads();
  }
  tot[0] = carry3[0]; tot[1] = carry3[1]; tot[2] = carry3[2];
  if (tid == 0) { out0[n] = tot[0]; out1[n] = tot[1]; out2[n] = tot[2]; }
  __syncthreads();
}

__global__ void k_init(TablesDev t, int num_nodes) {
  chain_enter();
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  const int stride = gridDim.x * blockDim.x;
  for (int v = i; v < num_nodes; v += stride) t.node_seg[v] = 0;
  for (int s = i; s < t.seg_cap; s += stride) t.grp_fill[s] = 0;
  if (i == 0) {
    Header h;
    h.bad_req = INT_MAX;
    h.num_segments = h.num_pairs = h.num_items = h.num_slots = h.mrg_total = 0;
    h.num_wide = 0;
    h.wide_units = 0;
    h.wide_list_n = 0;
    h.wide_work = 0;
    h.wide_tokens = 0;
    h.wide_tile_units = 0;
    h.stream_steps = 0;
    h.max_q_rows = 0;
    h.resident_tokens = h.materialised_tokens = h.num_q_rows = 0ull;
    *t.hdr = h;
  }
}

__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
  return v;
}

// One warp per request (lanes over path positions): validate the path, count the users of every
// non-empty node (node_seg[v] += 1, an integer count: order independent), total its context.
__global__ void k_validate(GraphDev g, TablesDev t, const int32_t* __restrict__ path_ptr,
                           const int32_t* __restrict__ path_node) {
  chain_enter();
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (r >= t.num_requests) return;
  const int b = path_ptr[r], e = path_ptr[r + 1];
  bool bad = (b < 0) || (e <= b) || (e > t.num_pairs_in) || (r == 0 && b != 0);
  if (!bad) {
    for (int i = b + lane; i < e; i += 32) {
      const int v = path_node[i];
      if (v < 0 || v >= g.num_nodes) bad = true;
    }
    bad = __any_sync(0xffffffffu, bad);
  }
  if (!bad) {
    for (int i = b + lane; i < e; i += 32) {
      const int a = path_node[i];
      for (int j = i + 1; j < e; ++j)
        if (path_node[j] == a) bad = true;
      if (i + 1 < e) {
        const int c = path_node[i + 1];
        if (a < g.num_shared_nodes && c < g.num_shared_nodes) {
          int lo = g.adj_ptr[a], hi = g.adj_ptr[a + 1];  // binary search c in the sorted row
          const int end = hi;
          while (lo < hi) {
            const int mid = (lo + hi) >> 1;
            if (g.adj_dst[mid] < c) lo = mid + 1; else hi = mid;
          }
          if (lo >= end || g.adj_dst[lo] != c) bad = true;
        }
      }
    }
    if (lane == 0 && t.mode == GF_MODE_EXTEND && g.node_len[path_node[e - 1]] <= 0) bad = true;
    if (t.mode == GF_MODE_EXTEND)  // extend streams whole extents: a state kept as base + residual has none of its own
      for (int i = b + lane; i < e; i += 32)
        if (g.node_res[path_node[i]] >= 0) bad = true;
    bad = __any_sync(0xffffffffu, bad);
  }
  if (bad) {
    if (lane == 0) {
      atomicMin(&t.hdr->bad_req, r);
      t.req_len[r] = 0; t.req_nseg[r] = 0; t.req_qrows[r] = 0;
    }
    return;
  }
  int len = 0, nseg = 0;
  for (int i = b + lane; i < e; i += 32) {
    const int v = path_node[i];
    const int l = g.node_len[v];
    if (l > 0) { len += l; ++nseg; atomicAdd(&t.node_seg[v], 1); }
  }
  len = warp_sum(len);
  nseg = warp_sum(nseg);
  if (lane == 0) {
    t.req_len[r] = len;
    t.req_nseg[r] = nseg;
    t.req_qrows[r] = (t.mode == GF_MODE_EXTEND) ? g.node_len[path_node[e - 1]] : 1;
    atomicAdd(&t.hdr->materialised_tokens, (unsigned long long)len);
  }
}

// One CTA.  User counts per node -> ascending segment list (T1) with group sizes; then the
// chunking policy per segment -> group, item and slot bases (T2 / T5 layout).
// Afterwards node_seg[v] is the exclusive segment index and node_seg[v+1]-node_seg[v] the flag.
__global__ void k_scan_nodes_segments(GraphDev g, TablesDev t, gf_policy_t pol) {
  chain_enter();
  if (t.hdr->bad_req != INT_MAX) return;
  __shared__ unsigned long long red[32];
  __shared__ int warp_tot[32];
  __shared__ int carry_s;
  __shared__ int wide_units, wide_work, wide_tokens, wide_tile_units, stream_steps;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  const int n = g.num_nodes;
  if (tid == 0) { carry_s = 0; wide_units = 0; wide_work = 0; wide_tokens = 0; wide_tile_units = 0; stream_steps = 0; }
  __syncthreads();
  unsigned long long sum = 0;
  for (int base = 0; base < n; base += blockDim.x) {
    const int v = base + tid;
    const int cnt = (v < n) ? t.node_seg[v] : 0;
    const int x = cnt > 0 ? 1 : 0;
    int incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (wid == 0) {
      int w = (lane < nw) ? warp_tot[lane] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, w, d);
        if (lane >= d) w += y;
      }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const int idx = carry_s + ((wid == 0) ? 0 : warp_tot[wid - 1]) + incl - x;
    if (v < n) {
      t.node_seg[v] = idx;
      if (x) {
        const int l = g.node_len[v];
        t.seg_node[idx] = v;
        t.seg_len[idx] = l;
        t.seg_off[idx] = g.node_off[v];
        t.grp_ptr[idx] = cnt;
        sum += (unsigned long long)l;
      }
    }
    __syncthreads();
    if (tid == 0) carry_s += warp_tot[nw - 1];
    __syncthreads();
  }
  const int S = carry_s;
  for (int d = 16; d > 0; d >>= 1) sum += __shfl_down_sync(0xffffffffu, sum, d);
  if (lane == 0) red[wid] = sum;
  __syncthreads();
  if (tid == 0) {
    unsigned long long tot = 0;
    for (int w = 0; w < nw; ++w) tot += red[w];
    t.node_seg[n] = S;
    t.hdr->resident_tokens = tot;
    t.hdr->num_segments = S;
  }
  for (int s = tid; s < S; s += blockDim.x) {
    const int G = t.grp_ptr[s];
    const int l = t.seg_len[s];
    const int mult = min(pol.max_chunk_mult, max(1, ceil_div(G, pol.group_unit)));
    const int n0 = ceil_div(l, pol.chunk_tokens * mult);
    const int chunk = kTile * ceil_div(ceil_div(l, n0), kTile);
    const int nchunk = ceil_div(l, chunk);
    t.seg_chunk[s] = chunk;
    t.seg_nchunk[s] = nchunk;
    t.seg_item_base[s] = nchunk * ceil_div(G, pol.group_tile);
    t.seg_part_base[s] = nchunk * G;
    // (a segment whose state is base + residual is patched in shared memory by the warp kernel only)
    if (G >= t.wide_probe_group && (t.wide_unit_req % pol.group_tile) == 0 && t.node_res[t.seg_node[s]] < 0) {
      atomicAdd(&wide_units, nchunk * ceil_div(G, t.wide_unit_req));  // CTAs' worth of work for the wide kernel, per KV head
      if (t.wide_min_group > 0) atomicAdd(&t.hdr->num_wide, nchunk * ceil_div(G, pol.group_tile));  // its items
      // its work: every 128-token stage of every chunk, once per 128-row tile of the stacked query rows
      const int stages = (nchunk - 1) * ceil_div(chunk, 128) + ceil_div(l - (nchunk - 1) * chunk, 128);
      atomicAdd(&wide_work, stages * ceil_div(G * (256 / t.wide_unit_req), 128));
      atomicAdd(&wide_tile_units, nchunk * ceil_div(G * (256 / t.wide_unit_req), 128));
      atomicAdd(&wide_tokens, l);
    } else {
      // the warp kernel's work: every 64-token tile once per 16-row group of the stacked query rows
      const int gqa = 256 / t.wide_unit_req;
      const int groups = (G / pol.group_tile) * ceil_div(pol.group_tile * gqa, 16) +
                         ceil_div((G % pol.group_tile) * gqa, 16);
      atomicAdd(&stream_steps, ceil_div(l, kTile) * groups);
    }
  }
  __syncthreads();
  // the tensor-memory kernel pays off only when its units can fill the GPU; otherwise every chunk
  // stays with the warp kernel.  The host keeps the unit count as a hint for builds it does not wait for.
  if (tid == 0) {
    t.hdr->wide_units = wide_units;
    t.hdr->wide_work = wide_work;
    t.hdr->wide_tokens = wide_tokens;
    t.hdr->wide_tile_units = wide_tile_units;
    t.hdr->stream_steps = stream_steps;
    if (wide_units < t.wide_min_units) t.hdr->num_wide = 0;
  }
  __syncthreads();
  int tot[3];
  block_exclusive_scan3(t.grp_ptr, t.grp_ptr, t.seg_item_base, t.seg_item_base, t.seg_part_base, t.seg_part_base, S, tot);
  if (tid == 0) { t.hdr->num_items = tot[1]; t.hdr->num_slots = tot[2]; }
}

__device__ __forceinline__ int seg_of_node(const TablesDev& t, int v) {
  const int idx = t.node_seg[v];
  return (t.node_seg[v + 1] != idx) ? idx : -1;
}

// One warp per request: append the request to the member list of each of its segments
// (unordered; sorted next), and count its partial slots.
__global__ void k_fill_groups(TablesDev t, const int32_t* __restrict__ path_ptr,
                              const int32_t* __restrict__ path_node) {
  chain_enter();
  if (t.hdr->bad_req != INT_MAX) return;
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (r >= t.num_requests) return;
  int nslot = 0;
  for (int i = path_ptr[r] + lane; i < path_ptr[r + 1]; i += 32) {
    const int s = seg_of_node(t, path_node[i]);
    if (s < 0) continue;
    const int pos = atomicAdd(&t.grp_fill[s], 1);
    if (GF_CHECK(t.grp_ptr[s] + pos < t.num_pairs_in, t.status, 301)) t.grp_tmp[t.grp_ptr[s] + pos] = r;
    nslot += t.seg_nchunk[s];
  }
  nslot = warp_sum(nslot);
  if (lane == 0) t.req_nslot[r] = nslot;
}

// Ascending order of every group's members (distinct request ids): unique result.  Small groups
// by rank counting; larger ones through a bitmap of request ids in shared memory: the rank of r is
// the number of set bits below it (word prefix counts + a popcount), O(n + R/32) per group.
constexpr int kSortCache = 4096;
constexpr int kBitmapWords = 2048;  // request ids below 65536
__device__ void sort_groups(const TablesDev& t, int first_block, int num_blocks) {
  __shared__ int32_t cache[kSortCache];  // bitmap words, then their exclusive popcount prefix
  __shared__ int wsum[32];
  const int S = t.hdr->num_segments;
  const int W = (t.num_requests + 31) >> 5;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  for (int s = (int)blockIdx.x - first_block; s < S; s += num_blocks) {
    const int b = t.grp_ptr[s], n = t.grp_ptr[s + 1] - b;
    const int32_t* src = t.grp_tmp + b;
    if (n <= 32) {
      if (tid < n) {
        const int v = src[tid];
        int rank = 0;
        for (int j = 0; j < n; ++j) rank += (src[j] < v);
        if (GF_CHECK(b + rank < t.num_pairs_in, t.status, 302)) t.grp_req[b + rank] = v;
      }
      continue;
    }
    __syncthreads();
    if (W <= kBitmapWords) {
      uint32_t* bm = reinterpret_cast<uint32_t*>(cache);
      int32_t* pre = cache + kBitmapWords;
      for (int w = tid; w < W; w += blockDim.x) bm[w] = 0u;
      __syncthreads();
      for (int i = tid; i < n; i += blockDim.x) {
        const int r = src[i];
        atomicOr(&bm[r >> 5], 1u << (r & 31));
      }
      __syncthreads();
      // exclusive prefix of the words' popcounts: each thread owns a run of consecutive words
      const int per = (W + blockDim.x - 1) / blockDim.x;
      const int w0 = min(W, tid * per), w1 = min(W, w0 + per);
      int local = 0;
      for (int w = w0; w < w1; ++w) local += __popc(bm[w]);
      int incl = local;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= d) incl += y;
      }
      if (lane == 31) wsum[wid] = incl;
      __syncthreads();
      if (wid == 0) {
        int v = (lane < nw) ? wsum[lane] : 0;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
          const int y = __shfl_up_sync(0xffffffffu, v, d);
          if (lane >= d) v += y;
        }
        wsum[lane] = v;
      }
      __syncthreads();
      int run = ((wid == 0) ? 0 : wsum[wid - 1]) + incl - local;
      for (int w = w0; w < w1; ++w) { pre[w] = run; run += __popc(bm[w]); }
      __syncthreads();
      for (int i = tid; i < n; i += blockDim.x) {
        const int r = src[i];
        const int rank = pre[r >> 5] + __popc(bm[r >> 5] & ((1u << (r & 31)) - 1u));
        if (GF_CHECK(b + rank < t.num_pairs_in, t.status, 303)) t.grp_req[b + rank] = r;
      }
      continue;
    }
    const bool cached = n <= kSortCache;
    if (cached) {
      for (int i = tid; i < n; i += blockDim.x) cache[i] = src[i];
      __syncthreads();
    }
    const int32_t* look = cached ? cache : src;
    for (int i = tid; i < n; i += blockDim.x) {
      const int v = look[i];
      int rank = 0;
      for (int j = 0; j < n; ++j) rank += (look[j] < v);
      if (GF_CHECK(b + rank < t.num_pairs_in, t.status, 304)) t.grp_req[b + rank] = v;
    }
  }
}

// One CTA: per-request scans (starts of the segment lists, of the merge map and of the query rows);
// the lists themselves are written by k_emit, a warp per request.
__device__ void scan_requests(const TablesDev& t, const int32_t* __restrict__ path_ptr,
                              const int32_t* __restrict__ path_node) {
  const int R = t.num_requests;
  int tot[3];
  block_exclusive_scan3(t.req_nseg, t.pseg_ptr, t.req_nslot, t.mrg_ptr, t.req_qrows, t.q_ptr, R, tot);
  if (threadIdx.x == 0) {
    t.hdr->num_pairs = tot[0];
    t.hdr->mrg_total = tot[1];
    t.hdr->num_q_rows = (unsigned long long)tot[2];
  }
  __syncthreads();
  if (t.mode != GF_MODE_EXTEND) return;
  // Extend launches walk whole paths, so their cost follows the context length: requests by
  // descending length (ties by id: a unique order), and the longest query block for the grid.
  int mq = 0;
  for (int r = threadIdx.x; r < R; r += blockDim.x) {
    const int len = t.req_len[r];
    int rank = 0;
    for (int o = 0; o < R; ++o) {
      const int lo = t.req_len[o];
      rank += (lo > len) || (lo == len && o < r);
    }
    t.req_order[rank] = r;
    mq = max(mq, t.req_qrows[r]);
  }
  atomicMax(&t.hdr->max_q_rows, mq);
}

// Two steps that need the unordered groups and nothing from each other, in one launch: block 0 does
// the per-request scans, the other blocks sort the groups.
__global__ void __launch_bounds__(kScanThreads) k_sort_groups_scan_requests(TablesDev t, const int32_t* __restrict__ path_ptr,
                                                                            const int32_t* __restrict__ path_node) {
  chain_enter();
  if (t.hdr->bad_req != INT_MAX) return;
  if (blockIdx.x == 0) scan_requests(t, path_ptr, path_node);
  else sort_groups(t, 1, (int)gridDim.x - 1);
}

// One item: (segment, chunk, group tile) from the item index (T5).
__device__ void emit_item(const TablesDev& t, const gf_policy_t& pol, int i, const int32_t* item_base) {
  const int S = t.hdr->num_segments;
  int lo = 0, hi = S;  // largest s with item_base[s] <= i (item_base: seg_item_base or its copy in shared memory)
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (item_base[mid] <= i) lo = mid; else hi = mid;
  }
  const int s = lo;
  const int G = t.grp_ptr[s + 1] - t.grp_ptr[s];
  const int ntile = ceil_div(G, pol.group_tile);
  const int local = i - t.seg_item_base[s];
  const int c = local / ntile, tl = local - c * ntile;
  const int chunk = t.seg_chunk[s];
  Item it;
  it.seg = s;
  it.tok_begin = c * chunk;
  it.tok_count = min(chunk, t.seg_len[s] - c * chunk);
  it.grp_begin = t.grp_ptr[s] + tl * pol.group_tile;
  it.grp_count = min(pol.group_tile, G - tl * pol.group_tile);
  it.part_base = t.seg_part_base[s] + c * G + tl * pol.group_tile;
  it.tile0 = (t.seg_off[s] + it.tok_begin) / kTile;
  // the group tiles of wide_unit_req / group_tile consecutive items form one unit of the wide kernel
  const int res = t.node_res[t.seg_node[s]];
  const bool wide = t.hdr->num_wide > 0 && G >= t.wide_min_group && (t.wide_unit_req % pol.group_tile) == 0 && res < 0;
  it.pad = (wide ? 1 : 0) | ((res + 1) << 8);
  t.items[i] = it;
  // the first item of every wide_unit_req requests of a wide chunk stands for a unit of the wide kernel
  if (wide && ((it.grp_begin - t.grp_ptr[s]) % t.wide_unit_req) == 0) {
    const int at = atomicAdd(&t.hdr->wide_list_n, 1);
    if (GF_CHECK(at < t.slot_cap, t.status, 305)) t.wide_list[at] = i;
  }
}

// The first item_blocks CTAs: one thread per item, (segment, chunk, group tile) from the item
// index (T5).  The remaining CTAs: one warp per request, its partial slots in item order (T6);
// items are ordered by segment then chunk, so slots follow ascending segment index.  The same warp
// first writes the request's segment list in path order (T7).
constexpr int kEmitCache = 4096;  // segment starts searched in shared memory when there are no more than this
__global__ void k_emit(TablesDev t, gf_policy_t pol, int item_blocks, const int32_t* __restrict__ path_ptr,
                       const int32_t* __restrict__ path_node) {
  __shared__ int32_t base_cache[kEmitCache];
  chain_enter();
  if (!tables_usable(*t.hdr, t.slot_cap)) return;
  if ((int)blockIdx.x < item_blocks) {
    const int num_items = t.hdr->num_items;
    // every item searches the segments' item starts: a dozen dependent loads, from shared memory when they fit
    const int S = t.hdr->num_segments;
    const int32_t* item_base = t.seg_item_base;
    if (S <= kEmitCache) {
      for (int s = threadIdx.x; s < S; s += blockDim.x) base_cache[s] = t.seg_item_base[s];
      __syncthreads();
      item_base = base_cache;
    }
    for (int i = blockIdx.x * blockDim.x + threadIdx.x; i < num_items; i += item_blocks * blockDim.x)
      emit_item(t, pol, i, item_base);
    return;
  }
  const int r = (((int)blockIdx.x - item_blocks) * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (r >= t.num_requests) return;
  // T7 first: the request's segment indices in path order (lanes over path positions, kept in order by
  // the rank of each lane among those whose node has a segment), and its own (last) segment
  {
    const int b = path_ptr[r], e = path_ptr[r + 1];
    int k = t.pseg_ptr[r];
    int last = -1;
    for (int i0 = b; i0 < e; i0 += 32) {
      const int i = i0 + lane;
      const int s = (i < e) ? seg_of_node(t, path_node[i]) : -1;
      const uint32_t have = __ballot_sync(0xffffffffu, s >= 0);
      if (s >= 0 && GF_CHECK(k + __popc(have & ((1u << lane) - 1u)) < t.num_pairs_in, t.status, 306))
        t.pseg[k + __popc(have & ((1u << lane) - 1u))] = s;
      k += __popc(have);
      if (e - 1 >= i0 && e - 1 < i0 + 32) last = __shfl_sync(0xffffffffu, s, e - 1 - i0);
    }
    if (lane == 0) t.self_seg[r] = last;
    __syncwarp();
  }
  const int pb = t.pseg_ptr[r], pe = t.pseg_ptr[r + 1];
  for (int i = pb + lane; i < pe; i += 32) {
    const int s = t.pseg[i];
    int k = t.mrg_ptr[r];  // slots of the request's segments with a smaller index come first
    for (int j = pb; j < pe; ++j) {
      const int c = t.pseg[j];
      if (c < s) k += t.seg_nchunk[c];
    }
    const int gb = t.grp_ptr[s], G = t.grp_ptr[s + 1] - gb;
    int lo = 0, hi = G;  // rank of r inside the ascending group
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (t.grp_req[gb + mid] < r) lo = mid + 1; else hi = mid;
    }
    const int nchunk = t.seg_nchunk[s];
    const int base = t.seg_part_base[s] + lo;
    for (int c = 0; c < nchunk; ++c)
      if (GF_CHECK(k + c < t.slot_cap && base + c * G < t.slot_cap, t.status, 307)) t.mrg_slot[k + c] = base + c * G;
  }
}

__global__ void k_set_node(GraphDev g, int node, int len, int off) {
  g.node_len[node] = len;
  g.node_off[node] = off;
}

__global__ void k_set_residual(ResidualEntry* slot, ResidualEntry value, int32_t* node_res, int node, int row) {
  if (slot != nullptr) *slot = value;
  node_res[node] = row;
}

inline int blocks_for(int n, int threads) { return n <= 0 ? 1 : (n + threads - 1) / threads; }

}  // namespace

int launch_graph_set_node(const GraphDev& g, int node, int len, int off, cudaStream_t st) {
  k_set_node<<<1, 1, 0, st>>>(g, node, len, off);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_set_residual(ResidualEntry* slot, const ResidualEntry& value, int32_t* node_res, int node, int row,
                        cudaStream_t st) {
  k_set_residual<<<1, 1, 0, st>>>(slot, value, node_res, node, row);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_tables_phase_a(const GraphDev& g, const TablesDev& t, const int32_t* path_ptr,
                          const int32_t* path_node, gf_policy_t pol, cudaStream_t st) {
  const int R = t.num_requests;
  const int span = (g.num_nodes + 1 > t.seg_cap) ? g.num_nodes + 1 : t.seg_cap;
  launch_chained(k_init, dim3(blocks_for(span, 256)), dim3(256), 0, st, t, g.num_nodes + 1);
  launch_chained(k_validate, dim3(blocks_for(R * 32, 128)), dim3(128), 0, st, g, t, path_ptr, path_node);
  launch_chained(k_scan_nodes_segments, dim3(1), dim3(kScanThreads), 0, st, g, t, pol);
  launch_chained(k_fill_groups, dim3(blocks_for(R * 32, 128)), dim3(128), 0, st, t, path_ptr, path_node);
  launch_chained(k_sort_groups_scan_requests, dim3(1 + 2 * t.num_sms), dim3(kScanThreads), 0, st, t, path_ptr, path_node);
  return cudaGetLastError() == cudaSuccess ? 5 : -1;
}

int launch_tables_phase_b(const TablesDev& t, const int32_t* path_ptr, const int32_t* path_node, gf_policy_t pol,
                          int num_items, cudaStream_t st) {
  const int wave = 2 * t.num_sms;  // two CTAs of 128 threads per multiprocessor
  const int item_blocks = (num_items >= 0 && num_items < wave * 128) ? blocks_for(num_items, 128) : wave;
  launch_chained(k_emit, dim3(item_blocks + blocks_for(t.num_requests * 32, 128)), dim3(128), 0, st, t, pol, item_blocks,
                 path_ptr, path_node);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
