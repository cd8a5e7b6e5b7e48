// Host side of the C ABI: handles, argument validation, workspace carving, launches.
#include <math.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <mutex>
#include <new>
#include <vector>

#include "gf_internal.h"

using namespace gf;

struct gf_tables {
  gf_wgraph* owner = nullptr;
  TablesDev dev{};
  gf_tables_info_t info{};
  gf_policy_t policy{};
  int32_t bad_req = -1;
  int32_t max_q_rows = 0;
  int32_t num_wide = -1;       // items flagged wide; -1: not known on the host (deferred, or phase B still to run)
  int32_t split_sms = 0;       // multiprocessors the tensor-memory decode kernel gets beside the warp kernel (0: one after the other)
  bool pending = false;        // deferred build: sizes and validity not read back yet
  cudaStream_t build_stream = nullptr;
  gf_status_t error = GF_OK;   // what a deferred build turned out to be
  bool built = false;
  uint64_t generation = 0;
};

// Tiles of the KV pool: extents are runs of consecutive tiles, handed out first fit (the free runs in
// ascending order, then the untouched tail) and joined with their free neighbours when they return.
struct TilePool {
  std::map<uint32_t, uint32_t> holes;  // free runs below `top`: first tile -> length
  uint32_t top = 0;                    // one past the last tile in use
  uint32_t cap = 0;
  uint32_t in_use = 0;
  uint32_t first_free() const { return holes.empty() ? top : holes.begin()->first; }
  bool take(uint32_t need, uint32_t* first) {
    if (need == 0) { *first = first_free(); return true; }
    for (auto it = holes.begin(); it != holes.end(); ++it) {
      if (it->second < need) continue;
      *first = it->first;
      const uint32_t rest = it->second - need;
      holes.erase(it);
      if (rest) holes[*first + need] = rest;
      in_use += need;
      return true;
    }
    if ((uint64_t)top + need > cap) return false;
    *first = top;
    top += need;
    in_use += need;
    return true;
  }
  void give(uint32_t first, uint32_t n) {
    if (n == 0) return;
    in_use -= n;
    auto next = holes.lower_bound(first);
    if (next != holes.begin()) {  // join with the free run that ends where this one starts
      auto prev = std::prev(next);
      if (prev->first + prev->second == first) { first = prev->first; n += prev->second; holes.erase(prev); }
    }
    if (next != holes.end() && first + n == next->first) { n += next->second; holes.erase(next); }
    if (first + n == top) top = first;  // the run reaches the untouched tail: it becomes part of it
    else holes[first] = n;
  }
};

struct gf_wgraph {
  gf_wgraph_desc_t desc{};
  PoolGeom pool{};
  AttnShape shape{};
  GraphDev gd{};
  int32_t* status_dev = nullptr;
  std::vector<int32_t> node_len;  // -1 = never written
  std::vector<int32_t> node_off;
  // nodes whose state is kept as a base node's tiles plus a sparse residual (no extent of their own)
  std::vector<int32_t> node_base;   // base node, -1: an ordinary node
  std::vector<int32_t> node_res;    // row of the residual table, -1: none
  std::vector<int32_t> variants_of; // how many such nodes name this node as their base
  std::vector<int32_t> free_res_rows;
  ResidualEntry* res_table_dev = nullptr;  // [num_layers][max_residual_nodes]
  ScoreGraphDev score_graph{};             // the task-conditioned graph for gf_edge_scores
  int32_t res_rows_in_use = 0;
  TilePool tiles;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  size_t ws_graph_end = 0;  // tables are carved after this offset
  gf_tables tables;
  uint64_t generation = 1;
  uint64_t launches = 0;
  int32_t num_sms = 148;
  int32_t last_bounds_site = 0;  // debug build: site code of the range check behind the last GF_ERR_BOUNDS
  bool wide_hint = true;  // the last batch whose sizes were read back had enough widely shared work
  int32_t split_hint = 0; // and this is how its two decode kernels shared the multiprocessors
  // Side stream and fork / join events for running the two decode kernels of a layer side by side.
  // Host objects, created on first use; no device memory is allocated for them by this library.
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  int32_t wide_min_group = 64;  // decode: segments shared this widely go to the tensor-memory kernel
  // optional per-kernel timing
  bool profiling = false;
  struct Span { cudaEvent_t a, b; int kind, launches; };
  std::vector<Span> spans;
  std::vector<cudaEvent_t> free_events;
  gf_profile_t prof{};
};

namespace {

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

struct Carver {
  char* base;
  size_t off, cap;
  bool ok = true;
  template <typename T>
  T* take(size_t count, size_t align = 16) {
    off = align_up(off, align);
    T* p = reinterpret_cast<T*>(base + off);
    off += count * sizeof(T);
    if (off > cap) ok = false;
    return p;
  }
};

size_t graph_region_bytes(int num_nodes, int num_shared, int num_edges, int residual_rows) {
  size_t b = 0;
  b = align_up(b + (size_t)(num_shared + 1) * 4, 16);
  b = align_up(b + (size_t)(num_edges > 0 ? num_edges : 1) * 4, 16);
  b = align_up(b + (size_t)num_nodes * 4, 16);
  b = align_up(b + (size_t)num_nodes * 4, 16);
  b = align_up(b + (size_t)num_nodes * 4, 16);
  b = align_up(b + (size_t)residual_rows * sizeof(ResidualEntry), 16);
  // the task-conditioned graph: symmetric neighbourhoods, 1 / sqrt(deg), edge endpoints
  b = align_up(b + (size_t)(num_shared + 1) * 4, 16);
  b = align_up(b + (size_t)(num_edges > 0 ? 2 * num_edges : 1) * 4, 16);
  b = align_up(b + (size_t)(num_shared + 1) * 4, 16);
  b = align_up(b + (size_t)(num_edges > 0 ? num_edges : 1) * 4, 16);
  b = align_up(b + 64, 256);
  return b;
}

size_t phase_a_bytes(int num_nodes, int R, int P) {
  const size_t seg_cap = (size_t)(num_nodes < P ? num_nodes : P);
  size_t b = 256;                                   // header
  b += align_up((size_t)(num_nodes + 1) * 4, 16);  // node_seg
  b += 3 * align_up(seg_cap * 4, 16);              // seg_node/len/off
  b += align_up((seg_cap + 1) * 4, 16);            // grp_ptr
  b += align_up(seg_cap * 4, 16);                  // grp_fill
  b += 2 * align_up((size_t)P * 4, 16);            // grp_tmp, grp_req
  b += 2 * align_up(seg_cap * 4, 16);              // seg_chunk, seg_nchunk
  b += 2 * align_up((seg_cap + 1) * 4, 16);        // item/part bases
  b += 7 * align_up((size_t)R * 4, 16);            // req_len/nseg/nslot/qrows, self_seg, req_order, ext_written
  b += 3 * align_up((size_t)(R + 1) * 4, 16);      // pseg_ptr, mrg_ptr, q_ptr
  b += align_up((size_t)P * 4, 16);                // pseg
  return b + 256;
}

enum { kSpanTables = 0, kSpanDecode, kSpanMerge, kSpanExtend };

cudaEvent_t take_event(gf_wgraph* g) {
  if (!g->free_events.empty()) {
    cudaEvent_t e = g->free_events.back();
    g->free_events.pop_back();
    return e;
  }
  cudaEvent_t e = nullptr;
  cudaEventCreate(&e);
  return e;
}

// Brackets one launcher call with events when profiling is on.
template <typename F>
int timed(gf_wgraph* g, int kind, cudaStream_t st, F&& launch) {
  if (!g->profiling) return launch();
  cudaEvent_t a = take_event(g), b = take_event(g);
  if (!a || !b) return launch();
  cudaEventRecord(a, st);
  const int n = launch();
  cudaEventRecord(b, st);
  g->spans.push_back({a, b, kind, n > 0 ? n : 0});
  return n;
}

void drain_spans(gf_wgraph* g) {
  for (auto& s : g->spans) {
    float ms = 0.f;
    if (cudaEventSynchronize(s.b) == cudaSuccess && cudaEventElapsedTime(&ms, s.a, s.b) == cudaSuccess) {
      double* tgt[4] = {&g->prof.tables_ms, &g->prof.decode_ms, &g->prof.merge_ms, &g->prof.extend_ms};
      uint64_t* cnt[4] = {&g->prof.tables_launches, &g->prof.decode_launches, &g->prof.merge_launches,
                          &g->prof.extend_launches};
      *tgt[s.kind] += ms;
      *cnt[s.kind] += (uint64_t)s.launches;
    }
    g->free_events.push_back(s.a);
    g->free_events.push_back(s.b);
  }
  g->spans.clear();
}

bool policy_ok(const gf_policy_t& p, int gqa) {
  return p.chunk_tokens >= kTile && p.chunk_tokens % kTile == 0 && p.chunk_tokens <= 65536 &&
         p.group_tile >= 1 && p.group_tile <= 16 && p.group_tile * gqa <= 64 && p.group_unit >= 1 &&
         p.max_chunk_mult >= 1 && p.max_chunk_mult <= 1024;
}

}  // namespace

extern "C" {

const char* gf_status_string(gf_status_t s) {
  switch (s) {
    case GF_OK: return "ok";
    case GF_ERR_INVALID_ARG: return "invalid argument";
    case GF_ERR_INVALID_GRAPH: return "invalid wGraph (bad edge or cycle)";
    case GF_ERR_INVALID_PATH: return "invalid request path";
    case GF_ERR_CAPACITY: return "KV pool or workspace too small";
    case GF_ERR_NOT_WRITTEN: return "node KV not written";
    case GF_ERR_NOT_BUILT: return "tables not built for this call";
    case GF_ERR_CUDA: return "CUDA runtime error";
    case GF_ERR_TIMEOUT: return "bounded device wait gave up";
    case GF_ERR_BOUNDS: return "a range check of the debug build failed";
  }
  return "unknown status";
}

uint64_t gf_pool_bytes_per_tile(int32_t head_dim) { return (uint64_t)2 * kTile * head_dim * 2; }

uint64_t gf_workspace_bytes(int32_t num_nodes, int32_t num_edges, int32_t max_requests,
                            int32_t max_pairs, int32_t max_items, int32_t max_slots,
                            int32_t num_q_heads, int32_t head_dim) {
  size_t b = graph_region_bytes(num_nodes, num_nodes, num_edges, 0);
  b += phase_a_bytes(num_nodes, max_requests, max_pairs);
  // The build carves items, merge slots, the wide-unit list and the partials for one common count
  // (there are never more items than slots), sized from what is left of the workspace.
  const size_t n = (size_t)(max_items > max_slots ? max_items : max_slots) + 1;
  b += n * (sizeof(Item) + 8 + (size_t)num_q_heads * (2 + head_dim) * 4);
  return (uint64_t)b + 4096;
}

gf_status_t gf_wgraph_create(const gf_wgraph_desc_t* d, gf_wgraph_t** out) {
  if (out == nullptr) return GF_ERR_INVALID_ARG;
  *out = nullptr;
  if (d == nullptr) return GF_ERR_INVALID_ARG;
  if (d->num_nodes < 1 || d->num_shared_nodes < 0 || d->num_shared_nodes > d->num_nodes ||
      d->num_edges < 0 || (d->num_edges > 0 && (!d->edge_src_host || !d->edge_dst_host)) ||
      d->max_residual_nodes < 0 || d->max_residual_nodes > (1 << 22))
    return GF_ERR_INVALID_ARG;
  if (d->num_layers < 1 || d->num_kv_heads < 1 || d->num_q_heads < d->num_kv_heads ||
      d->num_q_heads % d->num_kv_heads != 0)
    return GF_ERR_INVALID_ARG;
  const int gqa = d->num_q_heads / d->num_kv_heads;
  if (gqa != 1 && gqa != 2 && gqa != 4 && gqa != 8) return GF_ERR_INVALID_ARG;
  if (d->head_dim != 64 && d->head_dim != 128) return GF_ERR_INVALID_ARG;
  if (!(d->softmax_scale >= 0.f) || !isfinite(d->softmax_scale)) return GF_ERR_INVALID_ARG;
  if (!d->kv_pool_dev || !d->workspace_dev || ((uintptr_t)d->kv_pool_dev & 1023) ||
      ((uintptr_t)d->workspace_dev & 255))
    return GF_ERR_INVALID_ARG;

  // Sec. 3: the wGraph is a DAG.  Kahn's algorithm on the host.
  const int NS = d->num_shared_nodes, E = d->num_edges;
  std::vector<int32_t> adj_ptr(NS + 1, 0), adj_dst(E > 0 ? E : 1, 0), indeg(NS, 0);
  for (int e = 0; e < E; ++e) {
    const int a = d->edge_src_host[e], b = d->edge_dst_host[e];
    if (a < 0 || a >= NS || b < 0 || b >= NS || a == b) return GF_ERR_INVALID_GRAPH;
    adj_ptr[a + 1]++;
    indeg[b]++;
  }
  for (int v = 0; v < NS; ++v) adj_ptr[v + 1] += adj_ptr[v];
  {
    std::vector<int32_t> cur(adj_ptr.begin(), adj_ptr.end() - 1);
    for (int e = 0; e < E; ++e) adj_dst[cur[d->edge_src_host[e]]++] = d->edge_dst_host[e];
    for (int v = 0; v < NS; ++v) {  // ascending rows (insertion sort: rows are short)
      for (int i = adj_ptr[v] + 1; i < adj_ptr[v + 1]; ++i) {
        const int32_t key = adj_dst[i];
        int j = i - 1;
        while (j >= adj_ptr[v] && adj_dst[j] > key) { adj_dst[j + 1] = adj_dst[j]; --j; }
        adj_dst[j + 1] = key;
      }
    }
    std::vector<int32_t> queue;
    queue.reserve(NS);
    for (int v = 0; v < NS; ++v)
      if (indeg[v] == 0) queue.push_back(v);
    for (size_t h = 0; h < queue.size(); ++h) {
      const int v = queue[h];
      for (int i = adj_ptr[v]; i < adj_ptr[v + 1]; ++i)
        if (--indeg[adj_dst[i]] == 0) queue.push_back(adj_dst[i]);
    }
    if ((int)queue.size() != NS) return GF_ERR_INVALID_GRAPH;
  }

  gf_wgraph* g = new (std::nothrow) gf_wgraph();
  if (!g) return GF_ERR_INVALID_ARG;
  g->desc = *d;
  g->desc.edge_src_host = g->desc.edge_dst_host = nullptr;
  g->shape.num_q_heads = d->num_q_heads;
  g->shape.num_kv_heads = d->num_kv_heads;
  g->shape.head_dim = d->head_dim;
  const float scale = d->softmax_scale > 0.f ? d->softmax_scale : 1.f / sqrtf((float)d->head_dim);
  g->shape.scale_log2 = scale * 1.4426950408889634f;

  g->pool.base = (char*)d->kv_pool_dev;
  g->pool.tile_bytes = (uint32_t)gf_pool_bytes_per_tile(d->head_dim);
  const uint64_t per_tile_all = (uint64_t)g->pool.tile_bytes * d->num_kv_heads * d->num_layers;
  const uint64_t cap = d->kv_pool_bytes / per_tile_all;
  if (cap < 1 || cap > 0x7fffffffull / kTile) { delete g; return GF_ERR_CAPACITY; }
  g->pool.cap_tiles = (uint32_t)cap;
  g->tiles.cap = (uint32_t)cap;
  g->pool.head_stride = (uint64_t)g->pool.cap_tiles * g->pool.tile_bytes;
  g->pool.layer_stride = g->pool.head_stride * d->num_kv_heads;

  g->ws = (char*)d->workspace_dev;
  g->ws_bytes = d->workspace_bytes;
  if (graph_region_bytes(d->num_nodes, NS, E, d->max_residual_nodes * d->num_layers) > d->workspace_bytes) {
    delete g;
    return GF_ERR_CAPACITY;
  }
  Carver c{g->ws, 0, g->ws_bytes};
  int32_t* adj_ptr_dev = c.take<int32_t>(NS + 1);
  int32_t* adj_dst_dev = c.take<int32_t>(E > 0 ? E : 1);
  g->gd.node_len = c.take<int32_t>(d->num_nodes);
  g->gd.node_off = c.take<int32_t>(d->num_nodes);
  g->gd.node_res = c.take<int32_t>(d->num_nodes);
  g->res_table_dev = c.take<ResidualEntry>((size_t)d->max_residual_nodes * d->num_layers);
  // the task-conditioned graph of the scoring model (Sec. 4.1): operation edges in both directions,
  // duplicates dropped; deg = neighbours + the task node + the node itself
  std::vector<int32_t> sym_ptr(NS + 1, 0), sym_idx, e_src(E > 0 ? E : 1, 0);
  std::vector<float> inv_sqrt(NS + 1, 1.f);
  {
    std::vector<std::vector<int32_t>> nb(NS);
    for (int v = 0; v < NS; ++v)
      for (int i = adj_ptr[v]; i < adj_ptr[v + 1]; ++i) {
        e_src[i] = v;
        nb[v].push_back(adj_dst[i]);
        nb[adj_dst[i]].push_back(v);
      }
    for (int v = 0; v < NS; ++v) {
      std::sort(nb[v].begin(), nb[v].end());
      nb[v].erase(std::unique(nb[v].begin(), nb[v].end()), nb[v].end());
      sym_ptr[v + 1] = sym_ptr[v] + (int32_t)nb[v].size();
      sym_idx.insert(sym_idx.end(), nb[v].begin(), nb[v].end());
      inv_sqrt[v] = 1.f / sqrtf((float)(nb[v].size() + 2));
    }
    inv_sqrt[NS] = 1.f / sqrtf((float)(NS + 1));
    if (sym_idx.empty()) sym_idx.push_back(0);
  }
  int32_t* sym_ptr_dev = c.take<int32_t>(NS + 1);
  int32_t* sym_idx_dev = c.take<int32_t>(sym_idx.size());
  float* inv_sqrt_dev = c.take<float>(NS + 1);
  int32_t* e_src_dev = c.take<int32_t>(E > 0 ? E : 1);
  g->status_dev = c.take<int32_t>(kStatusWords);
  c.off = align_up(c.off, 256);
  if (!c.ok || c.off > c.cap) { delete g; return GF_ERR_CAPACITY; }
  g->ws_graph_end = c.off;
  g->gd.adj_ptr = adj_ptr_dev;
  g->gd.adj_dst = adj_dst_dev;
  g->gd.num_nodes = d->num_nodes;
  g->gd.num_shared_nodes = NS;
  bool ok = cudaMemcpy(adj_ptr_dev, adj_ptr.data(), (size_t)(NS + 1) * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(adj_dst_dev, adj_dst.data(), (size_t)(E > 0 ? E : 1) * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(sym_ptr_dev, sym_ptr.data(), (size_t)(NS + 1) * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(sym_idx_dev, sym_idx.data(), sym_idx.size() * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(inv_sqrt_dev, inv_sqrt.data(), (size_t)(NS + 1) * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  ok = ok && cudaMemcpy(e_src_dev, e_src.data(), (size_t)(E > 0 ? E : 1) * 4, cudaMemcpyHostToDevice) == cudaSuccess;
  g->score_graph = ScoreGraphDev{sym_ptr_dev, sym_idx_dev, inv_sqrt_dev, e_src_dev, adj_dst_dev, NS, E};
  ok = ok && cudaMemset(g->gd.node_len, 0xFF, (size_t)d->num_nodes * 4) == cudaSuccess;
  ok = ok && cudaMemset(g->gd.node_off, 0xFF, (size_t)d->num_nodes * 4) == cudaSuccess;
  ok = ok && cudaMemset(g->gd.node_res, 0xFF, (size_t)d->num_nodes * 4) == cudaSuccess;
  ok = ok && cudaMemset(g->status_dev, 0, kStatusWords * 4) == cudaSuccess;
  if (!ok) { delete g; return GF_ERR_CUDA; }
  g->node_len.assign(d->num_nodes, -1);
  g->node_off.assign(d->num_nodes, -1);
  g->node_base.assign(d->num_nodes, -1);
  g->node_res.assign(d->num_nodes, -1);
  g->variants_of.assign(d->num_nodes, 0);
  for (int r = d->max_residual_nodes - 1; r >= 0; --r) g->free_res_rows.push_back(r);
  {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
      g->num_sms = sms;
  }
  g->tables.owner = g;
  *out = g;
  return GF_OK;
}

gf_status_t gf_wgraph_destroy(gf_wgraph_t* g) {
  if (!g) return GF_ERR_INVALID_ARG;
  drain_spans(g);
  for (cudaEvent_t e : g->free_events) cudaEventDestroy(e);
  if (g->side_stream) {
    cudaStreamSynchronize(g->side_stream);
    cudaStreamDestroy(g->side_stream);
    cudaEventDestroy(g->ev_fork);
    cudaEventDestroy(g->ev_join);
  }
  delete g;
  return GF_OK;
}

// Gives an unwritten node its extent (first fit), or checks that a written one has this length.
// *fresh tells the caller that the device copy of the node's length and offset still has to be set.
static gf_status_t reserve_extent(gf_wgraph* g, int32_t node, int32_t n_tokens, bool* fresh) {
  *fresh = false;
  if (g->node_base[node] >= 0) return GF_ERR_INVALID_ARG;  // kept as base + residual: it has no extent to write
  if (g->node_len[node] >= 0) return g->node_len[node] == n_tokens ? GF_OK : GF_ERR_INVALID_ARG;
  uint32_t first = 0;
  if (!g->tiles.take((uint32_t)((n_tokens + kTile - 1) / kTile), &first)) return GF_ERR_CAPACITY;
  g->node_len[node] = n_tokens;
  g->node_off[node] = (int32_t)(first * kTile);
  g->generation++;  // lengths changed: built tables are stale
  *fresh = true;
  return GF_OK;
}

gf_status_t gf_node_kv_write(gf_wgraph_t* g, int32_t node, int32_t layer, const void* k_dev,
                             const void* v_dev, int32_t n_tokens, void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes || layer < 0 || layer >= g->desc.num_layers ||
      n_tokens < 0)
    return GF_ERR_INVALID_ARG;
  if (n_tokens > 0 && (!k_dev || !v_dev || ((uintptr_t)k_dev & 15) || ((uintptr_t)v_dev & 15)))
    return GF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  bool fresh = false;
  const gf_status_t rs = reserve_extent(g, node, n_tokens, &fresh);
  if (rs != GF_OK) return rs;
  // the copy kernel also records a fresh node's length and offset on the device; an empty node has no copy
  if (fresh && n_tokens == 0) {
    const int n = launch_graph_set_node(g->gd, node, n_tokens, g->node_off[node], st);
    if (n < 0) return GF_ERR_CUDA;
    g->launches += n;
  }
  int n = launch_kv_write(g->pool, layer, g->desc.num_kv_heads, g->desc.head_dim,
                          g->node_off[node] / kTile, k_dev, v_dev, n_tokens, fresh ? &g->gd : nullptr, node,
                          g->status_dev, st);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_node_kv_reserve(gf_wgraph_t* g, int32_t node, int32_t n_tokens, void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes || n_tokens < 0) return GF_ERR_INVALID_ARG;
  bool fresh = false;
  const gf_status_t rs = reserve_extent(g, node, n_tokens, &fresh);
  if (rs != GF_OK) return rs;
  if (fresh) {
    const int n = launch_graph_set_node(g->gd, node, n_tokens, g->node_off[node], (cudaStream_t)stream);
    if (n < 0) return GF_ERR_CUDA;
    g->launches += n;
  }
  return GF_OK;
}

gf_status_t gf_node_kv_release(gf_wgraph_t* g, int32_t node, void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes) return GF_ERR_INVALID_ARG;
  if (g->node_len[node] < 0) return GF_ERR_NOT_WRITTEN;
  if (g->variants_of[node] > 0) return GF_ERR_INVALID_ARG;  // states kept as this node's tiles + residual still exist
  cudaStream_t st = (cudaStream_t)stream;
  if (g->node_base[node] >= 0) {
    // a state kept as base + residual owns no tiles: only its row of the residual table comes back
    g->variants_of[g->node_base[node]]--;
    g->free_res_rows.push_back(g->node_res[node]);
    g->res_rows_in_use--;
    g->node_base[node] = -1;
    g->node_res[node] = -1;
    const int m = launch_set_residual(nullptr, ResidualEntry{}, g->gd.node_res, node, -1, st);
    if (m < 0) return GF_ERR_CUDA;
    g->launches += m;
  } else {
    g->tiles.give((uint32_t)(g->node_off[node] / kTile), (uint32_t)((g->node_len[node] + kTile - 1) / kTile));
  }
  g->node_len[node] = -1;
  g->node_off[node] = -1;
  g->generation++;  // built tables may name the node: stale
  const int n = launch_graph_set_node(g->gd, node, -1, -1, st);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_node_extent(const gf_wgraph_t* g, int32_t node, int32_t* n_tokens, int32_t* token_offset) {
  if (!g || node < 0 || node >= g->desc.num_nodes) return GF_ERR_INVALID_ARG;
  if (g->node_len[node] < 0) return GF_ERR_NOT_WRITTEN;
  if (n_tokens) *n_tokens = g->node_len[node];
  if (token_offset) *token_offset = g->node_off[node];
  return GF_OK;
}

gf_status_t gf_pool_info(const gf_wgraph_t* g, gf_pool_info_t* out) {
  if (!g || !out) return GF_ERR_INVALID_ARG;
  out->capacity_tiles = g->tiles.cap;
  out->tiles_in_use = g->tiles.in_use;
  out->high_water_tiles = g->tiles.top;
  return GF_OK;
}

gf_status_t gf_node_kv_read(gf_wgraph_t* g, int32_t node, int32_t layer, void* k_out_dev,
                            void* v_out_dev, void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes || layer < 0 || layer >= g->desc.num_layers)
    return GF_ERR_INVALID_ARG;
  if (g->node_len[node] < 0) return GF_ERR_NOT_WRITTEN;
  const int n_tokens = g->node_len[node];
  if (n_tokens > 0 && (!k_out_dev || !v_out_dev || ((uintptr_t)k_out_dev & 15) || ((uintptr_t)v_out_dev & 15)))
    return GF_ERR_INVALID_ARG;
  int n = launch_kv_read(g->pool, layer, g->desc.num_kv_heads, g->desc.head_dim, g->node_off[node] / kTile,
                         k_out_dev, v_out_dev, n_tokens, (cudaStream_t)stream);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

static bool residual_ok(const gf_residual_t* r) {
  if (!r) return true;
  if (r->nnz < 0 || r->nnz > 0x7fffffff || !r->bitmap_dev || !r->row_ptr_dev || (r->nnz > 0 && !r->values_dev)) return false;
  return (((uintptr_t)r->bitmap_dev & 15) | ((uintptr_t)r->row_ptr_dev & 3) | ((uintptr_t)r->values_dev & 1)) == 0;
}

gf_status_t gf_node_kv_reconstruct(gf_wgraph_t* g, int32_t node, int32_t layer, int32_t base_node,
                                   const gf_residual_t* k_res, const gf_residual_t* v_res,
                                   void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes || base_node < 0 || base_node >= g->desc.num_nodes ||
      node == base_node || layer < 0 || layer >= g->desc.num_layers || !residual_ok(k_res) || !residual_ok(v_res))
    return GF_ERR_INVALID_ARG;
  if (g->node_len[base_node] < 0) return GF_ERR_NOT_WRITTEN;
  const int n_tokens = g->node_len[base_node];
  if (((int64_t)n_tokens + kTile) * g->desc.num_kv_heads > 0x7fffffff) return GF_ERR_INVALID_ARG;  // rows are indexed with int32
  cudaStream_t st = (cudaStream_t)stream;
  bool fresh = false;
  const gf_status_t rs = reserve_extent(g, node, n_tokens, &fresh);
  if (rs != GF_OK) return rs;
  if (fresh) {
    const int n = launch_graph_set_node(g->gd, node, n_tokens, g->node_off[node], st);
    if (n < 0) return GF_ERR_CUDA;
    g->launches += n;
  }
  int n = launch_kv_reconstruct(g->pool, layer, g->desc.num_kv_heads, g->desc.head_dim,
                                g->node_off[node] / kTile, g->node_off[base_node] / kTile, k_res, v_res,
                                n_tokens, g->status_dev, st);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_node_kv_attach_residual(gf_wgraph_t* g, int32_t node, int32_t layer, int32_t base_node,
                                       const gf_residual_t* k_res, const gf_residual_t* v_res, void* stream) {
  if (!g || node < 0 || node >= g->desc.num_nodes || base_node < 0 || base_node >= g->desc.num_nodes ||
      node == base_node || layer < 0 || layer >= g->desc.num_layers || !residual_ok(k_res) || !residual_ok(v_res))
    return GF_ERR_INVALID_ARG;
  if (g->node_len[base_node] < 0) return GF_ERR_NOT_WRITTEN;
  if (g->node_base[base_node] >= 0) return GF_ERR_INVALID_ARG;  // the base must own its tiles
  const int n_tokens = g->node_len[base_node];
  if ((int64_t)n_tokens * g->desc.num_kv_heads > 0x7fffffff) return GF_ERR_INVALID_ARG;  // rows are indexed with int32
  cudaStream_t st = (cudaStream_t)stream;
  if (g->node_len[node] < 0) {
    if (g->free_res_rows.empty()) return GF_ERR_CAPACITY;
    const int row = g->free_res_rows.back();
    g->free_res_rows.pop_back();
    g->res_rows_in_use++;
    g->node_len[node] = n_tokens;
    g->node_off[node] = g->node_off[base_node];  // the node's tiles are the base node's
    g->node_base[node] = base_node;
    g->node_res[node] = row;
    g->variants_of[base_node]++;
    g->generation++;
    const int n = launch_graph_set_node(g->gd, node, n_tokens, g->node_off[node], st);
    if (n < 0) return GF_ERR_CUDA;
    g->launches += n;
  } else if (g->node_base[node] != base_node) {
    return GF_ERR_INVALID_ARG;  // written as an ordinary node, or attached to another base
  }
  ResidualEntry e{};
  e.k_nnz = e.v_nnz = -1;
  if (k_res) { e.k_bitmap = k_res->bitmap_dev; e.k_values = (const uint16_t*)k_res->values_dev; e.k_row_ptr = k_res->row_ptr_dev; e.k_nnz = (int32_t)k_res->nnz; }
  if (v_res) { e.v_bitmap = v_res->bitmap_dev; e.v_values = (const uint16_t*)v_res->values_dev; e.v_row_ptr = v_res->row_ptr_dev; e.v_nnz = (int32_t)v_res->nnz; }
  const int row = g->node_res[node];
  const int n = launch_set_residual(g->res_table_dev + (size_t)layer * g->desc.max_residual_nodes + row, e, g->gd.node_res,
                                    node, row, st);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

static bool residual_buf_ok(const gf_residual_buf_t* r, const void* full) {
  if (!r) return true;
  if (!full || ((uintptr_t)full & 15) || r->capacity < 0 || !r->bitmap_dev || !r->row_ptr_dev || !r->nnz_dev ||
      (r->capacity > 0 && !r->values_dev))
    return false;
  return (((uintptr_t)r->bitmap_dev & 15) | ((uintptr_t)r->row_ptr_dev & 3) | ((uintptr_t)r->values_dev & 1) |
          ((uintptr_t)r->nnz_dev & 7)) == 0;
}

gf_status_t gf_residual_encode(gf_wgraph_t* g, int32_t base_node, int32_t layer, const void* k_full_dev,
                               const void* v_full_dev, float threshold, const gf_residual_buf_t* k_out,
                               const gf_residual_buf_t* v_out, void* stream) {
  if (!g || base_node < 0 || base_node >= g->desc.num_nodes || layer < 0 || layer >= g->desc.num_layers ||
      !(threshold >= 0.f) || !residual_buf_ok(k_out, k_full_dev) || !residual_buf_ok(v_out, v_full_dev))
    return GF_ERR_INVALID_ARG;
  if (g->node_len[base_node] < 0) return GF_ERR_NOT_WRITTEN;
  const int n_tokens = g->node_len[base_node];
  if ((int64_t)n_tokens * g->desc.num_kv_heads > 0x7fffffff) return GF_ERR_INVALID_ARG;  // rows are indexed with int32
  int n = launch_residual_encode(g->pool, layer, g->desc.num_kv_heads, g->desc.head_dim,
                                 g->node_off[base_node] / kTile, k_full_dev, v_full_dev, n_tokens, threshold,
                                 k_out, v_out, g->status_dev, (cudaStream_t)stream);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_transition_counts(gf_wgraph_t* g, int32_t num_requests, int32_t num_path_nodes,
                                 const int32_t* path_ptr_dev, const int32_t* path_node_dev,
                                 int32_t* counts_dev, uint64_t* misses_dev, void* stream) {
  if (!g || num_requests < 0 || num_path_nodes < 0 || !misses_dev || (g->desc.num_edges > 0 && !counts_dev) ||
      (num_requests > 0 && (!path_ptr_dev || !path_node_dev)) || ((uintptr_t)misses_dev & 7))
    return GF_ERR_INVALID_ARG;
  int n = launch_transition_counts(g->gd, g->desc.num_edges, num_requests, num_path_nodes, path_ptr_dev,
                                   path_node_dev, counts_dev, (unsigned long long*)misses_dev, (cudaStream_t)stream);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_select_transitions(gf_wgraph_t* g, const int32_t* counts_dev, int32_t min_count,
                                  uint8_t* keep_dev, uint64_t* totals_dev, void* stream) {
  if (!g || !totals_dev || ((uintptr_t)totals_dev & 7) || (g->desc.num_edges > 0 && (!counts_dev || !keep_dev)))
    return GF_ERR_INVALID_ARG;
  int n = launch_select_transitions(counts_dev, g->desc.num_edges, min_count, keep_dev,
                                    (unsigned long long*)totals_dev, (cudaStream_t)stream);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

// How many multiprocessors the warp decode kernel leaves to the tensor-memory decode kernel while the
// two run side by side.  A model of both, fitted to measurements on the high-sharing and the full-depth
// workloads: the tensor-memory kernel costs about 0.8 us per (128-token stage x 128-row tile) plus 13 us
// per (chunk x tile) for loading its queries and writing its partials, spread over its multiprocessors;
// the warp kernel streams its segments at 6.2 TB/s when nearly every tile is used by one 16-row group
// and slower (down to 4.4) the more groups share a tile, and slows down with fewer multiprocessors the
// less it is bound by HBM.  The split balances the two times.  It need not be exact: the tensor-memory
// kernel is launched with a CTA for every multiprocessor, and those that find no room at first start when
// the warp kernel's CTAs leave.
static int decode_split(const gf_wgraph* g, const Header& h) {
  const int sms = g->num_sms;
  const double heads = g->desc.num_kv_heads;
  const double wide_sm_us = (0.80 * h.wide_work + 13.0 * h.wide_tile_units) * heads;  // us x multiprocessors
  const double stream_tokens = (double)h.resident_tokens - (double)h.wide_tokens;
  if (!(wide_sm_us > 0.0) || !(stream_tokens > 0.0)) return 0;
  const double steps_per_tile = (double)h.stream_steps / (stream_tokens / kTile);
  double rate = 6.2 - 2.46 * (steps_per_tile - 1.17);   // TB/s
  rate = rate < 4.4 ? 4.4 : (rate > 6.2 ? 6.2 : rate);
  double alpha = 0.1 + 0.72 * (steps_per_tile - 1.17);  // how much fewer multiprocessors slow the stream down
  alpha = alpha < 0.1 ? 0.1 : (alpha > 0.7 ? 0.7 : alpha);
  const double bytes_per_token = 2.0 * heads * g->desc.head_dim * 2.0;
  const double t_stream = stream_tokens * bytes_per_token / (rate * 1e6);  // us on every multiprocessor
  int best_x = 0;
  double best_t = 0.0;
  for (int x = 2; x <= sms / 2; ++x) {
    const double tw = wide_sm_us / x, ts = t_stream * pow((double)sms / (sms - x), alpha);
    const double t = tw > ts ? tw : ts;
    if (best_x == 0 || t < best_t) { best_x = x; best_t = t; }
  }
  return best_x;
}

// Waits for the build stream and reads the header: sizes, totals, validation result.
static gf_status_t read_back_tables(gf_tables* T) {
  Header h;
  if (cudaMemcpyAsync(&h, T->dev.hdr, sizeof(Header), cudaMemcpyDeviceToHost, T->build_stream) != cudaSuccess ||
      cudaStreamSynchronize(T->build_stream) != cudaSuccess)
    return GF_ERR_CUDA;
  if (h.bad_req != 0x7fffffff) {
    T->bad_req = h.bad_req;
    return GF_ERR_INVALID_PATH;
  }
  if (h.mrg_total != h.num_slots) return GF_ERR_CUDA;  // internal consistency
  if (!tables_usable(h, T->dev.slot_cap)) return GF_ERR_CAPACITY;
  T->info.num_segments = h.num_segments;
  T->info.num_pairs = h.num_pairs;
  T->info.num_items = h.num_items;
  T->info.num_slots = h.num_slots;
  T->info.resident_tokens = (int64_t)h.resident_tokens;
  T->info.materialised_tokens = (int64_t)h.materialised_tokens;
  T->info.num_q_rows = (int64_t)h.num_q_rows;
  T->max_q_rows = h.max_q_rows;
  T->num_wide = h.num_wide;
  T->owner->wide_hint = h.wide_units >= T->dev.wide_min_units;
  T->split_sms = h.num_wide > 0 ? decode_split(T->owner, h) : 0;
  T->owner->split_hint = T->split_sms;
  return GF_OK;
}

gf_status_t gf_build_path_tables(gf_wgraph_t* g, int32_t num_requests, int32_t num_path_nodes,
                                 const int32_t* path_ptr_dev, const int32_t* path_node_dev,
                                 int32_t mode, const gf_policy_t* policy, gf_tables_t** out,
                                 void* stream) {
  if (out) *out = nullptr;
  if (!g || !out || num_requests < 1 || num_path_nodes < num_requests || !path_ptr_dev ||
      !path_node_dev)
    return GF_ERR_INVALID_ARG;
  const bool deferred = (mode & GF_MODE_DEFERRED) != 0;
  mode &= ~GF_MODE_DEFERRED;
  if ((mode != GF_MODE_DECODE && mode != GF_MODE_EXTEND) || (deferred && mode != GF_MODE_DECODE))
    return GF_ERR_INVALID_ARG;
  if (mode == GF_MODE_EXTEND && num_requests > 65535) return GF_ERR_INVALID_ARG;  // requests are a grid dimension there
  gf_policy_t pol = policy ? *policy : gf_policy_t{256, 16, 2, 16};
  const int gqa = g->shape.num_q_heads / g->shape.num_kv_heads;
  if (!policy) while (pol.group_tile * gqa > 64) pol.group_tile >>= 1;
  if (!policy_ok(pol, gqa)) return GF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;

  gf_tables& T = g->tables;
  T.built = false;
  T.bad_req = -1;
  T.policy = pol;
  const int R = num_requests, P = num_path_nodes, N = g->desc.num_nodes;
  const int seg_cap = N < P ? N : P;
  Carver c{g->ws, g->ws_graph_end, g->ws_bytes};
  TablesDev& t = T.dev;
  t = TablesDev{};
  t.hdr = c.take<Header>(1, 256);
  t.node_seg = c.take<int32_t>(N + 1);
  t.seg_node = c.take<int32_t>(seg_cap);
  t.seg_len = c.take<int32_t>(seg_cap);
  t.seg_off = c.take<int32_t>(seg_cap);
  t.grp_ptr = c.take<int32_t>(seg_cap + 1);
  t.grp_fill = c.take<int32_t>(seg_cap);
  t.grp_tmp = c.take<int32_t>(P);
  t.grp_req = c.take<int32_t>(P);
  t.seg_chunk = c.take<int32_t>(seg_cap);
  t.seg_nchunk = c.take<int32_t>(seg_cap);
  t.seg_item_base = c.take<int32_t>(seg_cap + 1);
  t.seg_part_base = c.take<int32_t>(seg_cap + 1);
  t.req_len = c.take<int32_t>(R);
  t.req_nseg = c.take<int32_t>(R);
  t.req_nslot = c.take<int32_t>(R);
  t.req_qrows = c.take<int32_t>(R);
  t.self_seg = c.take<int32_t>(R);
  t.req_order = c.take<int32_t>(R);
  t.ext_written = c.take<int32_t>(R);
  t.pseg_ptr = c.take<int32_t>(R + 1);
  t.mrg_ptr = c.take<int32_t>(R + 1);
  t.q_ptr = c.take<int32_t>(R + 1);
  t.pseg = c.take<int32_t>(P);
  if (!c.ok) return GF_ERR_CAPACITY;
  t.status = g->status_dev;
  t.node_res = g->gd.node_res;
  t.seg_cap = seg_cap;
  t.num_requests = R;
  t.num_pairs_in = P;
  t.mode = mode;
  t.wide_min_group = (mode == GF_MODE_DECODE) ? g->wide_min_group : 0;
  t.wide_probe_group = g->wide_min_group;
  if (deferred && !g->wide_hint) t.wide_min_group = 0;  // nothing to launch blindly: every chunk goes to the warp kernel
  t.wide_min_units = (g->num_sms + g->desc.num_kv_heads - 1) / g->desc.num_kv_heads;
  t.num_sms = g->num_sms;
  t.wide_unit_req = 256 / gqa;

  // Items, merge slots and partials take the rest of the workspace; how many exist is only known on
  // the device until the header is read back, so the room is expressed as a slot capacity.
  {
    c.off = align_up(c.off, 256);
    const size_t per_slot = sizeof(Item) + 8 + (size_t)g->shape.num_q_heads * (2 + g->shape.head_dim) * 4;
    const size_t room = c.cap > c.off + 1024 ? c.cap - c.off - 1024 : 0;
    const size_t cap = room / per_slot < 0x7fffffffu ? room / per_slot : 0x7fffffffu;
    if (cap < 1) return GF_ERR_CAPACITY;
    t.slot_cap = (int32_t)cap;
    t.items = c.take<Item>(cap, 32);
    t.mrg_slot = c.take<int32_t>(cap);
    t.wide_list = c.take<int32_t>(cap);
    t.part_ml = c.take<float>(cap * g->shape.num_q_heads * 2, 256);
    t.part_o = c.take<float>(cap * g->shape.num_q_heads * g->shape.head_dim, 256);
    if (!c.ok) return GF_ERR_CAPACITY;
  }
  T.pending = false;
  T.num_wide = -1;
  T.error = GF_OK;
  T.build_stream = st;
  T.info = gf_tables_info_t{};
  T.info.num_requests = R;
  T.info.mode = mode;

  int n = timed(g, kSpanTables, st, [&] { return launch_tables_phase_a(g->gd, t, path_ptr_dev, path_node_dev, pol, st); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  *out = &T;
  if (deferred) {
    // (the wide decode kernel was enabled above only if the last batch whose sizes the host saw had work for it)
    // everything is enqueued without waiting: the kernels read the sizes on the device and do
    // nothing if a path is invalid or the workspace too small; the first call that needs the sizes
    // on the host (or gf_last_status) waits and reports
    n = timed(g, kSpanTables, st, [&] { return launch_tables_phase_b(t, path_ptr_dev, path_node_dev, pol, -1, st); });
    if (n < 0) return GF_ERR_CUDA;
    g->launches += n;
    T.pending = true;
    T.built = true;
    T.generation = g->generation;
    return GF_OK;
  }
  const gf_status_t fs = read_back_tables(&T);
  if (fs != GF_OK) return fs;
  n = timed(g, kSpanTables, st, [&] { return launch_tables_phase_b(t, path_ptr_dev, path_node_dev, pol, T.info.num_items, st); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  T.built = true;
  T.generation = g->generation;
  return GF_OK;
}

// Completes a deferred build on the host side; GF_OK when nothing is pending.
static gf_status_t finalize_tables(const gf_tables_t* ct) {
  gf_tables* T = const_cast<gf_tables*>(ct);
  if (!T->pending) return T->error;
  T->pending = false;
  T->error = read_back_tables(T);
  if (T->error != GF_OK) T->built = false;
  return T->error;
}

gf_status_t gf_tables_info(const gf_tables_t* t, gf_tables_info_t* info) {
  if (!t || !info) return GF_ERR_INVALID_ARG;
  if (t->pending) {
    const gf_status_t fs = finalize_tables(t);
    if (fs != GF_OK) return fs;
  }
  if (!t->built) return GF_ERR_NOT_BUILT;
  *info = t->info;
  return GF_OK;
}

int32_t gf_tables_bad_request(const gf_tables_t* t) {
  if (!t) return -1;
  if (t->pending) finalize_tables(t);
  return t->bad_req;
}

gf_status_t gf_tables_export(const gf_tables_t* t, gf_tables_host_t* o) {
  if (!t || !o) return GF_ERR_INVALID_ARG;
  if (t->pending) {
    const gf_status_t fs = finalize_tables(t);
    if (fs != GF_OK) return fs;
  }
  if (!t->built) return GF_ERR_NOT_BUILT;
  const TablesDev& d = t->dev;
  const gf_tables_info_t& i = t->info;
  bool ok = true;
  auto get = [&](int32_t* dst, const int32_t* src, size_t count) {
    if (dst && count)
      ok = ok && cudaMemcpy(dst, src, count * 4, cudaMemcpyDeviceToHost) == cudaSuccess;
  };
  get(o->seg_node, d.seg_node, i.num_segments);
  get(o->seg_len, d.seg_len, i.num_segments);
  get(o->seg_off, d.seg_off, i.num_segments);
  get(o->grp_ptr, d.grp_ptr, (size_t)i.num_segments + 1);
  get(o->grp_req, d.grp_req, i.num_pairs);
  get(o->req_len, d.req_len, i.num_requests);
  get(o->req_nseg, d.req_nseg, i.num_requests);
  get(o->mrg_ptr, d.mrg_ptr, (size_t)i.num_requests + 1);
  get(o->mrg_slot, d.mrg_slot, i.num_slots);
  get(o->pseg_ptr, d.pseg_ptr, (size_t)i.num_requests + 1);
  get(o->pseg, d.pseg, i.num_pairs);
  if (i.mode == GF_MODE_EXTEND) {
    get(o->q_ptr, d.q_ptr, (size_t)i.num_requests + 1);
    get(o->self_seg, d.self_seg, i.num_requests);
  }
  if (o->items && i.num_items) {
    std::vector<Item> tmp(i.num_items);
    ok = ok && cudaMemcpy(tmp.data(), d.items, (size_t)i.num_items * sizeof(Item), cudaMemcpyDeviceToHost) == cudaSuccess;
    for (int k = 0; ok && k < i.num_items; ++k) {
      int32_t* p = o->items + (size_t)k * 6;
      p[0] = tmp[k].seg; p[1] = tmp[k].tok_begin; p[2] = tmp[k].tok_count;
      p[3] = tmp[k].grp_begin; p[4] = tmp[k].grp_count; p[5] = tmp[k].part_base;
    }
  }
  return ok ? GF_OK : GF_ERR_CUDA;
}

static gf_status_t check_attention_args(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                        const void* q, void* out, int mode) {
  if (!g || !t || !q || !out || layer < 0 || layer >= g->desc.num_layers ||
      ((uintptr_t)q & 15) || ((uintptr_t)out & 15))
    return GF_ERR_INVALID_ARG;
  if (t != &g->tables || !t->built || t->generation != g->generation || t->info.mode != mode)
    return GF_ERR_NOT_BUILT;
  return GF_OK;
}

static bool ensure_side_stream(gf_wgraph* g) {
  if (g->side_stream) return true;
  cudaStream_t s = nullptr;
  cudaEvent_t a = nullptr, b = nullptr;
  if (cudaStreamCreateWithFlags(&s, cudaStreamNonBlocking) != cudaSuccess ||
      cudaEventCreateWithFlags(&a, cudaEventDisableTiming) != cudaSuccess ||
      cudaEventCreateWithFlags(&b, cudaEventDisableTiming) != cudaSuccess) {
    if (b) cudaEventDestroy(b);
    if (a) cudaEventDestroy(a);
    if (s) cudaStreamDestroy(s);
    return false;
  }
  g->side_stream = s;
  g->ev_fork = a;
  g->ev_join = b;
  return true;
}

// K2 of one layer with the tables `td` (partials possibly redirected): the warp kernel and, when the
// batch has widely shared chunks, the tensor-memory kernel.  The two work on disjoint items and share
// nothing but the tables, and one is bound by HBM while the other is bound by its MMAs, so they run
// side by side: the tensor-memory kernel on a side stream (forked after everything enqueued on `st` so
// far, joined before anything that follows), the warp kernel leaving it as many multiprocessors as
// decode_split says.  Returns the number of kernels enqueued, or -1.
static int launch_decode_kernels(gf_wgraph* g, const gf_tables* t, const TablesDev& td, int layer, const void* q,
                                 cudaStream_t st, bool* joined) {
  *joined = false;
  const int num_items = t->pending ? -1 : t->info.num_items;
  const ResidualEntry* residuals =
      g->res_rows_in_use > 0 ? g->res_table_dev + (size_t)layer * g->desc.max_residual_nodes : nullptr;
  const bool wide = td.wide_min_group > 0 && t->num_wide != 0;
  const int split = wide ? (t->pending ? g->split_hint : t->split_sms) : 0;
  if (wide && split > 0 && ensure_side_stream(g)) {
    if (cudaEventRecord(g->ev_fork, st) != cudaSuccess || cudaStreamWaitEvent(g->side_stream, g->ev_fork, 0) != cudaSuccess)
      return -1;
    // the warp kernel first: its CTAs are placed before the other kernel's, and those on the multiprocessors
    // it yields leave at once, so the tensor-memory kernel's first CTAs land there instead of ahead of it
    const int b = launch_decode(g->pool, g->shape, td, num_items, layer, q, g->status_dev, split, residuals, st);
    const int a = launch_decode_wide(g->pool, g->shape, td, num_items, layer, q, g->status_dev, 0, split, false, g->side_stream);
    if (a < 0 || cudaEventRecord(g->ev_join, g->side_stream) != cudaSuccess) return -1;
    if (cudaStreamWaitEvent(st, g->ev_join, 0) != cudaSuccess || b < 0) return -1;
    *joined = true;
    return a + b;
  }
  const int b = launch_decode(g->pool, g->shape, td, num_items, layer, q, g->status_dev, 0, residuals, st);
  if (b < 0) return -1;
  int a = 0;
  if (wide) a = launch_decode_wide(g->pool, g->shape, td, num_items, layer, q, g->status_dev, 0, 0, true, st);
  return a < 0 ? -1 : a + b;
}

gf_status_t gf_path_attention_decode(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                     const void* q_dev, void* out_dev, float* lse_dev, void* stream) {
  gf_status_t s = check_attention_args(g, t, layer, q_dev, out_dev, GF_MODE_DECODE);
  if (s != GF_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  bool joined = false;
  int n = timed(g, kSpanDecode, st, [&] { return launch_decode_kernels(g, t, t->dev, layer, q_dev, st, &joined); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  n = timed(g, kSpanMerge, st, [&] { return launch_merge(g->shape, t->dev, out_dev, lse_dev, !joined, st); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_path_attention_extend(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                     const void* q_dev, void* out_dev, float* lse_dev, void* stream) {
  gf_status_t s = check_attention_args(g, t, layer, q_dev, out_dev, GF_MODE_EXTEND);
  if (s != GF_OK) return s;
  cudaStream_t st = (cudaStream_t)stream;
  int n = timed(g, kSpanExtend, st, [&] {
    return launch_extend_tc(g->pool, g->shape, t->dev, layer, t->max_q_rows, t->info.num_q_rows, q_dev, nullptr, nullptr, out_dev, lse_dev,
                            g->status_dev, st);
  });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

gf_status_t gf_path_attention_extend_append(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                            const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                                            void* out_dev, float* lse_dev, void* stream) {
  gf_status_t s = check_attention_args(g, t, layer, q_dev, out_dev, GF_MODE_EXTEND);
  if (s != GF_OK) return s;
  if (!k_new_dev || !v_new_dev || ((uintptr_t)k_new_dev & 15) || ((uintptr_t)v_new_dev & 15)) return GF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int n = timed(g, kSpanExtend, st, [&] {
    return launch_extend_tc(g->pool, g->shape, t->dev, layer, t->max_q_rows, t->info.num_q_rows, q_dev, k_new_dev, v_new_dev, out_dev,
                            lse_dev, g->status_dev, st);
  });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}

static bool scorer_ok(const gf_scorer_t* m) {
  return m && m->d_in >= 1 && m->d_hidden >= 1 && m->d_hidden <= 4096 && m->d_mlp >= 32 && m->d_mlp <= 128 &&
         m->d_mlp % 32 == 0 && m->w_gcn1_dev && m->w_gcn2_dev && m->w_mlp1_dev && m->b_mlp1_dev && m->w_mlp2_dev &&
         m->b_mlp2_dev && m->w_mlp3_dev;
}

uint64_t gf_edge_scores_scratch_bytes(const gf_wgraph_t* g, const gf_scorer_t* m, int32_t num_tasks, int32_t per_pass) {
  if (!g || !scorer_ok(m) || num_tasks < 1 || per_pass < 1) return 0;
  if (per_pass > num_tasks) per_pass = num_tasks;
  return (uint64_t)edge_scores_scratch_floats(g->desc.num_shared_nodes, *m, num_tasks, per_pass) * 4;
}

gf_status_t gf_edge_scores(gf_wgraph_t* g, const gf_scorer_t* m, const float* x_op_dev, int32_t num_tasks,
                           const float* x_task_dev, float* scores_dev, void* scratch_dev, uint64_t scratch_bytes,
                           void* stream) {
  if (!g || !scorer_ok(m) || num_tasks < 0 || !x_op_dev || (num_tasks > 0 && (!x_task_dev || !scores_dev)) ||
      !scratch_dev || ((uintptr_t)scratch_dev & 15))
    return GF_ERR_INVALID_ARG;
  if (num_tasks == 0 || g->desc.num_edges == 0) return GF_OK;
  // as many tasks per pass as the scratch allows
  const int n = g->desc.num_shared_nodes;
  int per_pass = 0;
  for (int cand = num_tasks; cand >= 1; cand = cand > 1 ? (cand + 1) / 2 : 0)
    if ((uint64_t)edge_scores_scratch_floats(n, *m, num_tasks, cand) * 4 <= scratch_bytes) { per_pass = cand; break; }
  if (per_pass == 0) return GF_ERR_CAPACITY;
  const int k = launch_edge_scores(g->score_graph, *m, x_op_dev, num_tasks, x_task_dev, scores_dev, (float*)scratch_dev,
                                   per_pass, (cudaStream_t)stream);
  if (k < 0) return GF_ERR_CUDA;
  g->launches += k;
  return GF_OK;
}

gf_status_t gf_last_status(gf_wgraph_t* g, void* stream) {
  if (!g) return GF_ERR_INVALID_ARG;
  int32_t w[3] = {0, 0, 0};  // [kStatusReport], [kStatusGiveUp], [kStatusBounds]
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess ||
      cudaMemcpy(w, g->status_dev, 12, cudaMemcpyDeviceToHost) != cudaSuccess)
    return GF_ERR_CUDA;
  if (w[0] != 0 || w[1] != 0 || w[2] != 0) cudaMemset(g->status_dev, 0, 12);
  g->last_bounds_site = w[kStatusBounds];
  if (w[kStatusGiveUp] != 0) return GF_ERR_TIMEOUT;  // results of that launch are undefined: reported first
  if (w[kStatusBounds] != 0) return GF_ERR_BOUNDS;
  if (w[kStatusReport] != 0) return (gf_status_t)w[kStatusReport];
  if (g->tables.pending) return finalize_tables(&g->tables);
  return GF_OK;
}

gf_status_t gf_profile_enable(gf_wgraph_t* g, int32_t on) {
  if (!g) return GF_ERR_INVALID_ARG;
  g->profiling = on != 0;
  return GF_OK;
}

gf_status_t gf_profile_read(gf_wgraph_t* g, gf_profile_t* out) {
  if (!g || !out) return GF_ERR_INVALID_ARG;
  drain_spans(g);
  *out = g->prof;
  g->prof = gf_profile_t{};
  return GF_OK;
}

uint64_t gf_launch_count(const gf_wgraph_t* g) { return g ? g->launches : 0; }

int32_t gf_debug_bounds_enabled(void) { return GF_BOUNDS_ON; }
int32_t gf_debug_bounds_site(const gf_wgraph_t* g) { return g ? g->last_bounds_site : 0; }

gf_status_t gf_debug_counters(gf_wgraph_t* g, gf_debug_counters_t* out, void* stream) {
  if (!g || !out) return GF_ERR_INVALID_ARG;
  static_assert(kStatusReruns == kStatusRescales + 1, "the two counters are read with one copy");
  int32_t words[2] = {0, 0};
  if (cudaStreamSynchronize((cudaStream_t)stream) != cudaSuccess ||
      cudaMemcpy(words, g->status_dev + kStatusRescales, 8, cudaMemcpyDeviceToHost) != cudaSuccess ||
      cudaMemset(g->status_dev + kStatusRescales, 0, 8) != cudaSuccess)
    return GF_ERR_CUDA;
  out->softmax_reference_moves = (uint64_t)(uint32_t)words[0];
  out->exact_reruns = (uint64_t)(uint32_t)words[1];
  return GF_OK;
}

gf_status_t gf_debug_wait_probe(gf_wgraph_t* g, int64_t limit_cycles, int32_t* gave_up, void* stream) {
  if (!g || !gave_up || limit_cycles < 1 || limit_cycles > 100000000ll) return GF_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  int32_t seen = 0;
  if (cudaMemsetAsync(g->status_dev + kStatusProbe, 0, 4, st) != cudaSuccess) return GF_ERR_CUDA;
  const int n = launch_wait_probe(g->status_dev, limit_cycles, g->status_dev + kStatusProbe, st);
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  if (cudaMemcpyAsync(&seen, g->status_dev + kStatusProbe, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess ||
      cudaStreamSynchronize(st) != cudaSuccess)
    return GF_ERR_CUDA;
  *gave_up = seen == 2 ? 1 : 0;
  return GF_OK;
}

}  // extern "C"

// ---- decode for callers that cannot allocate: partials in a library-resident device array ----
//
// The array below is part of the library image: every GPU that loads the library holds these
// bytes until the process exits.  In host code `g_static_scratch` is only a stand-in for the
// symbol, not a device address, so the address is looked up once per device with
// cudaGetSymbolAddress (with that device current) and only that pointer is given to kernels.
namespace {
constexpr size_t kStaticScratchBytes = GF_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
void* g_static_scratch_ptr[kMaxDevices] = {};
std::mutex g_static_scratch_mu;

// Device address of the array on the current device; nullptr if the lookup fails.
void* static_scratch_for_current_device() {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_static_scratch_mu);
  if (g_static_scratch_ptr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || p == nullptr) return nullptr;
    g_static_scratch_ptr[dev] = p;
  }
  return g_static_scratch_ptr[dev];
}
}  // namespace

extern "C" gf_status_t gf_path_attention_decode_static(gf_wgraph_t* g, const gf_tables_t* t,
                                                       int32_t layer, const void* q_dev,
                                                       void* out_dev, float* lse_dev, void* stream) {
  gf_status_t s = check_attention_args(g, t, layer, q_dev, out_dev, GF_MODE_DECODE);
  if (s != GF_OK) return s;
  if (t->pending && (s = finalize_tables(t)) != GF_OK) return s;
  const size_t ml_bytes = align_up((size_t)t->info.num_slots * g->shape.num_q_heads * 2 * 4, 256);
  const size_t o_bytes = (size_t)t->info.num_slots * g->shape.num_q_heads * g->shape.head_dim * 4;
  if (ml_bytes + o_bytes > kStaticScratchBytes) return GF_ERR_CAPACITY;
  char* scratch = (char*)static_scratch_for_current_device();
  if (scratch == nullptr) return GF_ERR_CUDA;
  TablesDev td = t->dev;  // same tables, partials redirected into the resident array
  td.part_ml = reinterpret_cast<float*>(scratch);
  td.part_o = reinterpret_cast<float*>(scratch + ml_bytes);
  cudaStream_t st = (cudaStream_t)stream;
  bool joined = false;
  int n = timed(g, kSpanDecode, st, [&] { return launch_decode_kernels(g, t, td, layer, q_dev, st, &joined); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  n = timed(g, kSpanMerge, st, [&] { return launch_merge(g->shape, td, out_dev, lse_dev, !joined, st); });
  if (n < 0) return GF_ERR_CUDA;
  g->launches += n;
  return GF_OK;
}
