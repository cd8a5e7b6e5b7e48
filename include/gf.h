/*
 * gf.h -- C ABI of the path-attention library (sm_100a).
 *
 * Attention for many concurrent agent requests whose KV context is a path of
 * wGraph nodes.  The wGraph is the global DAG of atomic operations (paper,
 * Sec. 3 "Overview"); every operation node owns one precomputed KV segment and
 * a workflow's KV cache is assembled from the nodes it selects (Sec. 5,
 * "Topology-Aware State Management").  A segment is stored once and shared by
 * every request whose path passes through its node; this is the base-KV term
 * of the reconstruction rule in Sec. 5.1; gf_node_kv_reconstruct applies a
 * sparse per-prefix residual to it (Eq. 7), gf_residual_encode produces that
 * residual from the two states, and gf_transition_counts /
 * gf_select_transitions are the statistics of Sec. 5.2 that decide which
 * residuals are kept.
 *
 * Conventions
 *   - Every entry point returns a gf_status_t; nothing throws or aborts.
 *   - Pointers named *_dev are device pointers, *_host are host pointers.
 *   - The library never allocates device memory: the KV pool and the workspace
 *     are caller-allocated and caller-owned, and must outlive the handle.
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     gf_node_kv_write, gf_node_kv_read, gf_node_kv_reconstruct,
 *     gf_residual_encode, gf_transition_counts, gf_select_transitions,
 *     gf_path_attention_decode and gf_path_attention_extend only enqueue work.  gf_build_path_tables enqueues its kernels and then
 *     waits on the stream once, to read back four table sizes and the
 *     validation result.
 *   - Argument errors are detected on the host before anything is launched.
 *   - One handle is used from one host thread at a time.
 *   - bf16 everywhere for K, V, Q and the output; accumulation is fp32.
 */
#ifndef GF_H_
#define GF_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gf_wgraph gf_wgraph_t; /* library-owned host object; gf_wgraph_destroy frees it */
typedef struct gf_tables gf_tables_t; /* owned by its wGraph; valid until the next build or destroy */

typedef enum {
  GF_OK = 0,
  GF_ERR_INVALID_ARG = 1,   /* null pointer, size out of range, unsupported shape            */
  GF_ERR_INVALID_GRAPH = 2, /* edge endpoint out of range, self loop, or a cycle             */
  GF_ERR_INVALID_PATH = 3,  /* a request path failed validation (see gf_tables_bad_request)  */
  GF_ERR_CAPACITY = 4,      /* KV pool or workspace too small                                 */
  GF_ERR_NOT_WRITTEN = 5,   /* the call needs a node's KV state and that node was never written */
  GF_ERR_NOT_BUILT = 6,     /* tables missing, stale, or built in the other mode              */
  GF_ERR_CUDA = 7,          /* a CUDA runtime call failed                                     */
  GF_ERR_TIMEOUT = 8,       /* a bounded device-side wait gave up (see gf_last_status)        */
  GF_ERR_BOUNDS = 9         /* debug build (GF_DEBUG_BOUNDS): a table-derived index was out of range */
} gf_status_t;

enum { GF_MODE_DECODE = 0, GF_MODE_EXTEND = 1 };
/* OR-ed into mode (decode only): enqueue the whole build and return without waiting, see below. */
#define GF_MODE_DEFERRED 0x100

/* Tokens per pool tile: every node extent starts on a tile boundary. */
#define GF_TILE_TOKENS 64

typedef struct {
  int32_t num_nodes;          /* size of the node-id space, private nodes included            */
  int32_t num_shared_nodes;   /* ids below this are wGraph operation nodes; hops between two  */
                              /* of them must be wGraph edges.  Ids at or above it are private */
                              /* (a request's own suffix, or the new segment of an extend).    */
  int32_t num_edges;
  const int32_t* edge_src_host; /* [num_edges] valid dependencies (v_i, v_j) of Sec. 3         */
  const int32_t* edge_dst_host;
  int32_t num_layers;
  int32_t num_q_heads;        /* multiple of num_kv_heads; query head h reads KV head          */
  int32_t num_kv_heads;       /*   h / (num_q_heads / num_kv_heads)                            */
  int32_t head_dim;           /* 64 or 128                                                     */
  float softmax_scale;        /* 0 selects 1/sqrt(head_dim)                                    */
  void* kv_pool_dev;          /* 1024-byte aligned                                             */
  uint64_t kv_pool_bytes;     /* holds floor(bytes / gf_pool_bytes_per_tile / layers) tiles    */
  void* workspace_dev;        /* 256-byte aligned; graph CSR, tables and attention partials    */
  uint64_t workspace_bytes;
  int32_t max_residual_nodes; /* nodes that may be kept as base + residual at one time (see     */
                              /* gf_node_kv_attach_residual); each takes 64 * num_layers bytes   */
                              /* of the workspace on top of gf_workspace_bytes.  0: none.        */
} gf_wgraph_desc_t;

/* Work-list policy (pure integer formula, applied per segment of length l shared by G requests):
 *   mult = min(max_chunk_mult, max(1, ceil(G / group_unit)));  n0 = ceil(l / (chunk_tokens*mult));
 *   chunk = 64*ceil(ceil(l / n0) / 64);  chunks = ceil(l / chunk);  tiles = ceil(G / group_tile).
 * chunk_tokens is a positive multiple of 64, group_tile is 1..16, the others are >= 1. */
typedef struct {
  int32_t chunk_tokens;
  int32_t group_tile;
  int32_t group_unit;
  int32_t max_chunk_mult;
} gf_policy_t;

/* Host copy of the tables (test and inspection hook).  Every pointer is a caller-provided host
 * array of at least the stated length, or NULL to skip that array. */
typedef struct {
  int32_t* seg_node;  /* [num_segments]  ascending node ids with a non-empty segment on a path */
  int32_t* seg_len;   /* [num_segments]                                                       */
  int32_t* seg_off;   /* [num_segments]  token offset of the node's extent in the pool        */
  int32_t* grp_ptr;   /* [num_segments+1]                                                     */
  int32_t* grp_req;   /* [num_pairs]     ascending request ids per segment                    */
  int32_t* req_len;   /* [num_requests]                                                       */
  int32_t* req_nseg;  /* [num_requests]                                                       */
  int32_t* items;     /* [num_items*6]   seg, tok_begin, tok_count, grp_begin, grp_count, part_base */
  int32_t* mrg_ptr;   /* [num_requests+1]                                                     */
  int32_t* mrg_slot;  /* [num_slots]                                                          */
  int32_t* pseg_ptr;  /* [num_requests+1]                                                     */
  int32_t* pseg;      /* [num_pairs]     segment indices in path order                        */
  int32_t* q_ptr;     /* [num_requests+1] extend mode only                                    */
  int32_t* self_seg;  /* [num_requests]   extend mode only                                    */
} gf_tables_host_t;

typedef struct {
  int32_t num_requests;
  int32_t num_segments;
  int32_t num_pairs;      /* sum over segments of group size = sum over requests of req_nseg */
  int32_t num_items;
  int32_t num_slots;
  int32_t mode;
  int64_t resident_tokens;     /* sum of seg_len                                             */
  int64_t materialised_tokens; /* sum of req_len = what per-request (stateful) caching holds */
  int64_t num_q_rows;          /* num_requests (decode) or total new tokens (extend)         */
} gf_tables_info_t;

/* Bytes of pool one 64-token tile of one KV head occupies (K block then V block). */
uint64_t gf_pool_bytes_per_tile(int32_t head_dim);

/* Lower bound on workspace_bytes for a batch (graph CSR + tables + partials), so that callers can
 * size the workspace: max_pairs bounds sum of path lengths, max_slots the partial slots. */
uint64_t gf_workspace_bytes(int32_t num_nodes, int32_t num_edges, int32_t max_requests,
                            int32_t max_pairs, int32_t max_items, int32_t max_slots,
                            int32_t num_q_heads, int32_t head_dim);

/* Sec. 3: G_op = (V_op, E_op), a DAG.  Validates the edge list (Kahn's algorithm; a cycle, a self
 * loop or an endpoint outside [0, num_shared_nodes) gives GF_ERR_INVALID_GRAPH), copies the
 * adjacency to the workspace (synchronous), and records shapes.  *out is NULL on failure. */
gf_status_t gf_wgraph_create(const gf_wgraph_desc_t* desc, gf_wgraph_t** out);
gf_status_t gf_wgraph_destroy(gf_wgraph_t* g);

/* Sec. 5: attach the precomputed KV state of one operation node (one layer of it).
 * k_dev, v_dev: [n_tokens, num_kv_heads, head_dim] bf16, caller-owned, read in stream order and
 * never modified.  The first write of a node (any layer) fixes its length and reserves its extent
 * (the same tile range in every layer), rounded up to whole tiles, first fit (see
 * gf_node_kv_release; without releases that is first-write order); later
 * writes must pass the same n_tokens (GF_ERR_INVALID_ARG otherwise).  n_tokens = 0 records an
 * empty node.  GF_ERR_CAPACITY when the pool is full.  Writing a node invalidates built tables. */
gf_status_t gf_node_kv_write(gf_wgraph_t* g, int32_t node, int32_t layer, const void* k_dev,
                             const void* v_dev, int32_t n_tokens, void* stream);

/* Reserves a node's extent without data: fixes its length, takes the tiles (same rule as the first
 * gf_node_kv_write), and lets paths name the node, so that tables can be built before its K/V exist.
 * Meant for the new segment of an extend whose K/V are appended by gf_path_attention_extend_append;
 * until something writes the extent its contents are undefined.  A node already written or
 * reserved must have this length (then nothing happens).  GF_ERR_CAPACITY when no run of free tiles
 * is long enough. */
gf_status_t gf_node_kv_reserve(gf_wgraph_t* g, int32_t node, int32_t n_tokens, void* stream);

/* Sec. 5.2: only the states of frequently taken transitions stay materialised; a workflow on any
 * other transition computes its KV on the fly, and that state need not stay either.  Returns the
 * node's tiles (all layers) to the pool and makes the node unwritten again; built tables become
 * stale.  Extents are handed out first fit: the lowest run of free tiles that is long enough, free
 * runs that touch are one run.  The release is ordered on `stream` like a write: work enqueued
 * earlier on that stream may still read the extent, and whoever is given the tiles next writes them
 * on the same stream or after synchronising with it.  GF_ERR_NOT_WRITTEN for a node without an extent. */
gf_status_t gf_node_kv_release(gf_wgraph_t* g, int32_t node, void* stream);

/* Length and pool offset (both in tokens; the offset is what seg_off reports) of a node's extent.
 * Either pointer may be NULL.  GF_ERR_NOT_WRITTEN for a node without an extent. */
gf_status_t gf_node_extent(const gf_wgraph_t* g, int32_t node, int32_t* n_tokens_host, int32_t* token_offset_host);

typedef struct {
  uint32_t capacity_tiles;   /* tiles per (layer, KV head) the pool holds                       */
  uint32_t tiles_in_use;     /* tiles of live extents                                           */
  uint32_t high_water_tiles; /* one past the highest tile in use                                */
} gf_pool_info_t;
gf_status_t gf_pool_info(const gf_wgraph_t* g, gf_pool_info_t* out_host);

/* Copies one layer of a node's KV state from the pool back to the caller layout
 * ([n_tokens, num_kv_heads, head_dim] bf16 each, caller-owned device buffers of the node's
 * length), in stream order: the state a workflow would assemble from this node (Sec. 5).
 * GF_ERR_NOT_WRITTEN for a node that was never written. */
gf_status_t gf_node_kv_read(gf_wgraph_t* g, int32_t node, int32_t layer, void* k_out_dev,
                            void* v_out_dev, void* stream);

/* A sparse residual of one tensor (K or V) of one node under one prefix, Sec. 5.1.  The logical
 * tensor is [rows, head_dim] with rows = n_tokens * num_kv_heads in the caller layout of
 * gf_node_kv_write (row = token * num_kv_heads + kv_head).  The paper fixes no storage format;
 * this one is a bitmap plus packed values: bit j of word w of a row marks entry 32 * w + j, the
 * bf16 values of the marked entries follow in (row, entry) order, row_ptr is the exclusive prefix
 * sum of the rows' counts and nnz = row_ptr[rows].  All three arrays are device memory, caller-owned,
 * read in stream order.  A value index outside [0, nnz) is not read: the entry keeps its base value
 * and gf_last_status reports GF_ERR_INVALID_ARG. */
typedef struct gf_residual {
  const uint32_t* bitmap_dev; /* [rows, head_dim / 32], 16-byte aligned */
  const void* values_dev;     /* bf16 [nnz]             */
  const int32_t* row_ptr_dev; /* int32 [rows + 1]       */
  int64_t nnz;
} gf_residual_t;

/* Sec. 5.1, Eq. 7: KV(P, v) = KV_base(v) + dKV(P, v).  Writes one layer of `node`, the state of an
 * operation under one prefix, as the base node's state plus a sparse residual: an entry the bitmap
 * marks becomes the bf16 sum of base and residual value (one rounding, nearest even), every other
 * entry is the base bit for bit.  `node` gets an extent of its own like in gf_node_kv_write (length
 * = the base node's; a node already written must have that length), so paths can name it like any
 * node; ids at or above num_shared_nodes are not edge-checked, which is where prefix-conditioned
 * variants of an operation belong.  k_res or v_res NULL: that tensor is copied unchanged.
 * GF_ERR_NOT_WRITTEN when base_node was never written; GF_ERR_INVALID_ARG when node == base_node or
 * lengths differ. */
gf_status_t gf_node_kv_reconstruct(gf_wgraph_t* g, int32_t node, int32_t layer, int32_t base_node,
                                   const gf_residual_t* k_res, const gf_residual_t* v_res,
                                   void* stream);

/* Sec. 5.1, Eq. 7 applied inside the segment stream.  Declares layer `layer` of `node` to be the state
 * of base_node plus a sparse residual WITHOUT materialising it: the node gets no tiles of its own (its
 * length is the base node's, the pool holds the base once, the residual, about a third of the dense
 * size at the densities the section reports, stays in the caller's memory, which must stay valid and
 * unchanged while the node exists).  Decode over a path that names the node streams the base node's
 * tiles and completes them in shared memory before they are used: every marked entry becomes the bf16
 * sum rounded once, exactly the bits gf_node_kv_reconstruct would have stored, so the two give
 * identical results.  Requests with the same prefix name the same node and share the segment as
 * usual; variants of one base with neighbouring ids are worked on close together, so the base's tiles
 * tend to come from L2 for all but the first.  Call once per layer.  k_res / v_res NULL: that tensor
 * is the base's.  gf_node_kv_release(node) detaches it (a base cannot be released while such nodes
 * exist: GF_ERR_INVALID_ARG).  Limits: up to max_residual_nodes at a time (GF_ERR_CAPACITY); the base
 * must own its tiles; extend mode does not take paths through such nodes (GF_ERR_INVALID_PATH:
 * materialise the state with gf_node_kv_reconstruct for that); gf_node_kv_read / write do not apply. */
gf_status_t gf_node_kv_attach_residual(gf_wgraph_t* g, int32_t node, int32_t layer, int32_t base_node,
                                       const gf_residual_t* k_res, const gf_residual_t* v_res, void* stream);

/* Room for one tensor's residual, caller-owned device memory: bitmap_dev uint32 [rows, head_dim / 32]
 * (16-byte aligned), row_ptr_dev int32 [rows + 1], values_dev bf16 [capacity], and nnz_dev, one int64
 * that receives the number of values (8-byte aligned).  rows = n_tokens * num_kv_heads of the node. */
typedef struct gf_residual_buf {
  uint32_t* bitmap_dev;
  void* values_dev;
  int32_t* row_ptr_dev;
  int64_t capacity;
  int64_t* nnz_dev;
} gf_residual_buf_t;

/* Sec. 5.1, the other direction of Eq. 7: dKV(P, v) = KV(P, v) - KV_base(v), stored sparsely.  Given
 * one layer of the state of operation `base_node` computed under a prefix (k_full_dev, v_full_dev:
 * [n_tokens, num_kv_heads, head_dim] bf16 like in gf_node_kv_write, n_tokens = the node's length,
 * 16-byte aligned), writes for each tensor the residual against the node's stored base state in the
 * format gf_node_kv_reconstruct reads: the difference of every entry is rounded once to bf16, and it
 * is stored when the magnitude of that rounded value exceeds `threshold` (the section drops the
 * entries below a small threshold and names no value; 0 keeps every non-zero difference).  k_out or
 * v_out NULL skips that tensor.  When a tensor needs more than `capacity` values, the values beyond it
 * are not written, *nnz_dev still holds the number needed and gf_last_status reports
 * GF_ERR_CAPACITY.  GF_ERR_NOT_WRITTEN when base_node was never written.  Set-up work (three short
 * kernels per call); enqueued on `stream`. */
gf_status_t gf_residual_encode(gf_wgraph_t* g, int32_t base_node, int32_t layer, const void* k_full_dev,
                               const void* v_full_dev, float threshold, const gf_residual_buf_t* k_out,
                               const gf_residual_buf_t* v_out, void* stream);

/* Sec. 5.2 (effective path pruning), the statistics: how often every wGraph transition was taken by
 * a set of executed workflows.  Paths are given like in gf_build_path_tables (path_ptr_dev int32
 * [num_requests+1], path_node_dev int32 [num_path_nodes]).  counts_dev: int32 [num_edges], written in
 * ascending (source, destination) order of the edges given to gf_wgraph_create: entry e is the number
 * of hops u -> v over all paths with (u, v) the e-th edge in that order.  Hops that touch a node at or
 * above num_shared_nodes are not wGraph transitions and are skipped; a hop between two operation
 * nodes that is not an edge is counted in *misses_dev (uint64, device) and nowhere else.  Both outputs
 * are overwritten.  Enqueued on `stream`; nothing is waited for. */
gf_status_t gf_transition_counts(gf_wgraph_t* g, int32_t num_requests, int32_t num_path_nodes,
                                 const int32_t* path_ptr_dev, const int32_t* path_node_dev,
                                 int32_t* counts_dev, uint64_t* misses_dev, void* stream);

/* Sec. 5.2, the choice: the transitions whose residual KV states are kept are those taken at least
 * min_count times (the paper names no threshold; min_count is the caller's policy).  keep_dev: uint8
 * [num_edges], 1 = keep, in the order of counts_dev.  totals_dev: uint64 [3] = kept edges, traversals
 * on kept edges, traversals in total (what share of the executed hops finds its residual stored).
 * A workflow that takes any other transition falls back to computing that node's KV on the fly
 * (gf_path_attention_extend). */
gf_status_t gf_select_transitions(gf_wgraph_t* g, const int32_t* counts_dev, int32_t min_count,
                                  uint8_t* keep_dev, uint64_t* totals_dev, void* stream);

/* Sec. 3 (a workflow is a path over the wGraph's operation nodes, its edges the valid dependencies)
 * and Sec. 5 (a workflow's KV cache is assembled from the states of the nodes it selects): turns the
 * batch's node paths into deduplicated segment lists, request groups, the work list
 * and the merge map (tables T1..T7 of gf_tables_host_t), bit-exact integer work on the device.
 * A path may name a node that was never written: it is treated like an empty node (no segment, no
 * tokens; in extend mode an unwritten last node makes the path invalid).
 * path_ptr_dev: int32 [num_requests+1], path_node_dev: int32 [num_path_nodes] with
 * num_path_nodes = path_ptr[num_requests] (the caller knows it; passing it avoids a read-back).
 * mode GF_MODE_EXTEND: the last node of every path is the request's new segment (causal).
 * policy NULL selects {256, 16, 2, 16}.  Waits on `stream` once.  On an invalid path returns
 * GF_ERR_INVALID_PATH and *out still reports the offending request via gf_tables_bad_request;
 * GF_ERR_CAPACITY when tables + partials do not fit the workspace.
 * mode GF_MODE_DECODE | GF_MODE_DEFERRED: nothing is waited for.  The call returns GF_OK once the
 * kernels are enqueued, and gf_path_attention_decode may follow at once on the same stream (its
 * kernels read the table sizes on the device and leave `out` untouched if a path was invalid or the
 * workspace too small).  The outcome is reported by the first of gf_last_status, gf_tables_info,
 * gf_tables_bad_request or gf_tables_export, each of which then waits on the build's stream. */
gf_status_t gf_build_path_tables(gf_wgraph_t* g, int32_t num_requests, int32_t num_path_nodes,
                                 const int32_t* path_ptr_dev, const int32_t* path_node_dev,
                                 int32_t mode, const gf_policy_t* policy, gf_tables_t** out,
                                 void* stream);
gf_status_t gf_tables_info(const gf_tables_t* t, gf_tables_info_t* info_host);
int32_t gf_tables_bad_request(const gf_tables_t* t); /* -1 if all paths were valid */
gf_status_t gf_tables_export(const gf_tables_t* t, gf_tables_host_t* out_host); /* synchronous */

/* Sec. 5 (topology-aware state management: the states of a workflow's nodes, each stored once, are
 * what its next token attends over; Sec. 5.1's per-node base term).  One decode step of one layer:
 * request r's single query token attends over the concatenation of
 * the KV segments on its path (softmax(scale * q K^T) V, grouped-query head mapping).  Each
 * (segment chunk, group tile) item streams its K/V tiles once for the requests that share them
 * and writes per-request partial (o, m, l); a log-sum-exp merge then forms out.
 * q_dev/out_dev: [num_requests, num_q_heads, head_dim] bf16; lse_dev: optional fp32
 * [num_requests, num_q_heads] natural-log sum of exp of the scaled scores.  Asynchronous. */
gf_status_t gf_path_attention_decode(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                     const void* q_dev, void* out_dev, float* lse_dev,
                                     void* stream);

/* Decode for callers that must not allocate.  (The paper has no counterpart; this is a packaging
 * variant of gf_path_attention_decode.)  Some hosts of this library cannot provide scratch for the
 * attention partials: a serving loop whose device memory was carved up completely at start-up, a
 * plug-in that is handed only its input and output buffers, or code running where the CUDA
 * allocator must not be entered because it may synchronise the device or fail under a full pool.
 * For them the per-(slot, head) partials live in an array that is part of the library image,
 * GF_STATIC_SCRATCH_BYTES large, which every GPU that loads the library holds until the process
 * exits.  Same arguments, results and kernels as gf_path_attention_decode; the tables are still
 * the ones gf_build_path_tables left in the caller's workspace.
 *   - GF_ERR_CAPACITY when the partials do not fit: num_slots * num_q_heads * 2 * 4 bytes rounded up to
 *     a multiple of 256, plus num_slots * num_q_heads * head_dim * 4 bytes (the slot count is in
 *     gf_tables_info), must not exceed GF_STATIC_SCRATCH_BYTES; nothing is launched.
 *   - The workspace given to gf_wgraph_create is sized as for gf_path_attention_decode
 *     (gf_workspace_bytes, partials included): gf_build_path_tables lays out the same tables either
 *     way, this entry point only does not use the partials' part of it.
 *   - Calls no cudaMalloc / cudaFree or other allocating routine.  The first call on each device
 *     looks up the array's device address (cudaGetSymbolAddress, with the caller's current device,
 *     which must be the one that owns the pool); make that first call outside any stream capture.
 *   - The array is shared by every handle and every call on that GPU and keeps the previous call's
 *     contents.  Nothing in it has to start at zero: each launch overwrites every partial it later
 *     reads.  Two calls whose kernels overlap on the GPU (different streams, no ordering) race on
 *     it; order them. */
#define GF_STATIC_SCRATCH_BYTES (32u << 20)
gf_status_t gf_path_attention_decode_static(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                            const void* q_dev, void* out_dev, float* lse_dev,
                                            void* stream);

/* Extend / prefill of one layer (the on-the-fly path of Sec. 5.2 once the new segment's K/V are
 * in the pool): query token i of request r's new node attends over every token of the earlier
 * nodes on the path and tokens 0..i of the new node.  q_dev/out_dev: [num_q_rows, num_q_heads,
 * head_dim] bf16, request-major (request r owns rows q_ptr[r]..q_ptr[r+1]).  Asynchronous.
 * Two kernels are enqueued: the attention kernel, whose running softmax measures a stage's scores
 * against the maximum of the stages before it, and a second one that leaves at once unless the first
 * met a score more than 2^64 above that reference; in that case it computes the whole call again with
 * every stage's own maximum taken first and overwrites out_dev / lse_dev.  Any finite bf16 input is
 * therefore accepted; the same holds for the decode entry points' kernel over widely shared chunks. */
gf_status_t gf_path_attention_extend(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                     const void* q_dev, void* out_dev, float* lse_dev,
                                     void* stream);

/* Sec. 5.2, the on-the-fly branch end to end: a workflow on a transition whose state is not kept
 * computes the new node's K/V itself and appends them while it attends.  Same as
 * gf_path_attention_extend, except that the new segments' K/V do not have to be in the pool: they
 * arrive as k_new_dev / v_new_dev, [num_q_rows, num_kv_heads, head_dim] bf16 in the row order of
 * q_dev (request r's new tokens are rows q_ptr[r]..q_ptr[r+1]), and the same launch writes layer
 * `layer` of every request's new node (the last node of its path, reserved with gf_node_kv_reserve or
 * written before) while the queries attend over the prefix; the new segment is streamed once its
 * tiles are in the pool.  Afterwards the nodes hold those K/V like after gf_node_kv_write.  Two
 * requests must not name the same new node.  Inputs are read in stream order, never modified. */
gf_status_t gf_path_attention_extend_append(gf_wgraph_t* g, const gf_tables_t* t, int32_t layer,
                                            const void* q_dev, const void* k_new_dev, const void* v_new_dev,
                                            void* out_dev, float* lse_dev, void* stream);

/* Sec. 4.2 and the appendix "Network Architecture Details": the workflow construction model's
 * parameters, all fp32 device arrays, row-major, caller-owned.  The encoder is two graph-convolution
 * layers without bias (d_in -> d_hidden -> d_hidden, ReLU after each); the edge scorer is
 * Linear(3 d_hidden -> d_mlp) - ReLU - Linear(d_mlp -> d_mlp) - ReLU - Linear(d_mlp -> 1) - sigmoid.
 * The paper's sizes are d_in 384, d_hidden 256, d_mlp 128.  d_mlp is a multiple of 32, at most 128. */
typedef struct {
  int32_t d_in, d_hidden, d_mlp;
  const float* w_gcn1_dev; /* [d_in, d_hidden]                                                     */
  const float* w_gcn2_dev; /* [d_hidden, d_hidden]                                                 */
  const float* w_mlp1_dev; /* [3 * d_hidden, d_mlp]: rows for h_i, then h_j, then h_task           */
  const float* b_mlp1_dev; /* [d_mlp]                                                              */
  const float* w_mlp2_dev; /* [d_mlp, d_mlp]                                                       */
  const float* b_mlp2_dev; /* [d_mlp]                                                              */
  const float* w_mlp3_dev; /* [d_mlp]                                                              */
  float b_mlp3;
} gf_scorer_t;

/* Sec. 4.1, 4.2 (Eq. 5 and 6): task-aware compatibility scores of every wGraph edge for a batch of
 * tasks.  The wGraph given to gf_wgraph_create is extended by a virtual task node joined to every
 * operation node in both directions; every node i is encoded by two layers of
 * h_i' = ReLU(sum over j in N(i) and i of h_j W / sqrt(deg(i) deg(j))) (operation edges count in both
 * directions, deg counts the node itself), and edge (v_i, v_j) gets
 * s = sigmoid(MLP([h_i, h_j, h_task])).  x_op_dev: fp32 [num_shared_nodes, d_in] operation features;
 * x_task_dev: fp32 [num_tasks, d_in]; scores_dev: fp32 [num_tasks, num_edges], edges in ascending
 * (source, destination) order like gf_transition_counts.  scratch_dev: caller-owned, 16-byte aligned,
 * at least gf_edge_scores_scratch_bytes(g, model, num_tasks, 1) bytes; more lets more tasks be worked
 * on per pass (..., num_tasks, num_tasks) holds them all).  Enqueued on `stream`, nothing is waited for. */
uint64_t gf_edge_scores_scratch_bytes(const gf_wgraph_t* g, const gf_scorer_t* model, int32_t num_tasks,
                                      int32_t tasks_per_pass);
gf_status_t gf_edge_scores(gf_wgraph_t* g, const gf_scorer_t* model, const float* x_op_dev, int32_t num_tasks,
                           const float* x_task_dev, float* scores_dev, void* scratch_dev, uint64_t scratch_bytes,
                           void* stream);

/* Synchronises `stream` and returns what the kernels reported since the last call, then clears it:
 * GF_ERR_TIMEOUT if a bounded wait inside a kernel gave up (results of that launch are undefined;
 * reported before anything else), else the sticky report of a set-up kernel (GF_ERR_CAPACITY from
 * gf_residual_encode, GF_ERR_INVALID_ARG from gf_node_kv_reconstruct), else GF_OK.  Such a report
 * does not disturb attention calls enqueued before it is read.  After a deferred build the call also
 * completes that build and returns its outcome. */
gf_status_t gf_last_status(gf_wgraph_t* g, void* stream);

/* Optional per-kernel timing.  While enabled, every attention / table call brackets each kernel
 * it enqueues with CUDA events on the caller's stream (events are host objects; no device memory
 * is allocated).  gf_profile_read synchronises those events, adds their elapsed times into the
 * totals below, returns the totals accumulated since the last read and resets them. */
typedef struct {
  double tables_ms, decode_ms, merge_ms, extend_ms;
  uint64_t tables_launches, decode_launches, merge_launches, extend_launches;
} gf_profile_t;
gf_status_t gf_profile_enable(gf_wgraph_t* g, int32_t on);
gf_status_t gf_profile_read(gf_wgraph_t* g, gf_profile_t* out_host);

/* Number of kernels this library has launched on behalf of handle g since creation. */
uint64_t gf_launch_count(const gf_wgraph_t* g);

/* Diagnostics, for tests.  softmax_reference_moves: how many times, since the last read, a query tile
 * of the tensor-memory kernels (extend, and decode over widely shared chunks) moved the reference of
 * its running softmax after its first stage, i.e. rescaled its accumulated output because a later
 * stage's scores outgrew the running maximum by more than 2^8.  exact_reruns: how many times one of
 * their CTAs walked its piece of work a second time.  (The first walk forms the probabilities of a
 * stage against the maximum of the stages before it, which is exact as long as no score stands more
 * than 2^64 above that reference; when one does, the CTA discards the walk and repeats it with the
 * stage's own maximum taken first.)  Synchronises `stream`, then resets both. */
typedef struct {
  uint64_t softmax_reference_moves;
  uint64_t exact_reruns;
} gf_debug_counters_t;
gf_status_t gf_debug_counters(gf_wgraph_t* g, gf_debug_counters_t* out_host, void* stream);

/* Runs the library's bounded device wait once on a barrier that nothing ever completes, with a limit
 * of limit_cycles clock cycles (1 .. 10^8), and waits for the kernel: *gave_up_host becomes 1 when the
 * wait returned by giving up.  The next gf_last_status then reports GF_ERR_TIMEOUT (and clears it),
 * exactly as it would after a wait inside an attention kernel ran out.  The kernel is one warp and
 * ends by itself; nothing else on the GPU is involved. */
gf_status_t gf_debug_wait_probe(gf_wgraph_t* g, int64_t limit_cycles, int32_t* gave_up_host, void* stream);

/* The debug build (compiled with -DGF_DEBUG_BOUNDS) checks every index its kernels derive from the
 * tables against the size of what it indexes; a failed check is recorded instead of performed and
 * gf_last_status returns GF_ERR_BOUNDS.  gf_debug_bounds_enabled: 1 in that build, 0 otherwise.
 * gf_debug_bounds_site: the code of the check behind the last GF_ERR_BOUNDS that gf_last_status
 * returned (1xx decode kernel and merge, 2xx tensor-memory kernels, 3xx table builder, 4xx pool). */
int32_t gf_debug_bounds_enabled(void);
int32_t gf_debug_bounds_site(const gf_wgraph_t* g);

const char* gf_status_string(gf_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* GF_H_ */
