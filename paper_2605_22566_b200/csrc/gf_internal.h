// Internal declarations shared by the translation units of the path-attention library.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gf.h"

namespace gf {

constexpr int kTile = GF_TILE_TOKENS;  // tokens per pool tile
constexpr int kMaxDevices = 64;        // device ordinals for which per-device set-up is remembered

// The handle's status block: 16 int32 at the head of the workspace, all zero between launches.
enum StatusWord {
  kStatusReport = 0,       // sticky argument / capacity report of a set-up kernel (a gf_status_t)
  kStatusGiveUp = 1,       // non-zero: a bounded device wait gave up (GF_ERR_TIMEOUT)
  kStatusBounds = 2,       // debug build only: the largest site code of a range check that failed (GF_ERR_BOUNDS)
  kStatusDecodeQueue = 4,  // [0] next unit of the warp decode kernel, [1] its CTAs that finished
  kStatusWideQueue = 8,    // the same pair for the tensor-memory decode kernel
  kStatusProbe = 3,        // what the wait probe's waiter saw (gf_debug_wait_probe)
  kStatusRescales = 12,    // diagnostic: times a tensor-memory tile moved its softmax reference after its first stage
  kStatusReruns = 13,      // diagnostic: times the exact tensor-memory kernel redid the work of the launch before it
  kStatusOverflow = 14,    // raised by a tensor-memory kernel that met a score too far above its lagging maximum
  kStatusExactDone = 15,   // CTAs of the exact kernel that finished (the last one lowers the flag)
  kStatusWords = 16
};

// One work item: a chunk of one shared segment for one tile of the requests that share it.
struct __align__(32) Item {
  int32_t seg, tok_begin, tok_count, grp_begin, grp_count, part_base;
  int32_t tile0;  // pool tile index of the chunk's first token
  int32_t pad;    // bit 0: chunk of a widely shared segment, handled by the tensor-memory decode kernel;
                  // bits 8..: 1 + row of the residual table if the segment's state is base + residual
};

// Small block the table builder leaves for the host to read back.
struct Header {
  int32_t bad_req;    // INT_MAX while no bad request has been found
  int32_t num_segments;
  int32_t num_pairs;
  int32_t num_items;
  int32_t num_slots;
  int32_t mrg_total;  // must equal num_slots
  int32_t num_wide;   // items flagged wide
  int32_t max_q_rows;  // extend mode: most query rows of one request
  int32_t wide_units;  // units per KV head the wide decode kernel would get (whether or not it is enabled)
  int32_t wide_list_n; // heads of wide units listed for the wide kernel
  int32_t wide_work;   // work of the wide kernel per KV head, in (128-token stage x 128-row tile) units
  int32_t wide_tokens; // tokens of the segments the wide kernel handles (the warp kernel streams the rest)
  int32_t wide_tile_units;  // (chunk x 128-row tile) pairs of the wide kernel per KV head: each loads queries and writes partials
  int32_t stream_steps;     // work of the warp kernel per KV head, in (64-token tile x 16-row group) steps
  unsigned long long resident_tokens;
  unsigned long long materialised_tokens;
  unsigned long long num_q_rows;
};

// Device views (all int32 unless noted).  Filled by the host when it carves the workspace.
struct GraphDev {
  const int32_t* adj_ptr;  // [num_shared_nodes+1] CSR of E_op by source
  const int32_t* adj_dst;  // [num_edges] ascending within a row
  int32_t* node_len;       // [num_nodes] tokens; -1 = never written
  int32_t* node_off;       // [num_nodes] pool token offset (tile aligned)
  int32_t* node_res;       // [num_nodes] row of the residual table of a node whose state is base + residual; -1: none
  int32_t num_nodes, num_shared_nodes;
};

// One (variant node, layer) of the residual table: the sparse residual (Sec. 5.1) that turns the base
// node's tiles into this node's state while they sit in shared memory.  Pointers are the caller's.
struct __align__(16) ResidualEntry {
  const uint32_t* k_bitmap;
  const uint16_t* k_values;
  const int32_t* k_row_ptr;
  const uint32_t* v_bitmap;
  const uint16_t* v_values;
  const int32_t* v_row_ptr;
  int32_t k_nnz, v_nnz;  // -1: that tensor has no residual
};

struct TablesDev {
  Header* hdr;
  int32_t* node_seg;   // [num_nodes] flag, then segment index or -1
  int32_t* seg_node;   // [seg_cap]
  int32_t* seg_len;
  int32_t* seg_off;
  int32_t* grp_ptr;    // [seg_cap+1]
  int32_t* grp_fill;   // [seg_cap] counters
  int32_t* grp_tmp;    // [pairs]
  int32_t* grp_req;    // [pairs]
  int32_t* seg_chunk;  // [seg_cap] chunk length in tokens
  int32_t* seg_nchunk; // [seg_cap]
  int32_t* seg_item_base;  // [seg_cap+1]
  int32_t* seg_part_base;  // [seg_cap+1]
  int32_t* req_len;    // [R]
  int32_t* req_nseg;   // [R]
  int32_t* req_nslot;  // [R]
  int32_t* req_qrows;  // [R]
  int32_t* pseg_ptr;   // [R+1]
  int32_t* pseg;       // [pairs]
  int32_t* mrg_ptr;    // [R+1]
  int32_t* q_ptr;      // [R+1]
  int32_t* self_seg;   // [R]
  int32_t* req_order;  // [R] extend mode: requests by descending context length (longest work first)
  int32_t* ext_written; // [R] extend with append: tiles of every request's new node written so far
  Item* items;         // [num_items]   (carved after the read-back)
  int32_t* mrg_slot;   // [num_slots]   (carved after the read-back)
  int32_t* wide_list;  // [wide_list_n] item index of the first item of every wide unit, any order
  float* part_o;       // [num_slots, Hq, D] fp32 un-normalised partial outputs
  float* part_ml;      // [num_slots, Hq, 2] running max (log2 units) and sum
  const int32_t* node_res;  // [num_nodes] the graph's residual rows (see GraphDev)
  int32_t* status;     // the handle's status block (range checks of the debug build report there)
  int32_t seg_cap, num_requests, num_pairs_in, mode;
  int32_t slot_cap;    // items and partial slots the workspace has room for
  int32_t wide_min_group;  // segments shared by at least this many requests are flagged wide (0: none)
  int32_t wide_probe_group;  // group size counted as wide for the hint, even when wide_min_group is 0
  int32_t wide_min_units;  // ... provided the batch has at least this many wide units per KV head
  int32_t num_sms;         // multiprocessors of the device the handle lives on (grid sizing)
  int32_t wide_unit_req;   // requests per unit of the wide kernel: 256 stacked query rows / GQA group size
};

// True when the tables on the device are usable: every path valid and the items / partial slots fit
// the room the host carved for them.  Kernels that consume the tables do nothing otherwise.
__host__ __device__ inline bool tables_usable(const Header& h, int slot_cap) {
  return h.bad_req == 0x7fffffff && h.num_items <= slot_cap && h.num_slots <= slot_cap;
}

struct PoolGeom {
  char* base;
  uint64_t layer_stride;  // bytes between layers
  uint64_t head_stride;   // bytes between KV heads of one layer
  uint32_t tile_bytes;    // K block + V block of one 64-token tile of one head
  uint32_t cap_tiles;     // tiles per (layer, head)
};

struct AttnShape {
  int32_t num_q_heads, num_kv_heads, head_dim;
  float scale_log2;  // softmax scale * log2(e)
};

// The task-conditioned graph of the workflow construction model (Sec. 4.1) as the scoring kernels read
// it: symmetric neighbourhoods of the operation nodes (operation edges in both directions, without
// duplicates), 1 / sqrt(deg) of every node (the task node last; deg counts the node itself and, for an
// operation, the task node), and the wGraph's edges in the order of the scores.  Built by the host.
struct ScoreGraphDev {
  const int32_t* sym_ptr;   // [num_ops + 1]
  const int32_t* sym_idx;   // [sym_ptr[num_ops]]
  const float* inv_sqrt;    // [num_ops + 1]
  const int32_t* edge_src;  // [num_edges] ascending (source, destination), like gf_transition_counts
  const int32_t* edge_dst;  // [num_edges]
  int32_t num_ops, num_edges;
};

// ---- range checks of the debug build --------------------------------------------------------------
// Compiled with -DGF_DEBUG_BOUNDS, every index that a kernel derives from the tables (or from a table
// that a previous kernel wrote) is checked against the size of what it indexes before it is used.  A
// failed check never traps: it records its site code in the status block (gf_last_status then says
// GF_ERR_BOUNDS) and the access is skipped, or made at index 0 where something must be loaded for the
// control flow to go on.  In the normal build GF_CHECK is the constant true and its condition is not
// evaluated.
#ifdef GF_DEBUG_BOUNDS
#define GF_BOUNDS_ON 1
#else
#define GF_BOUNDS_ON 0
#endif
#ifdef __CUDACC__
__device__ __forceinline__ bool bounds_report(bool ok, int32_t* status, int site) {
  if (!ok) atomicMax(status + kStatusBounds, site);
  return ok;
}
#define GF_CHECK(ok, status, site) (GF_BOUNDS_ON ? ::gf::bounds_report((ok), (status), (site)) : true)
// the index if it is inside [0, n), else 0 (and the failure is recorded)
#define GF_CLAMP(i, n, status, site) (GF_CHECK((i) >= 0 && (long long)(i) < (long long)(n), (status), (site)) ? (i) : 0)
#endif

// ---- chained launches ----------------------------------------------------------------------------
// The kernels of a step depend on each other in stream order.  Launched with programmatic stream
// serialization, a kernel may be scheduled while its predecessor is still running; it first lets its
// own successor be scheduled, then waits until the predecessor has completed and its writes are
// visible, before it touches global memory.  What is saved is the launch and drain gap at every
// boundary of the chain (a decode step on config 1 is nine short kernels).
#ifdef __CUDACC__
__device__ __forceinline__ void chain_enter() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  asm volatile("griddepcontrol.wait;" ::: "memory");
}
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                  Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

// Opt-in to more than 48 KB of dynamic shared memory is a per-device attribute of a kernel: remembered
// per device ordinal, so that a process driving several GPUs sets it on each of them.
template <typename K>
inline bool ensure_dynamic_smem(K kernel, size_t bytes, bool (&done)[kMaxDevices]) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return false;
  const bool cacheable = dev >= 0 && dev < kMaxDevices;
  if (cacheable && done[dev]) return true;
  if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes) != cudaSuccess) return false;
  if (cacheable) done[dev] = true;
  return true;
}

// ---- launchers (each returns the number of kernels it enqueued, or -1 on a launch error) ----
int launch_graph_set_node(const GraphDev& g, int node, int len, int off, cudaStream_t st);
// set != nullptr: the kernel also records the node's length and pool offset on the device (first write).
int launch_kv_write(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0,
                    const void* k, const void* v, int n_tokens, const GraphDev* set, int node, int32_t* status,
                    cudaStream_t st);
int launch_kv_read(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0, void* k,
                   void* v, int n_tokens, cudaStream_t st);
int launch_kv_reconstruct(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0_dst,
                          int tile0_base, const gf_residual_t* rk, const gf_residual_t* rv, int n_tokens,
                          int32_t* status, cudaStream_t st);
int launch_residual_encode(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0,
                           const void* k_full, const void* v_full, int n_tokens, float threshold,
                           const gf_residual_buf_t* k_out, const gf_residual_buf_t* v_out, int32_t* status,
                           cudaStream_t st);
int launch_transition_counts(const GraphDev& g, int num_edges, int num_requests, int num_path_nodes,
                             const int32_t* path_ptr, const int32_t* path_node, int32_t* counts,
                             unsigned long long* misses, cudaStream_t st);
int launch_select_transitions(const int32_t* counts, int num_edges, int min_count, uint8_t* keep,
                              unsigned long long* totals, cudaStream_t st);
int launch_tables_phase_a(const GraphDev& g, const TablesDev& t, const int32_t* path_ptr,
                          const int32_t* path_node, gf_policy_t pol, cudaStream_t st);
// num_items < 0: not known on the host (deferred build); the kernels read the counts on the device.
int launch_tables_phase_b(const TablesDev& t, const int32_t* path_ptr, const int32_t* path_node, gf_policy_t pol,
                          int num_items, cudaStream_t st);
// yield_sms > 0: CTAs that find themselves on a multiprocessor with an id below it leave at once, so
// that the tensor-memory decode kernel, enqueued on another stream, can have those multiprocessors.
// residuals: the residual table rows of `layer` ([row] of ResidualEntry), or null when no node has one.
int launch_decode(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int num_items,
                  int layer, const void* q, int32_t* status, int yield_sms, const ResidualEntry* residuals,
                  cudaStream_t st);
int launch_set_residual(ResidualEntry* slot, const ResidualEntry& value, int32_t* node_res, int node, int row,
                        cudaStream_t st);
int launch_merge(const AttnShape& sh, const TablesDev& t, void* out, float* lse, bool chained, cudaStream_t st);
// Two launches: the kernel and, behind it, its exact variant, which leaves at once unless the first
// met scores beyond what its lagging softmax reference may keep.  num_ctas / exact_ctas <= 0: one per
// multiprocessor.  chained: launched with programmatic stream serialization (only when its
// predecessor in `st` is the kernel it depends on).
int launch_decode_wide(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int num_items, int layer,
                       const void* q, int32_t* status, int num_ctas, int exact_ctas, bool chained, cudaStream_t st);
size_t edge_scores_scratch_floats(int num_ops, const gf_scorer_t& m, int num_queries, int per_pass);
int launch_edge_scores(const ScoreGraphDev& g, const gf_scorer_t& m, const float* x_op, int num_queries,
                       const float* x_task, float* scores, float* scratch, int per_pass, cudaStream_t st);
int launch_wait_probe(int32_t* status, long long limit, int32_t* returned, cudaStream_t st);
// k_new / v_new non-null: the new segments' K/V (caller layout, request-major rows) are written to their
// pool extents by the same launch (extend with append).
int launch_extend_tc(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int layer,
                     int max_q_rows, long long num_q_rows, const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                     int32_t* status, cudaStream_t st);

}  // namespace gf
