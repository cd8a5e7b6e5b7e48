// K3 on the 5th-generation tensor cores: extend / prefill over a path of shared segments.
//
// Request r appends a new node whose tokens are the queries; token i attends over every token of
// the earlier nodes on the path and tokens 0..i of the new node (the on-the-fly branch of
// Sec. 5.2, once the new segment's K/V are in the pool).  The stacked queries (token x GQA head)
// of a request against a shared segment's K and V are two dense contractions, S = Q K^T and
// O += P V, and run as tcgen05 MMAs with accumulators in tensor memory:
//
//   CTA           two 128-row query tiles (A, B) = 2 * 128/g consecutive new tokens x the g query
//                 heads of one KV head; it walks the request's segment list in path order, 128 tokens
//                 per stage, and keeps (O, m, l) for the whole walk, so no partials are written.
//   warp 16       producer: bulk copies (TMA engine, no tensor map needed: the pool is already in
//                 the 128-byte-swizzled operand layout) of K and V stages into two rings.
//   warp 17       one thread issues every MMA.  Per stage j and tile t:  O_t += P_t(j-1) V(j-1)
//                 (A operand = P in tensor memory, B = V MN-major), then S_t(j) = Q_t K(j)^T (both
//                 K-major), so the tensor pipe works on one tile while the other tile's softmax runs.
//   warps 0-7     softmax of tile A, two threads per query row (64 score columns each): scores from
//   warps 8-15    tensor memory, kept in registers.  First the maximum of the thread's visible
//                 scores; the two threads of a row exchange it through shared memory (a barrier of
//                 their two warps only), so every stage knows its exact row maximum before anything
//                 is exponentiated.  The row's reference m moves only when the stage outgrew it by
//                 more than 2^8 (any reference is exact as long as P, l and O share it, and P never
//                 exceeds 2^8), in which case l and the row of O in tensor memory are rescaled.
//                 Then P = 2^(s - m) goes over S as bf16 pairs, l sums the unrounded values.
//
// Tensor memory (512 columns): S_A 0..127, S_B 128..255 (P of tokens 0..63 over S columns 0..31, P of
// tokens 64..127 over S columns 64..95: each softmax thread overwrites only scores it has read itself),
// O_A 256.., O_B 256+D...  Every wait is bounded (see mbar_wait).
#include "gf_internal.h"
#include "tc_device.cuh"

namespace gf {
namespace {

constexpr int kStageTokens = 128;
constexpr int kKStages = 2;
constexpr int kVStages = 2;
constexpr int kTcThreads = 640;   // warps 0-15: softmax (2 tiles x 8), 16: producer, 17: MMA issuer, 18-19: no role
constexpr int kServiceRegs = 56;  // registers per thread the last warpgroup keeps (setmaxnreg)
constexpr int kSoftmaxRegs = 104; // and what the softmax warpgroups grow to: 128 * (4 * 104 + 56) <= 640 * 96
constexpr float kRescaleThreshold = 8.f;  // log2 units: the exact walk keeps P below 2^8
constexpr float kOverflowMargin = 64.f;   // log2 units above its lagging reference at which the lagging walk gives up
constexpr int kMaxMeta = 48;              // path segments whose geometry is kept in shared memory

struct ExtendTcParams {
  const char* pool_layer;
  uint64_t head_stride;
  uint32_t tile_bytes;
  const int32_t* seg_off;
  const int32_t* seg_len;
  const int32_t* pseg_ptr;
  const int32_t* pseg;
  const int32_t* q_ptr;
  const int32_t* req_order;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int32_t num_requests, num_q_heads, gqa;
  float scale_log2;
  // decode mode: the widely shared chunks of the work list (items flagged by the table builder)
  const Item* items;
  const int32_t* grp_ptr;
  const int32_t* grp_req;
  float* part_o;
  float* part_ml;
  const Header* hdr;
  const int32_t* wide_list;
  int32_t* counters;  // [0] next (unit, head), [1] CTAs finished; zero between launches
  int32_t num_kv_heads;
  int32_t slot_cap;
  // extend with append: the new segments' K/V arrive in the caller layout and are written to the pool
  // by the first CTAs of this launch (see k_path_tc)
  const __nv_bfloat16* k_new;  // [num_q_rows, Hkv, D], request-major; null: plain extend
  const __nv_bfloat16* v_new;
  const int32_t* self_seg;     // [R] segment index of every request's new node
  int32_t* written;            // [R] 64-token tiles of the request's new node that are in the pool; zero at launch
  int32_t cap_tiles, num_pairs, seg_cap;  // sizes that table-derived indices are checked against (debug build)
  long long num_q_rows;
  int32_t writer_tiles;        // writer jobs per request: ceil(longest new segment / 64)
  int32_t grid_x, grid_y;      // the (query block, request) extent of the work grid, KV heads slowest
};

// Barrier among the 256 softmax threads of one query tile (lagging walk): named barriers 9 and 10.
__device__ __forceinline__ void tile_bar_sync(int t) {
  if (t == 0) asm volatile("bar.sync 9, 256;" ::: "memory");
  else asm volatile("bar.sync 10, 256;" ::: "memory");
}

// Barrier between the two softmax warps that share the rows of one quarter of a query tile (the two
// column halves): named barriers 1..8, 64 threads each; id 0 is __syncthreads.
__device__ __forceinline__ void pair_bar_sync(int id) {
  asm volatile("bar.sync %0, 64;" ::"r"(id) : "memory");
}

template <int D>
struct TcLayout {
  static constexpr int CB = D / 64;                          // 128-byte column blocks per row
  static constexpr uint32_t kCbStride = 128u * 128u;        // bytes between column blocks (128 rows)
  static constexpr uint32_t kTileBytes = CB * kCbStride;    // one Q tile, one K stage or one V stage
  static constexpr uint32_t kHalfBytes = 64u * 128u;        // one 64-token pool tile of one column block
  static constexpr uint32_t offQ = 0;
  static constexpr uint32_t offK = 2 * kTileBytes;
  static constexpr uint32_t offV = offK + kKStages * kTileBytes;
  static constexpr uint32_t offBar = offV + kVStages * kTileBytes;
  static constexpr uint32_t kTotal = offBar + 256 + 2 * 768 * 4 + 8 * kMaxMeta;
};

struct Bars {
  uint64_t q_full[2], s_full[2], p_full[2], o_full[2];
  uint64_t k_full[kKStages], k_empty[kKStages], v_full[kVStages], v_empty[kVStages];
  uint32_t tmem_base;
  int32_t next_unit;  // decode: the (unit, head) this CTA works on next
  float xch[2][768];  // per tile: [2 stage parities + 1][2 column halves][128 rows]
  int grow[2][2];     // lagging walk: per tile and stage parity, a row outgrew its running maximum
  int2 meta[kMaxMeta];
};

// The CTA's path, copied to shared memory once: (tokens, first pool tile) per segment, so that no
// role waits on global memory at a segment boundary.  Paths longer than kMaxMeta segments read the
// rest from global memory.
struct PathMeta {
  const int2* meta;  // shared memory, min(nseg, kMaxMeta) entries
  const ExtendTcParams* p;
  int pb, nseg, vis_len;
  bool last_is_self;  // extend: the last segment is the request's own, causal, vis_len tokens of it
  __device__ __forceinline__ int2 get(int k) const {
    if (k < kMaxMeta) return meta[k];
    const int s = GF_CLAMP(p->pseg[GF_CLAMP(pb + k, p->num_pairs, p->status, 205)], p->seg_cap, p->status, 206);
    return make_int2(p->seg_len[s], p->seg_off[s] / kTile);
  }
};

// Calls body(j, self, t0, nv, tile) for every 128-token stage of the walk: j counts stages,
// self marks the request's own (causal) segment, t0 is the stage's first token inside its segment,
// nv its number of tokens, tile the pool tile index of token t0.
template <typename F>
__device__ __forceinline__ int walk_stages(const PathMeta& pm, F&& body) {
  int j = 0;
  for (int k = 0; k < pm.nseg; ++k) {
    const int2 m = pm.get(k);
    const bool self = pm.last_is_self && (k == pm.nseg - 1);
    const int len = self ? pm.vis_len : m.x;
    for (int t0 = 0; t0 < len; t0 += kStageTokens, ++j)
      body(j, self, t0, min(kStageTokens, len - t0), m.y + t0 / kTile);
  }
  return j;
}

// What one pass of a CTA works on (uniform over the CTA).
struct Pass {
  int q0, T, tok0, ntok, vis_len, pb, nseg;                  // extend
  int unit_req0, unit_slot0, unit_tile0, unit_len;           // decode
  int kvh;
  int req;  // extend: the request
  bool has_b;
  uint32_t tbase;
};

// Start of a pass, executed by every thread of the CTA: picks the work (decode: the next (unit, KV
// head) pair from the shared counter).  Returns false when there is nothing left.
template <bool kDecode, bool kExact>
__device__ __forceinline__ bool pick_work(const ExtendTcParams& p, Bars* bars, int& pass, int num_items, int tpt,
                                          int bx, int by, int bz, Pass& w) {
  const int tpc = 2 * tpt;
  w = Pass{};
  if (kDecode) {
    __syncthreads();  // everyone has read the previous pass's unit
    if (threadIdx.x == 0) bars->next_unit = atomicAdd(&p.counters[0], 1);
    __syncthreads();
    const int u = bars->next_unit;
    if (u >= num_items) return false;
    w.kvh = u % p.num_kv_heads;
    const int listed = p.wide_list[GF_CLAMP(u / p.num_kv_heads, p.slot_cap, p.status, 201)];
    const Item it = p.items[GF_CLAMP(listed, p.slot_cap, p.status, 202)];
    w.unit_req0 = it.grp_begin;
    w.unit_slot0 = it.part_base;
    w.unit_tile0 = it.tile0;
    w.unit_len = it.tok_count;
    w.ntok = min(tpc, p.grp_ptr[it.seg + 1] - it.grp_begin);  // requests of the unit
    w.T = w.ntok;
    w.nseg = 1;
  } else {
    if (kExact) {
      // a fixed row of CTAs strides over the (query block, request, KV head) grid of the first launch
      for (;; ++pass) {
        const long long wk = (long long)pass * gridDim.x + blockIdx.x;
        if (wk >= (long long)p.grid_x * p.grid_y * p.num_kv_heads) return false;
        bx = (int)(wk % p.grid_x);
        by = (int)((wk / p.grid_x) % p.grid_y);
        bz = (int)(wk / ((long long)p.grid_x * p.grid_y));
        const int rr = p.req_order[by];
        if (bx * tpc < p.q_ptr[rr + 1] - p.q_ptr[rr]) break;
      }
    } else if (pass > 0) {
      return false;
    }
    const int r = p.req_order[by];
    w.req = r;
    w.kvh = bz;
    w.q0 = p.q_ptr[r];
    w.T = p.q_ptr[r + 1] - w.q0;
    w.tok0 = bx * tpc;
    w.ntok = min(tpc, w.T - w.tok0);
    w.vis_len = w.tok0 + w.ntok;  // causal: later tokens of the new segment are never needed
    w.pb = p.pseg_ptr[r];
    w.nseg = p.pseg_ptr[r + 1] - w.pb;
  }
  w.has_b = w.ntok > tpt;
  return true;
}

// Start of the work on a pass, executed by every thread of the CTA: re-arms the barriers and stages
// the path geometry in shared memory.
template <bool kDecode>
__device__ __forceinline__ void arm_pass(const ExtendTcParams& p, Bars* bars, bool first, Pass& w) {
  __syncthreads();  // the previous pass (if any) is completely done with the barriers and buffers
  if (threadIdx.x == 0) {
    bars->grow[0][0] = bars->grow[0][1] = bars->grow[1][0] = bars->grow[1][1] = 0;
    if (!first) {  // the previous pass's barriers are valid objects: they are invalidated before they are set up again
      for (int t = 0; t < 2; ++t) {
        mbar_inval(&bars->q_full[t]); mbar_inval(&bars->s_full[t]); mbar_inval(&bars->p_full[t]); mbar_inval(&bars->o_full[t]);
      }
      for (int s = 0; s < kKStages; ++s) { mbar_inval(&bars->k_full[s]); mbar_inval(&bars->k_empty[s]); }
      for (int s = 0; s < kVStages; ++s) { mbar_inval(&bars->v_full[s]); mbar_inval(&bars->v_empty[s]); }
    }
    for (int t = 0; t < 2; ++t) {
      mbar_init(&bars->q_full[t], 8);   // one arrival per softmax warp of the tile
      mbar_init(&bars->s_full[t], 1);
      mbar_init(&bars->p_full[t], 8);
      mbar_init(&bars->o_full[t], 1);
    }
    for (int s = 0; s < kKStages; ++s) { mbar_init(&bars->k_full[s], 1); mbar_init(&bars->k_empty[s], 1); }
    for (int s = 0; s < kVStages; ++s) { mbar_init(&bars->v_full[s], 1); mbar_init(&bars->v_empty[s], 1); }
    if (kDecode) bars->meta[0] = make_int2(w.unit_len, w.unit_tile0);
    mbar_fence_init();
  }
  if (!kDecode) {
    for (int k = threadIdx.x; k < min(w.nseg, kMaxMeta); k += kTcThreads) {
      const int sg = GF_CLAMP(p.pseg[GF_CLAMP(w.pb + k, p.num_pairs, p.status, 203)], p.seg_cap, p.status, 204);
      bars->meta[k] = make_int2(p.seg_len[sg], p.seg_off[sg] / kTile);
    }
  }
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  w.tbase = bars->tmem_base;
}

// The last CTA of a launch to get here re-arms the shared counters for the next launch.
__device__ __forceinline__ void cta_finished(const ExtendTcParams& p) {
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(&p.counters[1], 1) == (int)gridDim.x - 1) { p.counters[0] = 0; p.counters[1] = 0; }
  }
}

// Exact kernel: every CTA read the flag when it started, so the last one to finish may lower it.
__device__ __forceinline__ void exact_finished(const ExtendTcParams& p) {
  if (threadIdx.x == 0) {
    __threadfence();
    if (atomicAdd(p.status + kStatusExactDone, 1) == (int)gridDim.x - 1) {
      p.status[kStatusExactDone] = 0;
      p.status[kStatusOverflow] = 0;
      atomicAdd(p.status + kStatusReruns, 1);
    }
  }
}

// Writer job of an extend with append: tile `tile` (64 tokens) of request r's new node, every KV
// head, K and V, from the caller layout [row, Hkv, D] into the pool layout (rows past the node's
// length are zeros, like in a node write).  The whole CTA copies; then the tile is counted.
template <int D>
__device__ void append_tile(const ExtendTcParams& p, int r, int tile) {
  constexpr int cpr = D / 8;  // 16-byte chunks per row of one head
  const int q0 = p.q_ptr[r], T = p.q_ptr[r + 1] - q0;
  if (tile * kTile >= T) return;  // this request's new node is shorter: nothing to copy, nothing to count
  const int tile0 = p.seg_off[GF_CLAMP(p.self_seg[r], p.seg_cap, p.status, 207)] / kTile + tile;
  if (!GF_CHECK(tile0 >= 0 && tile0 < p.cap_tiles, p.status, 208)) return;
  const int total = kTile * p.num_kv_heads * cpr;
  char* pool = const_cast<char*>(p.pool_layer);
  for (int which = 0; which < 2; ++which) {
    const uint4* src = reinterpret_cast<const uint4*>(which ? p.v_new : p.k_new);
    const uint32_t block_off = which ? (p.tile_bytes >> 1) : 0u;
    for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
      const int c = idx % cpr;
      const int head = (idx / cpr) % p.num_kv_heads;
      const int row = idx / (cpr * p.num_kv_heads);  // token inside the tile
      const int token = tile * kTile + row;
      uint4 val = make_uint4(0u, 0u, 0u, 0u);
      if (token < T) val = src[((size_t)(q0 + token) * p.num_kv_heads + head) * cpr + c];
      char* dst = pool + (uint64_t)head * p.head_stride + (uint64_t)tile0 * p.tile_bytes + block_off +
                  (uint32_t)(c >> 3) * (kTile * 128u) + swz128((uint32_t)row, (uint32_t)c & 7u);
      *reinterpret_cast<uint4*>(dst) = val;
    }
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    __threadfence();  // the tile is in global memory before it is counted
    atomicAdd(&p.written[r], 1);
  }
}

// The producer's wait for the writers of request r's new node: bounded like every wait here.  The
// copies that follow read the pool through the async proxy, hence the proxy fence after the acquire.
__device__ __forceinline__ void wait_appended(const ExtendTcParams& p, int r, int tiles) {
  const long long t0 = clock64();
  while (*(volatile int32_t*)(p.written + r) < tiles) {
    __nanosleep(256);
    if (*(volatile int32_t*)(p.status + kStatusGiveUp) != 0) break;
    if (clock64() - t0 > kWaitCycles) {
      atomicExch(p.status + kStatusGiveUp, (int32_t)8 /* GF_ERR_TIMEOUT */);
      break;
    }
  }
  __threadfence();
  asm volatile("fence.proxy.async;" ::: "memory");
}

// kDecode = false: extend.  One CTA per (request, block of 2*128/g new tokens, KV head).
// kDecode = true : decode over widely shared chunks.  A unit is a chunk of a segment and up to 64 of
//   the requests that share it (the group tiles of four consecutive flagged items: their partial
//   slots are contiguous), i.e. up to 256 stacked query rows (request x GQA head) against the chunk's
//   K and V, no mask; the result is the fp32 partial (O, m, l) per (slot, head) for the merge.  The
//   table builder lists the units; one CTA per SM takes (unit, KV head) pairs from a shared counter.
//
// Registers.  The CTA is launched as five warpgroups of 96 registers per thread (20 warps: register
// files are handed out to four warps at a time, so 18 warps would cost the same), and that total,
// 640 * 96 = 61 440, is all the CTA can redistribute.  The last warpgroup (producer, MMA issuer, two
// warps without a role) keeps 56; the four softmax warpgroups grow to 104, which lets a thread hold
// its 64 scores of a stage in registers between taking their maximum and exponentiating them:
// 128 * (4 * 104 + 56) = 60 416.
//
// kExact.  The plain kernel (kExact = false) forms the probabilities of a stage against the maximum
// of the stages before it, which saves a pass over the scores and a barrier per stage and is exact
// as long as no score stands more than 2^64 above that reference.  A thread that meets such a score
// raises a flag in the status block.  The exact kernel (kExact = true) is launched behind every plain
// launch, leaves at once unless the flag is up, and otherwise redoes all of the launch's work with
// each stage's maximum taken before its probabilities, overwriting every result of the plain launch.
template <int D, bool kDecode, bool kExact>
__global__ void __launch_bounds__(kTcThreads, 1) k_path_tc(const ExtendTcParams p) {
  using L = TcLayout<D>;
  constexpr int CB = L::CB;
  extern __shared__ __align__(1024) unsigned char smem[];
  Bars* bars = reinterpret_cast<Bars*>(smem + L::offBar);
  chain_enter();  // nothing above touches global memory
  if (kExact && *(volatile int32_t*)(p.status + kStatusOverflow) == 0) return;  // uniform over the launch

  const int g = p.gqa;
  const int tpt = 128 / g;   // query tokens (extend) or requests (decode) per 128-row tile
  const int tpc = 2 * tpt;   // per CTA
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int num_items = 1;  // decode: (wide unit, KV head) pairs, taken from a shared counter
  int bx = blockIdx.x, by = blockIdx.y, bz = blockIdx.z;  // extend: (query block, request in launch order, KV head)
  if (kDecode) {
    if (!tables_usable(*p.hdr, p.slot_cap) || p.hdr->num_wide == 0) {  // nothing is flagged wide
      if (kExact) exact_finished(p);
      return;
    }
    num_items = p.hdr->wide_list_n * p.num_kv_heads;
  } else {
    if (p.k_new != nullptr) {
      // Extend with append.  CTAs take a ticket in the order in which they start.  The first
      // R * writer_tiles tickets are writer jobs: copy one 64-token tile of one request's new K/V
      // from the caller layout into its pool extent, then count it in written[request].  Later
      // tickets are the attention work in the usual order; their producer waits (bounded) for
      // written[request] before it streams the new segment, long after it has walked the prefix.
      // A writer never waits for anything and every writer has started before any worker exists,
      // so the waits end whatever the order in which CTAs are scheduled.
      if (threadIdx.x == 0) bars->next_unit = atomicAdd(&p.counters[0], 1);
      __syncthreads();
      const int ticket = bars->next_unit;
      const int n_writer = p.num_requests * p.writer_tiles;
      if (ticket < n_writer) {
        append_tile<D>(p, ticket / p.writer_tiles, ticket % p.writer_tiles);
        cta_finished(p);
        return;
      }
      const int wk = ticket - n_writer;
      bx = wk % p.grid_x;
      by = (wk / p.grid_x) % p.grid_y;
      bz = wk / (p.grid_x * p.grid_y);
    }
    // `by` walks the requests longest context first; leave before anything is allocated if this
    // block of query tokens does not exist
    if (!kExact) {
      const int r = p.req_order[by];
      if (bx * tpc >= p.q_ptr[r + 1] - p.q_ptr[r]) {
        if (p.k_new != nullptr) cta_finished(p);
        return;
      }
    }
  }
  if (warp == 17) tmem_alloc(&bars->tmem_base, 512);

  if (warp >= 16) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kServiceRegs));
    bool first = true;
    for (int pass = 0;; ++pass, first = false) {
      Pass w;
      if (!pick_work<kDecode, kExact>(p, bars, pass, num_items, tpt, bx, by, bz, w)) break;
      arm_pass<kDecode>(p, bars, first, w);
      const int kvh = w.kvh;
      const bool has_b = w.has_b;
      const uint32_t tbase = w.tbase;
      PathMeta pm;
      pm.meta = bars->meta; pm.p = &p; pm.pb = w.pb; pm.nseg = w.nseg; pm.vis_len = w.vis_len;
      pm.last_is_self = !kDecode;
  if (warp == 16) {
    // ------------------------------- producer -------------------------------
    if (lane == 0) {
      const char* head_base = p.pool_layer + (uint64_t)kvh * p.head_stride;
      walk_stages(pm, [&](int j, bool self, int t0, int nv, int tile) {
        if (!kDecode && self && t0 == 0 && p.k_new != nullptr) wait_appended(p, w.req, (w.T + kTile - 1) / kTile);
        const int nh = nv > kTile ? 2 : 1;  // 64-token pool tiles in this stage
        if (!GF_CHECK(tile >= 0 && tile + nh <= p.cap_tiles, p.status, 209)) tile = 0;
        const char* src = head_base + (uint64_t)tile * p.tile_bytes;
        {
          const int st = j % kKStages;
          if (j >= kKStages) mbar_wait(&bars->k_empty[st], ((j / kKStages) - 1) & 1, p.status);
          unsigned char* dst = smem + L::offK + st * L::kTileBytes;
          mbar_arrive_expect_tx(&bars->k_full[st], nh * CB * L::kHalfBytes);
          for (int h = 0; h < nh; ++h)
#pragma unroll
            for (int cb = 0; cb < CB; ++cb)
              bulk_g2s(dst + cb * L::kCbStride + h * L::kHalfBytes,
                       src + (uint64_t)h * p.tile_bytes + cb * L::kHalfBytes, L::kHalfBytes, &bars->k_full[st]);
        }
        {
          const int st = j % kVStages;
          if (j >= kVStages) mbar_wait(&bars->v_empty[st], ((j / kVStages) - 1) & 1, p.status);
          unsigned char* dst = smem + L::offV + st * L::kTileBytes;
          mbar_arrive_expect_tx(&bars->v_full[st], nh * CB * L::kHalfBytes);
          for (int h = 0; h < nh; ++h)
#pragma unroll
            for (int cb = 0; cb < CB; ++cb)
              bulk_g2s(dst + cb * L::kCbStride + h * L::kHalfBytes,
                       src + (uint64_t)h * p.tile_bytes + (CB + cb) * L::kHalfBytes, L::kHalfBytes,
                       &bars->v_full[st]);
        }
      });
    }
  } else if (warp == 17) {
    // ------------------------------- MMA issuer -------------------------------
    // One thread issues every MMA, alternating between the tiles, which keeps their softmax phases
    // half a period apart.  It sustains one 128x128x16 MMA per ~64 cycles only with a handful of
    // instructions between issues, hence the prebuilt descriptors and unrolled loops.
    if (lane == 0) {
      constexpr uint32_t idesc_s128 = tc_idesc_bf16(128, kStageTokens, false);
      constexpr uint32_t idesc_s64 = tc_idesc_bf16(128, kTile, false);  // a stage with one pool tile
      constexpr uint32_t idesc_o = tc_idesc_bf16(128, D, true);
      // The start address sits in the low bits of a descriptor, in units of 16 bytes: inside the
      // loops an MMA costs one 64-bit add and the issue.
      const uint64_t q_desc0 = tc_smem_desc(smem_u32(smem + L::offQ), 0, 1024);
      const uint64_t k_desc0 = tc_smem_desc(smem_u32(smem + L::offK), 0, 1024);
      const uint64_t v_desc0 = tc_smem_desc(smem_u32(smem + L::offV), L::kCbStride, 1024);
      const int ntile = has_b ? 2 : 1;
      for (int t = 0; t < ntile; ++t) mbar_wait(&bars->q_full[t], 0, p.status);
      int prev_nv = 0;
      // O_t += P_t(jp) V(jp) for the stage jp whose P the softmax warps have just finished
      auto issue_pv = [&](int t, int jp, int nv) {
        mbar_wait(&bars->p_full[t], jp & 1, p.status);
        tc_fence_after_sync();
        const uint64_t vd = v_desc0 + (uint64_t)((jp % kVStages) * (L::kTileBytes >> 4));
        const uint32_t d_o = tbase + 256 + t * D, a_p = tbase + t * 128;
        if (nv == kStageTokens) {
          umma_ts_kloop8(d_o, a_p, vd, idesc_o, jp > 0 ? 1u : 0u);
        } else {
          umma_ts(d_o, a_p, vd, idesc_o, jp > 0 ? 1u : 0u);
          const int ksteps = (nv + 15) >> 4;
          for (int ks = 1; ks < ksteps; ++ks)
            umma_ts(d_o, a_p + (ks >> 2) * 64 + (ks & 3) * 8, vd + ks * (2048 >> 4), idesc_o, 1u);
        }
      };
      // The pipe takes an MMA from this thread only shortly before it runs it (a few MMAs ahead at
      // most), so whatever the thread does between two MMAs beyond a couple of hundred cycles is
      // time the pipe stands idle.  The waits and commits of a stage are therefore spread over the
      // gaps between its four MMA blocks instead of being gathered at the stage's start.
      const int n = walk_stages(pm, [&](int j, bool, int, int nv, int) {
        const int st = j % kKStages;
        const uint64_t kd = k_desc0 + (uint64_t)(st * (L::kTileBytes >> 4));
        const uint32_t idesc_s = nv > kTile ? idesc_s128 : idesc_s64;
        for (int t = 0; t < ntile; ++t) {
          if (j > 0) {
            if (t == 0) mbar_wait(&bars->v_full[(j - 1) % kVStages], ((j - 1) / kVStages) & 1, p.status);
            issue_pv(t, j - 1, prev_nv);
            if (t == ntile - 1) tc_commit(&bars->v_empty[(j - 1) % kVStages]);
          }
          if (t == 0) {  // K(j) is first needed here, behind the MMAs just queued
            mbar_wait(&bars->k_full[st], (j / kKStages) & 1, p.status);
            tc_fence_after_sync();
          }
          const uint64_t qd = q_desc0 + (uint64_t)(t * (L::kTileBytes >> 4));
          umma_ss_kloop<CB>(tbase + t * 128, qd, kd, idesc_s);
          tc_commit(&bars->s_full[t]);
        }
        tc_commit(&bars->k_empty[st]);
        prev_nv = nv;
      });
      mbar_wait(&bars->v_full[(n - 1) % kVStages], ((n - 1) / kVStages) & 1, p.status);
      for (int t = 0; t < ntile; ++t) {
        issue_pv(t, n - 1, prev_nv);
        tc_commit(&bars->o_full[t]);
      }
    }
  }
    }  // passes of the service warps
  } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    bool first = true;
    for (int pass = 0;; ++pass, first = false) {
      Pass w;
      if (!pick_work<kDecode, kExact>(p, bars, pass, num_items, tpt, bx, by, bz, w)) break;
      arm_pass<kDecode>(p, bars, first, w);
      const int kvh = w.kvh, q0 = w.q0, T = w.T, tok0 = w.tok0, unit_req0 = w.unit_req0, unit_slot0 = w.unit_slot0;
      const bool has_b = w.has_b;
      const uint32_t tbase = w.tbase;
      PathMeta pm;
      pm.meta = bars->meta; pm.p = &p; pm.pb = w.pb; pm.nseg = w.nseg; pm.vis_len = w.vis_len;
      pm.last_is_self = !kDecode;
  {
    // ------------------------------- softmax + epilogue -------------------------------
    // Eight warps per tile: two threads share a query row, each owning 64 of the stage's 128
    // score columns and 64 of the D output columns.  A warp may only touch the tensor-memory
    // lanes of its quarter (warp index mod 4), so the two warps of a quarter split the columns.
    const int t = warp >> 3;                     // 0: tile A, 1: tile B
    if (t == 0 || has_b) {
      const int half = (warp >> 2) & 1;          // which 64 columns
      const int row = (warp & 3) * 32 + lane;    // row of the tile = tensor-memory lane
      const uint32_t lane_field = (uint32_t)((warp & 3) * 32) << 16;
      const int tok = tok0 + t * tpt + row / g;  // extend: token of the new segment; decode: request of the unit
      const bool valid = tok < T;
      const int lim = valid ? tok : -1;          // extend: newest visible token of the new segment
      const int tile_first_tok = tok0 + t * tpt;
      const int head = kvh * g + row % g;
      // row of Q (and, in extend, of out / lse) in global memory
      const size_t grow =
          kDecode ? (size_t)GF_CLAMP(valid ? p.grp_req[GF_CLAMP(unit_req0 + tok, p.num_pairs, p.status, 210)] : 0,
                                     p.num_requests, p.status, 211) * p.num_q_heads + head
                  : (size_t)(valid ? GF_CLAMP(q0 + tok, p.num_q_rows, p.status, 212) : 0) * p.num_q_heads + head;
      constexpr int DH = D / 2;                  // output columns of this thread

      // Stage the tile's query rows (zeros for rows past the end).  The rows are dealt out in 16-byte
      // pieces, 32 consecutive pieces (two whole rows at D = 128) per warp and load instruction, so that
      // a warp's load reads whole lines; which thread stages which piece has nothing to do with the row
      // the thread owns in the softmax.  Every load is issued before the first store.
      {
        unsigned char* qt = smem + L::offQ + t * L::kTileBytes;
        constexpr int CPR = D / 8;  // 16-byte pieces per row
        uint4 val[D / 16];
#pragma unroll
        for (int i = 0; i < D / 16; ++i) {
          const int id = (((warp & 7) * (D / 16) + i) << 5) + lane;
          const int r = id / CPR, c = id % CPR;
          const int tok_r = tok0 + t * tpt + r / g;
          const size_t grow_r =
              kDecode ? (size_t)GF_CLAMP(tok_r < T ? p.grp_req[GF_CLAMP(unit_req0 + tok_r, p.num_pairs, p.status, 210)] : 0,
                                         p.num_requests, p.status, 211) * p.num_q_heads + kvh * g + r % g
                      : (size_t)(tok_r < T ? GF_CLAMP(q0 + tok_r, p.num_q_rows, p.status, 212) : 0) * p.num_q_heads + kvh * g + r % g;
          val[i] = make_uint4(0u, 0u, 0u, 0u);
          if (tok_r < T) val[i] = __ldg(reinterpret_cast<const uint4*>(p.q + grow_r * D) + c);
        }
#pragma unroll
        for (int i = 0; i < D / 16; ++i) {
          const int id = (((warp & 7) * (D / 16) + i) << 5) + lane;
          const int r = id / CPR, c = id % CPR;
          *reinterpret_cast<uint4*>(qt + (c >> 3) * L::kCbStride + swz128(r, c & 7)) = val[i];
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->q_full[t]);
      }

      const uint32_t ts_row = tbase + t * 128 + lane_field + half * 64;        // this thread's S columns
      const uint32_t tp_row = ts_row;  // packed P goes over the first 32 of this thread's own S columns
      const uint32_t to_row = tbase + 256 + t * D + lane_field + half * DH;    // its O columns
      float* xch = bars->xch[t];  // [stage parity][half][row]: row maxima (and, at the end, row sums)
      const int pair_id = 1 + t * 4 + (warp & 3);
      float m_used = -INFINITY, l = 0.f;
      if constexpr (!kExact) {
      // ---- one pass over the scores per stage, against a maximum that lags one stage
      volatile int* grow_flag = bars->grow[t];  // [stage parity]: some row of the tile outgrew its maximum
      float mx_prev = -INFINITY;  // maximum of this thread's raw scores in the previous stage
      walk_stages(pm, [&](int j, bool self, int t0, int nv, int) {
        mbar_wait(&bars->s_full[t], j & 1, p.status);
        tc_fence_after_sync();
        const bool need_mask = (nv < kStageTokens) || (self && t0 + kStageTokens - 1 > tile_first_tok);
        // visible columns of this row, counted from this thread's first column (may be <= 0)
        const int ncol = (self ? min(nv, lim - t0 + 1) : nv) - half * 64;
        const int my_chunks = min(2, max(0, (nv - half * 64 + 31) >> 5));  // 32-column chunks the MMA wrote

        // The running maximum lags by one stage: P uses the maximum known so far (any reference
        // works as long as P, l and O share it), and only when some row's scores outgrew it by more
        // than 2^8 does the whole tile, one stage later, agree on new maxima and rescale l and O.
        // The first stage takes the same path to get an initial maximum from its own scores.
        const bool slow = (j == 0) || (grow_flag[(j - 1) & 1] != 0);  // uniform over the tile
        if (slow) {
          float mx = mx_prev;
          if (j == 0) {
            mx = -INFINITY;
            for (int c = 0; c < my_chunks; ++c) {
              uint32_t rg[32];
              tmem_ld32(ts_row + c * 32, rg);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) mx = (c * 32 + i < ncol) ? fmaxf(mx, __uint_as_float(rg[i])) : mx;
            }
          }
          float* slot = xch + (j & 1) * 256;
          slot[half * 128 + row] = mx;
          tile_bar_sync(t);
          mx = fmaxf(mx, slot[(half ^ 1) * 128 + row]);
          if (j > 0 && half == 0 && row == 0) grow_flag[(j - 1) & 1] = 0;
          const float m_new = fmaxf(m_used, mx * p.scale_log2);
          const float alpha = (m_new > m_used) ? ((m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_new)) : 1.f;
          l *= alpha;
          m_used = m_new;
          if (j > 0) {  // stage 0 overwrites O, nothing to rescale yet
            if (lane == 0 && half == 0) atomicAdd(p.status + kStatusRescales, 1);
#pragma unroll
            for (int c = 0; c < DH / 32; ++c) {
              uint32_t rg[32];
              tmem_ld32(to_row + c * 32, rg);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 32; ++i) rg[i] = __float_as_uint(__uint_as_float(rg[i]) * alpha);
              tmem_st32(to_row + c * 32, rg);
            }
          }
        }

        // one pass over this thread's scores: P = 2^(s*scale - m), row sum, bf16 pairs over S
        const float m_ref = (m_used == -INFINITY) ? 0.f : m_used;
        const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
        const uint64_t nm2 = f2_pack(-m_ref, -m_ref);
        uint64_t sum2 = f2_pack(0.f, 0.f);
        float sum = 0.f, mx = -INFINITY;
        for (int c = 0; c < my_chunks; ++c) {
          uint32_t rg[32], pk[16];
          tmem_ld32(ts_row + c * 32, rg);
          tmem_wait_ld();
          if (need_mask) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float s0 = __uint_as_float(rg[2 * i]), s1 = __uint_as_float(rg[2 * i + 1]);
              const bool v0 = c * 32 + 2 * i < ncol, v1 = c * 32 + 2 * i + 1 < ncol;
              mx = v0 ? fmaxf(mx, s0) : mx;
              mx = v1 ? fmaxf(mx, s1) : mx;
              const float p0 = v0 ? fast_exp2(fmaf(s0, p.scale_log2, -m_ref)) : 0.f;
              const float p1 = v1 ? fast_exp2(fmaf(s1, p.scale_log2, -m_ref)) : 0.f;
              sum += p0 + p1;
              pk[i] = pack_bf16(p0, p1);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float s0 = __uint_as_float(rg[2 * i]), s1 = __uint_as_float(rg[2 * i + 1]);
              mx = fmax3(mx, s0, s1);
              float x0, x1;
              f2_unpack(f2_fma(f2_pack(s0, s1), scale2, nm2), x0, x1);
              const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
              sum2 = f2_add(sum2, f2_pack(p0, p1));
              pk[i] = pack_bf16(p0, p1);
            }
          }
          tmem_st16(tp_row + c * 16, pk);
        }
        {
          float s0, s1;
          f2_unpack(sum2, s0, s1);
          l += sum + (s0 + s1);
        }
        mx_prev = mx;
        if (mx * p.scale_log2 > m_used + kRescaleThreshold) grow_flag[j & 1] = 1;
        // P was formed against a reference that lags.  A score this far above it is close to what
        // fp32 can exponentiate: nothing this launch computes is kept then, the exact kernel follows.
        if (mx * p.scale_log2 > m_used + kOverflowMargin) *(volatile int32_t*)(p.status + kStatusOverflow) = 1;
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();  // every lane's stores are done and fenced: one arrival stands for the warp
        if (lane == 0) mbar_arrive(&bars->p_full[t]);
      });

      } else {
      // ---- the stage's own maximum first, then the probabilities: two steps over scores held in registers
      walk_stages(pm, [&](int j, bool self, int t0, int nv, int) {
        mbar_wait(&bars->s_full[t], j & 1, p.status);
        tc_fence_after_sync();
        const bool need_mask = (nv < kStageTokens) || (self && t0 + kStageTokens - 1 > tile_first_tok);
        // visible columns of this row, counted from this thread's first column (may be <= 0)
        const int ncol = (self ? min(nv, lim - t0 + 1) : nv) - half * 64;
        const int my_chunks = min(2, max(0, (nv - half * 64 + 31) >> 5));  // 32-column chunks the MMA wrote

        // ---- this thread's scores (up to 64 columns) stay in registers for both steps below
        uint32_t r0[32], r1[32];
        if (my_chunks > 0) tmem_ld32(ts_row, r0);
        if (my_chunks > 1) tmem_ld32(ts_row + 32, r1);
        tmem_wait_ld();

        // ---- step 1: the row's maximum over this stage, exact, before anything is exponentiated
        float mx = -INFINITY;
        if (need_mask) {
          if (my_chunks > 0) {
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = (i < ncol) ? fmaxf(mx, __uint_as_float(r0[i])) : mx;
          }
          if (my_chunks > 1) {
#pragma unroll
            for (int i = 0; i < 32; ++i) mx = (32 + i < ncol) ? fmaxf(mx, __uint_as_float(r1[i])) : mx;
          }
        } else {  // a full stage: both chunks exist and every column is visible
#pragma unroll
          for (int i = 0; i < 16; ++i) {
            mx = fmax3(mx, __uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
            mx = fmax3(mx, __uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
          }
        }
        {
          float* slot = xch + (j & 1) * 256;
          slot[half * 128 + row] = mx;
          pair_bar_sync(pair_id);
          mx = fmaxf(mx, slot[(half ^ 1) * 128 + row]);
        }
        // Both threads of the row now hold the same maximum and the same reference, so they take the
        // same decision without further talk.  The reference moves when the stage outgrew it by more
        // than the threshold (always for the first visible score: m_used is -inf until then).
        const float m_stage = mx * p.scale_log2;
        const bool move = m_stage > m_used + kRescaleThreshold;
        if (__any_sync(0xffffffffu, move)) {  // the tensor-memory accesses below are warp-wide
          const float alpha = !move ? 1.f : ((m_used == -INFINITY) ? 0.f : fast_exp2(m_used - m_stage));
          if (move) { l *= alpha; m_used = m_stage; }
          if (j > 0) {  // stage 0 overwrites O, nothing to rescale yet
            for (int c = 0; c < DH / 16; ++c) {  // 16 columns at a time: the scores stay in registers meanwhile
              uint32_t rg[16];
              tmem_ld16(to_row + c * 16, rg);
              tmem_wait_ld();
#pragma unroll
              for (int i = 0; i < 16; ++i) rg[i] = __float_as_uint(__uint_as_float(rg[i]) * alpha);
              tmem_st16(to_row + c * 16, rg);
            }
            if (lane == 0 && half == 0) atomicAdd(p.status + kStatusRescales, 1);
          }
        }

        // ---- step 2: P = 2^(s*scale - m) as bf16 pairs over S, and the row sum
        const float m_ref = (m_used == -INFINITY) ? 0.f : m_used;
        const uint64_t scale2 = f2_pack(p.scale_log2, p.scale_log2);
        const uint64_t nm2 = f2_pack(-m_ref, -m_ref);
        uint64_t sum2 = f2_pack(0.f, 0.f);
        auto emit = [&](const uint32_t (&rg)[32], int c) {
          uint32_t pk[16];
          if (need_mask) {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              const float s0 = __uint_as_float(rg[2 * i]), s1 = __uint_as_float(rg[2 * i + 1]);
              const bool v0 = c * 32 + 2 * i < ncol, v1 = c * 32 + 2 * i + 1 < ncol;
              const float p0 = v0 ? fast_exp2(fmaf(s0, p.scale_log2, -m_ref)) : 0.f;
              const float p1 = v1 ? fast_exp2(fmaf(s1, p.scale_log2, -m_ref)) : 0.f;
              sum2 = f2_add(sum2, f2_pack(p0, p1));
              pk[i] = pack_bf16(p0, p1);
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float x0, x1;
              f2_unpack(f2_fma(f2_pack(__uint_as_float(rg[2 * i]), __uint_as_float(rg[2 * i + 1])), scale2, nm2), x0, x1);
              const float p0 = fast_exp2(x0), p1 = fast_exp2(x1);
              sum2 = f2_add(sum2, f2_pack(p0, p1));
              pk[i] = pack_bf16(p0, p1);
            }
          }
          tmem_st16(tp_row + c * 16, pk);
        };
        if (my_chunks > 0) emit(r0, 0);
        if (my_chunks > 1) emit(r1, 1);
        {
          float s0, s1;
          f2_unpack(sum2, s0, s1);
          l += s0 + s1;
        }
        tmem_wait_st();
        tc_fence_before_sync();
        __syncwarp();  // every lane's stores are done and fenced: one arrival stands for the warp
        if (lane == 0) mbar_arrive(&bars->p_full[t]);
      });

      }

      // epilogue: the row sum is the two halves' sums; O / l -> bf16, 64 columns per thread
      mbar_wait(&bars->o_full[t], 0, p.status);
      tc_fence_after_sync();
      {
        float* slot = xch + 512;  // not one of the per-stage slots
        slot[half * 128 + row] = l;
        pair_bar_sync(pair_id);
        l += slot[(half ^ 1) * 128 + row];
      }
      if (kDecode) {
        // fp32 partial for the merge: un-normalised O, m in scaled log2 units, l
        const size_t ph = (size_t)GF_CLAMP(valid ? unit_slot0 + tok : 0, p.slot_cap, p.status, 213) * p.num_q_heads + head;
#pragma unroll
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t rg[32];
          tmem_ld32(to_row + c * 32, rg);
          tmem_wait_ld();
          if (valid) {
            uint4* dst = reinterpret_cast<uint4*>(p.part_o + ph * D + half * DH + c * 32);
#pragma unroll
            for (int v4 = 0; v4 < 8; ++v4) dst[v4] = make_uint4(rg[4 * v4], rg[4 * v4 + 1], rg[4 * v4 + 2], rg[4 * v4 + 3]);
          }
        }
        if (half == 0 && valid) *reinterpret_cast<float2*>(p.part_ml + ph * 2) = make_float2(m_used, l);
      } else {
        const float inv = (l > 0.f) ? 1.f / l : 0.f;
#pragma unroll
        for (int c = 0; c < DH / 32; ++c) {
          uint32_t rg[32];
          tmem_ld32(to_row + c * 32, rg);
          tmem_wait_ld();
          if (valid) {
            uint4* dst = reinterpret_cast<uint4*>(p.out + grow * D + half * DH + c * 32);
#pragma unroll
            for (int v4 = 0; v4 < 4; ++v4) {
              uint4 o4;
              o4.x = pack_bf16(__uint_as_float(rg[8 * v4 + 0]) * inv, __uint_as_float(rg[8 * v4 + 1]) * inv);
              o4.y = pack_bf16(__uint_as_float(rg[8 * v4 + 2]) * inv, __uint_as_float(rg[8 * v4 + 3]) * inv);
              o4.z = pack_bf16(__uint_as_float(rg[8 * v4 + 4]) * inv, __uint_as_float(rg[8 * v4 + 5]) * inv);
              o4.w = pack_bf16(__uint_as_float(rg[8 * v4 + 6]) * inv, __uint_as_float(rg[8 * v4 + 7]) * inv);
              dst[v4] = o4;
            }
          }
        }
        if (half == 0 && valid && p.lse != nullptr)
          p.lse[grow] = (l > 0.f) ? (m_used + log2f(l)) * 0.6931471805599453f : -INFINITY;
      }
    }
  }
    }  // passes of the softmax warps
  }
  if (kDecode || p.k_new != nullptr) cta_finished(p);
  if (kExact) exact_finished(p);

  tc_fence_before_sync();
  __syncthreads();
  if (warp == 17) {
    __syncwarp();
    tmem_dealloc(bars->tmem_base, 512);
  }
}

}  // namespace

// Decode over the widely shared chunks (items the table builder flagged).  grid.x strides over the
// item list, whose length the kernel reads on the device.
// The plain kernel, then the exact kernel (which leaves at once unless the plain one raised the flag).
template <int D, bool kDecode>
bool launch_tc_pair(ExtendTcParams p, dim3 grid, dim3 grid_exact, bool chained, cudaStream_t st) {
  static bool optin[kMaxDevices] = {}, optin_exact[kMaxDevices] = {};
  if (!ensure_dynamic_smem(k_path_tc<D, kDecode, false>, TcLayout<D>::kTotal, optin)) return false;
  if (!ensure_dynamic_smem(k_path_tc<D, kDecode, true>, TcLayout<D>::kTotal, optin_exact)) return false;
  if (chained) launch_chained(k_path_tc<D, kDecode, false>, grid, dim3(kTcThreads), TcLayout<D>::kTotal, st, p);
  else k_path_tc<D, kDecode, false><<<grid, dim3(kTcThreads), TcLayout<D>::kTotal, st>>>(p);
  p.k_new = nullptr;  // an append has happened by now: the exact kernel reads the new segment from the pool
  p.v_new = nullptr;
  k_path_tc<D, kDecode, true><<<grid_exact, dim3(kTcThreads), TcLayout<D>::kTotal, st>>>(p);
  return true;
}

int launch_decode_wide(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int num_items, int layer,
                       const void* q, int32_t* status, int num_ctas, int exact_ctas, bool chained, cudaStream_t st) {
  if (num_items == 0) return 0;
  ExtendTcParams p{};
  p.pool_layer = pool.base + (uint64_t)layer * pool.layer_stride;
  p.head_stride = pool.head_stride;
  p.tile_bytes = pool.tile_bytes;
  p.q = (const __nv_bfloat16*)q;
  p.status = status;
  p.num_requests = t.num_requests;
  p.num_q_heads = sh.num_q_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  p.items = t.items;
  p.grp_ptr = t.grp_ptr;
  p.grp_req = t.grp_req;
  p.part_o = t.part_o;
  p.part_ml = t.part_ml;
  p.hdr = t.hdr;
  p.slot_cap = t.slot_cap;
  p.wide_list = t.wide_list;
  p.cap_tiles = (int32_t)pool.cap_tiles;
  p.num_pairs = t.num_pairs_in;
  p.seg_cap = t.seg_cap;
  p.counters = status + kStatusWideQueue;
  p.num_kv_heads = sh.num_kv_heads;
  const int sms = t.num_sms > 0 ? t.num_sms : 148;
  dim3 grid((unsigned)((num_ctas > 0 && num_ctas < sms) ? num_ctas : sms), 1, 1);  // persistent: at most one CTA per SM
  // the exact kernel behind it: as many CTAs as are sure to find a multiprocessor while another kernel runs beside
  dim3 grid_exact((unsigned)((exact_ctas > 0 && exact_ctas < sms) ? exact_ctas : sms), 1, 1);
  if (sh.head_dim == 128) {
    if (!launch_tc_pair<128, true>(p, grid, grid_exact, chained, st)) return -1;
  } else {
    if (!launch_tc_pair<64, true>(p, grid, grid_exact, chained, st)) return -1;
  }
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

int launch_extend_tc(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int layer,
                     int max_q_rows, long long num_q_rows, const void* q, const void* k_new, const void* v_new, void* out, float* lse,
                     int32_t* status, cudaStream_t st) {
  if (max_q_rows <= 0) return 0;
  ExtendTcParams p{};
  p.pool_layer = pool.base + (uint64_t)layer * pool.layer_stride;
  p.head_stride = pool.head_stride;
  p.tile_bytes = pool.tile_bytes;
  p.seg_off = t.seg_off;
  p.seg_len = t.seg_len;
  p.pseg_ptr = t.pseg_ptr;
  p.pseg = t.pseg;
  p.q_ptr = t.q_ptr;
  p.req_order = t.req_order;
  p.q = (const __nv_bfloat16*)q;
  p.out = (__nv_bfloat16*)out;
  p.lse = lse;
  p.status = status;
  p.num_requests = t.num_requests;
  p.num_q_heads = sh.num_q_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  p.cap_tiles = (int32_t)pool.cap_tiles;
  p.num_pairs = t.num_pairs_in;
  p.seg_cap = t.seg_cap;
  p.num_q_rows = num_q_rows;
  const int tpc = 256 / p.gqa;
  dim3 grid((unsigned)((max_q_rows + tpc - 1) / tpc), (unsigned)t.num_requests, (unsigned)sh.num_kv_heads);
  p.grid_x = (int)grid.x;
  p.grid_y = (int)grid.y;
  p.num_kv_heads = sh.num_kv_heads;
  const long long blocks = (long long)grid.x * grid.y * grid.z;
  const int sms = t.num_sms > 0 ? t.num_sms : 148;
  dim3 grid_exact((unsigned)(blocks < sms ? blocks : sms), 1, 1);
  if (k_new != nullptr) {
    // append: writer jobs first, then the same work in the same order, all as one row of CTAs that
    // take tickets (the counters are those of the tensor-memory decode kernel, idle in extend mode)
    p.k_new = (const __nv_bfloat16*)k_new;
    p.v_new = (const __nv_bfloat16*)v_new;
    p.self_seg = t.self_seg;
    p.written = t.ext_written;
    p.writer_tiles = (max_q_rows + kTile - 1) / kTile;
    p.counters = status + kStatusWideQueue;
    const long long total = (long long)t.num_requests * p.writer_tiles + blocks;
    if (total > 0x7fffffffll) return -1;
    if (cudaMemsetAsync(t.ext_written, 0, (size_t)t.num_requests * 4, st) != cudaSuccess) return -1;
    grid = dim3((unsigned)total, 1, 1);
  }
  if (sh.head_dim == 128) {
    if (!launch_tc_pair<128, false>(p, grid, grid_exact, true, st)) return -1;
  } else {
    if (!launch_tc_pair<64, false>(p, grid, grid_exact, true, st)) return -1;
  }
  return cudaGetLastError() == cudaSuccess ? 2 : -1;
}

}  // namespace gf
