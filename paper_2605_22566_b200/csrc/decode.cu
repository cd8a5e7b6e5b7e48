// K2: shared-segment decode, and K4: log-sum-exp merge.
//
// A work item is one chunk of one node's KV segment together with one tile (<= 16) of the
// requests whose workflow path passes through that node (Sec. 5: the node's KV state is stored
// once and assembled into every such request's context).  A unit of work is (item, KV head); its
// K/V tiles are streamed from the pool exactly once for all the queries of the tile.
//
// The kernel is persistent, two CTAs per SM, each a producer warp and four MMA warps around a 3-stage
// shared-memory ring of 64-token K|V tiles (192 KB per SM for head_dim 128).  Two producers per SM
// matter: one thread issuing every stage of an SM (header, bookkeeping, waits) was the pace setter.
// A CTA is launched as two warpgroups of 128 registers per thread and re-divides them: the MMA
// warpgroup runs with 216, the producer's with 40 (see the kernel).
//
//   MMA warps     : a warp owns 16 stacked query rows (request x GQA head) of one unit for the
//                   unit's whole chunk, so (O, m, l) never leave its registers and no warp ever
//                   waits for another: S^T = K * Q^T with tokens as the MMA M dimension and the
//                   query rows as N (query fragments come straight from global memory), online
//                   softmax on the fp32 scores with warp shuffles across the token lanes,
//                   O^T += V^T * P^T with P transposed in registers (movmatrix); at the end of the
//                   chunk the fp32 partial goes from registers to global memory in full 32-byte
//                   sectors.  A unit with up to 64 rows occupies 1..4 warps; up to eight units are
//                   in progress per SM (four per CTA), so one unit's start-up and write-back overlap the others.
//   producer warp : takes units from a global counter (item order: the long, heavily shared
//                   segments come first) when a warp is free or about to be, assigns each to free
//                   MMA warps, and issues the tiles of
//                   all units in progress round-robin as cp.async.bulk (TMA engine) copies,
//                   completion counted in bytes on mbarriers.  Every stage carries a header: the
//                   warps that consume it and the unit's geometry.  All four warps pass every
//                   stage in ring order (the ones it is not meant for just release it).
#include "attn_core.cuh"

namespace gf {
namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kDecodeThreads = 256;  // warps 0-3: MMA (one warpgroup), warp 4: producer, warps 5-7: give their registers away
constexpr int kProducerRegs = 40;    // registers per thread the second warpgroup keeps
constexpr int kConsumerRegs = 216;   // and what the MMA warpgroup grows to: 128 + (128 - 40)
constexpr int kClaimTiles = 3;  // a unit this close to its end lets the producer claim the next one

struct DecodeParams {
  const char* pool_layer;
  uint64_t head_stride;
  uint32_t tile_bytes;
  const Item* items;
  const int32_t* grp_req;
  const __nv_bfloat16* q;
  float* part_o;
  float* part_ml;
  int32_t* status;
  int32_t* counters;  // [0] next unit, [1] CTAs finished; both zero between launches
  const Header* hdr;  // table sizes and validity, read on the device (the host may not know them yet)
  int32_t slot_cap;
  int32_t num_q_heads, num_kv_heads, gqa;
  float scale_log2;
  const ResidualEntry* residuals;  // this layer's rows of the residual table (null: no node has one)
  int32_t cap_tiles, num_pairs, num_requests;  // sizes that table-derived indices are checked against (debug build)
  int32_t yield_sms;  // CTAs on a multiprocessor with an id below this leave at once (see launch_decode)
};

struct __align__(16) StageHeader {
  int32_t mask;  // bits 0..3: consumer warps this tile is for (0: no more work); bits 8..: 1 + row of the
                 // residual table to apply to the tile before use (0: none)
  int32_t tile, ntile;
  int32_t kvh;   // bits 0..7: KV head; bits 8..: first token of the unit's chunk inside its node, in tiles
  int32_t grp_begin, grp_count, part_base, tok_count;
};

// One unit in progress, as the producer sees it.
struct Stream {
  int32_t mask, t, ntile, kvh;
  int32_t grp_begin, grp_count, part_base, tok_count;
  int32_t tile0, res, tok_begin, pad2;
};

// Eq. 7 on a tile in shared memory: rows [0, nv) of the staged K and V blocks of one KV head become
// base + residual, every marked entry the bf16 sum rounded once (nearest even), like
// gf_node_kv_reconstruct writes it to the pool, so that attention over either is the same bit for bit.
// One warp.  What costs here is the latency of dependent global loads (bitmap and row start, then the
// values they point to), so they are issued in two waves: first the bitmaps and row starts of all of
// the tile's rows (both tensors) into a scratch area in shared memory, then, eight row passes at a
// time, every value those passes need, before any of them is used.  head_dim / 8 lanes share a row (a
// 16-byte chunk, eight entries, each).  A value index outside [0, nnz) is not read and is reported.
constexpr int kPatchRows = 2 * kTile;  // K rows then V rows of one tile
struct PatchScratch {
  uint32_t bm[kPatchRows][4];  // bitmap words of the row (head_dim / 32 of them are used)
  int32_t rp[kPatchRows];      // index of the row's first value
};

template <int D>
__device__ __forceinline__ void apply_residual(unsigned char* stage, PatchScratch* sc, const ResidualEntry& e, int tok0,
                                               int nv, int kvh, int num_kv_heads, int lane, int32_t* status) {
  constexpr int kWords = D / 32, kLanesPerRow = D / 8, kRowsPerPass = 32 / kLanesPerRow;
  constexpr uint32_t kBlk = (D / 64) * kTile * 128;
  constexpr int kBatch = 8;  // row passes whose values are requested together
  // ---- wave 1: bitmaps and row starts of every row of the tile
  for (int i = lane; i < kPatchRows; i += 32) {
    const int which = i / kTile, r = i % kTile;
    const uint32_t* bitmap = which ? e.v_bitmap : e.k_bitmap;
    const int32_t* row_ptr = which ? e.v_row_ptr : e.k_row_ptr;
    const bool on = r < nv && bitmap != nullptr && (which ? e.v_nnz : e.k_nnz) >= 0;
    const long long grow = (long long)(tok0 + r) * num_kv_heads + kvh;  // row of the node's [tokens x heads, D] tensor
#pragma unroll
    for (int x = 0; x < 4; ++x) sc->bm[i][x] = (on && x < kWords) ? bitmap[grow * kWords + x] : 0u;
    const int first = on ? row_ptr[grow] : 0;
    sc->rp[i] = first;
    // ask for the row's values now (they span at most head_dim entries: three 128-byte lines), so that
    // all rows' requests are under way together; wave 2 then finds them in L2
    if (on) {
      const uint16_t* v0 = (which ? e.v_values : e.k_values) + first;
      asm volatile("prefetch.global.L2 [%0];" ::"l"(v0));
      asm volatile("prefetch.global.L2 [%0];" ::"l"(v0 + 64));
    }
  }
  __syncwarp();
  // ---- wave 2: the values, kBatch passes at a time, then the sums
  const int sub = lane % kLanesPerRow, rsub = lane / kLanesPerRow;
  const int w = sub >> 2;
  const uint32_t sh = ((uint32_t)sub & 3u) * 8u;
  bool bad = false;
  const int passes = 2 * kTile / kRowsPerPass;  // over K then V
  for (int p0 = 0; p0 < passes; p0 += kBatch) {
    uint32_t d[kBatch][4];
    uint32_t todo = 0u;  // bit b: pass b has entries to add in this lane's chunk
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int i = (p0 + b) * kRowsPerPass + rsub;  // row of the scratch area: K rows, then V rows
      const int nnz = (i / kTile) ? e.v_nnz : e.k_nnz;
      const uint16_t* values = (i / kTile) ? e.v_values : e.k_values;
      const uint32_t bits = (sc->bm[i][w] >> sh) & 0xffu;
      int at = sc->rp[i];
#pragma unroll
      for (int x = 0; x < kWords; ++x)
        if (x < w) at += __popc(sc->bm[i][x]);
      at += __popc(sc->bm[i][w] & ((1u << sh) - 1u));
      if (bits != 0u) todo |= 1u << b;
      // Branch-free: entry k's value sits at `at` + (number of marked entries below k); every lane
      // requests all eight (clamped into the array) so that the loads of the whole batch are in flight
      // together, and keeps -0, which leaves an entry as it is, where entry k is not marked.
      uint32_t v[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        const int idx = at + __popc(bits & ((1u << k) - 1u));
        const bool marked = (bits >> k) & 1u;
        if (marked && (idx < 0 || idx >= nnz)) bad = true;
        v[k] = (nnz > 0) ? (uint32_t)values[min(max(idx, 0), nnz - 1)] : 0x8000u;
        v[k] = (marked && idx >= 0 && idx < nnz) ? v[k] : 0x8000u;
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) d[b][k] = v[2 * k] | (v[2 * k + 1] << 16);
    }
    if (todo == 0u) continue;
#pragma unroll
    for (int b = 0; b < kBatch; ++b) {
      const int i = (p0 + b) * kRowsPerPass + rsub;
      if (!((todo >> b) & 1u)) continue;
      unsigned char* blk = stage + (i / kTile) * kBlk;
      uint4* cell = reinterpret_cast<uint4*>(blk + (uint32_t)(sub >> 3) * (kTile * 128u) +
                                             swz128((uint32_t)(i % kTile), (uint32_t)sub & 7u));
      uint4 c = *cell;
      asm("add.rn.bf16x2 %0, %0, %1;" : "+r"(c.x) : "r"(d[b][0]));
      asm("add.rn.bf16x2 %0, %0, %1;" : "+r"(c.y) : "r"(d[b][1]));
      asm("add.rn.bf16x2 %0, %0, %1;" : "+r"(c.z) : "r"(d[b][2]));
      asm("add.rn.bf16x2 %0, %0, %1;" : "+r"(c.w) : "r"(d[b][3]));
      *cell = c;
    }
  }
  if (bad) atomicCAS(status + kStatusReport, 0, (int32_t)GF_ERR_INVALID_ARG);
}

// kRes: some node of the batch may be kept as base + residual (the tiles of such segments are completed
// in shared memory before use); the kernel without it carries none of that machinery.
template <int D, bool kRes>
__global__ void __launch_bounds__(kDecodeThreads, 2) k_decode(const DecodeParams p) {
  constexpr int CB = D / 64;                   // 128-byte column blocks per row
  constexpr uint32_t kBlk = CB * kTile * 128;  // bytes of one K (or V) block
  constexpr uint32_t kStageBytes = 2 * kBlk;

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stage_mem = smem;
  StageHeader* hdr = reinterpret_cast<StageHeader*>(smem + kStages * kStageBytes);
  Stream* streams = reinterpret_cast<Stream*>(hdr + kStages);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(streams + kConsumerWarps);
  uint64_t* empty_bar = full_bar + kStages;
  uint64_t* ready_bar = empty_bar + kStages;  // the tile's residual (if any) has been applied
  PatchScratch* patch = reinterpret_cast<PatchScratch*>(ready_bar + kStages + 1);  // one per MMA warp

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = p.gqa;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
      if (kRes) mbar_init(&ready_bar[s], 1);
    }
    mbar_fence_init();
  }
  chain_enter();  // nothing above touches global memory
  __syncthreads();

  // Multiprocessors with an id below yield_sms are left to the tensor-memory decode kernel, which runs
  // beside this one on another stream: a CTA that finds itself there only counts itself as finished.
  // Which CTAs leave does not matter for the result (the others take every unit from the counter).
  if (p.yield_sms > 0) {
    uint32_t smid;
    asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
    if ((int)smid < p.yield_sms) {
      if (threadIdx.x == 0) {
        __threadfence();
        if (atomicAdd(&p.counters[1], 1) == (int)gridDim.x - 1) {
          p.counters[0] = 0;
          p.counters[1] = 0;
        }
      }
      return;
    }
  }

  // The launch gives every thread 128 registers (two CTAs of 256 threads fill the register file).
  // The second warpgroup (the producer warp and three warps that have nothing else to do) keeps 40 of
  // them; the MMA warpgroup takes what that frees: with 216 registers the loads of the next MMAs are
  // in flight while the current ones issue, which the 168 a five-warp CTA allows did not permit (a
  // 64-token step of a 16-row group takes 1.6 K cycles instead of 2.9 K).  Every warp of a warpgroup
  // executes the same instruction, once; 4 * 32 * (40 + 216) = the CTA's 32 768 registers.
  if (warp >= kConsumerWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kProducerRegs));
    // ------------------------------- producer -------------------------------
    if (warp == kConsumerWarps && lane == 0) {
      const int num_units = tables_usable(*p.hdr, p.slot_cap) ? p.hdr->num_items * p.num_kv_heads : 0;
      int n = 0;                                            // stages issued so far
      uint32_t free_mask = (1u << kConsumerWarps) - 1, live_mask = 0;  // live: indexed by a unit's lowest warp
      // A unit is claimed (one atomic on the global counter) only when a warp is free or about to be:
      // a CTA busy with long chunks must not sit on units that an idle CTA could run.  The claim is
      // spread over passes of the loop below so that neither the counter's round trip nor the item's
      // load is waited for: pass k issues the atomic, pass k+1 reads its result and requests the item,
      // pass k+2 hands the unit to free warps.  Chunks flagged wide belong to the tensor-memory kernel
      // and are skipped.
      Item it;
      int u = 0;
      int claim = 0;           // 0: nothing claimed, 1: counter asked, 2: item requested
      bool exhausted = false;  // the counter has run past the last unit
      bool soon = true;        // a warp is free, or a unit in progress is within kClaimTiles of its end
      while (true) {
        if (claim == 2) {
          if (it.pad & 1) {
            u = atomicAdd(&p.counters[0], 1);
            claim = 1;
          } else {
            const int need = (it.grp_count * g + 15) >> 4;
            if (__popc(free_mask) >= need) {
              uint32_t mask = 0;
              for (int k = 0; k < need; ++k) {
                const uint32_t bit = free_mask & (0u - free_mask);
                mask |= bit;
                free_mask ^= bit;
              }
              const int slot = __ffs(mask) - 1;
              Stream sm;
              sm.mask = (int32_t)mask; sm.t = 0; sm.ntile = (it.tok_count + kTile - 1) / kTile;
              sm.kvh = u % p.num_kv_heads;
              sm.grp_begin = it.grp_begin; sm.grp_count = it.grp_count; sm.part_base = it.part_base;
              sm.tok_count = it.tok_count; sm.tile0 = it.tile0; sm.pad2 = 0;
              sm.res = (it.pad >> 8) - 1; sm.tok_begin = it.tok_begin;
              streams[slot] = sm;
              live_mask |= 1u << slot;
              claim = 0;
              soon = soon || free_mask != 0 || sm.ntile <= kClaimTiles;
            }
          }
        } else if (claim == 1) {
          if (u >= num_units) {
            exhausted = true;
            claim = 0;
          } else {
            it = p.items[GF_CLAMP(u / p.num_kv_heads, p.slot_cap, p.status, 101)];
            claim = 2;
          }
        }
        if (claim == 0 && !exhausted && soon) {
          u = atomicAdd(&p.counters[0], 1);
          claim = 1;
        }
        if (live_mask == 0) {
          if (exhausted && claim == 0) break;  // nothing in progress and nothing left
          continue;
        }
        // one tile of every unit in progress
        soon = free_mask != 0;
        for (uint32_t rest = live_mask; rest != 0; rest &= rest - 1) {
          const int slot = __ffs(rest) - 1;
          Stream sm = streams[slot];
          const int st = n % kStages;
          if (n >= kStages) mbar_wait(&empty_bar[st], ((n / kStages) - 1) & 1, p.status);
          StageHeader h;
          h.mask = sm.mask; h.tile = sm.t; h.ntile = sm.ntile; h.kvh = sm.kvh;
          h.grp_begin = sm.grp_begin; h.grp_count = sm.grp_count; h.part_base = sm.part_base;
          h.tok_count = sm.tok_count;
          if (kRes) {
            h.mask |= (sm.res + 1) << 8;
            h.kvh |= (sm.tok_begin / kTile) << 8;
          }
          hdr[st] = h;
          const int nv = min(kTile, sm.tok_count - sm.t * kTile);
          const int rf = min(kTile, (nv + 15) & ~15);
          unsigned char* dst = stage_mem + st * kStageBytes;
          const char* src = p.pool_layer + (uint64_t)sm.kvh * p.head_stride +
                            (uint64_t)GF_CLAMP(sm.tile0 + sm.t, p.cap_tiles, p.status, 102) * p.tile_bytes;
          if (rf == kTile) {
            mbar_arrive_expect_tx(&full_bar[st], kStageBytes);
            bulk_g2s(dst, src, kStageBytes, &full_bar[st]);
          } else {
            mbar_arrive_expect_tx(&full_bar[st], 2u * CB * rf * 128u);
#pragma unroll
            for (int b = 0; b < 2 * CB; ++b)
              bulk_g2s(dst + b * (kTile * 128), src + b * (kTile * 128), rf * 128u, &full_bar[st]);
          }
          ++n;
          if (++sm.t == sm.ntile) {
            live_mask &= ~(1u << slot);
            free_mask |= (uint32_t)sm.mask;
            soon = true;
          } else {
            streams[slot].t = sm.t;
            soon = soon || sm.ntile - sm.t <= kClaimTiles;
          }
        }
      }
      const int st = n % kStages;
      if (n >= kStages) mbar_wait(&empty_bar[st], ((n / kStages) - 1) & 1, p.status);
      StageHeader h{};
      hdr[st] = h;  // mask 0: stop
      mbar_arrive(&full_bar[st]);
      // the last CTA to run out of work re-arms the counters for the next launch
      __threadfence();
      if (atomicAdd(&p.counters[1], 1) == (int)gridDim.x - 1) {
        p.counters[0] = 0;
        p.counters[1] = 0;
      }
    }
    return;
  }

  // ------------------------------- MMA warps -------------------------------
  asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kConsumerRegs));
  WarpAttn<D> wa;
  int rows_here = 0;  // query rows of this warp's 16-row group that exist
  int row0 = 0;       // first stacked row of the group inside the item
  for (int n = 0;; ++n) {
    const int st = n % kStages;
    if (!mbar_wait(&full_bar[st], (n / kStages) & 1, p.status)) break;
    StageHeader h = hdr[st];
    if (h.mask == 0) break;
    const int res = kRes ? (h.mask >> 8) - 1 : -1;
    const int tok0 = kRes ? ((h.kvh >> 8) + h.tile) * kTile : 0;
    if (kRes) { h.mask &= 0xff; h.kvh &= 0xff; }
    const bool mine = (h.mask >> warp) & 1;
    if (mine && kRes) {
      // Differential KV inside the stream (Sec. 5.1, Eq. 7): the tile that arrived is the base node's; a
      // segment whose state is base + sparse residual is completed here, in shared memory, by the
      // unit's first warp, and the unit's other warps wait until that is done.  Every use of a stage
      // completes one phase of its ready barrier (the first warp arrives whether it patched or not).
      const bool first = (h.mask & ((1 << warp) - 1)) == 0;
      if (first) {
        if (res >= 0) {
          const int nvp = min(kTile, h.tok_count - h.tile * kTile);
          apply_residual<D>(stage_mem + st * kStageBytes, patch + warp, p.residuals[res], tok0, nvp, h.kvh,
                            p.num_kv_heads, lane, p.status);
          __syncwarp();
        }
        if (lane == 0) mbar_arrive(&ready_bar[st]);
      } else if (res >= 0) {
        mbar_wait(&ready_bar[st], (n / kStages) & 1, p.status);
      }
    }
    if (mine) {
      if (h.tile == 0) {
        // ---- begin a unit: this warp's row group, query fragments from global memory ----
        const int rg = __popc(h.mask & ((1 << warp) - 1));
        row0 = rg * 16;
        rows_here = min(16, h.grp_count * g - row0);
        wa.init();
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int row = j * 8 + (lane >> 2);
          const bool ok = row < rows_here;
          int req = ok ? p.grp_req[GF_CLAMP(h.grp_begin + (row0 + row) / g, p.num_pairs, p.status, 103)] : 0;
          req = GF_CLAMP(req, p.num_requests, p.status, 104);
          const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
              p.q + ((size_t)req * p.num_q_heads + h.kvh * g + (row0 + row) % g) * D);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            wa.qf[j][ks][0] = ok ? qrow[ks * 8 + (lane & 3)] : 0u;
            wa.qf[j][ks][1] = ok ? qrow[ks * 8 + 4 + (lane & 3)] : 0u;
          }
        }
      }
      const int nv = min(kTile, h.tok_count - h.tile * kTile);
      const uint32_t kb = smem_u32(stage_mem + st * kStageBytes), vb = kb + kBlk;
      if (rows_here <= 8) {
        if (nv == kTile) wa.template step<4, 1, false>(kb, vb, 0, nv, p.scale_log2, lane);
        else wa.template step<4, 1, true>(kb, vb, 0, nv, p.scale_log2, lane);
      } else {
        if (nv == kTile) wa.template step<4, 2, false>(kb, vb, 0, nv, p.scale_log2, lane);
        else wa.template step<4, 2, true>(kb, vb, 0, nv, p.scale_log2, lane);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[st]);
    if (!mine || h.tile != h.ntile - 1) continue;

    // ---- end of the unit: registers -> fp32 partials ----
    wa.finish_sums();
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int row = j * 8 + (lane & 3) * 2 + c;
        if (row < rows_here && GF_CHECK(h.part_base + (row0 + row) / g < p.slot_cap, p.status, 105)) {
          const int srow = row0 + row;
          const size_t ph = (size_t)(h.part_base + srow / g) * p.num_q_heads + h.kvh * g + srow % g;
          float* po = p.part_o + ph * D + (lane >> 2);
#pragma unroll
          for (int i = 0; i < D / 16; ++i) {
            po[i * 16] = wa.o[i][j][c];
            po[i * 16 + 8] = wa.o[i][j][2 + c];
          }
          if ((lane >> 2) == 0)
            *reinterpret_cast<float2*>(p.part_ml + ph * 2) = make_float2(wa.m_run[j][c], wa.l_run[j][c]);
        }
      }
  }
}

// K4.  One warp per (request, query head): out = sum_i w_i o_i / sum_i w_i l_i with
// w_i = 2^(m_i - max m) over the request's partial slots; lse in natural-log units.
template <int D>
__global__ void __launch_bounds__(256) k_merge(const float* __restrict__ part_o,
                                               const float* __restrict__ part_ml,
                                               const int32_t* __restrict__ mrg_ptr,
                                               const int32_t* __restrict__ mrg_slot, int num_requests,
                                               int num_q_heads, __nv_bfloat16* __restrict__ out,
                                               float* __restrict__ lse, const Header* __restrict__ hdr,
                                               int slot_cap, int32_t* status) {
  chain_enter();
  if (!tables_usable(*hdr, slot_cap)) return;
  const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (gw >= num_requests * num_q_heads) return;
  const int r = gw / num_q_heads, h = gw % num_q_heads;
  int b = mrg_ptr[r], e = mrg_ptr[r + 1];
  if (!GF_CHECK(b >= 0 && b <= e && e <= slot_cap, status, 110)) e = b = 0;
  constexpr int kLanes = D / 4;  // lanes that carry output columns
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float L = 0.f, M = -INFINITY;
  // 32 slots at a time: lane i fetches slot index and (m, l) of the i-th; the maximum of the batch is
  // folded into the running one, then the partial rows are read four at a time (independent loads).
  for (int base = b; base < e; base += 32) {
    const int cnt = min(32, e - base);
    int slot = 0;
    float2 ml = make_float2(-INFINITY, 0.f);
    if (lane < cnt) {
      slot = mrg_slot[base + lane];
      slot = GF_CLAMP(slot, slot_cap, status, 111);
      ml = *reinterpret_cast<const float2*>(part_ml + ((size_t)slot * num_q_heads + h) * 2);
    }
    float mb = ml.x;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) mb = fmaxf(mb, __shfl_xor_sync(0xffffffffu, mb, d));
    const float Mn = fmaxf(M, mb);
    const float resc = (M == -INFINITY) ? 0.f : fast_exp2(M - Mn);
    acc.x *= resc; acc.y *= resc; acc.z *= resc; acc.w *= resc;
    L *= resc;
    M = Mn;
    const float wl = (ml.x == -INFINITY) ? 0.f : fast_exp2(ml.x - M);
    float lsum = wl * ml.y;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) lsum += __shfl_xor_sync(0xffffffffu, lsum, d);
    L += lsum;
    for (int i0 = 0; i0 < cnt; i0 += 4) {
      float4 v[4];
      float w[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int i = min(i0 + k, cnt - 1);
        const int sl = __shfl_sync(0xffffffffu, slot, i);
        w[k] = (i0 + k < cnt) ? __shfl_sync(0xffffffffu, wl, i) : 0.f;
        v[k] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (lane < kLanes)
          v[k] = *reinterpret_cast<const float4*>(part_o + ((size_t)sl * num_q_heads + h) * D + lane * 4);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        acc.x += w[k] * v[k].x; acc.y += w[k] * v[k].y; acc.z += w[k] * v[k].z; acc.w += w[k] * v[k].w;
      }
    }
  }
  const float inv = (L > 0.f) ? 1.f / L : 0.f;
  if (lane < kLanes) {
    uint2 packed;
    packed.x = pack_bf16(acc.x * inv, acc.y * inv);
    packed.y = pack_bf16(acc.z * inv, acc.w * inv);
    *reinterpret_cast<uint2*>(out + ((size_t)r * num_q_heads + h) * D + lane * 4) = packed;
  }
  if (lse != nullptr && lane == 0)
    lse[(size_t)r * num_q_heads + h] = (L > 0.f) ? (M + log2f(L)) * 0.6931471805599453f : -INFINITY;
}

template <int D, bool kRes>
constexpr size_t decode_smem_bytes() {
  return (size_t)kStages * 2 * (D / 64) * kTile * 128 + kStages * sizeof(StageHeader) +
         kConsumerWarps * sizeof(Stream) + 3 * kStages * 8 + 8 + (kRes ? kConsumerWarps * sizeof(PatchScratch) : 0);
}

// CTAs of the persistent grid: two per SM of the current device.
int decode_grid_limit() {
  static int cached[kMaxDevices] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 2 * 148;
  if (cached[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    cached[dev] = 2 * sms;
  }
  return cached[dev];
}

}  // namespace

int launch_decode(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int num_items,
                  int layer, const void* q, int32_t* status, int yield_sms, const ResidualEntry* residuals,
                  cudaStream_t st) {
  if (num_items == 0) return 0;  // num_items < 0: not known on the host, the kernel reads it
  DecodeParams p;
  p.pool_layer = pool.base + (uint64_t)layer * pool.layer_stride;
  p.head_stride = pool.head_stride;
  p.tile_bytes = pool.tile_bytes;
  p.items = t.items;
  p.grp_req = t.grp_req;
  p.q = (const __nv_bfloat16*)q;
  p.part_o = t.part_o;
  p.part_ml = t.part_ml;
  p.status = status;
  p.counters = status + kStatusDecodeQueue;
  p.hdr = t.hdr;
  p.slot_cap = t.slot_cap;
  p.residuals = residuals;
  p.cap_tiles = (int32_t)pool.cap_tiles;
  p.num_pairs = t.num_pairs_in;
  p.num_requests = t.num_requests;
  const long long units = num_items < 0 ? (1ll << 40) : (long long)num_items * sh.num_kv_heads;
  p.num_q_heads = sh.num_q_heads;
  p.num_kv_heads = sh.num_kv_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  const int limit = decode_grid_limit();
  dim3 grid((unsigned)(units < limit ? units : limit), 1, 1);
  // multiprocessors are only given away by a grid that fills the whole GPU (two CTAs on every one)
  p.yield_sms = ((int)grid.x == limit && yield_sms > 0 && 2 * yield_sms < limit) ? yield_sms : 0;
  auto go = [&](auto kernel, size_t smem, bool (&optin)[kMaxDevices]) {
    if (!ensure_dynamic_smem(kernel, smem, optin)) return false;
    launch_chained(kernel, grid, dim3(kDecodeThreads), smem, st, p);
    return true;
  };
  static bool optin[4][kMaxDevices] = {};
  bool ok;
  if (sh.head_dim == 128)
    ok = residuals ? go(k_decode<128, true>, decode_smem_bytes<128, true>(), optin[0])
                   : go(k_decode<128, false>, decode_smem_bytes<128, false>(), optin[1]);
  else
    ok = residuals ? go(k_decode<64, true>, decode_smem_bytes<64, true>(), optin[2])
                   : go(k_decode<64, false>, decode_smem_bytes<64, false>(), optin[3]);
  if (!ok) return -1;
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_merge(const AttnShape& sh, const TablesDev& t, void* out, float* lse, bool chained, cudaStream_t st) {
  const long long warps = (long long)t.num_requests * sh.num_q_heads;
  if (warps <= 0) return 0;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  auto go = [&](auto kernel) {
    if (chained)
      launch_chained(kernel, dim3(blocks), dim3(256), 0, st, t.part_o, t.part_ml, t.mrg_ptr, t.mrg_slot, t.num_requests,
                     sh.num_q_heads, (__nv_bfloat16*)out, lse, t.hdr, t.slot_cap, t.status);
    else  // behind a join with another stream: must not be scheduled before that join is through
      kernel<<<dim3(blocks), dim3(256), 0, st>>>(t.part_o, t.part_ml, t.mrg_ptr, t.mrg_slot, t.num_requests, sh.num_q_heads,
                                                 (__nv_bfloat16*)out, lse, t.hdr, t.slot_cap, t.status);
  };
  if (sh.head_dim == 128) go(k_merge<128>);
  else go(k_merge<64>);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
