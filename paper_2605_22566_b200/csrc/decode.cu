// K2: shared-segment decode, and K4: log-sum-exp merge.
//
// A work item is one chunk of one node's KV segment together with one tile (<= 16) of the
// requests whose workflow path passes through that node (Sec. 5: the node's KV state is stored
// once and assembled into every such request's context).  A unit of work is (item, KV head); its
// K/V tiles are streamed from the pool exactly once for all the queries of the tile.
//
// The kernel is persistent: two CTAs per SM, each a producer warp plus four MMA warps around a
// 3-stage shared-memory ring of 64-token K|V tiles.
//
//   producer warp : takes the next unit from a global counter (units in item order, so the long,
//                   heavily shared segments come first), and issues cp.async.bulk (TMA engine)
//                   copies of the unit's tiles, completion counted in bytes on mbarriers.  It
//                   runs ahead across unit boundaries, so tiles of the next unit are already in
//                   flight while the MMA warps finish the previous one.  Each stage carries a
//                   small header (item, tile index, tile count, KV head) for the consumers.
//   4 MMA warps   : S^T = K * Q^T with tokens as the MMA M dimension and the stacked query rows
//                   (request x GQA head) as N, so 1..64 query rows cost 1..8 n-tiles; the query
//                   fragments are loaded straight from global memory into registers;
//                   online softmax on the fp32 scores with warp shuffles across the token lanes;
//                   O^T += V^T * P^T with P transposed in registers (movmatrix).
//   unit epilogue : warps that split the tokens of a tile combine their (O, m, l) through a small
//                   scratch area; the result goes from registers to the fp32 partials in full
//                   32-byte sectors.
//
// Warps split the work by rows when the tile is large (each warp owns 16 query rows) and by tokens
// when it is small (each warp owns a slice of every 64-token tile).
#include "attn_core.cuh"

namespace gf {
namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;
constexpr int kScratchBytes = 2 * 40 * 128;  // two warps x (32 O registers + 4 m + 4 l) x 32 lanes x 4 B

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
  int32_t num_units, num_q_heads, num_kv_heads, gqa;
  float scale_log2;
};

struct StageHeader {
  int32_t item, tile, ntile, kvh;  // item < 0: no more work
};

__device__ __forceinline__ void consumer_bar_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kDecodeThreads, 2) k_decode(const DecodeParams p) {
  constexpr int CB = D / 64;                   // 128-byte column blocks per row
  constexpr uint32_t kBlk = CB * kTile * 128;  // bytes of one K (or V) block
  constexpr uint32_t kStageBytes = 2 * kBlk;

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stage_mem = smem;
  float* scratch = reinterpret_cast<float*>(smem + kStages * kStageBytes);
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(smem + kStages * kStageBytes + kScratchBytes);
  uint64_t* empty_bar = full_bar + kStages;
  StageHeader* hdr = reinterpret_cast<StageHeader*>(empty_bar + kStages);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], kConsumerWarps);
    }
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------- producer -------------------------------
    if (lane == 0) {
      int n = 0;  // stages issued so far
      int u = atomicAdd(&p.counters[0], 1);
      Item it;
      if (u < p.num_units) it = p.items[u / p.num_kv_heads];
      while (u < p.num_units) {
        const int kvh = u % p.num_kv_heads;
        const int item = u / p.num_kv_heads;
        const int u_next = atomicAdd(&p.counters[0], 1);
        Item it_next = it;
        if (u_next < p.num_units) it_next = p.items[u_next / p.num_kv_heads];  // in flight during the copies
        const int ntile = (it.tok_count + kTile - 1) / kTile;
        const char* src0 = p.pool_layer + (uint64_t)kvh * p.head_stride + (uint64_t)it.tile0 * p.tile_bytes;
        for (int t = 0; t < ntile; ++t, ++n) {
          const int st = n % kStages;
          if (n >= kStages) mbar_wait(&empty_bar[st], ((n / kStages) - 1) & 1, p.status);
          hdr[st] = StageHeader{item, t, ntile, kvh};
          const int nv = min(kTile, it.tok_count - t * kTile);
          const int rf = min(kTile, (nv + 15) & ~15);
          unsigned char* dst = stage_mem + st * kStageBytes;
          const char* src = src0 + (uint64_t)t * p.tile_bytes;
          if (rf == kTile) {
            mbar_arrive_expect_tx(&full_bar[st], kStageBytes);
            bulk_g2s(dst, src, kStageBytes, &full_bar[st]);
          } else {
            mbar_arrive_expect_tx(&full_bar[st], 2u * CB * rf * 128u);
#pragma unroll
            for (int b = 0; b < 2 * CB; ++b)
              bulk_g2s(dst + b * (kTile * 128), src + b * (kTile * 128), rf * 128u, &full_bar[st]);
          }
        }
        u = u_next;
        it = it_next;
      }
      const int st = n % kStages;
      if (n >= kStages) mbar_wait(&empty_bar[st], ((n / kStages) - 1) & 1, p.status);
      hdr[st] = StageHeader{-1, 0, 0, 0};
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
  const int g = p.gqa;
  WarpAttn<D> wa;
  Item it;
  int rows = 0, nrg = 1, tsplit = 4, rg = 0, tpart = 0, kvh = 0;
  bool active = false;
  const int no_lim[2][2] = {{0, 0}, {0, 0}};
  for (int n = 0;; ++n) {
    const int st = n % kStages;
    if (!mbar_wait(&full_bar[st], (n / kStages) & 1, p.status)) break;
    const StageHeader h = hdr[st];
    if (h.item < 0) break;
    if (h.tile == 0) {
      // ---- begin a unit: shape of the split, query fragments from global memory ----
      it = p.items[h.item];
      kvh = h.kvh;
      rows = it.grp_count * g;          // stacked query rows of this item (<= 64)
      nrg = (rows + 15) >> 4;           // 16-row groups
      tsplit = nrg == 1 ? 4 : (nrg == 2 ? 2 : 1);
      rg = warp / tsplit;
      tpart = warp % tsplit;
      active = rg < nrg;
      wa.init();
      if (active) {
#pragma unroll
        for (int j = 0; j < 2; ++j) {
          const int row = rg * 16 + j * 8 + (lane >> 2);
          const bool ok = row < rows;
          const int req = ok ? p.grp_req[it.grp_begin + row / g] : 0;
          const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
              p.q + ((size_t)req * p.num_q_heads + kvh * g + row % g) * D);
#pragma unroll
          for (int ks = 0; ks < D / 16; ++ks) {
            wa.qf[j][ks][0] = ok ? qrow[ks * 8 + (lane & 3)] : 0u;
            wa.qf[j][ks][1] = ok ? qrow[ks * 8 + 4 + (lane & 3)] : 0u;
          }
        }
      }
    }
    if (active) {
      const int tok_per = kTile / tsplit, t0 = tpart * tok_per;
      const int nv = min(kTile, it.tok_count - h.tile * kTile);
      const uint32_t kb = smem_u32(stage_mem + st * kStageBytes);
      for (int ts = t0; ts < t0 + tok_per && ts < nv; ts += 16)
        wa.template step<false>(kb, kb + kBlk, ts, nv, p.scale_log2, lane, 0, no_lim);
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[st]);
    if (h.tile != h.ntile - 1) continue;

    // ---- end of the unit: combine token-split warps, write the partials ----
    if (active) wa.finish_sums();
    if (tsplit > 1) {
      // round 1: odd token parts hand their state to the even ones; round 2 (4-way split only):
      // part 2 hands its state to part 0.  Each hand-over moves half of O at a time.
      for (int round = 1; round < tsplit; round <<= 1) {
        const bool giver = active && (tpart & (2 * round - 1)) == round;
        const bool taker = active && (tpart & (2 * round - 1)) == 0;
        const int pair = (round == 1) ? (warp >> 1) : 0;  // scratch slot shared by giver and taker
        float* slot = scratch + pair * (40 * 32);
#pragma unroll
        for (int half = 0; half < 2; ++half) {
          if (giver) wa.hand_over(slot, half, lane);
          consumer_bar_sync();
          if (taker) wa.take_over(slot, half, lane);
          consumer_bar_sync();
        }
      }
    }
    if (active && tpart == 0) {
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int row = rg * 16 + j * 8 + (lane & 3) * 2 + c;
          if (row < rows) {
            const size_t ph = (size_t)(it.part_base + row / g) * p.num_q_heads + kvh * g + row % g;
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
}

// K4.  One warp per (request, query head): out = sum_i w_i o_i / sum_i w_i l_i with
// w_i = 2^(m_i - max m) over the request's partial slots; lse in natural-log units.
template <int D>
__global__ void __launch_bounds__(256) k_merge(const float* __restrict__ part_o,
                                               const float* __restrict__ part_ml,
                                               const int32_t* __restrict__ mrg_ptr,
                                               const int32_t* __restrict__ mrg_slot, int num_requests,
                                               int num_q_heads, __nv_bfloat16* __restrict__ out,
                                               float* __restrict__ lse) {
  const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (gw >= num_requests * num_q_heads) return;
  const int r = gw / num_q_heads, h = gw % num_q_heads;
  const int b = mrg_ptr[r], e = mrg_ptr[r + 1];
  float M = -INFINITY;
  for (int i = b + lane; i < e; i += 32)
    M = fmaxf(M, part_ml[((size_t)mrg_slot[i] * num_q_heads + h) * 2]);
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) M = fmaxf(M, __shfl_xor_sync(0xffffffffu, M, d));
  constexpr int kLanes = D / 4;  // lanes that carry output columns
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float L = 0.f;
  for (int i = b; i < e; ++i) {
    const size_t ph = (size_t)mrg_slot[i] * num_q_heads + h;
    const float2 ml = *reinterpret_cast<const float2*>(part_ml + ph * 2);
    const float w = fast_exp2(ml.x - M);
    L += w * ml.y;
    if (lane < kLanes) {
      const float4 v = *reinterpret_cast<const float4*>(part_o + ph * D + lane * 4);
      acc.x += w * v.x; acc.y += w * v.y; acc.z += w * v.z; acc.w += w * v.w;
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

template <int D>
constexpr size_t decode_smem_bytes() {
  return (size_t)kStages * 2 * (D / 64) * kTile * 128 + kScratchBytes + 2 * kStages * 8 +
         kStages * sizeof(StageHeader);
}

// CTAs of the persistent grid: two per SM of the current device.
int decode_grid_limit() {
  static int cached[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 2 * 148;
  if (cached[dev] == 0) {
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    cached[dev] = 2 * sms;
  }
  return cached[dev];
}

}  // namespace

int launch_decode(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int num_items,
                  int layer, const void* q, int32_t* status, cudaStream_t st) {
  if (num_items <= 0) return 0;
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
  p.counters = status + 4;
  p.num_units = num_items * sh.num_kv_heads;
  p.num_q_heads = sh.num_q_heads;
  p.num_kv_heads = sh.num_kv_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  const int limit = decode_grid_limit();
  dim3 grid((unsigned)(p.num_units < limit ? p.num_units : limit), 1, 1);
  cudaError_t err;
  if (sh.head_dim == 128) {
    static bool attr_done = false;
    if (!attr_done) {
      err = cudaFuncSetAttribute(k_decode<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)decode_smem_bytes<128>());
      if (err != cudaSuccess) return -1;
      attr_done = true;
    }
    k_decode<128><<<grid, kDecodeThreads, decode_smem_bytes<128>(), st>>>(p);
  } else {
    static bool attr_done = false;
    if (!attr_done) {
      err = cudaFuncSetAttribute(k_decode<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)decode_smem_bytes<64>());
      if (err != cudaSuccess) return -1;
      attr_done = true;
    }
    k_decode<64><<<grid, kDecodeThreads, decode_smem_bytes<64>(), st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_merge(const AttnShape& sh, const TablesDev& t, void* out, float* lse, cudaStream_t st) {
  const long long warps = (long long)t.num_requests * sh.num_q_heads;
  if (warps <= 0) return 0;
  const unsigned blocks = (unsigned)((warps * 32 + 255) / 256);
  if (sh.head_dim == 128)
    k_merge<128><<<blocks, 256, 0, st>>>(t.part_o, t.part_ml, t.mrg_ptr, t.mrg_slot, t.num_requests,
                                         sh.num_q_heads, (__nv_bfloat16*)out, lse);
  else
    k_merge<64><<<blocks, 256, 0, st>>>(t.part_o, t.part_ml, t.mrg_ptr, t.mrg_slot, t.num_requests,
                                        sh.num_q_heads, (__nv_bfloat16*)out, lse);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
