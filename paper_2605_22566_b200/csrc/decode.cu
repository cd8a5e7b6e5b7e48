// K2: shared-segment decode, and K4: log-sum-exp merge.
//
// A work item is one chunk of one node's KV segment together with one tile (<= 16) of the
// requests whose workflow path passes through that node (Sec. 5: the node's KV state is stored
// once and assembled into every such request's context).  One CTA per (item, KV head) streams the
// chunk's K/V tiles from the pool exactly once, for all the queries of the tile:
//
//   producer warp : cp.async.bulk (TMA) of 64-token K|V tiles into a 3-stage shared-memory ring,
//                   completion counted in bytes on mbarriers (only the rows that exist are copied);
//   4 MMA warps   : S^T = K * Q^T with tokens as the MMA M dimension and the stacked query rows
//                   (request x GQA head) as N, so 1..64 query rows cost 1..8 n-tiles;
//                   online softmax on the fp32 scores with warp shuffles across the token lanes;
//                   O^T += V^T * P^T with P transposed in registers (movmatrix);
//   epilogue      : the warps' partial (O, m, l) are combined through shared memory and written as
//                   one fp32 partial per (slot, query head) with 16-byte stores.
//
// Warps split the work by rows when the tile is large (each warp owns 16 query rows) and by tokens
// when it is small (each warp owns a slice of every 64-token tile).
#include "attn_core.cuh"

namespace gf {
namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kDecodeThreads = (kConsumerWarps + 1) * 32;

struct DecodeParams {
  const char* pool_layer;
  uint64_t head_stride;
  uint32_t tile_bytes;
  const Item* items;
  const int32_t* seg_off;
  const int32_t* grp_req;
  const __nv_bfloat16* q;
  float* part_o;
  float* part_ml;
  int32_t* status;
  int32_t num_q_heads, gqa;
  float scale_log2;
};

__device__ __forceinline__ void consumer_bar_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kDecodeThreads, 2) k_decode(const DecodeParams p) {
  constexpr int CB = D / 64;                   // 128-byte column blocks per row
  constexpr uint32_t kBlk = CB * kTile * 128;  // bytes of one K (or V) block
  constexpr uint32_t kStageBytes = 2 * kBlk;
  constexpr int kORow = D + 4;                 // padded fp32 row of the combine scratch

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stage_mem = smem;
  unsigned char* q_mem = smem + kStages * kStageBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(q_mem + kBlk);
  uint64_t* empty_bar = full_bar + kStages;

  const Item it = p.items[blockIdx.x];
  const int kvh = blockIdx.y;
  const int g = p.gqa;
  const int rows = it.grp_count * g;           // stacked query rows of this item (<= 64)
  const int nrg = (rows + 15) >> 4;            // 16-row groups
  const int tsplit = nrg == 1 ? 4 : (nrg == 2 ? 2 : 1);
  const int nactive = nrg * tsplit;            // MMA warps with work (3 or 4)
  const int ntile = (it.tok_count + kTile - 1) / kTile;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], nactive);
    }
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    // ------------------------------- producer -------------------------------
    if (lane == 0) {
      const char* src0 = p.pool_layer + (uint64_t)kvh * p.head_stride +
                         (uint64_t)((p.seg_off[it.seg] + it.tok_begin) / kTile) * p.tile_bytes;
      for (int t = 0; t < ntile; ++t) {
        const int st = t % kStages;
        if (t >= kStages) mbar_wait(&empty_bar[st], ((t / kStages) - 1) & 1, p.status);
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
    }
    return;
  }

  // ------------------------------- MMA warps -------------------------------
  // Stage the item's query rows in shared memory (16-byte loads), swizzled like a K block.
  for (int idx = threadIdx.x; idx < nrg * 16 * (D / 8); idx += kConsumerWarps * 32) {
    const int row = idx / (D / 8), c = idx % (D / 8);
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (row < rows) {
      const int req = p.grp_req[it.grp_begin + row / g];
      const int head = kvh * g + row % g;
      val = *reinterpret_cast<const uint4*>(p.q + ((size_t)req * p.num_q_heads + head) * D + c * 8);
    }
    *reinterpret_cast<uint4*>(q_mem + (c >> 3) * (kTile * 128) + swz128(row, c & 7)) = val;
  }
  consumer_bar_sync();

  const int rg = warp / tsplit, tpart = warp % tsplit;
  const bool active = rg < nrg;
  const int tok_per = kTile / tsplit, t0 = tpart * tok_per;

  WarpAttn<D> wa;
  wa.init();
  if (active) {
    wa.load_q(smem_u32(q_mem), rg * 16, lane);
    const int no_lim[2][2] = {{0, 0}, {0, 0}};
    for (int t = 0; t < ntile; ++t) {
      const int st = t % kStages;
      mbar_wait(&full_bar[st], (t / kStages) & 1, p.status);
      const int nv = min(kTile, it.tok_count - t * kTile);
      const uint32_t kb = smem_u32(stage_mem + st * kStageBytes);
      for (int ts = t0; ts < t0 + tok_per && ts < nv; ts += 16)
        wa.template step<false>(kb, kb + kBlk, ts, nv, p.scale_log2, lane, 0, no_lim);
      __syncwarp();
      if (lane == 0) mbar_arrive(&empty_bar[st]);
    }
    wa.finish_sums();
  }

  // ------------------------------- combine + write partials -------------------------------
  // All tiles have been consumed by every active warp once they pass this barrier, so the stage
  // ring can be reused as scratch.
  consumer_bar_sync();
  float* so = reinterpret_cast<float*>(stage_mem);                   // [4 warps][16][kORow]
  float* sml = so + kConsumerWarps * 16 * kORow;                     // [4 warps][16][2]
  if (active) wa.spill(so + warp * 16 * kORow, sml + warp * 32, kORow, lane);
  consumer_bar_sync();
  for (int idx = threadIdx.x; idx < nrg * 16 * (D / 4); idx += kConsumerWarps * 32) {
    const int row = idx / (D / 4), dc = idx % (D / 4);
    if (row >= rows) continue;
    const int w0 = (row >> 4) * tsplit, qi = row & 15;
    float M = -INFINITY;
    for (int tp = 0; tp < tsplit; ++tp) M = fmaxf(M, sml[((w0 + tp) * 16 + qi) * 2]);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    float L = 0.f;
    for (int tp = 0; tp < tsplit; ++tp) {
      const float wgt = fast_exp2(sml[((w0 + tp) * 16 + qi) * 2] - M);
      const float4 v = *reinterpret_cast<const float4*>(so + ((w0 + tp) * 16 + qi) * kORow + dc * 4);
      acc.x += wgt * v.x; acc.y += wgt * v.y; acc.z += wgt * v.z; acc.w += wgt * v.w;
      L += wgt * sml[((w0 + tp) * 16 + qi) * 2 + 1];
    }
    const size_t ph = (size_t)(it.part_base + row / g) * p.num_q_heads + kvh * g + row % g;
    *reinterpret_cast<float4*>(p.part_o + ph * D + dc * 4) = acc;
    if (dc == 0) *reinterpret_cast<float2*>(p.part_ml + ph * 2) = make_float2(M, L);
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
  return (size_t)kStages * 2 * (D / 64) * kTile * 128 + (size_t)(D / 64) * kTile * 128 + 2 * kStages * 8;
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
  p.seg_off = t.seg_off;
  p.grp_req = t.grp_req;
  p.q = (const __nv_bfloat16*)q;
  p.part_o = t.part_o;
  p.part_ml = t.part_ml;
  p.status = status;
  p.num_q_heads = sh.num_q_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  dim3 grid((unsigned)num_items, (unsigned)sh.num_kv_heads, 1);
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
