// K3 (warp-MMA variant): extend / prefill over a path of shared segments.
//
// Request r appends a new node whose tokens are the queries; token i attends over every token of
// the earlier nodes on the path and tokens 0..i of the new node (the on-the-fly branch of
// Sec. 5.2, after the new segment's K/V are in the pool).  One CTA owns a tile of 64 stacked query
// rows (64/g consecutive new tokens x the g query heads of one KV head), walks the request's
// segment list in path order, streams each segment's K/V tiles through the same bulk-copy ring as
// the decode kernel, and keeps (O, m, l) in registers for the whole walk, so no partials are
// written: the log-sum-exp merge across segments happens in the running softmax.
#include "attn_core.cuh"

namespace gf {
namespace {

constexpr int kStages = 3;
constexpr int kConsumerWarps = 4;
constexpr int kThreads = (kConsumerWarps + 1) * 32;

struct ExtendParams {
  const char* pool_layer;
  uint64_t head_stride;
  uint32_t tile_bytes;
  const int32_t* seg_off;
  const int32_t* seg_len;
  const int32_t* pseg_ptr;
  const int32_t* pseg;
  const int32_t* q_ptr;
  const __nv_bfloat16* q;
  __nv_bfloat16* out;
  float* lse;
  int32_t* status;
  int32_t num_requests, num_q_heads, gqa;
  float scale_log2;
};

__device__ __forceinline__ void consumer_bar_sync() {
  asm volatile("bar.sync 1, %0;" ::"n"(kConsumerWarps * 32) : "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads, 2) k_extend_mma(const ExtendParams p) {
  constexpr int CB = D / 64;
  constexpr uint32_t kBlk = CB * kTile * 128;
  constexpr uint32_t kStageBytes = 2 * kBlk;
  constexpr int kORow = D + 4;

  extern __shared__ __align__(1024) unsigned char smem[];
  unsigned char* stage_mem = smem;
  unsigned char* q_mem = smem + kStages * kStageBytes;
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(q_mem + kBlk);
  uint64_t* empty_bar = full_bar + kStages;

  const int g = p.gqa;
  const int qtt = 64 / g;  // query tokens per CTA
  // blockIdx.x enumerates (request, query tile) slots: request r owns slots starting at
  // q_ptr[r]/qtt + r, which leaves room for ceil(T_r/qtt) tiles.
  const int x = blockIdx.x;
  int lo = 0, hi = p.num_requests;
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (p.q_ptr[mid] / qtt + mid <= x) lo = mid; else hi = mid;
  }
  const int r = lo;
  const int q0 = p.q_ptr[r], T = p.q_ptr[r + 1] - q0;
  const int tok0 = (x - (q0 / qtt + r)) * qtt;
  if (tok0 >= T) return;
  const int ntok = min(qtt, T - tok0);
  const int rows = ntok * g;
  const int nrg = (rows + 15) >> 4;
  const int pb = p.pseg_ptr[r], pe = p.pseg_ptr[r + 1];
  const int kvh = blockIdx.y;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStages; ++s) {
      mbar_init(&full_bar[s], 1);
      mbar_init(&empty_bar[s], nrg);
    }
    mbar_fence_init();
  }
  __syncthreads();

  if (warp == kConsumerWarps) {
    if (lane == 0) {
      int n = 0;
      for (int k = pb; k < pe; ++k) {
        const int s = p.pseg[k];
        const int len = (k == pe - 1) ? tok0 + ntok : p.seg_len[s];  // causal: later tokens unseen
        const char* src0 = p.pool_layer + (uint64_t)kvh * p.head_stride +
                           (uint64_t)(p.seg_off[s] / kTile) * p.tile_bytes;
        for (int t = 0; t * kTile < len; ++t, ++n) {
          const int st = n % kStages;
          if (n >= kStages) mbar_wait(&empty_bar[st], ((n / kStages) - 1) & 1, p.status);
          const int nv = min(kTile, len - t * kTile);
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
    }
    return;
  }

  for (int idx = threadIdx.x; idx < nrg * 16 * (D / 8); idx += kConsumerWarps * 32) {
    const int row = idx / (D / 8), c = idx % (D / 8);
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (row < rows) {
      const size_t qrow = (size_t)(q0 + tok0 + row / g) * p.num_q_heads + kvh * g + row % g;
      val = *reinterpret_cast<const uint4*>(p.q + qrow * D + c * 8);
    }
    *reinterpret_cast<uint4*>(q_mem + (c >> 3) * (kTile * 128) + swz128(row, c & 7)) = val;
  }
  consumer_bar_sync();

  const bool active = warp < nrg;
  WarpAttn<D> wa;
  wa.init();
  if (active) {
    wa.load_q(smem_u32(q_mem), warp * 16, lane);
    // Newest token each of this thread's four columns may see, and the warp's maximum.
    int lim[2][2];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const int row = warp * 16 + j * 8 + (lane & 3) * 2 + c;
        lim[j][c] = (row < rows) ? tok0 + row / g : -1;
      }
    const int warp_lim = tok0 + min(ntok - 1, (warp * 16 + 15) / g);
    int n = 0;
    for (int k = pb; k < pe; ++k) {
      const int s = p.pseg[k];
      const bool self = (k == pe - 1);
      const int len = self ? tok0 + ntok : p.seg_len[s];
      for (int t = 0; t * kTile < len; ++t, ++n) {
        const int st = n % kStages;
        mbar_wait(&full_bar[st], (n / kStages) & 1, p.status);
        const int nv = min(kTile, len - t * kTile);
        const uint32_t kb = smem_u32(stage_mem + st * kStageBytes);
        if (self) {
          for (int ts = 0; ts < nv && t * kTile + ts <= warp_lim; ts += 16)
            wa.template step<true>(kb, kb + kBlk, ts, nv, p.scale_log2, lane, t * kTile, lim);
        } else {
          for (int ts = 0; ts < nv; ts += 16)
            wa.template step<false>(kb, kb + kBlk, ts, nv, p.scale_log2, lane, 0, lim);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty_bar[st]);
      }
    }
    wa.finish_sums();
  }

  consumer_bar_sync();  // every active warp has consumed every tile: the ring becomes scratch
  float* so = reinterpret_cast<float*>(stage_mem);
  float* sml = so + kConsumerWarps * 16 * kORow;
  if (active) {
    float* wo = so + warp * 16 * kORow;
    float* wml = sml + warp * 32;
    wa.spill(wo, wml, kORow, lane);
    __syncwarp();
    for (int qi = 0; qi < 16; ++qi) {
      const int row = warp * 16 + qi;
      if (row >= rows) break;
      const float m = wml[qi * 2], l = wml[qi * 2 + 1];
      const float inv = (l > 0.f) ? 1.f / l : 0.f;
      const size_t orow = (size_t)(q0 + tok0 + row / g) * p.num_q_heads + kvh * g + row % g;
      if (lane < D / 4) {
        const float4 v = *reinterpret_cast<const float4*>(wo + qi * kORow + lane * 4);
        uint2 packed;
        packed.x = pack_bf16(v.x * inv, v.y * inv);
        packed.y = pack_bf16(v.z * inv, v.w * inv);
        *reinterpret_cast<uint2*>(p.out + orow * D + lane * 4) = packed;
      }
      if (p.lse != nullptr && lane == 0)
        p.lse[orow] = (l > 0.f) ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
  }
}

template <int D>
constexpr size_t extend_smem_bytes() {
  return (size_t)kStages * 2 * (D / 64) * kTile * 128 + (size_t)(D / 64) * kTile * 128 + 2 * kStages * 8;
}

}  // namespace

int launch_extend(const PoolGeom& pool, const AttnShape& sh, const TablesDev& t, int layer,
                  int64_t num_q_rows, const void* q, void* out, float* lse, int32_t* status,
                  cudaStream_t st) {
  if (num_q_rows <= 0) return 0;
  ExtendParams p;
  p.pool_layer = pool.base + (uint64_t)layer * pool.layer_stride;
  p.head_stride = pool.head_stride;
  p.tile_bytes = pool.tile_bytes;
  p.seg_off = t.seg_off;
  p.seg_len = t.seg_len;
  p.pseg_ptr = t.pseg_ptr;
  p.pseg = t.pseg;
  p.q_ptr = t.q_ptr;
  p.q = (const __nv_bfloat16*)q;
  p.out = (__nv_bfloat16*)out;
  p.lse = lse;
  p.status = status;
  p.num_requests = t.num_requests;
  p.num_q_heads = sh.num_q_heads;
  p.gqa = sh.num_q_heads / sh.num_kv_heads;
  p.scale_log2 = sh.scale_log2;
  const int qtt = 64 / p.gqa;
  dim3 grid((unsigned)(num_q_rows / qtt + t.num_requests), (unsigned)sh.num_kv_heads, 1);
  cudaError_t err;
  if (sh.head_dim == 128) {
    static bool attr_done = false;
    if (!attr_done) {
      err = cudaFuncSetAttribute(k_extend_mma<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)extend_smem_bytes<128>());
      if (err != cudaSuccess) return -1;
      attr_done = true;
    }
    k_extend_mma<128><<<grid, kThreads, extend_smem_bytes<128>(), st>>>(p);
  } else {
    static bool attr_done = false;
    if (!attr_done) {
      err = cudaFuncSetAttribute(k_extend_mma<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)extend_smem_bytes<64>());
      if (err != cudaSuccess) return -1;
      attr_done = true;
    }
    k_extend_mma<64><<<grid, kThreads, extend_smem_bytes<64>(), st>>>(p);
  }
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
