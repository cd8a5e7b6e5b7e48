// Differential KV, the encoding side (Sec. 5.1): the sparse residual of a prefix-conditioned state
// against the base state of its node, dKV(P, v) = KV(P, v) - KV_base(v), entries below a threshold
// dropped, in the bitmap format gf_node_kv_reconstruct reads.  Set-up work (residuals are computed
// once, ahead of serving), so three plain passes:
//   mark : per row (token x KV head), head_dim/8 lanes of eight entries: the difference of every entry
//          rounded once to bf16, the bitmap of the entries whose stored magnitude exceeds the
//          threshold, and the row's count;
//   scan : counts -> exclusive row starts (one CTA), the total, and the capacity check;
//   fill : the kept differences written at row start + rank.
#include "gf_device.cuh"
#include "gf_internal.h"

namespace gf {
namespace {

constexpr int kEncThreads = 256;

__device__ __forceinline__ uint32_t sub_bf16x2_bits(uint32_t a, uint32_t b) {  // a - b, one rounding each
  uint32_t r;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b ^ 0x80008000u));
  return r;
}

// Differences of the lane's eight entries (bf16 bits, four pairs) and the byte of those kept.
__device__ __forceinline__ uint32_t diff_and_mask(const uint4& full, const uint4& base, float threshold, uint32_t (&d)[4]) {
  d[0] = sub_bf16x2_bits(full.x, base.x);
  d[1] = sub_bf16x2_bits(full.y, base.y);
  d[2] = sub_bf16x2_bits(full.z, base.z);
  d[3] = sub_bf16x2_bits(full.w, base.w);
  uint32_t bits = 0u;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float lo = fabsf(__uint_as_float(d[i] << 16)), hi = fabsf(__uint_as_float(d[i] & 0xffff0000u));
    bits |= (lo > threshold ? 1u : 0u) << (2 * i);
    bits |= (hi > threshold ? 1u : 0u) << (2 * i + 1);
  }
  return bits;
}

struct EncodeArgs {
  const char* layer_base;
  uint64_t head_stride;
  uint32_t tile_bytes;
  int tile0;
  const uint4* full[2];   // K, V of the prefix-conditioned state, caller layout [n_tokens, Hkv, D]
  uint32_t* bitmap[2];
  uint16_t* values[2];
  int32_t* row_ptr[2];
  long long capacity[2];
  long long* nnz[2];
  int n_tokens, num_kv_heads;
  float threshold;
  int32_t* status;
};

// kFill = false: bitmap and row counts (into row_ptr).  kFill = true: values at row_ptr + rank.
template <int D, bool kFill>
__global__ void __launch_bounds__(kEncThreads) k_residual_pass(const EncodeArgs a) {
  constexpr int kLanesPerRow = D / 8;
  constexpr int kRowsPerWarp = 32 / kLanesPerRow;
  const int t = blockIdx.y;  // 0: K, 1: V
  if (a.bitmap[t] == nullptr) return;
  const uint32_t block_off = t ? (a.tile_bytes >> 1) : 0u;
  const int lane = threadIdx.x & 31, sub = lane & (kLanesPerRow - 1);
  const int rows = a.n_tokens * a.num_kv_heads;
  const int group = ((blockIdx.x * kEncThreads + threadIdx.x) >> 5) * kRowsPerWarp + lane / kLanesPerRow;
  const int num_groups = ((gridDim.x * kEncThreads) >> 5) * kRowsPerWarp;
  // every lane of a warp runs the same number of passes (the shuffles below need the whole warp)
  const int passes = (rows + num_groups - 1) / num_groups;
  for (int it = 0; it < passes; ++it) {
    const int th = group + it * num_groups;
    const bool live = th < rows;
    uint32_t bits = 0u;
    uint32_t d[4] = {0u, 0u, 0u, 0u};
    if (live) {
      const int token = th / a.num_kv_heads, head = th - token * a.num_kv_heads;
      const char* src = a.layer_base + (uint64_t)head * a.head_stride + (uint64_t)(a.tile0 + (token >> 6)) * a.tile_bytes +
                        block_off + ((uint32_t)token & 63u) * 128u + (uint32_t)(sub >> 3) * (kTile * 128u) +
                        ((((uint32_t)sub & 7u) ^ ((uint32_t)token & 7u)) << 4);
      const uint4 base = *reinterpret_cast<const uint4*>(src);
      const uint4 full = a.full[t][(size_t)th * kLanesPerRow + sub];
      bits = diff_and_mask(full, base, a.threshold, d);
    }
    // the row's bitmap word of this lane's four-lane group, and the values before this lane in the row
    uint32_t word = bits << (((uint32_t)sub & 3u) * 8u);
    word |= __shfl_xor_sync(0xffffffffu, word, 1);
    word |= __shfl_xor_sync(0xffffffffu, word, 2);
    int incl = __popc(bits);
#pragma unroll
    for (int s = 1; s < kLanesPerRow; s <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, incl, s, kLanesPerRow);
      if (sub >= s) incl += y;
    }
    if (!live) continue;
    if (!kFill) {
      if ((sub & 3) == 0) a.bitmap[t][(size_t)th * (D / 32) + (sub >> 2)] = word;
      if (sub == kLanesPerRow - 1) a.row_ptr[t][th] = incl;  // the row's count; the scan turns it into a start
    } else {
      long long k = (long long)a.row_ptr[t][th] + (incl - __popc(bits));
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        if ((bits >> i) & 1u) {
          if (k < a.capacity[t]) a.values[t][k] = (uint16_t)((d[i >> 1] >> ((i & 1) * 16)) & 0xffffu);
          ++k;
        }
      }
    }
  }
}

// One CTA per tensor: row counts -> exclusive row starts, row_ptr[rows] = nnz, the capacity check.
__global__ void __launch_bounds__(1024) k_residual_scan(const EncodeArgs a) {
  const int t = blockIdx.x;
  if (a.bitmap[t] == nullptr) return;
  __shared__ long long warp_tot[32];
  __shared__ long long carry_s;
  const int rows = a.n_tokens * a.num_kv_heads;
  const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, nw = blockDim.x >> 5;
  int32_t* rp = a.row_ptr[t];
  if (tid == 0) carry_s = 0;
  __syncthreads();
  for (int base = 0; base < rows; base += blockDim.x) {
    const int i = base + tid;
    const long long x = (i < rows) ? rp[i] : 0;
    long long incl = x;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
      const long long y = __shfl_up_sync(0xffffffffu, incl, d);
      if (lane >= d) incl += y;
    }
    if (lane == 31) warp_tot[wid] = incl;
    __syncthreads();
    if (wid == 0) {
      long long w = (lane < nw) ? warp_tot[lane] : 0;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const long long y = __shfl_up_sync(0xffffffffu, w, d);
        if (lane >= d) w += y;
      }
      warp_tot[lane] = w;
    }
    __syncthreads();
    const long long start = carry_s + ((wid == 0) ? 0 : warp_tot[wid - 1]) + incl - x;
    if (i < rows) rp[i] = (int32_t)(start < 0x7fffffffll ? start : 0x7fffffffll);
    __syncthreads();
    if (tid == 0) carry_s += warp_tot[nw - 1];
    __syncthreads();
  }
  if (tid == 0) {
    const long long total = carry_s;
    rp[rows] = (int32_t)(total < 0x7fffffffll ? total : 0x7fffffffll);
    *a.nnz[t] = total;
    if (total > a.capacity[t] || total > 0x7fffffffll) atomicCAS(a.status, 0, (int32_t)GF_ERR_CAPACITY);
  }
}

}  // namespace

int launch_residual_encode(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0,
                           const void* k_full, const void* v_full, int n_tokens, float threshold,
                           const gf_residual_buf_t* k_out, const gf_residual_buf_t* v_out, int32_t* status,
                           cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  EncodeArgs a;
  a.layer_base = pool.base + (uint64_t)layer * pool.layer_stride;
  a.head_stride = pool.head_stride;
  a.tile_bytes = pool.tile_bytes;
  a.tile0 = tile0;
  const gf_residual_buf_t* outs[2] = {k_out, v_out};
  const void* fulls[2] = {k_full, v_full};
  for (int t = 0; t < 2; ++t) {
    const bool on = outs[t] != nullptr;
    a.full[t] = (const uint4*)fulls[t];
    a.bitmap[t] = on ? outs[t]->bitmap_dev : nullptr;
    a.values[t] = on ? (uint16_t*)outs[t]->values_dev : nullptr;
    a.row_ptr[t] = on ? outs[t]->row_ptr_dev : nullptr;
    a.capacity[t] = on ? (long long)outs[t]->capacity : 0;
    a.nnz[t] = on ? (long long*)outs[t]->nnz_dev : nullptr;
  }
  a.n_tokens = n_tokens;
  a.num_kv_heads = num_kv_heads;
  a.threshold = threshold;
  a.status = status;
  const int groups_per_block = kEncThreads / 32 * (head_dim == 128 ? 2 : 4);
  const long long rows = (long long)n_tokens * num_kv_heads;
  long long blocks = (rows + groups_per_block - 1) / groups_per_block;
  if (blocks > 148 * 8) blocks = 148 * 8;
  dim3 grid((unsigned)blocks, 2, 1);
  if (head_dim == 128) k_residual_pass<128, false><<<grid, kEncThreads, 0, st>>>(a);
  else k_residual_pass<64, false><<<grid, kEncThreads, 0, st>>>(a);
  k_residual_scan<<<2, 1024, 0, st>>>(a);
  if (head_dim == 128) k_residual_pass<128, true><<<grid, kEncThreads, 0, st>>>(a);
  else k_residual_pass<64, true><<<grid, kEncThreads, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? 3 : -1;
}

}  // namespace gf
