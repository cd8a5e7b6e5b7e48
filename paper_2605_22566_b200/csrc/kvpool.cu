// KV pool: one extent per wGraph node (Sec. 5: each operation node is associated with its
// precomputed KV states), stored once, in the layout the attention kernels stream.
//
// Layout.  pool[layer][kv_head][tile] where a tile holds 64 tokens of one head: a K block followed
// by a V block.  A block is head_dim/64 column blocks, each [64 rows (tokens)][128 bytes (64 bf16)]
// with the eight 16-byte chunks of a row XOR-swizzled by (row & 7).  A plain bulk copy of a block
// (or of the first n rows of each column block) therefore lands in shared memory already in the
// conflict-free / tensor-core operand layout, and the tiles of one (layer, head) are contiguous so
// an item streams one contiguous byte range.  Rows past a node's length are written as zeros so
// that ragged tails contribute exact zeros to P*V.
#include "gf_device.cuh"
#include "gf_internal.h"

namespace gf {
namespace {

__global__ void k_kv_write(char* __restrict__ layer_base, uint64_t head_stride, uint32_t tile_bytes,
                           int tile0, const uint4* __restrict__ k, const uint4* __restrict__ v,
                           int n_tokens, int n_pad, int num_kv_heads, int chunks_per_row, int32_t* node_len,
                           int32_t* node_off, int node, int cap_tiles, int32_t* status) {
  // the first write of a node also tells the device its length and where its extent starts
  if (node_len != nullptr && blockIdx.x == 0 && blockIdx.y == 0 && threadIdx.x == 0) {
    node_len[node] = n_tokens;
    node_off[node] = tile0 * kTile;
  }
  const long long total = (long long)n_pad * num_kv_heads * chunks_per_row;
  const uint4* __restrict__ src = blockIdx.y ? v : k;
  const uint32_t block_off = blockIdx.y ? (tile_bytes >> 1) : 0u;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks_per_row);
    const long long th = idx / chunks_per_row;
    const int head = (int)(th % num_kv_heads);
    const int token = (int)(th / num_kv_heads);
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (token < n_tokens) val = src[idx];
    const uint32_t row = (uint32_t)token & (kTile - 1);
    const uint64_t tile = (uint64_t)(tile0 + token / kTile);
    if (!GF_CHECK(tile < (uint64_t)cap_tiles, status, 401)) continue;
    char* dst = layer_base + (uint64_t)head * head_stride + tile * tile_bytes + block_off +
                (uint32_t)(c >> 3) * (kTile * 128u) + swz128(row, (uint32_t)c & 7u);
    *reinterpret_cast<uint4*>(dst) = val;
  }
}

// The inverse of k_kv_write: a node's extent back to the caller layout [n_tokens, Hkv, D].
__global__ void k_kv_read(const char* __restrict__ layer_base, uint64_t head_stride, uint32_t tile_bytes,
                          int tile0, uint4* __restrict__ k, uint4* __restrict__ v, int n_tokens,
                          int num_kv_heads, int chunks_per_row) {
  const long long total = (long long)n_tokens * num_kv_heads * chunks_per_row;
  uint4* __restrict__ dst = blockIdx.y ? v : k;
  const uint32_t block_off = blockIdx.y ? (tile_bytes >> 1) : 0u;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks_per_row);
    const long long th = idx / chunks_per_row;
    const int head = (int)(th % num_kv_heads);
    const int token = (int)(th / num_kv_heads);
    const uint32_t row = (uint32_t)token & (kTile - 1);
    const uint64_t tile = (uint64_t)(tile0 + token / kTile);
    const char* src = layer_base + (uint64_t)head * head_stride + tile * tile_bytes + block_off +
                      (uint32_t)(c >> 3) * (kTile * 128u) + swz128(row, (uint32_t)c & 7u);
    dst[idx] = *reinterpret_cast<const uint4*>(src);
  }
}

// Two bf16 sums, each rounded once (nearest, ties to even).
__device__ __forceinline__ uint32_t add_bf16x2_bits(uint32_t a, uint32_t b) {
  uint32_t r;
  asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
  return r;
}

struct ResidualDev {
  const uint32_t* bitmap;  // [rows, D/32]; null: the tensor has no residual
  const uint16_t* values;  // bf16 bits, (row, column) order
  const int32_t* row_ptr;  // [rows + 1]
  long long nnz;
};

constexpr int kReconThreads = 256;

// Eq. 7 of Sec. 5.1 for one layer of one node: the base node's extent plus the residual entries the
// bitmap marks, written to the new node's extent in the same pool layout.  A row (token x KV head) is
// handled by head_dim/8 lanes, one 16-byte chunk (eight adjacent entries) each, so a warp works on
// two rows (head_dim 128) or four (64) at a time: the lane's bitmap byte says which of its entries
// carry a value, and the popcount of the row's bitmap below it is the rank of its first value inside
// the row.  An entry without a value gets -0 added, which leaves every number (and the sign of a
// zero) as it was.  A group of lanes keeps its KV head and walks the tokens with a fixed stride, so no
// division is left in the loop, and the next row's bitmap and first-value index are requested before
// the current row is worked on.  Values are read only below nnz; an inconsistent residual sets the
// status word instead of reading out of bounds.
template <int D>
__global__ void __launch_bounds__(kReconThreads, 6) k_kv_reconstruct(
    char* layer_base, uint64_t head_stride, uint32_t tile_bytes, int tile0_dst, int tile0_base, ResidualDev rk,
    ResidualDev rv, int n_tokens, int n_pad, int num_kv_heads, int32_t* status) {
  constexpr int kWords = D / 32;        // bitmap words per row
  constexpr int kLanesPerRow = D / 8;   // 16 or 8
  constexpr int kRowsPerWarp = 32 / kLanesPerRow;
  const ResidualDev res = blockIdx.y ? rv : rk;
  const uint32_t block_off = blockIdx.y ? (tile_bytes >> 1) : 0u;
  const int lane = threadIdx.x & 31;
  const int sub = lane & (kLanesPerRow - 1);  // this lane's 16-byte chunk of its row: entries 8*sub .. 8*sub+7
  // a group of lanes = one KV head, tokens token0, token0 + stride, ...
  const int group = ((blockIdx.x * kReconThreads + threadIdx.x) >> 5) * kRowsPerWarp + lane / kLanesPerRow;
  const int num_groups = ((gridDim.x * kReconThreads) >> 5) * kRowsPerWarp;  // a multiple of num_kv_heads
  const int head = group % num_kv_heads;
  const int stride = num_groups / num_kv_heads;
  const bool has_res = res.bitmap != nullptr;
  const int nnz = (int)res.nnz;
  char* head_base = layer_base + (uint64_t)head * head_stride + block_off;
  const long long dst_minus_src = ((long long)tile0_dst - tile0_base) * (long long)tile_bytes;
  // byte offset of the lane's chunk inside an unswizzled row: column block, then chunk in it
  const uint32_t lane_cb = (uint32_t)(sub >> 3) * (kTile * 128u), lane_chunk = ((uint32_t)sub & 7u) << 4;
  const int w = sub >> 2;                        // the lane's bitmap word
  const uint32_t sh = ((uint32_t)sub & 3u) * 8u;  // and its byte inside it
  bool bad = false;

  uint32_t words[kWords];
  int rp = 0;
  auto load_meta = [&](int token) {
#pragma unroll
    for (int x = 0; x < kWords; ++x) words[x] = 0u;
    rp = 0;
    if (has_res && token < n_tokens) {
      const int th = token * num_kv_heads + head;
      if (kWords == 4) {
        const uint4 x = *reinterpret_cast<const uint4*>(res.bitmap + (size_t)th * 4);
        words[0] = x.x; words[1] = x.y; words[2 % kWords] = x.z; words[3 % kWords] = x.w;
      } else {
        const uint2 x = *reinterpret_cast<const uint2*>(res.bitmap + (size_t)th * 2);
        words[0] = x.x; words[1] = x.y;
      }
      rp = res.row_ptr[th];
    }
  };
  int token = group / num_kv_heads;
  load_meta(token);
  for (; token < n_pad; token += stride) {
    // this row's bitmap word, the count of values before it, and the next row's request
    uint32_t mine = words[0];
    int before = 0;
#pragma unroll
    for (int x = 1; x < kWords; ++x) {
      if (w >= x) { before += __popc(words[x - 1]); mine = words[x]; }
    }
    const int k = rp + before + __popc(mine & ((1u << sh) - 1u));
    const uint32_t bits = (mine >> sh) & 0xffu;
    load_meta(token + stride);

    const char* src = head_base + (uint64_t)(tile0_base + (token >> 6)) * tile_bytes + ((uint32_t)token & 63u) * 128u +
                      lane_cb + (lane_chunk ^ (((uint32_t)token & 7u) << 4));
    uint4 base = make_uint4(0u, 0u, 0u, 0u);
    if (token < n_tokens) base = *reinterpret_cast<const uint4*>(src);
    uint4 out = base;
    if (bits != 0u) {
      if (k < 0 || k + __popc(bits) > nnz) {
        bad = true;
      } else {
        // entry i takes the value whose rank is the number of marked entries before it
        uint32_t e[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          e[i] = 0x8000u;  // -0: x + (-0) = x
          if ((bits >> i) & 1u) e[i] = res.values[k + __popc(bits & ((1u << i) - 1u))];
        }
        out.x = add_bf16x2_bits(base.x, e[0] | (e[1] << 16));
        out.y = add_bf16x2_bits(base.y, e[2] | (e[3] << 16));
        out.z = add_bf16x2_bits(base.z, e[4] | (e[5] << 16));
        out.w = add_bf16x2_bits(base.w, e[6] | (e[7] << 16));
      }
    }
    *reinterpret_cast<uint4*>(const_cast<char*>(src) + dst_minus_src) = out;
  }
  if (bad) atomicCAS(status, 0, (int32_t)GF_ERR_INVALID_ARG);
}

}  // namespace

int launch_kv_write(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0,
                    const void* k, const void* v, int n_tokens, const GraphDev* set, int node, int32_t* status,
                    cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int n_pad = (n_tokens + kTile - 1) / kTile * kTile;
  const int cpr = head_dim / 8;
  const long long total = (long long)n_pad * num_kv_heads * cpr;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, 2, 1);
  k_kv_write<<<grid, 256, 0, st>>>(pool.base + (uint64_t)layer * pool.layer_stride, pool.head_stride,
                                   pool.tile_bytes, tile0, (const uint4*)k, (const uint4*)v,
                                   n_tokens, n_pad, num_kv_heads, cpr, set ? set->node_len : nullptr,
                                   set ? set->node_off : nullptr, node, (int)pool.cap_tiles, status);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_kv_read(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0, void* k,
                   void* v, int n_tokens, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int cpr = head_dim / 8;
  const long long total = (long long)n_tokens * num_kv_heads * cpr;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, 2, 1);
  k_kv_read<<<grid, 256, 0, st>>>(pool.base + (uint64_t)layer * pool.layer_stride, pool.head_stride,
                                  pool.tile_bytes, tile0, (uint4*)k, (uint4*)v, n_tokens, num_kv_heads, cpr);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

int launch_kv_reconstruct(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0_dst,
                          int tile0_base, const gf_residual_t* rk, const gf_residual_t* rv, int n_tokens,
                          int32_t* status, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int n_pad = (n_tokens + kTile - 1) / kTile * kTile;
  // groups (one row at a time each) per CTA; the grid holds a multiple of num_kv_heads groups so that
  // a group keeps its head, and no more CTAs than six per SM or than the rows need
  const int groups_per_block = kReconThreads / 32 * (head_dim == 128 ? 2 : 4);
  const long long rows = (long long)n_pad * num_kv_heads;
  long long blocks = (rows + groups_per_block - 1) / groups_per_block;
  if (blocks > 148 * 6) blocks = 148 * 6;
  while ((blocks * groups_per_block) % num_kv_heads != 0) ++blocks;
  dim3 grid((unsigned)blocks, 2, 1);
  ResidualDev dk{nullptr, nullptr, nullptr, 0}, dv{nullptr, nullptr, nullptr, 0};
  if (rk) dk = ResidualDev{rk->bitmap_dev, (const uint16_t*)rk->values_dev, rk->row_ptr_dev, (long long)rk->nnz};
  if (rv) dv = ResidualDev{rv->bitmap_dev, (const uint16_t*)rv->values_dev, rv->row_ptr_dev, (long long)rv->nnz};
  char* base = pool.base + (uint64_t)layer * pool.layer_stride;
  if (head_dim == 128)
    k_kv_reconstruct<128><<<grid, kReconThreads, 0, st>>>(base, pool.head_stride, pool.tile_bytes, tile0_dst,
                                                          tile0_base, dk, dv, n_tokens, n_pad, num_kv_heads, status);
  else
    k_kv_reconstruct<64><<<grid, kReconThreads, 0, st>>>(base, pool.head_stride, pool.tile_bytes, tile0_dst,
                                                         tile0_base, dk, dv, n_tokens, n_pad, num_kv_heads, status);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
