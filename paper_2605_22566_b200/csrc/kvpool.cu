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
                           int n_tokens, int n_pad, int num_kv_heads, int chunks_per_row) {
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

// One bf16 sum, rounded once (nearest, ties to even).
__device__ __forceinline__ uint32_t add_bf16_bits(uint32_t a, uint32_t b) {
  uint16_t r;
  asm("add.rn.bf16 %0, %1, %2;" : "=h"(r) : "h"((uint16_t)a), "h"((uint16_t)b));
  return r;
}

struct ResidualDev {
  const uint32_t* bitmap;  // [rows, D/32]; null: the tensor has no residual
  const uint16_t* values;  // bf16 bits, (row, column) order
  const int32_t* row_ptr;  // [rows + 1]
  long long nnz;
};

// Eq. 7 of Sec. 5.1 for one layer of one node: every 16-byte chunk (8 entries) of the base node's
// extent plus the residual entries its bitmap byte marks, written to the new node's extent in the
// same pool layout.  A thread handles one chunk: the rank of its first residual value inside the
// row is the popcount of the row's bitmap below the chunk.  Values are read only below nnz; an
// inconsistent residual sets the status word instead of reading out of bounds.
__global__ void k_kv_reconstruct(char* layer_base, uint64_t head_stride, uint32_t tile_bytes,
                                 int tile0_dst, int tile0_base, ResidualDev rk, ResidualDev rv, int n_tokens,
                                 int n_pad, int num_kv_heads, int chunks_per_row, int32_t* status) {
  const long long total = (long long)n_pad * num_kv_heads * chunks_per_row;
  const ResidualDev res = blockIdx.y ? rv : rk;
  const uint32_t block_off = blockIdx.y ? (tile_bytes >> 1) : 0u;
  const int words = chunks_per_row >> 2;  // bitmap words per row
  bool bad = false;
  for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
       idx += (long long)gridDim.x * blockDim.x) {
    const int c = (int)(idx % chunks_per_row);
    const long long th = idx / chunks_per_row;  // row of the residual: token * Hkv + head
    const int head = (int)(th % num_kv_heads);
    const int token = (int)(th / num_kv_heads);
    const uint32_t row = (uint32_t)token & (kTile - 1);
    const uint32_t in_tile = block_off + (uint32_t)(c >> 3) * (kTile * 128u) + swz128(row, (uint32_t)c & 7u);
    char* head_base = layer_base + (uint64_t)head * head_stride;
    uint4 val = make_uint4(0u, 0u, 0u, 0u);
    if (token < n_tokens) {
      val = *reinterpret_cast<const uint4*>(head_base + (uint64_t)(tile0_base + token / kTile) * tile_bytes + in_tile);
      if (res.bitmap != nullptr) {
        const uint32_t* bm = res.bitmap + th * words;
        const uint32_t word = bm[c >> 2];
        const uint32_t shift = (uint32_t)(c & 3) * 8u;
        uint32_t bits = (word >> shift) & 0xffu;
        if (bits != 0u) {
          int rank = __popc(word & ((1u << shift) - 1u));
          for (int w = 0; w < (c >> 2); ++w) rank += __popc(bm[w]);
          long long k = (long long)res.row_ptr[th] + rank;
          uint32_t e[4] = {val.x, val.y, val.z, val.w};
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            if ((bits >> j) & 1u) {
              uint32_t d = 0u;
              if (k >= 0 && k < res.nnz) d = res.values[k]; else bad = true;
              ++k;
              const uint32_t sh = (uint32_t)(j & 1) * 16u;
              const uint32_t sum = add_bf16_bits((e[j >> 1] >> sh) & 0xffffu, d);
              e[j >> 1] = (e[j >> 1] & ~(0xffffu << sh)) | (sum << sh);
            }
          }
          val = make_uint4(e[0], e[1], e[2], e[3]);
        }
      }
    }
    *reinterpret_cast<uint4*>(head_base + (uint64_t)(tile0_dst + token / kTile) * tile_bytes + in_tile) = val;
  }
  if (bad) atomicCAS(status, 0, (int32_t)GF_ERR_INVALID_ARG);
}

}  // namespace

int launch_kv_write(const PoolGeom& pool, int layer, int num_kv_heads, int head_dim, int tile0,
                    const void* k, const void* v, int n_tokens, cudaStream_t st) {
  if (n_tokens <= 0) return 0;
  const int n_pad = (n_tokens + kTile - 1) / kTile * kTile;
  const int cpr = head_dim / 8;
  const long long total = (long long)n_pad * num_kv_heads * cpr;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, 2, 1);
  k_kv_write<<<grid, 256, 0, st>>>(pool.base + (uint64_t)layer * pool.layer_stride, pool.head_stride,
                                   pool.tile_bytes, tile0, (const uint4*)k, (const uint4*)v,
                                   n_tokens, n_pad, num_kv_heads, cpr);
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
  const int cpr = head_dim / 8;
  const long long total = (long long)n_pad * num_kv_heads * cpr;
  long long blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  dim3 grid((unsigned)blocks, 2, 1);
  ResidualDev dk{nullptr, nullptr, nullptr, 0}, dv{nullptr, nullptr, nullptr, 0};
  if (rk) dk = ResidualDev{rk->bitmap_dev, (const uint16_t*)rk->values_dev, rk->row_ptr_dev, (long long)rk->nnz};
  if (rv) dv = ResidualDev{rv->bitmap_dev, (const uint16_t*)rv->values_dev, rv->row_ptr_dev, (long long)rv->nnz};
  k_kv_reconstruct<<<grid, 256, 0, st>>>(pool.base + (uint64_t)layer * pool.layer_stride, pool.head_stride,
                                         pool.tile_bytes, tile0_dst, tile0_base, dk, dv, n_tokens, n_pad,
                                         num_kv_heads, cpr, status);
  return cudaGetLastError() == cudaSuccess ? 1 : -1;
}

}  // namespace gf
