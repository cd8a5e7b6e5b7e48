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

}  // namespace gf
