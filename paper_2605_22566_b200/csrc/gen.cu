// Device-side copy of the synthetic value generator (inputs only; no attention arithmetic).
// Element i of stream `key` is tab[splitmix64(key + (i+1)*GOLDEN) & 0xFFFF], where tab is the
// caller-supplied 65 536-entry table of bf16 bit patterns.  Bit-identical to the numpy generator.
#include <cuda_runtime.h>
#include <stdint.h>

namespace {
__global__ void k_fill(const uint16_t* __restrict__ tab, unsigned long long key, unsigned long long start,
                       unsigned long long count, uint16_t* __restrict__ out) {
  for (unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; i < count;
       i += (unsigned long long)gridDim.x * blockDim.x) {
    unsigned long long z = key + (start + i + 1ull) * 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    z ^= z >> 31;
    out[i] = tab[z & 0xFFFFull];
  }
}
}  // namespace

extern "C" int gfgen_fill_bf16(const void* tab_dev, uint64_t key, uint64_t start, uint64_t count,
                               void* out_dev, void* stream) {
  if (count == 0) return 0;
  unsigned long long blocks = (count + 255) / 256;
  if (blocks > 148 * 32) blocks = 148 * 32;
  k_fill<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((const uint16_t*)tab_dev, key, start, count,
                                                             (uint16_t*)out_dev);
  return cudaGetLastError() == cudaSuccess ? 0 : 1;
}
