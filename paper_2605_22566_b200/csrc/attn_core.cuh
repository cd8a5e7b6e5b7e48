// Per-warp attention core of the decode kernel.
//
// A warp owns 8 or 16 stacked query rows (one or two MMA n-tiles of 8) and consumes MT*16 tokens
// per step from a K block and a V block staged in shared memory in the pool's swizzled layout:
//   S^T[MT*16 tokens x rows] = K * Q^T          (tokens are the MMA M dimension)
//   online softmax per query row (column of S^T): running max m (log2 units) and sum l
//   O^T[D x rows] += V^T * P^T                  (P transposed in registers with movmatrix)
// This is softmax(scale * q K^T) V over the tokens seen so far, in flash-attention form.  The
// MT m-tiles of a step are independent until the softmax, which gives the tensor pipe MT*NT
// accumulator chains to overlap and amortises the shuffles and the rescale over MT*16 tokens.
#pragma once
#include "gf_device.cuh"
#include "gf_internal.h"

namespace gf {

template <int D>
struct WarpAttn {
  static constexpr int KS = D / 16;
  uint32_t qf[2][KS][2];   // Q^T fragments (B operand): [n-tile][k step][2]
  float o[KS][2][4];       // O^T accumulators: [d tile][n-tile][4]
  float m_run[2][2], l_run[2][2];

  __device__ __forceinline__ void init() {
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) { m_run[j][c] = -INFINITY; l_run[j][c] = 0.f; }
#pragma unroll
    for (int i = 0; i < KS; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) o[i][j][e] = 0.f;
  }

  // One step over tokens ts .. ts+MT*16-1 of the staged tile (rows of the K and V blocks at kb, vb).
  // NT: n-tiles in use (1: query rows 0..7 only).  kMask: tokens >= nv are masked and m-tiles that
  // start at or after nv are skipped (their shared-memory rows were never copied).
  template <int MT, int NT, bool kMask>
  __device__ __forceinline__ void step(uint32_t kb, uint32_t vb, int ts, int nv, float scale_log2, int lane) {
    const int lr = lane & 7, mi = lane >> 3;
    float s[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int j = 0; j < NT; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) s[mt][j][e] = 0.f;
    const int nmt = kMask ? min(MT, (nv - ts + 15) >> 4) : MT;  // m-tiles with at least one token
    const uint32_t krow = ts + lr + ((mi & 1) << 3);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int chunk = 2 * ks + (mi >> 1);
      const uint32_t base = kb + (chunk >> 3) * (kTile * 128);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        if (kMask && mt >= nmt) continue;
        uint32_t a[4];
        ldmatrix_x4(a, base + swz128(krow + mt * 16, chunk & 7));
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_bf16(s[mt][j], a, qf[j][ks][0], qf[j][ks][1]);
      }
    }
    // scale, mask, column maxima (the token index lives in lane bits 2..4 and in mt / e>>1)
    float mx[NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) { mx[j][0] = -INFINITY; mx[j][1] = -INFINITY; }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const int tlo = ts + mt * 16 + (lane >> 2), thi = tlo + 8;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        if (kMask) {
          s[mt][j][0] = (tlo < nv) ? s[mt][j][0] * scale_log2 : -INFINITY;
          s[mt][j][1] = (tlo < nv) ? s[mt][j][1] * scale_log2 : -INFINITY;
          s[mt][j][2] = (thi < nv) ? s[mt][j][2] * scale_log2 : -INFINITY;
          s[mt][j][3] = (thi < nv) ? s[mt][j][3] * scale_log2 : -INFINITY;
        } else {
#pragma unroll
          for (int e = 0; e < 4; ++e) s[mt][j][e] *= scale_log2;
        }
        mx[j][0] = fmaxf(mx[j][0], fmaxf(s[mt][j][0], s[mt][j][2]));
        mx[j][1] = fmaxf(mx[j][1], fmaxf(s[mt][j][1], s[mt][j][3]));
      }
    }
    bool grew = false;
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v = mx[j][c];
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 4));
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
        v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 16));
        mx[j][c] = fmaxf(v, m_run[j][c]);
        grew |= mx[j][c] > m_run[j][c];
      }
    if (__any_sync(0xffffffffu, grew)) {  // rescale only when some running maximum moved
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        // a column whose maximum is still -inf has seen no visible token: keep it at zero
        const float a0 = (mx[j][0] == -INFINITY) ? 0.f : fast_exp2(m_run[j][0] - mx[j][0]);
        const float a1 = (mx[j][1] == -INFINITY) ? 0.f : fast_exp2(m_run[j][1] - mx[j][1]);
        l_run[j][0] *= a0; l_run[j][1] *= a1;
        m_run[j][0] = mx[j][0]; m_run[j][1] = mx[j][1];
#pragma unroll
        for (int i = 0; i < KS; ++i) {
          o[i][j][0] *= a0; o[i][j][1] *= a1; o[i][j][2] *= a0; o[i][j][3] *= a1;
        }
      }
    }
    uint32_t pb[MT][NT][2];
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      // (-inf) - (-inf) would be NaN: a fully masked column uses 0 as its reference instead
      const float r0 = (m_run[j][0] == -INFINITY) ? 0.f : m_run[j][0];
      const float r1 = (m_run[j][1] == -INFINITY) ? 0.f : m_run[j][1];
#pragma unroll
      for (int mt = 0; mt < MT; ++mt) {
        const float p0 = fast_exp2(s[mt][j][0] - r0);
        const float p1 = fast_exp2(s[mt][j][1] - r1);
        const float p2 = fast_exp2(s[mt][j][2] - r0);
        const float p3 = fast_exp2(s[mt][j][3] - r1);
        l_run[j][0] += p0 + p2;
        l_run[j][1] += p1 + p3;
        pb[mt][j][0] = movmatrix_trans(pack_bf16(p0, p1));  // P^T as the B operand: k = token, n = row
        pb[mt][j][1] = movmatrix_trans(pack_bf16(p2, p3));
      }
    }
    // m-tile outermost: consecutive MMAs then update different accumulators, so the tensor pipe
    // never waits on the one it has just been given
    const uint32_t vrow = ts + lr + ((mi & 2) << 2);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      if (kMask && mt >= nmt) continue;
#pragma unroll
      for (int i = 0; i < KS; ++i) {
        const int chunk = 2 * i + (mi & 1);
        uint32_t a[4];
        ldmatrix_x4_trans(a, vb + (chunk >> 3) * (kTile * 128) + swz128(vrow + mt * 16, chunk & 7));
#pragma unroll
        for (int j = 0; j < NT; ++j) mma_bf16(o[i][j], a, pb[mt][j][0], pb[mt][j][1]);
      }
    }
  }

  // Sum the per-thread partial row sums over the token lanes.
  __device__ __forceinline__ void finish_sums() {
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        float v = l_run[j][c];
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v += __shfl_xor_sync(0xffffffffu, v, 8);
        v += __shfl_xor_sync(0xffffffffu, v, 16);
        l_run[j][c] = v;
      }
  }
};

}  // namespace gf
