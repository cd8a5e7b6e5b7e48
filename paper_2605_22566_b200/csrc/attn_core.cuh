// Per-warp attention core shared by the decode and the (warp-MMA) extend kernels.
//
// A warp owns 16 stacked query rows (two MMA n-tiles of 8) and consumes 16 tokens per step from a
// K block and a V block staged in shared memory in the pool's swizzled layout:
//   S^T[16 tokens x 16 rows] = K * Q^T          (tokens are the MMA M dimension)
//   online softmax per query row (column of S^T): running max m (log2 units) and sum l
//   O^T[D x 16 rows] += V^T * P^T               (P transposed in registers with movmatrix)
// This is softmax(scale * q K^T) V over the tokens seen so far, in flash-attention form.
#pragma once
#include "gf_device.cuh"
#include "gf_internal.h"

namespace gf {

template <int D>
struct WarpAttn {
  static constexpr int KS = D / 16;
  uint32_t qf[2][KS][2];
  float o[KS][2][4];
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

  // Query rows row0..row0+15 from a swizzled [col block][row][128 B] staging area.
  __device__ __forceinline__ void load_q(uint32_t qbase, int row0, int lane) {
    const int row = row0 + (lane >> 4) * 8 + (lane & 7);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int chunk = 2 * ks + ((lane >> 3) & 1);
      uint32_t r[4];
      ldmatrix_x4(r, qbase + (chunk >> 3) * (kTile * 128) + swz128(row, chunk & 7));
      qf[0][ks][0] = r[0]; qf[0][ks][1] = r[1]; qf[1][ks][0] = r[2]; qf[1][ks][1] = r[3];
    }
  }

  // One 16-token step at rows ts..ts+15 of the staged tile.  Tokens >= nv are masked.  When
  // kCausal, token index tok_base+ts+i is visible to column (j,c) only if it is <= lim[j][c].
  template <bool kCausal>
  __device__ __forceinline__ void step(uint32_t kb, uint32_t vb, int ts, int nv, float scale_log2,
                                       int lane, int tok_base, const int (&lim)[2][2]) {
    const int lr = lane & 7, mi = lane >> 3;
    float s[2][4];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) s[j][e] = 0.f;
    const uint32_t krow = ts + lr + ((mi & 1) << 3);
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
      const int chunk = 2 * ks + (mi >> 1);
      uint32_t a[4];
      ldmatrix_x4(a, kb + (chunk >> 3) * (kTile * 128) + swz128(krow, chunk & 7));
      mma_bf16(s[0], a, qf[0][ks][0], qf[0][ks][1]);
      mma_bf16(s[1], a, qf[1][ks][0], qf[1][ks][1]);
    }
    const int tlo = ts + (lane >> 2), thi = tlo + 8;
    float mx[2][2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      bool v0 = tlo < nv, v1 = v0, v2 = thi < nv, v3 = v2;
      if (kCausal) {
        v0 = v0 && (tok_base + tlo <= lim[j][0]);
        v1 = v1 && (tok_base + tlo <= lim[j][1]);
        v2 = v2 && (tok_base + thi <= lim[j][0]);
        v3 = v3 && (tok_base + thi <= lim[j][1]);
      }
      s[j][0] = v0 ? s[j][0] * scale_log2 : -INFINITY;
      s[j][1] = v1 ? s[j][1] * scale_log2 : -INFINITY;
      s[j][2] = v2 ? s[j][2] * scale_log2 : -INFINITY;
      s[j][3] = v3 ? s[j][3] * scale_log2 : -INFINITY;
      mx[j][0] = fmaxf(s[j][0], s[j][2]);
      mx[j][1] = fmaxf(s[j][1], s[j][3]);
    }
    // Column maxima over the 16 tokens: the token index lives in lane bits 2..4.
    bool grew = false;
#pragma unroll
    for (int j = 0; j < 2; ++j)
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
      for (int j = 0; j < 2; ++j) {
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
    uint32_t pb0[2], pb1[2];
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      // (-inf) - (-inf) would be NaN: a fully masked column uses 0 as its reference instead
      const float r0 = (m_run[j][0] == -INFINITY) ? 0.f : m_run[j][0];
      const float r1 = (m_run[j][1] == -INFINITY) ? 0.f : m_run[j][1];
      const float p0 = fast_exp2(s[j][0] - r0);
      const float p1 = fast_exp2(s[j][1] - r1);
      const float p2 = fast_exp2(s[j][2] - r0);
      const float p3 = fast_exp2(s[j][3] - r1);
      l_run[j][0] += p0 + p2;
      l_run[j][1] += p1 + p3;
      pb0[j] = movmatrix_trans(pack_bf16(p0, p1));  // P^T as the B operand: k = token, n = row
      pb1[j] = movmatrix_trans(pack_bf16(p2, p3));
    }
    const uint32_t vrow = ts + lr + ((mi & 2) << 2);
#pragma unroll
    for (int i = 0; i < KS; ++i) {
      const int chunk = 2 * i + (mi & 1);
      uint32_t a[4];
      ldmatrix_x4_trans(a, vb + (chunk >> 3) * (kTile * 128) + swz128(vrow, chunk & 7));
      mma_bf16(o[i][0], a, pb0[0], pb1[0]);
      mma_bf16(o[i][1], a, pb0[1], pb1[1]);
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

  // Token-split warps hold partial (O, m, l) of the same 16 query rows in the same fragment
  // layout.  hand_over writes half of O (and m, l after finish_sums) as [register][lane] floats,
  // take_over merges it into this warp's state: both rescaled to the common maximum.
  __device__ __forceinline__ void hand_over(float* slot, int half, int lane) const {
#pragma unroll
    for (int i = 0; i < KS / 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) slot[((i * 2 + j) * 4 + e) * 32 + lane] = o[half * (KS / 2) + i][j][e];
    constexpr int kBase = (KS / 2) * 8;
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        slot[(kBase + j * 2 + c) * 32 + lane] = m_run[j][c];
        slot[(kBase + 4 + j * 2 + c) * 32 + lane] = l_run[j][c];
      }
  }
  __device__ __forceinline__ void take_over(const float* slot, int half, int lane) {
    constexpr int kBase = (KS / 2) * 8;
    float wa[2][2], wb[2][2];
#pragma unroll
    for (int j = 0; j < 2; ++j)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const float mb = slot[(kBase + j * 2 + c) * 32 + lane];
        const float lb = slot[(kBase + 4 + j * 2 + c) * 32 + lane];
        const float M = fmaxf(m_run[j][c], mb);
        wa[j][c] = (m_run[j][c] == -INFINITY) ? 0.f : fast_exp2(m_run[j][c] - M);
        wb[j][c] = (mb == -INFINITY) ? 0.f : fast_exp2(mb - M);
        if (half == 1) {  // m and l change once, after both halves of O used the old values
          l_run[j][c] = wa[j][c] * l_run[j][c] + wb[j][c] * lb;
          m_run[j][c] = M;
        }
      }
#pragma unroll
    for (int i = 0; i < KS / 2; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          float& dst = o[half * (KS / 2) + i][j][e];
          dst = wa[j][e & 1] * dst + wb[j][e & 1] * slot[((i * 2 + j) * 4 + e) * 32 + lane];
        }
  }

  // Spill O (as [16 rows][row_stride] fp32) and (m, l) (as [16][2]) to shared memory.
  __device__ __forceinline__ void spill(float* wo, float* wml, int row_stride, int lane) const {
#pragma unroll
    for (int i = 0; i < KS; ++i)
#pragma unroll
      for (int j = 0; j < 2; ++j) {
        const int qi = j * 8 + (lane & 3) * 2, d = i * 16 + (lane >> 2);
        wo[qi * row_stride + d] = o[i][j][0];
        wo[(qi + 1) * row_stride + d] = o[i][j][1];
        wo[qi * row_stride + d + 8] = o[i][j][2];
        wo[(qi + 1) * row_stride + d + 8] = o[i][j][3];
      }
    if (lane < 4) {
#pragma unroll
      for (int j = 0; j < 2; ++j)
#pragma unroll
        for (int c = 0; c < 2; ++c) {
          const int qi = j * 8 + lane * 2 + c;
          wml[qi * 2 + 0] = m_run[j][c];
          wml[qi * 2 + 1] = l_run[j][c];
        }
    }
  }
};

}  // namespace gf
