// Workflow generation scoring (Sec. 4.1, 4.2; appendix "Network Architecture Details"): for a batch of
// tasks, the task-conditioned graph (the wGraph plus a virtual task node joined to every operation) is
// encoded by a 2-layer graph convolution and every wGraph edge is scored by a 3-layer perceptron.
//
//   encoder layer   h_i' = ReLU( sum over j in N(i) and i itself of (h_j W) / sqrt(deg(i) deg(j)) ),
//                   operation edges taken in both directions, deg counting the node itself, no bias
//   edge (i, j)     s = sigmoid( w3 . ReLU( W2^T ReLU( W1^T [h_i, h_j, h_task] + b1 ) + b2 ) + b3 )
//
// Everything is fp32.  The first perceptron layer is linear in its three blocks, so it is applied to
// the node embeddings once per node (three narrow products) and an edge only adds three rows.  A
// second, small workload beside the attention path: plain tiled kernels, latency-bound at these sizes.
#include "gf_internal.h"

namespace gf {
namespace {

// C[m, n] = sum_k A[m, k] * W[k, n]; row-major with leading dimensions; 64 x 64 tiles, 256 threads.
constexpr int kTileM = 64, kTileN = 64, kTileK = 16;
__global__ void __launch_bounds__(256) k_linear(const float* __restrict__ A, int lda, const float* __restrict__ W, int ldw,
                                                float* __restrict__ C, int ldc, int M, int N, int K) {
  __shared__ float As[kTileK][kTileM + 1];
  __shared__ float Ws[kTileK][kTileN + 1];
  const int m0 = blockIdx.y * kTileM, n0 = blockIdx.x * kTileN;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;  // 16 x 16 threads, 4 x 4 outputs each
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += kTileK) {
    for (int i = threadIdx.x; i < kTileM * kTileK; i += 256) {
      const int m = i / kTileK, k = i % kTileK;
      As[k][m] = (m0 + m < M && k0 + k < K) ? A[(size_t)(m0 + m) * lda + k0 + k] : 0.f;
    }
    for (int i = threadIdx.x; i < kTileK * kTileN; i += 256) {
      const int k = i / kTileN, n = i % kTileN;
      Ws[k][n] = (k0 + k < K && n0 + n < N) ? W[(size_t)(k0 + k) * ldw + n0 + n] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < kTileK; ++k) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[k][ty * 4 + i]; w[i] = Ws[k][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < M && n < N) C[(size_t)m * ldc + n] = acc[i][j];
    }
}

// One encoder layer's aggregation for node i of task b (grid: node x task, one thread per feature):
// out[b][i] = ReLU( sum over j in N(i) and i of in(b, j) / sqrt(deg i deg j) ), where in(b, j) is row j of
// the operation rows (op + b * op_stride) for j < num_ops and the task row (task + b * task_stride) for
// the task node.  The task node's neighbourhood is every operation.
__global__ void k_aggregate(ScoreGraphDev g, const float* __restrict__ op, size_t op_stride, const float* __restrict__ task,
                            size_t task_stride, float* __restrict__ out, int d) {
  const int i = blockIdx.x, b = blockIdx.y, n = g.num_ops;
  const float* rows = op + (size_t)b * op_stride;
  const float* trow = task + (size_t)b * task_stride;
  const float wi = g.inv_sqrt[i];
  for (int f = threadIdx.x; f < d; f += blockDim.x) {
    float acc;
    if (i < n) {
      acc = rows[(size_t)i * d + f] * wi * wi + trow[f] * wi * g.inv_sqrt[n];
      for (int k = g.sym_ptr[i]; k < g.sym_ptr[i + 1]; ++k) {
        const int j = g.sym_idx[k];
        acc = fmaf(rows[(size_t)j * d + f], wi * g.inv_sqrt[j], acc);
      }
    } else {
      acc = trow[f] * wi * wi;
      for (int j = 0; j < n; ++j) acc = fmaf(rows[(size_t)j * d + f], wi * g.inv_sqrt[j], acc);
    }
    out[((size_t)b * (n + 1) + i) * d + f] = fmaxf(acc, 0.f);
  }
}

// The perceptron on every (task, edge) pair.  P holds, per task and node, the three partial products of
// the first layer ([h Wa | h Wb | h Wc], 3 * dm floats); a warp takes a pair, forms
// a1 = ReLU(Pa[src] + Pb[dst] + Pc[task] + b1) in shared memory, then every lane computes dm / 32
// outputs of the second layer from the copy of W2 in shared memory, and the warp reduces the third.
__global__ void __launch_bounds__(256) k_edge_mlp(ScoreGraphDev g, const float* __restrict__ P, const float* __restrict__ b1,
                                                  const float* __restrict__ w2, const float* __restrict__ b2,
                                                  const float* __restrict__ w3, float b3, float* __restrict__ scores,
                                                  int dm, int num_tasks, size_t score_stride) {
  extern __shared__ float sm[];
  float* w2s = sm;                      // [dm][dm]
  float* a1s = sm + (size_t)dm * dm;    // [8 warps][dm]
  for (int i = threadIdx.x; i < dm * dm; i += blockDim.x) w2s[i] = w2[i];
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  float* a1 = a1s + warp * dm;
  const int per = dm / 32;
  const long long pairs = (long long)num_tasks * g.num_edges;
  const size_t node_stride = (size_t)3 * dm, task_rows = (size_t)(g.num_ops + 1);
  for (long long pr = (long long)blockIdx.x * 8 + warp; pr < pairs; pr += (long long)gridDim.x * 8) {
    const int b = (int)(pr / g.num_edges), e = (int)(pr % g.num_edges);
    const float* base = P + (size_t)b * task_rows * node_stride;
    const float* pa = base + (size_t)g.edge_src[e] * node_stride;
    const float* pb = base + (size_t)g.edge_dst[e] * node_stride + dm;
    const float* pc = base + (size_t)g.num_ops * node_stride + 2 * dm;
    for (int k = lane; k < dm; k += 32) a1[k] = fmaxf(pa[k] + pb[k] + pc[k] + b1[k], 0.f);
    __syncwarp();
    float part = 0.f;
    for (int c = 0; c < per; ++c) {
      const int n = lane + 32 * c;
      float acc = b2[n];
      for (int k = 0; k < dm; ++k) acc = fmaf(a1[k], w2s[(size_t)k * dm + n], acc);
      part = fmaf(fmaxf(acc, 0.f), w3[n], part);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
    if (lane == 0) scores[(size_t)b * score_stride + e] = 1.f / (1.f + expf(-(part + b3)));
    __syncwarp();
  }
}

void linear(const float* A, int lda, const float* W, int ldw, float* C, int ldc, int M, int N, int K, cudaStream_t st) {
  if (M <= 0 || N <= 0) return;
  dim3 grid((unsigned)((N + kTileN - 1) / kTileN), (unsigned)((M + kTileM - 1) / kTileM));
  k_linear<<<grid, 256, 0, st>>>(A, lda, W, ldw, C, ldc, M, N, K);
}

}  // namespace

// Floats of scratch for `per_pass` tasks worked on at a time: the operations' and the tasks' first-layer
// products (shared by all passes), two node-embedding buffers and the first perceptron layer's partial
// products for the pass.
size_t edge_scores_scratch_floats(int num_ops, const gf_scorer_t& m, int num_queries, int per_pass) {
  const size_t dh = m.d_hidden, dm = m.d_mlp, rows = (size_t)per_pass * (num_ops + 1);
  return (size_t)num_ops * dh + (size_t)num_queries * dh + 2 * rows * dh + rows * 3 * dm;
}

int launch_edge_scores(const ScoreGraphDev& g, const gf_scorer_t& m, const float* x_op, int num_queries,
                       const float* x_task, float* scores, float* scratch, int per_pass, cudaStream_t st) {
  const int n = g.num_ops, dh = m.d_hidden, dm = m.d_mlp;
  if (num_queries <= 0 || g.num_edges <= 0) return 0;
  float* z_op = scratch;
  float* z_task = z_op + (size_t)n * dh;
  float* h = z_task + (size_t)num_queries * dh;            // [per_pass][n + 1][dh]: layer-1 output, then layer-2 output
  float* gbuf = h + (size_t)per_pass * (n + 1) * dh;       // [per_pass][n + 1][dh]: layer-1 output times W2
  float* pbuf = gbuf + (size_t)per_pass * (n + 1) * dh;    // [per_pass][n + 1][3 dm]
  static bool optin[kMaxDevices] = {};
  const size_t mlp_smem = ((size_t)dm * dm + 8 * (size_t)dm) * sizeof(float);
  if (!ensure_dynamic_smem(k_edge_mlp, mlp_smem, optin)) return -1;
  int launches = 0;
  // first encoder layer before aggregation: the operations' rows are the same for every task
  linear(x_op, m.d_in, m.w_gcn1_dev, dh, z_op, dh, n, dh, m.d_in, st);
  linear(x_task, m.d_in, m.w_gcn1_dev, dh, z_task, dh, num_queries, dh, m.d_in, st);
  launches += 2;
  const unsigned agg_threads = (unsigned)(dh < 256 ? ((dh + 31) / 32 * 32) : 256);
  for (int b0 = 0; b0 < num_queries; b0 += per_pass) {
    const int nb = num_queries - b0 < per_pass ? num_queries - b0 : per_pass;
    const size_t rows = (size_t)nb * (n + 1);
    k_aggregate<<<dim3((unsigned)(n + 1), (unsigned)nb), agg_threads, 0, st>>>(g, z_op, 0, z_task + (size_t)b0 * dh, (size_t)dh,
                                                                              h, dh);
    linear(h, dh, m.w_gcn2_dev, dh, gbuf, dh, (int)rows, dh, dh, st);
    k_aggregate<<<dim3((unsigned)(n + 1), (unsigned)nb), agg_threads, 0, st>>>(g, gbuf, (size_t)(n + 1) * dh,
                                                                              gbuf + (size_t)n * dh, (size_t)(n + 1) * dh, h, dh);
    for (int blk = 0; blk < 3; ++blk)  // [h Wa | h Wb | h Wc]
      linear(h, dh, m.w_mlp1_dev + (size_t)blk * dh * dm, dm, pbuf + (size_t)blk * dm, 3 * dm, (int)rows, dm, dh, st);
    const long long pairs = (long long)nb * g.num_edges;
    const unsigned blocks = (unsigned)((pairs + 7) / 8 < 148 * 2 ? (pairs + 7) / 8 : 148 * 2);
    k_edge_mlp<<<blocks, 256, mlp_smem, st>>>(g, pbuf, m.b_mlp1_dev, m.w_mlp2_dev, m.b_mlp2_dev, m.w_mlp3_dev, m.b_mlp3,
                                              scores + (size_t)b0 * g.num_edges, dm, nb, (size_t)g.num_edges);
    launches += 7;
  }
  return cudaGetLastError() == cudaSuccess ? launches : -1;
}

}  // namespace gf
