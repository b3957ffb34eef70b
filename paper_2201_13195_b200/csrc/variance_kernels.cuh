// Variance diagnostics of the randomized weight gradient (Section 2.3): the four sums that
// Lemma 1 (Eq. 9), Lemma 2 (Eq. 11) and Theorem 1 (Eq. 13) are written in,
//     a = |X|_F^2,  b = |dY|_F^2,  c = sum_n |x_n|^2 |dy_n|^2,  d = |X^T dY|_F^2,
// and the quantities derived from them.  a, b, c come from one streaming pass over the rows of X
// and dY (row_norms_kernel, bound by HBM: every element is read once, 2 (D_in + D_out) bytes per token); d is the squared norm of
// the exact gradient dY^T X, which the tensor-core contraction kernel accumulates in its
// epilogue from the fp32 accumulators.  All partial sums are combined in a fixed order, so the
// result does not change from run to run.
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

namespace rmm {

constexpr int VAR_THREADS = 256;              // 8 warps, one row at a time each
constexpr int VAR_WARPS = VAR_THREADS / 32;
constexpr int VAR_BLOCKS_PER_SM = 4;          // resident blocks the launch is sized for (<= 64 registers per thread)
constexpr int VAR_OUT = 8;                    // doubles written by variance_finish_kernel

__device__ __forceinline__ float sumsq8(const uint4& v) {
  const uint32_t w[4] = {v.x, v.y, v.z, v.w};
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float lo = __uint_as_float(w[j] << 16), hi = __uint_as_float(w[j] & 0xffff0000u);
    s0 = fmaf(lo, lo, s0);
    s1 = fmaf(hi, hi, s1);
  }
  return s0 + s1;
}

// Sum of squares of one bf16 row of d elements (d a multiple of 8, row 16-byte aligned), over the
// warp.  Eight independent 16-byte loads per lane are in flight at a time: with 32 resident warps
// that is 128 KB per SM, enough to cover the memory latency at full HBM bandwidth.
__device__ __forceinline__ float row_sumsq_bf16(const __nv_bfloat16* row, int64_t d, int lane) {
  const uint4* p = reinterpret_cast<const uint4*>(row);
  const int64_t chunks = d >> 3;
  float s = 0.f;
  int64_t i = lane;
  for (; i + 7 * 32 < chunks; i += 8 * 32) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) v[u] = __ldg(p + i + 32 * u);
#pragma unroll
    for (int u = 0; u < 8; ++u) s += sumsq8(v[u]);
  }
  for (; i < chunks; i += 32) s += sumsq8(__ldg(p + i));
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return s;
}

// partial[block][3] = (sum |x_n|^2, sum |dy_n|^2, sum |x_n|^2 |dy_n|^2) over the rows of the block.
// Every warp owns a contiguous range of rows (ranges differ by one row at most); the grid is the
// number of blocks that are resident at once, so there is no second wave.
__global__ void __launch_bounds__(VAR_THREADS, VAR_BLOCKS_PER_SM)
row_norms_kernel(const __nv_bfloat16* __restrict__ X, const __nv_bfloat16* __restrict__ dY, int64_t N, int64_t D_in,
                 int64_t D_out, double* __restrict__ partial) {
  __shared__ double sm[VAR_WARPS][3];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int64_t gw = (int64_t)blockIdx.x * VAR_WARPS + warp, nw = (int64_t)gridDim.x * VAR_WARPS;
  const int64_t r_begin = gw * N / nw, r_end = (gw + 1) * N / nw;
  double a = 0.0, b = 0.0, c = 0.0;
  for (int64_t n = r_begin; n < r_end; ++n) {
    const float sx = row_sumsq_bf16(X + n * D_in, D_in, lane);
    const float sy = row_sumsq_bf16(dY + n * D_out, D_out, lane);
    a += (double)sx;
    b += (double)sy;
    c += (double)sx * (double)sy;
  }
  if (lane == 0) { sm[warp][0] = a; sm[warp][1] = b; sm[warp][2] = c; }
  __syncthreads();
  if (threadIdx.x < 3) {
    double s = 0.0;
    for (int w = 0; w < VAR_WARPS; ++w) s += sm[w][threadIdx.x];
    partial[(int64_t)blockIdx.x * 3 + threadIdx.x] = s;
  }
}

// One warp: lane l adds elements l, l + 32, ... in order, then a fixed shuffle tree.
__device__ __forceinline__ double ordered_sum(const double* v, int n, int stride, int lane) {
  double s = 0.0;
  for (int i = lane; i < n; i += 32) s += v[(int64_t)i * stride];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  return s;
}

// out[0..3] = a, b, c, d;  out[4] = D^2_SGD (Eq. 9);  out[5] = D^2_RMM for the given sketch with
// the fourth moment of its entries kept;  out[6] = D^2_RMM as Eq. 11 prints it;  out[7] = alpha (Eq. 13).
__global__ void variance_finish_kernel(const double* __restrict__ row_partial, int row_blocks,
                                       const double* __restrict__ gemm_partial, int gemm_entries, int64_t N,
                                       int64_t b_proj, int dist, double* __restrict__ out) {
  const int lane = threadIdx.x & 31;
  const double a = ordered_sum(row_partial + 0, row_blocks, 3, lane);
  const double b = ordered_sum(row_partial + 1, row_blocks, 3, lane);
  const double c = ordered_sum(row_partial + 2, row_blocks, 3, lane);
  const double d = ordered_sum(gemm_partial, gemm_entries, 1, lane);
  if (threadIdx.x == 0) {
    const double n = (double)N, k = (double)b_proj;
    out[0] = a; out[1] = b; out[2] = c; out[3] = d;
    out[4] = n / (n - 1.0) * c - d / (n - 1.0);
    out[5] = dist == 0 ? (a * b + d) / k : dist == 1 ? (a * b + d - 2.0 * c) / k : 0.0;
    out[6] = (a * b - d) / k;
    out[7] = (a * b) > 0.0 ? d / (a * b) : 0.0;
  }
}

}  // namespace rmm
