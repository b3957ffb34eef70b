// Plain fp32-FMA kernels: the fp32 mode of the layer (whose 1e-5 tolerance rules out
// reduced-precision tensor-core inputs), the exact bias gradient, and the dump of S.
//
// One tiled kernel serves the five contractions of Algorithm 1:
//   C[m][n] = alpha * sum_k A(m,k) * B(n,k) (+ bias[n])
// with A and B addressed through element strides, or with A generated on the fly as
// A(m,k) = P[token k][sketch column m] (the transposed sketch matrix).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "sketch_rng.cuh"

namespace rmm {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct SimtGemmArgs {
  const void* A; int64_t a_sm, a_sk;   // A(m,k) = A[m*a_sm + k*a_sk]   (unused when generated)
  const void* B; int64_t b_sn, b_sk;   // B(n,k) = B[n*b_sn + k*b_sk]
  void* C; int64_t ldc;                // C[m*ldc + n]
  const void* bias;                    // [n] or nullptr
  int64_t M, N, K;
  float alpha;
  int dist;                            // generated A only
  uint32_t sors_mask;                  // dist 3: order of the Hadamard matrix - 1
};

// 32 x 64 output tiles (the layer's fp32 shapes are small: with 64 x 64 tiles the 512-token configuration gave
// 48 to 144 blocks for 148 SMs), 16-deep K slices; the next slice's global loads are issued into registers
// before the current slice is multiplied, so their latency overlaps the arithmetic.
constexpr int SIMT_BM = 32, SIMT_BN = 64, SIMT_BK = 16, SIMT_THREADS = 256;
constexpr int SIMT_A_PER_THREAD = SIMT_BM * SIMT_BK / SIMT_THREADS;   // 2
constexpr int SIMT_B_PER_THREAD = SIMT_BN * SIMT_BK / SIMT_THREADS;   // 4

template <typename T, bool GEN_A>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_gemm_kernel(SimtGemmArgs g, PhiloxKey pk) {
  __shared__ float As[SIMT_BK][SIMT_BM + 4];
  __shared__ float Bs[SIMT_BK][SIMT_BN + 4];
  const int tid = threadIdx.x;
  const int64_t m0 = (int64_t)blockIdx.y * SIMT_BM, n0 = (int64_t)blockIdx.x * SIMT_BN;
  const int tx = tid & 15, ty = tid >> 4;   // 16 x 16 threads, 2 x 4 outputs each
  float acc[2][4] = {};
  const T* A = reinterpret_cast<const T*>(g.A);
  const T* B = reinterpret_cast<const T*>(g.B);

  // element e of a slice of A / B -> (row in tile, k in slice); the orientation is chosen so that consecutive
  // threads walk the unit-stride index
  auto a_coord = [&](int e, int& mm, int& kk) {
    if (g.a_sk == 1) { kk = e % SIMT_BK; mm = e / SIMT_BK; } else { mm = e % SIMT_BM; kk = e / SIMT_BM; }
  };
  auto b_coord = [&](int e, int& nn, int& kk) {
    if (g.b_sk == 1) { kk = e % SIMT_BK; nn = e / SIMT_BK; } else { nn = e % SIMT_BN; kk = e / SIMT_BN; }
  };
  float ra[SIMT_A_PER_THREAD], rb[SIMT_B_PER_THREAD];
  auto fetch = [&](int64_t k0) {
    if (!GEN_A) {
#pragma unroll
      for (int i = 0; i < SIMT_A_PER_THREAD; ++i) {
        int mm, kk;
        a_coord(tid + i * SIMT_THREADS, mm, kk);
        const int64_t m = m0 + mm, k = k0 + kk;
        ra[i] = (m < g.M && k < g.K) ? to_f32<T>(A[m * g.a_sm + k * g.a_sk]) : 0.0f;
      }
    }
#pragma unroll
    for (int i = 0; i < SIMT_B_PER_THREAD; ++i) {
      int nn, kk;
      b_coord(tid + i * SIMT_THREADS, nn, kk);
      const int64_t n = n0 + nn, k = k0 + kk;
      rb[i] = (n < g.N && k < g.K) ? to_f32<T>(B[n * g.b_sn + k * g.b_sk]) : 0.0f;
    }
  };
  fetch(0);
  for (int64_t k0 = 0; k0 < g.K; k0 += SIMT_BK) {
    if (GEN_A) {
      // 32 sketch columns x 16 tokens: 64 tasks of 8 tokens each.
      if (tid < 2 * SIMT_BM) {
        const int r = tid >> 1, h = tid & 1;
        const int64_t j = m0 + r, n8 = k0 + 8 * h;
        float z[8];
        if (g.dist == 0) {
          gaussian_8(pk, (uint32_t)n8, (uint32_t)j, z);
          if (sizeof(T) == 2) {
#pragma unroll
            for (int i = 0; i < 8; ++i) z[i] = __bfloat162float(__float2bfloat16_rn(z[i]));
          }
        } else if (g.dist == 1) {
          uint32_t w[4];
          rademacher_128(pk, (uint32_t)(n8 >> 7), (uint32_t)j, w);
          const uint32_t bits = w[(n8 & 127) >> 5] >> (n8 & 31);
#pragma unroll
          for (int i = 0; i < 8; ++i) z[i] = ((bits >> i) & 1u) ? -1.0f : 1.0f;
        } else if (g.dist == 3) {
          const uint32_t bits = sors_sign_bits_8(pk, (uint32_t)n8, (uint32_t)j, g.sors_mask);
#pragma unroll
          for (int i = 0; i < 8; ++i) z[i] = ((bits >> i) & 1u) ? -1.0f : 1.0f;
        } else if (g.dist == 4) {
          dct_8(pk, (uint32_t)n8, (uint32_t)j, g.sors_mask, z);
          if (sizeof(T) == 2) {
#pragma unroll
            for (int i = 0; i < 8; ++i) z[i] = __bfloat162float(__float2bfloat16_rn(z[i]));
          }
        } else {
#pragma unroll
          for (int i = 0; i < 8; ++i) z[i] = (n8 + i == j) ? 1.0f : 0.0f;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) As[8 * h + i][r] = (j < g.M && n8 + i < g.K) ? z[i] : 0.0f;
      }
    } else {
#pragma unroll
      for (int i = 0; i < SIMT_A_PER_THREAD; ++i) {
        int mm, kk;
        a_coord(tid + i * SIMT_THREADS, mm, kk);
        As[kk][mm] = ra[i];
      }
    }
#pragma unroll
    for (int i = 0; i < SIMT_B_PER_THREAD; ++i) {
      int nn, kk;
      b_coord(tid + i * SIMT_THREADS, nn, kk);
      Bs[kk][nn] = rb[i];
    }
    __syncthreads();
    if (k0 + SIMT_BK < g.K) fetch(k0 + SIMT_BK);      // in flight while this slice is multiplied
#pragma unroll
    for (int kk = 0; kk < SIMT_BK; ++kk) {
      float a[2], b[4];
#pragma unroll
      for (int i = 0; i < 2; ++i) a[i] = As[kk][ty * 2 + i];
#pragma unroll
      for (int i = 0; i < 4; ++i) b[i] = Bs[kk][tx * 4 + i];
#pragma unroll
      for (int i = 0; i < 2; ++i)
#pragma unroll
        for (int jn = 0; jn < 4; ++jn) acc[i][jn] = fmaf(a[i], b[jn], acc[i][jn]);
    }
    __syncthreads();
  }
  T* C = reinterpret_cast<T*>(g.C);
  const T* bias = reinterpret_cast<const T*>(g.bias);
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int64_t m = m0 + ty * 2 + i;
    if (m >= g.M) continue;
#pragma unroll
    for (int jn = 0; jn < 4; ++jn) {
      const int64_t n = n0 + tx * 4 + jn;
      if (n >= g.N) continue;
      float v = acc[i][jn] * g.alpha;
      if (bias) v += to_f32<T>(bias[n]);
      C[m * g.ldc + n] = from_f32<T>(v);
    }
  }
}

// db partial sums (Eq. 3): block (x = group of 256 columns, y = row slice) adds its rows
// of dY column by column; warp shuffles are not needed across columns because every thread
// owns one column, the cross-slice sum is done by db_finish_kernel in a fixed order.
template <typename T>
__global__ void __launch_bounds__(256)
db_partial_kernel(const T* __restrict__ dY, int64_t N, int64_t D_out, int rows_per_slice, float* __restrict__ partial) {
  const int64_t col = (int64_t)blockIdx.x * 256 + threadIdx.x;
  if (col >= D_out) return;
  const int64_t r0 = (int64_t)blockIdx.y * rows_per_slice;
  const int64_t r1 = min(N, r0 + rows_per_slice);
  float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
  int64_t r = r0;
  for (; r + 3 < r1; r += 4) {
    acc0 += to_f32<T>(dY[r * D_out + col]);
    acc1 += to_f32<T>(dY[(r + 1) * D_out + col]);
    acc2 += to_f32<T>(dY[(r + 2) * D_out + col]);
    acc3 += to_f32<T>(dY[(r + 3) * D_out + col]);
  }
  for (; r < r1; ++r) acc0 += to_f32<T>(dY[r * D_out + col]);
  partial[(int64_t)blockIdx.y * D_out + col] = (acc0 + acc1) + (acc2 + acc3);
}

template <typename T>
__global__ void db_finish_kernel(const float* __restrict__ partial, int slices, int64_t D_out, T* __restrict__ db) {
  const int64_t col = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (col >= D_out) return;
  float acc = 0.f;
  for (int s = 0; s < slices; ++s) acc += partial[(int64_t)s * D_out + col];
  db[col] = from_f32<T>(acc);
}

// Dump of the unscaled sketch entries P [N, B_proj] (debug entry point).
template <typename T>
__global__ void dump_sketch_kernel(PhiloxKey pk, int dist, int64_t N, int64_t k, T* __restrict__ out) {
  const int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= N * k) return;
  const int64_t n = idx / k, j = idx % k;
  out[idx] = from_f32<T>(sketch_entry(pk, dist, n, j, sizeof(T) == 2, sors_mask_for(N)));
}

// The normal transform applied to caller-given words (debug entry point).
__global__ void gauss_words_kernel(const uint32_t* __restrict__ words, int64_t n, float* __restrict__ out) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float a, b;
  gauss_pair(words[i], a, b);
  out[2 * i] = a;
  out[2 * i + 1] = b;
}

}  // namespace rmm
