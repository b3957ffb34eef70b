// Fast path of the subsampled-Hadamard sketch (RMM_DIST_SORS_HADAMARD, bf16 mode):
//     out[j][:] = c * sum_n d_n * H[n][r_j] * B[n][:],   H[n][r] = (-1)^popcount(n & r),
// by a two-level Walsh-Hadamard transform over the token index instead of a dense contraction
// (Section 2.1 of the paper notes that such matrices have a fast matrix-by-vector product).
// With n = 128 a + b and r = 128 ra + rb the sign factors split, so
//     T[a][rb][:]  = sum_b H128[b][rb] * d_n * B[128 a + b][:]          (stage 1, inside 128-token blocks)
//     out[j][:]    = c * sum_a H_A[a][ra_j] * T[a][rb_j][:]             (stage 2, across the A = L/128 blocks)
// where L is the order of the Hadamard matrix (128 <= L <= 16384 here; other sizes take the dense
// kernel).  Both stages are the same shared-memory butterfly network on a [128 rows][64 columns]
// tile; they are bound by HBM: stage 1 reads B and writes T (bf16), stage 2 reads T once and
// writes only the B_proj rows that were drawn.  db (the column sums of B) is taken along in
// stage 1 per block and added up over the blocks, in order, by the rb = 0 CTAs of stage 2.
//
// S is the same matrix as in the dense kernels and in the CPU oracle: only the order of the
// floating-point additions differs (T is rounded to bf16 between the stages).
#pragma once
#include <cuda_bf16.h>
#include <stdint.h>

#include "sketch_rng.cuh"

namespace rmm {

constexpr int FW_ROWS = 128, FW_COLS = 64, FW_THREADS = 256;

// Drawn columns grouped by rb = r_j & 127: entries[offsets[rb] .. offsets[rb + 1]) = (j, ra_j).
struct SorsGroups {
  int* offsets;     // [129]
  int2* entries;    // [B_proj]
};

// One block: r_j for every sketch column, counted and scattered by rb.  The order inside a group
// depends on the order of the atomics; every entry is written out independently, so it does not
// affect the result.
__global__ void __launch_bounds__(1024)
sors_group_kernel(PhiloxKey pk, int64_t k, uint32_t mask, SorsGroups g, int* status, int clear_status) {
  __shared__ int count[128], start[129], fill[128];
  if (clear_status && threadIdx.x == 0) *status = 0;
  if (threadIdx.x < 128) { count[threadIdx.x] = 0; fill[threadIdx.x] = 0; }
  __syncthreads();
  for (int64_t j = threadIdx.x; j < k; j += blockDim.x) {
    uint32_t w[4];
    philox4x32_10(pk, (uint32_t)j, 0u, 0u, 3u, w);
    atomicAdd(&count[(w[0] & mask) & 127u], 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    int s = 0;
    for (int i = 0; i < 128; ++i) { start[i] = s; s += count[i]; }
    start[128] = s;
  }
  __syncthreads();
  if (threadIdx.x <= 128) g.offsets[threadIdx.x] = start[threadIdx.x];
  for (int64_t j = threadIdx.x; j < k; j += blockDim.x) {
    uint32_t w[4];
    philox4x32_10(pk, (uint32_t)j, 0u, 0u, 3u, w);
    const uint32_t r = w[0] & mask;
    const int rb = (int)(r & 127u);
    const int pos = start[rb] + atomicAdd(&fill[rb], 1);
    g.entries[pos] = make_int2((int)j, (int)(r >> 7));
  }
}

// Walsh-Hadamard transform over the rows of a [128][65] fp32 tile, all 64 columns at once.  Thread
// (rg, c) = (tid >> 6, tid & 63) takes the 32 rows 32 rg .. 32 rg + 31 of column c into registers
// (optionally negating the rows whose bit is set in dbits, and returning their plain sum), does the
// five stages over the low row bits there, writes them back, and after one barrier does the two
// stages over the high row bits for eight of the low indices: 6 passes over the tile in shared
// memory instead of 14.  `len` (a power of two <= 128) rows are transformed; rows >= len are not read.
__device__ __forceinline__ float fwht_tile(float (*tile)[FW_COLS + 1], int len, int tid, const uint32_t* dbits) {
  const int c = tid & 63, rg = tid >> 6;
  float sum = 0.f;
  const int low = len < 32 ? len : 32;           // rows per group that take part
  if (rg * 32 < len) {
    float x[32];
    const uint32_t bits = dbits ? dbits[rg] : 0u;
#pragma unroll
    for (int i = 0; i < 32; ++i) {
      x[i] = i < low ? tile[rg * 32 + i][c] : 0.f;
      sum += x[i];
      if ((bits >> i) & 1u) x[i] = -x[i];
    }
#pragma unroll
    for (int h = 1; h < 32; h <<= 1) {
      if (h < low) {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          if ((i & h) == 0) { const float u = x[i], v = x[i + h]; x[i] = u + v; x[i + h] = u - v; }
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 32; ++i)
      if (i < low) tile[rg * 32 + i][c] = x[i];
  }
  __syncthreads();
  if (len > 32) {
    const int groups = len / 32;                  // 2 or 4
#pragma unroll
    for (int q = 0; q < 8; ++q) {
      const int i = rg * 8 + q;
      float y0 = tile[i][c], y1 = tile[32 + i][c], y2 = groups == 4 ? tile[64 + i][c] : 0.f, y3 = groups == 4 ? tile[96 + i][c] : 0.f;
      const float s0 = y0 + y1, d0 = y0 - y1;
      if (groups == 4) {
        const float s1 = y2 + y3, d1 = y2 - y3;
        tile[i][c] = s0 + s1; tile[32 + i][c] = d0 + d1; tile[64 + i][c] = s0 - s1; tile[96 + i][c] = d0 - d1;
      } else {
        tile[i][c] = s0; tile[32 + i][c] = d0;
      }
    }
    __syncthreads();
  }
  return sum;
}

// Stage 1.  grid = (column slabs of 64, A blocks of 128 tokens).  B is [N][ldb] bf16 (this launch
// covers `width` columns starting at B); T is [A * 128][ldt] bf16; colsum (nullable) is [A][ldt] fp32.
__global__ void __launch_bounds__(FW_THREADS)
fwht_stage1_kernel(const __nv_bfloat16* __restrict__ B, int64_t ldb, int64_t N, int width, PhiloxKey pk,
                   __nv_bfloat16* __restrict__ T, int64_t ldt, float* __restrict__ colsum) {
  __shared__ float tile[FW_ROWS][FW_COLS + 1];
  __shared__ uint32_t dbits[4];
  const int tid = threadIdx.x;
  const int c0 = blockIdx.x * FW_COLS, a = blockIdx.y;
  if (tid == 0) {
    uint32_t w[4];
    philox4x32_10(pk, (uint32_t)a, 0u, 0u, 2u, w);      // the 128 sign bits of this block: tokens 128 a .. 128 a + 127
    dbits[0] = w[0]; dbits[1] = w[1]; dbits[2] = w[2]; dbits[3] = w[3];
  }
  __syncthreads();
  // 128 rows x 8 chunks of 8 columns; four chunks per thread
  for (int t = tid; t < FW_ROWS * 8; t += FW_THREADS) {
    const int b = t >> 3, ch = t & 7;
    const int64_t n = (int64_t)a * FW_ROWS + b;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (n < N && c0 + 8 * ch < width) v = __ldg(reinterpret_cast<const uint4*>(B + n * ldb + c0 + 8 * ch));
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      tile[b][8 * ch + 2 * i] = __uint_as_float(w[i] << 16);
      tile[b][8 * ch + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  __syncthreads();
  __shared__ float part[4][FW_COLS];
  const float psum = fwht_tile(tile, FW_ROWS, tid, dbits);     // signs d_n applied on the way in; psum = plain sum of 32 rows
  if (colsum != nullptr) {                                      // column sums of the block, the four row groups in order
    part[tid >> 6][tid & 63] = psum;
    __syncthreads();
    if (tid < FW_COLS && c0 + tid < width)
      colsum[(int64_t)a * ldt + c0 + tid] = (part[0][tid] + part[1][tid]) + (part[2][tid] + part[3][tid]);
  }
  for (int t = tid; t < FW_ROWS * 8; t += FW_THREADS) {
    const int rb = t >> 3, ch = t & 7;
    if (c0 + 8 * ch >= width) continue;
    uint32_t o[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      __nv_bfloat162 h = __floats2bfloat162_rn(tile[rb][8 * ch + 2 * i], tile[rb][8 * ch + 2 * i + 1]);
      o[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(T + ((int64_t)a * FW_ROWS + rb) * ldt + c0 + 8 * ch) = make_uint4(o[0], o[1], o[2], o[3]);
  }
}

// Stage 2.  grid = (column slabs of 64, 128 values of rb).  Transforms the A rows T[128 a + rb] over
// a and writes, for every drawn column j of this rb, out[j][c] = scale * U[ra_j][c]; the rb = 0
// CTAs also add the per-block column sums into ones_out (db).  out is [B_proj][ldo] bf16.
__global__ void __launch_bounds__(FW_THREADS)
fwht_stage2_kernel(const __nv_bfloat16* __restrict__ T, int64_t ldt, int A, int width, SorsGroups g, float scale,
                   __nv_bfloat16* __restrict__ out, int64_t ldo, const float* __restrict__ colsum,
                   __nv_bfloat16* __restrict__ ones_out) {
  __shared__ float tile[FW_ROWS][FW_COLS + 1];
  const int tid = threadIdx.x;
  const int c0 = blockIdx.x * FW_COLS, rb = blockIdx.y;
  const int j0 = g.offsets[rb], j1 = g.offsets[rb + 1];
  const bool do_db = (rb == 0 && colsum != nullptr && ones_out != nullptr);
  if (j0 == j1 && !do_db) return;
  if (j0 < j1) {
    for (int t = tid; t < A * 8; t += FW_THREADS) {
      const int a = t >> 3, ch = t & 7;
      uint4 v = make_uint4(0u, 0u, 0u, 0u);
      if (c0 + 8 * ch < width) v = *reinterpret_cast<const uint4*>(T + ((int64_t)a * FW_ROWS + rb) * ldt + c0 + 8 * ch);
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        tile[a][8 * ch + 2 * i] = __uint_as_float(w[i] << 16);
        tile[a][8 * ch + 2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
      }
    }
    __syncthreads();
    fwht_tile(tile, A, tid, nullptr);
    // 8 threads per output row (8 columns each), 32 rows per pass
    for (int e = j0 + (tid >> 3); e < j1; e += FW_THREADS / 8) {
      const int2 jr = g.entries[e];
      const int ch = tid & 7;
      if (c0 + 8 * ch >= width) continue;
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(tile[jr.y][8 * ch + 2 * i] * scale, tile[jr.y][8 * ch + 2 * i + 1] * scale);
        o[i] = *reinterpret_cast<uint32_t*>(&h);
      }
      *reinterpret_cast<uint4*>(out + (int64_t)jr.x * ldo + c0 + 8 * ch) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  }
  if (do_db && tid < FW_COLS && c0 + tid < width) {
    float s = 0.f;
    for (int a = 0; a < A; ++a) s += colsum[(int64_t)a * ldt + c0 + tid];
    ones_out[c0 + tid] = __float2bfloat16_rn(s);
  }
}

}  // namespace rmm
