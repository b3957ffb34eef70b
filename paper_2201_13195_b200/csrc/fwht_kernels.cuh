// Fast path of the subsampled-Hadamard sketch (RMM_DIST_SORS_HADAMARD, bf16 mode):
//     out[j][:] = c * sum_n d_n * H[n][r_j] * B[n][:],   H[n][r] = (-1)^popcount(n & r),
// by a two-level Walsh-Hadamard transform over the token index instead of a dense contraction
// (Section 2.1 of the paper notes that such matrices have a fast matrix-by-vector product).
// With n = 128 a + b and r = 128 ra + rb the sign factors split, so
//     T[a][rb][:]  = sum_b H128[b][rb] * d_n * B[128 a + b][:]          (stage 1, inside 128-token blocks)
//     out[j][:]    = c * sum_a H_A[a][ra_j] * T[a][rb_j][:]             (stage 2, across the A = L/128 blocks)
// where L is the order of the Hadamard matrix (128 <= L <= 16384 here; other sizes take the dense
// kernel).  Both stages are the same butterfly network (registers, one pass through shared memory)
// on a [128 rows][64 columns] tile; they are bound by HBM: stage 1 reads B and writes T (bf16), stage 2 reads T once and
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
// affect the result.  Run by the first block of the first stage-1 launch of a sketch (stage 2, which reads the
// groups, is a later launch on the same stream): the block is the first to be scheduled, and the few
// microseconds it spends here are over long before the other blocks of the launch are.
__device__ __forceinline__ void sors_group_block(const PhiloxKey& pk, int64_t k, uint32_t mask, SorsGroups g) {
  __shared__ int count[128], start[129], fill[128];
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
  __syncthreads();
}

// The 128-point Walsh-Hadamard transform of a [128 rows][64 columns] tile, rows = 16 g + i.
// A thread owns two adjacent columns (lane -> columns 2 lane, 2 lane + 1: a warp reads or writes
// one 128-byte row segment per instruction) and, in phase 1, the 16 rows i = 0..15 of group g = its
// warp: four butterfly stages in registers.  The tile then goes through shared memory once; in
// phase 2 warp w takes the rows i = 2 w, 2 w + 1 of all eight groups: three stages over g.
// Rows that do not exist are zeros: for the Sylvester matrix the first A outputs of the 128-point
// transform of a zero-padded vector are its A-point transform, so one code path serves every A.
__device__ __forceinline__ void wht16(float (&x)[16]) {
#pragma unroll
  for (int h = 1; h < 16; h <<= 1) {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if ((i & h) == 0) { const float u = x[i], v = x[i + h]; x[i] = u + v; x[i + h] = u - v; }
  }
}
__device__ __forceinline__ void wht8(float (&y)[8]) {
#pragma unroll
  for (int h = 1; h < 8; h <<= 1) {
#pragma unroll
    for (int g = 0; g < 8; ++g)
      if ((g & h) == 0) { const float u = y[g], v = y[g + h]; y[g] = u + v; y[g + h] = u - v; }
  }
}
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

// Stage 1.  grid = (column slabs of 64, A blocks of 128 tokens); block (0, 0) also builds the column groups.  B is [N][ldb] bf16 (this launch
// covers `width` columns starting at B); T is [A * 128][ldt] bf16; colsum (nullable) is [A][ldt] fp32.
__global__ void __launch_bounds__(FW_THREADS)
fwht_stage1_kernel(const __nv_bfloat16* __restrict__ B, int64_t ldb, int64_t N, int width, PhiloxKey pk,
                   __nv_bfloat16* __restrict__ T, int64_t ldt, float* __restrict__ colsum, SorsGroups groups, int64_t k,
                   uint32_t mask, int* status, int clear_status) {
  __shared__ float2 tile[FW_ROWS][FW_COLS / 2];
  __shared__ float2 part[FW_THREADS / 32][FW_COLS / 2];
  const int tid = threadIdx.x, w = tid >> 5, lane = tid & 31;
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    if (clear_status && tid == 0) *status = 0;
    if (groups.offsets != nullptr) sors_group_block(pk, k, mask, groups);   // only in the first launch of a sketch
  }
  const int c0 = blockIdx.x * FW_COLS, a = blockIdx.y;
  const int col = c0 + 2 * lane;
  const bool in_cols = col < width;                       // width is a multiple of 8: a column pair is all in or all out
  uint32_t dw[4];
  philox4x32_10(pk, (uint32_t)a, 0u, 0u, 2u, dw);         // the 128 sign bits of tokens 128 a .. 128 a + 127
  const uint32_t bits = (dw[w >> 1] >> ((w & 1) * 16)) & 0xffffu;   // those of rows 16 w .. 16 w + 15
  float x0[16], x1[16];
  uint32_t raw[16];
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    const int64_t n = (int64_t)a * FW_ROWS + 16 * w + i;
    raw[i] = (in_cols && n < N) ? __ldg(reinterpret_cast<const uint32_t*>(B + n * ldb + col)) : 0u;
  }
  float s0 = 0.f, s1 = 0.f;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    x0[i] = __uint_as_float(raw[i] << 16);
    x1[i] = __uint_as_float(raw[i] & 0xffff0000u);
    s0 += x0[i];
    s1 += x1[i];
    if ((bits >> i) & 1u) { x0[i] = -x0[i]; x1[i] = -x1[i]; }
  }
  wht16(x0);
  wht16(x1);
#pragma unroll
  for (int i = 0; i < 16; ++i) tile[16 * w + i][lane] = make_float2(x0[i], x1[i]);
  part[w][lane] = make_float2(s0, s1);
  __syncthreads();
  if (colsum != nullptr && w == 0 && in_cols) {            // column sums of the block: the eight row groups in order
    float t0 = 0.f, t1 = 0.f;
#pragma unroll
    for (int g = 0; g < FW_THREADS / 32; ++g) { t0 += part[g][lane].x; t1 += part[g][lane].y; }
    *reinterpret_cast<float2*>(colsum + (int64_t)a * ldt + col) = make_float2(t0, t1);
  }
#pragma unroll
  for (int ii = 0; ii < 2; ++ii) {
    const int i = 2 * w + ii;
    float y0[8], y1[8];
#pragma unroll
    for (int g = 0; g < 8; ++g) { const float2 v = tile[16 * g + i][lane]; y0[g] = v.x; y1[g] = v.y; }
    wht8(y0);
    wht8(y1);
    if (in_cols) {
#pragma unroll
      for (int g = 0; g < 8; ++g)
        *reinterpret_cast<uint32_t*>(T + ((int64_t)a * FW_ROWS + 16 * g + i) * ldt + col) = pack2_bf16(y0[g], y1[g]);
    }
  }
}

// Stage 2.  grid = (column slabs of 64, 128 values of rb).  Transforms the A rows T[128 a + rb] over
// a and writes, for every drawn column j of this rb, out[j][c] = scale * U[ra_j][c]; the rb = 0
// CTAs also add the per-block column sums into ones_out (db).  out is [B_proj][ldo] bf16.
__global__ void __launch_bounds__(FW_THREADS)
fwht_stage2_kernel(const __nv_bfloat16* __restrict__ T, int64_t ldt, int A, int width, SorsGroups g, float scale,
                   __nv_bfloat16* __restrict__ out, int64_t ldo, const float* __restrict__ colsum,
                   __nv_bfloat16* __restrict__ ones_out) {
  __shared__ float2 tile[FW_ROWS][FW_COLS / 2];
  const int tid = threadIdx.x, w = tid >> 5, lane = tid & 31;
  const int c0 = blockIdx.x * FW_COLS, rb = blockIdx.y;
  const int col = c0 + 2 * lane;
  const bool in_cols = col < width;
  const int j0 = g.offsets[rb], j1 = g.offsets[rb + 1];
  const bool do_db = (rb == 0 && colsum != nullptr && ones_out != nullptr);
  if (j0 == j1 && !do_db) return;
  if (j0 < j1) {
    float x0[16], x1[16];
    uint32_t raw[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
      const int a = 16 * w + i;
      raw[i] = (in_cols && a < A) ? *reinterpret_cast<const uint32_t*>(T + ((int64_t)a * FW_ROWS + rb) * ldt + col) : 0u;
    }
#pragma unroll
    for (int i = 0; i < 16; ++i) { x0[i] = __uint_as_float(raw[i] << 16); x1[i] = __uint_as_float(raw[i] & 0xffff0000u); }
    wht16(x0);
    wht16(x1);
#pragma unroll
    for (int i = 0; i < 16; ++i) tile[16 * w + i][lane] = make_float2(x0[i], x1[i]);
    __syncthreads();
    float y0[2][8], y1[2][8];
#pragma unroll
    for (int ii = 0; ii < 2; ++ii) {
#pragma unroll
      for (int q = 0; q < 8; ++q) { const float2 v = tile[16 * q + 2 * w + ii][lane]; y0[ii][q] = v.x; y1[ii][q] = v.y; }
      wht8(y0[ii]);
      wht8(y1[ii]);
    }
    __syncthreads();                                         // everyone has read its inputs: the tile takes the outputs
#pragma unroll
    for (int ii = 0; ii < 2; ++ii) {
#pragma unroll
      for (int q = 0; q < 8; ++q) tile[16 * q + 2 * w + ii][lane] = make_float2(y0[ii][q], y1[ii][q]);
    }
    __syncthreads();
    // the drawn rows of this rb: one warp per entry and pass, a 4-byte store per lane
    for (int e = j0 + w; e < j1; e += FW_THREADS / 32) {
      const int2 jr = g.entries[e];
      if (in_cols) {
        const float2 v = tile[jr.y][lane];
        *reinterpret_cast<uint32_t*>(out + (int64_t)jr.x * ldo + col) = pack2_bf16(v.x * scale, v.y * scale);
      }
    }
  }
  if (do_db && tid < FW_COLS && c0 + tid < width) {
    float s = 0.f;
    for (int a = 0; a < A; ++a) s += colsum[(int64_t)a * ldt + c0 + tid];
    ones_out[c0 + tid] = __float2bfloat16_rn(s);
  }
}

}  // namespace rmm
