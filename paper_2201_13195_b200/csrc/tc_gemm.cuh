// Tensor-core contraction kernel for the bf16 mode (sm_100a): C = alpha * A B^T (+ bias),
// bf16 operands, fp32 accumulation in tensor memory, persistent CTA pairs.
//
// The three dense contractions of Algorithm 1 whose operands all live in memory differ only
// in the operand layouts (the two sketch contractions are in tc_sketch.cuh):
//   A_K   : A[m][k] row-major (k contiguous), fetched by TMA           (Y: X,  dX: dY)
//   A_MN  : A given as [k][m] row-major (m contiguous), fetched by TMA (dW: G = S^T dY)
//   B_K   : B[n][k] row-major (k contiguous)                           (Y: W)
//   B_MN  : B given as [k][n] row-major (n contiguous)                 (dX: W, dW: X_proj)
// "MN-major" operands are consumed in place through the transpose bits of the tcgen05
// instruction descriptor; nothing is transposed in memory.
//
// CTA pairs.  Two CTAs on neighbouring SMs (a cluster of two) compute one 256 x 256 output tile
// with tcgen05.mma.cta_group::2: each CTA stages its own 128 rows of A and only half (128) of
// the tile's B columns, the hardware feeds both halves of B to both tensor cores, and each CTA
// keeps the 128 x 256 accumulator of its rows in its own tensor memory.  Per MMA this halves
// the B bytes an SM pulls from L2 and pushes through its shared memory, which is what limits a
// one-CTA 128 x 256 tile, and it makes room for six pipeline stages instead of four.
//
// Epilogue.  Each epilogue warp owns 32 rows of the accumulator.  Per 64 output columns it reads
// them out of tensor memory, applies alpha and the bias, rounds to bf16, writes a [32 rows][128 B]
// box into shared memory (128-byte swizzle) and hands it to a TMA store; two boxes per warp, so
// the conversion of one overlaps the store of the other.  The stores reach L2 as whole 128-byte
// lines (per-lane 16-byte stores of row fragments cost the Y GEMM a sixth of its time), and
// the tensor map clips rows and columns beyond the matrix.
//
// Warp roles per CTA: warp 0 = TMA producer (its halves), warp 1 = tensor-memory owner and, in
// the leader CTA (even rank), MMA issuer; warps 2..5 = epilogue.  Barriers: full (leader; TMA
// bytes of both CTAs landed), empty (both; tcgen05.commit from the leader: the MMAs that read
// the stage have retired), accfull (both; all MMAs of the tile retired), accempty (leader; the
// epilogues of both CTAs have read the accumulator buffer out of tensor memory).  Two
// accumulator buffers: the MMAs of tile i+1 overlap the epilogue of tile i.
#pragma once
#include "tc_common.cuh"

namespace rmm {
namespace tc {

constexpr int BM = 128;                       // rows of A (and of the accumulator) per CTA
constexpr int PAIR_M = 2 * BM;                // rows of a pair tile
constexpr int BN = 256, BK = 64, UMMA_K = 16;
constexpr int BN_HALF = BN / 2;               // B columns staged by each CTA
constexpr int STAGES = 6;
constexpr int A_BYTES = BM * BK * 2;          // 16 KiB
constexpr int B_BYTES = BN_HALF * BK * 2;     // 16 KiB
constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
constexpr int SLAB_BYTES = 64 * BK * 2;       // one [64 k][64 mn] MN-major slab, 8 KiB
constexpr int TMEM_COLS = 512;                // two 128 x 256 fp32 accumulators per CTA
constexpr int NEPI = 4;                       // epilogue warps: one per tensor-memory lane quarter
constexpr int EPI_COLS = 64;                  // output columns per store box: 128 bytes of bf16
constexpr int EPI_BOX_BYTES = 32 * EPI_COLS * 2;   // [32 rows][64 columns] = 4 KiB
constexpr int EPI_BYTES = NEPI * 2 * EPI_BOX_BYTES;   // two boxes per epilogue warp
constexpr int GEMM_SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 /*alignment slack*/ + 256 /*barriers*/;

enum : int { A_K = 0, A_MN = 1 };
enum : int { B_K = 0, B_MN = 1 };

struct GemmParams {
  int64_t M, N, K;
  const void* bias;   // bf16 [N] or nullptr
  float alpha;
  int* status;        // workspace status word
  int clear_status;   // first kernel of a call: reset the status word (a timeout can only be recorded seconds later)
  double* sumsq;      // nullptr, or [gridDim.x][NEPI]: every epilogue warp adds up the squares of the (scaled,
                      // biased, unrounded) results it converts, for |C|_F^2 (variance diagnostics)
};

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}

template <int AMODE, int BMODE>
__global__ void __launch_bounds__(64 + 32 * NEPI, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, GemmParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * STAGE_BYTES + EPI_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto accempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  MBAR_PEEK_DECLARE();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
  if (p.clear_status && blockIdx.x == 0 && threadIdx.x == 0) *p.status = 0;
  const bool leader = rank == 0;
  // Persistent: this pair takes pair tiles pair, pair + num_pairs, ...  Tile t is
  // (m = t / tiles_n, n = t % tiles_n): the pairs of one wave share a few A row blocks (the large,
  // token-sized operand is then read from HBM once) and sweep all of B (weights, L2 resident).
  const int pair = (int)(blockIdx.x >> 1), num_pairs = (int)(gridDim.x >> 1);
  const int tiles_n = (int)((p.N + BN - 1) / BN);
  const int num_tiles = (int)((p.M + PAIR_M - 1) / PAIR_M) * tiles_n;
  const int num_kb = (int)((p.K + BK - 1) / BK);

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accfull_bar(b), 1);
      mbar_init(accempty_bar(b), 2 * NEPI);     // one arrival per epilogue warp of either CTA
    }
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32(tmem_slot), TMEM_COLS);
    tmem_relinquish_pair();
  }
  tc_fence_before();
  cluster_sync_all();      // both CTAs' barriers and tensor memory exist before anyone signals across
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer: this CTA's halves
    if (lane == 0) {
      tma_prefetch_desc(&tmA);
      tma_prefetch_desc(&tmB);
      const uint32_t leader_delta = mapa_shared(bar0, 0) - bar0;   // 0 in the leader itself
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs) {
        const int m0 = (tile / tiles_n) * PAIR_M + (int)rank * BM;
        const int n0 = (tile % tiles_n) * BN + (int)rank * BN_HALF;
        for (int kb = 0; kb < num_kb; ++kb) {
          if (!mbar_wait_cluster(empty_bar(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
          const uint32_t a_smem = sbase + s * STAGE_BYTES, b_smem = a_smem + A_BYTES;
          if (leader) mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);   // bytes of both CTAs
          const uint32_t full_leader = full_bar(s) + leader_delta;
          const int k0 = kb * BK;
          if (AMODE == A_K) {
            tma_load_2d_pair(a_smem, &tmA, full_leader, k0, m0);
          } else {
#pragma unroll
            for (int sl = 0; sl < BM / 64; ++sl)
              tma_load_2d_pair(a_smem + sl * SLAB_BYTES, &tmA, full_leader, m0 + 64 * sl, k0);
          }
          if (BMODE == B_K) {
            tma_load_2d_pair(b_smem, &tmB, full_leader, k0, n0);
          } else {
#pragma unroll
            for (int sl = 0; sl < BN_HALF / 64; ++sl)
              tma_load_2d_pair(b_smem + sl * SLAB_BYTES, &tmB, full_leader, n0 + 64 * sl, k0);
          }
          if (++s == STAGES) { s = 0; ph ^= 1u; }
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    // ------------------------------------------------------------ MMA issuer (leader CTA only)
    // The whole warp runs the loop, so that descriptors and addresses stay warp-uniform (the
    // tcgen05 operands live in uniform registers); one elected lane issues.
    if (leader) {
      constexpr uint32_t idesc = instr_desc_bf16(PAIR_M, BN, AMODE == A_MN, BMODE == B_MN);
      // Descriptors are built once; a stage or K step only adds to the 14-bit start-address
      // field (16-byte units), which never carries out of it.  The same shared-memory offsets
      // are used in both CTAs.
      const uint64_t adesc0 = (AMODE == A_MN) ? smem_desc_sw128(sbase, SLAB_BYTES, 1024) : smem_desc_sw128(sbase, 16, 1024);
      const uint64_t bdesc0 = (BMODE == B_MN) ? smem_desc_sw128(sbase + A_BYTES, SLAB_BYTES, 1024)
                                              : smem_desc_sw128(sbase + A_BYTES, 16, 1024);
      constexpr uint32_t a_kstep = ((AMODE == A_MN) ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      constexpr uint32_t b_kstep = ((BMODE == B_MN) ? UMMA_K * 128 : UMMA_K * 2) >> 4;
      const uint32_t peer_delta = mapa_shared(bar0, 1) - bar0;
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;
      int it = 0;                               // tiles done by this pair
      MBAR_PEEK_CLUSTER(0, full_bar(0), 0u);    // every stage's barrier is tested one stage ahead
      for (int tile = pair; tile < num_tiles && ok; tile += num_pairs, ++it) {
        const int buf = it & 1;
        // the epilogues of both CTAs must have drained this accumulator buffer (two tiles ago)
        ok = (mbar_wait_cluster_warp(accempty_bar(buf), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag, p.status));
        if (!ok) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < num_kb; ++kb) {
          uint32_t ready;
          MBAR_PEEK_RESULT(0, ready);
          if (!__all_sync(0xffffffffu, ready != 0)) {
            ok = (mbar_wait_cluster_warp(full_bar(s), ph, abort_flag, p.status));
            if (!ok) break;
          }
          tc_fence_after();
          const uint64_t ad = adesc0 + (uint64_t)(s * (STAGE_BYTES >> 4));
          const uint64_t bd = bdesc0 + (uint64_t)(s * (STAGE_BYTES >> 4));
          const int s_next = (s + 1 == STAGES) ? 0 : s + 1;
          const uint32_t ph_next = (s_next == 0) ? (ph ^ 1u) : ph;
          const bool issuer = elect_one();
          if (issuer) {
#pragma unroll
            for (int j = 0; j < BK / UMMA_K; ++j)
              umma_bf16_pair(d_tmem, ad + j * a_kstep, bd + j * b_kstep, idesc, (kb | j) != 0 ? 1u : 0u);
          }
          MBAR_PEEK_CLUSTER(0, full_bar(s_next), ph_next);   // travels while the commits are issued
          if (issuer) {
            umma_commit_pair(empty_bar(s));
            umma_commit_pair(empty_bar(s) + peer_delta);
          }
          __syncwarp();
          s = s_next;
          ph = ph_next;
        }
        if (ok) {
          if (elect_one()) {
            umma_commit_pair(accfull_bar(buf));
            umma_commit_pair(accfull_bar(buf) + peer_delta);
          }
          __syncwarp();
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ epilogue (overlaps the next tile's MMAs)
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const __nv_bfloat16* bias = reinterpret_cast<const __nv_bfloat16*>(p.bias);
    const uint32_t accempty_leader0 = mapa_shared(accempty_bar(0), 0);
    const uint32_t box0 = sbase + STAGES * STAGE_BYTES + (uint32_t)(warp - 2) * 2 * EPI_BOX_BYTES;   // this warp's two boxes
    const uint32_t row_off = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
    if (lane == 0) tma_prefetch_desc(&tmC);
    int it = 0;
    uint32_t nbox = 0;                            // boxes filled so far: box nbox & 1 is next
    double sq = 0.0;                              // this lane's share of |C|_F^2 (only with p.sumsq)
    for (int tile = pair; tile < num_tiles; tile += num_pairs, ++it) {
      const int buf = it & 1;
      const bool acc_ready =
          (mbar_wait_cluster_warp(accfull_bar(buf), (uint32_t)(it >> 1) & 1u, abort_flag, p.status));
      if (!acc_ready) break;
      tc_fence_after();
      const int64_t m0 = (int64_t)(tile / tiles_n) * PAIR_M + (int64_t)rank * BM, n0 = (int64_t)(tile % tiles_n) * BN;
      const int64_t row0 = m0 + q * 32;           // first row of this warp's boxes
#pragma unroll 1
      for (int cb = 0; cb < BN / EPI_COLS; ++cb, ++nbox) {
        const uint32_t box = box0 + (nbox & 1u) * EPI_BOX_BYTES;
        // the store that read this box two boxes ago must have finished reading it
        if (lane == 0) bulk_wait_group_read<1>();
        __syncwarp();
#pragma unroll
        for (int h = 0; h < EPI_COLS / 32; ++h) {
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(buf * BN + cb * EPI_COLS + h * 32), v);
          tmem_ld_wait();
#pragma unroll
          for (int g = 0; g < 4; ++g) {
            const int64_t col = n0 + cb * EPI_COLS + h * 32 + g * 8;
            float f[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[g * 8 + i]) * p.alpha;
            if (bias && col < p.N) {              // N is a multiple of 8: a group of 8 columns is all in or all out
              const uint4 bv = *reinterpret_cast<const uint4*>(bias + col);
              const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                f[2 * i] += __uint_as_float(bw[i] << 16);
                f[2 * i + 1] += __uint_as_float(bw[i] & 0xffff0000u);
              }
            }
            if (p.sumsq) {                        // rows and columns out of range hold exact zeros (zero-filled operands)
#pragma unroll
              for (int i = 0; i < 8; ++i) sq += (double)f[i] * (double)f[i];
            }
            // row `lane` of the box, 16-byte chunk 4h + g, at its swizzled position
            const uint32_t dst = box + row_off + ((((uint32_t)(4 * h + g)) ^ sw) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "r"(pack_bf16x2(f[0], f[1])),
                         "r"(pack_bf16x2(f[2], f[3])), "r"(pack_bf16x2(f[4], f[5])), "r"(pack_bf16x2(f[6], f[7]))
                         : "memory");
          }
        }
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          const int64_t col0 = n0 + cb * EPI_COLS;
          if (row0 < p.M && col0 < p.N) tma_store_2d(&tmC, box, (int)col0, (int)row0);
          bulk_commit_group();
        }
      }
      // every read of the accumulator buffer is done: hand it back to the MMA issuer in the leader CTA
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(accempty_leader0 + 8u * buf);
    }
    if (p.sumsq) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xffffffffu, sq, o);
      if (lane == 0) p.sumsq[(size_t)blockIdx.x * NEPI + (warp - 2)] = sq;
    }
    if (lane == 0) bulk_wait_group_all();         // the boxes must outlive their stores
    __syncwarp();
  }
  // ---------------------------------------------------------------- teardown
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the CTA's shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) __nanosleep(1000);
  }
  tc_fence_before();
  cluster_sync_all();      // nobody leaves while its partner may still signal or read across
  if (warp == 1) tmem_dealloc_pair(tmem_base, TMEM_COLS);
}

}  // namespace tc
}  // namespace rmm
