// One pass of the layer as ONE persistent launch (bf16 mode, sm_100a).
//
// Algorithm 1 computes, in each pass, a dense product and a sketch from the same token-sized
// operand: FORWARD Y = X W^T + 1 b^T and X_proj = S^T X; BACKWARD dX = dY W and G = S^T dY (with
// db = dY^T 1 as one more row of S^T).  pass_kernel does both in one launch: every CTA pair of the
// grid first works on its share of the sketch, then on its share of the dense tiles, and at the
// end all warps of the grid add up the partial sketch tiles.  Both kinds of work run on the same
// pipeline (one TMA ring, tcgen05.mma.cta_group::2 throughout), so
// the dense tiles fill the time that the few, long sketch tiles would leave idle.
//
// Dense tiles: as in tc_gemm.cuh (256 x 256 pair tiles, K step 64, two accumulator buffers,
// TMA-store epilogue).
//
// Sketch units.  C[j][d] = sum_n P[n][j] B[n][d] is computed transposed: the token-sized operand
// B (X or dY, [tokens][d] row-major) is the M side of the MMA (MN-major, by TMA), the generated
// S^T tile (sketch rows j x tokens, K-major) is the N side.  A pair tile is 128 sketch rows x
// (nat x 256) data columns: per 16 tokens the leader issues nat MMAs of M 256 (128 data columns
// from each CTA) x N 128 (64 generated sketch rows from each CTA) into nat accumulators of 128
// tensor-memory columns.  Each CTA generates only its 64 rows of every S^T stage, and the tensor
// cores of both CTAs read both halves: every generated entry feeds nat x 256 multiply-adds
// without any copy between the CTAs.  A tile's token range is cut into `nb` blocks; block b of
// tile t is unit b * tiles + t, units are dealt round-robin to the pairs (all pairs that run at the
// same time walk the same token range, so the token-sized operand is read from HBM once), and
// every unit leaves one fp32 partial tile.
//
// Reduction.  When the warps of a CTA have stored their part of a unit's partial tile, the CTA raises
// the unit's completion flag: it writes the launch's tag (unique per launch, so flags need no reset
// between launches; a value left by an earlier launch reads as "not yet").  After its last unit
// every warp of the grid takes rows of the result, waits (bounded) until the flags of the row's tile
// are all raised, adds the partial tiles in block order, applies the scale c = 1/sqrt(B_proj)
// (Eq. 5), rounds to bf16 and stores.  Sketch units never wait for another pair, so this wait cannot
// deadlock; it normally finds the flags raised.
//
// Warp roles per CTA: warp 0 TMA producer; warp 1 tensor-memory owner and, in the leader CTA, MMA
// issuer (dense tiles; accumulators 0 and 1 of the sketch units); warp 14 second MMA issuer of the
// sketch units (accumulators 2 and 3); warps 2-5 epilogue of the dense tiles; warps 6-13 generators
// of S^T, four groups of two, group g filling S^T stage g; warps 2-13 drain the sketch accumulators.
// The generators of the leader CTA arrive on the leader's "S^T stage full" barrier; those of the peer
// signal it with one asynchronous 4-byte store per stage, counted on the same barrier.  Shared memory:
// ring of 6 stages of 32 KB (dense: 128 x 64 of A and of B; sketch: 32 tokens x nat x 128 data
// columns), and 32 KB that hold the four 64-token S^T stages while the CTA works on sketch units and
// the epilogue's store boxes afterwards.  All waits are bounded.
#pragma once
#include "sketch_rng.cuh"
#include "tc_common.cuh"
#include "tc_gemm.cuh"

namespace rmm {
namespace tc {

constexpr int PS_MAX_PAIRS = 74;
constexpr int PS_GEN_WARPS = 8;
constexpr int PS_WARPS = 2 + NEPI + PS_GEN_WARPS + 1;      // 15: the last one is the second MMA issuer of the sketch units
constexpr int PS_MMA2_WARP = PS_WARPS - 1;
constexpr int PS_THREADS = 32 * PS_WARPS;
constexpr int PS_DRAIN_WARPS = NEPI + PS_GEN_WARPS;        // warps 2..13
constexpr int PS_S_STAGES = 4;
constexpr int PS_GEN_GROUPS = PS_S_STAGES;                 // one generator group per S^T stage: group g fills stage g
constexpr int PS_GROUP_WARPS = PS_GEN_WARPS / PS_GEN_GROUPS;
constexpr int PS_GROUP_THREADS = 32 * PS_GROUP_WARPS;
constexpr int PS_CHUNKS = 64 * 8;                          // 16-byte chunks (row, 8 tokens) of a CTA's part of a stage
constexpr int PS_CHUNKS_PER_THREAD = PS_CHUNKS / PS_GROUP_THREADS;
static_assert(PS_GEN_WARPS % PS_GEN_GROUPS == 0 && PS_CHUNKS % PS_GROUP_THREADS == 0, "generator groups");
constexpr int PS_S_BYTES = 64 * 64 * 2;                    // 64 sketch rows x 64 tokens, 8 KiB
constexpr int PS_SLAB = 32 * 64 * 2;                       // [32 tokens][64 columns], 4 KiB
constexpr int PS_ROWS = 128;                               // sketch rows of a pair tile
constexpr int PS_MAX_NAT = 4;                              // accumulators of 128 columns in 512 columns of tensor memory
static_assert(PS_S_STAGES * PS_S_BYTES == EPI_BYTES, "the S^T ring and the store boxes share one region");
constexpr int PS_SMEM_BYTES = STAGES * STAGE_BYTES + EPI_BYTES + 1024 + 512;

// Static schedule, built on the host (make_pass_schedule in rmm_api.cu).
struct PassSchedule {
  int num_pairs;
  // dense part: pair p computes tiles [gemm_begin[p], gemm_begin[p + 1])
  int gemm_tiles, tiles_n, num_kb;
  int gemm_begin[PS_MAX_PAIRS + 2];
  // sketch part: tile t = group * tiles_m + row tile; unit i = block * tiles + t; pair p takes units p, p + num_pairs, ...
  int tiles_m, groups, nat, ksteps, nb, blen;
  __host__ __device__ int sk_tiles() const { return tiles_m * groups; }
  __host__ __device__ int sk_units() const { return sk_tiles() * nb; }
  __host__ __device__ int cwp() const { return nat * 256; }     // data columns of a pair tile
};

struct PassParams {
  // dense part: C[M][N] = A[M][K] B^T (+ bias)
  int64_t M, N, K;
  const void* bias;
  // sketch part
  long long rows;        // rows of S^T that are computed: B_proj (+ 1 with the row of ones)
  long long b_proj;      // index of the row of ones
  long long cols, tokens;
  float scale;
  int ones_row, slab_map;
  uint32_t sors_mask;
  float* partial;                 // [units][128][cwp] fp32
  unsigned long long* tickets;    // [units][2] flags: the CTA has stored its part of the unit's partial tile
  unsigned long long tag;         // unique per launch
  __nv_bfloat16* sk_out;          // [B_proj][cols]
  __nv_bfloat16* ones_out;        // [cols] or nullptr
  int* status;
  int clear_status;
  PassSchedule sched;
};

// Token step visited at position i of a block: blocks of different row tiles start at different
// offsets (and wrap around), so that pairs walking the same token range do not ask L2 for the same
// lines at the same instant.  A fixed function of the schedule: results stay reproducible.
__host__ __device__ inline int pass_step(int ks0, int ks1, int tile_m, int i) {
  const int len = ks1 - ks0;
  int k = i + (tile_m * 2) % len;
  if (k >= len) k -= len;
  return ks0 + k;
}

// Eight consecutive tokens (tok8 a multiple of 8) of sketch row j as packed bf16: one 16-byte
// chunk of an S^T stage.
template <int DIST>
__device__ __forceinline__ uint4 pass_chunk(const PhiloxKey& pk, const PassParams& p, long long j, long long tok8) {
  constexpr uint32_t kOnes = 0x3f803f80u;   // two bf16 1.0
  uint4 v;
  if (DIST == 0) {
    v = gaussian_8_bf16(pk, (uint32_t)tok8, (uint32_t)j);
  } else if (DIST == 1) {
    uint32_t w[4];
    rademacher_128(pk, (uint32_t)(tok8 >> 7), (uint32_t)j, w);
    const int t = (int)(tok8 & 127);
    uint32_t word = w[0];                    // select without dynamic indexing
    word = (t >> 5) == 1 ? w[1] : word;
    word = (t >> 5) == 2 ? w[2] : word;
    word = (t >> 5) == 3 ? w[3] : word;
    v = rademacher_8_bf16(word, (t & 31) >> 3);
  } else if (DIST == 3) {
    v = rademacher_8_bf16(sors_sign_bits_8(pk, (uint32_t)tok8, (uint32_t)j, p.sors_mask), 0);
  } else if (DIST == 4) {
    v = dct_8_bf16(pk, (uint32_t)tok8, (uint32_t)j, p.sors_mask);
  } else {
    const long long d = j - tok8;
    uint32_t q0 = 0, q1 = 0, q2 = 0, q3 = 0;
    if (d >= 0 && d < 8) {
      const uint32_t one = (d & 1) ? 0x3f800000u : 0x00003f80u;
      const int wi = (int)(d >> 1);
      q0 = wi == 0 ? one : 0u; q1 = wi == 1 ? one : 0u; q2 = wi == 2 ? one : 0u; q3 = wi == 3 ? one : 0u;
    }
    v = make_uint4(q0, q1, q2, q3);
  }
  if (p.ones_row && j == p.b_proj) v = make_uint4(kOnes, kOnes, kOnes, kOnes);
  return v;
}

__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y), "r"(z)
      : "memory");
}

#ifndef PS_EXP_GUARD
#define PS_EXP_GUARD
#endif
// trace slots: 0 kernel cycles; producer: 1 wait empty, 2 loop; MMA: 3 wait S^T, 4 wait data, 5 wait accumulator,
// 6 sketch loop, 7 dense loop; generator warp 6: 8 arithmetic, 9 wait free stage, 10 loop; warp 2: 11 wait sketch
// accumulator, 12 drain, 13 epilogue loop, 14 reduction (wait), 15 reduction (work)

template <int BMODE, int DIST>
__global__ void __launch_bounds__(PS_THREADS, 1)
pass_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
            const __grid_constant__ CUtensorMap tmC, const __grid_constant__ CUtensorMap tmD, PassParams p, PhiloxKey pk) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const uint32_t sbase = smem_u32(smem);
  uint8_t* aux = smem + STAGES * STAGE_BYTES;              // S^T ring, later the store boxes
  const uint32_t aux_base = sbase + STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(aux + EPI_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  auto full_bar = [&](int s) { return bar0 + 8u * s; };
  auto empty_bar = [&](int s) { return bar0 + 8u * (STAGES + s); };
  auto accfull_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + b); };
  auto accempty_bar = [&](int b) { return bar0 + 8u * (2 * STAGES + 2 + b); };
  auto fulls_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 4 + s); };
  auto emptys_bar = [&](int s) { return bar0 + 8u * (2 * STAGES + 4 + PS_S_STAGES + s); };
  const uint32_t skfull_bar = bar0 + 8u * (2 * STAGES + 4 + 2 * PS_S_STAGES);
  const uint32_t skempty_bar = skfull_bar + 8u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * STAGES + 4 + 2 * PS_S_STAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* drain_count = tmem_slot + 2;          // draining warps of this CTA that have stored their part of a unit
  uint32_t* gen_count = tmem_slot + 3;            // [PS_S_STAGES] generator warps of a group that have stored their part
  uint32_t* peer_flag = tmem_slot + 3 + PS_S_STAGES;   // [PS_S_STAGES] words the peer's "stage ready" signals land in

  MBAR_PEEK_DECLARE();
  PS_TRACE_T0(trace_kernel0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = leader of the pair
  const bool leader = rank == 0;
  if (p.clear_status && blockIdx.x == 0 && threadIdx.x == 0) *p.status = 0;
  const PassSchedule& sc = p.sched;
  const int pair = (int)(blockIdx.x >> 1), num_pairs = sc.num_pairs;
  const int sk_tiles = sc.sk_tiles(), sk_units = sc.sk_units();
  const int nat = sc.nat, cwp = sc.cwp();
  const int g_begin = sc.gemm_begin[pair], g_end = sc.gemm_begin[pair + 1];
  const int tiles_n = sc.tiles_n, num_kb = sc.num_kb;
  // sketch units of this pair: unit, unit + num_pairs, ...
  const int my_units = pair < sk_units ? (sk_units - pair + num_pairs - 1) / num_pairs : 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(empty_bar(s), 2);                 // two commits: one per MMA-issuing warp (dense tiles: both from warp 1)
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(accfull_bar(b), 1);
      mbar_init(accempty_bar(b), 2 * NEPI);     // one arrival per epilogue warp of either CTA
    }
    for (int s = 0; s < PS_S_STAGES; ++s) {
      mbar_init(fulls_bar(s), PS_GROUP_WARPS);   // the leader's warps of the stage's generator group + 4 bytes from the peer
      mbar_init(emptys_bar(s), 2);
      gen_count[s] = 0;
    }
    mbar_init(skfull_bar, 2);
    mbar_init(skempty_bar, 2 * PS_DRAIN_WARPS);    // one arrival per draining warp of either CTA
    *abort_flag = 0;
    *drain_count = 0;
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
    // ------------------------------------------------------------ TMA producer: this CTA's parts
    if (lane == 0) {
      if (my_units > 0) tma_prefetch_desc(&tmD);
      if (g_end > g_begin) { tma_prefetch_desc(&tmA); tma_prefetch_desc(&tmB); }
      const uint32_t leader_delta = mapa_shared(bar0, 0) - bar0;   // 0 in the leader itself
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      PS_TRACE_DECL(tr_wait);
      PS_TRACE_T0(tr_loop0);
      const uint32_t sk_stage_bytes = (uint32_t)nat * 2u * PS_SLAB;    // per CTA
      for (int u = pair; u < sk_units && ok; u += num_pairs) {
        const int t = u % sk_tiles, b = u / sk_tiles;
        const int g = t / sc.tiles_m, tm = t % sc.tiles_m;
        const int ks0 = b * sc.blen, ks1 = ks0 + sc.blen < sc.ksteps ? ks0 + sc.blen : sc.ksteps;
        const int col0 = g * cwp + (int)rank * nat * 128;             // this CTA's first data column
        for (int i = 0; i < ks1 - ks0 && ok; ++i) {
          const int ks = pass_step(ks0, ks1, tm, i);
#pragma unroll
          for (int half = 0; half < 2; ++half) {
            PS_TRACE_T0(tw);
            if (!mbar_wait_cluster(empty_bar(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
            PS_TRACE_ADD(tr_wait, tw);
            const uint32_t dst = sbase + s * STAGE_BYTES;
            if (leader) mbar_arrive_expect_tx(full_bar(s), 2 * sk_stage_bytes);
            const uint32_t full_leader = full_bar(s) + leader_delta;
            const int tok0 = ks * 64 + half * 32;
            if (p.slab_map) {
              tma_load_3d_pair(dst, &tmD, full_leader, 0, tok0, col0 >> 6);
            } else {
              for (int sl = 0; sl < 2 * nat; ++sl)
                tma_load_2d_pair(dst + sl * PS_SLAB, &tmD, full_leader, col0 + 64 * sl, tok0);
            }
            if (++s == STAGES) { s = 0; ph ^= 1u; }
          }
        }
      }
      for (int tile = g_begin; tile < g_end && ok; ++tile) {
        const int m0 = (tile / tiles_n) * PAIR_M + (int)rank * BM;
        const int n0 = (tile % tiles_n) * BN + (int)rank * BN_HALF;
        for (int kb = 0; kb < num_kb; ++kb) {
          PS_TRACE_T0(tw);
          if (!mbar_wait_cluster(empty_bar(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
          PS_TRACE_ADD(tr_wait, tw);
          const uint32_t a_smem = sbase + s * STAGE_BYTES, b_smem = a_smem + A_BYTES;
          if (leader) mbar_arrive_expect_tx(full_bar(s), 2 * STAGE_BYTES);   // bytes of both CTAs
          const uint32_t full_leader = full_bar(s) + leader_delta;
          const int k0 = kb * BK;
          tma_load_2d_pair(a_smem, &tmA, full_leader, k0, m0);
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
      PS_TRACE_PUT(1, tr_wait);
      PS_TRACE_PUT(2, clock64() - tr_loop0);
    }
    __syncwarp();
  } else if (warp == 1 || warp == PS_MMA2_WARP) {
    // ------------------------------------------------------------ MMA issuers (leader CTA only)
    // Sketch units: two issuing warps, warp 1 for the accumulators 0 and 1, the last warp for 2 and 3 (an
    // issuing thread has 64 cycles per MMA of M 256 x N 128 x K 16, and waits, barrier tests and commits come on
    // top).  Both wait on the same full barriers; a stage is free once both have committed.  Dense tiles: warp 1.
    if (leader) {
      bool ok = true;
      int s = 0;
      uint32_t ph = 0;
      MBAR_PEEK_CLUSTER(0, full_bar(0), 0u);    // every stage's barrier is tested one stage ahead
      PS_TRACE_DECL(tr_ws);
      PS_TRACE_DECL(tr_m_fe);
      PS_TRACE_DECL(tr_m_is);
      PS_TRACE_DECL(tr_m_co);
      PS_TRACE_DECL(tr_wd);
      PS_TRACE_DECL(tr_wa);
      PS_TRACE_T0(tr_sk0);
      // ---------------- sketch units
      {
        // The loop is kept to a handful of instructions per MMA: descriptors differ only in the low word (the
        // 14-bit start-address field never carries), the accumulator loop is unrolled with a uniform guard, every
        // barrier is tested one stage ahead, and one multicast commit signals both CTAs.
        constexpr uint32_t idesc = instr_desc_bf16(PAIR_M, PS_ROWS, true, false);
        const uint64_t adesc0 = smem_desc_sw128(sbase, PS_SLAB, 1024);         // data, MN-major: slabs of 64 columns
        const uint64_t bdesc0 = smem_desc_sw128(aux_base, 16, 1024);           // S^T, K-major
        const uint32_t a_lo0 = (uint32_t)adesc0, a_hi = (uint32_t)(adesc0 >> 32);
        const uint32_t b_lo0 = (uint32_t)bdesc0, b_hi = (uint32_t)(bdesc0 >> 32);
        auto desc64 = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | (uint64_t)lo; };
        const int a_first = warp == 1 ? 0 : 2;            // this warp's accumulators: a_first, a_first + 1
        int sa = 0;
        uint32_t pha = 0;
        int seg = 0;
        if (my_units > 0) MBAR_PEEK_CLUSTER(1, fulls_bar(0), 0u);
        for (int u = pair; u < sk_units && ok; u += num_pairs, ++seg) {
          const int b = u / sk_tiles;
          const int ks0 = b * sc.blen, ks1 = ks0 + sc.blen < sc.ksteps ? ks0 + sc.blen : sc.ksteps;
          if (seg > 0) {   // the previous unit's accumulators must have been drained
            PS_TRACE_T0(tw);
            ok = mbar_wait_cluster_warp(skempty_bar, (uint32_t)(seg - 1) & 1u, abort_flag, p.status);
            PS_TRACE_ADD(tr_wa, tw);
            if (!ok) break;
            tc_fence_after();
          }
          uint32_t acc = 0;
          for (int i = 0; i < ks1 - ks0 && ok; ++i) {
            uint32_t ready;
            MBAR_PEEK_RESULT(1, ready);
            if (!__all_sync(0xffffffffu, ready != 0)) {
              PS_TRACE_T0(tw);
              ok = mbar_wait_cluster_warp(fulls_bar(sa), pha, abort_flag, p.status);
              PS_TRACE_ADD(tr_ws, tw);
              if (!ok) break;
            }
            const uint32_t b_lo = b_lo0 + (uint32_t)(sa * (PS_S_BYTES >> 4));
            const int sa_next = (sa + 1 == PS_S_STAGES) ? 0 : sa + 1;
            const uint32_t pha_next = (sa_next == 0) ? (pha ^ 1u) : pha;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
              MBAR_PEEK_RESULT(0, ready);
              if (!__all_sync(0xffffffffu, ready != 0)) {
                PS_TRACE_T0(tw);
                ok = mbar_wait_cluster_warp(full_bar(s), ph, abort_flag, p.status);
                PS_TRACE_ADD(tr_wd, tw);
                if (!ok) break;
              }
              PS_TRACE_T0(tfa);
              tc_fence_after();
              PS_TRACE_ADD(tr_m_fe, tfa);
              const uint32_t a_lo = a_lo0 + (uint32_t)(s * (STAGE_BYTES >> 4));
              const int s_next = (s + 1 == STAGES) ? 0 : s + 1;
              const uint32_t ph_next = (s_next == 0) ? (ph ^ 1u) : ph;
              PS_TRACE_T0(tis);
              const bool issuer = elect_one();
              if (issuer) {
#pragma unroll
                for (int kk = 0; kk < 2; ++kk) {
#pragma unroll
                  for (int da = 0; da < 2; ++da) {
                    const int a = a_first + da;
                    if (a < nat PS_EXP_GUARD)
                      umma_bf16_pair(tmem_base + a * PS_ROWS, desc64(a_lo + (uint32_t)((a * 2 * PS_SLAB + kk * 2048) >> 4), a_hi),
                                     desc64(b_lo + (uint32_t)((half * 2 + kk) * 2), b_hi), idesc, kk == 0 ? acc : 1u);
                  }
                }
              }
              PS_TRACE_ADD(tr_m_is, tis);
              PS_TRACE_T0(tco);
              MBAR_PEEK_CLUSTER(0, full_bar(s_next), ph_next);   // travels while the commits are issued
              if (half == 1) MBAR_PEEK_CLUSTER(1, fulls_bar(sa_next), pha_next);
              if (issuer) {
                umma_commit_pair_multicast(empty_bar(s), (uint16_t)3);
                if (half == 1) umma_commit_pair_multicast(emptys_bar(sa), (uint16_t)3);
              }
              __syncwarp();
              PS_TRACE_ADD(tr_m_co, tco);
              acc = 1;
              s = s_next;
              ph = ph_next;
            }
            sa = sa_next;
            pha = pha_next;
          }
          if (ok) {
            if (elect_one()) umma_commit_pair_multicast(skfull_bar, (uint16_t)3);
            __syncwarp();
          }
        }
        if (ok && seg > 0 && g_end > g_begin && warp == 1) {   // the dense tiles reuse the tensor memory of the last unit
          PS_TRACE_T0(tw);
          ok = mbar_wait_cluster_warp(skempty_bar, (uint32_t)(seg - 1) & 1u, abort_flag, p.status);
          PS_TRACE_ADD(tr_wa, tw);
          tc_fence_after();
        }
      }
      if (warp == 1) {
      PS_TRACE_PUT(6, clock64() - tr_sk0);
      PS_TRACE_T0(tr_ge0);
      // ---------------- dense tiles
      {
        constexpr uint32_t idesc = instr_desc_bf16(PAIR_M, BN, false, BMODE == B_MN);
        const uint64_t adesc0 = smem_desc_sw128(sbase, 16, 1024);
        const uint64_t bdesc0 = (BMODE == B_MN) ? smem_desc_sw128(sbase + A_BYTES, SLAB_BYTES, 1024)
                                                : smem_desc_sw128(sbase + A_BYTES, 16, 1024);
        constexpr uint32_t a_kstep = (UMMA_K * 2) >> 4;
        constexpr uint32_t b_kstep = ((BMODE == B_MN) ? UMMA_K * 128 : UMMA_K * 2) >> 4;
        int it = 0;                               // tiles done by this pair
        for (int tile = g_begin; tile < g_end && ok; ++tile, ++it) {
          const int buf = it & 1;
          // the epilogues of both CTAs must have drained this accumulator buffer (two tiles ago)
          PS_TRACE_T0(twa);
          ok = (mbar_wait_cluster_warp(accempty_bar(buf), ((uint32_t)(it >> 1) & 1u) ^ 1u, abort_flag, p.status));
          PS_TRACE_ADD(tr_wa, twa);
          if (!ok) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + buf * BN;
          for (int kb = 0; kb < num_kb; ++kb) {
            uint32_t ready;
            MBAR_PEEK_RESULT(0, ready);
            if (!__all_sync(0xffffffffu, ready != 0)) {
              PS_TRACE_T0(tw);
              ok = (mbar_wait_cluster_warp(full_bar(s), ph, abort_flag, p.status));
              PS_TRACE_ADD(tr_wd, tw);
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
              umma_commit_pair_multicast(empty_bar(s), (uint16_t)3);      // the barrier counts two arrivals
              umma_commit_pair_multicast(empty_bar(s), (uint16_t)3);
            }
            __syncwarp();
            s = s_next;
            ph = ph_next;
          }
          if (ok) {
            if (elect_one()) umma_commit_pair_multicast(accfull_bar(buf), (uint16_t)3);
            __syncwarp();
          }
        }
      }
      if (lane == 0) {
        PS_TRACE_PUT(3, tr_ws); PS_TRACE_PUT(4, tr_wd); PS_TRACE_PUT(5, tr_wa);
        PS_TRACE_PUT(19, tr_m_fe); PS_TRACE_PUT(20, tr_m_is); PS_TRACE_PUT(21, tr_m_co);
        PS_TRACE_PUT(7, clock64() - tr_ge0);
      }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ generators, drain, epilogue
    const int q = warp & 3;                       // tensor-memory lane quarter this warp may read
    const int dw = warp - 2;                      // index among the draining warps
    const int dgroup = dw >> 2;                   // index among the three warps that share the quarter
    const bool is_gen = warp >= 2 + NEPI;
    const int grp = (warp - 2 - NEPI) / PS_GROUP_WARPS;                      // generators: this warp's group
    const int gtid = ((warp - 2 - NEPI) % PS_GROUP_WARPS) * 32 + lane;       // and the thread index within it
    const uint32_t fulls_leader0 = mapa_shared(fulls_bar(0), 0);
    const uint32_t peer_flag_leader0 = mapa_shared(smem_u32(peer_flag), 0);
    const uint32_t skempty_leader = mapa_shared(skempty_bar, 0);
    bool ok = true;
    PS_TRACE_DECL(tr_gen);
    PS_TRACE_DECL(tr_g_st);
    PS_TRACE_DECL(tr_g_fe);
    PS_TRACE_DECL(tr_g_ar);
    PS_TRACE_DECL(tr_gw);
    PS_TRACE_DECL(tr_gl);
    PS_TRACE_DECL(tr_dw);
    PS_TRACE_DECL(tr_dr);
    // ---------------- sketch units
    {
      int step0 = 0;                              // steps of earlier units of this pair
      int seg = 0;
      for (int u = pair; u < sk_units && ok; u += num_pairs, ++seg) {
        const int t = u % sk_tiles, b = u / sk_tiles;
        const int g = t / sc.tiles_m, tm = t % sc.tiles_m;
        const int ks0 = b * sc.blen, ks1 = ks0 + sc.blen < sc.ksteps ? ks0 + sc.blen : sc.ksteps;
        const int len = ks1 - ks0;
        if (is_gen) {
          // This CTA's 64 rows of every stage: 512 chunks (row, 8 tokens).  Group g produces the steps g,
          // g + groups, ... of this pair's sequence, all of which go into ring stage g; the groups run out of
          // phase, so the stores, the proxy fence and the barrier round trip of one are covered by the
          // arithmetic of the others.
          const long long j0 = (long long)tm * PS_ROWS + (long long)rank * 64;
          PS_TRACE_T0(tgl);
          for (int i = (grp + PS_GEN_GROUPS - step0 % PS_GEN_GROUPS) % PS_GEN_GROUPS; i < len; i += PS_GEN_GROUPS) {
            PS_TRACE_T0(tg0);
            const int ks = pass_step(ks0, ks1, tm, i);
            const int step = step0 + i;
            const int sa = grp;                                         // step % stages
            const uint32_t pha = (uint32_t)(step / PS_S_STAGES) & 1u;
            // Generate first, into registers: the entries do not depend on the ring, so the wait for
            // the free stage only covers the stores.
            uint4 v[PS_CHUNKS_PER_THREAD];
            uint32_t off[PS_CHUNKS_PER_THREAD];
#pragma unroll
            for (int it = 0; it < PS_CHUNKS_PER_THREAD; ++it) {
              const int task = it * PS_GROUP_THREADS + gtid;
              const int r = task >> 3, c = task & 7;
              v[it] = pass_chunk<DIST>(pk, p, j0 + r, (long long)ks * 64 + 8 * c);
              off[it] = (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
            }
            PS_TRACE_ADD(tr_gen, tg0);
            PS_TRACE_T0(tgw);
            if (!mbar_wait_cluster_warp(emptys_bar(sa), pha ^ 1u, abort_flag, p.status)) { ok = false; break; }
            PS_TRACE_ADD(tr_gw, tgw);
            uint8_t* const stage_ptr = aux + sa * PS_S_BYTES;
            PS_TRACE_T0(tst);
#pragma unroll
            for (int it = 0; it < PS_CHUNKS_PER_THREAD; ++it) *reinterpret_cast<uint4*>(stage_ptr + off[it]) = v[it];
            PS_TRACE_ADD(tr_g_st, tst);
            PS_TRACE_T0(tfe);
            fence_proxy_async_smem();
            PS_TRACE_ADD(tr_g_fe, tfe);
            PS_TRACE_T0(tar);
            __syncwarp();
            if (lane == 0) {
              if (leader) {
                // the stage is complete once this group's warps have arrived here and the peer's signal has landed
                if (gtid == 0) mbar_arrive_expect_tx(fulls_bar(sa), 4);
                else mbar_arrive(fulls_bar(sa));
              } else {
                // the warp of the group that stores last tells the leader, with an asynchronous store counted on the
                // leader's barrier (the counter only grows: a stage is reused after its barrier has completed)
                __threadfence_block();
                const uint32_t n = atomicAdd(&gen_count[sa], 1u);
                if ((n % PS_GROUP_WARPS) == PS_GROUP_WARPS - 1) {
                  __threadfence_block();
                  st_async_u32(peer_flag_leader0 + 4u * sa, 1u, fulls_leader0 + 8u * sa);
                }
              }
            }
            PS_TRACE_ADD(tr_g_ar, tar);
          }
          PS_TRACE_ADD(tr_gl, tgl);
          if (!ok) break;
        }
        step0 += len;
        // drain: this warp's 32-column chunks of the nat accumulators -> the unit's partial tile
        PS_TRACE_T0(tdw);
        ok = mbar_wait_cluster_warp(skfull_bar, (uint32_t)seg & 1u, abort_flag, p.status);
        PS_TRACE_ADD(tr_dw, tdw);
        if (!ok) break;
        tc_fence_after();
        PS_TRACE_T0(tdr);
        {
          float* tile_base = p.partial + (long long)u * PS_ROWS * cwp;
          const int pc0 = (int)rank * nat * 128 + q * 32 + lane;      // pair-local data column of this lane, accumulator 0
          const long long row_first = (long long)tm * PS_ROWS;
#pragma unroll 1
          for (int c = dgroup; c < nat * 4; c += PS_DRAIN_WARPS / 4) {
            const int a = c >> 2, cc = c & 3;
            if (row_first + cc * 32 >= p.rows) continue;                // rows beyond the result are never read
            if ((long long)g * cwp + (long long)rank * nat * 128 + a * 128 + q * 32 >= p.cols) continue;
            uint32_t v[32];
            tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(a * PS_ROWS + cc * 32), v);
            tmem_ld_wait();
            float* dst = tile_base + (long long)(cc * 32) * cwp + pc0 + a * 128;
#pragma unroll
            for (int r = 0; r < 32; ++r) __stcg(dst + (long long)r * cwp, __uint_as_float(v[r]));
          }
        }
        __threadfence();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) {
          // the warp of this CTA that stores last arrives on the tile's ticket for all of them (the counter only
          // grows: a unit's arrivals are complete before the next unit's begin, the MMAs wait for skempty)
          const uint32_t n = atomicAdd(drain_count, 1u);
          if ((n % PS_DRAIN_WARPS) == PS_DRAIN_WARPS - 1) {
            __threadfence();
            flag_raise(p.tickets + (long long)u * 2 + rank, p.tag);
          }
          mbar_arrive_cluster(skempty_leader);
        }
        PS_TRACE_ADD(tr_dr, tdr);
      }
    }
    if (lane == 0 && warp == 2 + NEPI) {
      PS_TRACE_PUT(8, tr_gen); PS_TRACE_PUT(9, tr_gw); PS_TRACE_PUT(10, tr_gl);
      PS_TRACE_PUT(16, tr_g_st); PS_TRACE_PUT(17, tr_g_fe); PS_TRACE_PUT(18, tr_g_ar);
    }
    if (lane == 0 && warp == 2) { PS_TRACE_PUT(11, tr_dw); PS_TRACE_PUT(12, tr_dr); }
    PS_TRACE_T0(tr_ep0);
    // ---------------- epilogue of the dense tiles (overlaps the next tile's MMAs)
    if (!is_gen && ok) {
      const __nv_bfloat16* bias = reinterpret_cast<const __nv_bfloat16*>(p.bias);
      const uint32_t accempty_leader0 = mapa_shared(accempty_bar(0), 0);
      const uint32_t box0 = aux_base + (uint32_t)(warp - 2) * 2 * EPI_BOX_BYTES;   // this warp's two boxes
      const uint32_t row_off = (uint32_t)lane * 128u, sw = (uint32_t)(lane & 7);
      if (lane == 0 && g_end > g_begin) tma_prefetch_desc(&tmC);
      int it = 0;
      uint32_t nbox = 0;                            // boxes filled so far: box nbox & 1 is next
      for (int tile = g_begin; tile < g_end; ++tile, ++it) {
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
            for (int gq = 0; gq < 4; ++gq) {
              const int64_t col = n0 + cb * EPI_COLS + h * 32 + gq * 8;
              float f[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) f[i] = __uint_as_float(v[gq * 8 + i]);
              if (bias && col < p.N) {              // N is a multiple of 8: a group of 8 columns is all in or all out
                const uint4 bv = *reinterpret_cast<const uint4*>(bias + col);
                const uint32_t bw[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                  f[2 * i] += __uint_as_float(bw[i] << 16);
                  f[2 * i + 1] += __uint_as_float(bw[i] & 0xffff0000u);
                }
              }
              // row `lane` of the box, 16-byte chunk 4h + gq, at its swizzled position
              const uint32_t dst = box + row_off + ((((uint32_t)(4 * h + gq)) ^ sw) << 4);
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
      if (lane == 0) bulk_wait_group_all();         // the boxes must outlive their stores
      __syncwarp();
      if (lane == 0 && warp == 2) PS_TRACE_PUT(13, clock64() - tr_ep0);
    }
  }
  // ---------------------------------------------------------------- reduction of the partial sketch tiles
  // Every warp of the grid takes rows (tile, row) of the result, round-robin.
  if (sk_units > 0) {
    __syncwarp();
    const int total_warps = (int)gridDim.x * PS_WARPS;
    int checked_tile = -1;
    bool ok = true;
    PS_TRACE_DECL(tr_rw);
    PS_TRACE_T0(tr_r0);
    for (int unit = (int)blockIdx.x * PS_WARPS + warp; unit < sk_tiles * PS_ROWS && ok; unit += total_warps) {
      const int t = unit >> 7, r = unit & 127;
      const int g = t / sc.tiles_m, tm = t % sc.tiles_m;
      const long long j = (long long)tm * PS_ROWS + r;
      if (j >= p.rows) continue;
      if (t != checked_tile) {
        // the flags of both CTAs of every unit (token block) of this tile: units t, t + tiles, ...
        PS_TRACE_T0(tw);
        ok = flags_wait_warp(p.tickets, (long long)t * 2, (long long)sk_tiles * 2, sc.nb, p.tag, abort_flag, p.status) &&
             flags_wait_warp(p.tickets, (long long)t * 2 + 1, (long long)sk_tiles * 2, sc.nb, p.tag, abort_flag, p.status);
        PS_TRACE_ADD(tr_rw, tw);
        if (!ok) break;
        checked_tile = t;
      }
      const bool is_ones = p.ones_row && j == p.b_proj;
      const float sc_f = is_ones ? 1.0f : p.scale;
      __nv_bfloat16* dst_row = is_ones ? p.ones_out : p.sk_out + j * p.cols;
      if (dst_row == nullptr) continue;
      const long long col_base = (long long)g * cwp;
      const float* src0 = p.partial + ((long long)t * PS_ROWS + r) * cwp;
      const long long unit_stride = (long long)sk_tiles * PS_ROWS * cwp;   // between the blocks of a tile
      for (int c = lane * 8; c < cwp; c += 256) {
        if (col_base + c >= p.cols) break;              // cols is a multiple of 8
        float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0;
        const float* src = src0 + c;
#pragma unroll 4
        for (int b = 0; b < sc.nb; ++b) {
          const float4 x0 = __ldcg(reinterpret_cast<const float4*>(src + (long long)b * unit_stride));
          const float4 x1 = __ldcg(reinterpret_cast<const float4*>(src + (long long)b * unit_stride + 4));
          a0.x += x0.x; a0.y += x0.y; a0.z += x0.z; a0.w += x0.w;
          a1.x += x1.x; a1.y += x1.y; a1.z += x1.z; a1.w += x1.w;
        }
        __nv_bfloat162 h0 = __floats2bfloat162_rn(a0.x * sc_f, a0.y * sc_f), h1 = __floats2bfloat162_rn(a0.z * sc_f, a0.w * sc_f);
        __nv_bfloat162 h2 = __floats2bfloat162_rn(a1.x * sc_f, a1.y * sc_f), h3 = __floats2bfloat162_rn(a1.z * sc_f, a1.w * sc_f);
        *reinterpret_cast<uint4*>(dst_row + col_base + c) =
            make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                       *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
      }
    }
    if (warp == 2 && lane == 0) { PS_TRACE_PUT(14, tr_rw); PS_TRACE_PUT(15, clock64() - tr_r0); }
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
  if (threadIdx.x == 0) PS_TRACE_PUT(0, clock64() - trace_kernel0);
}

}  // namespace tc
}  // namespace rmm
