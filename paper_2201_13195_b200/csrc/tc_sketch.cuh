// Sketch contraction on the tensor cores (bf16 mode, sm_100a):
//     C[j][d] = sum over tokens n of P[n][j] * B[n][d]
// i.e. X_proj = S^T X in the forward pass and G = S^T dY in the backward pass of
// Algorithm 1, with the 128 x 64 tiles of S^T generated in shared memory from the Philox
// seed by the CTA's own warps (S is never read from or written to memory) and B (X or
// dY, row-major [tokens][d]) streamed by TMA as an MN-major operand.
//
// Work decomposition.  An output tile is 128 sketch rows x 512 columns: the whole tensor
// memory of an SM (512 fp32 columns) accumulates it, so that every generated entry of S
// is used 512 times by the CTA that holds it.
//
// Sharing S across a cluster.  Generating the normals is plain ALU work (about 24
// instructions each) and takes about as many issue slots as the MMAs that consume them take
// tensor cycles.  CTAs that compute the same sketch rows for neighbouring 512-column blocks
// therefore form a thread-block cluster of C (1 or 2; with 4 too few such clusters are
// co-resident): each CTA generates 128/C rows of every S^T stage into its own operand ring and
// sends that block to the other CTAs with one bulk shared-to-shared copy each, counted on the
// destination's full barrier, so each generated entry feeds C x 512 columns.  Every CTA runs
// its own TMA ring for its B columns, its own MMAs and its own accumulator.
//
// Stream-K.  There are far fewer tiles than SMs and each has a long contraction (all tokens),
// so (tile group, 64-token step) units are distributed over the clusters by a static
// schedule (below).  A CTA accumulates each tile segment of its cluster's share in tensor
// memory and writes it as an fp32 partial tile; sketch_reduce_kernel adds the partial tiles
// of every output tile in a fixed order, applies the scale c = 1/sqrt(B_proj) (Eq. 5) and
// rounds to bf16.
//
// db for free: when ones_row is set, row index B_proj of S^T is a row of ones, so row
// B_proj of the result is sum_n dY[n][:] (Eq. 3); the reduce kernel stores it, unscaled.
//
// Warp roles: warp 0 TMA producer (B); warps 1-2 MMA issuers, one per 256-column half of the
// accumulator (warp 1 owns the tensor memory); warps 3..14 generate S tiles, in three groups of
// four that each own one ring stage, and drain the accumulator.  A ring: 3 stages of 64 tokens x
// 128 rows; B ring: 5 stages of 64 tokens x 256 columns, each consumed by one MMA warp (one barrier
// round per four MMAs).
// What limits the kernel (cycle counters of the RMM_PASS_TRACE build, 256-step segments): a 64-token
// step takes about 1400 cycles with the Gaussian sketch against 1024 cycles of tensor work.  The
// generators need about 930 cycles of arithmetic per step (three groups in turn) plus the hand-over
// of the stage (stores, proxy fence, count, bulk copy to the peer: 360 cycles), and the MMA warps
// wait about 450 cycles per step for S^T: the generation of the normals is the bound.  With the
// Rademacher sketch the generators are idle, but a step takes 1800 cycles: a stage is refilled the
// moment it is freed, while the tensor pipe reads operands at full rate (96 bytes per cycle of MMA
// operand reads plus 64 of TMA writes per SM), and the generators' ordinary stores into shared memory
// then complete slowly: the same hand-over takes 1700 cycles.  The tensor pipe itself runs every
// operand layout used here at its nominal 8192 FLOP per cycle and SM when fed from resident tiles.
// Barriers of a CTA: fullA[s] (the group's warps + the bytes copied in by the other CTAs: the
// stage is complete in this CTA's ring), emptyA[s] (2 C commits: every MMA warp of every CTA of the
// cluster has consumed the stage, so it may be overwritten everywhere), fullB / emptyB (TMA
// ring; one commit, by the warp the stage belongs to), accfull / accempty.  All waits are bounded.
#pragma once
#include "sketch_rng.cuh"
#include "tc_common.cuh"

namespace rmm {
namespace tc {

constexpr int SK_BM = 128, SK_BN = 512, SK_AK = 64;
constexpr int SK_BK = 64;                            // tokens of a B stage
constexpr int SK_BNH = 256;                          // columns of a B stage: one half of the tile, one MMA warp's
constexpr int SK_A_STAGES = 3, SK_B_STAGES = 5;
constexpr int SK_A_BYTES = SK_BM * SK_AK * 2;        // 16 KiB
constexpr int SK_B_BYTES = SK_BNH * SK_BK * 2;       // 32 KiB
constexpr int SK_B_SLAB = 64 * SK_BK * 2;            // [64 tokens][64 columns] = 8 KiB
constexpr int SK_STAGGER = 2;                        // steps by which neighbouring tile rows are offset
constexpr int SK_GEN_GROUPS = SK_A_STAGES;  // one generator warp group per ring stage: group g fills stage g.
// (A stage must have one producer group: barrier waits only see the parity of a phase, and two
// groups taking turns on one stage could get two phases apart.)
constexpr int SK_GEN_WARPS = 4 * SK_GEN_GROUPS;
constexpr int SK_GEN_THREADS = 32 * SK_GEN_WARPS;
constexpr int SK_MMA_WARPS = 2;            // each issues the MMAs of one 256-column half of the tile
constexpr int SK_THREADS = 32 * (1 + SK_MMA_WARPS) + SK_GEN_THREADS;
constexpr int SK_SMEM_BYTES = SK_A_STAGES * SK_A_BYTES + SK_B_STAGES * SK_B_BYTES + 1024 + 256;
constexpr int SK_TILE_ELEMS = SK_BM * SK_BN;         // fp32 elements of one partial tile
constexpr int SK_MAX_CTAS = 148;                     // CTAs (all clusters together) used for workspace sizing

// Static schedule shared by the sketch kernel, the reduce kernel and the host.
//
// A "tile" of the schedule is a tile group: 128 rows x (C x 512) columns, worked on by one
// cluster of C CTAs; "CTA" below means one such cluster.
// Units are (tile, 64-token step) pairs; every CTA gets `upc` consecutive units of a
// line that is ordered so that CTAs running at the same time read the same token rows
// of B (they then come out of L2 instead of being fetched from HBM once per tile row):
//   1. rounds: while at least num_ctas tiles are left, CTA i takes one whole tile;
//   2. the remaining `tiles_rem` tiles are cut along tokens into blocks of `upc` steps;
//      block b of tile t goes to CTA b * tiles_rem + t, so all CTAs of a block walk the
//      same token range in step;
//   3. the last, narrower block (width `w_last`) is laid out tile after tile and cut
//      into ranges of `upl` units, which may span several tiles; `upl` < `upc`, because each
//      extra segment costs a drain of the accumulator -- or, when that is cheaper, the tiles
//      are cut into equal blocks only (make_sketch_schedule compares the candidates).
// Every (CTA, tile) intersection is one segment = one fp32 partial tile (slot).
struct SketchSchedule {
  int cluster;             // C: CTAs per cluster = 512-column blocks per tile group
  int tiles_m, tiles_n, ksteps;   // tiles_n counts tile groups
  int num_ctas;            // number of clusters
  int rounds;              // whole-tile rounds
  int tiles_rem;           // tiles handled by the blocked part
  int upc;                 // units per CTA in the blocked part
  int full_blocks;         // blocks of width upc
  int w_last;              // width of the last block (0 if none)
  int upl;                 // units per CTA in the last block's line
  long long lcm_last;      // lcm(upl, w_last)
  long long est_steps;     // host only: estimated time of the busiest cluster, in 64-token steps (drains included)

  __host__ __device__ int tiles() const { return tiles_m * tiles_n; }
  __host__ __device__ long long num_slots() const { return (long long)tiles() + num_ctas; }
  // slot of the whole-tile segment of a round
  __host__ __device__ long long slot_round(int tile) const { return tile; }
  // slot of full block b of remainder tile t (CTA b * tiles_rem + t)
  __host__ __device__ long long slot_block(int b, int t) const {
    return (long long)rounds * num_ctas + (long long)b * tiles_rem + t;
  }
  // slot of a segment of the last block: CTA index ci and tile t, both relative to the last
  // block, seg_start = first unit of the segment in the last block's tile-major line.
  // Segments are numbered in line order; one starts at every CTA-range start and at every
  // tile start (a unit that is both counts once).
  __host__ __device__ long long slot_last(int ci, int t, long long seg_start) const {
    return (long long)rounds * num_ctas + (long long)full_blocks * tiles_rem + ci + t - seg_start / lcm_last;
  }
};

// Token step visited at position i of a segment.  Segments of different tile rows start at
// different offsets (and wrap around), so that the CTAs that walk the same token range do not all
// ask L2 for the same rows of B at the same moment.  The sum of a segment does not depend on the
// order of its steps up to fp32 rounding, and the order is a fixed function of the schedule.
__host__ __device__ inline int sketch_step(int ks0, int ks1, int tile_m, int i) {
  const int len = ks1 - ks0;
  int k = i + (tile_m * SK_STAGGER) % len;
  if (k >= len) k -= len;
  return ks0 + k;
}

// One segment of work of a CTA.
struct SketchSegment {
  int tile, ks0, ks1;
  long long slot;
};

// Enumerates the segments of CTA `cta` in execution order; returns false when exhausted.
// `it` and `cursor` are the iteration state (start both at 0).
__host__ __device__ inline bool sketch_next_segment(const SketchSchedule& sc, int cta, int& it, long long& cursor,
                                                    SketchSegment& seg) {
  if (it < sc.rounds) {                       // whole tiles
    seg.tile = it * sc.num_ctas + cta;
    seg.ks0 = 0; seg.ks1 = sc.ksteps;
    seg.slot = sc.slot_round(seg.tile);
    ++it;
    return true;
  }
  if (sc.tiles_rem == 0) return false;
  const int base_tile = sc.rounds * sc.num_ctas;
  const int nfull = sc.full_blocks * sc.tiles_rem;       // CTAs that own a full block
  if (cta < nfull) {
    if (it > sc.rounds) return false;
    const int b = cta / sc.tiles_rem, t = cta % sc.tiles_rem;
    seg.tile = base_tile + t;
    seg.ks0 = b * sc.upc;
    seg.ks1 = seg.ks0 + sc.upc < sc.ksteps ? seg.ks0 + sc.upc : sc.ksteps;   // the last block may be narrower
    seg.slot = sc.slot_block(b, t);
    ++it;
    return true;
  }
  if (sc.w_last == 0) return false;
  const int ci = cta - nfull;
  const long long total = (long long)sc.tiles_rem * sc.w_last;
  const long long begin = (long long)ci * sc.upl;
  const long long end = begin + sc.upl < total ? begin + sc.upl : total;
  if (it == sc.rounds) { cursor = begin; }
  if (cursor >= end) return false;
  const int t = (int)(cursor / sc.w_last);
  const int off = (int)(cursor % sc.w_last);
  const long long rem = end - cursor;
  const int len = (int)((sc.w_last - off < rem) ? sc.w_last - off : rem);
  seg.tile = base_tile + t;
  seg.ks0 = sc.full_blocks * sc.upc + off;
  seg.ks1 = seg.ks0 + len;
  seg.slot = sc.slot_last(ci, t, cursor);
  cursor += len;
  ++it;
  return true;
}

// Calls f(slot) for every partial tile of output tile `tile`, in schedule order (the order in
// which sketch_reduce_kernel adds them).
template <class F>
__host__ __device__ inline void sketch_for_each_slot_of_tile(const SketchSchedule& sc, int tile, F&& f) {
  const int base_tile = sc.rounds * sc.num_ctas;
  if (tile < base_tile) {
    f(sc.slot_round(tile));
    return;
  }
  const int t = tile - base_tile;
  for (int b = 0; b < sc.full_blocks; ++b) f(sc.slot_block(b, t));
  if (sc.w_last > 0) {
    const int ci_first = (int)(((long long)t * sc.w_last) / sc.upl);
    const int ci_last = (int)((((long long)t + 1) * sc.w_last - 1) / sc.upl);
    for (int ci = ci_first; ci <= ci_last; ++ci) {
      const long long cs = (long long)ci * sc.upl, ts = (long long)t * sc.w_last;
      f(sc.slot_last(ci, t, cs > ts ? cs : ts));
    }
  }
}

inline long long gcd_ll(long long a, long long b) { while (b) { long long t = a % b; a = b; b = t; } return a; }

// Cluster size for a result with `cols` columns: two CTAs (neighbouring 512-column blocks) share every
// generated S^T stage whenever there are at least two blocks.  With an odd number of blocks the last cluster's
// second CTA has no columns of its own: it still generates and sends its half of S^T, and skips the rest.
inline int sketch_cluster_size(long long cols) {
  const long long blocks = (cols + SK_BN - 1) / SK_BN;
  return blocks >= 2 ? 2 : 1;
}

inline SketchSchedule make_sketch_schedule(long long rows, long long cols, long long tokens, int cluster, int max_ctas) {
  SketchSchedule s;
  s.cluster = cluster;
  s.tiles_m = (int)((rows + SK_BM - 1) / SK_BM);
  s.tiles_n = (int)((cols + (long long)SK_BN * cluster - 1) / ((long long)SK_BN * cluster));
  s.ksteps = (int)((tokens + SK_AK - 1) / SK_AK);
  const int tiles = s.tiles_m * s.tiles_n;
  s.rounds = tiles / max_ctas;
  s.tiles_rem = tiles % max_ctas;
  s.num_ctas = max_ctas;
  s.upc = 0; s.full_blocks = 0; s.w_last = 0; s.upl = 1; s.lcm_last = 1;
  s.est_steps = (long long)s.rounds * (s.ksteps + 14);
  if (s.tiles_rem > 0) {
    // Every segment ends with a drain of the accumulator that the next segment has to wait for:
    // about kSegCost steps' worth.  CTAs of the last block's line work on several tiles, so they
    // get fewer units than the CTAs that own a full block.  Candidates: every full-block width
    // from the even share upwards (the rest of each tile forms the last block, shared by the
    // CTAs that are left), and equal blocks with no last block; the one whose busiest CTA
    // finishes first wins.
    constexpr int kSegCost = 14;
    const long long total = (long long)s.tiles_rem * s.ksteps;
    int upc0 = (int)((total + max_ctas - 1) / max_ctas);
    if (upc0 < 4 && upc0 < s.ksteps) upc0 = s.ksteps < 4 ? s.ksteps : 4;   // no slivers
    long long best_cost = -1;
    for (int u1 = upc0; u1 <= s.ksteps; ++u1) {
      const int fb = s.ksteps / u1;
      const int wl = s.ksteps - fb * u1;
      const long long left = (long long)max_ctas - (long long)fb * s.tiles_rem;   // CTAs for the last line
      long long cost;
      int u2 = 1;
      if (wl == 0) {
        if (left < 0) continue;
        cost = u1 + kSegCost;
      } else {
        if (left < 1) continue;
        u2 = (int)(((long long)s.tiles_rem * wl + left - 1) / left);
        const int segs = (u2 + wl - 1) / wl + 1;
        const long long c2 = u2 + (long long)kSegCost * segs;
        cost = u1 + kSegCost > c2 ? u1 + kSegCost : c2;
      }
      if (best_cost < 0 || cost < best_cost) {
        best_cost = cost;
        s.upc = u1; s.full_blocks = fb; s.w_last = wl; s.upl = u2;
      }
    }
    {   // equal blocks: every tile cut into nb blocks of the same width, one segment per CTA
      const int nb_max = max_ctas / s.tiles_rem;
      for (int nb = 1; nb <= nb_max && nb <= s.ksteps; ++nb) {
        const int ue = (s.ksteps + nb - 1) / nb;
        if (ue < 4 && ue < s.ksteps) break;
        const long long cost = ue + kSegCost;
        if (best_cost < 0 || cost <= best_cost) {
          best_cost = cost;
          s.upc = ue; s.full_blocks = (s.ksteps + ue - 1) / ue; s.w_last = 0; s.upl = 1;
        }
      }
    }
    s.est_steps += best_cost;
    if (s.w_last > 0) s.lcm_last = (long long)s.upl / gcd_ll(s.upl, s.w_last) * s.w_last;
    const long long last_ctas = s.w_last > 0 ? ((long long)s.tiles_rem * s.w_last + s.upl - 1) / s.upl : 0;
    const long long used = (long long)s.full_blocks * s.tiles_rem + last_ctas;
    if (s.rounds == 0) s.num_ctas = (int)used;          // never more than max_ctas by construction
  }
  return s;
}

struct SketchParams {
  long long rows;      // rows of S^T that are computed: B_proj (+1 with the ones row)
  long long b_proj;    // index of the ones row when ones_row != 0
  long long cols;      // columns of B and of the result
  long long tokens;    // contraction length
  float* partial;      // [num_slots][128][512] fp32
  int dist;
  int ones_row;
  int slab_map;        // tmB is the 3-D (column in slab, token, slab) view: needs cols % 64 == 0
  int* status;
  int clear_status;    // first kernel of a call: reset the status word
  uint32_t sors_mask;  // dist 3: order of the Hadamard matrix - 1
  SketchSchedule sched;
};

// Eight consecutive tokens (tok8 a multiple of 8) of sketch row j as packed bf16: one 16-byte
// chunk of the operand tile.  The distribution is a compile-time parameter: a run-time dispatch in
// this innermost routine costs the Gaussian path registers and about 2 % of the kernel's time.
template <int DIST>
__device__ __forceinline__ uint4 sketch_chunk(const PhiloxKey& pk, const SketchParams& p, long long j, long long tok8) {
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

// Layout of an S^T stage (128 rows x 64 tokens): K-major with the 128-byte swizzle: row r at
// byte 128 r, its 16-byte chunk c (tokens 8c .. 8c+7) stored at chunk position c ^ (r & 7).

template <int C, int DIST>
__global__ void __launch_bounds__(SK_THREADS, 1)
sketch_kernel(const __grid_constant__ CUtensorMap tmB, SketchParams p, PhiloxKey pk) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* a_ring = smem;
  uint8_t* b_ring = smem + SK_A_STAGES * SK_A_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(b_ring + SK_B_STAGES * SK_B_BYTES);
  const uint32_t bar0 = smem_u32(bars);
  auto fulla_bar = [&](int s) { return bar0 + 8u * s; };
  auto emptya_bar = [&](int s) { return bar0 + 8u * (SK_A_STAGES + s); };
  auto fullb_bar = [&](int s) { return bar0 + 8u * (2 * SK_A_STAGES + s); };
  auto emptyb_bar = [&](int s) { return bar0 + 8u * (2 * SK_A_STAGES + SK_B_STAGES + s); };
  const uint32_t accfull_bar = bar0 + 8u * (2 * SK_A_STAGES + 2 * SK_B_STAGES);
  const uint32_t accempty_bar = accfull_bar + 8u;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * SK_A_STAGES + 2 * SK_B_STAGES + 2);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  uint32_t* gen_count = tmem_slot + 2;           // generator warps that have stored their part of a stage

  // tasks = (row, 16-byte chunk) pairs of a stage; this CTA generates rows [rank*128/C, (rank+1)*128/C).
  // The generator warps form one group per ring stage: group g produces the K-steps g,
  // g + SK_A_STAGES, ... of this CTA's sequence, all of which go into ring stage g.  The groups
  // run out of phase, so the stores, fences and barrier round trips of one are covered by the
  // arithmetic of the others.
  constexpr int TASKS = SK_BM * 8 / C;                                         // per CTA and stage
  constexpr int GROUP_WARPS = SK_GEN_WARPS / SK_GEN_GROUPS;
  constexpr int GROUP_THREADS = 32 * GROUP_WARPS;
  constexpr int TASKS_PER_THREAD = TASKS / GROUP_THREADS;
  static_assert(SK_GEN_WARPS % SK_GEN_GROUPS == 0 && TASKS % GROUP_THREADS == 0, "generator groups");

  MBAR_PEEK_DECLARE();
  PS_TRACE_T0(trace_kernel0);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = (C == 1) ? 0u : cluster_ctarank();
  const SketchSchedule& sc = p.sched;
  const int cl = (int)(blockIdx.x / C);          // cluster index = worker index of the schedule
  if (p.clear_status && blockIdx.x == 0 && threadIdx.x == 0) *p.status = 0;

  if (threadIdx.x == 0) {
    for (int s = 0; s < SK_A_STAGES; ++s) {
      mbar_init(fulla_bar(s), GROUP_WARPS);   // C > 1: plus the bytes that the other CTAs copy in
      mbar_init(emptya_bar(s), C * SK_MMA_WARPS);
      gen_count[s] = 0;
    }
    for (int s = 0; s < SK_B_STAGES; ++s) {
      mbar_init(fullb_bar(s), 1);
      mbar_init(emptyb_bar(s), 1);              // a B stage belongs to one MMA warp
    }
    mbar_init(accfull_bar, SK_MMA_WARPS);
    mbar_init(accempty_bar, SK_GEN_WARPS);
    *abort_flag = 0;
    fence_barrier_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32(tmem_slot), 512);
    tmem_relinquish();
  }
  tc_fence_before();
  if (C == 1) __syncthreads(); else cluster_sync_all();   // every CTA's barriers exist before anyone signals across
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------ TMA producer (this CTA's B columns)
    if (lane == 0) {
      tma_prefetch_desc(&tmB);
      int s = 0;
      uint32_t ph = 0;
      bool ok = true;
      int seg_it = 0;
      long long cursor = 0;
      SketchSegment sg;
      PS_TRACE_DECL(tr_pw);
      PS_TRACE_T0(tr_pl);
      while (ok && sketch_next_segment(sc, cl, seg_it, cursor, sg)) {
        const int n0 = ((sg.tile % sc.tiles_n) * C + (int)rank) * SK_BN;
        for (int i = 0; i < sg.ks1 - sg.ks0 && ok; ++i) {
          const int ks = sketch_step(sg.ks0, sg.ks1, sg.tile / sc.tiles_n, i);
#pragma unroll
          for (int nh = 0; nh < 2; ++nh) {       // one stage per column half: 64 tokens x 256 columns
            if (n0 + nh * SK_BNH >= p.cols) continue;      // no such columns: the MMA warp of this half skips it too
            PS_TRACE_T0(tw);
            if (!mbar_wait(emptyb_bar(s), ph ^ 1u, abort_flag, p.status)) { ok = false; break; }
            PS_TRACE_ADD(tr_pw, tw);
            const uint32_t b_smem = smem_u32(b_ring) + s * SK_B_BYTES;
            mbar_arrive_expect_tx(fullb_bar(s), SK_B_BYTES);
            const int tok0 = ks * SK_AK;
            const int c0 = n0 + nh * SK_BNH;
            if (p.slab_map) {
              // one instruction for all four [64 tokens][64 columns] slabs of the stage
              tma_load_3d(b_smem, &tmB, fullb_bar(s), 0, tok0, c0 >> 6);
            } else {
#pragma unroll
              for (int sl = 0; sl < SK_BNH / 64; ++sl)
                tma_load_2d(b_smem + sl * SK_B_SLAB, &tmB, fullb_bar(s), c0 + 64 * sl, tok0);
            }
            if (++s == SK_B_STAGES) { s = 0; ph ^= 1u; }
          }
        }
      }
      PS_TRACE_PUT(1, tr_pw);
      PS_TRACE_PUT(2, clock64() - tr_pl);
    }
    __syncwarp();
  } else if (warp <= SK_MMA_WARPS) {
    // ------------------------------------------------------------ MMA issuers
    // Two warps, one per 256-column half of the accumulator.  The tensor pipe needs 128 cycles per MMA
    // (M 128 x N 256 x K 16); the issuing thread shares its scheduler with three generator warps, so its
    // loop is kept short: one barrier round (test, fence, election, commits) per four MMAs, each warp with
    // B stages of its own (64 tokens x its 256 columns), descriptors that differ only in the low word.
    // Both warps read the same S^T stages; an S^T stage is free once both (in every CTA) have committed.
    const int nh = warp - 1;
    // The whole warp runs the loop, so that descriptors and addresses stay warp-uniform (the
    // tcgen05 operands live in uniform registers); one elected lane issues.
    {
      constexpr uint32_t idesc = instr_desc_bf16(SK_BM, SK_BNH, false, true);
      // Descriptors are built once; stage and K-step offsets are added to the start-address field (16-byte
      // units, 14 bits: no carry into the high word).
      const uint64_t adesc0 = smem_desc_sw128(smem_u32(a_ring), 16, 1024);
      const uint64_t bdesc0 = smem_desc_sw128(smem_u32(b_ring), SK_B_SLAB, 1024);
      const uint32_t a_lo0 = (uint32_t)adesc0, a_hi = (uint32_t)(adesc0 >> 32);
      const uint32_t b_lo0 = (uint32_t)bdesc0, b_hi = (uint32_t)(bdesc0 >> 32);
      auto desc64 = [](uint32_t lo, uint32_t hi) { return ((uint64_t)hi << 32) | (uint64_t)lo; };
      uint32_t peer_emptya0[C];                  // emptyA[0] of every CTA of the cluster
#pragma unroll
      for (int r = 0; r < C; ++r) peer_emptya0[r] = (C == 1) ? emptya_bar(0) : mapa_shared(emptya_bar(0), r);
      // B ring: the producer fills one stage per step and column half that exists (a half that starts beyond
      // the last column is skipped); qs / qph = ring position and phase of the step's first stage.
      int sa = 0, qs = 0;
      uint32_t pha = 0, qph = 0;
      int seg = 0;
      bool ok = true;
      bool bpeek = false;                        // the B barrier of the coming step has been tested
      int seg_it = 0;
      long long cursor = 0;
      SketchSegment sg;
      // Each full barrier is tested one stage ahead (slot 0: S^T ring, slot 1: B ring).
      if (C == 1) { MBAR_PEEK(0, fulla_bar(0), 0u); } else { MBAR_PEEK_CLUSTER(0, fulla_bar(0), 0u); }
      PS_TRACE_DECL(tr_ws);
      PS_TRACE_DECL(tr_wd);
      PS_TRACE_DECL(tr_wa);
      PS_TRACE_DECL(tr_m_is);
      PS_TRACE_DECL(tr_m_co);
      PS_TRACE_T0(tr_sk0);
      for (; ok && sketch_next_segment(sc, cl, seg_it, cursor, sg); ++seg) {
        const long long n0 = (long long)((sg.tile % sc.tiles_n) * C + (int)rank) * SK_BN;
        const int live0 = n0 < p.cols ? 1 : 0, live1 = n0 + SK_BNH < p.cols ? 1 : 0;
        const bool mine = nh == 0 ? live0 != 0 : live1 != 0;      // this warp's half has columns
        const int myoff = (nh == 1 && live0) ? 1 : 0;
        if (seg > 0) {   // the previous segment's accumulator must have been drained
          PS_TRACE_T0(tw);
          ok = (mbar_wait_warp(accempty_bar, (uint32_t)(seg - 1) & 1u, abort_flag, p.status));
          PS_TRACE_ADD(tr_wa, tw);
          if (!ok) break;
          tc_fence_after();
        }
        uint32_t acc = 0;
        bpeek = false;
        for (int ks = sg.ks0; ks < sg.ks1 && ok; ++ks) {
          uint32_t ready;
          MBAR_PEEK_RESULT(0, ready);
          if (!__all_sync(0xffffffffu, ready != 0)) {
            PS_TRACE_T0(tw);
            ok = (C == 1) ? mbar_wait_warp(fulla_bar(sa), pha, abort_flag, p.status)
                          : mbar_wait_cluster_warp(fulla_bar(sa), pha, abort_flag, p.status);
            PS_TRACE_ADD(tr_ws, tw);
            if (!ok) break;
          }
          const int sa_next = (sa + 1 == SK_A_STAGES) ? 0 : sa + 1;
          const uint32_t pha_next = (sa_next == 0) ? (pha ^ 1u) : pha;
          int sb = qs + myoff;
          uint32_t phb = qph;
          if (sb >= SK_B_STAGES) { sb -= SK_B_STAGES; phb ^= 1u; }
          int qn = qs + live0 + live1;
          uint32_t qphn = qph;
          if (qn >= SK_B_STAGES) { qn -= SK_B_STAGES; qphn ^= 1u; }
          bool issuer = false;
          if (mine) {
            ready = 0;
            if (bpeek) MBAR_PEEK_RESULT(1, ready);
            if (!__all_sync(0xffffffffu, ready != 0)) {
              PS_TRACE_T0(tw);
              ok = (mbar_wait_warp(fullb_bar(sb), phb, abort_flag, p.status));
              PS_TRACE_ADD(tr_wd, tw);
              if (!ok) break;
            }
            tc_fence_after();
            const uint32_t a_lo = a_lo0 + (uint32_t)(sa * (SK_A_BYTES >> 4));
            const uint32_t b_lo = b_lo0 + (uint32_t)(sb * (SK_B_BYTES >> 4));
            PS_TRACE_T0(tis);
            issuer = elect_one();
            if (issuer) {
#pragma unroll
              for (int j = 0; j < SK_AK / 16; ++j)
                umma_bf16(tmem_base + nh * SK_BNH, desc64(a_lo + (uint32_t)(j * 2), a_hi),
                          desc64(b_lo + (uint32_t)((j * 2048) >> 4), b_hi), idesc, j == 0 ? acc : 1u);
            }
            PS_TRACE_ADD(tr_m_is, tis);
            // the tests of the next stages travel while the commits are issued
            bpeek = ks + 1 < sg.ks1;
            if (bpeek) {
              int sbn = qn + myoff;
              uint32_t phbn = qphn;
              if (sbn >= SK_B_STAGES) { sbn -= SK_B_STAGES; phbn ^= 1u; }
              MBAR_PEEK(1, fullb_bar(sbn), phbn);
            }
          } else {
            issuer = elect_one();
          }
          PS_TRACE_T0(tco);
          if (C == 1) { MBAR_PEEK(0, fulla_bar(sa_next), pha_next); } else { MBAR_PEEK_CLUSTER(0, fulla_bar(sa_next), pha_next); }
          if (issuer) {
            if (mine) umma_commit(emptyb_bar(sb));
            // tell every CTA of the cluster (all of them write into this stage) that this warp is done with it
#pragma unroll
            for (int r = 0; r < C; ++r) umma_commit(peer_emptya0[r] + 8u * sa);
          }
          __syncwarp();
          PS_TRACE_ADD(tr_m_co, tco);
          acc = 1;
          qs = qn;
          qph = qphn;
          sa = sa_next;
          pha = pha_next;
        }
        if (ok) {
          if (elect_one()) umma_commit(accfull_bar);
          __syncwarp();
        }
      }
      if (warp == 1 && lane == 0) {
        PS_TRACE_PUT(3, tr_ws); PS_TRACE_PUT(4, tr_wd); PS_TRACE_PUT(5, tr_wa); PS_TRACE_PUT(6, clock64() - tr_sk0);
        PS_TRACE_PUT(20, tr_m_is); PS_TRACE_PUT(21, tr_m_co);
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------ S generators + accumulator drain
    const int gw = warp - 1 - SK_MMA_WARPS;
    const int grp = gw / GROUP_WARPS;            // this warp's group
    const int gtid = (gw % GROUP_WARPS) * 32 + lane;   // thread index within the group
    constexpr uint32_t PART_BYTES = SK_A_BYTES / C;   // this CTA's rows of a stage: one contiguous block
    const uint32_t part_smem = smem_u32(a_ring) + rank * PART_BYTES;   // that block in stage 0 of this CTA's ring
    uint32_t peer_part[C];                       // the same place in the ring of every CTA of the cluster
    uint32_t peer_fulla[C];                      // fullA[0] of every CTA of the cluster
    if (C > 1) {
#pragma unroll
      for (int r = 0; r < C; ++r) {
        peer_part[r] = mapa_shared(part_smem, r);
        peer_fulla[r] = mapa_shared(fulla_bar(0), r);
      }
    }
    int step0 = 0;                               // position of the segment's first K-step in this CTA's sequence
    int seg = 0;
    bool ok = true;
    int seg_it = 0;
    long long cursor = 0;
    SketchSegment sg;
    PS_TRACE_DECL(tr_gen);
    PS_TRACE_DECL(tr_gw);
    PS_TRACE_DECL(tr_g_ar);
    PS_TRACE_DECL(tr_dw);
    PS_TRACE_DECL(tr_dr);
    PS_TRACE_T0(tr_gl0);
    for (; ok && sketch_next_segment(sc, cl, seg_it, cursor, sg); ++seg) {
      const int tile = sg.tile;
      const long long m0 = (long long)(tile / sc.tiles_n) * SK_BM;
      const int len = sg.ks1 - sg.ks0;
      // the group's first step of this segment: the first i with (step0 + i) % groups == grp
      for (int i = (grp + SK_GEN_GROUPS - step0 % SK_GEN_GROUPS) % SK_GEN_GROUPS; i < len; i += SK_GEN_GROUPS) {
        const int ks = sketch_step(sg.ks0, sg.ks1, tile / sc.tiles_n, i);
        const int step = step0 + i;
        const int sa = grp;                                         // ring stage of this step (step % stages)
        const uint32_t pha = (uint32_t)(step / SK_A_STAGES) & 1u;   // and its parity
        // Generate first, into registers: the entries do not depend on the ring, so the wait for
        // the free stage only covers the stores.
        PS_TRACE_T0(tg0);
        uint4 v[TASKS_PER_THREAD];
        uint32_t off[TASKS_PER_THREAD];
#pragma unroll
        for (int it = 0; it < TASKS_PER_THREAD; ++it) {
          const int t = it * GROUP_THREADS + gtid;
          const int r = (int)rank * (SK_BM / C) + (t >> 3), c = t & 7;
          v[it] = sketch_chunk<DIST>(pk, p, m0 + r, (long long)ks * SK_AK + 8 * c);
          off[it] = (uint32_t)(r * 128 + ((c ^ (r & 7)) << 4));
        }
        PS_TRACE_ADD(tr_gen, tg0);
        PS_TRACE_T0(tgw);
        const bool freed = (C == 1) ? mbar_wait_warp(emptya_bar(sa), pha ^ 1u, abort_flag, p.status)
                                    : mbar_wait_cluster_warp(emptya_bar(sa), pha ^ 1u, abort_flag, p.status);
        PS_TRACE_ADD(tr_gw, tgw);
        if (!freed) { ok = false; break; }
        PS_TRACE_T0(tar);
        uint8_t* const stage_ptr = a_ring + sa * SK_A_BYTES;
#pragma unroll
        for (int it = 0; it < TASKS_PER_THREAD; ++it) *reinterpret_cast<uint4*>(stage_ptr + off[it]) = v[it];
        fence_proxy_async_smem();
        __syncwarp();
        if (lane == 0) {
          if (C == 1) {
            mbar_arrive(fulla_bar(sa));
          } else {
            // The stage is complete here once the group's warps have arrived and the other CTAs'
            // rows have been copied in; the copies count their bytes on this barrier.
            if (gtid == 0) mbar_arrive_expect_tx(fulla_bar(sa), SK_A_BYTES - PART_BYTES);
            else mbar_arrive(fulla_bar(sa));
            // The warp that stores last sends this CTA's rows to the other CTAs with one bulk
            // copy each.  The counter only grows: a stage is reused after its barrier has
            // completed, so the counts of two uses never mix.
            __threadfence_block();
            const uint32_t n = atomicAdd(&gen_count[sa], 1u);
            if ((n % GROUP_WARPS) == GROUP_WARPS - 1) {
              __threadfence_block();
#pragma unroll
              for (int q = 0; q < C; ++q)
                if (q != (int)rank)
                  bulk_copy_to_cluster(peer_part[q] + sa * SK_A_BYTES, part_smem + sa * SK_A_BYTES, PART_BYTES,
                                       peer_fulla[q] + 8u * sa);
            }
          }
        }
        PS_TRACE_ADD(tr_g_ar, tar);
      }
      step0 += len;
      PS_TRACE_T0(tdw);
      ok = ok && mbar_wait_warp(accfull_bar, (uint32_t)seg & 1u, abort_flag, p.status);
      PS_TRACE_ADD(tr_dw, tdw);
      if (!ok) break;
      tc_fence_after();
      PS_TRACE_T0(tdr);
      {
        const int q = warp & 3;                 // tensor-memory lane quarter of this warp
        const int cgroup = gw >> 2;             // index among the SK_GEN_WARPS / 4 warps that share the quarter
        float* slot = p.partial + (sg.slot * C + rank) * (long long)SK_TILE_ELEMS;
        float* prow = slot + (long long)(q * 32 + lane) * 4;   // this lane's row, quad-major layout
        const long long n0d = (long long)((tile % sc.tiles_n) * C + (int)rank) * SK_BN;
        for (int c = cgroup; c < SK_BN / 32; c += SK_GEN_WARPS / 4) {   // 32-column chunks, dealt round-robin
          if (n0d + c * 32 >= p.cols) break;    // columns beyond the result: nothing was accumulated, nothing is read
          uint32_t v[32];
          tmem_ld_32x32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(c * 32), v);
          tmem_ld_wait();
#pragma unroll
          for (int g = 0; g < 8; ++g)
            *reinterpret_cast<uint4*>(prow + (long long)(c * 8 + g) * SK_BM * 4) = make_uint4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(accempty_bar);
      PS_TRACE_ADD(tr_dr, tdr);
    }
    if (warp == 1 + SK_MMA_WARPS && lane == 0) {
      PS_TRACE_PUT(8, tr_gen); PS_TRACE_PUT(9, tr_gw); PS_TRACE_PUT(10, clock64() - tr_gl0); PS_TRACE_PUT(18, tr_g_ar);
      PS_TRACE_PUT(11, tr_dw); PS_TRACE_PUT(12, tr_dr);
    }
  }
  // ---------------------------------------------------------------- teardown
  if (*abort_flag) {
    // give copies that may still be in flight time to land before the shared memory is released
    const long long t0 = clock64();
    while (clock64() - t0 < 2000000ll) __nanosleep(1000);
  }
  tc_fence_before();
  if (C == 1) __syncthreads(); else cluster_sync_all();   // nobody leaves while a neighbour may still store or signal here
  if (warp == 1) tmem_dealloc(tmem_base, 512);
  if (threadIdx.x == 0) PS_TRACE_PUT(0, clock64() - trace_kernel0);
}

// Layout of a partial tile (128 rows x 512 columns, fp32): column quads are outermost, element
// (r, col) sits at float index ((col / 4) * 128 + r) * 4 + col % 4.  The accumulator comes out
// of tensor memory one row per lane, so a warp's 16-byte stores of one quad are 512 contiguous
// bytes, and the reduce kernel, one row per thread, reads them back the same way.
__host__ __device__ inline long long sketch_partial_index(int r, int col) {
  return ((long long)(col >> 2) * SK_BM + r) * 4 + (col & 3);
}

// Adds the partial tiles of each output tile in schedule order, scales, rounds to bf16.
// grid = (tile groups * C, 32 column chunks), block = 128 threads: thread t owns row t of the
// tile and the 16 columns of the chunk; blockIdx.x = C * tile group + rank of the CTA that
// produced the 512-column block.  The kernel is bound by the latency of its loads (a few tens of
// MB, mostly out of L2), so a thread fetches its 16 columns of four partial tiles at a time (16
// independent 16-byte loads in flight) and then adds them in schedule order: the sum is the same
// fixed sequence of fp32 additions whatever the batching.
constexpr int SKR_CHUNK = 16;        // columns per block of the reduce kernel
constexpr int SKR_BATCH = 4;         // partial tiles fetched together
__global__ void __launch_bounds__(SK_BM)
sketch_reduce_kernel(SketchParams p, float scale, __nv_bfloat16* __restrict__ out, __nv_bfloat16* __restrict__ ones_out) {
  const SketchSchedule& sc = p.sched;
  const int per_tile = sc.cluster;      // partial tiles (CTAs) per schedule tile
  const int tile = blockIdx.x / per_tile, rank = blockIdx.x % per_tile;
  const long long m0 = (long long)(tile / sc.tiles_n) * SK_BM;
  const long long n0 = ((long long)(tile % sc.tiles_n) * sc.cluster + rank) * SK_BN;
  const int r = threadIdx.x;
  const long long j = m0 + r;
  const int col0 = blockIdx.y * SKR_CHUNK;
  if (j >= p.rows || n0 + col0 >= p.cols) return;
  constexpr int Q = SKR_CHUNK / 4;      // float4 per thread and partial tile
  float4 acc[Q];
#pragma unroll
  for (int g = 0; g < Q; ++g) acc[g] = make_float4(0.f, 0.f, 0.f, 0.f);
  const long long off = sketch_partial_index(r, col0);
  const float* pending[SKR_BATCH];
  int npending = 0;
  auto flush = [&]() {
    float4 v[SKR_BATCH][Q];
#pragma unroll
    for (int b = 0; b < SKR_BATCH; ++b) {
      if (b < npending) {
#pragma unroll
        for (int g = 0; g < Q; ++g) v[b][g] = __ldcs(reinterpret_cast<const float4*>(pending[b] + (long long)g * SK_BM * 4));
      }
    }
#pragma unroll
    for (int b = 0; b < SKR_BATCH; ++b) {
      if (b < npending) {
#pragma unroll
        for (int g = 0; g < Q; ++g) { acc[g].x += v[b][g].x; acc[g].y += v[b][g].y; acc[g].z += v[b][g].z; acc[g].w += v[b][g].w; }
      }
    }
    npending = 0;
  };
  sketch_for_each_slot_of_tile(sc, tile, [&](long long slot_index) {
    const float* src = p.partial + (slot_index * per_tile + rank) * (long long)SK_TILE_ELEMS + off;
    // constant indices only, so that the array stays in registers
#pragma unroll
    for (int b = 0; b < SKR_BATCH; ++b)
      if (b == npending) pending[b] = src;
    if (++npending == SKR_BATCH) flush();
  });
  flush();
  const bool is_ones = p.ones_row && j == p.b_proj;
  const float s = is_ones ? 1.0f : scale;
  __nv_bfloat16* dst = is_ones ? ones_out : out + j * p.cols;
  if (dst == nullptr) return;
  dst += n0 + col0;
  // cols is a multiple of 8: the 8 columns of a 16-byte store are all inside or all outside
#pragma unroll
  for (int g = 0; g < SKR_CHUNK / 8; ++g) {
    if (n0 + col0 + 8 * g >= p.cols) break;
    const float4 a = acc[2 * g], b = acc[2 * g + 1];
    __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x * s, a.y * s), h1 = __floats2bfloat162_rn(a.z * s, a.w * s);
    __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x * s, b.y * s), h3 = __floats2bfloat162_rn(b.z * s, b.w * s);
    *reinterpret_cast<uint4*>(dst + 8 * g) = make_uint4(*reinterpret_cast<uint32_t*>(&h0), *reinterpret_cast<uint32_t*>(&h1),
                                                        *reinterpret_cast<uint32_t*>(&h2), *reinterpret_cast<uint32_t*>(&h3));
  }
}

}  // namespace tc
}  // namespace rmm
