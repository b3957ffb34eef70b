// C ABI of the RMM linear layer (see include/rmm.h): argument checks, workspace
// layout, TMA tensor maps and kernel launches.  All arithmetic runs in the kernels.
#include "../../include/rmm.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>
#include <chrono>
#include <cstring>
#include <mutex>
#include <vector>

#include "simt_kernels.cuh"
#include "sketch_rng.cuh"
#include "tc_gemm.cuh"
#include "fwht_kernels.cuh"
#include "tc_sketch.cuh"
#include "tc_pass.cuh"
#include "variance_kernels.cuh"

namespace {

using namespace rmm;

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
inline size_t elem_bytes(rmm_dtype dt) { return dt == RMM_DTYPE_BF16 ? 2 : 4; }

// ------------------------------------------------------------------ workspace layout
// [status word | G = S^T dY | scratch], scratch = fp32 partial tiles of the sketch kernels
// (bf16 mode) or partial column sums of db (fp32 mode).
struct Workspace {
  size_t status_off, ticket_off, g_off, scratch_off, total;
  int db_rows_per_slice, db_slices;
};

// Geometry of the sketch part of a pass (tc_pass.cuh): a pair tile is 128 sketch rows x nat x 256 data
// columns; the column groups are balanced so that no group is mostly padding.
struct SketchGeometry {
  int tiles_m, groups, nat, ksteps;
  int tiles() const { return tiles_m * groups; }
  // Upper bound of the number of token blocks per tile, whatever the device: at most kMaxUnits units in all
  // (one or two per CTA pair of the largest grid) unless the tiles alone are more.
  static constexpr int kMaxUnits = 2 * tc::PS_MAX_PAIRS;
  int nb_cap() const {
    int c = kMaxUnits / tiles();
    if (c < 1) c = 1;
    return c < ksteps ? c : ksteps;
  }
  size_t scratch_bytes() const {
    return (size_t)tiles() * (size_t)nb_cap() * tc::PS_ROWS * (size_t)nat * 256 * sizeof(float);
  }
};

SketchGeometry sketch_geometry(int64_t rows, int64_t cols, int64_t tokens) {
  SketchGeometry g;
  const int64_t t256 = (cols + 255) / 256;
  g.groups = (int)((t256 + tc::PS_MAX_NAT - 1) / tc::PS_MAX_NAT);
  g.nat = (int)((t256 + g.groups - 1) / g.groups);
  g.tiles_m = (int)((rows + tc::PS_ROWS - 1) / tc::PS_ROWS);
  g.ksteps = (int)((tokens + 63) / 64);
  return g;
}

Workspace workspace_layout(int64_t N, int64_t D_in, int64_t D_out, int64_t k, rmm_dtype dt) {
  Workspace w;
  w.status_off = 0;
  w.ticket_off = kAlign;
  size_t off = w.ticket_off;
  size_t scratch_pass = 0;
  if (dt == RMM_DTYPE_BF16) {
    const SketchGeometry gf = sketch_geometry(k, D_in, N), gb = sketch_geometry(k + 1, D_out, N);
    const int tmax = gf.tiles() > gb.tiles() ? gf.tiles() : gb.tiles();
    // completion flags of the partial tiles: one per partial tile and CTA of a cluster (or pair)
    off += align_up(((size_t)tmax + 2 * tc::SK_MAX_CTAS) * 2 * sizeof(unsigned long long));
    scratch_pass = gf.scratch_bytes() > gb.scratch_bytes() ? gf.scratch_bytes() : gb.scratch_bytes();
  }
  w.g_off = off;
  off = w.g_off + align_up((size_t)k * (size_t)D_out * elem_bytes(dt));
  int64_t rps = 32;                       // rows per slice of the fp32 mode's db partial sums: at most 256 slices
  if ((N + rps - 1) / rps > 256) rps = (N + 255) / 256;
  w.db_rows_per_slice = (int)rps;
  w.db_slices = (int)((N + rps - 1) / rps);
  w.scratch_off = off;
  size_t scratch = (size_t)w.db_slices * (size_t)D_out * sizeof(float);
  if (dt == RMM_DTYPE_BF16) {
    // an upper bound over every grid the launch may use: one partial tile per (tile, CTA) pair at most
    // (512-column blocks are counted in pairs: a cluster of two CTAs has a slot for each of its CTAs)
    auto blocks2 = [](int64_t d) { const int64_t b = (d + tc::SK_BN - 1) / tc::SK_BN; return b >= 2 ? (b + 1) / 2 * 2 : b; };
    const long long tf = ((k + tc::SK_BM - 1) / tc::SK_BM) * blocks2(D_in);
    const long long tb = ((k + 1 + tc::SK_BM - 1) / tc::SK_BM) * blocks2(D_out);
    scratch = (size_t)((tf > tb ? tf : tb) + tc::SK_MAX_CTAS) * tc::SK_TILE_ELEMS * sizeof(float);
    if (scratch_pass > scratch) scratch = scratch_pass;
  }
  off += align_up(scratch);
  w.total = off;
  return w;
}

// ------------------------------------------------------------------ device / driver set-up
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct DeviceState {
  bool ok = false;
  EncodeTiledFn encode = nullptr;
  int num_sms = 0;
  int gemm_pairs = 0;                         // CTA pairs of the GEMM kernel resident at once
  int sketch_clusters[5] = {0, 0, 0, 0, 0};   // [C]: clusters of C CTAs of the sketch kernel resident at once
  int pass_pairs = 0;                         // CTA pairs of the pass kernel resident at once
  // side lanes for the two kernels of a pass that run at the same time: a stream and two events each
  static constexpr int kLanes = 8;
  cudaStream_t lane_stream[kLanes] = {};
  cudaEvent_t lane_fork[kLanes] = {}, lane_join[kLanes] = {};
  std::mutex lane_mutex[kLanes];
  std::atomic<unsigned> next_lane{0};
  bool lanes_ok = false;
};

template <typename K>
bool allow_big_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

constexpr int kNumDists = 5;     // rmm_dist values 0..4

// The sketch kernel for a cluster size (1 or 2) and a distribution (rmm_dist value).
typedef void (*SketchKernelFn)(const CUtensorMap, tc::SketchParams, PhiloxKey);
SketchKernelFn sketch_kernel_fn(int c, int dist) {
  static const SketchKernelFn table[2][kNumDists] = {
      {tc::sketch_kernel<1, 0>, tc::sketch_kernel<1, 1>, tc::sketch_kernel<1, 2>, tc::sketch_kernel<1, 3>,
       tc::sketch_kernel<1, 4>},
      {tc::sketch_kernel<2, 0>, tc::sketch_kernel<2, 1>, tc::sketch_kernel<2, 2>, tc::sketch_kernel<2, 3>,
       tc::sketch_kernel<2, 4>}};
  return table[c == 2 ? 1 : 0][dist >= 0 && dist < kNumDists ? dist : 0];
}

// The pass kernel for an operand mode of the dense part (B_K: Y = X W^T, B_MN: dX = dY W) and a distribution.
typedef void (*PassKernelFn)(const CUtensorMap, const CUtensorMap, const CUtensorMap, const CUtensorMap, tc::PassParams,
                             PhiloxKey);
PassKernelFn pass_kernel_fn(int bmode, int dist) {
  static const PassKernelFn table[2][kNumDists] = {
      {tc::pass_kernel<tc::B_K, 0>, tc::pass_kernel<tc::B_K, 1>, tc::pass_kernel<tc::B_K, 2>, tc::pass_kernel<tc::B_K, 3>,
       tc::pass_kernel<tc::B_K, 4>},
      {tc::pass_kernel<tc::B_MN, 0>, tc::pass_kernel<tc::B_MN, 1>, tc::pass_kernel<tc::B_MN, 2>,
       tc::pass_kernel<tc::B_MN, 3>, tc::pass_kernel<tc::B_MN, 4>}};
  return table[bmode == tc::B_MN ? 1 : 0][dist >= 0 && dist < kNumDists ? dist : 0];
}

// How many clusters of `c` CTAs of kernel `k` can be resident on the device at once.
template <typename K>
bool query_clusters(K k, int c, int* out, int threads = tc::SK_THREADS, int smem = tc::SK_SMEM_BYTES) {
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)c; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3((unsigned)(tc::SK_MAX_CTAS / c * c));
  cfg.blockDim = dim3((unsigned)threads);
  cfg.dynamicSmemBytes = (size_t)smem;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, k, &cfg) != cudaSuccess || n < 1) return false;
  *out = n < tc::SK_MAX_CTAS / c ? n : tc::SK_MAX_CTAS / c;
  return true;
}

// Per-device set-up, done at the first call made with that device current: the shared-memory opt-in
// of the kernels (a per-device function attribute) and the residency counts that size the grids.
constexpr int kMaxDevices = 64;

void init_device_state(DeviceState& st, int dev) {
  int major = 0, minor = 0;
  if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return;
  if (cudaDeviceGetAttribute(&minor, cudaDevAttrComputeCapabilityMinor, dev) != cudaSuccess) return;
  if (major != 10) return;  // the kernels are sm_100a only; there is no other path
  if (cudaDeviceGetAttribute(&st.num_sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess ||
      qres != cudaDriverEntryPointSuccess || fn == nullptr)
    return;
  st.encode = reinterpret_cast<EncodeTiledFn>(fn);
  bool a = true;
  a &= allow_big_smem(tc::gemm_kernel<tc::A_K, tc::B_K>, tc::GEMM_SMEM_BYTES);
  a &= allow_big_smem(tc::gemm_kernel<tc::A_K, tc::B_MN>, tc::GEMM_SMEM_BYTES);
  a &= allow_big_smem(tc::gemm_kernel<tc::A_MN, tc::B_MN>, tc::GEMM_SMEM_BYTES);
  for (int c = 1; c <= 2; ++c)
    for (int d = 0; d < kNumDists; ++d) a &= allow_big_smem(sketch_kernel_fn(c, d), tc::SK_SMEM_BYTES);
  for (int bm = 0; bm < 2; ++bm)
    for (int d = 0; d < kNumDists; ++d) a &= allow_big_smem(pass_kernel_fn(bm, d), tc::PS_SMEM_BYTES);
  if (a) {
    a &= query_clusters(tc::pass_kernel<tc::B_K, 0>, 2, &st.pass_pairs, tc::PS_THREADS, tc::PS_SMEM_BYTES);
    if (st.pass_pairs > tc::PS_MAX_PAIRS) st.pass_pairs = tc::PS_MAX_PAIRS;
    st.sketch_clusters[1] = st.num_sms < tc::SK_MAX_CTAS ? st.num_sms : tc::SK_MAX_CTAS;
    a &= query_clusters(tc::sketch_kernel<2, 0>, 2, &st.sketch_clusters[2]);   // the same for every distribution
    a &= query_clusters(tc::gemm_kernel<tc::A_K, tc::B_K>, 2, &st.gemm_pairs, 64 + 32 * tc::NEPI, tc::GEMM_SMEM_BYTES);
  }
  if (a) {
    bool l = true;
    for (int i = 0; i < DeviceState::kLanes && l; ++i) {
      l &= cudaStreamCreateWithFlags(&st.lane_stream[i], cudaStreamNonBlocking) == cudaSuccess;
      l &= cudaEventCreateWithFlags(&st.lane_fork[i], cudaEventDisableTiming) == cudaSuccess;
      l &= cudaEventCreateWithFlags(&st.lane_join[i], cudaEventDisableTiming) == cudaSuccess;
    }
    st.lanes_ok = l;
  }
  st.ok = a;
}

// State of the device that is current on the calling thread.  A device that cannot run the kernels (or an
// index beyond kMaxDevices) yields a state with ok == false, and the entry points return RMM_ERR_CUDA.
DeviceState& device_state() {
  static DeviceState states[kMaxDevices];
  static bool tried[kMaxDevices] = {};
  static DeviceState none;
  static std::mutex mu;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return none;
  std::lock_guard<std::mutex> lock(mu);
  if (!tried[dev]) {
    tried[dev] = true;
    init_device_state(states[dev], dev);
  }
  return states[dev];
}

// Tensor map of a row-major bf16 matrix [rows][cols] (cols contiguous), box = [box_rows][64 cols],
// 128-byte swizzle, out-of-range elements read as zero.
bool make_tmap(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  return device_state().encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box,
                               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Tensor map of a row-major bf16 matrix [rows][cols], cols a multiple of 64, viewed as
// (column in slab: 64, row, slab: cols / 64); box = [box_slabs][box_rows][64]: in shared memory the
// slabs ([box_rows][64 columns], 128-byte swizzle) follow one another, which is the MN-major
// operand layout, and one TMA instruction fetches all of them.  Rows out of range read as zero.
bool make_tmap_slabs(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows, int box_slabs) {
  cuuint64_t gdim[3] = {64u, (cuuint64_t)rows, (cuuint64_t)(cols / 64)};
  cuuint64_t gstride[2] = {(cuuint64_t)cols * 2, 128u};
  cuuint32_t box[3] = {64u, (cuuint32_t)box_rows, (cuuint32_t)box_slabs};
  cuuint32_t estr[3] = {1u, 1u, 1u};
  return device_state().encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box,
                               estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                               CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Kernels launched by rmm_forward / rmm_backward (and their host-buffer wrappers) since the library was loaded.
std::atomic<long long> g_layer_launches{0};
inline void note_launches(int n) { g_layer_launches.fetch_add(n, std::memory_order_relaxed); }

// ------------------------------------------------------------------ per-kernel timing (benchmarks)
struct ProfileRecord { int step; cudaEvent_t t0, t1; };
struct Profiler {
  std::vector<ProfileRecord> pool;
  size_t used = 0;
};
Profiler& profiler() {
  static Profiler p;
  return p;
}
// Brackets the launches made while it is alive with two events on the stream.
struct ScopedTiming {
  ProfileRecord* rec = nullptr;
  cudaStream_t stream;
  ScopedTiming(int step, cudaStream_t s) : stream(s) {
    Profiler& p = profiler();
    if (p.used < p.pool.size()) {
      rec = &p.pool[p.used++];
      rec->step = step;
      cudaEventRecord(rec->t0, stream);
    }
  }
  ~ScopedTiming() {
    if (rec) cudaEventRecord(rec->t1, stream);
  }
};

// ------------------------------------------------------------------ launches
// One contraction on the tensor cores.  a/b are row-major bf16 matrices:
//   A_K : a is [M][K]   A_MN: a is [K][M]
//   B_K : b is [N][K]   B_MN: b is [K][N]
// Number of CTAs launch_tc uses for an M x N result (the size of the optional sumsq array is NEPI times this).
int tc_grid_ctas(int64_t M, int64_t N) {
  const int64_t tiles = ((N + tc::BN - 1) / tc::BN) * ((M + tc::PAIR_M - 1) / tc::PAIR_M);
  const int max_pairs = device_state().gemm_pairs;
  return 2 * (int)(tiles < max_pairs ? tiles : max_pairs);
}

template <int AMODE, int BMODE>
rmm_status launch_tc(const void* a, const void* b, void* c, const void* bias, int64_t M, int64_t N, int64_t K,
                     float alpha, int* status, cudaStream_t stream, double* sumsq = nullptr, bool clear_status = false,
                     int pairs_limit = 0) {
  CUtensorMap tmA, tmB, tmC;
  bool ok = make_tmap(&tmC, c, M, N, 32);        // store boxes of the epilogue: [32 rows][64 columns]
  if (AMODE == tc::A_K) ok &= make_tmap(&tmA, a, M, K, tc::BM);
  if (AMODE == tc::A_MN) ok &= make_tmap(&tmA, a, K, M, tc::BK);
  if (BMODE == tc::B_K) ok &= make_tmap(&tmB, b, N, K, tc::BN_HALF);
  if (BMODE == tc::B_MN) ok &= make_tmap(&tmB, b, K, N, tc::BK);
  if (!ok) return RMM_ERR_CUDA;
  tc::GemmParams p;
  p.M = M; p.N = N; p.K = K;
  p.bias = bias; p.alpha = alpha; p.status = status; p.sumsq = sumsq; p.clear_status = clear_status ? 1 : 0;
  const int64_t tiles = ((N + tc::BN - 1) / tc::BN) * ((M + tc::PAIR_M - 1) / tc::PAIR_M);
  int max_pairs = device_state().gemm_pairs;
  if (pairs_limit > 0 && pairs_limit < max_pairs) max_pairs = pairs_limit;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(2 * (unsigned)(tiles < max_pairs ? tiles : max_pairs));   // persistent CTA pairs
  cfg.blockDim = dim3(64 + 32 * tc::NEPI);
  cfg.dynamicSmemBytes = tc::GEMM_SMEM_BYTES;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, tc::gemm_kernel<AMODE, BMODE>, tmA, tmB, tmC, p) != cudaSuccess) return RMM_ERR_CUDA;
  note_launches(1);
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

// Sketch contraction out[j][d] = c * sum_n P[n][j] * b[n][d] for j < k (b is [tokens][cols] bf16),
// and, when ones_out is given, ones_out[d] = sum_n b[n][d] from the extra row of ones.
// The subsampled-Hadamard sketch by a two-level Walsh-Hadamard transform (fwht_kernels.cuh).  Returns
// RMM_ERR_UNSUPPORTED when the shape is outside the fast path (the caller then takes the dense kernel).
// scratch holds, in this order: the grouped column list, the per-block column sums, the stage-1 result
// T for as many columns per round as fit.
// Layout of the fast path's scratch for a sketch of k rows over `cols` columns and `tokens` rows; false when the
// shape is outside the fast path (Hadamard order below 128 or above 16384, or scratch too small).
struct SorsFastPlan {
  uint32_t mask;
  int A;
  size_t entries_off, colsum_off, t_off;
  int64_t wslab;
};
bool sors_fast_plan(int64_t k, int64_t cols, int64_t tokens, size_t scratch_bytes, SorsFastPlan* plan) {
  const uint32_t mask = sors_mask_for(tokens);
  const int64_t L = (int64_t)mask + 1;
  if (L < FW_ROWS || L > (int64_t)FW_ROWS * FW_ROWS) return false;
  const int A = (int)(L / FW_ROWS);
  size_t off = align_up(129 * sizeof(int));
  const size_t entries_off = off;
  off += align_up((size_t)k * sizeof(int2));
  if (off + 2 * kAlign >= scratch_bytes) return false;
  const size_t per_col = (size_t)A * sizeof(float) + (size_t)L * 2;       // column sums + T, per column of a round
  const int64_t cols64 = (cols + FW_COLS - 1) / FW_COLS * FW_COLS;
  int64_t wslab = (int64_t)((scratch_bytes - off - 2 * kAlign) / per_col) / FW_COLS * FW_COLS;
  if (wslab > cols64) wslab = cols64;
  if (wslab < FW_COLS) return false;
  {   // rounds of equal width rather than full ones and a narrow last one
    const int64_t rounds = (cols64 + wslab - 1) / wslab;
    wslab = ((cols64 + rounds - 1) / rounds + FW_COLS - 1) / FW_COLS * FW_COLS;
  }
  if (plan) {
    plan->mask = mask; plan->A = A; plan->entries_off = entries_off; plan->colsum_off = off;
    plan->t_off = off + align_up((size_t)A * (size_t)wslab * sizeof(float));
    plan->wslab = wslab;
  }
  return true;
}
// Scratch with which the fast path takes all `cols` columns in one round (0 outside the fast path).
size_t sors_fast_full_scratch(int64_t k, int64_t cols, int64_t tokens) {
  const int64_t L = (int64_t)sors_mask_for(tokens) + 1;
  if (L < FW_ROWS || L > (int64_t)FW_ROWS * FW_ROWS) return 0;
  const int64_t cols64 = (cols + FW_COLS - 1) / FW_COLS * FW_COLS;
  const size_t off = align_up(129 * sizeof(int)) + align_up((size_t)k * sizeof(int2));
  return off + align_up((size_t)(L / FW_ROWS) * (size_t)cols64 * sizeof(float)) + (size_t)L * (size_t)cols64 * 2 + 4 * kAlign;
}
bool sors_fast_supported(int64_t k, int64_t cols, int64_t tokens, size_t scratch_bytes) {
  return sors_fast_plan(k, cols, tokens, scratch_bytes, nullptr);
}

rmm_status launch_sors_fast(const void* b, void* out, void* ones_out, int64_t k, int64_t cols, int64_t tokens, float c,
                            const PhiloxKey& pk, void* scratch, size_t scratch_bytes, int* status, cudaStream_t stream,
                            bool clear_status) {
  SorsFastPlan plan;
  if (!sors_fast_plan(k, cols, tokens, scratch_bytes, &plan)) return RMM_ERR_UNSUPPORTED;
  const uint32_t mask = plan.mask;
  const int A = plan.A;
  const int64_t wslab = plan.wslab;
  uint8_t* base = reinterpret_cast<uint8_t*>(scratch);
  SorsGroups g;
  g.offsets = reinterpret_cast<int*>(base);
  g.entries = reinterpret_cast<int2*>(base + plan.entries_off);
  float* colsum = reinterpret_cast<float*>(base + plan.colsum_off);
  __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(base + plan.t_off);
  const __nv_bfloat16* B = reinterpret_cast<const __nv_bfloat16*>(b);
  __nv_bfloat16* O = reinterpret_cast<__nv_bfloat16*>(out);
  __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(ones_out);
  for (int64_t c0 = 0; c0 < cols; c0 += wslab) {
    const int width = (int)(cols - c0 < wslab ? cols - c0 : wslab);
    const unsigned slabs = (unsigned)((width + FW_COLS - 1) / FW_COLS);
    SorsGroups build = g;                                   // the first launch also builds the column groups
    if (c0 != 0) { build.offsets = nullptr; build.entries = nullptr; }
    fwht_stage1_kernel<<<dim3(slabs, (unsigned)A), FW_THREADS, 0, stream>>>(B + c0, cols, tokens, width, pk, T, wslab,
                                                                           ones ? colsum : nullptr, build, k, mask, status,
                                                                           (clear_status && c0 == 0) ? 1 : 0);
    if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
    note_launches(2);
    fwht_stage2_kernel<<<dim3(slabs, FW_ROWS), FW_THREADS, 0, stream>>>(T, wslab, A, width, g, c, O + c0, cols,
                                                                       ones ? colsum : nullptr, ones ? ones + c0 : nullptr);
    if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
  }
  return RMM_OK;
}

// Tag of a launch: the completion flags of its partial tiles carry it, so that values left in a workspace by
// earlier launches (or never initialised) read as "not yet".  64 bits from a counter that starts at a
// time-dependent value: a stale word equals the tag of a later launch with probability 2^-64 per flag.
unsigned long long next_launch_tag() {
  static std::atomic<unsigned long long> counter{
      (unsigned long long)std::chrono::steady_clock::now().time_since_epoch().count() * 0x9E3779B97F4A7C15ull};
  return counter.fetch_add(0x9E3779B97F4A7C15ull) + 1;
}

rmm_status launch_sketch(const void* b, void* out, void* ones_out, int64_t k, int64_t cols, int64_t tokens, float c,
                         int dist, const PhiloxKey& pk, float* partial, int* status, cudaStream_t stream,
                         bool clear_status = false, int clusters_limit = 0) {
  CUtensorMap tmB;
  const bool slab_map = cols % 64 == 0;
  if (!(slab_map ? make_tmap_slabs(&tmB, b, tokens, cols, tc::SK_BK, tc::SK_BNH / 64)
                 : make_tmap(&tmB, b, tokens, cols, tc::SK_BK)))
    return RMM_ERR_CUDA;
  tc::SketchParams p;
  p.slab_map = slab_map ? 1 : 0;
  p.rows = k + (ones_out ? 1 : 0);
  p.b_proj = k;
  p.cols = cols;
  p.tokens = tokens;
  p.partial = partial;
  p.dist = dist;
  p.sors_mask = sors_mask_for(tokens);
  p.ones_row = ones_out ? 1 : 0;
  p.status = status;
  p.clear_status = clear_status ? 1 : 0;
  const int C = tc::sketch_cluster_size(cols);
  int max_clusters = device_state().sketch_clusters[C];
  if (clusters_limit > 0 && clusters_limit < max_clusters) max_clusters = clusters_limit;
  p.sched = tc::make_sketch_schedule(p.rows, cols, tokens, C, max_clusters);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)C; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3((unsigned)(C * p.sched.num_ctas));      // the schedule's workers are clusters
  cfg.blockDim = dim3(tc::SK_THREADS);
  cfg.dynamicSmemBytes = tc::SK_SMEM_BYTES;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  cudaError_t le = cudaLaunchKernelEx(&cfg, sketch_kernel_fn(C, dist), tmB, p, pk);
  if (le != cudaSuccess) return RMM_ERR_CUDA;
  note_launches(2);
  // The partial tiles are added up by a second, short kernel: measured against a reduction at the end of the sketch
  // kernel itself (completion flags per partial tile, every warp of the grid taking rows), the separate launch is
  // 5 us per pass faster on the 4096-token shapes (its blocks start as soon as SMs are free, and the sketch CTAs do
  // not sit on their SMs while the slowest cluster drains).
  dim3 rgrid((unsigned)(p.sched.tiles() * C), tc::SK_BN / tc::SKR_CHUNK);
  tc::sketch_reduce_kernel<<<rgrid, tc::SK_BM, 0, stream>>>(p, c, reinterpret_cast<__nv_bfloat16*>(out),
                                                      reinterpret_cast<__nv_bfloat16*>(ones_out));
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

// ------------------------------------------------------------------ one pass as one launch (tc_pass.cuh)
// Static schedule of a pass on `max_pairs` CTA pairs.  The sketch tiles are cut along the tokens into nb
// blocks each (unit = block * tiles + tile, dealt round-robin: the pairs that run at the same time walk the
// same token range); the dense tiles then go, one by one, to the pair that is least loaded.  nb is the
// candidate with the smallest estimated makespan, in units of tensor-pipe cycles of a pair.
tc::PassSchedule make_pass_schedule(bool with_gemm, int64_t gM, int64_t gN, int64_t gK, bool with_sketch, int64_t rows,
                                    int64_t cols, int64_t tokens, int max_pairs) {
  tc::PassSchedule s = {};
  if (max_pairs > tc::PS_MAX_PAIRS) max_pairs = tc::PS_MAX_PAIRS;
  if (max_pairs < 1) max_pairs = 1;
  s.tiles_n = 1; s.num_kb = 0; s.gemm_tiles = 0;
  if (with_gemm) {
    s.tiles_n = (int)((gN + tc::BN - 1) / tc::BN);
    s.gemm_tiles = (int)((gM + tc::PAIR_M - 1) / tc::PAIR_M) * s.tiles_n;
    s.num_kb = (int)((gK + tc::BK - 1) / tc::BK);
  }
  s.tiles_m = 0; s.groups = 1; s.nat = 1; s.ksteps = 0; s.nb = 1; s.blen = 1;
  SketchGeometry g = {};
  if (with_sketch) {
    g = sketch_geometry(rows, cols, tokens);
    s.tiles_m = g.tiles_m; s.groups = g.groups; s.nat = g.nat; s.ksteps = g.ksteps;
  }
  const int G = s.gemm_tiles, T = with_sketch ? g.tiles() : 0;
  // estimated costs (cycles of the pair's tensor pipe): a dense tile, a 64-token sketch step, the drain of a unit
  const long long cg = (long long)s.num_kb * 512 + 1500;
  const long long cs = (long long)s.nat * 256 + 64;
  const long long co = 3500;
  constexpr int kGreedyMax = 16384;
  int best_nb = 1, best_pairs = 1;
  long long best_cost = -1;
  std::vector<long long> load;
  const int nb_cap = with_sketch ? g.nb_cap() : 1;
  for (int nb_try = 1; nb_try <= nb_cap; ++nb_try) {
    int blen = 1, nb = 1;
    if (with_sketch) {
      blen = (s.ksteps + nb_try - 1) / nb_try;
      nb = (s.ksteps + blen - 1) / blen;
      if (nb != nb_try) continue;               // the same cut as a smaller candidate
      if (blen < 4 && nb > 1) break;            // no slivers
    }
    const long long units = (long long)T * nb;
    const int pairs = (int)(units + G < max_pairs ? (units + G > 0 ? units + G : 1) : max_pairs);
    load.assign((size_t)pairs, 0);
    for (long long u = 0; u < units; ++u) {
      const int b = (int)(u / T);
      const int len = (b + 1) * blen <= s.ksteps ? blen : s.ksteps - b * blen;
      load[(size_t)(u % pairs)] += (long long)len * cs + co;
    }
    for (int t = 0; t < G && G <= kGreedyMax; ++t) {
      size_t m = 0;
      for (size_t q = 1; q < load.size(); ++q)
        if (load[q] < load[m]) m = q;
      load[m] += cg;
    }
    if (G > kGreedyMax)                         // very many dense tiles: the sketch units no longer matter for the balance
      for (long long& v : load) v += (long long)((G + pairs - 1) / pairs) * cg;
    long long cost = 0;
    for (long long v : load) cost = v > cost ? v : cost;
    cost += (long long)nb * 40;                 // more blocks: more partial tiles to add up
    if (best_cost < 0 || cost < best_cost) {
      best_cost = cost; best_nb = nb; best_pairs = pairs;
    }
    if (!with_sketch) break;
  }
  s.nb = best_nb;
  s.blen = with_sketch ? (s.ksteps + best_nb - 1) / best_nb : 1;
  s.num_pairs = best_pairs;
  // dense tiles: counts by the same greedy rule, then consecutive ranges
  std::vector<int> count((size_t)best_pairs, 0);
  load.assign((size_t)best_pairs, 0);
  const long long units = (long long)T * s.nb;
  for (long long u = 0; u < units; ++u) {
    const int b = (int)(u / T);
    const int len = (b + 1) * s.blen <= s.ksteps ? s.blen : s.ksteps - b * s.blen;
    load[(size_t)(u % best_pairs)] += (long long)len * cs + co;
  }
  for (int t = 0; t < G && G <= kGreedyMax; ++t) {
    size_t m = 0;
    for (size_t q = 1; q < load.size(); ++q)
      if (load[q] < load[m]) m = q;
    load[m] += cg;
    ++count[m];
  }
  if (G > kGreedyMax)
    for (int q = 0; q < best_pairs; ++q) count[(size_t)q] = G / best_pairs + (q < G % best_pairs ? 1 : 0);
  int acc = 0;
  for (int q = 0; q <= tc::PS_MAX_PAIRS; ++q) {
    s.gemm_begin[q] = acc;
    if (q < best_pairs) acc += count[(size_t)q];
  }
  s.gemm_begin[tc::PS_MAX_PAIRS + 1] = acc;
  return s;
}

// One pass: optional dense part C = A B^T (+ bias), A [M][K]; B [N][K] (B_K) or [K][N] (B_MN); optional sketch
// part out[j][d] = c sum_n P[n][j] data[n][d] (+ ones_out[d] = sum_n data[n][d]).
struct PassArgs {
  // dense
  const void *a = nullptr, *b = nullptr, *bias = nullptr;
  void* c = nullptr;
  int64_t M = 0, N = 0, K = 0;
  int bmode = tc::B_K;
  // sketch
  const void* data = nullptr;
  void *out = nullptr, *ones_out = nullptr;
  int64_t k = 0, cols = 0, tokens = 0;
  float scale = 1.0f;
  int dist = 0;
};

rmm_status launch_pass(const PassArgs& a, const PhiloxKey& pk, float* partial, unsigned long long* tickets, int* status,
                       cudaStream_t stream, bool clear_status) {
  const bool with_gemm = a.c != nullptr, with_sketch = a.out != nullptr;
  if (!with_gemm && !with_sketch) return RMM_OK;
  const int64_t rows = a.k + (a.ones_out ? 1 : 0);
  tc::PassParams p = {};
  p.sched = make_pass_schedule(with_gemm, a.M, a.N, a.K, with_sketch, rows, a.cols, a.tokens, device_state().pass_pairs);
  CUtensorMap tmA, tmB, tmC, tmD;
  memset(&tmA, 0, sizeof(tmA)); memset(&tmB, 0, sizeof(tmB)); memset(&tmC, 0, sizeof(tmC)); memset(&tmD, 0, sizeof(tmD));
  bool ok = true;
  if (with_gemm) {
    ok &= make_tmap(&tmC, a.c, a.M, a.N, 32);
    ok &= make_tmap(&tmA, a.a, a.M, a.K, tc::BM);
    if (a.bmode == tc::B_K) ok &= make_tmap(&tmB, a.b, a.N, a.K, tc::BN_HALF);
    else ok &= make_tmap(&tmB, a.b, a.K, a.N, tc::BK);
  }
  const bool slab_map = a.cols % 64 == 0;
  if (with_sketch)
    ok &= slab_map ? make_tmap_slabs(&tmD, a.data, a.tokens, a.cols, 32, 2 * p.sched.nat)
                   : make_tmap(&tmD, a.data, a.tokens, a.cols, 32);
  if (!ok) return RMM_ERR_CUDA;
  p.M = a.M; p.N = a.N; p.K = a.K; p.bias = a.bias;
  p.rows = rows; p.b_proj = a.k; p.cols = a.cols; p.tokens = a.tokens;
  p.scale = a.scale; p.ones_row = a.ones_out ? 1 : 0; p.slab_map = slab_map ? 1 : 0;
  p.sors_mask = sors_mask_for(a.tokens > 0 ? a.tokens : 1);
  p.partial = partial; p.tickets = tickets; p.tag = next_launch_tag();
  p.sk_out = reinterpret_cast<__nv_bfloat16*>(a.out);
  p.ones_out = reinterpret_cast<__nv_bfloat16*>(a.ones_out);
  p.status = status; p.clear_status = clear_status ? 1 : 0;
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 2; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.gridDim = dim3(2 * (unsigned)p.sched.num_pairs);
  cfg.blockDim = dim3(tc::PS_THREADS);
  cfg.dynamicSmemBytes = tc::PS_SMEM_BYTES;
  cfg.stream = stream;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (cudaLaunchKernelEx(&cfg, pass_kernel_fn(a.bmode, a.dist), tmA, tmB, tmC, tmD, p, pk) != cudaSuccess)
    return RMM_ERR_CUDA;
  note_launches(1);
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

template <typename T, bool GEN_A>
rmm_status launch_simt(const SimtGemmArgs& g, const PhiloxKey& pk, cudaStream_t stream) {
  dim3 grid((unsigned)((g.N + SIMT_BN - 1) / SIMT_BN), (unsigned)((g.M + SIMT_BM - 1) / SIMT_BM));
  simt_gemm_kernel<T, GEN_A><<<grid, SIMT_THREADS, 0, stream>>>(g, pk);
  note_launches(1);
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

rmm_status simt_gemm_f32(bool gen_a, const void* A, int64_t a_sm, int64_t a_sk, const void* B, int64_t b_sn,
                         int64_t b_sk, void* C, const void* bias, int64_t M, int64_t N, int64_t K, float alpha,
                         int dist, const PhiloxKey& pk, cudaStream_t stream) {
  SimtGemmArgs g;
  g.A = A; g.a_sm = a_sm; g.a_sk = a_sk;
  g.B = B; g.b_sn = b_sn; g.b_sk = b_sk;
  g.C = C; g.ldc = N; g.bias = bias;
  g.M = M; g.N = N; g.K = K; g.alpha = alpha; g.dist = dist;
  g.sors_mask = sors_mask_for(K);      // generated A: K is the token count
  return gen_a ? launch_simt<float, true>(g, pk, stream) : launch_simt<float, false>(g, pk, stream);
}

template <typename T>
rmm_status launch_db(const void* dY, int64_t N, int64_t D_out, const Workspace& w, char* ws, void* db,
                     cudaStream_t stream) {
  float* partial = reinterpret_cast<float*>(ws + w.scratch_off);
  dim3 grid((unsigned)((D_out + 255) / 256), (unsigned)w.db_slices);
  note_launches(2);
  db_partial_kernel<T><<<grid, 256, 0, stream>>>(reinterpret_cast<const T*>(dY), N, D_out, w.db_rows_per_slice, partial);
  db_finish_kernel<T><<<(unsigned)((D_out + 255) / 256), 256, 0, stream>>>(partial, w.db_slices, D_out,
                                                                           reinterpret_cast<T*>(db));
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

// ------------------------------------------------------------------ a pass as two kernels that run at the same time
// The dense product and the sketch of a pass (Algorithm 1: Y and S^T X; dX and S^T dY) read the same token-sized
// operand and do not depend on each other.  Each is a persistent kernel whose static schedule is built for the
// number of CTA pairs / clusters it is given, so the two can share the GPU: the dense kernel gets `pairs` CTA
// pairs on the caller's stream, the sketch kernel the remaining clusters on a side stream that forks from and
// joins the caller's stream through events.  Short tails of one kernel are filled by the other, the fixed costs of
// the launches overlap, and the shared operand is in L2 for whichever reads it second.  If the device cannot hold
// both grids at once (other work running) the kernels simply run one after the other: neither waits for the other.
struct PassSplit {
  int gemm_pairs;       // 0: no split, both kernels get the whole device one after the other
  int sketch_clusters;
};

PassSplit plan_pass_split_uncached(int64_t gM, int64_t gN, int64_t gK, int64_t rows, int64_t cols, int64_t tokens,
                                   int64_t tail_m, int64_t tail_n, int64_t tail_k);

// The plan depends on the shape only (and on the device's residency counts, the same for every B200 of a process
// in practice): the last few shapes are remembered, so that a layer that is called again costs no search.
// tail_m x tail_n (contracted over tail_k; 0: none) is a dense product that follows the sketch on its side of the
// split (dW = G^T X_proj needs G = S^T dY, not dX).
PassSplit plan_pass_split(int64_t gM, int64_t gN, int64_t gK, int64_t rows, int64_t cols, int64_t tokens,
                          int64_t tail_m = 0, int64_t tail_n = 0, int64_t tail_k = 0) {
  struct Entry { int64_t key[9]; int dev; PassSplit plan; };
  static std::mutex mu;
  static std::vector<Entry> cache;
  int dev = 0;
  cudaGetDevice(&dev);
  const int64_t key[9] = {gM, gN, gK, rows, cols, tokens, tail_m, tail_n, tail_k};
  {
    std::lock_guard<std::mutex> lock(mu);
    for (const Entry& e : cache)
      if (e.dev == dev && memcmp(e.key, key, sizeof(key)) == 0) return e.plan;
  }
  const PassSplit plan = plan_pass_split_uncached(gM, gN, gK, rows, cols, tokens, tail_m, tail_n, tail_k);
  std::lock_guard<std::mutex> lock(mu);
  if (cache.size() >= 64) cache.erase(cache.begin());
  Entry e;
  memcpy(e.key, key, sizeof(key));
  e.dev = dev; e.plan = plan;
  cache.push_back(e);
  return plan;
}

PassSplit plan_pass_split_uncached(int64_t gM, int64_t gN, int64_t gK, int64_t rows, int64_t cols, int64_t tokens,
                                   int64_t tail_m, int64_t tail_n, int64_t tail_k) {
  PassSplit best = {0, 0};
  const DeviceState& ds = device_state();
  const int C = tc::sketch_cluster_size(cols);
  const int total = ds.gemm_pairs < ds.sketch_clusters[2] ? ds.gemm_pairs : ds.sketch_clusters[2];   // SM pairs
  if (total < 2 || !ds.lanes_ok) return best;
  const long long G = ((gN + tc::BN - 1) / tc::BN) * ((gM + tc::PAIR_M - 1) / tc::PAIR_M);
  const long long num_kb = (gK + tc::BK - 1) / tc::BK;
  // costs in SM cycles, from the launch lists under profiles/: a dense tile (about 500 cycles per K block of 64, plus
  // fill and epilogue), a 64-token sketch step (1415 cycles measured in steady state; 1300 here splits the 4096-token
  // shapes best and makes no difference on the 16384-token ones: 1300 / 1460 / 1600 / 1750 were timed back to back)
  const long long cg = num_kb * 500 + 800, cstep = 1300, fixed = 6000;
  auto gemm_cost = [&](int pairs) { return ((G + pairs - 1) / pairs) * cg + fixed; };
  const long long tail_tiles = tail_m > 0 ? ((tail_n + tc::BN - 1) / tc::BN) * ((tail_m + tc::PAIR_M - 1) / tc::PAIR_M) : 0;
  const long long tail_cg = ((tail_k + tc::BK - 1) / tc::BK) * 500 + 800;
  auto sketch_cost = [&](int clusters) {
    const tc::SketchSchedule sc = tc::make_sketch_schedule(rows, cols, tokens, C, C == 2 ? clusters : 2 * clusters);
    long long t = sc.est_steps * cstep + fixed + 9000;    // + the reduction kernel
    if (tail_tiles > 0) t += ((tail_tiles + clusters - 1) / clusters) * tail_cg + fixed;
    return t;
  };
  const long long serial = gemm_cost(total) + sketch_cost(total);
  long long best_cost = serial;
  for (int pg = 1; pg < total; ++pg) {
    const long long a = gemm_cost(pg), b = sketch_cost(total - pg);
    const long long c = (a > b ? a : b) + 1500;      // fork and join
    if (c < best_cost) { best_cost = c; best.gemm_pairs = pg; best.sketch_clusters = total - pg; }
  }
  return best;
}

// Runs `on_side` on a side stream that starts after everything queued on `stream` so far and that `stream` waits for
// afterwards; `on_main` is queued on `stream` in between.
template <class FSide, class FMain>
rmm_status fork_join(cudaStream_t stream, FSide&& on_side, FMain&& on_main) {
  DeviceState& ds = device_state();
  const unsigned lane = ds.next_lane.fetch_add(1) % DeviceState::kLanes;
  std::lock_guard<std::mutex> lock(ds.lane_mutex[lane]);
  cudaStream_t side = ds.lane_stream[lane];
  if (cudaEventRecord(ds.lane_fork[lane], stream) != cudaSuccess) return RMM_ERR_CUDA;
  if (cudaStreamWaitEvent(side, ds.lane_fork[lane], 0) != cudaSuccess) return RMM_ERR_CUDA;
  rmm_status st = on_side(side);
  // the join is queued even after an error, so that the side stream never runs ahead of the caller's stream
  const bool rec = cudaEventRecord(ds.lane_join[lane], side) == cudaSuccess;
  const rmm_status st2 = on_main(stream);
  const bool wait = rec && cudaStreamWaitEvent(stream, ds.lane_join[lane], 0) == cudaSuccess;
  if (st != RMM_OK) return st;
  if (st2 != RMM_OK) return st2;
  return wait ? RMM_OK : RMM_ERR_CUDA;
}

std::atomic<int> g_pass_mode{0};

// ------------------------------------------------------------------ allocation-free bias gradient
// Scratch for rmm_bias_grad_static: partial column sums, [slice][column].  The name below
// is only a host-side handle; kernels get the device address from cudaGetSymbolAddress.
static __device__ __align__(256) float g_bias_grad_scratch[RMM_BIAS_GRAD_STATIC_SLICES * RMM_BIAS_GRAD_STATIC_MAX_D_OUT];

float* g_bias_grad_scratch_addr[kMaxDevices] = {};
std::mutex g_bias_grad_mutex;

// Device address of the scratch array on the current device (looked up once per device).
rmm_status bias_grad_scratch(float** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return RMM_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_bias_grad_mutex);
  if (g_bias_grad_scratch_addr[dev] == nullptr) {
    float* ptr = nullptr;
    if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_bias_grad_scratch) != cudaSuccess || ptr == nullptr)
      return RMM_ERR_CUDA;
    g_bias_grad_scratch_addr[dev] = ptr;
  }
  *out = g_bias_grad_scratch_addr[dev];
  return RMM_OK;
}

// ------------------------------------------------------------------ argument checks
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

rmm_status check_common(int64_t N, int64_t D_in, int64_t D_out, int64_t k, rmm_dist dist, rmm_dtype dt) {
  if (N < 1 || D_in < 1 || D_out < 1 || k < 1 || k > N) return RMM_ERR_INVALID_ARG;
  if (N > (int64_t)1 << 31 || D_in > (int64_t)1 << 30 || D_out > (int64_t)1 << 30) return RMM_ERR_INVALID_ARG;
  if (dist != RMM_DIST_GAUSSIAN && dist != RMM_DIST_RADEMACHER && dist != RMM_DIST_IDENTITY &&
      dist != RMM_DIST_SORS_HADAMARD && dist != RMM_DIST_SORS_DCT)
    return RMM_ERR_INVALID_ARG;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_IDENTITY && k != N) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_SORS_DCT && N > ((int64_t)1 << 30)) return RMM_ERR_UNSUPPORTED;   // its index arithmetic is 32-bit
  if (dt == RMM_DTYPE_BF16 && (D_in % 8 != 0 || D_out % 8 != 0)) return RMM_ERR_UNSUPPORTED;
  return RMM_OK;
}

rmm_status check_workspace(const void* ws, size_t ws_bytes, const Workspace& w) {
  if (ws == nullptr || (reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return RMM_ERR_WORKSPACE;
  if (ws_bytes < w.total) return RMM_ERR_WORKSPACE;
  return RMM_OK;
}

}  // namespace

extern "C" {

size_t rmm_workspace_bytes(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt) {
  if (N < 1 || D_in < 1 || D_out < 1 || B_proj < 1 || B_proj > N) return 0;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return 0;
  return workspace_layout(N, D_in, D_out, B_proj, dt).total;
}

size_t rmm_workspace_bytes_for(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt, rmm_dist dist) {
  const size_t base = rmm_workspace_bytes(N, D_in, D_out, B_proj, dt);
  if (base == 0 || dist != RMM_DIST_SORS_HADAMARD || dt != RMM_DTYPE_BF16) return base;
  const Workspace w = workspace_layout(N, D_in, D_out, B_proj, dt);
  const size_t f = sors_fast_full_scratch(B_proj, D_in, N), b = sors_fast_full_scratch(B_proj, D_out, N);
  const size_t want = w.scratch_off + (f > b ? f : b);
  return want > base ? want : base;
}

rmm_status rmm_forward(const void* X, const void* W, const void* b, int64_t N, int64_t D_in, int64_t D_out,
                       uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt, void* Y, void* X_proj,
                       void* workspace, size_t workspace_bytes, void* cuda_stream) {
  rmm_status st = check_common(N, D_in, D_out, B_proj, dist, dt);
  if (st != RMM_OK) return st;
  if (!X || !W || !X_proj) return RMM_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(W) || !aligned16(b) || !aligned16(Y) || !aligned16(X_proj)) return RMM_ERR_INVALID_ARG;
  const Workspace w = workspace_layout(N, D_in, D_out, B_proj, dt);
  if ((st = check_workspace(workspace, workspace_bytes, w)) != RMM_OK) return st;
  if (!device_state().ok) return RMM_ERR_CUDA;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* ws = reinterpret_cast<char*>(workspace);
  int* status = reinterpret_cast<int*>(ws + w.status_off);
  const PhiloxKey pk = make_philox_key(seed);
  const float c = sketch_scale(B_proj, dist);

  if (dt == RMM_DTYPE_BF16) {
    float* scratch = reinterpret_cast<float*>(ws + w.scratch_off);
    unsigned long long* tickets = reinterpret_cast<unsigned long long*>(ws + w.ticket_off);
    const size_t scratch_bytes = workspace_bytes - w.scratch_off;   // all the caller gave: the fast Hadamard path uses the extra
    // the first kernel of the call resets the status word (no separate memset on the stream)
    if (dist == RMM_DIST_SORS_HADAMARD && sors_fast_supported(B_proj, D_in, N, scratch_bytes)) {
      // the subsampled-Hadamard sketch by its fast transform; the dense product on its own
      if (Y) {
        ScopedTiming t(RMM_STEP_Y, stream);
        st = launch_tc<tc::A_K, tc::B_K>(X, W, Y, b, N, D_out, D_in, 1.0f, status, stream, nullptr, true);
        if (st != RMM_OK) return st;
      }
      ScopedTiming t(RMM_STEP_SKETCH, stream);
      return launch_sors_fast(X, X_proj, nullptr, B_proj, D_in, N, c, pk, scratch, scratch_bytes, status, stream, Y == nullptr);
    }
    if (g_pass_mode.load(std::memory_order_relaxed) == 1) {
      // Y = X W^T + 1 b^T and X_proj = S^T X in one launch
      ScopedTiming t(RMM_STEP_FWD, stream);
      PassArgs a;
      if (Y) { a.a = X; a.b = W; a.bias = b; a.c = Y; a.M = N; a.N = D_out; a.K = D_in; a.bmode = tc::B_K; }
      a.data = X; a.out = X_proj; a.k = B_proj; a.cols = D_in; a.tokens = N; a.scale = c; a.dist = (int)dist;
      return launch_pass(a, pk, scratch, tickets, status, stream, true);
    }
    if (!Y) {
      ScopedTiming t(RMM_STEP_SKETCH, stream);
      return launch_sketch(X, X_proj, nullptr, B_proj, D_in, N, c, dist, pk, scratch, status, stream, true);
    }
    // Y = X W^T + 1 b^T and X_proj = S^T X: two kernels that share the device and the X stream
    const PassSplit split = g_pass_mode.load(std::memory_order_relaxed) == 2 ? PassSplit{0, 0}
                                                                              : plan_pass_split(N, D_out, D_in, B_proj, D_in, N);
    ScopedTiming t(RMM_STEP_FWD, stream);
    auto gemm = [&](cudaStream_t s_, int pairs) {
      return launch_tc<tc::A_K, tc::B_K>(X, W, Y, b, N, D_out, D_in, 1.0f, status, s_, nullptr, true, pairs);
    };
    auto sketch = [&](cudaStream_t s_, int clusters) {
      return launch_sketch(X, X_proj, nullptr, B_proj, D_in, N, c, dist, pk, scratch, status, s_, false, clusters);
    };
    if (split.gemm_pairs == 0) {
      st = gemm(stream, 0);
      return st != RMM_OK ? st : sketch(stream, 0);
    }
    return fork_join(stream, [&](cudaStream_t side) { return sketch(side, split.sketch_clusters); },
                     [&](cudaStream_t main_) { return gemm(main_, split.gemm_pairs); });
  }
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return RMM_ERR_CUDA;
  if (Y) {
    ScopedTiming t(RMM_STEP_Y, stream);
    st = simt_gemm_f32(false, X, D_in, 1, W, D_in, 1, Y, b, N, D_out, D_in, 1.0f, 0, pk, stream);
    if (st != RMM_OK) return st;
  }
  ScopedTiming t(RMM_STEP_SKETCH, stream);
  return simt_gemm_f32(true, nullptr, 0, 0, X, 1, D_in, X_proj, nullptr, B_proj, D_in, N, c, dist, pk, stream);
}

rmm_status rmm_backward(const void* dY, const void* W, const void* X_proj, int64_t N, int64_t D_in, int64_t D_out,
                        uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt, void* dX, void* dW, void* db,
                        void* workspace, size_t workspace_bytes, void* cuda_stream) {
  rmm_status st = check_common(N, D_in, D_out, B_proj, dist, dt);
  if (st != RMM_OK) return st;
  if (!dY || !W || !X_proj || !dW) return RMM_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(W) || !aligned16(X_proj) || !aligned16(dX) || !aligned16(dW) || !aligned16(db))
    return RMM_ERR_INVALID_ARG;
  const Workspace w = workspace_layout(N, D_in, D_out, B_proj, dt);
  if ((st = check_workspace(workspace, workspace_bytes, w)) != RMM_OK) return st;
  if (!device_state().ok) return RMM_ERR_CUDA;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  char* ws = reinterpret_cast<char*>(workspace);
  int* status = reinterpret_cast<int*>(ws + w.status_off);
  void* G = ws + w.g_off;
  const PhiloxKey pk = make_philox_key(seed);
  const float c = sketch_scale(B_proj, dist);

  if (dt == RMM_DTYPE_BF16) {
    float* scratch = reinterpret_cast<float*>(ws + w.scratch_off);
    unsigned long long* tickets = reinterpret_cast<unsigned long long*>(ws + w.ticket_off);
    const size_t scratch_bytes = workspace_bytes - w.scratch_off;   // all the caller gave: the fast Hadamard path uses the extra
    // the first kernel of the call resets the status word (no separate memset on the stream)
    if (dist == RMM_DIST_SORS_HADAMARD && sors_fast_supported(B_proj, D_out, N, scratch_bytes)) {
      if (dX) {
        ScopedTiming t(RMM_STEP_DX, stream);
        st = launch_tc<tc::A_K, tc::B_MN>(dY, W, dX, nullptr, N, D_in, D_out, 1.0f, status, stream, nullptr, true);
        if (st != RMM_OK) return st;
      }
      ScopedTiming t(RMM_STEP_SDY, stream);
      st = launch_sors_fast(dY, G, db, B_proj, D_out, N, c, pk, scratch, scratch_bytes, status, stream, dX == nullptr);
      if (st != RMM_OK) return st;
    } else if (g_pass_mode.load(std::memory_order_relaxed) == 1) {
      // dX = dY W, G = S^T dY and db = dY^T 1 (the row of ones of S^T) in one launch
      ScopedTiming t(RMM_STEP_BWD, stream);
      PassArgs a;
      if (dX) { a.a = dY; a.b = W; a.c = dX; a.M = N; a.N = D_in; a.K = D_out; a.bmode = tc::B_MN; }
      a.data = dY; a.out = G; a.ones_out = db; a.k = B_proj; a.cols = D_out; a.tokens = N; a.scale = c; a.dist = (int)dist;
      st = launch_pass(a, pk, scratch, tickets, status, stream, true);
      if (st != RMM_OK) return st;
    } else if (!dX) {
      ScopedTiming t(RMM_STEP_SDY, stream);
      st = launch_sketch(dY, G, db, B_proj, D_out, N, c, dist, pk, scratch, status, stream, true);
      if (st != RMM_OK) return st;
    } else {
      // dX = dY W and G = S^T dY (with db = dY^T 1 as the row of ones of S^T): two kernels that share the device and
      // the dY stream
      const PassSplit split = g_pass_mode.load(std::memory_order_relaxed) == 2
                                  ? PassSplit{0, 0}
                                  : plan_pass_split(N, D_in, D_out, B_proj + 1, D_out, N, D_out, D_in, B_proj);
      auto gemm = [&](cudaStream_t s_, int pairs) {
        return launch_tc<tc::A_K, tc::B_MN>(dY, W, dX, nullptr, N, D_in, D_out, 1.0f, status, s_, nullptr, true, pairs);
      };
      auto sketch = [&](cudaStream_t s_, int clusters) {
        return launch_sketch(dY, G, db, B_proj, D_out, N, c, dist, pk, scratch, status, s_, false, clusters);
      };
      if (split.gemm_pairs == 0) {
        ScopedTiming t(RMM_STEP_BWD, stream);
        st = gemm(stream, 0);
        if (st == RMM_OK) st = sketch(stream, 0);
      } else {
        // dW = G^T X_proj follows the sketch on the side stream, on the SMs that the sketch kernel leaves: it needs
        // G, not dX, so it runs beside the rest of the dX product
        ScopedTiming t(RMM_STEP_BWD, stream);
        return fork_join(stream,
                         [&](cudaStream_t side) {
                           rmm_status s1 = sketch(side, split.sketch_clusters);
                           if (s1 != RMM_OK) return s1;
                           return launch_tc<tc::A_MN, tc::B_MN>(G, X_proj, dW, nullptr, D_out, D_in, B_proj, 1.0f, status, side,
                                                                nullptr, false, split.sketch_clusters);
                         },
                         [&](cudaStream_t main_) { return gemm(main_, split.gemm_pairs); });
      }
      if (st != RMM_OK) return st;
    }
    ScopedTiming t(RMM_STEP_DW, stream);
    return launch_tc<tc::A_MN, tc::B_MN>(G, X_proj, dW, nullptr, D_out, D_in, B_proj, 1.0f, status, stream);
  }
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return RMM_ERR_CUDA;
  if (dX) {
    ScopedTiming t(RMM_STEP_DX, stream);
    st = simt_gemm_f32(false, dY, D_out, 1, W, 1, D_in, dX, nullptr, N, D_in, D_out, 1.0f, 0, pk, stream);
    if (st != RMM_OK) return st;
  }
  {
    ScopedTiming t(RMM_STEP_SDY, stream);
    st = simt_gemm_f32(true, nullptr, 0, 0, dY, 1, D_out, G, nullptr, B_proj, D_out, N, c, dist, pk, stream);
    if (st != RMM_OK) return st;
  }
  {
    ScopedTiming t(RMM_STEP_DW, stream);
    st = simt_gemm_f32(false, G, 1, D_out, X_proj, 1, D_in, dW, nullptr, D_out, D_in, B_proj, 1.0f, 0, pk, stream);
    if (st != RMM_OK) return st;
  }
  if (db) {
    ScopedTiming t(RMM_STEP_DB, stream);
    return launch_db<float>(dY, N, D_out, w, ws, db, stream);
  }
  return RMM_OK;
}

rmm_status rmm_debug_generate_s(uint64_t seed, int64_t N, int64_t B_proj, rmm_dist dist, rmm_dtype dt, void* S_out,
                                void* cuda_stream) {
  if (N < 1 || B_proj < 1 || B_proj > N || !S_out) return RMM_ERR_INVALID_ARG;
  if (dist != RMM_DIST_GAUSSIAN && dist != RMM_DIST_RADEMACHER && dist != RMM_DIST_IDENTITY &&
      dist != RMM_DIST_SORS_HADAMARD && dist != RMM_DIST_SORS_DCT)
    return RMM_ERR_INVALID_ARG;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_IDENTITY && B_proj != N) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_SORS_DCT && N > ((int64_t)1 << 30)) return RMM_ERR_UNSUPPORTED;
  if (!device_state().ok) return RMM_ERR_CUDA;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const PhiloxKey pk = make_philox_key(seed);
  const int64_t total = N * B_proj;
  const unsigned blocks = (unsigned)((total + 255) / 256);
  if (dt == RMM_DTYPE_BF16)
    dump_sketch_kernel<__nv_bfloat16><<<blocks, 256, 0, stream>>>(pk, (int)dist, N, B_proj,
                                                                  reinterpret_cast<__nv_bfloat16*>(S_out));
  else
    dump_sketch_kernel<float><<<blocks, 256, 0, stream>>>(pk, (int)dist, N, B_proj, reinterpret_cast<float*>(S_out));
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

rmm_status rmm_debug_gauss_words(const uint32_t* words, int64_t n, float* out, void* cuda_stream) {
  if (!words || !out || n < 1) return RMM_ERR_INVALID_ARG;
  if (!device_state().ok) return RMM_ERR_CUDA;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  gauss_words_kernel<<<(unsigned)((n + 255) / 256), 256, 0, stream>>>(words, n, out);
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

int64_t rmm_debug_sketch_schedule(int64_t rows, int64_t cols, int64_t tokens, int max_ctas, int mode, int64_t* records,
                                  int64_t cap, int64_t* info) {
  if (rows < 1 || cols < 1 || tokens < 1 || max_ctas < 1) return -1;
  const int C = tc::sketch_cluster_size(cols);
  const tc::SketchSchedule sc = tc::make_sketch_schedule(rows, cols, tokens, C, max_ctas / C > 0 ? max_ctas / C : 1);
  if (info) {
    info[0] = sc.tiles(); info[1] = sc.ksteps; info[2] = sc.num_ctas; info[3] = sc.num_slots(); info[4] = C;
    info[5] = sc.rounds; info[6] = sc.full_blocks; info[7] = sc.w_last;
  }
  int64_t n = 0;
  auto put = [&](int64_t a, int64_t b, int64_t c, int64_t d, int64_t e) {
    if (records && n < cap) {
      int64_t* r = records + 5 * n;
      r[0] = a; r[1] = b; r[2] = c; r[3] = d; r[4] = e;
    }
    ++n;
  };
  if (mode == 0) {
    for (int cta = 0; cta < sc.num_ctas; ++cta) {
      int it = 0;
      long long cursor = 0;
      tc::SketchSegment sg;
      while (tc::sketch_next_segment(sc, cta, it, cursor, sg)) put(cta, sg.tile, sg.ks0, sg.ks1, sg.slot);
    }
  } else {
    for (int tile = 0; tile < sc.tiles(); ++tile)
      tc::sketch_for_each_slot_of_tile(sc, tile, [&](long long slot) { put(tile, slot, 0, 0, 0); });
  }
  return n;
}

int rmm_debug_hadamard_plan(int64_t rows, int64_t cols, int64_t tokens, size_t scratch_bytes, int64_t* info) {
  if (rows < 1 || cols < 1 || tokens < 1 || info == nullptr) return -1;
  SorsFastPlan plan;
  if (!sors_fast_plan(rows, cols, tokens, scratch_bytes, &plan)) return 0;
  info[0] = (int64_t)plan.mask + 1;
  info[1] = plan.A;
  info[2] = plan.wslab;
  info[3] = (cols + plan.wslab - 1) / plan.wslab;
  return 1;
}

int64_t rmm_debug_pass_schedule(int64_t gemm_m, int64_t gemm_n, int64_t gemm_k, int64_t rows, int64_t cols, int64_t tokens,
                                int max_pairs, int64_t* out, int64_t cap) {
  if (max_pairs < 1 || gemm_m < 0 || rows < 0) return -1;
  const bool with_gemm = gemm_m > 0, with_sketch = rows > 0;
  if (with_gemm && (gemm_n < 1 || gemm_k < 1)) return -1;
  if (with_sketch && (cols < 1 || tokens < 1)) return -1;
  const tc::PassSchedule s = make_pass_schedule(with_gemm, gemm_m, gemm_n, gemm_k, with_sketch, rows, cols, tokens, max_pairs);
  const int64_t head[10] = {s.num_pairs, s.gemm_tiles, s.tiles_n, s.num_kb, s.tiles_m, s.groups, s.nat, s.ksteps, s.nb, s.blen};
  const int64_t n = 10 + s.num_pairs + 1;
  for (int64_t i = 0; i < n && i < cap && out; ++i) out[i] = i < 10 ? head[i] : s.gemm_begin[i - 10];
  return n;
}

rmm_status rmm_last_device_status(const void* workspace) {
  if (!workspace) return RMM_ERR_INVALID_ARG;
  int v = 0;
  if (cudaMemcpy(&v, workspace, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return RMM_ERR_CUDA;
  return v == 0 ? RMM_OK : RMM_ERR_TIMEOUT;
}

const char* rmm_status_string(rmm_status s) {
  switch (s) {
    case RMM_OK: return "RMM_OK";
    case RMM_ERR_INVALID_ARG: return "RMM_ERR_INVALID_ARG";
    case RMM_ERR_UNSUPPORTED: return "RMM_ERR_UNSUPPORTED";
    case RMM_ERR_WORKSPACE: return "RMM_ERR_WORKSPACE";
    case RMM_ERR_CUDA: return "RMM_ERR_CUDA";
    case RMM_ERR_TIMEOUT: return "RMM_ERR_TIMEOUT";
  }
  return "RMM_ERR_UNKNOWN";
}

// ------------------------------------------------------------------ variance diagnostics
namespace {
struct ProbeWorkspace {
  size_t status_off, row_off, gemm_off, dw_off, total;
  int row_blocks;
};
ProbeWorkspace probe_layout(int64_t N, int64_t D_in, int64_t D_out) {
  ProbeWorkspace w;
  const int64_t want = (N + VAR_WARPS - 1) / VAR_WARPS;  // at least one row per warp
  const int64_t cap = (int64_t)(device_state().num_sms > 0 ? device_state().num_sms : 148) * VAR_BLOCKS_PER_SM;
  w.row_blocks = (int)(want < cap ? want : cap);
  if (w.row_blocks > 4096) w.row_blocks = 4096;
  w.status_off = 0;
  w.row_off = kAlign;
  w.gemm_off = w.row_off + align_up((size_t)4096 * 3 * sizeof(double));   // room for any grid of row_norms_kernel
  w.dw_off = w.gemm_off + align_up((size_t)tc::SK_MAX_CTAS * tc::NEPI * sizeof(double));
  w.total = w.dw_off + align_up((size_t)D_out * (size_t)D_in * 2);
  return w;
}
}  // namespace

size_t rmm_variance_probe_workspace_bytes(int64_t N, int64_t D_in, int64_t D_out) {
  if (N < 2 || D_in < 1 || D_out < 1) return 0;
  return probe_layout(N, D_in, D_out).total;
}

rmm_status rmm_variance_probe(const void* X, const void* dY, int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj,
                              rmm_dist dist, rmm_dtype dt, double* out, void* dW_exact, void* workspace,
                              size_t workspace_bytes, void* cuda_stream) {
  if (N < 2) return RMM_ERR_INVALID_ARG;                       // Eq. 9 divides by N - 1
  rmm_status st = check_common(N, D_in, D_out, B_proj, dist, dt);
  if (st != RMM_OK) return st;
  if (dt != RMM_DTYPE_BF16) return RMM_ERR_UNSUPPORTED;
  if (dist == RMM_DIST_SORS_HADAMARD || dist == RMM_DIST_SORS_DCT) return RMM_ERR_UNSUPPORTED;   // no closed form here
  if (!X || !dY || !out) return RMM_ERR_INVALID_ARG;
  if (!aligned16(X) || !aligned16(dY) || !aligned16(out) || !aligned16(dW_exact)) return RMM_ERR_INVALID_ARG;
  const ProbeWorkspace w = probe_layout(N, D_in, D_out);
  if (workspace == nullptr || (reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0 || workspace_bytes < w.total)
    return RMM_ERR_WORKSPACE;
  if (!device_state().ok) return RMM_ERR_CUDA;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  uint8_t* ws = reinterpret_cast<uint8_t*>(workspace);
  int* status = reinterpret_cast<int*>(ws + w.status_off);
  double* row_partial = reinterpret_cast<double*>(ws + w.row_off);
  double* gemm_partial = reinterpret_cast<double*>(ws + w.gemm_off);
  void* dw = dW_exact ? dW_exact : static_cast<void*>(ws + w.dw_off);
  if (cudaMemsetAsync(status, 0, sizeof(int), stream) != cudaSuccess) return RMM_ERR_CUDA;
  row_norms_kernel<<<w.row_blocks, VAR_THREADS, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(X),
                                                             reinterpret_cast<const __nv_bfloat16*>(dY), N, D_in, D_out,
                                                             row_partial);
  if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
  // exact gradient dW* = dY^T X (Eq. 3) on the tensor cores; its epilogue leaves |dW*|_F^2 in gemm_partial
  st = launch_tc<tc::A_MN, tc::B_MN>(dY, X, dw, nullptr, D_out, D_in, N, 1.0f, status, stream, gemm_partial);
  if (st != RMM_OK) return st;
  variance_finish_kernel<<<1, 32, 0, stream>>>(row_partial, w.row_blocks, gemm_partial, tc_grid_ctas(D_out, D_in) * tc::NEPI,
                                              N, B_proj, (int)dist, out);
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

rmm_status rmm_bias_grad_static(const void* dY, int64_t N, int64_t D_out, rmm_dtype dt, void* db, void* cuda_stream) {
  if (!dY || !db || N < 1 || D_out < 1) return RMM_ERR_INVALID_ARG;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return RMM_ERR_INVALID_ARG;
  if (!aligned16(dY) || !aligned16(db)) return RMM_ERR_INVALID_ARG;
  if (D_out > RMM_BIAS_GRAD_STATIC_MAX_D_OUT) return RMM_ERR_UNSUPPORTED;  // would not fit the fixed scratch
  if (!device_state().ok) return RMM_ERR_CUDA;
  float* scratch = nullptr;
  rmm_status st = bias_grad_scratch(&scratch);
  if (st != RMM_OK) return st;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const int slices = (int)(N < RMM_BIAS_GRAD_STATIC_SLICES ? N : RMM_BIAS_GRAD_STATIC_SLICES);
  const int rows_per_slice = (int)((N + slices - 1) / slices);
  const int used = (int)((N + rows_per_slice - 1) / rows_per_slice);
  dim3 grid((unsigned)((D_out + 255) / 256), (unsigned)used);
  const unsigned fin_blocks = (unsigned)((D_out + 255) / 256);
  if (dt == RMM_DTYPE_BF16) {
    db_partial_kernel<__nv_bfloat16><<<grid, 256, 0, stream>>>(reinterpret_cast<const __nv_bfloat16*>(dY), N, D_out,
                                                                rows_per_slice, scratch);
    db_finish_kernel<__nv_bfloat16><<<fin_blocks, 256, 0, stream>>>(scratch, used, D_out,
                                                                     reinterpret_cast<__nv_bfloat16*>(db));
  } else {
    db_partial_kernel<float><<<grid, 256, 0, stream>>>(reinterpret_cast<const float*>(dY), N, D_out, rows_per_slice,
                                                        scratch);
    db_finish_kernel<float><<<fin_blocks, 256, 0, stream>>>(scratch, used, D_out, reinterpret_cast<float*>(db));
  }
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

#ifdef RMM_PASS_TRACE
// Trace build only: copies the cycle counters of the last pass launch ([148][32] int64) to host memory.
int rmm_debug_pass_trace(long long* host_out) {
  return cudaMemcpyFromSymbol(host_out, tc::g_pass_trace, sizeof(long long) * 148 * tc::PS_TRACE_SLOTS) ==
                 cudaSuccess ? 0 : 1;
}
#endif

rmm_status rmm_set_pass_mode(int mode) {
  if (mode < 0 || mode > 2) return RMM_ERR_INVALID_ARG;
  g_pass_mode.store(mode, std::memory_order_relaxed);
  return RMM_OK;
}

int64_t rmm_layer_launch_count(void) { return (int64_t)g_layer_launches.load(std::memory_order_relaxed); }

rmm_status rmm_profile_enable(int capacity) {
  Profiler& p = profiler();
  for (ProfileRecord& r : p.pool) {
    cudaEventDestroy(r.t0);
    cudaEventDestroy(r.t1);
  }
  p.pool.clear();
  p.used = 0;
  if (capacity <= 0) return RMM_OK;
  if (!device_state().ok) return RMM_ERR_CUDA;
  p.pool.reserve((size_t)capacity);
  for (int i = 0; i < capacity; ++i) {
    ProfileRecord r;
    r.step = -1;
    if (cudaEventCreate(&r.t0) != cudaSuccess) return RMM_ERR_CUDA;
    if (cudaEventCreate(&r.t1) != cudaSuccess) { cudaEventDestroy(r.t0); return RMM_ERR_CUDA; }
    p.pool.push_back(r);
  }
  return RMM_OK;
}

int rmm_profile_read(int* step_ids, float* milliseconds, int max_records) {
  Profiler& p = profiler();
  int n = 0;
  for (size_t i = 0; i < p.used && n < max_records; ++i) {
    float ms = 0.f;
    if (cudaEventSynchronize(p.pool[i].t1) != cudaSuccess) break;
    if (cudaEventElapsedTime(&ms, p.pool[i].t0, p.pool[i].t1) != cudaSuccess) break;
    if (step_ids) step_ids[n] = p.pool[i].step;
    if (milliseconds) milliseconds[n] = ms;
    ++n;
  }
  p.used = 0;
  return n;
}

// ------------------------------------------------------------------ host-buffer wrappers
size_t rmm_host_staging_bytes(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt, int backward,
                              int outputs) {
  if (N < 1 || D_in < 1 || D_out < 1 || B_proj < 1) return 0;
  const size_t e = elem_bytes(dt);
  const size_t x = align_up((size_t)N * D_in * e), w = align_up((size_t)D_out * D_in * e), bb = align_up((size_t)D_out * e);
  const size_t y = align_up((size_t)N * D_out * e), xp = align_up((size_t)B_proj * D_in * e);
  if (!backward) return outputs ? y + xp : x + w + bb;
  return outputs ? x + w + bb : y + w + xp;
}

rmm_status rmm_forward_host(const void* X, const void* W, const void* b, int64_t N, int64_t D_in, int64_t D_out,
                            uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt, void* Y, void* X_proj,
                            void* dev_in, void* dev_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
  rmm_status st = check_common(N, D_in, D_out, B_proj, dist, dt);
  if (st != RMM_OK) return st;
  if (!X || !W || !X_proj || !dev_in || !dev_out) return RMM_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t e = elem_bytes(dt);
  const size_t xb = (size_t)N * D_in * e, wb = (size_t)D_out * D_in * e, bb = (size_t)D_out * e;
  const size_t yb = (size_t)N * D_out * e, xpb = (size_t)B_proj * D_in * e;
  char* di = reinterpret_cast<char*>(dev_in);
  char* dout = reinterpret_cast<char*>(dev_out);
  char *dX = di, *dWt = dX + align_up(xb), *dB = dWt + align_up(wb);
  char *dYv = dout, *dXp = dYv + align_up(yb);
  bool ok = cudaMemcpyAsync(dX, X, xb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(dWt, W, wb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (b) ok = ok && cudaMemcpyAsync(dB, b, bb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (!ok) return RMM_ERR_CUDA;
  st = rmm_forward(dX, dWt, b ? dB : nullptr, N, D_in, D_out, seed, B_proj, dist, dt, Y ? dYv : nullptr, dXp,
                   workspace, workspace_bytes, cuda_stream);
  if (st != RMM_OK) return st;
  if (Y) ok = ok && cudaMemcpyAsync(Y, dYv, yb, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(X_proj, dXp, xpb, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  return ok ? RMM_OK : RMM_ERR_CUDA;
}

rmm_status rmm_backward_host(const void* dY, const void* W, const void* X_proj, int64_t N, int64_t D_in,
                             int64_t D_out, uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt, void* dX,
                             void* dW, void* db, void* dev_in, void* dev_out, void* workspace,
                             size_t workspace_bytes, void* cuda_stream) {
  rmm_status st = check_common(N, D_in, D_out, B_proj, dist, dt);
  if (st != RMM_OK) return st;
  if (!dY || !W || !X_proj || !dW || !dev_in || !dev_out) return RMM_ERR_INVALID_ARG;
  cudaStream_t stream = reinterpret_cast<cudaStream_t>(cuda_stream);
  const size_t e = elem_bytes(dt);
  const size_t xb = (size_t)N * D_in * e, wb = (size_t)D_out * D_in * e, bb = (size_t)D_out * e;
  const size_t yb = (size_t)N * D_out * e, xpb = (size_t)B_proj * D_in * e;
  char* di = reinterpret_cast<char*>(dev_in);
  char* dout = reinterpret_cast<char*>(dev_out);
  char *ddY = di, *dWt = ddY + align_up(yb), *dXp = dWt + align_up(wb);
  char *ddX = dout, *ddW = ddX + align_up(xb), *ddb = ddW + align_up(wb);
  bool ok = cudaMemcpyAsync(ddY, dY, yb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(dWt, W, wb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(dXp, X_proj, xpb, cudaMemcpyHostToDevice, stream) == cudaSuccess;
  if (!ok) return RMM_ERR_CUDA;
  st = rmm_backward(ddY, dWt, dXp, N, D_in, D_out, seed, B_proj, dist, dt, dX ? ddX : nullptr, ddW, db ? ddb : nullptr,
                    workspace, workspace_bytes, cuda_stream);
  if (st != RMM_OK) return st;
  if (dX) ok = ok && cudaMemcpyAsync(dX, ddX, xb, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  ok = ok && cudaMemcpyAsync(dW, ddW, wb, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  if (db) ok = ok && cudaMemcpyAsync(db, ddb, bb, cudaMemcpyDeviceToHost, stream) == cudaSuccess;
  ok = ok && cudaStreamSynchronize(stream) == cudaSuccess;
  return ok ? RMM_OK : RMM_ERR_CUDA;
}

}  // extern "C"
