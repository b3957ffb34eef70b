// C ABI of the RMM linear layer (see include/rmm.h): argument checks, workspace
// layout, TMA tensor maps and kernel launches.  All arithmetic runs in the kernels.
#include "../../include/rmm.h"

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <mutex>
#include <vector>

#include "simt_kernels.cuh"
#include "sketch_rng.cuh"
#include "tc_gemm.cuh"
#include "fwht_kernels.cuh"
#include "tc_sketch.cuh"
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
  size_t status_off, g_off, scratch_off, total;
  int db_rows_per_slice, db_slices;
};

Workspace workspace_layout(int64_t N, int64_t D_in, int64_t D_out, int64_t k, rmm_dtype dt) {
  Workspace w;
  w.status_off = 0;
  w.g_off = kAlign;
  size_t off = w.g_off + align_up((size_t)k * (size_t)D_out * elem_bytes(dt));
  int64_t rps = 256;
  if ((N + rps - 1) / rps > 256) rps = (N + 255) / 256;
  w.db_rows_per_slice = (int)rps;
  w.db_slices = (int)((N + rps - 1) / rps);
  w.scratch_off = off;
  size_t scratch = (size_t)w.db_slices * (size_t)D_out * sizeof(float);
  if (dt == RMM_DTYPE_BF16) {
    // an upper bound over every grid the launch may use: one partial tile per (tile, CTA) pair at most
    const long long tf = ((k + tc::SK_BM - 1) / tc::SK_BM) * ((D_in + tc::SK_BN - 1) / tc::SK_BN);
    const long long tb = ((k + 1 + tc::SK_BM - 1) / tc::SK_BM) * ((D_out + tc::SK_BN - 1) / tc::SK_BN);
    scratch = (size_t)((tf > tb ? tf : tb) + tc::SK_MAX_CTAS) * tc::SK_TILE_ELEMS * sizeof(float);
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
};

template <typename K>
bool allow_big_smem(K kernel, int bytes) {
  return cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, bytes) == cudaSuccess;
}

// The sketch kernel for a cluster size (1 or 2) and a distribution (rmm_dist value).
typedef void (*SketchKernelFn)(const CUtensorMap, tc::SketchParams, PhiloxKey);
SketchKernelFn sketch_kernel_fn(int c, int dist) {
  static const SketchKernelFn table[2][4] = {
      {tc::sketch_kernel<1, 0>, tc::sketch_kernel<1, 1>, tc::sketch_kernel<1, 2>, tc::sketch_kernel<1, 3>},
      {tc::sketch_kernel<2, 0>, tc::sketch_kernel<2, 1>, tc::sketch_kernel<2, 2>, tc::sketch_kernel<2, 3>}};
  return table[c == 2 ? 1 : 0][dist & 3];
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
    for (int d = 0; d < 4; ++d) a &= allow_big_smem(sketch_kernel_fn(c, d), tc::SK_SMEM_BYTES);
  if (a) {
    st.sketch_clusters[1] = st.num_sms < tc::SK_MAX_CTAS ? st.num_sms : tc::SK_MAX_CTAS;
    a &= query_clusters(tc::sketch_kernel<2, 0>, 2, &st.sketch_clusters[2]);   // the same for every distribution
    a &= query_clusters(tc::gemm_kernel<tc::A_K, tc::B_K>, 2, &st.gemm_pairs, 64 + 32 * tc::NEPI, tc::GEMM_SMEM_BYTES);
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
                     float alpha, int* status, cudaStream_t stream, double* sumsq = nullptr, bool clear_status = false) {
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
  const int max_pairs = device_state().gemm_pairs;
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
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

// Sketch contraction out[j][d] = c * sum_n P[n][j] * b[n][d] for j < k (b is [tokens][cols] bf16),
// and, when ones_out is given, ones_out[d] = sum_n b[n][d] from the extra row of ones.
// The subsampled-Hadamard sketch by a two-level Walsh-Hadamard transform (fwht_kernels.cuh).  Returns
// RMM_ERR_UNSUPPORTED when the shape is outside the fast path (the caller then takes the dense kernel).
// scratch holds, in this order: the grouped column list, the per-block column sums, the stage-1 result
// T for as many columns per round as fit.
rmm_status launch_sors_fast(const void* b, void* out, void* ones_out, int64_t k, int64_t cols, int64_t tokens, float c,
                            const PhiloxKey& pk, void* scratch, size_t scratch_bytes, int* status, cudaStream_t stream,
                            bool clear_status) {
  const uint32_t mask = sors_mask_for(tokens);
  const int64_t L = (int64_t)mask + 1;
  if (L < FW_ROWS || L > (int64_t)FW_ROWS * FW_ROWS) return RMM_ERR_UNSUPPORTED;
  const int A = (int)(L / FW_ROWS);
  uint8_t* base = reinterpret_cast<uint8_t*>(scratch);
  size_t off = 0;
  SorsGroups g;
  g.offsets = reinterpret_cast<int*>(base + off);
  off += align_up(129 * sizeof(int));
  g.entries = reinterpret_cast<int2*>(base + off);
  off += align_up((size_t)k * sizeof(int2));
  if (off + 2 * kAlign >= scratch_bytes) return RMM_ERR_UNSUPPORTED;
  const size_t per_col = (size_t)A * sizeof(float) + (size_t)L * 2;       // column sums + T, per column of a round
  const int64_t cols64 = (cols + FW_COLS - 1) / FW_COLS * FW_COLS;
  int64_t wslab = (int64_t)((scratch_bytes - off - 2 * kAlign) / per_col) / FW_COLS * FW_COLS;
  if (wslab > cols64) wslab = cols64;
  if (wslab < FW_COLS) return RMM_ERR_UNSUPPORTED;
  {   // rounds of equal width rather than full ones and a narrow last one
    const int64_t rounds = (cols64 + wslab - 1) / wslab;
    wslab = ((cols64 + rounds - 1) / rounds + FW_COLS - 1) / FW_COLS * FW_COLS;
  }
  float* colsum = reinterpret_cast<float*>(base + off);
  off += align_up((size_t)A * (size_t)wslab * sizeof(float));
  __nv_bfloat16* T = reinterpret_cast<__nv_bfloat16*>(base + off);
  sors_group_kernel<<<1, 1024, 0, stream>>>(pk, k, mask, g, status, clear_status ? 1 : 0);
  if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
  const __nv_bfloat16* B = reinterpret_cast<const __nv_bfloat16*>(b);
  __nv_bfloat16* O = reinterpret_cast<__nv_bfloat16*>(out);
  __nv_bfloat16* ones = reinterpret_cast<__nv_bfloat16*>(ones_out);
  for (int64_t c0 = 0; c0 < cols; c0 += wslab) {
    const int width = (int)(cols - c0 < wslab ? cols - c0 : wslab);
    const unsigned slabs = (unsigned)((width + FW_COLS - 1) / FW_COLS);
    fwht_stage1_kernel<<<dim3(slabs, (unsigned)A), FW_THREADS, 0, stream>>>(B + c0, cols, tokens, width, pk, T, wslab,
                                                                           ones ? colsum : nullptr);
    if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
    fwht_stage2_kernel<<<dim3(slabs, FW_ROWS), FW_THREADS, 0, stream>>>(T, wslab, A, width, g, c, O + c0, cols,
                                                                       ones ? colsum : nullptr, ones ? ones + c0 : nullptr);
    if (cudaGetLastError() != cudaSuccess) return RMM_ERR_CUDA;
  }
  return RMM_OK;
}

rmm_status launch_sketch(const void* b, void* out, void* ones_out, int64_t k, int64_t cols, int64_t tokens, float c,
                         int dist, const PhiloxKey& pk, float* partial, int* status, cudaStream_t stream,
                         bool clear_status = false, size_t scratch_bytes = 0) {
  if (dist == RMM_DIST_SORS_HADAMARD && scratch_bytes > 0) {
    const rmm_status fs = launch_sors_fast(b, out, ones_out, k, cols, tokens, c, pk, partial, scratch_bytes, status, stream,
                                           clear_status);
    if (fs != RMM_ERR_UNSUPPORTED) return fs;
  }
  CUtensorMap tmB;
  const bool slab_map = cols % 64 == 0;
  if (!(slab_map ? make_tmap_slabs(&tmB, b, tokens, cols, tc::SK_BK, tc::SK_BN / 64)
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
  p.sched = tc::make_sketch_schedule(p.rows, cols, tokens, C, device_state().sketch_clusters[C]);
  const int per_tile = C;
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
  dim3 rgrid((unsigned)(p.sched.tiles() * per_tile), tc::SK_BN / tc::SKR_CHUNK);
  tc::sketch_reduce_kernel<<<rgrid, tc::SK_BM, 0, stream>>>(p, c, reinterpret_cast<__nv_bfloat16*>(out),
                                                      reinterpret_cast<__nv_bfloat16*>(ones_out));
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

template <typename T, bool GEN_A>
rmm_status launch_simt(const SimtGemmArgs& g, const PhiloxKey& pk, cudaStream_t stream) {
  dim3 grid((unsigned)((g.N + SIMT_BN - 1) / SIMT_BN), (unsigned)((g.M + SIMT_BM - 1) / SIMT_BM));
  simt_gemm_kernel<T, GEN_A><<<grid, SIMT_THREADS, 0, stream>>>(g, pk);
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
  db_partial_kernel<T><<<grid, 256, 0, stream>>>(reinterpret_cast<const T*>(dY), N, D_out, w.db_rows_per_slice, partial);
  db_finish_kernel<T><<<(unsigned)((D_out + 255) / 256), 256, 0, stream>>>(partial, w.db_slices, D_out,
                                                                           reinterpret_cast<T*>(db));
  return cudaGetLastError() == cudaSuccess ? RMM_OK : RMM_ERR_CUDA;
}

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
      dist != RMM_DIST_SORS_HADAMARD)
    return RMM_ERR_INVALID_ARG;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_IDENTITY && k != N) return RMM_ERR_INVALID_ARG;
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
    // the first kernel of the call resets the status word (no separate memset on the stream)
    if (Y) {
      ScopedTiming t(RMM_STEP_Y, stream);
      st = launch_tc<tc::A_K, tc::B_K>(X, W, Y, b, N, D_out, D_in, 1.0f, status, stream, nullptr, true);
      if (st != RMM_OK) return st;
    }
    ScopedTiming t(RMM_STEP_SKETCH, stream);
    return launch_sketch(X, X_proj, nullptr, B_proj, D_in, N, c, dist, pk, reinterpret_cast<float*>(ws + w.scratch_off),
                         status, stream, Y == nullptr, w.total - w.scratch_off);
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
    // the first kernel of the call resets the status word (no separate memset on the stream)
    if (dX) {
      ScopedTiming t(RMM_STEP_DX, stream);
      st = launch_tc<tc::A_K, tc::B_MN>(dY, W, dX, nullptr, N, D_in, D_out, 1.0f, status, stream, nullptr, true);
      if (st != RMM_OK) return st;
    }
    {
      // db = dY^T 1 comes out of the same contraction as the extra row of ones of S^T
      ScopedTiming t(RMM_STEP_SDY, stream);
      st = launch_sketch(dY, G, db, B_proj, D_out, N, c, dist, pk, reinterpret_cast<float*>(ws + w.scratch_off), status,
                         stream, dX == nullptr, w.total - w.scratch_off);
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
      dist != RMM_DIST_SORS_HADAMARD)
    return RMM_ERR_INVALID_ARG;
  if (dt != RMM_DTYPE_BF16 && dt != RMM_DTYPE_F32) return RMM_ERR_INVALID_ARG;
  if (dist == RMM_DIST_IDENTITY && B_proj != N) return RMM_ERR_INVALID_ARG;
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
  if (dist == RMM_DIST_SORS_HADAMARD) return RMM_ERR_UNSUPPORTED;   // no closed form for its variance here
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
