/*
 * rmm.h - C ABI of the randomized-matrix-multiplication (RMM) linear layer for
 * NVIDIA B200 (sm_100a).
 *
 * The layer is the one of "Memory-Efficient Backpropagation through Large Linear
 * Layers" (arXiv 2201.13195), Section 2.1, Algorithm 1: the forward pass returns
 * Y = X W^T + 1 b^T (Eq. 1) and keeps, instead of X, the sketch X_proj = S^T X
 * together with the seed that S was drawn from; the backward pass regenerates S,
 * and returns the exact dX = dY W (Eq. 2), the randomized estimate
 * dW = (dY^T S) X_proj of dY^T X (Eq. 4) and the exact db = dY^T 1 (Eq. 3).
 *
 * Notation: N = number of token rows (the paper's batch dimension B), D_in / D_out =
 * the paper's N_in / N_out, B_proj = number of columns of S (Section 2.4.2).
 *
 * General conventions
 *   - Every tensor pointer is a DEVICE pointer owned by the caller, row-major,
 *     contiguous, 16-byte aligned.  The library allocates no device memory and never
 *     synchronises.  To the caller all work is ordered on the CUDA stream that is passed in
 *     (a cudaStream_t cast to void*, NULL = default stream); in the default pass mode part
 *     of a bf16 pass is queued on a stream of the library's own that forks from and joins
 *     that stream through events (rmm_set_pass_mode).  What the library keeps between
 *     calls, per process: per device the kernels' attributes, eight such side streams with
 *     two events each (created at the first call made with that device current) and the
 *     address of the fixed scratch of rmm_bias_grad_static; the last 64 pass plans by
 *     shape; a launch counter.  Results never depend on any of it.
 *   - Outputs are overwritten, never accumulated into.
 *   - dtype RMM_DTYPE_BF16: tensors are bfloat16, contractions run on the tensor
 *     cores with fp32 accumulation; D_in and D_out must be multiples of 8.
 *     dtype RMM_DTYPE_F32: tensors are fp32, contractions are plain fp32 FMA.
 *   - Errors are return codes.  Argument errors are detected on the host before any
 *     launch.  A device-side wait that does not complete within its iteration limit
 *     is recorded in the workspace and reported by rmm_last_device_status().
 *   - There is no CPU fallback: on a machine without a usable sm_100a device every
 *     compute entry point returns RMM_ERR_CUDA.
 *
 * The sketch matrix S (N x B_proj) is a pure function of (seed, dist, N-index,
 * column index, dtype); it does not depend on tile shapes, launch geometry or on
 * which pass asks for it.  S = c * P with c = fp32 1/sqrt(B_proj) and
 *   RMM_DIST_GAUSSIAN   P iid standard normal (Eq. 5): Philox4x32-10 with key =
 *                       (seed low word, seed high word) and counter
 *                       (n >> 3, j, 0, 0) gives four words; word i gives, by a
 *                       Box-Muller transform on its two 16-bit halves evaluated with
 *                       a fixed sequence of correctly rounded fp32 operations, the
 *                       entries P[8*(n>>3) + 2i][j] and P[8*(n>>3) + 2i + 1][j];
 *   RMM_DIST_RADEMACHER P = +-1 with probability 1/2 (Section 3.5): counter
 *                       (n >> 7, j, 0, 1) gives 128 bits, entry P[n][j] is -1 when
 *                       bit (n & 31) of word ((n & 127) >> 5) is set;
 *   RMM_DIST_SORS_HADAMARD  subsampled orthonormal matrix with random signs (Section 2.1 names the
 *                       family; the paper gives no construction, this one is this library's):
 *                       P[n][j] = d_n * H[n][r_j] with H the Sylvester Hadamard matrix of the
 *                       smallest power-of-two order >= N, H[n][r] = (-1)^popcount(n & r);
 *                       d_n = -1 when bit (n & 31) of word ((n & 127) >> 5) of counter
 *                       (n >> 7, 0, 0, 2) is set; r_j = first word of counter (j, 0, 0, 3)
 *                       modulo the order (columns drawn with replacement, so E[S S^T] = I
 *                       exactly).  In bf16 mode, for 128 <= order <= 16384, the sketches are
 *                       applied by a two-level Walsh-Hadamard transform over the token index
 *                       (O(N D log N)); otherwise by the same dense contraction as the other
 *                       distributions.  S is the same matrix either way;
 *   RMM_DIST_SORS_DCT   subsampled DCT-II matrix with random signs (Section 3.5 and Table 4 compare DCT
 *                       sketches; the construction is this library's): with L, d_n and r_j as above and C the
 *                       orthonormal DCT-II matrix of order L, P[n][j] = d_n * sqrt(L) * C[r_j][n], i.e. d_n for
 *                       r_j = 0 and d_n * sqrt(2) cos(pi (2n+1) r_j / (2L)) otherwise, the cosine evaluated by
 *                       a fixed fp32 sequence (exact integer quadrant reduction, two cubic polynomials with
 *                       fused multiply-adds).  E[S S^T] = I exactly up to that sequence's error of 2e-5.
 *                       Applied by the dense contraction kernels;
 *   RMM_DIST_IDENTITY   S = I (needs B_proj == N; c = 1): the case in which the
 *                       layer reduces to the exact linear layer; meant for tests.
 * In bf16 mode P is rounded to bfloat16 (nearest even) before it is used.
 */
#ifndef RMM_H_
#define RMM_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  RMM_OK = 0,
  RMM_ERR_INVALID_ARG = 1, /* null pointer, non-positive size, B_proj outside [1,N], bad enum, misalignment */
  RMM_ERR_UNSUPPORTED = 2, /* shape not supported in this dtype (D_in or D_out not a multiple of 8 in bf16) */
  RMM_ERR_WORKSPACE = 3,   /* workspace missing, misaligned or smaller than rmm_workspace_bytes() */
  RMM_ERR_CUDA = 4,        /* a CUDA runtime or driver call failed (including: no sm_100a device) */
  RMM_ERR_TIMEOUT = 5      /* a device-side wait gave up; results of that call are invalid */
} rmm_status;

typedef enum {
  RMM_DIST_GAUSSIAN = 0,
  RMM_DIST_RADEMACHER = 1,
  RMM_DIST_IDENTITY = 2,
  RMM_DIST_SORS_HADAMARD = 3,
  RMM_DIST_SORS_DCT = 4
} rmm_dist;
typedef enum { RMM_DTYPE_BF16 = 0, RMM_DTYPE_F32 = 1 } rmm_dtype;

/*
 * Bytes of scratch device memory that rmm_forward / rmm_backward need for these
 * sizes (the larger of the two).  The scratch holds the intermediate G = S^T dY
 * (B_proj x D_out), fp32 partial tiles of the sketches with their completion flags, and a
 * status word; it need not be initialised.  Returns 0 for invalid sizes.
 * The same workspace may be reused by later calls on the same stream; calls that may
 * overlap on the device need separate workspaces.
 */
size_t rmm_workspace_bytes(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt);

/*
 * The workspace size with which calls that use sketch `dist` run fastest; never less than
 * rmm_workspace_bytes(), and equal to it for every distribution but RMM_DIST_SORS_HADAMARD in bf16
 * mode with at most 16384 tokens.  There the fast transform (Section 2.1: structured sketches have a
 * fast matrix-by-vector product) keeps an intermediate of L x D bf16 values (L = the Hadamard order,
 * D = the wider of D_in and D_out) in the workspace; with less room it takes the columns in
 * several rounds of launches.  Any workspace of at least rmm_workspace_bytes() bytes is valid for
 * every call; the calls use all of the workspace_bytes they are given.
 */
size_t rmm_workspace_bytes_for(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt, rmm_dist dist);

/*
 * Algorithm 1, FORWARD (Eq. 1 and X_proj = S^T X, Section 2.1).
 *   in : X [N, D_in], W [D_out, D_in], b [D_out] or NULL (no bias)
 *   out: Y [N, D_out] = X W^T + 1 b^T ;  X_proj [B_proj, D_in] = S^T X
 * X_proj and seed are all the caller has to keep for the backward pass.  Use a fresh
 * seed for every layer and every step: S must be independent of dY (Section 2.1).
 * Y may be NULL (only the sketch is computed).
 */
rmm_status rmm_forward(const void* X, const void* W, const void* b,
                       int64_t N, int64_t D_in, int64_t D_out,
                       uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt,
                       void* Y, void* X_proj,
                       void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Algorithm 1, BACKWARD (Eq. 2, 3, 4).  (seed, B_proj, dist, N) must be the values
 * given to the forward call that produced X_proj.
 *   in : dY [N, D_out], W [D_out, D_in], X_proj [B_proj, D_in]
 *   out: dX [N, D_in] = dY W               (exact; NULL to skip)
 *        dW [D_out, D_in] = (S^T dY)^T X_proj   (unbiased estimate of dY^T X)
 *        db [D_out] = sum over rows of dY  (exact; NULL to skip)
 * The bias is not an input: Algorithm 1 lists it but no gradient depends on it.
 */
rmm_status rmm_backward(const void* dY, const void* W, const void* X_proj,
                        int64_t N, int64_t D_in, int64_t D_out,
                        uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt,
                        void* dX, void* dW, void* db,
                        void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * How the bf16 passes are executed (no counterpart in the paper; process-wide, takes effect for later calls).
 *   0 (default): the dense product and the sketch of a pass (Y and S^T X; dX and S^T dY) are two persistent
 *      kernels that run at the same time on disjoint sets of SMs; the sketch kernel is queued on a stream of the
 *      library's own that forks from and joins the caller's stream through events, so to the caller the pass is
 *      still ordered on its stream.  The library creates these side streams (eight per device) at its first call
 *      on a device and keeps them until the process exits.
 *   1: both parts of a pass in ONE launch (a kernel whose CTA pairs take sketch units and dense tiles from one
 *      static schedule).  Same results up to the order of the fp32 partial sums; slower on B200 for the Gaussian
 *      sketch (the generation of S does not keep up with two SMs that share every generated entry through the
 *      tensor cores' pair mode), kept as an alternative and for measurements.
 *   2: the two kernels of mode 0 one after the other on the caller's stream, each on the whole device.
 * Returns RMM_ERR_INVALID_ARG for any other value.
 */
rmm_status rmm_set_pass_mode(int mode);

/*
 * Writes the sketch matrix itself, S_out [N, B_proj] row-major in the given dtype
 * holding the UNSCALED entries P (multiply by fp32 1/sqrt(B_proj) to get S, Eq. 5).
 * Not part of the layer: it exists so that the generator can be compared bit for bit
 * with an independent implementation.
 */
rmm_status rmm_debug_generate_s(uint64_t seed, int64_t N, int64_t B_proj, rmm_dist dist, rmm_dtype dt,
                                void* S_out, void* cuda_stream);

/*
 * Applies the uniform -> normal map of RMM_DIST_GAUSSIAN to n given Philox output words
 * (device array): out[2i] and out[2i+1] (device, fp32) are the two normals that word i
 * yields, before any storage rounding.  Debug aid like rmm_debug_generate_s: lets a test
 * sweep all 2^16 radius inputs and all 2^16 angle inputs of the transform.
 */
rmm_status rmm_debug_gauss_words(const uint32_t* words, int64_t n, float* out, void* cuda_stream);

/*
 * Host-only testing aid (no device needed): the static work schedule of the sketch kernels
 * for a result of `rows` x `cols` contracted over `tokens`, on `max_ctas` CTAs.  CTAs work in
 * clusters of C (2 when the result has at least two 512-column blocks, else 1); a "tile" is
 * 128 rows x C 512-column blocks and a "cta" in the records is one cluster.
 *   mode 0: one record (cta, tile, first step, end step, slot) per work segment, in the
 *           order in which each CTA executes them;
 *   mode 1: one record (tile, slot, 0, 0, 0) per partial tile in the order in which the
 *           reduction adds them.
 * Writes at most `cap` records of five int64 to `records` (host memory) and returns the
 * number of records that exist; info[0..7] = tiles, 64-token steps per tile, clusters, slots, C, rounds of
 * whole tiles, full token blocks per remaining tile, width of the last block (0: none, the tiles are cut into
 * equal blocks only).
 */
int64_t rmm_debug_sketch_schedule(int64_t rows, int64_t cols, int64_t tokens, int max_ctas, int mode,
                                  int64_t* records, int64_t cap, int64_t* info);

/*
 * Host-only testing aid (no device needed): the static work schedule of one pass launch (Algorithm 1,
 * FORWARD or BACKWARD without its last product) on `max_pairs` CTA pairs.  The dense part is a
 * gemm_m x gemm_n result contracted over gemm_k (gemm_m = 0: none), in 256 x 256 tiles; the sketch part a
 * rows x cols result contracted over `tokens` (rows = 0: none), in tiles of 128 rows x nat x 256 columns cut
 * along the tokens into nb blocks of blen 64-token steps.  Writes to out (host memory, at most cap values):
 *   num_pairs, dense tiles, dense column tiles, K blocks, sketch row tiles, column groups, nat,
 *   64-token steps, nb, blen, then num_pairs + 1 values b[p]: pair p computes the dense tiles
 *   [b[p], b[p + 1]).  Sketch unit i = block * (row tiles * groups) + tile goes to pair i % num_pairs.
 * Returns the number of values that exist, or -1 for invalid arguments.
 */
int64_t rmm_debug_pass_schedule(int64_t gemm_m, int64_t gemm_n, int64_t gemm_k, int64_t rows, int64_t cols,
                                int64_t tokens, int max_pairs, int64_t* out, int64_t cap);

/*
 * Host-only testing aid (no device needed): how the fast transform of RMM_DIST_SORS_HADAMARD (bf16 mode) would
 * take a sketch of `rows` rows over a tokens x cols matrix with `scratch_bytes` bytes of scratch (the part of the
 * workspace that follows the status word, the flags and G).
 * Returns 1 and writes info[0..3] = Hadamard order L, L / 128, columns per round, rounds (two launches each);
 * 0 when the shape is outside the fast path (the dense sketch kernel is used); -1 for invalid arguments.
 */
int rmm_debug_hadamard_plan(int64_t rows, int64_t cols, int64_t tokens, size_t scratch_bytes, int64_t* info);

/*
 * Reads the status word that the kernels of the last call using this workspace left
 * there.  HOST-synchronous on the device-to-host copy of one word: the caller must
 * have synchronised the stream first.  Returns RMM_OK or RMM_ERR_TIMEOUT (or
 * RMM_ERR_CUDA if the copy fails).
 */
rmm_status rmm_last_device_status(const void* workspace);

/* Static, human-readable name of a status code. */
const char* rmm_status_string(rmm_status s);

/*
 * Per-kernel timing for benchmarks (no counterpart in the paper).  While enabled,
 * every kernel that rmm_forward / rmm_backward launch is bracketed by a pair of CUDA
 * events recorded on the caller's stream, up to `capacity` launches; further launches
 * are not recorded.  Event objects are created by rmm_profile_enable(capacity > 0)
 * and destroyed by rmm_profile_enable(0).  Process-wide, not thread-safe; meant for a
 * single benchmarking thread.
 *   rmm_profile_read: waits for the recorded events, writes for each recorded launch
 *   its step id (rmm_step below) and its duration in milliseconds, returns the
 *   number of records written (at most max_records) and clears the record list.
 */
typedef enum {
  RMM_STEP_Y = 0,       /* Y = X W^T + b            (Eq. 1) */
  RMM_STEP_SKETCH = 1,  /* X_proj = S^T X           (Section 2.1) */
  RMM_STEP_DX = 2,      /* dX = dY W                (Eq. 2) */
  RMM_STEP_SDY = 3,     /* G = S^T dY               (Algorithm 1, inner product of Eq. 4) */
  RMM_STEP_DW = 4,      /* dW = G^T X_proj          (Eq. 4) */
  RMM_STEP_DB = 5,      /* db = dY^T 1              (Eq. 3), partial sums and final sum */
  RMM_STEP_FWD = 6,     /* Y and X_proj in one launch       (Algorithm 1, FORWARD) */
  RMM_STEP_BWD = 7      /* dX, G = S^T dY and db in one launch (Algorithm 1, BACKWARD, all but the last product) */
} rmm_step;
rmm_status rmm_profile_enable(int capacity);
/* Number of kernels that rmm_forward / rmm_backward (and their host-buffer forms) have launched in this
 * process so far (no counterpart in the paper; a benchmark's launch count). */
int64_t rmm_layer_launch_count(void);
int rmm_profile_read(int* step_ids, float* milliseconds, int max_records);

/*
 * Bias gradient without any allocation (the paper has no counterpart; it computes the
 * same db = dY^T 1 of Eq. 3 that rmm_backward returns).
 *
 * For callers that hold no workspace and cannot obtain one: code running inside a
 * memory-pool or graph-replay region where cudaMalloc (and with it every allocating
 * library routine, PyTorch's caching allocator included) is forbidden, or late in a
 * step when the device is full.  rmm_backward needs caller-provided scratch for its
 * partial sums; this entry point keeps that scratch in a fixed array that is part of
 * the library image: RMM_BIAS_GRAD_STATIC_SLICES x RMM_BIAS_GRAD_STATIC_MAX_D_OUT
 * fp32 values = 256 KiB, resident on every GPU that loads the library until the process
 * exits.  It calls no cudaMalloc, cudaFree or other allocating routine.
 *   in : dY [N, D_out] (device, row-major, 16-byte aligned), dt = element type
 *   out: db [D_out] (device) = column sums of dY, accumulated in fp32
 * Returns RMM_ERR_UNSUPPORTED when D_out > RMM_BIAS_GRAD_STATIC_MAX_D_OUT, and
 * RMM_ERR_INVALID_ARG for null or misaligned pointers or non-positive sizes.
 * The first call on each device looks up the device address of the array (one driver
 * query, with that device current); make that first call outside any stream capture.
 * All calls on a device share the one array, which keeps the previous call's partial
 * sums: every value that is read is rewritten first, so nothing needs clearing, but two
 * calls that may run concurrently on the same device (different streams) race on it.
 */
#define RMM_BIAS_GRAD_STATIC_MAX_D_OUT 4096
#define RMM_BIAS_GRAD_STATIC_SLICES 16
rmm_status rmm_bias_grad_static(const void* dY, int64_t N, int64_t D_out, rmm_dtype dt, void* db,
                                void* cuda_stream);

/*
 * Variance diagnostics of the randomized weight gradient (Section 2.3).  For one layer's
 * actual X [N, D_in] and dY [N, D_out] (the paper's X and Y of Lemmas 1 and 2) it computes
 *   out[0] = |X|_F^2            out[1] = |dY|_F^2
 *   out[2] = sum_n |x_n|^2 |dy_n|^2
 *   out[3] = |X^T dY|_F^2       (the squared norm of the exact gradient, Eq. 3)
 *   out[4] = D^2_SGD = N/(N-1) out[2] - out[3]/(N-1)                        (Lemma 1, Eq. 9)
 *   out[5] = D^2_RMM = E |X^T S S^T dY - X^T dY|_F^2 for the given sketch with the fourth
 *            moment of its entries kept: (out[0] out[1] + out[3]) / B_proj for Gaussian S,
 *            (out[0] out[1] + out[3] - 2 out[2]) / B_proj for Rademacher S, 0 for S = I
 *   out[6] = (out[0] out[1] - out[3]) / B_proj, the expression Lemma 2, Eq. 11 prints
 *            (it drops the fourth moment; it equals out[5] only when X^T dY = 0)
 *   out[7] = alpha = out[3] / (out[0] out[1])                               (Theorem 1, Eq. 13)
 * It needs X, so it is a debugging aid for a probed layer, not part of a training step that
 * wants the memory saving (the paper, too, probes single layers: Section 3.3).
 *   in : X, dY (device, bf16 only: RMM_ERR_UNSUPPORTED for RMM_DTYPE_F32), N >= 2,
 *        1 <= B_proj <= N, dist as in rmm_forward except RMM_DIST_SORS_HADAMARD
 *        (RMM_ERR_UNSUPPORTED: its variance has no closed form among the above)
 *   out: out = 8 doubles in DEVICE memory (16-byte aligned), written on the stream;
 *        dW_exact (nullable) = the exact gradient dY^T X [D_out, D_in] in bf16, which the
 *        probe computes on the way
 *   workspace: at least rmm_variance_probe_workspace_bytes(N, D_in, D_out) bytes, 256-byte
 *        aligned, caller-owned; it also receives the device status word that
 *        rmm_last_device_status() reads.
 * Sums are accumulated in fp32 inside a row or a tensor-core tile and in fp64 across them,
 * in a fixed order (the result is reproducible).
 */
size_t rmm_variance_probe_workspace_bytes(int64_t N, int64_t D_in, int64_t D_out);
rmm_status rmm_variance_probe(const void* X, const void* dY, int64_t N, int64_t D_in, int64_t D_out,
                              int64_t B_proj, rmm_dist dist, rmm_dtype dt, double* out, void* dW_exact,
                              void* workspace, size_t workspace_bytes, void* cuda_stream);

/*
 * Host-buffer convenience wrappers (end-to-end path): the tensor arguments are HOST
 * pointers (pinned memory recommended); the device buffers dev_* and the workspace
 * are caller-owned DEVICE scratch of at least the tensors' sizes.  Each call copies
 * its inputs host->device, runs the device entry point above, and copies the outputs
 * device->host, all on cuda_stream, then synchronises that stream.
 *   rmm_forward_host : dev_in  >= bytes(X) + bytes(W) + bytes(b), dev_out >= bytes(Y) + bytes(X_proj)
 *   rmm_backward_host: dev_in  >= bytes(dY) + bytes(W) + bytes(X_proj), dev_out >= bytes(dX) + bytes(dW) + bytes(db)
 * Sizes are rounded up to multiples of 256 bytes per tensor; see rmm_host_staging_bytes().
 */
size_t rmm_host_staging_bytes(int64_t N, int64_t D_in, int64_t D_out, int64_t B_proj, rmm_dtype dt,
                              int backward, int outputs);
rmm_status rmm_forward_host(const void* X, const void* W, const void* b,
                            int64_t N, int64_t D_in, int64_t D_out,
                            uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt,
                            void* Y, void* X_proj,
                            void* dev_in, void* dev_out,
                            void* workspace, size_t workspace_bytes, void* cuda_stream);
rmm_status rmm_backward_host(const void* dY, const void* W, const void* X_proj,
                             int64_t N, int64_t D_in, int64_t D_out,
                             uint64_t seed, int64_t B_proj, rmm_dist dist, rmm_dtype dt,
                             void* dX, void* dW, void* db,
                             void* dev_in, void* dev_out,
                             void* workspace, size_t workspace_bytes, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RMM_H_ */
