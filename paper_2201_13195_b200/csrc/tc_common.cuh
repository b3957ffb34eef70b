// sm_100a building blocks: mbarrier, TMA (bulk tensor copies), tcgen05 (5th-generation
// tensor cores with accumulators in tensor memory) as thin inline-PTX wrappers, plus the
// shared-memory and instruction descriptors that tcgen05.mma consumes.
//
// Every wait in this file is bounded: a wait that neither completes nor is cancelled
// within its limit reports failure, the caller records RMM_ERR_TIMEOUT in the
// workspace status word, raises the CTA-wide abort flag and leaves through the normal
// teardown (tensor memory is freed, the kernel returns, the context stays usable).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace rmm {
namespace tc {

constexpr int kStatusTimeout = 5;                 // == RMM_ERR_TIMEOUT
constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s of SM clock per wait
constexpr uint32_t kWaitLimitPolls = 1u << 30;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile(
      "{\n .reg .pred p;\n elect.sync _|p, 0xffffffff;\n selp.u32 %0, 1, 0, p;\n}\n" : "=r"(pred));
  return pred != 0;
}

// ---------------------------------------------------------------- mbarrier
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait.  Returns false if the abort flag was raised by someone else or if the
// limit ran out (then it raises the flag itself and records the timeout).  The limit is
// counted in polls and in SM cycles (clock64 is a register read).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait(bar, parity)) return true;
  long long t0 = 0;
  for (uint32_t polls = 1; polls < kWaitLimitPolls; ++polls) {
    if (mbar_try_wait(bar, parity)) return true;
    if ((polls & 0x3f) == 0) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitCycles) break;
    }
  }
  *abort_flag = 1;
  if (status) atomicExch(status, kStatusTimeout);
  return false;
}

// Early test of a barrier phase ("peek").  A barrier test is a long round trip for the one warp
// that issues MMAs; started one stage ahead, it overlaps the MMA issue of the current stage, and
// the blocking wait is only entered when the early test said "not yet".  The predicate lives in
// a PTX register that MBAR_PEEK_DECLARE() declares once, in the entry block of the kernel;
// slot is a literal 0 or 1.  All lanes of the warp test the same address in one instruction, so
// they read the same answer.
#define MBAR_PEEK_DECLARE() asm volatile(".reg .pred mbar_peek0, mbar_peek1;")
#define MBAR_PEEK(slot, bar, parity) \
  asm volatile("mbarrier.test_wait.parity.shared::cta.b64 mbar_peek" #slot ", [%0], %1;" ::"r"(bar), "r"(parity) : "memory")
#define MBAR_PEEK_CLUSTER(slot, bar, parity)                                                                       \
  asm volatile("mbarrier.test_wait.parity.acquire.cluster.shared::cta.b64 mbar_peek" #slot ", [%0], %1;" ::"r"(bar), \
               "r"(parity)                                                                                          \
               : "memory")
#define MBAR_PEEK_RESULT(slot, out) asm volatile("selp.u32 %0, 1, 0, mbar_peek" #slot ";" : "=r"(out)::"memory")

// ---------------------------------------------------------------- thread-block clusters
__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// shared::cluster address of the same shared-memory location in the CTA of rank `rank`
__device__ __forceinline__ uint32_t mapa_shared(uint32_t local_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
  return r;
}
// all threads of all CTAs of the cluster
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// arrive on a barrier that may live in another CTA of the cluster (address from mapa_shared)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The same with the default semantics of mbarrier.arrive (release at CTA scope): for a producer that has made its
// shared-memory writes visible to the async proxy (fence_proxy_async_smem) and whose data is read by the tensor
// cores, not by the threads that wait on the barrier.  A cluster-scope release makes the arriving thread wait
// until all its earlier writes are visible cluster-wide, which costs thousands of cycles per arrival.
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// Asynchronous copy of `bytes` (a multiple of 16, both addresses 16-byte aligned) from this CTA's
// shared memory into the shared memory of a CTA of the cluster (address from mapa_shared). The
// bytes are counted on an mbarrier of the destination CTA, so the consumer's wait on that barrier
// covers the data. The source is read through the async proxy: writers fence with
// fence_proxy_async_smem() before the issuing thread is told that the data is there.
__device__ __forceinline__ void bulk_copy_to_cluster(uint32_t dst_cluster_addr, uint32_t src_cta_addr, uint32_t bytes,
                                                     uint32_t cluster_mbar) {
  asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(dst_cluster_addr), "r"(src_cta_addr), "r"(bytes), "r"(cluster_mbar)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait on a barrier of this CTA that other CTAs of the cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  long long t0 = 0;
  for (uint32_t polls = 1; polls < kWaitLimitPolls; ++polls) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((polls & 0x3f) == 0) {
      if (*abort_flag) return false;
      const long long now = clock64();
      if (t0 == 0) t0 = now;
      else if (now - t0 > kWaitLimitCycles) break;
    }
  }
  *abort_flag = 1;
  if (status) atomicExch(status, kStatusTimeout);
  return false;
}
// Warp-level waits: lane 0 polls, the other lanes park at the warp barrier.  A whole warp (or
// sixteen of them) spinning on try_wait floods the shared-memory pipe that the MMA issuer's own
// barrier and tcgen05 instructions go through.
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag, int* status) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait(bar, parity, abort_flag, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}
__device__ __forceinline__ bool mbar_wait_cluster_warp(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                       int* status) {
  int ok = 1;
  if ((threadIdx.x & 31) == 0) ok = mbar_wait_cluster(bar, parity, abort_flag, status) ? 1 : 0;
  return __shfl_sync(0xffffffffu, ok, 0) != 0;
}

// ---------------------------------------------------------------- CTA pairs (cta_group::2)
// Two CTAs of a cluster with consecutive ranks work as one MMA unit; the leader is the even one.
__device__ __forceinline__ void tmem_alloc_pair(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
// Tiled load into this CTA's shared memory whose completion bytes are counted on a barrier that
// may belong to the other CTA of the pair (bar_cluster_addr from mapa_shared).
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(bar_cluster_addr), "r"(x), "r"(y)
      : "memory");
}
// D[tensor memory of both CTAs] (+)= A * B over the pair: M = 256 (128 rows from each CTA's A tile),
// N columns of B of which each CTA holds half; issued by one thread of the leader CTA.
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive on a barrier (of any CTA of the cluster) once all pair MMAs issued so far have completed
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster_addr) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr)
               : "memory");
}

// The same arrival on the barriers at this shared-memory offset in every CTA of the pair named by `cta_mask`
// (bit r = CTA of rank r), with one instruction.
__device__ __forceinline__ void umma_commit_pair_multicast(uint32_t bar_local_addr, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
               ::"r"(bar_local_addr), "h"(cta_mask)
               : "memory");
}
// Asynchronous 4-byte store into the shared memory of a CTA of the cluster whose 4 bytes are counted on an mbarrier of
// that CTA (both addresses from mapa_shared).  Does not block the issuing thread: used as a signal across the pair
// where an mbarrier.arrive on a shared::cluster address stalls the arriving warp for thousands of cycles.
__device__ __forceinline__ void st_async_u32(uint32_t dst_cluster_addr, uint32_t value, uint32_t cluster_mbar) {
  asm volatile("st.async.shared::cluster.mbarrier::complete_tx::bytes.b32 [%0], %1, [%2];"
               ::"r"(dst_cluster_addr), "r"(value), "r"(cluster_mbar)
               : "memory");
}

// generic-proxy writes to shared memory -> visible to the async proxy (TMA, tcgen05)
__device__ __forceinline__ void fence_proxy_async_smem() {
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}

// ---------------------------------------------------------------- TMA
__device__ __forceinline__ void tma_prefetch_desc(const CUtensorMap* m) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(m) : "memory");
}
// 2-D tiled load global -> shared, completion counted in bytes on an mbarrier.
// x = innermost (contiguous) coordinate, y = row coordinate, both in elements.
__device__ __forceinline__ void tma_load_2d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar, int x, int y) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(bar), "r"(x), "r"(y)
      : "memory");
}

// 3-D tiled load (x innermost).  Used to fetch several [rows][64-column] slabs of a row-major
// matrix with one instruction: the matrix is viewed as (column in slab, row, slab).
__device__ __forceinline__ void tma_load_3d(uint32_t dst_smem, const CUtensorMap* map, uint32_t bar, int x, int y, int z) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
      ::"r"(dst_smem), "l"(map), "r"(bar), "r"(x), "r"(y), "r"(z)
      : "memory");
}

// 2-D tiled store shared -> global (bulk async group of the issuing thread).  The box is clipped
// at the tensor's bounds: rows and columns out of range are not written.  x must be a multiple of
// 8 elements (16 bytes) and neither coordinate negative.
__device__ __forceinline__ void tma_store_2d(const CUtensorMap* map, uint32_t src_smem, int x, int y) {
  asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];"
               ::"l"(map), "r"(src_smem), "r"(x), "r"(y)
               : "memory");
}
__device__ __forceinline__ void bulk_commit_group() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// Waits until at most N of the issuing thread's bulk groups still read their shared-memory source.
template <int N>
__device__ __forceinline__ void bulk_wait_group_read() {
  asm volatile("cp.async.bulk.wait_group.read %0;" ::"n"(N) : "memory");
}
// Waits until all of the issuing thread's bulk groups have completed.
__device__ __forceinline__ void bulk_wait_group_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

// ---------------------------------------------------------------- tensor memory
__device__ __forceinline__ void tmem_alloc(uint32_t slot_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(slot_smem), "r"(ncols)
               : "memory");
}
__device__ __forceinline__ void tmem_relinquish() {
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// D[tmem] (+)= A[smem] * B[smem], bf16 inputs, fp32 accumulate; issued by one thread.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// mbarrier arrive once every tcgen05.mma issued so far by this thread has completed.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// 32 lanes x 32 consecutive fp32 columns: thread i of the warp receives lane (base+i).
__device__ __forceinline__ void tmem_ld_32x32(uint32_t taddr, uint32_t v[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Optional cycle accounting (build with -DRMM_PASS_TRACE): per CTA, how long each role spent in its loops
// and in each kind of wait.  Read back with rmm_debug_pass_trace.  Not compiled into the product library.
#ifdef RMM_PASS_TRACE
constexpr int PS_TRACE_SLOTS = 32;
__device__ long long g_pass_trace[148][PS_TRACE_SLOTS];
#define PS_TRACE_DECL(name) long long name = 0
#define PS_TRACE_T0(name) const long long name = clock64()
#define PS_TRACE_ADD(acc, t0) acc += clock64() - (t0)
#define PS_TRACE_PUT(slot, value) g_pass_trace[blockIdx.x][slot] = (value)
#else
#define PS_TRACE_DECL(name)
#define PS_TRACE_T0(name)
#define PS_TRACE_ADD(acc, t0)
#define PS_TRACE_PUT(slot, value)
#endif

// ---------------------------------------------------------------- completion flags across CTAs
// A CTA that has stored a partial result raises its flag: it writes the launch's tag (unique per launch, so that
// values left by earlier launches, or never written, read as "not yet") with release semantics.  A reader polls
// the flags it needs with acquire loads.  No atomics: nothing to reset, no contention between the writers.
__device__ __forceinline__ void flag_raise(unsigned long long* f, unsigned long long tag) {
  asm volatile("st.release.gpu.global.u64 [%0], %1;" ::"l"(f), "l"(tag) : "memory");
}
__device__ __forceinline__ unsigned long long ld_acquire_gpu(const unsigned long long* p) {
  unsigned long long v;
  asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(v) : "l"(p) : "memory");
  return v;
}
// Bounded wait of a whole warp until the `count` flags f[first], f[first + stride], ... all carry `tag`
// (lane i polls the flags i, i + 32, ...).  Returns false on abort or when the limit runs out.
__device__ __forceinline__ bool flags_wait_warp(const unsigned long long* f, long long first, long long stride, int count,
                                                unsigned long long tag, volatile int* abort_flag, int* status) {
  const int lane = (int)(threadIdx.x & 31);
  const long long t0 = clock64();
  for (uint32_t polls = 0; polls < kWaitLimitPolls; ++polls) {
    bool mine = true;
    for (int i = lane; i < count; i += 32) mine = mine && ld_acquire_gpu(f + first + (long long)i * stride) == tag;
    if (__all_sync(0xffffffffu, mine)) return true;
    __nanosleep(100);
    if ((polls & 0xf) == 0xf) {
      const bool stop = *abort_flag != 0 || clock64() - t0 > kWaitLimitCycles;
      if (__any_sync(0xffffffffu, stop)) break;
    }
  }
  if (lane == 0 && *abort_flag == 0) {
    *abort_flag = 1;
    if (status) atomicExch(status, kStatusTimeout);
  }
  __syncwarp();
  return false;
}

// ---------------------------------------------------------------- descriptors
// Shared-memory matrix descriptor, 128-byte swizzle.  Bits: [0,14) start address >> 4,
// [16,30) leading byte offset >> 4, [32,46) stride byte offset >> 4, [46,48) version = 1,
// [61,64) layout = 2 (128-byte swizzle).
//   K-major tile (rows of 64 bf16 = 128 B, 8-row groups 1024 B apart): LBO unused (1), SBO = 1024.
//   MN-major tile (slabs of [K rows][64 bf16]): LBO = bytes between 64-element slabs along
//   M/N, SBO = bytes between groups of 8 K rows = 1024.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t saddr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
  uint64_t d = 0;
  d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
  d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFFu) << 16;
  d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFFu) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
// Instruction descriptor for kind::f16 with bf16 inputs and fp32 accumulation.
// Bits: [4,6) D format (1 = f32), [7,10) A format (1 = bf16), [10,13) B format,
// 15 A major (1 = MN), 16 B major, [17,23) N >> 3, [24,29) M >> 4.
__host__ __device__ constexpr uint32_t instr_desc_bf16(int m, int n, bool a_mn_major, bool b_mn_major) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((a_mn_major ? 1u : 0u) << 15) | ((b_mn_major ? 1u : 0u) << 16) |
         ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}

}  // namespace tc
}  // namespace rmm
