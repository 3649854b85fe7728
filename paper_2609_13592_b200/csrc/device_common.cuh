// Device-side building blocks shared by the kernels: mbarrier / bulk-copy / cp.async
// wrappers (inline PTX for sm_100a), bounded waits, bf16 unpacking, work queues.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/boost.h"

namespace boostk {

constexpr uint32_t kPageBytes = BOOST_PAGE_BYTES;

// Words at the start of every kernel workspace.
enum : uint32_t {
  kWsStatus = 0,    // sticky error bits, see kErr*
  kWsHostNext = 1,  // next item of the host-tier queue
  kWsHbmNext = 2,   // next item of the HBM queue
  kWsDone = 3,      // threadblocks that have finished (self-reset of the words above)
  // Host-written, read-only for the kernels (both 0 in normal use):
  kWsWaitLimit = 4,     // bounded waits give up after this many cycles instead of kWaitLimitCycles
  kWsSkipArrivals = 5,  // honoured only with a non-zero kWsWaitLimit: threadblocks [0, n) leave out their
                        // phase-boundary arrival, so that the others' waits run out (test of the wind-down)
  kWsLog = 6,           // two words: device address of a schedule log (boost_schedule_log_*), 0 = none
  kWsBar = 8,       // a weight product launched alone keeps its two grid-wide counters here
  kWsHeaderWords = 16
};
enum : uint32_t { kErrWaitTimeout = 1u, kErrBadIndex = 2u };

// A wait that cannot hang the GPU: give up after about a second and record it.
constexpr long long kWaitLimitCycles = 2000000000LL;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return (uint32_t)__cvta_generic_to_shared(p);
}

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void fence_barrier_init() {
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait on an mbarrier phase.  On a timeout the error is recorded in *status and the
// caller simply carries on (its data is wrong, the host sees the status word), so that no
// thread is left behind waiting for an arrival that never comes.
// Returns false when it gave up.
// `status` is the first word of the kernel's workspace header: the limit is read from the
// header (kWsWaitLimit; 0 = kWaitLimitCycles) only once the barrier has not completed at the
// first try, so callers carry no limit around.
__device__ __forceinline__ long long wait_limit_of(const uint32_t* ws) {
  const uint32_t v = __ldg(ws + kWsWaitLimit);
  return v ? (long long)v : kWaitLimitCycles;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t* status) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long limit = wait_limit_of(status);
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) {
      atomicOr(status, kErrWaitTimeout);
      return false;
    }
  }
  return true;
}

// Bulk asynchronous copy global -> shared through the TMA unit; completion is counted in
// bytes on `bar`.  All three addresses 16-byte aligned, bytes a multiple of 16.
__device__ __forceinline__ void bulk_copy_g2s(void* dst_smem, const void* src, uint32_t bytes,
                                              uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
          smem_u32(dst_smem)),
      "l"(src), "r"(bytes), "r"(smem_u32(bar))
      : "memory");
}

// Tiled (tensor-map) copy global -> shared through the TMA unit: the box of the map at
// coordinates (c0 = innermost, in elements; c1 = row); completion is counted in bytes on `bar`.
// c0 x element size must be a multiple of 16 bytes; elements outside the tensor arrive as zeros.
__device__ __forceinline__ void tma_load_2d(void* dst_smem, const void* tensor_map, int32_t c0, int32_t c1, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
          smem_u32(dst_smem)),
      "l"(tensor_map), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
      : "memory");
}

// Brings a tensor map into the descriptor cache ahead of its first use.
__device__ __forceinline__ void tma_prefetch_map(const void* tensor_map) {
  asm volatile("prefetch.tensormap [%0];" ::"l"(tensor_map) : "memory");
}

// Orders this thread's earlier generic-proxy view of memory (what it has acquired from other
// threads' ordinary stores) before its later copies through the asynchronous proxy (TMA).
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// 16-byte asynchronous copy through the load/store path (works on any mapped address,
// host-pinned pages included); src_bytes = 0 writes zeros.
__device__ __forceinline__ void cp_async_16(void* dst_smem, const void* src, uint32_t src_bytes) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(smem_u32(dst_smem)), "l"(src),
               "r"(src_bytes)
               : "memory");
}
// Arrive on `bar` once all cp.async issued so far by this thread have landed (the arrival
// is one of the barrier's expected arrivals).
__device__ __forceinline__ void cp_async_arrive_noinc(uint64_t* bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() { asm volatile("cp.async.wait_all;" ::: "memory"); }

// Programmatic dependent launch: let the next kernel of the stream start its prologue now,
// and wait (before touching anything an earlier kernel produces or still reads) until all
// earlier kernels have completed and their writes are visible.  No-ops when the kernel was
// launched without the programmatic-serialization attribute.
__device__ __forceinline__ void pdl_launch_dependents() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// Wait until the counter at `ctr` (raised once by every threadblock of the grid) reaches
// `target`: the grid barrier between two phases of one persistent kernel.  All threadblocks of
// such a kernel are resident at once (the host sizes the grid from the occupancy), so the
// counter always gets there; the wait is bounded all the same and records a timeout.
// Returns false when it gave up.  `status`: first word of the workspace header (see mbar_wait).
__device__ __forceinline__ bool grid_counter_wait(const uint32_t* ctr, uint32_t target, uint32_t* status) {
  const long long limit = wait_limit_of(status);
  const long long t0 = clock64();
  for (;;) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
    if (v >= target) return true;
    if (clock64() - t0 > limit) {
      atomicOr(status, kErrWaitTimeout);
      return false;
    }
    __nanosleep(32);
  }
}

// Named barrier among n_threads threads that also ORs a predicate over them: every participant
// gets the same answer.
__device__ __forceinline__ bool named_barrier_or(uint32_t id, uint32_t n_threads, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.b32 p, %3, 0;\n\t"
      "bar.red.or.pred q, %1, %2, p;\n\t"
      "selp.u32 %0, 1, 0, q;\n\t}"
      : "=r"(r)
      : "r"(id), "r"(n_threads), "r"((uint32_t)pred)
      : "memory");
  return r != 0u;
}

// Test hook (see kWsSkipArrivals): how many threadblocks leave out their phase-boundary arrival.
__device__ __forceinline__ uint32_t skip_arrivals_of(const uint32_t* ws) {
  return __ldg(ws + kWsWaitLimit) ? __ldg(ws + kWsSkipArrivals) : 0u;
}

__device__ __forceinline__ void named_barrier_sync(uint32_t id, uint32_t n_threads) {
  asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n_threads) : "memory");
}

__device__ __forceinline__ uint4 ld_stream_16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// ---- 5th-generation tensor cores (tcgen05): accumulators live in tensor memory (TMEM), the
// operands are read from shared memory through 64-bit matrix descriptors, one thread issues.

// Allocate n_cols (a power of two >= 32) TMEM columns; the base address lands in *dst_smem.
// Executed by one whole warp, which also frees them with tmem_dealloc.
__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t n_cols) {
  asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(n_cols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t n_cols) {
  asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(n_cols) : "memory");
}
__device__ __forceinline__ void tc_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Writes made through the load/store path (cp.async, st.shared) become visible to the
// asynchronous proxy, through which the tensor cores read shared memory.
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 tile in the 128-byte swizzle: rows of
// 128 bytes (64 values of k), 16-byte chunk c of row r stored at chunk c ^ (r & 7), groups of
// 8 rows 1024 bytes apart, tile base 1024-byte aligned.  `addr` may be advanced by 32 bytes
// per 16 values of k inside the row.
__device__ __forceinline__ uint64_t umma_desc_k_sw128(uint32_t addr) {
  return (uint64_t)((addr >> 4) & 0x3FFFu)   // start address
         | ((uint64_t)1 << 16)               // leading byte offset (unused inside one swizzle row): 16 B
         | ((uint64_t)(1024 >> 4) << 32)     // stride byte offset: 8-row groups 1024 B apart
         | ((uint64_t)1 << 46)               // descriptor version of this architecture
         | ((uint64_t)2 << 61);              // layout type: 128-byte swizzle
}
// Instruction descriptor: D fp32 = A bf16 (K-major, M rows) x B bf16 (K-major, N rows)^T.
__device__ __forceinline__ constexpr uint32_t umma_idesc_bf16_f32(uint32_t M, uint32_t N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((N >> 3) << 17) | ((M >> 4) << 24);
}
// D[tmem] (+)= A[smem] * B[smem]^T, K = 16; accumulate = 0 overwrites D.
__device__ __forceinline__ void umma_bf16(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, {%5, %5, %5, %5}, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate), "r"(0u)
      : "memory");
}
// Arrive (count one) on `bar` when every MMA this thread has issued so far has completed.
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar))
               : "memory");
}
// 16 consecutive fp32 columns of this thread's TMEM lane (lane = 32 * (warp % 4) + lane id).
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// kN = 16 or 32 consecutive columns of this warp's 32 TMEM lanes.
template <uint32_t kN>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, float (&v)[kN]) {
  static_assert(kN == 16 || kN == 32, "16 or 32 columns");
  uint32_t r[kN];
#pragma unroll
  for (uint32_t h = 0; h < kN / 16; ++h)
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[16 * h + 0]), "=r"(r[16 * h + 1]), "=r"(r[16 * h + 2]), "=r"(r[16 * h + 3]), "=r"(r[16 * h + 4]),
          "=r"(r[16 * h + 5]), "=r"(r[16 * h + 6]), "=r"(r[16 * h + 7]), "=r"(r[16 * h + 8]), "=r"(r[16 * h + 9]),
          "=r"(r[16 * h + 10]), "=r"(r[16 * h + 11]), "=r"(r[16 * h + 12]), "=r"(r[16 * h + 13]), "=r"(r[16 * h + 14]),
          "=r"(r[16 * h + 15])
        : "r"(taddr + 16 * h)
        : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (uint32_t i = 0; i < kN; ++i) v[i] = __uint_as_float(r[i]);
}

// Two bf16 packed in a 32-bit word -> two floats (bf16 is the top half of an fp32).
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ void ldmatrix_x4(uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3,
                                            uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(smem_addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3, uint32_t smem_addr) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3)
               : "r"(smem_addr));
}
// D (16x8, fp32) += A (16x16, bf16, row) * B (16x8, bf16, col)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                               uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
      "{%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// ---- Schedule log (opt-in; see boost_schedule_stats).  The host puts the device address of a
// log buffer into words kWsLog, kWsLog + 1 of a kernel's workspace header; the kernel then
// appends one record per work item: who streamed how many bytes of which tier, from the moment
// its first byte was requested to the moment its last byte had been consumed.  Buffer layout:
// uint64 count (records claimed so far, may exceed the capacity), uint64 capacity, two unused
// uint64, then the records.
struct SchedRecord {
  uint32_t kind_phase;   // BOOST_SCHED_KIND_* | phase of a chain << 8
  uint32_t cta_warp;     // threadblock | warp << 24
  uint32_t bytes;        // bytes of the item
  uint32_t host_bytes;   // of which from host-tier pages
  unsigned long long t_request;    // global timer, ns
  unsigned long long t_consumed;   // global timer, ns; 0 while the item is in flight
};
constexpr uint32_t kNoRecord = 0xFFFFFFu;   // record indices travel in 24 bits

__device__ __forceinline__ unsigned long long global_time_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ unsigned long long* sched_log_of(const uint32_t* ws) {
  return reinterpret_cast<unsigned long long*>(*reinterpret_cast<const unsigned long long*>(ws + kWsLog));
}
// Claim a record and fill in everything but the end time.  One thread.  Returns kNoRecord when
// there is no log or it is full.
__device__ __forceinline__ uint32_t sched_log_begin(unsigned long long* log, uint32_t kind_phase, uint32_t cta_warp,
                                                    uint32_t bytes, uint32_t host_bytes) {
  if (!log) return kNoRecord;
  const unsigned long long idx = atomicAdd(log, 1ull);
  if (idx >= log[1] || idx >= kNoRecord) return kNoRecord;
  SchedRecord* r = reinterpret_cast<SchedRecord*>(log + 4) + idx;
  r->kind_phase = kind_phase; r->cta_warp = cta_warp; r->bytes = bytes; r->host_bytes = host_bytes;
  r->t_consumed = 0ull;
  r->t_request = global_time_ns();
  return (uint32_t)idx;
}
__device__ __forceinline__ void sched_log_end(unsigned long long* log, uint32_t idx) {
  if (log && idx != kNoRecord) (reinterpret_cast<SchedRecord*>(log + 4) + idx)->t_consumed = global_time_ns();
}

// Two work queues: threadblocks with `host_first` take items of the host-tier queue
// [0, n_host_items) until it is empty and then help with the HBM queue
// [n_host_items, n_items); the others do the reverse.  Every threadblock owns its first
// item by position (no atomic on the critical path of a short kernel); later items come from
// two atomic counters in `ws`.  Returns the queue position or 0xFFFFFFFF when both queues are
// empty.  Called by one thread per threadblock.
struct TierQueues {
  uint32_t* ws;
  uint32_t n_host_items, n_hbm_items;
  uint32_t host_base, hbm_base;     // items handed out by position
  uint32_t first_host, first_hbm;   // this threadblock's own first items (or none)
  bool host_first;
  bool host_open, hbm_open;
  __device__ __forceinline__ void init(uint32_t* workspace, uint32_t n_host, uint32_t n_all, uint32_t n_host_ctas,
                                       uint32_t cta, uint32_t n_ctas) {
    ws = workspace; n_host_items = n_host; n_hbm_items = n_all - n_host;
    host_first = cta < n_host_ctas;
    host_base = min(n_host_ctas, n_host_items);
    hbm_base = min(n_ctas - n_host_ctas, n_hbm_items);
    first_host = (host_first && cta < n_host_items) ? cta : 0xFFFFFFFFu;
    first_hbm = (!host_first && cta - n_host_ctas < n_hbm_items) ? n_host_items + cta - n_host_ctas : 0xFFFFFFFFu;
    host_open = n_host_items > 0; hbm_open = n_hbm_items > 0;
  }
  __device__ __forceinline__ uint32_t take_host() {
    if (first_host != 0xFFFFFFFFu) { const uint32_t i = first_host; first_host = 0xFFFFFFFFu; return i; }
    if (!host_open) return 0xFFFFFFFFu;
    const uint32_t i = host_base + atomicAdd(ws + kWsHostNext, 1u);
    if (i < n_host_items) return i;
    host_open = false;
    return 0xFFFFFFFFu;
  }
  __device__ __forceinline__ uint32_t take_hbm() {
    if (first_hbm != 0xFFFFFFFFu) { const uint32_t i = first_hbm; first_hbm = 0xFFFFFFFFu; return i; }
    if (!hbm_open) return 0xFFFFFFFFu;
    const uint32_t i = hbm_base + atomicAdd(ws + kWsHbmNext, 1u);
    if (i < n_hbm_items) return n_host_items + i;
    hbm_open = false;
    return 0xFFFFFFFFu;
  }
  __device__ __forceinline__ uint32_t next() {
    uint32_t q = host_first ? take_host() : take_hbm();
    if (q == 0xFFFFFFFFu) q = host_first ? take_hbm() : take_host();
    return q;
  }
  // Last threadblock out puts the queue words back to zero for the next launch.
  __device__ __forceinline__ void finish(uint32_t n_ctas) {
    __threadfence();
    const uint32_t d = atomicAdd(ws + kWsDone, 1u);
    if (d == n_ctas - 1) {
      ws[kWsHostNext] = 0; ws[kWsHbmNext] = 0; ws[kWsDone] = 0;
      __threadfence();
    }
  }
};

}  // namespace boostk
