// Streaming kernels over paged buffers: the tiered stream-reduce (the "add" micro-benchmark
// of Sec. 2.6 with a sum as its compute) and the page scatter / gather copies used when a
// tensor is materialised into its tiers.
#include <cuda_runtime.h>

#include <mutex>

#include "device_common.cuh"
#include "host_common.h"

namespace boosth {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(cudaError_t e) { g_last_cuda_error = (int)e; }

int device_slot() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return -1;
  return dev;
}

int sm_count() {
  static int cached[kMaxDevices] = {0};
  const int dev = device_slot();
  if (dev < 0) return 0;
  if (cached[dev] == 0) {
    int n = 0;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return 0;
    cached[dev] = n;
  }
  return cached[dev];
}

}  // namespace boosth

extern "C" int boost_last_cuda_error(void) { return boosth::g_last_cuda_error; }

extern "C" int boost_host_device_pointer(void* pinned_host, void** device_ptr_out) {
  if (!pinned_host || !device_ptr_out) return BOOST_ERR_INVALID;
  cudaPointerAttributes attr;
  const int rc = boosth::check(cudaPointerGetAttributes(&attr, pinned_host));
  if (rc != BOOST_OK) return rc;
  if (attr.type != cudaMemoryTypeHost || attr.devicePointer == nullptr) return BOOST_ERR_INVALID;
  *device_ptr_out = attr.devicePointer;
  return BOOST_OK;
}

namespace {

using namespace boostk;

constexpr uint32_t kTileBytes = 128u * 1024u;
constexpr uint32_t kTilesPerPage = kPageBytes / kTileBytes;  // 16
constexpr uint32_t kReduceThreads = 256;
constexpr uint32_t kUnroll = 8;

__device__ __forceinline__ float sum8_bf16(const uint4& v) {
  return ((bf16_lo(v.x) + bf16_hi(v.x)) + (bf16_lo(v.y) + bf16_hi(v.y))) +
         ((bf16_lo(v.z) + bf16_hi(v.z)) + (bf16_lo(v.w) + bf16_hi(v.w)));
}

// Persistent grid.  Work item = one 128 KiB tile of one page; items of host pages sit at
// the front of the queue and `n_host_ctas` threadblocks start on them, so the link streams
// from the first cycle while every other threadblock reads HBM (Sec. 3.2: one tier per
// threadblock at a time, an alpha-sized share of the blocks on the host tier).
__global__ void __launch_bounds__(kReduceThreads, 4)
stream_reduce_kernel(const void* const* __restrict__ page_ptr, const uint32_t* __restrict__ order,
                     uint32_t n_pages, uint32_t n_host_pages, float* __restrict__ per_page_sum,
                     uint32_t* __restrict__ ws, uint32_t n_host_ctas) {
  __shared__ uint32_t s_item;
  __shared__ float s_warp[kReduceThreads / 32];
  uint32_t* page_cnt = ws + kWsHeaderWords;
  float* tile_part = reinterpret_cast<float*>(ws + kWsHeaderWords + n_pages);

  TierQueues q;
  q.init(ws, n_host_pages * kTilesPerPage, n_pages * kTilesPerPage, n_host_ctas, blockIdx.x, gridDim.x);
  const uint32_t tid = threadIdx.x;
  unsigned long long* const sched_log = tid == 0 ? sched_log_of(ws) : nullptr;
  uint32_t rec = kNoRecord;

  for (;;) {
    if (tid == 0) {
      s_item = q.next();
      if (s_item != 0xFFFFFFFFu)
        rec = sched_log_begin(sched_log, BOOST_SCHED_KIND_STREAM, blockIdx.x, kTileBytes,
                              s_item < n_host_pages * kTilesPerPage ? kTileBytes : 0u);
    }
    __syncthreads();
    const uint32_t item = s_item;
    if (item == 0xFFFFFFFFu) break;
    const uint32_t page = order[item / kTilesPerPage];
    const uint32_t tile = item % kTilesPerPage;
    const uint4* src = reinterpret_cast<const uint4*>(
        static_cast<const char*>(page_ptr[page]) + (size_t)tile * kTileBytes);
    float acc = 0.f;
    constexpr uint32_t kVecs = kTileBytes / 16;  // 8192
#pragma unroll 1
    for (uint32_t i = tid; i < kVecs; i += kReduceThreads * kUnroll) {
      uint4 v[kUnroll];
#pragma unroll
      for (uint32_t u = 0; u < kUnroll; ++u) v[u] = ld_stream_16(src + i + u * kReduceThreads);
#pragma unroll
      for (uint32_t u = 0; u < kUnroll; ++u) acc += sum8_bf16(v[u]);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if ((tid & 31) == 0) s_warp[tid >> 5] = acc;
    __syncthreads();
    if (tid == 0) {
      sched_log_end(sched_log, rec);
      float t = 0.f;
#pragma unroll
      for (uint32_t w = 0; w < kReduceThreads / 32; ++w) t += s_warp[w];
      __stcg(tile_part + (size_t)page * kTilesPerPage + tile, t);
      __threadfence();
      const uint32_t old = atomicAdd(page_cnt + page, 1u);
      if (old == kTilesPerPage - 1) {  // last tile of this page: combine in tile order
        __threadfence();
        float s = 0.f;
        for (uint32_t k = 0; k < kTilesPerPage; ++k) s += __ldcg(tile_part + (size_t)page * kTilesPerPage + k);
        per_page_sum[page] = s;
        page_cnt[page] = 0;
      }
    }
  }
  if (tid == 0) q.finish(gridDim.x);
}

__global__ void __launch_bounds__(256)
page_copy_kernel(uint4* __restrict__ flat, const void* const* __restrict__ page_ptr, size_t n_vec,
                 int to_pages) {
  constexpr size_t kVecPerPage = kPageBytes / 16;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
    uint4* in_page = reinterpret_cast<uint4*>(const_cast<void*>(page_ptr[i / kVecPerPage])) + (i % kVecPerPage);
    if (to_pages) *in_page = flat[i];
    else flat[i] = *in_page;
  }
}

int launch_page_copy(void* flat, size_t bytes, const void* const* page_ptr, size_t n_pages,
                     void* stream, int to_pages) {
  if (bytes == 0) return BOOST_OK;
  if (!flat || !page_ptr) return BOOST_ERR_INVALID;
  if (bytes % 16 != 0 || ((uintptr_t)flat % 16) != 0) return BOOST_ERR_ALIGN;
  if ((bytes + kPageBytes - 1) / kPageBytes > n_pages) return BOOST_ERR_CAPACITY;
  const size_t n_vec = bytes / 16;
  size_t blocks = (n_vec + 255) / 256;
  const size_t cap = (size_t)(boosth::sm_count() > 0 ? boosth::sm_count() : 148) * 16;
  if (blocks > cap) blocks = cap;
  page_copy_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((uint4*)flat, page_ptr, n_vec, to_pages);
  return boosth::check_launch();
}

}  // namespace

extern "C" int boost_scatter_pages(const void* src, size_t bytes, const void* const* page_ptr,
                                   size_t n_pages, void* stream) {
  return launch_page_copy(const_cast<void*>(src), bytes, page_ptr, n_pages, stream, 1);
}

extern "C" int boost_gather_pages(void* dst, size_t bytes, const void* const* page_ptr,
                                  size_t n_pages, void* stream) {
  return launch_page_copy(dst, bytes, page_ptr, n_pages, stream, 0);
}

extern "C" size_t boost_stream_reduce_workspace_bytes(size_t n_pages) {
  return (size_t)boostk::kWsHeaderWords * 4 + n_pages * 4 + n_pages * kTilesPerPage * 4;
}

extern "C" int boost_stream_reduce_tiered(const void* const* page_ptr, const uint32_t* order,
                                          size_t n_pages, size_t n_host_pages, float* per_page_sum,
                                          void* workspace, size_t workspace_bytes, void* stream) {
  if (n_pages == 0) return BOOST_OK;
  if (!page_ptr || !order || !per_page_sum || !workspace) return BOOST_ERR_INVALID;
  if (n_host_pages > n_pages || n_pages > (0xFFFFFFFFu / kTilesPerPage)) return BOOST_ERR_INVALID;
  if (workspace_bytes < boost_stream_reduce_workspace_bytes(n_pages)) return BOOST_ERR_CAPACITY;
  if ((uintptr_t)workspace % 16 != 0) return BOOST_ERR_ALIGN;
  const int sms = boosth::sm_count();
  if (sms <= 0) return BOOST_ERR_CUDA;
  const size_t n_items = n_pages * kTilesPerPage;
  size_t grid = (size_t)sms * 4;  // four resident threadblocks per SM: full waves
  if (grid > n_items) grid = n_items;
  uint32_t n_host_ctas = 0;
  if (n_host_pages) {
    // enough blocks on the link to keep it full, never more than the host tiles
    size_t want = 16;
    if (want > n_host_pages * kTilesPerPage) want = n_host_pages * kTilesPerPage;
    if (want > grid) want = grid;
    n_host_ctas = (uint32_t)want;
  }
  stream_reduce_kernel<<<(unsigned)grid, kReduceThreads, 0, (cudaStream_t)stream>>>(
      page_ptr, order, (uint32_t)n_pages, (uint32_t)n_host_pages, per_page_sum,
      static_cast<uint32_t*>(workspace), n_host_ctas);
  return boosth::check_launch();
}

// ---------------------------------------------------------------------------------------
// Stream reduce for callers that may not allocate.
//
// Some users of this library cannot obtain scratch memory at call time: a serving engine
// that has handed all of the GPU's memory to its own pools at start-up (a later cudaMalloc
// simply fails), a plug-in that runs under a host framework's allocator and is forbidden
// to go around it, or code on a path where the allocating CUDA calls are not permitted.
// For them the scratch of the stream-reduce kernel lives in a fixed array inside the
// library image.  Every GPU that loads the library carries these kStaticScratchBytes
// until the process exits, which is why the limit is modest.
constexpr size_t kStaticMaxPages = 4096;   // buffers of up to 8 GiB
constexpr size_t kStaticScratchBytes =
    (size_t)boostk::kWsHeaderWords * 4 + kStaticMaxPages * 4 + kStaticMaxPages * kTilesPerPage * 4;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

namespace {

// In host code `g_static_scratch` is only a handle for the runtime, not an address a kernel
// can use; the device address is looked up once per device, with that device current.
void* g_static_scratch_dev[64] = {nullptr};
std::mutex g_static_scratch_mutex;

int static_scratch_address(void** out) {
  int dev = 0;
  int rc = boosth::check(cudaGetDevice(&dev));
  if (rc != BOOST_OK) return rc;
  if (dev < 0 || dev >= 64) return BOOST_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
  if (g_static_scratch_dev[dev] == nullptr) {
    void* p = nullptr;
    rc = boosth::check(cudaGetSymbolAddress(&p, g_static_scratch));
    if (rc != BOOST_OK) return rc;
    if (p == nullptr) return BOOST_ERR_CUDA;
    g_static_scratch_dev[dev] = p;
  }
  *out = g_static_scratch_dev[dev];
  return BOOST_OK;
}

}  // namespace

extern "C" size_t boost_stream_reduce_static_max_pages(void) { return kStaticMaxPages; }

extern "C" int boost_stream_reduce_tiered_static(const void* const* page_ptr, const uint32_t* order,
                                                 size_t n_pages, size_t n_host_pages,
                                                 float* per_page_sum, void* stream) {
  if (n_pages == 0) return BOOST_OK;
  if (!page_ptr || !order || !per_page_sum) return BOOST_ERR_INVALID;
  if (n_host_pages > n_pages) return BOOST_ERR_INVALID;
  if (n_pages > kStaticMaxPages) return BOOST_ERR_CAPACITY;   // larger buffers need the caller's own workspace
  void* scratch = nullptr;
  int rc = static_scratch_address(&scratch);
  if (rc != BOOST_OK) return rc;
  // The array keeps whatever the previous call left.  The queue words and the per-page
  // counters must start at zero; the per-tile partial sums are overwritten before use.
  const size_t counters = (size_t)boostk::kWsHeaderWords * 4 + n_pages * 4;
  rc = boosth::check(cudaMemsetAsync(scratch, 0, counters, (cudaStream_t)stream));
  if (rc != BOOST_OK) return rc;
  return boost_stream_reduce_tiered(page_ptr, order, n_pages, n_host_pages, per_page_sum, scratch,
                                    kStaticScratchBytes, stream);
}
