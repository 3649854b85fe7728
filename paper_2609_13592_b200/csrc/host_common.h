// Host-side helpers shared by the .cu files: CUDA error capture, device facts.
#pragma once
#include <cuda_runtime.h>

#include "../../include/boost.h"

namespace boosth {

void set_last_cuda_error(cudaError_t e);

// Number of SMs of the current device (cached per device); 0 on failure.
int sm_count();

// What the launch paths set up once per device (function attributes, occupancy) is kept in
// arrays of this many slots indexed by the current device's ordinal.
constexpr int kMaxDevices = 64;
// Ordinal of the current device, or -1 (no device, or an ordinal beyond kMaxDevices).
int device_slot();

inline int check(cudaError_t e) {
  if (e == cudaSuccess) return BOOST_OK;
  set_last_cuda_error(e);
  return BOOST_ERR_CUDA;
}

// Launch a kernel of the decode chain with programmatic stream serialization allowed: it may
// start while its predecessor drains, and waits inside (griddepcontrol.wait) before it touches
// anything the predecessor produces.
template <typename... KArgs, typename... Args>
inline int launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t stream,
                          Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return check(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

// The same for a kernel whose threadblocks form clusters of cluster_x along x.
template <typename... KArgs, typename... Args>
inline int launch_chained_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, unsigned cluster_x,
                                  cudaStream_t stream, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return check(cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...));
}

// boost_gemv_tiered with a private set of queue words (16 zeroed uint32 that no other launch
// in flight uses): the kernel may then take work and stream weights before its predecessor
// has finished.  queue_words = nullptr gives the public behaviour.  header_row_tiles: size the
// counter area at the head of the workspace for this many row tiles (0 = the product's own),
// so that products of different shapes that share one workspace keep their counters clear of
// each other's partial sums.
int gemv_tiered_launch(const void* const* w_page_ptr, const uint32_t* w_order, size_t n_pages,
                       size_t n_host_pages, uint32_t N, uint32_t K, const void* x, uint32_t M_b, void* y,
                       int y_dtype, const void* residual, void* workspace, size_t workspace_bytes,
                       const boost_gemv_epilogue_t* epilogue, uint32_t* queue_words, uint32_t header_row_tiles,
                       void* stream, uint32_t* extra_launches = nullptr);

// A chain of 1..4 products in one launch (see boost_gemv_tiered_chain).  sync_words: 16 zeroed
// uint32 per product (its queue words) followed by 16 more (phase counters).  early = true: the
// words are private to this launch among the launches in flight (the caller rotates through
// several sets), so the weight warps may take work before the preceding kernel has finished;
// early = false: the preceding kernel on the stream may have used the same words.
// extra_launches (both calls, optional): incremented for every kernel launched beyond the first
// (the combine of the last product when it has a kernel of its own).
int gemv_chain_launch(const boost_gemv_call_t* calls, uint32_t n_calls, uint32_t M_b, void* workspace,
                      size_t workspace_bytes, uint32_t* sync_words, bool early, uint32_t header_row_tiles,
                      void* stream, uint32_t* extra_launches = nullptr);

// Bytes of the counter area for n_row_tiles row tiles, and of the partial sums of one product.
size_t gemv_header_bytes(uint32_t n_row_tiles);
size_t gemv_partial_bytes(uint32_t N, uint32_t K, uint32_t M_b);

// Launch check: picks up configuration errors of the launch just made.
inline int check_launch() { return check(cudaGetLastError()); }

// boost_paged_attn_decode_tiered with the choice of who plans the launch (see kernels_attn.cu).
enum { kAttnPlanOwn = 0, kAttnPlanOnly = 1, kAttnPlanReuse = 2 };
int paged_attn_launch(const void* q, const void* const* k_page_ptr, const void* const* v_page_ptr, const uint8_t* kv_tier,
                      size_t n_kv_pages, uint32_t n_pool_blocks, const int32_t* block_table, uint32_t max_blocks,
                      const int32_t* ctx_lens, uint32_t B, uint32_t Hq, uint32_t Hkv, uint32_t D, float scale, void* workspace,
                      size_t workspace_bytes, void* out, void* stream, int plan);

}  // namespace boosth
