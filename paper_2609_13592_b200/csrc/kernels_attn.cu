// Tiered paged decode attention (split-KV) over the KV cache of a boost_kv_pool, and the
// copies that move a logical [Hkv][N][16][D] cache into and out of its pages.
//
// A threadblock handles one KV-head chunk run: sequence b, KV head g, blocks
// [8 s, 8 s + 8) of the sequence (Sec. 3.3: attention threadblocks work on KV head
// chunks).  All K and V chunks of the run are requested at once - 4 KiB bulk copies through
// the TMA unit for HBM pages, 16-byte cp.async fans for host pages - so up to 64 KiB per
// threadblock are in flight; four warps then take blocks as they land, compute
// S = q K^T and O += P V with bf16 tensor-core MMAs (the query heads of the group are the
// rows of a 16-row tile) and an online softmax, merge through shared memory, and the last
// split of a (b, g) pair to finish combines all splits in split order.
// Threadblocks are numbered so that the heads held on the host tier start first.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "device_common.cuh"
#include "host_common.h"

namespace {

using namespace boostk;

constexpr uint32_t kD = 128;
constexpr uint32_t kTok = BOOST_KV_BLOCK_TOKENS;         // 16
constexpr uint32_t kChunkBytes = kTok * kD * 2;          // 4 KiB
constexpr uint32_t kChunksPerPage = kPageBytes / kChunkBytes;
constexpr uint32_t kSplitBlocks = 8;                     // blocks per threadblock
constexpr uint32_t kAttnWarps = 4;
constexpr uint32_t kAttnThreads = kAttnWarps * 32;
constexpr uint32_t kMaxGroup = 16;

struct AttnParams {
  const __nv_bfloat16* q;
  const void* const* k_page_ptr;
  const void* const* v_page_ptr;
  uint32_t first_host_page;   // pages >= this are host pages (linear placement)
  uint32_t n_pool_blocks;
  const int32_t* block_table;
  uint32_t max_blocks;
  const int32_t* ctx_lens;
  uint32_t B, Hq, Hkv, group, max_splits;
  float scale_log2e;
  uint32_t* ws;        // header + one counter per (b, g)
  float* part_ml;      // [B][Hq][max_splits][2]
  float* part_o;       // [B][Hq][max_splits][128]
  __nv_bfloat16* out;
};

__global__ void __launch_bounds__(kAttnThreads, 3) paged_attn_kernel(const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  uint8_t* k_sm = smem;                                   // [kSplitBlocks][4 KiB]
  uint8_t* v_sm = smem + kSplitBlocks * kChunkBytes;      // [kSplitBlocks][4 KiB]
  float* merge_o = reinterpret_cast<float*>(smem);        // [warps][16][128], reuses k_sm / v_sm
  __shared__ uint64_t bar[kSplitBlocks];
  __shared__ float merge_ml[kAttnWarps][kMaxGroup][2];
  __shared__ uint32_t s_old;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t* status = p.ws + kWsStatus;
  pdl_launch_dependents();
  pdl_wait();   // the newest K/V rows and q come from the kernel just before this one

  // threadblock -> (g, b, split); the highest-numbered KV heads (the host-resident ones
  // under linear placement) come first
  const uint32_t per_head = p.B * p.max_splits;
  const uint32_t g = p.Hkv - 1 - blockIdx.x / per_head;
  const uint32_t b = (blockIdx.x % per_head) / p.max_splits;
  const uint32_t split = blockIdx.x % p.max_splits;
  const uint32_t ctx = (uint32_t)max(p.ctx_lens[b], 0);
  const uint32_t n_blk = (ctx + kTok - 1) / kTok;
  const uint32_t n_splits = n_blk ? (n_blk + kSplitBlocks - 1) / kSplitBlocks : 1;
  if (split >= n_splits) return;
  const uint32_t blk0 = split * kSplitBlocks;
  const uint32_t my_blocks = min(kSplitBlocks, n_blk - min(n_blk, blk0));

  if (tid == 0) {
    for (uint32_t i = 0; i < kSplitBlocks; ++i) mbar_init(&bar[i], kAttnThreads + 1);
    fence_barrier_init();
  }
  __syncthreads();

  // ---- request every chunk of the run
  for (uint32_t i = 0; i < my_blocks; ++i) {
    const int32_t blk = p.block_table[(size_t)b * p.max_blocks + blk0 + i];
    uint32_t lin = g * p.n_pool_blocks + (uint32_t)blk;
    if (blk < 0 || (uint32_t)blk >= p.n_pool_blocks) {   // bad table entry: record, read block 0
      if (tid == 0) atomicOr(status, kErrBadIndex);
      lin = g * p.n_pool_blocks;
    }
    const uint32_t page = lin / kChunksPerPage;
    const size_t in_page = (size_t)(lin % kChunksPerPage) * kChunkBytes;
    const uint8_t* ksrc = static_cast<const uint8_t*>(p.k_page_ptr[page]) + in_page;
    const uint8_t* vsrc = static_cast<const uint8_t*>(p.v_page_ptr[page]) + in_page;
    uint8_t* kdst = k_sm + i * kChunkBytes;
    uint8_t* vdst = v_sm + i * kChunkBytes;
    const bool from_host = page >= p.first_host_page;
    if (from_host) {
#pragma unroll
      for (uint32_t c = tid; c < kChunkBytes / 16; c += kAttnThreads) {
        cp_async_16(kdst + c * 16, ksrc + c * 16, 16u);
        cp_async_16(vdst + c * 16, vsrc + c * 16, 16u);
      }
    }
    cp_async_arrive_noinc(&bar[i]);
    if (tid == 0) {
      if (from_host) {
        mbar_arrive(&bar[i]);
      } else {
        mbar_arrive_expect_tx(&bar[i], 2 * kChunkBytes);
        bulk_copy_g2s(kdst, ksrc, kChunkBytes, &bar[i]);
        bulk_copy_g2s(vdst, vsrc, kChunkBytes, &bar[i]);
      }
    }
  }

  // ---- query rows of this KV group as A fragments (rows >= group are zero)
  const uint32_t r0 = lane >> 2, r1 = r0 + 8, cpair = (lane & 3) * 2;
  uint32_t qa[8][4];
  {
    const uint32_t* q0 = reinterpret_cast<const uint32_t*>(p.q + ((size_t)b * p.Hq + g * p.group + r0) * kD);
    const uint32_t* q1 = reinterpret_cast<const uint32_t*>(p.q + ((size_t)b * p.Hq + g * p.group + r1) * kD);
#pragma unroll
    for (uint32_t ks = 0; ks < 8; ++ks) {
      const uint32_t w0 = (ks * 16 + cpair) / 2, w1 = (ks * 16 + 8 + cpair) / 2;
      qa[ks][0] = r0 < p.group ? q0[w0] : 0u;
      qa[ks][1] = r1 < p.group ? q1[w0] : 0u;
      qa[ks][2] = r0 < p.group ? q0[w1] : 0u;
      qa[ks][3] = r1 < p.group ? q1[w1] : 0u;
    }
  }

  float o[16][4];
#pragma unroll
  for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
  float m_run[2] = {-CUDART_INF_F, -CUDART_INF_F};
  float l_run[2] = {0.f, 0.f};

  for (uint32_t i = warp; i < my_blocks; i += kAttnWarps) {
    mbar_wait(&bar[i], 0u, status);
    const uint32_t kbase = smem_u32(k_sm + i * kChunkBytes);
    const uint32_t vbase = smem_u32(v_sm + i * kChunkBytes);
    // S = q K^T for 16 tokens: two n-tiles of 8 tokens
    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
    {
      const uint32_t tok = (lane & 7) + ((lane >> 4) << 3);
#pragma unroll
      for (uint32_t ks = 0; ks < 8; ++ks) {
        const uint32_t chunk = 2 * ks + ((lane >> 3) & 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4(b0, b1, b2, b3, kbase + tok * 256 + ((chunk ^ (tok & 7)) << 4));
        mma_bf16_16816(s[0], qa[ks], b0, b1);
        mma_bf16_16816(s[1], qa[ks], b2, b3);
      }
    }
    // mask the tail of the last block, scale into the log2 domain
    const uint32_t tok_base = (blk0 + i) * kTok;
#pragma unroll
    for (int nj = 0; nj < 2; ++nj)
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        const uint32_t t = tok_base + nj * 8 + cpair + (r & 1);
        s[nj][r] = (t < ctx) ? s[nj][r] * p.scale_log2e : -CUDART_INF_F;
      }
    // online softmax, rows r0 (regs 0,1) and r1 (regs 2,3)
    float p_frag[2][4];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      float mx = fmaxf(fmaxf(s[0][2 * h], s[0][2 * h + 1]), fmaxf(s[1][2 * h], s[1][2 * h + 1]));
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 2));
      const float m_new = fmaxf(m_run[h], mx);           // finite: a block has a valid token
      const float corr = exp2f(m_run[h] - m_new);        // exp2(-inf) = 0 on the first block
      float sum = 0.f;
#pragma unroll
      for (int nj = 0; nj < 2; ++nj)
#pragma unroll
        for (int e = 0; e < 2; ++e) {
          const float pv = exp2f(s[nj][2 * h + e] - m_new);
          p_frag[nj][2 * h + e] = pv;
          sum += pv;
        }
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 1);
      sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 2);
      l_run[h] = l_run[h] * corr + sum;
      m_run[h] = m_new;
#pragma unroll
      for (int nd = 0; nd < 16; ++nd) { o[nd][2 * h] *= corr; o[nd][2 * h + 1] *= corr; }
    }
    // P as the A operand (k = 16 tokens).  A single bf16 rounding of P would put an error of
    // 2^-9 * sqrt(sum p^2 v^2) on every output, far above 1 % of the outputs that are close
    // to zero; P is therefore split into three bf16 terms (hi + mid + lo carry 24 bits) and
    // multiplied term by term - the tensor pipe has the headroom, the kernel is HBM-bound.
    uint32_t pa[3][4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int nj = i >> 1, r = (i & 1) * 2;
      float x0 = p_frag[nj][r], x1 = p_frag[nj][r + 1];
#pragma unroll
      for (int t = 0; t < 3; ++t) {
        const __nv_bfloat162 h = __floats2bfloat162_rn(x0, x1);
        pa[t][i] = *reinterpret_cast<const uint32_t*>(&h);
        x0 -= __low2float(h);
        x1 -= __high2float(h);
      }
    }
    {
      const uint32_t mi = lane >> 3;
      const uint32_t tok = (lane & 7) + ((mi & 1) << 3);
#pragma unroll
      for (uint32_t jj = 0; jj < 8; ++jj) {
        const uint32_t chunk = 2 * jj + (mi >> 1);
        uint32_t b0, b1, b2, b3;
        ldmatrix_x4_trans(b0, b1, b2, b3, vbase + tok * 256 + ((chunk ^ (tok & 7)) << 4));
#pragma unroll
        for (int t = 2; t >= 0; --t) {
          mma_bf16_16816(o[2 * jj], pa[t], b0, b1);
          mma_bf16_16816(o[2 * jj + 1], pa[t], b2, b3);
        }
      }
    }
  }

  // ---- merge the warps (each holds a disjoint set of blocks) through shared memory;
  // the merge buffer overlays the K/V stages, so every warp must be done with them first
  __syncthreads();
  if ((lane & 3) == 0) {
    if (r0 < kMaxGroup) { merge_ml[warp][r0][0] = m_run[0]; merge_ml[warp][r0][1] = l_run[0]; }
    if (r1 < kMaxGroup) { merge_ml[warp][r1][0] = m_run[1]; merge_ml[warp][r1][1] = l_run[1]; }
  }
#pragma unroll
  for (int nd = 0; nd < 16; ++nd) {
    const uint32_t d = nd * 8 + cpair;
    if (r0 < p.group) *reinterpret_cast<float2*>(merge_o + ((size_t)warp * kMaxGroup + r0) * kD + d) = make_float2(o[nd][0], o[nd][1]);
    if (r1 < p.group) *reinterpret_cast<float2*>(merge_o + ((size_t)warp * kMaxGroup + r1) * kD + d) = make_float2(o[nd][2], o[nd][3]);
  }
  __syncthreads();

  const bool single = (n_splits == 1);
  // thread d of 128 owns output column d; loop over the query heads of the group
  for (uint32_t r = 0; r < p.group; ++r) {
    float m_all = -CUDART_INF_F;
#pragma unroll
    for (uint32_t w = 0; w < kAttnWarps; ++w) m_all = fmaxf(m_all, merge_ml[w][r][0]);
    float acc = 0.f, l_all = 0.f;
#pragma unroll
    for (uint32_t w = 0; w < kAttnWarps; ++w) {
      const float mw = merge_ml[w][r][0];
      const float f = (mw == -CUDART_INF_F) ? 0.f : exp2f(mw - m_all);
      acc += f * merge_o[((size_t)w * kMaxGroup + r) * kD + tid];
      l_all += f * merge_ml[w][r][1];
    }
    const uint32_t hq = g * p.group + r;
    if (single) {
      const float v = l_all > 0.f ? acc / l_all : 0.f;
      p.out[((size_t)b * p.Hq + hq) * kD + tid] = __float2bfloat16_rn(v);
    } else {
      const size_t slot = ((size_t)b * p.Hq + hq) * p.max_splits + split;
      __stcg(p.part_o + slot * kD + tid, acc);
      if (tid == 0) { __stcg(p.part_ml + slot * 2, m_all); __stcg(p.part_ml + slot * 2 + 1, l_all); }
    }
  }
  if (single) return;

  // ---- the last split of (b, g) to arrive combines all splits, in split order
  uint32_t* cnt = p.ws + kWsHeaderWords + b * p.Hkv + g;
  __threadfence();
  __syncthreads();
  if (tid == 0) s_old = atomicAdd(cnt, 1u);
  __syncthreads();
  if (s_old != n_splits - 1) return;
  __threadfence();
  for (uint32_t r = 0; r < p.group; ++r) {
    const uint32_t hq = g * p.group + r;
    const size_t slot0 = ((size_t)b * p.Hq + hq) * p.max_splits;
    float m_all = -CUDART_INF_F;
    for (uint32_t sp = 0; sp < n_splits; ++sp) m_all = fmaxf(m_all, __ldcg(p.part_ml + (slot0 + sp) * 2));
    float acc = 0.f, l_all = 0.f;
    for (uint32_t sp = 0; sp < n_splits; ++sp) {
      const float f = exp2f(__ldcg(p.part_ml + (slot0 + sp) * 2) - m_all);
      acc += f * __ldcg(p.part_o + (slot0 + sp) * kD + tid);
      l_all += f * __ldcg(p.part_ml + (slot0 + sp) * 2 + 1);
    }
    p.out[((size_t)b * p.Hq + hq) * kD + tid] = __float2bfloat16_rn(l_all > 0.f ? acc / l_all : 0.f);
  }
  if (tid == 0) *cnt = 0;
}

// Logical cache [Hkv][N][16][D] (contiguous, bf16) <-> pages.  Inside a 4 KiB chunk token t
// occupies 256 bytes at t*256 and its 16-byte piece c (8 values of d) sits at position
// c ^ (t & 7), so tensor-core loads of 8 consecutive tokens hit distinct banks.
__global__ void __launch_bounds__(256)
kv_copy_kernel(uint4* __restrict__ flat, const void* const* __restrict__ page_ptr, size_t n_vec,
               int to_pages) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_vec; i += stride) {
    const size_t chunk = i / (kChunkBytes / 16);
    const uint32_t in_chunk = (uint32_t)(i % (kChunkBytes / 16));
    const uint32_t t = in_chunk >> 4, c = in_chunk & 15;
    const size_t off = chunk * kChunkBytes + t * 256 + ((c ^ (t & 7)) << 4);
    uint4* in_page = reinterpret_cast<uint4*>(
        static_cast<uint8_t*>(const_cast<void*>(page_ptr[off / kPageBytes])) + off % kPageBytes);
    if (to_pages) *in_page = flat[i];
    else flat[i] = *in_page;
  }
}

int launch_kv_copy(void* flat, uint32_t n_kv_heads, uint32_t n_pool_blocks, uint32_t D,
                   const void* const* page_ptr, size_t n_pages, void* stream, int to_pages) {
  if (!flat || !page_ptr) return BOOST_ERR_INVALID;
  if (D != kD) return BOOST_ERR_UNSUPPORTED;
  if (((uintptr_t)flat % 16) != 0) return BOOST_ERR_ALIGN;
  const size_t bytes = (size_t)n_kv_heads * n_pool_blocks * kChunkBytes;
  if (bytes == 0) return BOOST_OK;
  if ((bytes + kPageBytes - 1) / kPageBytes > n_pages) return BOOST_ERR_CAPACITY;
  const size_t n_vec = bytes / 16;
  size_t blocks = (n_vec + 255) / 256;
  const size_t cap = (size_t)(boosth::sm_count() > 0 ? boosth::sm_count() : 148) * 16;
  if (blocks > cap) blocks = cap;
  kv_copy_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>((uint4*)flat, page_ptr, n_vec, to_pages);
  return boosth::check_launch();
}

size_t attn_header_bytes(uint32_t B, uint32_t Hkv_upper) {
  return ((size_t)(kWsHeaderWords + (size_t)B * Hkv_upper) * 4 + 255) / 256 * 256;
}

}  // namespace

extern "C" int boost_kv_scatter(const void* src, uint32_t n_kv_heads, uint32_t n_pool_blocks,
                                uint32_t D, const void* const* page_ptr, size_t n_pages, void* stream) {
  return launch_kv_copy(const_cast<void*>(src), n_kv_heads, n_pool_blocks, D, page_ptr, n_pages, stream, 1);
}

extern "C" int boost_kv_gather(void* dst, uint32_t n_kv_heads, uint32_t n_pool_blocks, uint32_t D,
                               const void* const* page_ptr, size_t n_pages, void* stream) {
  return launch_kv_copy(dst, n_kv_heads, n_pool_blocks, D, page_ptr, n_pages, stream, 0);
}

extern "C" size_t boost_paged_attn_workspace_bytes(uint32_t B, uint32_t Hq, uint32_t D,
                                                   uint32_t max_blocks) {
  if (D != kD || B == 0 || Hq == 0) return 0;
  const size_t max_splits = max_blocks ? (max_blocks + kSplitBlocks - 1) / kSplitBlocks : 1;
  // counters are per (b, KV head); Hq bounds the number of KV heads
  return attn_header_bytes(B, Hq) + (size_t)B * Hq * max_splits * (2 + kD) * 4;
}

extern "C" int boost_paged_attn_decode_tiered(const void* q, const void* const* k_page_ptr,
                                              const void* const* v_page_ptr, const uint8_t* kv_tier,
                                              size_t n_kv_pages, uint32_t n_pool_blocks,
                                              const int32_t* block_table, uint32_t max_blocks,
                                              const int32_t* ctx_lens, uint32_t B, uint32_t Hq,
                                              uint32_t Hkv, uint32_t D, float scale, void* workspace,
                                              size_t workspace_bytes, void* out, void* stream) {
  if (B == 0) return BOOST_OK;
  if (!q || !k_page_ptr || !v_page_ptr || !block_table || !ctx_lens || !workspace || !out)
    return BOOST_ERR_INVALID;
  if (D != kD) return BOOST_ERR_UNSUPPORTED;
  if (Hkv == 0 || Hq % Hkv != 0 || Hq / Hkv > kMaxGroup || max_blocks == 0 || n_pool_blocks == 0)
    return BOOST_ERR_INVALID;
  if (((uint64_t)n_pool_blocks * kChunkBytes) % kPageBytes != 0) return BOOST_ERR_INVALID;
  if ((uint64_t)Hkv * n_pool_blocks / kChunksPerPage != n_kv_pages) return BOOST_ERR_INVALID;
  if (((uintptr_t)q % 16) || ((uintptr_t)out % 16) || ((uintptr_t)workspace % 256)) return BOOST_ERR_ALIGN;
  if (workspace_bytes < boost_paged_attn_workspace_bytes(B, Hq, D, max_blocks)) return BOOST_ERR_CAPACITY;
  // linear placement: host pages are the tail of the range
  uint32_t first_host = (uint32_t)n_kv_pages;
  if (kv_tier) {
    size_t i = 0;
    while (i < n_kv_pages && kv_tier[i] == BOOST_TIER_HBM) ++i;
    first_host = (uint32_t)i;
    for (; i < n_kv_pages; ++i)
      if (kv_tier[i] != BOOST_TIER_HOST) return BOOST_ERR_UNSUPPORTED;
  }
  AttnParams p;
  p.q = static_cast<const __nv_bfloat16*>(q);
  p.k_page_ptr = k_page_ptr;
  p.v_page_ptr = v_page_ptr;
  p.first_host_page = first_host;
  p.n_pool_blocks = n_pool_blocks;
  p.block_table = block_table;
  p.max_blocks = max_blocks;
  p.ctx_lens = ctx_lens;
  p.B = B; p.Hq = Hq; p.Hkv = Hkv; p.group = Hq / Hkv;
  p.max_splits = (max_blocks + kSplitBlocks - 1) / kSplitBlocks;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.ws = static_cast<uint32_t*>(workspace);
  uint8_t* base = static_cast<uint8_t*>(workspace) + attn_header_bytes(B, Hq);
  p.part_ml = reinterpret_cast<float*>(base);
  p.part_o = p.part_ml + (size_t)B * Hq * p.max_splits * 2;
  p.out = static_cast<__nv_bfloat16*>(out);
  static_assert(2 * kSplitBlocks * kChunkBytes >= kAttnWarps * kMaxGroup * kD * 4, "merge buffer overlays K/V");
  const size_t smem = 2 * kSplitBlocks * kChunkBytes + 128;
  static bool configured = false;
  if (!configured) {
    const int rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    if (rc != BOOST_OK) return rc;
    configured = true;
  }
  const uint64_t grid = (uint64_t)Hkv * B * p.max_splits;
  if (grid > 0x7FFFFFFFull) return BOOST_ERR_INVALID;
  return boosth::launch_chained(paged_attn_kernel, dim3((unsigned)grid), dim3(kAttnThreads), smem,
                                (cudaStream_t)stream, p);
}
