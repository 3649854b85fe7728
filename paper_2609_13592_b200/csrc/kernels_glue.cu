// Small operators between the weight and attention kernels of a decode step: embedding
// gather, RMSNorm, rotary embedding + KV append into the paged cache, SwiGLU, argmax.
// The paper does not discuss them (weights take about 70 % and attention about 30 % of decode
// time, Sec. 5.4); they move < 0.1 % of the bytes of a step.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>

#include "device_common.cuh"
#include "host_common.h"

namespace {

using namespace boostk;

constexpr uint32_t kD = 128;
constexpr uint32_t kTok = BOOST_KV_BLOCK_TOKENS;
constexpr uint32_t kChunkBytes = kTok * kD * 2;

// ssq (optional): ssq[tile][b] = sum of squares of columns [128 tile, 128 tile + 128) of row b,
// the row statistics a following product needs for its RMS scale.  A tile is 16 vectors of 8
// values, read by 16 consecutive threads and summed with a fixed butterfly.
__global__ void __launch_bounds__(256)
embed_gather_kernel(const uint4* __restrict__ table, uint32_t vocab, uint32_t row_vecs,
                    const int32_t* __restrict__ tokens, uint4* __restrict__ out,
                    float* __restrict__ ssq, uint32_t ssq_stride) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t b = blockIdx.x;
  int32_t t = tokens[b];
  if (t < 0 || (uint32_t)t >= vocab) t = 0;
  const uint32_t n_iter = (row_vecs + blockDim.x - 1) / blockDim.x;
  for (uint32_t it = 0; it < n_iter; ++it) {
    const uint32_t i = it * blockDim.x + threadIdx.x;
    float sq = 0.f;
    if (i < row_vecs) {
      const uint4 v = table[(size_t)t * row_vecs + i];
      out[(size_t)b * row_vecs + i] = v;
      const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) { sq = fmaf(bf16_lo(w[j]), bf16_lo(w[j]), sq); sq = fmaf(bf16_hi(w[j]), bf16_hi(w[j]), sq); }
    }
    if (ssq) {
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 1);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 2);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 4);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 8);
      if (i < row_vecs && (i & 15u) == 0) ssq[(size_t)(i >> 4) * ssq_stride + b] = sq;
    }
  }
}

// out = x * rsqrt(mean(x^2) + eps) * w, one threadblock per row, fp32 arithmetic.
__global__ void __launch_bounds__(256)
rmsnorm_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
               uint32_t hidden, float eps, __nv_bfloat16* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float s_part[8];
  __shared__ float s_scale;
  const size_t row = (size_t)blockIdx.x * hidden;
  float ss = 0.f;
  for (uint32_t i = threadIdx.x * 2; i < hidden; i += blockDim.x * 2) {
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(x + row + i));
    ss = fmaf(v.x, v.x, ss);
    ss = fmaf(v.y, v.y, ss);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) ss += __shfl_xor_sync(0xFFFFFFFFu, ss, o);
  if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (uint32_t k = 0; k < blockDim.x / 32; ++k) t += s_part[k];
    s_scale = rsqrtf(t / (float)hidden + eps);
  }
  __syncthreads();
  const float sc = s_scale;
  for (uint32_t i = threadIdx.x * 2; i < hidden; i += blockDim.x * 2) {
    const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(x + row + i));
    const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(w + i));
    *reinterpret_cast<__nv_bfloat162*>(out + row + i) = __floats2bfloat162_rn(v.x * sc * g.x, v.y * sc * g.y);
  }
}

__device__ __forceinline__ size_t kv_elem_offset(uint32_t head, uint32_t n_pool_blocks, uint32_t blk,
                                                 uint32_t slot, uint32_t d) {
  // byte offset inside the K (or V) tensor: chunk (head, blk), token `slot`, element d
  return ((size_t)head * n_pool_blocks + blk) * kChunkBytes + slot * 256 + ((((d >> 3) ^ (slot & 7))) << 4) +
         (d & 7) * 2;
}

// One thread per (sequence, head, i < D/2).  Query heads: rotate and write to q_out.
// Key heads: rotate and write into the cache at position ctx-1.  Value heads: copy.
// Rotate-half pairing: element i pairs with i + D/2, angle = pos * base^(-2i/D), computed
// in double so that positions of several thousand radians keep full accuracy.
__global__ void __launch_bounds__(256)
rope_kv_append_kernel(const __nv_bfloat16* __restrict__ qkv, __nv_bfloat16* __restrict__ q_out,
                      const void* const* __restrict__ k_page_ptr, const void* const* __restrict__ v_page_ptr,
                      uint32_t n_pool_blocks, const int32_t* __restrict__ block_table, uint32_t max_blocks,
                      const int32_t* __restrict__ ctx_lens, uint32_t B, uint32_t Hq, uint32_t Hkv,
                      double log2_base, uint32_t* __restrict__ status) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t half = kD / 2;
  const uint32_t heads = Hq + 2 * Hkv;
  const uint32_t idx = blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= B * heads * half) return;
  const uint32_t i = idx % half;
  const uint32_t head = (idx / half) % heads;
  const uint32_t b = idx / (half * heads);
  const int32_t ctx = ctx_lens[b];
  if (ctx <= 0) return;
  const uint32_t pos = (uint32_t)ctx - 1;
  const __nv_bfloat16* src = qkv + ((size_t)b * heads + head) * kD;
  const float x1 = __bfloat162float(src[i]), x2 = __bfloat162float(src[i + half]);
  float y1 = x1, y2 = x2;
  if (head < Hq + Hkv) {
    const double inv_freq = exp2(-(double)(2 * i) / (double)kD * log2_base);
    double sn, cs;
    sincos((double)pos * inv_freq, &sn, &cs);
    y1 = (float)((double)x1 * cs - (double)x2 * sn);
    y2 = (float)((double)x2 * cs + (double)x1 * sn);
  }
  if (head < Hq) {
    __nv_bfloat16* dst = q_out + ((size_t)b * Hq + head) * kD;
    dst[i] = __float2bfloat16_rn(y1);
    dst[i + half] = __float2bfloat16_rn(y2);
    return;
  }
  const bool is_k = head < Hq + Hkv;
  const uint32_t kvh = is_k ? head - Hq : head - Hq - Hkv;
  // the table row is max_blocks wide: check the column before reading it
  const int32_t blk = pos / kTok < max_blocks ? block_table[(size_t)b * max_blocks + pos / kTok] : -1;
  if (blk < 0 || (uint32_t)blk >= n_pool_blocks) {
    atomicOr(status, kErrBadIndex);
    return;
  }
  const void* const* pages = is_k ? k_page_ptr : v_page_ptr;
  const uint32_t slot = pos % kTok;
  const size_t o1 = kv_elem_offset(kvh, n_pool_blocks, (uint32_t)blk, slot, i);
  const size_t o2 = kv_elem_offset(kvh, n_pool_blocks, (uint32_t)blk, slot, i + half);
  uint8_t* p1 = static_cast<uint8_t*>(const_cast<void*>(pages[o1 / kPageBytes])) + o1 % kPageBytes;
  uint8_t* p2 = static_cast<uint8_t*>(const_cast<void*>(pages[o2 / kPageBytes])) + o2 % kPageBytes;
  *reinterpret_cast<__nv_bfloat16*>(p1) = __float2bfloat16_rn(y1);
  *reinterpret_cast<__nv_bfloat16*>(p2) = __float2bfloat16_rn(y2);
}

// (cos, sin) of the rotary angles of the new token of every sequence, in double.
__global__ void __launch_bounds__(64)
rope_table_kernel(const int32_t* __restrict__ ctx_lens, double log2_base, float2* __restrict__ table) {
  pdl_launch_dependents();
  pdl_wait();
  const uint32_t b = blockIdx.x, i = threadIdx.x;
  const int32_t ctx = ctx_lens[b];
  const double pos = ctx > 0 ? (double)(ctx - 1) : 0.0;
  const double inv_freq = exp2(-(double)(2 * i) / (double)kD * log2_base);
  double sn, cs;
  sincos(pos * inv_freq, &sn, &cs);
  table[(size_t)b * (kD / 2) + i] = make_float2((float)cs, (float)sn);
}

// act = silu(gate) * up with gate = gu[:, :F], up = gu[:, F:]
__global__ void __launch_bounds__(256)
swiglu_kernel(const __nv_bfloat16* __restrict__ gu, uint32_t B, uint32_t F, __nv_bfloat16* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  const size_t n = (size_t)B * F / 2;
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const size_t e = i * 2;
    const size_t b = e / F, f = e % F;
    const float2 g = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gu + b * 2 * F + f));
    const float2 u = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(gu + b * 2 * F + F + f));
    const float a0 = g.x / (1.f + expf(-g.x)) * u.x;
    const float a1 = g.y / (1.f + expf(-g.y)) * u.y;
    *reinterpret_cast<__nv_bfloat162*>(out + b * F + f) = __floats2bfloat162_rn(a0, a1);
  }
}

// argmax over fp32 logits, lowest index on ties.  One cluster of kArgmaxCluster threadblocks
// per row: each scans a slice of the row, and the first block of the cluster reads the others'
// candidates out of their shared memory (distributed shared memory), so no scratch in global
// memory and no second launch are needed.
constexpr uint32_t kArgmaxCluster = 8;
constexpr uint32_t kArgmaxThreads = 512;

__device__ __forceinline__ void take_better(float& best, uint32_t& best_i, float v, uint32_t i) {
  if (v > best || (v == best && i < best_i)) { best = v; best_i = i; }
}

__global__ void __launch_bounds__(kArgmaxThreads)
argmax_kernel(const float* __restrict__ logits, uint32_t V, int32_t* __restrict__ out) {
  pdl_launch_dependents();
  pdl_wait();
  __shared__ float s_val[32];
  __shared__ uint32_t s_idx[32];
  __shared__ float s_best;
  __shared__ uint32_t s_best_i;
  uint32_t rank;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(rank));
  const float* row = logits + (size_t)blockIdx.y * V;
  const uint32_t slice = (V + kArgmaxCluster - 1) / kArgmaxCluster;
  const uint32_t i0 = rank * slice, i1 = min(V, i0 + slice);
  float best = -CUDART_INF_F;
  uint32_t best_i = 0xFFFFFFFFu;   // "nothing yet": loses every tie, and any value beats -inf or equals it
  uint32_t i = i0 + threadIdx.x;
  for (; i + 3 * kArgmaxThreads < i1; i += 4 * kArgmaxThreads) {   // four loads in flight
    const float v0 = row[i], v1 = row[i + kArgmaxThreads], v2 = row[i + 2 * kArgmaxThreads], v3 = row[i + 3 * kArgmaxThreads];
    take_better(best, best_i, v0, i);
    take_better(best, best_i, v1, i + kArgmaxThreads);
    take_better(best, best_i, v2, i + 2 * kArgmaxThreads);
    take_better(best, best_i, v3, i + 3 * kArgmaxThreads);
  }
  for (; i < i1; i += kArgmaxThreads) take_better(best, best_i, row[i], i);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, o);
    const uint32_t oi = __shfl_xor_sync(0xFFFFFFFFu, best_i, o);
    take_better(best, best_i, ov, oi);
  }
  if ((threadIdx.x & 31) == 0) { s_val[threadIdx.x >> 5] = best; s_idx[threadIdx.x >> 5] = best_i; }
  __syncthreads();
  if (threadIdx.x < 32) {
    const uint32_t n_warps = kArgmaxThreads / 32;
    best = threadIdx.x < n_warps ? s_val[threadIdx.x] : -CUDART_INF_F;
    best_i = threadIdx.x < n_warps ? s_idx[threadIdx.x] : 0xFFFFFFFFu;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xFFFFFFFFu, best, o);
      const uint32_t oi = __shfl_xor_sync(0xFFFFFFFFu, best_i, o);
      take_better(best, best_i, ov, oi);
    }
    if (threadIdx.x == 0) { s_best = best; s_best_i = best_i; }
  }
  // every block's candidate is in its shared memory: the first block of the cluster collects them
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
  if (rank == 0 && threadIdx.x == 0) {
    for (uint32_t r = 1; r < kArgmaxCluster; ++r) {
      uint32_t a_val, a_idx, ri;
      float rv;
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a_val) : "r"(smem_u32(&s_best)), "r"(r));
      asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a_idx) : "r"(smem_u32(&s_best_i)), "r"(r));
      asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(rv) : "r"(a_val) : "memory");
      asm volatile("ld.shared::cluster.u32 %0, [%1];" : "=r"(ri) : "r"(a_idx) : "memory");
      take_better(best, best_i, rv, ri);
    }
    out[blockIdx.y] = best_i == 0xFFFFFFFFu ? 0 : (int32_t)best_i;   // a row of NaNs: index 0
  }
  // nobody leaves (and gives up its shared memory) before the collector has read it
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

}  // namespace

extern "C" int boost_embed_gather(const void* table, uint32_t vocab, uint32_t hidden,
                                  const int32_t* tokens, uint32_t B, void* out, void* stream) {
  return boost_embed_gather_ssq(table, vocab, hidden, tokens, B, out, nullptr, 0, stream);
}

extern "C" int boost_embed_gather_ssq(const void* table, uint32_t vocab, uint32_t hidden,
                                      const int32_t* tokens, uint32_t B, void* out, float* ssq_out,
                                      uint32_t ssq_stride, void* stream) {
  if (B == 0) return BOOST_OK;
  if (!table || !tokens || !out || vocab == 0 || hidden == 0) return BOOST_ERR_INVALID;
  if (hidden % 8 != 0 || ((uintptr_t)table % 16) || ((uintptr_t)out % 16)) return BOOST_ERR_ALIGN;
  if (ssq_out && (hidden % 128 != 0 || ssq_stride < B)) return BOOST_ERR_INVALID;
  return boosth::launch_chained(embed_gather_kernel, dim3(B), dim3(256), 0, (cudaStream_t)stream,
                                static_cast<const uint4*>(table), vocab, hidden / 8, tokens, static_cast<uint4*>(out),
                                ssq_out, ssq_stride);
}

extern "C" int boost_rmsnorm(const void* x, const void* weight, uint32_t B, uint32_t hidden, float eps,
                             void* out, void* stream) {
  if (B == 0) return BOOST_OK;
  if (!x || !weight || !out || hidden == 0) return BOOST_ERR_INVALID;
  if (hidden % 2 != 0 || ((uintptr_t)x % 4) || ((uintptr_t)out % 4) || ((uintptr_t)weight % 4)) return BOOST_ERR_ALIGN;
  return boosth::launch_chained(rmsnorm_kernel, dim3(B), dim3(256), 0, (cudaStream_t)stream,
                                static_cast<const __nv_bfloat16*>(x), static_cast<const __nv_bfloat16*>(weight),
                                hidden, eps, static_cast<__nv_bfloat16*>(out));
}

extern "C" int boost_rope_kv_append(const void* qkv, void* q_out, const void* const* k_page_ptr,
                                    const void* const* v_page_ptr, uint32_t n_pool_blocks,
                                    const int32_t* block_table, uint32_t max_blocks,
                                    const int32_t* ctx_lens, uint32_t B, uint32_t Hq, uint32_t Hkv,
                                    uint32_t D, float rope_base, void* status_word, void* stream) {
  if (B == 0) return BOOST_OK;
  if (!qkv || !q_out || !k_page_ptr || !v_page_ptr || !block_table || !ctx_lens || !status_word)
    return BOOST_ERR_INVALID;
  if (D != kD) return BOOST_ERR_UNSUPPORTED;
  if (Hq == 0 || Hkv == 0 || max_blocks == 0 || n_pool_blocks == 0 || !(rope_base > 1.f)) return BOOST_ERR_INVALID;
  const uint64_t n = (uint64_t)B * (Hq + 2 * Hkv) * (kD / 2);
  if (n > 0x7FFFFFFFull) return BOOST_ERR_INVALID;
  return boosth::launch_chained(rope_kv_append_kernel, dim3((unsigned)((n + 255) / 256)), dim3(256), 0,
                                (cudaStream_t)stream, static_cast<const __nv_bfloat16*>(qkv),
                                static_cast<__nv_bfloat16*>(q_out), k_page_ptr, v_page_ptr, n_pool_blocks,
                                block_table, max_blocks, ctx_lens, B, Hq, Hkv, log2((double)rope_base),
                                static_cast<uint32_t*>(status_word));
}

extern "C" int boost_rope_table(const int32_t* ctx_lens, uint32_t B, uint32_t D, float rope_base, float* table,
                                void* stream) {
  if (B == 0) return BOOST_OK;
  if (!ctx_lens || !table || !(rope_base > 1.f)) return BOOST_ERR_INVALID;
  if (D != kD) return BOOST_ERR_UNSUPPORTED;
  if ((uintptr_t)table % 16) return BOOST_ERR_ALIGN;
  return boosth::launch_chained(rope_table_kernel, dim3(B), dim3(kD / 2), 0, (cudaStream_t)stream, ctx_lens,
                                log2((double)rope_base), reinterpret_cast<float2*>(table));
}

extern "C" int boost_swiglu(const void* gate_up, uint32_t B, uint32_t F, void* out, void* stream) {
  if (B == 0 || F == 0) return BOOST_OK;
  if (!gate_up || !out) return BOOST_ERR_INVALID;
  if (F % 2 != 0 || ((uintptr_t)gate_up % 4) || ((uintptr_t)out % 4)) return BOOST_ERR_ALIGN;
  const size_t n = (size_t)B * F / 2;
  size_t blocks = (n + 255) / 256;
  const size_t cap = (size_t)(boosth::sm_count() > 0 ? boosth::sm_count() : 148) * 8;
  if (blocks > cap) blocks = cap;
  return boosth::launch_chained(swiglu_kernel, dim3((unsigned)blocks), dim3(256), 0, (cudaStream_t)stream,
                                static_cast<const __nv_bfloat16*>(gate_up), B, F, static_cast<__nv_bfloat16*>(out));
}

extern "C" int boost_argmax(const float* logits, uint32_t B, uint32_t V, int32_t* out, void* stream) {
  if (B == 0) return BOOST_OK;
  if (!logits || !out || V == 0) return BOOST_ERR_INVALID;
  if (B > 65535) return BOOST_ERR_UNSUPPORTED;
  return boosth::launch_chained_cluster(argmax_kernel, dim3(kArgmaxCluster, B), dim3(kArgmaxThreads), 0, kArgmaxCluster,
                                        (cudaStream_t)stream, logits, V, out);
}
