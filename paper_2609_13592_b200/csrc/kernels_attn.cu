// Tiered paged decode attention (split-KV) over the KV cache of a boost_kv_pool, and the
// copies that move a logical [Hkv][N][16][D] cache into and out of its pages.
//
// Persistent threadblocks, two per SM.  A work item is a KV-head chunk run: sequence b, KV
// head g, blocks [16 s, 16 s + 16) of the sequence (Sec. 3.3: attention threadblocks work
// on KV head chunks); items of the highest-numbered heads - the ones linear placement puts
// on the host tier - are handed out first.  A producer warp walks the items and fills a
// ring of 8 KiB stages, one KV block (K chunk + V chunk) per stage: two 4 KiB bulk copies
// through the TMA unit for HBM pages, a fan of 16-byte cp.async loads for host pages; the
// query rows of the item ride along with its first block.  Four consumer warps take the
// blocks of an item round-robin, each with its own running softmax state.  The products
// are bf16 tensor-core MMAs with the 16 tokens of a block as the 16-row dimension and the
// query heads of the group as the 8-wide dimension (S^T = K q^T, O^T += V^T P^T, so a group of
// four heads wastes half a tile instead of three quarters); P goes in as three bf16 terms,
// transposed in registers with movmatrix; the online softmax is fp32.  At the end of
// an item the warps merge through shared memory, and the last split of a (b, g) pair to
// finish combines all splits in split order.
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
constexpr uint32_t kItemBlocks = 16;                     // KV blocks per work item
constexpr uint32_t kStageBytes = 2 * kChunkBytes;        // K chunk + V chunk
constexpr uint32_t kAttnWarps = 4;                       // consumer warps
constexpr uint32_t kConsumerThreads = kAttnWarps * 32;
constexpr uint32_t kAttnThreads = kConsumerThreads + 32; // + producer warp
constexpr uint32_t kMaxGroup = 16;
constexpr uint32_t kMaxStages = 12;
constexpr uint32_t kQRowStride = 272;                    // 256 data bytes + 16: rows hit distinct banks
constexpr uint32_t kAttnSmemBudget3 = 74u * 1024u;       // three threadblocks per SM (groups up to 8)
constexpr uint32_t kAttnSmemBudget2 = 111u * 1024u;      // two per SM (groups up to 16)

enum : uint32_t { kAFirst = 1u, kALast = 2u, kAStop = 4u, kANoData = 8u };

struct AttnParams {
  const __nv_bfloat16* q;
  const void* const* k_page_ptr;
  const void* const* v_page_ptr;
  uint32_t first_host_page;   // pages >= this are host pages (linear placement)
  uint32_t n_pool_blocks;
  const int32_t* block_table;
  uint32_t max_blocks;
  const int32_t* ctx_lens;
  uint32_t B, Hq, Hkv, group, max_splits, n_items, n_stages;
  float scale_log2e;
  uint32_t* ws;        // header (status, item counter, done counter) + one counter per (b, g)
  float* part_ml;      // [B][Hq][max_splits][2]
  float* part_o;       // [B][Hq][max_splits][128]
  __nv_bfloat16* out;
};

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// NH = number of 8-head tiles of a KV group (1: up to 8 query heads per KV head, 2: up to 16)
template <int NH>
__global__ void __launch_bounds__(kAttnThreads, (NH == 1 ? 3 : 2)) paged_attn_kernel(const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  const uint32_t n_stages = p.n_stages;
  uint8_t* stage_sm = smem;                                        // [n_stages][K 4 KiB | V 4 KiB]
  uint8_t* q_sm = smem + (size_t)n_stages * kStageBytes;           // [n_stages][group][kQRowStride]
  const uint32_t q_slot_bytes = p.group * kQRowStride;             // query rows travel with an item's first stage
  float* merge_o = reinterpret_cast<float*>(q_sm + (size_t)n_stages * q_slot_bytes);  // [warps][group][128]
  __shared__ uint64_t full_bar[kMaxStages];
  __shared__ uint64_t empty_bar[kMaxStages];
  __shared__ uint4 meta[kMaxStages];
  __shared__ uint32_t meta_ctx[kMaxStages];
  __shared__ float merge_ml[kAttnWarps][kMaxGroup][2];
  __shared__ uint32_t s_old;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t* status = p.ws + kWsStatus;
  pdl_launch_dependents();
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 33);   // 32 cp.async arrivals + the arrive.expect_tx
      mbar_init(&empty_bar[s], kAttnWarps);
    }
    fence_barrier_init();
  }
  pdl_wait();   // q and the newest K/V rows come from the kernels just before this one
  __syncthreads();

  if (warp == kAttnWarps) {
    // ------------------------------------------------------------------ producer warp
    uint32_t stage = 0, phase = 0;
    uint32_t id = blockIdx.x;   // first item by position, later ones from the counter
    const uint32_t per_head = p.B * p.max_splits;
    while (id < p.n_items) {
      const uint32_t g = p.Hkv - 1 - id / per_head;     // host-resident heads first
      const uint32_t b = (id % per_head) / p.max_splits;
      const uint32_t split = id % p.max_splits;
      const uint32_t ctx = (uint32_t)max(p.ctx_lens[b], 0);
      const uint32_t n_blk = (ctx + kTok - 1) / kTok;
      const uint32_t n_splits = n_blk ? (n_blk + kItemBlocks - 1) / kItemBlocks : 1;
      if (split < n_splits) {
        const uint32_t blk0 = split * kItemBlocks;
        const uint32_t nb = min(kItemBlocks, n_blk - min(n_blk, blk0));
        // every lane resolves one block of the item: table entry, page, addresses
        const uint8_t* ksrc = nullptr;
        const uint8_t* vsrc = nullptr;
        uint32_t host_bit = 0;
        if (lane < nb) {
          int32_t blk = p.block_table[(size_t)b * p.max_blocks + blk0 + lane];
          if (blk < 0 || (uint32_t)blk >= p.n_pool_blocks) {   // bad table entry: record, read block 0
            atomicOr(status, kErrBadIndex);
            blk = 0;
          }
          const uint32_t lin = g * p.n_pool_blocks + (uint32_t)blk;
          const uint32_t page = lin / kChunksPerPage;
          const size_t in_page = (size_t)(lin % kChunksPerPage) * kChunkBytes;
          ksrc = static_cast<const uint8_t*>(p.k_page_ptr[page]) + in_page;
          vsrc = static_cast<const uint8_t*>(p.v_page_ptr[page]) + in_page;
          host_bit = page >= p.first_host_page ? 1u : 0u;
        }
        const uint32_t n_emit = nb ? nb : 1u;   // an empty sequence still gets one (data-less) stage
        for (uint32_t i = 0; i < n_emit; ++i) {
          const uint8_t* ks = reinterpret_cast<const uint8_t*>(__shfl_sync(0xFFFFFFFFu, (unsigned long long)ksrc, i));
          const uint8_t* vs = reinterpret_cast<const uint8_t*>(__shfl_sync(0xFFFFFFFFu, (unsigned long long)vsrc, i));
          const bool from_host = __shfl_sync(0xFFFFFFFFu, host_bit, i) != 0;
          uint8_t* kdst = stage_sm + (size_t)stage * kStageBytes;
          uint8_t* vdst = kdst + kChunkBytes;
          if (lane == 0) {
            mbar_wait(&empty_bar[stage], phase ^ 1u, status);
            const uint32_t flags = (i == 0 ? kAFirst : 0u) | (i + 1 == n_emit ? kALast : 0u) | (nb ? 0u : kANoData);
            meta[stage] = make_uint4(b, g | (split << 16), (blk0 + i) * kTok, flags | (i << 16));
            meta_ctx[stage] = ctx;
            const bool bulk = nb && !from_host;
            mbar_arrive_expect_tx(&full_bar[stage], bulk ? kStageBytes : 0u);
            if (bulk) {
              bulk_copy_g2s(kdst, ks, kChunkBytes, &full_bar[stage]);
              bulk_copy_g2s(vdst, vs, kChunkBytes, &full_bar[stage]);
            }
          }
          __syncwarp();
          if (nb && from_host) {
#pragma unroll
            for (uint32_t c = lane; c < kChunkBytes / 16; c += 32) {
              cp_async_16(kdst + c * 16, ks + c * 16, 16u);
              cp_async_16(vdst + c * 16, vs + c * 16, 16u);
            }
          }
          if (i == 0) {
            // the item's query rows: group x 256 bytes into this item's slot
            const uint8_t* qsrc = reinterpret_cast<const uint8_t*>(p.q + ((size_t)b * p.Hq + g * p.group) * kD);
            uint8_t* qdst = q_sm + (size_t)stage * q_slot_bytes;
            for (uint32_t c = lane; c < p.group * 16; c += 32)
              cp_async_16(qdst + (c >> 4) * kQRowStride + (c & 15) * 16, qsrc + c * 16, 16u);
          }
          cp_async_arrive_noinc(&full_bar[stage]);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
        }
      }
      uint32_t nxt = 0;
      if (lane == 0) nxt = gridDim.x + atomicAdd(p.ws + kWsHbmNext, 1u);
      id = __shfl_sync(0xFFFFFFFFu, nxt, 0);
    }
    // tell the consumers to stop, then the last threadblock out resets the counters
    if (lane == 0) {
      mbar_wait(&empty_bar[stage], phase ^ 1u, status);
      meta[stage] = make_uint4(0u, 0u, 0u, kAStop);
      mbar_arrive(&full_bar[stage]);
    }
    __syncwarp();
    cp_async_arrive_noinc(&full_bar[stage]);
    if (lane == 0) {
      __threadfence();
      const uint32_t d = atomicAdd(p.ws + kWsDone, 1u);
      if (d == gridDim.x - 1) { p.ws[kWsHbmNext] = 0; p.ws[kWsDone] = 0; __threadfence(); }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  // Fragment coordinates: rows g, g+8 (tokens for S^T, d for O^T), columns c0, c0+1 (heads).
  const uint32_t gq = lane >> 2, c0 = (lane & 3) * 2;
  uint32_t qb[NH][8][2];      // q^T as the B operand: k = d, n = head
  float o[NH][8][4];          // O^T: 8 tiles of 16 d, columns = heads
  float m_run[NH][2], l_run[NH][2];
  uint32_t stage = 0, phase = 0;
  for (;;) {
    mbar_wait(&full_bar[stage], phase, status);
    const uint4 mt = meta[stage];
    const uint32_t flags = mt.w & 0xFFu;
    if (flags & kAStop) break;
    if (flags & kAFirst) {
      // the item's query rows sit in the slot of its first stage, ours until we release it
      const uint8_t* qs = q_sm + (size_t)stage * q_slot_bytes;
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        const uint32_t head = nh * 8 + gq;
#pragma unroll
        for (uint32_t ks = 0; ks < 8; ++ks) {
          const uint8_t* src = qs + head * kQRowStride + (ks * 16 + c0) * 2;
          qb[nh][ks][0] = head < p.group ? *reinterpret_cast<const uint32_t*>(src) : 0u;
          qb[nh][ks][1] = head < p.group ? *reinterpret_cast<const uint32_t*>(src + 16) : 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[nh][i][0] = o[nh][i][1] = o[nh][i][2] = o[nh][i][3] = 0.f; }
        m_run[nh][0] = m_run[nh][1] = -CUDART_INF_F;
        l_run[nh][0] = l_run[nh][1] = 0.f;
      }
    }
    const uint32_t b = mt.x, g = mt.y & 0xFFFFu, split = mt.y >> 16;
    const uint32_t ctx = meta_ctx[stage];
    if (!(flags & kANoData) && ((mt.w >> 16) & 3u) == warp) {
      const uint32_t kbase = smem_u32(stage_sm + (size_t)stage * kStageBytes);
      const uint32_t vbase = kbase + kChunkBytes;
      const uint32_t tok = (lane & 7) + ((lane >> 4) << 3);     // ldmatrix row of this lane
      const uint32_t sub = (lane >> 3) & 1;                     // which 16-byte chunk of a pair
      // S^T = K q^T: rows = 16 tokens, columns = heads
      float s[NH][4], s2[NH][4];   // two accumulation chains, added at the end
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        s[nh][0] = s[nh][1] = s[nh][2] = s[nh][3] = 0.f;
        s2[nh][0] = s2[nh][1] = s2[nh][2] = s2[nh][3] = 0.f;
      }
#pragma unroll
      for (uint32_t ks = 0; ks < 8; ++ks) {
        // A fragment of K: m0 tokens 0-7 / chunk 2ks, m1 tokens 8-15 / chunk 2ks, m2, m3 chunk 2ks+1
        const uint32_t a_tok = (lane & 7) + (((lane >> 3) & 1) << 3);
        const uint32_t a_chunk = 2 * ks + (lane >> 4);
        uint32_t a[4];
        ldmatrix_x4(a[0], a[1], a[2], a[3], kbase + a_tok * 256 + ((a_chunk ^ (a_tok & 7)) << 4));
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) mma_bf16_16816((ks & 1) ? s2[nh] : s[nh], a, qb[nh][ks][0], qb[nh][ks][1]);
      }
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int r = 0; r < 4; ++r) s[nh][r] += s2[nh][r];
      // mask the tail of the last block, scale into the log2 domain; online softmax per head
      const uint32_t t_lo = mt.z + gq, t_hi = t_lo + 8;
      uint32_t pa[NH][3][2];
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        float pf[4];
#pragma unroll
        for (int r = 0; r < 4; ++r) {
          const uint32_t t = (r & 2) ? t_hi : t_lo;
          s[nh][r] = (t < ctx) ? s[nh][r] * p.scale_log2e : -CUDART_INF_F;
        }
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          float mx = fmaxf(s[nh][h], s[nh][2 + h]);
          mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 4));
          mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 8));
          mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, 16));
          const float m_new = fmaxf(m_run[nh][h], mx);      // finite: a block has a valid token
          const float corr = exp2f(m_run[nh][h] - m_new);   // exp2(-inf) = 0 on the first block
          pf[h] = exp2f(s[nh][h] - m_new);
          pf[2 + h] = exp2f(s[nh][2 + h] - m_new);
          float sum = pf[h] + pf[2 + h];
          sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 4);
          sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 8);
          sum += __shfl_xor_sync(0xFFFFFFFFu, sum, 16);
          l_run[nh][h] = l_run[nh][h] * corr + sum;
          m_run[nh][h] = m_new;
#pragma unroll
          for (int i = 0; i < 8; ++i) { o[nh][i][h] *= corr; o[nh][i][2 + h] *= corr; }
        }
        // P^T as the B operand (k = token, n = head).  A single bf16 rounding of P would put
        // an error of 2^-9 * sqrt(sum p^2 v^2) on every output, far above 1 % of the outputs
        // that are close to zero; P is split into three bf16 terms (24 bits) multiplied term by
        // term.  The accumulator layout (token rows) is turned into the operand layout (token
        // as k) by an 8x8 transpose across the warp.
        float x0 = pf[0], x1 = pf[1], x2 = pf[2], x3 = pf[3];
#pragma unroll
        for (int t = 0; t < 3; ++t) {
          const __nv_bfloat162 lo = __floats2bfloat162_rn(x0, x1), hi = __floats2bfloat162_rn(x2, x3);
          pa[nh][t][0] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&lo));   // tokens 0-7
          pa[nh][t][1] = movmatrix_trans(*reinterpret_cast<const uint32_t*>(&hi));   // tokens 8-15
          x0 -= __low2float(lo); x1 -= __high2float(lo);
          x2 -= __low2float(hi); x3 -= __high2float(hi);
        }
      }
      // O^T += V^T P^T: rows = d (8 tiles of 16), k = 16 tokens
#pragma unroll
      for (uint32_t dt = 0; dt < 8; ++dt) {
        // A fragment of V^T: m0 d-chunk 2dt / tokens 0-7, m1 chunk 2dt+1 / tokens 0-7, m2, m3 tokens 8-15
        const uint32_t chunk = 2 * dt + sub;
        uint32_t a[4];
        ldmatrix_x4_trans(a[0], a[1], a[2], a[3], vbase + tok * 256 + ((chunk ^ (tok & 7)) << 4));
#pragma unroll
        for (int nh = 0; nh < NH; ++nh)
#pragma unroll
          for (int t = 2; t >= 0; --t) mma_bf16_16816(o[nh][dt], a, pa[nh][t][0], pa[nh][t][1]);
      }
    }
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);
    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
    if (!(flags & kALast)) continue;

    // ---- end of the item: merge the warps (disjoint sets of blocks) through shared memory
#pragma unroll
    for (int nh = 0; nh < NH; ++nh)
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t head = nh * 8 + c0 + h;
        if (head < p.group) {
          if (gq == 0) { merge_ml[warp][head][0] = m_run[nh][h]; merge_ml[warp][head][1] = l_run[nh][h]; }
          float* dst = merge_o + ((size_t)warp * p.group + head) * kD;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            dst[i * 16 + gq] = o[nh][i][h];
            dst[i * 16 + gq + 8] = o[nh][i][2 + h];
          }
        }
      }
    named_barrier_sync(1, kConsumerThreads);

    const uint32_t n_blk = (ctx + kTok - 1) / kTok;
    const uint32_t n_splits = n_blk ? (n_blk + kItemBlocks - 1) / kItemBlocks : 1;
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
        acc += f * merge_o[((size_t)w * p.group + r) * kD + tid];
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
    if (!single) {
      // the last split of (b, g) to arrive combines all splits, in split order
      uint32_t* cnt = p.ws + kWsHeaderWords + b * p.Hkv + g;
      named_barrier_sync(1, kConsumerThreads);
      if (tid == 0) {
        __threadfence();   // cumulative: publishes the partials of all 128 threads (ordered by the barrier)
        s_old = atomicAdd(cnt, 1u);
      }
      named_barrier_sync(1, kConsumerThreads);
      if (s_old == n_splits - 1) {
        __threadfence();
        for (uint32_t r = 0; r < p.group; ++r) {
          const uint32_t hq = g * p.group + r;
          const size_t slot0 = ((size_t)b * p.Hq + hq) * p.max_splits;
          float m_all = -CUDART_INF_F;
          for (uint32_t sp = 0; sp < n_splits; ++sp) m_all = fmaxf(m_all, __ldcg(p.part_ml + (slot0 + sp) * 2));
          float acc = 0.f, l_all = 0.f;
          for (uint32_t sp = 0; sp < n_splits; ++sp) {
            const float ms = __ldcg(p.part_ml + (slot0 + sp) * 2);
            const float f = (ms == -CUDART_INF_F) ? 0.f : exp2f(ms - m_all);
            acc += f * __ldcg(p.part_o + (slot0 + sp) * kD + tid);
            l_all += f * __ldcg(p.part_ml + (slot0 + sp) * 2 + 1);
          }
          p.out[((size_t)b * p.Hq + hq) * kD + tid] = __float2bfloat16_rn(l_all > 0.f ? acc / l_all : 0.f);
        }
        if (tid == 0) *cnt = 0;
      }
    }
    named_barrier_sync(1, kConsumerThreads);   // the merge buffers are free again
  }
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
  const size_t max_splits = max_blocks ? (max_blocks + kItemBlocks - 1) / kItemBlocks : 1;
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
  p.max_splits = (max_blocks + kItemBlocks - 1) / kItemBlocks;
  const uint64_t n_items = (uint64_t)Hkv * B * p.max_splits;
  if (n_items > 0x7FFFFFFFull) return BOOST_ERR_INVALID;
  p.n_items = (uint32_t)n_items;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.ws = static_cast<uint32_t*>(workspace);
  uint8_t* base = static_cast<uint8_t*>(workspace) + attn_header_bytes(B, Hq);
  p.part_ml = reinterpret_cast<float*>(base);
  p.part_o = p.part_ml + (size_t)B * Hq * p.max_splits * 2;
  p.out = static_cast<__nv_bfloat16*>(out);
  const size_t fixed = (size_t)kAttnWarps * p.group * kD * 4 + 128;
  const uint32_t budget = p.group <= 8 ? kAttnSmemBudget3 : kAttnSmemBudget2;
  uint32_t n_stages = (uint32_t)((budget - fixed) / (kStageBytes + p.group * kQRowStride));
  if (n_stages > kMaxStages) n_stages = kMaxStages;
  p.n_stages = n_stages;
  const size_t smem = (size_t)n_stages * (kStageBytes + p.group * kQRowStride) + fixed;
  static bool configured = false;
  if (!configured) {
    int rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemBudget2));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kAttnSmemBudget2));
    if (rc != BOOST_OK) return rc;
    configured = true;
  }
  const int sms = boosth::sm_count();
  if (sms <= 0) return BOOST_ERR_CUDA;
  uint32_t grid = (uint32_t)sms * (p.group <= 8 ? 3 : 2);
  if (grid > p.n_items) grid = p.n_items;
  if (p.group <= 8)
    return boosth::launch_chained(paged_attn_kernel<1>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p);
  return boosth::launch_chained(paged_attn_kernel<2>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p);
}
