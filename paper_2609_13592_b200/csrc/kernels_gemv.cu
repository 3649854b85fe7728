// Tiered weight-streaming product y = x W^T (GEMV at batch 1, skinny GEMM above) and the
// kernel that packs a row-major weight into its paged 16 KiB-block form.
//
// Persistent threadblocks (two per SM for the mma.sync kernel, one for the tcgen05 kernel).  A
// weight producer warp fills a ring of shared-memory stages, one 16 KiB weight block per bulk copy
// through the TMA unit; an activation producer warp adds the matching 64-column slice of x.
// Consumer warps multiply from shared memory: on CUDA cores with warp-shuffle reductions for
// batches of 1 and 2, with mma.sync bf16 tensor-core MMAs up to 32 rows, with tcgen05 MMAs into
// tensor memory above.  Two schedules.  The default cuts every weight evenly over the
// threadblocks, a contiguous share of the packed matrix each; blocks that lie in host pages are
// read in place by the same bulk copies (they read pinned host memory as they read HBM), more
// slowly, by whichever threadblock's share holds them - modulo placement spreads the host pages
// over the matrix, so the link works from the start of the launch.  The other is the paper's
// (Sec. 3.2; boost_gemv_set_tier_schedule): a weight with host pages is cut into work items (runs
// of blocks of one row tile inside one page) in two queues, host-tier items first and fetched by
// deep fans of 16-byte cp.async loads, so a threadblock reads one tier at a time.  Split-K partial
// sums meet in L2 and are combined in a fixed order.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdlib.h>

#include "device_common.cuh"
#include "host_common.h"

namespace {

using namespace boostk;

constexpr uint32_t kBlockRows = 128;
constexpr uint32_t kBlockK = 64;
constexpr uint32_t kBlockBytes = kBlockRows * kBlockK * 2;      // 16 KiB
constexpr uint32_t kBlocksPerPage = kPageBytes / kBlockBytes;   // 128
constexpr uint32_t kConsumerWarps = 8;
constexpr uint32_t kConsumerThreads = kConsumerWarps * 32;
constexpr uint32_t kGemvThreads = kConsumerThreads + 64;   // + weight producer warp + x producer warp
constexpr uint32_t kMaxStages = 16;
constexpr uint32_t kSmemBudget = 224u * 1024u;
constexpr uint32_t kXRowStride = 144;  // 128 data bytes + 16: 8 consecutive rows hit distinct banks

enum : uint32_t { kFlagFirst = 1u, kFlagLast = 2u, kFlagStop = 4u, kFlagPhaseEnd = 8u, kFlagPair = 16u, kFlagSecond = 32u, kFlagHost = 64u };
constexpr uint32_t kMaxPhases = 4;
// Grid-wide counters of a launch, zero at rest: threadblocks that have left; per phase the
// threadblocks whose partial sums are in memory, and the threadblocks that have finished the phase.
enum : uint32_t { kBarExit = 0u, kBarPartials = 1u, kBarPhase = 1u + kMaxPhases, kBarWords = 1u + 2u * kMaxPhases };
// From this many partial sums per row tile on, a phase combines all its tiles at its end, spread
// over all threadblocks, instead of tile by tile in the threadblock that delivers the last one.
constexpr uint32_t kEndCombineMinSegments = 4;
enum : uint32_t { kEpiPlain = 0u, kEpiSwiglu = 1u, kEpiRope = 2u };


struct GemvParams {
  const void* const* w_page_ptr;
  const uint32_t* w_order;
  uint32_t n_pages, n_host_pages;
  uint32_t N, K, n_row_tiles, k_blocks, run, splits, items_per_page, n_items;
  const __nv_bfloat16* x;
  uint32_t M_b;
  void* y;
  int y_dtype;
  const __nv_bfloat16* residual;
  uint32_t* ws;        // header, then one counter per row tile
  uint32_t* queue;     // queue words: the header, or a private set (then weights may stream early)
  uint32_t early;      // 1: private queue words
  // epilogue
  uint32_t epi;              // kEpiPlain / kEpiSwiglu / kEpiRope
  const float* ssq_in;       // [ssq_in_tiles][ssq_stride]: sums of squares of the rows of x by 128-column tile, or null
  uint32_t ssq_in_tiles, ssq_stride, x_cols;
  float rms_eps;
  float* ssq_out;            // [n_row_tiles][ssq_stride]: the same for the rows of y (plain epilogue, bf16 output), or null
  __nv_bfloat16* q_out;      // rope epilogue: rotated queries [M_b, Hq, 128]
  const void* const* k_page_ptr;
  const void* const* v_page_ptr;
  const void* const* k_page_ptr2;   // optional second copy of the cache (staged host pages)
  const void* const* v_page_ptr2;
  const int32_t* block_table;
  const int32_t* ctx_lens;
  uint32_t n_pool_blocks, max_blocks, Hq, Hkv;
  const float* rope_table;   // rope epilogue: (cos, sin) [M_b][64] of this step's positions
  float* partials;     // [row_tile][split][x_rows][128]
  uint32_t n_host_ctas;
  uint32_t n_stages;
  uint32_t active_ctas;   // threadblocks [0, active_ctas) take this product's items (an even share each)
  // Even partition (weights with no host page): threadblock c of active_ctas streams the blocks
  // [c T / G, (c + 1) T / G) of the packed matrix, T = total_blocks, cut into segments at row-tile
  // boundaries; a row tile's partial sums then come from the consecutive threadblocks that
  // touch it.  Every SM carries the same number of bytes, which is what HBM-bound work needs.
  uint32_t even_part, total_blocks;
  uint32_t max_seg;       // partial-sum slots per row tile (= splits with the queues)
  uint32_t tiles_per_unit;   // tcgen05 kernel, even partition: 1, or 2 = adjacent row tiles share an activation tile
  // 1: the partial sums of all row tiles are combined when the phase ends, every warp of the grid
  // taking (row tile, batch row) units in turn (combine_units); 0: tile by tile as they complete
  uint32_t end_combine;
  // end_combine phases only.  1: this launch leaves the combine to a small kernel that follows it
  // on the stream (gemv_combine_kernel) - the last phase of a launch, whose threadblocks then leave
  // as soon as their partial sums are stored and make room for the next kernel's threadblocks
  uint32_t defer_combine;
};

// Counter updates that publish this threadblock's earlier writes (release) and, where the old
// value decides who reads the others' writes, also order those reads after it (acquire).
__device__ __forceinline__ uint32_t atom_add_acq_rel(uint32_t* p, uint32_t v) {
  uint32_t old;
  asm volatile("atom.acq_rel.gpu.global.add.u32 %0, [%1], %2;" : "=r"(old) : "l"(p), "r"(v) : "memory");
  return old;
}
__device__ __forceinline__ void red_add_release(uint32_t* p, uint32_t v) {
  asm volatile("red.release.gpu.global.add.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// First / last threadblock of the even partition that holds a block of row tile `t`.
__device__ __forceinline__ uint32_t part_owner(uint64_t block, uint32_t G, uint32_t T) {
  return (uint32_t)(((block + 1) * G - 1) / T);
}

// Partial sums of row tile `row_tile` under the even partition: one per threadblock (of the G that
// share the product) whose range holds some of the tile's blocks.
__device__ __forceinline__ uint32_t even_part_segments(const GemvParams& p, uint32_t row_tile) {
  const uint32_t tpu = p.tiles_per_unit;
  const uint32_t T2 = ((p.n_row_tiles + tpu - 1) / tpu) * p.k_blocks;
  const uint64_t u0 = (uint64_t)(row_tile / tpu) * p.k_blocks;
  return part_owner(u0 + p.k_blocks - 1, p.active_ctas, T2) - part_owner(u0, p.active_ctas, T2) + 1;
}

// Schedule log only: bytes of blocks [b, b + n) (one row tile's consecutive blocks) that lie in
// host-tier pages.  The host pages of a weight are the first n_host_pages entries of w_order.
__device__ __noinline__ uint32_t host_bytes_of_blocks(const GemvParams& p, uint32_t b, uint32_t n) {
  uint32_t bytes = 0;
  while (n) {
    const uint32_t page = b / kBlocksPerPage;
    const uint32_t here = min(n, kBlocksPerPage - b % kBlocksPerPage);
    bool host = false;
    for (uint32_t i = 0; i < p.n_host_pages && !host; ++i) host = p.w_order[i] == page;
    if (host) bytes += here * kBlockBytes;
    b += here;
    n -= here;
  }
  return bytes;
}

// A launch runs one product, or a chain of up to kMaxPhases products in which each takes the
// previous one's output (as its x, its residual or its row statistics).  The threadblocks stay
// resident; between two phases they meet at a grid-wide counter, and because weights do not
// depend on activations the weight warps stream the next phase's blocks into their rings
// while the tail of the current phase (last items, partial sums, combine) is still running.
// M_b, ws, n_stages and early are those of phase 0.
struct ChainParams {
  uint32_t n_phases;

  uint32_t* bar;   // n_phases > 1: counters [kMaxPhases + 1], zero at rest (one per phase boundary, one for the exit)
  GemvParams ph[kMaxPhases];
};

// tcgen05 kernel: the chain, and the activations of each phase as a tiled tensor map (box = 64
// columns x the padded batch, 128-byte swizzle: the B operand's shared-memory layout as the copy lands)
struct TcChainParams {
  ChainParams chain;
  alignas(64) CUtensorMap x_map[kMaxPhases];
};

__host__ __device__ constexpr uint32_t x_rows_of(int NT, int MB) { return NT > 0 ? NT * 8 : MB; }
__host__ __device__ constexpr uint32_t stage_bytes_of(int NT, int MB) {
  return kBlockBytes + ((x_rows_of(NT, MB) * kXRowStride + 1023u) / 1024u) * 1024u;
}

__device__ __forceinline__ void store_out(const GemvParams& p, uint32_t m, uint32_t n, float v) {
  const size_t idx = (size_t)m * p.N + n;
  if (p.residual) v += bf16_lo((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p.residual) + idx));
  if (p.y_dtype == 0) static_cast<float*>(p.y)[idx] = v;
  else static_cast<__nv_bfloat16*>(p.y)[idx] = __float2bfloat16_rn(v);
}

__device__ __forceinline__ uint2 pack4_bf16(float a, float b, float c, float d) {
  const __nv_bfloat162 lo = __floats2bfloat162_rn(a, b), hi = __floats2bfloat162_rn(c, d);
  uint2 o;
  o.x = *reinterpret_cast<const uint32_t*>(&lo);
  o.y = *reinterpret_cast<const uint32_t*>(&hi);
  return o;
}
__device__ __forceinline__ float round_bf16(float v) { return __bfloat162float(__float2bfloat16_rn(v)); }

// Second half of a combine pass for one thread: its sums (lo = columns [4 v, 4 v + 4) of batch row m,
// hi = their partners 64 columns on) are scaled by the row statistics, paired up and stored as the
// epilogue of the product says (see combine_units).  Called by whole warps: it shuffles.
// What the RoPE epilogue reads besides the sums, requested ahead of them by callers that have the
// registers for it (have = true): the context length, the block-table entry of the new token, the
// cos / sin pairs.  Otherwise finish_pair loads them itself, after the sums.
struct RopeOperands {
  bool have = false;
  int32_t ctx = 0, blk = -1;
  float4 cs01 = make_float4(0.f, 0.f, 0.f, 0.f), cs23 = make_float4(0.f, 0.f, 0.f, 0.f);
  // K / V heads with a valid block: where the two halves of the new row go (second pair: the
  // optional second copy of the cache), looked up through the page tables
  uint8_t* dst[4] = {nullptr, nullptr, nullptr, nullptr};
};
// Byte offsets, inside the K (or V) tensor, of the two 8-byte pieces a lane writes for the new
// token of a sequence: chunk (kvh, blk), token `slot` at slot * 256, 16-byte piece c at position
// c ^ (slot & 7); the lane holds d = 4 v .. 4 v + 3 and d + 64.
__device__ __forceinline__ void kv_append_offsets(const GemvParams& p, uint32_t kvh, uint32_t blk, uint32_t pos, uint32_t v,
                                                  size_t& off1, size_t& off2) {
  const uint32_t slot = pos % BOOST_KV_BLOCK_TOKENS, d = v * 4;
  const size_t chunk = ((size_t)kvh * p.n_pool_blocks + blk) * 4096u + slot * 256u;
  off1 = chunk + ((((d >> 3) ^ (slot & 7u))) << 4) + (d & 7u) * 2u;
  off2 = chunk + (((((d + 64) >> 3) ^ (slot & 7u))) << 4) + (d & 7u) * 2u;
}
// Two parts.  Where the new row goes (context length -> block-table entry -> page addresses:
// three dependent look-ups) depends only on the caller's inputs and the page tables, which no
// kernel of this library writes: it may be fetched before the wait on the product.  The cos / sin
// pairs come from a table that an earlier kernel of the same step writes: after the wait.
__device__ __forceinline__ void load_rope_table(const GemvParams& p, uint32_t row_tile, uint32_t m, uint32_t v, RopeOperands& r) {
  if (row_tile < p.Hq + p.Hkv) {
    r.cs01 = __ldg(reinterpret_cast<const float4*>(p.rope_table + ((size_t)m * 64 + v * 4) * 2));
    r.cs23 = __ldg(reinterpret_cast<const float4*>(p.rope_table + ((size_t)m * 64 + v * 4 + 2) * 2));
  }
}
__device__ __forceinline__ RopeOperands load_rope_operands(const GemvParams& p, uint32_t row_tile, uint32_t m, uint32_t v) {
  RopeOperands r;
  r.have = true;
  r.ctx = p.ctx_lens[m];
  if (row_tile >= p.Hq && r.ctx > 0) {
    const uint32_t bi = ((uint32_t)r.ctx - 1u) / BOOST_KV_BLOCK_TOKENS;
    r.blk = bi < p.max_blocks ? p.block_table[(size_t)m * p.max_blocks + bi] : -1;
    if (r.blk >= 0 && (uint32_t)r.blk < p.n_pool_blocks) {
      const bool is_k = row_tile < p.Hq + p.Hkv;
      size_t off1, off2;
      kv_append_offsets(p, is_k ? row_tile - p.Hq : row_tile - p.Hq - p.Hkv, (uint32_t)r.blk, (uint32_t)r.ctx - 1u, v, off1, off2);
      const void* const* pages = is_k ? p.k_page_ptr : p.v_page_ptr;
      r.dst[0] = static_cast<uint8_t*>(const_cast<void*>(pages[off1 / kPageBytes])) + off1 % kPageBytes;
      r.dst[1] = static_cast<uint8_t*>(const_cast<void*>(pages[off2 / kPageBytes])) + off2 % kPageBytes;
      const void* const* pages2 = is_k ? p.k_page_ptr2 : p.v_page_ptr2;
      if (pages2) {
        r.dst[2] = static_cast<uint8_t*>(const_cast<void*>(pages2[off1 / kPageBytes])) + off1 % kPageBytes;
        r.dst[3] = static_cast<uint8_t*>(const_cast<void*>(pages2[off2 / kPageBytes])) + off2 % kPageBytes;
      }
    }
  }
  return r;
}

template <uint32_t kXRows>
__device__ __forceinline__ void finish_pair(const GemvParams& p, uint32_t row_tile, uint32_t m, uint32_t v, bool valid,
                                            float4 lo, float4 hi, float ss, float ss0, float ss1, const uint2 (&res)[2],
                                            bool vec_out, uint32_t* status, const RopeOperands& pre = RopeOperands()) {
  if (p.ssq_in) {
    ss += ss0 + ss1;
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 4);
    ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 8);
    const float rs = rsqrtf(ss / (float)p.x_cols + p.rms_eps);
    lo.x *= rs; lo.y *= rs; lo.z *= rs; lo.w *= rs;
    hi.x *= rs; hi.y *= rs; hi.z *= rs; hi.w *= rs;
  }
  if (p.epi == kEpiPlain) {
    float sq = 0.f;
    if (valid) {
      const float4 val[2] = {lo, hi};
#pragma unroll
      for (int half = 0; half < 2; ++half) {
        const uint32_t n = row_tile * kBlockRows + half * 64 + v * 4;
        float e[4] = {val[half].x, val[half].y, val[half].z, val[half].w};
        if (n + 3 < p.N && vec_out) {
          const size_t idx = (size_t)m * p.N + n;
          if (p.residual) {
            const uint2 r = res[half];
            e[0] += bf16_lo(r.x); e[1] += bf16_hi(r.x); e[2] += bf16_lo(r.y); e[3] += bf16_hi(r.y);
          }
          if (p.y_dtype == 0) {
            *reinterpret_cast<float4*>(static_cast<float*>(p.y) + idx) = make_float4(e[0], e[1], e[2], e[3]);
          } else {
            *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.y) + idx) = pack4_bf16(e[0], e[1], e[2], e[3]);
#pragma unroll
            for (int j = 0; j < 4; ++j) { const float b = round_bf16(e[j]); sq = fmaf(b, b, sq); }
          }
        } else {
#pragma unroll
          for (int j = 0; j < 4; ++j)
            if (n + j < p.N) {
              float x = e[j];
              if (p.residual) x += bf16_lo((uint32_t)__ldcg(reinterpret_cast<const unsigned short*>(p.residual) + (size_t)m * p.N + n + j));
              if (p.y_dtype == 0) static_cast<float*>(p.y)[(size_t)m * p.N + n + j] = x;
              else {
                static_cast<__nv_bfloat16*>(p.y)[(size_t)m * p.N + n + j] = __float2bfloat16_rn(x);
                const float b = round_bf16(x);
                sq = fmaf(b, b, sq);
              }
            }
        }
      }
    }
    if (p.ssq_out) {   // sum over the 16 threads that share row m (a fixed butterfly order)
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 1);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 2);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 4);
      sq += __shfl_xor_sync(0xFFFFFFFFu, sq, 8);
      if (valid && v == 0) p.ssq_out[(size_t)row_tile * p.ssq_stride + m] = sq;
    }
  } else if (p.epi == kEpiSwiglu) {
    if (valid) {
      const float g[4] = {round_bf16(lo.x), round_bf16(lo.y), round_bf16(lo.z), round_bf16(lo.w)};
      const float u[4] = {round_bf16(hi.x), round_bf16(hi.y), round_bf16(hi.z), round_bf16(hi.w)};
      float a[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) a[j] = g[j] / (1.f + expf(-g[j])) * u[j];
      const size_t idx = (size_t)m * (p.N / 2) + row_tile * 64 + v * 4;
      *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(p.y) + idx) = pack4_bf16(a[0], a[1], a[2], a[3]);
    }
  } else {   // kEpiRope
    const int32_t ctx = valid ? (pre.have ? pre.ctx : p.ctx_lens[m]) : 0;
    if (valid && ctx > 0) {
      const uint32_t pos = (uint32_t)ctx - 1u;
      const uint32_t head = row_tile;
      float x1[4] = {round_bf16(lo.x), round_bf16(lo.y), round_bf16(lo.z), round_bf16(lo.w)};
      float x2[4] = {round_bf16(hi.x), round_bf16(hi.y), round_bf16(hi.z), round_bf16(hi.w)};
      if (head < p.Hq + p.Hkv) {
        // cos / sin of position * base^(-2i/128) for i = 4v .. 4v+3, from the step's table
        const float4 cs01 = pre.have ? pre.cs01 : __ldg(reinterpret_cast<const float4*>(p.rope_table + ((size_t)m * 64 + v * 4) * 2));
        const float4 cs23 = pre.have ? pre.cs23 : __ldg(reinterpret_cast<const float4*>(p.rope_table + ((size_t)m * 64 + v * 4 + 2) * 2));
        const float cs[4] = {cs01.x, cs01.z, cs23.x, cs23.z}, sn[4] = {cs01.y, cs01.w, cs23.y, cs23.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float y1 = x1[j] * cs[j] - x2[j] * sn[j];
          const float y2 = x2[j] * cs[j] + x1[j] * sn[j];
          x1[j] = y1; x2[j] = y2;
        }
      }
      const uint2 o1 = pack4_bf16(x1[0], x1[1], x1[2], x1[3]), o2 = pack4_bf16(x2[0], x2[1], x2[2], x2[3]);
      const uint32_t d = v * 4;
      if (head < p.Hq) {
        __nv_bfloat16* dst = p.q_out + ((size_t)m * p.Hq + head) * kBlockRows;
        *reinterpret_cast<uint2*>(dst + d) = o1;
        *reinterpret_cast<uint2*>(dst + d + 64) = o2;
      } else {
        const bool is_k = head < p.Hq + p.Hkv;
        const uint32_t kvh = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
        const uint32_t bi = pos / BOOST_KV_BLOCK_TOKENS;
        const int32_t blk = pre.have ? pre.blk : (bi < p.max_blocks ? p.block_table[(size_t)m * p.max_blocks + bi] : -1);
        if (blk < 0 || (uint32_t)blk >= p.n_pool_blocks) {
          atomicOr(status, kErrBadIndex);
        } else if (pre.have) {
          *reinterpret_cast<uint2*>(pre.dst[0]) = o1;
          *reinterpret_cast<uint2*>(pre.dst[1]) = o2;
          if (pre.dst[2]) {
            *reinterpret_cast<uint2*>(pre.dst[2]) = o1;
            *reinterpret_cast<uint2*>(pre.dst[3]) = o2;
          }
        } else {
          const void* const* pages = is_k ? p.k_page_ptr : p.v_page_ptr;
          size_t off1, off2;
          kv_append_offsets(p, kvh, (uint32_t)blk, pos, v, off1, off2);
          *reinterpret_cast<uint2*>(static_cast<uint8_t*>(const_cast<void*>(pages[off1 / kPageBytes])) + off1 % kPageBytes) = o1;
          *reinterpret_cast<uint2*>(static_cast<uint8_t*>(const_cast<void*>(pages[off2 / kPageBytes])) + off2 % kPageBytes) = o2;
          const void* const* pages2 = is_k ? p.k_page_ptr2 : p.v_page_ptr2;
          if (pages2) {
            *reinterpret_cast<uint2*>(static_cast<uint8_t*>(const_cast<void*>(pages2[off1 / kPageBytes])) + off1 % kPageBytes) = o1;
            *reinterpret_cast<uint2*>(static_cast<uint8_t*>(const_cast<void*>(pages2[off2 / kPageBytes])) + off2 % kPageBytes) = o2;
          }
        }
      }
    }
  }
}

// What a combine does with the sums of a (batch row m, columns [4 v, 4 v + 4) and their partners
// 64 columns on) - the partners are what SwiGLU (gate / up) and the rotary embedding (d / d + 64)
// pair up:
//   plain   y = sum (* row scale) (+ residual); optionally the sum of squares of the bf16
//           outputs per row, for the RMS scale of the next product;
//   swiglu  rows 0..63 of the tile are gate rows, 64..127 the matching up rows:
//           out[m, 64 t + j] = silu(bf16(gate)) * bf16(up);
//   rope    the tile is one head of [q heads | k heads | v heads]: q and k are rotated
//           (rotate-half pairing, cos / sin from the step's table), q goes to q_out, k and v
//           into the paged cache at the position of the new token.
// The row scale is rsqrt(mean(x^2) + eps) from per-tile sums of squares of the rows of x:
// RMSNorm whose weight has been folded into the packed matrix.
//
// The combine, warp by warp: one row tile (the threadblock that
// delivered its last partial sum: first / step = warp index / warps of the threadblock), or all
// row tiles of a product once every threadblock's partial sums are in memory (the caller has
// waited for that: first / step = warp index / warps of the whole grid).  A warp takes one slot
// per pass.  With few partial sums per tile (at most kPer) a slot is two batch rows, one per
// half-warp, each lane summing all segments of its columns; with many, a slot is one batch row,
// the half-warps take the even and the odd segments and the sums meet through a shuffle - eight
// segments per round trip to L2.  Lane -> v = lane
// % 16: columns [4 v, 4 v + 4) and their partners 64 on.  Sum order (fixed): ascending within a
// lane, even segments + odd segments.  Short products (output, down, next qkv) have ten or so
// partial sums per tile and all their tiles complete together at the end of the phase anyway:
// combining them there, spread over all warps of the grid, replaces six dependent round trips in
// 32 threadblocks by two in all of them.
constexpr uint32_t kAllTiles = 0xFFFFFFFFu;
template <uint32_t kXRows>
__device__ __forceinline__ constexpr uint32_t combine_per_round() { return kXRows == 32 ? 6u : 5u; }
// Slots of one row tile (see combine_units): pairs of batch rows, or single batch rows.
template <uint32_t kXRows>
__device__ __forceinline__ uint32_t combine_slots_per_tile(const GemvParams& p) {
  return p.max_seg <= combine_per_round<kXRows>() ? (p.M_b + 1) / 2 : p.M_b;
}
template <uint32_t kXRows, bool kRopeAhead = false>
__device__ __forceinline__ void combine_units(const GemvParams& p, uint32_t first, uint32_t step, uint32_t tile_or_all,
                                              uint32_t lane, uint32_t* status) {
  constexpr uint32_t kVecRow = kBlockRows / 4;   // float4 per batch row
  // partial sums per lane and round: what the register budget of the instantiation leaves room for
  constexpr uint32_t kPer = combine_per_round<kXRows>();
  const uint32_t v = lane & 15u, half = lane >> 4;
  const bool pair_mode = p.max_seg <= kPer;      // no tile of the product has more partial sums than that
  const uint32_t slots_per_tile = combine_slots_per_tile<kXRows>(p);
  const uint32_t n_slots = tile_or_all == kAllTiles ? p.n_row_tiles * slots_per_tile : slots_per_tile;
  const bool vec_out = (p.N & 3u) == 0;
  bool waited = false;   // (kRopeAhead: the caller has not waited for the product yet)
  for (uint32_t s = first; s < n_slots; s += step) {
    const uint32_t row_tile = tile_or_all == kAllTiles ? s / slots_per_tile : tile_or_all;
    const uint32_t i = tile_or_all == kAllTiles ? s - row_tile * slots_per_tile : s;
    const uint32_t m = pair_mode ? 2 * i + half : i;
    const bool live = m < p.M_b;                       // (the second batch row of the last pair may not exist)
    const bool valid = pair_mode ? live : half == 0;   // these lanes finish outputs
    const uint32_t n_seg = p.even_part ? even_part_segments(p, row_tile) : p.splits;
    const float4* base = reinterpret_cast<const float4*>(p.partials + (size_t)row_tile * p.max_seg * kXRows * kBlockRows) +
                         (live ? m : 0u) * kVecRow + v;
    // everything a lane needs from memory is requested before the first use
    RopeOperands pre;
    if constexpr (kRopeAhead) {
      // Where the RoPE epilogue puts the new K / V row - context length, block-table entry, page
      // addresses - is not written by the product or anything before it on the stream's chain of
      // kernels: it is fetched (three dependent look-ups) while the product is still running, and
      // only then does the warp wait for the product (once: later slots find it complete).
      if (p.epi == kEpiRope && valid) pre = load_rope_operands(p, row_tile, m, v);
      if (!waited) {
        pdl_wait();
        waited = true;
      }
      if (p.epi == kEpiRope && valid) load_rope_table(p, row_tile, m, v, pre);
    }
    float ss = 0.f, ss0 = 0.f, ss1 = 0.f;
    if (p.ssq_in && valid) {
      if (v < p.ssq_in_tiles) ss0 = __ldcg(p.ssq_in + (size_t)v * p.ssq_stride + m);
      if (v + 16 < p.ssq_in_tiles) ss1 = __ldcg(p.ssq_in + (size_t)(v + 16) * p.ssq_stride + m);
      for (uint32_t t0 = v + 32; t0 < p.ssq_in_tiles; t0 += 16) ss += __ldcg(p.ssq_in + (size_t)t0 * p.ssq_stride + m);
    }
    uint2 res[2] = {make_uint2(0u, 0u), make_uint2(0u, 0u)};
    if (valid && p.epi == kEpiPlain && p.residual && vec_out) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const uint32_t n = row_tile * kBlockRows + h * 64 + v * 4;
        if (n < p.N) res[h] = __ldcg(reinterpret_cast<const uint2*>(p.residual + (size_t)m * p.N + n));   // L2: an earlier phase may have rewritten it
      }
    }
    float4 lo = make_float4(0.f, 0.f, 0.f, 0.f), hi = lo;
    const uint32_t seg_first = pair_mode ? 0u : half, seg_step = pair_mode ? 1u : 2u;
    for (uint32_t s0 = seg_first; s0 < n_seg; s0 += kPer * seg_step) {
      float4 t0[kPer], t1[kPer];
#pragma unroll
      for (uint32_t j = 0; j < kPer; ++j) {
        const uint32_t seg = s0 + j * seg_step;
        if (seg < n_seg && live) {
          const float4* src = base + (size_t)seg * kXRows * kVecRow;
          t0[j] = __ldcg(src);
          t1[j] = __ldcg(src + 16);
        }
      }
#pragma unroll
      for (uint32_t j = 0; j < kPer; ++j) {
        if (s0 + j * seg_step < n_seg && live) {
          lo.x += t0[j].x; lo.y += t0[j].y; lo.z += t0[j].z; lo.w += t0[j].w;
          hi.x += t1[j].x; hi.y += t1[j].y; hi.z += t1[j].z; hi.w += t1[j].w;
        }
      }
    }
    if (!pair_mode) {   // lanes 0..15 take the odd segments' sums from lanes 16..31
      lo.x += __shfl_down_sync(0xFFFFFFFFu, lo.x, 16); lo.y += __shfl_down_sync(0xFFFFFFFFu, lo.y, 16);
      lo.z += __shfl_down_sync(0xFFFFFFFFu, lo.z, 16); lo.w += __shfl_down_sync(0xFFFFFFFFu, lo.w, 16);
      hi.x += __shfl_down_sync(0xFFFFFFFFu, hi.x, 16); hi.y += __shfl_down_sync(0xFFFFFFFFu, hi.y, 16);
      hi.z += __shfl_down_sync(0xFFFFFFFFu, hi.z, 16); hi.w += __shfl_down_sync(0xFFFFFFFFu, hi.w, 16);
    }
    finish_pair<kXRows>(p, row_tile, live ? m : 0u, v, valid, lo, hi, ss, ss0, ss1, res, vec_out, status, pre);
  }
}

// NT > 0: tensor-core path with NT batch tiles of 8; NT == 0: CUDA-core path for MB rows.
template <int NT, int MB>
__global__ void __launch_bounds__(kGemvThreads, (NT >= 8 ? 1 : 2)) gemv_tiered_kernel(const __grid_constant__ ChainParams cp) {
  constexpr uint32_t kXRows = x_rows_of(NT, MB);
  constexpr uint32_t kStageBytes = stage_bytes_of(NT, MB);
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[kMaxStages];
  __shared__ uint64_t empty_bar[kMaxStages];
  __shared__ uint4 meta[kMaxStages];
  __shared__ uint64_t item_full[4];
  __shared__ uint64_t item_empty[4];
  __shared__ uint32_t item_ring[4];
  __shared__ uint32_t s_old;
  __shared__ volatile uint32_t s_abort;    // a bounded wait ran out somewhere: every role leaves

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t n_stages = cp.ph[0].n_stages;
  const uint32_t n_phases = cp.n_phases;
  uint32_t* status = cp.ph[0].ws + kWsStatus;

  pdl_launch_dependents();
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 65);              // 2 x 32 cp.async arrivals + the arrive.expect_tx
      mbar_init(&empty_bar[s], kConsumerWarps);
      meta[s] = make_uint4(0u, 0u, 0u, 0u);     // a consumer whose wait ran out reads nothing wild
    }
    for (uint32_t s = 0; s < 4; ++s) {
      mbar_init(&item_full[s], 1);
      mbar_init(&item_empty[s], 1);
    }
    s_abort = 0u;
    fence_barrier_init();
  }
  __syncthreads();

  // Bounded waits.  On a timeout the status word gets kErrWaitTimeout, s_abort is raised and the
  // warp leaves the kernel; the other roles see the flag (or run into their own limit) and leave
  // too, so nothing is read or written on the strength of a wait that did not succeed.
  auto lane0_wait = [&](uint64_t* bar, uint32_t parity) -> bool {   // lane 0 waits, the warp learns the outcome
    uint32_t ok = 1u;
    if (lane == 0) ok = (!s_abort && mbar_wait(bar, parity, status)) ? 1u : 0u;
    ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
    if (!ok) s_abort = 1u;
    return ok != 0u;
  };
  auto warp_wait = [&](uint64_t* bar, uint32_t parity) -> bool {    // all lanes wait
    const bool ok = !s_abort && mbar_wait(bar, parity, status);
    const bool all_ok = __all_sync(0xFFFFFFFFu, ok);
    if (!all_ok) s_abort = 1u;
    return all_ok;
  };

  if (warp >= kConsumerWarps) {
    // ------------------------------------------------------------------ producer warps
    // Warp 8 owns the work queue and the weight blocks; warp 9 follows the same item
    // sequence (handed over through a four-slot ring) and loads the matching slices of x.
    // Two warps, because a lone warp's instruction latency would cap the fill rate.
    const bool leader = (warp == kConsumerWarps);
    uint32_t stage = 0, phase = 0, icount = 0;
    unsigned long long* const sched_log = (leader && lane == 0) ? sched_log_of(cp.ph[0].ws) : nullptr;
    uint32_t rec = kNoRecord;   // schedule-log record of the item in production (weight warp, lane 0)
    // Leaving after a timeout: this warp's own copies into the ring must have landed before the
    // threadblock's shared memory goes away.  The cp.async fans can be waited for; a bulk copy
    // reports only to its stage's barrier, which in this situation may never complete, so the
    // weight warp allows a grace period far longer than a copy takes (16 KiB from HBM: about a
    // microsecond, over the host link: a few) - and in practice it got here through a wait that
    // had already lasted the whole limit.
    auto leave = [&]() {
      cp_async_wait_all();
      if (leader) {
        const long long t0 = clock64();
        while (clock64() - t0 < 100000) __nanosleep(1000);   // ~50 us
      }
      __syncwarp();
    };
    for (uint32_t ph = 0; ph < n_phases; ++ph) {
      const GemvParams& p = cp.ph[ph];
      const uint32_t n_host_items = p.n_host_pages * p.items_per_page;
      TierQueues q;
      const bool active = blockIdx.x < p.active_ctas;
      if (active && !p.even_part) q.init(p.queue, n_host_items, p.n_pages * p.items_per_page, p.n_host_ctas, blockIdx.x, p.active_ctas);
      if (ph == 0) {
        // Weights are never written by the decode chain, so with private queue words the weight
        // warp starts streaming while the previous kernel is still running; x is produced by
        // that kernel, so the x warp (and the consumers) wait for it.
        if (!leader || !p.early) pdl_wait();
      } else if (!leader) {
        // x of this phase is what the previous phase wrote: wait until every threadblock has
        // finished it.  The weight warp does not wait: it fills the ring meanwhile.
        uint32_t ok = 1u;
        if (lane == 0) ok = (!s_abort && grid_counter_wait(cp.bar + kBarPhase + (ph - 1), gridDim.x, status)) ? 1u : 0u;
        ok = __shfl_sync(0xFFFFFFFFu, ok, 0);
        if (!ok) { s_abort = 1u; leave(); return; }
      }
      if (p.even_part) {
        // Even partition: both warps walk the same static block range, no queue.
        const uint32_t G = p.active_ctas, T = p.total_blocks;
        if (blockIdx.x < G) {
          const uint32_t b0 = (uint32_t)((uint64_t)blockIdx.x * T / G), b1 = (uint32_t)((uint64_t)(blockIdx.x + 1) * T / G);
          uint32_t row_tile = b0 / p.k_blocks, kb = b0 % p.k_blocks;
          uint32_t seg = blockIdx.x - part_owner((uint64_t)row_tile * p.k_blocks, G, T);
          const uint32_t c = lane & 7, m0 = lane >> 3;
          // the page address is looked up once per page, not once per block: a table look-up per
          // block would put an L2 round trip between any two copies of this warp
          const uint8_t* page_base = nullptr;
          uint32_t page_of_base = 0xFFFFFFFFu;
          for (uint32_t b = b0; b < b1; ++b) {
            const bool seg_first = (b == b0) || kb == 0, seg_last = (b + 1 == b1) || (kb + 1 == p.k_blocks);
            if (leader) {
              uint8_t* wdst = smem + (size_t)stage * kStageBytes;
              if (!lane0_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
              if (lane == 0) {
                if (b / kBlocksPerPage != page_of_base) {
                  page_of_base = b / kBlocksPerPage;
                  page_base = static_cast<const uint8_t*>(p.w_page_ptr[page_of_base]);
                }
                const uint8_t* src = page_base + (size_t)(b % kBlocksPerPage) * kBlockBytes;
                if (seg_first && sched_log) {   // the segment: blocks up to the end of the row tile or of this threadblock's range
                  const uint32_t n_seg_blocks = min(b1 - b, p.k_blocks - kb);
                  rec = sched_log_begin(sched_log, BOOST_SCHED_KIND_GEMV | (ph << 8), blockIdx.x | (warp << 24),
                                        n_seg_blocks * kBlockBytes, p.n_host_pages ? host_bytes_of_blocks(p, b, n_seg_blocks) : 0u);
                }
                meta[stage] = make_uint4(row_tile, seg, (seg_first ? kFlagFirst : 0u) | (seg_last ? kFlagLast : 0u) | (rec << 8), ph);
                mbar_arrive_expect_tx(&full_bar[stage], kBlockBytes);
                bulk_copy_g2s(wdst, src, kBlockBytes, &full_bar[stage]);
              }
              __syncwarp();
              cp_async_arrive_noinc(&full_bar[stage]);
            } else {
              if (!warp_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
              uint8_t* xdst = smem + (size_t)stage * kStageBytes + kBlockBytes + m0 * kXRowStride + c * 16;
              const uint32_t k = kb * kBlockK + c * 8;
              const bool k_ok = k < p.K;
              const __nv_bfloat16* xs = p.x + (size_t)m0 * p.K + (k_ok ? k : 0u);
#pragma unroll 4
              for (uint32_t m = m0; m < kXRows; m += 4) {
                cp_async_16(xdst, xs, (k_ok && m < p.M_b) ? 16u : 0u);
                xdst += 4 * kXRowStride;
                if (m + 4 < p.M_b) xs += (size_t)4 * p.K;
              }
              cp_async_arrive_noinc(&full_bar[stage]);
            }
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
            if (++kb == p.k_blocks) { kb = 0; ++row_tile; seg = 0; }
          }
        }
      } else
      for (;;) {
        const uint32_t slot = icount & 3u, iphase = (icount >> 2) & 1u;
        uint32_t qi = 0;
        if (leader) {
          if (lane == 0) {
            for (;;) {   // skip the unused tail of the last page
              qi = active ? q.next() : 0xFFFFFFFFu;
              if (qi == 0xFFFFFFFFu) break;
              if (p.w_order[qi / p.items_per_page] * p.items_per_page + qi % p.items_per_page < p.n_items) break;
            }
          }
          if (!lane0_wait(&item_empty[slot], iphase ^ 1u)) { leave(); return; }
          if (lane == 0) {
            item_ring[slot] = qi;
            mbar_arrive(&item_full[slot]);
          }
          qi = __shfl_sync(0xFFFFFFFFu, qi, 0);
        } else {
          if (!warp_wait(&item_full[slot], iphase)) { leave(); return; }
          qi = item_ring[slot];
          __syncwarp();
          if (lane == 0) mbar_arrive(&item_empty[slot]);
        }
        ++icount;
        if (qi == 0xFFFFFFFFu) break;
        const uint32_t page = p.w_order[qi / p.items_per_page];
        const uint32_t first_blk = (page * p.items_per_page + qi % p.items_per_page) * p.run;
        const uint32_t row_tile = first_blk / p.k_blocks;
        const uint32_t kb0 = first_blk % p.k_blocks;
        const bool from_host = qi < n_host_items;
        if (leader) {
          const uint8_t* src = static_cast<const uint8_t*>(p.w_page_ptr[page]) +
                               (size_t)(first_blk % kBlocksPerPage) * kBlockBytes;
          for (uint32_t j = 0; j < p.run; ++j, src += kBlockBytes) {
            uint8_t* wdst = smem + (size_t)stage * kStageBytes;
            // (the other lanes must not run ahead of lane 0's wait on the stage)
            if (!lane0_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
            if (lane == 0) {
              if (j == 0)
                rec = sched_log_begin(sched_log, BOOST_SCHED_KIND_GEMV | (ph << 8), blockIdx.x | (warp << 24),
                                      p.run * kBlockBytes, from_host ? p.run * kBlockBytes : 0u);
              meta[stage] = make_uint4(row_tile, kb0 / p.run,
                                       (j == 0 ? kFlagFirst : 0u) | (j + 1 == p.run ? kFlagLast : 0u) | (rec << 8), ph);
              mbar_arrive_expect_tx(&full_bar[stage], from_host ? 0u : kBlockBytes);
              if (!from_host) bulk_copy_g2s(wdst, src, kBlockBytes, &full_bar[stage]);
            }
            __syncwarp();
            if (from_host) {
              // host page: a fan of 16-byte loads through the load/store path keeps many
              // requests on the link at once (Sec. 3.2: this threadblock is a host-tier block)
#pragma unroll 8
              for (uint32_t idx = lane; idx < kBlockBytes / 16; idx += 32)
                cp_async_16(wdst + idx * 16, src + idx * 16, 16u);
            }
            cp_async_arrive_noinc(&full_bar[stage]);
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
          }
        } else {
          // lane -> (row m0 + 4 i, 16-byte chunk c); pointers advance by constants
          const uint32_t c = lane & 7, m0 = lane >> 3;
          for (uint32_t j = 0; j < p.run; ++j) {
            if (!warp_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
            uint8_t* xdst = smem + (size_t)stage * kStageBytes + kBlockBytes + m0 * kXRowStride + c * 16;
            const uint32_t k = (kb0 + j) * kBlockK + c * 8;
            const bool k_ok = k < p.K;
            const __nv_bfloat16* xs = p.x + (size_t)m0 * p.K + (k_ok ? k : 0u);
#pragma unroll 4
            for (uint32_t m = m0; m < kXRows; m += 4) {
              cp_async_16(xdst, xs, (k_ok && m < p.M_b) ? 16u : 0u);
              xdst += 4 * kXRowStride;
              if (m + 4 < p.M_b) xs += (size_t)4 * p.K;
            }
            cp_async_arrive_noinc(&full_bar[stage]);
            if (++stage == n_stages) { stage = 0; phase ^= 1u; }
          }
        }
      }
      // a stage without data tells the consumers that the phase (or the launch) is over
      if (leader) {
        if (!lane0_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
        if (lane == 0) {
          meta[stage] = make_uint4(0u, 0u, ph + 1 == n_phases ? kFlagStop : kFlagPhaseEnd, ph);
          mbar_arrive(&full_bar[stage]);
        }
        __syncwarp();
        cp_async_arrive_noinc(&full_bar[stage]);
        if (lane == 0 && active && !p.even_part) q.finish(p.active_ctas);
      } else {
        if (!warp_wait(&empty_bar[stage], phase ^ 1u)) { leave(); return; }
        cp_async_arrive_noinc(&full_bar[stage]);
      }
      if (++stage == n_stages) { stage = 0; phase ^= 1u; }
    }
    return;
  }

  // -------------------------------------------------------------------- consumer warps
  constexpr int kAccN = NT > 0 ? NT : 4;
  constexpr int kAccM = NT > 0 ? 4 : MB;
  float acc[kAccN][kAccM];
#pragma unroll
  for (int i = 0; i < kAccN; ++i)
#pragma unroll
    for (int j = 0; j < kAccM; ++j) acc[i][j] = 0.f;

  // The consumer warps meet at named barrier 1, which also ORs their views of s_abort, so all of
  // them take the same way out.  A hardware barrier has no time limit, so the wind-down after a
  // failed wait must leave nobody in it: a warp whose (bounded) wait ran out arrives ONCE more,
  // with "abort", before it leaves (end of this function).  Every other warp arrives once more too -
  // at its next group_sync, or the same way after a failed wait of its own (once s_abort is up
  // every wait fails at once) - so that barrier generation completes and tells everybody to leave.
  // False: leave, without a further arrival.
  auto group_sync = [&]() -> bool { return !named_barrier_or(1, kConsumerThreads, s_abort != 0u); };
  uint32_t* tile_cnt = cp.ph[0].ws + kWsHeaderWords;
  uint32_t stage = 0, phase = 0;
  bool wait_failed = false;   // this warp's own wait ran out (as opposed to: it saw s_abort after a barrier)
  pdl_wait();
  // Outer loop: one round per phase.  The inner loop consumes stages until the marker stage that
  // ends the phase; what follows a phase (the combine of all tiles, the grid-wide counters) stays
  // outside the inner loop, so that its register needs do not weigh on the streaming code.
  for (;;) {
  uint4 mk = make_uint4(0u, 0u, 0u, 0u);
  bool failed = false;
  // Opaque copies of the warp and lane numbers, renewed for every phase: the shared-memory
  // addresses the streaming loop derives from them are loop invariants that the compiler keeps in
  // registers, and this keeps them from staying alive across the code that follows a phase.
  uint32_t lw = warp, ll = lane;
  asm volatile("" : "+r"(lw), "+r"(ll));
  for (;;) {
    if (!warp_wait(&full_bar[stage], phase)) { wait_failed = true; failed = true; break; }
    const uint4 mt = meta[stage];
    if (mt.z & (kFlagStop | kFlagPhaseEnd)) { mk = mt; break; }
    if (mt.z & kFlagFirst) {
#pragma unroll
      for (int i = 0; i < kAccN; ++i)
#pragma unroll
        for (int j = 0; j < kAccM; ++j) acc[i][j] = 0.f;
    }
    const uint8_t* wsm = smem + (size_t)stage * kStageBytes;
    const uint8_t* xsm = wsm + kBlockBytes;
    if constexpr (NT > 0) {
      const uint32_t wbase = smem_u32(wsm), xbase = smem_u32(xsm);
      const uint32_t a_row = lw * 16 + (ll & 7) + ((ll >> 3) & 1) * 8;
      const uint32_t b_row0 = ((ll >> 4) << 3) + (ll & 7);
#pragma unroll
      for (uint32_t ks = 0; ks < 4; ++ks) {
        uint32_t a[4];
        const uint32_t a_chunk = ks * 2 + (ll >> 4);
        ldmatrix_x4(a[0], a[1], a[2], a[3], wbase + a_row * 128 + ((a_chunk ^ (a_row & 7)) << 4));
        const uint32_t b_chunk = ks * 2 + ((ll >> 3) & 1);
#pragma unroll
        for (int n2 = 0; n2 < NT / 2; ++n2) {
          const uint32_t b_row = n2 * 16 + b_row0;
          uint32_t b0, b1, b2, b3;
          ldmatrix_x4(b0, b1, b2, b3, xbase + b_row * kXRowStride + (b_chunk << 4));
          mma_bf16_16816(acc[2 * n2], a, b0, b1);
          mma_bf16_16816(acc[2 * n2 + 1], a, b2, b3);
        }
      }
    } else {
      // lanes 8g..8g+7 share weight row (lw*16 + 4j + g) and split its 64 columns
      const uint32_t c = ll & 7, g = ll >> 3;
      float wf[4][8];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t row = lw * 16 + 4 * j + g;
        const uint4 w = *reinterpret_cast<const uint4*>(wsm + row * 128 + ((c ^ (row & 7)) << 4));
        wf[j][0] = bf16_lo(w.x); wf[j][1] = bf16_hi(w.x); wf[j][2] = bf16_lo(w.y); wf[j][3] = bf16_hi(w.y);
        wf[j][4] = bf16_lo(w.z); wf[j][5] = bf16_hi(w.z); wf[j][6] = bf16_lo(w.w); wf[j][7] = bf16_hi(w.w);
      }
#pragma unroll
      for (int m = 0; m < MB; ++m) {
        const uint4 xv = *reinterpret_cast<const uint4*>(xsm + m * kXRowStride + (c << 4));
        const float xf[8] = {bf16_lo(xv.x), bf16_hi(xv.x), bf16_lo(xv.y), bf16_hi(xv.y),
                             bf16_lo(xv.z), bf16_hi(xv.z), bf16_lo(xv.w), bf16_hi(xv.w)};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          float s = acc[j][m];
#pragma unroll
          for (int e = 0; e < 8; ++e) s = fmaf(wf[j][e], xf[e], s);
          acc[j][m] = s;
        }
      }
    }
    // Every read of the stage must have been performed before the stage is released: the loads
    // went through the generic proxy, the refill is a bulk copy through the async proxy, and the
    // release alone does not keep the refill behind loads that are still in flight (the MMAs
    // that use them may be scheduled after it).  Seen on B200 as torn weight rows in one launch
    // in four when threadblocks have an SM to themselves and the producer reacts at once.  A
    // CTA-scope fence in every reading thread closes it (1.3 % of the step; fence.proxy.async in
    // the same place also does, at 2.4 %).
    __threadfence_block();
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);
    if (++stage == n_stages) { stage = 0; phase ^= 1u; }

    if (mt.z & kFlagLast) {
      if (warp == 0 && lane == 0 && (mt.z >> 8) != kNoRecord) sched_log_end(sched_log_of(cp.ph[0].ws), mt.z >> 8);
      const GemvParams& p = cp.ph[mt.w];
      const uint32_t row_tile = mt.x, split = mt.y;
      if constexpr (NT == 0) {
        // finish the dot products: sum over the 8 lanes that share a row
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
          for (int m = 0; m < MB; ++m) {
            float s = acc[j][m];
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 1);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 2);
            s += __shfl_xor_sync(0xFFFFFFFFu, s, 4);
            acc[j][m] = s;
          }
      }
      // partial sums of this row tile: one per split of the queue items, or one per
      // threadblock of the even partition that holds some of its blocks
      const uint32_t n_seg = p.even_part ? even_part_segments(p, row_tile) : p.splits;
      // without splits (and without a row scale, pairing or row statistics) the sums go straight out
      const bool direct = (n_seg == 1) && p.epi == kEpiPlain && !p.ssq_in && !p.ssq_out && !p.end_combine;
      float* part = p.partials + ((size_t)row_tile * p.max_seg + split) * kXRows * kBlockRows;
      if constexpr (NT > 0) {
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const uint32_t m = nt * 8 + (lane & 3) * 2 + (r & 1);
            const uint32_t nl = warp * 16 + (lane >> 2) + (r >> 1) * 8;
            if (direct) {
              const uint32_t n = row_tile * kBlockRows + nl;
              if (m < p.M_b && n < p.N) store_out(p, m, n, acc[nt][r]);
            } else {
              __stcg(part + m * kBlockRows + nl, acc[nt][r]);
            }
          }
      } else {
        if ((lane & 7) == 0) {
#pragma unroll
          for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int m = 0; m < MB; ++m) {
              const uint32_t nl = warp * 16 + 4 * j + (lane >> 3);
              if (direct) {
                const uint32_t n = row_tile * kBlockRows + nl;
                if ((uint32_t)m < p.M_b && n < p.N) store_out(p, m, n, acc[j][m]);
              } else {
                __stcg(part + m * kBlockRows + nl, acc[j][m]);
              }
            }
        }
      }
      if (!direct && !p.end_combine) {
        // the threadblock that delivers the last partial sum of a row tile adds them up (in a
        // fixed order: deterministic) and writes the output
        if (!group_sync()) { failed = true; break; }
        if (tid == 0) {
          // release: publishes the partials of all consumer threads (ordered by the barrier);
          // acquire: the last to arrive reads the others' partials after this
          s_old = atom_add_acq_rel(tile_cnt + row_tile, 1u);
        }
        if (!group_sync()) { failed = true; break; }
        if (s_old == n_seg - 1) {   // ours was the last: leave the streaming loop for the combine
          mk = make_uint4(row_tile, 0u, 0u, mt.w);
          break;
        }
      }
    }
  }
  if (failed) break;
  // ---- outside the streaming loop: a row tile to combine (mk.z == 0: tile mk.x of phase mk.w),
  // or the marker that ends a phase or the launch.  One call of the combine serves both.
  // (the accumulators hold nothing here: saying so frees their registers for the combine)
#pragma unroll
  for (int i = 0; i < kAccN; ++i)
#pragma unroll
    for (int j = 0; j < kAccM; ++j) acc[i][j] = 0.f;
  {
    const uint4 mt = mk;
    const GemvParams& p = cp.ph[mt.w];
    const bool phase_end = (mt.z & (kFlagStop | kFlagPhaseEnd)) != 0;
    // Slots go to the warps of the grid in order, so only the first threadblocks have any; one
    // without has nothing to wait for once its own partial sums are out (after the last phase it
    // leaves at once and makes room for the next kernel's threadblocks).
    bool combines = !phase_end;
    const uint32_t combine_ctas = gridDim.x;
    if (phase_end && p.end_combine && !p.defer_combine) {
      // every threadblock's partial sums of this phase in memory -> all tiles combined, by all
      if (!group_sync()) break;
      combines = blockIdx.x < combine_ctas && blockIdx.x * kConsumerWarps < p.n_row_tiles * combine_slots_per_tile<kXRows>(p);
      if (tid == 0) {
        red_add_release(cp.bar + kBarPartials + mt.w, 1u);
        if (combines && !grid_counter_wait(cp.bar + kBarPartials + mt.w, gridDim.x, status)) s_abort = 1u;
      }
      if (combines && !group_sync()) break;
    }
    if (combines) {
      __threadfence();
      const bool all = phase_end;
      combine_units<kXRows>(p, all ? blockIdx.x * kConsumerWarps + warp : warp, all ? combine_ctas * kConsumerWarps : kConsumerWarps,
                            all ? kAllTiles : mt.x, lane, status);
    }
    if (!phase_end) {
      if (tid == 0) tile_cnt[mt.x] = 0;
      if (!group_sync()) break;   // (s_old may be rewritten, the tile's slots reused)
      continue;
    }
    // every consumer thread has finished this phase's items, combines included: publish
    // them and tell the grid (the x warps of all threadblocks wait for the count)
    if (!group_sync()) break;
    if (tid == 0) {
      if (mt.z & kFlagPhaseEnd) {
        if (blockIdx.x >= skip_arrivals_of(cp.ph[0].ws)) red_add_release(cp.bar + kBarPhase + mt.w, 1u);
      } else {
        __threadfence();
        // last threadblock out puts the counters back to zero for the next launch; by then
        // every warp of every threadblock has passed every counter it waits for
        const uint32_t old = atomicAdd(cp.bar + kBarExit, 1u);
        if (old == gridDim.x - 1) {
          for (uint32_t i = 0; i < (n_phases > 1 ? kBarWords : kBarPartials + 1); ++i) cp.bar[i] = 0u;
          __threadfence();
        }
      }
    }
    if (mt.z & kFlagStop) break;
    __syncwarp();
    if (lane == 0) mbar_arrive(&empty_bar[stage]);
    if (++stage == n_stages) { stage = 0; phase ^= 1u; }
  }
  }
  if (wait_failed) named_barrier_or(1, kConsumerThreads, true);   // the arrival the others' next group_sync counts on
}

// The combine of a product whose launch left it out (defer_combine): every row tile at once, the
// warps of this small grid taking slots in turn.  It follows the product on the stream with
// programmatic dependent launch, so its threadblocks are in place when the product's last
// threadblock leaves, and the kernel after it (attention, in a decode step) finds the SMs free:
// the product's threadblocks do not stay around for a combine that a handful of warps can do.
template <uint32_t kXRows>
__global__ void __launch_bounds__(kConsumerThreads) gemv_combine_kernel(const __grid_constant__ GemvParams p) {
  pdl_launch_dependents();
  // (combine_units waits for the product - its partial sums in memory - after it has requested
  // what does not depend on it)
  combine_units<kXRows, true>(p, blockIdx.x * kConsumerWarps + (threadIdx.x >> 5), gridDim.x * kConsumerWarps, kAllTiles,
                              threadIdx.x & 31u, p.ws + kWsStatus);
}

// ---------------------------------------------------------------------------------------------
// The same product on the 5th-generation tensor cores, for batches where it is a real dense
// contraction.  A packed weight block is already the A operand the hardware wants (128 rows,
// K-major, 128-byte swizzle); the activations of the block's 64 columns are staged as the B
// operand (NPAD rows, same layout); one thread issues four tcgen05.mma (K = 16 each) per block
// and the 128 x NPAD fp32 accumulator lives in tensor memory, double-buffered so that the
// next segment accumulates while the epilogue warps read the finished one back
// (tcgen05.ld), write the partial sums and run the same combine as the kernel above.
// Warps: 0-11 epilogue (warp w reads TMEM lanes 32 (w % 4) .. + 31 = weight rows, and the third
// w / 4 of the accumulator's 16-column chunks), 12 MMA issue and TMEM allocation, 13 weight
// producer (bulk copies; under the two-queue schedule 16-byte copies of all its lanes for
// host-tier blocks), 14 activation
// producer (one thread: a tiled TMA copy per stage lands x[:, 64 kb .. + 64) in the B operand's
// swizzled layout, rows beyond the batch as zeros).  Twelve epilogue warps because the combine of
// the partial sums is bound by what the warps of an SM can pull from L2 (eight: 163 us per chain
// of four products at batch 128, twelve: 154, sixteen - 96 registers per thread - 155).  Fifteen
// warps, four to an SM sub-partition at most: 128 registers per thread.  One threadblock per SM
// (the driver keeps kernels that allocate tensor memory at one per SM at this shared-memory size)
// with nearly all shared memory as its ring: no warp reads an operand back, so the ring's
// bandwidth is all HBM's.
constexpr uint32_t kTcEpiWarps = 12;
constexpr uint32_t kTcGroups = kTcEpiWarps / 4;   // warps w, w + 4, w + 8 share TMEM lanes 32 (w % 4) .. + 31 and split the columns
constexpr uint32_t kTcEpiThreads = kTcEpiWarps * 32;
constexpr uint32_t kTcThreads = kTcEpiThreads + 96;   // + MMA warp, weight producer, activation producer
// ring memory: what the epilogue's static arrays (row scales, the gate / up exchange buffer) leave
constexpr uint32_t kTcSmemBudget = kSmemBudget - 14u * 1024u;

// a stage: two weight blocks (the same 64 columns of two adjacent row tiles) and one activation tile
// (at 256 batch rows the activation tile alone is 32 KiB and tensor memory holds two accumulators
// of that width, not four: one weight block per stage, no pairs)
__host__ __device__ constexpr uint32_t tc_weight_slots(uint32_t npad) { return npad <= 128 ? 2u : 1u; }
__host__ __device__ constexpr uint32_t tc_stage_bytes(uint32_t npad) { return tc_weight_slots(npad) * kBlockBytes + npad * 128u; }

// A row tile finished from tensor memory by the threadblock that delivered its last partial sum:
// its own accumulator never goes to memory, the other segments' partial sums are added to it
// in the order the combine above uses for products with few partial sums per tile (ascending
// segments), and the epilogue runs in the accumulator's own layout - thread = weight row (TMEM
// lane), 32 batch rows at a time (16 for small batches).  For the epilogues that
// need nothing across weight rows but the gate / up partner 64 rows on, which changes hands
// through shared memory: SwiGLU, and plain without sums of squares of the output.
// s_rs: row scales of the phase (filled by the caller when the product has row statistics);
// s_exch: kTcGroups x tc_finish_cols x 64 floats.  Called by all epilogue warps.
// columns (batch rows) per pass of tc_finish_tile
template <uint32_t NPAD>
__host__ __device__ constexpr uint32_t tc_finish_cols() { return 16u; }

template <uint32_t NPAD>
__device__ __forceinline__ void tc_finish_tile(const GemvParams& p, uint32_t row_tile, uint32_t my_seg, uint32_t n_seg,
                                               uint32_t taddr, uint32_t warp, uint32_t lane, const float* s_rs,
                                               float* s_exch) {
  constexpr uint32_t kC = tc_finish_cols<NPAD>();
  const uint32_t quarter = warp & 3u, group = warp >> 2;
  const uint32_t nl = quarter * 32u + lane;
  // the column chunks of the accumulator, shared out between the groups of four warps
  constexpr uint32_t kChunks = NPAD / kC;
  const uint32_t c_begin = kChunks * group / kTcGroups * kC, c_end = kChunks * (group + 1) / kTcGroups * kC;
  const float* part0 = p.partials + (size_t)row_tile * p.max_seg * NPAD * kBlockRows + nl;
  for (uint32_t c0 = c_begin; c0 < c_end; c0 += kC) {
    float acc[kC];
#pragma unroll
    for (uint32_t j = 0; j < kC; ++j) acc[j] = 0.f;
    for (uint32_t seg = 0; seg < n_seg; ++seg) {
      // from memory, or (this threadblock's own) from tensor memory
      float v[kC];
      if (seg != my_seg) {
        const float* ps = part0 + ((size_t)seg * NPAD + c0) * kBlockRows;
#pragma unroll
        for (uint32_t j = 0; j < kC; ++j) v[j] = __ldcg(ps + j * kBlockRows);
      } else {
        tmem_ld<kC>(taddr + c0, v);
      }
#pragma unroll
      for (uint32_t j = 0; j < kC; ++j) acc[j] += v[j];
    }
    if (p.ssq_in) {
#pragma unroll
      for (uint32_t j = 0; j < kC; ++j) acc[j] *= s_rs[c0 + j];
    }
    if (p.epi == kEpiSwiglu) {
      // rows 64 .. 127 of the tile are the up rows of the gate rows 0 .. 63
      float* ex = s_exch + group * (kC * 64u);
      if (quarter >= 2) {
#pragma unroll
        for (uint32_t j = 0; j < kC; ++j) ex[j * 64u + (nl - 64u)] = acc[j];
      }
      named_barrier_sync(3 + group, 128);
      if (quarter < 2) {
        __nv_bfloat16* out = static_cast<__nv_bfloat16*>(p.y) + (size_t)row_tile * 64u + nl;
#pragma unroll
        for (uint32_t j = 0; j < kC; ++j) {
          const uint32_t m = c0 + j;
          if (m < p.M_b) {
            const float g = round_bf16(acc[j]), u = round_bf16(ex[j * 64u + nl]);
            out[(size_t)m * (p.N / 2)] = __float2bfloat16_rn(g / (1.f + expf(-g)) * u);
          }
        }
      }
      named_barrier_sync(3 + group, 128);   // (the next pass overwrites the exchange buffer)
    } else {
      const uint32_t n = row_tile * kBlockRows + nl;
#pragma unroll
      for (uint32_t j = 0; j < kC; ++j) {
        const uint32_t m = c0 + j;
        if (m < p.M_b && n < p.N) store_out(p, m, n, acc[j]);
      }
    }
  }
}

template <uint32_t NPAD>
__global__ void __launch_bounds__(kTcThreads, 1) gemv_tc_kernel(const __grid_constant__ TcChainParams tp) {
  const ChainParams& cp = tp.chain;
  constexpr uint32_t kStageBytes = tc_stage_bytes(NPAD);
  constexpr uint32_t kSlots = tc_weight_slots(NPAD);
  constexpr uint32_t kTmemCols = 2 * kSlots * NPAD < 32 ? 32 : 2 * kSlots * NPAD;   // one accumulator per weight slot, double-buffered
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  __shared__ uint64_t full_bar[kMaxStages];
  __shared__ uint64_t empty_bar[kMaxStages];
  __shared__ uint4 meta[kMaxStages];
  __shared__ uint64_t item_full[4];
  __shared__ uint64_t item_empty[4];
  __shared__ uint32_t item_ring[4];
  __shared__ uint64_t acc_full[2];
  __shared__ uint64_t acc_empty[2];
  __shared__ uint4 acc_meta[2];
  __shared__ uint32_t s_tmem;
  __shared__ uint32_t s_go[2];          // epilogue: thread 0's wait on an accumulator succeeded
  __shared__ volatile uint32_t s_abort; // a bounded wait ran out somewhere: everybody winds down
  __shared__ uint32_t s_rs_phase;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t n_stages = cp.ph[0].n_stages;
  const uint32_t n_phases = cp.n_phases;
  uint32_t* status = cp.ph[0].ws + kWsStatus;

  pdl_launch_dependents();
  if (tid == 0) {
    for (uint32_t s = 0; s < n_stages; ++s) {
      mbar_init(&full_bar[s], 34);   // the two producers' arrive.expect_tx + the cp.async arrivals of the weight warp
      mbar_init(&empty_bar[s], 1);   // the commit of the MMAs that read the stage
    }
    for (uint32_t s = 0; s < 4; ++s) {
      mbar_init(&item_full[s], 1);
      mbar_init(&item_empty[s], 1);
    }
    for (uint32_t s = 0; s < 2; ++s) {
      mbar_init(&acc_full[s], 1);
      mbar_init(&acc_empty[s], kTcEpiWarps);
    }
    s_abort = 0;
    s_rs_phase = 0xFFFFFFFFu;
    fence_barrier_init();
  }
  if (warp == kTcEpiWarps) tmem_alloc(&s_tmem, kTmemCols);
  tc_fence_before_sync();
  __syncthreads();
  tc_fence_after_sync();
  const uint32_t tmem_base = s_tmem;

  if (warp > kTcEpiWarps) {
    // ------------------------------------------------------------------ producer warps (as above)
    const bool leader = (warp == kTcEpiWarps + 1);
    if (!leader && lane == 0)   // the phases' tensor maps: fetched now, not at each phase's first copy
      for (uint32_t ph = 0; ph < n_phases; ++ph) tma_prefetch_map(&tp.x_map[ph]);
    uint32_t stage = 0, phase = 0, icount = 0;
    unsigned long long* const sched_log = (leader && lane == 0) ? sched_log_of(cp.ph[0].ws) : nullptr;
    uint32_t rec = kNoRecord;   // schedule-log record of the item in production (weight warp, lane 0)
    for (uint32_t ph = 0; ph < n_phases; ++ph) {
      const GemvParams& p = cp.ph[ph];
      const uint32_t n_host_items = p.n_host_pages * p.items_per_page;
      TierQueues q;
      const bool active = blockIdx.x < p.active_ctas;
      if (active && !p.even_part) q.init(p.queue, n_host_items, p.n_pages * p.items_per_page, p.n_host_ctas, blockIdx.x, p.active_ctas);
      if (ph == 0) {
        if (!leader || !p.early) pdl_wait();
      } else if (!leader) {
        if (lane == 0 && !grid_counter_wait(cp.bar + kBarPhase + (ph - 1), gridDim.x, status)) s_abort = 1;
        __syncwarp();
      }
      // (the activations were written with ordinary stores, by this launch or the one before,
      // and are read through the TMA unit)
      if (!leader) fence_proxy_async_all();
      // one stage: the weight warp copies the weight block (two blocks in pair mode), the
      // activation producer requests x[:, 64 kb .. 64 kb + 64) as NPAD rows of 128 bytes in the
      // 128-byte swizzle (rows >= M_b are zero)
      auto produce = [&](const uint8_t* src, const uint8_t* src1, bool from_host, uint32_t row_tile, uint32_t seg,
                         uint32_t flags, uint32_t kb) {
        if (s_abort) return;
        if (leader) {
          uint8_t* wdst = smem + (size_t)stage * kStageBytes;
          if (lane == 0) {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1u, status)) s_abort = 1;
            meta[stage] = make_uint4(row_tile, seg, flags | (from_host ? kFlagHost : 0u) | (rec << 8), ph);
            mbar_arrive_expect_tx(&full_bar[stage], from_host ? 0u : ((flags & kFlagSecond) ? 2 * kBlockBytes : kBlockBytes));
            if (!from_host) {
              bulk_copy_g2s(wdst, src, kBlockBytes, &full_bar[stage]);
              if (flags & kFlagSecond) bulk_copy_g2s(wdst + kBlockBytes, src1, kBlockBytes, &full_bar[stage]);
            }
          }
          __syncwarp();
          if (from_host) {
#pragma unroll 8
            for (uint32_t idx = lane; idx < kBlockBytes / 16; idx += 32) cp_async_16(wdst + idx * 16, src + idx * 16, 16u);
          }
          cp_async_arrive_noinc(&full_bar[stage]);
        } else {
          if (lane == 0) {
            if (!mbar_wait(&empty_bar[stage], phase ^ 1u, status)) s_abort = 1;
            mbar_arrive_expect_tx(&full_bar[stage], NPAD * 128u);
            tma_load_2d(smem + (size_t)stage * kStageBytes + kSlots * kBlockBytes, &tp.x_map[ph], (int32_t)(kb * kBlockK), 0,
                        &full_bar[stage]);
          }
          __syncwarp();
        }
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
      };
      if (p.even_part) {
        // The unit is (row tile, kb) or, for long matrices, (pair of adjacent row tiles, kb): both
        // weight blocks then meet the same activation tile, which halves the activation traffic
        // from L2 and its share of the ring (short matrices keep single tiles: pairs would double
        // the partial sums per tile).  Threadblock c of G takes units [c T2 / G, (c + 1) T2 / G).
        const uint32_t G = p.active_ctas, tpu = p.tiles_per_unit;
        const uint32_t n_pairs = (p.n_row_tiles + tpu - 1) / tpu, T2 = n_pairs * p.k_blocks;
        if (blockIdx.x < G) {
          const uint32_t u0 = (uint32_t)((uint64_t)blockIdx.x * T2 / G), u1 = (uint32_t)((uint64_t)(blockIdx.x + 1) * T2 / G);
          uint32_t pair = u0 / p.k_blocks, kb = u0 % p.k_blocks;
          uint32_t seg = blockIdx.x - part_owner((uint64_t)pair * p.k_blocks, G, T2);
          const uint8_t* page_base[2] = {nullptr, nullptr};   // looked up once per page (an L2 round trip)
          uint32_t page_of_base[2] = {0xFFFFFFFFu, 0xFFFFFFFFu};
          for (uint32_t u = u0; u < u1; ++u) {
            const bool seg_first = (u == u0) || kb == 0, seg_last = (u + 1 == u1) || (kb + 1 == p.k_blocks);
            const bool second = tpu == 2 && 2 * pair + 1 < p.n_row_tiles;
            const uint8_t* src[2] = {nullptr, nullptr};
            if (leader && lane == 0) {
#pragma unroll
              for (uint32_t h = 0; h < 2; ++h) {
                if (h == 1 && !second) break;
                const uint32_t b = (tpu * pair + h) * p.k_blocks + kb;
                if (b / kBlocksPerPage != page_of_base[h]) {
                  page_of_base[h] = b / kBlocksPerPage;
                  page_base[h] = static_cast<const uint8_t*>(p.w_page_ptr[page_of_base[h]]);
                }
                src[h] = page_base[h] + (size_t)(b % kBlocksPerPage) * kBlockBytes;
              }
              if (seg_first && sched_log) {   // the segment: units up to the end of the row tile (pair) or of this threadblock's range
                const uint32_t n_seg_units = min(u1 - u, p.k_blocks - kb);
                uint32_t host_bytes = 0;
                if (p.n_host_pages) {
                  host_bytes = host_bytes_of_blocks(p, tpu * pair * p.k_blocks + kb, n_seg_units);
                  if (second) host_bytes += host_bytes_of_blocks(p, (tpu * pair + 1) * p.k_blocks + kb, n_seg_units);
                }
                rec = sched_log_begin(sched_log, BOOST_SCHED_KIND_GEMV | (ph << 8), blockIdx.x | (warp << 24),
                                      n_seg_units * (second ? 2u : 1u) * kBlockBytes, host_bytes);
              }
            }
            produce(src[0], src[1], false, tpu * pair, seg,
                    kFlagPair | (second ? kFlagSecond : 0u) | (seg_first ? kFlagFirst : 0u) | (seg_last ? kFlagLast : 0u), kb);
            if (++kb == p.k_blocks) { kb = 0; ++pair; seg = 0; }
          }
        }
      } else {
        for (;;) {
          const uint32_t slot = icount & 3u, iphase = (icount >> 2) & 1u;
          uint32_t qi = 0;
          if (leader) {
            if (lane == 0) {
              for (;;) {   // skip the unused tail of the last page
                qi = active ? q.next() : 0xFFFFFFFFu;
                if (qi == 0xFFFFFFFFu) break;
                if (p.w_order[qi / p.items_per_page] * p.items_per_page + qi % p.items_per_page < p.n_items) break;
              }
              if (!mbar_wait(&item_empty[slot], iphase ^ 1u, status)) { s_abort = 1; qi = 0xFFFFFFFFu; }
              item_ring[slot] = qi;
              mbar_arrive(&item_full[slot]);
            }
            qi = __shfl_sync(0xFFFFFFFFu, qi, 0);
          } else {
            const bool got = mbar_wait(&item_full[slot], iphase, status);
            qi = got ? item_ring[slot] : 0xFFFFFFFFu;
            if (!got) s_abort = 1;
            __syncwarp();
            if (lane == 0) mbar_arrive(&item_empty[slot]);
          }
          ++icount;
          if (qi == 0xFFFFFFFFu) break;
          const uint32_t page = p.w_order[qi / p.items_per_page];
          const uint32_t first_blk = (page * p.items_per_page + qi % p.items_per_page) * p.run;
          const uint32_t row_tile = first_blk / p.k_blocks, kb0 = first_blk % p.k_blocks;
          const bool from_host = qi < n_host_items;
          const uint8_t* src = static_cast<const uint8_t*>(p.w_page_ptr[page]) + (size_t)(first_blk % kBlocksPerPage) * kBlockBytes;
          if (leader && lane == 0)
            rec = sched_log_begin(sched_log, BOOST_SCHED_KIND_GEMV | (ph << 8), blockIdx.x | (warp << 24), p.run * kBlockBytes,
                                  from_host ? p.run * kBlockBytes : 0u);
          for (uint32_t j = 0; j < p.run; ++j, src += kBlockBytes)
            produce(src, nullptr, from_host, row_tile, kb0 / p.run, (j == 0 ? kFlagFirst : 0u) | (j + 1 == p.run ? kFlagLast : 0u), kb0 + j);
        }
      }
      // a stage without data tells the MMA warp that the phase (or the launch) is over
      if (leader) {
        if (lane == 0) {
          mbar_wait(&empty_bar[stage], phase ^ 1u, status);
          meta[stage] = make_uint4(0u, 0u, ph + 1 == n_phases ? kFlagStop : kFlagPhaseEnd, ph);
          mbar_arrive(&full_bar[stage]);
        }
        __syncwarp();
        cp_async_arrive_noinc(&full_bar[stage]);
        if (lane == 0 && active && !p.even_part) q.finish(p.active_ctas);
      } else {
        if (lane == 0) {
          mbar_wait(&empty_bar[stage], phase ^ 1u, status);
          mbar_arrive(&full_bar[stage]);
        }
        __syncwarp();
      }
      if (++stage == n_stages) { stage = 0; phase ^= 1u; }
    }
    return;
  }

  if (warp == kTcEpiWarps) {
    // ------------------------------------------------------------------ MMA warp: one thread issues
    if (lane == 0) {
      constexpr uint32_t idesc = umma_idesc_bf16_f32(kBlockRows, NPAD);
      uint32_t stage = 0, phase = 0, buf = 0, buf_phase = 0, accumulate = 0;
      for (;;) {
        if (s_abort || !mbar_wait(&full_bar[stage], phase, status)) { s_abort = 1; break; }
        const uint4 mt = meta[stage];
        if (mt.z & (kFlagStop | kFlagPhaseEnd)) {
          // hand the marker to the epilogue warps in order with the segments
          if (!mbar_wait(&acc_empty[buf], buf_phase ^ 1u, status)) { s_abort = 1; break; }
          acc_meta[buf] = mt;
          mbar_arrive(&acc_full[buf]);
          if (++buf == 2) { buf = 0; buf_phase ^= 1u; }
          mbar_arrive(&empty_bar[stage]);
          if (++stage == n_stages) { stage = 0; phase ^= 1u; }
          if (mt.z & kFlagStop) break;
          continue;
        }
        if (mt.z & kFlagFirst) {
          if (!mbar_wait(&acc_empty[buf], buf_phase ^ 1u, status)) { s_abort = 1; break; }   // the epilogue has read this accumulator
          accumulate = 0;
        }
        fence_proxy_async_smem();   // x (and host-tier weight blocks) were written through the load/store path
        tc_fence_after_sync();
        const uint32_t wbase = smem_u32(smem + (size_t)stage * kStageBytes);
        const uint32_t xbase = wbase + kSlots * kBlockBytes;
        const uint32_t d0 = tmem_base + buf * kSlots * NPAD;   // accumulator of the first row tile; the second follows it
#pragma unroll
        for (uint32_t ks = 0; ks < kBlockK / 16; ++ks) {
          const uint64_t xdesc = umma_desc_k_sw128(xbase + ks * 32);
          umma_bf16(d0, umma_desc_k_sw128(wbase + ks * 32), xdesc, idesc, accumulate);
          if (mt.z & kFlagSecond) umma_bf16(d0 + NPAD, umma_desc_k_sw128(wbase + kBlockBytes + ks * 32), xdesc, idesc, accumulate);
          accumulate = 1;
        }
        umma_commit(&empty_bar[stage]);   // the stage is free once these MMAs have read it
        if (mt.z & kFlagLast) {
          acc_meta[buf] = mt;
          umma_commit(&acc_full[buf]);    // the accumulator is complete once they have finished
          if (++buf == 2) { buf = 0; buf_phase ^= 1u; }
        }
        if (++stage == n_stages) { stage = 0; phase ^= 1u; }
      }
    }
    __syncwarp();
    named_barrier_sync(2, kTcEpiThreads + 32);   // the epilogue warps have read everything
    tmem_dealloc(tmem_base, kTmemCols);
    return;
  }

  // -------------------------------------------------------------------- epilogue warps
  // Each round of the loop takes one accumulator (or phase marker) from the MMA warp and ends
  // with at most two combines - the row tiles of the accumulator whose last partial sum this
  // threadblock delivered, or all tiles of a phase at its end - through ONE call of the combine,
  // so that its code (and register needs) exist once in the kernel.
  uint32_t* tile_cnt = cp.ph[0].ws + kWsHeaderWords;
  __shared__ uint32_t s_last[2];
  __shared__ float s_rs[NPAD];           // row scales of phase s_rs_phase (tc_finish_tile)
  __shared__ float s_exch[kTcGroups * tc_finish_cols<NPAD>() * 64];
  uint32_t buf = 0, buf_phase = 0;
  pdl_wait();
  for (;;) {
    // thread 0 waits for the accumulator (or marker) and tells the others, so that all 256
    // threads take the same way out if the wait runs out
    if (tid == 0) {
      const bool ok = mbar_wait(&acc_full[buf], buf_phase, status);
      if (!ok) s_abort = 1;
      s_go[buf] = ok ? 1u : 0u;
    }
    named_barrier_sync(1, kTcEpiThreads);
    if (!s_go[buf]) break;
    const uint4 mt = acc_meta[buf];
    const GemvParams& p = cp.ph[mt.w];
    const bool phase_end = (mt.z & (kFlagStop | kFlagPhaseEnd)) != 0;
    uint32_t n_jobs = 0, job[2] = {0u, 0u};   // row tiles to combine, or kAllTiles
    if (phase_end) {
      if (p.end_combine && !p.defer_combine) {
        // every threadblock's partial sums of this phase in memory -> all tiles combined, by the
        // epilogue warps of the whole grid (see combine_units)
        const bool combines = blockIdx.x * kTcEpiWarps < p.n_row_tiles * combine_slots_per_tile<NPAD>(p);
        if (tid == 0) {
          red_add_release(cp.bar + kBarPartials + mt.w, 1u);   // (the barrier above ordered everybody's stores before this)
          bool ok = true;
          if (combines && !grid_counter_wait(cp.bar + kBarPartials + mt.w, gridDim.x, status)) { s_abort = 1; ok = false; }
          s_go[buf] = ok ? 1u : 0u;
        }
        named_barrier_sync(1, kTcEpiThreads);
        if (!s_go[buf]) break;
        if (combines) job[n_jobs++] = kAllTiles;
      }
    } else {
      tc_fence_after_sync();
      if (tid == 0 && (mt.z >> 8) != kNoRecord) sched_log_end(sched_log_of(cp.ph[0].ws), mt.z >> 8);
      const uint32_t split = mt.y;
      const uint32_t n_tiles = (mt.z & kFlagSecond) ? 2u : 1u;   // row tiles in this accumulator
      const uint32_t n_seg = p.even_part ? even_part_segments(p, mt.x) : p.splits;   // (the same for both tiles of a pair)
      const uint32_t quarter = warp & 3u, group = warp >> 2;
      const uint32_t nl = quarter * 32 + lane;                                 // weight row of this thread = its TMEM lane
      // the accumulator's columns in chunks of 16, shared out between the groups of four warps
      constexpr uint32_t kChunks = NPAD / 16;
      const uint32_t c_begin = kChunks * group / kTcGroups * 16, c_end = kChunks * (group + 1) / kTcGroups * 16;
      // Tile by tile, with an epilogue that works in the accumulator's layout: whoever holds
      // the last partial sum of a tile keeps it in tensor memory and finishes the tile from
      // there (tc_finish_tile); the others write theirs out.  A tile's counter holds the
      // arrivals in its low half and the partial sums in memory in its high half.
      const bool native = !p.end_combine && p.max_seg <= combine_per_round<NPAD>() &&
                          (p.epi == kEpiSwiglu || (p.epi == kEpiPlain && !p.ssq_out));
      if (native && n_seg > 1) {
        if (tid < n_tiles) s_last[tid] = ((atomicAdd(tile_cnt + mt.x + tid, 1u) & 0xFFFFu) == n_seg - 1) ? 1u : 0u;
        named_barrier_sync(1, kTcEpiThreads);
      }
      bool stored = false;
      for (uint32_t ti = 0; ti < n_tiles; ++ti) {
        if (native && (n_seg == 1 || s_last[ti])) continue;
        stored = true;
        const uint32_t row_tile = mt.x + ti;
        float* part = p.partials + ((size_t)row_tile * p.max_seg + split) * NPAD * kBlockRows;
        const uint32_t taddr = tmem_base + ((quarter * 32u) << 16) + buf * kSlots * NPAD + ti * NPAD;
        for (uint32_t c0 = c_begin; c0 < c_end; c0 += 16) {
          float v[16];
          tmem_ld16(taddr + c0, v);
#pragma unroll
          for (uint32_t j = 0; j < 16; ++j) __stcg(part + (c0 + j) * kBlockRows + nl, v[j]);   // batch row = accumulator column
        }
      }
      if (native) {
        if (stored) {
          named_barrier_sync(1, kTcEpiThreads);   // everybody's stores come before the release
          if (tid < n_tiles && !s_last[tid] && blockIdx.x >= skip_arrivals_of(cp.ph[0].ws)) red_add_release(tile_cnt + mt.x + tid, 0x10000u);
        }
        bool gave_up = false;
        for (uint32_t ti = 0; ti < n_tiles; ++ti) {
          if (n_seg > 1 && !s_last[ti]) continue;
          const uint32_t row_tile = mt.x + ti;
          if (n_seg > 1) {
            // the other segments' partial sums: all in memory?  (their threadblocks are past
            // their arrival and wait for nothing on the way to the release)
            if (tid == 0) {
              const bool ok = grid_counter_wait(tile_cnt + row_tile, (n_seg - 1) << 16, status);
              if (!ok) s_abort = 1;
              s_go[buf] = ok ? 1u : 0u;
            }
            named_barrier_sync(1, kTcEpiThreads);
            if (!s_go[buf]) { gave_up = true; break; }
            __threadfence();
          }
          if (p.ssq_in) {
            // row scales of this phase's activations, once per phase (in the combine's order of sums)
            named_barrier_sync(1, kTcEpiThreads);
            if (s_rs_phase != mt.w) {
              const uint32_t v = tid & 15u;
              for (uint32_t m_base = 0; m_base < NPAD; m_base += kTcEpiThreads / 16) {   // (every warp the same number of passes: it shuffles)
                const uint32_t m = m_base + (tid >> 4);
                float ss = 0.f, ss0 = 0.f, ss1 = 0.f;
                if (m < p.M_b && m < NPAD) {
                  if (v < p.ssq_in_tiles) ss0 = __ldcg(p.ssq_in + (size_t)v * p.ssq_stride + m);
                  if (v + 16 < p.ssq_in_tiles) ss1 = __ldcg(p.ssq_in + (size_t)(v + 16) * p.ssq_stride + m);
                  for (uint32_t t0 = v + 32; t0 < p.ssq_in_tiles; t0 += 16) ss += __ldcg(p.ssq_in + (size_t)t0 * p.ssq_stride + m);
                }
                ss += ss0 + ss1;
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 1);
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 2);
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 4);
                ss += __shfl_xor_sync(0xFFFFFFFFu, ss, 8);
                if (v == 0 && m < NPAD) s_rs[m] = rsqrtf(ss / (float)p.x_cols + p.rms_eps);
              }
              named_barrier_sync(1, kTcEpiThreads);
              if (tid == 0) s_rs_phase = mt.w;
            }
          }
          tc_finish_tile<NPAD>(p, row_tile, split, n_seg, tmem_base + ((quarter * 32u) << 16) + buf * kSlots * NPAD + ti * NPAD, warp,
                               lane, s_rs, s_exch);
          if (n_seg > 1 && tid == 0) tile_cnt[row_tile] = 0;
        }
        if (gave_up) break;
      }
      // the accumulators may be overwritten
      tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
      if (++buf == 2) { buf = 0; buf_phase ^= 1u; }
      if (!native && !p.end_combine) {
        // the threadblock that delivers the last partial sum of a row tile combines it
        named_barrier_sync(1, kTcEpiThreads);
        if (tid < n_tiles) s_last[tid] = atom_add_acq_rel(tile_cnt + mt.x + tid, 1u) == n_seg - 1 ? 1u : 0u;   // release ours, acquire the others'
        named_barrier_sync(1, kTcEpiThreads);
        for (uint32_t ti = 0; ti < n_tiles; ++ti)
          if (s_last[ti]) job[n_jobs++] = mt.x + ti;
      }
    }
    for (uint32_t j = 0; j < n_jobs; ++j) {
      const bool all = job[j] == kAllTiles;
      __threadfence();
      combine_units<NPAD>(p, all ? blockIdx.x * kTcEpiWarps + warp : warp, all ? gridDim.x * kTcEpiWarps : kTcEpiWarps, job[j], lane,
                          status);
      if (!all && tid == 0) tile_cnt[job[j]] = 0;
    }
    if (n_jobs && !phase_end) named_barrier_sync(1, kTcEpiThreads);   // (s_last may be rewritten, the tiles' slots reused)
    if (phase_end) {
      named_barrier_sync(1, kTcEpiThreads);
      if (tid == 0) {
        if (mt.z & kFlagPhaseEnd) {
          if (blockIdx.x >= skip_arrivals_of(cp.ph[0].ws)) red_add_release(cp.bar + kBarPhase + mt.w, 1u);
        } else {
          __threadfence();
          const uint32_t old = atomicAdd(cp.bar + kBarExit, 1u);
          if (old == gridDim.x - 1) {
            for (uint32_t i = 0; i < (n_phases > 1 ? kBarWords : kBarPartials + 1); ++i) cp.bar[i] = 0u;
            __threadfence();
          }
        }
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(&acc_empty[buf]);
      if (++buf == 2) { buf = 0; buf_phase ^= 1u; }
      if (mt.z & kFlagStop) break;
    }
  }
  named_barrier_sync(2, kTcEpiThreads + 32);
}

// Packed form: 16-byte chunk `pos` of row r of block (t, kb) holds columns
// [64 kb + 8 c, +8) of packed row 128 t + r with c = pos ^ (r & 7).  Packed row -> weight row:
// identity, or (row_mode 1) rows 0..63 of a tile = rows [64 t, 64 t + 64) of the first half of
// W and rows 64..127 the same rows of the second half (gate and up rows side by side).
// col_scale (bf16 [K], optional) multiplies column k: an RMSNorm weight folded into W.
__global__ void __launch_bounds__(256)
pack_weights_kernel(const uint4* __restrict__ w, uint32_t N, uint32_t K, uint32_t k_blocks,
                    size_t n_chunks, const void* const* __restrict__ page_ptr, int row_mode,
                    const uint4* __restrict__ col_scale) {
  const size_t stride = (size_t)gridDim.x * blockDim.x;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_chunks; i += stride) {
    const size_t blk = i / (kBlockBytes / 16);
    const uint32_t in_blk = (uint32_t)(i % (kBlockBytes / 16));
    const uint32_t r = in_blk >> 3, pos = in_blk & 7, c = pos ^ (r & 7);
    const uint32_t t = (uint32_t)(blk / k_blocks), kb = (uint32_t)(blk % k_blocks);
    uint32_t row = t * kBlockRows + r;
    if (row_mode == 1) row = (r < 64) ? t * 64 + r : N / 2 + t * 64 + (r - 64);
    const uint32_t k = kb * kBlockK + c * 8;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (row < N && k < K) {
      v = w[((size_t)row * K + k) / 8];
      if (col_scale) {
        const uint4 g = col_scale[k / 8];
        const uint32_t wv[4] = {v.x, v.y, v.z, v.w}, gv[4] = {g.x, g.y, g.z, g.w};
        uint32_t o[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const __nv_bfloat162 pr = __floats2bfloat162_rn(bf16_lo(wv[j]) * bf16_lo(gv[j]), bf16_hi(wv[j]) * bf16_hi(gv[j]));
          o[j] = *reinterpret_cast<const uint32_t*>(&pr);
        }
        v = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
    const size_t off = i * 16;
    uint4* dst = reinterpret_cast<uint4*>(static_cast<uint8_t*>(const_cast<void*>(page_ptr[off / kPageBytes])) +
                                          off % kPageBytes);
    *dst = v;
  }
}

uint32_t pick_run(uint32_t n_row_tiles, uint32_t k_blocks) {
  // Run length of a work item in blocks: a power of two that divides the row tile's
  // k_blocks (and so the 128 blocks of a page).  Every run ends with a split-K partial sum
  // that is written, fenced and later re-read, and on B200 that costs more than a coarse
  // split of the work (measured): take the longest run that still leaves one item per SM,
  // else the longest that leaves 64 items, else single blocks.
  const uint64_t total = (uint64_t)n_row_tiles * k_blocks;
  const uint64_t wanted[2] = {148, 64};
  for (int pass = 0; pass < 2; ++pass)
    for (uint32_t run = 32; run >= 1; run >>= 1)
      if (k_blocks % run == 0 && total / run >= wanted[pass]) return run;
  return 1;
}

// Combine-at-phase-end on (1) or off (0: every tile by its last arriver), for measurements; and
// whether the last phase's combine goes to a kernel of its own.
// 0: host pages are read in place under the even partition; 1: two queues of work items, host pages first
uint32_t g_tier_schedule = 0;
uint32_t g_end_combine = 1;
uint32_t g_defer_combine = 1;

// Common launch path of the two kernels: ring depth from the shared-memory budget, grid and
// per-phase threadblock counts, host-tier threadblocks.  `state` keeps what is set up once per
// kernel instantiation.
struct KernelState {
  bool configured = false;
  int resident = 0;   // threadblocks of the kernel that one SM holds at its shared-memory size
};

// pairs: the even partition counts (pair of row tiles, k block) units instead of blocks.
template <typename KernelParams, typename Wrap>
int launch_planned(void (*kernel)(KernelParams), Wrap wrap, void (*combine_kernel)(GemvParams), uint32_t x_rows, KernelState& state,
                   uint32_t threads, uint32_t stage_bytes, uint32_t smem_budget, uint32_t ctas_per_sm, bool pairs, bool end_combine_allowed,
                   const ChainParams& chain, int sms, cudaStream_t stream, uint32_t* extra_launches) {
  ChainParams c = chain;
  uint32_t n_stages = (smem_budget / ctas_per_sm - 1024) / stage_bytes;
  if (n_stages > kMaxStages) n_stages = kMaxStages;
  const size_t smem = (size_t)n_stages * stage_bytes + 1024;
  if (!state.configured) {
    int rc = boosth::check(cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(smem_budget + 1024)));
    if (rc != BOOST_OK) return rc;
    rc = boosth::check(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&state.resident, kernel, (int)threads, smem));
    if (rc != BOOST_OK) return rc;
    state.configured = true;
  }
  // The phases of a chain, and the threadblocks of a product that combines its tiles at the end,
  // meet at grid-wide counters: every threadblock must be resident.
  if (state.resident < 1) return BOOST_ERR_UNSUPPORTED;
  if ((uint32_t)state.resident < ctas_per_sm) ctas_per_sm = (uint32_t)state.resident;
  const uint32_t max_ctas = (uint32_t)sms * ctas_per_sm;
  uint32_t grid = 0;
  for (uint32_t i = 0; i < c.n_phases; ++i) {
    GemvParams& q = c.ph[i];
    q.n_stages = n_stages;
    // Threadblocks share HBM bandwidth, so what has to be even is the number of items per
    // threadblock: use as many blocks as give every block the same count (rounded up).
    const uint32_t queue_len = q.n_pages * q.items_per_page;
    const uint32_t items = q.n_items ? q.n_items : 1;
    const uint32_t per_cta = (items + max_ctas - 1) / max_ctas;
    uint32_t g = (items + per_cta - 1) / per_cta;
    if (g > queue_len) g = queue_len;
    if (q.even_part) {
      // at least one unit per threadblock: the partial-sum slots of a row tile are sized for that
      // pairs of row tiles wherever every threadblock still gets two units or more: a stage then
      // carries two weight blocks, and a single tile would leave half of the ring empty
      // (measured, batch 64, down product 4096 x 14336: 61 -> 46 us inside a chain)
      q.tiles_per_unit = (pairs && (uint64_t)((q.n_row_tiles + 1) / 2) * q.k_blocks >= 2ull * max_ctas) ? 2u : 1u;
      const uint32_t units = ((q.n_row_tiles + q.tiles_per_unit - 1) / q.tiles_per_unit) * q.k_blocks;
      g = units < max_ctas ? units : max_ctas;
    }
    q.active_ctas = g;
    if (g > grid) grid = g;
    // Partial sums per row tile, typically: with ten or so (short products cut over the whole
    // machine) all tiles complete together at the end of the phase, and they are combined then.
    uint32_t typical_seg = q.splits;
    if (q.even_part) {
      const uint32_t units = ((q.n_row_tiles + q.tiles_per_unit - 1) / q.tiles_per_unit) * q.k_blocks;
      const uint32_t per_cta2 = units / g ? units / g : 1;
      typical_seg = (q.k_blocks + per_cta2 - 1) / per_cta2;
    }
    // From 64 batch rows on (tcgen05 kernel) a tile's combine takes a threadblock's eight warps
    // ten microseconds and more; where a threadblock holds under two units, every tile's combine
    // would wait at the end of the phase behind its last partial sum anyway: all at once, then.
    bool few_units = false;
    if (q.even_part && x_rows >= 64) {
      const uint32_t units = ((q.n_row_tiles + q.tiles_per_unit - 1) / q.tiles_per_unit) * q.k_blocks;
      few_units = units < 2u * g * q.k_blocks;   // (a unit = one k block of a tile or pair)
    }
    q.end_combine = (end_combine_allowed && (typical_seg >= kEndCombineMinSegments || few_units)) ? 1u : 0u;
    q.defer_combine = (q.end_combine && i + 1 == c.n_phases && g_defer_combine) ? 1u : 0u;
  }
  // a chain keeps one grid for all phases: the full machine, so that threadblocks that run
  // out of items in one phase stream ahead in the next
  if (c.n_phases > 1) grid = max_ctas;
  for (uint32_t i = 0; i < c.n_phases; ++i) {
    GemvParams& q = c.ph[i];
    uint32_t n_host_ctas = 0;
    if (q.n_host_pages) {
      n_host_ctas = 8;
      if (n_host_ctas > q.n_host_pages * q.items_per_page) n_host_ctas = q.n_host_pages * q.items_per_page;
      if (n_host_ctas > q.active_ctas) n_host_ctas = q.active_ctas;
    }
    q.n_host_ctas = n_host_ctas;
  }
  int rc = boosth::launch_chained(kernel, dim3(grid), dim3(threads), smem, stream, wrap(c));
  const GemvParams& last = c.ph[c.n_phases - 1];
  if (rc == BOOST_OK && last.defer_combine) {
    // one slot per warp where the machine has the warps for it (two small threadblocks per SM)
    const uint32_t slots = last.n_row_tiles * (last.max_seg <= (x_rows == 32 ? 6u : 5u) ? (last.M_b + 1) / 2 : last.M_b);
    uint32_t cgrid = (slots + kConsumerWarps - 1) / kConsumerWarps;
    if (cgrid > 2u * (uint32_t)sms) cgrid = 2u * (uint32_t)sms;
    if (cgrid == 0) cgrid = 1;
    rc = boosth::launch_chained(combine_kernel, dim3(cgrid), dim3(kConsumerThreads), 0, stream, last);
    if (rc == BOOST_OK && extra_launches) ++*extra_launches;
  }
  return rc;
}


// Two threadblocks per SM where registers allow: a second ring hides the producer / consumer
// hand-over latency of the first (measured: +25 % bandwidth on B200).
template <int NT, int MB>
int launch_gemv(const ChainParams& chain, int sms, cudaStream_t stream, uint32_t* extra_launches) {
  static KernelState states[boosth::kMaxDevices];   // attributes and occupancy are per device
  const int slot = boosth::device_slot();
  if (slot < 0) return BOOST_ERR_CUDA;
  KernelState& state = states[slot];
  return launch_planned(gemv_tiered_kernel<NT, MB>, [](const ChainParams& c) -> const ChainParams& { return c; },
                        gemv_combine_kernel<x_rows_of(NT, MB)>, x_rows_of(NT, MB), state, kGemvThreads,
                        stage_bytes_of(NT, MB), kSmemBudget, (NT >= 8) ? 1 : 2, false, g_end_combine != 0, chain, sms, stream, extra_launches);
}

// Tensor map of a phase's activations x [M_b, K] (bf16, row-major) for the tcgen05 kernel: boxes of
// 64 columns x npad rows in the 128-byte swizzle; rows and columns beyond the tensor read as zero.
// The driver's encoder is looked up at run time (no link-time dependency on the driver library).
int encode_x_map(CUtensorMap* map, const void* x, uint32_t M_b, uint32_t K, uint32_t npad) {
  using Encode = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                              const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                              CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static Encode encode = [] {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult st;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &st) != cudaSuccess ||
        st != cudaDriverEntryPointSuccess)
      fn = nullptr;
    return reinterpret_cast<Encode>(fn);
  }();
  if (!encode) return BOOST_ERR_UNSUPPORTED;
  const cuuint64_t dims[2] = {K, M_b};
  const cuuint64_t strides[1] = {(cuuint64_t)K * 2};
  const cuuint32_t box[2] = {kBlockK, npad};
  const cuuint32_t elem[2] = {1, 1};
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, elem,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? BOOST_OK : BOOST_ERR_ALIGN;
}

template <uint32_t NPAD>
int launch_gemv_tc(const ChainParams& chain, int sms, cudaStream_t stream, uint32_t* extra_launches) {
  static KernelState states[boosth::kMaxDevices];
  const int slot = boosth::device_slot();
  if (slot < 0) return BOOST_ERR_CUDA;
  KernelState& state = states[slot];
  TcChainParams tp;
  for (uint32_t i = 0; i < chain.n_phases; ++i) {
    const GemvParams& q = chain.ph[i];
    const int rc = encode_x_map(&tp.x_map[i], q.x, q.M_b, q.K, NPAD);
    if (rc != BOOST_OK) return rc;
  }
  auto wrap = [&tp](const ChainParams& c) -> const TcChainParams& {
    tp.chain = c;
    return tp;
  };
  return launch_planned(gemv_tc_kernel<NPAD>, wrap, gemv_combine_kernel<NPAD>, NPAD, state, kTcThreads, tc_stage_bytes(NPAD), kTcSmemBudget, 1,
                        tc_weight_slots(NPAD) == 2,
                        g_end_combine != 0, chain, sms, stream, extra_launches);
}

}  // namespace

extern "C" int boost_weight_layout(uint32_t N, uint32_t K, boost_weight_layout_t* out) {
  if (!out || N == 0 || K == 0) return BOOST_ERR_INVALID;
  out->n_row_tiles = (N + kBlockRows - 1) / kBlockRows;
  out->k_blocks = (K + kBlockK - 1) / kBlockK;
  out->blocks_per_item = pick_run(out->n_row_tiles, out->k_blocks);
  out->splits = out->k_blocks / out->blocks_per_item;
  out->bytes = (uint64_t)out->n_row_tiles * out->k_blocks * kBlockBytes;
  out->n_pages = (out->bytes + kPageBytes - 1) / kPageBytes;
  return BOOST_OK;
}

extern "C" int boost_pack_weights_ex(const void* w_row_major, uint32_t N, uint32_t K,
                                     const void* const* w_page_ptr, size_t n_pages, int row_mode,
                                     const void* col_scale, void* stream) {
  boost_weight_layout_t lay;
  const int rc = boost_weight_layout(N, K, &lay);
  if (rc != BOOST_OK) return rc;
  if (!w_row_major || !w_page_ptr) return BOOST_ERR_INVALID;
  if (row_mode != 0 && row_mode != 1) return BOOST_ERR_INVALID;
  if (row_mode == 1 && N % 128 != 0) return BOOST_ERR_INVALID;
  if (K % 8 != 0 || ((uintptr_t)w_row_major % 16) != 0 || ((uintptr_t)col_scale % 16) != 0) return BOOST_ERR_ALIGN;
  if (n_pages < lay.n_pages) return BOOST_ERR_CAPACITY;
  const size_t n_chunks = lay.bytes / 16;
  size_t blocks = (n_chunks + 255) / 256;
  const size_t cap = (size_t)(boosth::sm_count() > 0 ? boosth::sm_count() : 148) * 16;
  if (blocks > cap) blocks = cap;
  pack_weights_kernel<<<(unsigned)blocks, 256, 0, (cudaStream_t)stream>>>(
      static_cast<const uint4*>(w_row_major), N, K, lay.k_blocks, n_chunks, w_page_ptr, row_mode,
      static_cast<const uint4*>(col_scale));
  return boosth::check_launch();
}

extern "C" int boost_pack_weights(const void* w_row_major, uint32_t N, uint32_t K,
                                  const void* const* w_page_ptr, size_t n_pages, void* stream) {
  return boost_pack_weights_ex(w_row_major, N, K, w_page_ptr, n_pages, 0, nullptr, stream);
}

static uint32_t gemv_x_rows(uint32_t M_b) {
  // rows of x staged per block: 1 or 2 on the CUDA-core path, else batch tiles of 8 for the
  // tensor cores (which outrun the CUDA cores from three rows up: the kernel is HBM-bound and
  // the tensor pipe is otherwise idle)
  if (M_b <= 1) return 1;
  if (M_b <= 2) return 2;
  if (M_b <= 16) return 16;
  if (M_b <= 32) return 32;
  if (M_b <= 64) return 64;
  if (M_b <= 128) return 128;
  return 256;
}

size_t boosth::gemv_header_bytes(uint32_t n_row_tiles) {
  return ((size_t)(kWsHeaderWords + n_row_tiles) * 4 + 255) / 256 * 256;
}

// Partial-sum slots per row tile: the splits of the queue items, or (even partition over G
// threadblocks, each at least floor(T / G) blocks long) the most threadblocks a tile can touch.
static uint32_t partial_slots(const boost_weight_layout_t& lay, uint32_t M_b) {
  int sms = boosth::sm_count();
  if (sms <= 0) sms = 148;
  const uint64_t T = (uint64_t)lay.n_row_tiles * lay.k_blocks;
  uint64_t G = (uint64_t)sms * 2;   // the most threadblocks any of the kernels keeps on an SM
  if (G > T) G = T;
  const uint32_t per = (uint32_t)(T / G);
  const uint32_t even = (lay.k_blocks + per - 1) / per + 1;
  return even > lay.splits ? even : lay.splits;
}

size_t boosth::gemv_partial_bytes(uint32_t N, uint32_t K, uint32_t M_b) {
  boost_weight_layout_t lay;
  if (boost_weight_layout(N, K, &lay) != BOOST_OK || M_b == 0 || M_b > 256) return 0;
  return (size_t)lay.n_row_tiles * partial_slots(lay, M_b) * gemv_x_rows(M_b) * kBlockRows * 4;
}

extern "C" size_t boost_gemv_workspace_bytes(uint32_t N, uint32_t K, uint32_t M_b) {
  boost_weight_layout_t lay;
  if (boost_weight_layout(N, K, &lay) != BOOST_OK || M_b == 0 || M_b > 256) return 0;
  return boosth::gemv_header_bytes(lay.n_row_tiles) + boosth::gemv_partial_bytes(N, K, M_b);
}

extern "C" int boost_gemv_tiered(const void* const* w_page_ptr, const uint32_t* w_order,
                                 size_t n_pages, size_t n_host_pages, uint32_t N, uint32_t K,
                                 const void* x, uint32_t M_b, void* y, int y_dtype,
                                 const void* residual, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  return boosth::gemv_tiered_launch(w_page_ptr, w_order, n_pages, n_host_pages, N, K, x, M_b, y, y_dtype,
                                    residual, workspace, workspace_bytes, nullptr, nullptr, 0, stream);
}

extern "C" int boost_gemv_tiered_fused(const void* const* w_page_ptr, const uint32_t* w_order,
                                       size_t n_pages, size_t n_host_pages, uint32_t N, uint32_t K,
                                       const void* x, uint32_t M_b, void* y, int y_dtype,
                                       const void* residual, const boost_gemv_epilogue_t* epilogue,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  return boosth::gemv_tiered_launch(w_page_ptr, w_order, n_pages, n_host_pages, N, K, x, M_b, y, y_dtype,
                                    residual, workspace, workspace_bytes, epilogue, nullptr, 0, stream);
}

namespace {

// Checks one product's arguments and fills its kernel parameters.  `header` = bytes of the
// counter area at the head of the workspace (the same for all products that share it).
int fill_params(GemvParams& p, const void* const* w_page_ptr, const uint32_t* w_order, size_t n_pages,
                size_t n_host_pages, uint32_t N, uint32_t K, const void* x, uint32_t M_b, void* y, int y_dtype,
                const void* residual, void* workspace, size_t workspace_bytes, const boost_gemv_epilogue_t* epi,
                uint32_t* queue_words, bool early, uint32_t header_row_tiles) {
  const int mode = epi ? epi->mode : BOOST_EPI_PLAIN;
  if (!w_page_ptr || !w_order || !x || !workspace) return BOOST_ERR_INVALID;
  if (!y && mode != BOOST_EPI_ROPE_APPEND) return BOOST_ERR_INVALID;
  if (mode != BOOST_EPI_PLAIN && mode != BOOST_EPI_SWIGLU && mode != BOOST_EPI_ROPE_APPEND) return BOOST_ERR_INVALID;
  if (mode == BOOST_EPI_SWIGLU && (N % 128 != 0 || y_dtype != 1 || residual)) return BOOST_ERR_INVALID;
  if (mode == BOOST_EPI_ROPE_APPEND) {
    if (!epi->q_out || !epi->k_page_ptr || !epi->v_page_ptr || !epi->block_table || !epi->ctx_lens ||
        epi->n_pool_blocks == 0 || epi->max_blocks == 0 || !epi->rope_table || residual)
      return BOOST_ERR_INVALID;
    if ((uint64_t)(epi->n_q_heads + 2 * epi->n_kv_heads) * 128 != N) return BOOST_ERR_INVALID;
  }
  if (epi && epi->ssq_in && (epi->ssq_in_tiles == 0 || epi->ssq_stride < M_b)) return BOOST_ERR_INVALID;
  if (epi && epi->ssq_out && (mode != BOOST_EPI_PLAIN || y_dtype != 1 || epi->ssq_stride < M_b)) return BOOST_ERR_INVALID;
  if (M_b == 0 || M_b > 256 || (y_dtype != 0 && y_dtype != 1)) return BOOST_ERR_INVALID;
  boost_weight_layout_t lay;
  const int rc = boost_weight_layout(N, K, &lay);
  if (rc != BOOST_OK) return rc;
  if (n_pages != lay.n_pages || n_host_pages > n_pages) return BOOST_ERR_INVALID;
  if (K % 8 != 0 || ((uintptr_t)x % 16) != 0 || ((uintptr_t)workspace % 256) != 0) return BOOST_ERR_ALIGN;
  const size_t header =
      boosth::gemv_header_bytes(header_row_tiles > lay.n_row_tiles ? header_row_tiles : lay.n_row_tiles);
  if (workspace_bytes < header + boosth::gemv_partial_bytes(N, K, M_b)) return BOOST_ERR_CAPACITY;

  p.w_page_ptr = w_page_ptr;
  p.w_order = w_order;
  p.n_pages = (uint32_t)n_pages;
  p.n_host_pages = (uint32_t)n_host_pages;
  p.N = N; p.K = K;
  p.n_row_tiles = lay.n_row_tiles;
  p.k_blocks = lay.k_blocks;
  p.run = lay.blocks_per_item;
  p.splits = lay.splits;
  p.even_part = (n_host_pages == 0 || g_tier_schedule == 0) ? 1u : 0u;
  p.total_blocks = lay.n_row_tiles * lay.k_blocks;
  p.max_seg = partial_slots(lay, M_b);
  p.tiles_per_unit = 1;
  p.items_per_page = kBlocksPerPage / lay.blocks_per_item;
  p.n_items = (uint32_t)((uint64_t)lay.n_row_tiles * lay.k_blocks / lay.blocks_per_item);
  p.x = static_cast<const __nv_bfloat16*>(x);
  p.M_b = M_b;
  p.y = y; p.y_dtype = y_dtype;
  p.residual = static_cast<const __nv_bfloat16*>(residual);
  p.ws = static_cast<uint32_t*>(workspace);
  p.queue = queue_words ? queue_words : p.ws;
  p.early = (queue_words && early) ? 1u : 0u;
  p.epi = (uint32_t)mode;
  p.ssq_in = epi ? epi->ssq_in : nullptr;
  p.ssq_in_tiles = epi ? epi->ssq_in_tiles : 0;
  p.ssq_stride = epi ? epi->ssq_stride : 0;
  p.x_cols = K;
  p.rms_eps = epi ? epi->rms_eps : 0.f;
  p.ssq_out = epi ? epi->ssq_out : nullptr;
  p.q_out = epi ? static_cast<__nv_bfloat16*>(epi->q_out) : nullptr;
  p.k_page_ptr = epi ? epi->k_page_ptr : nullptr;
  p.v_page_ptr = epi ? epi->v_page_ptr : nullptr;
  p.k_page_ptr2 = epi ? epi->k_page_ptr2 : nullptr;
  p.v_page_ptr2 = epi ? epi->v_page_ptr2 : nullptr;
  p.block_table = epi ? epi->block_table : nullptr;
  p.ctx_lens = epi ? epi->ctx_lens : nullptr;
  p.n_pool_blocks = epi ? epi->n_pool_blocks : 0;
  p.max_blocks = epi ? epi->max_blocks : 0;
  p.Hq = epi ? epi->n_q_heads : 0;
  p.Hkv = epi ? epi->n_kv_heads : 0;
  p.rope_table = epi ? epi->rope_table : nullptr;
  p.partials = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + header);
  p.n_host_ctas = 0; p.n_stages = 0;
  p.end_combine = 0;
  return BOOST_OK;
}

// Batches from this size on take the tcgen05 kernel, smaller ones (from 3 rows) mma.sync.
// Measured on B200 on Llama-3-8B-shaped matrices: up to 32 rows the mma.sync kernel (two
// threadblocks per SM) streams faster; at 64 rows the tcgen05 kernel is 1.5 x, at 128 rows
// 1.8 x faster, because the mma.sync kernel re-reads the activation tile from shared memory in
// every warp.
uint32_t g_tc_min_batch = 33;

int launch_routed(const ChainParams& c, uint32_t M_b, void* stream, uint32_t* extra_launches = nullptr) {
  const int sms = boosth::sm_count();
  if (sms <= 0) return BOOST_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  const bool tc = M_b >= g_tc_min_batch;
  switch (gemv_x_rows(M_b)) {
    case 1: return launch_gemv<0, 1>(c, sms, st, extra_launches);
    case 2: return launch_gemv<0, 2>(c, sms, st, extra_launches);
    case 16: return tc ? launch_gemv_tc<16>(c, sms, st, extra_launches) : launch_gemv<2, 0>(c, sms, st, extra_launches);
    case 32: return tc ? launch_gemv_tc<32>(c, sms, st, extra_launches) : launch_gemv<4, 0>(c, sms, st, extra_launches);
    case 64: return tc ? launch_gemv_tc<64>(c, sms, st, extra_launches) : launch_gemv<8, 0>(c, sms, st, extra_launches);
    case 128: return tc ? launch_gemv_tc<128>(c, sms, st, extra_launches) : launch_gemv<16, 0>(c, sms, st, extra_launches);
    default: return launch_gemv_tc<256>(c, sms, st, extra_launches);   // 129 - 256 rows: the tcgen05 kernel only
  }
}

}  // namespace

int boosth::gemv_tiered_launch(const void* const* w_page_ptr, const uint32_t* w_order, size_t n_pages,
                               size_t n_host_pages, uint32_t N, uint32_t K, const void* x, uint32_t M_b,
                               void* y, int y_dtype, const void* residual, void* workspace,
                               size_t workspace_bytes, const boost_gemv_epilogue_t* epi,
                               uint32_t* queue_words, uint32_t header_row_tiles, void* stream, uint32_t* extra_launches) {
  ChainParams c;
  c.n_phases = 1;
  c.bar = static_cast<uint32_t*>(workspace) + kWsBar;   // a lone product's two counters live in the header
  const int rc = fill_params(c.ph[0], w_page_ptr, w_order, n_pages, n_host_pages, N, K, x, M_b, y, y_dtype, residual,
                             workspace, workspace_bytes, epi, queue_words, queue_words != nullptr, header_row_tiles);
  if (rc != BOOST_OK) return rc;
  return launch_routed(c, M_b, stream, extra_launches);
}

int boosth::gemv_chain_launch(const boost_gemv_call_t* calls, uint32_t n_calls, uint32_t M_b, void* workspace,
                              size_t workspace_bytes, uint32_t* sync_words, bool early, uint32_t header_row_tiles,
                              void* stream, uint32_t* extra_launches) {
  if (!calls || n_calls == 0 || n_calls > kMaxPhases || !sync_words) return BOOST_ERR_INVALID;
  uint32_t tiles = header_row_tiles;
  for (uint32_t i = 0; i < n_calls; ++i) {
    const uint32_t t = (calls[i].w.N + kBlockRows - 1) / kBlockRows;
    tiles = t > tiles ? t : tiles;
  }
  ChainParams c;
  c.n_phases = n_calls;
  c.bar = sync_words + 16 * n_calls;
  for (uint32_t i = 0; i < n_calls; ++i) {
    const boost_gemv_call_t& g = calls[i];
    const int rc = fill_params(c.ph[i], g.w.page_ptr, g.w.order, (size_t)g.w.n_pages, (size_t)g.w.n_host_pages, g.w.N,
                               g.w.K, g.x, M_b, g.y, g.y_dtype, g.residual, workspace, workspace_bytes,
                               g.has_epilogue ? &g.epilogue : nullptr, sync_words + 16 * i, early, tiles);
    if (rc != BOOST_OK) return rc;
  }
  return launch_routed(c, M_b, stream, extra_launches);
}

extern "C" size_t boost_gemv_chain_workspace_bytes(const boost_gemv_call_t* calls, uint32_t n_calls, uint32_t M_b) {
  if (!calls || n_calls == 0 || n_calls > kMaxPhases) return 0;
  uint32_t tiles = 0;
  size_t partial = 0;
  for (uint32_t i = 0; i < n_calls; ++i) {
    const uint32_t t = (calls[i].w.N + kBlockRows - 1) / kBlockRows;
    tiles = t > tiles ? t : tiles;
    const size_t b = boosth::gemv_partial_bytes(calls[i].w.N, calls[i].w.K, M_b);
    if (b == 0) return 0;
    partial = b > partial ? b : partial;
  }
  return boosth::gemv_header_bytes(tiles) + (partial + 255) / 256 * 256 + 64 * (size_t)(n_calls + 1);
}

extern "C" int boost_gemv_tiered_chain(const boost_gemv_call_t* calls, uint32_t n_calls, uint32_t M_b,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  const size_t need = boost_gemv_chain_workspace_bytes(calls, n_calls, M_b);
  if (need == 0) return BOOST_ERR_INVALID;
  if (!workspace) return BOOST_ERR_INVALID;
  if (((uintptr_t)workspace % 256) != 0) return BOOST_ERR_ALIGN;
  if (workspace_bytes < need) return BOOST_ERR_CAPACITY;
  // the tail of the workspace holds the queue words of every product and the phase counters
  const size_t sync_bytes = 64 * (size_t)(n_calls + 1);
  const size_t usable = (workspace_bytes - sync_bytes) & ~(size_t)255;
  uint32_t* sync_words = reinterpret_cast<uint32_t*>(static_cast<uint8_t*>(workspace) + usable);
  // The sync words sit at a fixed place of the caller's workspace, and the header lets the next
  // call reuse the workspace on the same stream: that call's threadblocks may become resident
  // while this one drains, so none of them may touch the words before this launch has completed
  // (early = false: the weight warps also wait for the preceding kernel).
  return boosth::gemv_chain_launch(calls, n_calls, M_b, workspace, usable, sync_words, false, 0, stream);
}

// Routing threshold between the two tensor-core kernels (measurement and tests).
extern "C" int boost_gemv_set_tc_min_batch(uint32_t m_b) {
  g_tc_min_batch = m_b;
  return BOOST_OK;
}

// Where the partial sums of a product are combined (measurement and tests): 1 = at the end of
// the phase by all threadblocks when a row tile has many (the default), 0 = always tile by tile.
extern "C" int boost_gemv_set_end_combine(uint32_t on) {
  g_end_combine = on ? 1u : 0u;
  return BOOST_OK;
}

// How a weight with host pages is scheduled (measurement and tests): 0 = its host pages are read
// in place by the threadblocks whose share of the even partition holds them (the default), 1 = two
// queues of work items, host pages first.
extern "C" int boost_gemv_set_tier_schedule(uint32_t two_queues) {
  g_tier_schedule = two_queues ? 1u : 0u;
  return BOOST_OK;
}
