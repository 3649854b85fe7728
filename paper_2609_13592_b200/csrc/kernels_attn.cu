// Tiered paged decode attention (split-KV) over the KV cache of a boost_kv_pool, and the
// copies that move a logical [Hkv][N][16][D] cache into and out of its pages.
//
// Persistent grid.  A work item is a KV-head chunk run: sequence b, KV head g, a run of
// consecutive blocks of the sequence (Sec. 3.3: threadblocks work on KV head chunks); items
// of the highest-numbered heads - the ones linear placement puts on the host tier - are
// handed out first.  The four warps of a threadblock take a quarter of the run each and
// stream it on their own, through their own two-stage rings in shared memory: per block two
// 4 KiB bulk copies through the TMA unit (K chunk, V chunk) when the page is in HBM, a fan of
// 16-byte cp.async loads when it is host memory.  Twelve such warps per SM keep about
// 150 KiB in flight with no producer warp and no barrier while they stream.  The products
// are bf16 tensor-core MMAs with the 16 tokens of a block as the 16-row dimension and the
// query heads of the group as the 8-wide dimension (S^T = K q^T, O^T += V^T P^T: a group of
// four heads wastes half a tile instead of three quarters); P goes in as three bf16 terms,
// transposed in registers with movmatrix; the online softmax is fp32.  The four quarters are
// merged in shared memory; only a sequence longer than one item leaves partial results in
// global memory, and the last of its items to finish combines them in run order.
// The run length is not fixed by the host: every threadblock derives it, and a dense list of
// the items, from the context lengths when it starts (before the wait on the preceding
// kernel), so the decomposition follows the batch's real mix of lengths.
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdlib.h>

#include "device_common.cuh"
#include "host_common.h"

namespace {

using namespace boostk;

constexpr uint32_t kD = 128;
constexpr uint32_t kTok = BOOST_KV_BLOCK_TOKENS;         // 16
constexpr uint32_t kChunkBytes = kTok * kD * 2;          // 4 KiB
constexpr uint32_t kChunksPerPage = kPageBytes / kChunkBytes;
constexpr uint32_t kMaxItemBlocks = 64;                  // KV blocks per warp and work item: at most (one lane resolves two blocks)
constexpr uint32_t kMinItemBlocks = 4;
constexpr uint32_t kStageBytes = 2 * kChunkBytes;        // K chunk + V chunk
constexpr uint32_t kAttnWarps = 4;                       // warps per threadblock
constexpr uint32_t kAttnThreads = kAttnWarps * 32;
constexpr uint32_t kWarpStages = 2;                      // ring depth of one warp
constexpr uint32_t kMaxGroup = 16;
constexpr uint32_t kParkStride = kD + 4;                 // floats per parked head: 128 outputs, m, l, padding
constexpr uint32_t kMaxListedSeqs = 1024;                // batches up to this size get a dense item list
constexpr uint32_t kMaxSmemPages = 256;                   // page tables up to this size are staged in shared memory
constexpr uint32_t kWsPlan = 12;                         // workspace header word: the plan of attn_plan_kernel (0: none yet)
constexpr uint32_t kTailPieces = 4;                      // the runs of the last KV head are cut in this many items


struct AttnParams {
  const __nv_bfloat16* q;
  const void* const* k_page_ptr;
  const void* const* v_page_ptr;
  uint32_t first_host_page;   // pages >= this are host pages (linear placement)
  uint32_t n_pool_blocks;
  const int32_t* block_table;
  uint32_t max_blocks;
  const int32_t* ctx_lens;
  uint32_t B, Hq, Hkv, group;
  uint32_t cta_slots;         // threadblocks the device holds at once (the balance target)
  uint32_t smem_pages;        // > 0: the K and V page tables (this many entries each) are staged in shared memory
  float scale_log2e;
  uint32_t* ws;        // header (status, item counter, done counter) + one counter per (b, g)
  float* part_ml;      // [B][Hq][max_splits][2], max_splits from the run length chosen on the device
  float* part_o;       // [B][Hq][max_splits][128]
  __nv_bfloat16* out;
};

// Cached tokens of sequence b, kept inside what its row of the block table can describe (a
// length outside it is recorded in the status word where the sequence's items are processed).
__device__ __forceinline__ uint32_t seq_len(const AttnParams& p, uint32_t b) {
  return min((uint32_t)max(p.ctx_lens[b], 0), p.max_blocks * kTok);
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}

// Run length for sequences about equally long, each cut into s runs: the slots take the items in
// rounds; a full round streams at the HBM rate, the last one at the rate its items can draw (a
// threadblock alone gets 1 / (55 % of the slots) of it), and every round costs a hand-over (table
// look-up, query load, merge: about 5 us = 4000 block times).  In units of the time HBM takes for
// one KV block: cost = run x (full rounds x slots + max(55 % of slots, items of the last round))
// + 4000 x rounds.  Candidates: 1 .. 4 runs per sequence, and one run per slot over 4 / 7 of the
// slots (runs of 1.75 times the blocks a slot gets on average: what long sequences in small
// batches need).  Returns the blocks per warp of the cheapest.
__device__ __forceinline__ uint32_t item_blocks_by_cost(uint32_t total_blocks, uint32_t longest, uint32_t B, uint32_t Hkv,
                                                     uint32_t slots) {
  const float sat = 0.55f * (float)slots, inv_slots = 1.f / (float)slots;
  const uint32_t mean = (total_blocks + B - 1) / B;
  const uint32_t per_slot = (total_blocks * Hkv * 7u + slots * 4u - 1u) / (slots * 4u);
  float best = 3.0e38f;
  uint32_t item_blocks = kMaxItemBlocks;
#pragma unroll 1
  for (uint32_t s = 0; s <= 4; ++s) {
    const uint32_t run = s ? (longest + s - 1) / s : per_slot;
    const uint32_t ib = min(kMaxItemBlocks, max(kMinItemBlocks, (run + kAttnWarps - 1) / kAttnWarps));
    const uint32_t n_spl = mean ? (mean + kAttnWarps * ib - 1) / (kAttnWarps * ib) : 1u;
    const float len = mean ? (float)((mean + n_spl - 1) / n_spl) : 0.f;
    const float items = (float)(B * Hkv * n_spl);
    const float full = floorf(items * inv_slots + 1e-4f), tail = items - full * (float)slots;
    const float cost = len * (full * (float)slots + (tail > 0.5f ? fmaxf(sat, tail) : 0.f)) + 4000.f * (full + (tail > 0.5f ? 1.f : 0.f));
    if (cost < best) { best = cost; item_blocks = ib; }
  }
  return item_blocks;
}

// The plan of a launch - blocks per warp and work item in the low half, bit 31: a mix of lengths -
// from the sum and the maximum of the sequences' block counts.  An item costs a table look-up,
// a query load and, when a sequence needs several items, a partial result in global memory,
// so long runs are better; but the kernel ends with its longest item, and about 55 % of the
// threadblocks the device holds saturate HBM (measured on B200: about a thousand warps with
// 16 KiB in flight each).  With u KV blocks per threadblock slot on average: a mix of lengths
// (longest above 1.25 times the mean) -> runs of at most u, a few items per slot to even out
// through the queue; sequences about equally long -> runs of at most 1.75 u where one run per
// sequence fills one round of the slots well (between 55 % of them and all), else what the cost
// model picks.
constexpr uint32_t kPlanMixed = 0x80000000u;
__device__ __forceinline__ uint32_t attn_plan_word(uint64_t total_blocks, uint32_t longest, uint32_t B, uint32_t Hkv, uint32_t slots) {
  const bool mixed = (uint64_t)longest * B * 4 > total_blocks * 5;
  const uint64_t quarters = mixed ? 4 : 7;   // run cap in quarters of u
  const uint64_t run_cap = (total_blocks * Hkv * quarters + (uint64_t)slots * 4 - 1) / ((uint64_t)slots * 4);
  uint32_t item_blocks = (uint32_t)min((uint64_t)kMaxItemBlocks, max((uint64_t)kMinItemBlocks, (run_cap + kAttnWarps - 1) / kAttnWarps));
  const uint32_t whole = B * Hkv;
  if (!mixed && !(longest <= kAttnWarps * kMaxItemBlocks && whole <= slots && whole * 20u >= slots * 11u))
    item_blocks = item_blocks_by_cost((uint32_t)total_blocks, longest, B, Hkv, slots);
  return item_blocks | (mixed ? kPlanMixed : 0u);
}

// Sum and maximum of the sequences' block counts over a threadblock of kAttnThreads threads
// (scratch: two arrays of kAttnWarps words).  Every thread gets the result.
__device__ __forceinline__ void attn_block_counts(const AttnParams& p, uint32_t* s_sum, uint32_t* s_max, uint64_t& total_blocks,
                                                  uint32_t& longest) {
  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint32_t my_blocks = 0, my_max = 0;
  for (uint32_t b = tid; b < p.B; b += kAttnThreads) {
    const uint32_t n = (seq_len(p, b) + kTok - 1) / kTok;
    my_blocks += n;
    my_max = max(my_max, n);
  }
#pragma unroll
  for (int sh = 16; sh >= 1; sh >>= 1) {
    my_blocks += __shfl_xor_sync(0xFFFFFFFFu, my_blocks, sh);
    my_max = max(my_max, __shfl_xor_sync(0xFFFFFFFFu, my_max, sh));
  }
  if (lane == 0) { s_sum[warp] = my_blocks; s_max[warp] = my_max; }
  __syncthreads();
  total_blocks = 0;
  longest = 0;
#pragma unroll
  for (uint32_t w = 0; w < kAttnWarps; ++w) { total_blocks += s_sum[w]; longest = max(longest, s_max[w]); }
}

// The plan as a kernel of its own (one threadblock): a decode step runs it once, ahead of its
// attention launches, which then read the word instead of each deriving it (kOwnPlan = false).
// It does not release its dependents early: whatever is launched behind it starts after it.
__global__ void __launch_bounds__(kAttnThreads) attn_plan_kernel(const AttnParams p) {
  __shared__ uint32_t s_sum[kAttnWarps], s_max[kAttnWarps];
  pdl_wait();
  uint64_t total_blocks;
  uint32_t longest;
  attn_block_counts(p, s_sum, s_max, total_blocks, longest);
  if (threadIdx.x == 0) p.ws[kWsPlan] = attn_plan_word(total_blocks, longest, p.B, p.Hkv, p.cta_slots);
}

// NH = number of 8-head tiles of a KV group (1: up to 8 query heads per KV head, 2: up to 16);
// kOwnPlan: the kernel derives its plan itself (every threadblock sums the context lengths), or
// reads the word attn_plan_kernel left in the workspace.
template <int NH, bool kOwnPlan>
__global__ void __launch_bounds__(kAttnThreads, (NH == 1 ? 3 : 2)) paged_attn_kernel(const AttnParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
  __shared__ uint64_t full_bar[kAttnWarps][kWarpStages];

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  uint8_t* ring = smem + (size_t)warp * kWarpStages * kStageBytes;   // this warp's stages
  // Small page tables are copied into shared memory once: a block's address is then one
  // dependent global load (its table entry) away instead of two.
  unsigned long long* s_pages = reinterpret_cast<unsigned long long*>(smem + (size_t)kAttnWarps * kWarpStages * kStageBytes);
  for (uint32_t i = tid; i < p.smem_pages; i += kAttnThreads) {
    s_pages[i] = reinterpret_cast<unsigned long long>(p.k_page_ptr[i]);
    s_pages[p.smem_pages + i] = reinterpret_cast<unsigned long long>(p.v_page_ptr[i]);
  }
  uint32_t* status = p.ws + kWsStatus;
  pdl_launch_dependents();
  if (lane == 0) {
    for (uint32_t s = 0; s < kWarpStages; ++s) mbar_init(&full_bar[warp][s], 33);   // 32 cp.async arrivals + arrive.expect_tx
    fence_barrier_init();
  }
  __syncwarp();
  // The kernels just before this one produce q and the newest K / V row of every sequence
  // (in its last block).  Context lengths, block tables and all older blocks are not theirs:
  // the first item's look-ups, and its first blocks unless one of them is the sequence's
  // last, are requested before the wait on those kernels.
  bool waited = false;

  // Fragment coordinates: rows gq, gq+8 (tokens for S^T, d for O^T), columns c0, c0+1 (heads).
  const uint32_t gq = lane >> 2, c0 = (lane & 3) * 2;
  uint32_t phase_mask = 0;                       // bit s = phase to wait for on stage s
  // A work item belongs to the threadblock: (sequence b, KV head g, a run of blocks); its four
  // warps take a quarter of the run each and stream it on their own; their results meet in
  // shared memory.  First item by position, later ones from the counter.
  __shared__ uint32_t s_next, s_old;
  __shared__ uint32_t s_warp_sum[kAttnWarps], s_warp_max[kAttnWarps];
  __shared__ uint32_t s_first_item[kMaxListedSeqs + 1];   // first item of every sequence within a head

  // ---- run length.  Every threadblock works with the same decomposition of the sequences into
  // items (see attn_plan_word).
  uint32_t plan;
  if constexpr (kOwnPlan) {
    uint64_t total_blocks;
    uint32_t longest;
    attn_block_counts(p, s_warp_sum, s_warp_max, total_blocks, longest);
    plan = attn_plan_word(total_blocks, longest, p.B, p.Hkv, p.cta_slots);
  } else {
    plan = __ldcg(p.ws + kWsPlan);
  }
  const bool mixed = (plan & kPlanMixed) != 0;
  const uint32_t item_blocks = min(kMaxItemBlocks, max(kMinItemBlocks, plan & 0xFFFFu));
  const uint32_t cta_max = kAttnWarps * item_blocks;
  const uint32_t max_splits = (p.max_blocks + cta_max - 1) / cta_max;
  // ---- item list.  Up to kMaxListedSeqs sequences: items are numbered densely, sequence by
  // sequence (s_first_item = running count of runs), so no threadblock draws an empty item.
  // Larger batches: every sequence has max_splits numbers and the unused ones are skipped.
  const bool listed = p.B <= kMaxListedSeqs;
  if (!listed && p.smem_pages) __syncthreads();   // (the listed path below has barriers of its own)
  uint32_t per_head = p.B * max_splits;
  if (listed) {
    uint32_t carry = 0;
    for (uint32_t b0 = 0; b0 < p.B; b0 += kAttnThreads) {
      const uint32_t b = b0 + tid;
      const uint32_t n_blk = b < p.B ? (seq_len(p, b) + kTok - 1) / kTok : 0;
      const uint32_t mine = b < p.B ? (n_blk ? (n_blk + cta_max - 1) / cta_max : 1u) : 0u;
      uint32_t incl = mine;
#pragma unroll
      for (int sh = 1; sh < 32; sh <<= 1) {
        const uint32_t up = __shfl_up_sync(0xFFFFFFFFu, incl, sh);
        if ((int)lane >= sh) incl += up;
      }
      __syncthreads();   // s_warp_sum is free again
      if (lane == 31) s_warp_sum[warp] = incl;
      __syncthreads();
      uint32_t before = carry, round_total = 0;
#pragma unroll
      for (uint32_t w = 0; w < kAttnWarps; ++w) {
        if (w < warp) before += s_warp_sum[w];
        round_total += s_warp_sum[w];
      }
      if (b < p.B) s_first_item[b] = before + incl - mine;
      carry += round_total;
    }
    if (tid == 0) s_first_item[p.B] = carry;
    __syncthreads();
    per_head = carry;
  }
  // The queue ends with KV head 0.  With a mix of lengths its runs are cut in kTailPieces
  // items each, so the threadblocks run out of work within a short item of one another.
  const uint32_t tail_k = mixed ? kTailPieces : 1u;
  const uint32_t n_long = (p.Hkv - 1) * per_head;
  const uint32_t n_items = n_long + per_head * tail_k;
  const uint32_t slots_per = max_splits * tail_k;      // partial results of one (sequence, query head)
  uint32_t id = blockIdx.x;

  while (id < n_items) {
    const bool tail = id >= n_long;
    const uint32_t g = tail ? 0u : p.Hkv - 1 - id / per_head;     // host-resident heads first
    const uint32_t k_pieces = tail ? tail_k : 1u;
    const uint32_t in_head = tail ? (id - n_long) / tail_k : id % per_head;
    const uint32_t piece = tail ? (id - n_long) % tail_k : 0u;
    uint32_t b, split;
    if (listed) {
      // the sequence whose range of items holds in_head: last b with s_first_item[b] <= in_head
      uint32_t lo = 0, hi = p.B;
      while (hi - lo > 1) {
        const uint32_t mid = (lo + hi) >> 1;
        if (s_first_item[mid] <= in_head) lo = mid; else hi = mid;
      }
      b = lo;
      split = in_head - s_first_item[lo];
    } else {
      b = in_head / max_splits;
      split = in_head % max_splits;
    }
    if (tid == 0 && (p.ctx_lens[b] < 0 || (uint32_t)p.ctx_lens[b] > p.max_blocks * kTok)) atomicOr(status, kErrBadIndex);
    const uint32_t ctx = seq_len(p, b);
    const uint32_t n_blk = (ctx + kTok - 1) / kTok;
    const uint32_t n_splits = n_blk ? (n_blk + cta_max - 1) / cta_max : 1;
    if (split < n_splits) {
      // the sequence's blocks in n_splits runs of equal length (the last may be shorter by a
      // few), each run in four quarters
      const uint32_t run_len = n_blk ? (n_blk + n_splits - 1) / n_splits : 0;
      const uint32_t rblk0 = split * run_len;
      const uint32_t rnb = min(run_len, n_blk - min(n_blk, rblk0));
      const uint32_t piece_len = (rnb + k_pieces - 1) / k_pieces;
      const uint32_t cblk0 = rblk0 + piece * piece_len;
      const uint32_t cnb = min(piece_len, rnb - min(rnb, piece * piece_len));
      const uint32_t sub_len = (cnb + kAttnWarps - 1) / kAttnWarps;
      const uint32_t blk0 = cblk0 + warp * sub_len;
      const uint32_t nb = min(sub_len, cnb - min(cnb, warp * sub_len));
      // every lane resolves up to two blocks of the warp's run (lane and lane + 32): table
      // entry, page, addresses (K and V sit at the same offset of their tensors)
      const uint8_t* ksrc[2] = {nullptr, nullptr};
      size_t v_minus_k[2] = {0, 0};
      uint32_t host_bits = 0;
#pragma unroll
      for (uint32_t h = 0; h < 2; ++h) {
        if (lane + 32 * h < nb) {
          int32_t blk = p.block_table[(size_t)b * p.max_blocks + blk0 + lane + 32 * h];
          if (blk < 0 || (uint32_t)blk >= p.n_pool_blocks) {   // bad table entry: record, read block 0
            atomicOr(status, kErrBadIndex);
            blk = 0;
          }
          const uint32_t lin = g * p.n_pool_blocks + (uint32_t)blk;
          const uint32_t page = lin / kChunksPerPage;
          const size_t in_page = (size_t)(lin % kChunksPerPage) * kChunkBytes;
          const uint8_t* kpage = p.smem_pages ? reinterpret_cast<const uint8_t*>(s_pages[page]) : static_cast<const uint8_t*>(p.k_page_ptr[page]);
          const uint8_t* vpage = p.smem_pages ? reinterpret_cast<const uint8_t*>(s_pages[p.smem_pages + page])
                                              : static_cast<const uint8_t*>(p.v_page_ptr[page]);
          ksrc[h] = kpage + in_page;
          v_minus_k[h] = (size_t)(vpage + in_page - ksrc[h]);
          host_bits |= (page >= p.first_host_page ? 1u : 0u) << h;
        }
      }
      // request block i of the run into stage i % kWarpStages
      auto request = [&](uint32_t i) {
        const uint32_t st = i % kWarpStages;
        const uint32_t h = i >> 5, src_lane = i & 31u;
        const unsigned long long k_all = (unsigned long long)(h ? ksrc[1] : ksrc[0]);
        const unsigned long long d_all = (unsigned long long)(h ? v_minus_k[1] : v_minus_k[0]);
        const uint8_t* ks = reinterpret_cast<const uint8_t*>(__shfl_sync(0xFFFFFFFFu, k_all, src_lane));
        const uint8_t* vs = ks + __shfl_sync(0xFFFFFFFFu, d_all, src_lane);
        const bool from_host = ((__shfl_sync(0xFFFFFFFFu, host_bits, src_lane) >> h) & 1u) != 0;
        uint8_t* kdst = ring + (size_t)st * kStageBytes;
        uint8_t* vdst = kdst + kChunkBytes;
        if (lane == 0) {
          mbar_arrive_expect_tx(&full_bar[warp][st], from_host ? 0u : kStageBytes);
          if (!from_host) {
            bulk_copy_g2s(kdst, ks, kChunkBytes, &full_bar[warp][st]);
            bulk_copy_g2s(vdst, vs, kChunkBytes, &full_bar[warp][st]);
          }
        }
        if (from_host) {
          // host page: a fan of 16-byte loads through the load/store path (Sec. 3.2)
#pragma unroll
          for (uint32_t c = lane; c < kChunkBytes / 16; c += 32) {
            cp_async_16(kdst + c * 16, ks + c * 16, 16u);
            cp_async_16(vdst + c * 16, vs + c * 16, 16u);
          }
        }
        cp_async_arrive_noinc(&full_bar[warp][st]);
      };
      // schedule log (opt-in): one record per warp and item, the warp's quarter of the run
      uint32_t rec = kNoRecord;
      if (nb) {
        const uint32_t host_blocks = __popc(__ballot_sync(0xFFFFFFFFu, (host_bits & 1u) != 0)) +
                                     __popc(__ballot_sync(0xFFFFFFFFu, (host_bits & 2u) != 0));
        if (lane == 0)
          rec = sched_log_begin(sched_log_of(p.ws), BOOST_SCHED_KIND_ATTN, blockIdx.x | (warp << 24), nb * kStageBytes,
                                host_blocks * kStageBytes);
      }
      const uint32_t n_first = min(nb, kWarpStages);
      const bool early = !waited && blk0 + n_first + 1 <= n_blk;   // none of them is the last block
      if (early)
        for (uint32_t i = 0; i < n_first; ++i) request(i);
      if (!waited) {
        pdl_wait();
        waited = true;
      }
      if (!early)
        for (uint32_t i = 0; i < n_first; ++i) request(i);

      // q^T as the B operand (k = d, n = head), straight from global while the blocks fly
      uint32_t qb[NH][8][2];
      float o[NH][8][4];          // O^T: 8 tiles of 16 d, columns = heads
      float m_run[NH][2], l_run[NH][2];
#pragma unroll
      for (int nh = 0; nh < NH; ++nh) {
        const uint32_t head = nh * 8 + gq;
        const uint8_t* qs = reinterpret_cast<const uint8_t*>(p.q + ((size_t)b * p.Hq + g * p.group + head) * kD);
#pragma unroll
        for (uint32_t ks = 0; ks < 8; ++ks) {
          qb[nh][ks][0] = head < p.group ? *reinterpret_cast<const uint32_t*>(qs + (ks * 16 + c0) * 2) : 0u;
          qb[nh][ks][1] = head < p.group ? *reinterpret_cast<const uint32_t*>(qs + (ks * 16 + c0) * 2 + 16) : 0u;
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[nh][i][0] = o[nh][i][1] = o[nh][i][2] = o[nh][i][3] = 0.f; }
        m_run[nh][0] = m_run[nh][1] = -CUDART_INF_F;
        l_run[nh][0] = l_run[nh][1] = 0.f;
      }

      for (uint32_t i = 0; i < nb; ++i) {
        const uint32_t st = i % kWarpStages;
        mbar_wait(&full_bar[warp][st], (phase_mask >> st) & 1u, status);
        phase_mask ^= 1u << st;
        const uint32_t kbase = smem_u32(ring + (size_t)st * kStageBytes);
        const uint32_t vbase = kbase + kChunkBytes;
        const uint32_t tok = (lane & 7) + ((lane >> 4) << 3);     // ldmatrix row of this lane (V^T)
        const uint32_t sub = (lane >> 3) & 1;                     // which 16-byte chunk of a pair
        // S^T = K q^T: rows = 16 tokens, columns = heads; two accumulation chains
        float s[NH][4], s2[NH][4];
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
        // mask the tail of the last block, scale into the log2 domain; online softmax per head
        const uint32_t t_lo = (blk0 + i) * kTok + gq, t_hi = t_lo + 8;
        uint32_t pa[NH][3][2];
#pragma unroll
        for (int nh = 0; nh < NH; ++nh) {
          float pf[4];
#pragma unroll
          for (int r = 0; r < 4; ++r) {
            const uint32_t t = (r & 2) ? t_hi : t_lo;
            const float v = s[nh][r] + s2[nh][r];
            s[nh][r] = (t < ctx) ? v * p.scale_log2e : -CUDART_INF_F;
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
            for (int j = 0; j < 8; ++j) { o[nh][j][h] *= corr; o[nh][j][2 + h] *= corr; }
          }
          // P^T as the B operand (k = token, n = head).  A single bf16 rounding of P would put
          // an error of 2^-9 * sqrt(sum p^2 v^2) on every output, far above 1 % of the outputs
          // that are close to zero; P is split into three bf16 terms (24 bits) multiplied term
          // by term.  The accumulator layout (token rows) becomes the operand layout (token as
          // k) by an 8x8 transpose across the warp.
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
        // Every lane is done with this stage before it is refilled, and its loads have been
        // performed: they went through the generic proxy, the refill is a bulk copy through the
        // async proxy, which nothing else keeps behind loads still in flight.
        __threadfence_block();
        __syncwarp();
        if (i + kWarpStages < nb) request(i + kWarpStages);
      }
      if (lane == 0 && rec != kNoRecord) sched_log_end(sched_log_of(p.ws), rec);

      // ---- end of the run: the four warps' (m, l, O) meet in shared memory.  Each warp parks
      // its result in its own (now idle) ring space: per head 128 outputs, then m and l.
      float* park = reinterpret_cast<float*>(ring);
#pragma unroll
      for (int nh = 0; nh < NH; ++nh)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const uint32_t head = nh * 8 + c0 + h;
          if (head >= p.group) continue;
          float* dst = park + head * kParkStride;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            dst[j * 16 + gq] = o[nh][j][h];
            dst[j * 16 + gq + 8] = o[nh][j][2 + h];
          }
          if (gq == 0) { dst[kD] = m_run[nh][h]; dst[kD + 1] = l_run[nh][h]; }
        }
      __syncthreads();
      // warp w merges heads w, w + 4, ...: lane = four consecutive outputs
      const uint32_t n_parts = n_splits * k_pieces;   // items of this (sequence, KV head)
      const bool single = (n_parts == 1);
      for (uint32_t r = warp; r < p.group; r += kAttnWarps) {
        const uint32_t hq = g * p.group + r;
        float mw[kAttnWarps], lw[kAttnWarps];
        float m_all = -CUDART_INF_F;
#pragma unroll
        for (uint32_t w = 0; w < kAttnWarps; ++w) {
          const float* src = reinterpret_cast<const float*>(smem + (size_t)w * kWarpStages * kStageBytes) + r * kParkStride;
          mw[w] = src[kD]; lw[w] = src[kD + 1];
          m_all = fmaxf(m_all, mw[w]);
        }
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        float l_all = 0.f;
#pragma unroll
        for (uint32_t w = 0; w < kAttnWarps; ++w) {
          if (mw[w] == -CUDART_INF_F) continue;   // a quarter without blocks
          const float f = exp2f(mw[w] - m_all);
          const float4 v = *(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(smem + (size_t)w * kWarpStages * kStageBytes) + r * kParkStride) + lane);
          acc.x += f * v.x; acc.y += f * v.y; acc.z += f * v.z; acc.w += f * v.w;
          l_all += f * lw[w];
        }
        if (single) {
          const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
          const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
          const __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
          uint2 ov;
          ov.x = *reinterpret_cast<const uint32_t*>(&lo);
          ov.y = *reinterpret_cast<const uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(p.out + ((size_t)b * p.Hq + hq) * kD + lane * 4) = ov;
        } else {
          const size_t slot = ((size_t)b * p.Hq + hq) * slots_per + split * k_pieces + piece;
          __stcg(reinterpret_cast<float4*>(p.part_o + slot * kD) + lane, acc);
          if (lane == 0) { __stcg(p.part_ml + slot * 2, m_all); __stcg(p.part_ml + slot * 2 + 1, l_all); }
        }
      }
      if (!single) {
        // the last run of (b, g) to arrive combines all runs, in run order
        uint32_t* cnt = p.ws + kWsHeaderWords + b * p.Hkv + g;
        __syncthreads();
        if (tid == 0) {
          __threadfence();   // cumulative: publishes the partial results of the whole threadblock
          s_old = atomicAdd(cnt, 1u);
        }
        __syncthreads();
        if (s_old == n_parts - 1) {
          __threadfence();
          for (uint32_t r = warp; r < p.group; r += kAttnWarps) {
            const uint32_t hq = g * p.group + r;
            const size_t slot0 = ((size_t)b * p.Hq + hq) * slots_per;
            // lane i looks after the (m, l) pair of runs i, i + 32, ...; the outputs are summed
            // in run order, eight loads in flight at a time
            float m_all = -CUDART_INF_F;
            for (uint32_t sp = lane; sp < n_parts; sp += 32) m_all = fmaxf(m_all, __ldcg(p.part_ml + (slot0 + sp) * 2));
#pragma unroll
            for (int sh = 16; sh >= 1; sh >>= 1) m_all = fmaxf(m_all, __shfl_xor_sync(0xFFFFFFFFu, m_all, sh));
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            float l_all = 0.f;
            for (uint32_t base = 0; base < n_parts; base += 32) {
              float f_mine = 0.f, lf = 0.f;
              if (base + lane < n_parts) {
                const float2 ml = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (slot0 + base + lane) * 2));
                f_mine = (ml.x == -CUDART_INF_F) ? 0.f : exp2f(ml.x - m_all);
                lf = f_mine * ml.y;
              }
#pragma unroll
              for (int sh = 16; sh >= 1; sh >>= 1) lf += __shfl_xor_sync(0xFFFFFFFFu, lf, sh);
              l_all += lf;
              const uint32_t n_here = min(32u, n_parts - base);
              for (uint32_t j0 = 0; j0 < n_here; j0 += 8) {
                float4 v[8];
#pragma unroll
                for (uint32_t u = 0; u < 8; ++u)
                  if (j0 + u < n_here) v[u] = __ldcg(reinterpret_cast<const float4*>(p.part_o + (slot0 + base + j0 + u) * kD) + lane);
#pragma unroll
                for (uint32_t u = 0; u < 8; ++u) {
                  const float f = __shfl_sync(0xFFFFFFFFu, f_mine, (j0 + u) & 31u);
                  if (j0 + u < n_here) { acc.x += f * v[u].x; acc.y += f * v[u].y; acc.z += f * v[u].z; acc.w += f * v[u].w; }
                }
              }
            }
            const float inv = l_all > 0.f ? 1.f / l_all : 0.f;
            const __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
            const __nv_bfloat162 hi = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
            uint2 ov;
            ov.x = *reinterpret_cast<const uint32_t*>(&lo);
            ov.y = *reinterpret_cast<const uint32_t*>(&hi);
            *reinterpret_cast<uint2*>(p.out + ((size_t)b * p.Hq + hq) * kD + lane * 4) = ov;
          }
          if (tid == 0) *cnt = 0;
        }
      }
      // the ring is written by bulk copies again: every thread orders its reads and writes of the
      // parked values before them (proxy fence), then all meet
      fence_proxy_async_smem();
      __syncthreads();
    } else if (!waited) {
      pdl_wait();   // keep every thread's first pass through the dependency wait
      waited = true;
    }
    if (tid == 0) s_next = gridDim.x + atomicAdd(p.ws + kWsHbmNext, 1u);
    __syncthreads();
    id = s_next;
    __syncthreads();
  }
  // the last threadblock out resets the counters for the next launch
  if (tid == 0) {
    __threadfence();
    const uint32_t d = atomicAdd(p.ws + kWsDone, 1u);
    if (d == gridDim.x - 1) { p.ws[kWsHbmNext] = 0; p.ws[kWsDone] = 0; __threadfence(); }
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

// Partial results a (sequence, query head) can have: the shortest runs, each cut in pieces.
size_t partial_slots(uint32_t max_blocks) {
  const size_t runs = max_blocks ? (max_blocks + kAttnWarps * kMinItemBlocks - 1) / (kAttnWarps * kMinItemBlocks) : 1;
  return runs * kTailPieces;
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
  const size_t max_splits = partial_slots(max_blocks);
  // counters are per (b, KV head); Hq bounds the number of KV heads
  return attn_header_bytes(B, Hq) + (size_t)B * Hq * max_splits * (2 + kD) * 4;
}

// plan: who decides the run length of the items.  kAttnPlanOwn: the attention kernel itself, every
// threadblock from the context lengths (a call on its own); kAttnPlanOnly: no attention, only the
// one-threadblock kernel that leaves the plan in the workspace (a decode step runs it first of
// all, several launches ahead of the first attention kernel, which reads the word before its
// dependency wait); kAttnPlanReuse: attention with the plan such a call left there for the same
// batch and context lengths.
int boosth::paged_attn_launch(const void* q, const void* const* k_page_ptr, const void* const* v_page_ptr,
                              const uint8_t* kv_tier, size_t n_kv_pages, uint32_t n_pool_blocks,
                              const int32_t* block_table, uint32_t max_blocks, const int32_t* ctx_lens, uint32_t B,
                              uint32_t Hq, uint32_t Hkv, uint32_t D, float scale, void* workspace, size_t workspace_bytes,
                              void* out, void* stream, int plan) {
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
  const int sms = boosth::sm_count();
  if (sms <= 0) return BOOST_ERR_CUDA;
  const uint32_t ctas_per_sm = p.group <= 8 ? 3 : 2;
  p.cta_slots = (uint32_t)sms * ctas_per_sm;
  // every sequence is at least one item per KV head, at most one per kMinItemBlocks-long quarter run
  const uint64_t max_items = (uint64_t)Hkv * B * partial_slots(max_blocks);
  if (max_items > 0x7FFFFFFFull) return BOOST_ERR_INVALID;
  p.scale_log2e = scale * 1.4426950408889634f;
  p.ws = static_cast<uint32_t*>(workspace);
  uint8_t* base = static_cast<uint8_t*>(workspace) + attn_header_bytes(B, Hq);
  p.part_ml = reinterpret_cast<float*>(base);
  // room for the shortest runs; the kernel indexes with the max_splits of the run length it picks
  p.part_o = p.part_ml + (size_t)B * Hq * partial_slots(max_blocks) * 2;
  p.out = static_cast<__nv_bfloat16*>(out);
  // page tables of up to 256 entries ride in shared memory (three threadblocks per SM still fit)
  p.smem_pages = n_kv_pages <= kMaxSmemPages ? (uint32_t)n_kv_pages : 0u;
  const size_t smem_max = (size_t)kAttnWarps * kWarpStages * kStageBytes + 128 + (size_t)kMaxSmemPages * 16;
  const size_t smem = (size_t)kAttnWarps * kWarpStages * kStageBytes + 128 + (size_t)p.smem_pages * 16;
  static bool configured_on[boosth::kMaxDevices] = {false};   // function attributes are per device
  const int slot = boosth::device_slot();
  if (slot < 0) return BOOST_ERR_CUDA;
  bool& configured = configured_on[slot];
  if (!configured) {
    int rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<1, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<2, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<1, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
    if (rc == BOOST_OK)
      rc = boosth::check(cudaFuncSetAttribute(paged_attn_kernel<2, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max));
    if (rc != BOOST_OK) return rc;
    configured = true;
  }
  uint32_t grid = p.cta_slots;
  if (grid > max_items) grid = (uint32_t)max_items;
  if (plan == boosth::kAttnPlanOnly)
    return boosth::launch_chained(attn_plan_kernel, dim3(1), dim3(kAttnThreads), 0, (cudaStream_t)stream, p);
  const bool own = plan == boosth::kAttnPlanOwn;
  if (p.group <= 8)
    return own ? boosth::launch_chained(paged_attn_kernel<1, true>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p)
               : boosth::launch_chained(paged_attn_kernel<1, false>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p);
  return own ? boosth::launch_chained(paged_attn_kernel<2, true>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p)
             : boosth::launch_chained(paged_attn_kernel<2, false>, dim3(grid), dim3(kAttnThreads), smem, (cudaStream_t)stream, p);
}

extern "C" int boost_paged_attn_decode_tiered(const void* q, const void* const* k_page_ptr,
                                              const void* const* v_page_ptr, const uint8_t* kv_tier,
                                              size_t n_kv_pages, uint32_t n_pool_blocks,
                                              const int32_t* block_table, uint32_t max_blocks,
                                              const int32_t* ctx_lens, uint32_t B, uint32_t Hq,
                                              uint32_t Hkv, uint32_t D, float scale, void* workspace,
                                              size_t workspace_bytes, void* out, void* stream) {
  return boosth::paged_attn_launch(q, k_page_ptr, v_page_ptr, kv_tier, n_kv_pages, n_pool_blocks, block_table, max_blocks,
                                   ctx_lens, B, Hq, Hkv, D, scale, workspace, workspace_bytes, out, stream, boosth::kAttnPlanOwn);
}
