/*
 * boost.h - C ABI of the tiered decode hot path (BOOST, arxiv 2609.13592) for NVIDIA B200.
 *
 * Every buffer is cut into 2 MiB pages that live in one of two tiers: HBM, or
 * pinned host memory that the GPU reads with ordinary loads over the CPU-GPU
 * link.  Pages are placed so that every wave of threadblocks reads both tiers
 * at once and in proportion to their bandwidths; each threadblock stays on one
 * tier for a whole work item.
 *
 * Conventions
 *   - plain C; every call returns BOOST_OK (0) or a negative BOOST_ERR_* code;
 *     no exception crosses the boundary;
 *   - the library never allocates or frees device or pinned memory: callers
 *     pass pointers and sizes.  "host" / "device" beside an argument says in
 *     which address space the pointer must be valid for the library's own
 *     reads and writes (host = dereferenced on the CPU inside the call;
 *     device = dereferenced by kernels);
 *   - kernel launches are asynchronous on the given stream (a cudaStream_t
 *     passed as void*; NULL is the default stream);
 *   - `workspace` arguments are scratch in device memory owned by the caller.
 *     A workspace must be zero-filled once before its first use; kernels leave
 *     the counters in it at zero when they finish, so the same workspace can be
 *     reused by later calls on the same stream.  Calls that may overlap on the
 *     GPU need separate workspaces;
 *   - the first 16 32-bit words of every workspace are its header.  Word 0 is the status
 *     word: kernels OR error bits into it and never clear it (bit 0: a bounded wait ran out
 *     and the kernel wound down early - its outputs are not valid; bit 1: a table index out
 *     of range was skipped).  A non-zero status word means: zero-fill the whole workspace
 *     before it is used again (counters may have been left mid-count).  Words 4 - 7 are the
 *     caller's, read by the kernels and 0 in normal use: word 4 replaces the limit of every
 *     bounded wait (GPU clock cycles; the default is about a second), word 5 - honoured only
 *     with a non-zero word 4 - makes that many threadblocks withhold their arrival at the end
 *     of a product of a chain, and their announcement that a row tile's partial sum is in
 *     memory (a test hook: it makes the others' waits run out), words 6 - 7
 *     hold the device address of a schedule log (see boost_schedule_stats).  The other
 *     header words belong to the kernels;
 *   - every wait inside a kernel is bounded: none can hang the GPU;
 *   - what the launch paths set up once (function attributes, occupancy) is kept per device,
 *     indexed by the device that is current at the call, so one process may drive several
 *     GPUs; handles (boost_kv_pool_t) are not thread safe;
 *   - limits: head dimension 128; at most 16 query heads per KV head; the KV range of a
 *     tensor must be placed linearly (host pages at its tail, as the pool places it);
 *     weight products and the whole decode step take 1 - 256 batch rows (sequences).
 */
#ifndef BOOST_H_
#define BOOST_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BOOST_PAGE_BYTES 2097152u /* 2 MiB pages (Sec. 1, Sec. 2.6) */
#define BOOST_KV_BLOCK_TOKENS 16u /* tokens per KV block (Sec. 4.3) */

enum {
  BOOST_OK = 0,
  BOOST_ERR_INVALID = -1,  /* bad argument, unknown request, double free */
  BOOST_ERR_NOMEM = -2,    /* KV pool exhausted: the scheduler must decide (Sec. 4.3) */
  BOOST_ERR_ALIGN = -3,    /* pointer or size not aligned as documented */
  BOOST_ERR_CUDA = -4,     /* a CUDA runtime call failed; see boost_last_cuda_error() */
  BOOST_ERR_CAPACITY = -5, /* an output or workspace buffer is too small */
  BOOST_ERR_UNSUPPORTED = -6
};

enum { BOOST_TIER_HBM = 0, BOOST_TIER_HOST = 1 };

enum {
  BOOST_POLICY_MODULO = 0,     /* K pages HBM, then one page host, repeating (Sec. 3.1) */
  BOOST_POLICY_CONTIGUOUS = 1, /* head of the range HBM, tail host (Sec. 4.2, Sec. 5.7) */
  BOOST_POLICY_RANDOM = 2      /* every page host with the target probability (Sec. 2.6) */
};

/* boost_place_pages flag: a wave of `wave_size` pages is shorter than one period, so
 * not every wave can contain a host page (the precondition of Sec. 3.1 fails). */
#define BOOST_FLAG_WAVE_SHORTER_THAN_PERIOD 1u

/* CUDA error code (cudaError_t as int) of the most recent BOOST_ERR_CUDA on this thread. */
int boost_last_cuda_error(void);

/* ------------------------------------------------------------------ placement */

/* Period M of the modulo rule for a host share of all pages `host_ratio` (= 1/M):
 * the smallest M with 1/M <= host_ratio * (1 + 2^-40), so the host share never
 * exceeds the request (rounding rule of Sec. 4.4).  host_ratio = 0 gives M = 0
 * (no host pages).  host_ratio must be 0 or lie in [2^-30, 1/2]. */
int boost_modulus_from_ratio(double host_ratio, uint32_t* modulus_out /*host*/);

/* M = ceil(hbm_bw / link_bw) + 1: K = ceil(1/alpha) pages of HBM, then one host page
 * (Sec. 3.1, Sec. 4.4).  Any unit, both > 0. */
int boost_modulus_from_bandwidths(double hbm_bw, double link_bw, uint32_t* modulus_out /*host*/);

/* Page-to-tier table of one tensor under modulo placement (Sec. 3.1).
 *   buffer      only checked for 2 MiB alignment (may be NULL to skip the check);
 *   bytes       size of the tensor; P = ceil(bytes / 2 MiB) pages;
 *   host_ratio  share of all pages that go to the host tier (see above);
 *   wave_size   pages one wave of threadblocks covers; does not change the table,
 *               only sets BOOST_FLAG_WAVE_SHORTER_THAN_PERIOD (0 = unknown);
 *   tier_out    host array of tier_cap bytes; entry i = BOOST_TIER_* of page i;
 *   n_pages_out receives P.
 * Page i is a host page iff (i mod M) == M-1.  The function keeps no state, so the
 * pattern restarts for every tensor (Sec. 3.1).
 * Errors: INVALID (null outputs, bad ratio), ALIGN, CAPACITY (tier_cap < P). */
int boost_place_pages(const void* buffer, size_t bytes, double host_ratio, uint32_t wave_size,
                      uint8_t* tier_out /*host*/, size_t tier_cap, size_t* n_pages_out /*host*/);

/* As boost_place_pages with the comparison policies and superpages.
 *   policy           BOOST_POLICY_*;
 *   seed             used by RANDOM only: page i is host iff
 *                    mix(seed + (i+1)*0x9E3779B97F4A7C15) < floor(2^64 / M), mix being the
 *                    SplitMix64 output function;
 *   superpage_pages  S >= 1: groups of S consecutive pages share a tier and the modulo
 *                    rule runs over groups (Sec. 3.2, Sec. 4.4); MODULO only;
 *   flags_out        may be NULL.
 * CONTIGUOUS puts floor(P/M) pages, the last ones, on the host. */
int boost_place_pages_ex(const void* buffer, size_t bytes, double host_ratio, uint32_t wave_size,
                         int policy, uint64_t seed, uint32_t superpage_pages,
                         uint8_t* tier_out /*host*/, size_t tier_cap, size_t* n_pages_out /*host*/,
                         uint32_t* flags_out /*host*/);

/* Host share of every wave when tiles are handed out in address order (Sec. 2.2, Sec. 2.6). */
typedef struct {
  uint64_t n_waves;
  uint64_t n_host_pages;
  uint64_t n_zero_waves; /* waves that touch no host tile */
  uint64_t n_over_waves; /* waves whose host share exceeds host_ratio */
  double mean, var, min, max; /* of the per-wave host share; var is the population variance */
} boost_wave_stats_t;

/* tile_bytes must divide 2 MiB; wave w holds tiles [w*G, (w+1)*G), G = ctas_per_wave; the
 * last wave may be short (Sec. 4.4). */
int boost_wave_stats(const uint8_t* tier /*host*/, size_t n_pages, size_t tile_bytes,
                     uint32_t ctas_per_wave, double host_ratio, boost_wave_stats_t* out /*host*/);

/* ---- The schedule a kernel realised (Sec. 2.6, Sec. 3.1: the host share of every wave is what
 * placement is about; Sec. 3.2: with threadblocks specialised by tier it is the hand-out order,
 * not the address order, that decides it).  The tier-aware kernels hand out host-tier work first
 * from queues of their own, so what each wave of work, and each stretch of time, really read from
 * which tier is a property of the run.  Opt-in: put the device address of a log buffer into words
 * 6 and 7 (one 64-bit value) of a kernel's zero-filled workspace header before the launch; every
 * work item then appends one record.  Log buffer: boost_schedule_log_bytes(capacity) bytes of
 * device memory, zero-filled, with the capacity stored in its second 64-bit word (the first
 * counts the records claimed; more than the capacity means records were dropped).  The decode
 * step's products share one workspace, its attention kernels another. */
#define BOOST_SCHED_KIND_STREAM 1u /* stream reduce: a 128 KiB tile */
#define BOOST_SCHED_KIND_GEMV 2u   /* weight product: a queue item, or a threadblock's segment of a row tile */
#define BOOST_SCHED_KIND_ATTN 3u   /* attention: one warp's quarter of a run of KV blocks */
typedef struct {
  uint32_t kind_phase;  /* BOOST_SCHED_KIND_* | (phase of a chain << 8) */
  uint32_t cta_warp;    /* threadblock | (warp << 24) */
  uint32_t bytes;       /* bytes the item streams */
  uint32_t host_bytes;  /* of which from host-tier pages */
  uint64_t t_request;   /* GPU global timer (ns) when the item's first byte was requested */
  uint64_t t_consumed;  /* ... when its last byte had been consumed; 0 = never finished */
} boost_schedule_record_t;
size_t boost_schedule_log_bytes(size_t capacity);
/* Statistics of a log copied to host memory (log = the whole buffer, header included).
 *   kind             only records of this BOOST_SCHED_KIND_* (0 = all);
 *   items_per_wave   records are ordered by t_request (ties: cta_warp, then kind_phase) and cut
 *                    into waves of this many consecutive starts; a wave's host share is its
 *                    host_bytes / bytes -> wave_out (n_over_waves counts shares above host_ratio);
 *   window_ns        the time from the first request to the last consumption is cut into windows
 *                    of this length; a record's bytes are spread evenly over [t_request,
 *                    t_consumed] (at least 1 ns) and a window's host share is host / all bytes
 *                    that fall into it; windows without traffic are left out -> window_out;
 *   n_records_out    records that passed the filter (unfinished ones are skipped).
 * n_host_pages of the outputs holds the number of records with host_bytes > 0.
 * Errors: INVALID (null pointers, zero items_per_wave or window_ns, a log shorter than its
 * header says). */
int boost_schedule_stats(const void* log /*host*/, size_t log_bytes, uint32_t kind, uint32_t items_per_wave,
                         uint64_t window_ns, double host_ratio, boost_wave_stats_t* wave_out /*host*/,
                         boost_wave_stats_t* window_out /*host*/, uint64_t* n_records_out /*host*/);

/* Visit order for tier-specialised kernels: host pages first (ascending), then HBM pages
 * (ascending).  Each threadblock works on one tier at a time (Sec. 3.2); handing out the
 * slow tier's pages first keeps both tiers busy for the whole kernel.
 * order_out: host array of n_pages entries; n_host_out receives the number of host pages. */
int boost_tier_order(const uint8_t* tier /*host*/, size_t n_pages, uint32_t* order_out /*host*/,
                     size_t* n_host_out /*host*/);

/* ------------------------------------------------------------ materialisation */

/* One virtual address range over both tiers.  The paper's kernels are unmodified library
 * kernels: they read an ordinary address range whose 2 MiB pages have been placed on one tier
 * or the other underneath them (Sec. 2.3: the GPU and the host memory share one address space;
 * Sec. 4.4: the allocator binds each page of a tensor to its tier).  boost_va_buffer_create
 * builds that on this machine with the CUDA virtual-memory API: it reserves n_pages * 2 MiB of
 * device-visible address space and maps page i to a fresh HBM page (tier[i] = BOOST_TIER_HBM)
 * or to a pinned page of host memory on NUMA node host_numa_node (BOOST_TIER_HOST).  The range
 * is then one flat buffer for anything on the current device - cudaMemcpy, kernels of other
 * libraries, this library's kernels through boost_va_buffer_page_table (page i at base +
 * i * 2 MiB) - while every page lives where the tier table says.
 *   tier   host array of n_pages entries (from boost_place_pages*); ownership stays with the caller;
 *   out    receives the handle; release with boost_va_buffer_destroy (unmaps and frees all).
 * Errors: INVALID, CAPACITY (out of HBM), UNSUPPORTED (the driver or the platform has no
 * virtual-memory management for the tier, e.g. no host-NUMA allocations). Not thread safe. */
typedef struct boost_va_buffer boost_va_buffer_t;
int boost_va_buffer_create(const uint8_t* tier /*host*/, size_t n_pages, int host_numa_node,
                           boost_va_buffer_t** out /*host*/);
void* boost_va_buffer_base(const boost_va_buffer_t* buffer);   /* device address of page 0 */
int boost_va_buffer_page_table(const boost_va_buffer_t* buffer, void** page_ptr_out /*host*/, size_t cap);
int boost_va_buffer_destroy(boost_va_buffer_t* buffer);


/* Device-visible address of a pinned (page-locked) host allocation; INVALID when the
 * pointer is not pinned host memory that the current device can address. */
int boost_host_device_pointer(void* pinned_host, void** device_ptr_out /*host*/);

/* A peer GPU's HBM as the second tier ("Bandwidth Ratio Ablation with NVLinks": the same
 * placement with the second tier behind NVLink instead of the CPU link, where the bandwidth
 * ratio is around 10 % instead of 1 %).  Pages of the second tier then live in a slab on
 * peer_device; their addresses go into the page table through boost_page_table's host_slab
 * argument and every kernel of this library reads them as it reads pinned host memory: each
 * threadblock with its own copies into its own shared memory.  The modulus for such a tier is
 * boost_modulus_from_bandwidths(hbm, link) with the measured peer-read bandwidth.
 *   boost_peer_tier_open   lets kernels of the current device read peer_device's memory
 *                          (idempotent);
 *   boost_peer_tier_alloc  allocates `bytes` in peer_device's HBM; slab_out receives the
 *                          address (valid on both devices once opened; the caller aligns it to
 *                          2 MiB as for any slab); the caller's current device is unchanged;
 *   boost_peer_tier_free   releases such a slab (NULL is accepted).
 * Errors: INVALID (peer_device out of range or the current device itself, NULL / zero
 * arguments), UNSUPPORTED (no peer access between the two devices), CAPACITY (out of memory
 * on the peer), CUDA.  One process per GPU: the peer's slab is owned by the process that
 * allocated it. */
int boost_peer_tier_open(int peer_device);
int boost_peer_tier_alloc(int peer_device, size_t bytes, void** slab_out /*host*/);
int boost_peer_tier_free(int peer_device, void* slab /*device*/);

/* Page base addresses for a placed tensor (the analogue of binding each 2 MiB region to a
 * memory node, Sec. 4.4).  HBM pages take consecutive 2 MiB slots of hbm_slab, host pages
 * consecutive slots of host_slab, both in page order.
 *   hbm_slab / host_slab  device-visible base addresses, 2 MiB aligned; a slab may be NULL
 *                         when its tier holds no page; *_slab_bytes are their capacities;
 *   page_ptr_out          host array of n_pages pointers. */
int boost_page_table(const uint8_t* tier /*host*/, size_t n_pages, void* hbm_slab,
                     size_t hbm_slab_bytes, void* host_slab, size_t host_slab_bytes,
                     void** page_ptr_out /*host*/);

/* Copy a contiguous device buffer of `bytes` into its pages (page i receives bytes
 * [i*2MiB, (i+1)*2MiB)), or back.  src/dst device; page_ptr device array. bytes % 16 == 0. */
int boost_scatter_pages(const void* src /*device*/, size_t bytes,
                        const void* const* page_ptr /*device*/, size_t n_pages, void* stream);
int boost_gather_pages(void* dst /*device*/, size_t bytes, const void* const* page_ptr /*device*/,
                       size_t n_pages, void* stream);

/* ------------------------------------------------------------------- KV pool */

typedef struct boost_kv_pool boost_kv_pool_t;

typedef struct {
  uint32_t n_blocks, n_kv_heads, host_modulus, chunk_bytes;
  uint32_t n_pages;          /* pages of one K (or V) tensor of one layer */
  uint32_t n_host_pages;     /* the last n_host_pages pages are host pages (Sec. 4.2) */
  uint32_t host_heads_lo;    /* host heads of a "lo" block; a "hi" block has one more */
  uint32_t first_hi_block;   /* blocks >= this index are "hi" blocks */
  uint32_t free_lo, free_hi; /* free blocks of each kind */
  uint32_t live_blocks, n_requests;
  uint64_t live_host_chunks, live_chunks; /* (head, block) chunks of live blocks */
} boost_kv_pool_info_t;

/* Wave-aware pool of KV blocks (Sec. 4.3, Sec. 4.5).
 * Geometry: per layer and per K/V the cache is [n_kv_heads][n_blocks][16 tokens][D] with
 * heads outermost; chunk (h, b) is chunk_bytes long at byte offset (h*n_blocks + b) *
 * chunk_bytes.  n_blocks*chunk_bytes must be a multiple of 2 MiB so heads never share a
 * page.  The tensor is placed linearly: its last floor(P/host_modulus) pages are host
 * pages (host_modulus 0 = none; 1 is rejected).  A block therefore has host_heads_lo or
 * host_heads_lo+1 of its heads on the host ("lo" and "hi" blocks).
 * Policy: one FIFO free list per kind, ascending at start.  A request's first allocation
 * fixes its kind: "hi" iff free_hi / (free_lo+free_hi) exceeds the target share of hi
 * blocks (n_kv_heads - host_heads_lo*host_modulus) / host_modulus, else "lo".  Blocks
 * come from the list of the request's kind; when that list is empty the block comes from
 * the other list and the request keeps that kind from then on. */
int boost_kv_pool_create(uint32_t n_blocks, uint32_t n_kv_heads, uint32_t host_modulus,
                         uint32_t chunk_bytes, boost_kv_pool_t** pool_out /*host*/);

/* Give `n` (>= 1) blocks to `request_id`, creating the request on first use.
 * block_ids_out: host array of n entries.  NOMEM when fewer than n blocks are free in
 * total; the pool is then unchanged. */
int boost_kv_pool_alloc(boost_kv_pool_t* pool, uint64_t request_id, uint32_t n,
                        int32_t* block_ids_out /*host*/);

/* Return all blocks of a request to the tail of their lists, in the order they were
 * handed out.  INVALID for an unknown (or already freed) request. */
int boost_kv_pool_free(boost_kv_pool_t* pool, uint64_t request_id);

int boost_kv_pool_query(const boost_kv_pool_t* pool, boost_kv_pool_info_t* info_out /*host*/);

/* Kind (0 = lo, 1 = hi) a live request currently draws from. */
int boost_kv_pool_request_kind(const boost_kv_pool_t* pool, uint64_t request_id,
                               int* kind_out /*host*/);

/* Tier of every page of one K (or V) tensor of one layer. */
int boost_kv_pool_page_tiers(const boost_kv_pool_t* pool, uint8_t* tier_out /*host*/,
                             size_t tier_cap, size_t* n_pages_out /*host*/);

int boost_kv_pool_destroy(boost_kv_pool_t* pool);

/* ------------------------------------------------------------------- kernels */

/* Streaming read of a paged bf16 buffer: per_page_sum[i] = sum of the 1 Mi bf16 values of
 * page i, accumulated in fp32 (the "add" micro-benchmark of Sec. 2.6 with a sum as its
 * trivial compute).  Threadblocks take 128 KiB tiles of pages in `order`; a fixed share of
 * the blocks starts on the host pages (Sec. 3.2) and all tiles of a page are combined in
 * a fixed order, so results do not depend on scheduling.
 *   page_ptr      device array of n_pages page addresses;
 *   order         device array from boost_tier_order (host pages first);
 *   per_page_sum  device array of n_pages floats;
 *   workspace     device, >= boost_stream_reduce_workspace_bytes(n_pages). */
size_t boost_stream_reduce_workspace_bytes(size_t n_pages);
int boost_stream_reduce_tiered(const void* const* page_ptr /*device*/,
                               const uint32_t* order /*device*/, size_t n_pages,
                               size_t n_host_pages, float* per_page_sum /*device*/,
                               void* workspace /*device*/, size_t workspace_bytes, void* stream);

/* boost_stream_reduce_tiered for callers that cannot allocate.  (The paper has no
 * counterpart: this entry point exists for integration, not for the method.)
 * Who needs it: an engine that gave all device memory to its own pools at start-up, so a
 * later cudaMalloc fails; a plug-in that must stay inside a host framework's allocator; any
 * caller on a path where allocating CUDA calls are not allowed.  The scratch that the
 * kernel needs lives in a fixed array inside the library (about 272 KiB, held by every GPU
 * that loads the library until the process exits), so the call allocates nothing - no
 * cudaMalloc, cudaFree or allocating library routine - and takes no workspace argument.
 *   - n_pages may be at most boost_stream_reduce_static_max_pages() (4096 pages, 8 GiB);
 *     larger buffers return BOOST_ERR_CAPACITY and must use boost_stream_reduce_tiered.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call outside any stream capture.
 *   - All calls on a device share the one array: the call clears the counters it needs on
 *     `stream` before the kernel, but two calls that overlap on the GPU (different streams,
 *     or a graph replayed concurrently) race on it and give wrong sums.
 * Inputs, outputs and results are those of boost_stream_reduce_tiered. */
size_t boost_stream_reduce_static_max_pages(void);
int boost_stream_reduce_tiered_static(const void* const* page_ptr /*device*/,
                                      const uint32_t* order /*device*/, size_t n_pages,
                                      size_t n_host_pages, float* per_page_sum /*device*/,
                                      void* stream);

/* Weight tensors are stored in pages as a stream of 16 KiB blocks.  Block (t, kb) holds
 * rows [128 t, 128 t + 128) and columns [64 kb, 64 kb + 64) of the row-major [N, K] bf16
 * matrix W (zero padded), at byte offset (t * ceil(K/64) + kb) * 16 KiB of the tensor; row
 * r of the block occupies 128 bytes at r*128 and its 16-byte chunk c sits at position
 * c ^ (r & 7) (the 128-byte shared-memory swizzle), so one bulk copy brings a block into
 * shared memory ready for the tensor cores.  A threadblock streams a run of blocks of one
 * row tile from one page, i.e. a contiguous region of one tier (Sec. 3.1, Sec. 3.2). */
typedef struct {
  uint32_t n_row_tiles;     /* ceil(N / 128) */
  uint32_t k_blocks;        /* ceil(K / 64) */
  uint32_t blocks_per_item; /* run length L: divides 128 and k_blocks */
  uint32_t splits;          /* k_blocks / L partial sums per row tile */
  uint64_t bytes;           /* n_row_tiles * k_blocks * 16 KiB */
  uint64_t n_pages;
} boost_weight_layout_t;

int boost_weight_layout(uint32_t N, uint32_t K, boost_weight_layout_t* out /*host*/);

/* Write the packed form of row-major W [N, K] (device, bf16) into its pages. */
int boost_pack_weights(const void* w_row_major /*device*/, uint32_t N, uint32_t K,
                       const void* const* w_page_ptr /*device*/, size_t n_pages, void* stream);

/* boost_pack_weights with two load-time transformations that let the small operators of a
 * decode step disappear into the products (the paper does not discuss those operators):
 *   row_mode 1  rows 0..63 of packed row tile t are rows [64 t, 64 t + 64) of the first half of
 *               W and rows 64..127 the same rows of the second half, so that gate row j and up
 *               row j of a [gate; up] matrix meet in one threadblock (N % 128 == 0);
 *   col_scale   bf16 [K] or NULL: W[n, k] is multiplied by col_scale[k] and rounded to bf16 -
 *               an RMSNorm weight folded into the matrix it feeds. */
int boost_pack_weights_ex(const void* w_row_major /*device*/, uint32_t N, uint32_t K,
                          const void* const* w_page_ptr /*device*/, size_t n_pages, int row_mode,
                          const void* col_scale /*device*/, void* stream);

/* y[m, n] = sum_k x[m, k] * W[n, k] (+ residual[m, n]), fp32 accumulation: the
 * weight-streaming product that dominates decode (Sec. 2.1, Sec. 3.1; the two-pointer
 * handwritten matmul of Sec. 3.1 is the closest thing the paper describes).
 *   w_page_ptr, w_order  device arrays for the packed weight (n_pages entries; order from
 *                        boost_tier_order, host pages first);
 *   x          device, bf16 row-major [M_b, K];  1 <= M_b <= 256;
 *   y          device, row-major [M_b, N]; y_dtype 0 = fp32, 1 = bf16;
 *   residual   device bf16 [M_b, N] added before the final rounding, or NULL;
 *   workspace  device, >= boost_gemv_workspace_bytes(N, K, M_b).
 * M_b <= 2 runs on CUDA cores with warp-shuffle reductions; larger batches use the tensor
 * cores (mma.sync up to 32 rows, tcgen05 with accumulators in tensor memory above; see
 * boost_gemv_set_tc_min_batch).  The blocks of a weight are cut evenly over the threadblocks;
 * host pages are read in place, by the same bulk copies, by the threadblocks whose share holds
 * them (boost_gemv_set_tier_schedule selects the two-queue schedule that hands host pages out
 * first instead).  Split-K
 * partial sums meet in L2 and are combined in a fixed order - tile by tile in the threadblock
 * that delivers a tile's last partial sum, or, for a product cut so finely that a tile has four
 * or more, all tiles at the end of the product spread over the warps of the grid (see
 * boost_gemv_set_end_combine; after the last product of a launch that combine runs as a small
 * kernel of its own right behind it on the stream) - so the result is deterministic (to the bit
 * for a given placement, device and batch; across placements the order of the fp32 sums, hence
 * the last bits, may differ).
 * Errors: INVALID, ALIGN (x not 16-byte, workspace not 256-byte aligned, K % 8 != 0), CAPACITY,
 * UNSUPPORTED (the device cannot hold one threadblock of the kernel), CUDA.  Status bits in
 * word 0 of the workspace: see the conventions at the top (bit 1 here: a block index out of
 * range in the RoPE / KV-append epilogue). */
size_t boost_gemv_workspace_bytes(uint32_t N, uint32_t K, uint32_t M_b);
int boost_gemv_tiered(const void* const* w_page_ptr /*device*/, const uint32_t* w_order /*device*/,
                      size_t n_pages, size_t n_host_pages, uint32_t N, uint32_t K,
                      const void* x /*device*/, uint32_t M_b, void* y /*device*/, int y_dtype,
                      const void* residual /*device*/, void* workspace /*device*/,
                      size_t workspace_bytes, void* stream);

/* Epilogues of boost_gemv_tiered_fused.  All are applied by the threadblock that combines the
 * split-K partial sums of a row tile, in fixed order. */
enum {
  BOOST_EPI_PLAIN = 0,      /* y = acc (* row scale) (+ residual) */
  BOOST_EPI_SWIGLU = 1,     /* weight packed with row_mode 1 from [gate; up]: y[m, j] =
                               silu(bf16(gate_j)) * bf16(up_j), y bf16 [M_b, N/2] */
  BOOST_EPI_ROPE_APPEND = 2 /* N = (Hq + 2 Hkv) * 128, row tile = head: rotate q and k heads
                               (as boost_rope_kv_append), write q to q_out and k, v into the
                               paged cache; y is not written */
};

typedef struct {
  int mode;
  /* Row scale rsqrt(sum_t ssq_in[t][m] / K + rms_eps): RMSNorm of x whose weight was folded
   * into W (boost_pack_weights_ex col_scale).  ssq_in [ssq_in_tiles][ssq_stride] fp32 holds,
   * per 128-column tile of x, the sum of squares of row m; NULL = no scale. */
  const float* ssq_in; /* device */
  uint32_t ssq_in_tiles, ssq_stride;
  float rms_eps;
  /* PLAIN with bf16 output only: ssq_out[t][m] = sum of squares of the (rounded) outputs of
   * row tile t, i.e. the ssq_in of a product that consumes y.  NULL = not wanted. */
  float* ssq_out; /* device */
  /* ROPE_APPEND only */
  void* q_out;                   /* device bf16 [M_b, Hq, 128] */
  const void* const* k_page_ptr; /* device */
  const void* const* v_page_ptr; /* device */
  uint32_t n_pool_blocks;
  const int32_t* block_table;    /* device [M_b, max_blocks] */
  uint32_t max_blocks;
  const int32_t* ctx_lens;       /* device [M_b], new token included */
  uint32_t n_q_heads, n_kv_heads;
  const float* rope_table;       /* device, from boost_rope_table: (cos, sin) [M_b][64] */
  /* Optional second pair of page tables of the same cache: the new K / V rows are written
   * through both (the prefetch-to-HBM variant keeps a staged copy of host pages in HBM). */
  const void* const* k_page_ptr2; /* device or NULL */
  const void* const* v_page_ptr2; /* device or NULL */
} boost_gemv_epilogue_t;

/* Batches of at least m_b rows run on the tcgen05 kernel (operands from shared memory through
 * matrix descriptors, accumulators in tensor memory), smaller ones down to 3 rows on the
 * mma.sync kernel; 1 and 2 rows always use the CUDA cores.  Process-wide; the results of the
 * two tensor-core kernels agree to fp32 rounding.  Default 33 (measured crossover on B200).  The paper has no counterpart
 * (its matrix products are library kernels, Sec. 4.1). */
int boost_gemv_set_tc_min_batch(uint32_t m_b);

/* Where the split-K partial sums of a product are combined.  on = 1 (default): a product cut so
 * finely that a row tile has four or more partial sums (the short products of a decode layer
 * spread over the whole machine) combines all its tiles when its last block has been consumed,
 * every threadblock taking a share of the (row tile, batch row) units and requesting all partial
 * sums of a unit at once; other products, and every product with on = 0, combine each row tile in
 * the threadblock that delivers its last partial sum.  Both orders of summation are fixed, so
 * either setting is deterministic; they differ from each other in fp32 rounding.  Process-wide;
 * for measurement and tests.  The paper has no counterpart (its products are library kernels,
 * Sec. 4.1). */
int boost_gemv_set_end_combine(uint32_t on);

/* How a weight with host pages is scheduled.  0 (the default): the even partition of a weight
 * that is entirely in HBM, with every host-tier block read in place by the threadblock whose
 * contiguous share holds it - both tiers stream for as long as such shares last, no queue, no
 * specialised threadblocks.  1: the schedule of Sec. 3.2 and Sec. 3.1 - work items of one page
 * each in two queues, host-tier items handed out first to a few threadblocks that stay on that
 * tier while it has items (16-byte copies through the load/store path), the others on the HBM
 * queue.  Measured on a B200 whose host link carries 0.8 % of the HBM bandwidth, the in-place
 * form is as fast or faster for every Llama-3-8B matrix, batch size and host share tried, which
 * is why it is the default.  Under 0 the result of a product does not depend on where its pages
 * live (the same bits for every tier table); results differ between the two settings in fp32
 * rounding (other partial sums).  Process-wide; for measurement, tests and the comparison with the paper's schedule. */
int boost_gemv_set_tier_schedule(uint32_t two_queues);

/* boost_gemv_tiered with an epilogue descriptor (NULL = plain). */
int boost_gemv_tiered_fused(const void* const* w_page_ptr /*device*/, const uint32_t* w_order /*device*/,
                            size_t n_pages, size_t n_host_pages, uint32_t N, uint32_t K,
                            const void* x /*device*/, uint32_t M_b, void* y /*device*/, int y_dtype,
                            const void* residual /*device*/, const boost_gemv_epilogue_t* epilogue /*host*/,
                            void* workspace /*device*/, size_t workspace_bytes, void* stream);

/* A packed, tiered weight as consumed by boost_gemv_tiered. */
typedef struct {
  const void* const* page_ptr; /* device */
  const uint32_t* order;       /* device */
  uint64_t n_pages, n_host_pages;
  uint32_t N, K;
} boost_weight_t;

/* One product of a chain: y = x W^T with the epilogue of boost_gemv_tiered_fused
 * (has_epilogue = 0: plain). */
typedef struct {
  boost_weight_t w;
  const void* x;        /* device, bf16 [M_b, w.K] */
  void* y;              /* device (see boost_gemv_tiered_fused) */
  int y_dtype;
  const void* residual; /* device or NULL */
  int has_epilogue;
  boost_gemv_epilogue_t epilogue;
} boost_gemv_call_t;

/* A chain of 1..4 weight products in ONE launch, each of which may take what the previous
 * ones wrote (as its x, its residual or its row statistics): the results equal those of the
 * same calls of boost_gemv_tiered_fused made one after the other.  Sec. 2.1 describes decode as
 * a chain of weight-streaming products; because weights do not depend on activations, the
 * persistent threadblocks stream the next product's weight pages (both tiers, host pages
 * first, as in boost_gemv_tiered) while the tail of the current product drains, and meet at
 * a grid-wide counter between products.  All calls share M_b and the workspace.
 *   workspace  device, 256-byte aligned, >= boost_gemv_chain_workspace_bytes, zero-filled
 *              once (the kernel leaves its counters at zero, so calls that follow one another
 *              on a stream may reuse it with nothing in between); word 0 collects error bits
 *              (bit 0: a bounded wait ran out, including the waits between products).
 * Errors: INVALID (n_calls outside 1..4, a call that boost_gemv_tiered_fused would reject),
 * ALIGN, CAPACITY, UNSUPPORTED (the device cannot hold one threadblock), CUDA. */
size_t boost_gemv_chain_workspace_bytes(const boost_gemv_call_t* calls /*host*/, uint32_t n_calls, uint32_t M_b);
int boost_gemv_tiered_chain(const boost_gemv_call_t* calls /*host*/, uint32_t n_calls, uint32_t M_b,
                            void* workspace /*device*/, size_t workspace_bytes, void* stream);

/* Copy a logical KV cache [n_kv_heads][n_pool_blocks][16][D] (contiguous device buffer,
 * bf16) into the pages of a K or V tensor, or back.  Chunk (h, b) lands at byte offset
 * (h*n_pool_blocks + b) * 4 KiB of the tensor; inside a chunk token t occupies 256 bytes at
 * t*256 and its 16-byte piece c (8 values of d) sits at position c ^ (t & 7), which keeps
 * tensor-core loads of 8 consecutive tokens on distinct shared-memory banks.  D = 128. */
int boost_kv_scatter(const void* src /*device*/, uint32_t n_kv_heads, uint32_t n_pool_blocks,
                     uint32_t D, const void* const* page_ptr /*device*/, size_t n_pages, void* stream);
int boost_kv_gather(void* dst /*device*/, uint32_t n_kv_heads, uint32_t n_pool_blocks, uint32_t D,
                    const void* const* page_ptr /*device*/, size_t n_pages, void* stream);

/* One decode step of softmax attention over the paged KV cache of a boost_kv_pool
 * (Sec. 3.3: threadblocks work on KV head chunks; chunks of host-resident heads are
 * started first).
 *   q            device bf16 [B, Hq, D];  D = 128;  Hq/Hkv in 1..16;
 *   k_page_ptr, v_page_ptr  device arrays of page addresses of the K and V tensors, each
 *                laid out [Hkv][n_pool_blocks][16][D] (chunk (h, b) at (h*n_pool_blocks+b)*4 KiB,
 *                chunk-internal layout as written by boost_kv_scatter);
 *   kv_tier      host array, tier of each of the n_kv_pages pages, or NULL (all HBM); must be
 *                a linear placement (HBM pages, then host pages), else UNSUPPORTED;
 *   block_table  device int32 [B, max_blocks]; ctx_lens device int32 [B] (tokens cached,
 *                the current one included); query head j reads KV head j / (Hq/Hkv);
 *                the kernel cuts the sequences into work items from ctx_lens itself, and
 *                reads ctx_lens and block_table before it waits for the kernel launched
 *                just before it on the stream when that kernel is one of this library's
 *                (which write neither); the newest K / V rows and q are read after it;
 *   out          device bf16 [B, Hq, D];
 *   workspace    device, >= boost_paged_attn_workspace_bytes(B, Hq, D, max_blocks); its first
 *                word collects error bits (1 = a bounded wait gave up, 2 = a block index
 *                outside the pool or a context length outside [0, 16 * max_blocks]: such a
 *                block is read as block 0, such a length is clamped) and is 0 after a clean run. */
size_t boost_paged_attn_workspace_bytes(uint32_t B, uint32_t Hq, uint32_t D, uint32_t max_blocks);
int boost_paged_attn_decode_tiered(const void* q /*device*/, const void* const* k_page_ptr /*device*/,
                                   const void* const* v_page_ptr /*device*/,
                                   const uint8_t* kv_tier /*host*/, size_t n_kv_pages,
                                   uint32_t n_pool_blocks, const int32_t* block_table /*device*/,
                                   uint32_t max_blocks, const int32_t* ctx_lens /*device*/,
                                   uint32_t B, uint32_t Hq, uint32_t Hkv, uint32_t D, float scale,
                                   void* workspace /*device*/, size_t workspace_bytes,
                                   void* out /*device*/, void* stream);

/* --------------------------------------------------- glue of a decode step
 * The paper does not describe these operators (it treats decode as weight kernels plus
 * attention, Sec. 2.1, Sec. 5.4); shapes follow the public Llama-3 architecture.  All
 * tensors are bf16 row-major in device memory unless stated otherwise. */

/* out[b, :] = table[tokens[b], :];  table [vocab, hidden]; tokens device int32 [B]. */
int boost_embed_gather(const void* table /*device*/, uint32_t vocab, uint32_t hidden,
                       const int32_t* tokens /*device*/, uint32_t B, void* out /*device*/, void* stream);

/* As boost_embed_gather; also writes ssq_out[t][b] (fp32, row pitch ssq_stride >= B) = sum of
 * squares of columns [128 t, 128 t + 128) of row b, the row statistics a following
 * boost_gemv_tiered_fused needs for its RMS scale.  hidden % 128 == 0. */
int boost_embed_gather_ssq(const void* table /*device*/, uint32_t vocab, uint32_t hidden,
                           const int32_t* tokens /*device*/, uint32_t B, void* out /*device*/,
                           float* ssq_out /*device*/, uint32_t ssq_stride, void* stream);

/* out = x * rsqrt(mean(x^2) + eps) * weight, row by row; x, out [B, hidden]; weight [hidden]. */
int boost_rmsnorm(const void* x /*device*/, const void* weight /*device*/, uint32_t B, uint32_t hidden,
                  float eps, void* out /*device*/, void* stream);

/* Rotary embedding and KV append.  qkv [B, (Hq + 2 Hkv) * D] holds the query heads, then the
 * key heads, then the value heads of the new token of every sequence; its position is
 * ctx_lens[b] - 1.  Queries and keys are rotated (rotate-half pairing: element i with
 * i + D/2, angle = position * rope_base^(-2i/D)); rotated queries go to q_out [B, Hq, D];
 * rotated keys and the values are written into the paged cache (layout of
 * boost_kv_scatter) at block_table[b][pos / 16], slot pos % 16.  status_word: device
 * uint32 that receives error bits (bit 1 = a block index out of range).  D = 128. */
int boost_rope_kv_append(const void* qkv /*device*/, void* q_out /*device*/,
                         const void* const* k_page_ptr /*device*/, const void* const* v_page_ptr /*device*/,
                         uint32_t n_pool_blocks, const int32_t* block_table /*device*/, uint32_t max_blocks,
                         const int32_t* ctx_lens /*device*/, uint32_t B, uint32_t Hq, uint32_t Hkv,
                         uint32_t D, float rope_base, void* status_word /*device*/, void* stream);

/* table[b][i] = (cos, sin) of (ctx_lens[b] - 1) * rope_base^(-2i/D), i < D/2, fp32 pairs,
 * evaluated in double: the rotary angles of the new token of every sequence.  They are the
 * same for all layers of a step, so a step computes them once.  D = 128. */
int boost_rope_table(const int32_t* ctx_lens /*device*/, uint32_t B, uint32_t D, float rope_base,
                     float* table /*device, B * D/2 * 2 floats*/, void* stream);

/* out[b, f] = silu(gate_up[b, f]) * gate_up[b, F + f];  gate_up [B, 2F]; out [B, F]. */
int boost_swiglu(const void* gate_up /*device*/, uint32_t B, uint32_t F, void* out /*device*/, void* stream);

/* out[b] = index of the largest of logits[b, :] (fp32), lowest index on ties. */
int boost_argmax(const float* logits /*device*/, uint32_t B, uint32_t V, int32_t* out /*device*/,
                 void* stream);

/* ------------------------------------------------------- whole decode step */

typedef struct {
  boost_weight_t wqkv; /* [(Hq + 2 Hkv) D, hidden]: query, key, value rows; packed with col_scale = norm-1 weight */
  boost_weight_t wo;   /* [hidden, Hq D] */
  boost_weight_t wgu;  /* [2 F, hidden]: gate rows then up rows; packed with row_mode 1, col_scale = norm-2 weight */
  boost_weight_t wd;   /* [hidden, F] */
  const void* const* k_page_ptr; /* device: pages of this layer's K tensor */
  const void* const* v_page_ptr;
} boost_llama_layer_t;

typedef struct {
  uint32_t n_layers, hidden, ffn, n_q_heads, n_kv_heads, head_dim, vocab;
  float rms_eps, rope_base;
  const void* embed;      /* device bf16 [vocab, hidden] */
  boost_weight_t lm_head; /* [vocab, hidden]; packed with col_scale = final norm weight */
  const boost_llama_layer_t* layers; /* host array of n_layers entries */
  const uint8_t* kv_tier;            /* host: tier of every page of a K (or V) tensor, or NULL */
  uint64_t n_kv_pages;
  uint32_t n_pool_blocks;
} boost_llama_model_t;

/* Device scratch of a decode step for up to ssq_stride sequences (bf16 unless noted):
 * h [B, hidden] (residual stream); q_rot, attn [B, Hq D]; act [B, F]; logits fp32 [B, vocab];
 * ssq_a, ssq_b fp32 [hidden / 128][ssq_stride] (row statistics for the RMS scales); rope_table
 * fp32 [B][64][2];
 * gemv_ws >= boost_llama_gemv_workspace_bytes(model, B) (counters sized for the widest
 * product, the largest set of partial sums, one set of queue words per launch); attn_ws >=
 * boost_paged_attn_workspace_bytes; both zero-filled once and 256-byte aligned; tokens_dev /
 * ctx_dev / next_dev int32 [B] and table_dev int32 [B, max_blocks] are staging buffers used by
 * boost_llama_decode_step_host only. */
typedef struct {
  void *h, *q_rot, *attn, *act;
  float* logits;
  float *ssq_a, *ssq_b;
  uint32_t ssq_stride;
  float* rope_table; /* fp32 [B][64][2] */
  void* gemv_ws;
  size_t gemv_ws_bytes;
  void* attn_ws;
  size_t attn_ws_bytes;
  int32_t *tokens_dev, *ctx_dev, *table_dev, *next_dev;
} boost_llama_scratch_t;

/* Prefetch-to-HBM comparison variant (Sec. 2.5: the alternative to concurrent access is to
 * copy host-resident data into HBM ahead of its use; its gain is bounded by 1 - alpha).  The
 * host pages of every layer's K and V tensor occupy one contiguous range of the pinned slab
 * (boost_page_table puts them in consecutive slots); the copy engine brings that range into
 * one of two staging buffers in HBM while earlier layers compute, and the attention kernel
 * reads the staged copy through a second page table in which host pages point into the
 * staging buffer.  The new token's K / V rows are written to both copies.
 *   host_bytes                 bytes of host pages per tensor (a multiple of 2 MiB; the same
 *                              for every layer: the pool places all layers alike);
 *   k_stage / v_stage          device, two staging buffers of host_bytes each, 2 MiB aligned;
 *   layers[l].k_host_src ...   host (pinned) address of the first host page of layer l;
 *   layers[l].k_page_ptr_staged  device array like the layer's k_page_ptr with every host
 *                              page replaced by its slot in staging buffer l % 2. */
typedef struct {
  const void* k_host_src; /* pinned host */
  const void* v_host_src;
  const void* const* k_page_ptr_staged; /* device */
  const void* const* v_page_ptr_staged;
} boost_kv_prefetch_layer_t;

typedef struct {
  uint64_t host_bytes;
  void* k_stage[2];
  void* v_stage[2];
  const boost_kv_prefetch_layer_t* layers; /* host array of n_layers entries */
} boost_kv_prefetch_t;

/* Copy stream and events of the prefetch variant; one per model instance. */
typedef struct boost_prefetch_ctx boost_prefetch_ctx;
int boost_prefetch_ctx_create(uint32_t n_layers, boost_prefetch_ctx** out /*host*/);
void boost_prefetch_ctx_destroy(boost_prefetch_ctx* ctx);

/* boost_llama_decode_step with the host pages of the KV cache staged into HBM by the copy
 * engine, layer l + 2 while layers l and l + 1 compute.  Same results as
 * boost_llama_decode_step (the attention kernel reads identical bytes from another address).
 * model->kv_tier may name host pages; they are never read by the SMs in this variant. */
int boost_llama_decode_step_prefetch(const boost_llama_model_t* model /*host*/,
                                     const boost_llama_scratch_t* scratch /*host*/,
                                     const boost_kv_prefetch_t* prefetch /*host*/, boost_prefetch_ctx* ctx,
                                     const int32_t* tokens /*device*/, const int32_t* block_table /*device*/,
                                     uint32_t max_blocks, const int32_t* ctx_lens /*device*/, uint32_t B,
                                     int32_t* next_tokens /*device*/, uint32_t* n_launches_out /*host*/,
                                     void* stream);

/* Size of scratch->gemv_ws for steps of up to B sequences of this model (Sec. 2.1 treats the
 * step as a chain of weight products; they share one workspace).  0 on invalid arguments. */
size_t boost_llama_gemv_workspace_bytes(const boost_llama_model_t* model /*host*/, uint32_t B);

/* One decode step for B sequences (Sec. 2.1: a chain of weight-streaming products and
 * attention kernels): embedding, n_layers x (RMSNorm, QKV product, RoPE + KV append, paged
 * attention, output product + residual, RMSNorm, gate/up product, SwiGLU, down product +
 * residual), final RMSNorm, LM head, argmax - as 4 + 2 n_layers launches: RoPE table,
 * embedding gather, the first layer's QKV product, then per layer the attention kernel and
 * ONE chain launch (boost_gemv_tiered_chain) for the output, gate/up and down products and the
 * next layer's QKV product (the LM head after the last layer), then argmax.  Every small
 * operator rides in the epilogue of a weight product (RMSNorm as a row scale with its weight
 * folded into the matrix, RoPE + KV append after the QKV product, SwiGLU after the gate/up
 * product, the row statistics of the residual stream after the output and down products).
 * Activations between kernels are bf16; logits fp32.  tokens, block_table [B, max_blocks],
 * ctx_lens (new token included) and next_tokens are device arrays.  Launches are
 * asynchronous on stream.  Returns the number of kernels launched in *n_launches_out when
 * it is not NULL.  Errors: INVALID, UNSUPPORTED (head_dim != 128, hidden % 128 != 0),
 * CAPACITY (scratch->gemv_ws too small), CUDA. */
int boost_llama_decode_step(const boost_llama_model_t* model /*host*/,
                            const boost_llama_scratch_t* scratch /*host*/,
                            const int32_t* tokens /*device*/, const int32_t* block_table /*device*/,
                            uint32_t max_blocks, const int32_t* ctx_lens /*device*/, uint32_t B,
                            int32_t* next_tokens /*device*/, uint32_t* n_launches_out /*host*/,
                            void* stream);

/* Measurement aid: runs one step as boost_llama_decode_step does, with a pair of CUDA
 * events around every launch, waits for the stream and returns the summed device time and
 * the number of launches per kind of kernel: [0] weight products (boost_gemv_tiered),
 * [1] attention, [2] everything else.  kind_ms_out / kind_launches_out: host arrays of 3.
 * Creates and destroys its events; not for use inside a timed region. */
int boost_llama_decode_step_profile(const boost_llama_model_t* model /*host*/,
                                    const boost_llama_scratch_t* scratch /*host*/,
                                    const int32_t* tokens /*device*/, const int32_t* block_table /*device*/,
                                    uint32_t max_blocks, const int32_t* ctx_lens /*device*/, uint32_t B,
                                    int32_t* next_tokens /*device*/, float* kind_ms_out /*host*/,
                                    uint32_t* kind_launches_out /*host*/, void* stream);

/* As above with HOST buffers (pinned memory recommended): copies tokens, block_table and
 * ctx_lens to the staging buffers of `scratch`, runs the step, copies next_tokens back and
 * waits for the stream, so the result is valid on return. */
int boost_llama_decode_step_host(const boost_llama_model_t* model /*host*/,
                                 const boost_llama_scratch_t* scratch /*host*/,
                                 const int32_t* tokens /*host*/, const int32_t* block_table /*host*/,
                                 uint32_t max_blocks, const int32_t* ctx_lens /*host*/, uint32_t B,
                                 int32_t* next_tokens /*host*/, uint32_t* n_launches_out /*host*/,
                                 void* stream);

#ifdef __cplusplus
}
#endif
#endif /* BOOST_H_ */
