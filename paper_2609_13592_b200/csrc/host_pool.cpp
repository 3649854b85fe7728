// Host side of the library: the wave-aware pool of free KV blocks.
// Free lists are fixed-capacity ring buffers over block indices; the kind of a block
// follows from one threshold index derived in closed form from the linear placement.
#include <cstdint>
#include <new>
#include <unordered_map>
#include <vector>

#include "../../include/boost.h"

namespace {

struct Ring {
  std::vector<int32_t> slot;
  uint32_t head = 0, count = 0;
  void init(uint32_t capacity) { slot.assign(capacity ? capacity : 1, 0); head = 0; count = 0; }
  void push(int32_t b) { slot[(head + count) % slot.size()] = b; ++count; }
  int32_t pop() { const int32_t b = slot[head]; head = (head + 1) % slot.size(); --count; return b; }
};

struct Request {
  std::vector<int32_t> blocks;
  int kind = 0;
};

}  // namespace

struct boost_kv_pool {
  uint32_t n_blocks, n_kv_heads, host_modulus, chunk_bytes;
  uint32_t n_pages, n_host_pages, host_heads_lo, first_hi_block;
  Ring ring[2];  // [0] = lo, [1] = hi
  std::unordered_map<uint64_t, Request> requests;
  uint64_t live_blocks = 0, live_hi_blocks = 0;
};

extern "C" int boost_kv_pool_create(uint32_t n_blocks, uint32_t n_kv_heads, uint32_t host_modulus,
                                    uint32_t chunk_bytes, boost_kv_pool_t** pool_out) {
  if (!pool_out || n_blocks == 0 || n_kv_heads == 0 || chunk_bytes == 0 || host_modulus == 1)
    return BOOST_ERR_INVALID;
  if (BOOST_PAGE_BYTES % chunk_bytes != 0) return BOOST_ERR_INVALID;
  const uint64_t head_bytes = (uint64_t)n_blocks * chunk_bytes;
  if (head_bytes % BOOST_PAGE_BYTES != 0) return BOOST_ERR_INVALID;
  const uint64_t pages_per_head = head_bytes / BOOST_PAGE_BYTES;
  const uint64_t n_pages = pages_per_head * n_kv_heads;
  if (n_pages > 0xFFFFFFFFull || n_blocks > 0x7FFFFFFFu) return BOOST_ERR_INVALID;
  boost_kv_pool* p = new (std::nothrow) boost_kv_pool();
  if (!p) return BOOST_ERR_NOMEM;
  p->n_blocks = n_blocks;
  p->n_kv_heads = n_kv_heads;
  p->host_modulus = host_modulus;
  p->chunk_bytes = chunk_bytes;
  p->n_pages = (uint32_t)n_pages;
  const uint64_t n_host = host_modulus ? n_pages / host_modulus : 0;
  p->n_host_pages = (uint32_t)n_host;
  // The last n_host pages are host pages.  Whole heads at the top are entirely on the
  // host; the head below them has its last (n_host mod pages_per_head) pages there.
  p->host_heads_lo = (uint32_t)(n_host / pages_per_head);
  const uint64_t partial_pages = n_host % pages_per_head;
  const uint64_t chunks_per_page = BOOST_PAGE_BYTES / chunk_bytes;
  p->first_hi_block = (uint32_t)(n_blocks - partial_pages * chunks_per_page);
  p->ring[0].init(p->first_hi_block);
  p->ring[1].init(n_blocks - p->first_hi_block);
  for (uint32_t b = 0; b < p->first_hi_block; ++b) p->ring[0].push((int32_t)b);
  for (uint32_t b = p->first_hi_block; b < n_blocks; ++b) p->ring[1].push((int32_t)b);
  *pool_out = p;
  return BOOST_OK;
}

extern "C" int boost_kv_pool_alloc(boost_kv_pool_t* pool, uint64_t request_id, uint32_t n,
                                   int32_t* block_ids_out) {
  if (!pool || !block_ids_out || n == 0) return BOOST_ERR_INVALID;
  const uint64_t free_lo = pool->ring[0].count, free_hi = pool->ring[1].count;
  if (free_lo + free_hi < n) return BOOST_ERR_NOMEM;
  auto it = pool->requests.find(request_id);
  if (it == pool->requests.end()) {
    int kind = 0;
    if (pool->host_modulus != 0) {
      // hi iff free_hi / free > (H - k_lo*M) / M, in integers (no division)
      const uint64_t target_num =
          (uint64_t)pool->n_kv_heads - (uint64_t)pool->host_heads_lo * pool->host_modulus;
      if (free_hi * pool->host_modulus > target_num * (free_lo + free_hi)) kind = 1;
    }
    it = pool->requests.emplace(request_id, Request()).first;
    it->second.kind = kind;
  }
  Request& rq = it->second;
  rq.blocks.reserve(rq.blocks.size() + n);
  for (uint32_t i = 0; i < n; ++i) {
    if (pool->ring[rq.kind].count == 0) rq.kind ^= 1;  // borrow, and keep the new kind
    const int32_t b = pool->ring[rq.kind].pop();
    rq.blocks.push_back(b);
    block_ids_out[i] = b;
    pool->live_hi_blocks += ((uint32_t)b >= pool->first_hi_block);
  }
  pool->live_blocks += n;
  return BOOST_OK;
}

extern "C" int boost_kv_pool_free(boost_kv_pool_t* pool, uint64_t request_id) {
  if (!pool) return BOOST_ERR_INVALID;
  auto it = pool->requests.find(request_id);
  if (it == pool->requests.end()) return BOOST_ERR_INVALID;
  for (int32_t b : it->second.blocks) {
    const int hi = ((uint32_t)b >= pool->first_hi_block);
    pool->ring[hi].push(b);
    pool->live_hi_blocks -= hi;
  }
  pool->live_blocks -= it->second.blocks.size();
  pool->requests.erase(it);
  return BOOST_OK;
}

extern "C" int boost_kv_pool_query(const boost_kv_pool_t* pool, boost_kv_pool_info_t* o) {
  if (!pool || !o) return BOOST_ERR_INVALID;
  o->n_blocks = pool->n_blocks;
  o->n_kv_heads = pool->n_kv_heads;
  o->host_modulus = pool->host_modulus;
  o->chunk_bytes = pool->chunk_bytes;
  o->n_pages = pool->n_pages;
  o->n_host_pages = pool->n_host_pages;
  o->host_heads_lo = pool->host_heads_lo;
  o->first_hi_block = pool->first_hi_block;
  o->free_lo = pool->ring[0].count;
  o->free_hi = pool->ring[1].count;
  o->live_blocks = (uint32_t)pool->live_blocks;
  o->n_requests = (uint32_t)pool->requests.size();
  o->live_host_chunks = pool->live_blocks * pool->host_heads_lo + pool->live_hi_blocks;
  o->live_chunks = pool->live_blocks * pool->n_kv_heads;
  return BOOST_OK;
}

extern "C" int boost_kv_pool_request_kind(const boost_kv_pool_t* pool, uint64_t request_id,
                                          int* kind_out) {
  if (!pool || !kind_out) return BOOST_ERR_INVALID;
  auto it = pool->requests.find(request_id);
  if (it == pool->requests.end()) return BOOST_ERR_INVALID;
  *kind_out = it->second.kind;
  return BOOST_OK;
}

extern "C" int boost_kv_pool_page_tiers(const boost_kv_pool_t* pool, uint8_t* tier_out,
                                        size_t tier_cap, size_t* n_pages_out) {
  if (!pool || !n_pages_out) return BOOST_ERR_INVALID;
  *n_pages_out = pool->n_pages;
  if (!tier_out) return BOOST_ERR_INVALID;
  if (tier_cap < pool->n_pages) return BOOST_ERR_CAPACITY;
  const uint32_t first_host = pool->n_pages - pool->n_host_pages;
  for (uint32_t i = 0; i < pool->n_pages; ++i)
    tier_out[i] = (i >= first_host) ? BOOST_TIER_HOST : BOOST_TIER_HBM;
  return BOOST_OK;
}

extern "C" int boost_kv_pool_destroy(boost_kv_pool_t* pool) {
  if (!pool) return BOOST_ERR_INVALID;
  delete pool;
  return BOOST_OK;
}
