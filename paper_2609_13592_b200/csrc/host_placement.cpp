// Host side of the library: page placement, per-wave statistics, visit order and
// page-pointer tables.  Integer logic only; no CUDA calls in this file.
#include <cmath>
#include <cstdint>
#include <algorithm>
#include <cstring>
#include <vector>
#include <limits>

#include "../../include/boost.h"

namespace {

typedef unsigned __int128 u128;

// Smallest M with 1/M <= r * (1 + 2^-40), decided exactly: with r = mant * 2^e
// (53-bit integer mantissa) the test is  2^40 <= M * mant * (2^40 + 1) * 2^e.
bool ratio_admits(uint64_t m, uint64_t mant, int e) {
  // e is negative for every r <= 1/2: compare 2^(40 - e) with m * mant * (2^40 + 1).
  const int shift = 40 - e;  // <= 40 + 30 + 53 = 123 for r >= 2^-30
  if (shift >= 127) return false;
  const u128 lhs = (u128)1 << shift;
  const u128 rhs = (u128)m * (u128)mant * (((u128)1 << 40) + 1);
  return lhs <= rhs;
}

int modulus_from_ratio(double r, uint32_t* out) {
  if (!(r == r)) return BOOST_ERR_INVALID;
  if (r == 0.0) { *out = 0; return BOOST_OK; }
  if (r < std::ldexp(1.0, -30) || r > 0.5) return BOOST_ERR_INVALID;
  int e2 = 0;
  const double frac = std::frexp(r, &e2);            // r = frac * 2^e2, frac in [0.5, 1)
  const uint64_t mant = (uint64_t)std::ldexp(frac, 53);  // exact 53-bit integer
  const int e = e2 - 53;
  // start near 1/r and walk to the exact boundary
  uint64_t m = (uint64_t)(1.0 / r);
  if (m < 1) m = 1;
  while (!ratio_admits(m, mant, e)) ++m;
  while (m > 1 && ratio_admits(m - 1, mant, e)) --m;
  if (m > 0xFFFFFFFFull) return BOOST_ERR_INVALID;
  *out = (uint32_t)m;
  return BOOST_OK;
}

inline uint64_t splitmix_out(uint64_t z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}

}  // namespace

extern "C" int boost_modulus_from_ratio(double host_ratio, uint32_t* modulus_out) {
  if (!modulus_out) return BOOST_ERR_INVALID;
  return modulus_from_ratio(host_ratio, modulus_out);
}

extern "C" int boost_modulus_from_bandwidths(double hbm_bw, double link_bw, uint32_t* modulus_out) {
  if (!modulus_out || !(hbm_bw > 0.0) || !(link_bw > 0.0)) return BOOST_ERR_INVALID;
  const double q = hbm_bw / link_bw;
  if (!(q < 4.0e9)) return BOOST_ERR_INVALID;
  uint64_t k = (uint64_t)q;
  // ceil(hbm/link) without trusting the rounded quotient: k*link >= hbm must hold
  while ((double)k * link_bw < hbm_bw) ++k;
  while (k > 0 && (double)(k - 1) * link_bw >= hbm_bw) --k;
  *modulus_out = (uint32_t)(k + 1);
  return BOOST_OK;
}

extern "C" int boost_place_pages_ex(const void* buffer, size_t bytes, double host_ratio,
                                    uint32_t wave_size, int policy, uint64_t seed,
                                    uint32_t superpage_pages, uint8_t* tier_out, size_t tier_cap,
                                    size_t* n_pages_out, uint32_t* flags_out) {
  if (!n_pages_out) return BOOST_ERR_INVALID;
  if (buffer && ((uintptr_t)buffer % BOOST_PAGE_BYTES) != 0) return BOOST_ERR_ALIGN;
  if (superpage_pages < 1) return BOOST_ERR_INVALID;
  if (policy != BOOST_POLICY_MODULO && policy != BOOST_POLICY_CONTIGUOUS &&
      policy != BOOST_POLICY_RANDOM)
    return BOOST_ERR_INVALID;
  if (policy != BOOST_POLICY_MODULO && superpage_pages != 1) return BOOST_ERR_INVALID;
  uint32_t m = 0;
  const int rc = modulus_from_ratio(host_ratio, &m);
  if (rc != BOOST_OK) return rc;
  const size_t p = bytes / BOOST_PAGE_BYTES + ((bytes % BOOST_PAGE_BYTES) ? 1 : 0);
  *n_pages_out = p;
  if (flags_out) *flags_out = (m != 0 && wave_size != 0 && wave_size < m) ? BOOST_FLAG_WAVE_SHORTER_THAN_PERIOD : 0u;
  if (p == 0) return BOOST_OK;
  if (!tier_out) return BOOST_ERR_INVALID;
  if (tier_cap < p) return BOOST_ERR_CAPACITY;
  std::memset(tier_out, BOOST_TIER_HBM, p);
  if (m == 0) return BOOST_OK;
  if (policy == BOOST_POLICY_MODULO) {
    // host groups are groups m-1, 2m-1, ...; mark their pages without dividing per page
    const size_t s = superpage_pages;
    for (size_t first = (size_t)(m - 1) * s; first < p; first += (size_t)m * s) {
      const size_t last = (first + s < p) ? first + s : p;
      std::memset(tier_out + first, BOOST_TIER_HOST, last - first);
    }
  } else if (policy == BOOST_POLICY_CONTIGUOUS) {
    const size_t n_host = p / m;
    std::memset(tier_out + (p - n_host), BOOST_TIER_HOST, n_host);
  } else {
    const uint64_t threshold = std::numeric_limits<uint64_t>::max() / m +
                               ((std::numeric_limits<uint64_t>::max() % m) == (uint64_t)(m - 1) ? 1 : 0);
    uint64_t state = seed;
    for (size_t i = 0; i < p; ++i) {
      state += 0x9E3779B97F4A7C15ull;  // seed + (i+1) * gamma
      if (splitmix_out(state) < threshold) tier_out[i] = BOOST_TIER_HOST;
    }
  }
  return BOOST_OK;
}

extern "C" int boost_place_pages(const void* buffer, size_t bytes, double host_ratio,
                                 uint32_t wave_size, uint8_t* tier_out, size_t tier_cap,
                                 size_t* n_pages_out) {
  return boost_place_pages_ex(buffer, bytes, host_ratio, wave_size, BOOST_POLICY_MODULO, 0, 1,
                              tier_out, tier_cap, n_pages_out, nullptr);
}

extern "C" int boost_wave_stats(const uint8_t* tier, size_t n_pages, size_t tile_bytes,
                                uint32_t ctas_per_wave, double host_ratio,
                                boost_wave_stats_t* out) {
  if (!out || (!tier && n_pages) || tile_bytes == 0 || ctas_per_wave == 0) return BOOST_ERR_INVALID;
  if (BOOST_PAGE_BYTES % tile_bytes != 0) return BOOST_ERR_INVALID;
  if (!(host_ratio >= 0.0)) return BOOST_ERR_INVALID;
  const uint64_t tpp = BOOST_PAGE_BYTES / tile_bytes;
  const uint64_t n_tiles = (uint64_t)n_pages * tpp;
  const uint64_t g = ctas_per_wave;
  std::memset(out, 0, sizeof(*out));
  for (size_t i = 0; i < n_pages; ++i) out->n_host_pages += (tier[i] == BOOST_TIER_HOST);
  if (n_tiles == 0) return BOOST_OK;
  // prefix count of host tiles at page granularity: host tiles before tile t
  //   = tpp * hostpages_before(page(t)) + (tier[page] ? t % tpp : 0)
  // walk waves with a running page cursor instead of storing the prefix array
  const double slack = host_ratio * (1.0 + std::ldexp(1.0, -40));
  double sum = 0.0, sumsq_dev = 0.0, mn = 2.0, mx = -1.0;
  const uint64_t n_waves = (n_tiles + g - 1) / g;
  // two passes (mean, then variance) over per-wave counts recomputed on the fly
  for (int pass = 0; pass < 2; ++pass) {
    const double mean = (pass == 1) ? sum / (double)n_waves : 0.0;
    uint64_t page = 0, host_before_page = 0;  // cursor state for tile index `t0`
    uint64_t host_before_t0 = 0;
    for (uint64_t w = 0; w < n_waves; ++w) {
      const uint64_t t1 = ((w + 1) * g < n_tiles) ? (w + 1) * g : n_tiles;
      // advance the cursor to tile t1
      const uint64_t page1 = t1 / tpp;
      while (page < page1) { host_before_page += (tier[page] == BOOST_TIER_HOST); ++page; }
      uint64_t host_before_t1 = host_before_page * tpp;
      if (page1 < n_pages && tier[page1] == BOOST_TIER_HOST) host_before_t1 += t1 % tpp;
      const uint64_t host = host_before_t1 - host_before_t0;
      const uint64_t size = t1 - w * g;
      const double f = (double)host / (double)size;
      if (pass == 0) {
        sum += f;
        if (f < mn) mn = f;
        if (f > mx) mx = f;
        if (host == 0) ++out->n_zero_waves;
        if (f > slack) ++out->n_over_waves;
      } else {
        sumsq_dev += (f - mean) * (f - mean);
      }
      host_before_t0 = host_before_t1;
    }
  }
  out->n_waves = n_waves;
  out->mean = sum / (double)n_waves;
  out->var = sumsq_dev / (double)n_waves;
  out->min = mn;
  out->max = mx;
  return BOOST_OK;
}

extern "C" int boost_tier_order(const uint8_t* tier, size_t n_pages, uint32_t* order_out,
                                size_t* n_host_out) {
  if (!n_host_out || (n_pages && (!tier || !order_out))) return BOOST_ERR_INVALID;
  if (n_pages > 0xFFFFFFFFull) return BOOST_ERR_INVALID;
  size_t n_host = 0;
  for (size_t i = 0; i < n_pages; ++i) n_host += (tier[i] == BOOST_TIER_HOST);
  size_t h = 0, d = n_host;  // two write cursors: host part, then HBM part
  for (size_t i = 0; i < n_pages; ++i) {
    if (tier[i] == BOOST_TIER_HOST) order_out[h++] = (uint32_t)i;
    else order_out[d++] = (uint32_t)i;
  }
  *n_host_out = n_host;
  return BOOST_OK;
}

extern "C" int boost_page_table(const uint8_t* tier, size_t n_pages, void* hbm_slab,
                                size_t hbm_slab_bytes, void* host_slab, size_t host_slab_bytes,
                                void** page_ptr_out) {
  if (n_pages && (!tier || !page_ptr_out)) return BOOST_ERR_INVALID;
  if (((uintptr_t)hbm_slab % BOOST_PAGE_BYTES) || ((uintptr_t)host_slab % BOOST_PAGE_BYTES))
    return BOOST_ERR_ALIGN;
  size_t n_host = 0;
  for (size_t i = 0; i < n_pages; ++i) n_host += (tier[i] == BOOST_TIER_HOST);
  const size_t n_hbm = n_pages - n_host;
  if (n_hbm && (!hbm_slab || hbm_slab_bytes / BOOST_PAGE_BYTES < n_hbm)) return BOOST_ERR_CAPACITY;
  if (n_host && (!host_slab || host_slab_bytes / BOOST_PAGE_BYTES < n_host)) return BOOST_ERR_CAPACITY;
  char* next_hbm = (char*)hbm_slab;
  char* next_host = (char*)host_slab;
  for (size_t i = 0; i < n_pages; ++i) {
    if (tier[i] == BOOST_TIER_HOST) { page_ptr_out[i] = next_host; next_host += BOOST_PAGE_BYTES; }
    else { page_ptr_out[i] = next_hbm; next_hbm += BOOST_PAGE_BYTES; }
  }
  return BOOST_OK;
}

// ---- statistics of a schedule log (see boost.h)

extern "C" size_t boost_schedule_log_bytes(size_t capacity) {
  return 32 + capacity * sizeof(boost_schedule_record_t);
}

namespace {

struct ShareStats {
  uint64_t n = 0, n_zero = 0, n_over = 0;
  std::vector<double> f;
  void add(double host, double all, double slack) {
    const double v = host / all;
    f.push_back(v);
    ++n;
    if (host == 0.0) ++n_zero;
    if (v > slack) ++n_over;
  }
  void fill(boost_wave_stats_t* out, uint64_t n_host_items) const {
    std::memset(out, 0, sizeof(*out));
    out->n_waves = n;
    out->n_host_pages = n_host_items;
    out->n_zero_waves = n_zero;
    out->n_over_waves = n_over;
    if (!n) return;
    double sum = 0.0, mn = f[0], mx = f[0];
    for (double v : f) { sum += v; mn = v < mn ? v : mn; mx = v > mx ? v : mx; }
    const double mean = sum / (double)n;
    double dev = 0.0;
    for (double v : f) dev += (v - mean) * (v - mean);
    out->mean = mean; out->var = dev / (double)n; out->min = mn; out->max = mx;
  }
};

}  // namespace

extern "C" int boost_schedule_stats(const void* log, size_t log_bytes, uint32_t kind, uint32_t items_per_wave,
                                    uint64_t window_ns, double host_ratio, boost_wave_stats_t* wave_out,
                                    boost_wave_stats_t* window_out, uint64_t* n_records_out) {
  if (!log || !wave_out || !window_out || !n_records_out || items_per_wave == 0 || window_ns == 0) return BOOST_ERR_INVALID;
  if (log_bytes < 32 || !(host_ratio >= 0.0)) return BOOST_ERR_INVALID;
  const uint64_t* head = static_cast<const uint64_t*>(log);
  const uint64_t claimed = head[0], capacity = head[1];
  const uint64_t n_all = claimed < capacity ? claimed : capacity;
  if (log_bytes < 32 + n_all * sizeof(boost_schedule_record_t)) return BOOST_ERR_INVALID;
  const boost_schedule_record_t* rec = reinterpret_cast<const boost_schedule_record_t*>(head + 4);
  std::vector<const boost_schedule_record_t*> r;
  for (uint64_t i = 0; i < n_all; ++i) {
    if (kind && (rec[i].kind_phase & 0xFFu) != kind) continue;
    if (rec[i].t_consumed == 0 || rec[i].bytes == 0) continue;
    r.push_back(rec + i);
  }
  std::sort(r.begin(), r.end(), [](const boost_schedule_record_t* a, const boost_schedule_record_t* b) {
    if (a->t_request != b->t_request) return a->t_request < b->t_request;
    if (a->cta_warp != b->cta_warp) return a->cta_warp < b->cta_warp;
    return a->kind_phase < b->kind_phase;
  });
  *n_records_out = r.size();
  uint64_t n_host_items = 0;
  for (const auto* x : r) n_host_items += x->host_bytes > 0;
  const double slack = host_ratio * (1.0 + std::ldexp(1.0, -40));
  // waves of consecutive starts
  ShareStats waves;
  for (size_t i = 0; i < r.size(); i += items_per_wave) {
    uint64_t host = 0, all = 0;
    for (size_t j = i; j < r.size() && j < i + items_per_wave; ++j) { host += r[j]->host_bytes; all += r[j]->bytes; }
    waves.add((double)host, (double)all, slack);
  }
  waves.fill(wave_out, n_host_items);
  // time windows: a record's bytes spread evenly over its interval
  ShareStats windows;
  if (!r.empty()) {
    uint64_t t0 = r[0]->t_request, t1 = 0;
    for (const auto* x : r) {
      const uint64_t e = x->t_consumed > x->t_request ? x->t_consumed : x->t_request + 1;
      t1 = e > t1 ? e : t1;
    }
    const uint64_t n_win = (t1 - t0 + window_ns - 1) / window_ns;
    std::vector<double> host(n_win, 0.0), all(n_win, 0.0);
    for (const auto* x : r) {
      const uint64_t a = x->t_request - t0;
      const uint64_t e = (x->t_consumed > x->t_request ? x->t_consumed : x->t_request + 1) - t0;
      const double dur = (double)(e - a);
      for (uint64_t w = a / window_ns; w * window_ns < e; ++w) {
        const uint64_t lo = w * window_ns > a ? w * window_ns : a;
        const uint64_t hi = (w + 1) * window_ns < e ? (w + 1) * window_ns : e;
        const double part = (double)(hi - lo) / dur;
        host[w] += part * (double)x->host_bytes;
        all[w] += part * (double)x->bytes;
      }
    }
    for (uint64_t w = 0; w < n_win; ++w)
      if (all[w] > 0.0) windows.add(host[w], all[w], slack);
  }
  windows.fill(window_out, n_host_items);
  return BOOST_OK;
}

