// One virtual address range over both tiers, through the CUDA virtual-memory API.
//
// The paper's system presents kernels with an ordinary address range whose 2 MiB pages the
// operating system has placed on one tier or the other (Sec. 2.3 on the unified address space,
// Sec. 4.4 on how the allocator binds pages); kernels are not modified and see no page table.
// The rest of this library hands its kernels a table of page addresses instead.  This file
// provides the paper's form on this machine: a reserved virtual range into which HBM pages and
// pinned host pages are mapped page by page, so that anything written for a flat buffer - a
// copy, a kernel of another library - reads a tiered one.  Host code only; the driver entry
// points are looked up at run time, so the library has no link-time dependency on the driver.
#include <cuda.h>
#include <cuda_runtime.h>

#include <new>
#include <vector>

#include "host_common.h"

namespace {

struct Driver {
  CUresult (*AddressReserve)(CUdeviceptr*, size_t, size_t, CUdeviceptr, unsigned long long) = nullptr;
  CUresult (*AddressFree)(CUdeviceptr, size_t) = nullptr;
  CUresult (*Create)(CUmemGenericAllocationHandle*, size_t, const CUmemAllocationProp*, unsigned long long) = nullptr;
  CUresult (*Release)(CUmemGenericAllocationHandle) = nullptr;
  CUresult (*Map)(CUdeviceptr, size_t, size_t, CUmemGenericAllocationHandle, unsigned long long) = nullptr;
  CUresult (*Unmap)(CUdeviceptr, size_t) = nullptr;
  CUresult (*SetAccess)(CUdeviceptr, size_t, const CUmemAccessDesc*, size_t) = nullptr;
  CUresult (*Granularity)(size_t*, const CUmemAllocationProp*, CUmemAllocationGranularity_flags) = nullptr;
  bool ok = false;
};

template <typename F>
bool lookup(const char* name, F& fn) {
  void* p = nullptr;
  cudaDriverEntryPointQueryResult st;
  if (cudaGetDriverEntryPoint(name, &p, cudaEnableDefault, &st) != cudaSuccess || st != cudaDriverEntryPointSuccess || !p)
    return false;
  fn = reinterpret_cast<F>(p);
  return true;
}

const Driver& driver() {
  static Driver d = [] {
    Driver x;
    x.ok = lookup("cuMemAddressReserve", x.AddressReserve) && lookup("cuMemAddressFree", x.AddressFree) &&
           lookup("cuMemCreate", x.Create) && lookup("cuMemRelease", x.Release) && lookup("cuMemMap", x.Map) &&
           lookup("cuMemUnmap", x.Unmap) && lookup("cuMemSetAccess", x.SetAccess) &&
           lookup("cuMemGetAllocationGranularity", x.Granularity);
    return x;
  }();
  return d;
}

struct Run {
  CUmemGenericAllocationHandle handle;
  size_t offset, bytes;
  bool mapped;
};

}  // namespace

struct boost_va_buffer {
  CUdeviceptr base = 0;
  size_t bytes = 0;
  std::vector<Run> runs;   // maximal runs of consecutive pages of one tier: one allocation each
};

extern "C" int boost_va_buffer_destroy(boost_va_buffer* b) {
  if (!b) return BOOST_ERR_INVALID;
  const Driver& d = driver();
  if (d.ok) {
    for (Run& r : b->runs) {
      if (r.mapped) d.Unmap(b->base + r.offset, r.bytes);
      d.Release(r.handle);
    }
    if (b->base) d.AddressFree(b->base, b->bytes);
  }
  delete b;
  return BOOST_OK;
}

extern "C" int boost_va_buffer_create(const uint8_t* tier, size_t n_pages, int host_numa_node, boost_va_buffer** out) {
  if (!tier || !out || n_pages == 0 || host_numa_node < 0) return BOOST_ERR_INVALID;
  *out = nullptr;
  const Driver& d = driver();
  int dev = 0;
  if (!d.ok || cudaGetDevice(&dev) != cudaSuccess) return BOOST_ERR_UNSUPPORTED;
  if (cudaFree(nullptr) != cudaSuccess) return BOOST_ERR_CUDA;   // (makes sure the device's context exists)
  CUmemAllocationProp prop[2] = {};
  prop[BOOST_TIER_HBM].type = CU_MEM_ALLOCATION_TYPE_PINNED;
  prop[BOOST_TIER_HBM].location.type = CU_MEM_LOCATION_TYPE_DEVICE;
  prop[BOOST_TIER_HBM].location.id = dev;
  prop[BOOST_TIER_HOST].type = CU_MEM_ALLOCATION_TYPE_PINNED;
  prop[BOOST_TIER_HOST].location.type = CU_MEM_LOCATION_TYPE_HOST_NUMA;
  prop[BOOST_TIER_HOST].location.id = host_numa_node;
  bool any[2] = {false, false};
  for (size_t i = 0; i < n_pages; ++i) {
    if (tier[i] > BOOST_TIER_HOST) return BOOST_ERR_INVALID;
    any[tier[i]] = true;
  }
  // a page (2 MiB) must be a whole number of the allocation granules of its tier
  for (int t = 0; t < 2; ++t) {
    if (!any[t]) continue;
    size_t g = 0;
    if (d.Granularity(&g, &prop[t], CU_MEM_ALLOC_GRANULARITY_MINIMUM) != CUDA_SUCCESS || g == 0 || BOOST_PAGE_BYTES % g != 0)
      return BOOST_ERR_UNSUPPORTED;
  }
  boost_va_buffer* b = new (std::nothrow) boost_va_buffer;
  if (!b) return BOOST_ERR_INVALID;
  b->bytes = n_pages * (size_t)BOOST_PAGE_BYTES;
  int rc = BOOST_OK;
  if (d.AddressReserve(&b->base, b->bytes, BOOST_PAGE_BYTES, 0, 0) != CUDA_SUCCESS) {
    b->base = 0;
    rc = BOOST_ERR_UNSUPPORTED;
  }
  for (size_t i = 0; i < n_pages && rc == BOOST_OK;) {
    size_t j = i;
    while (j < n_pages && tier[j] == tier[i]) ++j;
    Run r = {0, i * (size_t)BOOST_PAGE_BYTES, (j - i) * (size_t)BOOST_PAGE_BYTES, false};
    if (d.Create(&r.handle, r.bytes, &prop[tier[i]], 0) != CUDA_SUCCESS) {
      rc = tier[i] == BOOST_TIER_HOST ? BOOST_ERR_UNSUPPORTED : BOOST_ERR_CAPACITY;
      break;
    }
    b->runs.push_back(r);
    if (d.Map(b->base + r.offset, r.bytes, 0, r.handle, 0) != CUDA_SUCCESS) { rc = BOOST_ERR_UNSUPPORTED; break; }
    b->runs.back().mapped = true;
    i = j;
  }
  if (rc == BOOST_OK) {
    CUmemAccessDesc acc = {};
    acc.location.type = CU_MEM_LOCATION_TYPE_DEVICE;
    acc.location.id = dev;
    acc.flags = CU_MEM_ACCESS_FLAGS_PROT_READWRITE;
    if (d.SetAccess(b->base, b->bytes, &acc, 1) != CUDA_SUCCESS) rc = BOOST_ERR_UNSUPPORTED;
  }
  if (rc != BOOST_OK) {
    boost_va_buffer_destroy(b);
    return rc;
  }
  *out = b;
  return BOOST_OK;
}

extern "C" void* boost_va_buffer_base(const boost_va_buffer* b) {
  return b ? reinterpret_cast<void*>(b->base) : nullptr;
}

extern "C" int boost_va_buffer_page_table(const boost_va_buffer* b, void** page_ptr_out, size_t cap) {
  if (!b || !page_ptr_out) return BOOST_ERR_INVALID;
  const size_t n = b->bytes / BOOST_PAGE_BYTES;
  if (cap < n) return BOOST_ERR_CAPACITY;
  for (size_t i = 0; i < n; ++i) page_ptr_out[i] = reinterpret_cast<void*>(b->base + i * (size_t)BOOST_PAGE_BYTES);
  return BOOST_OK;
}
