// A peer GPU's HBM as the second tier (the bandwidth-ratio ablation over NVLink, "Bandwidth Ratio
// Ablation with NVLinks"): host-side set-up only.  The kernels need nothing new - a page table
// holds device-visible addresses, and a page that lives in a peer's memory is read like a page in
// pinned host memory: by the threadblock that owns it, with its own plain or bulk copies (one threadblock, one
// destination), over NVLink instead of the CPU link.  The placement modulus for such a tier
// comes from boost_modulus_from_bandwidths(hbm, nvlink).
#include <cuda_runtime.h>

#include "host_common.h"

namespace {

// Runs f with `device` current and puts the caller's device back.
template <typename F>
int on_device(int device, F f) {
  int cur = -1;
  int rc = boosth::check(cudaGetDevice(&cur));
  if (rc != BOOST_OK) return rc;
  rc = boosth::check(cudaSetDevice(device));
  if (rc != BOOST_OK) return rc;
  rc = f();
  const int back = boosth::check(cudaSetDevice(cur));
  return rc != BOOST_OK ? rc : back;
}

int check_peer(int peer_device, int* cur_out) {
  int cur = -1, n = 0;
  int rc = boosth::check(cudaGetDevice(&cur));
  if (rc != BOOST_OK) return rc;
  rc = boosth::check(cudaGetDeviceCount(&n));
  if (rc != BOOST_OK) return rc;
  if (peer_device < 0 || peer_device >= n || peer_device == cur) return BOOST_ERR_INVALID;
  *cur_out = cur;
  return BOOST_OK;
}

}  // namespace

extern "C" int boost_peer_tier_open(int peer_device) {
  int cur = -1;
  int rc = check_peer(peer_device, &cur);
  if (rc != BOOST_OK) return rc;
  int can = 0;
  rc = boosth::check(cudaDeviceCanAccessPeer(&can, cur, peer_device));
  if (rc != BOOST_OK) return rc;
  if (!can) return BOOST_ERR_UNSUPPORTED;
  const cudaError_t e = cudaDeviceEnablePeerAccess(peer_device, 0);
  if (e == cudaErrorPeerAccessAlreadyEnabled) {
    (void)cudaGetLastError();   // not an error for the caller: clear it
    return BOOST_OK;
  }
  return boosth::check(e);
}

extern "C" int boost_peer_tier_alloc(int peer_device, size_t bytes, void** slab_out) {
  if (!slab_out || bytes == 0) return BOOST_ERR_INVALID;
  int cur = -1;
  int rc = check_peer(peer_device, &cur);
  if (rc != BOOST_OK) return rc;
  void* ptr = nullptr;
  // cudaMalloc returns allocations of this size aligned to 2 MiB and more on current drivers, but
  // nothing promises it: one page of slack, and the caller aligns (as for every slab)
  rc = on_device(peer_device, [&]() {
    const cudaError_t e = cudaMalloc(&ptr, bytes);
    if (e == cudaErrorMemoryAllocation) {
      (void)cudaGetLastError();
      return (int)BOOST_ERR_CAPACITY;
    }
    return boosth::check(e);
  });
  if (rc != BOOST_OK) return rc;
  *slab_out = ptr;
  return BOOST_OK;
}

extern "C" int boost_peer_tier_free(int peer_device, void* slab) {
  if (!slab) return BOOST_OK;
  int cur = -1;
  const int rc = check_peer(peer_device, &cur);
  if (rc != BOOST_OK) return rc;
  return on_device(peer_device, [&]() { return boosth::check(cudaFree(slab)); });
}
