// Host-side helpers shared by the .cu files: CUDA error capture, device facts.
#pragma once
#include <cuda_runtime.h>

#include "../../include/boost.h"

namespace boosth {

void set_last_cuda_error(cudaError_t e);

// Number of SMs of the current device (cached per device); 0 on failure.
int sm_count();

inline int check(cudaError_t e) {
  if (e == cudaSuccess) return BOOST_OK;
  set_last_cuda_error(e);
  return BOOST_ERR_CUDA;
}

// Launch check: picks up configuration errors of the launch just made.
inline int check_launch() { return check(cudaGetLastError()); }

}  // namespace boosth
