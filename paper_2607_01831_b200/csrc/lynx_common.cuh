// Shared host/device helpers of the Lynx CUDA library (sm_100a).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>

#include "lynx.h"

#define LYNX_D 128

namespace lynx {

__host__ inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Status of the launch just made.  With LYNX_DEBUG set in the environment the CUDA error text
// goes to stderr.
__host__ inline lynx_status launch_status() {
  const cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) return LYNX_OK;
  if (getenv("LYNX_DEBUG")) fprintf(stderr, "lynx: CUDA error at launch: %s\n", cudaGetErrorString(e));
  return LYNX_ERR_CUDA;
}

// Number of SMs of the current device (cached per device id).
__host__ int sm_count();

// Workspace header (first 256 bytes): word 0 = status flags set by kernels.
constexpr int kWsHeaderBytes = 256;
constexpr uint32_t kFlagBadBlock = 1u;
constexpr uint32_t kFlagTimeout = 2u;
constexpr uint32_t kFlagRange = 4u;

}  // namespace lynx
