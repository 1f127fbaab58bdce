// Launch interface between the C ABI (api.cu) and the sm_100a kernels (kernels.cu).
#pragma once

#include <cuda_runtime.h>

#include <cstdint>

#include "bcp.h"

namespace bcp {

// Device-side control words of one plan (zero-initialised once; the kernel restores the
// first two to zero before it exits, so every launch starts from the same state).
struct Control {
  uint32_t ticket;  // next work unit to hand out
  uint32_t done;    // CTAs that have left the work loop
  uint32_t status;  // 0 or a bcp_status raised on the device
  uint32_t pad;
};

struct LaunchArgs {
  const bcp_tile* tiles;      // device: n_big CTA-wide units followed by n_small warp units
  uint32_t n_big;
  uint32_t n_small;
  const void* const* src;     // device table of source base pointers
  void* const* dst;           // device table of target base pointers
  Control* ctrl;              // device
  uint32_t block_threads;
  uint32_t grid;
  uint32_t cache_hints;       // 1 streaming, 2 plain
};

// Largest useful persistent grid for the copy kernel on the current device.
cudaError_t copy_kernel_max_grid(uint32_t block_threads, uint32_t ctas_per_sm, uint32_t* grid);

// Enqueue the multi-region copy on `stream`.
cudaError_t launch_copy(const LaunchArgs& a, cudaStream_t stream);

}  // namespace bcp
