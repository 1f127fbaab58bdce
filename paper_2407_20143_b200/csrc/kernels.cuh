// Launch interface between the C ABI (api.cu) and the sm_100a kernels (kernels.cu, tma_kernel.cu,
// convert_kernel.cu).
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
  uint32_t unroll;            // 4 or 8
  uint32_t warp_workers;      // 1: every warp is an independent worker (256-thread CTAs); 0: CTA-wide units
};

struct TmaLaunchArgs {
  const bcp_tile* tiles;  // device: n_tiles units, all eligible for bulk copies
  uint32_t n_tiles;
  uint32_t n_tail;        // units right behind them in the list that the warps copy through registers
  const void* const* src;
  void* const* dst;
  Control* ctrl;          // device, separate from the register kernel's
  uint32_t stage_bytes;   // shared-memory stage, multiple of 128
  uint32_t n_stages;      // 2..8
  uint32_t grid;
  uint64_t wait_ns;       // how long a CTA waits for one stage before it gives up (global timer)
  uint32_t test_stall;    // test hook: CTA 0 over-arms its first stage so that one wait runs out
  uint32_t cache_hints;   // 3: evict-first stores; 4: evict-first loads too; else none
  const void* maps;       // device: two 128-byte tensor maps (source view, target view) per tensor-map rectangle
};

struct ConvertLaunchArgs {
  const bcp_tile* tiles;  // device: n_units converting units (BCP_TILE_CVT_MASK set)
  uint32_t n_units;
  const void* const* src;
  void* const* dst;
  Control* ctrl;          // device, separate from the other kernels'
  uint32_t grid;
};

struct ConvertStagedLaunchArgs {
  const bcp_tile* tiles;  // device: the same n_units converting units; this kernel takes those marked BCP_TILE_TMA
  uint32_t n_units;
  const void* const* src;
  void* const* dst;
  Control* ctrl;          // device, separate from the other kernels'
  uint32_t stage_bytes;   // shared-memory stage, multiple of 128
  uint32_t n_stages;      // 2..8
  uint32_t grid;
  uint64_t wait_ns;       // how long a CTA waits for one stage before it gives up (global timer)
  uint32_t test_stall;    // test hook: CTA 0 over-arms its first stage so that one wait runs out
};

// Persistent grid of the staged converting kernel (one warp per CTA) for a stage geometry.
cudaError_t convert_staged_max_grid(uint32_t stage_bytes, uint32_t n_stages, uint32_t ctas_per_sm, uint32_t* grid);

// Enqueue the staged converting kernel on `stream`.
cudaError_t launch_convert_staged(const ConvertStagedLaunchArgs& a, cudaStream_t stream);

// Persistent grid of the converting kernel (256-thread CTAs, every warp a worker).
cudaError_t convert_kernel_max_grid(uint32_t* grid);

// Enqueue the converting kernel on `stream`.
cudaError_t launch_convert(const ConvertLaunchArgs& a, cudaStream_t stream);

// Persistent grid of the TMA staging kernel (one warp per CTA) for a stage geometry.
cudaError_t tma_kernel_max_grid(uint32_t stage_bytes, uint32_t n_stages, uint32_t ctas_per_sm, uint32_t* grid);

// Enqueue the TMA staging kernel on `stream`.
cudaError_t launch_tma(const TmaLaunchArgs& a, cudaStream_t stream);

// Persistent grid of the warp-worker form of the copy kernel (256-thread CTAs).
cudaError_t warp_kernel_max_grid(uint32_t ctas_per_sm, uint32_t* grid);

// Largest useful persistent grid for the copy kernel on the current device.
cudaError_t copy_kernel_max_grid(uint32_t block_threads, uint32_t ctas_per_sm, uint32_t* grid);

// Enqueue the multi-region copy on `stream`.
cudaError_t launch_copy(const LaunchArgs& a, cudaStream_t stream);

}  // namespace bcp
