// Register (LDG/STG) kernels that execute the resharding work list, or the part of it that the
// TMA staging kernel (tma_kernel.cu) does not take: pieces that are not 16-byte aligned in two
// dimensions, rows too short for bulk copies, zero fills, and units under 4 KiB.
//
// One persistent kernel runs its whole list (Sec. 3.3 Step 5 of arXiv 2407.20143: every
// matched segment is copied into its target shard).  CTAs draw work units from an atomic
// ticket counter; a unit is either one CTA-wide tile (up to tile_bytes of payload, a run or a
// strided rectangle) or a batch of small tiles, one per warp.  Every tile carries the widest
// power-of-two access width (1..16 bytes) that divides its offsets, row length and pitches;
// the copy loops are instantiated for each width and keep U independent loads in flight per
// thread before the first store.
#include "kernels.cuh"
#include "copy_loops.cuh"

namespace bcp {
namespace {

// ---------------------------------------------------------------- the persistent kernel
template <int NT, int U, int HINT>
__global__ void __launch_bounds__(NT, 1024 / NT) bcp_copy_kernel(const bcp_tile* __restrict__ tiles, uint32_t n_big,
                                                        uint32_t n_small, const void* const* __restrict__ src,
                                                        void* const* __restrict__ dst, Control* ctrl) {
  __shared__ uint32_t s_unit[2];
  const uint32_t tid = threadIdx.x;
  constexpr uint32_t nwarps = NT >> 5;
  const uint32_t n_units = n_big + (n_small + nwarps - 1) / nwarps;
  if (tid == 0) s_unit[0] = atomicAdd(&ctrl->ticket, 1u);
  __syncthreads();
  for (uint32_t it = 0;; ++it) {
    const uint32_t u = s_unit[it & 1];
    if (u >= n_units) break;
    // draw the next ticket now so that its latency hides behind this unit's copy
    if (tid == 0) s_unit[(it + 1) & 1] = atomicAdd(&ctrl->ticket, 1u);
    if (u < n_big) {
      const bcp_tile t = load_tile(tiles + u);
      copy_tile<U, HINT, NT>(t, src, dst, tid);
    } else {
      const uint32_t i = (u - n_big) * nwarps + (tid >> 5);
      if (i < n_small) {
        const bcp_tile t = load_tile(tiles + n_big + i);
        copy_tile<2, HINT, 32>(t, src, dst, tid & 31);
      }
    }
    __syncthreads();
  }
  // every CTA draws exactly one ticket past the end; the last CTA to leave rewinds the
  // counters so that the next launch starts from zero
  if (tid == 0) {
    __threadfence();
    const uint32_t left = atomicAdd(&ctrl->done, 1u);
    if (left == gridDim.x - 1) {
      ctrl->ticket = 0;
      ctrl->done = 0;
      __threadfence();
    }
  }
}

// ---------------------------------------------------------------- warp workers
// The same work list with every warp as an independent worker: a warp draws a unit (CTA-wide
// and small units alike), copies it alone with U x 512 bytes in flight, and moves on.  No
// CTA-wide barrier, and the ticket and the record of the next unit are fetched while the
// current unit is being copied, so the dependent chain ticket -> record -> base pointers ->
// data never stalls the SM: 32 warps per SM are at different points of it.
template <int U, int HINT>
__global__ void __launch_bounds__(256, 4) bcp_copy_kernel_warps(const bcp_tile* __restrict__ tiles, uint32_t n_units,
                                                                const void* const* __restrict__ src,
                                                                void* const* __restrict__ dst, Control* ctrl) {
  const uint32_t lane = threadIdx.x & 31;
  uint32_t pending = 0;  // lane 0: ticket drawn but not yet used
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
  uint32_t u = __shfl_sync(0xffffffffu, pending, 0);
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
  bcp_tile t;
  if (u < n_units) t = load_tile(tiles + u);
  while (u < n_units) {
    const uint32_t next = __shfl_sync(0xffffffffu, pending, 0);
    if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);  // for the unit after the next
    bcp_tile tn;
    if (next < n_units) tn = load_tile(tiles + next);  // in flight while this unit is copied
    copy_tile<U, HINT, 32>(t, src, dst, lane);
    u = next;
    t = tn;
  }
  // every warp has drawn tickets past the end; the last warp to leave rewinds the counters
  if (lane == 0) {
    __threadfence();
    const uint32_t left = atomicAdd(&ctrl->done, 1u);
    if (left == gridDim.x * (blockDim.x >> 5) - 1) {
      ctrl->ticket = 0;
      ctrl->done = 0;
      __threadfence();
    }
  }
}

template <int NT, int HINT>
cudaError_t launch_as(const LaunchArgs& a, cudaStream_t stream) {
  if (a.unroll == 8) {
    bcp_copy_kernel<NT, 8, HINT><<<a.grid, NT, 0, stream>>>(a.tiles, a.n_big, a.n_small, a.src, a.dst, a.ctrl);
  } else {
    bcp_copy_kernel<NT, 4, HINT><<<a.grid, NT, 0, stream>>>(a.tiles, a.n_big, a.n_small, a.src, a.dst, a.ctrl);
  }
  return cudaGetLastError();
}

template <int HINT>
cudaError_t launch_hint(const LaunchArgs& a, cudaStream_t stream) {
  if (a.warp_workers) {
    const uint32_t n_units = a.n_big + a.n_small;
    if (a.unroll == 8) {
      bcp_copy_kernel_warps<8, HINT><<<a.grid, 256, 0, stream>>>(a.tiles, n_units, a.src, a.dst, a.ctrl);
    } else {
      bcp_copy_kernel_warps<4, HINT><<<a.grid, 256, 0, stream>>>(a.tiles, n_units, a.src, a.dst, a.ctrl);
    }
    return cudaGetLastError();
  }
  switch (a.block_threads) {
    case 256: return launch_as<256, HINT>(a, stream);
    case 512: return launch_as<512, HINT>(a, stream);
    case 1024: return launch_as<1024, HINT>(a, stream);
    default: return cudaErrorInvalidConfiguration;
  }
}

}  // namespace

cudaError_t warp_kernel_max_grid(uint32_t ctas_per_sm, uint32_t* grid) {
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_copy_kernel_warps<8, 1>, 256, 0);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  const uint32_t k = ctas_per_sm < uint32_t(per_sm) ? ctas_per_sm : uint32_t(per_sm);
  *grid = uint32_t(sms) * k;
  return cudaSuccess;
}

cudaError_t copy_kernel_max_grid(uint32_t block_threads, uint32_t ctas_per_sm, uint32_t* grid) {
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  switch (block_threads) {
    case 256: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_copy_kernel<256, 4, 1>, 256, 0); break;
    case 512: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_copy_kernel<512, 4, 1>, 512, 0); break;
    case 1024: e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_copy_kernel<1024, 4, 1>, 1024, 0); break;
    default: return cudaErrorInvalidConfiguration;
  }
  if (e != cudaSuccess) return e;
  if (per_sm < 1) per_sm = 1;
  const uint32_t k = ctas_per_sm < uint32_t(per_sm) ? ctas_per_sm : uint32_t(per_sm);
  *grid = uint32_t(sms) * k;
  return cudaSuccess;
}

cudaError_t launch_copy(const LaunchArgs& a, cudaStream_t stream) {
  if (a.n_big + a.n_small == 0) return cudaSuccess;
  if (a.cache_hints == 2) return launch_hint<2>(a, stream);
  return launch_hint<1>(a, stream);
}

}  // namespace bcp
