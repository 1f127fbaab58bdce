// The plan object behind bcp_plan_t and the internal calls shared by the files of the C ABI
// (api.cu: planning, execution, pack; plan_image.cu: images; host_path.cu: host buffers).
#pragma once

#include <cstring>
#include <vector>

#include <cuda.h>

#include "kernels.cuh"
#include "plan.hpp"

struct bcp_plan_s {
  bcp::Options opt;
  bcp_plan_stats_t stats;
  bcp::TileVec tiles;  // TMA units, then other CTA-wide units, then warp units, then converting units
  size_t n_tma = 0, n_big = 0, n_cvt = 0;
  size_t n_small() const { return tiles.size() - n_tma - n_big - n_cvt; }
  std::vector<uint64_t> src_bytes, dst_bytes;
  std::vector<bcp::Rect> rects;  // rectangles staged through tensor maps (two descriptors each)
  std::vector<bcp::Gap> gaps;    // target bytes no entry names (zeroed by the host-buffer call)
  std::vector<uint32_t> used_src;  // bcp_plan only: indices of the saved entries the work list reads
  bool has_used_src = false;
  std::vector<CUtensorMap> h_maps;
  CUtensorMap* d_maps = nullptr;
  // device side, created by the first execution
  int device = -1;
  bcp_tile* d_tiles = nullptr;
  bcp_tile* d_fan_tiles = nullptr;  // the same list with replica groups marked (in-place host path)
  void** d_ptrs = nullptr;  // source table followed by target table
  bcp::Control* d_ctrl = nullptr;  // [0] register kernel, [1] TMA kernel, [2] converting kernel, [3] staged converting kernel
  uint32_t grid = 0, tma_grid = 0, cvt_grid = 0, cvt_staged_grid = 0;
  uint32_t cvt_stage_bytes = 0, cvt_stages = 0;  // stage geometry of the staged converting kernel
  size_t n_cvt_staged = 0;  // converting units marked for the staged kernel (counted when the plan is bound)
  cudaStream_t last_stream = nullptr;
  cudaEvent_t ev_switch = nullptr;  // orders an execution after the previous one when the stream changes
  bool ran = false;
  std::vector<void*> h_ptrs;
  bool table_current = false;  // the device pointer table already holds h_ptrs
  // bcp_reshard_host: device staging plus a second copy of the work list grouped by target
  // buffer, so that uploads, kernels and downloads of different target buffers overlap
  struct Group {  // units of one target buffer inside d_host_tiles
    size_t first = 0, n_tma = 0, n_big = 0, n_small = 0, n_cvt = 0;
    std::vector<uint32_t> needs;  // source buffers its units read
  };
  std::vector<void*> stage_src, stage_dst;
  bcp_tile* d_host_tiles = nullptr;
  std::vector<Group> groups;     // one per target buffer
  std::vector<uint32_t> order;   // target buffers in processing order
  cudaStream_t s_h2d = nullptr, s_d2h = nullptr;
  std::vector<cudaEvent_t> ev_src, ev_dst;
};

#define BCP_CUDA(call)                                                                       \
  do {                                                                                       \
    cudaError_t e_ = (call);                                                                 \
    if (e_ != cudaSuccess) return bcp::fail(BCP_ERR_CUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

namespace bcp {

// First execution of a plan: upload the work list to the current device and size the grids.
int bind_device(bcp_plan_t* p);
// Upload the pointer table in h_ptrs and, for tensor-map rectangles, descriptors for those addresses.
int upload_tables(bcp_plan_t* p, cudaStream_t stream);
// Enqueue the kernels for a slice of a device work list laid out as [TMA | CTA-wide | warp | converting units].
int launch_units(bcp_plan_t* p, const bcp_tile* tiles, size_t n_tma, size_t n_big, size_t n_small, size_t n_cvt, cudaStream_t stream);
// Validate the buffers, refresh the tables if an address changed, enqueue the kernels (`list`: another device copy of the work list).
int execute(bcp_plan_t* p, const void* const* src, size_t ns, void* const* dst, size_t nd, cudaStream_t stream,
            const bcp_tile* list = nullptr);

}  // namespace bcp
