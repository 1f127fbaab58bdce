// Internal structures shared by the host planner, the C ABI and the kernel launcher.
#pragma once

#include <cstdarg>
#include <cstdint>
#include <memory>
#include <new>
#include <string>
#include <utility>
#include <vector>

#include "bcp.h"

namespace bcp {

// Thread-local error text behind bcp_last_error().
std::string& last_error();
int fail(int code, const char* fmt, ...);

// A copy (or zero-fill) request before it is cut into work units: rows x row_bytes bytes.
struct Item {
  uint64_t src_off = 0, dst_off = 0;
  uint64_t src_pitch = 0, dst_pitch = 0;
  uint64_t row_bytes = 0;  // may exceed 4 GiB; cut into tiles later
  uint64_t rows = 1;
  uint32_t src_buf = 0, dst_buf = 0;
  bool zero = false;  // no source: write zeros
  uint8_t cvt = 0;    // BCP_CONVERT_*: row_bytes counts target bytes, the source row holds the same elements
  // bytes of one source row
  uint64_t src_row_bytes() const { return cvt == BCP_CONVERT_F32_TO_BF16 ? row_bytes * 2 : cvt == BCP_CONVERT_BF16_TO_F32 ? row_bytes / 2 : row_bytes; }
};

struct Options {
  uint32_t tile_bytes = 65536;
  uint32_t run_tile_bytes = 0;  // unit size of 16-byte aligned contiguous runs; 0: chosen from the work list (see build_tiles)
  uint32_t small_bytes = 4096;
  uint32_t block_threads = 512;
  uint32_t ctas_per_sm = 0;  // 0: chosen from the work list
  uint32_t order = 0;  // 0: chosen from the work list (see build_tiles)
  uint32_t path_mask = 0;  // 0: decided from the work list
  uint32_t cache_hints = 1;
  uint32_t tma_stage_bytes = 0;  // 0: chosen from the work list (see build_tiles)
  uint32_t tma_stages = 0;
  uint32_t tma_ctas_per_sm = 0;
  uint32_t unroll = 4;
  uint32_t worker = 0;  // 0: chosen from the work list
  uint32_t tma_min_row_bytes = 512;
  uint32_t allow_replicas = 0;
  uint32_t tma_wait_ms = 2000;
  uint32_t test_stall = 0;
  uint32_t fanout = 1;  // 1 on, 2 off
  uint32_t convert = 0, convert_src_tag = 0, convert_dst_tag = 0;
  uint32_t src_buf_first = 0, src_buf_count = 0;  // count 0: pieces from every source buffer are executed
};

// A strided rectangle that is staged with 2-D tensor-map copies.  Its two descriptors (source
// view, target view) depend on buffer addresses and are encoded when the plan is executed.
struct Rect {
  uint64_t src_off, dst_off, src_pitch, dst_pitch, rows;
  uint32_t row_bytes, src_buf, dst_buf, box_rows;
};

// Bytes of a target buffer that no target entry names.
struct Gap {
  uint64_t off, len;
  uint32_t buf, pad;
};

int parse_options(const bcp_plan_opts* in, Options* out);

// Irregular-tensor decomposition (Sec. 3.2): boxes relative to the local tensor, flat order.
struct RelBox {
  int64_t off[BCP_MAX_NDIM];
  int64_t len[BCP_MAX_NDIM];
};
void decompose(const int64_t* lengths, uint32_t ndim, int64_t a, int64_t b, std::vector<RelBox>* out);

// Matching (Sec. 3.3 Step 2) + lowering: metas -> items.  Fills the entry / intersection
// counters of `stats` and, if asked, the ascending indices of the saved entries the items read.
int match_and_lower(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes, size_t n_src_bufs,
                    const bcp_shard_meta* dst, size_t n_dst, const uint64_t* dst_buf_bytes, size_t n_dst_bufs,
                    const Options& opt, std::vector<Item>* items, std::vector<Gap>* gaps, bcp_plan_stats_t* stats,
                    std::vector<uint32_t>* used_src);

// Coalesce adjacent items, cut them into work units, classify and order them.
// tiles = [TMA units..., other CTA-wide units..., warp units..., converting units...].
// Mark groups of TMA units (ordered by source address) that read the same source bytes.
void mark_followers(bcp_tile* tma, size_t n);

// A work list can hold a million units: a vector whose resize() leaves the new elements
// uninitialised, so that the threads which fill it are the first to touch its pages.
template <class T>
struct NoInitAlloc : std::allocator<T> {
  template <class U>
  struct rebind {
    using other = NoInitAlloc<U>;
  };
  NoInitAlloc() = default;
  template <class U>
  NoInitAlloc(const NoInitAlloc<U>&) {}
  template <class U>
  void construct(U* p) {
    ::new (static_cast<void*>(p)) U;
  }
  template <class U, class... A>
  void construct(U* p, A&&... a) {
    ::new (static_cast<void*>(p)) U(std::forward<A>(a)...);
  }
};
using TileVec = std::vector<bcp_tile, NoInitAlloc<bcp_tile>>;

// src_bytes: sizes of the source buffers (bounds for over-reading aligned supersets).
// Large lists are built by several host threads (at most 8; the environment variable
// BCP_PLAN_THREADS overrides the count); the result does not depend on how many.
void build_tiles(std::vector<Item>& items, Options& opt, const std::vector<uint64_t>* src_bytes, TileVec* tiles,
                 size_t* n_tma, size_t* n_big, size_t* n_cvt, std::vector<Rect>* rects, bcp_plan_stats_t* stats);

}  // namespace bcp
