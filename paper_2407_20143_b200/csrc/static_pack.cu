// bcp_pack_static: the pack operation for callers that must not allocate.
//
// Some hosts of this library run with every byte of device memory already handed out to
// their own pool (an inference server, a training job sized to the last megabyte) or call us
// from a point where an allocation would synchronise the device or is simply forbidden by
// the embedding framework.  bcp_pack allocates its device-side work list on first use;
// this entry point does not: work list, pointer table and the kernel's control words live in
// one fixed array in device memory that is part of the library image, and the host-side
// staging copy of it is a fixed array too.  The price is a size limit and shared state.
#include <cstring>
#include <mutex>

#include "kernels.cuh"
#include "plan.hpp"

namespace {

using namespace bcp;

// Limits of one call.  BCP_STATIC_MAX_UNITS work units of at most 64 MiB bound the payload
// far above any real blob; the tensor count is the limit callers meet in practice.
constexpr uint32_t kMaxTensors = BCP_STATIC_MAX_TENSORS;
constexpr uint32_t kMaxUnits = BCP_STATIC_MAX_UNITS;

struct StaticScratch {
  Control ctrl;                       // ticket counter, exit counter, status
  unsigned char pad[256 - sizeof(Control)];
  void* ptrs[kMaxTensors + 1 + 31];   // tensor bases, then the blob base (padded to 256 bytes)
  bcp_tile tiles[kMaxUnits];
};
static_assert(sizeof(StaticScratch) <= (1u << 20), "the scratch array is meant to stay near 1 MiB");

// Device memory that exists from the moment the library is loaded on a GPU until the process
// exits (about 0.8 MiB per GPU).  In host code this name is only a handle: the address a kernel
// can use comes from cudaGetSymbolAddress, per device.
static __device__ __align__(256) unsigned char g_scratch[sizeof(StaticScratch)];

// Host mirror of the scratch, filled per call and copied to the device; fixed storage as well.
StaticScratch g_host;
std::mutex g_mu;

constexpr int kMaxDevices = 64;
unsigned char* g_dev_ptr[kMaxDevices];  // device address of g_scratch on each device, once known

// One-time set-up per device, with that device current.
int scratch_address(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(BCP_ERR_CUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
  if (dev < 0 || dev >= kMaxDevices) return fail(BCP_ERR_INVALID, "device index %d is outside [0, %d)", dev, kMaxDevices);
  if (!g_dev_ptr[dev]) {
    unsigned char* p = nullptr;
    e = cudaGetSymbolAddress(reinterpret_cast<void**>(&p), g_scratch);
    if (e != cudaSuccess || !p)
      return fail(BCP_ERR_CUDA, "cudaGetSymbolAddress(static scratch) on device %d: %s", dev, cudaGetErrorString(e));
    g_dev_ptr[dev] = p;
  }
  *out = g_dev_ptr[dev];
  return BCP_OK;
}

// The work list is produced in two passes over the same cutting rule: a counting pass (store ==
// false) that only sizes the two groups, then a writing pass that puts CTA-wide units at
// tiles[0, n_big) and warp units at tiles[small_base, small_base + n_small), each in emission
// order.  No unit is ever moved inside the fixed array.
struct UnitWriter {
  uint32_t n_big = 0, n_small = 0;
  uint32_t small_base = 0;  // writing pass: where the warp units start (= the counted n_big)
  bool store = false;
  bool overflow = false;

  void emit(uint64_t src_off, uint64_t dst_off, uint64_t bytes, uint32_t src_buf, bool zero, uint32_t small_bytes) {
    if (bytes == 0) return;
    if (n_big + n_small >= kMaxUnits) {
      overflow = true;
      return;
    }
    if (!store) {
      if (bytes < small_bytes) ++n_small; else ++n_big;
      return;
    }
    bcp_tile t;
    memset(&t, 0, sizeof t);
    t.src_off = zero ? 0 : src_off;
    t.dst_off = dst_off;
    t.rows = 1;
    t.row_bytes = uint32_t(bytes);
    t.src_buf = src_buf;
    t.dst_buf = 0;
    uint64_t bits = dst_off | bytes | (zero ? 0 : src_off);
    uint32_t g = 0;
    while (g < 4 && !((bits >> g) & 1)) ++g;
    t.flags = g | (zero ? BCP_TILE_ZERO : 0u);
    if (bytes < small_bytes) {
      t.flags |= BCP_TILE_SMALL;
      g_host.tiles[small_base + n_small++] = t;
    } else {
      g_host.tiles[n_big++] = t;
    }
  }

  // same cutting rule as the planner: peel a ragged head and tail when both sides share their
  // remainder mod 16, then pieces of tile_bytes
  void run(uint64_t so, uint64_t dof, uint64_t n, uint32_t src_buf, bool zero, uint64_t tile_bytes, uint32_t small_bytes) {
    if (n == 0) return;
    if ((zero || ((so ^ dof) & 15) == 0) && n >= 32) {
      const uint64_t head = (16 - (dof & 15)) & 15;
      if (head) {
        emit(so, dof, head, src_buf, zero, small_bytes);
        so += head, dof += head, n -= head;
      }
      const uint64_t tail = n & 15;
      if (tail) {
        emit(so + n - tail, dof + n - tail, tail, src_buf, zero, small_bytes);
        n -= tail;
      }
    }
    while (n) {
      const uint64_t c = n < tile_bytes ? n : tile_bytes;
      emit(so, dof, c, src_buf, zero, small_bytes);
      so += c, dof += c, n -= c;
    }
  }
};

}  // namespace

extern "C" int bcp_pack_static(const void* const* tensors, const bcp_pack_meta* metas, size_t n, void* blob,
                               uint64_t blob_bytes, void* stream_) {
  cudaStream_t stream = static_cast<cudaStream_t>(stream_);
  if ((n && (!tensors || !metas)) || (blob_bytes && !blob)) return fail(BCP_ERR_INVALID, "bcp_pack_static: NULL argument");
  if (n > kMaxTensors)
    return fail(BCP_ERR_CAPACITY, "bcp_pack_static: %zu tensors, the fixed scratch holds at most %u (use bcp_pack)", n, kMaxTensors);
  uint64_t pos = 0;
  for (size_t i = 0; i < n; ++i) {
    if (metas[i].byte_offset < pos) return fail(BCP_ERR_INVALID, "bcp_pack_static: meta %zu overlaps the previous tensor", i);
    if (metas[i].byte_offset > blob_bytes || metas[i].byte_length > blob_bytes - metas[i].byte_offset)
      return fail(BCP_ERR_BOUNDS, "bcp_pack_static: meta %zu reaches past the blob (%llu bytes)", i, (unsigned long long)blob_bytes);
    if (metas[i].byte_length && !tensors[i]) return fail(BCP_ERR_INVALID, "bcp_pack_static: tensor %zu is NULL", i);
    pos = metas[i].byte_offset + metas[i].byte_length;
  }
  // The uploads below read the shared host mirror when they execute.  Recorded by a stream
  // capture they would read it again at every replay, after later calls have rewritten it, while
  // the kernel node keeps this call's unit counts: refused rather than silently wrong.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(stream, &capturing) != cudaSuccess) {
    cudaGetLastError();
    return fail(BCP_ERR_CUDA, "bcp_pack_static: cudaStreamIsCapturing failed");
  }
  if (capturing != cudaStreamCaptureStatusNone)
    return fail(BCP_ERR_INVALID, "bcp_pack_static: the stream is being captured; its uploads come from a host array that every call rewrites");
  std::lock_guard<std::mutex> lock(g_mu);
  unsigned char* dev = nullptr;
  if (int rc = scratch_address(&dev)) return rc;
  StaticScratch* d = reinterpret_cast<StaticScratch*>(dev);

  // addresses: rounded down to 16 bytes, the remainder goes into the offsets
  const uintptr_t blob_addr = reinterpret_cast<uintptr_t>(blob);
  const uint64_t blob_res = blob_addr & 15;
  for (size_t i = 0; i < n; ++i) g_host.ptrs[i] = reinterpret_cast<void*>(reinterpret_cast<uintptr_t>(tensors[i]) & ~uintptr_t(15));
  g_host.ptrs[n] = reinterpret_cast<void*>(blob_addr & ~uintptr_t(15));

  // work list; the unit size doubles until the list fits
  const uint32_t small_bytes = 4096;
  auto cut = [&](UnitWriter& w, uint64_t tile_bytes) {
    uint64_t at = 0;
    for (size_t i = 0; i < n; ++i) {
      w.run(0, blob_res + at, metas[i].byte_offset - at, 0, true, tile_bytes, small_bytes);  // padding -> zeros
      const uint64_t res = reinterpret_cast<uintptr_t>(tensors[i]) & 15;
      w.run(res, blob_res + metas[i].byte_offset, metas[i].byte_length, uint32_t(i), false, tile_bytes, small_bytes);
      at = metas[i].byte_offset + metas[i].byte_length;
    }
    w.run(0, blob_res + at, blob_bytes - at, 0, true, tile_bytes, small_bytes);
  };
  UnitWriter counted;
  uint64_t tile_bytes = 65536;
  for (;; tile_bytes *= 2) {
    counted = UnitWriter();
    cut(counted, tile_bytes);
    if (!counted.overflow) break;
    if (tile_bytes >= (64u << 20))
      return fail(BCP_ERR_CAPACITY, "bcp_pack_static: more than %u work units even at 64 MiB per unit (use bcp_pack)", kMaxUnits);
  }
  if (counted.n_big + counted.n_small == 0) return BCP_OK;
  UnitWriter w;
  w.store = true;
  w.small_base = counted.n_big;
  cut(w, tile_bytes);
  if (w.overflow || w.n_big != counted.n_big || w.n_small != counted.n_small)
    return fail(BCP_ERR_INVALID, "bcp_pack_static: the two passes over the layout disagree (arguments changed during the call?)");
  memset(&g_host.ctrl, 0, sizeof g_host.ctrl);

#define BCP_S_CUDA(call)                                                                             \
  do {                                                                                               \
    cudaError_t e_ = (call);                                                                         \
    if (e_ != cudaSuccess) return fail(BCP_ERR_CUDA, "bcp_pack_static: %s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)
  // The control words must start at zero for every launch; the pointer table and the work
  // list are overwritten as far as this call uses them.  Outside a capture (checked above)
  // pageable sources are staged by the runtime before the call returns, so g_host may be
  // reused right after.
  BCP_S_CUDA(cudaMemcpyAsync(&d->ctrl, &g_host.ctrl, sizeof(Control), cudaMemcpyHostToDevice, stream));
  BCP_S_CUDA(cudaMemcpyAsync(d->ptrs, g_host.ptrs, (n + 1) * sizeof(void*), cudaMemcpyHostToDevice, stream));
  BCP_S_CUDA(cudaMemcpyAsync(d->tiles, g_host.tiles, size_t(w.n_big + w.n_small) * sizeof(bcp_tile), cudaMemcpyHostToDevice, stream));
  LaunchArgs a;
  a.tiles = d->tiles;
  a.n_big = w.n_big;
  a.n_small = w.n_small;
  a.src = reinterpret_cast<const void* const*>(d->ptrs);
  a.dst = reinterpret_cast<void* const*>(d->ptrs + n);
  a.ctrl = &d->ctrl;
  a.block_threads = 512;
  a.cache_hints = 1;
  a.unroll = 4;
  a.warp_workers = 0;
  uint32_t grid = 0;
  BCP_S_CUDA(copy_kernel_max_grid(a.block_threads, 2, &grid));
  const uint64_t units = uint64_t(a.n_big) + (a.n_small + 15) / 16;
  a.grid = uint32_t(units < grid ? units : grid);
  BCP_S_CUDA(launch_copy(a, stream));
#undef BCP_S_CUDA
  return BCP_OK;
}
