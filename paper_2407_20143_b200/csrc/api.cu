// C ABI of the resharding engine: plan objects, execution, pack / unpack.
// (Plan images are in plan_image.cu, the host-buffer call in host_path.cu.)
#include <chrono>
#include <cstdio>
#include <cstdlib>
#include <mutex>
#include <new>

#include "plan_object.hpp"

using namespace bcp;

namespace bcp {

// Only warp units (under 4 KiB each) ride along: one warp copies such a unit in a round trip or two,
// while a CTA-wide unit of 64 KiB would keep a single warp busy for tens of microseconds.
constexpr size_t kFoldMaxSmall = 8192;
inline bool folds(size_t n_tma, size_t n_big, size_t n_small) { return n_tma && n_big == 0 && n_small > 0 && n_small <= kFoldMaxSmall; }
constexpr int kControls = 4;  // control blocks of a plan, one per kernel
// Stage geometry of the staged converting kernel.  The warp converts out of shared memory itself,
// so what counts is how many warps an SM has at work: six one-warp CTAs with two 16 KiB stages each
// (192 KiB of shared memory per SM, like the copy) measured best on the full-size 8B merge
// (7.02 ms; four CTAs with three stages 7.61 ms, two CTAs with three 32 KiB stages 11.6 ms).
constexpr uint32_t kCvtStageBytes = 16384, kCvtStages = 2, kCvtCtasPerSm = 6;

int bind_device_alloc(bcp_plan_t* p) {
  const size_t n_ptrs = p->src_bytes.size() + p->dst_bytes.size();
  if (!p->tiles.empty()) {
    BCP_CUDA(cudaMalloc(&p->d_tiles, p->tiles.size() * sizeof(bcp_tile)));
    BCP_CUDA(cudaMemcpy(p->d_tiles, p->tiles.data(), p->tiles.size() * sizeof(bcp_tile), cudaMemcpyHostToDevice));
  }
  BCP_CUDA(cudaMalloc(&p->d_ptrs, (n_ptrs ? n_ptrs : 1) * sizeof(void*)));
  if (!p->rects.empty()) {
    BCP_CUDA(cudaMalloc(&p->d_maps, p->rects.size() * 2 * sizeof(CUtensorMap)));
    p->h_maps.resize(p->rects.size() * 2);
  }
  BCP_CUDA(cudaMalloc(&p->d_ctrl, kControls * sizeof(Control)));
  BCP_CUDA(cudaMemset(p->d_ctrl, 0, kControls * sizeof(Control)));
  if (p->opt.worker == 2) {
    BCP_CUDA(warp_kernel_max_grid(p->opt.ctas_per_sm, &p->grid));
  } else {
    BCP_CUDA(copy_kernel_max_grid(p->opt.block_threads, p->opt.ctas_per_sm, &p->grid));
  }
  if (p->n_tma)
    BCP_CUDA(tma_kernel_max_grid(p->opt.tma_stage_bytes, p->opt.tma_stages, p->opt.tma_ctas_per_sm, &p->tma_grid));
  if (p->n_cvt) {
    BCP_CUDA(convert_kernel_max_grid(&p->cvt_grid));
    p->n_cvt_staged = 0;
    for (size_t i = p->tiles.size() - p->n_cvt; i < p->tiles.size(); ++i) p->n_cvt_staged += (p->tiles[i].flags & BCP_TILE_TMA) != 0;
    if (p->n_cvt_staged) {
      p->cvt_stage_bytes = kCvtStageBytes, p->cvt_stages = kCvtStages;
      uint32_t per_sm = kCvtCtasPerSm;
      if (const char* g = getenv("BCP_CVT_GEOMETRY")) {  // tuning override: "stage_bytes,stages,ctas_per_sm"
        unsigned a = 0, b = 0, c = 0;
        if (sscanf(g, "%u,%u,%u", &a, &b, &c) == 3 && a >= 1024 && a % 128 == 0 && b >= 2 && b <= 8 && c >= 1 && c <= 16)
          p->cvt_stage_bytes = a, p->cvt_stages = b, per_sm = c;
      }
      BCP_CUDA(convert_staged_max_grid(p->cvt_stage_bytes, p->cvt_stages, per_sm, &p->cvt_staged_grid));
    }
  }
  p->h_ptrs.resize(n_ptrs);
  return BCP_OK;
}

// First execution of a plan: upload the work list to the current device and size the grids.
int bind_device(bcp_plan_t* p) {
  int dev = 0;
  BCP_CUDA(cudaGetDevice(&dev));
  if (p->device >= 0) {
    if (p->device != dev) return fail(BCP_ERR_INVALID, "plan is bound to device %d but device %d is current", p->device, dev);
    return BCP_OK;
  }
  if (int rc = bind_device_alloc(p)) {  // leave nothing half-built behind
    cudaFree(p->d_tiles);
    cudaFree(p->d_ptrs);
    cudaFree(p->d_ctrl);
    cudaFree(p->d_maps);
    p->d_maps = nullptr;
    p->d_tiles = nullptr;
    p->d_ptrs = nullptr;
    p->d_ctrl = nullptr;
    cudaGetLastError();
    return rc;
  }
  p->device = dev;
  return BCP_OK;
}

// Tensor maps are encoded by the driver; the entry point is looked up once (no link against libcuda).
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
int encode_fn(EncodeTiledFn* out) {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* sym = nullptr;
    cudaDriverEntryPointQueryResult q;
    BCP_CUDA(cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &sym, cudaEnableDefault, &q));
    if (q != cudaDriverEntryPointSuccess || !sym) return fail(BCP_ERR_CUDA, "cuTensorMapEncodeTiled is not available in this driver");
    fn = reinterpret_cast<EncodeTiledFn>(sym);
  }
  *out = fn;
  return BCP_OK;
}

// One view of a rectangle: `rows` rows of row_bytes bytes, `pitch` apart, as a 2-D tensor of
// 8-byte elements; a box is the whole row width times box_rows rows.
int encode_view(EncodeTiledFn fn, CUtensorMap* map, void* base, const Rect& r, uint64_t pitch) {
  if (reinterpret_cast<uintptr_t>(base) & 15) return fail(BCP_ERR_INVALID, "rectangle base address is not 16-byte aligned");
  const cuuint64_t dims[2] = {r.row_bytes / 8, r.rows};
  const cuuint64_t strides[1] = {pitch};
  const cuuint32_t box[2] = {r.row_bytes / 8, r.box_rows};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult rc = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, base, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (rc != CUDA_SUCCESS) return fail(BCP_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", int(rc));
  return BCP_OK;
}

// Upload the pointer table in h_ptrs and, for tensor-map rectangles, descriptors for those addresses.
int upload_tables(bcp_plan_t* p, cudaStream_t stream) {
  const size_t ns = p->src_bytes.size(), nd = p->dst_bytes.size();
  p->table_current = false;
  if (!p->rects.empty()) {
    EncodeTiledFn fn;
    if (int rc = encode_fn(&fn)) return rc;
    for (size_t i = 0; i < p->rects.size(); ++i) {
      const Rect& r = p->rects[i];
      char* sb = static_cast<char*>(p->h_ptrs[r.src_buf]) + r.src_off;
      char* db = static_cast<char*>(p->h_ptrs[ns + r.dst_buf]) + r.dst_off;
      if (int rc = encode_view(fn, &p->h_maps[2 * i], sb, r, r.src_pitch)) return rc;
      if (int rc = encode_view(fn, &p->h_maps[2 * i + 1], db, r, r.dst_pitch)) return rc;
    }
    BCP_CUDA(cudaMemcpyAsync(p->d_maps, p->h_maps.data(), p->h_maps.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, stream));
  }
  // pageable sources: the runtime stages them before returning, so the host copies may be reused
  BCP_CUDA(cudaMemcpyAsync(p->d_ptrs, p->h_ptrs.data(), (ns + nd) * sizeof(void*), cudaMemcpyHostToDevice, stream));
  p->table_current = true;
  return BCP_OK;
}

// Enqueue the kernels for a slice of a device work list laid out as [TMA | CTA-wide | warp | converting units].
int launch_units(bcp_plan_t* p, const bcp_tile* tiles, size_t n_tma, size_t n_big, size_t n_small, size_t n_cvt,
                 cudaStream_t stream) {
  const size_t ns = p->src_bytes.size();
  // A rest of nothing but a few thousand warp units rides along in the staging kernel (one launch
  // instead of two); anything more is better served by the register kernel's many warps.
  const bool fold = folds(n_tma, n_big, n_small);
  if (n_tma) {
    TmaLaunchArgs t;
    t.tiles = tiles;
    t.n_tiles = uint32_t(n_tma);
    t.n_tail = fold ? uint32_t(n_big + n_small) : 0u;
    t.src = reinterpret_cast<const void* const*>(p->d_ptrs);
    t.dst = reinterpret_cast<void* const*>(p->d_ptrs + ns);
    t.ctrl = p->d_ctrl + 1;
    t.stage_bytes = p->opt.tma_stage_bytes;
    t.n_stages = p->opt.tma_stages;
    t.grid = uint32_t(n_tma < p->tma_grid ? n_tma : p->tma_grid);
    t.wait_ns = uint64_t(p->opt.tma_wait_ms) * 1000000ull;
    t.test_stall = p->opt.test_stall;
    t.cache_hints = p->opt.cache_hints;
    t.maps = p->d_maps;
    BCP_CUDA(launch_tma(t, stream));
  }
  LaunchArgs a;
  a.tiles = tiles + n_tma;
  a.n_big = uint32_t(n_big);
  a.n_small = uint32_t(n_small);
  a.src = reinterpret_cast<const void* const*>(p->d_ptrs);
  a.dst = reinterpret_cast<void* const*>(p->d_ptrs + ns);
  a.ctrl = p->d_ctrl;
  a.block_threads = p->opt.block_threads;
  a.warp_workers = p->opt.worker == 2;
  const uint32_t nwarps = a.block_threads / 32;
  uint64_t units = uint64_t(a.n_big) + (a.n_small + nwarps - 1) / nwarps;  // CTA-wide units + batches of warp units
  uint64_t ctas = units;
  if (a.warp_workers) {
    units = uint64_t(a.n_big) + a.n_small;
    ctas = (units + 7) / 8;  // 8 warps per CTA
  }
  a.grid = uint32_t(ctas < p->grid ? ctas : p->grid);
  a.cache_hints = p->opt.cache_hints;
  a.unroll = p->opt.unroll;
  if (units && !fold) BCP_CUDA(launch_copy(a, stream));
  // converting units: both kernels walk the same list; the staged one takes the units marked
  // BCP_TILE_TMA, the register one the rest (a kernel that would find nothing is not launched)
  if (n_cvt && p->n_cvt_staged) {
    ConvertStagedLaunchArgs c;
    c.tiles = tiles + n_tma + n_big + n_small;
    c.n_units = uint32_t(n_cvt);
    c.src = a.src;
    c.dst = a.dst;
    c.ctrl = p->d_ctrl + 3;
    c.stage_bytes = p->cvt_stage_bytes;
    c.n_stages = p->cvt_stages;
    c.grid = p->cvt_staged_grid;
    c.wait_ns = uint64_t(p->opt.tma_wait_ms) * 1000000ull;
    c.test_stall = p->opt.test_stall;
    BCP_CUDA(launch_convert_staged(c, stream));
  }
  if (n_cvt && p->n_cvt_staged < p->n_cvt) {
    ConvertLaunchArgs c;
    c.tiles = tiles + n_tma + n_big + n_small;
    c.n_units = uint32_t(n_cvt);
    c.src = a.src;
    c.dst = a.dst;
    c.ctrl = p->d_ctrl + 2;
    c.grid = p->cvt_grid;
    BCP_CUDA(launch_convert(c, stream));
  }
  return BCP_OK;
}

int execute(bcp_plan_t* p, const void* const* src, size_t ns, void* const* dst, size_t nd, cudaStream_t stream,
            const bcp_tile* list) {
  if (!p) return fail(BCP_ERR_INVALID, "plan is NULL");
  if (ns != p->src_bytes.size() || nd != p->dst_bytes.size())
    return fail(BCP_ERR_INVALID, "buffer counts (%zu, %zu) differ from the planned (%zu, %zu)", ns, nd, p->src_bytes.size(),
                p->dst_bytes.size());
  if ((ns && !src) || (nd && !dst)) return fail(BCP_ERR_INVALID, "pointer array is NULL");
  for (size_t i = 0; i < ns; ++i)
    if (!src[i] && p->src_bytes[i]) return fail(BCP_ERR_INVALID, "source buffer %zu is NULL", i);
  for (size_t i = 0; i < nd; ++i)
    if (!dst[i] && p->dst_bytes[i]) return fail(BCP_ERR_INVALID, "target buffer %zu is NULL", i);
  // the access width of every work unit was derived from byte offsets, so bases must be 16-byte aligned
  for (size_t i = 0; i < ns; ++i)
    if (reinterpret_cast<uintptr_t>(src[i]) & 15) return fail(BCP_ERR_INVALID, "source buffer %zu is not 16-byte aligned", i);
  for (size_t i = 0; i < nd; ++i)
    if (reinterpret_cast<uintptr_t>(dst[i]) & 15) return fail(BCP_ERR_INVALID, "target buffer %zu is not 16-byte aligned", i);
  if (int rc = bind_device(p)) return rc;
  if (p->tiles.empty()) return BCP_OK;
  // Executions of a plan share its pointer tables and ticket counters.  On the same stream they
  // are ordered anyway; when the stream changes (two users of one cached pack layout, say) the
  // new stream is made to wait for everything queued on the previous one.  Not during a stream
  // capture, which must not depend on outside work: there the caller orders the executions.
  if (p->ran && p->last_stream != stream) {
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone) {
      if (!p->ev_switch) BCP_CUDA(cudaEventCreateWithFlags(&p->ev_switch, cudaEventDisableTiming));
      if (cudaEventRecord(p->ev_switch, p->last_stream) == cudaSuccess) {
        BCP_CUDA(cudaStreamWaitEvent(stream, p->ev_switch, 0));
      } else {
        cudaGetLastError();  // the previous stream no longer exists (then its work is done) or is being captured
      }
    } else {
      cudaGetLastError();
    }
  }
  // The device pointer table is refreshed only when a base address changed since the last
  // execution (executions of a plan are ordered, so the previous upload has been consumed).
  bool same = p->table_current;
  for (size_t i = 0; same && i < ns; ++i) same = p->h_ptrs[i] == src[i];
  for (size_t i = 0; same && i < nd; ++i) same = p->h_ptrs[ns + i] == dst[i];
  if (!same) {
    for (size_t i = 0; i < ns; ++i) p->h_ptrs[i] = const_cast<void*>(src[i]);
    for (size_t i = 0; i < nd; ++i) p->h_ptrs[ns + i] = dst[i];
    if (int rc = upload_tables(p, stream)) return rc;
  }
  if (int rc = launch_units(p, list ? list : p->d_tiles, p->n_tma, p->n_big, p->n_small(), p->n_cvt, stream)) return rc;
  p->last_stream = stream;
  p->ran = true;
  return BCP_OK;
}

}  // namespace bcp

namespace {

bcp_plan_t* finish_plan(std::vector<Item>& items, const Options& opt, bcp_plan_stats_t stats,
                      std::vector<uint64_t> src_bytes, std::vector<uint64_t> dst_bytes) {
  bcp_plan_t* p = new (std::nothrow) bcp_plan_t;
  if (!p) return nullptr;
  p->opt = opt;
  p->stats = stats;
  p->src_bytes = std::move(src_bytes);
  p->dst_bytes = std::move(dst_bytes);
  build_tiles(items, p->opt, &p->src_bytes, &p->tiles, &p->n_tma, &p->n_big, &p->n_cvt, &p->rects, &p->stats);
  return p;
}

double ms_since(std::chrono::steady_clock::time_point t0) {
  return std::chrono::duration<double, std::milli>(std::chrono::steady_clock::now() - t0).count();
}

// ------------------------------------------------------------------ pack / unpack plan cache
struct PackEntry {
  bool unpack;
  int device;  // plans are bound to the device they first ran on
  uint64_t blob_bytes;
  std::vector<uint8_t> residues;  // address mod 16 of every tensor, then of the blob
  std::vector<bcp_pack_meta> metas;
  bcp_plan_t* plan;
  uint64_t stamp;
};
std::mutex g_pack_mu;
std::vector<PackEntry> g_pack_cache;
uint64_t g_pack_stamp = 0;
const size_t kPackCacheMax = 16;

// Tensor and blob addresses need no alignment: each is rounded down to a 16-byte boundary
// and the remainder (`residues`) becomes part of the planned byte offsets, so the access
// width of every unit accounts for it.  A layout is cached per set of remainders.
int pack_plan(bool unpack, const bcp_pack_meta* metas, size_t n, uint64_t blob_bytes,
              const std::vector<uint8_t>& residues, bcp_plan_t** out) {
  int device = 0;
  BCP_CUDA(cudaGetDevice(&device));
  for (PackEntry& e : g_pack_cache) {
    if (e.unpack == unpack && e.device == device && e.blob_bytes == blob_bytes && e.metas.size() == n && e.residues == residues &&
        (n == 0 || memcmp(e.metas.data(), metas, n * sizeof(bcp_pack_meta)) == 0)) {
      e.stamp = ++g_pack_stamp;
      *out = e.plan;
      return BCP_OK;
    }
  }
  uint64_t pos = 0;
  for (size_t i = 0; i < n; ++i) {
    if (metas[i].byte_offset < pos)
      return fail(BCP_ERR_INVALID, "pack meta %zu starts at %llu, before the end (%llu) of the previous tensor", i,
                  (unsigned long long)metas[i].byte_offset, (unsigned long long)pos);
    if (metas[i].byte_offset > blob_bytes || metas[i].byte_length > blob_bytes - metas[i].byte_offset)
      return fail(BCP_ERR_BOUNDS, "pack meta %zu reaches past the blob (%llu bytes)", i, (unsigned long long)blob_bytes);
    pos = metas[i].byte_offset + metas[i].byte_length;
  }
  const auto t0 = std::chrono::steady_clock::now();
  std::vector<Item> items;
  const uint64_t blob_res = residues[n];
  std::vector<uint64_t> tensor_bytes(n), blob(1, blob_bytes + blob_res);
  pos = 0;
  for (size_t i = 0; i < n; ++i) {
    tensor_bytes[i] = metas[i].byte_length + residues[i];
    Item it;
    it.row_bytes = metas[i].byte_length;
    if (!unpack) {
      if (metas[i].byte_offset > pos) {  // padding before this tensor is written as zeros
        Item z;
        z.zero = true;
        z.dst_off = blob_res + pos;
        z.row_bytes = metas[i].byte_offset - pos;
        items.push_back(z);
      }
      it.src_buf = uint32_t(i);
      it.src_off = residues[i];
      it.dst_off = blob_res + metas[i].byte_offset;
    } else {
      it.dst_buf = uint32_t(i);
      it.dst_off = residues[i];
      it.src_off = blob_res + metas[i].byte_offset;
    }
    items.push_back(it);
    pos = metas[i].byte_offset + metas[i].byte_length;
  }
  if (!unpack && pos < blob_bytes) {
    Item z;
    z.zero = true;
    z.dst_off = blob_res + pos;
    z.row_bytes = blob_bytes - pos;
    items.push_back(z);
  }
  Options opt;
  opt.order = 2;
  bcp_plan_stats_t st;
  memset(&st, 0, sizeof st);
  st.n_src_entries = unpack ? 1 : n;
  st.n_dst_entries = unpack ? n : 1;
  st.n_intersections = n;
  bcp_plan_t* p = unpack ? finish_plan(items, opt, st, blob, tensor_bytes) : finish_plan(items, opt, st, tensor_bytes, blob);
  if (!p) return fail(BCP_ERR_NOMEM, "out of host memory");
  uint64_t uniq = 0;
  for (size_t i = 0; i < n; ++i) uniq += metas[i].byte_length;
  p->stats.bytes_src_unique = uniq;
  p->stats.plan_ms = ms_since(t0);
  if (g_pack_cache.size() >= kPackCacheMax) {
    size_t victim = 0;
    for (size_t i = 1; i < g_pack_cache.size(); ++i)
      if (g_pack_cache[i].stamp < g_pack_cache[victim].stamp) victim = i;
    bcp_plan_destroy(g_pack_cache[victim].plan);
    g_pack_cache.erase(g_pack_cache.begin() + victim);
  }
  g_pack_cache.push_back(PackEntry{unpack, device, blob_bytes, residues, std::vector<bcp_pack_meta>(metas, metas + n), p, ++g_pack_stamp});
  *out = p;
  return BCP_OK;
}

// address -> (address rounded down to 16 bytes, remainder)
void* split_addresses(const void* const* tensors, size_t n, void* blob, std::vector<uint8_t>* res,
                      std::vector<const void*>* bases) {
  res->resize(n + 1);
  bases->resize(n ? n : 1);
  for (size_t i = 0; i < n; ++i) {
    const uintptr_t a = reinterpret_cast<uintptr_t>(tensors[i]);
    (*res)[i] = uint8_t(a & 15);
    (*bases)[i] = reinterpret_cast<const void*>(a & ~uintptr_t(15));
  }
  const uintptr_t b = reinterpret_cast<uintptr_t>(blob);
  (*res)[n] = uint8_t(b & 15);
  return reinterpret_cast<void*>(b & ~uintptr_t(15));
}

}  // namespace

extern "C" {

int bcp_version(void) { return 202; }  // 0.2.2: plan options (and so plan images) carry the source-buffer range and the run unit size

const char* bcp_last_error(void) { return last_error().c_str(); }

int bcp_decompose(const int64_t* lengths, uint32_t ndim, int64_t flat_begin, int64_t flat_end,
                  int64_t (*out_off)[BCP_MAX_NDIM], int64_t (*out_len)[BCP_MAX_NDIM], size_t cap, size_t* n) {
  if (!n || (ndim && !lengths) || ndim > BCP_MAX_NDIM) return fail(BCP_ERR_INVALID, "bcp_decompose: bad arguments");
  int64_t vol = 1;
  for (uint32_t k = 0; k < ndim; ++k) {
    if (lengths[k] < 0) return fail(BCP_ERR_INVALID, "bcp_decompose: negative length");
    vol *= lengths[k];
  }
  if (flat_begin < 0 || flat_end < flat_begin || flat_end > vol)
    return fail(BCP_ERR_INVALID, "bcp_decompose: range [%lld, %lld) outside %lld elements", (long long)flat_begin,
                (long long)flat_end, (long long)vol);
  std::vector<RelBox> boxes;
  decompose(lengths, ndim, flat_begin, flat_end, &boxes);
  *n = boxes.size();
  if (boxes.size() > cap) return fail(BCP_ERR_CAPACITY, "bcp_decompose: %zu boxes, room for %zu", boxes.size(), cap);
  if (!boxes.empty() && (!out_off || !out_len)) return fail(BCP_ERR_INVALID, "bcp_decompose: output arrays are NULL");
  for (size_t i = 0; i < boxes.size(); ++i)
    for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) {
      out_off[i][k] = k < ndim ? boxes[i].off[k] : 0;
      out_len[i][k] = k < ndim ? boxes[i].len[k] : 0;
    }
  return BCP_OK;
}

int bcp_dedup_assign(const uint64_t* shard_bytes, const uint64_t* holder_offsets, const uint32_t* holders, size_t n_shards,
                     size_t n_ranks, uint64_t* rank_load, uint32_t* out_owner) {
  if (n_shards && (!shard_bytes || !holder_offsets || !holders || !out_owner)) return fail(BCP_ERR_INVALID, "bcp_dedup_assign: NULL argument");
  if (n_ranks && !rank_load) return fail(BCP_ERR_INVALID, "bcp_dedup_assign: rank_load is NULL");
  // validate everything first: a failing call must leave its outputs untouched
  for (size_t i = 0; i < n_shards; ++i) {
    if (holder_offsets[i + 1] <= holder_offsets[i]) return fail(BCP_ERR_INVALID, "bcp_dedup_assign: shard %zu has no holder", i);
    for (uint64_t k = holder_offsets[i]; k < holder_offsets[i + 1]; ++k)
      if (holders[k] >= n_ranks) return fail(BCP_ERR_BOUNDS, "bcp_dedup_assign: shard %zu is held by rank %u of %zu", i, holders[k], n_ranks);
  }
  for (size_t i = 0; i < n_shards; ++i) {
    uint32_t best = holders[holder_offsets[i]];
    for (uint64_t k = holder_offsets[i] + 1; k < holder_offsets[i + 1]; ++k) {
      const uint32_t r = holders[k];
      if (rank_load[r] < rank_load[best] || (rank_load[r] == rank_load[best] && r < best)) best = r;
    }
    rank_load[best] += shard_bytes[i];
    out_owner[i] = best;
  }
  return BCP_OK;
}

int bcp_plan(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes, size_t n_src_bufs,
             const bcp_shard_meta* dst, size_t n_dst, const uint64_t* dst_buf_bytes, size_t n_dst_bufs,
             const bcp_plan_opts* opts, bcp_plan_t** out_plan) {
  if (!out_plan) return fail(BCP_ERR_INVALID, "out_plan is NULL");
  const auto t0 = std::chrono::steady_clock::now();
  Options opt;
  if (int rc = parse_options(opts, &opt)) return rc;
  try {
    std::vector<Item> items;
    std::vector<Gap> gaps;
    bcp_plan_stats_t st;
    memset(&st, 0, sizeof st);
    std::vector<uint32_t> used;
    if (int rc = match_and_lower(src, n_src, src_buf_bytes, n_src_bufs, dst, n_dst, dst_buf_bytes, n_dst_bufs, opt, &items, &gaps, &st, &used))
      return rc;
    bcp_plan_t* p = finish_plan(items, opt, st, std::vector<uint64_t>(src_buf_bytes, src_buf_bytes + n_src_bufs),
                              std::vector<uint64_t>(dst_buf_bytes, dst_buf_bytes + n_dst_bufs));
    if (!p) return fail(BCP_ERR_NOMEM, "out of host memory");
    p->gaps = std::move(gaps);
    p->used_src = std::move(used);
    p->has_used_src = true;
    if (p->tiles.size() > 0xFFFF0000ull) {
      delete p;
      return fail(BCP_ERR_INVALID, "work list too long for one launch");
    }
    p->stats.plan_ms = ms_since(t0);
    *out_plan = p;
  } catch (const std::bad_alloc&) {
    return fail(BCP_ERR_NOMEM, "out of host memory");
  }
  return BCP_OK;
}

int bcp_plan_stats(const bcp_plan_t* plan, bcp_plan_stats_t* out) {
  if (!plan || !out) return fail(BCP_ERR_INVALID, "bcp_plan_stats: NULL argument");
  *out = plan->stats;
  size_t staged = 0;
  for (size_t i = plan->tiles.size() - plan->n_cvt; i < plan->tiles.size(); ++i) staged += (plan->tiles[i].flags & BCP_TILE_TMA) != 0;
  const size_t rest = plan->n_big + plan->n_small();
  out->n_kernels = (plan->n_tma > 0) + (rest > 0 && !folds(plan->n_tma, plan->n_big, plan->n_small())) + (staged > 0) +
                   (staged < plan->n_cvt);
  return BCP_OK;
}

int bcp_plan_used_sources(const bcp_plan_t* plan, uint32_t* out, size_t cap, size_t* n) {
  if (!plan || !n || (cap && !out)) return fail(BCP_ERR_INVALID, "bcp_plan_used_sources: NULL argument");
  if (!plan->has_used_src) return fail(BCP_ERR_INVALID, "bcp_plan_used_sources: this plan was not built by bcp_plan (images and pack layouts do not record it)");
  *n = plan->used_src.size();
  const size_t k = cap < plan->used_src.size() ? cap : plan->used_src.size();
  if (k) memcpy(out, plan->used_src.data(), k * sizeof(uint32_t));
  return BCP_OK;
}

int bcp_plan_tiles(const bcp_plan_t* plan, bcp_tile* out, size_t cap, size_t* n) {
  if (!plan || !n || (cap && !out)) return fail(BCP_ERR_INVALID, "bcp_plan_tiles: NULL argument");
  *n = plan->tiles.size();
  const size_t k = cap < plan->tiles.size() ? cap : plan->tiles.size();
  if (k) memcpy(out, plan->tiles.data(), k * sizeof(bcp_tile));
  return BCP_OK;
}

int bcp_reshard(bcp_plan_t* plan, const void* const* src_blobs, size_t n_src_bufs, void* const* dst_bufs,
                size_t n_dst_bufs, void* stream) {
  return execute(plan, src_blobs, n_src_bufs, dst_bufs, n_dst_bufs, static_cast<cudaStream_t>(stream));
}

int bcp_plan_device_status(bcp_plan_t* plan, void* stream) {
  if (!plan) return fail(BCP_ERR_INVALID, "plan is NULL");
  if (plan->device < 0) return BCP_OK;
  BCP_CUDA(cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
  Control c[kControls];
  BCP_CUDA(cudaMemcpy(c, plan->d_ctrl, sizeof c, cudaMemcpyDeviceToHost));
  uint32_t status = 0;
  for (const Control& k : c)
    if (!status) status = k.status;
  if (status) {
    BCP_CUDA(cudaMemset(plan->d_ctrl, 0, sizeof c));  // counters of an aborted launch are stale: start clean
    return fail(BCP_ERR_DEVICE_TIMEOUT, "a bounded wait of a staging kernel gave up (device status %d); "
                "the targets of that execution are incomplete", int(status));
  }
  return BCP_OK;
}

int bcp_plan_destroy(bcp_plan_t* plan) {
  if (!plan) return BCP_OK;
  int rc = BCP_OK;
  if (plan->device >= 0) {
    int cur = 0;
    cudaGetDevice(&cur);
    if (cur != plan->device) cudaSetDevice(plan->device);
    if (plan->ran && cudaStreamSynchronize(plan->last_stream) != cudaSuccess) {
      cudaGetLastError();
      cudaDeviceSynchronize();
    }
    if (plan->s_h2d) cudaStreamSynchronize(plan->s_h2d);
    if (plan->s_d2h) cudaStreamSynchronize(plan->s_d2h);
    if (plan->ev_switch) cudaEventDestroy(plan->ev_switch);
    for (cudaEvent_t e : plan->ev_src)
      if (e) cudaEventDestroy(e);
    for (cudaEvent_t e : plan->ev_dst)
      if (e) cudaEventDestroy(e);
    if (plan->s_h2d) cudaStreamDestroy(plan->s_h2d);
    if (plan->s_d2h) cudaStreamDestroy(plan->s_d2h);
    for (void* q : plan->stage_src) cudaFree(q);
    for (void* q : plan->stage_dst) cudaFree(q);
    cudaFree(plan->d_host_tiles);
    cudaFree(plan->d_tiles);
    cudaFree(plan->d_fan_tiles);
    cudaFree(plan->d_ptrs);
    cudaFree(plan->d_ctrl);
    cudaFree(plan->d_maps);
    if (cudaGetLastError() != cudaSuccess) rc = fail(BCP_ERR_CUDA, "bcp_plan_destroy: a CUDA call failed");
    if (cur != plan->device) cudaSetDevice(cur);
  }
  delete plan;
  return rc;
}

int bcp_pack_layout(const uint64_t* tensor_bytes, size_t n, uint64_t align, uint64_t* out_offsets, uint64_t* out_blob_bytes) {
  if ((n && (!tensor_bytes || !out_offsets)) || !out_blob_bytes) return fail(BCP_ERR_INVALID, "bcp_pack_layout: NULL argument");
  if (align < 16 || (align & (align - 1))) return fail(BCP_ERR_INVALID, "bcp_pack_layout: align must be a power of two >= 16");
  uint64_t pos = 0;
  for (size_t i = 0; i < n; ++i) {
    pos = (pos + align - 1) & ~(align - 1);
    out_offsets[i] = pos;
    pos += tensor_bytes[i];
  }
  *out_blob_bytes = (pos + align - 1) & ~(align - 1);
  return BCP_OK;
}

int bcp_pack(const void* const* tensors, const bcp_pack_meta* metas, size_t n, void* blob, uint64_t blob_bytes, void* stream) {
  if ((n && (!tensors || !metas)) || (blob_bytes && !blob)) return fail(BCP_ERR_INVALID, "bcp_pack: NULL argument");
  std::lock_guard<std::mutex> lock(g_pack_mu);
  std::vector<uint8_t> res;
  std::vector<const void*> bases;
  void* blob_base = split_addresses(tensors, n, blob, &res, &bases);
  bcp_plan_t* p = nullptr;
  if (int rc = pack_plan(false, metas, n, blob_bytes, res, &p)) return rc;
  void* dst[1] = {blob_base};
  return execute(p, bases.data(), n, dst, 1, static_cast<cudaStream_t>(stream));
}

int bcp_unpack(const void* blob, uint64_t blob_bytes, const bcp_pack_meta* metas, size_t n, void* const* tensors, void* stream) {
  if ((n && (!tensors || !metas)) || (blob_bytes && !blob)) return fail(BCP_ERR_INVALID, "bcp_unpack: NULL argument");
  std::lock_guard<std::mutex> lock(g_pack_mu);
  std::vector<uint8_t> res;
  std::vector<const void*> bases;
  const void* blob_base = split_addresses(tensors, n, const_cast<void*>(blob), &res, &bases);
  bcp_plan_t* p = nullptr;
  if (int rc = pack_plan(true, metas, n, blob_bytes, res, &p)) return rc;
  const void* src[1] = {blob_base};
  return execute(p, src, 1, const_cast<void* const*>(bases.data()), n, static_cast<cudaStream_t>(stream));
}

int bcp_pack_cache_clear(void) {
  std::lock_guard<std::mutex> lock(g_pack_mu);
  int rc = BCP_OK;
  for (PackEntry& e : g_pack_cache)
    if (int r = bcp_plan_destroy(e.plan)) rc = r;
  g_pack_cache.clear();
  return rc;
}

}  // extern "C"
