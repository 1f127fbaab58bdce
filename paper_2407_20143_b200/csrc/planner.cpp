// Host planner: metadata -> flat work list.
//
// Follows the load-time resharding workflow of the paper (arXiv 2407.20143):
//   Sec. 3.2 "Decomposing irregular tensors": an irregular (flat) shard becomes several
//            regular boxes;
//   Sec. 3.3 Step 2: every wanted shard is matched against the saved shards of the same
//            FQN; each matching segment becomes one piece of the load plan.
// Everything here is int64 arithmetic on the host; no CUDA.
#include <algorithm>
#include <atomic>
#include <chrono>
#include <cstdlib>
#include <memory>
#include <thread>
#include <cstdio>
#include <cstring>
#include <string>
#include <string_view>
#include <unordered_map>
#include <unordered_set>

#include "plan.hpp"

namespace bcp {

std::string& last_error() {
  thread_local std::string s;
  return s;
}

int fail(int code, const char* fmt, ...) {
  char buf[768];
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(buf, sizeof buf, fmt, ap);
  va_end(ap);
  last_error() = buf;
  return code;
}

int parse_options(const bcp_plan_opts* in, Options* out) {
  Options o;
  if (in) {
    if (in->tile_bytes) o.tile_bytes = in->tile_bytes;
    if (in->small_bytes) o.small_bytes = in->small_bytes;
    if (in->block_threads) o.block_threads = in->block_threads;
    if (in->ctas_per_sm) o.ctas_per_sm = in->ctas_per_sm;
    if (in->order) o.order = in->order;
    if (in->path_mask) o.path_mask = in->path_mask;
    if (in->cache_hints) o.cache_hints = in->cache_hints;
    if (in->tma_stage_bytes) o.tma_stage_bytes = in->tma_stage_bytes;
    if (in->tma_stages) o.tma_stages = in->tma_stages;
    if (in->tma_ctas_per_sm) o.tma_ctas_per_sm = in->tma_ctas_per_sm;
    if (in->unroll) o.unroll = in->unroll;
    if (in->worker) o.worker = in->worker;
    if (in->tma_min_row_bytes) o.tma_min_row_bytes = in->tma_min_row_bytes;
    o.allow_replicas = in->allow_replicas;
    if (in->tma_wait_ms) o.tma_wait_ms = in->tma_wait_ms;
    o.test_stall = in->test_stall;
    if (in->fanout) o.fanout = in->fanout;
    o.convert = in->convert;
    o.convert_src_tag = in->convert_src_tag;
    o.convert_dst_tag = in->convert_dst_tag;
  }
  if (o.tile_bytes % 4096 || o.tile_bytes < 4096 || o.tile_bytes > (64u << 20))
    return fail(BCP_ERR_INVALID, "tile_bytes must be a multiple of 4096 in [4096, 64 MiB]");
  if (o.small_bytes > o.tile_bytes) return fail(BCP_ERR_INVALID, "small_bytes must not exceed tile_bytes");
  if (o.block_threads != 256 && o.block_threads != 512 && o.block_threads != 1024)
    return fail(BCP_ERR_INVALID, "block_threads must be 256, 512 or 1024");
  if (o.ctas_per_sm > 16) return fail(BCP_ERR_INVALID, "ctas_per_sm must be in [1, 16]");
  if (o.order < 1 || o.order > 2) return fail(BCP_ERR_INVALID, "order must be 1 or 2");
  if (o.path_mask != 0 && o.path_mask != 1 && o.path_mask != 3 && o.path_mask != 7)
    return fail(BCP_ERR_INVALID, "path_mask must be 0, 1, 3 or 7");
  if (o.tma_stage_bytes && (o.tma_stage_bytes % 128 || o.tma_stage_bytes < 1024 || o.tma_stage_bytes > 65536))
    return fail(BCP_ERR_INVALID, "tma_stage_bytes must be a multiple of 128 in [1024, 65536]");
  if (o.tma_stages && (o.tma_stages < 2 || o.tma_stages > 8)) return fail(BCP_ERR_INVALID, "tma_stages must be in [2, 8]");
  if (uint64_t(o.tma_stage_bytes ? o.tma_stage_bytes : 32768) * (o.tma_stages ? o.tma_stages : 4) > 200 * 1024)
    return fail(BCP_ERR_INVALID, "tma_stage_bytes * tma_stages must not exceed 200 KiB");
  if (o.tma_ctas_per_sm > 16) return fail(BCP_ERR_INVALID, "tma_ctas_per_sm must be in [1, 16]");
  if (o.cache_hints < 1 || o.cache_hints > 4) return fail(BCP_ERR_INVALID, "cache_hints must be in [1, 4]");
  if (o.unroll != 4 && o.unroll != 8) return fail(BCP_ERR_INVALID, "unroll must be 4 or 8");
  if (o.allow_replicas > 1) return fail(BCP_ERR_INVALID, "allow_replicas must be 0 or 1");
  if (o.test_stall > 1) return fail(BCP_ERR_INVALID, "test_stall must be 0 or 1");
  if (o.fanout != 1 && o.fanout != 2) return fail(BCP_ERR_INVALID, "fanout must be 0, 1 or 2");
  if (o.tma_wait_ms > 60000) return fail(BCP_ERR_INVALID, "tma_wait_ms must not exceed 60000");
  if (o.worker > 2) return fail(BCP_ERR_INVALID, "worker must be 0, 1 or 2");
  if (o.convert > BCP_CONVERT_BF16_TO_F32) return fail(BCP_ERR_INVALID, "convert must be 0, 1 or 2");
  if (o.convert && o.convert_src_tag == o.convert_dst_tag)
    return fail(BCP_ERR_INVALID, "convert needs two different dtype tags (convert_src_tag, convert_dst_tag)");
  if (!o.convert && (o.convert_src_tag || o.convert_dst_tag))
    return fail(BCP_ERR_INVALID, "convert_src_tag / convert_dst_tag are set but convert is 0");
  if (o.tma_min_row_bytes < 16 || o.tma_min_row_bytes % 16 || o.tma_min_row_bytes > 65536)
    return fail(BCP_ERR_INVALID, "tma_min_row_bytes must be a multiple of 16 in [16, 65536]");
  *out = o;
  return BCP_OK;
}

// ------------------------------------------------------------------------------ decomposition
namespace {

int64_t volume(const int64_t* len, uint32_t from, uint32_t ndim) {
  int64_t v = 1;
  for (uint32_t k = from; k < ndim; ++k) v *= len[k];
  return v;
}

// Range [a, b) of the C-order flattening of dims d..ndim-1; dims before d are fixed in `pre`.
void decompose_rec(const int64_t* L, uint32_t ndim, uint32_t d, int64_t a, int64_t b, RelBox pre,
                   std::vector<RelBox>* out) {
  if (a >= b) return;
  if (d == ndim) {  // a single element (scalar tensor, or all dims fixed)
    out->push_back(pre);
    return;
  }
  if (d + 1 == ndim) {  // innermost dim: one run
    pre.off[d] = a;
    pre.len[d] = b - a;
    out->push_back(pre);
    return;
  }
  const int64_t inner = volume(L, d + 1, ndim);  // elements in one slab of dim d
  const int64_t i0 = a / inner, i1 = (b - 1) / inner;
  const int64_t ra = a - i0 * inner;  // where the range starts inside slab i0
  const int64_t rb = b - i1 * inner;  // where it ends inside slab i1, in (0, inner]
  auto full = [&](int64_t first, int64_t count) {
    RelBox box = pre;
    box.off[d] = first;
    box.len[d] = count;
    for (uint32_t k = d + 1; k < ndim; ++k) {
      box.off[k] = 0;
      box.len[k] = L[k];
    }
    out->push_back(box);
  };
  if (i0 == i1 && !(ra == 0 && rb == inner)) {  // inside one slab: go one dim deeper
    pre.off[d] = i0;
    pre.len[d] = 1;
    decompose_rec(L, ndim, d + 1, ra, rb, pre, out);
    return;
  }
  int64_t fs = i0, fe = i1 + 1;  // slabs [fs, fe) are complete
  if (ra != 0) {                 // partial head slab
    RelBox h = pre;
    h.off[d] = i0;
    h.len[d] = 1;
    decompose_rec(L, ndim, d + 1, ra, inner, h, out);
    fs = i0 + 1;
  }
  if (rb != inner) fe = i1;
  if (fe > fs) full(fs, fe - fs);
  if (rb != inner) {  // partial tail slab
    RelBox t = pre;
    t.off[d] = i1;
    t.len[d] = 1;
    decompose_rec(L, ndim, d + 1, 0, rb, t, out);
  }
}

}  // namespace

void decompose(const int64_t* lengths, uint32_t ndim, int64_t a, int64_t b, std::vector<RelBox>* out) {
  RelBox pre;
  for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) {
    pre.off[k] = 0;
    pre.len[k] = 1;
  }
  decompose_rec(lengths, ndim, 0, a, b, pre, out);
}

// ------------------------------------------------------------------------------ matching
namespace {

struct Entry {  // one regular box with its bytes
  int64_t off[BCP_MAX_NDIM];
  int64_t len[BCP_MAX_NDIM];
  int64_t vol;
  uint64_t byte_off;
  uint32_t buf;
  uint32_t meta;  // index of the meta it came from
};

struct Family {
  const char* fqn;
  uint32_t itemsize, dtype_tag, ndim;  // of the saved side (of the wanted side while nothing is saved)
  uint32_t d_itemsize, d_tag;          // of the wanted side (differs only under a conversion)
  uint32_t cvt;                        // BCP_CONVERT_* applied to this tensor
  bool has_src, has_dst;
  int64_t shape[BCP_MAX_NDIM];
  std::vector<Entry> src, dst;
  std::vector<uint32_t> src_metas, dst_metas;  // input entries of this tensor, expanded into src / dst when it is matched
};

const int64_t kMaxElems = int64_t(1) << 60;

int check_meta(const bcp_shard_meta& m, const char* side, size_t i, const uint64_t* buf_bytes, size_t n_bufs,
               int64_t* count) {
  if (!m.fqn) return fail(BCP_ERR_INVALID, "%s[%zu]: fqn is NULL", side, i);
  if (m.itemsize != 1 && m.itemsize != 2 && m.itemsize != 4 && m.itemsize != 8)
    return fail(BCP_ERR_INVALID, "%s[%zu] %s: itemsize %u is not 1, 2, 4 or 8", side, i, m.fqn, m.itemsize);
  if (m.ndim > BCP_MAX_NDIM) return fail(BCP_ERR_INVALID, "%s[%zu] %s: ndim %u > %d", side, i, m.fqn, m.ndim, BCP_MAX_NDIM);
  if (m.kind != BCP_BOX && m.kind != BCP_FLAT_SLICE)
    return fail(BCP_ERR_INVALID, "%s[%zu] %s: unknown kind %u", side, i, m.fqn, m.kind);
  if (m.reserved) return fail(BCP_ERR_INVALID, "%s[%zu] %s: reserved must be 0", side, i, m.fqn);
  int64_t vol = 1, gvol = 1;
  for (uint32_t k = 0; k < m.ndim; ++k) {
    const int64_t g = m.global_shape[k], o = m.offsets[k], l = m.lengths[k];
    if (g < 0 || o < 0 || l < 0 || o > g || l > g - o)
      return fail(BCP_ERR_INVALID, "%s[%zu] %s: dim %u box [%lld, +%lld) outside global extent %lld", side, i, m.fqn, k,
                  (long long)o, (long long)l, (long long)g);
    if (g > 0 && gvol > kMaxElems / g) return fail(BCP_ERR_INVALID, "%s[%zu] %s: global shape too large", side, i, m.fqn);
    gvol *= g;
    vol *= l;
  }
  int64_t n = vol;
  if (m.kind == BCP_FLAT_SLICE) {
    if (m.flat_begin < 0 || m.flat_end < m.flat_begin || m.flat_end > vol)
      return fail(BCP_ERR_INVALID, "%s[%zu] %s: flat range [%lld, %lld) outside local box of %lld elements", side, i,
                  m.fqn, (long long)m.flat_begin, (long long)m.flat_end, (long long)vol);
    n = m.flat_end - m.flat_begin;
  }
  if (m.byte_length != uint64_t(n) * m.itemsize)
    return fail(BCP_ERR_INVALID, "%s[%zu] %s: byte_length %llu != %lld elements * %u", side, i, m.fqn,
                (unsigned long long)m.byte_length, (long long)n, m.itemsize);
  if (n > 0) {
    if (m.buf_index >= n_bufs)
      return fail(BCP_ERR_BOUNDS, "%s[%zu] %s: buf_index %u >= %zu buffers", side, i, m.fqn, m.buf_index, n_bufs);
    if (m.byte_offset > buf_bytes[m.buf_index] || m.byte_length > buf_bytes[m.buf_index] - m.byte_offset)
      return fail(BCP_ERR_BOUNDS, "%s[%zu] %s: bytes [%llu, +%llu) outside buffer %u of %llu bytes", side, i, m.fqn,
                  (unsigned long long)m.byte_offset, (unsigned long long)m.byte_length, m.buf_index,
                  (unsigned long long)buf_bytes[m.buf_index]);
  }
  *count = n;
  return BCP_OK;
}

void expand(const bcp_shard_meta& m, uint32_t meta_index, int64_t count, std::vector<Entry>* out,
            std::vector<RelBox>* scratch) {
  if (count == 0) return;
  if (m.kind == BCP_BOX) {
    Entry e;
    for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) {
      e.off[k] = k < m.ndim ? m.offsets[k] : 0;
      e.len[k] = k < m.ndim ? m.lengths[k] : 1;
    }
    e.vol = count;
    e.byte_off = m.byte_offset;
    e.buf = m.buf_index;
    e.meta = meta_index;
    out->push_back(e);
    return;
  }
  std::vector<RelBox>& boxes = *scratch;
  boxes.clear();
  decompose(m.lengths, m.ndim, m.flat_begin, m.flat_end, &boxes);
  uint64_t pos = m.byte_offset;  // sub-boxes occupy consecutive byte ranges, in flat order
  for (const RelBox& b : boxes) {
    Entry e;
    for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) {
      e.off[k] = k < m.ndim ? m.offsets[k] + b.off[k] : 0;
      e.len[k] = k < m.ndim ? b.len[k] : 1;
    }
    e.vol = volume(e.len, 0, m.ndim);
    e.byte_off = pos;
    e.buf = m.buf_index;
    e.meta = meta_index;
    pos += uint64_t(e.vol) * m.itemsize;
    out->push_back(e);
  }
}

// Intersection of two boxes; false if empty.
inline bool intersect(const Entry& a, const Entry& b, uint32_t ndim, int64_t* off, int64_t* len) {
  for (uint32_t k = 0; k < ndim; ++k) {
    const int64_t lo = std::max(a.off[k], b.off[k]);
    const int64_t hi = std::min(a.off[k] + a.len[k], b.off[k] + b.len[k]);
    if (hi <= lo) return false;
    off[k] = lo;
    len[k] = hi - lo;
  }
  return true;
}

// One matched segment -> copy items.  The segment `off/len` lies inside both the saved box s
// and the wanted box d, each stored densely in C order.
void lower(const Entry& s, const Entry& d, uint32_t ndim, uint32_t s_isz, uint32_t d_isz, uint32_t cvt, const int64_t* off,
           const int64_t* len, std::vector<Item>* items) {
  // element strides of the containing boxes and byte offsets of the segment's origin
  int64_t ss[BCP_MAX_NDIM], ds[BCP_MAX_NDIM];
  int64_t sacc = 1, dacc = 1;
  for (int k = int(ndim) - 1; k >= 0; --k) {
    ss[k] = sacc;
    ds[k] = dacc;
    sacc *= s.len[k];
    dacc *= d.len[k];
  }
  uint64_t so = s.byte_off, dof = d.byte_off;
  for (uint32_t k = 0; k < ndim; ++k) {
    so += uint64_t(off[k] - s.off[k]) * uint64_t(ss[k]) * s_isz;
    dof += uint64_t(off[k] - d.off[k]) * uint64_t(ds[k]) * d_isz;
  }
  // dims of extent > 1, outer to inner, with byte strides
  struct Dim {
    uint64_t n, sp, dp;
  };
  Dim dims[BCP_MAX_NDIM + 1];
  int nd = 0;
  for (uint32_t k = 0; k < ndim; ++k)
    if (len[k] > 1) dims[nd++] = Dim{uint64_t(len[k]), uint64_t(ss[k]) * s_isz, uint64_t(ds[k]) * d_isz};
  // the innermost dim must be a dense run of elements on both sides; otherwise add a run of one element
  if (nd == 0 || dims[nd - 1].sp != s_isz || dims[nd - 1].dp != d_isz) dims[nd++] = Dim{1, s_isz, d_isz};
  // merge a dim into the run (counted in elements) while it is dense on both sides
  uint64_t run = dims[nd - 1].n;
  --nd;
  while (nd > 0 && dims[nd - 1].sp == run * s_isz && dims[nd - 1].dp == run * d_isz) {
    run *= dims[nd - 1].n;
    --nd;
  }
  // merge neighbouring outer dims that stride densely over each other
  for (int k = nd - 1; k > 0; --k) {
    if (dims[k - 1].sp == dims[k].n * dims[k].sp && dims[k - 1].dp == dims[k].n * dims[k].dp) {
      dims[k - 1].n *= dims[k].n;
      dims[k - 1].sp = dims[k].sp;
      dims[k - 1].dp = dims[k].dp;
      for (int j = k; j + 1 < nd; ++j) dims[j] = dims[j + 1];
      --nd;
    }
  }
  Item it;
  it.src_buf = s.buf;
  it.dst_buf = d.buf;
  it.row_bytes = run * d_isz;
  it.cvt = uint8_t(cvt);
  if (nd == 0) {
    it.src_off = so;
    it.dst_off = dof;
    items->push_back(it);
    return;
  }
  // the innermost remaining dim becomes the rows of a 2-D item; outer dims are enumerated
  const Dim rowdim = dims[nd - 1];
  it.rows = rowdim.n;
  it.src_pitch = rowdim.sp;
  it.dst_pitch = rowdim.dp;
  uint64_t idx[BCP_MAX_NDIM] = {0};
  const int no = nd - 1;
  for (;;) {
    uint64_t a = so, b = dof;
    for (int k = 0; k < no; ++k) {
      a += idx[k] * dims[k].sp;
      b += idx[k] * dims[k].dp;
    }
    it.src_off = a;
    it.dst_off = b;
    items->push_back(it);
    int k = no - 1;
    for (; k >= 0; --k) {
      if (++idx[k] < dims[k].n) break;
      idx[k] = 0;
    }
    if (k < 0) break;
  }
}

// Identity of a matched segment on the saved side (for the unique-bytes count): the saved box
// and the positions of the segment's first and last element in that box's C order, which fix
// the segment's box.
struct SegKey {
  uint64_t src, first, last, bytes;
  bool operator<(const SegKey& o) const {
    if (src != o.src) return src < o.src;
    return first != o.first ? first < o.first : last < o.last;
  }
  bool operator==(const SegKey& o) const { return src == o.src && first == o.first && last == o.last; }
};

}  // namespace

namespace {

// Host threads for large work lists.  The result never depends on the count.
unsigned plan_threads(size_t n_units) {
  if (n_units < 32768) return 1;
  unsigned n = 0;
  if (const char* e = getenv("BCP_PLAN_THREADS")) n = unsigned(strtoul(e, nullptr, 10));
  if (!n) n = std::min(8u, std::thread::hardware_concurrency());
  return std::max(1u, std::min(n, 64u));
}

// job(0) .. job(n_jobs - 1), handed out by a counter to the caller and up to threads - 1 helpers.
// Jobs must not throw; if helpers cannot be started the caller does all the work.
template <class F>
void parallel_jobs(size_t n_jobs, unsigned threads, F&& job) {
  std::atomic<size_t> next{0};
  auto worker = [&] {
    for (size_t j; (j = next.fetch_add(1)) < n_jobs;) job(j);
  };
  std::vector<std::thread> pool;
  if (threads > 1 && n_jobs > 1) {
    try {
      pool.reserve(threads - 1);
      for (unsigned t = 1; t < threads && t < n_jobs; ++t) pool.emplace_back(worker);
    } catch (...) {
    }
  }
  worker();
  for (std::thread& t : pool) t.join();
}

}  // namespace

int match_and_lower(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes, size_t n_src_bufs,
                    const bcp_shard_meta* dst, size_t n_dst, const uint64_t* dst_buf_bytes, size_t n_dst_bufs,
                    const Options& opt, std::vector<Item>* items, std::vector<Gap>* gaps, bcp_plan_stats_t* stats) {
  const bool allow_replicas = opt.allow_replicas != 0;
  if ((n_src && !src) || (n_dst && !dst) || (n_src_bufs && !src_buf_bytes) || (n_dst_bufs && !dst_buf_bytes))
    return fail(BCP_ERR_INVALID, "bcp_plan: NULL array with non-zero count");
  std::unordered_map<std::string_view, uint32_t> ids;  // keys point into the caller's metas
  std::vector<Family> fams;
  const char* const kDiffers = "%s[%zu] %s: itemsize, dtype_tag, ndim or global shape differs from an earlier entry";
  auto family_of = [&](const bcp_shard_meta& m, const char* side, size_t i, bool wanted, uint32_t* id) -> int {
    const std::string_view name(m.fqn);
    auto it = ids.find(name);
    if (it == ids.end()) {
      Family f;
      f.fqn = m.fqn;
      f.itemsize = f.d_itemsize = m.itemsize;
      f.dtype_tag = f.d_tag = m.dtype_tag;
      f.cvt = 0;
      f.has_src = !wanted;
      f.has_dst = wanted;
      f.ndim = m.ndim;
      for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) f.shape[k] = k < m.ndim ? m.global_shape[k] : 1;
      *id = uint32_t(fams.size());
      ids.emplace(name, *id);
      fams.push_back(std::move(f));
      return BCP_OK;
    }
    Family& f = fams[it->second];
    *id = it->second;
    bool same = f.ndim == m.ndim;
    for (uint32_t k = 0; same && k < m.ndim; ++k) same = f.shape[k] == m.global_shape[k];
    if (!same) return fail(BCP_ERR_MISMATCH, kDiffers, side, i, m.fqn);
    if (!wanted || f.has_dst) {  // later entries of a side repeat that side's dtype
      const bool ok = wanted ? (f.d_itemsize == m.itemsize && f.d_tag == m.dtype_tag) : (f.itemsize == m.itemsize && f.dtype_tag == m.dtype_tag);
      return ok ? BCP_OK : fail(BCP_ERR_MISMATCH, kDiffers, side, i, m.fqn);
    }
    // first wanted entry of a saved tensor: same dtype, or the pair the caller asked to convert
    f.has_dst = true;
    f.d_itemsize = m.itemsize;
    f.d_tag = m.dtype_tag;
    if (f.itemsize == m.itemsize && f.dtype_tag == m.dtype_tag) return BCP_OK;
    const uint32_t s_isz = opt.convert == BCP_CONVERT_F32_TO_BF16 ? 4 : 2, d_isz = 6 - s_isz;
    if (opt.convert && f.dtype_tag == opt.convert_src_tag && m.dtype_tag == opt.convert_dst_tag && f.itemsize == s_isz &&
        m.itemsize == d_isz) {
      f.cvt = opt.convert;
      return BCP_OK;
    }
    return fail(BCP_ERR_MISMATCH, kDiffers, side, i, m.fqn);
  };
  // A plan may cover a few target ranks against the saved metadata of a whole job (partial loads):
  // saved entries of tensors that no wanted entry names are validated but take no further part.
  std::unordered_set<std::string_view> wanted;
  wanted.reserve(n_dst);
  for (size_t i = 0; i < n_dst; ++i)
    if (dst[i].fqn) wanted.emplace(dst[i].fqn);
  std::vector<int64_t> src_count(n_src), dst_count(n_dst);  // elements of every input entry
  for (size_t i = 0; i < n_src; ++i) {
    uint32_t f;
    if (int rc = check_meta(src[i], "src", i, src_buf_bytes, n_src_bufs, &src_count[i])) return rc;
    if (!wanted.count(src[i].fqn)) continue;
    if (int rc = family_of(src[i], "src", i, false, &f)) return rc;
    fams[f].src_metas.push_back(uint32_t(i));
  }
  // target byte ranges must not overlap inside a buffer
  {
    struct Range {
      uint64_t lo, hi;
      uint32_t buf, meta;
    };
    std::vector<Range> rs;
    rs.reserve(n_dst);
    for (size_t i = 0; i < n_dst; ++i) {
      uint32_t f;
      if (int rc = check_meta(dst[i], "dst", i, dst_buf_bytes, n_dst_bufs, &dst_count[i])) return rc;
      if (int rc = family_of(dst[i], "dst", i, true, &f)) return rc;
      fams[f].dst_metas.push_back(uint32_t(i));
      const int64_t n = dst_count[i];
      if (n > 0) rs.push_back(Range{dst[i].byte_offset, dst[i].byte_offset + dst[i].byte_length, dst[i].buf_index, uint32_t(i)});
    }
    std::sort(rs.begin(), rs.end(), [](const Range& a, const Range& b) { return a.buf != b.buf ? a.buf < b.buf : a.lo < b.lo; });
    for (size_t i = 1; i < rs.size(); ++i)
      if (rs[i].buf == rs[i - 1].buf && rs[i].lo < rs[i - 1].hi)
        return fail(BCP_ERR_DST_ALIAS, "dst[%u] %s and dst[%u] %s write overlapping bytes of buffer %u", rs[i - 1].meta,
                    dst[rs[i - 1].meta].fqn, rs[i].meta, dst[rs[i].meta].fqn, rs[i].buf);
    if (gaps) {  // what no entry names: between the sorted ranges, and whole buffers without entries
      size_t i = 0;
      for (uint32_t b = 0; b < n_dst_bufs; ++b) {
        uint64_t pos = 0;
        for (; i < rs.size() && rs[i].buf == b; ++i) {
          if (rs[i].lo > pos) gaps->push_back(Gap{pos, rs[i].lo - pos, b, 0});
          pos = rs[i].hi;
        }
        if (dst_buf_bytes[b] > pos) gaps->push_back(Gap{pos, dst_buf_bytes[b] - pos, b, 0});
      }
    }
  }
  struct Scratch {
    std::vector<SegKey> segs;    // matched segments of the family at hand
    std::vector<int64_t> reach;  // reach[i] = largest end (along dim 0) among the family's saved boxes 0..i
    std::vector<RelBox> boxes;   // decomposition of one flat slice
    uint64_t n_se = 0, n_de = 0; // boxes after decomposition
  };
  // One tensor: check its saved boxes, match every wanted box, lower the matches.  Families are
  // independent, so large jobs hand blocks of them to several threads.
  auto match_family = [&](Family& f, Scratch& sc, std::vector<Item>* items, uint64_t* n_inter_out, uint64_t* uniq_out) -> int {
    std::vector<SegKey>& segs = sc.segs;
    std::vector<int64_t>& reach = sc.reach;
    uint64_t n_inter = 0, uniq = 0;
    const uint32_t nd = f.ndim;
    for (uint32_t i : f.src_metas) expand(src[i], i, src_count[i], &f.src, &sc.boxes);
    for (uint32_t i : f.dst_metas) expand(dst[i], i, dst_count[i], &f.dst, &sc.boxes);
    sc.n_se += f.src.size();
    sc.n_de += f.dst.size();
    if (allow_replicas && f.src.size() > 1) {
      // identical boxes are replicas of one shard: keep the one that came first in the input
      std::sort(f.src.begin(), f.src.end(), [nd](const Entry& a, const Entry& b) {
        for (uint32_t k = 0; k < nd; ++k) {
          if (a.off[k] != b.off[k]) return a.off[k] < b.off[k];
          if (a.len[k] != b.len[k]) return a.len[k] < b.len[k];
        }
        return a.meta < b.meta;
      });
      size_t kept = 0;
      for (size_t i = 0; i < f.src.size(); ++i) {
        bool same = kept > 0;
        for (uint32_t k = 0; same && k < nd; ++k)
          same = f.src[i].off[k] == f.src[kept - 1].off[k] && f.src[i].len[k] == f.src[kept - 1].len[k];
        if (!same) f.src[kept++] = f.src[i];
      }
      f.src.resize(kept);
    }
    // saved boxes of one tensor must be pairwise disjoint (each element is stored once)
    std::sort(f.src.begin(), f.src.end(), [](const Entry& a, const Entry& b) { return a.off[0] < b.off[0]; });
    for (size_t i = 0; i < f.src.size(); ++i) {
      const int64_t end0 = f.src[i].off[0] + f.src[i].len[0];
      for (size_t j = i + 1; j < f.src.size() && f.src[j].off[0] < end0; ++j) {
        int64_t o[BCP_MAX_NDIM], l[BCP_MAX_NDIM];
        if (intersect(f.src[i], f.src[j], nd, o, l))
          return fail(BCP_ERR_OVERLAP, "%s: saved entries src[%u] and src[%u] hold the same element", f.fqn, f.src[i].meta,
                      f.src[j].meta);
      }
    }
    if (f.cvt) {  // a converting unit reads and writes whole elements at their natural alignment
      for (const Entry& e : f.src)
        if (e.byte_off % f.itemsize)
          return fail(BCP_ERR_INVALID, "%s: src[%u] is converted, so its byte_offset must be a multiple of %u", f.fqn, e.meta, f.itemsize);
      for (const Entry& e : f.dst)
        if (e.byte_off % f.d_itemsize)
          return fail(BCP_ERR_INVALID, "%s: dst[%u] is converted, so its byte_offset must be a multiple of %u", f.fqn, e.meta, f.d_itemsize);
    }
    reach.resize(f.src.size());
    for (size_t i = 0; i < f.src.size(); ++i)
      reach[i] = std::max(i ? reach[i - 1] : INT64_MIN, f.src[i].off[0] + f.src[i].len[0]);
    segs.clear();
    for (const Entry& d : f.dst) {
      int64_t covered = 0;
      const int64_t dend0 = d.off[0] + d.len[0];
      // boxes before `first` all end at or before the wanted box's first row
      const uint32_t first = uint32_t(std::upper_bound(reach.begin(), reach.end(), d.off[0]) - reach.begin());
      for (uint32_t si = first; si < f.src.size(); ++si) {
        const Entry& s = f.src[si];
        if (s.off[0] >= dend0) break;  // sorted by first offset
        int64_t o[BCP_MAX_NDIM], l[BCP_MAX_NDIM];
        if (!intersect(s, d, nd, o, l)) continue;
        covered += volume(l, 0, nd);
        ++n_inter;
        lower(s, d, nd, f.itemsize, f.d_itemsize, f.cvt, o, l, items);
        SegKey key = {si, 0, 0, uint64_t(volume(l, 0, nd)) * f.itemsize};
        for (uint32_t k = 0; k < nd; ++k) {
          key.first = key.first * uint64_t(s.len[k]) + uint64_t(o[k] - s.off[k]);
          key.last = key.last * uint64_t(s.len[k]) + uint64_t(o[k] + l[k] - 1 - s.off[k]);
        }
        segs.push_back(key);
      }
      if (covered != d.vol)
        return fail(BCP_ERR_UNCOVERED, "%s: dst[%u] wants %lld elements, saved entries hold %lld of them", f.fqn, d.meta,
                    (long long)d.vol, (long long)covered);
    }
    // distinct source bytes: a segment wanted by several target entries (replicas) counts once
    std::sort(segs.begin(), segs.end());
    segs.erase(std::unique(segs.begin(), segs.end()), segs.end());
    for (const SegKey& k : segs) uniq += k.bytes;
    *n_inter_out += n_inter;
    *uniq_out += uniq;
    return BCP_OK;
  };
  uint64_t n_inter = 0, uniq = 0, n_se = 0, n_de = 0;
  const unsigned threads = plan_threads(n_src + n_dst);
  if (threads == 1) {
    Scratch sc;
    for (Family& f : fams)
      if (int rc = match_family(f, sc, items, &n_inter, &uniq)) return rc;
    n_se = sc.n_se, n_de = sc.n_de;
  } else {
    // blocks of consecutive families with about the same number of entries; a block stops at its
    // first error, and the error of the earliest family wins, as in the serial order
    struct Block {
      size_t begin, end;
      std::vector<Item> items;
      uint64_t n_inter = 0, uniq = 0, n_se = 0, n_de = 0;
      int rc = BCP_OK;
      std::string err;
    };
    std::vector<Block> blocks;
    const uint64_t per_block = uint64_t(n_src + n_dst) / (uint64_t(threads) * 8) + 1;
    uint64_t acc = 0;
    size_t begin = 0;
    for (size_t fi = 0; fi < fams.size(); ++fi) {
      acc += fams[fi].src_metas.size() + fams[fi].dst_metas.size();
      if (acc >= per_block || fi + 1 == fams.size()) {
        Block b;
        b.begin = begin, b.end = fi + 1;
        blocks.push_back(std::move(b));
        begin = fi + 1, acc = 0;
      }
    }
    parallel_jobs(blocks.size(), threads, [&](size_t j) {
      Block& b = blocks[j];
      try {
        Scratch sc;
        for (size_t fi = b.begin; fi < b.end && b.rc == BCP_OK; ++fi) {
          b.rc = match_family(fams[fi], sc, &b.items, &b.n_inter, &b.uniq);
          if (b.rc) b.err = last_error();  // the message lives in this thread
        }
        b.n_se = sc.n_se, b.n_de = sc.n_de;
      } catch (const std::bad_alloc&) {
        b.rc = BCP_ERR_NOMEM, b.err = "out of host memory";
      }
    });
    for (const Block& b : blocks)  // blocks are in family order
      if (b.rc) {
        last_error() = b.err;
        return b.rc;
      }
    size_t total = items->size();
    for (const Block& b : blocks) total += b.items.size();
    items->reserve(total);
    for (Block& b : blocks) {
      items->insert(items->end(), b.items.begin(), b.items.end());
      n_inter += b.n_inter;
      uniq += b.uniq;
      n_se += b.n_se;
      n_de += b.n_de;
    }
  }
  stats->n_src_entries = n_se;
  stats->n_dst_entries = n_de;
  stats->n_fqns = fams.size();
  stats->n_intersections = n_inter;
  stats->bytes_src_unique = uniq;
  return BCP_OK;
}

// ------------------------------------------------------------------------------ work units
namespace {

inline uint32_t gran_log2(uint64_t bits) {
  uint32_t g = 0;
  while (g < 4 && !((bits >> g) & 1)) ++g;
  return g;  // 0..4 -> 1..16 bytes
}

enum { kTma = 0, kBig = 1, kSmall = 2, kCvt = 3, kClasses = 4 };  // unit classes, in the order of the final list

struct Tally {
  uint64_t bytes_copied = 0, bytes_misaligned = 0, n_strided = 0;
  uint64_t tma_bytes = 0;   // payload of the TMA class ...
  uint64_t tma_busy = 0;    // ... in shifted runs and rectangles with rows under 2 KiB (the warp issues a lot)
  uint64_t tma_boxed = 0;   // ... in tensor-map boxes
  uint64_t cvt_bytes = 0;   // target bytes written by converting units
  void add(const Tally& o) {
    bytes_copied += o.bytes_copied, bytes_misaligned += o.bytes_misaligned, n_strided += o.n_strided;
    tma_bytes += o.tma_bytes, tma_busy += o.tma_busy, tma_boxed += o.tma_boxed, cvt_bytes += o.cvt_bytes;
  }
};

// Cuts items into units.  Used twice: a counting pass (out[] null) that sizes the arrays, then
// a writing pass in which every block of items starts at its own, precomputed positions.
struct Cutter {
  const Options& opt;
  const std::vector<uint64_t>* src_bytes;  // source buffer sizes (may be null: unknown)
  bool demote;                             // small job: TMA-eligible units go to the register kernel
  bcp_tile* out[kClasses];
  Rect* rects_out;
  size_t pos[kClasses];
  size_t rect_pos;
  Tally st;

  void put(int cls, const bcp_tile& t) {
    if (out[cls]) out[cls][pos[cls]] = t;
    ++pos[cls];
  }

  void emit(const Item& it, uint64_t src_off, uint64_t dst_off, uint64_t rows, uint64_t row_bytes) {
    bcp_tile t;
    memset(&t, 0, sizeof t);
    t.src_off = it.zero ? 0 : src_off;
    t.dst_off = dst_off;
    t.rows = uint32_t(rows);
    t.row_bytes = uint32_t(row_bytes);
    t.src_buf = it.src_buf;
    t.dst_buf = it.dst_buf;
    if (rows > 1) {
      t.src_pitch = it.src_pitch;
      t.dst_pitch = it.dst_pitch;
    }
    uint64_t bits = t.dst_off | t.row_bytes | t.dst_pitch;
    if (!it.zero) bits |= t.src_off | t.src_pitch;
    const uint32_t g = gran_log2(bits);
    t.flags = g;
    if (it.zero) t.flags |= BCP_TILE_ZERO;
    const uint64_t payload = rows * row_bytes;
    if (g < 4) st.bytes_misaligned += payload;
    if (rows > 1) ++st.n_strided;
    st.bytes_copied += payload;
    if (payload < opt.small_bytes) {
      t.flags |= BCP_TILE_SMALL;
      put(kSmall, t);
      return;
    }
    // TMA staging: whole 16-byte units between 16-byte aligned addresses (runs and rectangles),
    // or a run / rectangle of any alignment whose 16-byte aligned supersets stay inside the source buffer
    bool eligible = !it.zero && opt.path_mask != 1 && row_bytes >= opt.tma_min_row_bytes;
    if (eligible && g < 4) {  // the superset of the last row must not reach past the source buffer
      const uint64_t end16 = (src_off + (rows - 1) * (rows > 1 ? it.src_pitch : 0) + row_bytes + 15) & ~uint64_t(15);
      eligible = src_bytes && it.src_buf < src_bytes->size() && end16 <= (*src_bytes)[it.src_buf];
    }
    if (eligible) {
      st.tma_bytes += payload;
      if (g < 4 || (rows > 1 && row_bytes < 2048)) st.tma_busy += payload;
      if (!demote) {
        t.flags |= BCP_TILE_TMA;
        put(kTma, t);
        return;
      }
    }
    put(kBig, t);
  }

  // contiguous run: peel a ragged head / tail when source and target are co-aligned, then
  // cut the body so that later units start on a 256-byte boundary of the target
  void cut_run(const Item& it, uint64_t so, uint64_t dof, uint64_t n) {
    if (n == 0) return;
    const bool co = it.zero || ((so ^ dof) & 15) == 0;
    if (co && n >= 32) {
      const uint64_t head = (16 - (dof & 15)) & 15;
      if (head) {
        emit(it, so, dof, 1, head);
        so += head, dof += head, n -= head;
      }
      const uint64_t tail = n & 15;
      if (tail) {
        emit(it, so + n - tail, dof + n - tail, 1, tail);
        n -= tail;
      }
    }
    uint64_t first = opt.tile_bytes;
    if (n > opt.tile_bytes && (dof & 255)) first = opt.tile_bytes - (dof & 255);
    while (n) {
      const uint64_t c = std::min<uint64_t>(n, first);
      emit(it, so, dof, 1, c);
      so += c, dof += c, n -= c;
      first = opt.tile_bytes;
    }
  }

  // Rectangle with short rows -> units made of whole boxes of a 2-D tensor map (8-byte elements,
  // one box = all of a row x box_rows rows, at most 16 KiB).  Returns false if it does not qualify.
  bool cut_rect(const Item& it) {
    if ((opt.path_mask != 7 && opt.path_mask != 0) || it.zero || it.row_bytes < 16 || it.row_bytes > 2048 || it.rows >= (uint64_t(1) << 31)) return false;
    if ((it.src_off | it.dst_off | it.row_bytes | it.src_pitch | it.dst_pitch) & 15) return false;
    if (it.src_pitch >= (uint64_t(1) << 40) || it.dst_pitch >= (uint64_t(1) << 40)) return false;
    if (it.rows * it.row_bytes < 32768) return false;  // not worth two descriptors
    uint64_t cap = std::min<uint64_t>(16384, opt.tile_bytes);
    if (opt.tma_stage_bytes) cap = std::min<uint64_t>(cap, opt.tma_stage_bytes);
    const uint64_t box_rows = std::min<uint64_t>(256, cap / it.row_bytes);
    if (box_rows == 0) return false;
    const uint64_t rpt = std::max<uint64_t>(box_rows, opt.tile_bytes / it.row_bytes / box_rows * box_rows);
    if (!demote) {
      if (rects_out) {
        Rect& rc = rects_out[rect_pos];
        rc.src_off = it.src_off, rc.dst_off = it.dst_off, rc.src_pitch = it.src_pitch, rc.dst_pitch = it.dst_pitch;
        rc.rows = it.rows, rc.row_bytes = uint32_t(it.row_bytes), rc.src_buf = it.src_buf, rc.dst_buf = it.dst_buf;
        rc.box_rows = uint32_t(box_rows);
      }
      ++rect_pos;
    }
    for (uint64_t r = 0; r < it.rows; r += rpt) {
      const uint64_t nr = std::min(rpt, it.rows - r);
      bcp_tile t;
      memset(&t, 0, sizeof t);
      t.src_off = it.src_off + r * it.src_pitch;
      t.dst_off = it.dst_off + r * it.dst_pitch;
      t.src_pitch = it.src_pitch, t.dst_pitch = it.dst_pitch;
      t.rows = uint32_t(nr), t.row_bytes = uint32_t(it.row_bytes);
      t.src_buf = it.src_buf, t.dst_buf = it.dst_buf;
      t.flags = 4u;
      ++st.n_strided;
      st.bytes_copied += nr * it.row_bytes;
      st.tma_bytes += nr * it.row_bytes;
      st.tma_boxed += nr * it.row_bytes;
      if (demote) {
        put(kBig, t);
        continue;
      }
      t.flags |= BCP_TILE_TMA | BCP_TILE_TMA2D;
      t.reserved[0] = uint32_t(rect_pos);  // index + 1
      t.reserved[1] = uint32_t(r);
      t.reserved[2] = uint32_t(box_rows);
      put(kTma, t);
    }
    return true;
  }

  // Converting units: rows x row_bytes TARGET bytes each; no staging path, no warp path.
  void emit_cvt(const Item& it, uint64_t src_off, uint64_t dst_off, uint64_t rows, uint64_t row_bytes) {
    bcp_tile t;
    memset(&t, 0, sizeof t);
    t.src_off = src_off;
    t.dst_off = dst_off;
    t.rows = uint32_t(rows);
    t.row_bytes = uint32_t(row_bytes);
    t.src_buf = it.src_buf;
    t.dst_buf = it.dst_buf;
    if (rows > 1) {
      t.src_pitch = it.src_pitch;
      t.dst_pitch = it.dst_pitch;
      ++st.n_strided;
    }
    const uint32_t g = gran_log2(t.src_off | t.dst_off | t.row_bytes | t.src_pitch | t.dst_pitch);
    t.flags = g | (uint32_t(it.cvt) << BCP_TILE_CVT_SHIFT);
    if (g < 4) st.bytes_misaligned += rows * row_bytes;
    st.bytes_copied += rows * row_bytes;
    st.cvt_bytes += rows * row_bytes;
    put(kCvt, t);
  }

  void cut_cvt(const Item& it) {
    const uint64_t unit = opt.tile_bytes;
    auto src_bytes_of = [&](uint64_t dst_bytes) { return it.cvt == BCP_CONVERT_F32_TO_BF16 ? dst_bytes * 2 : dst_bytes / 2; };
    if (it.rows > 1 && it.row_bytes < unit) {  // groups of whole rows
      const uint64_t rpt = std::max<uint64_t>(1, unit / it.row_bytes);
      for (uint64_t r = 0; r < it.rows; r += rpt)
        emit_cvt(it, it.src_off + r * it.src_pitch, it.dst_off + r * it.dst_pitch, std::min(rpt, it.rows - r), it.row_bytes);
      return;
    }
    for (uint64_t r = 0; r < it.rows; ++r) {  // every row is a run, cut so that later units start 256-byte aligned
      uint64_t so = it.src_off + r * it.src_pitch, dof = it.dst_off + r * it.dst_pitch, n = it.row_bytes;
      uint64_t first = unit;
      if (n > unit && (dof & 255)) first = unit - (dof & 255);
      while (n) {
        const uint64_t c = std::min(n, first);
        emit_cvt(it, so, dof, 1, c);
        so += src_bytes_of(c), dof += c, n -= c;
        first = unit;
      }
    }
  }

  void cut(const Item& it) {
    if (it.cvt) {
      cut_cvt(it);
      return;
    }
    if (it.rows <= 1 || it.row_bytes == 0) {
      cut_run(it, it.src_off, it.dst_off, it.rows ? it.row_bytes : 0);
      return;
    }
    if (cut_rect(it)) return;
    if (it.row_bytes >= opt.tile_bytes) {  // long rows: each row is a run of its own
      for (uint64_t r = 0; r < it.rows; ++r) cut_run(it, it.src_off + r * it.src_pitch, it.dst_off + r * it.dst_pitch, it.row_bytes);
      return;
    }
    const uint64_t rpt = std::max<uint64_t>(1, opt.tile_bytes / it.row_bytes);
    for (uint64_t r = 0; r < it.rows; r += rpt) {
      const uint64_t nr = std::min(rpt, it.rows - r);
      emit(it, it.src_off + r * it.src_pitch, it.dst_off + r * it.dst_pitch, nr, it.row_bytes);
    }
  }
};

}  // namespace

// Read once, write many: TMA units that read exactly the same source bytes (the replicas of a
// target shard) sit next to each other in a list ordered by source address.  All but the first
// of such a group (up to 8 members) are marked as followers and the first one records how many
// follow; the kernel stages the source once and stores it to every member's target.
void mark_followers(bcp_tile* tma, size_t n) {
  size_t head = 0;
  for (size_t i = 1; i < n; ++i) {
    const bcp_tile& a = tma[i - 1];
    bcp_tile& b = tma[i];
    const uint32_t plain = ~(BCP_TILE_FOLLOW | (7u << BCP_TILE_FAN_SHIFT));
    // (equal flags include the access width, so one copy-out width suits every member's target)
    const bool same = a.src_buf == b.src_buf && a.src_off == b.src_off && a.rows == b.rows && a.row_bytes == b.row_bytes &&
                      a.src_pitch == b.src_pitch && (a.flags & plain) == (b.flags & plain) && (b.flags & BCP_TILE_TMA) &&
                      (!(b.flags & BCP_TILE_TMA2D) || a.reserved[2] == b.reserved[2]);
    if (same && i - head < 8) {
      b.flags |= BCP_TILE_FOLLOW;
      tma[head].flags = (tma[head].flags & ~(7u << BCP_TILE_FAN_SHIFT)) | (uint32_t(i - head) << BCP_TILE_FAN_SHIFT);
    } else {
      head = i;
    }
  }
}

namespace {

// Sort key of a unit: (a_buf, a_off) is the side the list is ordered by, (b_buf, b_off) breaks
// ties between units that read the same source bytes (replicas); idx = position before sorting.
struct Key {
  uint64_t a_off, b_off;
  uint32_t a_buf, b_buf, idx, pad;
};
inline bool key_less(const Key& x, const Key& y) {
  if (x.a_buf != y.a_buf) return x.a_buf < y.a_buf;
  if (x.a_off != y.a_off) return x.a_off < y.a_off;
  return x.b_buf != y.b_buf ? x.b_buf < y.b_buf : x.b_off < y.b_off;
}

// Merge sort over `threads` chunks; returns whichever of the two arrays holds the result.
// Every merge of two runs is itself split into parts (cut one run evenly, find the matching
// cut of the other by binary search), so that all rounds keep every thread busy.
template <class T, class Less>
T* parallel_sort(T* k, T* tmp, size_t n, unsigned threads, Less less) {
  const size_t chunks = std::max<size_t>(1, std::min<size_t>(threads, n / 8192));
  auto bound = [&](size_t i) { return n * std::min(i, chunks) / chunks; };
  parallel_jobs(chunks, threads, [&](size_t c) { std::sort(k + bound(c), k + bound(c + 1), less); });
  T *from = k, *to = tmp;
  for (size_t w = 1; w < chunks; w *= 2) {
    const size_t pairs = (chunks + 2 * w - 1) / (2 * w);
    const size_t parts = std::max<size_t>(1, (threads + pairs - 1) / pairs);
    parallel_jobs(pairs * parts, threads, [&](size_t job) {
      const size_t j = job / parts, part = job % parts;
      const size_t lo = bound(2 * j * w), mid = bound(2 * j * w + w), hi = bound(2 * j * w + 2 * w);
      const T *a = from + lo, *b = from + mid;
      const size_t na = mid - lo, nb = hi - mid;
      auto cut_b = [&](size_t ia) { return ia >= na ? nb : size_t(std::lower_bound(b, b + nb, a[ia], less) - b); };
      const size_t a0 = na * part / parts, a1 = na * (part + 1) / parts;
      const size_t b0 = part == 0 ? 0 : cut_b(a0), b1 = part + 1 == parts ? nb : cut_b(a1);
      std::merge(a + a0, a + a1, b + b0, b + b1, to + lo + a0 + b0, less);
    });
    std::swap(from, to);
  }
  return from;
}

}  // namespace

void build_tiles(std::vector<Item>& items, Options& opt, const std::vector<uint64_t>* src_bytes, TileVec* tiles,
                 size_t* n_tma, size_t* n_big, size_t* n_cvt, std::vector<Rect>* rects, bcp_plan_stats_t* stats) {
  // coalesce runs that are adjacent on both sides (e.g. the sub-boxes of one flat slice)
  auto by_target = [](const Item& a, const Item& b) { return a.dst_buf != b.dst_buf ? a.dst_buf < b.dst_buf : a.dst_off < b.dst_off; };
  const Item* sorted_items = items.data();
  std::vector<Item> item_tmp;
  if (const unsigned st = plan_threads(items.size()); st > 1) {
    item_tmp.resize(items.size());
    sorted_items = parallel_sort(items.data(), item_tmp.data(), items.size(), st, by_target);
  } else {
    std::sort(items.begin(), items.end(), by_target);
  }
  std::vector<Item> merged;
  merged.reserve(items.size());
  for (size_t ii = 0; ii < items.size(); ++ii) {
    const Item& it = sorted_items[ii];
    if (it.rows * it.row_bytes == 0) continue;
    if (!merged.empty()) {
      Item& p = merged.back();
      if (p.rows == 1 && it.rows == 1 && p.zero == it.zero && p.cvt == it.cvt && p.dst_buf == it.dst_buf &&
          p.dst_off + p.row_bytes == it.dst_off &&
          (it.zero || (p.src_buf == it.src_buf && p.src_off + p.src_row_bytes() == it.src_off))) {
        p.row_bytes += it.row_bytes;
        continue;
      }
    }
    merged.push_back(it);
  }
  const size_t n_items = merged.size();
  stats->n_items = n_items;

  // Pass 1: how many units of each class (and rectangles) every item gives.  A rough unit count
  // decides whether helpers are worth starting.
  uint64_t rough = 0;
  for (const Item& it : merged) rough += it.rows * it.row_bytes / opt.tile_bytes + (it.row_bytes >= opt.tile_bytes ? it.rows : 1);
  const unsigned threads = plan_threads(size_t(std::min<uint64_t>(rough, SIZE_MAX)));
  struct Count {
    size_t n[kClasses], rects;
  };
  std::vector<Count> cnt(n_items + 1);
  const size_t kBlock = 16;
  std::vector<Tally> tally((n_items + kBlock - 1) / kBlock);
  parallel_jobs(tally.size(), threads, [&](size_t j) {
    Cutter c{opt, src_bytes, false, {nullptr, nullptr, nullptr, nullptr}, nullptr, {0, 0, 0, 0}, 0, Tally()};
    for (size_t i = j * kBlock; i < std::min(n_items, (j + 1) * kBlock); ++i) {
      const Count before = {{c.pos[0], c.pos[1], c.pos[2], c.pos[3]}, c.rect_pos};
      c.cut(merged[i]);
      cnt[i] = {{c.pos[0] - before.n[0], c.pos[1] - before.n[1], c.pos[2] - before.n[2], c.pos[3] - before.n[3]},
                c.rect_pos - before.rects};
    }
    tally[j] = c.st;
  });
  Tally all;
  for (const Tally& t : tally) all.add(t);
  // small jobs are launch-bound: keep them in one kernel
  const bool demote = opt.path_mask == 0 && all.tma_bytes < (128u << 20);
  if (demote) {
    for (size_t i = 0; i < n_items; ++i) cnt[i].n[kBig] += cnt[i].n[kTma], cnt[i].n[kTma] = 0, cnt[i].rects = 0;
    all.tma_bytes = all.tma_busy = all.tma_boxed = 0;
  }
  Count run = {{0, 0, 0, 0}, 0};  // counts -> positions of each item's first unit inside its class
  for (size_t i = 0; i <= n_items; ++i) {
    const Count c = i < n_items ? cnt[i] : Count{{0, 0, 0, 0}, 0};
    cnt[i] = run;
    for (int k = 0; k < kClasses; ++k) run.n[k] += c.n[k];
    run.rects += c.rects;
  }
  const size_t total = run.n[0] + run.n[1] + run.n[2] + run.n[3];

  // Pass 2: write the units, blocks of items of about equal size in parallel
  std::unique_ptr<bcp_tile[]> raw(new bcp_tile[total ? total : 1]);
  bcp_tile* const cls[kClasses] = {raw.get(), raw.get() + run.n[0], raw.get() + run.n[0] + run.n[1],
                                   raw.get() + run.n[0] + run.n[1] + run.n[2]};
  std::vector<Rect> rc(run.rects);
  std::vector<size_t> cuts(1, 0);  // item index where each block starts
  {
    auto units_before = [&](size_t i) { return cnt[i].n[0] + cnt[i].n[1] + cnt[i].n[2] + cnt[i].n[3]; };
    const size_t per_block = std::max<size_t>(4096, total / (size_t(threads) * 8) + 1);
    for (size_t i = 1; i < n_items; ++i)
      if (units_before(i) - units_before(cuts.back()) >= per_block) cuts.push_back(i);
    cuts.push_back(n_items);
  }
  parallel_jobs(cuts.size() - 1, threads, [&](size_t j) {
    const Count& at = cnt[cuts[j]];
    Cutter c{opt, src_bytes, demote, {cls[0], cls[1], cls[2], cls[3]}, rc.data(), {at.n[0], at.n[1], at.n[2], at.n[3]}, at.rects, Tally()};
    for (size_t i = cuts[j]; i < cuts[j + 1]; ++i) c.cut(merged[i]);
  });
  stats->bytes_copied = all.bytes_copied;
  stats->bytes_misaligned = all.bytes_misaligned;
  stats->n_strided_tiles = all.n_strided;
  stats->n_tma_tiles = run.n[kTma];

  // Stage geometry of the TMA kernel when the caller left it open.  Long aligned runs only need
  // a few copy commands per stage, so two CTAs with 32 KiB stages per SM are enough; shifted
  // runs (copied out of shared memory by the warp itself) and rectangles with rows under 2 KiB
  // (one copy command per row) are limited by what one warp can issue and want four CTAs with
  // 16 KiB stages.  Both fill 192 KiB of shared memory per SM.
  {
    const uint64_t busy = all.tma_busy, boxed = all.tma_boxed, sum = all.tma_bytes;
    const bool many_busy = busy * 8 >= sum && sum > 0;
    const bool many_boxed = !many_busy && boxed * 8 >= sum && sum > 0;  // boxes are at most 16 KiB: deeper ring
    if (!opt.tma_stage_bytes) opt.tma_stage_bytes = (many_busy || many_boxed) ? 16384 : 32768;
    if (!opt.tma_ctas_per_sm) opt.tma_ctas_per_sm = many_busy ? 4 : 2;
    if (!opt.tma_stages) opt.tma_stages = many_boxed ? 4 : 3;
  }
  // Register kernel: a CTA per unit for small jobs (fewer, fatter workers start faster); every
  // warp its own worker once the kernel has a lot to move (no barriers, deeper overlap).
  if (!opt.worker) {
    opt.worker = all.bytes_copied - all.tma_bytes - all.cvt_bytes >= (128u << 20) ? 2 : 1;
    if (opt.worker == 2 && !opt.ctas_per_sm) opt.ctas_per_sm = 4;
  }
  if (!opt.ctas_per_sm) opt.ctas_per_sm = 2;

  // Order every class by source address (order 1: the reads of replicas meet in L2) or by target
  // address, through compact keys, and gather the units into the final list.
  std::unique_ptr<Key[]> keys(new Key[total ? total : 1]), spare(new Key[total ? total : 1]);
  const bool by_src = opt.order == 1;
  const size_t kChunk = 65536;
  parallel_jobs((total + kChunk - 1) / kChunk, threads, [&](size_t j) {
    for (size_t i = j * kChunk; i < std::min(total, (j + 1) * kChunk); ++i) {
      const bcp_tile& t = raw[i];
      const int k = i < run.n[0] ? 0 : i < run.n[0] + run.n[1] ? 1 : i < run.n[0] + run.n[1] + run.n[2] ? 2 : 3;
      const uint32_t idx = uint32_t(i - (cls[k] - raw.get()));
      keys[i] = by_src ? Key{t.src_off, t.dst_off, t.src_buf, t.dst_buf, idx, 0} : Key{t.dst_off, 0, t.dst_buf, 0, idx, 0};
    }
  });
  tiles->clear();
  tiles->resize(total);
  size_t base = 0;
  for (int k = 0; k < kClasses; ++k) {
    const size_t n = run.n[k];
    const Key* sorted = parallel_sort(keys.get() + base, spare.get() + base, n, threads, key_less);
    bcp_tile* dst = tiles->data() + base;
    const bcp_tile* src = cls[k];
    parallel_jobs((n + kChunk - 1) / kChunk, threads, [&](size_t j) {
      for (size_t i = j * kChunk; i < std::min(n, (j + 1) * kChunk); ++i) dst[i] = src[sorted[i].idx];
    });
    base += n;
  }
  if (opt.order == 1 && opt.fanout == 1) mark_followers(tiles->data(), run.n[kTma]);
  stats->n_tiles = run.n[kTma] + run.n[kBig];
  stats->n_small_tiles = run.n[kSmall];
  *n_tma = run.n[kTma];
  *n_big = run.n[kBig];
  *n_cvt = run.n[kCvt];
  stats->n_cvt_tiles = run.n[kCvt];
  if (rects) *rects = std::move(rc);
}

}  // namespace bcp
