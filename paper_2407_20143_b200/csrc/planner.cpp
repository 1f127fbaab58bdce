// Host planner, first half: metadata -> copy items (validation, decomposition, matching,
// lowering).  The second half (items -> flat work list) is units.cpp.
//
// Follows the load-time resharding workflow of the paper (arXiv 2407.20143):
//   Sec. 3.2 "Decomposing irregular tensors": an irregular (flat) shard becomes several
//            regular boxes;
//   Sec. 3.3 Step 2: every wanted shard is matched against the saved shards of the same
//            FQN; each matching segment becomes one piece of the load plan.
// Everything here is int64 arithmetic on the host; no CUDA.
#include <algorithm>
#include <cstdio>
#include <cstring>
#include <string>
#include <string_view>
#include <unordered_map>
#include <unordered_set>

#include "host_threads.hpp"
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
    if (in->tile_bytes) o.tile_bytes = o.run_tile_bytes = in->tile_bytes;
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
    o.src_buf_first = in->src_buf_first;
    o.src_buf_count = in->src_buf_count;
  }
  if (o.tile_bytes % 4096 || o.tile_bytes < 4096 || o.tile_bytes > (64u << 20))
    return fail(BCP_ERR_INVALID, "tile_bytes must be a multiple of 4096 in [4096, 64 MiB]");
  if (o.small_bytes > o.tile_bytes) return fail(BCP_ERR_INVALID, "small_bytes must not exceed tile_bytes");
  if (o.block_threads != 256 && o.block_threads != 512 && o.block_threads != 1024)
    return fail(BCP_ERR_INVALID, "block_threads must be 256, 512 or 1024");
  if (o.ctas_per_sm > 16) return fail(BCP_ERR_INVALID, "ctas_per_sm must be in [1, 16]");
  if (o.order > 3) return fail(BCP_ERR_INVALID, "order must be 0, 1, 2 or 3");
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
  if (!o.src_buf_count && o.src_buf_first) return fail(BCP_ERR_INVALID, "src_buf_first is set but src_buf_count is 0");
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


int match_and_lower(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes, size_t n_src_bufs,
                    const bcp_shard_meta* dst, size_t n_dst, const uint64_t* dst_buf_bytes, size_t n_dst_bufs,
                    const Options& opt, std::vector<Item>* items, std::vector<Gap>* gaps, bcp_plan_stats_t* stats,
                    std::vector<uint32_t>* used_src) {
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
  const uint32_t keep_first = opt.src_buf_first, keep_count = opt.src_buf_count;
  if (keep_count && (keep_first > n_src_bufs || keep_count > n_src_bufs - keep_first))
    return fail(BCP_ERR_INVALID, "source buffers [%u, %u + %u) are not among the %zu given", keep_first, keep_first, keep_count, n_src_bufs);
  std::vector<uint8_t> src_used(n_src ? n_src : 1, 0);  // saved entries that a kept piece reads
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
        // a plan restricted to some source buffers matches and checks coverage against all of
        // them, and keeps the pieces that are read from the chosen ones
        if (keep_count && (s.buf < keep_first || s.buf - keep_first >= keep_count)) continue;
        src_used[s.meta] = 1;  // (a saved entry belongs to one tensor, so no two threads write the same flag)
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
  if (used_src) {
    used_src->clear();
    for (size_t i = 0; i < n_src; ++i)
      if (src_used[i]) used_src->push_back(uint32_t(i));
  }
  stats->n_src_entries = n_se;
  stats->n_dst_entries = n_de;
  stats->n_fqns = fams.size();
  stats->n_intersections = n_inter;
  stats->bytes_src_unique = uniq;
  return BCP_OK;
}

}  // namespace bcp
