// Host planner: metadata -> flat work list.
//
// Follows the load-time resharding workflow of the paper (arXiv 2407.20143):
//   Sec. 3.2 "Decomposing irregular tensors": an irregular (flat) shard becomes several
//            regular boxes;
//   Sec. 3.3 Step 2: every wanted shard is matched against the saved shards of the same
//            FQN; each matching segment becomes one piece of the load plan.
// Everything here is int64 arithmetic on the host; no CUDA.
#include <algorithm>
#include <chrono>
#include <cstdio>
#include <cstring>
#include <string>
#include <unordered_map>

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
  uint32_t itemsize, dtype_tag, ndim;
  int64_t shape[BCP_MAX_NDIM];
  std::vector<Entry> src, dst;
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

void expand(const bcp_shard_meta& m, uint32_t meta_index, int64_t count, std::vector<Entry>* out) {
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
  std::vector<RelBox> boxes;
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
void lower(const Entry& s, const Entry& d, uint32_t ndim, uint32_t isz, const int64_t* off, const int64_t* len,
           std::vector<Item>* items) {
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
    so += uint64_t(off[k] - s.off[k]) * uint64_t(ss[k]) * isz;
    dof += uint64_t(off[k] - d.off[k]) * uint64_t(ds[k]) * isz;
  }
  // dims of extent > 1, outer to inner, with byte strides
  struct Dim {
    uint64_t n, sp, dp;
  };
  Dim dims[BCP_MAX_NDIM + 1];
  int nd = 0;
  for (uint32_t k = 0; k < ndim; ++k)
    if (len[k] > 1) dims[nd++] = Dim{uint64_t(len[k]), uint64_t(ss[k]) * isz, uint64_t(ds[k]) * isz};
  // the innermost dim must be a dense run of elements on both sides; otherwise add a run of one element
  if (nd == 0 || dims[nd - 1].sp != isz || dims[nd - 1].dp != isz) dims[nd++] = Dim{1, isz, isz};
  // merge a dim into the run while it is dense on both sides
  uint64_t run = dims[nd - 1].n * isz;
  --nd;
  while (nd > 0 && dims[nd - 1].sp == run && dims[nd - 1].dp == run) {
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
  it.row_bytes = run;
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

struct SegKey {  // identity of a matched segment on the saved side (for the unique-bytes count)
  uint32_t fam, src;
  int64_t off[BCP_MAX_NDIM], len[BCP_MAX_NDIM];
  bool operator<(const SegKey& o) const { return memcmp(this, &o, sizeof *this) < 0; }
  bool operator==(const SegKey& o) const { return memcmp(this, &o, sizeof *this) == 0; }
};

}  // namespace

int match_and_lower(const bcp_shard_meta* src, size_t n_src, const uint64_t* src_buf_bytes, size_t n_src_bufs,
                    const bcp_shard_meta* dst, size_t n_dst, const uint64_t* dst_buf_bytes, size_t n_dst_bufs,
                    bool allow_replicas, std::vector<Item>* items, std::vector<Gap>* gaps, bcp_plan_stats_t* stats) {
  if ((n_src && !src) || (n_dst && !dst) || (n_src_bufs && !src_buf_bytes) || (n_dst_bufs && !dst_buf_bytes))
    return fail(BCP_ERR_INVALID, "bcp_plan: NULL array with non-zero count");
  std::unordered_map<std::string, uint32_t> ids;
  std::vector<Family> fams;
  auto family_of = [&](const bcp_shard_meta& m, const char* side, size_t i, uint32_t* id) -> int {
    auto it = ids.find(m.fqn);
    if (it == ids.end()) {
      Family f;
      f.fqn = m.fqn;
      f.itemsize = m.itemsize;
      f.dtype_tag = m.dtype_tag;
      f.ndim = m.ndim;
      for (uint32_t k = 0; k < BCP_MAX_NDIM; ++k) f.shape[k] = k < m.ndim ? m.global_shape[k] : 1;
      *id = uint32_t(fams.size());
      ids.emplace(m.fqn, *id);
      fams.push_back(std::move(f));
      return BCP_OK;
    }
    const Family& f = fams[it->second];
    bool same = f.itemsize == m.itemsize && f.dtype_tag == m.dtype_tag && f.ndim == m.ndim;
    for (uint32_t k = 0; same && k < m.ndim; ++k) same = f.shape[k] == m.global_shape[k];
    if (!same)
      return fail(BCP_ERR_MISMATCH, "%s[%zu] %s: itemsize, dtype_tag, ndim or global shape differs from an earlier entry",
                  side, i, m.fqn);
    *id = it->second;
    return BCP_OK;
  };
  for (size_t i = 0; i < n_src; ++i) {
    int64_t n;
    uint32_t f;
    if (int rc = check_meta(src[i], "src", i, src_buf_bytes, n_src_bufs, &n)) return rc;
    if (int rc = family_of(src[i], "src", i, &f)) return rc;
    expand(src[i], uint32_t(i), n, &fams[f].src);
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
      int64_t n;
      uint32_t f;
      if (int rc = check_meta(dst[i], "dst", i, dst_buf_bytes, n_dst_bufs, &n)) return rc;
      if (int rc = family_of(dst[i], "dst", i, &f)) return rc;
      expand(dst[i], uint32_t(i), n, &fams[f].dst);
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
  std::vector<SegKey> segs;
  uint64_t n_inter = 0, n_se = 0, n_de = 0;
  for (uint32_t fi = 0; fi < fams.size(); ++fi) {
    Family& f = fams[fi];
    n_se += f.src.size();
    n_de += f.dst.size();
    const uint32_t nd = f.ndim;
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
    for (const Entry& d : f.dst) {
      int64_t covered = 0;
      const int64_t dend0 = d.off[0] + d.len[0];
      for (uint32_t si = 0; si < f.src.size(); ++si) {
        const Entry& s = f.src[si];
        if (s.off[0] >= dend0) break;  // sorted by first offset
        int64_t o[BCP_MAX_NDIM], l[BCP_MAX_NDIM];
        if (!intersect(s, d, nd, o, l)) continue;
        covered += volume(l, 0, nd);
        ++n_inter;
        lower(s, d, nd, f.itemsize, o, l, items);
        SegKey key;
        memset(&key, 0, sizeof key);
        key.fam = fi;
        key.src = si;
        for (uint32_t k = 0; k < nd; ++k) {
          key.off[k] = o[k];
          key.len[k] = l[k];
        }
        segs.push_back(key);
      }
      if (covered != d.vol)
        return fail(BCP_ERR_UNCOVERED, "%s: dst[%u] wants %lld elements, saved entries hold %lld of them", f.fqn, d.meta,
                    (long long)d.vol, (long long)covered);
    }
  }
  std::sort(segs.begin(), segs.end());
  segs.erase(std::unique(segs.begin(), segs.end()), segs.end());
  uint64_t uniq = 0;
  for (const SegKey& k : segs) uniq += uint64_t(volume(k.len, 0, fams[k.fam].ndim)) * fams[k.fam].itemsize;
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

struct Cutter {
  const Options& opt;
  const std::vector<uint64_t>* src_bytes;  // source buffer sizes (may be null: unknown)
  std::vector<bcp_tile> tma, big, small;
  std::vector<Rect> rects;
  bcp_plan_stats_t* st;

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
    if (g < 4) st->bytes_misaligned += payload;
    if (rows > 1) ++st->n_strided_tiles;
    st->bytes_copied += payload;
    if (payload < opt.small_bytes) {
      t.flags |= BCP_TILE_SMALL;
      small.push_back(t);
    } else {
      // TMA staging: whole 16-byte units between 16-byte aligned addresses (runs and rectangles),
      // or a run / rectangle of any alignment whose 16-byte aligned supersets stay inside the source buffer
      bool eligible = !it.zero && opt.path_mask != 1 && row_bytes >= opt.tma_min_row_bytes;
      if (eligible && g < 4) {  // the superset of the last row must not reach past the source buffer
        const uint64_t end16 = (src_off + (rows - 1) * (rows > 1 ? it.src_pitch : 0) + row_bytes + 15) & ~uint64_t(15);
        eligible = src_bytes && it.src_buf < src_bytes->size() && end16 <= (*src_bytes)[it.src_buf];
      }
      if (eligible) {
        t.flags |= BCP_TILE_TMA;
        ++st->n_tma_tiles;
        tma.push_back(t);
      } else {
        big.push_back(t);
      }
    }
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
    Rect rc;
    rc.src_off = it.src_off, rc.dst_off = it.dst_off, rc.src_pitch = it.src_pitch, rc.dst_pitch = it.dst_pitch;
    rc.rows = it.rows, rc.row_bytes = uint32_t(it.row_bytes), rc.src_buf = it.src_buf, rc.dst_buf = it.dst_buf;
    rc.box_rows = uint32_t(box_rows);
    rects.push_back(rc);
    for (uint64_t r = 0; r < it.rows; r += rpt) {
      const uint64_t nr = std::min(rpt, it.rows - r);
      bcp_tile t;
      memset(&t, 0, sizeof t);
      t.src_off = it.src_off + r * it.src_pitch;
      t.dst_off = it.dst_off + r * it.dst_pitch;
      t.src_pitch = it.src_pitch, t.dst_pitch = it.dst_pitch;
      t.rows = uint32_t(nr), t.row_bytes = uint32_t(it.row_bytes);
      t.src_buf = it.src_buf, t.dst_buf = it.dst_buf;
      t.flags = 4u | BCP_TILE_TMA | BCP_TILE_TMA2D;
      t.reserved[0] = uint32_t(rects.size());  // index + 1
      t.reserved[1] = uint32_t(r);
      t.reserved[2] = uint32_t(box_rows);
      ++st->n_strided_tiles;
      ++st->n_tma_tiles;
      st->bytes_copied += nr * it.row_bytes;
      tma.push_back(t);
    }
    return true;
  }

  void cut(const Item& it) {
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

void build_tiles(std::vector<Item>& items, Options& opt, const std::vector<uint64_t>* src_bytes,
                 std::vector<bcp_tile>* tiles, size_t* n_tma, size_t* n_big, std::vector<Rect>* rects,
                 bcp_plan_stats_t* stats) {
  // coalesce runs that are adjacent on both sides (e.g. the sub-boxes of one flat slice)
  std::sort(items.begin(), items.end(), [](const Item& a, const Item& b) {
    return a.dst_buf != b.dst_buf ? a.dst_buf < b.dst_buf : a.dst_off < b.dst_off;
  });
  std::vector<Item> merged;
  merged.reserve(items.size());
  for (const Item& it : items) {
    if (it.rows * it.row_bytes == 0) continue;
    if (!merged.empty()) {
      Item& p = merged.back();
      if (p.rows == 1 && it.rows == 1 && p.zero == it.zero && p.dst_buf == it.dst_buf &&
          p.dst_off + p.row_bytes == it.dst_off &&
          (it.zero || (p.src_buf == it.src_buf && p.src_off + p.row_bytes == it.src_off))) {
        p.row_bytes += it.row_bytes;
        continue;
      }
    }
    merged.push_back(it);
  }
  stats->n_items = merged.size();
  stats->bytes_copied = 0;
  stats->bytes_misaligned = 0;
  stats->n_strided_tiles = 0;
  stats->n_tma_tiles = 0;
  Cutter c{opt, src_bytes, {}, {}, {}, {}, stats};
  for (const Item& it : merged) c.cut(it);
  if (opt.path_mask == 0) {  // small jobs are launch-bound: keep them in one kernel
    uint64_t eligible = 0;
    for (const bcp_tile& t : c.tma) eligible += uint64_t(t.rows) * t.row_bytes;
    if (eligible < (128u << 20)) {
      for (bcp_tile& t : c.tma) {
        t.flags &= ~(BCP_TILE_TMA | BCP_TILE_TMA2D);
        t.reserved[0] = t.reserved[1] = t.reserved[2] = 0;
      }
      c.rects.clear();
      c.big.insert(c.big.end(), c.tma.begin(), c.tma.end());
      c.tma.clear();
      stats->n_tma_tiles = 0;
    }
  }
  auto by_src = [](const bcp_tile& a, const bcp_tile& b) {
    if (a.src_buf != b.src_buf) return a.src_buf < b.src_buf;
    if (a.src_off != b.src_off) return a.src_off < b.src_off;
    return a.dst_buf != b.dst_buf ? a.dst_buf < b.dst_buf : a.dst_off < b.dst_off;
  };
  auto by_dst = [](const bcp_tile& a, const bcp_tile& b) {
    return a.dst_buf != b.dst_buf ? a.dst_buf < b.dst_buf : a.dst_off < b.dst_off;
  };
  // Stage geometry of the TMA kernel when the caller left it open.  Long aligned runs only need
  // a few copy commands per stage, so two CTAs with 32 KiB stages per SM are enough; shifted
  // runs (copied out of shared memory by the warp itself) and rectangles with rows under 2 KiB
  // (one copy command per row) are limited by what one warp can issue and want four CTAs with
  // 16 KiB stages.  Both fill 192 KiB of shared memory per SM.
  {
    uint64_t total = 0, busy = 0, boxed = 0;
    for (const bcp_tile& t : c.tma) {
      const uint64_t n = uint64_t(t.rows) * t.row_bytes;
      total += n;
      if (t.flags & BCP_TILE_TMA2D) {
        boxed += n;
      } else if ((t.flags & BCP_TILE_GRAN_MASK) < 4 || (t.rows > 1 && t.row_bytes < 2048)) {
        busy += n;
      }
    }
    const bool many_busy = busy * 8 >= total && total > 0;
    const bool many_boxed = !many_busy && boxed * 8 >= total && total > 0;  // boxes are at most 16 KiB: deeper ring
    if (!opt.tma_stage_bytes) opt.tma_stage_bytes = (many_busy || many_boxed) ? 16384 : 32768;
    if (!opt.tma_ctas_per_sm) opt.tma_ctas_per_sm = many_busy ? 4 : 2;
    if (!opt.tma_stages) opt.tma_stages = many_boxed ? 4 : 3;
  }
  // Register kernel: a CTA per unit for small jobs (fewer, fatter workers start faster); every
  // warp its own worker once the kernel has a lot to move (no barriers, deeper overlap).
  if (!opt.worker) {
    uint64_t reg_bytes = 0;
    for (const bcp_tile& t : c.big) reg_bytes += uint64_t(t.rows) * t.row_bytes;
    for (const bcp_tile& t : c.small) reg_bytes += uint64_t(t.rows) * t.row_bytes;
    opt.worker = reg_bytes >= (128u << 20) ? 2 : 1;
    if (opt.worker == 2 && !opt.ctas_per_sm) opt.ctas_per_sm = 4;
  }
  if (!opt.ctas_per_sm) opt.ctas_per_sm = 2;
  for (std::vector<bcp_tile>* v : {&c.tma, &c.big, &c.small}) {
    if (opt.order == 1) {
      std::sort(v->begin(), v->end(), by_src);
    } else {
      std::sort(v->begin(), v->end(), by_dst);
    }
  }
  if (opt.order == 1 && opt.fanout == 1) mark_followers(c.tma.data(), c.tma.size());
  stats->n_tiles = c.tma.size() + c.big.size();
  stats->n_small_tiles = c.small.size();
  *n_tma = c.tma.size();
  *n_big = c.big.size();
  if (rects) *rects = std::move(c.rects);
  tiles->clear();
  tiles->reserve(c.tma.size() + c.big.size() + c.small.size());
  tiles->insert(tiles->end(), c.tma.begin(), c.tma.end());
  tiles->insert(tiles->end(), c.big.begin(), c.big.end());
  tiles->insert(tiles->end(), c.small.begin(), c.small.end());
}

}  // namespace bcp
