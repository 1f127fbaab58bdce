// Plan images: a plan as a position-independent byte string for reuse in another process
// (the paper's plan cache, Sec. 4.1), verified before use because a work list drives device copies.
#include <algorithm>
#include <new>

#include "plan_object.hpp"

using namespace bcp;

namespace {
const char kMagic[8] = {'B', 'C', 'P', 'P', 'L', 'A', 'N', '1'};
struct ImageHeader {
  char magic[8];
  uint32_t version, tile_size;
  Options opt;
  bcp_plan_stats_t stats;
  uint64_t n_src_bufs, n_dst_bufs, n_tma, n_big, n_tiles, n_rects, n_gaps, n_cvt;
};
uint64_t fnv1a(const unsigned char* p, size_t n) {
  uint64_t h = 1469598103934665603ull;
  for (size_t i = 0; i < n; ++i) h = (h ^ p[i]) * 1099511628211ull;
  return h;
}
// A unit is safe to execute if it stays inside its buffers and its flags match its geometry.
bool tile_ok(const bcp_tile& t, const std::vector<uint64_t>& sb, const std::vector<uint64_t>& db, const std::vector<Rect>& rects,
             const Options& opt) {
  if (t.rows == 0 || t.row_bytes == 0 || t.dst_buf >= db.size()) return false;
  if (const uint32_t kind = (t.flags & BCP_TILE_CVT_MASK) >> BCP_TILE_CVT_SHIFT) {
    // converting unit: element-aligned on both sides, source rows hold the same number of elements
    if (kind > BCP_CONVERT_BF16_TO_F32 || (t.flags & ~(BCP_TILE_GRAN_MASK | BCP_TILE_CVT_MASK | BCP_TILE_TMA)) || t.src_buf >= sb.size())
      return false;
    const uint64_t s_isz = kind == BCP_CONVERT_F32_TO_BF16 ? 4 : 2, d_isz = 6 - s_isz;
    const uint64_t s_row = uint64_t(t.row_bytes) / d_isz * s_isz;
    if (t.row_bytes % d_isz || t.dst_off % d_isz || t.dst_pitch % d_isz || t.src_off % s_isz || t.src_pitch % s_isz) return false;
    if (t.rows > 1 && (t.dst_pitch < t.row_bytes || t.src_pitch < s_row)) return false;
    const uint64_t span_d = uint64_t(t.rows - 1) * t.dst_pitch + t.row_bytes, span_s = uint64_t(t.rows - 1) * t.src_pitch + s_row;
    if (t.dst_off > db[t.dst_buf] || span_d > db[t.dst_buf] - t.dst_off) return false;
    if (t.src_off > sb[t.src_buf] || span_s > sb[t.src_buf] - t.src_off) return false;
    // staged conversion fetches the 16-byte aligned superset of every source row
    if ((t.flags & BCP_TILE_TMA) && (s_row < 16 || ((t.src_off + span_s + 15) & ~uint64_t(15)) > sb[t.src_buf])) return false;
    return uint64_t(t.rows) * t.row_bytes <= opt.tile_bytes;
  }
  const bool zero = t.flags & BCP_TILE_ZERO;
  const uint64_t span_d = uint64_t(t.rows - 1) * t.dst_pitch + t.row_bytes;
  if (t.dst_off > db[t.dst_buf] || span_d > db[t.dst_buf] - t.dst_off) return false;
  if (t.rows > 1 && t.dst_pitch < t.row_bytes) return false;
  uint64_t bits = t.dst_off | t.row_bytes | t.dst_pitch;
  if (!zero) {
    if (t.src_buf >= sb.size()) return false;
    const uint64_t span_s = uint64_t(t.rows - 1) * t.src_pitch + t.row_bytes;
    if (t.src_off > sb[t.src_buf] || span_s > sb[t.src_buf] - t.src_off) return false;
    bits |= t.src_off | t.src_pitch;
  }
  uint32_t g = 0;
  while (g < 4 && !((bits >> g) & 1)) ++g;
  if ((t.flags & BCP_TILE_GRAN_MASK) > g) return false;  // a wider access than the offsets allow would fault
  if (t.flags & BCP_TILE_TMA2D) {  // must be a whole number of boxes of the rectangle it names
    if (!(t.flags & BCP_TILE_TMA) || zero || g < 4 || t.reserved[0] == 0 || t.reserved[0] > rects.size()) return false;
    const Rect& r = rects[t.reserved[0] - 1];
    const uint64_t row0 = t.reserved[1];
    if (t.reserved[2] != r.box_rows || r.box_rows == 0 || row0 % r.box_rows || row0 + t.rows > r.rows) return false;
    if (t.rows % r.box_rows && row0 + t.rows != r.rows) return false;
    if (t.src_buf != r.src_buf || t.dst_buf != r.dst_buf || t.row_bytes != r.row_bytes || t.src_pitch != r.src_pitch ||
        t.dst_pitch != r.dst_pitch || t.src_off != r.src_off + row0 * r.src_pitch || t.dst_off != r.dst_off + row0 * r.dst_pitch)
      return false;
    if (uint64_t(r.box_rows) * r.row_bytes > opt.tma_stage_bytes) return false;
    return uint64_t(t.rows) * t.row_bytes <= std::max<uint64_t>(opt.tile_bytes, uint64_t(r.box_rows) * r.row_bytes);
  }
  if (t.flags & BCP_TILE_TMA) {
    if (zero || t.row_bytes < 16) return false;
    if (g < 4) {  // shifted run or rectangle: the aligned superset of the last row stays inside the source buffer
      if (((t.src_off + uint64_t(t.rows - 1) * t.src_pitch + t.row_bytes + 15) & ~uint64_t(15)) > sb[t.src_buf]) return false;
    }
  }
  return uint64_t(t.rows) * t.row_bytes <= opt.tile_bytes;
}
// A rectangle's two views must stay inside their buffers and satisfy the tensor-map rules.
bool rect_ok(const Rect& r, const std::vector<uint64_t>& sb, const std::vector<uint64_t>& db) {
  if (r.src_buf >= sb.size() || r.dst_buf >= db.size() || r.rows == 0 || r.rows >= (uint64_t(1) << 31)) return false;
  if (r.row_bytes < 16 || r.row_bytes > 2048 || r.box_rows == 0 || r.box_rows > 256) return false;
  if ((r.src_off | r.dst_off | r.row_bytes | r.src_pitch | r.dst_pitch) & 15) return false;
  if (r.src_pitch < r.row_bytes || r.dst_pitch < r.row_bytes || r.src_pitch >= (uint64_t(1) << 40) || r.dst_pitch >= (uint64_t(1) << 40))
    return false;
  const uint64_t ss = (r.rows - 1) * r.src_pitch + r.row_bytes, ds = (r.rows - 1) * r.dst_pitch + r.row_bytes;
  return r.src_off <= sb[r.src_buf] && ss <= sb[r.src_buf] - r.src_off && r.dst_off <= db[r.dst_buf] && ds <= db[r.dst_buf] - r.dst_off;
}
}  // namespace

extern "C" {

int bcp_plan_serialize(const bcp_plan_t* plan, void* out, size_t cap, size_t* n) {
  if (!plan || !n) return fail(BCP_ERR_INVALID, "bcp_plan_serialize: NULL argument");
  const size_t need = sizeof(ImageHeader) + (plan->src_bytes.size() + plan->dst_bytes.size()) * sizeof(uint64_t) +
                      plan->tiles.size() * sizeof(bcp_tile) + plan->rects.size() * sizeof(Rect) + plan->gaps.size() * sizeof(Gap) +
                      sizeof(uint64_t);
  *n = need;
  if (!out || cap < need) return fail(BCP_ERR_CAPACITY, "bcp_plan_serialize: image needs %zu bytes, room for %zu", need, out ? cap : size_t(0));
  ImageHeader h;
  memset(static_cast<void*>(&h), 0, sizeof h);  // padding bytes too: images are compared and checksummed
  memcpy(h.magic, kMagic, 8);
  h.version = uint32_t(bcp_version());
  h.tile_size = sizeof(bcp_tile);
  h.opt = plan->opt;
  h.stats = plan->stats;
  h.n_src_bufs = plan->src_bytes.size();
  h.n_dst_bufs = plan->dst_bytes.size();
  h.n_tma = plan->n_tma;
  h.n_big = plan->n_big;
  h.n_cvt = plan->n_cvt;
  h.n_tiles = plan->tiles.size();
  h.n_rects = plan->rects.size();
  h.n_gaps = plan->gaps.size();
  unsigned char* p = static_cast<unsigned char*>(out);
  memcpy(p, &h, sizeof h);
  p += sizeof h;
  if (h.n_src_bufs) memcpy(p, plan->src_bytes.data(), h.n_src_bufs * sizeof(uint64_t));
  p += h.n_src_bufs * sizeof(uint64_t);
  if (h.n_dst_bufs) memcpy(p, plan->dst_bytes.data(), h.n_dst_bufs * sizeof(uint64_t));
  p += h.n_dst_bufs * sizeof(uint64_t);
  if (h.n_tiles) memcpy(p, plan->tiles.data(), h.n_tiles * sizeof(bcp_tile));
  p += h.n_tiles * sizeof(bcp_tile);
  if (h.n_rects) memcpy(p, plan->rects.data(), h.n_rects * sizeof(Rect));
  p += h.n_rects * sizeof(Rect);
  if (h.n_gaps) memcpy(p, plan->gaps.data(), h.n_gaps * sizeof(Gap));
  p += h.n_gaps * sizeof(Gap);
  const uint64_t sum = fnv1a(static_cast<unsigned char*>(out), size_t(p - static_cast<unsigned char*>(out)));
  memcpy(p, &sum, sizeof sum);
  return BCP_OK;
}

int bcp_plan_deserialize(const void* image, size_t n, bcp_plan_t** out_plan) {
  if (!image || !out_plan) return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: NULL argument");
  if (n < sizeof(ImageHeader) + sizeof(uint64_t)) return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: image too short");
  ImageHeader h;
  memcpy(&h, image, sizeof h);
  if (memcmp(h.magic, kMagic, 8) != 0) return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: not a plan image");
  if (h.version != uint32_t(bcp_version()) || h.tile_size != sizeof(bcp_tile))
    return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: image of library version %u, this is %d", h.version, bcp_version());
  const uint64_t lim = uint64_t(1) << 32;
  if (h.n_src_bufs >= lim || h.n_dst_bufs >= lim || h.n_tiles >= lim || h.n_rects >= lim || h.n_gaps >= lim || h.n_tma > h.n_tiles ||
      h.n_big > h.n_tiles - h.n_tma || h.n_cvt > h.n_tiles - h.n_tma - h.n_big)
    return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: implausible counts");
  const uint64_t need = sizeof(ImageHeader) + (h.n_src_bufs + h.n_dst_bufs) * sizeof(uint64_t) + h.n_tiles * sizeof(bcp_tile) +
                        h.n_rects * sizeof(Rect) + h.n_gaps * sizeof(Gap) + sizeof(uint64_t);
  if (need != n) return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: image is %zu bytes, its header implies %llu", n, (unsigned long long)need);
  const unsigned char* base = static_cast<const unsigned char*>(image);
  uint64_t sum;
  memcpy(&sum, base + n - sizeof sum, sizeof sum);
  if (sum != fnv1a(base, n - sizeof sum)) return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: checksum mismatch");
  {  // the options were validated when the plan was made; re-check what the launch code relies on
    const Options& o = h.opt;
    if ((o.block_threads != 256 && o.block_threads != 512 && o.block_threads != 1024) || o.ctas_per_sm < 1 || o.ctas_per_sm > 16 ||
        o.tile_bytes < 4096 || o.tile_bytes > (64u << 20) || (o.unroll != 4 && o.unroll != 8) || (o.worker != 1 && o.worker != 2) || o.tma_stages < 2 || o.tma_stages > 8 ||
        o.tma_stage_bytes % 128 || o.tma_stage_bytes < 1024 || o.tma_stage_bytes > 65536 ||
        uint64_t(o.tma_stage_bytes) * o.tma_stages > 200 * 1024 || o.tma_ctas_per_sm < 1 || o.tma_ctas_per_sm > 16 || o.cache_hints < 1 ||
        o.cache_hints > 4)
      return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: options out of range");
  }
  bcp_plan_t* p = new (std::nothrow) bcp_plan_t;
  if (!p) return fail(BCP_ERR_NOMEM, "out of host memory");
  try {
    const unsigned char* q = base + sizeof h;
    p->opt = h.opt;
    p->stats = h.stats;
    p->src_bytes.resize(h.n_src_bufs);
    p->dst_bytes.resize(h.n_dst_bufs);
    p->tiles.resize(h.n_tiles);
    if (h.n_src_bufs) memcpy(p->src_bytes.data(), q, h.n_src_bufs * sizeof(uint64_t));
    q += h.n_src_bufs * sizeof(uint64_t);
    if (h.n_dst_bufs) memcpy(p->dst_bytes.data(), q, h.n_dst_bufs * sizeof(uint64_t));
    q += h.n_dst_bufs * sizeof(uint64_t);
    if (h.n_tiles) memcpy(p->tiles.data(), q, h.n_tiles * sizeof(bcp_tile));
    q += h.n_tiles * sizeof(bcp_tile);
    p->rects.resize(h.n_rects);
    if (h.n_rects) memcpy(p->rects.data(), q, h.n_rects * sizeof(Rect));
    q += h.n_rects * sizeof(Rect);
    p->gaps.resize(h.n_gaps);
    if (h.n_gaps) memcpy(p->gaps.data(), q, h.n_gaps * sizeof(Gap));
    p->n_tma = h.n_tma;
    p->n_big = h.n_big;
    p->n_cvt = h.n_cvt;
  } catch (const std::bad_alloc&) {
    delete p;
    return fail(BCP_ERR_NOMEM, "out of host memory");
  }
  for (const Gap& g : p->gaps) {  // gaps are zeroed in host memory: they must stay inside their buffer
    if (g.buf >= p->dst_bytes.size() || g.off > p->dst_bytes[g.buf] || g.len > p->dst_bytes[g.buf] - g.off) {
      delete p;
      return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: a gap lies outside its target buffer");
    }
  }
  for (size_t i = 0; i < p->rects.size(); ++i) {
    if (!rect_ok(p->rects[i], p->src_bytes, p->dst_bytes)) {
      delete p;
      return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: rectangle %zu is inconsistent with the recorded buffers", i);
    }
  }
  {  // replica groups must be exactly what the planner would mark: a follower is never staged itself
    std::vector<bcp_tile> again(p->tiles.begin(), p->tiles.begin() + p->n_tma);
    for (bcp_tile& t : again) t.flags &= ~(BCP_TILE_FOLLOW | (7u << BCP_TILE_FAN_SHIFT));
    if (p->opt.fanout == 1 && p->opt.order != 2) mark_followers(again.data(), again.size());
    bool ok = true;
    for (size_t i = 0; ok && i < p->tiles.size(); ++i)
      ok = i < p->n_tma ? again[i].flags == p->tiles[i].flags : !(p->tiles[i].flags & (BCP_TILE_FOLLOW | (7u << BCP_TILE_FAN_SHIFT)));
    if (!ok) {
      delete p;
      return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: replica groups of the work list are inconsistent");
    }
  }
  for (size_t i = 0; i < p->tiles.size(); ++i) {
    const bcp_tile& t = p->tiles[i];
    const bool in_tma = i < p->n_tma, in_cvt = i >= p->tiles.size() - p->n_cvt, in_small = i >= p->n_tma + p->n_big && !in_cvt;
    if (!tile_ok(t, p->src_bytes, p->dst_bytes, p->rects, p->opt) || (!in_cvt && bool(t.flags & BCP_TILE_TMA) != in_tma) ||
        bool(t.flags & BCP_TILE_SMALL) != in_small || bool(t.flags & BCP_TILE_CVT_MASK) != in_cvt) {
      delete p;
      return fail(BCP_ERR_INVALID, "bcp_plan_deserialize: work unit %zu is inconsistent with the recorded buffers", i);
    }
  }
  *out_plan = p;
  return BCP_OK;
}

}  // extern "C"
