// Host planner, second half: copy items -> flat work list (coalesce, cut into units, classify,
// order).  The first half (metadata -> items) is planner.cpp.
#include <algorithm>
#include <cstdint>
#include <cstring>
#include <memory>
#include <vector>

#include "host_threads.hpp"
#include "plan.hpp"

namespace bcp {

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
  uint64_t cvt_staged = 0;  // source + target bytes of converting units that qualify for the staged kernel
  void add(const Tally& o) {
    bytes_copied += o.bytes_copied, bytes_misaligned += o.bytes_misaligned, n_strided += o.n_strided;
    tma_bytes += o.tma_bytes, tma_busy += o.tma_busy, tma_boxed += o.tma_boxed, cvt_bytes += o.cvt_bytes;
    cvt_staged += o.cvt_staged;
  }
};

// Cuts items into units.  Used twice: a counting pass (out[] null) that sizes the arrays, then
// a writing pass in which every block of items starts at its own, precomputed positions.
struct Cutter {
  const Options& opt;
  const std::vector<uint64_t>* src_bytes;  // source buffer sizes (may be null: unknown)
  bool demote;                             // small job: TMA-eligible units go to the register kernel
  bool demote_cvt;                         // small converting job: no unit is marked for the staged converting kernel
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
    const uint64_t unit = (co && !it.zero && ((so | dof) & 15) == 0) ? opt.run_tile_bytes : opt.tile_bytes;
    uint64_t first = unit;
    if (n > unit && (dof & 255)) first = unit - (dof & 255);
    while (n) {
      const uint64_t c = std::min<uint64_t>(n, first);
      emit(it, so, dof, 1, c);
      so += c, dof += c, n -= c;
      first = unit;
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

  // Converting units: rows x row_bytes TARGET bytes each; no warp path.  A unit whose source rows
  // are long enough, and whose 16-byte aligned supersets stay inside the source buffer, is marked
  // BCP_TILE_TMA: the staged converting kernel takes it, the register one skips it.
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
    const uint64_t src_row = it.cvt == BCP_CONVERT_F32_TO_BF16 ? row_bytes * 2 : row_bytes / 2;
    bool staged = opt.path_mask != 1 && src_row >= opt.tma_min_row_bytes;
    if (staged) {
      const uint64_t end16 = (src_off + (rows - 1) * (rows > 1 ? it.src_pitch : 0) + src_row + 15) & ~uint64_t(15);
      staged = src_bytes && it.src_buf < src_bytes->size() && end16 <= (*src_bytes)[it.src_buf];
    }
    if (staged) {
      st.cvt_staged += rows * (row_bytes + src_row);
      if (!demote_cvt) t.flags |= BCP_TILE_TMA;
    }
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

  // Unit size of aligned contiguous runs when the caller left tile_bytes open.  Measured on the staging
  // kernel: plans that move every source byte once (or nearly) run 0.5-1.1 % faster when such runs are cut
  // into units of one stage (32 KiB) instead of two -- its CTAs then sweep a narrower window of memory at
  // any time; plans that write DP replicas of their sources (replica groups: one staged copy, several
  // stores) are 0.6 % slower that way, and so are shifted runs and rectangles, which keep tile_bytes.
  uint64_t written = 0;  // source bytes the list reads, replicas counted every time (= target bytes unless converted)
  for (const Item& it : merged)
    if (!it.zero) written += it.rows * it.src_row_bytes();
  const uint64_t uniq = stats->bytes_src_unique;  // 0 when the caller does not know (pack layouts: nothing is read twice)
  if (!opt.run_tile_bytes) {
    const bool replicated = uniq && written > uniq + uniq / 4;
    opt.run_tile_bytes = replicated || opt.convert ? opt.tile_bytes : std::min<uint32_t>(opt.tile_bytes, 32768);
  }
  // Order of the units when the caller left it open: 1 as soon as source bytes are wanted more than once
  // (replicas of a piece must sit side by side to be staged once and to hit L2), else 2 (by target address:
  // the pieces that make up one stretch of a target -- the column blocks of a row-parallel weight, say, which
  // come from several saved shards -- are then written at about the same time; measured: cfg3 1.2 %, cfg4 0.6 %,
  // the converting 8B merge 0.8 % faster than in source order; cfg5, where an eighth of the target bytes are
  // replicas, 5 % slower).  Under order 1 the staged units get both: replicas side by side, and these groups in
  // the order of their first member's target address; that pays when the plan has rectangles, whose target rows
  // are completed by pieces from several shards (cfg2 6.66 -> 6.59 ms), and costs a little when it has only runs
  // (cfg5 17.00 -> 17.08 ms), which stay in plain source order (3).  Decided after the counting pass below.
  const bool choose_order = !opt.order;
  const bool reads_twice = uniq && written > uniq + uniq / 50;

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
    Cutter c{opt, src_bytes, false, false, {nullptr, nullptr, nullptr, nullptr}, nullptr, {0, 0, 0, 0}, 0, Tally()};
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
  if (choose_order) opt.order = !reads_twice ? 2 : all.n_strided ? 1 : 3;
  // Tiny jobs stay in the register kernel.  From 4 MiB of stageable payload on the staging kernel is
  // the faster one (measured with L2 flushed, runs of 1 MiB..1 GiB: 10-12 us against 12 us up to 4 MiB,
  // 14 / 16 us at 16 MiB, 31 / 33 us at 64 MiB, 90 / 94 us at 256 MiB; rectangles with 2 KiB rows: 14 / 21 us
  // at 16 MiB, 32 / 49 us at 64 MiB), and the warp units of such a job ride along in the same launch.
  const bool demote = opt.path_mask == 0 && all.tma_bytes < (4u << 20);
  if (demote) {
    for (size_t i = 0; i < n_items; ++i) cnt[i].n[kBig] += cnt[i].n[kTma], cnt[i].n[kTma] = 0, cnt[i].rects = 0;
    all.tma_bytes = all.tma_busy = all.tma_boxed = 0;
  }
  // converting units: the staged kernel was the faster one at every size measured (2-4 KiB source rows, L2
  // flushed: 1 MiB 33 vs 51 us, 64 MiB 37 vs 57 us, 1 GiB 272 vs 311 us; widening 16 vs 37, 45 vs 82, 500 vs 563 us)
  const bool demote_cvt = opt.path_mask == 0 && all.cvt_staged < (1u << 20);
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
    Cutter c{opt, src_bytes, demote, demote_cvt, {cls[0], cls[1], cls[2], cls[3]}, rc.data(), {at.n[0], at.n[1], at.n[2], at.n[3]}, at.rects, Tally()};
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
  const bool by_src = opt.order != 2;
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
    std::unique_ptr<Key[]> again, again_spare;
    if (k == kTma && opt.order == 1 && n > 1) {
      // Second key of the staged class: units that read the same source bytes (neighbours in source order) form
      // a group; a group is keyed by the target address of its first member, a member by its place in the group.
      again.reset(new Key[n]);
      again_spare.reset(new Key[n]);
      size_t head = 0;
      for (size_t i = 0; i < n; ++i) {
        const bcp_tile& t = src[sorted[i].idx];
        const bcp_tile& h = src[sorted[head].idx];
        if (i && !(t.src_buf == h.src_buf && t.src_off == h.src_off && t.rows == h.rows && t.row_bytes == h.row_bytes &&
                   t.src_pitch == h.src_pitch))
          head = i;
        const bcp_tile& g = src[sorted[head].idx];
        again[i] = Key{g.dst_off, uint64_t(i), g.dst_buf, 0, sorted[i].idx, 0};
      }
      sorted = parallel_sort(again.get(), again_spare.get(), n, threads, key_less);
    }
    parallel_jobs((n + kChunk - 1) / kChunk, threads, [&](size_t j) {
      for (size_t i = j * kChunk; i < std::min(n, (j + 1) * kChunk); ++i) dst[i] = src[sorted[i].idx];
    });
    base += n;
  }
  if (opt.order != 2 && opt.fanout == 1) mark_followers(tiles->data(), run.n[kTma]);
  stats->n_tiles = run.n[kTma] + run.n[kBig];
  stats->n_small_tiles = run.n[kSmall];
  *n_tma = run.n[kTma];
  *n_big = run.n[kBig];
  *n_cvt = run.n[kCvt];
  stats->n_cvt_tiles = run.n[kCvt];
  if (rects) *rects = std::move(rc);
}

}  // namespace bcp
