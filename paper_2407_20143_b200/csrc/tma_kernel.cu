// TMA staging path: global -> shared -> global with bulk asynchronous copies.
//
// A CTA is one warp that only issues copy commands; the payload never enters registers.
// Work units (tiles whose offsets, row length and pitches are multiples of 16 bytes) are
// drawn from an atomic ticket counter and cut into chunks of at most one shared-memory
// stage.  A chunk is a run (one bulk copy) or a group of rows of a strided rectangle (one
// bulk copy per row, issued by different lanes, addresses computed here: no descriptors, so a
// plan stays independent of buffer addresses).  Loads complete on a per-stage mbarrier;
// stores are tracked with bulk groups.  With S stages, S-1 loads and up to 2 stores are in
// flight per CTA.  Every wait on an mbarrier is bounded: if it gives up, the CTA records
// BCP_ERR_DEVICE_TIMEOUT, stops taking work and leaves after its stores have drained.
// Every copy has one destination CTA (its own); no thread-block clusters.
//
// Runs whose source and target addresses are not both 16-byte aligned, or differ mod 16 (odd
// element cuts of ZeRO / FSDP flat shards, odd shapes), are staged too: the bulk load fetches
// the 16-byte aligned superset of the source piece, and the warp itself copies the payload out
// of shared memory with coalesced stores of the run's natural width (1, 2, 4 or 8 bytes), so
// global reads stay full-width and writes stay contiguous whatever the relative shift.  Strided
// rectangles with such offsets or pitches are handled the same way, several rows per stage,
// each row in a slot of its own.
//
// Rectangles with short rows can instead be staged with 2-D tensor-map copies
// (cp.async.bulk.tensor.2d): one command moves a box of up to 256 rows, where the per-row form
// would need one command per row and becomes issue-bound.  The two descriptors of a rectangle
// (source view, target view; 8-byte elements, no swizzle) live in global memory, are encoded
// by the host for the buffer addresses of the call, and are read through the tensormap proxy
// after an acquire fence.
//
// The few units of a plan that cannot be staged (pieces under 4 KiB, short unaligned rows, zero
// fills) may ride along as a tail of the ticket range: whoever draws such a ticket copies the
// unit with the warp's own loads and stores while its staged chunks are in flight, which saves a
// second kernel launch behind this one.
#include "kernels.cuh"
#include "copy_loops.cuh"
#include "tma_ptx.cuh"

namespace bcp {
namespace {

constexpr int kMaxFan = 7;  // followers a unit can carry (targets written from the same staged bytes)

struct Chunk {  // what one stage holds: rows x row_bytes, dense in shared memory
  const char* src;
  char* dst;
  uint64_t sp, dp;
  uint32_t rows, row_bytes;
  uint32_t shift;  // shifted run only: payload starts `shift` bytes into the stage
  uint32_t width;  // 0: aligned chunk, stored with bulk copies; 1..4: shifted run, log2 of the store width + 1;
                   // kTensor: one box of a tensor map (src / dst hold the descriptors, rows = box rows, shift = first row)
  // replicas: nf further targets receive the same bytes; their addresses live in fan slot `slot`, and
  // this chunk starts at row r0, byte c0 of the unit
  uint32_t nf, slot, r0, c0;
};

// Follower targets of one unit (same geometry as the head, own address / descriptor and pitch).
struct Fan {
  char* dst[kMaxFan];      // target base address (tensor-map rectangles: target descriptor)
  uint64_t pitch[kMaxFan];
  uint32_t row0[kMaxFan];  // tensor-map rectangles: first row of the unit inside the follower's rectangle
};
constexpr uint32_t kShiftedRows = 4;  // width codes 5..8: several shifted rows per chunk, `shift` = bytes per row slot
constexpr uint32_t kTensor = 9;

// Cuts the current tile into chunks.  All lanes hold the same state.
struct TileCursor {
  const char* s;
  char* d;
  uint64_t sp, dp;
  uint32_t rows, row_bytes;
  uint32_t r, c;  // next row, next byte inside the row
  uint32_t width;  // 0 aligned tile; 1..4 log2(access width) + 1 of a shifted run; kTensor: tensor-map rectangle
  uint32_t box_rows, row0;  // tensor-map rectangle: rows per box, first row of this unit inside the rectangle
  uint32_t nf, slot;        // followers of this unit and the fan slot that holds their targets
  bool live;

  __device__ __forceinline__ void fan(Chunk* out, uint32_t row, uint32_t col) const {
    out->nf = nf;
    out->slot = slot;
    out->r0 = row;
    out->c0 = col;
  }

  __device__ __forceinline__ bool next(uint32_t stage_bytes, Chunk* out) {
    if (!live) return false;
    out->shift = 0;
    out->width = 0;
    if (width == kTensor) {  // boxes of box_rows rows; the last box of a rectangle is clipped by the descriptor
      out->src = s;
      out->dst = d;
      out->rows = box_rows;
      out->row_bytes = row_bytes;
      out->sp = out->dp = 0;
      out->shift = row0 + r;
      out->width = kTensor;
      fan(out, r, 0);
      r += min(box_rows, rows - r);
      if (r == rows) live = false;
      return true;
    }
    if (width) {  // shifted run or rectangle: every row is fetched as its 16-byte aligned superset
      const uint32_t slot = (row_bytes + 45u) & ~15u;  // room for the superset of a row, whatever its shift
      if (rows > 1 && slot <= stage_bytes) {           // several whole rows, one slot each
        const uint32_t k = min(stage_bytes / slot, rows - r);
        out->src = s + uint64_t(r) * sp;
        out->dst = d + uint64_t(r) * dp;
        out->rows = k;
        out->row_bytes = row_bytes;
        out->sp = sp;
        out->dp = dp;
        out->shift = slot;
        out->width = width + kShiftedRows;
        fan(out, r, 0);
        r += k;
        if (r == rows) live = false;
        return true;
      }
      // pieces of one row that leave room for the aligned superset
      const uint32_t n = min(stage_bytes - 32, row_bytes - c);
      out->src = s + uint64_t(r) * sp + c;
      out->dst = d + uint64_t(r) * dp + c;
      out->rows = 1;
      out->row_bytes = n;
      out->sp = out->dp = 0;
      out->shift = uint32_t(reinterpret_cast<uintptr_t>(out->src) & 15);
      out->width = width;
      fan(out, r, c);
      c += n;
      if (c == row_bytes) {
        c = 0;
        ++r;
      }
      if (r == rows) live = false;
      return true;
    }
    if (row_bytes > stage_bytes || rows == 1) {  // pieces of one row
      const uint32_t n = min(stage_bytes, row_bytes - c);
      out->src = s + uint64_t(r) * sp + c;
      out->dst = d + uint64_t(r) * dp + c;
      out->rows = 1;
      out->row_bytes = n;
      out->sp = out->dp = 0;
      fan(out, r, c);
      c += n;
      if (c == row_bytes) {
        c = 0;
        ++r;
      }
    } else {  // whole rows
      const uint32_t k = min(stage_bytes / row_bytes, rows - r);
      out->src = s + uint64_t(r) * sp;
      out->dst = d + uint64_t(r) * dp;
      out->rows = k;
      out->row_bytes = row_bytes;
      out->sp = sp;
      out->dp = dp;
      fan(out, r, 0);
      r += k;
    }
    if (r == rows) live = false;
    return true;
  }
};

// Copy n bytes from shared memory (generic loads) to global memory, one warp, elements of V.
template <typename V>
__device__ __forceinline__ void warp_store_out(const unsigned char* smem, char* dst, uint32_t n, uint32_t lane) {
  const V* sv = reinterpret_cast<const V*>(smem);
  V* dv = reinterpret_cast<V*>(dst);
  const uint32_t ne = n / sizeof(V);
  uint32_t i = lane;
  for (; i + 7 * 32 < ne; i += 8 * 32) {
    V v[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) v[k] = sv[i + k * 32];
#pragma unroll
    for (int k = 0; k < 8; ++k) __stcs(dv + i + k * 32, v[k]);
  }
  for (; i < ne; i += 32) __stcs(dv + i, sv[i]);
}

__global__ void __launch_bounds__(32) bcp_tma_kernel(const bcp_tile* __restrict__ tiles, uint32_t n_tiles, uint32_t n_tail,
                                                     const void* const* __restrict__ src, void* const* __restrict__ dst,
                                                     Control* ctrl, uint32_t stage_bytes, uint32_t n_stages,
                                                     uint64_t wait_ns, uint32_t hints, const unsigned char* maps,
                                                     uint32_t test_stall) {
  extern __shared__ __align__(128) unsigned char stage_mem[];
  __shared__ __align__(8) uint64_t full[kMaxStages];
  __shared__ Chunk held[kMaxStages];
  __shared__ Fan fans[kMaxStages + 1];  // chunks in flight span at most n_stages units
  uint32_t fan_next = 0;
  const uint32_t lane = threadIdx.x;
  const uint64_t pol = policy_evict_first();
  const bool hint_st = hints >= 3, hint_ld = hints >= 4;  // 3: stores evict-first; 4: loads too
  if (lane == 0) {
    for (uint32_t i = 0; i < n_stages; ++i) mbar_init(smem_u32(&full[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  TileCursor cur;
  cur.live = false;
  uint32_t pending = 0;  // lane 0: the next ticket, drawn one tile ahead so that its latency is hidden
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
  bool drained = false;  // no more tickets
  bool failed = false;

  // returns false when the work list is exhausted
  auto produce = [&](Chunk* ch) -> bool {
    while (!cur.live) {
      if (drained) return false;
      const uint32_t ticket = __shfl_sync(0xffffffffu, pending, 0);
      if (ticket >= n_tiles + n_tail) {
        drained = true;
        return false;
      }
      const bcp_tile* t = tiles + ticket;
      if (ticket >= n_tiles) {  // a unit of the tail: copied through registers, here and now
        if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
        const bcp_tile u = load_tile(t);
        copy_tile<2, 1, 32>(u, src, dst, lane);
        continue;
      }
      const uint4 e = __ldg(reinterpret_cast<const uint4*>(t) + 3);  // flags, reserved[0..2]
      if (e.x & BCP_TILE_FOLLOW) {  // written by the CTA that stages the head of its group
        if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
        continue;
      }
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(t));
      const uint4 b = __ldg(reinterpret_cast<const uint4*>(t) + 1);
      const uint4 c = __ldg(reinterpret_cast<const uint4*>(t) + 2);
      cur.s = static_cast<const char*>(src[c.z]) + (uint64_t(a.x) | (uint64_t(a.y) << 32));
      cur.d = static_cast<char*>(dst[c.w]) + (uint64_t(a.z) | (uint64_t(a.w) << 32));
      cur.sp = uint64_t(b.x) | (uint64_t(b.y) << 32);
      cur.dp = uint64_t(b.z) | (uint64_t(b.w) << 32);
      cur.row_bytes = c.x;
      cur.rows = c.y;
      cur.r = cur.c = 0;
      cur.live = cur.rows > 0 && cur.row_bytes > 0;
      // a piece that is not 16-byte aligned on both sides, in length and in its pitches is staged shifted
      const uint32_t all = a.x | a.z | c.x | b.x | b.z;  // low bits (bases are 16-byte aligned)
      cur.width = 0;
      if (all & 15) cur.width = (all & 1) ? 1 : (all & 2) ? 2 : (all & 4) ? 3 : 4;
      if (e.x & BCP_TILE_TMA2D) {  // s / d name the rectangle's descriptors instead of addresses
        cur.width = kTensor;
        cur.s = reinterpret_cast<const char*>(maps + uint64_t(e.y - 1) * 256);
        cur.d = const_cast<char*>(cur.s) + 128;
        cur.row0 = e.z;
        cur.box_rows = e.w;
        if (lane == 0) {
          tensormap_acquire(cur.s);
          tensormap_acquire(cur.d);
        }
      }
      // followers: the head's flags say how many of the units right behind it read the same source bytes
      cur.nf = (e.x >> BCP_TILE_FAN_SHIFT) & 7u;
      if (cur.nf) {
        cur.slot = fan_next;
        fan_next = fan_next == n_stages ? 0 : fan_next + 1;
        if (lane < cur.nf) {
          const bcp_tile* f = tiles + ticket + 1 + lane;
          const uint4 fe = __ldg(reinterpret_cast<const uint4*>(f) + 3);
          const uint4 fa = __ldg(reinterpret_cast<const uint4*>(f));
          const uint4 fb = __ldg(reinterpret_cast<const uint4*>(f) + 1);
          const uint4 fc = __ldg(reinterpret_cast<const uint4*>(f) + 2);
          Fan& fn = fans[cur.slot];
          fn.pitch[lane] = uint64_t(fb.z) | (uint64_t(fb.w) << 32);
          if (fe.x & BCP_TILE_TMA2D) {
            fn.dst[lane] = const_cast<char*>(reinterpret_cast<const char*>(maps + uint64_t(fe.y - 1) * 256 + 128));
            fn.row0[lane] = fe.z;
            tensormap_acquire(fn.dst[lane]);
          } else {
            fn.dst[lane] = static_cast<char*>(dst[fc.w]) + (uint64_t(fa.z) | (uint64_t(fa.w) << 32));
            fn.row0[lane] = 0;
          }
        }
        __syncwarp();
      }
      if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);  // consumed when this tile is used up
    }
    return cur.next(stage_bytes, ch);
  };

  uint32_t issued = 0, stored = 0;  // chunks whose load / store has been issued
  auto issue_load = [&](uint32_t stage, const Chunk& ch) {
    const uint32_t bar = smem_u32(&full[stage]);
    const uint32_t base = smem_u32(stage_mem) + stage * stage_bytes;
    if (ch.width == kTensor) {  // one box; the transaction count is the full box even when it is clipped
      if (lane == 0) {
        held[stage] = ch;
        mbar_expect_tx(bar, ch.rows * ch.row_bytes);
        tensor_load_2d(base, ch.src, 0, int(ch.shift), bar);
      }
      __syncwarp();
      return;
    }
    if (ch.width > kShiftedRows) {  // shifted rows: one superset per row, each into its own slot
      uint32_t mine = 0;
      for (uint32_t r = lane; r < ch.rows; r += 32) {
        const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(ch.src + uint64_t(r) * ch.sp) & 15);
        mine += (sh + ch.row_bytes + 15u) & ~15u;
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
      if (lane == 0) {
        held[stage] = ch;
        mbar_expect_tx(bar, mine);
      }
      __syncwarp();
      for (uint32_t r = lane; r < ch.rows; r += 32) {
        const char* a = ch.src + uint64_t(r) * ch.sp;
        const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(a) & 15);
        bulk_load(base + r * ch.shift, a - sh, (sh + ch.row_bytes + 15u) & ~15u, bar);
      }
      return;
    }
    if (ch.width) {  // aligned superset of a shifted run, one bulk copy
      const uint32_t bytes = (ch.shift + ch.row_bytes + 15u) & ~15u;
      if (lane == 0) {
        held[stage] = ch;
        mbar_expect_tx(bar, bytes);
        bulk_load(base, ch.src - ch.shift, bytes, bar);
      }
      __syncwarp();
      return;
    }
    if (lane == 0) {
      held[stage] = ch;
      // test hook: the very first stage of CTA 0 is armed for 16 bytes that never arrive
      mbar_expect_tx(bar, ch.rows * ch.row_bytes + ((test_stall && blockIdx.x == 0 && issued == 0) ? 16u : 0u));
    }
    __syncwarp();
    for (uint32_t r = lane; r < ch.rows; r += 32) {
      if (hint_ld) {
        bulk_load_hint(base + r * ch.row_bytes, ch.src + uint64_t(r) * ch.sp, ch.row_bytes, bar, pol);
      } else {
        bulk_load(base + r * ch.row_bytes, ch.src + uint64_t(r) * ch.sp, ch.row_bytes, bar);
      }
    }
  };

  Chunk ch;
  while (issued + 1 < n_stages && produce(&ch)) {  // prologue: S-1 loads in flight
    issue_load(issued % n_stages, ch);
    ++issued;
  }
  while (stored < issued) {
    const uint32_t stage = stored % n_stages;
    const uint32_t parity = (stored / n_stages) & 1;
    const uint32_t bar = smem_u32(&full[stage]);
    if (!mbar_try_wait(bar, parity)) {  // bounded by the global timer, whatever one poll costs
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(bar, parity)) {
        if (global_timer_ns() - t0 > wait_ns) {
          failed = true;
          break;
        }
      }
    }
    if (failed) {
      // give the loads still in flight a bounded chance to land before the CTA leaves
      const uint64_t t0 = global_timer_ns();
      for (uint32_t k = stored + 1; k < issued; ++k) {
        const uint32_t b2 = smem_u32(&full[k % n_stages]);
        while (!mbar_try_wait(b2, (k / n_stages) & 1) && global_timer_ns() - t0 <= wait_ns) {
        }
      }
      break;
    }
    __syncwarp();
    const Chunk h = held[stage];
    const uint32_t base = smem_u32(stage_mem) + stage * stage_bytes;
    // the head's target, then every follower's, all from the same staged bytes
    for (uint32_t m = 0; m <= h.nf; ++m) {
      char* mdst = h.dst;
      uint64_t mdp = h.dp;
      uint32_t mrow = h.shift;
      if (m) {
        const Fan& fn = fans[h.slot];
        mdp = fn.pitch[m - 1];
        mdst = fn.dst[m - 1];
        if (h.width == kTensor) {
          mrow = fn.row0[m - 1] + h.r0;
        } else {
          mdst += uint64_t(h.r0) * mdp + h.c0;
        }
      }
      if (h.width == kTensor) {
        if (lane == 0) tensor_store_2d(mdst, 0, int(mrow), base);
      } else if (h.width > kShiftedRows) {  // shifted rows: the warp copies row after row out of its slot
        for (uint32_t r = 0; r < h.rows; ++r) {
          const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(h.src + uint64_t(r) * h.sp) & 15);
          const unsigned char* p = stage_mem + stage * stage_bytes + r * h.shift + sh;
          char* q = mdst + uint64_t(r) * mdp;
          switch (h.width - kShiftedRows) {
            case 4: warp_store_out<uint2>(p, q, h.row_bytes, lane); break;
            case 3: warp_store_out<unsigned int>(p, q, h.row_bytes, lane); break;
            case 2: warp_store_out<unsigned short>(p, q, h.row_bytes, lane); break;
            default: warp_store_out<unsigned char>(p, q, h.row_bytes, lane); break;
          }
        }
      } else if (h.width) {  // shifted run: the warp copies the payload out of the stage
        const unsigned char* p = stage_mem + stage * stage_bytes + h.shift;
        switch (h.width) {
          case 4: warp_store_out<uint2>(p, mdst, h.row_bytes, lane); break;
          case 3: warp_store_out<unsigned int>(p, mdst, h.row_bytes, lane); break;
          case 2: warp_store_out<unsigned short>(p, mdst, h.row_bytes, lane); break;
          default: warp_store_out<unsigned char>(p, mdst, h.row_bytes, lane); break;
        }
      } else {  // aligned rows: one bulk store per row
        for (uint32_t r = lane; r < h.rows; r += 32) {
          if (hint_st) {
            bulk_store_hint(mdst + uint64_t(r) * mdp, base + r * h.row_bytes, h.row_bytes, pol);
          } else {
            bulk_store(mdst + uint64_t(r) * mdp, base + r * h.row_bytes, h.row_bytes);
          }
        }
      }
    }
    if (h.width && h.width != kTensor) __syncwarp();
    bulk_commit();
    ++stored;
    // the stage of the previous store is free once that store has read its shared memory
    bulk_wait_read<1>();
    __syncwarp();
    if (produce(&ch)) {
      issue_load(issued % n_stages, ch);
      ++issued;
    }
  }
  bulk_wait_all();
  __syncwarp();
  if (lane == 0) {
    if (failed) atomicExch(&ctrl->status, uint32_t(BCP_ERR_DEVICE_TIMEOUT));
    // tickets: every CTA draws until it sees one past the end; a CTA that gave up early may
    // hold an unprocessed ticket, which the status word reports
    __threadfence();
    const uint32_t left = atomicAdd(&ctrl->done, 1u);
    if (left == gridDim.x - 1) {
      ctrl->ticket = 0;
      ctrl->done = 0;
      __threadfence();
    }
  }
}

}  // namespace

cudaError_t tma_kernel_max_grid(uint32_t stage_bytes, uint32_t n_stages, uint32_t ctas_per_sm, uint32_t* grid) {
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  const size_t smem = size_t(stage_bytes) * n_stages;
  // The opt-in limit is a property of the kernel, not of a plan: raise it to the device maximum
  // once, so that plans with different ring sizes can be executed in any order.
  int optin = 0;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, bcp_tma_kernel);
  if (e != cudaSuccess) return e;
  const int room = optin - int(fa.sharedSizeBytes);  // what the kernel's static shared memory leaves
  if (room <= 0 || smem > size_t(room)) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(bcp_tma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, room);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_tma_kernel, 32, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  const uint32_t k = ctas_per_sm < uint32_t(per_sm) ? ctas_per_sm : uint32_t(per_sm);
  *grid = uint32_t(sms) * k;
  return cudaSuccess;
}

cudaError_t launch_tma(const TmaLaunchArgs& a, cudaStream_t stream) {
  if (a.n_tiles == 0) return cudaSuccess;
  if (a.n_stages < 2 || a.n_stages > kMaxStages || a.stage_bytes % 128 || a.stage_bytes == 0) return cudaErrorInvalidValue;
  const size_t smem = size_t(a.stage_bytes) * a.n_stages;
  bcp_tma_kernel<<<a.grid, 32, smem, stream>>>(a.tiles, a.n_tiles, a.n_tail, a.src, a.dst, a.ctrl, a.stage_bytes, a.n_stages,
                                               a.wait_ns, a.cache_hints, static_cast<const unsigned char*>(a.maps),
                                               a.test_stall);
  return cudaGetLastError();
}

}  // namespace bcp
