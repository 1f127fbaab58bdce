// Converting copy for sm_100a: work units that change the element type while they move it
// (binary32 -> bfloat16 with round-to-nearest-even, bfloat16 -> binary32 exactly).
//
// The paper's resharding moves bytes only; these kernels serve plans built with
// bcp_plan_opts.convert (fp32 master weights handed to a bf16 evaluation job and back).
// HBM-bound like the plain copy: 6 bytes of traffic per element.
//
// Two kernels share the row loops below, which differ only in where the source row lies:
//
//   bcp_convert_staged_kernel  units marked BCP_TILE_TMA (source rows of at least
//       tma_min_row_bytes whose 16-byte aligned supersets stay inside the source buffer).
//       Persistent one-warp CTAs with a ring of shared-memory stages, like the staging copy
//       kernel: lanes issue one cp.async.bulk per row for the aligned superset of the source
//       rows of a chunk, completion is counted on the stage's mbarrier (bounded wait), and the
//       warp converts the rows out of shared memory with 16-byte streaming stores while the
//       loads of the next stages are in flight.  No registers hold data in flight across the
//       DRAM latency, so a few warps per SM keep the memory system full.
//   bcp_convert_kernel  every other converting unit (short rows, small jobs).  Persistent grid
//       of 256-thread CTAs; every warp is a worker of its own that draws units from an atomic
//       ticket counter (next unit's record in flight during the current one) and reads the
//       source rows with streaming global loads.
//
// A row is converted in three parts: leading elements until the 16-byte side is aligned, a
// body of wide groups, and the rest element by element.  Narrowing: 8 elements per group (two
// 16-byte loads, one 16-byte store).  Widening: 4 elements per group (one 8-byte load, one
// 16-byte store, so a warp writes 512 contiguous bytes per instruction).  When the two sides
// cannot be aligned together the body runs on pairs of elements (8-byte / 4-byte accesses,
// still fully coalesced).  Four groups per lane are in flight.
#include "kernels.cuh"
#include "tma_ptx.cuh"

namespace bcp {
namespace {

// binary32 bits -> bfloat16 bits: nearest, ties to even; NaN -> 0x7FC0.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(uint32_t x) {
  if ((x & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u;
  return (x + 0x7FFFu + ((x >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ uint32_t pack2_exact(uint32_t lo, uint32_t hi) { return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16); }
__device__ __noinline__ uint4 narrow8_exact(uint4 a, uint4 b) {
  return make_uint4(pack2_exact(a.x, a.y), pack2_exact(a.z, a.w), pack2_exact(b.x, b.y), pack2_exact(b.z, b.w));
}
// Two / eight values at once.  The hardware conversion (one instruction per pair) rounds to
// nearest even, keeps subnormals and overflows to infinity exactly like the integer form above;
// only what it makes of a NaN is not ours to choose, so a group with a NaN in it (one predicate
// per group, never taken on real weights) is redone in the integer form, out of line.
__device__ __forceinline__ uint32_t pack2(uint32_t lo, uint32_t hi) {
  uint32_t out, any_nan;
  asm("{\n\t.reg .pred p;\n\t"
      "setp.nan.f32 p, %2, %3;\n\t"
      "cvt.rn.bf16x2.f32 %0, %3, %2;\n\t"
      "selp.u32 %1, 1, 0, p;\n\t}"
      : "=r"(out), "=r"(any_nan)
      : "f"(__uint_as_float(lo)), "f"(__uint_as_float(hi)));
  if (__builtin_expect(any_nan != 0, 0)) out = narrow8_exact(make_uint4(lo, hi, 0, 0), make_uint4(0, 0, 0, 0)).x;
  return out;
}
__device__ __forceinline__ uint4 narrow8(uint4 a, uint4 b) {
  uint4 o;
  uint32_t any_nan;
  asm("{\n\t.reg .pred p;\n\t"
      "setp.nan.f32 p, %5, %6;\n\t"
      "setp.nan.or.f32 p, %7, %8, p;\n\t"
      "setp.nan.or.f32 p, %9, %10, p;\n\t"
      "setp.nan.or.f32 p, %11, %12, p;\n\t"
      "cvt.rn.bf16x2.f32 %0, %6, %5;\n\t"
      "cvt.rn.bf16x2.f32 %1, %8, %7;\n\t"
      "cvt.rn.bf16x2.f32 %2, %10, %9;\n\t"
      "cvt.rn.bf16x2.f32 %3, %12, %11;\n\t"
      "selp.u32 %4, 1, 0, p;\n\t}"
      : "=r"(o.x), "=r"(o.y), "=r"(o.z), "=r"(o.w), "=r"(any_nan)
      : "f"(__uint_as_float(a.x)), "f"(__uint_as_float(a.y)), "f"(__uint_as_float(a.z)), "f"(__uint_as_float(a.w)),
        "f"(__uint_as_float(b.x)), "f"(__uint_as_float(b.y)), "f"(__uint_as_float(b.z)), "f"(__uint_as_float(b.w)));
  if (__builtin_expect(any_nan != 0, 0)) o = narrow8_exact(a, b);
  return o;
}

// Where a source row is read from.
struct FromGlobal {  // read once: bypass L1
  static __device__ __forceinline__ uint4 ld16(const char* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
  }
  static __device__ __forceinline__ uint2 ld8(const char* p) {
    uint2 v;
    asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
    return v;
  }
  static __device__ __forceinline__ uint32_t ld4(const char* p) {
    uint32_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
    return v;
  }
  static __device__ __forceinline__ uint32_t ld2(const char* p) {
    uint16_t v;
    asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
    return v;
  }
};
struct FromShared {  // a stage filled by bulk copies (p is a generic pointer into shared memory)
  static __device__ __forceinline__ uint4 ld16(const char* p) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(smem_u32(p)));
    return v;
  }
  static __device__ __forceinline__ uint2 ld8(const char* p) {
    uint2 v;
    asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(smem_u32(p)));
    return v;
  }
  static __device__ __forceinline__ uint32_t ld4(const char* p) {
    uint32_t v;
    asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)));
    return v;
  }
  static __device__ __forceinline__ uint32_t ld2(const char* p) {
    uint16_t v;
    asm volatile("ld.shared.u16 %0, [%1];" : "=h"(v) : "r"(smem_u32(p)));
    return v;
  }
};

// ---- binary32 -> bfloat16: n elements from s (4-byte aligned) to d (2-byte aligned), one warp
template <class L>
__device__ __noinline__ void narrow_row(const char* __restrict__ s, char* __restrict__ d, uint64_t n, uint32_t lane) {
  // leading elements until d is 16-byte aligned; if s is not 16-byte aligned there, the body
  // runs on pairs, which only need d 4-byte aligned
  uint64_t lead = ((16 - (reinterpret_cast<uintptr_t>(d) & 15)) & 15) >> 1;
  const bool wide = lead <= n && ((reinterpret_cast<uintptr_t>(s) + 4 * lead) & 15) == 0;
  if (!wide) lead = (reinterpret_cast<uintptr_t>(d) >> 1) & 1;
  if (lead > n) lead = n;
  if (lane < lead) *reinterpret_cast<uint16_t*>(d + 2 * lane) = uint16_t(f32_to_bf16_bits(L::ld4(s + 4 * lane)));
  s += 4 * lead, d += 2 * lead, n -= lead;
  uint64_t done = 0;
  if (wide) {
    const uint64_t groups = n >> 3;  // 8 elements: 32 bytes in, 16 bytes out
    for (uint64_t g = lane; g < groups; g += 128) {  // four groups per lane in flight (the last round may hold fewer)
      uint4 a[4], b[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (g + 32 * k < groups) {
          a[k] = L::ld16(s + (g + 32 * k) * 32);
          b[k] = L::ld16(s + (g + 32 * k) * 32 + 16);
        }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (g + 32 * k < groups) __stcs(reinterpret_cast<uint4*>(d + (g + 32 * k) * 16), narrow8(a[k], b[k]));
    }
    done = groups << 3;
  } else {
    const uint64_t pairs = n >> 1;
    const bool s8 = (reinterpret_cast<uintptr_t>(s) & 7) == 0;
    uint64_t p = lane;
    for (; p + 96 < pairs; p += 128) {
      uint2 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const char* q = s + (p + 32 * k) * 8;
        v[k] = s8 ? L::ld8(q) : make_uint2(L::ld4(q), L::ld4(q + 4));
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) __stcs(reinterpret_cast<uint32_t*>(d + (p + 32 * k) * 4), pack2(v[k].x, v[k].y));
    }
    for (; p < pairs; p += 32) {
      const char* q = s + p * 8;
      const uint2 v = s8 ? L::ld8(q) : make_uint2(L::ld4(q), L::ld4(q + 4));
      __stcs(reinterpret_cast<uint32_t*>(d + p * 4), pack2(v.x, v.y));
    }
    done = pairs << 1;
  }
  for (uint64_t i = done + lane; i < n; i += 32) *reinterpret_cast<uint16_t*>(d + 2 * i) = uint16_t(f32_to_bf16_bits(L::ld4(s + 4 * i)));
}

// ---- bfloat16 -> binary32: n elements from s (2-byte aligned) to d (4-byte aligned), one warp
template <class L>
__device__ __noinline__ void widen_row(const char* __restrict__ s, char* __restrict__ d, uint64_t n, uint32_t lane) {
  // leading elements until d is 16-byte aligned; if s is not 8-byte aligned there, the body
  // runs on pairs, which only need s 4-byte aligned
  uint64_t lead = ((16 - (reinterpret_cast<uintptr_t>(d) & 15)) & 15) >> 2;
  const bool wide = lead <= n && ((reinterpret_cast<uintptr_t>(s) + 2 * lead) & 7) == 0;
  if (!wide) lead = (reinterpret_cast<uintptr_t>(s) >> 1) & 1;
  if (lead > n) lead = n;
  if (lane < lead) *reinterpret_cast<uint32_t*>(d + 4 * lane) = L::ld2(s + 2 * lane) << 16;
  s += 2 * lead, d += 4 * lead, n -= lead;
  uint64_t done = 0;
  if (wide) {
    const uint64_t groups = n >> 2;  // 4 elements: 8 bytes in, 16 bytes out, both contiguous across the warp
    for (uint64_t g = lane; g < groups; g += 128) {
      uint2 a[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (g + 32 * k < groups) a[k] = L::ld8(s + (g + 32 * k) * 8);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (g + 32 * k < groups)
          __stcs(reinterpret_cast<uint4*>(d + (g + 32 * k) * 16),
                 make_uint4(a[k].x << 16, a[k].x & 0xFFFF0000u, a[k].y << 16, a[k].y & 0xFFFF0000u));
    }
    done = groups << 2;
  } else {
    const uint64_t pairs = n >> 1;
    const bool d8 = (reinterpret_cast<uintptr_t>(d) & 7) == 0;
    uint64_t p = lane;
    for (; p + 96 < pairs; p += 128) {
      uint32_t v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = L::ld4(s + (p + 32 * k) * 4);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        char* q = d + (p + 32 * k) * 8;
        if (d8) {
          __stcs(reinterpret_cast<uint2*>(q), make_uint2(v[k] << 16, v[k] & 0xFFFF0000u));
        } else {
          __stcs(reinterpret_cast<uint32_t*>(q), v[k] << 16);
          __stcs(reinterpret_cast<uint32_t*>(q + 4), v[k] & 0xFFFF0000u);
        }
      }
    }
    for (; p < pairs; p += 32) {
      const uint32_t v = L::ld4(s + p * 4);
      char* q = d + p * 8;
      if (d8) {
        __stcs(reinterpret_cast<uint2*>(q), make_uint2(v << 16, v & 0xFFFF0000u));
      } else {
        __stcs(reinterpret_cast<uint32_t*>(q), v << 16);
        __stcs(reinterpret_cast<uint32_t*>(q + 4), v & 0xFFFF0000u);
      }
    }
    done = pairs << 1;
  }
  for (uint64_t i = done + lane; i < n; i += 32) *reinterpret_cast<uint32_t*>(d + 4 * i) = L::ld2(s + 2 * i) << 16;
}

struct Unit {
  uint64_t src_off, dst_off, src_pitch, dst_pitch;
  uint32_t row_bytes, rows, src_buf, dst_buf, flags;
};
__device__ __forceinline__ Unit load_unit(const bcp_tile* p) {
  const uint4* q = reinterpret_cast<const uint4*>(p);
  const uint4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
  Unit t;
  t.src_off = uint64_t(a.x) | (uint64_t(a.y) << 32);
  t.dst_off = uint64_t(a.z) | (uint64_t(a.w) << 32);
  t.src_pitch = uint64_t(b.x) | (uint64_t(b.y) << 32);
  t.dst_pitch = uint64_t(b.z) | (uint64_t(b.w) << 32);
  t.row_bytes = c.x;
  t.rows = c.y;
  t.src_buf = c.z;
  t.dst_buf = c.w;
  t.flags = __ldg(&p->flags);
  return t;
}

__device__ __forceinline__ void convert_unit(const Unit& t, const void* const* __restrict__ src, void* const* __restrict__ dst,
                                             uint32_t lane) {
  const char* s = static_cast<const char*>(src[t.src_buf]) + t.src_off;
  char* d = static_cast<char*>(dst[t.dst_buf]) + t.dst_off;
  const uint32_t kind = (t.flags & BCP_TILE_CVT_MASK) >> BCP_TILE_CVT_SHIFT;
  for (uint32_t r = 0; r < t.rows; ++r) {
    if (kind == BCP_CONVERT_F32_TO_BF16) {
      narrow_row<FromGlobal>(s + r * t.src_pitch, d + r * t.dst_pitch, t.row_bytes >> 1, lane);
    } else {
      widen_row<FromGlobal>(s + r * t.src_pitch, d + r * t.dst_pitch, t.row_bytes >> 2, lane);
    }
  }
}

__global__ void __launch_bounds__(256, 4) bcp_convert_kernel(const bcp_tile* __restrict__ tiles, uint32_t n_units,
                                                             const void* const* __restrict__ src, void* const* __restrict__ dst,
                                                             Control* ctrl) {
  const uint32_t lane = threadIdx.x & 31;
  uint32_t pending = 0;  // lane 0: ticket drawn but not yet used
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
  uint32_t u = __shfl_sync(0xffffffffu, pending, 0);
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
  Unit t;
  if (u < n_units) t = load_unit(tiles + u);
  while (u < n_units) {
    const uint32_t next = __shfl_sync(0xffffffffu, pending, 0);
    if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);  // for the unit after the next
    Unit tn;
    if (next < n_units) tn = load_unit(tiles + next);  // in flight while this unit is converted
    if (!(t.flags & BCP_TILE_TMA)) convert_unit(t, src, dst, lane);  // marked units belong to the staged kernel
    u = next;
    t = tn;
  }
  // the last warp to leave rewinds the counters so that the next launch starts from zero
  if (lane == 0) {
    __threadfence();
    const uint32_t left = atomicAdd(&ctrl->done, 1u);
    if (left == gridDim.x * (blockDim.x >> 5) - 1) {
      ctrl->ticket = 0;
      ctrl->done = 0;
      __threadfence();
    }
  }
}

// Several short rows of a stage at once (narrowing, every row 16-byte aligned in shared memory and
// at the target, whole 8-element groups): four rows are in flight per lane, so rows far shorter
// than what one warp covers in a round still keep several loads outstanding.
__device__ __forceinline__ void narrow_rows_aligned(const char* base, uint32_t slot, char* d, uint64_t dp, uint32_t rows,
                                                    uint32_t groups_per_row, uint32_t lane) {
  for (uint32_t r = 0; r < rows; r += 4) {
    for (uint32_t c = lane; c < groups_per_row; c += 32) {
      uint4 a[4], b[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k < rows) {
          a[k] = FromShared::ld16(base + (r + k) * slot + c * 32);
          b[k] = FromShared::ld16(base + (r + k) * slot + c * 32 + 16);
        }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (r + k < rows) __stcs(reinterpret_cast<uint4*>(d + uint64_t(r + k) * dp + c * 16), narrow8(a[k], b[k]));
    }
  }
}

// ------------------------------------------------------------------------------ staged form
struct CvtChunk {  // what one stage holds: `rows` source rows of `ne` elements, each in a slot of `slot` bytes
  const char* src;  // first element of the first row (global)
  char* dst;
  uint64_t sp, dp;
  uint32_t rows, ne, slot, kind;
};

__global__ void __launch_bounds__(32) bcp_convert_staged_kernel(const bcp_tile* __restrict__ tiles, uint32_t n_units,
                                                                const void* const* __restrict__ src, void* const* __restrict__ dst,
                                                                Control* ctrl, uint32_t stage_bytes, uint32_t n_stages,
                                                                uint64_t wait_ns, uint32_t test_stall) {
  extern __shared__ __align__(128) unsigned char stage_mem[];
  __shared__ __align__(8) uint64_t full[kMaxStages];
  __shared__ CvtChunk held[kMaxStages];
  const uint32_t lane = threadIdx.x;
  if (lane == 0) {
    for (uint32_t i = 0; i < n_stages; ++i) mbar_init(smem_u32(&full[i]), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncwarp();

  // the unit being cut into chunks (all lanes hold the same state)
  const char* us = nullptr;
  char* ud = nullptr;
  uint64_t usp = 0, udp = 0;
  uint32_t urows = 0, une = 0, ur = 0, uc = 0, ukind = 0;
  bool live = false, drained = false, failed = false;
  uint32_t pending = 0;  // lane 0: the next ticket, drawn one unit ahead
  if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);

  auto produce = [&](CvtChunk* ch) -> bool {
    while (!live) {
      if (drained) return false;
      const uint32_t ticket = __shfl_sync(0xffffffffu, pending, 0);
      if (ticket >= n_units) {
        drained = true;
        return false;
      }
      if (lane == 0) pending = atomicAdd(&ctrl->ticket, 1u);
      const bcp_tile* t = tiles + ticket;
      const uint4 e = __ldg(reinterpret_cast<const uint4*>(t) + 3);  // flags, reserved
      if (!(e.x & BCP_TILE_TMA)) continue;                           // the register kernel's unit
      const uint4 a = __ldg(reinterpret_cast<const uint4*>(t));
      const uint4 b = __ldg(reinterpret_cast<const uint4*>(t) + 1);
      const uint4 c = __ldg(reinterpret_cast<const uint4*>(t) + 2);
      ukind = (e.x & BCP_TILE_CVT_MASK) >> BCP_TILE_CVT_SHIFT;
      us = static_cast<const char*>(src[c.z]) + (uint64_t(a.x) | (uint64_t(a.y) << 32));
      ud = static_cast<char*>(dst[c.w]) + (uint64_t(a.z) | (uint64_t(a.w) << 32));
      usp = uint64_t(b.x) | (uint64_t(b.y) << 32);
      udp = uint64_t(b.z) | (uint64_t(b.w) << 32);
      une = ukind == BCP_CONVERT_F32_TO_BF16 ? c.x >> 1 : c.x >> 2;  // row_bytes counts target bytes
      urows = c.y;
      ur = uc = 0;
      live = urows > 0 && une > 0;
    }
    const uint32_t s_isz = ukind == BCP_CONVERT_F32_TO_BF16 ? 4u : 2u, d_isz = 6u - s_isz;
    const uint32_t slot = (une * s_isz + 45u) & ~15u;  // room for the aligned superset of a row, whatever its shift
    ch->kind = ukind;
    if (urows > 1 && slot <= stage_bytes) {  // several whole rows, one slot each
      const uint32_t k = min(stage_bytes / slot, urows - ur);
      ch->src = us + uint64_t(ur) * usp;
      ch->dst = ud + uint64_t(ur) * udp;
      ch->sp = usp, ch->dp = udp;
      ch->rows = k, ch->ne = une, ch->slot = slot;
      ur += k;
    } else {  // pieces of one row; a multiple of 8 elements keeps the alignment phase of both sides
      const uint32_t cap = ((stage_bytes - 32u) / s_isz) & ~7u;
      const uint32_t n = min(cap, une - uc);
      ch->src = us + uint64_t(ur) * usp + uint64_t(uc) * s_isz;
      ch->dst = ud + uint64_t(ur) * udp + uint64_t(uc) * d_isz;
      ch->sp = ch->dp = 0;
      ch->rows = 1, ch->ne = n, ch->slot = stage_bytes;
      uc += n;
      if (uc == une) uc = 0, ++ur;
    }
    if (ur == urows) live = false;
    return true;
  };

  bool first_load = true;
  auto issue_load = [&](uint32_t stage, const CvtChunk& ch) {
    const uint32_t bar = smem_u32(&full[stage]);
    const uint32_t base = smem_u32(stage_mem) + stage * stage_bytes;
    const uint32_t row_src = ch.ne * (ch.kind == BCP_CONVERT_F32_TO_BF16 ? 4u : 2u);
    uint32_t mine = 0;
    for (uint32_t r = lane; r < ch.rows; r += 32) {
      const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(ch.src + uint64_t(r) * ch.sp) & 15);
      mine += (sh + row_src + 15u) & ~15u;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
    if (lane == 0) {
      held[stage] = ch;
      // test hook: the very first stage of CTA 0 is armed for 16 bytes that never arrive
      mbar_expect_tx(bar, mine + ((test_stall && blockIdx.x == 0 && first_load) ? 16u : 0u));
    }
    first_load = false;
    __syncwarp();
    for (uint32_t r = lane; r < ch.rows; r += 32) {
      const char* a = ch.src + uint64_t(r) * ch.sp;
      const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(a) & 15);
      bulk_load(base + r * ch.slot, a - sh, (sh + row_src + 15u) & ~15u, bar);
    }
  };

  uint32_t issued = 0, consumed = 0;
  CvtChunk ch;
  while (issued + 1 < n_stages && produce(&ch)) {  // prologue: S-1 loads in flight
    issue_load(issued % n_stages, ch);
    ++issued;
  }
  while (consumed < issued) {
    const uint32_t stage = consumed % n_stages;
    const uint32_t parity = (consumed / n_stages) & 1;
    const uint32_t bar = smem_u32(&full[stage]);
    if (!mbar_try_wait(bar, parity)) {  // bounded by the global timer
      const uint64_t t0 = global_timer_ns();
      while (!mbar_try_wait(bar, parity)) {
        if (global_timer_ns() - t0 > wait_ns) {
          failed = true;
          break;
        }
      }
    }
    if (failed) {  // give the loads still in flight a bounded chance to land before the CTA leaves
      const uint64_t t0 = global_timer_ns();
      for (uint32_t k = consumed + 1; k < issued; ++k) {
        const uint32_t b2 = smem_u32(&full[k % n_stages]);
        while (!mbar_try_wait(b2, (k / n_stages) & 1) && global_timer_ns() - t0 <= wait_ns) {
        }
      }
      break;
    }
    __syncwarp();
    // refill the stage that was freed by the previous iteration before converting this one
    if (produce(&ch)) {
      issue_load(issued % n_stages, ch);
      ++issued;
    }
    const CvtChunk h = held[stage];
    const char* stage_base = reinterpret_cast<const char*>(stage_mem) + stage * stage_bytes;
    const bool quads = h.rows > 1 && h.kind == BCP_CONVERT_F32_TO_BF16 && (h.ne & 7) == 0 &&
                       ((reinterpret_cast<uintptr_t>(h.src) | reinterpret_cast<uintptr_t>(h.dst) | h.sp | h.dp) & 15) == 0;
    if (quads) narrow_rows_aligned(stage_base, h.slot, h.dst, h.dp, h.rows, h.ne >> 3, lane);
    for (uint32_t r = quads ? h.rows : 0; r < h.rows; ++r) {
      const uint32_t sh = uint32_t(reinterpret_cast<uintptr_t>(h.src + uint64_t(r) * h.sp) & 15);
      const char* p = stage_base + r * h.slot + sh;
      char* q = h.dst + uint64_t(r) * h.dp;
      if (h.kind == BCP_CONVERT_F32_TO_BF16) {
        narrow_row<FromShared>(p, q, h.ne, lane);
      } else {
        widen_row<FromShared>(p, q, h.ne, lane);
      }
    }
    __syncwarp();  // every lane has read its part of the stage: it may be overwritten
    ++consumed;
  }
  __syncwarp();
  if (lane == 0) {
    if (failed) atomicExch(&ctrl->status, uint32_t(BCP_ERR_DEVICE_TIMEOUT));
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

cudaError_t convert_kernel_max_grid(uint32_t* grid) {
  int dev = 0, sms = 0, per_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_convert_kernel, 256, 0);
  if (e != cudaSuccess) return e;
  if (per_sm > 4) per_sm = 4;
  *grid = uint32_t(sms) * uint32_t(per_sm > 0 ? per_sm : 1);
  return cudaSuccess;
}

cudaError_t launch_convert(const ConvertLaunchArgs& a, cudaStream_t stream) {
  if (a.n_units == 0) return cudaSuccess;
  const uint32_t ctas = (a.n_units + 7) / 8;  // 8 warps per CTA
  bcp_convert_kernel<<<ctas < a.grid ? ctas : a.grid, 256, 0, stream>>>(a.tiles, a.n_units, a.src, a.dst, a.ctrl);
  return cudaGetLastError();
}

cudaError_t convert_staged_max_grid(uint32_t stage_bytes, uint32_t n_stages, uint32_t ctas_per_sm, uint32_t* grid) {
  int dev = 0, sms = 0, per_sm = 0, optin = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  if (e != cudaSuccess) return e;
  cudaFuncAttributes fa;
  e = cudaFuncGetAttributes(&fa, bcp_convert_staged_kernel);
  if (e != cudaSuccess) return e;
  const size_t smem = size_t(stage_bytes) * n_stages;
  const int room = optin - int(fa.sharedSizeBytes);
  if (room <= 0 || smem > size_t(room)) return cudaErrorInvalidValue;
  e = cudaFuncSetAttribute(bcp_convert_staged_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, room);
  if (e != cudaSuccess) return e;
  e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, bcp_convert_staged_kernel, 32, smem);
  if (e != cudaSuccess) return e;
  if (per_sm < 1) return cudaErrorInvalidConfiguration;
  *grid = uint32_t(sms) * (ctas_per_sm < uint32_t(per_sm) ? ctas_per_sm : uint32_t(per_sm));
  return cudaSuccess;
}

cudaError_t launch_convert_staged(const ConvertStagedLaunchArgs& a, cudaStream_t stream) {
  if (a.n_units == 0) return cudaSuccess;
  if (a.n_stages < 2 || a.n_stages > uint32_t(kMaxStages) || a.stage_bytes % 128 || a.stage_bytes < 1024) return cudaErrorInvalidValue;
  const size_t smem = size_t(a.stage_bytes) * a.n_stages;
  const uint32_t grid = a.n_units < a.grid ? a.n_units : a.grid;
  bcp_convert_staged_kernel<<<grid, 32, smem, stream>>>(a.tiles, a.n_units, a.src, a.dst, a.ctrl, a.stage_bytes, a.n_stages, a.wait_ns,
                                                        a.test_stall);
  return cudaGetLastError();
}

}  // namespace bcp
