// Converting copy for sm_100a: work units that change the element type while they move it
// (binary32 -> bfloat16 with round-to-nearest-even, bfloat16 -> binary32 exactly).
//
// The paper's resharding moves bytes only; this kernel serves plans built with
// bcp_plan_opts.convert (fp32 master weights handed to a bf16 evaluation job and back).
// HBM-bound like the plain copy: 6 bytes of traffic per element.
//
// Persistent grid of 256-thread CTAs; every warp is a worker of its own that draws units
// from an atomic ticket counter (next unit's record in flight during the current one).
// A row is converted in three parts: leading elements until the 16-byte side is aligned,
// a body of 8-element groups (two 16-byte accesses on the binary32 side, one on the
// bfloat16 side, four groups in flight per lane), and the rest element by element.  When
// the two sides cannot be 16-byte aligned together the body runs on pairs of elements
// (8-byte / 4-byte accesses, still fully coalesced).
#include "kernels.cuh"

namespace bcp {
namespace {

// binary32 bits -> bfloat16 bits: nearest, ties to even; NaN -> 0x7FC0.
__device__ __forceinline__ uint32_t f32_to_bf16_bits(uint32_t x) {
  if ((x & 0x7FFFFFFFu) > 0x7F800000u) return 0x7FC0u;
  return (x + 0x7FFFu + ((x >> 16) & 1u)) >> 16;
}
__device__ __forceinline__ uint32_t pack2(uint32_t lo, uint32_t hi) { return f32_to_bf16_bits(lo) | (f32_to_bf16_bits(hi) << 16); }

__device__ __forceinline__ uint4 ld16(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ uint2 ld8(const void* p) {
  uint2 v;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld4(const void* p) {
  uint32_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u32 %0, [%1];" : "=r"(v) : "l"(p));
  return v;
}
__device__ __forceinline__ uint32_t ld2(const void* p) {
  uint16_t v;
  asm volatile("ld.global.nc.L1::no_allocate.u16 %0, [%1];" : "=h"(v) : "l"(p));
  return v;
}

// ---- binary32 -> bfloat16: n elements from s (4-byte aligned) to d (2-byte aligned), one warp
__device__ __noinline__ void narrow_row(const char* __restrict__ s, char* __restrict__ d, uint64_t n, uint32_t lane) {
  // leading elements until d is 16-byte aligned; if s is not 16-byte aligned there, the body
  // runs on pairs, which only need d 4-byte aligned
  uint64_t lead = ((16 - (reinterpret_cast<uintptr_t>(d) & 15)) & 15) >> 1;
  const bool wide = lead <= n && ((reinterpret_cast<uintptr_t>(s) + 4 * lead) & 15) == 0;
  if (!wide) lead = (reinterpret_cast<uintptr_t>(d) >> 1) & 1;
  if (lead > n) lead = n;
  if (lane < lead) *reinterpret_cast<uint16_t*>(d + 2 * lane) = uint16_t(f32_to_bf16_bits(ld4(s + 4 * lane)));
  s += 4 * lead, d += 2 * lead, n -= lead;
  uint64_t done = 0;
  if (wide) {
    const uint64_t groups = n >> 3;  // 8 elements: 32 bytes in, 16 bytes out
    uint64_t g = lane;
    for (; g + 96 < groups; g += 128) {  // four groups per lane in flight
      uint4 a[4], b[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        a[k] = ld16(s + (g + 32 * k) * 32);
        b[k] = ld16(s + (g + 32 * k) * 32 + 16);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k)
        __stcs(reinterpret_cast<uint4*>(d + (g + 32 * k) * 16),
               make_uint4(pack2(a[k].x, a[k].y), pack2(a[k].z, a[k].w), pack2(b[k].x, b[k].y), pack2(b[k].z, b[k].w)));
    }
    for (; g < groups; g += 32) {
      const uint4 a = ld16(s + g * 32), b = ld16(s + g * 32 + 16);
      __stcs(reinterpret_cast<uint4*>(d + g * 16), make_uint4(pack2(a.x, a.y), pack2(a.z, a.w), pack2(b.x, b.y), pack2(b.z, b.w)));
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
        v[k] = s8 ? ld8(q) : make_uint2(ld4(q), ld4(q + 4));
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) __stcs(reinterpret_cast<uint32_t*>(d + (p + 32 * k) * 4), pack2(v[k].x, v[k].y));
    }
    for (; p < pairs; p += 32) {
      const char* q = s + p * 8;
      const uint2 v = s8 ? ld8(q) : make_uint2(ld4(q), ld4(q + 4));
      __stcs(reinterpret_cast<uint32_t*>(d + p * 4), pack2(v.x, v.y));
    }
    done = pairs << 1;
  }
  for (uint64_t i = done + lane; i < n; i += 32) *reinterpret_cast<uint16_t*>(d + 2 * i) = uint16_t(f32_to_bf16_bits(ld4(s + 4 * i)));
}

// ---- bfloat16 -> binary32: n elements from s (2-byte aligned) to d (4-byte aligned), one warp
__device__ __noinline__ void widen_row(const char* __restrict__ s, char* __restrict__ d, uint64_t n, uint32_t lane) {
  // leading elements until s is 16-byte aligned; if d is not 16-byte aligned there, the body
  // runs on pairs, which only need s 4-byte aligned
  uint64_t lead = ((16 - (reinterpret_cast<uintptr_t>(s) & 15)) & 15) >> 1;
  const bool wide = lead <= n && ((reinterpret_cast<uintptr_t>(d) + 4 * lead) & 15) == 0;
  if (!wide) lead = (reinterpret_cast<uintptr_t>(s) >> 1) & 1;
  if (lead > n) lead = n;
  if (lane < lead) *reinterpret_cast<uint32_t*>(d + 4 * lane) = ld2(s + 2 * lane) << 16;
  s += 2 * lead, d += 4 * lead, n -= lead;
  uint64_t done = 0;
  if (wide) {
    const uint64_t groups = n >> 3;  // 8 elements: 16 bytes in, 32 bytes out
    uint64_t g = lane;
    for (; g + 96 < groups; g += 128) {
      uint4 a[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) a[k] = ld16(s + (g + 32 * k) * 16);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        char* q = d + (g + 32 * k) * 32;
        __stcs(reinterpret_cast<uint4*>(q), make_uint4(a[k].x << 16, a[k].x & 0xFFFF0000u, a[k].y << 16, a[k].y & 0xFFFF0000u));
        __stcs(reinterpret_cast<uint4*>(q + 16), make_uint4(a[k].z << 16, a[k].z & 0xFFFF0000u, a[k].w << 16, a[k].w & 0xFFFF0000u));
      }
    }
    for (; g < groups; g += 32) {
      const uint4 a = ld16(s + g * 16);
      char* q = d + g * 32;
      __stcs(reinterpret_cast<uint4*>(q), make_uint4(a.x << 16, a.x & 0xFFFF0000u, a.y << 16, a.y & 0xFFFF0000u));
      __stcs(reinterpret_cast<uint4*>(q + 16), make_uint4(a.z << 16, a.z & 0xFFFF0000u, a.w << 16, a.w & 0xFFFF0000u));
    }
    done = groups << 3;
  } else {
    const uint64_t pairs = n >> 1;
    const bool d8 = (reinterpret_cast<uintptr_t>(d) & 7) == 0;
    uint64_t p = lane;
    for (; p + 96 < pairs; p += 128) {
      uint32_t v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k) v[k] = ld4(s + (p + 32 * k) * 4);
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
      const uint32_t v = ld4(s + p * 4);
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
  for (uint64_t i = done + lane; i < n; i += 32) *reinterpret_cast<uint32_t*>(d + 4 * i) = ld2(s + 2 * i) << 16;
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
      narrow_row(s + r * t.src_pitch, d + r * t.dst_pitch, t.row_bytes >> 1, lane);
    } else {
      widen_row(s + r * t.src_pitch, d + r * t.dst_pitch, t.row_bytes >> 2, lane);
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
    convert_unit(t, src, dst, lane);
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

}  // namespace bcp
