// Register (LDG/STG) copy loops for one work unit, shared by the register kernels (kernels.cu)
// and by the staging kernel (tma_kernel.cu), whose warps execute the few units of a plan that
// cannot be staged.  A unit carries the widest power-of-two access width (1..16 bytes) that
// divides its offsets, row length and pitches; the loops are instantiated for each width and
// keep U independent loads in flight per thread before the first store.
#pragma once

#include <cstdint>

#include "bcp.h"

namespace bcp {
namespace {

// ---------------------------------------------------------------- memory access with hints
template <int HINT, typename V>
__device__ __forceinline__ V ld(const V* p) {
  if constexpr (HINT == 1) {
    if constexpr (sizeof(V) == 16) {
      uint4 v;
      asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                   : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                   : "l"(p));
      return v;
    } else {
      return __ldg(p);
    }
  } else {
    return *p;
  }
}

template <int HINT, typename V>
__device__ __forceinline__ void st(V* p, const V& v) {
  if constexpr (HINT == 1) {
    __stcs(p, v);
  } else {
    *p = v;
  }
}

template <typename V>
__device__ __forceinline__ V zero_of() {
  if constexpr (sizeof(V) == 16) {
    return make_uint4(0, 0, 0, 0);
  } else if constexpr (sizeof(V) == 8) {
    return make_uint2(0, 0);
  } else {
    return V(0);
  }
}

// ---------------------------------------------------------------- copy loops for one group
// A "group" is the set of threads that cooperate on a tile: a whole CTA (tid in [0, nt)) or
// one warp (tid = lane, nt = 32).

// contiguous run of n elements of V
template <typename V, int U, int HINT, uint32_t nt>
__device__ __forceinline__ void copy_run(const V* __restrict__ s, V* __restrict__ d, uint32_t n, uint32_t tid) {
  uint32_t base = tid;
  constexpr uint32_t step = nt * U;
  // full batches: U loads in flight, then U stores
  for (; base + (U - 1) * nt < n; base += step) {
    V v[U];
#pragma unroll
    for (int i = 0; i < U; ++i) v[i] = ld<HINT>(s + base + i * nt);
#pragma unroll
    for (int i = 0; i < U; ++i) st<HINT>(d + base + i * nt, v[i]);
  }
  // ragged rest
  V v[U];
#pragma unroll
  for (int i = 0; i < U; ++i)
    if (base + i * nt < n) v[i] = ld<HINT>(s + base + i * nt);
#pragma unroll
  for (int i = 0; i < U; ++i)
    if (base + i * nt < n) st<HINT>(d + base + i * nt, v[i]);
}

template <typename V, int HINT, uint32_t nt>
__device__ __forceinline__ void zero_run(V* d, uint32_t n, uint32_t tid) {
  const V z = zero_of<V>();
  for (uint32_t i = tid; i < n; i += nt) st<HINT>(d + i, z);
}

// rows x re elements with byte pitches; rows of at least one warp's width: each warp takes
// 32-element chunks of a row, so a warp's accesses stay contiguous
template <typename V, int U, int HINT, uint32_t nt>
__device__ __forceinline__ void copy_rows_wide(const char* __restrict__ s, char* __restrict__ d, uint32_t rows,
                                               uint32_t re, uint64_t sp, uint64_t dp, uint32_t tid) {
  const uint32_t lane = tid & 31, w = tid >> 5;
  constexpr uint32_t nw = nt >> 5;
  const uint32_t cpr = (re + 31) >> 5;  // chunks per row
  const uint32_t nchunks = rows * cpr;
  for (uint32_t k0 = w; k0 < nchunks; k0 += nw * U) {
    V v[U];
    uint64_t doff[U];
    bool ok[U];
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const uint32_t k = k0 + i * nw;
      const uint32_t r = k / cpr;
      const uint32_t c = ((k - r * cpr) << 5) + lane;
      ok[i] = k < nchunks && c < re;
      doff[i] = uint64_t(r) * dp + uint64_t(c) * sizeof(V);
      if (ok[i]) v[i] = ld<HINT>(reinterpret_cast<const V*>(s + uint64_t(r) * sp + uint64_t(c) * sizeof(V)));
    }
#pragma unroll
    for (int i = 0; i < U; ++i)
      if (ok[i]) st<HINT>(reinterpret_cast<V*>(d + doff[i]), v[i]);
  }
}

// rows x re elements, short rows: elements are numbered row-major and dealt out linearly
template <typename V, int U, int HINT, uint32_t nt>
__device__ __forceinline__ void copy_rows_narrow(const char* __restrict__ s, char* __restrict__ d, uint32_t rows,
                                                 uint32_t re, uint64_t sp, uint64_t dp, uint32_t tid) {
  const uint32_t n = rows * re;
  for (uint32_t e0 = tid; e0 < n; e0 += nt * U) {
    V v[U];
    uint64_t doff[U];
    bool ok[U];
#pragma unroll
    for (int i = 0; i < U; ++i) {
      const uint32_t e = e0 + i * nt;
      const uint32_t r = e / re;
      const uint32_t c = e - r * re;
      ok[i] = e < n;
      doff[i] = uint64_t(r) * dp + uint64_t(c) * sizeof(V);
      if (ok[i]) v[i] = ld<HINT>(reinterpret_cast<const V*>(s + uint64_t(r) * sp + uint64_t(c) * sizeof(V)));
    }
#pragma unroll
    for (int i = 0; i < U; ++i)
      if (ok[i]) st<HINT>(reinterpret_cast<V*>(d + doff[i]), v[i]);
  }
}

template <typename V, int U, int HINT, uint32_t nt>
__device__ __forceinline__ void copy_tile_as(uint32_t flags, uint32_t rows, uint32_t row_bytes, uint64_t sp, uint64_t dp,
                                             const char* s, char* d, uint32_t tid) {
  constexpr uint32_t W = sizeof(V);
  const uint32_t re = row_bytes / W;
  if (flags & BCP_TILE_ZERO) {
    zero_run<V, HINT, nt>(reinterpret_cast<V*>(d), re, tid);
  } else if (rows == 1) {
    copy_run<V, U, HINT, nt>(reinterpret_cast<const V*>(s), reinterpret_cast<V*>(d), re, tid);
  } else if (re >= 32) {
    copy_rows_wide<V, U, HINT, nt>(s, d, rows, re, sp, dp, tid);
  } else {
    copy_rows_narrow<V, U, HINT, nt>(s, d, rows, re, sp, dp, tid);
  }
}

// Out-of-line bodies, so that each gets its own register allocation (ptxas -v lists them
// one by one) and the work loop of the kernel stays small.
template <int U, int HINT, uint32_t nt>
__device__ __noinline__ void run16(const uint4* __restrict__ s, uint4* __restrict__ d, uint32_t n, uint32_t tid) {
  copy_run<uint4, U, HINT, nt>(s, d, n, tid);
}

template <int U, int HINT, uint32_t nt>
__device__ __noinline__ void rows16(const char* __restrict__ s, char* __restrict__ d, uint32_t rows, uint32_t re, uint64_t sp,
                                    uint64_t dp, uint32_t tid) {
  if (re >= 32) {
    copy_rows_wide<uint4, U, HINT, nt>(s, d, rows, re, sp, dp, tid);
  } else {
    copy_rows_narrow<uint4, U, HINT, nt>(s, d, rows, re, sp, dp, tid);
  }
}

// Tiles whose offsets, row length or pitches are not all multiples of 16 bytes (odd shapes,
// odd byte offsets), and zero fills: the same loops with a narrower element.
template <int HINT, uint32_t nt>
__device__ __noinline__ void other(uint32_t flags, uint32_t rows, uint32_t row_bytes, uint64_t sp, uint64_t dp,
                                   const char* s, char* d, uint32_t tid) {
  switch (flags & BCP_TILE_GRAN_MASK) {
    case 4: copy_tile_as<uint4, 2, HINT, nt>(flags, rows, row_bytes, sp, dp, s, d, tid); break;
    case 3: copy_tile_as<uint2, 2, HINT, nt>(flags, rows, row_bytes, sp, dp, s, d, tid); break;
    case 2: copy_tile_as<unsigned int, 2, HINT, nt>(flags, rows, row_bytes, sp, dp, s, d, tid); break;
    case 1: copy_tile_as<unsigned short, 2, HINT, nt>(flags, rows, row_bytes, sp, dp, s, d, tid); break;
    default: copy_tile_as<unsigned char, 2, HINT, nt>(flags, rows, row_bytes, sp, dp, s, d, tid); break;
  }
}

template <int U, int HINT, uint32_t nt>
__device__ __forceinline__ void copy_tile(const bcp_tile& t, const void* const* __restrict__ src,
                                          void* const* __restrict__ dst, uint32_t tid) {
  const bool zero = t.flags & BCP_TILE_ZERO;
  const char* s = zero ? nullptr : static_cast<const char*>(src[t.src_buf]) + t.src_off;
  char* d = static_cast<char*>(dst[t.dst_buf]) + t.dst_off;
  if ((t.flags & (BCP_TILE_GRAN_MASK | BCP_TILE_ZERO)) == 4) {
    if (t.rows == 1) {
      run16<U, HINT, nt>(reinterpret_cast<const uint4*>(s), reinterpret_cast<uint4*>(d), t.row_bytes >> 4, tid);
    } else {
      rows16<U, HINT, nt>(s, d, t.rows, t.row_bytes >> 4, t.src_pitch, t.dst_pitch, tid);
    }
  } else {
    other<HINT, nt>(t.flags, t.rows, t.row_bytes, t.src_pitch, t.dst_pitch, s, d, tid);
  }
}

__device__ __forceinline__ bcp_tile load_tile(const bcp_tile* p) {
  // 64-byte record, 16-byte aligned: four vector loads, identical for every thread of the group
  static_assert(sizeof(bcp_tile) == 64, "tile record must be 64 bytes");
  const uint4* q = reinterpret_cast<const uint4*>(p);
  const uint4 a = __ldg(q), b = __ldg(q + 1), c = __ldg(q + 2);
  bcp_tile t;
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

}  // namespace
}  // namespace bcp
