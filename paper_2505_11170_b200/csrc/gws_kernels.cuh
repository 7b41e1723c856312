// Device code of the sampling pass for sm_100a.
//
// The pass is elementwise plus a small per-group reduction, so it is bound by HBM
// bandwidth first and by the integer pipe (Philox + decode) second.  Every kernel
// therefore moves 16-byte vectors of 8 BF16 elements (one Philox call serves exactly
// one such vector), issues all loads of a thread before the first use, and reduces
// inside a warp with shuffles.  Three tilings cover the fast cases:
//
//   flat      group = 8 << k contiguous elements (k = 0..5) of a dense tensor: the tensor is
//             a flat run of vectors, a group is 1 << k adjacent lanes of a warp.
//   row-warp  group = one row of up to 4096 elements: one warp per row, up to 16 vectors
//             per lane kept in registers between the max and the add (single pass over W).
//   row-cta   group = one row of up to 65536 elements: one 512-thread block per row.
//
// and a general kernel (one block per group, scalar accesses) handles every other shape.
// All kernels read their tensor from a table so that one launch serves many tensors.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gws_math.cuh"

namespace gws {

enum Mode { kAbsmax = 0, kFwd = 1, kBwd = 2 };
enum KernelClass { kFlat = 0, kRowWarp = 1, kRowCta = 2, kGeneral = 3 };

// One tensor of a launch.  `in`/`out`/`gin`/`gout` change meaning with the mode:
//   absmax: in = w,           gout = absmax
//   fwd:    in = w,           out = w_hat,           gin = bt,    gout = scale_out or null
//   bwd:    in = grad_w_hat,  out = grad_w or null,  gin = scale, gout = grad_bt
struct __align__(16) Entry {
  const void* in;
  void* out;
  const float* gin;
  float* gout;
  int64_t rows, cols, ld;
  int32_t group_rows, group_cols;  // group_cols resolved: never 0
  uint64_t elem_offset;
  uint64_t n_vec;                  // rows*cols/8 (fast classes)
  uint32_t seed_lo, seed_hi;
  uint32_t vpr;                    // vectors per row (row classes)
  uint32_t lanes_log2;             // flat: log2(group_cols / 8)
  int64_t tile_begin;              // first tile of this tensor inside its launch
};
static_assert(sizeof(Entry) == 112, "Entry layout");

constexpr int kFlatThreads = 256, kFlatVecs = 4;        // 1024 vectors = 16 KiB of BF16 per tile
constexpr int kRowWarpThreads = 256, kRowWarpVecs = 16; // 8 rows per tile, <= 512 vectors per row
constexpr int kRowCtaThreads = 512, kRowCtaVecs = 16;   // 1 row per tile, <= 8192 vectors per row
constexpr int kGeneralThreads = 128;
constexpr float kLn2 = 0.693147180559945309f;

// ---- global memory accessors ---------------------------------------------------------------------
// Every access to caller memory goes through these.  In the self-checking build
// (-DGWS_SELF_CHECK) each address is first tested against a caller-declared window; an address
// outside it is recorded (first violation wins: kind, address, block, thread) and the access is
// skipped, so a wrong pointer or index shows up as a report instead of a fault.

#ifdef GWS_SELF_CHECK
struct CheckState {
  unsigned long long lo, hi;        // allowed window [lo, hi)
  unsigned long long violations;    // count
  unsigned long long first[4];      // kind, address, blockIdx.x, threadIdx.x of the first one
};
__device__ CheckState g_check;

__device__ __noinline__ bool check_access(const void* p, unsigned bytes, unsigned kind) {
  const unsigned long long a = reinterpret_cast<unsigned long long>(p);
  if (a >= g_check.lo && a + bytes <= g_check.hi) return true;
  if (atomicAdd(&g_check.violations, 1ull) == 0ull) {
    g_check.first[0] = kind;
    g_check.first[1] = a;
    g_check.first[2] = blockIdx.x;
    g_check.first[3] = threadIdx.x;
  }
  return false;
}
#define GWS_CHECK(p, bytes, kind, fallback) \
  if (!check_access((p), (bytes), (kind))) return fallback
#else
#define GWS_CHECK(p, bytes, kind, fallback)
#endif

__device__ __forceinline__ uint4 ld_vec(const void* base, uint64_t v) {
  const uint4* p = reinterpret_cast<const uint4*>(base) + v;
  GWS_CHECK(p, 16, 1, make_uint4(0, 0, 0, 0));
  return __ldg(p);
}
__device__ __forceinline__ void st_vec(void* base, uint64_t v, const uint4& x) {
  uint4* p = reinterpret_cast<uint4*>(base) + v;
  GWS_CHECK(p, 16, 2, );
  *p = x;
}
__device__ __forceinline__ float ld_f32(const float* base, uint64_t i) {
  GWS_CHECK(base + i, 4, 3, 0.0f);
  return __ldg(base + i);
}
__device__ __forceinline__ void st_f32(float* base, uint64_t i, float x) {
  GWS_CHECK(base + i, 4, 4, );
  base[i] = x;
}
__device__ __forceinline__ uint16_t ld_u16(const uint16_t* base, int64_t i) {
  GWS_CHECK(base + i, 2, 5, 0);
  return base[i];
}
__device__ __forceinline__ void st_u16(uint16_t* base, int64_t i, uint16_t x) {
  GWS_CHECK(base + i, 2, 6, );
  base[i] = x;
}

__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
  // max of two packed pairs of non-negative BF16 values
  __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
  return *reinterpret_cast<uint32_t*>(&r);
}

// Packed pair whose both halves hold ... partial maxima of |x| over the vector; the caller
// finishes with absmax_finish() after any cross-lane reduction.
__device__ __forceinline__ uint32_t absmax_vec(const uint4& x) {
  const uint32_t m = 0x7FFF7FFFu;
  return bmax2(bmax2(x.x & m, x.y & m), bmax2(x.z & m, x.w & m));
}
__device__ __forceinline__ float absmax_finish(uint32_t pair) {
  const uint32_t both = bmax2(pair, __byte_perm(pair, pair, 0x1032));  // max(lo, hi) in both halves
  return __uint_as_float(both << 16);
}

// 2^(1 - b): exact for integer-valued b, double exp2 rounded to float otherwise.
__device__ __forceinline__ float pow2_one_minus(float b) {
  if (b == truncf(b) && b >= -126.0f && b <= 127.0f) {
    const int e = 1 - static_cast<int>(b);
    return __int_as_float((127 + e) << 23);
  }
  return static_cast<float>(exp2(1.0 - static_cast<double>(b)));
}

__device__ __forceinline__ uint32_t pack_bf16_rne(float lo, float hi) {
  __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);  // cvt.rn.bf16x2.f32: IEEE round-to-nearest-even
  return *reinterpret_cast<uint32_t*>(&r);
}

// Eq. 3 + cast for one vector: 8 x ( bf16_rne( fl32(w + R*s) ) ).
// The decode gives float(R) * 2^-126 as a bit pattern; two exact multiplies rebuild R*s.
// w + 0.0f turns a -0.0 weight into +0.0 first, so that a signed zero noise term adds
// nothing (R == 0 must contribute +0.0).
__device__ __forceinline__ uint4 sample_vec(const uint4& w, const Words4& r, float s) {
  uint32_t p[4];
  decode4(r.o[0], r.o[1], p[0], p[1]);
  decode4(r.o[2], r.o[3], p[2], p[3]);
  const uint32_t wi[4] = {w.x, w.y, w.z, w.w};
  uint32_t o[4];
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float wl = __uint_as_float(wi[j] << 16);
    const float wh = __uint_as_float(wi[j] & 0xFFFF0000u);
    const float fl = __fmul_rn(__uint_as_float(p[j] << 16), 0x1p126f);
    const float fh = __fmul_rn(__uint_as_float(p[j] & 0xFFFF0000u), 0x1p126f);
    const float yl = __fadd_rn(__fadd_rn(wl, 0.0f), __fmul_rn(fl, s));
    const float yh = __fadd_rn(__fadd_rn(wh, 0.0f), __fmul_rn(fh, s));
    o[j] = pack_bf16_rne(yl, yh);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// sum over the vector of float(g) * R, accumulated in element order.
__device__ __forceinline__ float dot_vec(const uint4& g, const Words4& r) {
  uint32_t p[4];
  decode4(r.o[0], r.o[1], p[0], p[1]);
  decode4(r.o[2], r.o[3], p[2], p[3]);
  const uint32_t gi[4] = {g.x, g.y, g.z, g.w};
  float acc = 0.0f;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float gl = __uint_as_float(gi[j] << 16);
    const float gh = __uint_as_float(gi[j] & 0xFFFF0000u);
    const float fl = __fmul_rn(__uint_as_float(p[j] << 16), 0x1p126f);
    const float fh = __fmul_rn(__uint_as_float(p[j] & 0xFFFF0000u), 0x1p126f);
    acc = __fmaf_rn(gl, fl, acc);
    acc = __fmaf_rn(gh, fh, acc);
  }
  return acc;
}

__device__ __forceinline__ Words4 philox_vec(const Entry& e, uint64_t vec_in_tensor, uint32_t step_lo, uint32_t step_hi) {
  return philox_for_vector((e.elem_offset >> 3) + vec_in_tensor, step_lo, step_hi, e.seed_lo, e.seed_hi);
}

// Finds the tensor that owns tile `tile` of a multi-tensor launch (tile_begin is increasing).
__device__ __forceinline__ int locate(const Entry* __restrict__ table, int n, int64_t tile) {
  int lo = 0, hi = n - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if (table[mid].tile_begin <= tile) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// The tensor of this thread block.  MULTI is a compile-time switch: a single-tensor launch reads its
// entry from the kernel parameters, a multi-tensor launch from the table in global memory.  (A run-time
// choice between the two sources inside one kernel produced entries mixed from both on sm_100a.)
#define GWS_RESOLVE_ENTRY(e, tile)                                   \
  Entry e;                                                           \
  int64_t tile = static_cast<int64_t>(blockIdx.x);                   \
  if (MULTI) {                                                       \
    e = table[locate(table, n, tile)];                               \
    tile -= e.tile_begin;                                            \
  } else {                                                           \
    e = single;                                                      \
  }

// Diagnostic: what locate() resolves for a list of tile indices.  Reads the table only.
// out[6*k ..] = {in, out, gin, gout, local tile, tensor rows} for tiles[k].
__global__ void k_locate_probe(const Entry* __restrict__ table, int n, const int64_t* __restrict__ tiles, int n_tiles,
                               uint64_t* __restrict__ out) {
  const int k = blockIdx.x * blockDim.x + threadIdx.x;
  if (k >= n_tiles) return;
  const Entry e = table[locate(table, n, tiles[k])];
  const int64_t local = tiles[k] - e.tile_begin;
  out[6 * k + 0] = reinterpret_cast<uint64_t>(e.in);
  out[6 * k + 1] = reinterpret_cast<uint64_t>(e.out);
  out[6 * k + 2] = reinterpret_cast<uint64_t>(e.gin);
  out[6 * k + 3] = reinterpret_cast<uint64_t>(e.gout);
  out[6 * k + 4] = static_cast<uint64_t>(local);
  out[6 * k + 5] = static_cast<uint64_t>(e.rows);
}

// ---- flat groups ------------------------------------------------------------------------------

template <int MODE, bool MULTI>
__global__ void __launch_bounds__(kFlatThreads) k_flat(const __grid_constant__ Entry single,
                                                       const Entry* __restrict__ table, int n, uint32_t step_lo,
                                                       uint32_t step_hi) {
  constexpr int T = kFlatThreads, V = kFlatVecs;
  GWS_RESOLVE_ENTRY(e, tile)
  const uint32_t ll = e.lanes_log2;
  const uint32_t L = 1u << ll;
  const uint32_t lane_in_group = threadIdx.x & (L - 1u);
  const uint64_t base = static_cast<uint64_t>(tile) * (T * V) + threadIdx.x;

  uint4 x[V];
  float gv[V];
  bool ok[V];
#pragma unroll
  for (int k = 0; k < V; ++k) {
    const uint64_t v = base + static_cast<uint64_t>(k) * T;
    ok[k] = v < e.n_vec;
    x[k] = ok[k] ? ld_vec(e.in, v) : make_uint4(0, 0, 0, 0);
    gv[k] = 0.0f;
    if (MODE != kAbsmax && ok[k]) gv[k] = ld_f32(e.gin, v >> ll);
  }
#pragma unroll
  for (int k = 0; k < V; ++k) {
    const uint64_t v = base + static_cast<uint64_t>(k) * T;
    const uint64_t g = v >> ll;
    if (MODE == kBwd) {
      float acc = dot_vec(x[k], philox_vec(e, v, step_lo, step_hi));
      for (uint32_t o = 1; o < L; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
      if (ok[k]) {
        if (lane_in_group == 0) st_f32(e.gout, g, __fmul_rn(__fmul_rn(-kLn2, gv[k]), acc));
        if (e.out != nullptr) st_vec(e.out, v, x[k]);
      }
    } else {
      uint32_t m = absmax_vec(x[k]);
      for (uint32_t o = 1; o < L; o <<= 1) m = bmax2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      const float a = absmax_finish(m);
      if (MODE == kAbsmax) {
        if (ok[k] && lane_in_group == 0) st_f32(e.gout, g, a);
      } else {
        const float s = __fmul_rn(a, pow2_one_minus(gv[k]));
        const uint4 y = sample_vec(x[k], philox_vec(e, v, step_lo, step_hi), s);
        if (ok[k]) {
          st_vec(e.out, v, y);
          if (e.gout != nullptr && lane_in_group == 0) st_f32(e.gout, g, s);
        }
      }
    }
  }
}

// ---- one warp per row ---------------------------------------------------------------------------

template <int MODE, bool MULTI>
__global__ void __launch_bounds__(kRowWarpThreads) k_row_warp(const __grid_constant__ Entry single,
                                                              const Entry* __restrict__ table, int n,
                                                              uint32_t step_lo, uint32_t step_hi) {
  constexpr int V = kRowWarpVecs, ROWS = kRowWarpThreads / 32;
  GWS_RESOLVE_ENTRY(e, tile)
  const uint32_t lane = threadIdx.x & 31u;
  const int64_t row = tile * ROWS + (threadIdx.x >> 5);
  const bool okr = row < e.rows;
  const uint32_t vpr = e.vpr;
  const uint64_t vbase = static_cast<uint64_t>(row) * vpr;

  uint4 x[V];
#pragma unroll
  for (int k = 0; k < V; ++k) {
    x[k] = make_uint4(0, 0, 0, 0);
    if (k * 32u < vpr) {
      const uint32_t j = k * 32u + lane;
      if (okr && j < vpr) x[k] = ld_vec(e.in, vbase + j);
    }
  }
  const float gvr = (MODE != kAbsmax && okr) ? ld_f32(e.gin, row) : 0.0f;

  if (MODE == kBwd) {
    float acc = 0.0f;
#pragma unroll
    for (int k = 0; k < V; ++k) {
      if (k * 32u < vpr) {
        const uint32_t j = k * 32u + lane;
        const bool ok = okr && j < vpr;
        const float part = dot_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi));
        if (ok) {
          acc += part;
          if (e.out != nullptr) st_vec(e.out, vbase + j, x[k]);
        }
      }
    }
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (okr && lane == 0) st_f32(e.gout, row, __fmul_rn(__fmul_rn(-kLn2, gvr), acc));
  } else {
    uint32_t m = 0;
#pragma unroll
    for (int k = 0; k < V; ++k)
      if (k * 32u < vpr) m = bmax2(m, absmax_vec(x[k]));
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) m = bmax2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    const float a = absmax_finish(m);
    if (MODE == kAbsmax) {
      if (okr && lane == 0) st_f32(e.gout, row, a);
    } else {
      const float s = __fmul_rn(a, pow2_one_minus(gvr));
#pragma unroll
      for (int k = 0; k < V; ++k) {
        if (k * 32u < vpr) {
          const uint32_t j = k * 32u + lane;
          const uint4 y = sample_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), s);
          if (okr && j < vpr) st_vec(e.out, vbase + j, y);
        }
      }
      if (okr && lane == 0 && e.gout != nullptr) st_f32(e.gout, row, s);
    }
  }
}

// ---- one thread block per row ---------------------------------------------------------------------

template <int MODE, bool MULTI>
__global__ void __launch_bounds__(kRowCtaThreads) k_row_cta(const __grid_constant__ Entry single,
                                                            const Entry* __restrict__ table, int n,
                                                            uint32_t step_lo, uint32_t step_hi) {
  constexpr int T = kRowCtaThreads, V = kRowCtaVecs, WARPS = T / 32;
  __shared__ uint32_t red_u[WARPS];
  __shared__ float red_f[WARPS];
  GWS_RESOLVE_ENTRY(e, tile)
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const int64_t row = tile;
  const uint32_t vpr = e.vpr;
  const uint64_t vbase = static_cast<uint64_t>(row) * vpr;

  uint4 x[V];
#pragma unroll
  for (int k = 0; k < V; ++k) {
    x[k] = make_uint4(0, 0, 0, 0);
    if (static_cast<uint32_t>(k) * T < vpr) {
      const uint32_t j = k * T + threadIdx.x;
      if (j < vpr) x[k] = ld_vec(e.in, vbase + j);
    }
  }
  const float gvr = (MODE != kAbsmax) ? ld_f32(e.gin, row) : 0.0f;

  if (MODE == kBwd) {
    float acc = 0.0f;
#pragma unroll
    for (int k = 0; k < V; ++k) {
      if (static_cast<uint32_t>(k) * T < vpr) {
        const uint32_t j = k * T + threadIdx.x;
        const float part = dot_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi));
        if (j < vpr) {
          acc += part;
          if (e.out != nullptr) st_vec(e.out, vbase + j, x[k]);
        }
      }
    }
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) red_f[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      float total = 0.0f;
      for (int w = 0; w < WARPS; ++w) total += red_f[w];  // fixed order
      st_f32(e.gout, row, __fmul_rn(__fmul_rn(-kLn2, gvr), total));
    }
  } else {
    uint32_t m = 0;
#pragma unroll
    for (int k = 0; k < V; ++k)
      if (static_cast<uint32_t>(k) * T < vpr) m = bmax2(m, absmax_vec(x[k]));
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) m = bmax2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    if (lane == 0) red_u[warp] = m;
    __syncthreads();
    uint32_t mm = red_u[0];
#pragma unroll
    for (int w = 1; w < WARPS; ++w) mm = bmax2(mm, red_u[w]);
    const float a = absmax_finish(mm);
    if (MODE == kAbsmax) {
      if (threadIdx.x == 0) st_f32(e.gout, row, a);
    } else {
      const float s = __fmul_rn(a, pow2_one_minus(gvr));
#pragma unroll
      for (int k = 0; k < V; ++k) {
        if (static_cast<uint32_t>(k) * T < vpr) {
          const uint32_t j = k * T + threadIdx.x;
          const uint4 y = sample_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), s);
          if (j < vpr) st_vec(e.out, vbase + j, y);
        }
      }
      if (threadIdx.x == 0 && e.gout != nullptr) st_f32(e.gout, row, s);
    }
  }
}

// ---- general shapes: one thread block per group, scalar accesses ---------------------------------

template <int MODE, bool MULTI>
__global__ void __launch_bounds__(kGeneralThreads) k_general(const __grid_constant__ Entry single,
                                                             const Entry* __restrict__ table, int index,
                                                             uint32_t step_lo, uint32_t step_hi) {
  constexpr int T = kGeneralThreads, WARPS = T / 32;
  __shared__ float red[WARPS];
  __shared__ float bcast;
  Entry e;
  if (MULTI) e = table[index]; else e = single;
  const uint16_t* in = reinterpret_cast<const uint16_t*>(e.in);
  uint16_t* out = reinterpret_cast<uint16_t*>(e.out);
  const int64_t gr = e.group_rows, gc = e.group_cols;
  const int64_t gpr = (e.cols + gc - 1) / gc;
  const int64_t n_groups = ((e.rows + gr - 1) / gr) * gpr;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;

  for (int64_t g = blockIdx.x; g < n_groups; g += gridDim.x) {
    const int64_t r0 = (g / gpr) * gr, c0 = (g % gpr) * gc;
    const int64_t h = min(gr, e.rows - r0), wd = min(gc, e.cols - c0);
    const int64_t count = h * wd;
    float scale = 0.0f;
    if (MODE != kBwd) {
      float m = 0.0f;
      for (int64_t k = threadIdx.x; k < count; k += T) {
        const int64_t i = r0 + k / wd, j = c0 + k % wd;
        m = fmaxf(m, fabsf(__uint_as_float(static_cast<uint32_t>(ld_u16(in, i * e.ld + j)) << 16)));
      }
#pragma unroll
      for (uint32_t o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      if (lane == 0) red[warp] = m;
      __syncthreads();
      if (threadIdx.x == 0) {
        float a = red[0];
        for (int w = 1; w < WARPS; ++w) a = fmaxf(a, red[w]);
        if (MODE == kAbsmax) {
          st_f32(e.gout, g, a);
        } else {
          const float s = __fmul_rn(a, pow2_one_minus(ld_f32(e.gin, g)));
          if (e.gout != nullptr) st_f32(e.gout, g, s);
          bcast = s;
        }
      }
      __syncthreads();
      if (MODE == kFwd) scale = bcast;
    }
    if (MODE != kAbsmax) {
      float acc = 0.0f;
      for (int64_t k = threadIdx.x; k < count; k += T) {
        const int64_t i = r0 + k / wd, j = c0 + k % wd;
        const uint64_t el = e.elem_offset + static_cast<uint64_t>(i * e.cols + j);
        const Words4 words = philox_for_vector(el >> 3, step_lo, step_hi, e.seed_lo, e.seed_hi);
        const int r = decode_field(field_of(words, static_cast<unsigned>(el & 7u)));
        const uint16_t bits = ld_u16(in, i * e.ld + j);
        const float val = __uint_as_float(static_cast<uint32_t>(bits) << 16);
        if (MODE == kFwd) {
          const float q = __fmul_rn(static_cast<float>(r), scale);
          const float y = __fadd_rn(val, q);
          st_u16(out, i * e.ld + j, static_cast<uint16_t>(pack_bf16_rne(y, 0.0f) & 0xFFFFu));
        } else {
          acc = __fmaf_rn(val, static_cast<float>(r), acc);
          if (out != nullptr) st_u16(out, i * e.ld + j, bits);
        }
      }
      if (MODE == kBwd) {
#pragma unroll
        for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        if (lane == 0) red[warp] = acc;
        __syncthreads();
        if (threadIdx.x == 0) {
          float total = 0.0f;
          for (int w = 0; w < WARPS; ++w) total += red[w];
          st_f32(e.gout, g, __fmul_rn(__fmul_rn(-kLn2, ld_f32(e.gin, g)), total));
        }
      }
    }
    __syncthreads();  // red / bcast are reused by the next group
  }
}

// ---- noise words, raw Philox words, arithmetic probe ----------------------------------------------

__global__ void __launch_bounds__(256) k_noise(uint32_t* __restrict__ out, uint64_t n_words, uint64_t n_elems,
                                               uint64_t vec0, uint32_t seed_lo, uint32_t seed_hi, uint32_t step_lo,
                                               uint32_t step_hi) {
  const uint64_t v = static_cast<uint64_t>(blockIdx.x) * 256u + threadIdx.x;
  if (v >= n_words) return;
  uint32_t word = pack_nibbles(philox_for_vector(vec0 + v, step_lo, step_hi, seed_lo, seed_hi));
  const uint64_t remaining = n_elems - v * 8u;
  if (remaining < 8u) word &= (1u << (4u * static_cast<uint32_t>(remaining))) - 1u;
  out[v] = word;
}

// Same arithmetic as k_noise, 8 words per thread, one stored word per block.
__global__ void __launch_bounds__(256) k_noise_probe(uint32_t* __restrict__ sink, uint64_t n_words, uint64_t vec0,
                                                     uint32_t seed_lo, uint32_t seed_hi, uint32_t step_lo,
                                                     uint32_t step_hi) {
  __shared__ uint32_t red[8];
  uint32_t acc = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint64_t v = (static_cast<uint64_t>(blockIdx.x) * 8u + k) * 256u + threadIdx.x;
    if (v < n_words) acc ^= pack_nibbles(philox_for_vector(vec0 + v, step_lo, step_hi, seed_lo, seed_hi));
  }
#pragma unroll
  for (uint32_t o = 16; o > 0; o >>= 1) acc ^= __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if ((threadIdx.x & 31u) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    uint32_t t = 0;
    for (int w = 0; w < 8; ++w) t ^= red[w];
    sink[blockIdx.x] = t;
  }
}

__global__ void __launch_bounds__(256) k_philox_words(uint4* __restrict__ out, uint64_t n_vec, uint64_t first_vec,
                                                      uint32_t seed_lo, uint32_t seed_hi, uint32_t step_lo,
                                                      uint32_t step_hi) {
  const uint64_t v = static_cast<uint64_t>(blockIdx.x) * 256u + threadIdx.x;
  if (v >= n_vec) return;
  const Words4 w = philox_for_vector(first_vec + v, step_lo, step_hi, seed_lo, seed_hi);
  out[v] = make_uint4(w.o[0], w.o[1], w.o[2], w.o[3]);
}

}  // namespace gws
