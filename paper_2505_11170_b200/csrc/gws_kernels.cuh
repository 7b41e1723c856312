// Device code of the sampling pass for sm_100a.
//
// The pass is elementwise plus a small per-group reduction.  Its algorithmic cost is 4 bytes per
// element forward and 2 backward, but every element also needs 16 random bits (Philox4x32-10: 18
// wide multiplies + 19 three-input XORs per 8 elements once the launch-uniform part is hoisted).
// On B200 that generation alone runs at about 2.8 T elements/s: well above the HBM bound of the
// forward pass (1.6 T), below that of the backward pass (3.1 T).  So forward is HBM-bound, backward
// is bound by instruction issue, and everything besides Philox is written for instruction count:
//
//   * one Philox call and one whole-word decode serve the 8 elements of a 16-byte vector;
//   * the noise reaches the FP32 pipe as a BF16 bit pattern (2R); high halves (and in backward
//     both halves) are consumed directly by the mixed-precision add / fma of sm_100;
//   * a thread owns 64 contiguous bytes (a chunk: 4 vectors, 32 elements), moved with two 32-byte
//     accesses, so a group of 128 elements is 4 lanes and needs two shuffle steps;
//   * |w| maxima are taken on packed BF16 pairs (max.xorsign.abs), never widened;
//   * the tensors of a launch are described by compact records passed BY VALUE in the kernel
//     parameters, so a thread block (a few microseconds of work) finds its tensor without a
//     global-memory access.
//
// Kernels:
//   k_flat    group = 8 << k contiguous elements (k = 0..5) of a dense tensor: the tensor is a flat
//             run of chunks; groups up to a chunk live inside the thread.
//   k_row     group = one row (a multiple of 32 elements, up to 32768): 1..32 lanes or one block
//             share a row, whose chunks stay in registers between the max and the add.
//   k_square  group = the paper's 32 x 32 block: a warp per pair of neighbouring blocks, 16 lanes per block.
//   k_row_warp / k_row_cta   whole rows the chunk kernel does not take (16-byte vectors), one tensor
//             per launch;  k_general  every other shape: one block per group, scalar accesses,
//             tensor record read from a device table in multi-tensor plans.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "gws_math.cuh"

namespace gws {

// kFwdScaled: forward with the per-group factor s_g supplied (in `gin`) instead of derived from this tensor's own
// maxima: the add and cast of Eq. 3 for a tensor whose groups reach into memory this call does not see.
enum Mode { kAbsmax = 0, kFwd = 1, kBwd = 2, kFwdScaled = 3, kFwdMx8 = 4, kFwdMx6 = 5, kQuantMx8 = 6, kQuantMx6 = 7, kFwdMx8b = 8, kQuantMx8b = 9 };
// kFwdMx*: the forward pass with w_hat written as MX floating point (E4M3 or E3M2 elements, one E8M0 scale per 32
// elements) instead of BF16; kQuantMx*: that conversion alone, from a BF16 w_hat in `in`.
enum MxFormat { kMxE4M3 = 0, kMxE3M2 = 1, kMxE3M4 = 2 };   // Mx8 = E4M3, Mx6 = E3M2, Mx8b = E3M4
__host__ __device__ constexpr bool mode_is_mx_fwd(int m) { return m == kFwdMx8 || m == kFwdMx6 || m == kFwdMx8b; }
__host__ __device__ constexpr bool mode_is_mx_quant(int m) { return m == kQuantMx8 || m == kQuantMx6 || m == kQuantMx8b; }
__host__ __device__ constexpr bool mode_is_fwd(int m) { return m == kFwd || mode_is_mx_fwd(m); }            // takes maxima of w, writes scale_out
__host__ __device__ constexpr int mode_mx_format(int m) {
  return (m == kFwdMx8 || m == kQuantMx8) ? kMxE4M3 : ((m == kFwdMx8b || m == kQuantMx8b) ? kMxE3M4 : kMxE3M2);
}
__host__ __device__ constexpr bool mode_reads_group_input(int m) { return m != kAbsmax && !mode_is_mx_quant(m); }
enum KernelClass { kFlat = 0, kRowWarp = 1, kRowCta = 2, kGeneral = 3 };

// Full description of one tensor: the record of the multi-tensor tables and the parameter of the
// vector and general kernels.  `in`/`out`/`gin`/`gout` change meaning with the mode:
//   absmax: in = w,           gout = absmax
//   fwd:    in = w,           out = w_hat,           gin = bt,    gout = scale_out or null
//   scaled: in = w,           out = w_hat,           gout = scale (read only): the forward record serves both forms
//   fwd mx: as fwd, out = the MX buffer (element codes, then the scale bytes at the offset the record states)
//   quant:  in = w_hat (BF16), out = the MX buffer
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

// First statement of the chunk kernels after their index arithmetic (which reads kernel parameters only) and before their
// first access to global memory.  In a launch that was allowed to overlap the end of the kernel before it on the stream
// (programmatic stream serialization), a block may become resident while that kernel's last blocks still run; it stops here
// until that kernel has completed and its writes are visible.  In an ordinary launch both instructions do nothing.
__device__ __forceinline__ void wait_for_previous_kernel() {
  asm volatile("griddepcontrol.launch_dependents;");   // the next launch may become resident once all blocks of this one have started
  asm volatile("griddepcontrol.wait;" ::: "memory");
}

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
// 32-byte (sm_100) accesses; `byte_off` from a 32-byte aligned base.
struct __align__(32) Vec32 {
  uint32_t v[8];
};
__device__ __forceinline__ Vec32 ld_vec32(const void* base, uint64_t byte_off) {
  const char* p = reinterpret_cast<const char*>(base) + byte_off;
  Vec32 r;
#ifdef GWS_SELF_CHECK
  if (!check_access(p, 32, 1)) {
#pragma unroll
    for (int i = 0; i < 8; ++i) r.v[i] = 0;
    return r;
  }
#endif
  asm volatile("ld.global.nc.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r.v[0]), "=r"(r.v[1]), "=r"(r.v[2]), "=r"(r.v[3]), "=r"(r.v[4]), "=r"(r.v[5]), "=r"(r.v[6]), "=r"(r.v[7])
               : "l"(p));
  return r;
}
__device__ __forceinline__ void st_vec32(void* base, uint64_t byte_off, const uint32_t* x) {
  char* p = reinterpret_cast<char*>(base) + byte_off;
  GWS_CHECK(p, 32, 2, );
  asm volatile("st.global.v8.u32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"l"(p), "r"(x[0]), "r"(x[1]), "r"(x[2]), "r"(x[3]), "r"(x[4]),
               "r"(x[5]), "r"(x[6]), "r"(x[7])
               : "memory");
}
__device__ __forceinline__ void st_vec8(void* base, uint64_t byte_off, uint32_t a, uint32_t b) {
  char* p = reinterpret_cast<char*>(base) + byte_off;
  GWS_CHECK(p, 8, 2, );
  *reinterpret_cast<uint2*>(p) = make_uint2(a, b);
}
__device__ __forceinline__ void st_u32(void* base, uint64_t byte_off, uint32_t x) {
  char* p = reinterpret_cast<char*>(base) + byte_off;
  GWS_CHECK(p, 4, 2, );
  *reinterpret_cast<uint32_t*>(p) = x;
}
__device__ __forceinline__ void st_u8(void* base, uint64_t byte_off, uint32_t x) {
  uint8_t* p = reinterpret_cast<uint8_t*>(base) + byte_off;
  GWS_CHECK(p, 1, 7, );
  *p = static_cast<uint8_t>(x);
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

// Packed pair holding max(|a|, |b|) per BF16 half in its magnitude bits (the sign bits are the XOR
// of the operands' signs and are dropped by absmax_finish).
__device__ __forceinline__ uint32_t maxabs2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.xorsign.abs.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t absmax_vec(const uint4& x) { return maxabs2(maxabs2(x.x, x.y), maxabs2(x.z, x.w)); }
// max over both halves, as the FP32 value of that BF16 magnitude
__device__ __forceinline__ float absmax_finish(uint32_t pair) {
  const uint32_t both = maxabs2(pair, __byte_perm(pair, pair, 0x1032));
  return __uint_as_float((both << 16) & 0x7FFF0000u);
}

// 2^(1 - b): exact for integer-valued b, double exp2 rounded to float otherwise.
__device__ __noinline__ float pow2_one_minus_slow(float b) { return static_cast<float>(exp2(1.0 - static_cast<double>(b))); }
__device__ __forceinline__ float pow2_one_minus(float b) {
  if (b >= -126.0f && b <= 127.0f) {
    const int bi = __float2int_rz(b);
    if (static_cast<float>(bi) == b) return __int_as_float((128 - bi) << 23);
  }
  return pow2_one_minus_slow(b);
}

__device__ __forceinline__ uint32_t pack_bf16_rne(float lo, float hi) {
  __nv_bfloat162 r = __floats2bfloat162_rn(lo, hi);  // cvt.rn.bf16x2.f32: IEEE round-to-nearest-even
  return *reinterpret_cast<uint32_t*>(&r);
}

// Mixed-precision operations of sm_100: BF16 operands widened exactly, one FP32 rounding.
__device__ __forceinline__ float fma_bf16(uint16_t a, uint16_t b, float c) {
  float d;
  asm("fma.rn.f32.bf16 %0, %1, %2, %3;" : "=f"(d) : "h"(a), "h"(b), "f"(c));
  return d;
}
__device__ __forceinline__ float add_bf16(uint16_t a, float c) {
  float d;
  asm("add.rn.f32.bf16 %0, %1, %2;" : "=f"(d) : "h"(a), "f"(c));
  return d;
}
__device__ __forceinline__ uint16_t hi16(uint32_t x) { return static_cast<uint16_t>(x >> 16); }

// The per-group factor in the forms the forward pass needs.  The decode delivers 2R, so the
// multiplier is s/2; halving is exact unless s is below 2^-125, where the product is formed as
// (2R * 0.5) * s instead (both roundings then match R * s).
// When s/2 has at most 8 significant bits (always for integer bit-widths: the group maximum is a BF16 number and
// 2^(1-b) a power of two) it is itself a BF16 number, and w + 2R * (s/2) is one mixed-precision fma per element: the
// product is exact, so the single rounding of the fma is the rounding of the separate add.
struct Scale {
  float s, half;
  bool tiny, half_is_bf16;
};
__device__ __forceinline__ Scale make_scale(float s) {
  Scale k;
  k.s = s;
  k.half = __fmul_rn(s, 0.5f);
  k.tiny = s < 0x1p-120f;
  k.half_is_bf16 = !k.tiny && (__float_as_uint(k.half) & 0xFFFFu) == 0u;
  return k;
}
// FORM: 0 = one multiply per element; 1 = tiny scale; 2 = s/2 is a BF16 number
template <int FORM>
__device__ __forceinline__ float noise_term(float two_r, const Scale& k) {
  return FORM == 1 ? __fmul_rn(__fmul_rn(two_r, 0.5f), k.s) : __fmul_rn(two_r, k.half);
}

// Eq. 3 + cast for one pair word: 2 x ( bf16_rne( fl32(w + R*s) ) ).  R*s is exact, the add rounds
// once in FP32 (a separate instruction: never contracted), the pack rounds to nearest even.
template <int FORM>
__device__ __forceinline__ uint32_t sample_pair_t(uint32_t w, uint32_t pair, const Scale& k) {
  if (FORM == 2) {
    const uint16_t hb = hi16(__float_as_uint(k.half));
    return pack_bf16_rne(fma_bf16(static_cast<uint16_t>(pair & 0xFFFFu), hb, __uint_as_float(w << 16)),
                         fma_bf16(hi16(pair), hb, __uint_as_float(w & 0xFFFF0000u)));
  }
  const float ql = noise_term<FORM>(__uint_as_float(pair << 16), k);
  const float qh = noise_term<FORM>(__uint_as_float(pair & 0xFFFF0000u), k);
  return pack_bf16_rne(__fadd_rn(__uint_as_float(w << 16), ql), add_bf16(hi16(w), qh));
}
template <int FORM>
__device__ __forceinline__ uint4 sample_vec_t(const uint4& w, const Words4& r, const Scale& k) {
  uint32_t p[4];
  decode8(r, p);
  return make_uint4(sample_pair_t<FORM>(w.x, p[0], k), sample_pair_t<FORM>(w.y, p[1], k), sample_pair_t<FORM>(w.z, p[2], k),
                    sample_pair_t<FORM>(w.w, p[3], k));
}
// The form is chosen once per vector / chunk (it is a property of the group), so the common path carries one
// fma (or one multiply and one add) per element.
__device__ __forceinline__ uint4 sample_vec(const uint4& w, const Words4& r, const Scale& k) {
  return k.half_is_bf16 ? sample_vec_t<2>(w, r, k) : (k.tiny ? sample_vec_t<1>(w, r, k) : sample_vec_t<0>(w, r, k));
}
// One 64-byte chunk whose first vector has the (low) Philox counter word v0.  y may be x (word j depends on word j alone).
template <int FORM>
__device__ __forceinline__ void sample_chunk_t(const uint32_t* x, uint32_t v0, uint32_t k0, uint32_t k1, const PhiloxPre& pre,
                                               const Scale& sc, uint32_t* y) {
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const Words4 r = philox4x32_10_pre(v0 + k, k0, k1, pre);
    uint32_t p[4];
    decode8(r, p);
#pragma unroll
    for (int j = 0; j < 4; ++j) y[4 * k + j] = sample_pair_t<FORM>(x[4 * k + j], p[j], sc);
  }
}
// Half a chunk: 16 elements, two Philox vectors.
template <int FORM>
__device__ __forceinline__ void sample_half_t(const uint32_t* x, uint32_t v0, uint32_t k0, uint32_t k1, const PhiloxPre& pre,
                                              const Scale& sc, uint32_t* y) {
#pragma unroll
  for (int k = 0; k < 2; ++k) {
    const Words4 r = philox4x32_10_pre(v0 + k, k0, k1, pre);
    uint32_t p[4];
    decode8(r, p);
#pragma unroll
    for (int j = 0; j < 4; ++j) y[4 * k + j] = sample_pair_t<FORM>(x[4 * k + j], p[j], sc);
  }
}
__device__ __forceinline__ void sample_half(const uint32_t* x, uint32_t v0, uint32_t k0, uint32_t k1, const PhiloxPre& pre,
                                            const Scale& sc, uint32_t* y) {
  if (sc.half_is_bf16) sample_half_t<2>(x, v0, k0, k1, pre, sc, y);
  else if (sc.tiny) sample_half_t<1>(x, v0, k0, k1, pre, sc, y);
  else sample_half_t<0>(x, v0, k0, k1, pre, sc, y);
}
__device__ __forceinline__ void sample_chunk(const uint32_t* x, uint32_t v0, uint32_t k0, uint32_t k1, const PhiloxPre& pre,
                                             const Scale& sc, uint32_t* y) {
  if (sc.half_is_bf16) sample_chunk_t<2>(x, v0, k0, k1, pre, sc, y);
  else if (sc.tiny) sample_chunk_t<1>(x, v0, k0, k1, pre, sc, y);
  else sample_chunk_t<0>(x, v0, k0, k1, pre, sc, y);
}

// Running sum of float(g) * 2R: low and high BF16 halves of every pair go to their own accumulator
// (two independent FMA chains), both through fma.rn.f32.bf16, which widens the operands exactly
// and takes them straight from the halves of the 32-bit words.  The order is fixed, so results
// repeat bit for bit.
struct DotAcc {
  float lo = 0.0f, hi = 0.0f;
  __device__ __forceinline__ float total() const { return __fadd_rn(lo, hi); }
};
__device__ __forceinline__ void dot_pair(uint32_t g, uint32_t pair, DotAcc& acc) {
  acc.lo = fma_bf16(static_cast<uint16_t>(g & 0xFFFFu), static_cast<uint16_t>(pair & 0xFFFFu), acc.lo);
  acc.hi = fma_bf16(hi16(g), hi16(pair), acc.hi);
}
__device__ __forceinline__ void dot_vec(const uint4& g, const Words4& r, DotAcc& acc) {
  uint32_t p[4];
  decode8_signed_zero(r, p);   // g * (-0) adds a zero of either sign to the running sum: the sum is the same number
  dot_pair(g.x, p[0], acc);
  dot_pair(g.y, p[1], acc);
  dot_pair(g.z, p[2], acc);
  dot_pair(g.w, p[3], acc);
}
// dL/db_t of a group from its scale and the sum of g * 2R.
__device__ __forceinline__ float grad_bt_of(float scale, float sum_g_2r) {
  return __fmul_rn(__fmul_rn(-kLn2, scale), __fmul_rn(sum_g_2r, 0.5f));
}

// ---- w_hat as MX floating point ------------------------------------------------------------------------
//
// OCP Microscaling conversion of the BF16 w_hat with one scale per sampling group (Section 3.2: vectors of a
// square block share their scale): scale byte = max(E - emax, 0), E the biased exponent of the group's largest
// |w_hat| (so the shared exponent floor(log2 max) - emax is clamped at -127), elements = w_hat * 2^(127 - byte)
// rounded to nearest even onto the element grid and clamped to its largest normal, which is what
// cvt.rn.satfinite does.  The multiplication by a power of two is exact.
// Buffer: element codes from byte 0 in chunk order (E4M3: 32 bytes per 32-element chunk; E3M2: 24, code k of the
// chunk at bits [6k, 6k+5] of a little-endian bit stream), scale bytes from byte 16 * scales_off16, one per chunk.
// E3M4 (1-3-4, bias 3, every code finite, largest normal 31) has no conversion instruction: round to nearest even in
// integer arithmetic.  Below the smallest normal (2^-2) the codes are multiples of 2^-6: adding 2^17 makes the FP32
// adder round to that spacing.  From there up the mantissa is cut at bit 19 with the usual round-to-even increment,
// a carry moves into the exponent, and anything beyond the last code is clamped to it.
__device__ __forceinline__ uint32_t cvt_e3m4(float x) {
  const uint32_t bits = __float_as_uint(x), sign = (bits >> 24) & 0x80u;
  const float a = fabsf(x);
  uint32_t mag;
  if (a < 0.25f) {
    mag = __float_as_uint(__fadd_rn(a, 0x1p17f)) - __float_as_uint(0x1p17f);
  } else {
    uint32_t ab = bits & 0x7FFFFFFFu;
    ab += 0x3FFFFu + ((ab >> 19) & 1u);
    mag = min((ab >> 19) - ((127u - 3u) << 4), 0x7Fu);
  }
  return sign | mag;
}
template <int FMT>
__device__ __forceinline__ uint32_t cvt_mx_x2(float upper, float lower) {
  if (FMT == kMxE3M4) return (cvt_e3m4(upper) << 8) | cvt_e3m4(lower);
  uint16_t d;
  if (FMT == kMxE4M3) asm("cvt.rn.satfinite.e4m3x2.f32 %0, %1, %2;" : "=h"(d) : "f"(upper), "f"(lower));
  else asm("cvt.rn.satfinite.e3m2x2.f32 %0, %1, %2;" : "=h"(d) : "f"(upper), "f"(lower));
  return d;
}
// Scale byte of a group whose largest |w_hat| is `amax`, and the bits of the multiplier 2^(127 - byte).
template <int FMT>
__device__ __forceinline__ uint32_t mx_scale_byte(float amax) {
  constexpr int kEmax = FMT == kMxE4M3 ? 8 : 4;   // E3M2 and E3M4: 4
  return static_cast<uint32_t>(max(static_cast<int>(__float_as_uint(amax) >> 23) - kEmax, 0));   // amax >= 0: no sign bit
}
__device__ __forceinline__ uint32_t mx_mult_bits(uint32_t byte) { return (254u - byte) << 23; }

// Codes of 16 elements (8 packed BF16 pairs): E4M3 / E3M4 -> 4 words, E3M2 -> 3 words (four 6-bit codes per 3 bytes).
template <int FMT>
__device__ __forceinline__ void mx_encode_half(const uint32_t* y, uint32_t mult_bits, uint32_t* out) {
  const float mult = __uint_as_float(mult_bits);
  uint32_t q[8];                                                           // two codes each, element 2j in the low byte
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const float lo = __fmul_rn(__uint_as_float(y[j] << 16), mult);
    const float hi = fma_bf16(hi16(y[j]), hi16(mult_bits), -0.0f);         // + (-0): keeps the sign of a zero product
    q[j] = cvt_mx_x2<FMT>(hi, lo);
  }
  if (FMT != kMxE3M2) {   // one byte per code
#pragma unroll
    for (int k = 0; k < 4; ++k) out[k] = q[2 * k] | (q[2 * k + 1] << 16);
  } else {
    uint32_t v[4];                                                         // 24 bits: four codes
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t a = q[2 * k], b = q[2 * k + 1];
      v[k] = (a & 0x3Fu) | ((a >> 2) & 0xFC0u) | ((b & 0x3Fu) << 12) | (((b >> 2) & 0xFC0u) << 12);
    }
    out[0] = v[0] | (v[1] << 24);
    out[1] = (v[1] >> 8) | (v[2] << 16);
    out[2] = (v[2] >> 16) | (v[3] << 8);
  }
}
// One whole 32-element vector (chunk) held by one thread.
template <int FMT>
__device__ __forceinline__ void mx_write(void* out, uint32_t scales_off16, uint32_t chunk, const uint32_t* y, float amax) {
  const uint32_t byte = mx_scale_byte<FMT>(amax), mult_bits = mx_mult_bits(byte);
  if (FMT != kMxE3M2) {
    uint32_t w[8];
    mx_encode_half<FMT>(y, mult_bits, w);
    mx_encode_half<FMT>(y + 8, mult_bits, w + 4);
    st_vec32(out, static_cast<uint64_t>(chunk) * 32u, w);
  } else {
    uint32_t w[6];
    mx_encode_half<FMT>(y, mult_bits, w);
    mx_encode_half<FMT>(y + 8, mult_bits, w + 3);
    const uint64_t at = static_cast<uint64_t>(chunk) * 24u;
    st_vec8(out, at, w[0], w[1]);
    st_vec8(out, at + 8u, w[2], w[3]);
    st_vec8(out, at + 16u, w[4], w[5]);
  }
  st_u8(out, static_cast<uint64_t>(scales_off16) * 16u + chunk, byte);
}
// Half `h` (16 elements) of the vector `chunk`; the thread with the first half also writes the scale byte.
template <int FMT>
__device__ __forceinline__ void mx_write_half(void* out, uint32_t scales_off16, uint32_t chunk, uint32_t h, const uint32_t* y, float amax) {
  const uint32_t byte = mx_scale_byte<FMT>(amax), mult_bits = mx_mult_bits(byte);
  if (FMT != kMxE3M2) {
    uint32_t w[4];
    mx_encode_half<FMT>(y, mult_bits, w);
    st_vec(out, static_cast<uint64_t>(chunk) * 2u + h, make_uint4(w[0], w[1], w[2], w[3]));
  } else {
    uint32_t w[3];
    mx_encode_half<FMT>(y, mult_bits, w);
    const uint64_t at = static_cast<uint64_t>(chunk) * 24u + h * 12u;
    st_u32(out, at, w[0]);
    st_u32(out, at + 4u, w[1]);
    st_u32(out, at + 8u, w[2]);
  }
  if (h == 0u) st_u8(out, static_cast<uint64_t>(scales_off16) * 16u + chunk, byte);
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
//
// Tile = 256 threads x one 64-byte chunk (4 vectors, 32 elements) = 1024 vectors.  Groups of
// 32..256 elements are 1..8 neighbouring lanes (shuffle reduction); groups of 8 or 16 elements are
// handled inside the thread.  Only those small groups can leave a last chunk partly filled.

// One tensor of a flat-group launch.  The records travel BY VALUE in the kernel parameters (constant
// bank): a thread block finds its tensor without touching global memory, which matters because a
// block lives for only a few microseconds.  Pointer meanings as in Entry.
struct FlatRec {
  const void* in;
  void* out;
  const float* gin;
  float* gout;
  uint32_t vec_lo, vec_hi;  // elem_offset / 8: Philox counter of the first vector; vec_hi is the same for every vector
  uint32_t n_vec;
  uint32_t lanes_log2;      // log2(vectors per group)
  int32_t tile_begin;       // first tile of this tensor inside its launch
  uint32_t k0, k1;          // seed
  PhiloxPre pre;            // the step- and seed-dependent constants of the first two Philox rounds
  uint32_t pad;             // MX modes: byte offset of the scale bytes inside `out`, in units of 16
};
static_assert(sizeof(FlatRec) == 80, "FlatRec layout");
constexpr int kFlatHint = 128;
// hint[t >> hint_shift] is the record that owns tile (t >> hint_shift) << hint_shift; the owner of t
// is that record or one a few places further on.
template <int CAP>
struct FlatBatch {
  int32_t n;
  uint32_t hint_shift;
  uint32_t pad[2];
  uint16_t hint[kFlatHint];
  FlatRec e[CAP];
};
constexpr int kFlatCapSmall = 4, kFlatCapLarge = 192;   // 0.6 KiB and 15.3 KiB of parameters
enum FlatVariant { kWide32 = 0, kWide16 = 1, kNarrow = 2 };

struct Chunk {
  uint32_t x[16];
};

// USE32: both tensor pointers are 32-byte aligned, so a chunk moves as two 32-byte accesses.
template <bool USE32>
__device__ __forceinline__ Chunk load_chunk(const void* base, uint64_t chunk, uint32_t n_valid) {
  Chunk c;
  if (USE32) {
    const Vec32 a = ld_vec32(base, chunk * 64u), b = ld_vec32(base, chunk * 64u + 32u);
#pragma unroll
    for (int i = 0; i < 8; ++i) { c.x[i] = a.v[i]; c.x[8 + i] = b.v[i]; }
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint4 t = (static_cast<uint32_t>(k) < n_valid) ? ld_vec(base, chunk * 4u + k) : make_uint4(0, 0, 0, 0);
      c.x[4 * k] = t.x; c.x[4 * k + 1] = t.y; c.x[4 * k + 2] = t.z; c.x[4 * k + 3] = t.w;
    }
  }
  return c;
}
template <bool USE32>
__device__ __forceinline__ void store_chunk(void* base, uint64_t chunk, uint32_t n_valid, const Chunk& c) {
  if (USE32) {
    st_vec32(base, chunk * 64u, c.x);
    st_vec32(base, chunk * 64u + 32u, c.x + 8);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (static_cast<uint32_t>(k) < n_valid)
        st_vec(base, chunk * 4u + k, make_uint4(c.x[4 * k], c.x[4 * k + 1], c.x[4 * k + 2], c.x[4 * k + 3]));
  }
}
__device__ __forceinline__ uint32_t absmax_words4(const uint32_t* x) { return maxabs2(maxabs2(x[0], x[1]), maxabs2(x[2], x[3])); }
__device__ __forceinline__ uint32_t absmax_chunk(const uint32_t* x) {
  return maxabs2(maxabs2(absmax_words4(x), absmax_words4(x + 4)), maxabs2(absmax_words4(x + 8), absmax_words4(x + 12)));
}

// Groups of at least one chunk: `lanes` = chunks per group (1, 2, 4 or 8 neighbouring lanes).
// A thread handles CPT chunks, 256 chunks apart, all loaded before the first is used.
template <int MODE, bool USE32, int CPT>
__device__ __forceinline__ void flat_wide(const FlatRec& e, uint32_t first_chunk, uint32_t lanes, uint32_t lanes_log2) {
  const uint32_t n_chunks = e.n_vec >> 2;
  const bool writer_lane = (threadIdx.x & (lanes - 1u)) == 0u;
  uint32_t chunk[CPT];
  bool ok[CPT];
  Chunk c[CPT];
  float gv[CPT];
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const uint32_t chunk0 = first_chunk + static_cast<uint32_t>(i) * kFlatThreads;
    ok[i] = chunk0 < n_chunks;
    chunk[i] = ok[i] ? chunk0 : n_chunks - 1u;   // keeps the warp whole for the shuffles
    c[i] = load_chunk<USE32>(e.in, chunk[i], 4);
    gv[i] = mode_reads_group_input(MODE) ? ld_f32(MODE == kFwdScaled ? e.gout : e.gin, chunk[i] >> lanes_log2) : 0.0f;
  }
#pragma unroll
  for (int i = 0; i < CPT; ++i) {
    const uint32_t g = chunk[i] >> lanes_log2;
    const bool writer = ok[i] && writer_lane;
    const uint32_t v0 = e.vec_lo + chunk[i] * 4u;
    if (MODE == kBwd) {
      DotAcc dot;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const Words4 r = philox4x32_10_pre(v0 + k, e.k0, e.k1, e.pre);
        dot_vec(make_uint4(c[i].x[4 * k], c[i].x[4 * k + 1], c[i].x[4 * k + 2], c[i].x[4 * k + 3]), r, dot);
      }
      float acc = dot.total();
      for (uint32_t o = 1; o < lanes; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
      if (writer) st_f32(e.gout, g, grad_bt_of(gv[i], acc));
      if (ok[i] && e.out != nullptr) store_chunk<USE32>(e.out, chunk[i], 4, c[i]);
      continue;
    }
    if (MODE == kFwdScaled) {
      Chunk y;
      sample_chunk(c[i].x, v0, e.k0, e.k1, e.pre, make_scale(gv[i]), y.x);
      if (ok[i]) store_chunk<USE32>(e.out, chunk[i], 4, y);
      continue;
    }
    uint32_t m = absmax_chunk(c[i].x);
    for (uint32_t o = 1; o < lanes; o <<= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    const float a = absmax_finish(m);
    if (MODE == kAbsmax) {
      if (writer) st_f32(e.gout, g, a);
      continue;
    }
    if (mode_is_mx_quant(MODE)) {   // the chunk is w_hat itself
      if (ok[i]) mx_write<mode_mx_format(MODE)>(e.out, e.pad, chunk[i], c[i].x, a);
      continue;
    }
    const Scale sc = make_scale(__fmul_rn(a, pow2_one_minus(gv[i])));
    Chunk y;
    sample_chunk(c[i].x, v0, e.k0, e.k1, e.pre, sc, y.x);
    if (mode_is_mx_fwd(MODE)) {
      uint32_t my = absmax_chunk(y.x);
      for (uint32_t o = 1; o < lanes; o <<= 1) my = maxabs2(my, __shfl_xor_sync(0xFFFFFFFFu, my, o));
      if (ok[i]) mx_write<mode_mx_format(MODE)>(e.out, e.pad, chunk[i], y.x, absmax_finish(my));
    } else if (ok[i]) {
      store_chunk<USE32>(e.out, chunk[i], 4, y);
    }
    if (writer && e.gout != nullptr) st_f32(e.gout, g, sc.s);
  }
}

// Groups of one or two vectors (8 or 16 elements): 4 or 2 groups inside the thread's chunk.
template <int MODE>
__device__ __forceinline__ void flat_narrow(const FlatRec& e, uint32_t chunk, uint32_t ll) {
  if (chunk > (e.n_vec - 1u) >> 2) return;
  const uint32_t first = chunk * 4u;
  const uint32_t n_valid = min(4u, e.n_vec - first);
  const Chunk c = load_chunk<false>(e.in, chunk, n_valid);
  const uint32_t v0 = e.vec_lo + first;
  Chunk y;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    if (static_cast<uint32_t>(k) >= n_valid) break;
    const uint32_t g = (first + k) >> ll;
    const bool writer = ll == 0u || (k & 1) == 0;
    const uint4 xv = make_uint4(c.x[4 * k], c.x[4 * k + 1], c.x[4 * k + 2], c.x[4 * k + 3]);
    const int mate = k ^ 1;   // the other vector of a two-vector group (always inside the chunk)
    const Words4 r = philox4x32_10_pre(v0 + k, e.k0, e.k1, e.pre);
    if (MODE == kBwd) {
      if (writer) {
        DotAcc dot;
        dot_vec(xv, r, dot);
        if (ll == 1u) {
          const Words4 r2 = philox4x32_10_pre(v0 + mate, e.k0, e.k1, e.pre);
          dot_vec(make_uint4(c.x[4 * mate], c.x[4 * mate + 1], c.x[4 * mate + 2], c.x[4 * mate + 3]), r2, dot);
        }
        const float acc = dot.total();
        st_f32(e.gout, g, grad_bt_of(ld_f32(e.gin, g), acc));
      }
      continue;
    }
    if (MODE == kFwdScaled) {
      const uint4 yv = sample_vec(xv, r, make_scale(ld_f32(e.gout, g)));
      y.x[4 * k] = yv.x; y.x[4 * k + 1] = yv.y; y.x[4 * k + 2] = yv.z; y.x[4 * k + 3] = yv.w;
      continue;
    }
    uint32_t m = absmax_vec(xv);
    if (ll == 1u) m = maxabs2(m, absmax_words4(c.x + 4 * mate));
    const float a = absmax_finish(m);
    if (MODE == kAbsmax) {
      if (writer) st_f32(e.gout, g, a);
      continue;
    }
    const Scale sc = make_scale(__fmul_rn(a, pow2_one_minus(ld_f32(e.gin, g))));
    const uint4 yv = sample_vec(xv, r, sc);
    y.x[4 * k] = yv.x; y.x[4 * k + 1] = yv.y; y.x[4 * k + 2] = yv.z; y.x[4 * k + 3] = yv.w;
    if (writer && e.gout != nullptr) st_f32(e.gout, g, sc.s);
  }
  if (MODE == kFwd || MODE == kFwdScaled) store_chunk<false>(e.out, chunk, n_valid, y);
  if (MODE == kBwd && e.out != nullptr) store_chunk<false>(e.out, chunk, n_valid, c);
}

// VARIANT: kWide32 / kWide16 = groups of 32..256 elements with 32-byte / 16-byte accesses (the
// former needs every tensor pointer of the launch 32-byte aligned); kNarrow = groups of 8 or 16.
// A tile is 256 threads x CPT chunks (CPT = 1 for narrow groups).
template <int MODE, int VARIANT, int CAP, int CPT>
__global__ void __launch_bounds__(kFlatThreads) k_flat(const __grid_constant__ FlatBatch<CAP> b) {
  const int32_t tile = static_cast<int32_t>(blockIdx.x);
  int idx = b.hint[tile >> b.hint_shift];
  while (idx + 1 < b.n && b.e[idx + 1].tile_begin <= tile) ++idx;
  const FlatRec& e = b.e[idx];
  const uint32_t chunk = static_cast<uint32_t>(tile - e.tile_begin) * (kFlatThreads * CPT) + threadIdx.x;
  wait_for_previous_kernel();
  if (VARIANT == kNarrow) {
    flat_narrow<MODE>(e, chunk, e.lanes_log2);
  } else {
    const uint32_t lanes_log2 = e.lanes_log2 - 2u;
    flat_wide<MODE, VARIANT == kWide32, CPT>(e, chunk, 1u << lanes_log2, lanes_log2);
  }
}

// Host side: copies `count` records into a parameter block for the pass of gradient-update counter
// (step_lo, step_hi), numbers their tiles and builds the tile hint.  Returns the number of tiles.
template <int CAP>
inline int64_t fill_flat_batch(FlatBatch<CAP>& b, const FlatRec* recs, int count, int chunks_per_thread, uint32_t step_lo,
                               uint32_t step_hi) {
  b.n = count;
  b.hint_shift = 0;
  const int64_t per_tile = static_cast<int64_t>(kFlatThreads) * 4 * chunks_per_thread;   // vectors
  int64_t tiles = 0;
  for (int k = 0; k < count; ++k) {
    b.e[k] = recs[k];
    b.e[k].tile_begin = static_cast<int32_t>(tiles);
    b.e[k].pre = philox_pre(recs[k].vec_hi, step_lo, step_hi, recs[k].k0, recs[k].k1);
    tiles += (static_cast<int64_t>(recs[k].n_vec) + per_tile - 1) / per_tile;
    if (tiles > 2147483647LL) return -1;
  }
  while (tiles > 0 && ((tiles - 1) >> b.hint_shift) >= kFlatHint) ++b.hint_shift;
  int owner = 0;
  for (int h = 0; h < kFlatHint; ++h) {
    const int64_t t = static_cast<int64_t>(h) << b.hint_shift;
    while (owner + 1 < count && b.e[owner + 1].tile_begin <= t) ++owner;
    b.hint[h] = static_cast<uint16_t>(owner);
  }
  return tiles;
}

// ---- the paper's square blocks: 32 x 32 elements (Eq. 3, b_l = 32) -------------------------------------
//
// A 32 x 32 block is 64 bytes in each of 32 consecutive rows.  A warp takes two neighbouring blocks (128
// contiguous bytes per row) and reads 8 rows per access, four lanes per row, so an access touches 8 cache
// lines; with a lane per row it touched 32, and the L1 data pipe, not HBM, set the pace.  The 16 lanes of a
// block reduce its maximum and its gradient sum with four shuffle steps.  The 8 warps of a thread block
// take 16 neighbouring blocks of the same 32 rows (1 KiB contiguous per row).  Tensors with whole blocks
// only (rows and cols multiples of 32), dense and 32-byte aligned; the general kernel covers the rest.
struct SquareRec {
  const void* in;
  void* out;
  const float* gin;
  float* gout;
  uint32_t vec_lo, vec_hi;
  uint32_t cpr;             // chunks per row = blocks per row band = cols / 32
  uint32_t tiles_per_band;  // ceil(cpr / (8 * CPT))
  int32_t tile_begin;
  uint32_t k0, k1;
  PhiloxPre pre;
  uint32_t pad;
};
static_assert(sizeof(SquareRec) == 80, "SquareRec layout");
template <int CAP>
struct SquareBatch {
  int32_t n;
  uint32_t hint_shift;
  uint32_t pad[2];
  uint16_t hint[kFlatHint];
  SquareRec e[CAP];
};
constexpr int kSquareCpt = 2;

template <int MODE, int CAP>
__global__ void __launch_bounds__(kFlatThreads) k_square(const __grid_constant__ SquareBatch<CAP> b) {
  const int32_t tile = static_cast<int32_t>(blockIdx.x);
  int idx = b.hint[tile >> b.hint_shift];
  while (idx + 1 < b.n && b.e[idx + 1].tile_begin <= tile) ++idx;
  const SquareRec& e = b.e[idx];
  const uint32_t local = static_cast<uint32_t>(tile - e.tile_begin);
  const uint32_t band = local / e.tiles_per_band, in_band = local - band * e.tiles_per_band;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t cpr = e.cpr;
  // A warp takes two neighbouring blocks: 128 contiguous bytes of each of 32 rows.  One access covers 8 rows: lanes
  // 4r..4r+3 read the four 32-byte pieces of row r, so the warp touches 8 cache lines instead of 32.  A lane holds
  // one piece (16 elements: half of a block's row) of rows 8k + (lane >> 2), k = 0..3, all in the block `blk`.
  const uint32_t blk0 = in_band * (8u * kSquareCpt) + warp * 2u + ((lane & 3u) >> 1);
  const uint32_t half = lane & 1u;
  const bool ok = blk0 < cpr;                     // the same for the 16 lanes that share a block
  const uint32_t blk = ok ? blk0 : cpr - 1u;      // lanes past the last block redo it and store nothing
  const uint32_t g = band * cpr + blk;
  const bool writer = ok && (lane & ~2u) == 0u;   // lanes 0 and 2: first piece of each block
  const uint32_t piece0 = ((band * 32u + (lane >> 2)) * cpr + blk) * 2u + half, piece_step = 16u * cpr;   // 8 rows on
  uint32_t piece[4];                              // index of the 32-byte piece in the tensor
  uint32_t x[4][8];
  wait_for_previous_kernel();
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    piece[k] = piece0 + static_cast<uint32_t>(k) * piece_step;
    const Vec32 v = ld_vec32(e.in, static_cast<uint64_t>(piece[k]) * 32u);
#pragma unroll
    for (int i = 0; i < 8; ++i) x[k][i] = v.v[i];
  }
  const float gv = mode_reads_group_input(MODE) ? ld_f32(MODE == kFwdScaled ? e.gout : e.gin, g) : 0.0f;
  // shuffles over the 16 lanes of a block: they differ in bit 0 (half) and bits 2..4 (row)
  auto block_max = [](uint32_t m) {
    m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
#pragma unroll
    for (uint32_t o = 4; o < 32u; o <<= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    return m;
  };

  if (MODE == kBwd) {
    DotAcc dot;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      const uint32_t v0 = e.vec_lo + piece[k] * 2u;
#pragma unroll
      for (int v = 0; v < 2; ++v) {
        const Words4 r = philox4x32_10_pre(v0 + v, e.k0, e.k1, e.pre);
        dot_vec(make_uint4(x[k][4 * v], x[k][4 * v + 1], x[k][4 * v + 2], x[k][4 * v + 3]), r, dot);
      }
      if (ok && e.out != nullptr) st_vec32(e.out, static_cast<uint64_t>(piece[k]) * 32u, x[k]);
    }
    float acc = dot.total();
    acc += __shfl_xor_sync(0xFFFFFFFFu, acc, 1);
#pragma unroll
    for (uint32_t o = 4; o < 32u; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (writer) st_f32(e.gout, g, grad_bt_of(gv, acc));
    return;
  }

  float a = 0.0f;
  if (MODE != kFwdScaled) {
    uint32_t m = 0u;
#pragma unroll
    for (int k = 0; k < 4; ++k) m = maxabs2(m, maxabs2(absmax_words4(x[k]), absmax_words4(x[k] + 4)));
    a = absmax_finish(block_max(m));
  }
  if (MODE == kAbsmax) {
    if (writer) st_f32(e.gout, g, a);
    return;
  }
  if (mode_is_mx_quant(MODE)) {   // the pieces are w_hat itself
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (ok) mx_write_half<mode_mx_format(MODE)>(e.out, e.pad, piece[k] >> 1, half, x[k], a);
    return;
  }
  const Scale sc = make_scale(MODE == kFwdScaled ? gv : __fmul_rn(a, pow2_one_minus(gv)));
  if (mode_is_mx_fwd(MODE)) {
    uint32_t my = 0u;               // w_hat replaces w in the registers until the block maximum is known
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      sample_half(x[k], e.vec_lo + piece[k] * 2u, e.k0, e.k1, e.pre, sc, x[k]);
      my = maxabs2(my, maxabs2(absmax_words4(x[k]), absmax_words4(x[k] + 4)));
    }
    const float ay = absmax_finish(block_max(my));
#pragma unroll
    for (int k = 0; k < 4; ++k)
      if (ok) mx_write_half<mode_mx_format(MODE)>(e.out, e.pad, piece[k] >> 1, half, x[k], ay);
  } else {
#pragma unroll
    for (int k = 0; k < 4; ++k) {
      uint32_t y[8];
      sample_half(x[k], e.vec_lo + piece[k] * 2u, e.k0, e.k1, e.pre, sc, y);
      if (ok) st_vec32(e.out, static_cast<uint64_t>(piece[k]) * 32u, y);
    }
  }
  if (mode_is_fwd(MODE) && writer && e.gout != nullptr) st_f32(e.gout, g, sc.s);
}

// Host side: `bands[k]` = rows / 32 of record k.  Returns the number of tiles.
template <int CAP>
inline int64_t fill_square_batch(SquareBatch<CAP>& b, const SquareRec* recs, const uint32_t* bands, int count, uint32_t step_lo,
                                 uint32_t step_hi) {
  b.n = count;
  b.hint_shift = 0;
  int64_t tiles = 0;
  for (int k = 0; k < count; ++k) {
    b.e[k] = recs[k];
    b.e[k].tile_begin = static_cast<int32_t>(tiles);
    b.e[k].tiles_per_band = (recs[k].cpr + 8u * kSquareCpt - 1u) / (8u * kSquareCpt);
    b.e[k].pre = philox_pre(recs[k].vec_hi, step_lo, step_hi, recs[k].k0, recs[k].k1);
    tiles += static_cast<int64_t>(bands[k]) * b.e[k].tiles_per_band;
    if (tiles > 2147483647LL) return -1;
  }
  while (tiles > 0 && ((tiles - 1) >> b.hint_shift) >= kFlatHint) ++b.hint_shift;
  int owner = 0;
  for (int h = 0; h < kFlatHint; ++h) {
    const int64_t t = static_cast<int64_t>(h) << b.hint_shift;
    while (owner + 1 < count && b.e[owner + 1].tile_begin <= t) ++owner;
    b.hint[h] = static_cast<uint16_t>(owner);
  }
  return tiles;
}

// ---- whole-row groups on 64-byte chunks --------------------------------------------------------------
//
// Rows of a multiple of 32 elements, 32-byte aligned tensors.  T threads share a row (T = 1..32, a power
// of two: several rows per warp, shuffle reductions only; or T = 256: one row per block, one
// shared-memory step), each holding up to 4 chunks, T chunks apart, in registers between the max
// and the add, so W is read once.  Records by value in the kernel parameters, as for flat groups.
struct RowRec {
  const void* in;
  void* out;
  const float* gin;
  float* gout;
  uint32_t vec_lo, vec_hi;
  uint32_t rows, cpr;        // chunks per row = cols / 32
  uint32_t tpr_log2, cpt;    // threads per row (log2; 8 for the block kernel), chunks per thread (1..4)
  int32_t tile_begin;
  uint32_t k0, k1;
  PhiloxPre pre;
  uint32_t pad;
};
static_assert(sizeof(RowRec) == 88, "RowRec layout");
template <int CAP>
struct RowBatch {
  int32_t n;
  uint32_t hint_shift;
  uint32_t pad[2];
  uint16_t hint[kFlatHint];
  RowRec e[CAP];
};
constexpr int kRowCapSmall = 4, kRowCapLarge = 168;
constexpr int kRowThreads = 256, kRowMaxCpt = 4;

// Maximum over a row of the per-thread packed maxima: shuffles inside the `span` lanes that share the row, then (BLOCK)
// one shared-memory step.  AGAIN: red_u may still be read from an earlier use in this block.
template <bool BLOCK, bool AGAIN>
__device__ __forceinline__ uint32_t row_maxabs(uint32_t m, uint32_t span, uint32_t lane, uint32_t warp, uint32_t* red_u) {
  for (uint32_t o = 1; o < span; o <<= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
  if (BLOCK) {
    if (AGAIN) __syncthreads();
    if (lane == 0) red_u[warp] = m;
    __syncthreads();
    m = red_u[0];
#pragma unroll
    for (int w = 1; w < kRowThreads / 32; ++w) m = maxabs2(m, red_u[w]);
  }
  return m;
}

// MAXCPT (1..4): the chunks a thread holds in this launch; sizes the register arrays.
template <int MODE, bool BLOCK, int CAP, int MAXCPT>
__global__ void __launch_bounds__(kRowThreads) k_row(const __grid_constant__ RowBatch<CAP> b) {
  __shared__ uint32_t red_u[kRowThreads / 32];
  __shared__ float red_f[kRowThreads / 32];
  const int32_t tile = static_cast<int32_t>(blockIdx.x);
  int idx = b.hint[tile >> b.hint_shift];
  while (idx + 1 < b.n && b.e[idx + 1].tile_begin <= tile) ++idx;
  const RowRec& e = b.e[idx];
  const uint32_t tpr_log2 = BLOCK ? 8u : e.tpr_log2, tpr = 1u << tpr_log2;
  const uint32_t local = static_cast<uint32_t>(tile - e.tile_begin);
  const uint32_t row0 = BLOCK ? local : local * (kRowThreads >> tpr_log2) + (threadIdx.x >> tpr_log2);
  const uint32_t t = threadIdx.x & (tpr - 1u);
  const bool okr = row0 < e.rows;
  const uint32_t row = okr ? row0 : e.rows - 1u;   // keeps warps whole for the shuffles; nothing is stored for it
  const uint32_t cpr = e.cpr, cpt = e.cpt;
  const uint32_t row_chunk0 = row * cpr;
  wait_for_previous_kernel();

  Chunk c[MAXCPT];
  bool ok[MAXCPT];
#pragma unroll
  for (int k = 0; k < MAXCPT; ++k) {
    const uint32_t q = static_cast<uint32_t>(k) * tpr + t;
    ok[k] = static_cast<uint32_t>(k) < cpt && q < cpr;
    if (ok[k]) {
      c[k] = load_chunk<true>(e.in, row_chunk0 + q, 4);
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i) c[k].x[i] = 0u;
    }
  }
  const float gv = mode_reads_group_input(MODE) ? ld_f32(MODE == kFwdScaled ? e.gout : e.gin, row) : 0.0f;
  const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
  const uint32_t span = BLOCK ? 32u : tpr;   // lanes of this warp that share the row

  if (MODE == kBwd) {
    DotAcc dot;
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k) {
      if (!ok[k]) continue;
      const uint32_t chunk = row_chunk0 + static_cast<uint32_t>(k) * tpr + t;
      const uint32_t v0 = e.vec_lo + chunk * 4u;
#pragma unroll
      for (int v = 0; v < 4; ++v) {
        const Words4 r = philox4x32_10_pre(v0 + v, e.k0, e.k1, e.pre);
        dot_vec(make_uint4(c[k].x[4 * v], c[k].x[4 * v + 1], c[k].x[4 * v + 2], c[k].x[4 * v + 3]), r, dot);
      }
      if (okr && e.out != nullptr) store_chunk<true>(e.out, chunk, 4, c[k]);
    }
    float acc = dot.total();
    for (uint32_t o = 1; o < span; o <<= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (BLOCK) {
      if (lane == 0) red_f[warp] = acc;
      __syncthreads();
      acc = 0.0f;
#pragma unroll
      for (int w = 0; w < kRowThreads / 32; ++w) acc += red_f[w];   // fixed order
    }
    if (okr && t == 0u) st_f32(e.gout, row, grad_bt_of(gv, acc));
    return;
  }

  float a = 0.0f;
  if (MODE != kFwdScaled) {
    uint32_t m = 0u;
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k) m = maxabs2(m, absmax_chunk(c[k].x));
    a = absmax_finish(row_maxabs<BLOCK, false>(m, span, lane, warp, red_u));
  }
  if (MODE == kAbsmax) {
    if (okr && t == 0u) st_f32(e.gout, row, a);
    return;
  }
  if (mode_is_mx_quant(MODE)) {   // the chunks are w_hat itself
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k)
      if (ok[k] && okr) mx_write<mode_mx_format(MODE)>(e.out, e.pad, row_chunk0 + static_cast<uint32_t>(k) * tpr + t, c[k].x, a);
    return;
  }
  const Scale sc = make_scale(MODE == kFwdScaled ? gv : __fmul_rn(a, pow2_one_minus(gv)));
  if (mode_is_mx_fwd(MODE)) {
    // w_hat replaces w in the registers; its row maximum is known only after every chunk has been sampled
    uint32_t my = 0u;
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k) {
      if (!ok[k]) continue;
      const uint32_t chunk = row_chunk0 + static_cast<uint32_t>(k) * tpr + t;
      sample_chunk(c[k].x, e.vec_lo + chunk * 4u, e.k0, e.k1, e.pre, sc, c[k].x);
      my = maxabs2(my, absmax_chunk(c[k].x));
    }
    const float ay = absmax_finish(row_maxabs<BLOCK, true>(my, span, lane, warp, red_u));
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k)
      if (ok[k] && okr) mx_write<mode_mx_format(MODE)>(e.out, e.pad, row_chunk0 + static_cast<uint32_t>(k) * tpr + t, c[k].x, ay);
  } else {
#pragma unroll
    for (int k = 0; k < MAXCPT; ++k) {
      if (!ok[k]) continue;
      const uint32_t chunk = row_chunk0 + static_cast<uint32_t>(k) * tpr + t;
      const uint32_t v0 = e.vec_lo + chunk * 4u;
      Chunk y;
      sample_chunk(c[k].x, v0, e.k0, e.k1, e.pre, sc, y.x);
      if (okr) store_chunk<true>(e.out, chunk, 4, y);
    }
  }
  if (mode_is_fwd(MODE) && okr && t == 0u && e.gout != nullptr) st_f32(e.gout, row, sc.s);
}

// Host side: as fill_flat_batch.  Tiles: rows per block for shared rows (256 / threads per row), one row per block else.
template <int CAP>
inline int64_t fill_row_batch(RowBatch<CAP>& b, const RowRec* recs, int count, bool block, uint32_t step_lo, uint32_t step_hi) {
  b.n = count;
  b.hint_shift = 0;
  int64_t tiles = 0;
  for (int k = 0; k < count; ++k) {
    b.e[k] = recs[k];
    b.e[k].tile_begin = static_cast<int32_t>(tiles);
    b.e[k].pre = philox_pre(recs[k].vec_hi, step_lo, step_hi, recs[k].k0, recs[k].k1);
    const int64_t rows_per_tile = block ? 1 : (kRowThreads >> recs[k].tpr_log2);
    tiles += (static_cast<int64_t>(recs[k].rows) + rows_per_tile - 1) / rows_per_tile;
    if (tiles > 2147483647LL) return -1;
  }
  while (tiles > 0 && ((tiles - 1) >> b.hint_shift) >= kFlatHint) ++b.hint_shift;
  int owner = 0;
  for (int h = 0; h < kFlatHint; ++h) {
    const int64_t t = static_cast<int64_t>(h) << b.hint_shift;
    while (owner + 1 < count && b.e[owner + 1].tile_begin <= t) ++owner;
    b.hint[h] = static_cast<uint16_t>(owner);
  }
  return tiles;
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
  const float gvr = (MODE != kAbsmax && okr) ? ld_f32(MODE == kFwdScaled ? e.gout : e.gin, row) : 0.0f;

  if (MODE == kBwd) {
    DotAcc dot;
#pragma unroll
    for (int k = 0; k < V; ++k) {
      if (k * 32u < vpr) {
        const uint32_t j = k * 32u + lane;
        const bool ok = okr && j < vpr;
        // vectors past the end of the row are all zero and add nothing
        dot_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), dot);
        if (ok && e.out != nullptr) st_vec(e.out, vbase + j, x[k]);
      }
    }
    float acc = dot.total();
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (okr && lane == 0) st_f32(e.gout, row, grad_bt_of(gvr, acc));
  } else {
    float a = 0.0f;
    if (MODE != kFwdScaled) {
      uint32_t m = 0;
#pragma unroll
      for (int k = 0; k < V; ++k)
        if (k * 32u < vpr) m = maxabs2(m, absmax_vec(x[k]));
#pragma unroll
      for (uint32_t o = 16; o > 0; o >>= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      a = absmax_finish(m);
    }
    if (MODE == kAbsmax) {
      if (okr && lane == 0) st_f32(e.gout, row, a);
    } else {
      const Scale s = make_scale(MODE == kFwdScaled ? gvr : __fmul_rn(a, pow2_one_minus(gvr)));
#pragma unroll
      for (int k = 0; k < V; ++k) {
        if (k * 32u < vpr) {
          const uint32_t j = k * 32u + lane;
          const uint4 y = sample_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), s);
          if (okr && j < vpr) st_vec(e.out, vbase + j, y);
        }
      }
      if (MODE == kFwd && okr && lane == 0 && e.gout != nullptr) st_f32(e.gout, row, s.s);
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
  const float gvr = (MODE != kAbsmax) ? ld_f32(MODE == kFwdScaled ? e.gout : e.gin, row) : 0.0f;

  if (MODE == kBwd) {
    DotAcc dot;
#pragma unroll
    for (int k = 0; k < V; ++k) {
      if (static_cast<uint32_t>(k) * T < vpr) {
        const uint32_t j = k * T + threadIdx.x;
        dot_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), dot);   // zero vectors past the row add nothing
        if (j < vpr && e.out != nullptr) st_vec(e.out, vbase + j, x[k]);
      }
    }
    float acc = dot.total();
#pragma unroll
    for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
    if (lane == 0) red_f[warp] = acc;
    __syncthreads();
    if (threadIdx.x == 0) {
      float total = 0.0f;
      for (int w = 0; w < WARPS; ++w) total += red_f[w];  // fixed order
      st_f32(e.gout, row, grad_bt_of(gvr, total));
    }
  } else {
    float a = 0.0f;
    if (MODE != kFwdScaled) {
      uint32_t m = 0;
#pragma unroll
      for (int k = 0; k < V; ++k)
        if (static_cast<uint32_t>(k) * T < vpr) m = maxabs2(m, absmax_vec(x[k]));
#pragma unroll
      for (uint32_t o = 16; o > 0; o >>= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
      if (lane == 0) red_u[warp] = m;
      __syncthreads();
      uint32_t mm = red_u[0];
#pragma unroll
      for (int w = 1; w < WARPS; ++w) mm = maxabs2(mm, red_u[w]);
      a = absmax_finish(mm);
    }
    if (MODE == kAbsmax) {
      if (threadIdx.x == 0) st_f32(e.gout, row, a);
    } else {
      const Scale s = make_scale(MODE == kFwdScaled ? gvr : __fmul_rn(a, pow2_one_minus(gvr)));
#pragma unroll
      for (int k = 0; k < V; ++k) {
        if (static_cast<uint32_t>(k) * T < vpr) {
          const uint32_t j = k * T + threadIdx.x;
          const uint4 y = sample_vec(x[k], philox_vec(e, vbase + j, step_lo, step_hi), s);
          if (j < vpr) st_vec(e.out, vbase + j, y);
        }
      }
      if (MODE == kFwd && threadIdx.x == 0 && e.gout != nullptr) st_f32(e.gout, row, s.s);
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
    if (MODE == kFwdScaled) scale = ld_f32(e.gout, g);
    if (MODE == kAbsmax || MODE == kFwd) {
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
        uint32_t pairs[4];
        decode8(words, pairs);
        const int r = r_from_pairs(pairs, static_cast<unsigned>(el & 7u));
        const uint16_t bits = ld_u16(in, i * e.ld + j);
        const float val = __uint_as_float(static_cast<uint32_t>(bits) << 16);
        if (MODE == kFwd || MODE == kFwdScaled) {
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

// The arithmetic the forward and backward kernels spend on noise (hoisted Philox rounds + whole-word decode)
// with no memory traffic: 8 vectors per thread, one stored word per block.
__global__ void __launch_bounds__(256) k_noise_probe(uint32_t* __restrict__ sink, uint64_t n_words, uint64_t vec0,
                                                     uint32_t seed_lo, uint32_t seed_hi, uint32_t step_lo,
                                                     uint32_t step_hi) {
  __shared__ uint32_t red[8];
  uint32_t acc = 0;
  // one set of hoisted constants per block, as in the sampling kernels (its 2048 vectors share the high counter
  // word unless the block straddles a multiple of 2^32, which only changes the value of this probe's sink)
  const uint64_t block_vec0 = vec0 + static_cast<uint64_t>(blockIdx.x) * 2048u;
  const PhiloxPre pre = philox_pre(static_cast<uint32_t>(block_vec0 >> 32), step_lo, step_hi, seed_lo, seed_hi);
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const uint64_t v = (static_cast<uint64_t>(blockIdx.x) * 8u + k) * 256u + threadIdx.x;
    if (v < n_words) {
      const uint64_t vec = vec0 + v;
      uint32_t p[4];
      decode8(philox4x32_10_pre(static_cast<uint32_t>(vec), seed_lo, seed_hi, pre), p);
      acc ^= p[0] ^ p[1] ^ p[2] ^ p[3];
    }
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

// s_g = fl32(absmax_g * 2^(1 - b_g)) for a run of groups whose maxima were taken (and, for a sharded tensor,
// reduced across shards) beforehand: the factor of Eq. 3 as the fused forward kernels form it.
__global__ void __launch_bounds__(256) k_scale(const float* __restrict__ absmax, const float* __restrict__ bt,
                                               float* __restrict__ scale, int64_t n) {
  for (int64_t k = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; k < n; k += static_cast<int64_t>(gridDim.x) * 256)
    st_f32(scale, k, __fmul_rn(ld_f32(absmax, k), pow2_one_minus(ld_f32(bt, k))));
}

// ---- bit-width parametrisation (Eq. 11), its loss term (Eq. 12) and the chain rule back to b_i ----------

// b_t = fl(b_target + fl(b_i * delta)), delta = fl(b_init - b_target): one rounding per operation.
__global__ void __launch_bounds__(256) k_bitwidth(const float* __restrict__ bi, float delta, float b_target, float* __restrict__ bt,
                                                  int64_t n) {
  for (int64_t k = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; k < n; k += static_cast<int64_t>(gridDim.x) * 256)
    st_f32(bt, k, __fadd_rn(b_target, __fmul_rn(ld_f32(bi, k), delta)));
}

// dL'/db_i = delta * (dL/db_t + lam_over_m * sign(b_t - b_target)); sign(0) = 0.
__global__ void __launch_bounds__(256) k_bitwidth_grad(const float* __restrict__ grad_bt, const float* __restrict__ bt, float delta,
                                                       float b_target, float lam_over_m, float* __restrict__ grad_bi, int64_t n) {
  for (int64_t k = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x; k < n; k += static_cast<int64_t>(gridDim.x) * 256) {
    const float x = __fsub_rn(ld_f32(bt, k), b_target);
    const float sign = x > 0.0f ? 1.0f : (x < 0.0f ? -1.0f : 0.0f);
    st_f32(grad_bi, k, __fmul_rn(delta, __fadd_rn(ld_f32(grad_bt, k), __fmul_rn(lam_over_m, sign))));
  }
}

// mean_k |b_t,k - b_target| of one layer: one block, every thread a strided partial sum, combined in a fixed order.
__global__ void __launch_bounds__(1024) k_bitwidth_loss(const float* __restrict__ bt, float b_target, float* __restrict__ out,
                                                        int64_t m) {
  __shared__ float red[32];
  float acc = 0.0f;
  for (int64_t k = threadIdx.x; k < m; k += 1024) acc += fabsf(__fsub_rn(ld_f32(bt, k), b_target));
#pragma unroll
  for (uint32_t o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
  if ((threadIdx.x & 31u) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float total = 0.0f;
    for (int w = 0; w < 32; ++w) total += red[w];
    st_f32(out, 0, total / static_cast<float>(m));
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
