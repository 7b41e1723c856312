// Inline arithmetic of the sampling pass: Philox4x32-10, the AND/OR noise decode of
// Eq. 9 / Eq. 10 and the nibble packing of Section 3.4.  Integer-only, so the same
// code runs in kernels and (for host-side tests of the bit tricks) on the CPU.
#pragma once
#include <stdint.h>

#if defined(__CUDACC__)
#define GWS_HD __host__ __device__ __forceinline__
#else
#define GWS_HD inline
#endif

namespace gws {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

struct Words4 {
  uint32_t o[4];
};

// Ten rounds of the Philox4x32 block function.  Counter (c0..c3), key (k0, k1).
GWS_HD Words4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c0;
    const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * c2;
    // round key r is k + r*W (mod 2^32); r*W folds to a constant after unrolling
    const uint32_t rk0 = k0 + static_cast<uint32_t>(r) * kPhiloxW0;
    const uint32_t rk1 = k1 + static_cast<uint32_t>(r) * kPhiloxW1;
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ rk0;
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ rk1;
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
  }
  Words4 w;
  w.o[0] = c0; w.o[1] = c1; w.o[2] = c2; w.o[3] = c3;
  return w;
}

// Random words of the 8-element vector number `vec` (vec = logical element index >> 3).
GWS_HD Words4 philox_for_vector(uint64_t vec, uint32_t step_lo, uint32_t step_hi, uint32_t seed_lo, uint32_t seed_hi) {
  return philox4x32_10(static_cast<uint32_t>(vec), static_cast<uint32_t>(vec >> 32), step_lo, step_hi, seed_lo, seed_hi);
}

// Byte permute with the semantics of the PTX prmt instruction in its default mode,
// selector nibbles restricted to 0..7 (no sign replication).
GWS_HD uint32_t byte_perm(uint32_t a, uint32_t b, uint32_t sel) {
#if defined(__CUDA_ARCH__)
  return __byte_perm(a, b, sel);
#else
  const uint64_t both = (static_cast<uint64_t>(b) << 32) | a;
  uint32_t out = 0;
  for (int k = 0; k < 4; ++k) {
    const uint32_t idx = (sel >> (4 * k)) & 7u;
    out |= static_cast<uint32_t>((both >> (8 * idx)) & 0xFFu) << (8 * k);
  }
  return out;
#endif
}

// Decode four 16-bit fields (two Philox words) at once, one byte lane per field.
//
// Field bits x0..x15; hi byte y = x8..x15, lo byte l = x0..x7.
//   m2 = (l == 0xFF) & (x8|x9)          |R| = 2
//   m1 = (x10|x11) & (x12|x13) & x14    |R| = 1 unless m2
// Output: two words, each holding two elements as the upper halves of FP32 bit patterns,
// element (2k) in bits 0..15 and element (2k+1) in bits 16..31 of p[k]:
//   bit 15: x15 (raw sign), bit 8: m2, bit 7: m1 & ~m2, all other bits 0.
// Shifted into the top of a 32-bit word this is sign | exponent field 2 or 1, i.e.
// +-2^-125 or +-2^-126 (or +-0): multiply by 2^126 to get float(R) (with R = 0 possibly -0.0).
GWS_HD void decode4(uint32_t wa, uint32_t wb, uint32_t& p01, uint32_t& p23) {
  const uint32_t H = byte_perm(wa, wb, 0x7531u);  // hi bytes of fields 0..3
  const uint32_t L = byte_perm(wa, wb, 0x6420u);  // lo bytes of fields 0..3
  const uint32_t a = H | (H >> 1);                // per byte: bit0 = x8|x9, bit2 = x10|x11, bit4 = x12|x13
  const uint32_t M1 = (a << 4) & (a << 2) & H;    // per byte bit 6 = m1
  const uint32_t c = (L & 0x7F7F7F7Fu) + 0x01010101u;  // per byte bit 7 = (x0..x6 all ones)
  const uint32_t M2 = c & L & (a << 7);           // per byte bit 7 = m2
  const uint32_t C = (H & 0x80808080u) | ((M2 >> 7) & 0x01010101u);  // sign at bit 7, m2 at bit 0
  const uint32_t A = ((M1 << 1) & ~M2) & 0x80808080u;                // m1 & ~m2 at bit 7
  p01 = byte_perm(C, A, 0x1504u);
  p23 = byte_perm(C, A, 0x3726u);
}

// Plain per-field decode, straight from the definition (used by the general kernel,
// the noise packer and as the cross-check of decode4).
GWS_HD int decode_field(uint32_t x) {
  const bool m2 = ((x & 0xFFu) == 0xFFu) && ((x & 0x300u) != 0u);
  const bool m1 = ((x & 0xC00u) != 0u) && ((x & 0x3000u) != 0u) && ((x & 0x4000u) != 0u);
  const int mag = m2 ? 2 : (m1 ? 1 : 0);
  return (x & 0x8000u) ? -mag : mag;
}

GWS_HD uint32_t field_of(const Words4& w, unsigned t) { return (w.o[t >> 1] >> (16u * (t & 1u))) & 0xFFFFu; }

// R of field t (0..7) recovered from the decode4 outputs.
GWS_HD int r_from_pair(uint32_t pair, unsigned odd) {
  const uint32_t h = (pair >> (16u * odd)) & 0xFFFFu;
  const int mag = static_cast<int>((h >> 7) & 3u);  // 1 or 2 (never 3)
  return (h & 0x8000u) ? -mag : mag;
}

// Packed sign-magnitude nibbles of 8 elements; zero is never negative.
GWS_HD uint32_t pack_nibbles(const Words4& w) {
  uint32_t p[4];
  decode4(w.o[0], w.o[1], p[0], p[1]);
  decode4(w.o[2], w.o[3], p[2], p[3]);
  uint32_t out = 0;
#pragma unroll
  for (unsigned t = 0; t < 8; ++t) {
    const uint32_t h = (p[t >> 1] >> (16u * (t & 1u))) & 0xFFFFu;
    const uint32_t mag = (h >> 7) & 3u;
    const uint32_t neg = (mag != 0u) ? (h >> 15) : 0u;
    out |= ((neg << 3) | mag) << (4u * t);
  }
  return out;
}

}  // namespace gws
