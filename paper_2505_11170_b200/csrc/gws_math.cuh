// Inline integer arithmetic of the sampling pass: Philox4x32-10, the AND/OR noise decode of
// Eq. 9 / Eq. 10 on whole random words, and the nibble packing of Section 3.4.  Integer-only,
// so the same code runs in kernels and (for host-side tests of the bit tricks) on the CPU.
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

// Rounds of the Philox4x32 block function.  The library, its oracle and every test use 10.  The switch
// exists only to measure how much of the backward pass is random-bit generation (a build with another
// value has no oracle to be checked against).
#ifndef GWS_PHILOX_ROUNDS
#define GWS_PHILOX_ROUNDS 10
#endif
static_assert(GWS_PHILOX_ROUNDS >= 2, "the hoisted form below takes rounds 1 and 2 apart");

// Ten rounds of the Philox4x32 block function.  Counter (c0..c3), key (k0, k1).
GWS_HD Words4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1) {
#pragma unroll
  for (int r = 0; r < GWS_PHILOX_ROUNDS; ++r) {
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

// The same function with the launch-uniform part of the first two rounds taken out.  Of the counter
// (v_lo, v_hi, step_lo, step_hi) only v_lo differs between the vectors of one tensor (a tensor whose
// vectors straddle a multiple of 2^32 is not given to the kernels that use this).  Round 1 then needs
// one of its two multiplies (M1 * step_lo is uniform), and its new c0 is uniform, so round 2 needs
// one as well: 18 wide multiplies and 19 XORs per call instead of 20 and 20.
struct PhiloxPre {
  uint32_t x3;   // step_hi ^ k1                          -> c2 after round 1 = hi(M0 * v_lo) ^ x3
  uint32_t y0;   // lo(M1 * step_lo) ^ (k0 + W0)          -> c0 after round 2 = hi(M1 * c2) ^ y0
  uint32_t y2;   // hi(M0 * a0) ^ (k1 + W1)               -> c2 after round 2 = c3 ^ y2
  uint32_t l3;   // lo(M0 * a0)                           =  c3 after round 2,  a0 = hi(M1*step_lo) ^ v_hi ^ k0
};
GWS_HD PhiloxPre philox_pre(uint32_t v_hi, uint32_t step_lo, uint32_t step_hi, uint32_t k0, uint32_t k1) {
  const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * step_lo;
  const uint32_t a0 = static_cast<uint32_t>(p1 >> 32) ^ v_hi ^ k0;
  const uint64_t pa = static_cast<uint64_t>(kPhiloxM0) * a0;
  PhiloxPre q;
  q.x3 = step_hi ^ k1;
  q.y0 = static_cast<uint32_t>(p1) ^ (k0 + kPhiloxW0);
  q.y2 = static_cast<uint32_t>(pa >> 32) ^ (k1 + kPhiloxW1);
  q.l3 = static_cast<uint32_t>(pa);
  return q;
}
GWS_HD Words4 philox4x32_10_pre(uint32_t v_lo, uint32_t k0, uint32_t k1, const PhiloxPre& q) {
  // round 1
  const uint64_t r1 = static_cast<uint64_t>(kPhiloxM0) * v_lo;
  uint32_t c2 = static_cast<uint32_t>(r1 >> 32) ^ q.x3;
  uint32_t c3 = static_cast<uint32_t>(r1);
  // round 2
  const uint64_t r2 = static_cast<uint64_t>(kPhiloxM1) * c2;
  uint32_t c0 = static_cast<uint32_t>(r2 >> 32) ^ q.y0;
  uint32_t c1 = static_cast<uint32_t>(r2);
  c2 = c3 ^ q.y2;
  c3 = q.l3;
#pragma unroll
  for (int r = 2; r < GWS_PHILOX_ROUNDS; ++r) {
    const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c0;
    const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * c2;
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ (k0 + static_cast<uint32_t>(r) * kPhiloxW0);
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ (k1 + static_cast<uint32_t>(r) * kPhiloxW1);
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
  }
  Words4 w;
  w.o[0] = c0; w.o[1] = c1; w.o[2] = c2; w.o[3] = c3;
  return w;
}

// ---- noise decode on whole words ------------------------------------------------------------------
//
// Element t of a vector (j = t >> 1, h = t & 1) owns four bit columns of the four output words
// o0..o3:  A = 16h + 14 - 2j,  S = A + 1,  M = A - 7,  F = A - 8.  With o_k[c] = bit c of word k:
//
//   |R| = 2  iff  o0[M] & o1[M] & o2[M] & o3[M] & o1[F] & o2[F] & o3[F] & o0[S] & (o1[S] | o2[S])   Pr = 2^-8 * 3/4
//   |R| = 1  iff  not that, and (o0[A] | o1[A]) & (o2[A] | o3[A]) & o0[F]                           Pr = (3/4)^2 / 2
//   R < 0    iff  o3[S] and |R| != 0
//
// Every AND / OR below therefore evaluates one term of Eq. 10 for all eight elements at once; shifts
// only line up columns (M + 7 = A, F + 8 = A, S - 8 = M, F + 1 = M).  The columns are laid out so
// that `Z << 2j` brings the three flags of elements 2j (low half) and 2j+1 (high half) to bits
// 15 (sign), 14 (non-zero) and 7 (|R| = 2) of each 16-bit half: with all other bits cleared that
// half is the BF16 number 2R (0x4000 = 2.0, 0x4080 = 4.0, sign on top), and zero is always +0.
constexpr uint32_t kColsM = 0x00AA00AAu;   // bit columns M of the eight elements
constexpr uint32_t kColsS = 0xAA00AA00u;   // bit columns S
constexpr uint32_t kPairMask = 0xC080C080u;

GWS_HD void decode8(const Words4& r, uint32_t (&pair)[4]) {
  const uint32_t o0 = r.o[0], o1 = r.o[1], o2 = r.o[2], o3 = r.o[3];
  const uint32_t t1 = o1 & o2 & o3;
  const uint32_t and7 = t1 & o0 & (t1 << 1);        // at M: o0..o3[M] & o1..o3[F]
  const uint32_t top = o0 & (o1 | o2);              // at S: o0[S] & (o1[S] | o2[S])
  const uint32_t m2 = and7 & (top >> 8);            // at M
  const uint32_t m1 = (o0 | o1) & (o0 << 8) & (o2 | o3);   // at A
  const uint32_t any = m1 | (m2 << 7);              // at A
  const uint32_t z1 = (any & ~kColsM) | (m2 & kColsM);
  const uint32_t sgn = o3 & (any << 1);             // at S; zero noise keeps a positive sign
  const uint32_t z = (sgn & kColsS) | (z1 & ~kColsS);
  pair[0] = z & kPairMask;
  pair[1] = (z << 2) & kPairMask;
  pair[2] = (z << 4) & kPairMask;
  pair[3] = (z << 6) & kPairMask;
}

// The same decode for consumers that only multiply by the noise (the gradient sum of Eq. 4): a zero may come out as
// -0, because the sign column is taken as it is instead of being cleared where |R| = 0.  Two operations fewer.
GWS_HD void decode8_signed_zero(const Words4& r, uint32_t (&pair)[4]) {
  const uint32_t o0 = r.o[0], o1 = r.o[1], o2 = r.o[2], o3 = r.o[3];
  const uint32_t t1 = o1 & o2 & o3;
  const uint32_t and7 = t1 & o0 & (t1 << 1);
  const uint32_t top = o0 & (o1 | o2);
  const uint32_t m2 = and7 & (top >> 8);
  const uint32_t m1 = (o0 | o1) & (o0 << 8) & (o2 | o3);
  const uint32_t any = m1 | (m2 << 7);
  const uint32_t z1 = (any & ~kColsM) | (m2 & kColsM);
  const uint32_t z = (o3 & kColsS) | (z1 & ~kColsS);
  pair[0] = z & kPairMask;
  pair[1] = (z << 2) & kPairMask;
  pair[2] = (z << 4) & kPairMask;
  pair[3] = (z << 6) & kPairMask;
}

// R of element t (0..7) from the pair words of its vector.
GWS_HD int r_from_pairs(const uint32_t (&pair)[4], unsigned t) {
  const uint32_t h = (pair[t >> 1] >> (16u * (t & 1u))) & 0xFFFFu;
  const int mag = static_cast<int>(((h >> 14) & 1u) + ((h >> 7) & 1u));
  return (h & 0x8000u) ? -mag : mag;
}

// Packed sign-magnitude nibbles of 8 elements (nibble t = sign << 3 | |R|); zero is never negative.
GWS_HD uint32_t pack_nibbles(const Words4& w) {
  uint32_t pair[4];
  decode8(w, pair);
  uint32_t out = 0;
#pragma unroll
  for (unsigned t = 0; t < 8; ++t) {
    const uint32_t h = (pair[t >> 1] >> (16u * (t & 1u))) & 0xFFFFu;
    const uint32_t mag = ((h >> 14) & 1u) + ((h >> 7) & 1u);
    out |= (((h >> 15) << 3) | mag) << (4u * t);
  }
  return out;
}

}  // namespace gws
