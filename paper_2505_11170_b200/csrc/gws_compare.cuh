// Comparison noises on the forward pass: the same kernel shape as the flat-group forward (a thread owns 64-byte chunks, the
// lanes of a group reduce its maximum by shuffles, 32-byte accesses), with the noise of Eq. 3 replaced by
//   * BF16 U(-0.5, 0.5): the paper's "DiffQ" extension (Section 4, first paragraph).  Element e takes the 16-bit field at bits
//     [16 (e & 1), +16) of word (e >> 1) & 3 of the Philox output of vector e >> 3; u = bf16((x + 1/2) / 2^16 - 1/2);
//   * the rounded normal itself, R = round-half-even(N(0, 1) / 2), with the normals from the Box-Muller transform (Section 3.4;
//     the "bm" series of the paper's forward benchmark).  One Philox call, counter e >> 2, serves 4 elements: words (o0, o1)
//     give elements 4c and 4c + 1, (o2, o3) give 4c + 2 and 4c + 3; u1 = ((a >> 8) + 1) / 2^24, u2 = (b >> 8) / 2^24,
//     z = sqrt(-2 ln u1) * (cos, sin)(2 pi u2), evaluated in FP32.
// These exist to time the method's AND / OR generation against what it replaces, on one harness; they are not part of the
// sampling pass.  w_hat = bf16( fl32( float(w) + fl32( noise * s_g ) ) ) with s_g as in the forward pass.
#pragma once
#include "gws_kernels.cuh"

namespace gws {

enum NoiseKind { kNoiseUniformBf16 = 0, kNoiseBoxMuller = 1 };

__device__ __forceinline__ uint32_t uniform_bf16_bits(uint32_t x16) {
  // (2x + 1 - 65536) / 2^17 is exact in FP32; one rounding to BF16
  const float f = __fmul_rn(__int2float_rn(static_cast<int>(2u * x16 + 1u) - 65536), 0x1p-17f);
  return pack_bf16_rne(f, 0.0f) & 0xFFFFu;
}
__device__ __forceinline__ void box_muller(uint32_t a, uint32_t b, float& z0, float& z1) {
  const float u1 = __fmul_rn(__uint2float_rn((a >> 8) + 1u), 0x1p-24f), u2 = __fmul_rn(__uint2float_rn(b >> 8), 0x1p-24f);
  const float radius = sqrtf(__fmul_rn(-2.0f, logf(u1)));
  float s, c;
  sincospif(__fmul_rn(2.0f, u2), &s, &c);
  z0 = __fmul_rn(radius, c);
  z1 = __fmul_rn(radius, s);
}
__device__ __forceinline__ float rounded_half(float z) { return rintf(__fmul_rn(0.5f, z)); }

// Noise of the 8 elements of vector `k` of a chunk as FP32 numbers.  Uniform: ctr0 counts vectors (e >> 3); Box-Muller: ctr0
// counts quadruples (e >> 2), two calls per vector.
template <int KIND>
__device__ __forceinline__ void noise8(uint32_t ctr0, uint32_t k, uint32_t k0, uint32_t k1, const PhiloxPre& pre, float (&r)[8]) {
  if (KIND == kNoiseUniformBf16) {
    const Words4 o = philox4x32_10_pre(ctr0 + k, k0, k1, pre);
#pragma unroll
    for (int t = 0; t < 8; ++t) r[t] = __uint_as_float(uniform_bf16_bits((o.o[t >> 1] >> (16 * (t & 1))) & 0xFFFFu) << 16);
  } else {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const Words4 o = philox4x32_10_pre(ctr0 + 2u * k + h, k0, k1, pre);
      float z0, z1;
      box_muller(o.o[0], o.o[1], z0, z1);
      r[4 * h + 0] = rounded_half(z0);
      r[4 * h + 1] = rounded_half(z1);
      box_muller(o.o[2], o.o[3], z0, z1);
      r[4 * h + 2] = rounded_half(z0);
      r[4 * h + 3] = rounded_half(z1);
    }
  }
}

struct CompareArgs {
  const void* w;
  const float* bt;
  void* w_hat;
  float* scale_out;
  uint32_t n_chunks, lanes_log2;   // chunks of 32 elements; log2(chunks per group)
  uint32_t ctr_lo;                 // low counter word of the tensor's first vector (uniform) or quadruple (Box-Muller)
  uint32_t k0, k1;
  PhiloxPre pre;
};

template <int KIND>
__global__ void __launch_bounds__(kFlatThreads) k_compare_fwd(const __grid_constant__ CompareArgs a) {
  constexpr int kCpt = 2;
  const uint32_t first = blockIdx.x * (kFlatThreads * kCpt) + threadIdx.x;
  const uint32_t lanes = 1u << a.lanes_log2;
  const bool writer_lane = (threadIdx.x & (lanes - 1u)) == 0u;
  uint32_t chunk[kCpt];
  bool ok[kCpt];
  Chunk c[kCpt];
  float bits[kCpt];
#pragma unroll
  for (int i = 0; i < kCpt; ++i) {
    const uint32_t chunk0 = first + static_cast<uint32_t>(i) * kFlatThreads;
    ok[i] = chunk0 < a.n_chunks;
    chunk[i] = ok[i] ? chunk0 : a.n_chunks - 1u;   // keeps the warp whole for the shuffles
    c[i] = load_chunk<true>(a.w, chunk[i], 4);
    bits[i] = ld_f32(a.bt, chunk[i] >> a.lanes_log2);
  }
#pragma unroll
  for (int i = 0; i < kCpt; ++i) {
    uint32_t m = absmax_chunk(c[i].x);
    for (uint32_t o = 1; o < lanes; o <<= 1) m = maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
    const float s = __fmul_rn(absmax_finish(m), pow2_one_minus(bits[i]));
    const uint32_t ctr0 = a.ctr_lo + chunk[i] * (KIND == kNoiseUniformBf16 ? 4u : 8u);
    Chunk y;
#pragma unroll
    for (uint32_t k = 0; k < 4; ++k) {
      float r[8];
      noise8<KIND>(ctr0, k, a.k0, a.k1, a.pre, r);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint32_t wv = c[i].x[4 * k + j];
        const float lo = __fadd_rn(__uint_as_float(wv << 16), __fmul_rn(r[2 * j], s));
        const float hi = __fadd_rn(__uint_as_float(wv & 0xFFFF0000u), __fmul_rn(r[2 * j + 1], s));
        y.x[4 * k + j] = pack_bf16_rne(lo, hi);
      }
    }
    if (ok[i]) store_chunk<true>(a.w_hat, chunk[i], 4, y);
    if (ok[i] && writer_lane && a.scale_out != nullptr) st_f32(a.scale_out, chunk[i] >> a.lanes_log2, s);
  }
}

// The noise alone.  Uniform: one BF16 pattern per element (u16 [n]); Box-Muller: sign-magnitude nibbles, 8 per u32 (|R| <= 3),
// nibble t of word e >> 3 at bits [4t, 4t + 3], zero never negative: the packed format of Section 3.4.
template <int KIND>
__global__ void __launch_bounds__(256) k_compare_noise(void* __restrict__ out, uint32_t n_vec, uint32_t ctr_lo, uint32_t k0, uint32_t k1,
                                                       PhiloxPre pre) {
  const uint32_t v = blockIdx.x * 256u + threadIdx.x;
  if (v >= n_vec) return;
  float r[8];
  noise8<KIND>(ctr_lo, v, k0, k1, pre, r);
  if (KIND == kNoiseUniformBf16) {
    uint32_t p[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) p[j] = (__float_as_uint(r[2 * j]) >> 16) | (__float_as_uint(r[2 * j + 1]) & 0xFFFF0000u);
    st_vec(out, v, make_uint4(p[0], p[1], p[2], p[3]));
  } else {
    uint32_t word = 0;
#pragma unroll
    for (int t = 0; t < 8; ++t) {
      const int ri = __float2int_rn(r[t]);
      const uint32_t mag = static_cast<uint32_t>(ri < 0 ? -ri : ri);
      word |= ((ri < 0 ? 8u : 0u) | mag) << (4 * t);
    }
    st_u32(out, static_cast<uint64_t>(v) * 4u, word);
  }
}

}  // namespace gws
