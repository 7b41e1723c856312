// Issue-cost probes: how many cycles an SM sub-partition needs per warp instruction for the instruction kinds the
// sampling pass is made of, alone and mixed, and for the arithmetic of the backward pass with no memory traffic.
//
// The passes spend their time on Philox4x32-10 (per 8 elements 18 multiplies 32 x 32 -> 64 and 19 three-input XORs)
// and on the AND / OR decode of Eq. 10.  These kernels measure what that instruction mix costs on the chip at hand, so
// that the arithmetic ceiling quoted for the backward pass is a sum of measured per-instruction costs and not the rate
// of another kernel of this library.  Every chain is data dependent on its own previous result, every result is
// consumed, every thread runs 4 independent chains of each kind and every SM holds 64 warps.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "gws_kernels.cuh"

namespace gws {

// One step of one chain = NW multiplies 32 x 32 -> 64 by a constant + NW XORs of the high half with the other state
// word and a round key (NW = 2: one Philox round), K more three-input logic operations, F FP32 fused multiply-adds,
// B mixed-precision (FP32 += BF16 * BF16) fused multiply-adds, I integer additions, P byte permutes.
template <int NW, int K, int F, int B, int I, int P>
__global__ void __launch_bounds__(256) k_issue_probe(uint32_t* __restrict__ sink, uint32_t k0, uint32_t k1, float f0, int iterations) {
  uint32_t c0[4], c1[4], c2[4], c3[4], x[4], y[4], z[4], q[4];
  float f[4], h[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    c0[i] = threadIdx.x * 7u + i + blockIdx.x;
    c1[i] = threadIdx.x * 13u + i;
    c2[i] = c0[i] ^ 0x5555u;
    c3[i] = c1[i] + 77u;
    x[i] = c0[i] + 5u;
    y[i] = c1[i] ^ 0x77u;
    z[i] = x[i] * 3u;
    q[i] = y[i] + 9u;
    f[i] = static_cast<float>(threadIdx.x + i);
    h[i] = f[i] + 1.0f;
  }
  unsigned long long ns0 = 0, ns1 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns0));
  const long long t0 = clock64();
#pragma unroll 1
  for (int it = 0; it < iterations; ++it) {
#pragma unroll
    for (int r = 0; r < 8; ++r) {
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (NW == 2) {
          const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c0[i];
          const uint64_t p1 = static_cast<uint64_t>(kPhiloxM1) * c2[i];
          const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1[i] ^ (k0 + static_cast<uint32_t>(r) * kPhiloxW0);
          const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3[i] ^ (k1 + static_cast<uint32_t>(r) * kPhiloxW1);
          c1[i] = static_cast<uint32_t>(p1);
          c3[i] = static_cast<uint32_t>(p0);
          c0[i] = n0;
          c2[i] = n2;
        } else if (NW == 1) {
          const uint64_t p0 = static_cast<uint64_t>(kPhiloxM0) * c0[i];
          c0[i] = static_cast<uint32_t>(p0 >> 32) ^ c1[i] ^ (k0 + static_cast<uint32_t>(r) * kPhiloxW0);
          c1[i] = static_cast<uint32_t>(p0);
        }
#pragma unroll
        for (int l = 0; l < K; ++l) asm volatile("lop3.b32 %0, %0, %1, %2, 0xE8;" : "+r"(x[i]) : "r"(y[i]), "r"(k0));
#pragma unroll
        for (int l = 0; l < F; ++l) asm volatile("fma.rn.f32 %0, %0, %1, %1;" : "+f"(f[i]) : "f"(f0));
#pragma unroll
        for (int l = 0; l < B; ++l)
          asm volatile("{ .reg .b16 lo, hi; mov.b32 {lo, hi}, %1; fma.rn.f32.bf16 %0, lo, hi, %0; }" : "+f"(h[i]) : "r"(y[i]));
#pragma unroll
        for (int l = 0; l < I; ++l) asm volatile("add.u32 %0, %0, %1;" : "+r"(z[i]) : "r"(y[i]));
#pragma unroll
        for (int l = 0; l < P; ++l) asm volatile("prmt.b32 %0, %0, %1, 0x1032;" : "+r"(q[i]) : "r"(y[i]));
      }
    }
  }
  const long long t1 = clock64();
  uint32_t acc = 0;
  float facc = 0.0f;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    acc ^= c0[i] ^ c1[i] ^ c2[i] ^ c3[i] ^ x[i] ^ z[i] ^ q[i];
    facc += f[i] + h[i];
  }
  if (acc == k1 && facc == f0) sink[4] = acc;   // never true in practice: keeps every chain alive
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    sink[0] = static_cast<uint32_t>(t1 - t0);              // SM cycles of one warp from first to last step
    sink[1] = static_cast<uint32_t>(ns1 - ns0);            // the same span in nanoseconds: sink[0] / sink[1] = SM clock in GHz
  }
}

// The arithmetic of one pass over `vectors` 8-element vectors per thread with no memory traffic.
// PIECES: 1 = Philox4x32-10 (hoisted form), 2 = decode of the gradient sum, 4 = the 8 mixed-precision FMAs of the sum,
// 8 = forward instead: decode with the sign of zero cleared, Eq. 3's add (one FMA per element) and the BF16 packing.
template <int PIECES>
__global__ void __launch_bounds__(256) k_body_probe(uint32_t* __restrict__ sink, uint32_t k0, uint32_t k1, PhiloxPre pre, uint32_t g0,
                                                    int vectors) {
  uint32_t gw[4] = {g0 ^ threadIdx.x, g0 * 3u + threadIdx.x, g0 + 0x3F803F80u, g0 ^ 0x40004000u};
  DotAcc acc;
  uint32_t xacc = 0;
  const Scale sc = make_scale(__uint_as_float(0x3C000000u + (threadIdx.x << 16)));
  unsigned long long ns0 = 0, ns1 = 0;
  if (blockIdx.x == 0 && threadIdx.x == 0) asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns0));
  const long long t0 = clock64();
  uint32_t v = (blockIdx.x * 256u + threadIdx.x) * static_cast<uint32_t>(vectors);
#pragma unroll 1
  for (int it = 0; it < vectors; it += 4) {
#pragma unroll
    for (int s = 0; s < 4; ++s) {
      Words4 w;
      if (PIECES & 1) {
        w = philox4x32_10_pre(v + s, k0, k1, pre);
      } else {
        w.o[0] = v + s; w.o[1] = (v + s) * 3u; w.o[2] = (v + s) ^ k0; w.o[3] = (v + s) + k1;
      }
      uint32_t p[4];
      if (PIECES & 8) {
        decode8(w, p);
#pragma unroll
        for (int j = 0; j < 4; ++j) xacc ^= sample_pair_t<2>(gw[j], p[j], sc);
      } else {
        if (PIECES & 2) decode8_signed_zero(w, p);
        else { p[0] = w.o[0]; p[1] = w.o[1]; p[2] = w.o[2]; p[3] = w.o[3]; }
        if (PIECES & 4) {
#pragma unroll
          for (int j = 0; j < 4; ++j) dot_pair(gw[j], p[j], acc);
        } else {
          xacc ^= p[0] ^ p[1] ^ p[2] ^ p[3];
        }
      }
    }
    v += 4;
  }
  const long long t1 = clock64();
  if (acc.total() == 1.2345f || xacc == 0x1234567u) sink[4] = xacc;
  if (blockIdx.x == 0 && threadIdx.x == 0) {
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(ns1));
    sink[0] = static_cast<uint32_t>(t1 - t0);
    sink[1] = static_cast<uint32_t>(ns1 - ns0);
  }
}

}  // namespace gws
