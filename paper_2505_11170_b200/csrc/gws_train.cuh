// Eq. 11 and the gradient of Eq. 11 / Eq. 12 for many layers in one launch.
//
// A model has one b_i vector per linear layer (one entry per group), a few thousand to a few hundred thousand floats each:
// one launch per layer is all launch latency.  Here the layers' records travel by value in the kernel parameters, as in the
// sampling kernels, and a thread block of 256 threads takes 1024 consecutive entries of one layer.  The arithmetic is that
// of k_bitwidth and k_bitwidth_grad, operation for operation (one rounding each), so the results are the same bits.
#pragma once
#include "gws_kernels.cuh"

namespace gws {

struct BitwidthRec {
  const float* bi;        // Eq. 11 input (forward call)
  float* bt;              // written by the forward call, read by the gradient call
  const float* grad_bt;   // gradient call
  float* grad_bi;         // gradient call
  uint32_t n;             // entries = groups of the layer
  uint32_t block_begin;   // first thread block of this layer inside the launch
  float delta;            // b_init - b_target
  float b_target;
  float lam_over_m;       // lambda / (groups of the layer): Eq. 12's mean over the layer's blocks
  uint32_t accumulate;    // gradient call: add to grad_bi instead of overwriting it
};
static_assert(sizeof(BitwidthRec) == 56, "BitwidthRec layout");

constexpr int kBitwidthCap = 64;            // layers per launch: 3.5 KiB of kernel parameters
constexpr uint32_t kBitwidthPerBlock = 1024;

struct BitwidthBatch {
  int32_t n;
  int32_t pad;
  BitwidthRec e[kBitwidthCap];
};

template <bool GRAD>
__global__ void __launch_bounds__(256) k_bitwidth_multi(const __grid_constant__ BitwidthBatch b) {
  int idx = 0;
  while (idx + 1 < b.n && b.e[idx + 1].block_begin <= blockIdx.x) ++idx;
  const BitwidthRec& e = b.e[idx];
  const uint32_t first = (blockIdx.x - e.block_begin) * kBitwidthPerBlock + threadIdx.x;
#pragma unroll
  for (uint32_t j = 0; j < kBitwidthPerBlock / 256u; ++j) {
    const uint32_t k = first + j * 256u;
    if (k >= e.n) break;
    if (!GRAD) {
      st_f32(e.bt, k, __fadd_rn(e.b_target, __fmul_rn(ld_f32(e.bi, k), e.delta)));
    } else {
      const float x = __fsub_rn(ld_f32(e.bt, k), e.b_target);
      const float sign = x > 0.0f ? 1.0f : (x < 0.0f ? -1.0f : 0.0f);
      const float g = __fmul_rn(e.delta, __fadd_rn(ld_f32(e.grad_bt, k), __fmul_rn(e.lam_over_m, sign)));
      st_f32(e.grad_bi, k, e.accumulate != 0u ? __fadd_rn(e.grad_bi[k], g) : g);
    }
  }
}

}  // namespace gws
