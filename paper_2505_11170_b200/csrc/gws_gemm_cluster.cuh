// Fused sample-into-GEMM, cluster form:  Y[M, N] = X[M, K] * W_hat[N, K]^T  with every tile of W_hat sampled ONCE per
// thread-block cluster and shared through distributed shared memory, and the sampling of the next steps running while
// the tensor core works on the current one.
//
// A cluster is C thread blocks stacked along M (C = 1, 2 or 4); each block computes 256 rows x 128 columns of Y, so a
// sampled tile of W (128 rows of W x 128 along K = one sampling group per row) serves 256 * C rows of X.  Per step
// along K every block samples 128 / C rows of the tile (Eq. 3 + the BF16 cast, the arithmetic of the flat-group
// forward kernel; a thread takes 8 elements, 16 lanes a group) and stores them, K-major with the 128-byte swizzle,
// into the shared memory of ALL blocks of the cluster with st.async (a store that signals its bytes on the
// destination's mbarrier when they land, so the sampling threads never wait for a neighbour); a block's own X tiles
// arrive by TMA.  Three stages of W (96 KiB), two of X (128 KiB).  Roles:
//
//   sampler warps (16)    wait w_empty[s] (the MMAs of every block of the cluster have finished with stage s), sample,
//                         st.async to every block of the cluster
//   relay thread          expects the 32 KiB of a W stage on w_full[s], waits for them, fence.proxy.async (the tile was
//                         written through the generic proxy, the tensor core reads through the async proxy; the fence
//                         costs most of a thousand cycles, which is why it is not on a thread that issues MMAs),
//                         arrives on w_ready[s]
//   TMA thread            waits x_empty[s], starts the loads of the X tiles of the step onto x_full[s]
//   two MMA threads       one per 128-row tile of X: wait w_ready[s] and x_full[s], issue 8 tcgen05.mma (M = 128, N = 128,
//                         K = 16; FP32 accumulators in tensor memory), commit to x_empty[s] (this block) and, multicast, to
//                         w_empty[s] of every block of the cluster
//   sampler warps again   epilogue: tcgen05.ld, one rounding to BF16, 16-byte stores
//
// What bounds it (measured on B200): an MMA of this shape runs for 64 cycles and reads 8 KiB of shared memory, i.e. all
// 128 bytes per cycle an SM's shared memory delivers, while TMA and the neighbours' stores write another ~100 bytes per
// cycle into it; and issuing an MMA costs its thread about 46 cycles, a wait on a completed mbarrier 150 to 300.  A block
// therefore gets through a step along K in about 2,600 cycles instead of the 1,024 the tensor core would need.
//
// No load is multicast: the only cluster-wide operations are the st.async stores (with their mbarrier signals) and the
// multicast of tcgen05.commit.  Every mbarrier wait is bounded (about a second); a wait that runs out sets the status
// word and the block skips the rest of its work.  No block leaves before all blocks of its cluster have passed the
// final cluster barrier.
#pragma once

namespace {

constexpr int kClSamplerWarps = 16;
constexpr int kClThreads = (kClSamplerWarps + 4) * 32;   // samplers, the TMA warp, tensor-core warp 0, the W relay warp, tensor-core warp 1
constexpr int kClMT = 2;                                   // 128-row tiles of X per block
constexpr int kClStagesX = 2, kClStagesW = 3;
constexpr uint32_t kClStageXBytes = kClMT * kTileBytes;     // X: kClMT tiles of 128 rows x 128 along K per stage
constexpr uint32_t kClStageWBytes = kTileBytes;             // W: 128 rows x 128 along K (one sampling group per row)
constexpr uint32_t kClSmemBytes = kClStagesX * kClStageXBytes + kClStagesW * kClStageWBytes;

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
// 16 bytes into the shared memory of a block of the cluster (or this one), asynchronously: the store signals its 16
// bytes on the destination's mbarrier when they have landed, the storing thread does not wait for anything.
__device__ __forceinline__ void st_async_v4(uint32_t cluster_addr, uint32_t cluster_bar, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.v4.b32 [%0], {%1, %2, %3, %4}, [%5];" ::"r"(cluster_addr), "r"(a),
               "r"(b), "r"(c), "r"(d), "r"(cluster_bar)
               : "memory");
}
// As mbar_wait, with acquire semantics at cluster scope: what other blocks stored before they arrived is visible.
template <bool BACKOFF>
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (done) return true;
    if (clock64() - t0 > kWaitCycles) return false;
    if (BACKOFF) __nanosleep(64);   // sixteen warps wait here while one thread of the block feeds the tensor core: leave it the issue slots
  }
}
// tcgen05.mma with the accumulate flag as an immediate (no predicate set-up per instruction).
__device__ __forceinline__ void mma_bf16_acc(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d), "l"(a_desc),
               "l"(b_desc), "r"(kInstrDesc));
}
__device__ __forceinline__ void mma_bf16_first(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d), "l"(a_desc),
               "l"(b_desc), "r"(kInstrDesc));
}
__device__ __forceinline__ void mma_commit_cluster(uint64_t* bar, uint16_t cta_mask) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(smem_u32(bar)),
               "h"(cta_mask)
               : "memory");
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

template <int C>
__global__ void __launch_bounds__(kClThreads, 1) k_gemm_cluster(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment of the shared-window offset (identical in every block of the cluster): the swizzle pattern
  // is a function of address bits 7..9
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem_x = smem_raw + (((raw + 1023u) & ~1023u) - raw);
  uint8_t* smem_w = smem_x + kClStagesX * kClStageXBytes;
  __shared__ uint64_t x_full[kClStagesX], x_empty[kClStagesX], w_full[kClStagesW], w_ready[kClStagesW], w_empty[kClStagesW], acc_full;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int failed;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31u;
  const uint32_t rank = C > 1 ? cluster_rank() : 0u;
  const uint32_t n0 = blockIdx.x * kTileN, m0 = blockIdx.y * (kClMT * kTileM);
  const uint32_t steps = a.k / kTileK;        // steps of 128 along K: one W tile and one stage of X each
  constexpr uint32_t kTmemCols = kClMT * kTileN;
  constexpr uint32_t kSamplers = kClSamplerWarps * 32;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kClStagesX; ++s) {
      mbar_init(&x_full[s], 1);
      mbar_init(&x_empty[s], kClMT);          // one commit per tensor-core thread
    }
#pragma unroll
    for (int s = 0; s < kClStagesW; ++s) {
      mbar_init(&w_full[s], 1);               // the relay thread's expect_tx; the bytes come from the whole cluster
      mbar_init(&w_ready[s], 1);              // the relay thread, once the tile may be read through the async proxy
      mbar_init(&w_empty[s], kClMT * C);      // the tensor-core threads of every block
    }
    mbar_init(&acc_full, kClMT);
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kClSamplerWarps + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (C > 1) cluster_sync_all();   // every block's barriers exist before any store from outside signals them
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;
  uint32_t copies_started = 0;     // TMA thread: stages of X whose copies have been started

  if (warp < kClSamplerWarps) {
    // ---- samplers: rows [rank * 128 / C, (rank + 1) * 128 / C) of the W tile; a thread takes 16-byte vectors (8
    // elements, one Philox call), the 16 lanes of a row form its 128-element group ----
    constexpr uint32_t kRowsPerBlock = 128u / C;                  // rows of the tile this block samples
    constexpr uint32_t kVecsPerThread = kRowsPerBlock * 16u / kSamplers;   // 4 (C = 1), 2, 1
    uint32_t r[kVecsPerThread], vec0[kVecsPerThread], grp0[kVecsPerThread];
    uint4 w_next[kVecsPerThread];
    float bt_next[kVecsPerThread];
    const uint32_t unit = tid & 15u;                              // which 16 bytes of the row's 256
#pragma unroll
    for (uint32_t q = 0; q < kVecsPerThread; ++q) {
      r[q] = rank * kRowsPerBlock + q * (kSamplers / 16u) + (tid >> 4);   // row of the tile
      const uint32_t row = n0 + r[q];
      vec0[q] = (row * a.k) / 8u + unit;                          // step j: + 16 * j
      grp0[q] = row * steps;                                    // step j: + j
      w_next[q] = gws::ld_vec(a.w, vec0[q]);
      bt_next[q] = gws::ld_f32(a.bt, grp0[q]);
    }
    for (uint32_t j = 0; j < steps; ++j) {
      const uint32_t s = j % kClStagesW;
      if (j >= kClStagesW && !mbar_wait_cluster<true>(&w_empty[s], ((j / kClStagesW) - 1u) & 1u)) failed = 1;
      if (__any_sync(0xFFFFFFFFu, failed != 0)) break;   // a whole warp stays or leaves: the shuffles below need all lanes
      const uint32_t stage_w = smem_u32(smem_w + s * kClStageWBytes), bar = smem_u32(&w_full[s]);
#pragma unroll
      for (uint32_t q = 0; q < kVecsPerThread; ++q) {
        const uint32_t vec = vec0[q] + 16u * j;
        const uint4 wv = w_next[q];
        const float bits = bt_next[q];
        if (j + 1u < steps) {
          w_next[q] = gws::ld_vec(a.w, vec + 16u);
          bt_next[q] = gws::ld_f32(a.bt, grp0[q] + j + 1u);
        }
        uint32_t m = gws::absmax_vec(wv);
#pragma unroll
        for (uint32_t o = 1; o < 16u; o <<= 1) m = gws::maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        const gws::Scale sc = gws::make_scale(__fmul_rn(gws::absmax_finish(m), gws::pow2_one_minus(bits)));
        const uint4 y = gws::sample_vec(wv, gws::philox4x32_10_pre(a.vec_lo + vec, a.k0, a.k1, a.pre), sc);
        const uint32_t dst = stage_w + (unit >> 3) * kAtomBytes + (r[q] >> 3) * 1024u + (r[q] & 7u) * 128u + (((unit & 7u) ^ (r[q] & 7u)) << 4);
#pragma unroll
        for (uint32_t d = 0; d < static_cast<uint32_t>(C); ++d)
          st_async_v4(C > 1 ? map_to_rank(dst, d) : dst, C > 1 ? map_to_rank(bar, d) : bar, y.x, y.y, y.z, y.w);
        if (blockIdx.y < static_cast<uint32_t>(C)) {   // the first cluster along M exports the sampled weights
          if (a.w_hat_out != nullptr) gws::st_vec(a.w_hat_out, vec, y);
          if (a.scale_out != nullptr && unit == 0u) gws::st_f32(a.scale_out, grp0[q] + j, sc.s);
        }
      }
    }
  } else if (warp == kClSamplerWarps) {
    // ---- X tiles by TMA: a stage is kClMT tiles of 128 rows x 128 along K ----
    if (lane == 0) {
      for (uint32_t i = 0; i < steps; ++i) {
        const uint32_t s = i % kClStagesX;
        if (i >= kClStagesX && !mbar_wait(&x_empty[s], ((i / kClStagesX) - 1u) & 1u)) failed = 1;
        if (failed) break;
        uint8_t* stage_x = smem_x + s * kClStageXBytes;
        copies_started = i + 1u;
        mbar_expect_tx(&x_full[s], kClStageXBytes);
#pragma unroll
        for (int mt = 0; mt < kClMT; ++mt)
#pragma unroll
          for (int atom = 0; atom < 2; ++atom)
            tma_load_2d(stage_x + mt * kTileBytes + atom * kAtomBytes, &x_map, &x_full[s], static_cast<int32_t>(i * kTileK + atom * 64),
                        static_cast<int32_t>(m0 + mt * kTileM));
      }
    }
  } else if (warp == kClSamplerWarps + 1 || warp == kClSamplerWarps + 3) {
    // ---- tensor core: one issuing thread per 128-row tile of X (issuing an MMA costs its thread about 46 cycles and an
    // MMA of this shape runs for 64, so a single thread that also waits and commits cannot keep the pipe full) ----
    if (lane == 0) {
      const uint32_t mt = warp == kClSamplerWarps + 1 ? 0u : 1u;
      const uint64_t x_desc0 = smem_desc(smem_u32(smem_x) + mt * kTileBytes), w_desc0 = smem_desc(smem_u32(smem_w));
      const uint32_t acc = tmem_base + mt * kTileN;
      bool gave_up = false;
      for (uint32_t i = 0; i < steps; ++i) {
        const uint32_t sx = i % kClStagesX, sw = i % kClStagesW;
        if (!mbar_wait(&w_ready[sw], (i / kClStagesW) & 1u)) gave_up = true;
        if (!gave_up && !mbar_wait(&x_full[sx], (i / kClStagesX) & 1u)) gave_up = true;
        if (gave_up) break;   // another role's failure shows up here as a wait that runs out
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        // descriptors of the step: the stage's base descriptor plus byte offsets >> 4 in the address field
        const uint64_t xd = x_desc0 + static_cast<uint64_t>(sx * (kClStageXBytes >> 4));
        const uint64_t wd = w_desc0 + static_cast<uint64_t>(sw * (kClStageWBytes >> 4));
#pragma unroll
        for (uint32_t kk = 0; kk < kTileK / 16; ++kk) {
          const uint64_t off = static_cast<uint64_t>((kk >> 2) * (kAtomBytes >> 4) + (kk & 3u) * 2u);
          if (kk == 0 && i == 0) mma_bf16_first(acc, xd + off, wd + off);
          else mma_bf16_acc(acc, xd + off, wd + off);
        }
        mma_commit(&x_empty[sx]);
        if (C > 1) mma_commit_cluster(&w_empty[sw], static_cast<uint16_t>((1u << C) - 1u));
        else mma_commit(&w_empty[sw]);
      }
      if (gave_up) failed = 1;
      else mma_commit(&acc_full);
    }
  } else if (warp == kClSamplerWarps + 2) {
    // ---- W relay: waits until the whole tile of a step has landed (stores of every block of the cluster), orders those
    // generic-proxy stores before the tensor core's async-proxy reads, and hands the stage to the tensor-core thread.
    // The fence costs several hundred cycles; here it is off the thread that keeps the tensor core fed ----
    if (lane == 0) {
      for (uint32_t j = 0; j < steps; ++j) {
        const uint32_t s = j % kClStagesW, ph = (j / kClStagesW) & 1u;
        mbar_expect_tx(&w_full[s], kClStageWBytes);   // this block's copy of what every block of the cluster samples
        if (!mbar_wait_cluster<false>(&w_full[s], ph)) { failed = 1; break; }
        asm volatile("fence.proxy.async;" ::: "memory");
        asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&w_ready[s])) : "memory");
      }
    }
  }
  __syncthreads();
  // a block that gave up may still have copies of X in flight towards its shared memory: the thread that started them
  // waits (bounded) for the last copy of each stage before the shared memory is given up
  if (failed && warp == kClSamplerWarps && lane == 0) {
    for (uint32_t back = 0; back < kClStagesX && back < copies_started; ++back) {
      const uint32_t i = copies_started - 1u - back;
      (void)mbar_wait(&x_full[i % kClStagesX], (i / kClStagesX) & 1u);
    }
  }
  bool ok = !failed;
  if (ok && steps > 0 && !mbar_wait(&acc_full, 0)) ok = false;
  ok = __syncthreads_and(ok) != 0;   // the tensor-memory loads below are warp-collective: one decision for the block
  if (ok && warp < kClSamplerWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint16_t* y = reinterpret_cast<uint16_t*>(a.y);
    const uint32_t quarter_rows = (warp & 3u) * 32u;   // a warp reads the quarter (warp % 4) of the 128 accumulator rows
#pragma unroll 1
    for (uint32_t idx = warp >> 2; idx < kClMT * (kTileN / 32); idx += kClSamplerWarps / 4) {
      const uint32_t mt = idx / (kTileN / 32), cb = idx % (kTileN / 32);
      const uint64_t row = static_cast<uint64_t>(m0) + mt * kTileM + quarter_rows + lane;
      uint32_t acc[32];
      tmem_ld32(tmem_base + (quarter_rows << 16) + mt * kTileN + cb * 32u, acc);
      uint4* out = reinterpret_cast<uint4*>(y + row * a.n + n0 + cb * 32u);
#pragma unroll
      for (int q = 0; q < 4; ++q) {
        uint32_t p[4];
#pragma unroll
        for (int e = 0; e < 4; ++e)
          p[e] = gws::pack_bf16_rne(__uint_as_float(acc[8 * q + 2 * e]), __uint_as_float(acc[8 * q + 2 * e + 1]));
        out[q] = make_uint4(p[0], p[1], p[2], p[3]);
      }
    }
  } else if (!ok && tid == 0 && a.status != nullptr) {
    atomicExch(a.status, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (C > 1) cluster_sync_all();   // nobody leaves while a neighbour may still store into this block's shared memory
  if (warp == kClSamplerWarps + 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

template <int C>
int launch_gemm_cluster(const CUtensorMap& map, const GemmArgs& args, int64_t m, cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(kClSmemBytes) + 1024;
  cudaError_t err = cudaFuncSetAttribute(k_gemm_cluster<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) { g_gemm_error = std::string("shared memory size: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(args.n / kTileN, static_cast<unsigned>(m / (kClMT * kTileM)));
  cfg.blockDim = dim3(kClThreads);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = 1;
  attr[0].val.clusterDim.y = C;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  err = cudaLaunchKernelEx(&cfg, k_gemm_cluster<C>, map, args);
  if (err != cudaSuccess) { (void)cudaGetLastError(); g_gemm_error = std::string("fused GEMM (cluster) launch: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  return GWS_OK;
}

}  // namespace
