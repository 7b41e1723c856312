// Fused sample-into-GEMM, wide form:  Y[M, N] = X[M, K] * W_hat[N, K]^T  with 256 x 256 tiles of Y per thread block.
//
// In the cluster form with 128-column tiles a tcgen05.mma of 128 x 128 x 16 reads 8 KiB of shared memory in the 64 cycles
// it runs, all an SM's shared memory delivers, with the tile traffic of the pipeline on top.  With N = 256 an instruction
// runs for 128 cycles and reads 12 KiB (the X operand is read once for twice the columns): 96 bytes per cycle, and half as
// many instructions to issue per unit of tensor-core work.  The price: both accumulators of a block (2 x 128 rows x 256
// columns of FP32) take all 512 columns of tensor memory.
//
// A cluster is C blocks stacked along M (C = 1, 2, 4).  Per 128 elements along K (one sampling group per row of W) every
// block samples 256 / C rows of the 256-row tile of W into its OWN shared memory (64-byte chunks per thread, plain stores:
// the arithmetic of the flat-group forward kernel), and one thread then copies that share into the same place of every
// other block of the cluster with cp.async.bulk (shared memory to shared memory of the cluster, signalling the bytes on the
// destination's mbarrier); X arrives by TMA in steps of 64 along K.  Shared memory: two stages of W (256 rows x 128 along
// K = 64 KiB each, as two 128-byte-swizzled halves of 64 along K) and three stages of X (2 x 128 rows x 64 along K = 32 KiB
// each).  Roles: 16 sampling warps, a TMA thread, a relay thread (waits for the block's own share, fences the generic-proxy
// stores against async-proxy reads, starts the bulk copies, waits for the other blocks' shares, hands the stage to the
// tensor core), two MMA-issuing threads (one per accumulator).
//
// What it showed (B200, 16384 x 2048 by 5632 x 2048): 593 us for clusters of 2 against 617 us for the 128-column form, so
// shared-memory bandwidth and instruction issue were not what held that form back; and an earlier version of this kernel
// whose sampling threads stored every vector into every block with st.async (twice the sampling cost per stage) took
// 595 us, so the sampling rate is not it either.  Cycle stamps in a copy of this kernel: a block spends about 120,000 cycles
// on its tile, 95,000 of them in the 16 steps of 128 along K (5,900 each against 2,048 of tensor-core work).  A stage of W
// goes round in about 12,000 cycles (wait for the tensor cores of every block of the cluster to release it, sample 4,300,
// fence and copy 2,000 to 3,000, two MMA steps 2,500), and only two such stages fit beside three of X in 227 KiB: the
// tensor core is fed a third of the time.  First operands are ready 10,000 cycles after the block starts, the epilogue
// takes 10,000 and the last cluster barrier 3,000 to 4,000.
//
// No load from global memory is multicast and no TMA load touches another block's memory: the only transfers between blocks
// are the bulk copies from a block's own shared memory, and the multicast of tcgen05.commit.  Every mbarrier wait is bounded;
// a wait that runs out sets the status word and the block skips the rest of its work.  No block leaves before all blocks of
// its cluster have passed the final cluster barrier.
#pragma once

namespace {

constexpr int kWdN = 256;                                   // columns of Y (rows of W) per block
constexpr int kWdMT = 2;                                    // 128-row tiles of X per block
constexpr int kWdStepK = 64;                                // X arrives and is multiplied in steps of 64 along K
constexpr int kWdStagesX = 3, kWdStagesW = 2;
constexpr uint32_t kWdXTileBytes = 128u * 128u;             // 128 rows x 64 along K
constexpr uint32_t kWdStageXBytes = kWdMT * kWdXTileBytes;  // 32 KiB
constexpr uint32_t kWdHalfWBytes = kWdN * 128u;             // 256 rows x 64 along K
constexpr uint32_t kWdStageWBytes = 2u * kWdHalfWBytes;     // 256 rows x 128 along K: 64 KiB
constexpr uint32_t kWdSmemBytes = kWdStagesX * kWdStageXBytes + kWdStagesW * kWdStageWBytes;
// Instruction descriptor: FP32 accumulator, BF16 A and B, both K-major, N = 256, M = 128.
constexpr uint32_t kWdInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kWdN >> 3) << 17) | ((kTileM >> 4) << 24);

// tcgen05.ld of 32 lanes x 32 columns without the wait (the caller waits once for several of them).
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,"
      "%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
}

template <bool ACCUMULATE>
__device__ __forceinline__ void mma_bf16_wide(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc) {
  if (ACCUMULATE)
    asm volatile("{\n\t.reg .pred p;\n\tsetp.eq.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
                 "l"(a_desc), "l"(b_desc), "r"(kWdInstrDesc));
  else
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, 0, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
                 "l"(a_desc), "l"(b_desc), "r"(kWdInstrDesc));
}

template <int C>
__global__ void __launch_bounds__(kClThreads, 1) k_gemm_wide(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  uint8_t* smem_x = smem_raw + (((raw + 1023u) & ~1023u) - raw);   // the same offset in every block of the cluster
  uint8_t* smem_w = smem_x + kWdStagesX * kWdStageXBytes;
  __shared__ uint64_t x_full[kWdStagesX], x_empty[kWdStagesX], w_full[kWdStagesW], w_ready[kWdStagesW], w_empty[kWdStagesW], w_local[kWdStagesW], acc_full;
  __shared__ uint32_t tmem_slot;
  __shared__ volatile int failed;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31u;
  const uint32_t rank = C > 1 ? cluster_rank() : 0u;
  const uint32_t n0 = blockIdx.x * kWdN, m0 = blockIdx.y * (kWdMT * kTileM);
  const uint32_t pairs = a.k / 128u;             // sampling groups along K = stages of W
  const uint32_t steps = a.k / kWdStepK;         // stages of X = 2 * pairs
  constexpr uint32_t kTmemCols = kWdMT * kWdN;   // 512: all of it
  constexpr uint32_t kSamplers = kClSamplerWarps * 32;

  if (tid == 0) {
#pragma unroll
    for (int s = 0; s < kWdStagesX; ++s) {
      mbar_init(&x_full[s], 1);
      mbar_init(&x_empty[s], kWdMT);
    }
#pragma unroll
    for (int s = 0; s < kWdStagesW; ++s) {
      mbar_init(&w_full[s], 1);
      mbar_init(&w_ready[s], 1);
      mbar_init(&w_empty[s], kWdMT * C);
      mbar_init(&w_local[s], kClSamplerWarps);   // one arrival per sampling warp: this block's share of the stage is in its own shared memory
    }
    mbar_init(&acc_full, kWdMT);
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kClSamplerWarps + 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (C > 1) cluster_sync_all();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;
  uint32_t copies_started = 0;

  if (warp < kClSamplerWarps) {
    // ---- samplers: rows [rank * 256 / C, (rank + 1) * 256 / C) of the W tile into this block's OWN shared memory with plain
    // stores; the relay thread then copies the share to the other blocks of the cluster in bulk.  A thread takes kVecs
    // neighbouring 16-byte vectors of a row (4 = a 64-byte chunk for C <= 2, 2 for C = 4), 16 / kVecs lanes form the group ----
    constexpr uint32_t kRowsPerBlock = static_cast<uint32_t>(kWdN) / C;
    constexpr uint32_t kVecs = C == 4 ? 2u : 4u;
    constexpr uint32_t kLanesPerRow = 16u / kVecs;                       // 4 or 8
    constexpr uint32_t kRowsPerPass = kSamplers / kLanesPerRow;          // 128 or 64
    constexpr uint32_t kItems = kRowsPerBlock / kRowsPerPass;            // 2 (C = 1), 1, 1
    static_assert(kItems * kRowsPerPass == kRowsPerBlock, "share of the tile");
    const uint32_t part = tid % kLanesPerRow, unit0 = part * kVecs;      // first 16-byte unit of the row's 16
    uint32_t r[kItems], vec0[kItems], grp0[kItems];
    uint32_t x_next[kItems][4 * kVecs];
    float bt_next[kItems];
    auto load_item = [&](uint32_t (&x)[4 * kVecs], uint32_t vec) {
#pragma unroll
      for (uint32_t h = 0; h < kVecs / 2u; ++h) {
        const gws::Vec32 v = gws::ld_vec32(a.w, static_cast<uint64_t>(vec + 2u * h) * 16u);
#pragma unroll
        for (int i = 0; i < 8; ++i) x[8 * h + i] = v.v[i];
      }
    };
#pragma unroll
    for (uint32_t q = 0; q < kItems; ++q) {
      r[q] = rank * kRowsPerBlock + q * kRowsPerPass + tid / kLanesPerRow;
      const uint32_t row = n0 + r[q];
      vec0[q] = (row * a.k) / 8u + unit0;        // pair j: + 16 * j
      grp0[q] = row * pairs;                     // pair j: + j
      load_item(x_next[q], vec0[q]);
      bt_next[q] = gws::ld_f32(a.bt, grp0[q]);
    }
    for (uint32_t j = 0; j < pairs; ++j) {
      const uint32_t s = j % kWdStagesW;
      if (j >= kWdStagesW && !mbar_wait_cluster<true>(&w_empty[s], ((j / kWdStagesW) - 1u) & 1u)) failed = 1;
      if (__any_sync(0xFFFFFFFFu, failed != 0)) break;   // a whole warp stays or leaves: the shuffles below need all lanes
      uint8_t* stage_w = smem_w + s * kWdStageWBytes;
#pragma unroll
      for (uint32_t q = 0; q < kItems; ++q) {
        const uint32_t vec = vec0[q] + 16u * j;
        uint32_t x[4 * kVecs];
#pragma unroll
        for (uint32_t i = 0; i < 4 * kVecs; ++i) x[i] = x_next[q][i];
        const float bits = bt_next[q];
        if (j + 1u < pairs) {
          load_item(x_next[q], vec + 16u);
          bt_next[q] = gws::ld_f32(a.bt, grp0[q] + j + 1u);
        }
        uint32_t m = gws::absmax_words4(x);
#pragma unroll
        for (uint32_t i = 1; i < kVecs; ++i) m = gws::maxabs2(m, gws::absmax_words4(x + 4 * i));
#pragma unroll
        for (uint32_t o = 1; o < kLanesPerRow; o <<= 1) m = gws::maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, o));
        const gws::Scale sc = gws::make_scale(__fmul_rn(gws::absmax_finish(m), gws::pow2_one_minus(bits)));
        uint32_t y[4 * kVecs];
        if (kVecs == 4u) gws::sample_chunk(x, a.vec_lo + vec, a.k0, a.k1, a.pre, sc, y);
        else gws::sample_half(x, a.vec_lo + vec, a.k0, a.k1, a.pre, sc, y);
        uint8_t* row_base = stage_w + (unit0 >> 3) * kWdHalfWBytes + (r[q] >> 3) * 1024u + (r[q] & 7u) * 128u;
#pragma unroll
        for (uint32_t i = 0; i < kVecs; ++i)
          *reinterpret_cast<uint4*>(row_base + ((((unit0 + i) & 7u) ^ (r[q] & 7u)) << 4)) = make_uint4(y[4 * i], y[4 * i + 1], y[4 * i + 2], y[4 * i + 3]);
        if (blockIdx.y < static_cast<uint32_t>(C)) {   // the first cluster along M exports the sampled weights
          if (a.w_hat_out != nullptr) {
#pragma unroll
            for (uint32_t h = 0; h < kVecs / 2u; ++h) gws::st_vec32(a.w_hat_out, static_cast<uint64_t>(vec + 2u * h) * 16u, y + 8 * h);
          }
          if (a.scale_out != nullptr && part == 0u) gws::st_f32(a.scale_out, grp0[q] + j, sc.s);
        }
      }
      __syncwarp();
      if (lane == 0) asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&w_local[s])) : "memory");
    }
  } else if (warp == kClSamplerWarps) {
    // ---- X by TMA: a stage is kWdMT tiles of 128 rows x 64 along K ----
    if (lane == 0) {
      for (uint32_t i = 0; i < steps; ++i) {
        const uint32_t s = i % kWdStagesX;
        if (i >= kWdStagesX && !mbar_wait(&x_empty[s], ((i / kWdStagesX) - 1u) & 1u)) failed = 1;
        if (failed) break;
        uint8_t* stage_x = smem_x + s * kWdStageXBytes;
        copies_started = i + 1u;
        mbar_expect_tx(&x_full[s], kWdStageXBytes);
#pragma unroll
        for (int mt = 0; mt < kWdMT; ++mt)
          tma_load_2d(stage_x + mt * kWdXTileBytes, &x_map, &x_full[s], static_cast<int32_t>(i * kWdStepK), static_cast<int32_t>(m0 + mt * kTileM));
      }
    }
  } else if (warp == kClSamplerWarps + 1 || warp == kClSamplerWarps + 3) {
    // ---- tensor core: one issuing thread per accumulator; per step of 64 along K four MMAs of 128 x 256 x 16 ----
    if (lane == 0) {
      const uint32_t mt = warp == kClSamplerWarps + 1 ? 0u : 1u;
      const uint64_t x_desc0 = smem_desc(smem_u32(smem_x) + mt * kWdXTileBytes), w_desc0 = smem_desc(smem_u32(smem_w));
      const uint32_t acc = tmem_base + mt * kWdN;
      bool gave_up = false;
      for (uint32_t i = 0; i < steps; ++i) {
        const uint32_t sx = i % kWdStagesX, p = i >> 1, half = i & 1u, sw = p % kWdStagesW;
        if (half == 0u && !mbar_wait(&w_ready[sw], (p / kWdStagesW) & 1u)) gave_up = true;
        if (!gave_up && !mbar_wait(&x_full[sx], (i / kWdStagesX) & 1u)) gave_up = true;
        if (gave_up) break;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t xd = x_desc0 + static_cast<uint64_t>(sx * (kWdStageXBytes >> 4));
        const uint64_t wd = w_desc0 + static_cast<uint64_t>(sw * (kWdStageWBytes >> 4) + half * (kWdHalfWBytes >> 4));
#pragma unroll
        for (uint32_t kk = 0; kk < kWdStepK / 16; ++kk) {
          if (kk == 0 && i == 0) mma_bf16_wide<false>(acc, xd, wd);
          else mma_bf16_wide<true>(acc, xd + kk * 2u, wd + kk * 2u);
        }
        mma_commit(&x_empty[sx]);
        if (half == 1u) {
          if (C > 1) mma_commit_cluster(&w_empty[sw], static_cast<uint16_t>((1u << C) - 1u));
          else mma_commit(&w_empty[sw]);
        }
      }
      if (gave_up) failed = 1;
      else mma_commit(&acc_full);
    }
  } else if (warp == kClSamplerWarps + 2) {
    // ---- W relay: when this block's share of a stage is complete in its own shared memory, orders those generic-proxy stores
    // before async-proxy reads, copies the share in bulk into the same place of every other block of the cluster (two copies per
    // block: the share is contiguous in each half along K), waits for the other blocks' shares and hands the stage on ----
    if (lane == 0) {
      constexpr uint32_t kRowsPerBlock = static_cast<uint32_t>(kWdN) / C;
      constexpr uint32_t kShareBytes = kRowsPerBlock * 128u;    // per half along K
      for (uint32_t j = 0; j < pairs; ++j) {
        const uint32_t s = j % kWdStagesW, ph = (j / kWdStagesW) & 1u;
        if (C > 1) mbar_expect_tx(&w_full[s], (C - 1) * 2u * kShareBytes);
        if (!mbar_wait(&w_local[s], ph)) { failed = 1; break; }
        asm volatile("fence.proxy.async;" ::: "memory");
        if (C > 1) {
          const uint32_t src0 = smem_u32(smem_w + s * kWdStageWBytes) + rank * kShareBytes, bar = smem_u32(&w_full[s]);
#pragma unroll
          for (uint32_t d = 0; d < static_cast<uint32_t>(C); ++d) {
            if (d == rank) continue;
            const uint32_t rbar = map_to_rank(bar, d);
#pragma unroll
            for (uint32_t h = 0; h < 2; ++h) {
              const uint32_t src = src0 + h * kWdHalfWBytes;
              asm volatile("cp.async.bulk.shared::cluster.shared::cta.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(map_to_rank(src, d)),
                           "r"(src), "r"(kShareBytes), "r"(rbar)
                           : "memory");
            }
          }
          if (!mbar_wait_cluster<false>(&w_full[s], ph)) { failed = 1; break; }
        }
        asm volatile("mbarrier.arrive.release.cta.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&w_ready[s])) : "memory");
      }
    }
  }
  __syncthreads();
  if (failed && warp == kClSamplerWarps && lane == 0) {   // copies of X that may still be in flight: bounded waits
    for (uint32_t back = 0; back < kWdStagesX && back < copies_started; ++back) {
      const uint32_t i = copies_started - 1u - back;
      (void)mbar_wait(&x_full[i % kWdStagesX], (i / kWdStagesX) & 1u);
    }
  }
  bool ok = !failed;
  if (ok && steps > 0 && !mbar_wait(&acc_full, 0)) ok = false;
  ok = __syncthreads_and(ok) != 0;
  if (ok && warp < kClSamplerWarps) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint16_t* y = reinterpret_cast<uint16_t*>(a.y);
    const uint32_t quarter_rows = (warp & 3u) * 32u;
    // a warp owns 4 of the 16 column blocks (32 columns) of its quarter of the rows; two loads from tensor memory are in flight
    // before the first is converted and stored
#pragma unroll 1
    for (uint32_t idx = warp >> 2; idx < kWdMT * (kWdN / 32); idx += 2u * (kClSamplerWarps / 4)) {
      uint32_t acc[2][32];
#pragma unroll
      for (uint32_t h = 0; h < 2; ++h) {
        const uint32_t id = idx + h * (kClSamplerWarps / 4), mt = id / (kWdN / 32), cb = id % (kWdN / 32);
        tmem_ld32_issue(tmem_base + (quarter_rows << 16) + mt * kWdN + cb * 32u, acc[h]);
      }
      asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
      for (uint32_t h = 0; h < 2; ++h) {
        const uint32_t id = idx + h * (kClSamplerWarps / 4), mt = id / (kWdN / 32), cb = id % (kWdN / 32);
        const uint64_t row = static_cast<uint64_t>(m0) + mt * kTileM + quarter_rows + lane;
        uint4* out = reinterpret_cast<uint4*>(y + row * a.n + n0 + cb * 32u);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
          uint32_t p[4];
#pragma unroll
          for (int e = 0; e < 4; ++e)
            p[e] = gws::pack_bf16_rne(__uint_as_float(acc[h][8 * q + 2 * e]), __uint_as_float(acc[h][8 * q + 2 * e + 1]));
          out[q] = make_uint4(p[0], p[1], p[2], p[3]);
        }
      }
    }
  } else if (!ok && tid == 0 && a.status != nullptr) {
    atomicExch(a.status, 1);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (C > 1) cluster_sync_all();
  if (warp == kClSamplerWarps + 1) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

template <int C>
int launch_gemm_wide(const CUtensorMap& map, const GemmArgs& args, int64_t m, cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(kWdSmemBytes) + 1024;
  cudaError_t err = cudaFuncSetAttribute(k_gemm_wide<C>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) { g_gemm_error = std::string("shared memory size: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(args.n / kWdN, static_cast<unsigned>(m / (kWdMT * kTileM)));
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
  err = cudaLaunchKernelEx(&cfg, k_gemm_wide<C>, map, args);
  if (err != cudaSuccess) { (void)cudaGetLastError(); g_gemm_error = std::string("fused GEMM (wide) launch: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  return GWS_OK;
}

}  // namespace
