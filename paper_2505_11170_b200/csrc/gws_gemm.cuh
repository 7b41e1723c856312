// Fused sample-into-GEMM for sm_100a:  Y[M, N] = X[M, K] * W_hat[N, K]^T  with W_hat sampled from W (Eq. 3 + the BF16
// cast) tile by tile in the prologue of a tcgen05 GEMM, never written to global memory.  Section 3.5 of the paper keeps
// sampling and GEMM apart; this is the variant it decided against, built to be measured.
//
// One thread block (512 threads) computes MT x 128 rows by 128 columns of Y.  Per step along K (128 elements = one
// sampling group per row of W):
//   * one thread starts the TMA loads of the X tiles (MT x 128 rows x 128 K, 128-byte swizzle) onto an mbarrier;
//   * all threads sample the W tile (128 rows of W x 128 K; four lanes per row, exactly the arithmetic of the flat-group
//     forward kernel) and store it to shared memory in the same K-major 128-byte-swizzled layout;
//   * one thread issues the tcgen05.mma instructions (M = 128, N = 128, K = 16 each; BF16 x BF16 -> FP32 in tensor
//     memory) and commits them to a second mbarrier, which releases the shared memory for the next step.
// The accumulators (MT x 128 columns of tensor memory) are read back with tcgen05.ld, rounded to BF16 and stored.
// A larger MT re-uses each sampled tile for more rows of X: the sampling work per block is what this kernel is bound by.
//
// Every wait is bounded: a wait that runs out sets the status word, the block skips its remaining work, frees its
// tensor memory and returns.
//
// Included at the end of gws_api.cu (one translation unit: the kernels share the accessors and, in the self-checking
// build, the access window of gws_kernels.cuh).
#pragma once
#include <cuda.h>

namespace {

constexpr int kTileM = 128, kTileN = 128, kTileK = 128;
constexpr int kGemmThreads = 512;   // one 64-byte chunk of the W tile per thread and step
constexpr uint32_t kAtomBytes = 128u * 128u;        // 128 rows x 128 bytes (64 BF16 along K): one swizzle atom column
constexpr uint32_t kTileBytes = 2u * kAtomBytes;    // 128 rows x 128 K
constexpr long long kWaitCycles = 2000000000LL;     // about a second

struct GemmArgs {
  const void* w;
  const float* bt;
  void* y;
  void* w_hat_out;      // optional: the sampled weights, written by the blocks of the first row of tiles
  float* scale_out;     // optional
  int* status;          // optional: set to 1 by a block whose wait ran out
  uint32_t n, k;        // rows and cols of W
  uint32_t vec_lo, k0, k1;
  gws::PhiloxPre pre;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Waits for the phase with the given parity; false if it did not complete within kWaitCycles.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
  const long long t0 = clock64();
  for (;;) {
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    if (done) return true;
    if (clock64() - t0 > kWaitCycles) return false;
  }
}

__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, uint64_t* bar, int32_t c0, int32_t c1) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];" ::"r"(
                   smem_u32(dst)),
               "l"(reinterpret_cast<uint64_t>(map)), "r"(smem_u32(bar)), "r"(c0), "r"(c1)
               : "memory");
}

// Shared-memory matrix descriptor of a K-major operand stored with the 128-byte swizzle: start address, stride of
// 1024 bytes between groups of 8 rows, descriptor version 1, layout type 2 (128-byte swizzle).
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  return static_cast<uint64_t>((addr & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024u >> 4) << 32) | (1ull << 46) |
         (2ull << 61);
}
// Instruction descriptor: FP32 accumulator, BF16 A and B, both K-major, N = 128, M = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((kTileN >> 3) << 17) | ((kTileM >> 4) << 24);

__device__ __forceinline__ void mma_bf16(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\ttcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(tmem_d),
      "l"(a_desc), "l"(b_desc), "r"(kInstrDesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t* r) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,"
      "%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
        "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
        "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
        "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

template <int MT>
__global__ void __launch_bounds__(kGemmThreads, MT == 4 ? 1 : 2) k_gemm_fused(const __grid_constant__ CUtensorMap x_map, const __grid_constant__ GemmArgs a) {
  extern __shared__ uint8_t smem_raw[];
  // 1024-byte alignment: the swizzle pattern is a function of the address bits 7..9
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023u) & ~static_cast<uintptr_t>(1023u));
  uint8_t* smem_x = smem;                              // MT tiles of X
  uint8_t* smem_w = smem + MT * kTileBytes;            // one sampled tile of W
  __shared__ uint64_t bar_x, bar_mma;
  __shared__ uint32_t tmem_slot;
  __shared__ int failed;

  const uint32_t tid = threadIdx.x, warp = tid >> 5, lane = tid & 31u;
  const uint32_t n0 = blockIdx.x * kTileN, m0 = blockIdx.y * (MT * kTileM);
  const uint32_t k_tiles = a.k / kTileK;
  constexpr uint32_t kTmemCols = MT * kTileN;

  if (tid == 0) {
    mbar_init(&bar_x, 1);
    mbar_init(&bar_mma, 1);
    failed = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_slot)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = tmem_slot;

  const uint32_t quarter = tid & 3u;                    // which 32 elements of the 128-element group
  static_assert(kGemmThreads == 512, "one chunk of the W tile per thread and step");
  const uint32_t r = tid >> 2, row = n0 + r;
  const uint32_t chunk0 = (row * a.k) / 32u + quarter;  // this thread's chunk of step 0; step kt: + 4 * kt
  // the chunk and bit-width of the next step are fetched before the current step's arithmetic starts
  gws::Chunk c_next = gws::load_chunk<true>(a.w, chunk0, 4);
  float bt_next = gws::ld_f32(a.bt, row * k_tiles);
  bool copy_pending = false;       // thread 0: a copy of X has been started and not yet seen to land
  uint32_t copy_parity = 0;
  for (uint32_t kt = 0; kt < k_tiles; ++kt) {
    // the tensor core must have finished reading the previous step's tiles before they are overwritten
    if (kt > 0 && !mbar_wait(&bar_mma, (kt - 1u) & 1u)) failed = 1;
    __syncthreads();
    if (failed) break;
    if (tid == 0) {
      mbar_expect_tx(&bar_x, MT * kTileBytes);
#pragma unroll
      for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int atom = 0; atom < 2; ++atom)
          tma_load_2d(smem_x + mt * kTileBytes + atom * kAtomBytes, &x_map, &bar_x, static_cast<int32_t>(kt * kTileK + atom * 64),
                      static_cast<int32_t>(m0 + mt * kTileM));
      copy_pending = true;
      copy_parity = kt & 1u;
    }
    // sample the W tile: four lanes per row (one 128-element group)
    {
      const uint32_t chunk = chunk0 + 4u * kt;
      const gws::Chunk c = c_next;
      const float bits = bt_next;
      if (kt + 1u < k_tiles) {
        c_next = gws::load_chunk<true>(a.w, chunk + 4u, 4);
        bt_next = gws::ld_f32(a.bt, row * k_tiles + kt + 1u);
      }
      uint32_t m = gws::absmax_chunk(c.x);
      m = gws::maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, 1));
      m = gws::maxabs2(m, __shfl_xor_sync(0xFFFFFFFFu, m, 2));
      const uint32_t g = row * k_tiles + kt;
      const gws::Scale sc = gws::make_scale(__fmul_rn(gws::absmax_finish(m), gws::pow2_one_minus(bits)));
      gws::Chunk y;
      gws::sample_chunk(c.x, a.vec_lo + chunk * 4u, a.k0, a.k1, a.pre, sc, y.x);
      uint8_t* dst = smem_w + (quarter >> 1) * kAtomBytes + (r >> 3) * 1024u + (r & 7u) * 128u;
      const uint32_t unit0 = (quarter & 1u) * 4u;
#pragma unroll
      for (uint32_t i = 0; i < 4; ++i)
        *reinterpret_cast<uint4*>(dst + (((unit0 + i) ^ (r & 7u)) << 4)) = make_uint4(y.x[4 * i], y.x[4 * i + 1], y.x[4 * i + 2], y.x[4 * i + 3]);
      if (blockIdx.y == 0) {
        if (a.w_hat_out != nullptr) gws::store_chunk<true>(a.w_hat_out, chunk, 4, y);
        if (a.scale_out != nullptr && quarter == 0u) gws::st_f32(a.scale_out, g, sc.s);
      }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads shared memory through the async proxy
    __syncthreads();
    if (tid == 0) {
      if (!mbar_wait(&bar_x, kt & 1u)) {
        failed = 1;
      } else {
        copy_pending = false;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
          for (uint32_t j = 0; j < kTileK / 16; ++j) {
            const uint32_t off = (j >> 2) * kAtomBytes + (j & 3u) * 32u;
            mma_bf16(tmem_base + mt * kTileN, smem_desc(smem_u32(smem_x + mt * kTileBytes) + off), smem_desc(smem_u32(smem_w) + off),
                     (kt > 0 || j > 0) ? 1u : 0u);
          }
        mma_commit(&bar_mma);
      }
    }
  }
  if (!failed && k_tiles > 0 && !mbar_wait(&bar_mma, (k_tiles - 1u) & 1u)) failed = 1;
  __syncthreads();
  if (!failed) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    uint16_t* y = reinterpret_cast<uint16_t*>(a.y);
    // a warp reads the quarter (warp % 4) of the 128 accumulator rows; the warps of a quarter share its column blocks
    const uint32_t quarter_rows = (warp & 3u) * 32u;
#pragma unroll 1
    for (uint32_t idx = warp >> 2; idx < MT * (kTileN / 32); idx += kGemmThreads / 128) {
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
  } else if (tid == 0) {
    if (a.status != nullptr) atomicExch(a.status, 1);
    // a copy that may still be in flight gets one more bounded wait before the shared memory is given up
    if (copy_pending) (void)mbar_wait(&bar_x, copy_parity);
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
}

// The bounded wait on its own: one thread waits on an mbarrier that nothing will ever complete, gives up after
// kWaitCycles and reports it the way the GEMM does.  status[0] = 1: gave up; status[1] = SM cycles waited / 1024.
__global__ void k_wait_probe(int* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const long long t0 = clock64();
    const bool completed = mbar_wait(&bar, 0);
    status[0] = completed ? 0 : 1;
    status[1] = static_cast<int>(((clock64() - t0) >> 10) & 0x7FFFFFFF);
  }
}

using EncodeTiled = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

thread_local std::string g_gemm_error;

template <int MT>
int launch_gemm(const CUtensorMap& map, const GemmArgs& args, int64_t m, cudaStream_t stream) {
  const size_t smem = static_cast<size_t>(MT + 1) * kTileBytes + 1024;
  cudaError_t err = cudaFuncSetAttribute(k_gemm_fused<MT>, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
  if (err != cudaSuccess) { g_gemm_error = std::string("shared memory size: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  const dim3 grid(args.n / kTileN, static_cast<unsigned>(m / (MT * kTileM)));
  k_gemm_fused<MT><<<grid, kGemmThreads, smem, stream>>>(map, args);
  err = cudaGetLastError();
  if (err != cudaSuccess) { g_gemm_error = std::string("fused GEMM launch: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  return GWS_OK;
}

}  // namespace

extern "C" {

const char* gws_gemm_last_error(void) { return g_gemm_error.c_str(); }

int gws_gemm_wait_probe(int* status2, void* stream) {
  if (status2 == nullptr) return GWS_ERR_NULL;
  if ((reinterpret_cast<uintptr_t>(status2) % 4) != 0) return GWS_ERR_ALIGN;
  k_wait_probe<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status2);
  const cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) { g_gemm_error = std::string("wait probe launch: ") + cudaGetErrorString(err); return GWS_ERR_CUDA; }
  return GWS_OK;
}

}  // extern "C"

// Validation, tensor map of X and kernel arguments shared by both forms of the fused GEMM.  `row_multiple`: m must be a
// multiple of it.  Returns 1 when there is nothing to do.
static int gemm_prepare(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y, void* w_hat_out,
                        float* scale_out, int* status, int64_t row_multiple, CUtensorMap& map, GemmArgs& args) {
  if (wdesc == nullptr) return GWS_ERR_NULL;
  if (m < 0 || wdesc->rows < 0 || wdesc->cols < 0) return GWS_ERR_SHAPE;
  if (m == 0 || wdesc->rows == 0 || wdesc->cols == 0) return 1;
  if (x == nullptr || w == nullptr || bt == nullptr || y == nullptr) return GWS_ERR_NULL;
  const int64_t n = wdesc->rows, k = wdesc->cols;
  if (wdesc->group_rows != 1 || wdesc->group_cols != kTileK || wdesc->ld != k || k % kTileK != 0 || n % kTileN != 0 ||
      m % row_multiple != 0 || wdesc->elem_offset % 8 != 0)
    return GWS_ERR_UNSUPPORTED;
  const uint64_t first_vec = wdesc->elem_offset >> 3, last_vec = first_vec + static_cast<uint64_t>(n * k / 8) - 1;
  if ((first_vec >> 32) != (last_vec >> 32) || n * k > 0xFFFFFFFFLL || m * k > (1LL << 40)) return GWS_ERR_UNSUPPORTED;
  auto misaligned = [](const void* p, size_t al) { return (reinterpret_cast<uintptr_t>(p) % al) != 0; };
  if (misaligned(x, 16) || misaligned(w, 32) || misaligned(y, 16) || misaligned(bt, 4) || misaligned(w_hat_out, 32) || misaligned(scale_out, 4) ||
      misaligned(status, 4))
    return GWS_ERR_ALIGN;
  // An output laid over an input would be overwritten while other thread blocks still read it (every block along M
  // re-reads W, every block along N re-reads X): refused like in gws_sample_fwd.
  const size_t x_bytes = static_cast<size_t>(m) * static_cast<size_t>(k) * 2u, w_bytes = static_cast<size_t>(n) * static_cast<size_t>(k) * 2u;
  const size_t y_bytes = static_cast<size_t>(m) * static_cast<size_t>(n) * 2u, s_bytes = static_cast<size_t>(n) * static_cast<size_t>(k / kTileK) * 4u;
  if (overlaps(y, y_bytes, x, x_bytes) || overlaps(y, y_bytes, w, w_bytes) || overlaps(y, y_bytes, bt, s_bytes)) return GWS_ERR_ALIAS;
  if (w_hat_out != nullptr &&
      (overlaps(w_hat_out, w_bytes, w, w_bytes) || overlaps(w_hat_out, w_bytes, x, x_bytes) || overlaps(w_hat_out, w_bytes, y, y_bytes) ||
       overlaps(w_hat_out, w_bytes, bt, s_bytes)))
    return GWS_ERR_ALIAS;
  if (scale_out != nullptr &&
      (overlaps(scale_out, s_bytes, w, w_bytes) || overlaps(scale_out, s_bytes, x, x_bytes) || overlaps(scale_out, s_bytes, y, y_bytes) ||
       overlaps(scale_out, s_bytes, bt, s_bytes) || (w_hat_out != nullptr && overlaps(scale_out, s_bytes, w_hat_out, w_bytes))))
    return GWS_ERR_ALIAS;

  static EncodeTiled encode = nullptr;
  if (encode == nullptr) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult found;
    const cudaError_t err = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &found);
    if (err != cudaSuccess || found != cudaDriverEntryPointSuccess || fn == nullptr) {
      g_gemm_error = "cuTensorMapEncodeTiled is not available from this driver";
      return GWS_ERR_CUDA;
    }
    encode = reinterpret_cast<EncodeTiled>(fn);
  }
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(k), static_cast<cuuint64_t>(m)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(k) * 2u};
  const cuuint32_t box[2] = {64u, static_cast<cuuint32_t>(kTileM)};
  const cuuint32_t elem_strides[2] = {1u, 1u};
  const CUresult res = encode(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(x), dims, strides, box, elem_strides,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (res != CUDA_SUCCESS) {
    g_gemm_error = "cuTensorMapEncodeTiled failed with CUresult " + std::to_string(static_cast<int>(res));
    return GWS_ERR_CUDA;
  }

  std::memset(&args, 0, sizeof args);
  args.w = w;
  args.bt = bt;
  args.y = y;
  args.w_hat_out = w_hat_out;
  args.scale_out = scale_out;
  args.status = status;
  args.n = static_cast<uint32_t>(n);
  args.k = static_cast<uint32_t>(k);
  args.vec_lo = static_cast<uint32_t>(first_vec);
  args.k0 = static_cast<uint32_t>(wdesc->seed);
  args.k1 = static_cast<uint32_t>(wdesc->seed >> 32);
  args.pre = gws::philox_pre(static_cast<uint32_t>(first_vec >> 32), static_cast<uint32_t>(wdesc->step), static_cast<uint32_t>(wdesc->step >> 32),
                             args.k0, args.k1);
  return GWS_OK;
}

extern "C" {

int gws_gemm_fused(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y, void* w_hat_out,
                   float* scale_out, int* status, int rows_per_block, void* stream) {
  if (rows_per_block != 128 && rows_per_block != 256 && rows_per_block != 512) return wdesc == nullptr ? GWS_ERR_NULL : GWS_ERR_UNSUPPORTED;
  CUtensorMap map;
  GemmArgs args;
  const int st = gemm_prepare(wdesc, m, x, w, bt, y, w_hat_out, scale_out, status, rows_per_block, map, args);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (rows_per_block == 128) return launch_gemm<1>(map, args, m, s);
  if (rows_per_block == 256) return launch_gemm<2>(map, args, m, s);
  return launch_gemm<4>(map, args, m, s);
}

}  // extern "C"

#include "gws_gemm_cluster.cuh"

extern "C" {

int gws_gemm_fused_cluster(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y, void* w_hat_out,
                           float* scale_out, int* status, int cluster_blocks, void* stream) {
  if (cluster_blocks != 1 && cluster_blocks != 2 && cluster_blocks != 4) return wdesc == nullptr ? GWS_ERR_NULL : GWS_ERR_UNSUPPORTED;
  CUtensorMap map;
  GemmArgs args;
  const int st = gemm_prepare(wdesc, m, x, w, bt, y, w_hat_out, scale_out, status, static_cast<int64_t>(kClMT) * kTileM * cluster_blocks, map, args);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cluster_blocks == 1) return launch_gemm_cluster<1>(map, args, m, s);
  if (cluster_blocks == 2) return launch_gemm_cluster<2>(map, args, m, s);
  return launch_gemm_cluster<4>(map, args, m, s);
}

}  // extern "C"

#include "gws_gemm_wide.cuh"

extern "C" {

int gws_gemm_fused_wide(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y, void* w_hat_out,
                        float* scale_out, int* status, int cluster_blocks, void* stream) {
  if (cluster_blocks != 1 && cluster_blocks != 2 && cluster_blocks != 4) return wdesc == nullptr ? GWS_ERR_NULL : GWS_ERR_UNSUPPORTED;
  if (wdesc != nullptr && wdesc->rows > 0 && wdesc->rows % kWdN != 0) return GWS_ERR_UNSUPPORTED;
  CUtensorMap map;
  GemmArgs args;
  const int st = gemm_prepare(wdesc, m, x, w, bt, y, w_hat_out, scale_out, status, static_cast<int64_t>(kWdMT) * kTileM * cluster_blocks, map, args);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (cluster_blocks == 1) return launch_gemm_wide<1>(map, args, m, s);
  if (cluster_blocks == 2) return launch_gemm_wide<2>(map, args, m, s);
  return launch_gemm_wide<4>(map, args, m, s);
}

}  // extern "C"
