/*
 * gws.h - C ABI of the B200 (sm_100a) Gaussian-weight-sampling library.
 *
 * The library runs the per-step weight-sampling pass of GaussWS pseudo-quantization
 * training on one GPU:
 *
 *   forward  (Eq. 3 + the BF16 cast of Section 3.3):
 *       w_hat = bf16_rne( w + R * broadcast( max_group|w| * 2^(1 - b_t) ) )
 *   backward (Eq. 4):
 *       dL/dw = dL/dw_hat,   dL/db_t = -ln2 * max_group|w| * 2^(1-b_t) * sum_group( dL/dw_hat * R )
 *   noise    (Section 3.4, Eq. 9 / Eq. 10): R in {-2,-1,0,1,2}, built from AND / OR of
 *       independent random bits, regenerated in backward from the same counter (Section 3.5,
 *       "GPU memory"; Section 3.6, "Managing seed") instead of being stored.
 *
 * Conventions shared by every entry point
 *   - All data pointers are DEVICE pointers unless a parameter says "host".  The caller owns
 *     every buffer; the library allocates nothing, frees nothing, never synchronises the
 *     device and only enqueues work on `stream` (a cudaStream_t passed as void*; NULL is the
 *     legacy default stream); the one exception is gws_multi_prepare, which waits for its own
 *     table upload.  Inputs are never written.
 *   - A tensor is row-major [rows, cols] of BF16 with `ld` elements between rows (ld >= cols).
 *   - A group is group_rows x group_cols elements; group_cols == 0 means "the whole row".
 *     Groups are numbered row-major over the ceil(rows/group_rows) x ceil(cols/group_cols)
 *     grid, the shape the paper gives b_t under Eq. 3.  Per-group arrays (b_t, scale, absmax,
 *     grad_bt) are dense FP32 in that order.  Edge groups may be ragged.
 *   - Random bits: Philox4x32 with 10 rounds (Section 3.4 names Philox).  Element (i, j) has
 *     the logical index e = elem_offset + i*cols + j (independent of ld).  Counter =
 *     (lo32(e>>3), hi32(e>>3), lo32(step), hi32(step)), key = (lo32(seed), hi32(seed)).  One
 *     call yields four 32-bit words = 128 bits, 16 for each of 8 consecutive elements.
 *     Section 3.4 combines whole random integers with AND / OR, one bit position per element,
 *     so an element's 16 bits are bit columns of the four words, not a run inside one word:
 *     element t = e & 7 (j = t >> 1, h = t & 1) owns columns c+1, c, c-7, c-8 of every word,
 *     c = 16h + 14 - 2j.  Its field bit x_k is bit c + D[k] of word W[k] with
 *     W = {0,1,2,3, 1,2,3, 0,1,2, 0,1,2,3, 0, 3},  D = {-7,-7,-7,-7, -8,-8,-8, 1,1,1, 0,0,0,0, -8, 1}.
 *   - Field bits x0 .. x15:  m2 = x0&...&x7&(x8|x9);  m1 = (x10|x11)&(x12|x13)&x14;
 *     |R| = 2 if m2 else 1 if m1 else 0;  R is negative iff x15 is set and |R| != 0.
 *     This gives exactly Eq. 10: Pr(+-2) = 3/4 * 2^-9 each, Pr(+-1) = (3/4)^2 * 2^-2 *
 *     (1 - 3/1024) each.
 *   - scale_g = fl32( absmax_g * 2^(1 - b_g) ); 2^(1-b) is exact for integer-valued b and is
 *     computed in double then rounded to float otherwise.
 *   - sample: y = fl32( float(w) + float(R) * scale_g ) (the product is exact, no FMA
 *     contraction), w_hat = IEEE round-to-nearest-even of y to BF16.  R == 0 adds +0.0.
 *   - Fast kernels cover dense tensors (ld == cols) with 16-byte aligned pointers, cols % 8 == 0,
 *     elem_offset % 8 == 0 and: group_rows == 1 with group_cols in {8,16,32,64,128,256} dividing
 *     cols; whole-row groups with cols <= 65536; the paper's 32 x 32 blocks when rows and cols are
 *     multiples of 32.  They are fastest with 32-byte aligned pointers (and, for whole rows, cols a
 *     multiple of 32 up to 32768).  Every other legal shape (ragged groups, ld > cols, other 2-D
 *     groups, odd cols, a tensor whose element indices straddle a multiple of 2^35) runs on a
 *     slower general kernel with identical results.
 *   - NaN / Inf in the inputs give unspecified values but never a fault.
 *
 * Every function returns 0 (GWS_OK) or a negative gws_status.  Arguments are validated on
 * the host before anything is launched: a call that fails validation has enqueued nothing.  The
 * calls that issue several launches (the *_multi family, gws_sample_step_host) can also fail in
 * the middle with GWS_ERR_CUDA or GWS_ERR_LIMIT, when the runtime rejects one launch; the launches
 * before it are then already enqueued and their outputs should be treated as unspecified.
 */
#ifndef GWS_H_
#define GWS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum gws_status {
  GWS_OK = 0,
  GWS_ERR_NULL = -1,      /* a required pointer is NULL                                        */
  GWS_ERR_SHAPE = -2,     /* rows/cols < 0, ld < cols, elem_offset % 8 != 0, n < 0             */
  GWS_ERR_GROUP = -3,     /* group_rows < 1 or group_cols < 0                                  */
  GWS_ERR_ALIGN = -4,     /* BF16 pointer not 2-byte aligned / FP32 or u32 pointer not 4-byte  */
  GWS_ERR_ALIAS = -5,     /* output overlaps an input it must not overlap                      */
  GWS_ERR_WORKSPACE = -6, /* workspace NULL, misaligned (256 B) or too small                   */
  GWS_ERR_CUDA = -7,      /* a CUDA runtime call failed; see gws_last_cuda_error()             */
  GWS_ERR_LIMIT = -8,     /* size beyond a documented maximum                                  */
  GWS_ERR_UNSUPPORTED = -9 /* the call needs a different build of the library, or the tensor is
                              outside what the call supports (MX output), or the plan was
                              prepared for another kind of output                              */
} gws_status;

/* One tensor and its noise stream. */
typedef struct gws_desc {
  int64_t rows, cols;   /* logical shape; cols contiguous; 0 rows or cols = nothing to do      */
  int64_t ld;           /* elements between consecutive rows, >= cols                          */
  int32_t group_rows;   /* >= 1; the paper's square block is 32 (Eq. 3, b_l = 32)              */
  int32_t group_cols;   /* >= 1, or 0 for "whole row"                                          */
  uint64_t seed;        /* per-layer seed (output of the layer PRNG of Section 3.6)            */
  uint64_t step;        /* gradient-update counter; same value in forward and backward         */
  uint64_t elem_offset; /* logical index of element (0,0); multiple of 8; 0 unless the tensor
                           is a shard of a larger one whose noise stream it must reproduce     */
} gws_desc;

/* Number of groups of a descriptor (0 if rows or cols is 0, negative gws_status on error). */
int64_t gws_n_groups(const gws_desc* desc);

/*
 * Group absolute maximum, the max_{b_l}(|w|) of Eq. 3.
 *   w       device, BF16 [rows, ld], read only
 *   absmax  device, FP32 [n_groups], written; exact (a BF16 magnitude widened to FP32)
 */
int gws_group_absmax(const gws_desc* desc, const void* w, float* absmax, void* stream);

/*
 * The noise R of Section 3.4 in the packed format of that section's last paragraph:
 * sign-magnitude, 4 bits per element, 8 elements per 32-bit word (0.5 byte per element).
 *   r_packed  device, u32 [ceil(rows*cols/8)], written.  Element k (logical order, no ld)
 *             sits in word k>>3 at bits [4*(k&7), 4*(k&7)+3]; nibble = sign<<3 | |R|; zero is
 *             never negative; unused nibbles of a last partial word are 0.
 * Uses rows, cols, seed, step, elem_offset of the descriptor; ld and the group shape are ignored.
 */
int gws_noise(const gws_desc* desc, uint32_t* r_packed, void* stream);

/*
 * Forward sampling, Eq. 3 followed by the BF16 cast, in one pass over W.
 *   w          device, BF16 [rows, ld], read only
 *   bt         device, FP32 [n_groups], the bit-width b_t of each group, read only
 *   w_hat      device, BF16 [rows, ld], written (padding columns ld > cols are not touched);
 *              must not overlap w
 *   scale_out  device, FP32 [n_groups] or NULL; receives absmax * 2^(1-b_t), the factor the
 *              backward pass needs (W does not change between the two)
 */
int gws_sample_fwd(const gws_desc* desc, const void* w, const float* bt, void* w_hat, float* scale_out,
                   void* stream);

/*
 * Backward, Eq. 4, with R regenerated from (seed, step, element index).
 *   grad_w_hat  device, BF16 [rows, ld], dL/dw_hat, read only
 *   scale       device, FP32 [n_groups], as written by gws_sample_fwd for the same step
 *   grad_w      device, BF16 [rows, ld], NULL or == grad_w_hat: dL/dw is dL/dw_hat itself and
 *               nothing is copied; any other (non-overlapping) pointer receives a bit copy
 *   grad_bt     device, FP32 [n_groups], written: -ln2 * scale * sum_group(grad * R).  The sum
 *               is accumulated in FP32 in a fixed order (run-to-run identical bits).
 */
int gws_sample_bwd(const gws_desc* desc, const void* grad_w_hat, const float* scale, void* grad_w,
                   float* grad_bt, void* stream);

/* ---- tensors held in parts (shards) ---------------------------------------------------------
 * Section 3.5 leaves the 2 bytes per parameter of w_hat to training parallelism: each rank then
 * holds a run of a tensor's elements, and a group can reach across two ranks.  Eq. 3 needs the
 * maximum over the WHOLE group and Eq. 4 the sum over the whole group, so the fused calls above
 * are right only for groups a rank holds completely.  For the others the steps are taken apart:
 * gws_group_absmax on the part (a partial maximum), a MAX reduction between the ranks (the
 * caller's: NCCL or any other), gws_scale_from_absmax, gws_sample_fwd_scaled on the part; in
 * backward gws_sample_bwd on the part with that scale (a partial gradient: Eq. 4 is linear in
 * the group sum) and a SUM reduction.  A part states the logical index of its first element in
 * elem_offset, so it draws the noise the uncut tensor would: the result has the uncut tensor's bits.
 */

/*
 * The per-group factor of Eq. 3, s_g = fl32(absmax_g * 2^(1 - b_g)), from maxima taken earlier:
 * bit-identical to what gws_sample_fwd writes to scale_out for the same maxima and bit-widths.
 *   absmax, bt  device, FP32 [n_groups], read only
 *   scale       device, FP32 [n_groups], written (may be absmax itself)
 * n_groups == 0 does nothing; negative is GWS_ERR_SHAPE.
 */
int gws_scale_from_absmax(int64_t n_groups, const float* absmax, const float* bt, float* scale, void* stream);

/*
 * Forward sampling with the per-group factor supplied: noise, add and BF16 cast of Eq. 3, no
 * maximum taken.  Arguments as gws_sample_fwd, except
 *   scale  device, FP32 [n_groups of desc], read only: s_g of each group of the descriptor.
 * With scale as written by gws_sample_fwd the output equals that call's w_hat bit for bit.
 */
int gws_sample_fwd_scaled(const gws_desc* desc, const void* w, const float* scale, void* w_hat, void* stream);

/* ---- w_hat in a microscaling (MX) floating-point format -----------------------------------------
 * Section 3.1 names MX formats with low-precision FP elements as the target of the method and
 * Table C.1 lists the element types that hold w_hat (FP8_e4m3 up to b_t = 5, FP6_e3m2 up to
 * b_t = 4); the paper itself stores w_hat in BF16 and defines no conversion.  These calls apply
 * the conversion of the OCP Microscaling Formats (MX) specification v1.0 to the BF16 w_hat of
 * Eq. 3, with the sharing rule of Section 3.2: the scaling block is the sampling group, i.e. all
 * 32-element row vectors of a group (a 32 x 32 block, a 1 x G group, a row) carry the same
 * scale, which keeps a square block consistent under transposition.
 *   scale byte (E8M0)  max(E - emax, 0), E = biased exponent of max_group |w_hat|: the shared
 *                      exponent floor(log2 max) - emax clamped below at -127 (emax = 8 for E4M3, else 4)
 *   element            w_hat / 2^(byte - 127), round to nearest even onto the element grid
 *                      (subnormals included), clamped to the largest normal (448 / 28 / 31); the
 *                      sign of zero is kept
 * GWS_MX_FP8_E3M4 is Table C.1's FP8_e3m4, which the paper names without defining and which is not
 * an OCP element type: it is read by analogy with E3M2 (bias 3, every code finite, largest normal 31,
 * emax 4) and converted in integer arithmetic (the GPU has no instruction for it).
 * Buffer layout (one device allocation per tensor, 32-byte aligned, see gws_mx_layout):
 *   [0, codes_bytes)            element codes in logical row-major order.  E4M3 / E3M4: one byte each.
 *                               E3M2: a little-endian bit stream, element k at bits [6k, 6k+5]
 *                               (4 elements in 3 bytes, a 32-element vector in 24).
 *   [scales_offset, total)      one scale byte per 32 elements, [rows, cols/32] row-major;
 *                               scales_offset = codes_bytes rounded up to 256.
 * Supported tensors (anything else: GWS_ERR_UNSUPPORTED, nothing launched): dense (ld == cols),
 * cols a multiple of 32, 32-byte aligned pointers, elem_offset as for the fast kernels, and
 * groups of 1 x {32, 64, 128, 256}, whole rows up to 32768 elements, or 32 x 32 blocks with rows
 * a multiple of 32.
 */
typedef enum gws_mx_format { GWS_MX_FP8_E4M3 = 0, GWS_MX_FP6_E3M2 = 1, GWS_MX_FP8_E3M4 = 2 } gws_mx_format;

/* Sizes of the MX buffer of a tensor; any of the three outputs may be NULL.  Host arithmetic only. */
int gws_mx_layout(const gws_desc* desc, int format, size_t* codes_bytes, size_t* scales_offset, size_t* total_bytes);

/* BF16 w_hat (device, read only) -> MX buffer (device, written).  seed / step are not used. */
int gws_mx_quantize(const gws_desc* desc, int format, const void* w_hat, void* mx_out, void* stream);

/* gws_sample_fwd with the result written as MX instead of BF16, in one pass over W: exactly
 * gws_mx_quantize applied to the w_hat gws_sample_fwd would have written.  scale_out as there. */
int gws_sample_fwd_mx(const gws_desc* desc, int format, const void* w, const float* bt, void* mx_out,
                      float* scale_out, void* stream);

/* ---- sampling fused into the GEMM that consumes w_hat --------------------------------------------
 * Section 3.5 ("Separate kernels") keeps the sampling kernels and the GEMM apart; this entry point is
 * the variant the paper decided against, so that the decision can be measured on this GPU:
 *     Y[m, n] = X[m, k] * W_hat[n, k]^T,   W_hat = Eq. 3 + BF16 cast of W, sampled tile by tile in the
 * prologue of a tcgen05 / TMA GEMM (FP32 accumulation in tensor memory, Y rounded to BF16 once) and
 * never written to global memory unless w_hat_out is given.  W_hat has the bits gws_sample_fwd gives.
 *   wdesc           W: rows = n (a multiple of 128), cols = k (a multiple of 128), dense, groups 1 x 128
 *   m               rows of X and Y, a multiple of rows_per_block
 *   x               device, BF16 [m, k] row-major, 16-byte aligned, read only (through a TMA tensor map)
 *   w, bt           as for gws_sample_fwd; w 32-byte aligned
 *   y               device, BF16 [m, n] row-major, written
 *   w_hat_out       device, BF16 [n, k] or NULL: the sampled weights (written by one block per tile)
 *   scale_out       device, FP32 [n * k / 128] or NULL
 *   status          device, one int or NULL: set to 1 if a block gave up waiting for a copy or for the
 *                   tensor core (about a second); its part of Y is then not written.  Never set otherwise.
 *   rows_per_block  128, 256 or 512: rows of X per thread block; every sampled tile of W is used for that
 *                   many rows, so a larger value repeats less sampling work (512 takes all tensor memory
 *                   and 161 KiB of shared memory of an SM).
 * Other shapes: GWS_ERR_UNSUPPORTED.  An output (y, w_hat_out, scale_out) that overlaps an input (x, w, bt) or
 * another output: GWS_ERR_ALIAS (thread blocks re-read W and X while others write).
 * gws_gemm_last_error() describes a GWS_ERR_CUDA of this call.
 */
int gws_gemm_fused(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y,
                   void* w_hat_out, float* scale_out, int* status, int rows_per_block, void* stream);

/* The same product with every sampled tile of W shared by a cluster of thread blocks (Section 3.5's decision, measured
 * a second way): `cluster_blocks` (1, 2 or 4) blocks of 256 rows of X each, stacked along M, sample 128 / cluster_blocks
 * rows of each 128 x 128 tile of W and store them into the shared memory of all blocks of the cluster, so a tile is
 * sampled once per 256 * cluster_blocks rows of X; the sampling of the next step along K overlaps the tensor-core
 * work of the current one (two stages).  Arguments, results, bits of w_hat_out / scale_out and error behaviour as
 * for gws_gemm_fused; m must be a multiple of 256 * cluster_blocks.  No load is multicast; the blocks of a cluster
 * exchange data only through shared-memory stores and mbarrier arrivals, every wait is bounded as above. */
int gws_gemm_fused_cluster(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y,
                           void* w_hat_out, float* scale_out, int* status, int cluster_blocks, void* stream);

/* The cluster form with 256 x 256 tiles of Y per thread block: tcgen05.mma instructions of N = 256 read a third less
 * shared memory per unit of tensor-core work than those of N = 128 (the X operand is read once for twice the columns) and
 * halve the number of instructions to issue; both accumulators of a block take all 512 columns of an SM's tensor memory.
 * `cluster_blocks` (1, 2 or 4) blocks stacked along M sample 256 / cluster_blocks rows of each 256 x 128 tile of W each, into
 * their own shared memory, and copy that share in bulk into the shared memory of the other blocks of the cluster; X arrives
 * by TMA in steps of 64 along K (three stages).
 * Arguments, results, bits of w_hat_out / scale_out and error behaviour as for gws_gemm_fused; wdesc->rows must be a
 * multiple of 256 and m a multiple of 256 * cluster_blocks.  No load is multicast; every wait is bounded as above. */
int gws_gemm_fused_wide(const gws_desc* wdesc, int64_t m, const void* x, const void* w, const float* bt, void* y,
                        void* w_hat_out, float* scale_out, int* status, int cluster_blocks, void* stream);
const char* gws_gemm_last_error(void);
/* Diagnostic: runs the fused GEMM's bounded wait on an mbarrier that nothing completes (one thread, about a
 * second).  status2: device, two ints, written: [0] = 1 (the wait gave up, as it must), [1] = SM cycles waited / 1024. */
int gws_gemm_wait_probe(int* status2, void* stream);

/* ---- many tensors per launch ---------------------------------------------------------------
 * One linear layer of a 1B-parameter model is a few microseconds of HBM time, so a training
 * step samples all layers with as few launches as possible: tensors that run on the same kernel
 * share a launch.  The tensor set is described once (gws_multi_prepare); each step then calls
 * gws_sample_fwd_multi / gws_sample_bwd_multi with only the step counter changing.
 */

/* Host arrays of n device pointers each; the meaning of every pointer is that of the
 * single-tensor call.  scale is written by forward and read by backward.  grad_w_hat, grad_w and
 * grad_bt may be NULL arrays if backward is never called; w, bt, w_hat if forward is not (bt alone may be NULL
 * in a plan with MX outputs that is only used by gws_mx_quantize_multi). */
typedef struct gws_multi_ptrs {
  const void* const* w;
  const float* const* bt;
  void* const* w_hat;
  float* const* scale;
  const void* const* grad_w_hat;
  void* const* grad_w; /* array may be NULL, and so may each entry: identity, no copy */
  float* const* grad_bt;
  int32_t w_hat_kind;  /* what the w_hat pointers are: 0 = BF16 tensors; 1 + gws_mx_format = MX buffers
                          (gws_mx_layout), to be written by gws_sample_fwd_mx_multi only */
} gws_multi_ptrs;

/* Caller-owned, filled by gws_multi_prepare, read by the *_multi calls.  Plain data. */
typedef struct gws_multi_plan {
  void* workspace;
  const void* host_tables; /* the host copy of the tables (host_workspace of gws_multi_prepare)          */
  int32_t n_tensors;
  int32_t has_fwd, has_bwd;
  int32_t count[4];     /* tensors per class: flat groups, rows <= 4096, rows <= 65536, general (gws_kernel_class) */
  int64_t tiles[4];     /* size of each class in its table's units: 1024-vector tiles, 8-row tiles, rows, blocks  */
  int64_t fwd_offset[4], bwd_offset[4]; /* byte offsets of the class tables inside both workspaces          */
  int64_t total_elements;
  int32_t w_hat_kind;   /* copied from gws_multi_ptrs: a forward call for the other kind of output is refused */
  int32_t reserved;
} gws_multi_plan;

/* Bytes gws_multi_prepare needs for n tensors, both of device workspace (256-byte aligned base) and
 * of host workspace. */
size_t gws_workspace_bytes(int n_tensors);

/*
 * Validate n descriptors and pointer sets, build the tile tables, keep one copy in `host_workspace`
 * (HOST memory, caller-owned, at least gws_workspace_bytes(n)) and copy them into `workspace`
 * (DEVICE memory) on `stream`; the call waits for that copy, so call it outside the training loop.
 * desc[i].step is ignored.  Both workspaces must stay untouched for as long as the plan is used.
 * Launches take their tensor records from the host copy and pass them by value in the kernel
 * parameters (up to 192 flat-group or 168 whole-row records per launch), so that a thread block
 * finds its tensor without a memory access; only the general kernel (ragged groups, padded rows,
 * odd shapes) reads its record from the device copy.
 */
int gws_multi_prepare(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, void* workspace,
                      size_t workspace_bytes, void* host_workspace, size_t host_workspace_bytes,
                      gws_multi_plan* plan_out, void* stream);

/* The bytes gws_multi_prepare would upload, written to HOST memory instead (nothing touches the
 * GPU): lets a caller or a test inspect the tables.  Returns the image size in bytes (pass
 * host_image = NULL to query it) or a negative gws_status.  The image holds, at the byte offsets
 * recorded in the plan, arrays of 112-byte records: in, out, gin, gout (pointers), rows, cols, ld
 * (int64), group_rows, group_cols (int32), elem_offset, n_vec (uint64), seed_lo, seed_hi,
 * vectors_per_row, log2(lanes per group) (uint32), first tile of the tensor in its launch (int64). */
int64_t gws_multi_table_image(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, void* workspace,
                              size_t workspace_bytes, gws_multi_plan* plan_out, void* host_image,
                              size_t host_image_bytes);

/* Diagnostic: resolves n_tiles thread-block indices of one launch (kernel_class 1..2, forward or
 * backward table) to their tensors on the device.  tiles: device, int64 [n_tiles], each inside
 * [0, plan->tiles[kernel_class]).  out: device, u64 [6*n_tiles] = {in, out, gin, gout pointers,
 * tile index inside the tensor, rows of the tensor} per tile.  Reads the tables only. */
int gws_multi_locate_probe(const gws_multi_plan* plan, int backward, int kernel_class, const int64_t* tiles,
                           int n_tiles, uint64_t* out, void* stream);

/* Kernel launches one forward (backward != 0: backward) pass of the plan enqueues.  Tensors that share
 * a kernel share a launch (up to 192 flat-group or 168 whole-row tensors each): flat groups of 32..256
 * elements; flat groups of 8 / 16; rows up to 4096 elements and rows up to 32768 elements, each split
 * by how many 64-byte chunks a thread holds (1 to 4); tensors of whole 32 x 32 blocks.  Whole-row
 * tensors whose rows are not a multiple of 32 elements, are longer, or are not 32-byte aligned, and
 * general-class tensors, take one launch each. */
int gws_multi_launch_count(const gws_multi_plan* plan, int backward);

/* Forward / backward of every tensor of the plan for gradient-update counter `step`. */
int gws_sample_fwd_multi(const gws_multi_plan* plan, uint64_t step, void* stream);
int gws_sample_bwd_multi(const gws_multi_plan* plan, uint64_t step, void* stream);

/* gws_sample_fwd_scaled for every tensor of the plan, with the launches of gws_sample_fwd_multi: the
 * `scale` array each tensor was prepared with is READ (the per-group factor, e.g. after a reduction
 * between ranks) instead of written; `bt` is not used.  GWS_ERR_NULL if the plan has no forward side
 * or a tensor was prepared without a scale array. */
int gws_sample_fwd_scaled_multi(const gws_multi_plan* plan, uint64_t step, void* stream);

/* gws_sample_fwd_mx for every tensor of a plan prepared with w_hat_kind = 1 + format, i.e. whose
 * `w_hat` pointers are MX buffers (gws_mx_layout) instead of BF16 tensors.  GWS_ERR_UNSUPPORTED, with
 * nothing launched, if the plan was prepared for another kind of output or any tensor of it is outside
 * what the MX calls support; gws_sample_fwd_multi and gws_sample_fwd_scaled_multi refuse such a plan
 * the same way (they would write 2 bytes per element). */
int gws_sample_fwd_mx_multi(const gws_multi_plan* plan, int format, uint64_t step, void* stream);

/* gws_mx_quantize for every tensor of such a plan, one launch per kernel class: the plan's `w` pointers are then the
 * BF16 w_hat tensors to convert (read only) and its `w_hat` pointers the MX buffers; `bt` and `scale` are not used and
 * the plan may have been prepared with bt = NULL (gws_sample_fwd_mx_multi then returns GWS_ERR_NULL for it).  Same
 * refusals as gws_sample_fwd_mx_multi. */
int gws_mx_quantize_multi(const gws_multi_plan* plan, int format, void* stream);

/* ---- bit-width parametrisation and seeds (Section 3.6, "Bitwidth" and "Managing seed") ---------------
 *
 * Eq. 11: b_t = b_target + b_i * (b_init - b_target), one trainable b_i per group (initialised to 1,
 * pulled towards 0 by weight decay).  FP32, one rounding per operation (delta = fl(b_init - b_target),
 * fl(b_i * delta), fl(b_target + that)): b_t feeds 2^(1 - b_t), so its bits matter.
 *   bi, bt   device, FP32 [n_groups]; bt may be bi (in place)
 */
int gws_bitwidth(int64_t n_groups, const float* bi, float b_init, float b_target, float* bt, void* stream);

/* One layer's term of Eq. 12 without lambda: loss_out[0] = mean over the layer's m groups of
 * |b_t - b_target| (FP32, summed in a fixed order; 0 for m == 0).  bt, loss_out: device. */
int gws_bitwidth_loss(int64_t m, const float* bt, float b_target, float* loss_out, void* stream);

/* Chain rule back to b_i for one layer of m groups:
 *   grad_bi = (b_init - b_target) * ( grad_bt + lambda / m * sign(b_t - b_target) ),  sign(0) = 0,
 * i.e. Eq. 4's dL/db_t plus the derivative of the layer's Eq. 12 term, through Eq. 11.  lambda = 0
 * gives the plain chain rule.  All arrays device, FP32 [m]; grad_bi may be grad_bt (in place). */
int gws_bitwidth_grad(int64_t m, const float* grad_bt, const float* bt, float b_init, float b_target, double lambda,
                      float* grad_bi, void* stream);

/* Eq. 11 and the chain rule above for many layers at once.  A model has one b_i vector per linear layer, each a few
 * thousand floats: a launch per layer is all launch latency, so these two calls take a host array of items, one per
 * layer, and run them in one launch per 64 layers (the items travel in the kernel parameters; nothing is allocated or
 * copied).  Results are bit for bit those of gws_bitwidth / gws_bitwidth_grad called layer by layer.
 *   gws_bitwidth_multi       uses bi, bt, n, b_init, b_target of every item:   bt = b_target + bi * (b_init - b_target)
 *   gws_bitwidth_grad_multi  uses grad_bt, bt, grad_bi, n, b_init, b_target, lambda, accumulate:
 *                            grad_bi (+)= (b_init - b_target) * (grad_bt + lambda / n * sign(bt - b_target));
 *                            accumulate != 0 adds to what grad_bi holds (gradient accumulation), 0 overwrites it
 * All pointers device, FP32 [n], 4-byte aligned; n is the layer's number of groups (Eq. 12's mean is over them); items with
 * n == 0 are skipped.  items: host memory, read during the call.  Every item is validated before the first launch
 * (GWS_ERR_NULL, GWS_ERR_SHAPE for n < 0, GWS_ERR_LIMIT for n >= 2^31, GWS_ERR_ALIGN). */
typedef struct gws_bitwidth_item {
  const float* bi;
  float* bt;
  const float* grad_bt;
  float* grad_bi;
  int64_t n;
  float b_init, b_target;
  double lambda;
  int32_t accumulate;
  int32_t reserved;
} gws_bitwidth_item;
int gws_bitwidth_multi(int n_items, const gws_bitwidth_item* items, void* stream);
int gws_bitwidth_grad_multi(int n_items, const gws_bitwidth_item* items, void* stream);

/* Host only.  The seed of layer `layer` under the user's seed: the first 64 output bits of
 * Philox4x32-10 with counter (lo32(layer), hi32(layer), 0, 0) and key (lo32(user_seed), hi32(user_seed)).
 * The per-update change of a layer's PRNG state is the `step` of its descriptor. */
uint64_t gws_layer_seed(uint64_t user_seed, uint64_t layer);

/* ---- forward over many tensors for callers that cannot allocate device memory --------------------
 * (No counterpart in the paper: this entry point exists for the way the library gets embedded.)
 *
 * Some callers have nowhere to get the table workspace from: code that runs inside a framework's
 * allocator hooks or out-of-memory handlers, plug-ins that are handed tensors but no allocator, and
 * processes that have given all device memory to a pool at start-up and must not call cudaMalloc
 * afterwards (it would fail, or synchronise the device in the middle of a step).  For them the tensor
 * table lives in an array compiled into the library: sizeof = GWS_STATIC_MAX_TENSORS * 224 + 2048
 * bytes (about 59 KB) of device memory on every GPU that loads the library, held until the process
 * exits.  The call does what gws_multi_prepare followed by gws_sample_fwd_multi does, for the
 * forward pass only, and allocates no device memory, frees none and calls no allocating library
 * routine.
 *   n, descs, ptrs   as for gws_multi_prepare; only w, bt, w_hat and scale of `ptrs` are used
 *                    (scale, and each of its entries, may be NULL) and w_hat must be BF16 tensors
 *                    (w_hat_kind = 0, anything else is GWS_ERR_UNSUPPORTED).  n > GWS_STATIC_MAX_TENSORS
 *                    returns GWS_ERR_LIMIT.  Every error found while validating the arguments is
 *                    returned before the array is touched and before anything is enqueued.
 *   stream           must not be recording (cudaStreamBeginCapture): the call then returns
 *                    GWS_ERR_UNSUPPORTED with nothing enqueued, because its table upload reads host
 *                    memory that lives only for the duration of the call.
 *   step             gradient-update counter, as for gws_sample_fwd_multi
 * Results are bit-identical to gws_sample_fwd_multi.  Things to know:
 *   - The first call on each device looks up the array's device address (with that device current).
 *     Make that first call outside any stream capture.
 *   - Every call on a device rewrites the same array before launching, in stream order.  Two calls
 *     whose work can overlap on the GPU (different streams without an ordering between them, or
 *     different host threads doing so) race on it: keep all calls on one stream, or order them
 *     with events.  Nothing in the array has to be cleared between calls: each call overwrites all
 *     of what its own kernels read.
 *   - The table is uploaded from pageable host memory on `stream`, so the call may wait for earlier
 *     work on that stream; gws_multi_prepare + gws_sample_fwd_multi avoid that per-step cost and
 *     remain the better choice for callers that can allocate.
 */
#define GWS_STATIC_MAX_TENSORS 256
int gws_sample_fwd_multi_static(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, uint64_t step,
                                void* stream);

/* ---- host-buffer step (end-to-end path) --------------------------------------------------------
 * One forward + backward of one tensor whose data lives in HOST memory (pinned memory makes the
 * copies asynchronous).  Copies w, bt, grad_w_hat to the device staging buffers, runs
 * gws_sample_fwd and gws_sample_bwd, copies w_hat, scale and grad_bt back, all on `stream`;
 * returns without synchronising.
 *   h_w, h_bt, h_grad_w_hat   host inputs  (BF16 [rows, ld], FP32 [n_groups], BF16 [rows, ld])
 *   h_w_hat, h_scale, h_grad_bt  host outputs
 *   d_w, d_w_hat, d_grad      device staging, each rows*ld BF16; d_bt, d_scale, d_grad_bt device
 *                             staging, each n_groups FP32
 */
int gws_sample_step_host(const gws_desc* desc, const void* h_w, const float* h_bt, const void* h_grad_w_hat,
                         void* h_w_hat, float* h_scale, float* h_grad_bt, void* d_w, void* d_w_hat, void* d_grad,
                         float* d_bt, float* d_scale, float* d_grad_bt, void* stream);

/* ---- comparison noises ----------------------------------------------------------------------------
 * The forward pass of Eq. 3 with the noise R replaced by what the paper measures its generation against, on the same
 * kernel shape, so that the cost of the noise can be compared on one harness (Section 4.2 "Overhead": forward unit
 * benchmark with the series "ours" and "bm"; Section 4, first paragraph: "DiffQ" = the method with BF16 U(-0.5, 0.5)
 * in place of R).  Not part of the sampling pass.
 *   GWS_NOISE_UNIFORM_BF16   u = bf16_rne((x + 1/2) / 2^16 - 1/2), x the 16-bit field at bits [16 (e & 1), +16) of
 *                            word (e >> 1) & 3 of Philox4x32-10(counter = (e >> 3, step), key = seed)
 *   GWS_NOISE_BOX_MULLER     R = round-half-even(z / 2), z the Box-Muller normal of element e: one Philox call with
 *                            counter (e >> 2, step) serves 4 elements, words (o0, o1) give elements 4c, 4c + 1 and
 *                            (o2, o3) give 4c + 2, 4c + 3; u1 = ((a >> 8) + 1) / 2^24, u2 = (b >> 8) / 2^24,
 *                            z = sqrt(-2 ln u1) * (cos, sin)(2 pi u2) in FP32 (so an R may differ from an FP64
 *                            evaluation where z / 2 is within rounding of k + 1/2)
 * w_hat = bf16( fl32( float(w) + fl32( noise * scale_g ) ) ), scale_g as in gws_sample_fwd.
 * Shapes: dense, group_rows = 1, group_cols in {32, 64, 128, 256} dividing cols, elem_offset % 32 == 0, w and w_hat
 * 32-byte aligned; anything else GWS_ERR_UNSUPPORTED.  Arguments as gws_sample_fwd. */
typedef enum gws_noise_kind { GWS_NOISE_UNIFORM_BF16 = 0, GWS_NOISE_BOX_MULLER = 1 } gws_noise_kind;
int gws_sample_fwd_compare(const gws_desc* desc, int noise_kind, const void* w, const float* bt, void* w_hat,
                           float* scale_out, void* stream);
/* The comparison noise alone for rows * cols elements (a multiple of 8, as is elem_offset).  out: device, 16-byte aligned;
 * GWS_NOISE_UNIFORM_BF16: one BF16 pattern per element (u16 [rows * cols]); GWS_NOISE_BOX_MULLER: sign-magnitude nibbles
 * as written by gws_noise (u32 [rows * cols / 8], |R| <= 3). */
int gws_noise_compare(const gws_desc* desc, int noise_kind, void* out, void* stream);

/* ---- diagnostics -----------------------------------------------------------------------------*/

/* Raw Philox4x32-10 output words for vectors first_vec .. first_vec+n_vec-1 (4 words each):
 * the random bits of Section 3.4 before decoding.  out4: device, u32 [4*n_vec]. */
int gws_philox_words(uint64_t seed, uint64_t step, uint64_t first_vec, int64_t n_vec, uint32_t* out4,
                     void* stream);

/* Generates and decodes the noise of the descriptor with the arithmetic gws_sample_fwd / gws_sample_bwd
 * spend on it (Philox4x32-10 and the AND / OR decode of Eq. 10) but stores only one word per thread
 * block (an XOR of what it decoded): the rate of random-bit generation without memory traffic, which
 * the backward pass (2 bytes per element) cannot exceed.  sink: device, u32 [gws_noise_alu_probe_words(desc)]. */
int gws_noise_alu_probe(const gws_desc* desc, uint32_t* sink, void* stream);
int64_t gws_noise_alu_probe_words(const gws_desc* desc);

/* Issue cost of the instruction kinds the passes are made of (Section 3.4's generation is integer work: per 8
 * elements Philox4x32-10 takes 18 multiplies 32 x 32 -> 64 and 19 three-input XORs once its launch-uniform part is
 * hoisted, the AND / OR decode of Eq. 10 another 14 logic operations).  gws_issue_probe runs `iterations` x 32 steps
 * per thread of instruction mix `mix` on 64 warps per SM with no memory traffic; the caller times the launch.
 *   gws_issue_probe_mix(mix, counts7)  host only: instructions per step {multiply 32x32->64, XOR fed by it, other
 *       logic, FP32 FMA, FP32 += BF16*BF16 FMA, integer add, byte permute}; returns the steps per thread and
 *       iteration (32), or GWS_ERR_UNSUPPORTED for an unknown mix.  mix = 100 + pieces runs the arithmetic of a pass
 *       instead (pieces 1: Philox; 3: + gradient decode; 7: + the gradient sum's FMAs, i.e. the backward pass; 9:
 *       Philox + forward decode + Eq. 3's add and BF16 packing); `iterations` then counts 8-element vectors per
 *       thread (a multiple of 4) and the return value is 1.
 *   sink        device, u32 [8]: [0] SM cycles and [1] nanoseconds one warp spent in the loop (their ratio is the SM
 *               clock in GHz during the probe)
 *   host_info2  host, int32 [2]: thread blocks launched (of 256 threads), SMs of the device */
int gws_issue_probe_mix(int mix, int32_t* counts7);
int gws_issue_probe(int mix, int iterations, uint32_t* sink, int32_t* host_info2, void* stream);

/* Host-side evaluation of the same inline decode / Philox code the kernels use (no GPU needed):
 * r8 receives R for the 8 fields of the 4 words; packed receives the nibble word. */
void gws_host_decode8(const uint32_t* words4, int8_t* r8, uint32_t* packed);
/* The decode's raw output, four words holding the BF16 patterns of 2R for elements (2j, 2j+1), from the form the
 * forward pass uses (a zero is always +0) and from the form the gradient sum of Eq. 4 uses (a zero may be -0). */
void gws_host_decode8_pairs(const uint32_t* words4, uint32_t* pairs4, uint32_t* pairs4_signed_zero);
void gws_host_philox(uint64_t seed, uint64_t step, uint64_t vec, uint32_t* out4);

/* Self-checking build (compiled with -DGWS_SELF_CHECK; gws_selfcheck_enabled() returns 1): every
 * kernel access to caller memory is tested against the window [base, base+bytes) declared here; an
 * access outside it is counted, the first one recorded, and skipped instead of performed.  Both calls
 * synchronise the device.  report: out5 (host) = {violations, kind of the first (1 vector load,
 * 2 vector store, 3 float load, 4 float store, 5 element load, 6 element store), its address, block,
 * thread}.  In the normal build both return GWS_ERR_UNSUPPORTED. */
int gws_selfcheck_enabled(void);
int gws_selfcheck_set_window(const void* base, size_t bytes);
int gws_selfcheck_report(uint64_t* out5);

/* Which kernel class a descriptor with fully aligned pointers would use:
 * 0 flat groups, 1 warp per row, 2 thread block per row, 3 general; negative gws_status on error. */
int gws_kernel_class(const gws_desc* desc);

const char* gws_status_string(int status);
/* Text of the last CUDA error this thread saw inside the library ("" if none). */
const char* gws_last_cuda_error(void);
/* Count of kernel launches the library has enqueued since load (all threads). */
uint64_t gws_launch_count(void);

/* Launch overlap (off when the library is loaded; the setting is process-wide and read at every launch).
 *
 * The sampling pass on a small weight set is a handful of launches of some tens of microseconds each, and every launch
 * spends several microseconds filling the GPU and several more draining it (the per-step cost Section 3.5 counts as
 * "separate kernels").  With the overlap enabled, the kernels of the flat-group, whole-row and square-block classes are
 * launched with programmatic stream serialization: the blocks of a launch may become resident while the last blocks of
 * the kernel BEFORE it on the same stream still run.  They read nothing but their kernel parameters until that kernel
 * has completed and its writes are visible (griddepcontrol.wait stands before their first access to global memory), so
 * every result is bit for bit that of an ordinary launch and stream order still holds between any two kernels; only the
 * fill of one launch now overlaps the drain of the one before.  The vector and general kernels are launched as before,
 * and so is every kernel enqueued on a stream that is recording a CUDA graph.
 *
 * enable: 0 = ordinary launches, anything else = overlapping launches.  Returns the previous setting (0 or 1); never
 * fails and enqueues nothing.  A kernel of another library that follows one of these on the stream is unaffected (it is
 * not launched with the attribute); one that precedes them is simply waited for. */
int gws_set_launch_overlap(int enable);

#ifdef __cplusplus
}
#endif
#endif /* GWS_H_ */
