// Host side of the C ABI declared in gws.h: argument validation, choice of kernel class,
// launch geometry, the multi-tensor table.  No device memory is allocated here.
#include <algorithm>
#include <atomic>
#include <cstdio>
#include <cstring>
#include <string>
#include <vector>

#include "gws.h"
#ifndef GWS_FLAT_CPT_FWD
#define GWS_FLAT_CPT_FWD 2
#endif
#ifndef GWS_FLAT_CPT_BWD
#define GWS_FLAT_CPT_BWD 2
#endif
#include "gws_kernels.cuh"
#include "gws_probe.cuh"
#include "gws_compare.cuh"
#include "gws_train.cuh"

namespace {

using gws::Entry;

thread_local std::string g_last_cuda_error;
std::atomic<uint64_t> g_launches{0};

constexpr int64_t kMaxGrid = 2147483647LL;
constexpr int kGeneralGrid = 148 * 8;

int cuda_fail(cudaError_t err, const char* what) {
  g_last_cuda_error = std::string(what) + ": " + cudaGetErrorString(err);
  return GWS_ERR_CUDA;
}

int check_launch(const char* what) {
  g_launches.fetch_add(1, std::memory_order_relaxed);
  const cudaError_t err = cudaGetLastError();
  return err == cudaSuccess ? GWS_OK : cuda_fail(err, what);
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

int validate_desc(const gws_desc* d) {
  if (d == nullptr) return GWS_ERR_NULL;
  if (d->rows < 0 || d->cols < 0) return GWS_ERR_SHAPE;
  if (d->rows > 0 && d->cols > 0 && d->ld < d->cols) return GWS_ERR_SHAPE;
  if (d->elem_offset % 8 != 0) return GWS_ERR_SHAPE;
  if (d->group_rows < 1 || d->group_cols < 0) return GWS_ERR_GROUP;
  if (d->rows > 0 && d->cols > 0 && (d->rows > (INT64_MAX / 4) / d->cols || d->rows > (INT64_MAX / 4) / d->ld))
    return GWS_ERR_LIMIT;
  return GWS_OK;
}

bool is_empty(const gws_desc* d) { return d->rows == 0 || d->cols == 0; }

int64_t resolved_group_cols(const gws_desc* d) { return d->group_cols == 0 ? d->cols : d->group_cols; }

int64_t n_groups_of(const gws_desc* d) {
  if (is_empty(d)) return 0;
  const int64_t gc = resolved_group_cols(d);
  return ((d->rows + d->group_rows - 1) / d->group_rows) * ((d->cols + gc - 1) / gc);
}

// Bytes spanned by a [rows, ld] BF16 tensor with `cols` used columns.
size_t span_bytes(const gws_desc* d) { return static_cast<size_t>((d->rows - 1) * d->ld + d->cols) * 2u; }

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
  const uintptr_t x = reinterpret_cast<uintptr_t>(a), y = reinterpret_cast<uintptr_t>(b);
  return x < y + nb && y < x + na;
}

// Kernel class for a descriptor; `vec_ok` says whether every tensor pointer is 16-byte aligned.
int classify(const gws_desc* d, bool vec_ok) {
  const int64_t gc = resolved_group_cols(d);
  const bool dense = vec_ok && d->ld == d->cols && d->cols % 8 == 0 && d->group_rows == 1;
  if (!dense) return gws::kGeneral;
  // flat kernels keep the high word of the Philox counter uniform: the tensor's vectors must not straddle 2^32
  const uint64_t first_vec = d->elem_offset >> 3, last_vec = first_vec + static_cast<uint64_t>(d->rows * d->cols / 8) - 1;
  const bool uniform_hi = (first_vec >> 32) == (last_vec >> 32) && (last_vec - first_vec) < 0xFFFFFFFFull;
  if (gc <= 256 && gc >= 8 && (gc & (gc - 1)) == 0 && d->cols % gc == 0 && uniform_hi) return gws::kFlat;
  if (gc == d->cols) {
    const int64_t vpr = d->cols / 8;
    if (vpr <= 32 * gws::kRowWarpVecs) return gws::kRowWarp;
    if (vpr <= static_cast<int64_t>(gws::kRowCtaThreads) * gws::kRowCtaVecs) return gws::kRowCta;
  }
  return gws::kGeneral;
}

int64_t tiles_of(const gws_desc* d, int cls) {
  switch (cls) {
    case gws::kFlat: {
      const int64_t n_vec = d->rows * d->cols / 8;
      const int64_t per = static_cast<int64_t>(gws::kFlatThreads) * gws::kFlatVecs;
      return (n_vec + per - 1) / per;
    }
    case gws::kRowWarp:
      return (d->rows + (gws::kRowWarpThreads / 32) - 1) / (gws::kRowWarpThreads / 32);
    case gws::kRowCta:
      return d->rows;
    default: {
      const int64_t ng = n_groups_of(d);
      return ng < kGeneralGrid ? ng : kGeneralGrid;
    }
  }
}

Entry make_entry(const gws_desc* d, int cls, const void* in, void* out, const float* gin, float* gout) {
  Entry e;
  std::memset(&e, 0, sizeof e);
  e.in = in;
  e.out = out;
  e.gin = gin;
  e.gout = gout;
  e.rows = d->rows;
  e.cols = d->cols;
  e.ld = d->ld;
  e.group_rows = d->group_rows;
  e.group_cols = static_cast<int32_t>(resolved_group_cols(d) > INT32_MAX ? INT32_MAX : resolved_group_cols(d));
  e.elem_offset = d->elem_offset;
  e.n_vec = static_cast<uint64_t>(d->rows * d->cols / 8);
  e.seed_lo = static_cast<uint32_t>(d->seed);
  e.seed_hi = static_cast<uint32_t>(d->seed >> 32);
  e.vpr = static_cast<uint32_t>(d->cols / 8);
  e.lanes_log2 = 0;
  if (cls == gws::kFlat) {
    int64_t lanes = resolved_group_cols(d) / 8;
    while (lanes > 1) { lanes >>= 1; ++e.lanes_log2; }
  }
  e.tile_begin = 0;
  return e;
}

// ---- layout of an MX buffer ----------------------------------------------------------------------------
// Element codes first (E4M3: one byte per element; E3M2: 6 bits per element), then, from the next multiple of
// 256 bytes, one E8M0 scale byte per 32 elements.
size_t mx_codes_bytes(int64_t n_elements, int format) {
  return format == gws::kMxE3M2 ? static_cast<size_t>(n_elements) / 4u * 3u : static_cast<size_t>(n_elements);
}
size_t mx_scales_offset(int64_t n_elements, int format) { return (mx_codes_bytes(n_elements, format) + 255u) & ~static_cast<size_t>(255u); }
size_t mx_total_bytes(int64_t n_elements, int format) { return mx_scales_offset(n_elements, format) + static_cast<size_t>(n_elements) / 32u; }

// The `pad` field of a record: where the scale bytes start inside the output buffer, in units of 16 bytes (MX modes only).
template <int MODE>
uint32_t mx_scales_off16(const Entry& e) {
  if (!(gws::mode_is_mx_fwd(MODE) || gws::mode_is_mx_quant(MODE))) return 0u;
  return static_cast<uint32_t>(mx_scales_offset(e.rows * e.cols, gws::mode_mx_format(MODE)) / 16u);
}

// ---- launches of the chunk kernels (flat groups, rows, square blocks) ----------------------------------

// When set, the chunk kernels are launched with programmatic stream serialization: their blocks may become resident while
// the last blocks of the kernel before them on the stream still run, and wait there (griddepcontrol.wait, before their first
// access to global memory) until that kernel has completed.  Results are those of an ordinary launch; what changes is that the
// start of one launch overlaps the end of the one before it.
std::atomic<int> g_launch_overlap{0};

template <typename Kernel, typename Batch>
void launch_chunk_kernel(Kernel kernel, unsigned grid, unsigned block, cudaStream_t stream, const Batch& batch) {
  cudaLaunchConfig_t cfg;
  std::memset(&cfg, 0, sizeof cfg);
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(block);
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 0;
  if (g_launch_overlap.load(std::memory_order_relaxed) != 0) {   // a stream that records a graph gets ordinary launches
    cudaStreamCaptureStatus capture = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing(stream, &capture) == cudaSuccess && capture == cudaStreamCaptureStatusNone) cfg.numAttrs = 1;
  }
  cudaLaunchKernelEx(&cfg, kernel, batch);   // the error, if any, is read by check_launch
}

// ---- flat-group launches: tensor records by value in the kernel parameters ---------------------------

gws::FlatRec to_flat_rec(const Entry& e) {
  gws::FlatRec r;
  std::memset(&r, 0, sizeof r);
  r.in = e.in;
  r.out = e.out;
  r.gin = e.gin;
  r.gout = e.gout;
  r.vec_lo = static_cast<uint32_t>(e.elem_offset >> 3);
  r.vec_hi = static_cast<uint32_t>(e.elem_offset >> 35);
  r.n_vec = static_cast<uint32_t>(e.n_vec);   // classify() keeps tensors of 2^32 vectors or more out of this class
  r.k0 = e.seed_lo;
  r.k1 = e.seed_hi;
  r.lanes_log2 = e.lanes_log2;
  return r;
}

// Chunks (64 bytes) a thread handles in each mode.
template <int MODE, int VARIANT>
constexpr int flat_cpt() {
  return VARIANT == gws::kNarrow ? 1 : (MODE == gws::kBwd ? GWS_FLAT_CPT_BWD : GWS_FLAT_CPT_FWD);
}

template <int MODE, int VARIANT, int CAP>
int launch_flat_batch(gws::FlatRec* recs, int count, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  constexpr int CPT = flat_cpt<MODE, VARIANT>();
  gws::FlatBatch<CAP> b;
  std::memset(&b, 0, sizeof b);
  const int64_t tiles = gws::fill_flat_batch<CAP>(b, recs, count, CPT, lo, hi);
  if (tiles < 0) return GWS_ERR_LIMIT;
  if (tiles == 0) return GWS_OK;
  launch_chunk_kernel(gws::k_flat<MODE, VARIANT, CAP, CPT>, static_cast<unsigned>(tiles), gws::kFlatThreads, stream, b);
  return check_launch("flat-group kernel");
}

template <int MODE, int VARIANT>
int launch_flat_variant(std::vector<gws::FlatRec>& recs, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  for (size_t first = 0; first < recs.size(); first += gws::kFlatCapLarge) {
    const int count = static_cast<int>(std::min(recs.size() - first, static_cast<size_t>(gws::kFlatCapLarge)));
    const int st = count <= gws::kFlatCapSmall
                       ? launch_flat_batch<MODE, VARIANT, gws::kFlatCapSmall>(recs.data() + first, count, lo, hi, stream)
                       : launch_flat_batch<MODE, VARIANT, gws::kFlatCapLarge>(recs.data() + first, count, lo, hi, stream);
    if (st != GWS_OK) return st;
  }
  return GWS_OK;
}

// Launches needed for `count` flat-class entries: groups of 8 / 16 elements run apart from the wider ones.
template <int MODE>
int launch_flat(const Entry* entries, int count, uint64_t step, cudaStream_t stream) {
  std::vector<gws::FlatRec> wide, narrow;
  bool all32 = true;
  for (int k = 0; k < count; ++k) {
    const gws::FlatRec r = to_flat_rec(entries[k]);
    if (r.lanes_log2 < 2u) { narrow.push_back(r); continue; }
    wide.push_back(r);
    all32 = all32 && aligned(r.in, 32) && aligned(r.out, 32);
  }
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  int st = all32 ? launch_flat_variant<MODE, gws::kWide32>(wide, lo, hi, stream)
                 : launch_flat_variant<MODE, gws::kWide16>(wide, lo, hi, stream);
  if (st != GWS_OK) return st;
  return launch_flat_variant<MODE, gws::kNarrow>(narrow, lo, hi, stream);
}

// ---- whole-row launches on chunks -------------------------------------------------------------------

// The chunk kernel takes rows of a multiple of 32 elements up to 32768, 32-byte aligned, whose Philox
// counters share one high word; everything else of the row classes runs on the vector kernels.
bool row_chunk_eligible(const Entry& e) {
  if (e.cols % 32 != 0 || e.cols > 32768 || e.ld != e.cols || e.group_rows != 1 || e.group_cols != e.cols) return false;
  if (!aligned(e.in, 32) || !aligned(e.out, 32)) return false;
  const uint64_t first = e.elem_offset >> 3, last = first + e.n_vec - 1;
  return (first >> 32) == (last >> 32) && (last - first) < 0xFFFFFFFFull;
}

gws::RowRec to_row_rec(const Entry& e) {
  gws::RowRec r;
  std::memset(&r, 0, sizeof r);
  r.in = e.in;
  r.out = e.out;
  r.gin = e.gin;
  r.gout = e.gout;
  r.vec_lo = static_cast<uint32_t>(e.elem_offset >> 3);
  r.vec_hi = static_cast<uint32_t>(e.elem_offset >> 35);
  r.rows = static_cast<uint32_t>(e.rows);
  r.cpr = static_cast<uint32_t>(e.cols / 32);
  r.k0 = e.seed_lo;
  r.k1 = e.seed_hi;
  if (r.cpr > 128u) {   // one block per row
    r.tpr_log2 = 8;
    r.cpt = (r.cpr + gws::kRowThreads - 1) / gws::kRowThreads;
  } else {              // 1..32 threads per row: the (threads, chunks per thread) pair with the fewest idle slots
    uint32_t best_slots = ~0u;
    for (uint32_t cpt = 1; cpt <= static_cast<uint32_t>(gws::kRowMaxCpt); ++cpt) {
      uint32_t need = (r.cpr + cpt - 1) / cpt, log2 = 0;
      while ((1u << log2) < need) ++log2;
      if (log2 > 5u) continue;
      const uint32_t slots = (1u << log2) * cpt;
      if (slots < best_slots) { best_slots = slots; r.tpr_log2 = log2; r.cpt = cpt; }
    }
  }
  return r;
}

template <int MODE, bool BLOCK, int CAP, int MAXCPT>
int launch_row_batch(const gws::RowRec* recs, int count, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  gws::RowBatch<CAP> b;
  std::memset(&b, 0, sizeof b);
  const int64_t tiles = gws::fill_row_batch<CAP>(b, recs, count, BLOCK, lo, hi);
  if (tiles < 0) return GWS_ERR_LIMIT;
  if (tiles == 0) return GWS_OK;
  launch_chunk_kernel(gws::k_row<MODE, BLOCK, CAP, MAXCPT>, static_cast<unsigned>(tiles), gws::kRowThreads, stream, b);
  return check_launch("row kernel");
}

// Register-array size class of a record: its chunks per thread (1..4).
int row_cpt_class(const gws::RowRec& r) { return static_cast<int>(r.cpt < 1u ? 1u : r.cpt); }

template <int MODE, bool BLOCK, int MAXCPT>
int launch_row_chunks_of(const std::vector<gws::RowRec>& all, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  std::vector<gws::RowRec> recs;
  for (const gws::RowRec& r : all)
    if (row_cpt_class(r) == MAXCPT) recs.push_back(r);
  for (size_t first = 0; first < recs.size(); first += gws::kRowCapLarge) {
    const int count = static_cast<int>(std::min(recs.size() - first, static_cast<size_t>(gws::kRowCapLarge)));
    const int st = count <= gws::kRowCapSmall
                       ? launch_row_batch<MODE, BLOCK, gws::kRowCapSmall, MAXCPT>(recs.data() + first, count, lo, hi, stream)
                       : launch_row_batch<MODE, BLOCK, gws::kRowCapLarge, MAXCPT>(recs.data() + first, count, lo, hi, stream);
    if (st != GWS_OK) return st;
  }
  return GWS_OK;
}

template <int MODE, bool BLOCK>
int launch_row_chunks(const std::vector<gws::RowRec>& recs, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  int st = launch_row_chunks_of<MODE, BLOCK, 1>(recs, lo, hi, stream);
  if (st == GWS_OK) st = launch_row_chunks_of<MODE, BLOCK, 2>(recs, lo, hi, stream);
  if (st == GWS_OK) st = launch_row_chunks_of<MODE, BLOCK, 3>(recs, lo, hi, stream);
  if (st == GWS_OK) st = launch_row_chunks_of<MODE, BLOCK, 4>(recs, lo, hi, stream);
  return st;
}

template <int MODE>
int launch(int cls, const Entry& single, const Entry* table, int n_or_index, int64_t tiles, uint64_t step,
           cudaStream_t stream);

// All entries of a row class (kRowWarp or kRowCta): chunk kernel where it applies, else one launch each.
template <int MODE>
int launch_rows(int cls, const Entry* entries, int count, uint64_t step, cudaStream_t stream) {
  std::vector<gws::RowRec> shared_rows, block_rows;
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  for (int k = 0; k < count; ++k) {
    if (row_chunk_eligible(entries[k])) {
      const gws::RowRec r = to_row_rec(entries[k]);
      (r.tpr_log2 == 8u ? block_rows : shared_rows).push_back(r);
    } else {
      Entry e = entries[k];
      e.tile_begin = 0;
      const int64_t tiles = cls == gws::kRowWarp ? (e.rows + (gws::kRowWarpThreads / 32) - 1) / (gws::kRowWarpThreads / 32) : e.rows;
      const int st = launch<MODE>(cls, e, nullptr, -1, tiles, step, stream);
      if (st != GWS_OK) return st;
    }
  }
  const int st = launch_row_chunks<MODE, false>(shared_rows, lo, hi, stream);
  if (st != GWS_OK) return st;
  return launch_row_chunks<MODE, true>(block_rows, lo, hi, stream);
}

// ---- 32 x 32 square blocks --------------------------------------------------------------------------

bool square_eligible(const Entry& e) {
  if (e.group_rows != 32 || e.group_cols != 32 || e.rows % 32 != 0 || e.cols % 32 != 0 || e.ld != e.cols) return false;
  if (!aligned(e.in, 32) || !aligned(e.out, 32)) return false;
  const uint64_t n_vec = static_cast<uint64_t>(e.rows) * static_cast<uint64_t>(e.cols) / 8u;
  const uint64_t first = e.elem_offset >> 3, last = first + n_vec - 1;
  return (first >> 32) == (last >> 32) && (last - first) < 0xFFFFFFFFull;
}

template <int MODE, int CAP>
int launch_square_batch(const Entry* const* entries, int count, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  gws::SquareBatch<CAP> b;
  std::memset(&b, 0, sizeof b);
  gws::SquareRec recs[CAP];
  uint32_t bands[CAP];
  for (int k = 0; k < count; ++k) {
    const Entry& e = *entries[k];
    gws::SquareRec& r = recs[k];
    std::memset(&r, 0, sizeof r);
    r.in = e.in;
    r.out = e.out;
    r.gin = e.gin;
    r.gout = e.gout;
    r.vec_lo = static_cast<uint32_t>(e.elem_offset >> 3);
    r.vec_hi = static_cast<uint32_t>(e.elem_offset >> 35);
    r.cpr = static_cast<uint32_t>(e.cols / 32);
    r.k0 = e.seed_lo;
    r.k1 = e.seed_hi;
    r.pad = mx_scales_off16<MODE>(e);
    bands[k] = static_cast<uint32_t>(e.rows / 32);
  }
  const int64_t tiles = gws::fill_square_batch<CAP>(b, recs, bands, count, lo, hi);
  if (tiles < 0) return GWS_ERR_LIMIT;
  if (tiles == 0) return GWS_OK;
  launch_chunk_kernel(gws::k_square<MODE, CAP>, static_cast<unsigned>(tiles), gws::kFlatThreads, stream, b);
  return check_launch("square-block kernel");
}

template <int MODE>
int launch_squares(const std::vector<const Entry*>& entries, uint64_t step, cudaStream_t stream) {
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  for (size_t first = 0; first < entries.size(); first += gws::kFlatCapLarge) {
    const int count = static_cast<int>(std::min(entries.size() - first, static_cast<size_t>(gws::kFlatCapLarge)));
    const int st = count <= gws::kFlatCapSmall
                       ? launch_square_batch<MODE, gws::kFlatCapSmall>(entries.data() + first, count, lo, hi, stream)
                       : launch_square_batch<MODE, gws::kFlatCapLarge>(entries.data() + first, count, lo, hi, stream);
    if (st != GWS_OK) return st;
  }
  return GWS_OK;
}

// ---- MX output (element codes + scale bytes instead of BF16) -----------------------------------------------
//
// Only the kernels that work on 64-byte chunks write MX (a chunk is one 32-element MX vector): flat groups of 32
// to 256 elements, whole rows of a multiple of 32 elements up to 32768, whole 32 x 32 blocks; dense, 32-byte
// aligned.  Everything else is GWS_ERR_UNSUPPORTED, decided before anything is launched.
bool mx_entry_ok(int cls, const Entry& e) {
  if (e.cols % 32 != 0 || e.ld != e.cols || !aligned(e.in, 32) || !aligned(e.out, 32)) return false;
  if (cls == gws::kFlat) return e.lanes_log2 >= 2u;
  if (cls == gws::kRowWarp || cls == gws::kRowCta) return row_chunk_eligible(e);
  return square_eligible(e);
}

// `count` entries of one kernel class, all of them passing mx_entry_ok.
template <int MODE>
int launch_mx(int cls, const Entry* entries, int count, uint64_t step, cudaStream_t stream) {
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  if (cls == gws::kFlat) {
    std::vector<gws::FlatRec> recs;
    for (int k = 0; k < count; ++k) {
      gws::FlatRec r = to_flat_rec(entries[k]);
      r.pad = mx_scales_off16<MODE>(entries[k]);
      recs.push_back(r);
    }
    return launch_flat_variant<MODE, gws::kWide32>(recs, lo, hi, stream);
  }
  if (cls == gws::kRowWarp || cls == gws::kRowCta) {
    std::vector<gws::RowRec> shared_rows, block_rows;
    for (int k = 0; k < count; ++k) {
      gws::RowRec r = to_row_rec(entries[k]);
      r.pad = mx_scales_off16<MODE>(entries[k]);
      (r.tpr_log2 == 8u ? block_rows : shared_rows).push_back(r);
    }
    const int st = launch_row_chunks<MODE, false>(shared_rows, lo, hi, stream);
    return st != GWS_OK ? st : launch_row_chunks<MODE, true>(block_rows, lo, hi, stream);
  }
  std::vector<const Entry*> squares;
  for (int k = 0; k < count; ++k) squares.push_back(&entries[k]);
  return launch_squares<MODE>(squares, step, stream);
}

// One tensor on the vector kernels (row classes) or the general kernel.  The general kernel alone also
// reads its tensor from the device table (entry `index`) in multi-tensor plans.
template <int MODE>
int launch_single(int cls, const Entry& single, unsigned grid, uint32_t lo, uint32_t hi, cudaStream_t stream) {
  switch (cls) {
    case gws::kRowWarp:
      gws::k_row_warp<MODE, false><<<grid, gws::kRowWarpThreads, 0, stream>>>(single, nullptr, 0, lo, hi);
      return check_launch("warp-per-row kernel");
    case gws::kRowCta:
      gws::k_row_cta<MODE, false><<<grid, gws::kRowCtaThreads, 0, stream>>>(single, nullptr, 0, lo, hi);
      return check_launch("block-per-row kernel");
    default:
      gws::k_general<MODE, false><<<grid, gws::kGeneralThreads, 0, stream>>>(single, nullptr, 0, lo, hi);
      return check_launch("general kernel");
  }
}
template <int MODE>
int launch_general_from_table(const Entry& none, const Entry* table, int index, unsigned grid, uint32_t lo, uint32_t hi,
                              cudaStream_t stream) {
  gws::k_general<MODE, true><<<grid, gws::kGeneralThreads, 0, stream>>>(none, table, index, lo, hi);
  return check_launch("general kernel");
}

// table == nullptr: one tensor, described by `single`; otherwise entry n_or_index of `table` (general class only).
template <int MODE>
int launch(int cls, const Entry& single, const Entry* table, int n_or_index, int64_t tiles, uint64_t step,
           cudaStream_t stream) {
  if (tiles <= 0) return GWS_OK;
  if (tiles > kMaxGrid) return GWS_ERR_LIMIT;
  if (cls == gws::kFlat) return launch_flat<MODE>(&single, 1, step, stream);   // single-tensor calls only
  if ((cls == gws::kRowWarp || cls == gws::kRowCta) && table == nullptr && n_or_index != -1)
    return launch_rows<MODE>(cls, &single, 1, step, stream);
  if (cls == gws::kGeneral && table == nullptr && square_eligible(single)) {
    const std::vector<const Entry*> one{&single};
    return launch_squares<MODE>(one, step, stream);
  }
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  const unsigned grid = static_cast<unsigned>(tiles);
  return table == nullptr ? launch_single<MODE>(cls, single, grid, lo, hi, stream)
                          : launch_general_from_table<MODE>(single, table, n_or_index, grid, lo, hi, stream);
}

// Shared checks of the single-tensor calls.  Returns 1 if there is nothing to do.
int precheck(const gws_desc* d) {
  const int st = validate_desc(d);
  if (st != GWS_OK) return st;
  return is_empty(d) ? 1 : GWS_OK;
}

struct ClassTables {
  std::vector<Entry> fwd[4], bwd[4];
};

}  // namespace

extern "C" {

int64_t gws_n_groups(const gws_desc* desc) {
  const int st = validate_desc(desc);
  if (st != GWS_OK) return st;
  return n_groups_of(desc);
}

int gws_kernel_class(const gws_desc* desc) {
  const int st = validate_desc(desc);
  if (st != GWS_OK) return st;
  return classify(desc, true);
}

int gws_group_absmax(const gws_desc* desc, const void* w, float* absmax, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (w == nullptr || absmax == nullptr) return GWS_ERR_NULL;
  if (!aligned(w, 2) || !aligned(absmax, 4)) return GWS_ERR_ALIGN;
  const int cls = classify(desc, aligned(w, 16));
  const Entry e = make_entry(desc, cls, w, nullptr, nullptr, absmax);
  return launch<gws::kAbsmax>(cls, e, nullptr, 0, tiles_of(desc, cls), desc->step, static_cast<cudaStream_t>(stream));
}

int gws_sample_fwd(const gws_desc* desc, const void* w, const float* bt, void* w_hat, float* scale_out, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (w == nullptr || bt == nullptr || w_hat == nullptr) return GWS_ERR_NULL;
  if (!aligned(w, 2) || !aligned(w_hat, 2) || !aligned(bt, 4) || !aligned(scale_out, 4)) return GWS_ERR_ALIGN;
  if (overlaps(w, span_bytes(desc), w_hat, span_bytes(desc))) return GWS_ERR_ALIAS;
  const int cls = classify(desc, aligned(w, 16) && aligned(w_hat, 16));
  const Entry e = make_entry(desc, cls, w, w_hat, bt, scale_out);
  return launch<gws::kFwd>(cls, e, nullptr, 0, tiles_of(desc, cls), desc->step, static_cast<cudaStream_t>(stream));
}

int gws_scale_from_absmax(int64_t n_groups, const float* absmax, const float* bt, float* scale, void* stream) {
  if (n_groups < 0) return GWS_ERR_SHAPE;
  if (n_groups == 0) return GWS_OK;
  if (absmax == nullptr || bt == nullptr || scale == nullptr) return GWS_ERR_NULL;
  if (!aligned(absmax, 4) || !aligned(bt, 4) || !aligned(scale, 4)) return GWS_ERR_ALIGN;
  const int64_t blocks = std::min<int64_t>((n_groups + 255) / 256, 148 * 8);
  gws::k_scale<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(absmax, bt, scale, n_groups);
  return check_launch("scale kernel");
}

int gws_sample_fwd_scaled(const gws_desc* desc, const void* w, const float* scale, void* w_hat, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (w == nullptr || scale == nullptr || w_hat == nullptr) return GWS_ERR_NULL;
  if (!aligned(w, 2) || !aligned(w_hat, 2) || !aligned(scale, 4)) return GWS_ERR_ALIGN;
  if (overlaps(w, span_bytes(desc), w_hat, span_bytes(desc))) return GWS_ERR_ALIAS;
  const int cls = classify(desc, aligned(w, 16) && aligned(w_hat, 16));
  const Entry e = make_entry(desc, cls, w, w_hat, nullptr, const_cast<float*>(scale));   // this mode only reads it
  return launch<gws::kFwdScaled>(cls, e, nullptr, 0, tiles_of(desc, cls), desc->step, static_cast<cudaStream_t>(stream));
}

int gws_mx_layout(const gws_desc* desc, int format, size_t* codes_bytes, size_t* scales_offset, size_t* total_bytes) {
  const int st = validate_desc(desc);
  if (st != GWS_OK) return st;
  if (format != GWS_MX_FP8_E4M3 && format != GWS_MX_FP6_E3M2 && format != GWS_MX_FP8_E3M4) return GWS_ERR_UNSUPPORTED;
  if (desc->cols % 32 != 0) return GWS_ERR_UNSUPPORTED;
  const int64_t n = desc->rows * desc->cols;
  if (codes_bytes) *codes_bytes = mx_codes_bytes(n, format);
  if (scales_offset) *scales_offset = mx_scales_offset(n, format);
  if (total_bytes) *total_bytes = mx_total_bytes(n, format);
  return GWS_OK;
}

int gws_mx_quantize(const gws_desc* desc, int format, const void* w_hat, void* mx_out, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (format != GWS_MX_FP8_E4M3 && format != GWS_MX_FP6_E3M2 && format != GWS_MX_FP8_E3M4) return GWS_ERR_UNSUPPORTED;
  if (w_hat == nullptr || mx_out == nullptr) return GWS_ERR_NULL;
  if (!aligned(w_hat, 2)) return GWS_ERR_ALIGN;
  if (desc->cols % 32 != 0) return GWS_ERR_UNSUPPORTED;
  if (overlaps(w_hat, span_bytes(desc), mx_out, mx_total_bytes(desc->rows * desc->cols, format))) return GWS_ERR_ALIAS;
  const int cls = classify(desc, aligned(w_hat, 16) && aligned(mx_out, 16));
  const Entry e = make_entry(desc, cls, w_hat, mx_out, nullptr, nullptr);
  if (!mx_entry_ok(cls, e)) return GWS_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (format == GWS_MX_FP8_E4M3) return launch_mx<gws::kQuantMx8>(cls, &e, 1, desc->step, s);
  if (format == GWS_MX_FP8_E3M4) return launch_mx<gws::kQuantMx8b>(cls, &e, 1, desc->step, s);
  return launch_mx<gws::kQuantMx6>(cls, &e, 1, desc->step, s);
}

int gws_sample_fwd_mx(const gws_desc* desc, int format, const void* w, const float* bt, void* mx_out, float* scale_out,
                      void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (format != GWS_MX_FP8_E4M3 && format != GWS_MX_FP6_E3M2 && format != GWS_MX_FP8_E3M4) return GWS_ERR_UNSUPPORTED;
  if (w == nullptr || bt == nullptr || mx_out == nullptr) return GWS_ERR_NULL;
  if (!aligned(w, 2) || !aligned(bt, 4) || !aligned(scale_out, 4)) return GWS_ERR_ALIGN;
  if (desc->cols % 32 != 0) return GWS_ERR_UNSUPPORTED;
  if (overlaps(w, span_bytes(desc), mx_out, mx_total_bytes(desc->rows * desc->cols, format))) return GWS_ERR_ALIAS;
  const int cls = classify(desc, aligned(w, 16) && aligned(mx_out, 16));
  const Entry e = make_entry(desc, cls, w, mx_out, bt, scale_out);
  if (!mx_entry_ok(cls, e)) return GWS_ERR_UNSUPPORTED;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (format == GWS_MX_FP8_E4M3) return launch_mx<gws::kFwdMx8>(cls, &e, 1, desc->step, s);
  if (format == GWS_MX_FP8_E3M4) return launch_mx<gws::kFwdMx8b>(cls, &e, 1, desc->step, s);
  return launch_mx<gws::kFwdMx6>(cls, &e, 1, desc->step, s);
}

int gws_sample_bwd(const gws_desc* desc, const void* grad_w_hat, const float* scale, void* grad_w, float* grad_bt,
                   void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (grad_w_hat == nullptr || scale == nullptr || grad_bt == nullptr) return GWS_ERR_NULL;
  if (!aligned(grad_w_hat, 2) || !aligned(grad_w, 2) || !aligned(scale, 4) || !aligned(grad_bt, 4)) return GWS_ERR_ALIGN;
  if (grad_w == grad_w_hat) grad_w = nullptr;  // identity: nothing to copy
  if (grad_w != nullptr && overlaps(grad_w_hat, span_bytes(desc), grad_w, span_bytes(desc))) return GWS_ERR_ALIAS;
  const int cls = classify(desc, aligned(grad_w_hat, 16) && aligned(grad_w, 16));
  const Entry e = make_entry(desc, cls, grad_w_hat, grad_w, scale, grad_bt);
  return launch<gws::kBwd>(cls, e, nullptr, 0, tiles_of(desc, cls), desc->step, static_cast<cudaStream_t>(stream));
}

int gws_noise(const gws_desc* desc, uint32_t* r_packed, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (r_packed == nullptr) return GWS_ERR_NULL;
  if (!aligned(r_packed, 4)) return GWS_ERR_ALIGN;
  const uint64_t n_elems = static_cast<uint64_t>(desc->rows * desc->cols);
  const uint64_t n_words = (n_elems + 7u) / 8u;
  const uint64_t blocks = (n_words + 255u) / 256u;
  if (blocks > static_cast<uint64_t>(kMaxGrid)) return GWS_ERR_LIMIT;
  gws::k_noise<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      r_packed, n_words, n_elems, desc->elem_offset >> 3, static_cast<uint32_t>(desc->seed),
      static_cast<uint32_t>(desc->seed >> 32), static_cast<uint32_t>(desc->step), static_cast<uint32_t>(desc->step >> 32));
  return check_launch("noise kernel");
}

int64_t gws_noise_alu_probe_words(const gws_desc* desc) {
  const int st = validate_desc(desc);
  if (st != GWS_OK) return st;
  const uint64_t n_words = (static_cast<uint64_t>(desc->rows * desc->cols) + 7u) / 8u;
  return static_cast<int64_t>((n_words + 2047u) / 2048u);
}

int gws_noise_alu_probe(const gws_desc* desc, uint32_t* sink, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (sink == nullptr) return GWS_ERR_NULL;
  if (!aligned(sink, 4)) return GWS_ERR_ALIGN;
  const uint64_t n_words = (static_cast<uint64_t>(desc->rows * desc->cols) + 7u) / 8u;
  const uint64_t blocks = (n_words + 2047u) / 2048u;
  if (blocks > static_cast<uint64_t>(kMaxGrid)) return GWS_ERR_LIMIT;
  gws::k_noise_probe<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      sink, n_words, desc->elem_offset >> 3, static_cast<uint32_t>(desc->seed), static_cast<uint32_t>(desc->seed >> 32),
      static_cast<uint32_t>(desc->step), static_cast<uint32_t>(desc->step >> 32));
  return check_launch("noise arithmetic probe");
}

// Instruction mixes of gws_issue_probe: {multiplies 32x32->64, XORs fed by them, other three-input logic operations,
// FP32 FMAs, mixed-precision FMAs, integer additions, byte permutes} per step of one chain.
static const int32_t kIssueMixes[][7] = {
    {2, 2, 0, 0, 0, 0, 0},  //  0  one Philox round
    {2, 2, 1, 0, 0, 0, 0},  //  1  ... + 1 logic operation
    {2, 2, 2, 0, 0, 0, 0},  //  2
    {2, 2, 4, 0, 0, 0, 0},  //  3
    {2, 2, 0, 1, 0, 0, 0},  //  4  ... + 1 FP32 FMA
    {2, 2, 0, 2, 0, 0, 0},  //  5
    {2, 2, 0, 4, 0, 0, 0},  //  6
    {2, 2, 0, 0, 1, 0, 0},  //  7  ... + 1 mixed-precision FMA
    {2, 2, 0, 0, 2, 0, 0},  //  8
    {2, 2, 0, 0, 0, 2, 0},  //  9  ... + 2 integer additions
    {0, 0, 1, 0, 0, 0, 0},  // 10  logic alone
    {0, 0, 0, 1, 0, 0, 0},  // 11  FP32 FMA alone
    {0, 0, 0, 0, 1, 0, 0},  // 12  mixed-precision FMA alone
    {0, 0, 0, 0, 0, 1, 0},  // 13  integer addition alone
    {0, 0, 0, 0, 0, 0, 1},  // 14  byte permute alone
    {0, 0, 1, 1, 0, 0, 0},  // 15  logic + FP32 FMA
    {0, 0, 1, 0, 1, 0, 0},  // 16  logic + mixed-precision FMA
    {1, 1, 0, 0, 0, 0, 0},  // 17  half a round
    {1, 1, 1, 0, 0, 0, 0},  // 18
    {1, 1, 2, 0, 0, 0, 0},  // 19
};
constexpr int kIssueMixCount = static_cast<int>(sizeof(kIssueMixes) / sizeof(kIssueMixes[0]));
constexpr int kBodyProbeBase = 100;   // mix = 100 + pieces: the arithmetic of a pass without its memory traffic

int gws_issue_probe_mix(int mix, int32_t* counts7) {
  if (counts7 == nullptr) return GWS_ERR_NULL;
  if (mix >= 0 && mix < kIssueMixCount) {
    for (int k = 0; k < 7; ++k) counts7[k] = kIssueMixes[mix][k];
    return 32;   // steps per thread and iteration: 4 chains x 8
  }
  const int pieces = mix - kBodyProbeBase;
  if (pieces == 1 || pieces == 3 || pieces == 7 || pieces == 9) {
    for (int k = 0; k < 7; ++k) counts7[k] = 0;
    return 1;    // "iterations" counts 8-element vectors per thread
  }
  return GWS_ERR_UNSUPPORTED;
}

int gws_issue_probe(int mix, int iterations, uint32_t* sink, int32_t* host_info2, void* stream) {
  int32_t counts[7];
  const int steps = gws_issue_probe_mix(mix, counts);
  if (steps < 0) return steps;
  if (iterations <= 0 || iterations > (1 << 20)) return GWS_ERR_SHAPE;
  if (sink == nullptr || host_info2 == nullptr) return GWS_ERR_NULL;
  if (!aligned(sink, 4)) return GWS_ERR_ALIGN;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err == cudaSuccess) err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return cuda_fail(err, "device query");
  const unsigned blocks = static_cast<unsigned>(sms) * 8u;   // 2048 threads per SM: 16 warps on every sub-partition
  host_info2[0] = static_cast<int32_t>(blocks);
  host_info2[1] = sms;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint32_t k0 = 0x1234567u, k1 = 0x89ABCDEFu;
  const float f0 = 1.0001f;
#define GWS_ISSUE_CASE(ID, NW, K, F, B, I, P) \
  case ID: gws::k_issue_probe<NW, K, F, B, I, P><<<blocks, 256, 0, s>>>(sink, k0, k1, f0, iterations); break;
  if (mix < kBodyProbeBase) {
    switch (mix) {
      GWS_ISSUE_CASE(0, 2, 0, 0, 0, 0, 0) GWS_ISSUE_CASE(1, 2, 1, 0, 0, 0, 0) GWS_ISSUE_CASE(2, 2, 2, 0, 0, 0, 0)
      GWS_ISSUE_CASE(3, 2, 4, 0, 0, 0, 0) GWS_ISSUE_CASE(4, 2, 0, 1, 0, 0, 0) GWS_ISSUE_CASE(5, 2, 0, 2, 0, 0, 0)
      GWS_ISSUE_CASE(6, 2, 0, 4, 0, 0, 0) GWS_ISSUE_CASE(7, 2, 0, 0, 1, 0, 0) GWS_ISSUE_CASE(8, 2, 0, 0, 2, 0, 0)
      GWS_ISSUE_CASE(9, 2, 0, 0, 0, 2, 0) GWS_ISSUE_CASE(10, 0, 1, 0, 0, 0, 0) GWS_ISSUE_CASE(11, 0, 0, 1, 0, 0, 0)
      GWS_ISSUE_CASE(12, 0, 0, 0, 1, 0, 0) GWS_ISSUE_CASE(13, 0, 0, 0, 0, 1, 0) GWS_ISSUE_CASE(14, 0, 0, 0, 0, 0, 1)
      GWS_ISSUE_CASE(15, 0, 1, 1, 0, 0, 0) GWS_ISSUE_CASE(16, 0, 1, 0, 1, 0, 0) GWS_ISSUE_CASE(17, 1, 0, 0, 0, 0, 0)
      GWS_ISSUE_CASE(18, 1, 1, 0, 0, 0, 0) GWS_ISSUE_CASE(19, 1, 2, 0, 0, 0, 0)
      default: return GWS_ERR_UNSUPPORTED;
    }
  } else {
    if (iterations % 4 != 0) return GWS_ERR_SHAPE;
    const gws::PhiloxPre pre = gws::philox_pre(0u, 3u, 0u, k0, k1);
    switch (mix - kBodyProbeBase) {
      case 1: gws::k_body_probe<1><<<blocks, 256, 0, s>>>(sink, k0, k1, pre, 0x3C003C00u, iterations); break;
      case 3: gws::k_body_probe<3><<<blocks, 256, 0, s>>>(sink, k0, k1, pre, 0x3C003C00u, iterations); break;
      case 7: gws::k_body_probe<7><<<blocks, 256, 0, s>>>(sink, k0, k1, pre, 0x3C003C00u, iterations); break;
      case 9: gws::k_body_probe<9><<<blocks, 256, 0, s>>>(sink, k0, k1, pre, 0x3C003C00u, iterations); break;
      default: return GWS_ERR_UNSUPPORTED;
    }
  }
#undef GWS_ISSUE_CASE
  return check_launch("issue probe");
}

// ---- comparison noises (not part of the sampling pass: timed beside it) -----------------------------------------

// Shapes the comparison kernels take: dense tensors, groups of 32, 64, 128 or 256 contiguous elements that divide the row,
// 32-byte aligned pointers, and counters that do not cross a multiple of 2^32 inside the tensor.
static int compare_counters(const gws_desc* d, int kind, uint32_t* ctr_lo, gws::PhiloxPre* pre) {
  const int shift = kind == gws::kNoiseUniformBf16 ? 3 : 2;
  const uint64_t n = static_cast<uint64_t>(d->rows) * static_cast<uint64_t>(d->cols);
  const uint64_t first = d->elem_offset >> shift, last = (d->elem_offset + n - 1u) >> shift;
  if ((first >> 32) != (last >> 32) || n > 0xFFFFFFFFull) return GWS_ERR_UNSUPPORTED;
  *ctr_lo = static_cast<uint32_t>(first);
  *pre = gws::philox_pre(static_cast<uint32_t>(first >> 32), static_cast<uint32_t>(d->step), static_cast<uint32_t>(d->step >> 32),
                         static_cast<uint32_t>(d->seed), static_cast<uint32_t>(d->seed >> 32));
  return GWS_OK;
}

int gws_sample_fwd_compare(const gws_desc* desc, int noise_kind, const void* w, const float* bt, void* w_hat, float* scale_out,
                           void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (noise_kind != gws::kNoiseUniformBf16 && noise_kind != gws::kNoiseBoxMuller) return GWS_ERR_UNSUPPORTED;
  if (w == nullptr || bt == nullptr || w_hat == nullptr) return GWS_ERR_NULL;
  if (!aligned(w, 2) || !aligned(w_hat, 2) || !aligned(bt, 4) || !aligned(scale_out, 4)) return GWS_ERR_ALIGN;
  if (overlaps(w, span_bytes(desc), w_hat, span_bytes(desc))) return GWS_ERR_ALIAS;
  const int64_t gc = resolved_group_cols(desc);
  if (desc->group_rows != 1 || desc->ld != desc->cols || (gc != 32 && gc != 64 && gc != 128 && gc != 256) || desc->cols % gc != 0 ||
      desc->elem_offset % 32 != 0 || !aligned(w, 32) || !aligned(w_hat, 32))
    return GWS_ERR_UNSUPPORTED;
  gws::CompareArgs a;
  std::memset(&a, 0, sizeof a);
  const int cst = compare_counters(desc, noise_kind, &a.ctr_lo, &a.pre);
  if (cst != GWS_OK) return cst;
  a.w = w;
  a.bt = bt;
  a.w_hat = w_hat;
  a.scale_out = scale_out;
  a.n_chunks = static_cast<uint32_t>(desc->rows * desc->cols / 32);
  a.lanes_log2 = gc == 32 ? 0u : (gc == 64 ? 1u : (gc == 128 ? 2u : 3u));
  a.k0 = static_cast<uint32_t>(desc->seed);
  a.k1 = static_cast<uint32_t>(desc->seed >> 32);
  const unsigned blocks = (a.n_chunks + 2u * gws::kFlatThreads - 1u) / (2u * gws::kFlatThreads);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (noise_kind == gws::kNoiseUniformBf16) gws::k_compare_fwd<gws::kNoiseUniformBf16><<<blocks, gws::kFlatThreads, 0, s>>>(a);
  else gws::k_compare_fwd<gws::kNoiseBoxMuller><<<blocks, gws::kFlatThreads, 0, s>>>(a);
  return check_launch("comparison forward kernel");
}

int gws_noise_compare(const gws_desc* desc, int noise_kind, void* out, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (noise_kind != gws::kNoiseUniformBf16 && noise_kind != gws::kNoiseBoxMuller) return GWS_ERR_UNSUPPORTED;
  if (out == nullptr) return GWS_ERR_NULL;
  if (!aligned(out, 16)) return GWS_ERR_ALIGN;
  const uint64_t n = static_cast<uint64_t>(desc->rows) * static_cast<uint64_t>(desc->cols);
  if (n % 8 != 0 || desc->elem_offset % 8 != 0) return GWS_ERR_UNSUPPORTED;
  uint32_t ctr_lo;
  gws::PhiloxPre pre;
  const int cst = compare_counters(desc, noise_kind, &ctr_lo, &pre);
  if (cst != GWS_OK) return cst;
  const uint32_t n_vec = static_cast<uint32_t>(n / 8);
  const unsigned blocks = (n_vec + 255u) / 256u;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const uint32_t k0 = static_cast<uint32_t>(desc->seed), k1 = static_cast<uint32_t>(desc->seed >> 32);
  if (noise_kind == gws::kNoiseUniformBf16) gws::k_compare_noise<gws::kNoiseUniformBf16><<<blocks, 256, 0, s>>>(out, n_vec, ctr_lo, k0, k1, pre);
  else gws::k_compare_noise<gws::kNoiseBoxMuller><<<blocks, 256, 0, s>>>(out, n_vec, ctr_lo, k0, k1, pre);
  return check_launch("comparison noise kernel");
}

int gws_philox_words(uint64_t seed, uint64_t step, uint64_t first_vec, int64_t n_vec, uint32_t* out4, void* stream) {
  if (n_vec < 0) return GWS_ERR_SHAPE;
  if (n_vec == 0) return GWS_OK;
  if (out4 == nullptr) return GWS_ERR_NULL;
  if (!aligned(out4, 16)) return GWS_ERR_ALIGN;
  const uint64_t blocks = (static_cast<uint64_t>(n_vec) + 255u) / 256u;
  if (blocks > static_cast<uint64_t>(kMaxGrid)) return GWS_ERR_LIMIT;
  gws::k_philox_words<<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<uint4*>(out4), static_cast<uint64_t>(n_vec), first_vec, static_cast<uint32_t>(seed),
      static_cast<uint32_t>(seed >> 32), static_cast<uint32_t>(step), static_cast<uint32_t>(step >> 32));
  return check_launch("philox words kernel");
}

// ---- many tensors -------------------------------------------------------------------------------

size_t gws_workspace_bytes(int n_tensors) {
  if (n_tensors < 0) return 0;
  // two tables (forward, backward) of at most n entries, each of the 8 class tables 256-byte aligned
  return static_cast<size_t>(n_tensors) * 2u * sizeof(Entry) + 8u * 256u;
}

// Builds the table image (all class tables, forward then backward, each 256-byte aligned) in host
// memory and fills the plan.  `workspace` is only recorded, never dereferenced.
static int build_tables(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, void* workspace, size_t workspace_bytes,
                        gws_multi_plan* plan_out, std::vector<char>& image) {
  if (n < 0) return GWS_ERR_SHAPE;
  if (descs == nullptr || ptrs == nullptr || plan_out == nullptr) return GWS_ERR_NULL;
  const bool has_fwd = ptrs->w != nullptr;
  const bool has_bwd = ptrs->grad_w_hat != nullptr;
  if (!has_fwd && !has_bwd) return GWS_ERR_NULL;
  // a plan with MX outputs may come without bit-widths: it then serves gws_mx_quantize_multi only
  if (has_fwd && (ptrs->w_hat == nullptr || (ptrs->bt == nullptr && ptrs->w_hat_kind == 0))) return GWS_ERR_NULL;
  if (has_bwd && (ptrs->scale == nullptr || ptrs->grad_bt == nullptr)) return GWS_ERR_NULL;
  if (workspace == nullptr || !aligned(workspace, 256) || workspace_bytes < gws_workspace_bytes(n)) return GWS_ERR_WORKSPACE;
  const int kind = ptrs->w_hat_kind;
  if (kind < 0 || kind > 1 + GWS_MX_FP8_E3M4) return GWS_ERR_UNSUPPORTED;
  if (kind != 0 && !has_fwd) return GWS_ERR_NULL;

  ClassTables t;
  int64_t total = 0;
  for (int i = 0; i < n; ++i) {
    const gws_desc* d = &descs[i];
    const int st = validate_desc(d);
    if (st != GWS_OK) return st;
    if (is_empty(d)) continue;
    bool vec_ok = true;
    float* scale = ptrs->scale ? ptrs->scale[i] : nullptr;
    if (has_fwd) {
      const void* w = ptrs->w[i];
      void* w_hat = ptrs->w_hat[i];
      const float* bt = ptrs->bt ? ptrs->bt[i] : nullptr;
      if (w == nullptr || w_hat == nullptr || (bt == nullptr && ptrs->bt != nullptr)) return GWS_ERR_NULL;
      if (!aligned(w, 2) || !aligned(w_hat, 2) || !aligned(bt, 4) || !aligned(scale, 4)) return GWS_ERR_ALIGN;
      if (kind != 0 && d->cols % 32 != 0) return GWS_ERR_UNSUPPORTED;
      const size_t out_bytes = kind == 0 ? span_bytes(d) : mx_total_bytes(d->rows * d->cols, kind - 1);
      if (overlaps(w, span_bytes(d), w_hat, out_bytes)) return GWS_ERR_ALIAS;
      vec_ok = vec_ok && aligned(w, 16) && aligned(w_hat, 16);
    }
    void* gw = nullptr;
    if (has_bwd) {
      const void* g = ptrs->grad_w_hat[i];
      gw = ptrs->grad_w ? ptrs->grad_w[i] : nullptr;
      float* gbt = ptrs->grad_bt[i];
      if (g == nullptr || scale == nullptr || gbt == nullptr) return GWS_ERR_NULL;
      if (!aligned(g, 2) || !aligned(gw, 2) || !aligned(scale, 4) || !aligned(gbt, 4)) return GWS_ERR_ALIGN;
      if (gw == g) gw = nullptr;
      if (gw != nullptr && overlaps(g, span_bytes(d), gw, span_bytes(d))) return GWS_ERR_ALIAS;
      vec_ok = vec_ok && aligned(g, 16) && aligned(gw, 16);
    }
    const int cls = classify(d, vec_ok);
    const int64_t tiles = tiles_of(d, cls);
    total += d->rows * d->cols;
    if (has_fwd) {
      Entry e = make_entry(d, cls, ptrs->w[i], ptrs->w_hat[i], ptrs->bt ? ptrs->bt[i] : nullptr, scale);
      e.tile_begin = tiles;  // turned into a prefix sum below
      t.fwd[cls].push_back(e);
    }
    if (has_bwd) {
      Entry e = make_entry(d, cls, ptrs->grad_w_hat[i], gw, scale, ptrs->grad_bt[i]);
      e.tile_begin = tiles;
      t.bwd[cls].push_back(e);
    }
  }

  gws_multi_plan plan;
  std::memset(&plan, 0, sizeof plan);
  plan.workspace = workspace;
  plan.n_tensors = n;
  plan.has_fwd = has_fwd ? 1 : 0;
  plan.has_bwd = has_bwd ? 1 : 0;
  plan.total_elements = total;
  plan.w_hat_kind = kind;
  image.clear();
  auto place = [&](std::vector<Entry>& v, int cls, int64_t* where) -> int {
    int64_t running = 0;
    for (Entry& e : v) {
      const int64_t tiles = e.tile_begin;
      e.tile_begin = running;
      running += tiles;
    }
    if (cls != gws::kGeneral && running > kMaxGrid) return GWS_ERR_LIMIT;
    plan.count[cls] = static_cast<int32_t>(v.size());
    plan.tiles[cls] = running;
    *where = static_cast<int64_t>(image.size());
    const size_t bytes = v.size() * sizeof(Entry);
    const size_t padded = (bytes + 255u) & ~static_cast<size_t>(255u);
    image.resize(image.size() + padded, 0);
    if (bytes) std::memcpy(image.data() + *where, v.data(), bytes);
    return GWS_OK;
  };
  for (int cls = 0; cls < 4; ++cls) {
    int st = GWS_OK;
    if (has_fwd) st = place(t.fwd[cls], cls, &plan.fwd_offset[cls]);
    if (st != GWS_OK) return st;
    if (has_bwd) st = place(t.bwd[cls], cls, &plan.bwd_offset[cls]);
    if (st != GWS_OK) return st;
  }
  if (image.size() > workspace_bytes) return GWS_ERR_WORKSPACE;
  *plan_out = plan;
  return GWS_OK;
}

int gws_multi_prepare(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, void* workspace, size_t workspace_bytes,
                      void* host_workspace, size_t host_workspace_bytes, gws_multi_plan* plan_out, void* stream) {
  if (host_workspace == nullptr || host_workspace_bytes < gws_workspace_bytes(n)) return GWS_ERR_WORKSPACE;
  std::vector<char> image;
  gws_multi_plan plan;
  const int st = build_tables(n, descs, ptrs, workspace, workspace_bytes, &plan, image);
  if (st != GWS_OK) return st;
  if (!image.empty()) {
    // The host copy stays with the plan: flat-group launches pass their records by value from it.
    std::memcpy(host_workspace, image.data(), image.size());
    cudaError_t err = cudaMemcpyAsync(workspace, host_workspace, image.size(), cudaMemcpyHostToDevice,
                                      static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return cuda_fail(err, "table upload");
    // The caller may reuse the stream at once and the host copy may be pageable: wait for the upload.
    err = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (err != cudaSuccess) return cuda_fail(err, "table upload");
  }
  plan.host_tables = host_workspace;
  *plan_out = plan;
  return GWS_OK;
}

int64_t gws_multi_table_image(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, void* workspace,
                              size_t workspace_bytes, gws_multi_plan* plan_out, void* host_image, size_t host_image_bytes) {
  std::vector<char> image;
  const int st = build_tables(n, descs, ptrs, workspace, workspace_bytes, plan_out, image);
  if (st != GWS_OK) return st;
  if (host_image != nullptr) {
    if (host_image_bytes < image.size()) return GWS_ERR_WORKSPACE;
    std::memcpy(host_image, image.data(), image.size());
  }
  return static_cast<int64_t>(image.size());
}

}  // extern "C" (a template cannot have C linkage)

// One pass over the tensors of a plan.  MODE kFwd and kFwdScaled read the forward tables, kBwd the backward ones.
template <int MODE>
static int run_multi(const gws_multi_plan* plan, uint64_t step, void* stream) {
  constexpr bool backward = MODE == gws::kBwd;
  if (plan == nullptr) return GWS_ERR_NULL;
  if (plan->workspace == nullptr || plan->host_tables == nullptr) return GWS_ERR_WORKSPACE;
  if (backward ? !plan->has_bwd : !plan->has_fwd) return GWS_ERR_NULL;
  if (!backward && plan->w_hat_kind != 0) return GWS_ERR_UNSUPPORTED;   // the outputs are MX buffers: too small for BF16
  const Entry none{};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  auto host_table = [&](int cls) {
    return reinterpret_cast<const Entry*>(static_cast<const char*>(plan->host_tables) +
                                          (backward ? plan->bwd_offset[cls] : plan->fwd_offset[cls]));
  };
  if (MODE == gws::kFwdScaled)   // every tensor must come with its scale array
    for (int cls = 0; cls < 4; ++cls)
      for (int i = 0; i < plan->count[cls]; ++i)
        if (host_table(cls)[i].gout == nullptr) return GWS_ERR_NULL;
  for (int cls = 0; cls < 4; ++cls) {
    const int count = plan->count[cls];
    if (count == 0) continue;
    const Entry* table = reinterpret_cast<const Entry*>(static_cast<const char*>(plan->workspace) +
                                                        (backward ? plan->bwd_offset[cls] : plan->fwd_offset[cls]));
    const Entry* host = host_table(cls);
    if (cls == gws::kFlat) {
      const int st = launch_flat<MODE>(host, count, step, s);
      if (st != GWS_OK) return st;
    } else if (cls != gws::kGeneral) {
      const int st = launch_rows<MODE>(cls, host, count, step, s);
      if (st != GWS_OK) return st;
    } else {
      // whole 32 x 32 blocks share launches of the square-block kernel; every other shape: one launch per tensor
      std::vector<const Entry*> squares;
      for (int i = 0; i < count; ++i) {
        if (square_eligible(host[i])) { squares.push_back(&host[i]); continue; }
        const int st = launch<MODE>(cls, none, table, i, kGeneralGrid, step, s);
        if (st != GWS_OK) return st;
      }
      const int st = launch_squares<MODE>(squares, step, s);
      if (st != GWS_OK) return st;
    }
  }
  return GWS_OK;
}

// Forward pass of a plan with MX output: the w_hat pointers the plan was prepared with are MX buffers.
template <int MODE>
static int run_multi_mx(const gws_multi_plan* plan, uint64_t step, void* stream) {
  if (plan == nullptr) return GWS_ERR_NULL;
  if (plan->workspace == nullptr || plan->host_tables == nullptr) return GWS_ERR_WORKSPACE;
  if (!plan->has_fwd) return GWS_ERR_NULL;
  if (plan->w_hat_kind != 1 + gws::mode_mx_format(MODE)) return GWS_ERR_UNSUPPORTED;
  auto host_table = [&](int cls) {
    return reinterpret_cast<const Entry*>(static_cast<const char*>(plan->host_tables) + plan->fwd_offset[cls]);
  };
  for (int cls = 0; cls < 4; ++cls)
    for (int i = 0; i < plan->count[cls]; ++i) {
      if (!mx_entry_ok(cls, host_table(cls)[i])) return GWS_ERR_UNSUPPORTED;
      if (gws::mode_is_mx_fwd(MODE) && host_table(cls)[i].gin == nullptr) return GWS_ERR_NULL;   // sampling needs the bit-widths
    }
  for (int cls = 0; cls < 4; ++cls) {
    if (plan->count[cls] == 0) continue;
    const int st = launch_mx<MODE>(cls, host_table(cls), plan->count[cls], step, static_cast<cudaStream_t>(stream));
    if (st != GWS_OK) return st;
  }
  return GWS_OK;
}

extern "C" {

int gws_sample_fwd_mx_multi(const gws_multi_plan* plan, int format, uint64_t step, void* stream) {
  if (format == GWS_MX_FP8_E4M3) return run_multi_mx<gws::kFwdMx8>(plan, step, stream);
  if (format == GWS_MX_FP6_E3M2) return run_multi_mx<gws::kFwdMx6>(plan, step, stream);
  if (format == GWS_MX_FP8_E3M4) return run_multi_mx<gws::kFwdMx8b>(plan, step, stream);
  return GWS_ERR_UNSUPPORTED;
}

int gws_mx_quantize_multi(const gws_multi_plan* plan, int format, void* stream) {
  if (format == GWS_MX_FP8_E4M3) return run_multi_mx<gws::kQuantMx8>(plan, 0, stream);
  if (format == GWS_MX_FP6_E3M2) return run_multi_mx<gws::kQuantMx6>(plan, 0, stream);
  if (format == GWS_MX_FP8_E3M4) return run_multi_mx<gws::kQuantMx8b>(plan, 0, stream);
  return GWS_ERR_UNSUPPORTED;
}

int gws_multi_launch_count(const gws_multi_plan* plan, int backward) {
  if (plan == nullptr) return GWS_ERR_NULL;
  if (plan->host_tables == nullptr) return GWS_ERR_WORKSPACE;
  if (backward ? !plan->has_bwd : !plan->has_fwd) return 0;
  auto host = [&](int cls) {
    return reinterpret_cast<const Entry*>(static_cast<const char*>(plan->host_tables) +
                                          (backward ? plan->bwd_offset[cls] : plan->fwd_offset[cls]));
  };
  auto batches = [](int count, int cap) { return (count + cap - 1) / cap; };
  int wide = 0, narrow = 0, single = 0, rows[2][5] = {{0}};
  for (int k = 0; k < plan->count[0]; ++k) (host(0)[k].lanes_log2 < 2u ? narrow : wide) += 1;
  for (int cls = 1; cls <= 2; ++cls)
    for (int k = 0; k < plan->count[cls]; ++k) {
      if (!row_chunk_eligible(host(cls)[k])) { ++single; continue; }
      const gws::RowRec r = to_row_rec(host(cls)[k]);
      rows[r.tpr_log2 == 8u ? 1 : 0][row_cpt_class(r)] += 1;
    }
  int squares = 0;
  for (int k = 0; k < plan->count[3]; ++k) squares += square_eligible(host(3)[k]) ? 1 : 0;
  int total = batches(wide, gws::kFlatCapLarge) + batches(narrow, gws::kFlatCapLarge) + single + (plan->count[3] - squares) +
              batches(squares, gws::kFlatCapLarge);
  for (int blk = 0; blk < 2; ++blk)
    for (int c = 1; c <= 4; ++c) total += batches(rows[blk][c], gws::kRowCapLarge);
  return total;
}

int gws_sample_fwd_multi(const gws_multi_plan* plan, uint64_t step, void* stream) {
  return run_multi<gws::kFwd>(plan, step, stream);
}

int gws_sample_bwd_multi(const gws_multi_plan* plan, uint64_t step, void* stream) {
  return run_multi<gws::kBwd>(plan, step, stream);
}

int gws_sample_fwd_scaled_multi(const gws_multi_plan* plan, uint64_t step, void* stream) {
  return run_multi<gws::kFwdScaled>(plan, step, stream);
}

int gws_multi_locate_probe(const gws_multi_plan* plan, int backward, int kernel_class, const int64_t* tiles, int n_tiles,
                           uint64_t* out, void* stream) {
  if (plan == nullptr || tiles == nullptr || out == nullptr) return GWS_ERR_NULL;
  if (kernel_class < 1 || kernel_class > 2 || n_tiles < 0) return GWS_ERR_SHAPE;   // flat groups carry no device table
  if (plan->workspace == nullptr) return GWS_ERR_WORKSPACE;
  if (n_tiles == 0 || plan->count[kernel_class] == 0) return GWS_OK;
  const Entry* table = reinterpret_cast<const Entry*>(
      static_cast<const char*>(plan->workspace) + (backward ? plan->bwd_offset[kernel_class] : plan->fwd_offset[kernel_class]));
  gws::k_locate_probe<<<(n_tiles + 127) / 128, 128, 0, static_cast<cudaStream_t>(stream)>>>(
      table, plan->count[kernel_class], tiles, n_tiles, out);
  return check_launch("locate probe");
}

// ---- self-checking build ----------------------------------------------------------------------------

int gws_selfcheck_enabled(void) {
#ifdef GWS_SELF_CHECK
  return 1;
#else
  return 0;
#endif
}

int gws_selfcheck_set_window(const void* base, size_t bytes) {
#ifdef GWS_SELF_CHECK
  gws::CheckState st;
  std::memset(&st, 0, sizeof st);
  st.lo = reinterpret_cast<unsigned long long>(base);
  st.hi = st.lo + bytes;
  const cudaError_t err = cudaMemcpyToSymbol(gws::g_check, &st, sizeof st);
  return err == cudaSuccess ? GWS_OK : cuda_fail(err, "self-check window");
#else
  (void)base; (void)bytes;
  return GWS_ERR_UNSUPPORTED;
#endif
}

int gws_selfcheck_report(uint64_t* out5) {
#ifdef GWS_SELF_CHECK
  if (out5 == nullptr) return GWS_ERR_NULL;
  gws::CheckState st;
  const cudaError_t err = cudaMemcpyFromSymbol(&st, gws::g_check, sizeof st);
  if (err != cudaSuccess) return cuda_fail(err, "self-check report");
  out5[0] = st.violations;
  for (int k = 0; k < 4; ++k) out5[1 + k] = st.first[k];
  return GWS_OK;
#else
  (void)out5;
  return GWS_ERR_UNSUPPORTED;
#endif
}

// ---- host-buffer step ---------------------------------------------------------------------------

int gws_sample_step_host(const gws_desc* desc, const void* h_w, const float* h_bt, const void* h_grad_w_hat,
                         void* h_w_hat, float* h_scale, float* h_grad_bt, void* d_w, void* d_w_hat, void* d_grad,
                         float* d_bt, float* d_scale, float* d_grad_bt, void* stream) {
  const int st = precheck(desc);
  if (st != GWS_OK) return st < 0 ? st : GWS_OK;
  if (!h_w || !h_bt || !h_grad_w_hat || !h_w_hat || !h_scale || !h_grad_bt || !d_w || !d_w_hat || !d_grad || !d_bt ||
      !d_scale || !d_grad_bt)
    return GWS_ERR_NULL;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const size_t tb = span_bytes(desc), gb = static_cast<size_t>(n_groups_of(desc)) * sizeof(float);
  cudaError_t err;
  if ((err = cudaMemcpyAsync(d_w, h_w, tb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(err, "copy w");
  if ((err = cudaMemcpyAsync(d_bt, h_bt, gb, cudaMemcpyHostToDevice, s)) != cudaSuccess) return cuda_fail(err, "copy bt");
  if ((err = cudaMemcpyAsync(d_grad, h_grad_w_hat, tb, cudaMemcpyHostToDevice, s)) != cudaSuccess)
    return cuda_fail(err, "copy grad");
  int r = gws_sample_fwd(desc, d_w, d_bt, d_w_hat, d_scale, stream);
  if (r != GWS_OK) return r;
  r = gws_sample_bwd(desc, d_grad, d_scale, nullptr, d_grad_bt, stream);
  if (r != GWS_OK) return r;
  if ((err = cudaMemcpyAsync(h_w_hat, d_w_hat, tb, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
    return cuda_fail(err, "copy w_hat");
  if ((err = cudaMemcpyAsync(h_scale, d_scale, gb, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
    return cuda_fail(err, "copy scale");
  if ((err = cudaMemcpyAsync(h_grad_bt, d_grad_bt, gb, cudaMemcpyDeviceToHost, s)) != cudaSuccess)
    return cuda_fail(err, "copy grad_bt");
  return GWS_OK;
}

// ---- forward over many tensors without any device allocation ----------------------------------------
//
// The multi-tensor kernels read a table of tensor records from global memory.  Everywhere else that
// table sits in a workspace the caller allocated; here it sits in a fixed array that is part of the
// library image, so a caller that has no way to obtain device memory can still use one launch per
// kernel class.  The array exists once per GPU that loads the library and is shared by every call.

constexpr int kStaticMaxTensors = GWS_STATIC_MAX_TENSORS;
constexpr size_t kStaticTableBytes = static_cast<size_t>(kStaticMaxTensors) * 2u * sizeof(Entry) + 8u * 256u;
static __device__ __align__(256) unsigned char g_static_tables[kStaticTableBytes];

// In host code `g_static_tables` is only a handle for the runtime, not an address a kernel can use: the
// device address is looked up once per device, with that device current, and cached here.
constexpr int kMaxDevices = 64;
static void* g_static_tables_addr[kMaxDevices];
static std::atomic<int> g_static_tables_ready[kMaxDevices];

static int static_tables_address(void** out) {
  int dev = -1;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return cuda_fail(err, "current device");
  if (dev < 0 || dev >= kMaxDevices) return GWS_ERR_LIMIT;
  if (g_static_tables_ready[dev].load(std::memory_order_acquire) == 0) {
    void* p = nullptr;
    err = cudaGetSymbolAddress(&p, g_static_tables);
    if (err != cudaSuccess) return cuda_fail(err, "address of the built-in table array");
    if (p == nullptr || !aligned(p, 256)) return GWS_ERR_WORKSPACE;
    g_static_tables_addr[dev] = p;  // every thread that gets here stores the same value
    g_static_tables_ready[dev].store(1, std::memory_order_release);
  }
  *out = g_static_tables_addr[dev];
  return GWS_OK;
}

int gws_sample_fwd_multi_static(int n, const gws_desc* descs, const gws_multi_ptrs* ptrs, uint64_t step, void* stream) {
  if (n < 0) return GWS_ERR_SHAPE;
  if (n > kStaticMaxTensors) return GWS_ERR_LIMIT;  // more tensors than the built-in table holds
  if (descs == nullptr || ptrs == nullptr) return GWS_ERR_NULL;
  if (ptrs->w == nullptr) return GWS_ERR_NULL;  // forward pointers are required
  gws_multi_ptrs fwd_only = *ptrs;              // the backward arrays are ignored
  fwd_only.grad_w_hat = nullptr;
  fwd_only.grad_w = nullptr;
  fwd_only.grad_bt = nullptr;
  if (ptrs->w_hat_kind != 0) return GWS_ERR_UNSUPPORTED;   // BF16 w_hat only; refused before anything is uploaded
  // The table upload below reads host memory that dies with this call and the launches carry this call's step and
  // pointers by value: a stream that is recording work for later replay would replay neither correctly.
  cudaStreamCaptureStatus capturing = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(static_cast<cudaStream_t>(stream), &capturing) != cudaSuccess) {
    (void)cudaGetLastError();
    return GWS_ERR_UNSUPPORTED;
  }
  if (capturing != cudaStreamCaptureStatusNone) return GWS_ERR_UNSUPPORTED;
  void* table = nullptr;
  int st = static_tables_address(&table);
  if (st != GWS_OK) return st;
  std::vector<char> image;
  gws_multi_plan plan;
  st = build_tables(n, descs, &fwd_only, table, kStaticTableBytes, &plan, image);
  if (st != GWS_OK) return st;
  if (image.empty()) return GWS_OK;
  // Overwrites whatever the previous call left in the array.  The source is pageable host memory: the
  // runtime stages it before returning, so `image` may die with this call.
  const cudaError_t err = cudaMemcpyAsync(table, image.data(), image.size(), cudaMemcpyHostToDevice,
                                          static_cast<cudaStream_t>(stream));
  if (err != cudaSuccess) return cuda_fail(err, "upload into the built-in table array");
  plan.host_tables = image.data();   // lives until the launches below have copied their parameters
  return run_multi<gws::kFwd>(&plan, step, stream);
}

// ---- bit-width parametrisation and seeds (Section 3.6) ------------------------------------------------

static unsigned elementwise_grid(int64_t n) {
  const int64_t blocks = (n + 255) / 256;
  return static_cast<unsigned>(std::min<int64_t>(blocks, 148 * 16));
}

int gws_bitwidth(int64_t n_groups, const float* bi, float b_init, float b_target, float* bt, void* stream) {
  if (n_groups < 0) return GWS_ERR_SHAPE;
  if (n_groups == 0) return GWS_OK;
  if (bi == nullptr || bt == nullptr) return GWS_ERR_NULL;
  if (!aligned(bi, 4) || !aligned(bt, 4)) return GWS_ERR_ALIGN;
  gws::k_bitwidth<<<elementwise_grid(n_groups), 256, 0, static_cast<cudaStream_t>(stream)>>>(bi, b_init - b_target, b_target, bt,
                                                                                           n_groups);
  return check_launch("bit-width kernel");
}

int gws_bitwidth_loss(int64_t m, const float* bt, float b_target, float* loss_out, void* stream) {
  if (m < 0) return GWS_ERR_SHAPE;
  if (bt == nullptr && m > 0) return GWS_ERR_NULL;
  if (loss_out == nullptr) return GWS_ERR_NULL;
  if (!aligned(bt, 4) || !aligned(loss_out, 4)) return GWS_ERR_ALIGN;
  if (m == 0) {
    const cudaError_t err = cudaMemsetAsync(loss_out, 0, sizeof(float), static_cast<cudaStream_t>(stream));
    return err == cudaSuccess ? GWS_OK : cuda_fail(err, "bit-width loss");
  }
  gws::k_bitwidth_loss<<<1, 1024, 0, static_cast<cudaStream_t>(stream)>>>(bt, b_target, loss_out, m);
  return check_launch("bit-width loss kernel");
}

int gws_bitwidth_grad(int64_t m, const float* grad_bt, const float* bt, float b_init, float b_target, double lambda,
                      float* grad_bi, void* stream) {
  if (m < 0) return GWS_ERR_SHAPE;
  if (m == 0) return GWS_OK;
  if (grad_bt == nullptr || bt == nullptr || grad_bi == nullptr) return GWS_ERR_NULL;
  if (!aligned(grad_bt, 4) || !aligned(bt, 4) || !aligned(grad_bi, 4)) return GWS_ERR_ALIGN;
  gws::k_bitwidth_grad<<<elementwise_grid(m), 256, 0, static_cast<cudaStream_t>(stream)>>>(
      grad_bt, bt, b_init - b_target, b_target, static_cast<float>(lambda / static_cast<double>(m)), grad_bi, m);
  return check_launch("bit-width gradient kernel");
}

// Shared by the two multi-layer calls: validation of every item first, then one launch per kBitwidthCap layers.
static int bitwidth_multi(int n_items, const gws_bitwidth_item* items, bool grad, void* stream) {
  if (n_items < 0) return GWS_ERR_SHAPE;
  if (n_items == 0) return GWS_OK;
  if (items == nullptr) return GWS_ERR_NULL;
  for (int k = 0; k < n_items; ++k) {
    const gws_bitwidth_item& it = items[k];
    if (it.n < 0) return GWS_ERR_SHAPE;
    if (it.n > 0x7FFFFFFFLL) return GWS_ERR_LIMIT;
    if (it.n == 0) continue;
    if (it.bt == nullptr || (grad ? (it.grad_bt == nullptr || it.grad_bi == nullptr) : it.bi == nullptr)) return GWS_ERR_NULL;
    if (!aligned(it.bt, 4) || !aligned(it.bi, 4) || !aligned(it.grad_bt, 4) || !aligned(it.grad_bi, 4)) return GWS_ERR_ALIGN;
  }
  int k = 0;
  while (k < n_items) {
    gws::BitwidthBatch b;
    std::memset(&b, 0, sizeof b);
    uint64_t blocks = 0;
    while (k < n_items && b.n < gws::kBitwidthCap) {
      const gws_bitwidth_item& it = items[k++];
      if (it.n == 0) continue;
      const uint64_t need = (static_cast<uint64_t>(it.n) + gws::kBitwidthPerBlock - 1) / gws::kBitwidthPerBlock;
      if (blocks + need > static_cast<uint64_t>(kMaxGrid)) { --k; break; }   // the next launch takes it
      gws::BitwidthRec& r = b.e[b.n++];
      r.bi = it.bi;
      r.bt = it.bt;
      r.grad_bt = it.grad_bt;
      r.grad_bi = it.grad_bi;
      r.n = static_cast<uint32_t>(it.n);
      r.block_begin = static_cast<uint32_t>(blocks);
      r.delta = it.b_init - it.b_target;
      r.b_target = it.b_target;
      r.lam_over_m = static_cast<float>(it.lambda / static_cast<double>(it.n));
      r.accumulate = it.accumulate != 0 ? 1u : 0u;
      blocks += need;
    }
    if (b.n == 0) {
      if (k < n_items && blocks == 0) return GWS_ERR_LIMIT;   // a single layer beyond the grid limit
      continue;
    }
    if (grad) gws::k_bitwidth_multi<true><<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(b);
    else gws::k_bitwidth_multi<false><<<static_cast<unsigned>(blocks), 256, 0, static_cast<cudaStream_t>(stream)>>>(b);
    const int st = check_launch("multi-layer bit-width kernel");
    if (st != GWS_OK) return st;
  }
  return GWS_OK;
}

int gws_bitwidth_multi(int n_items, const gws_bitwidth_item* items, void* stream) { return bitwidth_multi(n_items, items, false, stream); }

int gws_bitwidth_grad_multi(int n_items, const gws_bitwidth_item* items, void* stream) { return bitwidth_multi(n_items, items, true, stream); }

uint64_t gws_layer_seed(uint64_t user_seed, uint64_t layer) {
  const gws::Words4 w = gws::philox4x32_10(static_cast<uint32_t>(layer), static_cast<uint32_t>(layer >> 32), 0u, 0u,
                                           static_cast<uint32_t>(user_seed), static_cast<uint32_t>(user_seed >> 32));
  return static_cast<uint64_t>(w.o[0]) | (static_cast<uint64_t>(w.o[1]) << 32);
}

// ---- diagnostics ----------------------------------------------------------------------------------

void gws_host_decode8(const uint32_t* words4, int8_t* r8, uint32_t* packed) {
  gws::Words4 w;
  for (int k = 0; k < 4; ++k) w.o[k] = words4[k];
  uint32_t p[4];
  gws::decode8(w, p);
  for (unsigned t = 0; t < 8; ++t) r8[t] = static_cast<int8_t>(gws::r_from_pairs(p, t));
  if (packed) *packed = gws::pack_nibbles(w);
}

void gws_host_decode8_pairs(const uint32_t* words4, uint32_t* pairs4, uint32_t* pairs4_signed_zero) {
  gws::Words4 w;
  for (int k = 0; k < 4; ++k) w.o[k] = words4[k];
  uint32_t p[4], q[4];
  gws::decode8(w, p);
  gws::decode8_signed_zero(w, q);
  for (int k = 0; k < 4; ++k) {
    pairs4[k] = p[k];
    pairs4_signed_zero[k] = q[k];
  }
}

void gws_host_philox(uint64_t seed, uint64_t step, uint64_t vec, uint32_t* out4) {
  const gws::Words4 w = gws::philox_for_vector(vec, static_cast<uint32_t>(step), static_cast<uint32_t>(step >> 32),
                                               static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32));
  for (int k = 0; k < 4; ++k) out4[k] = w.o[k];
}

const char* gws_status_string(int status) {
  switch (status) {
    case GWS_OK: return "ok";
    case GWS_ERR_NULL: return "a required pointer is NULL";
    case GWS_ERR_SHAPE: return "bad shape: negative size, ld < cols, or elem_offset not a multiple of 8";
    case GWS_ERR_GROUP: return "bad group shape: group_rows < 1 or group_cols < 0";
    case GWS_ERR_ALIGN: return "pointer not aligned to its element type";
    case GWS_ERR_ALIAS: return "output overlaps an input";
    case GWS_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case GWS_ERR_CUDA: return "CUDA runtime error (see gws_last_cuda_error)";
    case GWS_ERR_LIMIT: return "size beyond a documented maximum";
    case GWS_ERR_UNSUPPORTED: return "not supported: by this build of the library, or for this shape or kind of output";
    default: return "unknown status";
  }
}

const char* gws_last_cuda_error(void) { return g_last_cuda_error.c_str(); }

uint64_t gws_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int gws_set_launch_overlap(int enable) { return g_launch_overlap.exchange(enable != 0 ? 1 : 0, std::memory_order_relaxed); }

}  // extern "C"

#include "gws_gemm.cuh"   // gws_gemm_fused: the tcgen05 GEMM with sampling in its prologue
