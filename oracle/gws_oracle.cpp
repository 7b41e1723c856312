// GaussWS sampling oracle: a plain, slow, single-threaded CPU statement of the
// weight-sampling pass of Gaussian weight sampling (Eq. 3 forward, Eq. 4
// backward, Section 3.4 noise law of Eq. 9 / Eq. 10, packed format of
// Section 3.4's last paragraph).
//
// THIS FILE IS TEST INFRASTRUCTURE.  It exists to be checked by eye against
// the paper and to check the CUDA library.  It shares no code with the CUDA
// path, nothing in the product imports it, and it is never tuned for speed.
// Only the test suite, the smoke check and the CPU-baseline leg of the
// benchmark may call it.
//
// Build: g++ -std=c++17 -O2 -ffp-contract=off -fno-fast-math -shared -fPIC
// (no FMA contraction, so every float operation below rounds exactly once).
//
// Conventions (the paper leaves them open; both sides implement this list):
//   * A tensor is row-major [rows, cols] BF16 with `ld` elements between rows.
//   * A group is group_rows x group_cols elements (group_cols == 0: the whole
//     row).  Groups are numbered row-major over the ceil(rows/group_rows) x
//     ceil(cols/group_cols) grid, the shape the paper gives b_t below Eq. 3.
//   * PRNG: Philox4x32 with 10 rounds (the paper names Philox in Section 3.4).
//     Element (i, j) has the logical index e = elem_offset + i*cols + j.  The
//     Philox counter is (lo32(e>>3), hi32(e>>3), lo32(step), hi32(step)), the
//     key is (lo32(seed), hi32(seed)).  One call serves 8 consecutive
//     elements.  Section 3.4 treats every bit of the random integers as one
//     "bitwise random variable" and combines whole integers with AND / OR, so
//     the 16 random bits of an element are 16 bit positions spread over the
//     four output words, not 16 neighbouring bits of one word: element
//     t = e & 7 (j = t >> 1, h = t & 1) owns the four bit columns c+1, c, c-7
//     and c-8 with c = 16h + 14 - 2j, in each of the four words.  Bit x_k of
//     its field is bit (c + kFieldColumn[k]) of word kFieldWord[k] (tables
//     below); the eight fields of a vector use each of the 128 bits once.
//   * Noise decode (Eq. 9 / Eq. 10), field bits x0 (LSB) .. x15:
//       m2 = x0 & x1 & ... & x7 & (x8 | x9)          Pr = 2^-8 * 3/4
//       m1 = (x10 | x11) & (x12 | x13) & x14         Pr = (3/4)^2 * 1/2
//       |R| = 2 if m2, else 1 if m1, else 0;  R = -|R| if x15 else +|R|.
//   * scale s_g = fl32(absmax_g * 2^(1 - b_g)); 2^(1-b) is computed in
//     double and rounded to float (exact for integer b).
//   * sample: y = fl32(float(w) + float(R) * s_g)  (the product is exact),
//     w_hat = BF16 round-to-nearest-even of y.  R == 0 adds +0.0f.
//   * backward: grad_w = upstream gradient unchanged; grad_b_g =
//     float(-ln 2 * s_g * sum_g(float(g) * R)), the sum taken in double in
//     row-major order inside the group.
//
// Pins (tests/test_oracle_*.py): Philox known-answer vectors; exhaustive
// decode counts against Eq. 10; closed-form moments; KS / chi-square over
// 10^7 draws; hand-computed add-then-cast cases; library BF16 casts;
// finite-difference gradients; the Lemma 1 and Proposition 2 invariants;
// the given-scale forward against the fused one and a numpy restatement, and
// the facts a sharded pass rests on (partial maxima, partial sums); the MX
// element grids against their definition, brute-force nearest-even rounding
// and a library FP8 cast, the shared exponent against its formula, and the
// transposition property of square blocks.
// The only thing left unpinned is which of the equally valid bit assignments
// the authors' own kernels used; their stream cannot be reproduced.

#include <cmath>
#include <cstdint>
#include <cstring>

namespace {

// ---- BF16 <-> FP32 by bit manipulation ------------------------------------

float bf16_to_f32(uint16_t h) {
  uint32_t u = static_cast<uint32_t>(h) << 16;
  float f;
  std::memcpy(&f, &u, sizeof f);
  return f;
}

// IEEE round-to-nearest, ties-to-even, onto the upper 16 bits of a float.
uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, sizeof u);
  const uint32_t exponent = (u >> 23) & 0xFFu;
  const uint32_t fraction = u & 0x007FFFFFu;
  if (exponent == 0xFFu && fraction != 0) {
    // NaN: keep it a NaN after truncation.
    return static_cast<uint16_t>((u >> 16) | 0x0040u);
  }
  uint32_t kept = u >> 16;            // sign, exponent, 7 fraction bits
  const uint32_t dropped = u & 0xFFFFu;  // the 16 bits that are cut off
  const uint32_t half = 0x8000u;
  if (dropped > half) {
    kept += 1;                        // above the midpoint: round away
  } else if (dropped == half) {
    if (kept & 1u) kept += 1;         // exactly the midpoint: to even
  }
  // A carry out of the fraction moves into the exponent, which is the right
  // result (next binade, or infinity at the top).
  return static_cast<uint16_t>(kept);
}

// ---- Philox4x32-10 ----------------------------------------------------------

constexpr uint32_t PHILOX_M0 = 0xD2511F53u;
constexpr uint32_t PHILOX_M1 = 0xCD9E8D57u;
constexpr uint32_t PHILOX_W0 = 0x9E3779B9u;
constexpr uint32_t PHILOX_W1 = 0xBB67AE85u;

void philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  uint32_t k0 = key[0], k1 = key[1];
  for (int round = 0; round < 10; ++round) {
    const uint64_t p0 = static_cast<uint64_t>(PHILOX_M0) * c0;
    const uint64_t p1 = static_cast<uint64_t>(PHILOX_M1) * c2;
    const uint32_t hi0 = static_cast<uint32_t>(p0 >> 32), lo0 = static_cast<uint32_t>(p0);
    const uint32_t hi1 = static_cast<uint32_t>(p1 >> 32), lo1 = static_cast<uint32_t>(p1);
    const uint32_t n0 = hi1 ^ c1 ^ k0;
    const uint32_t n1 = lo1;
    const uint32_t n2 = hi0 ^ c3 ^ k1;
    const uint32_t n3 = lo0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += PHILOX_W0;
    k1 += PHILOX_W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// The four output words for the 8-element vector number `vec`.
void philox_for_vector(uint64_t seed, uint64_t step, uint64_t vec, uint32_t out[4]) {
  const uint32_t ctr[4] = {static_cast<uint32_t>(vec), static_cast<uint32_t>(vec >> 32),
                           static_cast<uint32_t>(step), static_cast<uint32_t>(step >> 32)};
  const uint32_t key[2] = {static_cast<uint32_t>(seed), static_cast<uint32_t>(seed >> 32)};
  philox4x32_10(ctr, key, out);
}

// ---- noise decode (Eq. 9 / Eq. 10) -----------------------------------------

int decode_field(uint32_t field) {
  int x[16];
  for (int k = 0; k < 16; ++k) x[k] = static_cast<int>((field >> k) & 1u);
  int low_byte_all_ones = 1;
  for (int k = 0; k < 8; ++k) low_byte_all_ones &= x[k];
  const int m2 = low_byte_all_ones & (x[8] | x[9]);
  const int m1 = (x[10] | x[11]) & (x[12] | x[13]) & x[14];
  const int magnitude = m2 ? 2 : (m1 ? 1 : 0);
  return x[15] ? -magnitude : magnitude;
}

// Where the 16 field bits of an element come from: x_k is bit (c + column[k])
// of output word word[k], with c = 16*(t & 1) + 14 - 2*(t >> 1) for element t
// of the vector.  x0..x7 (the eight-input AND of |R| = 2) sit in the two low
// columns c-7, c-8 and in word 0 of the top column; x8, x9 (its OR) and the
// sign x15 are the rest of the top column c+1; x10..x13 (the two ORs of
// |R| = 1) are column c, x14 the remaining bit of column c-8.
constexpr int kFieldWord[16] = {0, 1, 2, 3, 1, 2, 3, 0, 1, 2, 0, 1, 2, 3, 0, 3};
constexpr int kFieldColumn[16] = {-7, -7, -7, -7, -8, -8, -8, +1, +1, +1, 0, 0, 0, 0, -8, +1};

uint32_t field_of_element(const uint32_t o[4], unsigned t) {
  const int c = 16 * static_cast<int>(t & 1u) + 14 - 2 * static_cast<int>(t >> 1);
  uint32_t field = 0;
  for (int k = 0; k < 16; ++k) field |= ((o[kFieldWord[k]] >> (c + kFieldColumn[k])) & 1u) << k;
  return field;
}

// Noise of the element with logical index e.
int noise_of_element(uint64_t seed, uint64_t step, uint64_t e) {
  uint32_t o[4];
  philox_for_vector(seed, step, e >> 3, o);
  return decode_field(field_of_element(o, static_cast<unsigned>(e & 7u)));
}

// ---- group geometry ----------------------------------------------------------

struct Geometry {
  int64_t rows, cols, ld, group_rows, group_cols, groups_per_row_band, n_groups;
};

Geometry make_geometry(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols) {
  Geometry g;
  g.rows = rows;
  g.cols = cols;
  g.ld = ld;
  g.group_rows = group_rows;
  g.group_cols = (group_cols == 0) ? cols : group_cols;
  g.groups_per_row_band = (cols + g.group_cols - 1) / g.group_cols;
  g.n_groups = ((rows + group_rows - 1) / group_rows) * g.groups_per_row_band;
  return g;
}

int64_t group_of(const Geometry& g, int64_t i, int64_t j) {
  return (i / g.group_rows) * g.groups_per_row_band + (j / g.group_cols);
}

float scale_of(float absmax, float bits) {
  const float pow2 = static_cast<float>(std::exp2(1.0 - static_cast<double>(bits)));
  return absmax * pow2;
}

}  // namespace

extern "C" {

float gwso_bf16_to_f32(uint16_t h) { return bf16_to_f32(h); }
uint16_t gwso_f32_to_bf16_rne(float f) { return f32_to_bf16_rne(f); }

void gwso_philox4x32_10(const uint32_t* ctr4, const uint32_t* key2, uint32_t* out4) {
  philox4x32_10(ctr4, key2, out4);
}

// out4 receives 4 words for each of the n_vec vectors first_vec, first_vec+1, ...
void gwso_philox_words(uint64_t seed, uint64_t step, uint64_t first_vec, int64_t n_vec, uint32_t* out4) {
  for (int64_t k = 0; k < n_vec; ++k) philox_for_vector(seed, step, first_vec + static_cast<uint64_t>(k), out4 + 4 * k);
}

int gwso_decode_field(uint32_t field16) { return decode_field(field16 & 0xFFFFu); }

// The 16-bit field of element t (0..7) of a vector whose four output words are words4.
uint32_t gwso_field_of_element(const uint32_t* words4, uint32_t t) { return field_of_element(words4, t & 7u); }

int64_t gwso_n_groups(int64_t rows, int64_t cols, int64_t group_rows, int64_t group_cols) {
  return make_geometry(rows, cols, cols, group_rows, group_cols).n_groups;
}

// R for the n elements with logical indices first_elem, first_elem+1, ...
void gwso_noise_r(uint64_t seed, uint64_t step, uint64_t first_elem, int64_t n, int8_t* r) {
  for (int64_t k = 0; k < n; ++k)
    r[k] = static_cast<int8_t>(noise_of_element(seed, step, first_elem + static_cast<uint64_t>(k)));
}

// Packed sign-magnitude nibbles, 8 elements per 32-bit word: element k of the
// run sits in word k>>3 at bits [4*(k&7), 4*(k&7)+3]; nibble = sign<<3 | |R|,
// and R == 0 is always stored as 0 (no negative zero).  first_elem must be a
// multiple of 8; a final partial word has its unused nibbles zero.
void gwso_noise_packed(uint64_t seed, uint64_t step, uint64_t first_elem, int64_t n, uint32_t* packed) {
  const int64_t n_words = (n + 7) / 8;
  for (int64_t v = 0; v < n_words; ++v) packed[v] = 0;
  for (int64_t k = 0; k < n; ++k) {
    const int r = noise_of_element(seed, step, first_elem + static_cast<uint64_t>(k));
    const uint32_t magnitude = static_cast<uint32_t>(r < 0 ? -r : r);
    const uint32_t nibble = (r < 0 ? 8u : 0u) | magnitude;
    packed[k >> 3] |= nibble << (4 * (k & 7));
  }
}

// absmax[g] = max over group g of |w| (exact: BF16 magnitudes widen to FP32 exactly).
void gwso_group_absmax(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                       const uint16_t* w, float* absmax) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  for (int64_t g = 0; g < geo.n_groups; ++g) absmax[g] = 0.0f;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const float a = std::fabs(bf16_to_f32(w[i * ld + j]));
      const int64_t g = group_of(geo, i, j);
      if (a > absmax[g]) absmax[g] = a;
    }
}

void gwso_scale(int64_t n_groups, const float* absmax, const float* bt, float* scale) {
  for (int64_t g = 0; g < n_groups; ++g) scale[g] = scale_of(absmax[g], bt[g]);
}

// Eq. 3 followed by the BF16 cast, with R supplied by the caller
// (r[i*cols + j], values in -2..2).  scale_out may be null.
void gwso_sample_fwd_injected(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                              const uint16_t* w, const float* bt, const int8_t* r, uint16_t* w_hat,
                              float* scale_out, float* absmax_scratch) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  gwso_group_absmax(rows, cols, ld, group_rows, group_cols, w, absmax_scratch);
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const int64_t g = group_of(geo, i, j);
      const float s = scale_of(absmax_scratch[g], bt[g]);
      const float pqn = static_cast<float>(r[i * cols + j]) * s;
      const float y = bf16_to_f32(w[i * ld + j]) + pqn;
      w_hat[i * ld + j] = f32_to_bf16_rne(y);
    }
  if (scale_out)
    for (int64_t g = 0; g < geo.n_groups; ++g) scale_out[g] = scale_of(absmax_scratch[g], bt[g]);
}

// Eq. 3 + cast with R drawn from the counter-based generator.
void gwso_sample_fwd(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                     uint64_t seed, uint64_t step, uint64_t elem_offset, const uint16_t* w, const float* bt,
                     uint16_t* w_hat, float* scale_out, float* absmax_scratch) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  gwso_group_absmax(rows, cols, ld, group_rows, group_cols, w, absmax_scratch);
  uint64_t cached_vec = ~static_cast<uint64_t>(0);
  uint32_t o[4] = {0, 0, 0, 0};
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const uint64_t e = elem_offset + static_cast<uint64_t>(i * cols + j);
      if ((e >> 3) != cached_vec) {  // same call as noise_of_element, made once per vector
        cached_vec = e >> 3;
        philox_for_vector(seed, step, cached_vec, o);
      }
      const int r = decode_field(field_of_element(o, static_cast<unsigned>(e & 7u)));
      const int64_t g = group_of(geo, i, j);
      const float s = scale_of(absmax_scratch[g], bt[g]);
      const float pqn = static_cast<float>(r) * s;
      const float y = bf16_to_f32(w[i * ld + j]) + pqn;
      w_hat[i * ld + j] = f32_to_bf16_rne(y);
    }
  if (scale_out)
    for (int64_t g = 0; g < geo.n_groups; ++g) scale_out[g] = scale_of(absmax_scratch[g], bt[g]);
}

// Eq. 3 + cast for a tensor whose group maxima were taken elsewhere: scale[g]
// is s_g = max_g|w| * 2^(1 - b_g) as the caller has it (for a tensor cut into
// shards the maximum runs over the whole group, parts held by other shards
// included).  Same noise, add and cast as gwso_sample_fwd; nothing is reduced.
void gwso_sample_fwd_scaled(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                            uint64_t seed, uint64_t step, uint64_t elem_offset, const uint16_t* w,
                            const float* scale, uint16_t* w_hat) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const uint64_t e = elem_offset + static_cast<uint64_t>(i * cols + j);
      const int r = noise_of_element(seed, step, e);
      const float pqn = static_cast<float>(r) * scale[group_of(geo, i, j)];
      const float y = bf16_to_f32(w[i * ld + j]) + pqn;
      w_hat[i * ld + j] = f32_to_bf16_rne(y);
    }
}

// Eq. 4 with R supplied.  grad_w (may be null) receives the upstream gradient
// unchanged; grad_bt[g] = -ln2 * scale[g] * sum_g(grad * R).
void gwso_sample_bwd_injected(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                              const uint16_t* grad_w_hat, const float* scale, const int8_t* r,
                              uint16_t* grad_w, float* grad_bt, double* acc_scratch) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  for (int64_t g = 0; g < geo.n_groups; ++g) acc_scratch[g] = 0.0;
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const uint16_t gbits = grad_w_hat[i * ld + j];
      if (grad_w) grad_w[i * ld + j] = gbits;
      acc_scratch[group_of(geo, i, j)] +=
          static_cast<double>(bf16_to_f32(gbits)) * static_cast<double>(r[i * cols + j]);
    }
  const double ln2 = 0.6931471805599453;
  for (int64_t g = 0; g < geo.n_groups; ++g)
    grad_bt[g] = static_cast<float>(-ln2 * static_cast<double>(scale[g]) * acc_scratch[g]);
}

// Eq. 4 with R regenerated from (seed, step, element index).
void gwso_sample_bwd(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                     uint64_t seed, uint64_t step, uint64_t elem_offset, const uint16_t* grad_w_hat,
                     const float* scale, uint16_t* grad_w, float* grad_bt, double* acc_scratch) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  for (int64_t g = 0; g < geo.n_groups; ++g) acc_scratch[g] = 0.0;
  uint64_t cached_vec = ~static_cast<uint64_t>(0);
  uint32_t o[4] = {0, 0, 0, 0};
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const uint64_t e = elem_offset + static_cast<uint64_t>(i * cols + j);
      if ((e >> 3) != cached_vec) {
        cached_vec = e >> 3;
        philox_for_vector(seed, step, cached_vec, o);
      }
      const int r = decode_field(field_of_element(o, static_cast<unsigned>(e & 7u)));
      const uint16_t gbits = grad_w_hat[i * ld + j];
      if (grad_w) grad_w[i * ld + j] = gbits;
      acc_scratch[group_of(geo, i, j)] += static_cast<double>(bf16_to_f32(gbits)) * static_cast<double>(r);
    }
  const double ln2 = 0.6931471805599453;
  for (int64_t g = 0; g < geo.n_groups; ++g)
    grad_bt[g] = static_cast<float>(-ln2 * static_cast<double>(scale[g]) * acc_scratch[g]);
}

// ---- w_hat in a microscaling (MX) floating-point format ------------------------------------------------
//
// Section 3.1 targets MX formats whose elements are low-precision FP (MXFP), Section 3.2 notes that a
// square block whose 32-element vectors share one scale is MX-compliant, and Table C.1 lists FP8_e4m3 and
// FP6_e3m2 as the datatypes that hold w_hat for b_t <= 5 and b_t <= 4.  The paper defines no conversion;
// this one is the conversion of the OCP Microscaling Formats (MX) specification v1.0 applied to the BF16
// w_hat, with the paper's sharing rule:
//   * the scaling block is the sampling group (Eq. 3's b_l x b_l block, or the 1 x G group): every
//     32-element row vector of a group carries the same scale, so a square block stays consistent under
//     transposition;
//   * shared exponent = floor(log2(max_group |w_hat|)) - emax_elem, clamped to the E8M0 range
//     [-127, 127]; the scale byte is that exponent + 127 (an all-zero or subnormal-only group gets 0);
//   * element = w_hat / 2^shared_exponent rounded to nearest, ties to even, onto the element grid
//     (subnormals included); magnitudes beyond the largest normal are clamped to it; the sign of zero
//     is kept.
// Element formats: E4M3 = 1 sign, 4 exponent (bias 7), 3 mantissa bits, largest normal 448 = 1.75 * 2^8
// (emax 8; the code S.1111.111 is NaN and never produced from finite input); E3M2 = 1 sign, 3 exponent
// (bias 3), 2 mantissa bits, largest normal 28 = 1.75 * 2^4 (emax 4), no NaN or infinity.  Format 2 is
// Table C.1's FP8_e3m4, which the paper names without defining and which is not an OCP element type; it is
// read by analogy with E3M2: 1 sign, 3 exponent (bias 3), 4 mantissa bits, every code finite, largest
// normal 31 = 1.9375 * 2^4 (emax 4).

struct MxElement {
  int exponent_bits, mantissa_bits, bias, emax;
  double max_normal;
};

static MxElement mx_element(int format) {
  if (format == 0) return MxElement{4, 3, 7, 8, 448.0};
  if (format == 2) return MxElement{3, 4, 3, 4, 31.0};
  return MxElement{3, 2, 3, 4, 28.0};
}

// Value of a code of the element format (sign in the top bit of the code's width).
double gwso_mx_decode(int format, uint32_t code) {
  const MxElement f = mx_element(format);
  const int width = 1 + f.exponent_bits + f.mantissa_bits;
  const uint32_t sign = (code >> (width - 1)) & 1u;
  const uint32_t e = (code >> f.mantissa_bits) & ((1u << f.exponent_bits) - 1u);
  const uint32_t m = code & ((1u << f.mantissa_bits) - 1u);
  double v;
  if (format == 0 && e == 15u && m == 7u) return std::nan("");
  if (e == 0)
    v = std::ldexp(static_cast<double>(m), 1 - f.bias - f.mantissa_bits);
  else
    v = std::ldexp(1.0 + std::ldexp(static_cast<double>(m), -f.mantissa_bits), static_cast<int>(e) - f.bias);
  return sign ? -v : v;
}

// x (finite) rounded to the element grid: nearest, ties to even, clamped to the largest normal.
uint32_t gwso_mx_encode(int format, double x) {
  const MxElement f = mx_element(format);
  const int width = 1 + f.exponent_bits + f.mantissa_bits;
  const uint32_t sign = std::signbit(x) ? 1u : 0u;
  const double a = std::fabs(x);
  uint32_t magnitude = 0;
  if (a > 0.0) {
    int e = static_cast<int>(std::floor(std::log2(a)));
    if (std::ldexp(1.0, e) > a) --e;          // guard the floating-point log at exact powers of two
    if (std::ldexp(1.0, e + 1) <= a) ++e;
    const int e_min = 1 - f.bias;             // exponent of the smallest normal; subnormals share its spacing
    const int spacing_exp = (e < e_min ? e_min : e) - f.mantissa_bits;
    const double steps = std::nearbyint(std::ldexp(a, -spacing_exp));   // default rounding mode: ties to even
    double value = std::ldexp(steps, spacing_exp);
    if (value > f.max_normal) value = f.max_normal;
    if (value < std::ldexp(1.0, e_min)) {
      magnitude = static_cast<uint32_t>(std::ldexp(value, f.bias - 1 + f.mantissa_bits));   // subnormal: exponent field 0
    } else {
      int ev = static_cast<int>(std::floor(std::log2(value)));
      if (std::ldexp(1.0, ev) > value) --ev;
      if (std::ldexp(1.0, ev + 1) <= value) ++ev;
      const double frac = std::ldexp(value, -ev) - 1.0;
      magnitude = (static_cast<uint32_t>(ev + f.bias) << f.mantissa_bits) |
                  static_cast<uint32_t>(std::ldexp(frac, f.mantissa_bits));
    }
  }
  return (sign << (width - 1)) | magnitude;
}

// codes[i*cols + j]: one element code per byte (logical order, no ld); scales[i*(cols/32) + j/32]: the
// E8M0 byte of the 32-element vector.  cols and the resolved group_cols must be multiples of 32.
void gwso_mx_emit(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols, int format,
                  const uint16_t* w_hat, uint8_t* codes, uint8_t* scales, float* absmax_scratch) {
  const MxElement f = mx_element(format);
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  gwso_group_absmax(rows, cols, ld, group_rows, group_cols, w_hat, absmax_scratch);
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const float amax = absmax_scratch[group_of(geo, i, j)];
      int shared = -127;
      if (amax > 0.0f) {
        int e2;
        std::frexp(amax, &e2);                 // amax = m * 2^e2 with m in [0.5, 1): floor(log2) = e2 - 1
        shared = (e2 - 1) - f.emax;
        if (shared < -127) shared = -127;
        if (shared > 127) shared = 127;
      }
      const double scaled = std::ldexp(static_cast<double>(bf16_to_f32(w_hat[i * ld + j])), -shared);
      codes[i * cols + j] = static_cast<uint8_t>(gwso_mx_encode(format, scaled));
      if (j % 32 == 0) scales[i * (cols / 32) + j / 32] = static_cast<uint8_t>(shared + 127);
    }
}

// Six-bit codes as a little-endian bit stream: code k occupies bits [6k, 6k + 5] of the stream, so 4
// codes fill 3 bytes and a 32-element vector 24.  n must be a multiple of 4.
void gwso_mx_pack6(int64_t n, const uint8_t* codes, uint8_t* packed) {
  for (int64_t b = 0; b < n * 3 / 4; ++b) packed[b] = 0;
  for (int64_t k = 0; k < n; ++k)
    for (int bit = 0; bit < 6; ++bit)
      if ((codes[k] >> bit) & 1u) {
        const int64_t pos = 6 * k + bit;
        packed[pos >> 3] |= static_cast<uint8_t>(1u << (pos & 7));
      }
}

// ---- bit-width parametrisation and seeds (Section 3.6) ------------------------------------------------

// Eq. 11: b_t = b_target + b_i * (b_init - b_target), in FP32 with one rounding per operation (the
// result feeds 2^(1 - b_t), so its bits matter): delta = fl(b_init - b_target), then fl(b_i * delta),
// then fl(b_target + that).
void gwso_bitwidth(int64_t n, const float* bi, float b_init, float b_target, float* bt) {
  const float delta = b_init - b_target;
  for (int64_t k = 0; k < n; ++k) {
    const float scaled = bi[k] * delta;
    bt[k] = b_target + scaled;
  }
}

// One layer's term of Eq. 12 without its lambda: the mean over the layer's m blocks of |b_t - b_target|.
double gwso_bitwidth_loss(int64_t m, const float* bt, float b_target) {
  double sum = 0.0;
  for (int64_t k = 0; k < m; ++k) sum += std::fabs(static_cast<double>(bt[k]) - static_cast<double>(b_target));
  return m > 0 ? sum / static_cast<double>(m) : 0.0;
}

// dL'/db_i for one layer: Eq. 12 adds lambda/m * sign(b_t - b_target) to dL/db_t (the derivative of |x|,
// taken as 0 at x = 0), and Eq. 11 multiplies by db_t/db_i = b_init - b_target.
void gwso_bitwidth_grad(int64_t m, const float* grad_bt, const float* bt, float b_init, float b_target, double lambda,
                        double* grad_bi) {
  const double delta = static_cast<double>(b_init) - static_cast<double>(b_target);
  for (int64_t k = 0; k < m; ++k) {
    const double x = static_cast<double>(bt[k]) - static_cast<double>(b_target);
    const double sign = x > 0.0 ? 1.0 : (x < 0.0 ? -1.0 : 0.0);
    grad_bi[k] = delta * (static_cast<double>(grad_bt[k]) + lambda / static_cast<double>(m) * sign);
  }
}

// "Managing seed": the seed generator started from the user's seed gives every layer its own seed.
// Reading: layer l gets the first 64 output bits of Philox4x32-10 with counter (lo32(l), hi32(l), 0, 0)
// and key (lo32(user_seed), hi32(user_seed)); the per-update change of the layer's PRNG state is the
// gradient-update counter `step` that goes into the sampling counter.
uint64_t gwso_layer_seed(uint64_t user_seed, uint64_t layer) {
  const uint32_t ctr[4] = {static_cast<uint32_t>(layer), static_cast<uint32_t>(layer >> 32), 0u, 0u};
  const uint32_t key[2] = {static_cast<uint32_t>(user_seed), static_cast<uint32_t>(user_seed >> 32)};
  uint32_t o[4];
  philox4x32_10(ctr, key, o);
  return static_cast<uint64_t>(o[0]) | (static_cast<uint64_t>(o[1]) << 32);
}

// ---- comparison noises (Section 4, first paragraph: "DiffQ" = this method with BF16 U(-0.5, 0.5) in place of R; Section 3.4
// and the "bm" series of the forward benchmark: R = round(N(0,1) / 2) with the normals from the Box-Muller transform) -----------

// BF16 U(-0.5, 0.5): element e takes the 16-bit field x at bits [16 (e & 1), +16) of word (e >> 1) & 3 of the Philox output
// for vector e >> 3; u = ((x + 1/2) / 2^16 - 1/2) rounded to BF16 (nearest even).  (x + 1/2) / 2^16 is the midpoint rule for
// "random integer divided by its maximum": symmetric about 0 and never exactly -1/2 before rounding.
static uint16_t uniform_bf16_of_field(uint32_t x) {
  const double u = (static_cast<double>(x & 0xFFFFu) + 0.5) / 65536.0 - 0.5;
  return f32_to_bf16_rne(static_cast<float>(u));   // u is a multiple of 2^-17 below 1 in magnitude: exact in float
}

void gwso_noise_uniform(uint64_t seed, uint64_t step, uint64_t first_elem, int64_t n, uint16_t* u_bf16) {
  for (int64_t k = 0; k < n; ++k) {
    const uint64_t e = first_elem + static_cast<uint64_t>(k);
    uint32_t o[4];
    philox_for_vector(seed, step, e >> 3, o);
    const unsigned t = static_cast<unsigned>(e & 7u);
    u_bf16[k] = uniform_bf16_of_field((o[t >> 1] >> (16u * (t & 1u))) & 0xFFFFu);
  }
}

// Box-Muller: one Philox call (counter = e >> 2 in place of the vector index) serves 4 elements; words (o0, o1) give the
// normals of elements 4c and 4c + 1, words (o2, o3) those of 4c + 2 and 4c + 3:
//   u1 = ((a >> 8) + 1) / 2^24 in (0, 1],  u2 = (b >> 8) / 2^24 in [0, 1),
//   z0 = sqrt(-2 ln u1) cos(2 pi u2),  z1 = sqrt(-2 ln u1) sin(2 pi u2).
static void box_muller_pair(uint32_t a, uint32_t b, double* z0, double* z1) {
  const double u1 = (static_cast<double>(a >> 8) + 1.0) / 16777216.0, u2 = static_cast<double>(b >> 8) / 16777216.0;
  const double radius = std::sqrt(-2.0 * std::log(u1)), angle = 6.283185307179586476925286766559 * u2;
  *z0 = radius * std::cos(angle);
  *z1 = radius * std::sin(angle);
}

void gwso_noise_bm_z(uint64_t seed, uint64_t step, uint64_t first_elem, int64_t n, double* z) {
  for (int64_t k = 0; k < n; ++k) {
    const uint64_t e = first_elem + static_cast<uint64_t>(k);
    uint32_t o[4];
    philox_for_vector(seed, step, e >> 2, o);
    double z0, z1;
    box_muller_pair(o[(e & 2u) ? 2 : 0], o[(e & 2u) ? 3 : 1], &z0, &z1);
    z[k] = (e & 1u) ? z1 : z0;
  }
}

// R = round-half-even(z / 2), the rounded normal the method approximates (Section 3.4).
void gwso_noise_bm_r(uint64_t seed, uint64_t step, uint64_t first_elem, int64_t n, int8_t* r) {
  for (int64_t k = 0; k < n; ++k) {
    double z;
    gwso_noise_bm_z(seed, step, first_elem + static_cast<uint64_t>(k), 1, &z);
    r[k] = static_cast<int8_t>(std::nearbyint(0.5 * z));   // default rounding mode: to nearest, ties to even
  }
}

// Eq. 3 + the BF16 cast with a real-valued noise u given as BF16 bit patterns, one per element in logical order:
// w_hat = bf16( fl32( float(w) + fl32( float(u) * s_g ) ) ), s_g as in gwso_sample_fwd.
void gwso_sample_fwd_bf16_noise(int64_t rows, int64_t cols, int64_t ld, int64_t group_rows, int64_t group_cols,
                                const uint16_t* w, const float* bt, const uint16_t* u_bf16, uint16_t* w_hat,
                                float* scale_out, float* absmax_scratch) {
  const Geometry geo = make_geometry(rows, cols, ld, group_rows, group_cols);
  gwso_group_absmax(rows, cols, ld, group_rows, group_cols, w, absmax_scratch);
  for (int64_t i = 0; i < rows; ++i)
    for (int64_t j = 0; j < cols; ++j) {
      const int64_t g = group_of(geo, i, j);
      const float s = scale_of(absmax_scratch[g], bt[g]);
      const float pqn = bf16_to_f32(u_bf16[i * cols + j]) * s;
      const float y = bf16_to_f32(w[i * ld + j]) + pqn;
      w_hat[i * ld + j] = f32_to_bf16_rne(y);
    }
  if (scale_out)
    for (int64_t g = 0; g < geo.n_groups; ++g) scale_out[g] = scale_of(absmax_scratch[g], bt[g]);
}

}  // extern "C"
