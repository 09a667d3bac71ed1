// CPU oracle for the im2win convolution hot path.  TEST INFRASTRUCTURE ONLY.
//
// Plain, slow, fp64 restatement of what the paper's method computes.  It is
// built and called only by the test-suite, by the smoke check and by the
// benchmark's cpu-baseline leg; the product library never links, imports or
// executes it, and it shares no source, header, table or helper with the CUDA
// path.
//
// What is restated here, each from the paper's text:
//   * the 2-D convolution of Eq. 1 (cross-correlation, no kernel flip), with
//     the stride that Eq. 2 and Table 1 imply and a symmetric zero padding
//     restored, as seven nested loops (Section "Im2win Convolution");
//   * the im2win data transformation of Eq. 2, 0-based:
//         win[n][c][ho][k*Kh + u] = xpad[n][c][ho*s + u][k]
//     for k in [0, W+2p), u in [0, Kh), where xpad is x with p zero rows and
//     columns on every side;
//   * the im2win convolution of Eq. 3: every sliding window is the contiguous
//     run win[n][c][ho][(wo*s)*Kh : (wo*s)*Kh + Kh*Kw], multiplied with a
//     filter stored "height before width" (fp[co][c][v*Kh + u]);
//   * the GEMM view of Algorithm 1 (M = Co, N = batch*Ho*Wo, K = C*Kh*Kw) only
//     fixes the set of terms; the oracle sums them in the plain loop order.
//
//   * the last step of Algorithm 1 with the options the paper leaves open
//     (bias, ReLU, binary16 or binary32 store, NCHW or NHWC store) and the
//     channel-innermost form of the im2win tensor that the paper's tensor-core
//     section works on: see the second half of this file.
//
// Pins (see tests/test_oracle_*.py): Table 1's twelve output sizes, the shapes
// of Fig. 1, a hand-computed worked example, brute force of the two routes
// against each other, an independent library convolution, a delta filter,
// the 1x1 = GEMM special case, bilinearity, the closed-form tensor sizes and
// an exhaustive check of the binary16 rounding routines; for the epilogue a
// hand-computed example, bias as an extra all-ones channel, ReLU's defining
// properties and the single-rounding case that a detour through binary32 gets
// wrong; for the NHWC form an index-decoding test built with numpy slicing,
// its relation to the NCHW tensor and brute force against Eq. 1.
// Parity unpinned: the numerical output of the paper's own kernels (the paper
// prints no element values, checksums or error figures).

#include <cmath>
#include <cstdint>
#include <cstring>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

extern "C" {

typedef struct {
  int32_t N, C, H, W, Co, Kh, Kw, stride, pad;
} oracle_shape;

// Output size: Ho = floor((H + 2p - Kh) / s) + 1 (Table 1 lists only p = 0).
int oracle_out_dims(const oracle_shape* s, int32_t* Ho, int32_t* Wo) {
  if (!s || s->N < 1 || s->C < 1 || s->H < 1 || s->W < 1 || s->Co < 1 || s->Kh < 1 ||
      s->Kw < 1 || s->stride < 1 || s->pad < 0)
    return 1;
  const int64_t hs = (int64_t)s->H + 2 * (int64_t)s->pad - s->Kh;
  const int64_t ws = (int64_t)s->W + 2 * (int64_t)s->pad - s->Kw;
  if (hs < 0 || ws < 0) return 1;
  *Ho = (int32_t)(hs / s->stride) + 1;
  *Wo = (int32_t)(ws / s->stride) + 1;
  return 0;
}

// Element count of the im2win tensor: N*C*Ho*Kh*(W+2p)  (Eq. 2's index range).
int64_t oracle_window_elems(const oracle_shape* s) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return -1;
  return (int64_t)s->N * s->C * Ho * s->Kh * ((int64_t)s->W + 2 * s->pad);
}

// Element count of the im2col matrix: one row of C*Kh*Kw per output position.
int64_t oracle_im2col_elems(const oracle_shape* s) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return -1;
  return (int64_t)s->N * s->C * s->Kh * s->Kw * Ho * Wo;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

// Eq. 2 on raw storage: elements are elem_bytes-wide bit patterns (2 or 4)
// copied verbatim; padding positions hold the all-zero pattern (+0).
int oracle_transform(const void* x, void* win, const oracle_shape* s, int32_t elem_bytes) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  if (elem_bytes != 2 && elem_bytes != 4) return 2;
  const int64_t Wp = (int64_t)s->W + 2 * s->pad;
  const int64_t strip = (int64_t)s->Kh * Wp;
  const unsigned char* xi = (const unsigned char*)x;
  unsigned char* wo = (unsigned char*)win;
  std::memset(wo, 0, (size_t)(oracle_window_elems(s) * elem_bytes));
  for (int64_t n = 0; n < s->N; ++n)
    for (int64_t c = 0; c < s->C; ++c)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t k = 0; k < Wp; ++k)
          for (int64_t u = 0; u < s->Kh; ++u) {
            const int64_t h = m * s->stride + u - s->pad;  // row in the unpadded input
            const int64_t w = k - s->pad;                  // column in the unpadded input
            if (h < 0 || h >= s->H || w < 0 || w >= s->W) continue;
            const int64_t src = ((n * s->C + c) * s->H + h) * s->W + w;
            const int64_t dst = ((n * s->C + c) * Ho + m) * strip + k * s->Kh + u;
            std::memcpy(wo + dst * elem_bytes, xi + src * elem_bytes, (size_t)elem_bytes);
          }
  return 0;
}

// One output element of Eq. 1 (stride and zero padding restored), in fp64.
static inline void direct_point(const float* x, const float* f, const oracle_shape* s, int64_t n,
                                int64_t j, int64_t m, int64_t q, double* y, double* a) {
  double acc = 0.0, mag = 0.0;
  for (int64_t r = 0; r < s->C; ++r)
    for (int64_t u = 0; u < s->Kh; ++u)
      for (int64_t v = 0; v < s->Kw; ++v) {
        const int64_t h = m * s->stride + u - s->pad;
        const int64_t w = q * s->stride + v - s->pad;
        if (h < 0 || h >= s->H || w < 0 || w >= s->W) continue;
        const double xv = (double)x[((n * s->C + r) * s->H + h) * s->W + w];
        const double fv = (double)f[((j * s->C + r) * s->Kh + u) * s->Kw + v];
        acc += xv * fv;
        mag += std::fabs(xv) * std::fabs(fv);
      }
  *y = acc;
  *a = mag;
}

// Eq. 1 as the seven-loop direct convolution.  y and a (= sum |x||f| over the
// same terms, the tolerance denominator) are [N][Co][Ho][Wo] doubles.
int oracle_conv_direct(const float* x, const float* f, const oracle_shape* s, double* y,
                       double* a) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  for (int64_t n = 0; n < s->N; ++n)
    for (int64_t j = 0; j < s->Co; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t q = 0; q < Wo; ++q) {
          const int64_t o = ((n * s->Co + j) * Ho + m) * Wo + q;
          direct_point(x, f, s, n, j, m, q, &y[o], &a[o]);
        }
  return 0;
}

// Eq. 1 at chosen flat output indices only (for spot checks at full size).
int oracle_conv_direct_points(const float* x, const float* f, const oracle_shape* s,
                              const int64_t* flat, int64_t count, double* y, double* a) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  const int64_t total = (int64_t)s->N * s->Co * Ho * Wo;
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < count; ++i) {
    int64_t o = flat[i];
    if (o < 0 || o >= total) {
      y[i] = a[i] = NAN;
      continue;
    }
    const int64_t q = o % Wo;
    o /= Wo;
    const int64_t m = o % Ho;
    o /= Ho;
    const int64_t j = o % s->Co;
    const int64_t n = o / s->Co;
    direct_point(x, f, s, n, j, m, q, &y[i], &a[i]);
  }
  return 0;
}

// The im2win route: Eq. 2 into an fp64 window tensor, the filter repacked
// height-before-width, then Eq. 3's contiguous window x filter dot products.
// Images [n_begin, n_end) only, so that a bounded slice can be timed; y and a
// are indexed for the whole batch.  OpenMP over (n, co, ho).
int oracle_conv_im2win_range(const float* x, const float* f, const oracle_shape* s,
                             int32_t n_begin, int32_t n_end, double* y, double* a) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  if (n_begin < 0 || n_end > s->N || n_begin > n_end) return 2;
  const int64_t C = s->C, Kh = s->Kh, Kw = s->Kw, st = s->stride, p = s->pad;
  const int64_t Wp = (int64_t)s->W + 2 * p;
  const int64_t strip = Kh * Wp, T = Kh * Kw;
  const int64_t nimg = n_end - n_begin;

  // Eq. 2 (values widened to double; zeros where the padding is).
  std::vector<double> win((size_t)(nimg * C * Ho * strip), 0.0);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < nimg; ++n)
    for (int64_t c = 0; c < C; ++c)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t k = 0; k < Wp; ++k)
          for (int64_t u = 0; u < Kh; ++u) {
            const int64_t h = m * st + u - p, w = k - p;
            if (h < 0 || h >= s->H || w < 0 || w >= s->W) continue;
            win[(size_t)(((n * C + c) * Ho + m) * strip + k * Kh + u)] =
                (double)x[(((n + n_begin) * C + c) * s->H + h) * s->W + w];
          }

  // Filter with the height index fastest: fp[co][c][v*Kh + u] = f[co][c][u][v].
  std::vector<double> fp((size_t)((int64_t)s->Co * C * T));
  for (int64_t j = 0; j < s->Co; ++j)
    for (int64_t c = 0; c < C; ++c)
      for (int64_t u = 0; u < Kh; ++u)
        for (int64_t v = 0; v < Kw; ++v)
          fp[(size_t)((j * C + c) * T + v * Kh + u)] = (double)f[((j * C + c) * Kh + u) * Kw + v];

  // Eq. 3: outer loops over the output, inner loops over channel and window.
#pragma omp parallel for collapse(3) schedule(static)
  for (int64_t n = 0; n < nimg; ++n)
    for (int64_t j = 0; j < s->Co; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t q = 0; q < Wo; ++q) {
          double acc = 0.0, mag = 0.0;
          for (int64_t c = 0; c < C; ++c) {
            const double* wrow = &win[(size_t)(((n * C + c) * Ho + m) * strip + (q * st) * Kh)];
            const double* frow = &fp[(size_t)((j * C + c) * T)];
            for (int64_t t = 0; t < T; ++t) {
              acc += wrow[t] * frow[t];
              mag += std::fabs(wrow[t]) * std::fabs(frow[t]);
            }
          }
          const int64_t o = (((n + n_begin) * s->Co + j) * Ho + m) * Wo + q;
          y[o] = acc;
          if (a) a[o] = mag;
        }
  return 0;
}

int oracle_conv_im2win(const float* x, const float* f, const oracle_shape* s, double* y,
                       double* a) {
  return oracle_conv_im2win_range(x, f, s, 0, s ? s->N : 0, y, a);
}

// IEEE-754 binary32 -> binary16, round to nearest, ties to even, done on the
// bit patterns: subnormal halves are kept, values at or beyond 65520 become
// infinity, NaNs stay NaNs (quiet), signs are preserved.
static inline uint16_t f32_to_f16_bits(float v) {
  uint32_t b;
  std::memcpy(&b, &v, 4);
  const uint16_t sign = (uint16_t)((b >> 16) & 0x8000u);
  const uint32_t mag = b & 0x7fffffffu;
  if (mag >= 0x7f800000u) {                       // inf or NaN
    if (mag == 0x7f800000u) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | 0x7e00u | ((mag >> 13) & 0x3ffu));
  }
  const int32_t e = (int32_t)(mag >> 23) - 127;   // unbiased exponent
  uint32_t m = mag & 0x7fffffu;
  if (e >= 16) return (uint16_t)(sign | 0x7c00u); // too large for any finite half
  if (e >= -14) {                                 // normal half (before rounding)
    uint32_t h = ((uint32_t)(e + 15) << 10) | (m >> 13);
    const uint32_t rest = m & 0x1fffu;            // 13 dropped bits
    if (rest > 0x1000u || (rest == 0x1000u && (h & 1u))) ++h;  // may carry into inf: correct
    return (uint16_t)(sign | h);
  }
  if (e < -25) return sign;                       // below half of the smallest subnormal
  // subnormal half: value = (1.m) * 2^e, unit 2^-24
  m |= 0x800000u;                                 // 24-bit significand, weight 2^(e-23)
  const int32_t shift = -e - 1;                   // in [14, 24]: bits dropped to reach unit 2^-24
  uint32_t h = m >> shift;
  const uint32_t rest = m & ((1u << shift) - 1u);
  const uint32_t half = 1u << (shift - 1);
  if (rest > half || (rest == half && (h & 1u))) ++h;
  return (uint16_t)(sign | h);
}

static inline double f16_bits_to_f64(uint16_t h) {
  const int sign = (h >> 15) & 1;
  const int e = (h >> 10) & 0x1f;
  const int m = h & 0x3ff;
  double v;
  if (e == 0)
    v = std::ldexp((double)m, -24);
  else if (e == 31)
    v = m ? NAN : INFINITY;
  else
    v = std::ldexp((double)(m | 0x400), e - 25);
  return sign ? -v : v;
}

// Rounds n floats to binary16; writes the half bit patterns and, when asked,
// the rounded values widened back to float (exact).
void oracle_round_to_f16(const float* in, int64_t n, uint16_t* bits, float* back) {
#pragma omp parallel for schedule(static)
  for (int64_t i = 0; i < n; ++i) {
    const uint16_t h = f32_to_f16_bits(in[i]);
    if (bits) bits[i] = h;
    if (back) back[i] = (float)f16_bits_to_f64(h);
  }
}

void oracle_f16_bits_to_f64(const uint16_t* bits, int64_t n, double* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = f16_bits_to_f64(bits[i]);
}


// ---------------------------------------------------------------------------
// Last step of Algorithm 1 ("write C_reg to C") with the options the paper
// leaves open: the accumulator may leave as binary32 or binary16, a per-output-
// channel bias may be added and a ReLU applied first, and the output may be
// stored NCHW or NHWC.  The paper fixes none of these; the readings taken are
//   y = conv (Eq. 1, fp64)  ->  y += bias[co]  ->  y = max(y, 0)  ->  store,
// with a binary16 store rounding the fp64 value ONCE, to nearest, ties to even.

// IEEE-754 binary64 -> binary16 in one rounding (no detour through binary32,
// which could round twice), on the bit pattern.
static inline uint16_t f64_to_f16_bits(double v) {
  uint64_t b;
  std::memcpy(&b, &v, 8);
  const uint16_t sign = (uint16_t)((b >> 48) & 0x8000u);
  const uint64_t mag = b & 0x7fffffffffffffffull;
  if (mag >= 0x7ff0000000000000ull) {             // inf or NaN
    if (mag == 0x7ff0000000000000ull) return (uint16_t)(sign | 0x7c00u);
    return (uint16_t)(sign | 0x7e00u | ((mag >> 42) & 0x3ffu));
  }
  const int32_t e = (int32_t)(mag >> 52) - 1023;  // unbiased exponent (-1023 for zero/subnormal doubles)
  uint64_t m = mag & 0xfffffffffffffull;          // 52 fraction bits
  if (e >= 16) return (uint16_t)(sign | 0x7c00u);
  if (e >= -14) {                                 // normal half before rounding: keep 10 of 52 bits
    uint32_t h = ((uint32_t)(e + 15) << 10) | (uint32_t)(m >> 42);
    const uint64_t rest = m & ((1ull << 42) - 1);
    const uint64_t half = 1ull << 41;
    if (rest > half || (rest == half && (h & 1u))) ++h;        // a carry into the exponent is correct
    return (uint16_t)(sign | h);
  }
  if (e < -25) return sign;                       // below half of the smallest subnormal half (or zero)
  m |= 1ull << 52;                                // 53-bit significand, weight 2^(e-52)
  const int32_t shift = -e + 28;                  // bits dropped to reach the unit 2^-24: in [43, 53]
  uint32_t h = (uint32_t)(m >> shift);
  const uint64_t rest = m & ((1ull << shift) - 1);
  const uint64_t half = 1ull << (shift - 1);
  if (rest > half || (rest == half && (h & 1u))) ++h;
  return (uint16_t)(sign | h);
}

void oracle_round_f64_to_f16(const double* in, int64_t n, uint16_t* bits, double* back) {
  for (int64_t i = 0; i < n; ++i) {
    const uint16_t h = f64_to_f16_bits(in[i]);
    if (bits) bits[i] = h;
    if (back) back[i] = f16_bits_to_f64(h);
  }
}

// Applies the epilogue to y[N][Co][Ho][Wo] (fp64, NCHW) in place and, when
// asked, also writes the NHWC arrangement y_nhwc[N][Ho][Wo][Co].  a (the
// tolerance denominator, sum |x||f|) gets |bias| added.  bias may be null.
int oracle_epilogue(double* y, double* a, const oracle_shape* s, const float* bias, int32_t relu,
                    int32_t out16, double* y_nhwc) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  for (int64_t n = 0; n < s->N; ++n)
    for (int64_t j = 0; j < s->Co; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t q = 0; q < Wo; ++q) {
          const int64_t o = ((n * s->Co + j) * Ho + m) * Wo + q;
          double v = y[o];
          if (bias) {
            v += (double)bias[j];
            if (a) a[o] += std::fabs((double)bias[j]);
          }
          if (relu && v < 0.0) v = 0.0;           // NaN stays NaN
          if (out16) v = f16_bits_to_f64(f64_to_f16_bits(v));
          y[o] = v;
          if (y_nhwc) y_nhwc[((n * Ho + m) * Wo + q) * s->Co + j] = v;
        }
  return 0;
}

// ---------------------------------------------------------------------------
// Channel-innermost (NHWC) form of the im2win tensor.  The paper's tensor-core
// kernel works on NHWC data (Section "Im2win Convolution on Tensor Cores") but
// prints the index map only for NCHW (Eq. 2); the reading taken is Eq. 2 with
// the channel moved to the fastest position:
//     win[n][ho][k][u][c] = xpad[n][c][ho*s + u][k],   c in [0, Cp),
// where Cp >= C is the stored channel count (channels C..Cp-1 hold zeros).
// A sliding window (ho, wo) is then the contiguous run of Kw*Kh*Cp elements
// starting at (wo*s)*Kh*Cp of strip (n, ho), in the order (v, u, c): height
// before width as in Eq. 3, the channel below both.
// x_layout: 0 = x is [N][C][H][W], 1 = x is [N][H][W][C].
static inline int64_t x_index(const oracle_shape* s, int32_t x_layout, int64_t n, int64_t c, int64_t h, int64_t w) {
  return x_layout == 0 ? ((n * s->C + c) * s->H + h) * s->W + w : ((n * s->H + h) * s->W + w) * s->C + c;
}

int64_t oracle_window_elems_nhwc(const oracle_shape* s, int32_t Cp) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo) || Cp < s->C) return -1;
  return (int64_t)s->N * Ho * ((int64_t)s->W + 2 * s->pad) * s->Kh * Cp;
}

int oracle_transform_nhwc(const void* x, void* win, const oracle_shape* s, int32_t elem_bytes,
                          int32_t x_layout, int32_t Cp) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  if (elem_bytes != 2 && elem_bytes != 4) return 2;
  if (Cp < s->C || (x_layout != 0 && x_layout != 1)) return 3;
  const int64_t Wp = (int64_t)s->W + 2 * s->pad;
  const unsigned char* xi = (const unsigned char*)x;
  unsigned char* wo = (unsigned char*)win;
  std::memset(wo, 0, (size_t)(oracle_window_elems_nhwc(s, Cp) * elem_bytes));
  for (int64_t n = 0; n < s->N; ++n)
    for (int64_t m = 0; m < Ho; ++m)
      for (int64_t k = 0; k < Wp; ++k)
        for (int64_t u = 0; u < s->Kh; ++u)
          for (int64_t c = 0; c < s->C; ++c) {
            const int64_t h = m * s->stride + u - s->pad;
            const int64_t w = k - s->pad;
            if (h < 0 || h >= s->H || w < 0 || w >= s->W) continue;
            const int64_t src = x_index(s, x_layout, n, c, h, w);
            const int64_t dst = ((((n * Ho + m) * Wp + k) * s->Kh + u) * Cp) + c;
            std::memcpy(wo + dst * elem_bytes, xi + src * elem_bytes, (size_t)elem_bytes);
          }
  return 0;
}

// The NHWC im2win route: the tensor above in fp64, the filter repacked to
// fp[co][(v*Kh + u)*Cp + c] = f[co][c][u][v] (zeros for c >= C), then one
// contiguous dot product of length Kw*Kh*Cp per output.  y and a are written
// NCHW ([N][Co][Ho][Wo]) for images [n_begin, n_end) of the whole-batch arrays.
int oracle_conv_im2win_nhwc_range(const float* x, const float* f, const oracle_shape* s, int32_t x_layout,
                                  int32_t Cp, int32_t n_begin, int32_t n_end, double* y, double* a) {
  int32_t Ho, Wo;
  if (oracle_out_dims(s, &Ho, &Wo)) return 1;
  if (n_begin < 0 || n_end > s->N || n_begin > n_end) return 2;
  if (Cp < s->C || (x_layout != 0 && x_layout != 1)) return 3;
  const int64_t C = s->C, Kh = s->Kh, Kw = s->Kw, st = s->stride, p = s->pad;
  const int64_t Wp = (int64_t)s->W + 2 * p;
  const int64_t strip = Wp * Kh * Cp, run = Kw * Kh * Cp;
  const int64_t nimg = n_end - n_begin;
  std::vector<double> win((size_t)(nimg * Ho * strip), 0.0);
#pragma omp parallel for collapse(2) schedule(static)
  for (int64_t n = 0; n < nimg; ++n)
    for (int64_t m = 0; m < Ho; ++m)
      for (int64_t k = 0; k < Wp; ++k)
        for (int64_t u = 0; u < Kh; ++u)
          for (int64_t c = 0; c < C; ++c) {
            const int64_t h = m * st + u - p, w = k - p;
            if (h < 0 || h >= s->H || w < 0 || w >= s->W) continue;
            win[(size_t)((((n * Ho + m) * Wp + k) * Kh + u) * Cp + c)] =
                (double)x[x_index(s, x_layout, n + n_begin, c, h, w)];
          }
  std::vector<double> fp((size_t)((int64_t)s->Co * run), 0.0);
  for (int64_t j = 0; j < s->Co; ++j)
    for (int64_t c = 0; c < C; ++c)
      for (int64_t u = 0; u < Kh; ++u)
        for (int64_t v = 0; v < Kw; ++v)
          fp[(size_t)(j * run + (v * Kh + u) * Cp + c)] = (double)f[((j * C + c) * Kh + u) * Kw + v];
#pragma omp parallel for collapse(3) schedule(static)
  for (int64_t n = 0; n < nimg; ++n)
    for (int64_t j = 0; j < s->Co; ++j)
      for (int64_t m = 0; m < Ho; ++m)
        for (int64_t q = 0; q < Wo; ++q) {
          const double* wrow = &win[(size_t)((n * Ho + m) * strip + (q * st) * Kh * Cp)];
          const double* frow = &fp[(size_t)(j * run)];
          double acc = 0.0, mag = 0.0;
          for (int64_t t = 0; t < run; ++t) {
            acc += wrow[t] * frow[t];
            mag += std::fabs(wrow[t]) * std::fabs(frow[t]);
          }
          const int64_t o = (((n + n_begin) * s->Co + j) * Ho + m) * Wo + q;
          y[o] = acc;
          if (a) a[o] = mag;
        }
  return 0;
}

}  // extern "C"
