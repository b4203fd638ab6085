/*
 * rev oracle -- TEST INFRASTRUCTURE, NOT THE PRODUCT.
 *
 * A plain, slow, obviously-correct CPU statement of the memory kernels of the reversible
 * networks of Section III: the additive coupling of a reversible residual block (Eq. revnet4)
 * and its inverse (Eq. revnet5), and the invertible down-sampling that rearranges
 * C x F x T into r^2 C x F/r x T/r (Section III-B "Type II RevNets", Eq. revnet6).
 *
 * Only the tests, the smoke check and the benchmark's cpu-baseline leg may call this file.  It
 * shares no code, table, header or helper with the CUDA library and must never be linked or
 * imported by it.
 *
 * Precision: activations are binary32 in the paper (Section II), so the coupling is one IEEE
 * binary32 addition (or subtraction) per element; the rearrangement moves values unchanged.
 *
 * Layout (a reading; the paper gives shapes, not memory order): an activation is a
 * contiguous N x C x F x T array, T fastest.  "Split evenly along the channel dimension"
 * (Section III-B): x1 is channels [0, C/2), x2 is channels [C/2, C) of every sample.  The
 * residual branches F and G are the caller's: their outputs arrive as contiguous
 * N x C/2 x F x T arrays.
 *
 * Down-sampling (a reading): Section III-B describes cutting every channel into 2 x 2 blocks
 * and reshaping each C x 2 x 2 block into 4C x 1 x 1.  Flattening a C x r x r block row-major
 * puts input channel c, row offset df, column offset dt at output channel c*r*r + df*r + dt:
 *
 *     y[n, c*r*r + df*r + dt, fo, to] = x[n, c, fo*r + df, to*r + dt]
 *
 * The other common order ((df*r + dt)*C + c) holds the same values in permuted channels; the
 * paper does not say which it uses.  Parity unpinned against the authors' channel order; the
 * map is pinned as a bijection, by hand-computed cases, and against a library routine that
 * implements the row-major reading.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -shared -fPIC
 */
#include <stdint.h>

/* One half of Eq. revnet4 (sign = +1):  out_half = in_half + t
 * or of Eq. revnet5 (sign = -1):        out_half = in_half - t
 * `in` and `out` are N x C x F x T arrays seen as N samples of two halves of `half` elements
 * each (half = C/2 * F * T); `which` selects the half (0: channels [0, C/2), 1: the rest);
 * `t` is the branch output, N x half, contiguous.  The other half of `out` is not touched. */
int revo_couple_half(const float *in, const float *t, float *out, int64_t batch, int64_t half,
                     int which, int sign) {
  if (batch < 0 || half < 0 || (which != 0 && which != 1) || (sign != 1 && sign != -1)) return 1;
  for (int64_t n = 0; n < batch; ++n) {
    const float *a = in + (2 * n + which) * half;
    const float *b = t + n * half;
    float *o = out + (2 * n + which) * half;
    for (int64_t i = 0; i < half; ++i) o[i] = sign > 0 ? a[i] + b[i] : a[i] - b[i];
  }
  return 0;
}

/* Eq. revnet6, forward: x is N x C x F x T, y is N x (r*r*C) x (F/r) x (T/r). */
int revo_space_to_depth(const float *x, int64_t N, int64_t C, int64_t F, int64_t T, int r,
                        float *y) {
  if (N < 0 || C < 0 || F < 0 || T < 0 || r < 1 || F % r || T % r) return 1;
  const int64_t Fo = F / r, To = T / r;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t c = 0; c < C; ++c)
      for (int64_t f = 0; f < F; ++f)
        for (int64_t t = 0; t < T; ++t) {
          const int64_t fo = f / r, df = f % r, to = t / r, dt = t % r;
          const int64_t co = c * r * r + df * r + dt;
          y[((n * (C * r * r) + co) * Fo + fo) * To + to] = x[((n * C + c) * F + f) * T + t];
        }
  return 0;
}

/* The inverse rearrangement: y is N x (r*r*C) x Fo x To, x is N x C x (Fo*r) x (To*r). */
int revo_depth_to_space(const float *y, int64_t N, int64_t C, int64_t Fo, int64_t To, int r,
                        float *x) {
  if (N < 0 || C < 0 || Fo < 0 || To < 0 || r < 1) return 1;
  const int64_t F = Fo * r, T = To * r;
  for (int64_t n = 0; n < N; ++n)
    for (int64_t co = 0; co < C * r * r; ++co)
      for (int64_t fo = 0; fo < Fo; ++fo)
        for (int64_t to = 0; to < To; ++to) {
          const int64_t c = co / (r * r), df = (co % (r * r)) / r, dt = co % r;
          x[((n * C + c) * F + fo * r + df) * T + to * r + dt] =
              y[((n * (C * r * r) + co) * Fo + fo) * To + to];
        }
  return 0;
}
