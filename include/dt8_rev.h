/*
 * dt8_rev -- memory kernels of the reversible networks (CUDA, sm_100a), part of libdt8.
 *
 * Section III-B of "Memory-Efficient Training for Deep Speaker Embedding Learning in Speaker
 * Verification" (arXiv 2412.01195) removes the stored activations of a residual network in two
 * ways: a residual block becomes an additive coupling whose input can be recomputed from its
 * output (Eq. revnet4, Eq. revnet5, Alg. 1), and the strided down-sampling becomes a
 * rearrangement C x F x T -> r^2 C x F/r x T/r that loses nothing (Eq. revnet6).  The residual
 * branches F and G (convolutions, batch-norm, ReLU) are the caller's; these entry points are the
 * element-wise and permutation steps around them.  Each moves every byte once.
 *
 * Conventions: those of dt8.h (status codes, device pointers of the current device owned by the
 * caller, asynchronous on `stream`, no allocation, nothing launched on an error).  Activations
 * are binary32 (Section II), contiguous N x C x F x T arrays with T fastest.  The two halves of
 * a coupling are the channel ranges [0, C/2) and [C/2, C) of every sample (Section III-B: the
 * input is split evenly along the channel dimension); a branch output is a contiguous
 * N x C/2 x F x T array.  Pointers need 4-byte alignment; 16-byte-aligned tensors whose rows
 * allow it take 16-byte accesses.
 */
#ifndef DT8_REV_H_
#define DT8_REV_H_

#include <stdint.h>

#include "dt8.h"

#ifdef __cplusplus
extern "C" {
#endif

/*
 * One half of the additive coupling, Eq. revnet4:  y_half = x_half + t  (t = F(x2) for half 0,
 * t = G(y1) for half 1), one binary32 addition per element.  Also the two sums of Alg. 1,
 * dL/dz1 = dL/dy1 + (dG/dz1)^T dL/dy2 and dL/dx2 = dL/dy2 + (dF/dx2)^T dL/dz1, with the
 * gradient tensors in the place of x and y and the vector-Jacobian product in the place of t.
 *   x      device, const float[batch * 2 * half]   input activation (both halves)
 *   t      device, const float[batch * half]       branch output
 *   y      device, float[batch * 2 * half]         output activation; only half `which` is written;
 *                                                   y == x (in place) is allowed
 *   half   elements of one half of one sample (C/2 * F * T);  which  0 or 1
 * batch < 0, half < 0, which not 0 / 1 or a NULL pointer with work to do: DT8_ERR_INVALID_ARG.
 */
int dt8_rev_coupling_forward(const float *x, const float *t, float *y, int64_t batch, int64_t half,
                             int which, void *stream);

/*
 * One half of the inverse coupling, Eq. revnet5:  x_half = y_half - t  (t = G(z1) for half 1,
 * then t = F(x2) for half 0), one binary32 subtraction per element.  Arguments as above with the
 * roles of x and y exchanged; x == y (in place) is allowed.  The recovered input equals the
 * original up to the two roundings fl(fl(a + t) - t); it is exact whenever a + t is
 * representable.
 */
int dt8_rev_coupling_inverse(const float *y, const float *t, float *x, int64_t batch, int64_t half,
                             int which, void *stream);

/*
 * Invertible down-sampling with ratio r = 2 (Eq. revnet6, the ratio of every "rev_ds" layer of
 * the paper's Type II networks):  x is N x C x F x T, y is N x 4C x F/2 x T/2 with
 *     y[n, 4c + 2 df + dt, fo, to] = x[n, c, 2 fo + df, 2 to + dt],
 * i.e. every C x 2 x 2 block flattened row-major into 4C x 1 x 1 (the paper gives the shapes;
 * this order within the 4C channels is this library's reading of it).  F and T must be even;
 * x and y must not overlap.  Odd F or T: DT8_ERR_INVALID_ARG.  More than 2^33 elements:
 * DT8_ERR_UNSUPPORTED.
 */
int dt8_rev_space_to_depth(const float *x, int64_t N, int64_t C, int64_t F, int64_t T, float *y,
                           void *stream);

/* The inverse rearrangement: y is N x 4C x Fo x To, x is N x C x 2Fo x 2To. */
int dt8_rev_depth_to_space(const float *y, int64_t N, int64_t C, int64_t Fo, int64_t To, float *x,
                           void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DT8_REV_H_ */
