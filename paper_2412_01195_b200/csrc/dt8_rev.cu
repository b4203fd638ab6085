// Memory kernels of the reversible networks (Section III-B): additive coupling (Eq. revnet4),
// its inverse (Eq. revnet5) and the invertible down-sampling with ratio 2 (Eq. revnet6).
// All three are pure streaming work: 12 bytes per element for a coupling half (two reads, one
// write), 8 for the rearrangement; the bound is HBM bandwidth.
#include <cuda_runtime.h>

#include <cstdint>

#include "dt8_launch.h"
#include "dt8_rev.h"

namespace dt8 {
namespace {

bool aligned_to(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// ---------------------------------------------------------------------------------------------
// coupling: out[(2n + which) * half + i] = in[(2n + which) * half + i] + sign * t[n * half + i]
// One sample per blockIdx.y (strided when the batch exceeds the grid), `half` walked in units of
// VEC floats with kCoupleUnroll independent loads per operand in flight per thread.
// ---------------------------------------------------------------------------------------------
constexpr int kCoupleThreads = 256;
constexpr int kCoupleUnroll = 4;

template <int VEC> struct VecOf;
template <> struct VecOf<4> { typedef float4 type; };
template <> struct VecOf<1> { typedef float type; };

template <bool SUB>
__device__ __forceinline__ float combine(float a, float b) { return SUB ? __fsub_rn(a, b) : __fadd_rn(a, b); }
template <bool SUB>
__device__ __forceinline__ float4 combine(float4 a, float4 b) {
  return make_float4(combine<SUB>(a.x, b.x), combine<SUB>(a.y, b.y), combine<SUB>(a.z, b.z),
                     combine<SUB>(a.w, b.w));
}

template <int VEC, bool SUB>
__global__ void __launch_bounds__(kCoupleThreads)
coupling_kernel(const float* in, const float* __restrict__ t, float* out, int64_t batch, int64_t half,
                int which) {
  typedef typename VecOf<VEC>::type V;
  const int64_t units = half / VEC;   // half % VEC == 0 on this path
  const int64_t tile = static_cast<int64_t>(kCoupleThreads) * kCoupleUnroll;
  for (int64_t n = blockIdx.y; n < batch; n += gridDim.y) {
    const V* a = reinterpret_cast<const V*>(in + (2 * n + which) * half);
    const V* b = reinterpret_cast<const V*>(t + n * half);
    V* o = reinterpret_cast<V*>(out + (2 * n + which) * half);
    for (int64_t base = static_cast<int64_t>(blockIdx.x) * tile; base < units;
         base += static_cast<int64_t>(gridDim.x) * tile) {
      V va[kCoupleUnroll], vb[kCoupleUnroll];
#pragma unroll
      for (int k = 0; k < kCoupleUnroll; ++k) {
        const int64_t i = base + k * kCoupleThreads + threadIdx.x;
        if (i < units) {
          va[k] = __ldcs(a + i);   // each byte is used once: streaming loads and stores
          vb[k] = __ldcs(b + i);
        }
      }
#pragma unroll
      for (int k = 0; k < kCoupleUnroll; ++k) {
        const int64_t i = base + k * kCoupleThreads + threadIdx.x;
        if (i < units) __stcs(o + i, combine<SUB>(va[k], vb[k]));
      }
    }
  }
}

template <bool SUB>
int launch_coupling(const float* in, const float* t, float* out, int64_t batch, int64_t half, int which,
                    void* stream) {
  if (batch < 0 || half < 0 || (which != 0 && which != 1)) return DT8_ERR_INVALID_ARG;
  if (batch == 0 || half == 0) return DT8_OK;
  if (!in || !t || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned_to(in, 4) || !aligned_to(t, 4) || !aligned_to(out, 4)) return DT8_ERR_ALIGNMENT;
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e);
  const bool vec = (half % 4 == 0) && aligned_to(in, 16) && aligned_to(t, 16) && aligned_to(out, 16);
  const int64_t units = vec ? half / 4 : half;
  const int64_t tile = static_cast<int64_t>(kCoupleThreads) * kCoupleUnroll;
  const int64_t want_x = (units + tile - 1) / tile;
  const int64_t gy = batch < 65535 ? batch : 65535;
  // enough CTAs to fill the machine several times over, no more
  const int64_t cap_x = (static_cast<int64_t>(sms) * 16 + gy - 1) / gy;
  const int64_t gx = want_x < cap_x ? want_x : cap_x;
  const dim3 grid(static_cast<unsigned>(gx < 1 ? 1 : gx), static_cast<unsigned>(gy));
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  if (vec)
    coupling_kernel<4, SUB><<<grid, kCoupleThreads, 0, s>>>(in, t, out, batch, half, which);
  else
    coupling_kernel<1, SUB><<<grid, kCoupleThreads, 0, s>>>(in, t, out, batch, half, which);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

// ---------------------------------------------------------------------------------------------
// invertible down-sampling, r = 2.  In the N x C x F x T layout the two input rows 2fo, 2fo + 1 of
// a channel are adjacent, and the four output channels of an input channel start at the same
// offset as the input channel itself (4 * Fo * To == F * T).  A thread takes VEC consecutive
// elements of one input row (VEC = 8, 4 or 2, the largest that divides T): the even ones go to
// output channel 2 df, the odd ones to 2 df + 1, at column (t / 2) of row fo.  Consecutive threads
// take consecutive pieces of the flat input, so loads and stores are whole lines per warp.
// ---------------------------------------------------------------------------------------------
// n / d for 32-bit n by multiply-high and shifts (Granlund-Montgomery); d >= 1.
struct FastDiv {
  uint32_t d, m, s1, s2;
  __host__ explicit FastDiv(uint32_t div) : d(div) {
    uint32_t l = 0;
    while ((1ull << l) < div) ++l;                       // l = ceil(log2 d)
    m = static_cast<uint32_t>(((1ull << 32) * ((1ull << l) - div)) / div + 1);
    s1 = l < 1 ? l : 1;
    s2 = l == 0 ? 0 : l - 1;
  }
  __host__ __device__ __forceinline__ uint32_t div(uint32_t n) const {
#if defined(__CUDA_ARCH__)
    const uint32_t t = __umulhi(m, n);
#else
    const uint32_t t = static_cast<uint32_t>((static_cast<uint64_t>(m) * n) >> 32);
#endif
    return (t + ((n - t) >> s1)) >> s2;
  }
};

constexpr int kShuffleThreads = 256;
constexpr int kShuffleUnroll = 4;

// A piece: VEC consecutive elements of a flat row (In) and the VEC / 2 even or odd ones (Out).
struct Float8 {
  float4 a, b;
};
template <int VEC> struct Piece;
template <> struct Piece<8> {
  typedef Float8 In;
  typedef float4 Out;
  static __device__ __forceinline__ In load_in(const float* p) {
    In v;
    v.a = __ldcs(reinterpret_cast<const float4*>(p));
    v.b = __ldcs(reinterpret_cast<const float4*>(p) + 1);
    return v;
  }
  static __device__ __forceinline__ void store_in(float* p, In v) {
    __stcs(reinterpret_cast<float4*>(p), v.a);
    __stcs(reinterpret_cast<float4*>(p) + 1, v.b);
  }
  static __device__ __forceinline__ Out load_out(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
  static __device__ __forceinline__ void store_out(float* p, Out v) { __stcs(reinterpret_cast<float4*>(p), v); }
  static __device__ __forceinline__ Out even(In v) { return make_float4(v.a.x, v.a.z, v.b.x, v.b.z); }
  static __device__ __forceinline__ Out odd(In v) { return make_float4(v.a.y, v.a.w, v.b.y, v.b.w); }
  static __device__ __forceinline__ In merge(Out e, Out o) {
    In v;
    v.a = make_float4(e.x, o.x, e.y, o.y);
    v.b = make_float4(e.z, o.z, e.w, o.w);
    return v;
  }
};
template <> struct Piece<4> {
  typedef float4 In;
  typedef float2 Out;
  static __device__ __forceinline__ In load_in(const float* p) { return __ldcs(reinterpret_cast<const float4*>(p)); }
  static __device__ __forceinline__ void store_in(float* p, In v) { __stcs(reinterpret_cast<float4*>(p), v); }
  static __device__ __forceinline__ Out load_out(const float* p) { return __ldcs(reinterpret_cast<const float2*>(p)); }
  static __device__ __forceinline__ void store_out(float* p, Out v) { __stcs(reinterpret_cast<float2*>(p), v); }
  static __device__ __forceinline__ Out even(In v) { return make_float2(v.x, v.z); }
  static __device__ __forceinline__ Out odd(In v) { return make_float2(v.y, v.w); }
  static __device__ __forceinline__ In merge(Out e, Out o) { return make_float4(e.x, o.x, e.y, o.y); }
};
template <> struct Piece<2> {
  typedef float2 In;
  typedef float Out;
  static __device__ __forceinline__ In load_in(const float* p) { return __ldcs(reinterpret_cast<const float2*>(p)); }
  static __device__ __forceinline__ void store_in(float* p, In v) { __stcs(reinterpret_cast<float2*>(p), v); }
  static __device__ __forceinline__ Out load_out(const float* p) { return __ldcs(p); }
  static __device__ __forceinline__ void store_out(float* p, Out v) { __stcs(p, v); }
  static __device__ __forceinline__ Out even(In v) { return v.x; }
  static __device__ __forceinline__ Out odd(In v) { return v.y; }
  static __device__ __forceinline__ In merge(Out e, Out o) { return make_float2(e, o); }
};

// Where piece `i` of the flat N x C x F x T array lives in the rearranged array: the offset (in
// floats) of its even elements; the odd ones are one output channel (Fo * To floats) further.
struct ShuffleMap {
  FastDiv per_row;   // pieces per input row (T / VEC)
  FastDiv rows;      // F
  uint32_t T, F;
  template <int VEC>
  __device__ __forceinline__ int64_t deep_offset(uint32_t i) const {
    const uint32_t row = per_row.div(i);               // (n * C + c) * F + f
    const uint32_t q = i - row * per_row.d;            // piece inside the row
    const uint32_t plane = rows.div(row);
    const uint32_t f = row - plane * F;
    const uint32_t To = T >> 1, Fo = F >> 1;
    const int64_t chan = static_cast<int64_t>(plane) * 4 + (f & 1u) * 2;
    return (chan * Fo + (f >> 1)) * To + q * (VEC / 2);
  }
};

// TO_DEPTH: flat -> rearranged (Eq. revnet6); otherwise the inverse.
template <int VEC, bool TO_DEPTH>
__global__ void __launch_bounds__(kShuffleThreads)
shuffle_kernel(const float* __restrict__ src, float* __restrict__ dst, uint32_t pieces, ShuffleMap map) {
  typedef Piece<VEC> P;
  const int64_t chan_stride = static_cast<int64_t>(map.F >> 1) * (map.T >> 1);
  const uint32_t tile = kShuffleThreads * kShuffleUnroll;
  // pieces < 2^31 (checked by the host), so base + tile cannot wrap
  for (uint32_t base = blockIdx.x * tile; base < pieces; base += gridDim.x * tile) {
    typename P::In flat[kShuffleUnroll];
    typename P::Out ev[kShuffleUnroll], od[kShuffleUnroll];
    int64_t off[kShuffleUnroll];
#pragma unroll
    for (int k = 0; k < kShuffleUnroll; ++k) {
      const uint32_t i = base + k * kShuffleThreads + threadIdx.x;
      if (i < pieces) {
        off[k] = map.deep_offset<VEC>(i);
        if (TO_DEPTH) {
          flat[k] = P::load_in(src + static_cast<int64_t>(i) * VEC);
        } else {
          ev[k] = P::load_out(src + off[k]);
          od[k] = P::load_out(src + off[k] + chan_stride);
        }
      }
    }
#pragma unroll
    for (int k = 0; k < kShuffleUnroll; ++k) {
      const uint32_t i = base + k * kShuffleThreads + threadIdx.x;
      if (i < pieces) {
        if (TO_DEPTH) {
          P::store_out(dst + off[k], P::even(flat[k]));
          P::store_out(dst + off[k] + chan_stride, P::odd(flat[k]));
        } else {
          P::store_in(dst + static_cast<int64_t>(i) * VEC, P::merge(ev[k], od[k]));
        }
      }
    }
  }
}

// Rows that are not a multiple of 4 floats (T = 50 in the paper's last down-sampling stage) leave
// the output rows at 4-byte alignment only.  A channel plane, however, occupies the same
// contiguous range on both sides (F * T floats, a multiple of 4), so small planes are permuted in
// shared memory: a CTA copies a run of whole planes in with 16-byte loads, and writes the same
// range out with 16-byte stores, each output element gathered from its source position.
constexpr int kPlaneThreads = 256;
constexpr int kPlaneTileFloats = 6144;    // 24 KB of dynamic shared memory: eight CTAs per SM

struct PlaneMap {
  FastDiv plane;   // F * T
  FastDiv chan;    // Fo * To
  FastDiv row;     // To (to depth) or T (from depth)
  uint32_t F, T;
};

template <bool TO_DEPTH>
__global__ void __launch_bounds__(kPlaneThreads)
shuffle_planes_kernel(const float* __restrict__ src, float* __restrict__ dst, int64_t planes,
                      int planes_per_tile, PlaneMap m) {
  extern __shared__ __align__(16) float plane_buf[];
  const uint32_t PS = m.plane.d, To = m.T >> 1, Fo = m.F >> 1;
  const int64_t tiles = (planes + planes_per_tile - 1) / planes_per_tile;
  for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const int64_t first = tile * planes_per_tile;
    const int64_t left = planes - first;
    const uint32_t count = static_cast<uint32_t>(left < planes_per_tile ? left : planes_per_tile) * PS;
    const float4* in4 = reinterpret_cast<const float4*>(src + first * PS);
    float4* out4 = reinterpret_cast<float4*>(dst + first * PS);
    // four independent loads in flight per thread
    for (uint32_t i0 = threadIdx.x; i0 < count / 4; i0 += 4 * kPlaneThreads) {
      float4 v[4];
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (i0 + k * kPlaneThreads < count / 4) v[k] = __ldcs(in4 + i0 + k * kPlaneThreads);
#pragma unroll
      for (int k = 0; k < 4; ++k)
        if (i0 + k * kPlaneThreads < count / 4) reinterpret_cast<float4*>(plane_buf)[i0 + k * kPlaneThreads] = v[k];
    }
    __syncthreads();
    for (uint32_t i = threadIdx.x; i < count / 4; i += kPlaneThreads) {
      const uint32_t e = 4 * i;
      const uint32_t p = m.plane.div(e);
      uint32_t r = e - p * PS;
      const float* base = plane_buf + p * PS;
      float v[4];
      if (TO_DEPTH) {
        // output position (q, fo, to) of the plane <- input position (2 fo + q / 2, 2 to + q % 2)
        uint32_t q = m.chan.div(r);
        r -= q * m.chan.d;
        uint32_t fo = m.row.div(r), to = r - fo * To;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          v[k] = base[(2 * fo + (q >> 1)) * m.T + 2 * to + (q & 1)];
          if (++to == To) {
            to = 0;
            if (++fo == Fo) {
              fo = 0;
              ++q;
            }
          }
        }
      } else {
        // output position (f, t) of the plane <- rearranged position (2 (f % 2) + t % 2, f / 2, t / 2)
        uint32_t f = m.row.div(r), t = r - f * m.T;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          v[k] = base[((2 * (f & 1) + (t & 1)) * Fo + (f >> 1)) * To + (t >> 1)];
          if (++t == m.T) {
            t = 0;
            ++f;
          }
        }
      }
      __stcs(out4 + i, make_float4(v[0], v[1], v[2], v[3]));
    }
    __syncthreads();
  }
}

// `flat` is the N x C x F x T side, `deep` the N x 4C x F/2 x T/2 side.
template <bool TO_DEPTH>
int launch_shuffle(const float* src, float* dst, int64_t N, int64_t C, int64_t F, int64_t T, void* stream) {
  if (N < 0 || C < 0 || F < 0 || T < 0 || (F & 1) || (T & 1)) return DT8_ERR_INVALID_ARG;
  if (N == 0 || C == 0 || F == 0 || T == 0) return DT8_OK;
  if (!src || !dst) return DT8_ERR_INVALID_ARG;
  if (F > 0x7FFFFFFF || T > 0x7FFFFFFF) return DT8_ERR_UNSUPPORTED;
  // total elements, guarded against overflow
  const int64_t lim = int64_t(1) << 33;
  if (N > lim / C || N * C > lim / F || N * C * F > lim / T) return DT8_ERR_UNSUPPORTED;
  const int64_t total = N * C * F * T;
  const float* flat = TO_DEPTH ? src : dst;
  const float* deep = TO_DEPTH ? dst : src;
  // 16-byte pieces need rows of a multiple of 4 floats (then output rows are a multiple of 2)
  const bool vec8 = (T % 8 == 0) && aligned_to(flat, 16) && aligned_to(deep, 16);
  const bool vec4 = vec8 || ((T % 4 == 0) && aligned_to(flat, 16) && aligned_to(deep, 8));
  if (!vec4 && !(aligned_to(flat, 8) && aligned_to(deep, 4))) return DT8_ERR_ALIGNMENT;
  const int vec = vec8 ? 8 : vec4 ? 4 : 2;
  const int64_t pieces = total / vec;
  if (pieces >= (int64_t(1) << 31) || N * C * F >= (int64_t(1) << 32)) return DT8_ERR_UNSUPPORTED;
  int dev = 0, sms = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t plane = F * T;
  if (!vec4 && plane <= kPlaneTileFloats && aligned_to(src, 16) && aligned_to(dst, 16)) {
    // short rows, small planes: permute whole planes in shared memory
    const int per_tile = static_cast<int>(kPlaneTileFloats / plane);
    const uint32_t To = static_cast<uint32_t>(T / 2), Fo = static_cast<uint32_t>(F / 2);
    PlaneMap pm{FastDiv(static_cast<uint32_t>(plane)), FastDiv(Fo * To),
                FastDiv(TO_DEPTH ? To : static_cast<uint32_t>(T)), static_cast<uint32_t>(F),
                static_cast<uint32_t>(T)};
    const int64_t planes = N * C;
    const int64_t tiles = (planes + per_tile - 1) / per_tile;
    const int64_t cap = static_cast<int64_t>(sms) * 8;
    const unsigned g = static_cast<unsigned>(tiles < cap ? tiles : cap);
    const size_t smem = static_cast<size_t>(per_tile) * plane * sizeof(float);
    shuffle_planes_kernel<TO_DEPTH><<<g, kPlaneThreads, smem, s>>>(src, dst, planes, per_tile, pm);
    e = cudaGetLastError();
    return e == cudaSuccess ? DT8_OK : cuda_fail(e);
  }
  ShuffleMap map{FastDiv(static_cast<uint32_t>(T / vec)), FastDiv(static_cast<uint32_t>(F)),
                 static_cast<uint32_t>(T), static_cast<uint32_t>(F)};
  const int64_t tile = static_cast<int64_t>(kShuffleThreads) * kShuffleUnroll;
  const int64_t want = (pieces + tile - 1) / tile;
  const int64_t cap = static_cast<int64_t>(sms) * 16;
  const unsigned grid = static_cast<unsigned>(want < cap ? want : cap);
  if (vec8)
    shuffle_kernel<8, TO_DEPTH><<<grid, kShuffleThreads, 0, s>>>(src, dst, static_cast<uint32_t>(pieces), map);
  else if (vec4)
    shuffle_kernel<4, TO_DEPTH><<<grid, kShuffleThreads, 0, s>>>(src, dst, static_cast<uint32_t>(pieces), map);
  else
    shuffle_kernel<2, TO_DEPTH><<<grid, kShuffleThreads, 0, s>>>(src, dst, static_cast<uint32_t>(pieces), map);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

}  // namespace
}  // namespace dt8

using namespace dt8;

extern "C" {

int dt8_rev_coupling_forward(const float* x, const float* t, float* y, int64_t batch, int64_t half,
                             int which, void* stream) {
  return launch_coupling<false>(x, t, y, batch, half, which, stream);
}

int dt8_rev_coupling_inverse(const float* y, const float* t, float* x, int64_t batch, int64_t half,
                             int which, void* stream) {
  return launch_coupling<true>(y, t, x, batch, half, which, stream);
}

int dt8_rev_space_to_depth(const float* x, int64_t N, int64_t C, int64_t F, int64_t T, float* y,
                           void* stream) {
  return launch_shuffle<true>(x, y, N, C, F, T, stream);
}

int dt8_rev_depth_to_space(const float* y, int64_t N, int64_t C, int64_t Fo, int64_t To, float* x,
                           void* stream) {
  if (Fo > (int64_t(1) << 30) || To > (int64_t(1) << 30)) return DT8_ERR_UNSUPPORTED;
  return launch_shuffle<false>(y, x, N, C, Fo < 0 ? Fo : 2 * Fo, To < 0 ? To : 2 * To, stream);
}

}  // extern "C"
