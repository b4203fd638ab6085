// Host-side interface between the translation units of the dt8 library.  The kernels are
// instantiated in several files so that they compile in parallel; the C ABI (dt8_api.cu) checks
// the arguments and calls the launchers declared here.
#pragma once
#include <cuda_runtime.h>

#include <atomic>
#include <cstdint>

#include "dt8.h"
#include "dt8_kernels.cuh"

namespace dt8 {

// What a launcher needs to know about the current device and call.
struct LaunchCtx {
  int device;
  int sm_count;
  EncMeta em;
  const DeviceTables* tables;   // device address of the constant tables on `device`
  cudaStream_t stream;
};

// Records the CUDA error for dt8_last_cuda_error and returns DT8_ERR_CUDA.
int cuda_fail(cudaError_t e);

// The kernels index quantization blocks with 32 bits (next block = block + grid stride).
constexpr int64_t kMaxBlocksPerLaunch = 0x7FFF0000;

inline int grid_for(int64_t blocks, int groups_per_cta, int sm_count) {
  const int64_t want = (blocks + groups_per_cta - 1) / groups_per_cta;
  return static_cast<int>(want < sm_count ? want : sm_count);
}

// Opt a kernel in to its dynamic shared memory size, once per device.  `done` is the caller's
// per-kernel flag word (one bit per device).
template <class K>
cudaError_t allow_smem(std::atomic<uint64_t>& done, K kernel, int device, size_t bytes) {
  const uint64_t bit = 1ull << device;
  if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(bytes));
  if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_release);
  return e;
}

// Values per thread and threads per CTA for each operation and block size.  A group (B / VPT
// threads) is a whole number of warps, or half a warp, and the groups tile the CTA.
template <int B, int VPT_WANTED, int THREADS_WANTED> struct GeometryOf {
  static constexpr int VPT = (B / VPT_WANTED >= 16) ? VPT_WANTED : B / 16;
  static constexpr int THREADS = (THREADS_WANTED % (B / VPT) == 0) ? THREADS_WANTED : (B / VPT);
  static_assert(VPT % 4 == 0 && THREADS <= kCtaThreads && THREADS % (B / VPT) == 0, "bad geometry");
};
// The steps run 512 threads x 16 values.  At block 256 that makes a group half a warp, so a warp
// works on two blocks at once (0.95 of the copy bandwidth for Adam, against 0.83 with one warp per
// block and 8 values per thread).  Block 512 is the one size that measured better with 768 threads
// x 8 values (0.90 against 0.89).
template <int B> struct AdamGeometry : GeometryOf<B, 16, 512> {};
template <> struct AdamGeometry<512> : GeometryOf<512, 8, 768> {};
template <int B> struct SgdGeometry : GeometryOf<B, 16, 512> {};
// The light quantize operation prefers one warp per block at block 256 (0.93 against 0.85).
template <int B> struct QuantGeometry : GeometryOf<B, 16, 1024> {};
template <> struct QuantGeometry<256> : GeometryOf<256, 8, 1024> {};

// Launchers.  p_dtype / g_dtype are dt8_dtype values, block_size one of the supported sizes,
// `blocks` the number of quantization blocks of the launch (<= kMaxBlocksPerLaunch), `mode` one
// of kAdamWFast ... kAdamWSmall.  Each returns a dt8_status.
int launch_adam(const SingleArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype, int mode,
                const AdamHyper& h, const LaunchCtx& ctx);
int launch_adam(const MultiArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype, int mode,
                const AdamHyper& h, const LaunchCtx& ctx);
int launch_sgd(const SingleArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
               const SgdHyper& h, const LaunchCtx& ctx);
int launch_sgd(const MultiArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
               const SgdHyper& h, const LaunchCtx& ctx);
int launch_quantize(const float* x, int64_t n, int block_size, int is_signed, uint8_t* codes,
                    float* absmax, const LaunchCtx& ctx);
int launch_dequantize(const uint8_t* codes, const float* absmax, int64_t n, int block_size,
                      int is_signed, float* out, const LaunchCtx& ctx);

// Per-dtype instantiations of the Adam launchers (one translation unit each).
template <bool GBF16, bool PBF16, class Args>
int launch_adam_typed(const Args& a, int64_t blocks, int block_size, int mode, const AdamHyper& h,
                      const LaunchCtx& ctx);

}  // namespace dt8
