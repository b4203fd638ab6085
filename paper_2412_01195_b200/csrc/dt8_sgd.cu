// Fused 8-bit SGD-with-momentum step: kernel instantiations and launch.
#include "dt8_launch.h"

namespace dt8 {
namespace {

template <class Args, int B, bool GBF16, bool PBF16>
int launch_sgd_kernel(const Args& args, int64_t blocks, const SgdHyper& h, const LaunchCtx& ctx) {
  constexpr int VPT = SgdGeometry<B>::VPT, THREADS = SgdGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<SgdOp<B, VPT, THREADS, GBF16, PBF16>, Args>;
  const size_t smem = smem_bytes(ctx.em, true, false, true, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, ctx.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  kernel<<<grid_for(blocks, GROUPS, ctx.sm_count), THREADS, smem, ctx.stream>>>(args, h, ctx.em, ctx.tables);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

template <class Args, int B>
int launch_sgd_dtype(const Args& a, int64_t blocks, int p_dtype, int g_dtype, const SgdHyper& h,
                     const LaunchCtx& ctx) {
  const bool gb = g_dtype == DT8_BF16, pb = p_dtype == DT8_BF16;
  if (gb && pb) return launch_sgd_kernel<Args, B, true, true>(a, blocks, h, ctx);
  if (gb) return launch_sgd_kernel<Args, B, true, false>(a, blocks, h, ctx);
  if (pb) return launch_sgd_kernel<Args, B, false, true>(a, blocks, h, ctx);
  return launch_sgd_kernel<Args, B, false, false>(a, blocks, h, ctx);
}

template <class Args>
int launch_sgd_any(const Args& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
                   const SgdHyper& h, const LaunchCtx& ctx) {
  switch (block_size) {
    case 256: return launch_sgd_dtype<Args, 256>(a, blocks, p_dtype, g_dtype, h, ctx);
    case 512: return launch_sgd_dtype<Args, 512>(a, blocks, p_dtype, g_dtype, h, ctx);
    case 1024: return launch_sgd_dtype<Args, 1024>(a, blocks, p_dtype, g_dtype, h, ctx);
    case 2048: return launch_sgd_dtype<Args, 2048>(a, blocks, p_dtype, g_dtype, h, ctx);
    case 4096: return launch_sgd_dtype<Args, 4096>(a, blocks, p_dtype, g_dtype, h, ctx);
  }
  return DT8_ERR_UNSUPPORTED;
}

}  // namespace

int launch_sgd(const SingleArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
               const SgdHyper& h, const LaunchCtx& ctx) {
  return launch_sgd_any(a, blocks, block_size, p_dtype, g_dtype, h, ctx);
}

int launch_sgd(const MultiArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
               const SgdHyper& h, const LaunchCtx& ctx) {
  return launch_sgd_any(a, blocks, block_size, p_dtype, g_dtype, h, ctx);
}

}  // namespace dt8
