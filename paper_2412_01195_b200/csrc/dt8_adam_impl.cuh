// Launch code of the fused 8-bit Adam step for one (gradient dtype, parameter dtype) pair;
// included by dt8_adam_*.cu, each of which instantiates one pair.
#pragma once
#include "dt8_launch.h"

namespace dt8 {

template <class Args, int B, bool GBF16, bool PBF16, int MODE>
int launch_adam_kernel(const Args& args, int64_t blocks, const AdamHyper& h, const LaunchCtx& ctx) {
  constexpr int VPT = AdamGeometry<B>::VPT, THREADS = AdamGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<AdamOp<B, VPT, THREADS, GBF16, PBF16, MODE>, Args>;
  const size_t smem = smem_bytes(ctx.em, true, true, true, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, ctx.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  kernel<<<grid_for(blocks, GROUPS, ctx.sm_count), THREADS, smem, ctx.stream>>>(args, h, ctx.em, ctx.tables);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

template <class Args, int B, bool GBF16, bool PBF16>
int launch_adam_mode(const Args& args, int64_t blocks, int mode, const AdamHyper& h, const LaunchCtx& ctx) {
  switch (mode) {
    case kAdamWFast: return launch_adam_kernel<Args, B, GBF16, PBF16, kAdamWFast>(args, blocks, h, ctx);
    case kAdamWSmall: return launch_adam_kernel<Args, B, GBF16, PBF16, kAdamWSmall>(args, blocks, h, ctx);
    case kAdamWIeee: return launch_adam_kernel<Args, B, GBF16, PBF16, kAdamWIeee>(args, blocks, h, ctx);
    default: return launch_adam_kernel<Args, B, GBF16, PBF16, kAdamL2>(args, blocks, h, ctx);
  }
}

template <bool GBF16, bool PBF16, class Args>
int launch_adam_typed(const Args& a, int64_t blocks, int block_size, int mode, const AdamHyper& h,
                      const LaunchCtx& ctx) {
  switch (block_size) {
    case 256: return launch_adam_mode<Args, 256, GBF16, PBF16>(a, blocks, mode, h, ctx);
    case 512: return launch_adam_mode<Args, 512, GBF16, PBF16>(a, blocks, mode, h, ctx);
    case 1024: return launch_adam_mode<Args, 1024, GBF16, PBF16>(a, blocks, mode, h, ctx);
    case 2048: return launch_adam_mode<Args, 2048, GBF16, PBF16>(a, blocks, mode, h, ctx);
    case 4096: return launch_adam_mode<Args, 4096, GBF16, PBF16>(a, blocks, mode, h, ctx);
  }
  return DT8_ERR_UNSUPPORTED;
}

#define DT8_INSTANTIATE_ADAM(GBF16, PBF16)                                                          \
  template int launch_adam_typed<GBF16, PBF16, SingleArgs>(const SingleArgs&, int64_t, int, int,   \
                                                           const AdamHyper&, const LaunchCtx&);    \
  template int launch_adam_typed<GBF16, PBF16, MultiArgs>(const MultiArgs&, int64_t, int, int,     \
                                                          const AdamHyper&, const LaunchCtx&);

}  // namespace dt8
