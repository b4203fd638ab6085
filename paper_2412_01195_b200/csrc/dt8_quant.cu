// Stand-alone block-wise quantize (Eq. quant1 + quant2) and dequantize (Eq. quant3): kernel
// instantiations and launch.
#include "dt8_launch.h"

namespace dt8 {
namespace {

template <int B, bool SIGNED>
int launch_quantize_kernel(const float* x, int64_t n, uint8_t* codes, float* absmax, const LaunchCtx& ctx) {
  constexpr int VPT = QuantGeometry<B>::VPT, THREADS = QuantGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<QuantOp<B, VPT, THREADS, SIGNED>, SingleArgs>;
  const size_t smem = smem_bytes(ctx.em, SIGNED, !SIGNED, false, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, ctx.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  SingleArgs a;
  a.t = TensorDesc{nullptr, x, codes, absmax, nullptr, nullptr, n};
  a.nb = (n + B - 1) / B;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  kernel<<<grid_for(a.nb, GROUPS, ctx.sm_count), THREADS, smem, ctx.stream>>>(a, NoHyper{0}, ctx.em, ctx.tables);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int log2_int(int v) {
  int s = 0;
  while ((1 << s) < v) ++s;
  return s;
}

}  // namespace

int launch_quantize(const float* x, int64_t n, int block_size, int is_signed, uint8_t* codes,
                    float* absmax, const LaunchCtx& ctx) {
#define DT8_Q_CASE(BS)                                                              \
  case BS:                                                                          \
    return is_signed ? launch_quantize_kernel<BS, true>(x, n, codes, absmax, ctx)   \
                     : launch_quantize_kernel<BS, false>(x, n, codes, absmax, ctx);
  switch (block_size) {
    DT8_Q_CASE(256)
    DT8_Q_CASE(512)
    DT8_Q_CASE(1024)
    DT8_Q_CASE(2048)
    DT8_Q_CASE(4096)
  }
#undef DT8_Q_CASE
  return DT8_ERR_UNSUPPORTED;
}

int launch_dequantize(const uint8_t* codes, const float* absmax, int64_t n, int block_size,
                      int is_signed, float* out, const LaunchCtx& ctx) {
  // whole tiles: the bulk-store kernel; what is left (less than one tile): per-thread stores
  const int shift = log2_int(block_size);
  const int64_t tiles = n / kDeqBulkTile;
  if (tiles > 0) {
    static std::atomic<uint64_t> ok_s{0}, ok_u{0};
    cudaError_t e = is_signed ? allow_smem(ok_s, dequantize_bulk_kernel<true>, ctx.device, kDeqBulkSmemBytes)
                              : allow_smem(ok_u, dequantize_bulk_kernel<false>, ctx.device, kDeqBulkSmemBytes);
    if (e != cudaSuccess) return cuda_fail(e);
    const int64_t resident = static_cast<int64_t>(kDeqBulkCtasPerSm) * ctx.sm_count;
    const int g = static_cast<int>(tiles < resident ? tiles : resident);
    if (is_signed)
      dequantize_bulk_kernel<true><<<g, kDeqBulkThreads, kDeqBulkSmemBytes, ctx.stream>>>(codes, absmax, out, tiles, shift, ctx.tables);
    else
      dequantize_bulk_kernel<false><<<g, kDeqBulkThreads, kDeqBulkSmemBytes, ctx.stream>>>(codes, absmax, out, tiles, shift, ctx.tables);
    e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e);
    const int64_t done = tiles * kDeqBulkTile;     // a multiple of every block size
    codes += done;
    out += done;
    absmax += done >> shift;
    n -= done;
    if (n == 0) return DT8_OK;
  }
  const int64_t quads = (n + 3) / 4;
  const int64_t per_cta = static_cast<int64_t>(kDeqThreads) * kDeqUnroll;
  const int64_t ctas = (quads + per_cta - 1) / per_cta;
  const int64_t resident = static_cast<int64_t>(kDeqCtasPerSm) * ctx.sm_count;
  const int grid = static_cast<int>(ctas < resident ? ctas : resident);
  if (is_signed)
    dequantize_kernel<true><<<grid, kDeqThreads, kDeqSmemBytes, ctx.stream>>>(codes, absmax, out, n, shift, ctx.tables);
  else
    dequantize_kernel<false><<<grid, kDeqThreads, kDeqSmemBytes, ctx.stream>>>(codes, absmax, out, n, shift, ctx.tables);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

}  // namespace dt8
