// C ABI of the dt8 library: argument checks, table upload, kernel selection and launch.
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstring>
#include <initializer_list>
#include <mutex>

#include "dt8.h"
#include "dt8_kernels.cuh"

namespace dt8 {
namespace {

thread_local int tl_last_cuda_error = 0;

int cuda_fail(cudaError_t e) {
  tl_last_cuda_error = static_cast<int>(e);
  return DT8_ERR_CUDA;
}

constexpr int kMaxDevices = 64;

struct DeviceInfo {
  int device = -1;
  int sm_count = 0;
};

std::mutex g_init_mutex;
std::atomic<bool> g_uploaded[kMaxDevices];
int g_sm_count[kMaxDevices];

// Makes sure the current device holds the constant tables; returns the device's SM count.
int ensure_device(DeviceInfo* info, EncMeta* em) {
  const Tables* ht = host_tables();
  if (!ht) return DT8_ERR_UNSUPPORTED;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return DT8_ERR_UNSUPPORTED;
  if (!g_uploaded[dev].load(std::memory_order_acquire)) {
    std::lock_guard<std::mutex> lock(g_init_mutex);
    if (!g_uploaded[dev].load(std::memory_order_relaxed)) {
      static DeviceTables staging;  // guarded by g_init_mutex
      std::memcpy(staging.dec_s, ht->dec_signed, sizeof(staging.dec_s));
      std::memcpy(staging.dec_u, ht->dec_unsigned, sizeof(staging.dec_u));
      std::memset(staging.enc_s, 0, sizeof(staging.enc_s));
      std::memset(staging.enc_u, 0, sizeof(staging.enc_u));
      std::memcpy(staging.enc_s, ht->enc_signed.entries, sizeof(uint32_t) * ht->enc_signed.num_entries);
      std::memcpy(staging.enc_u, ht->enc_unsigned.entries, sizeof(uint32_t) * ht->enc_unsigned.num_entries);
      e = cudaMemcpyToSymbol(g_tables, &staging, sizeof(staging));
      if (e != cudaSuccess) return cuda_fail(e);
      // The kernels address their shared-memory tables absolutely: check once that this build's
      // tables fit the layout and that dynamic shared memory starts low enough on this device.
      EncMeta probe_em;
      probe_em.s_first = ht->enc_signed.first_key;
      probe_em.u_first = ht->enc_unsigned.first_key;
      probe_em.s_n = ht->enc_signed.num_entries;
      probe_em.u_n = ht->enc_unsigned.num_entries;
      if (!layout_ok(probe_em)) return DT8_ERR_UNSUPPORTED;
      const int probe_smem = static_cast<int>(smem_bytes(probe_em, true, true, true, true));
      e = cudaFuncSetAttribute(smem_start_probe, cudaFuncAttributeMaxDynamicSharedMemorySize, probe_smem);
      if (e != cudaSuccess) return cuda_fail(e);
      smem_start_probe<<<1, 32, probe_smem>>>();
      e = cudaGetLastError();
      if (e != cudaSuccess) return cuda_fail(e);
      uint32_t smem_start = 0xFFFFFFFFu;
      e = cudaMemcpyFromSymbol(&smem_start, g_smem_start, sizeof(smem_start));
      if (e != cudaSuccess) return cuda_fail(e);
      if (smem_start > kMaxSmemStart) return DT8_ERR_UNSUPPORTED;
      int sms = 0;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return cuda_fail(e);
      g_sm_count[dev] = sms;
      g_uploaded[dev].store(true, std::memory_order_release);
    }
  }
  info->device = dev;
  info->sm_count = g_sm_count[dev];
  em->s_first = ht->enc_signed.first_key;
  em->u_first = ht->enc_unsigned.first_key;
  em->s_n = ht->enc_signed.num_entries;
  em->u_n = ht->enc_unsigned.num_entries;
  return DT8_OK;
}

// Opt a kernel in to its dynamic shared memory size, once per device.  `done` is the caller's
// per-kernel flag word (kernels of different template arguments can share a pointer type, so the
// flag cannot live in this function).
template <class K>
cudaError_t allow_smem(std::atomic<uint64_t>& done, K kernel, int device, size_t bytes) {
  const uint64_t bit = 1ull << device;
  if (done.load(std::memory_order_acquire) & bit) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(bytes));
  if (e == cudaSuccess) done.fetch_or(bit, std::memory_order_release);
  return e;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

// The kernels index quantization blocks with 32 bits (next block = block + grid stride).
constexpr int64_t kMaxBlocksPerLaunch = 0x7FFF0000;

bool block_size_ok(int B) { return B == 256 || B == 512 || B == 1024 || B == 2048 || B == 4096; }

int log2_int(int v) {
  int s = 0;
  while ((1 << s) < v) ++s;
  return s;
}

int grid_for(int64_t blocks, int groups_per_cta, int sm_count) {
  const int64_t want = (blocks + groups_per_cta - 1) / groups_per_cta;
  return static_cast<int>(want < sm_count ? want : sm_count);
}

// Values per thread and threads per CTA for each operation and block size.  A group (B / VPT
// threads) is at least one warp, and the groups tile the CTA.
template <int B, int VPT_WANTED, int THREADS_WANTED> struct GeometryOf {
  static constexpr int VPT = (B / VPT_WANTED >= 32) ? VPT_WANTED : B / 32;
  static constexpr int THREADS = (THREADS_WANTED % (B / VPT) == 0) ? THREADS_WANTED : (B / VPT);
  static_assert(VPT % 4 == 0 && THREADS <= kCtaThreads && THREADS % (B / VPT) == 0, "bad geometry");
};
// The steps run 512 threads x 16 values.  Small blocks are latency-bound rather than issue-bound
// (one warp owns a block): 768 threads with 8 values each measured 1-5 % faster there.
template <int B> struct AdamGeometry : GeometryOf<B, 16, 512> {};
template <> struct AdamGeometry<256> : GeometryOf<256, 8, 768> {};
template <> struct AdamGeometry<512> : GeometryOf<512, 8, 768> {};
template <int B> struct SgdGeometry : GeometryOf<B, 16, 512> {};
template <> struct SgdGeometry<256> : GeometryOf<256, 8, 768> {};
template <int B> using QuantGeometry = GeometryOf<B, 16, 1024>;

// Hyper-parameters are checked before anything is launched: non-finite values and decay rates
// outside [0, 1) (1 - beta^step would be 0 or negative) are argument errors.
bool finite_all(std::initializer_list<float> v) {
  for (float x : v)
    if (!std::isfinite(x)) return false;
  return true;
}

bool adam_hyper_ok(float lr, float beta1, float beta2, float eps, float wd) {
  return finite_all({lr, beta1, beta2, eps, wd}) && beta1 >= 0.0f && beta1 < 1.0f && beta2 >= 0.0f &&
         beta2 < 1.0f && eps >= 0.0f;
}

bool sgd_hyper_ok(float lr, float momentum, float wd) {
  return finite_all({lr, momentum, wd}) && momentum >= 0.0f;
}

int check_tensor(const TensorDesc& d, int g_dtype, bool adam) {
  if (d.n < 0) return DT8_ERR_INVALID_ARG;
  if (d.n == 0) return DT8_OK;
  if (!d.p || !d.g || !d.mc || !d.ma) return DT8_ERR_INVALID_ARG;
  if (adam && (!d.rc || !d.ra)) return DT8_ERR_INVALID_ARG;
  if (!aligned(d.p, 16) || !aligned(d.g, g_dtype == DT8_F32 ? 16 : 8) || !aligned(d.mc, 4) ||
      !aligned(d.ma, 4))
    return DT8_ERR_ALIGNMENT;
  if (adam && (!aligned(d.rc, 4) || !aligned(d.ra, 4))) return DT8_ERR_ALIGNMENT;
  return DT8_OK;
}

// ---- launchers -------------------------------------------------------------------------------
template <class Args, int B, bool GBF16, int MODE>
int launch_adam(const Args& args, int64_t blocks, const AdamHyper& h, const EncMeta& em,
                const DeviceInfo& di, cudaStream_t stream) {
  constexpr int VPT = AdamGeometry<B>::VPT, THREADS = AdamGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<AdamOp<B, VPT, THREADS, GBF16, MODE>, Args>;
  const size_t smem = smem_bytes(em, true, true, true, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, di.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  kernel<<<grid_for(blocks, GROUPS, di.sm_count), THREADS, smem, stream>>>(args, h, em);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

template <class Args, int B, bool GBF16>
int dispatch_adam_mode(const Args& args, int64_t blocks, int mode, const AdamHyper& h,
                       const EncMeta& em, const DeviceInfo& di, cudaStream_t s) {
  switch (mode) {
    case kAdamWFast: return launch_adam<Args, B, GBF16, kAdamWFast>(args, blocks, h, em, di, s);
    case kAdamWIeee: return launch_adam<Args, B, GBF16, kAdamWIeee>(args, blocks, h, em, di, s);
    case kAdamWSmall: return launch_adam<Args, B, GBF16, kAdamWSmall>(args, blocks, h, em, di, s);
    default: return launch_adam<Args, B, GBF16, kAdamL2>(args, blocks, h, em, di, s);
  }
}

template <class Args, int B>
int dispatch_adam(const Args& args, int64_t blocks, int g_dtype, int mode, const AdamHyper& h,
                  const EncMeta& em, const DeviceInfo& di, cudaStream_t s) {
  return g_dtype == DT8_BF16 ? dispatch_adam_mode<Args, B, true>(args, blocks, mode, h, em, di, s)
                             : dispatch_adam_mode<Args, B, false>(args, blocks, mode, h, em, di, s);
}

template <class Args>
int dispatch_adam_b(const Args& args, int64_t blocks, int B, int g_dtype, int mode,
                    const AdamHyper& h, const EncMeta& em, const DeviceInfo& di, cudaStream_t s) {
  switch (B) {
    case 256: return dispatch_adam<Args, 256>(args, blocks, g_dtype, mode, h, em, di, s);
    case 512: return dispatch_adam<Args, 512>(args, blocks, g_dtype, mode, h, em, di, s);
    case 1024: return dispatch_adam<Args, 1024>(args, blocks, g_dtype, mode, h, em, di, s);
    case 2048: return dispatch_adam<Args, 2048>(args, blocks, g_dtype, mode, h, em, di, s);
    case 4096: return dispatch_adam<Args, 4096>(args, blocks, g_dtype, mode, h, em, di, s);
  }
  return DT8_ERR_UNSUPPORTED;
}

template <class Args, int B, bool GBF16>
int launch_sgd(const Args& args, int64_t blocks, const SgdHyper& h, const EncMeta& em,
               const DeviceInfo& di, cudaStream_t stream) {
  constexpr int VPT = SgdGeometry<B>::VPT, THREADS = SgdGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<SgdOp<B, VPT, THREADS, GBF16>, Args>;
  const size_t smem = smem_bytes(em, true, false, true, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, di.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  kernel<<<grid_for(blocks, GROUPS, di.sm_count), THREADS, smem, stream>>>(args, h, em);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

template <class Args>
int dispatch_sgd_b(const Args& args, int64_t blocks, int B, int g_dtype, const SgdHyper& h,
                   const EncMeta& em, const DeviceInfo& di, cudaStream_t s) {
#define DT8_SGD_CASE(BS)                                                        \
  case BS:                                                                      \
    return g_dtype == DT8_BF16 ? launch_sgd<Args, BS, true>(args, blocks, h, em, di, s) \
                               : launch_sgd<Args, BS, false>(args, blocks, h, em, di, s);
  switch (B) {
    DT8_SGD_CASE(256)
    DT8_SGD_CASE(512)
    DT8_SGD_CASE(1024)
    DT8_SGD_CASE(2048)
    DT8_SGD_CASE(4096)
  }
#undef DT8_SGD_CASE
  return DT8_ERR_UNSUPPORTED;
}

template <int B, bool SIGNED>
int launch_quantize(const float* x, int64_t n, uint8_t* codes, float* absmax, const EncMeta& em,
                    const DeviceInfo& di, cudaStream_t stream) {
  constexpr int VPT = QuantGeometry<B>::VPT, THREADS = QuantGeometry<B>::THREADS;
  constexpr int GROUPS = THREADS / (B / VPT);
  auto kernel = block_kernel<QuantOp<B, VPT, THREADS, SIGNED>, SingleArgs>;
  const size_t smem = smem_bytes(em, SIGNED, !SIGNED, false, true);
  static std::atomic<uint64_t> smem_ok{0};
  cudaError_t e = allow_smem(smem_ok, kernel, di.device, smem);
  if (e != cudaSuccess) return cuda_fail(e);
  SingleArgs a;
  a.t = TensorDesc{nullptr, x, codes, absmax, nullptr, nullptr, n};
  a.nb = (n + B - 1) / B;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  kernel<<<grid_for(a.nb, GROUPS, di.sm_count), THREADS, smem, stream>>>(a, NoHyper{0}, em);
  e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

// Correctly rounded binary32 reciprocal of a positive normal binary32 number, on the host.  The
// binary64 quotient rounded to binary32 can be one unit off (double rounding), so its two
// neighbours are compared as well: |d*y - 1| is exact in binary64 (a 48-bit product, then a
// difference of nearby numbers) and smallest for the nearest y.
float reciprocal_rn(float d) {
  const double dd = static_cast<double>(d);
  const float y0 = static_cast<float>(1.0 / dd);
  float best = y0;
  double best_err = std::fabs(dd * static_cast<double>(y0) - 1.0);
  const float cand[2] = {std::nextafterf(y0, 0.0f), std::nextafterf(y0, INFINITY)};
  for (float y : cand) {
    const double err = std::fabs(dd * static_cast<double>(y) - 1.0);
    if (err < best_err) {
      best_err = err;
      best = y;
    }
  }
  return best;
}

ConstDivisor make_const_divisor(float d) {
  ConstDivisor cd;
  cd.d = d;
  cd.usable = d >= kConstDivMinDivisor && d <= kConstDivMaxDivisor;
  cd.rd = cd.usable ? reciprocal_rn(d) : 0.0f;
  return cd;
}

AdamHyper make_adam_hyper(float lr, float beta1, float beta2, float eps, float wd, int64_t step,
                          uint32_t flags) {
  AdamHyper h;
  h.beta1 = beta1;
  h.beta2 = beta2;
  h.omb1 = 1.0f - beta1;
  h.omb2 = 1.0f - beta2;
  h.lr = lr;
  h.eps = eps;
  h.wd = wd;
  h.decay = 1.0f - lr * wd;
  if (flags & DT8_ADAM_BIAS_CORRECTION) {
    h.bc1 = static_cast<float>(1.0 - std::pow(static_cast<double>(beta1), static_cast<double>(step)));
    h.bc2 = static_cast<float>(1.0 - std::pow(static_cast<double>(beta2), static_cast<double>(step)));
  } else {
    h.bc1 = 1.0f;
    h.bc2 = 1.0f;
  }
  const double root_bc2 = std::sqrt(static_cast<double>(h.bc2));
  const double ss = static_cast<double>(lr) * root_bc2 / static_cast<double>(h.bc1);
  h.eps_scaled = static_cast<float>(static_cast<double>(eps) * root_bc2);
  h.inv_step = static_cast<float>(1.0 / ss);
  h.eps_over_step = static_cast<float>(static_cast<double>(eps) * root_bc2 / ss);
  const ConstDivisor d1 = make_const_divisor(h.bc1), d2 = make_const_divisor(h.bc2);
  h.rbc1 = d1.rd;
  h.rbc2 = d2.rd;
  h.const_div = (d1.usable && d2.usable) ? 1 : 0;
  return h;
}

// The single-instruction root and reciprocal flush subnormal numbers to zero; a flushed root
// (below 1.1e-19) is invisible next to the scaled eps only while that is well above it.  Below
// that the forms that keep subnormals are used.
constexpr float kMinEpsForFlushedRoot = 1e-12f;

// Coupled decay makes the parameters an input of the states, so they must then be computed with
// IEEE operations; without decay the two forms coincide and the approximate parameter path applies.
int adam_mode(uint32_t flags, const AdamHyper& h) {
  if (!(flags & DT8_ADAM_DECOUPLED_WD) && h.wd != 0.0f) return kAdamL2;
  // the approximate paths divide by the step size, so that must be a normal, moderate number
  const bool moderate = h.lr >= 1e-20f && h.lr <= 1e20f && std::isfinite(h.inv_step) &&
                        std::isfinite(h.eps_over_step) && h.inv_step >= 1e-30f;
  if (!moderate) return kAdamWIeee;
  const bool flush_ok = h.eps_scaled >= kMinEpsForFlushedRoot && h.eps_over_step >= 1e-30f;
  return flush_ok ? kAdamWFast : kAdamWSmall;
}

}  // namespace
}  // namespace dt8

using namespace dt8;

extern "C" {

const char* dt8_status_string(int status) {
  switch (status) {
    case DT8_OK: return "DT8_OK";
    case DT8_ERR_INVALID_ARG: return "DT8_ERR_INVALID_ARG: bad pointer, size, step, dtype or flag";
    case DT8_ERR_UNSUPPORTED: return "DT8_ERR_UNSUPPORTED: block size must be 256, 512, 1024, 2048 or 4096 (or the device cannot hold the shared-memory table layout)";
    case DT8_ERR_ALIGNMENT: return "DT8_ERR_ALIGNMENT: fp32 tensors need 16-byte, bf16 8-byte, codes and absmax 4-byte alignment";
    case DT8_ERR_CUDA: return "DT8_ERR_CUDA: a CUDA runtime call failed (see dt8_last_cuda_error)";
  }
  return "unknown dt8 status";
}

int dt8_last_cuda_error(void) { return tl_last_cuda_error; }

int dt8_codebook(int is_signed, float* out_host) {
  if (!out_host) return DT8_ERR_INVALID_ARG;
  build_codebook(is_signed != 0, out_host);
  return DT8_OK;
}

int64_t dt8_state_bytes(int64_t n, int block_size) {
  if (n < 0 || !block_size_ok(block_size)) return -1;
  return n + 4 * ((n + block_size - 1) / block_size);
}

int dt8_selfcheck_encode_host(int is_signed, const float* v_host, int64_t n, uint8_t* out_host) {
  if (n < 0 || (n > 0 && (!v_host || !out_host))) return DT8_ERR_INVALID_ARG;
  const Tables* ht = host_tables();
  if (!ht) return DT8_ERR_UNSUPPORTED;
  const EncTable& e = is_signed ? ht->enc_signed : ht->enc_unsigned;
  const EncBounds bounds = make_bounds(e.first_key, e.num_entries);
  const HostFetch fetch{e.entries, bounds.lo4};
  // groups of four, as the kernels do; the tail is padded with zeros
  for (int64_t i = 0; i < n; i += 4) {
    uint32_t bits[4] = {0, 0, 0, 0};
    const int cnt = static_cast<int>(n - i < 4 ? n - i : 4);
    std::memcpy(bits, v_host + i, 4 * static_cast<size_t>(cnt));
    uint32_t packed;
    if (is_signed) {
      packed = finish_signed4(lookup_signed<true>(fetch, bounds, bits[0]),
                              lookup_signed<true>(fetch, bounds, bits[1]),
                              lookup_signed<true>(fetch, bounds, bits[2]),
                              lookup_signed<true>(fetch, bounds, bits[3]), bits[0], bits[1], bits[2],
                              bits[3]);
    } else {
      packed = finish_unsigned4(lookup_unsigned<true>(fetch, bounds, bits[0]),
                                lookup_unsigned<true>(fetch, bounds, bits[1]),
                                lookup_unsigned<true>(fetch, bounds, bits[2]),
                                lookup_unsigned<true>(fetch, bounds, bits[3]));
    }
    for (int j = 0; j < cnt; ++j) out_host[i + j] = static_cast<uint8_t>(packed >> (8 * j));
  }
  return DT8_OK;
}

int dt8_init(void) {
  DeviceInfo di;
  EncMeta em;
  return ensure_device(&di, &em);
}

int dt8_selfcheck_divide(const float* s, const float* N, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!s || !N || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(s, 4) || !aligned(N, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  DeviceInfo di;
  EncMeta em;
  int rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * di.sm_count ? ctas : 8 * di.sm_count);
  divide_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(s, N, out, n);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_selfcheck_divide_const(const float* s, float d, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!s || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(s, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  DeviceInfo di;
  EncMeta em;
  int rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * di.sm_count ? ctas : 8 * di.sm_count);
  divide_const_kernel<<<grid, 256, 0, static_cast<cudaStream_t>(stream)>>>(s, make_const_divisor(d), out, n);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_quantize_blockwise(const float* x, int64_t n, int block_size, int is_signed, uint8_t* codes,
                           float* absmax, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  if (n == 0) return DT8_OK;
  if (!x || !codes || !absmax) return DT8_ERR_INVALID_ARG;
  if (!aligned(x, 16) || !aligned(codes, 4) || !aligned(absmax, 4)) return DT8_ERR_ALIGNMENT;
  DeviceInfo di;
  EncMeta em;
  int rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
#define DT8_Q_CASE(BS)                                                                  \
  case BS:                                                                              \
    return is_signed ? launch_quantize<BS, true>(x, n, codes, absmax, em, di, s)        \
                     : launch_quantize<BS, false>(x, n, codes, absmax, em, di, s);
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

int dt8_dequantize_blockwise(const uint8_t* codes, const float* absmax, int64_t n, int block_size,
                             int is_signed, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  if (n == 0) return DT8_OK;
  if (!codes || !absmax || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(out, 16) || !aligned(codes, 4) || !aligned(absmax, 4)) return DT8_ERR_ALIGNMENT;
  DeviceInfo di;
  EncMeta em;
  int rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int64_t quads = (n + 3) / 4;
  const int64_t per_cta = static_cast<int64_t>(kDeqThreads) * kDeqUnroll;
  const int64_t ctas = (quads + per_cta - 1) / per_cta;
  const int64_t resident = static_cast<int64_t>(kDeqCtasPerSm) * di.sm_count;
  const int grid = static_cast<int>(ctas < resident ? ctas : resident);
  const int shift = log2_int(block_size);
  if (is_signed)
    dequantize_kernel<true><<<grid, kDeqThreads, kDeqSmemBytes, s>>>(codes, absmax, out, n, shift);
  else
    dequantize_kernel<false><<<grid, kDeqThreads, kDeqSmemBytes, s>>>(codes, absmax, out, n, shift);
  const cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_sgd_step(float* p, const void* g, int g_dtype, uint8_t* m_codes, float* m_absmax, int64_t n,
                 float lr, float momentum, float weight_decay, int64_t step, int block_size,
                 void* stream) {
  if (g_dtype != DT8_F32 && g_dtype != DT8_BF16) return DT8_ERR_INVALID_ARG;
  if (step < 1 || !sgd_hyper_ok(lr, momentum, weight_decay)) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  SingleArgs a;
  a.t = TensorDesc{p, g, m_codes, m_absmax, nullptr, nullptr, n};
  int rc = check_tensor(a.t, g_dtype, false);
  if (rc != DT8_OK || n == 0) return rc;
  a.nb = (n + block_size - 1) / block_size;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  DeviceInfo di;
  EncMeta em;
  rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  const SgdHyper h{lr, momentum, weight_decay};
  return dispatch_sgd_b(a, a.nb, block_size, g_dtype, h, em, di, static_cast<cudaStream_t>(stream));
}

int dt8_adam_step(float* p, const void* g, int g_dtype, uint8_t* m_codes, float* m_absmax,
                  uint8_t* r_codes, float* r_absmax, int64_t n, float lr, float beta1, float beta2,
                  float eps, float weight_decay, int64_t step, int block_size, uint32_t flags,
                  void* stream) {
  if (g_dtype != DT8_F32 && g_dtype != DT8_BF16) return DT8_ERR_INVALID_ARG;
  if (step < 1 || (flags & ~3u)) return DT8_ERR_INVALID_ARG;
  if (!adam_hyper_ok(lr, beta1, beta2, eps, weight_decay)) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  SingleArgs a;
  a.t = TensorDesc{p, g, m_codes, m_absmax, r_codes, r_absmax, n};
  int rc = check_tensor(a.t, g_dtype, true);
  if (rc != DT8_OK || n == 0) return rc;
  a.nb = (n + block_size - 1) / block_size;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  DeviceInfo di;
  EncMeta em;
  rc = ensure_device(&di, &em);
  if (rc != DT8_OK) return rc;
  const AdamHyper h = make_adam_hyper(lr, beta1, beta2, eps, weight_decay, step, flags);
  return dispatch_adam_b(a, a.nb, block_size, g_dtype, adam_mode(flags, h), h, em, di,
                         static_cast<cudaStream_t>(stream));
}

}  // extern "C"

namespace dt8 {
namespace {

// Shared front end of the two pointer-list entry points: validates every tensor first (so that a
// bad entry means nothing was launched), then launches one kernel per kMaxTensorsPerLaunch
// non-empty tensors.  Every tensor that passed the checks fits a launch of its own, so after the
// checks only the CUDA runtime can fail (DT8_ERR_CUDA), possibly after earlier launches of the
// same call were queued.
template <class Launch>
int run_multi(int num_tensors, float* const* p, const void* const* g, int g_dtype,
              uint8_t* const* mc, float* const* ma, uint8_t* const* rc, float* const* ra,
              const int64_t* n, int block_size, bool adam, Launch launch) {
  if (num_tensors < 0) return DT8_ERR_INVALID_ARG;
  if (g_dtype != DT8_F32 && g_dtype != DT8_BF16) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  if (num_tensors == 0) return DT8_OK;
  if (!p || !g || !mc || !ma || !n || (adam && (!rc || !ra))) return DT8_ERR_INVALID_ARG;
  for (int i = 0; i < num_tensors; ++i) {
    const TensorDesc d{p[i], g[i], mc[i], ma[i], adam ? rc[i] : nullptr, adam ? ra[i] : nullptr, n[i]};
    const int st = check_tensor(d, g_dtype, adam);
    if (st != DT8_OK) return st;
    if ((n[i] + block_size - 1) / block_size > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  }
  DeviceInfo di;
  EncMeta em;
  int st = ensure_device(&di, &em);
  if (st != DT8_OK) return st;
  static thread_local MultiArgs args;
  int i = 0;
  while (i < num_tensors) {
    args.num = 0;
    args.blk_start[0] = 0;
    int64_t blocks = 0;
    while (i < num_tensors && args.num < kMaxTensorsPerLaunch) {
      if (n[i] > 0) {
        const int64_t nb = (n[i] + block_size - 1) / block_size;
        if (blocks + nb > kMaxBlocksPerLaunch) break;   // args.num > 0 here: nb alone fits
        args.t[args.num] = TensorDesc{p[i], g[i], mc[i], ma[i], adam ? rc[i] : nullptr,
                                      adam ? ra[i] : nullptr, n[i]};
        blocks += nb;
        args.blk_start[++args.num] = static_cast<int>(blocks);
      }
      ++i;
    }
    if (args.num == 0) continue;
    st = launch(args, blocks, em, di);
    if (st != DT8_OK) return st;
  }
  return DT8_OK;
}

}  // namespace
}  // namespace dt8

extern "C" {

int dt8_sgd_step_multi(int num_tensors, float* const* p, const void* const* g, int g_dtype,
                       uint8_t* const* m_codes, float* const* m_absmax, const int64_t* n, float lr,
                       float momentum, float weight_decay, int64_t step, int block_size,
                       void* stream) {
  if (step < 1 || !sgd_hyper_ok(lr, momentum, weight_decay)) return DT8_ERR_INVALID_ARG;
  const SgdHyper h{lr, momentum, weight_decay};
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return run_multi(num_tensors, p, g, g_dtype, m_codes, m_absmax, nullptr, nullptr, n, block_size,
                   false, [&](const MultiArgs& a, int64_t blocks, const EncMeta& em, const DeviceInfo& di) {
                     return dispatch_sgd_b(a, blocks, block_size, g_dtype, h, em, di, s);
                   });
}

int dt8_adam_step_multi(int num_tensors, float* const* p, const void* const* g, int g_dtype,
                        uint8_t* const* m_codes, float* const* m_absmax, uint8_t* const* r_codes,
                        float* const* r_absmax, const int64_t* n, float lr, float beta1, float beta2,
                        float eps, float weight_decay, int64_t step, int block_size, uint32_t flags,
                        void* stream) {
  if (step < 1 || (flags & ~3u)) return DT8_ERR_INVALID_ARG;
  if (!adam_hyper_ok(lr, beta1, beta2, eps, weight_decay)) return DT8_ERR_INVALID_ARG;
  const AdamHyper h = make_adam_hyper(lr, beta1, beta2, eps, weight_decay, step, flags);
  const int mode = adam_mode(flags, h);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  return run_multi(num_tensors, p, g, g_dtype, m_codes, m_absmax, r_codes, r_absmax, n, block_size,
                   true, [&](const MultiArgs& a, int64_t blocks, const EncMeta& em, const DeviceInfo& di) {
                     return dispatch_adam_b(a, blocks, block_size, g_dtype, mode, h, em, di, s);
                   });
}

}  // extern "C"
