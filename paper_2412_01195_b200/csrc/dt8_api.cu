// C ABI of the dt8 library: argument checks, table upload and the calls into the launchers of
// the other translation units.
#include <cuda_runtime.h>

#include <atomic>
#include <cmath>
#include <cstring>
#include <initializer_list>
#include <mutex>

#include "dt8.h"
#include "dt8_launch.h"

namespace dt8 {

namespace {
thread_local int tl_last_cuda_error = 0;
}  // namespace

int cuda_fail(cudaError_t e) {
  tl_last_cuda_error = static_cast<int>(e);
  return DT8_ERR_CUDA;
}

namespace {

// The constant tables, one copy per device (this translation unit owns them; the kernels of the
// other units receive the address).
__device__ DeviceTables g_tables;

// Shared-memory address at which a kernel's dynamic shared memory starts, written by
// smem_start_probe and read back once per device.
__device__ uint32_t g_smem_start;

__global__ void smem_start_probe() {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  if (threadIdx.x == 0) g_smem_start = static_cast<uint32_t>(__cvta_generic_to_shared(smem_raw));
}

// Diagnostic: s_i / d by the constant-divisor routine of the IEEE Adam update.
__global__ void __launch_bounds__(256)
divide_const_kernel(const float* __restrict__ s, ConstDivisor cd, float* __restrict__ out, int64_t n) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride)
  {
    const float a = fabsf(s[i]);
    const bool fast = cd.usable && a >= kConstDivMinDividend && a <= kConstDivMaxDividend;
    // the packed form the step kernel uses (both lanes carry the same dividend here)
    out[i] = fast ? lo2(cd.div2<true>(pack2(s[i], s[i]))) : cd.div<false>(s[i]);
  }
}

// Diagnostic: the normalising division of the encoder applied to arbitrary operand pairs.
__global__ void __launch_bounds__(256)
divide_kernel(const float* __restrict__ s, const float* __restrict__ N, float* __restrict__ out,
              int64_t n) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const Normaliser nz(N[i]);
    out[i] = nz.fast ? nz.div<true>(s[i]) : nz.div<false>(s[i]);
  }
}

// Diagnostic: the square root of the fast IEEE parameter update.
__global__ void __launch_bounds__(256)
root_kernel(const float* __restrict__ x, float* __restrict__ out, int64_t n) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const float v = x[i];
    out[i] = (v >= kFastRootMin && v <= kFastRootMax) ? sqrt_rn_inrange(v) : 0.0f;
  }
}

// Diagnostic: the reciprocal the normalising division starts from.
__global__ void __launch_bounds__(256)
reciprocal_kernel(const float* __restrict__ N, float* __restrict__ out, int64_t n) {
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += stride) {
    const Normaliser nz(N[i]);
    out[i] = nz.fast ? nz.rN : 0.0f;
  }
}

constexpr int kMaxDevices = 64;

std::mutex g_init_mutex;
std::atomic<bool> g_uploaded[kMaxDevices];
int g_sm_count[kMaxDevices];
const DeviceTables* g_tables_addr[kMaxDevices];

// Makes sure the current device holds the constant tables and fills the launch context.
int ensure_device(LaunchCtx* ctx, void* stream) {
  const Tables* ht = host_tables();
  if (!ht) return DT8_ERR_UNSUPPORTED;
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e);
  if (dev < 0 || dev >= kMaxDevices) return DT8_ERR_UNSUPPORTED;
  EncMeta em;
  em.s_first = ht->enc_signed.first_key;
  em.u_first = ht->enc_unsigned.first_key;
  em.s_n = ht->enc_signed.num_entries;
  em.u_n = ht->enc_unsigned.num_entries;
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
      // the shared-memory image of the step kernels: encode tables at their byte addresses (the
      // unsigned one shifted by kEncUOffset), decode tables replicated once per lane
      std::memset(staging.image, 0, sizeof(staging.image));
      if (layout_ok(em)) {
        const EncBounds bs = make_bounds(em.s_first, em.s_n), bu = make_bounds(em.u_first, em.u_n);
        uint32_t* img = staging.image;
        for (int i = 0; i < em.s_n; ++i) img[(bs.lo4 - kImageBase) / 4 + i] = staging.enc_s[i];
        for (int i = 0; i < em.u_n; ++i)
          img[(static_cast<int64_t>(bu.lo4) + kEncUOffset - kImageBase) / 4 + i] = staging.enc_u[i];
        for (int i = 0; i < 256 * 64; ++i) {   // code = i / 64, table = (i / 32) % 2, lane = i % 32
          const float v = (i & 32) ? staging.dec_u[i >> 6] : staging.dec_s[i >> 6];
          std::memcpy(&img[(kDecodeAddr - kImageBase) / 4 + i], &v, 4);
        }
      }
      e = cudaMemcpyToSymbol(g_tables, &staging, sizeof(staging));
      if (e != cudaSuccess) return cuda_fail(e);
      void* addr = nullptr;
      e = cudaGetSymbolAddress(&addr, g_tables);
      if (e != cudaSuccess) return cuda_fail(e);
      // The kernels address their shared-memory tables absolutely: check once that this build's
      // tables fit the layout and that dynamic shared memory starts low enough on this device.
      if (!layout_ok(em)) return DT8_ERR_UNSUPPORTED;
      const int probe_smem = static_cast<int>(smem_bytes(em, true, true, true, true));
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
      g_tables_addr[dev] = static_cast<const DeviceTables*>(addr);
      g_uploaded[dev].store(true, std::memory_order_release);
    }
  }
  ctx->device = dev;
  ctx->sm_count = g_sm_count[dev];
  ctx->em = em;
  ctx->tables = g_tables_addr[dev];
  ctx->stream = static_cast<cudaStream_t>(stream);
  return DT8_OK;
}

bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }

bool block_size_ok(int B) { return B == 256 || B == 512 || B == 1024 || B == 2048 || B == 4096; }

bool dtype_ok(int d) { return d == DT8_F32 || d == DT8_BF16; }

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

int check_tensor(const TensorDesc& d, int p_dtype, int g_dtype, bool adam) {
  if (d.n < 0) return DT8_ERR_INVALID_ARG;
  if (d.n == 0) return DT8_OK;
  if (!d.p || !d.g || !d.mc || !d.ma) return DT8_ERR_INVALID_ARG;
  if (adam && (!d.rc || !d.ra)) return DT8_ERR_INVALID_ARG;
  if (!aligned(d.p, p_dtype == DT8_F32 ? 16 : 8) || !aligned(d.g, g_dtype == DT8_F32 ? 16 : 8) ||
      !aligned(d.mc, 4) || !aligned(d.ma, 4))
    return DT8_ERR_ALIGNMENT;
  if (adam && (!aligned(d.rc, 4) || !aligned(d.ra, 4))) return DT8_ERR_ALIGNMENT;
  return DT8_OK;
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
  h.const_div = (d1.usable && d2.usable && eps <= kFastUpdateMaxEps) ? 1 : 0;
  h.neg_zero = -0.0f;
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

template <class Args>
static int launch_adam_any(const Args& a, int64_t blocks, int block_size, int p_dtype, int g_dtype,
                           int mode, const AdamHyper& h, const LaunchCtx& ctx) {
  const bool gb = g_dtype == DT8_BF16, pb = p_dtype == DT8_BF16;
  if (gb && pb) return launch_adam_typed<true, true, Args>(a, blocks, block_size, mode, h, ctx);
  if (gb) return launch_adam_typed<true, false, Args>(a, blocks, block_size, mode, h, ctx);
  if (pb) return launch_adam_typed<false, true, Args>(a, blocks, block_size, mode, h, ctx);
  return launch_adam_typed<false, false, Args>(a, blocks, block_size, mode, h, ctx);
}

int launch_adam(const SingleArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype, int mode,
                const AdamHyper& h, const LaunchCtx& ctx) {
  return launch_adam_any(a, blocks, block_size, p_dtype, g_dtype, mode, h, ctx);
}

int launch_adam(const MultiArgs& a, int64_t blocks, int block_size, int p_dtype, int g_dtype, int mode,
                const AdamHyper& h, const LaunchCtx& ctx) {
  return launch_adam_any(a, blocks, block_size, p_dtype, g_dtype, mode, h, ctx);
}

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


int dt8_selfcheck_layout_fits(uint32_t s_first, int s_entries, uint32_t u_first, int u_entries) {
  if (s_entries < 1 || u_entries < 1 || s_first < 1 || u_first < 1) return 0;
  EncMeta em;
  em.s_first = s_first;
  em.u_first = u_first;
  em.s_n = s_entries;
  em.u_n = u_entries;
  return layout_ok(em) ? 1 : 0;
}

int dt8_selfcheck_table_extents(uint32_t* s_first, int* s_entries, uint32_t* u_first, int* u_entries) {
  const Tables* ht = host_tables();
  if (!ht || !s_first || !s_entries || !u_first || !u_entries) return DT8_ERR_INVALID_ARG;
  *s_first = ht->enc_signed.first_key;
  *s_entries = ht->enc_signed.num_entries;
  *u_first = ht->enc_unsigned.first_key;
  *u_entries = ht->enc_unsigned.num_entries;
  return DT8_OK;
}

int dt8_init(void) {
  LaunchCtx ctx;
  return ensure_device(&ctx, nullptr);
}

int dt8_selfcheck_divide(const float* s, const float* N, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!s || !N || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(s, 4) || !aligned(N, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * ctx.sm_count ? ctas : 8 * ctx.sm_count);
  divide_kernel<<<grid, 256, 0, ctx.stream>>>(s, N, out, n);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_selfcheck_reciprocal(const float* N, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!N || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(N, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * ctx.sm_count ? ctas : 8 * ctx.sm_count);
  reciprocal_kernel<<<grid, 256, 0, ctx.stream>>>(N, out, n);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_selfcheck_root(const float* x, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!x || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(x, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * ctx.sm_count ? ctas : 8 * ctx.sm_count);
  root_kernel<<<grid, 256, 0, ctx.stream>>>(x, out, n);
  cudaError_t e = cudaGetLastError();
  return e == cudaSuccess ? DT8_OK : cuda_fail(e);
}

int dt8_selfcheck_divide_const(const float* s, float d, int64_t n, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (n == 0) return DT8_OK;
  if (!s || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(s, 4) || !aligned(out, 4)) return DT8_ERR_ALIGNMENT;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const int64_t ctas = (n + 255) / 256;
  const int grid = static_cast<int>(ctas < 8 * ctx.sm_count ? ctas : 8 * ctx.sm_count);
  divide_const_kernel<<<grid, 256, 0, ctx.stream>>>(s, make_const_divisor(d), out, n);
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
  if ((n + block_size - 1) / block_size > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  return launch_quantize(x, n, block_size, is_signed, codes, absmax, ctx);
}

int dt8_dequantize_blockwise(const uint8_t* codes, const float* absmax, int64_t n, int block_size,
                             int is_signed, float* out, void* stream) {
  if (n < 0) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  if (n == 0) return DT8_OK;
  if (!codes || !absmax || !out) return DT8_ERR_INVALID_ARG;
  if (!aligned(out, 16) || !aligned(codes, 4) || !aligned(absmax, 4)) return DT8_ERR_ALIGNMENT;
  LaunchCtx ctx;
  int rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  return launch_dequantize(codes, absmax, n, block_size, is_signed, out, ctx);
}

int dt8_sgd_step_ex(void* p, int p_dtype, const void* g, int g_dtype, uint8_t* m_codes,
                    float* m_absmax, int64_t n, float lr, float momentum, float weight_decay,
                    int64_t step, int block_size, void* stream) {
  if (!dtype_ok(g_dtype) || !dtype_ok(p_dtype)) return DT8_ERR_INVALID_ARG;
  if (step < 1 || !sgd_hyper_ok(lr, momentum, weight_decay)) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  SingleArgs a;
  a.t = TensorDesc{p, g, m_codes, m_absmax, nullptr, nullptr, n};
  int rc = check_tensor(a.t, p_dtype, g_dtype, false);
  if (rc != DT8_OK || n == 0) return rc;
  a.nb = (n + block_size - 1) / block_size;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  LaunchCtx ctx;
  rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const SgdHyper h{lr, momentum, weight_decay, -0.0f};
  return launch_sgd(a, a.nb, block_size, p_dtype, g_dtype, h, ctx);
}

int dt8_sgd_step(float* p, const void* g, int g_dtype, uint8_t* m_codes, float* m_absmax, int64_t n,
                 float lr, float momentum, float weight_decay, int64_t step, int block_size,
                 void* stream) {
  return dt8_sgd_step_ex(p, DT8_F32, g, g_dtype, m_codes, m_absmax, n, lr, momentum, weight_decay,
                         step, block_size, stream);
}

int dt8_adam_step_ex(void* p, int p_dtype, const void* g, int g_dtype, uint8_t* m_codes,
                     float* m_absmax, uint8_t* r_codes, float* r_absmax, int64_t n, float lr,
                     float beta1, float beta2, float eps, float weight_decay, int64_t step,
                     int block_size, uint32_t flags, void* stream) {
  if (!dtype_ok(g_dtype) || !dtype_ok(p_dtype)) return DT8_ERR_INVALID_ARG;
  if (step < 1 || (flags & ~3u)) return DT8_ERR_INVALID_ARG;
  if (!adam_hyper_ok(lr, beta1, beta2, eps, weight_decay)) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  SingleArgs a;
  a.t = TensorDesc{p, g, m_codes, m_absmax, r_codes, r_absmax, n};
  int rc = check_tensor(a.t, p_dtype, g_dtype, true);
  if (rc != DT8_OK || n == 0) return rc;
  a.nb = (n + block_size - 1) / block_size;
  if (a.nb > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  LaunchCtx ctx;
  rc = ensure_device(&ctx, stream);
  if (rc != DT8_OK) return rc;
  const AdamHyper h = make_adam_hyper(lr, beta1, beta2, eps, weight_decay, step, flags);
  return launch_adam(a, a.nb, block_size, p_dtype, g_dtype, adam_mode(flags, h), h, ctx);
}

int dt8_adam_step(float* p, const void* g, int g_dtype, uint8_t* m_codes, float* m_absmax,
                  uint8_t* r_codes, float* r_absmax, int64_t n, float lr, float beta1, float beta2,
                  float eps, float weight_decay, int64_t step, int block_size, uint32_t flags,
                  void* stream) {
  return dt8_adam_step_ex(p, DT8_F32, g, g_dtype, m_codes, m_absmax, r_codes, r_absmax, n, lr, beta1,
                          beta2, eps, weight_decay, step, block_size, flags, stream);
}

}  // extern "C"

namespace dt8 {
namespace {

// Shared front end of the pointer-list entry points: validates every tensor first (so that a
// bad entry means nothing was launched), then launches one kernel per kMaxTensorsPerLaunch
// non-empty tensors.  Every tensor that passed the checks fits a launch of its own, so after the
// checks only the CUDA runtime can fail (DT8_ERR_CUDA), possibly after earlier launches of the
// same call were queued.
template <class Launch>
int run_multi(int num_tensors, void* const* p, int p_dtype, const void* const* g, int g_dtype,
              uint8_t* const* mc, float* const* ma, uint8_t* const* rc, float* const* ra,
              const int64_t* n, int block_size, bool adam, void* stream, Launch launch) {
  if (num_tensors < 0) return DT8_ERR_INVALID_ARG;
  if (!dtype_ok(g_dtype) || !dtype_ok(p_dtype)) return DT8_ERR_INVALID_ARG;
  if (!block_size_ok(block_size)) return DT8_ERR_UNSUPPORTED;
  if (num_tensors == 0) return DT8_OK;
  if (!p || !g || !mc || !ma || !n || (adam && (!rc || !ra))) return DT8_ERR_INVALID_ARG;
  for (int i = 0; i < num_tensors; ++i) {
    const TensorDesc d{p[i], g[i], mc[i], ma[i], adam ? rc[i] : nullptr, adam ? ra[i] : nullptr, n[i]};
    const int st = check_tensor(d, p_dtype, g_dtype, adam);
    if (st != DT8_OK) return st;
    if ((n[i] + block_size - 1) / block_size > kMaxBlocksPerLaunch) return DT8_ERR_UNSUPPORTED;
  }
  LaunchCtx ctx;
  int st = ensure_device(&ctx, stream);
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
    st = launch(args, blocks, ctx);
    if (st != DT8_OK) return st;
  }
  return DT8_OK;
}

}  // namespace
}  // namespace dt8

extern "C" {

int dt8_sgd_step_multi_ex(int num_tensors, void* const* p, int p_dtype, const void* const* g,
                          int g_dtype, uint8_t* const* m_codes, float* const* m_absmax,
                          const int64_t* n, float lr, float momentum, float weight_decay,
                          int64_t step, int block_size, void* stream) {
  if (step < 1 || !sgd_hyper_ok(lr, momentum, weight_decay)) return DT8_ERR_INVALID_ARG;
  const SgdHyper h{lr, momentum, weight_decay, -0.0f};
  return run_multi(num_tensors, p, p_dtype, g, g_dtype, m_codes, m_absmax, nullptr, nullptr, n,
                   block_size, false, stream,
                   [&](const MultiArgs& a, int64_t blocks, const LaunchCtx& ctx) {
                     return launch_sgd(a, blocks, block_size, p_dtype, g_dtype, h, ctx);
                   });
}

int dt8_sgd_step_multi(int num_tensors, float* const* p, const void* const* g, int g_dtype,
                       uint8_t* const* m_codes, float* const* m_absmax, const int64_t* n, float lr,
                       float momentum, float weight_decay, int64_t step, int block_size,
                       void* stream) {
  return dt8_sgd_step_multi_ex(num_tensors, reinterpret_cast<void* const*>(p), DT8_F32, g, g_dtype,
                               m_codes, m_absmax, n, lr, momentum, weight_decay, step, block_size,
                               stream);
}

int dt8_adam_step_multi_ex(int num_tensors, void* const* p, int p_dtype, const void* const* g,
                           int g_dtype, uint8_t* const* m_codes, float* const* m_absmax,
                           uint8_t* const* r_codes, float* const* r_absmax, const int64_t* n,
                           float lr, float beta1, float beta2, float eps, float weight_decay,
                           int64_t step, int block_size, uint32_t flags, void* stream) {
  if (step < 1 || (flags & ~3u)) return DT8_ERR_INVALID_ARG;
  if (!adam_hyper_ok(lr, beta1, beta2, eps, weight_decay)) return DT8_ERR_INVALID_ARG;
  const AdamHyper h = make_adam_hyper(lr, beta1, beta2, eps, weight_decay, step, flags);
  const int mode = adam_mode(flags, h);
  return run_multi(num_tensors, p, p_dtype, g, g_dtype, m_codes, m_absmax, r_codes, r_absmax, n,
                   block_size, true, stream,
                   [&](const MultiArgs& a, int64_t blocks, const LaunchCtx& ctx) {
                     return launch_adam(a, blocks, block_size, p_dtype, g_dtype, mode, h, ctx);
                   });
}

int dt8_adam_step_multi(int num_tensors, float* const* p, const void* const* g, int g_dtype,
                        uint8_t* const* m_codes, float* const* m_absmax, uint8_t* const* r_codes,
                        float* const* r_absmax, const int64_t* n, float lr, float beta1, float beta2,
                        float eps, float weight_decay, int64_t step, int block_size, uint32_t flags,
                        void* stream) {
  return dt8_adam_step_multi_ex(num_tensors, reinterpret_cast<void* const*>(p), DT8_F32, g, g_dtype,
                                m_codes, m_absmax, r_codes, r_absmax, n, lr, beta1, beta2, eps,
                                weight_decay, step, block_size, flags, stream);
}

}  // extern "C"
