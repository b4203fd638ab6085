/*
 * dt8 -- fused 8-bit optimizer step over the dynamic-tree 8-bit data type (CUDA, sm_100a).
 *
 * C ABI of the library.  Plain pointers and sizes only; no framework types.
 *
 * The method is Section IV of "Memory-Efficient Training for Deep Speaker Embedding Learning
 * in Speaker Verification" (arXiv 2412.01195): optimizer states are stored as uint8 indices into
 * a 256-entry code book with one fp32 absolute maximum per block of B elements; a step
 * dequantizes the states to 32-bit, applies the 32-bit SGD-momentum / Adam update to the
 * parameters, and quantizes the new states back (Section I; Section IV-B; Eq. sgd, Eq. adam,
 * Eq. quant1, quant2, quant3).
 *
 * Conventions shared by every entry point
 *   - Return value: a dt8_status.  On any status other than DT8_OK nothing was launched and no
 *     caller buffer was written, with one exception: a pointer-list call that needs several
 *     launches (more than 256 tensors) can return DT8_ERR_CUDA from a later launch after the
 *     earlier ones were queued.  Every argument check is made before the first launch.
 *   - "device" pointers are CUDA device pointers of the current device, owned by the caller and
 *     valid until the work queued on `stream` has run.  "host" pointers are ordinary host memory.
 *   - Calls are asynchronous on `stream` (a cudaStream_t passed as void*; NULL is the default
 *     stream).  They never synchronise and never allocate device memory.
 *   - The first call on a device (or dt8_init) uploads the constant tables of the data type with
 *     a blocking copy and runs a one-warp probe kernel on the default stream that reports where
 *     dynamic shared memory starts (the kernels keep their tables at fixed shared-memory
 *     addresses); make that call outside any stream capture.  A device on which the layout does
 *     not fit gives DT8_ERR_UNSUPPORTED.
 *   - Layout: a tensor is a flat array of n elements, cut into nb = ceil(n / block_size) blocks;
 *     block b covers elements [b*block_size, min(n, (b+1)*block_size)).  `codes` holds n bytes,
 *     `absmax` holds nb floats (Section IV-B, "Tensor chunking").  Blocks never span tensors.
 *   - block_size is one of 256, 512, 1024, 2048, 4096 (the paper uses 2048), else
 *     DT8_ERR_UNSUPPORTED.  A tensor may have at most 2^31 - 2^16 blocks (4.4e12 elements at
 *     block_size 2048), in the single-tensor and the pointer-list forms alike, else
 *     DT8_ERR_UNSUPPORTED.
 *   - Alignment: fp32 tensors 16 bytes, bf16 tensors 8 bytes, code arrays 4 bytes, absmax arrays
 *     4 bytes, at each tensor's base; else DT8_ERR_ALIGNMENT.  Nothing more is assumed: a code
 *     array at a 4-byte-only offset or a parameter tensor at a 16-byte-only offset is fine.
 *   - n == 0 (or num_tensors == 0) is a successful no-op.  n < 0, a NULL tensor pointer with
 *     n > 0, step < 1, or an unknown dtype / flag gives DT8_ERR_INVALID_ARG.  So do non-finite
 *     hyper-parameters, beta1 or beta2 outside [0, 1), a negative eps and a negative momentum.
 *   - A state whose absmax entries are all 0 is the zero state (Eq. adam: r_0 = m_0 = 0); its code
 *     bytes are then ignored on input.
 *   - Codes are indices into the ASCENDING table (Section IV-B, "Indexing").
 *     The signed table has two zero entries, 127 and 128; the quantizer emits 127.
 *   - Arithmetic: everything that decides a code -- dequantized state, new state, block maximum,
 *     normalised value -- is computed in IEEE binary32, one rounding per written operation, no
 *     fused multiply-add, true division by the block maximum.
 *   - Non-finite inputs are outside the contract; they cannot cause an out-of-bounds access.
 */
#ifndef DT8_H_
#define DT8_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  DT8_OK = 0,
  DT8_ERR_INVALID_ARG = 1,
  DT8_ERR_UNSUPPORTED = 2,
  DT8_ERR_ALIGNMENT = 3,
  DT8_ERR_CUDA = 4
} dt8_status;

/* Element type of gradients and, in the _ex entry points, of parameters. */
typedef enum { DT8_F32 = 0, DT8_BF16 = 1 } dt8_dtype;

/* Flags of dt8_adam_step.  The default used by the Python binding is both bits set (AdamW with
 * bias correction, the optimizer the paper trains its DF-ResNets with, Section V).  With both
 * bits clear and weight_decay = 0 the update is Eq. adam exactly as printed. */
enum {
  DT8_ADAM_BIAS_CORRECTION = 1, /* divide m by 1-beta1^step and r by 1-beta2^step          */
  DT8_ADAM_DECOUPLED_WD = 2     /* w <- w(1 - lr*wd) (AdamW); clear: g <- g + wd*w (L2)     */
};

/* Human-readable name of a status code (static storage, never NULL). */
const char *dt8_status_string(int status);

/* Last CUDA error code (a cudaError_t as int) seen by a call that returned DT8_ERR_CUDA on this
 * host thread, 0 if none. */
int dt8_last_cuda_error(void);

/*
 * Code book of the dynamic-tree 8-bit data type (Section IV-B, "Nearest value searching",
 * Fig. dynamic_tree): sign bit, a run of E zero bits = decimal exponent 10^-E, an indicator bit,
 * and F fraction bits holding k, with value 10^-E * (0.1 + 0.9*(k+1)/2^F), rounded to binary32.
 * is_signed != 0: 7-bit magnitude behind a sign bit, values in [-1, 1], used for the momentum and
 * the Adam first moment.  is_signed == 0: 8-bit magnitude, values in [0, 1], used for the Adam
 * second moment.  Pure host function; writes 256 ascending floats to out_host (host memory).
 * DT8_ERR_INVALID_ARG if out_host is NULL.
 */
int dt8_codebook(int is_signed, float *out_host);

/*
 * Bytes of one 8-bit state of n elements: n code bytes plus one binary32 maximum per block
 * (Section IV-B, "Tensor chunking"), i.e. n + 4*ceil(n / block_size); a 32-bit state takes 4*n
 * (Section I: 4 bytes per weight for SGD, 8 for Adam's two states), which is where the paper's
 * "75 %" saving comes from (74.95 % at block_size 2048).  Pure host function.  Returns -1 for
 * n < 0 or an unsupported block_size.
 */
int64_t dt8_state_bytes(int64_t n, int block_size);

/*
 * Diagnostic, host only: runs the kernels' table-driven nearest-code search (the device code of
 * Eq. quant2, compiled for the host) on n already-normalised values in host memory and writes the
 * codes to out_host.  It exists so that the encode tables can be checked without a GPU; no step,
 * quantize or dequantize call uses it.
 */
int dt8_selfcheck_encode_host(int is_signed, const float *v_host, int64_t n, uint8_t *out_host);

/*
 * Diagnostic, device: out_i = s_i / N_i computed by the routine the kernels use for Eq. quant1's
 * normalisation (a correctly rounded reciprocal of N and a residual correction; the IEEE division
 * when N is 0 or outside 2^-76 .. 2^100).  The method needs the correctly rounded quotient for
 * |s_i| <= N_i; this entry point lets a test compare the routine with the true quotient on
 * operands of its choice.  No step, quantize or dequantize call uses it.
 *   s, N   device, const float[n];   out  device, float[n]
 */
int dt8_selfcheck_divide(const float *s, const float *N, int64_t n, float *out, void *stream);

/*
 * Diagnostic, device: out_i = the reciprocal of N_i that the routine above starts from (Eq. quant1:
 * one reciprocal per block, then one multiply and two fused multiply-adds per element).  The
 * residual correction is exact only when that reciprocal is the correctly rounded one, so a test
 * checks it for every binary32 mantissa.  out_i = 0 where the routine takes the IEEE division
 * instead (N_i = 0 included).  No step, quantize or dequantize call uses it.
 *   N  device, const float[n];   out  device, float[n]
 */
int dt8_selfcheck_reciprocal(const float *N, int64_t n, float *out, void *stream);

/*
 * Diagnostic, device: out_i = the square root of x_i as the IEEE form of the Adam parameter
 * update (Eq. adam, the root of the bias-corrected second moment) computes it when its operands
 * are in range: a reciprocal-root approximation and one fused correction, which must be the
 * correctly rounded root.  It depends on the mantissa and the parity of the exponent alone, so a
 * test checks all 2^24 cases.  out_i = 0 for x_i outside 2^-80 .. 2^80, where the step uses the
 * IEEE root instead.  No step, quantize or dequantize call uses it.
 *   x  device, const float[n];   out  device, float[n]
 */
int dt8_selfcheck_root(const float *x, int64_t n, float *out, void *stream);

/*
 * Diagnostic, device: out_i = s_i / d computed by the routine the IEEE form of the Adam parameter
 * update uses for Eq. adam's bias corrections m'/(1 - beta1^step), r'/(1 - beta2^step), whose
 * divisor is one number per launch: the host supplies the correctly rounded reciprocal of d and
 * the kernel corrects the product with two fused multiply-adds; for d outside 2^-20 .. 2^20 or
 * |s_i| outside 2^-60 .. 2^60 (zero included) it is the IEEE division.  The result must equal the
 * correctly rounded quotient; this entry point lets a test check that on divisors and dividends
 * of its choice.  No step, quantize or dequantize call uses it.
 *   s  device, const float[n];   d  the divisor;   out  device, float[n]
 */
int dt8_selfcheck_divide_const(const float *s, float d, int64_t n, float *out, void *stream);

/*
 * Diagnostics, host only.  The kernels keep their encode tables at fixed shared-memory addresses
 * (the table of bucket key k at byte 4*k, the unsigned one shifted below the signed one), so a
 * table set must fit between the reduction scratch and the decode tables without overlap; the
 * library checks that once per device and answers DT8_ERR_UNSUPPORTED otherwise.
 * dt8_selfcheck_table_extents writes the first bucket key and the number of entries of this
 * build's signed and unsigned encode tables; dt8_selfcheck_layout_fits answers 1 if tables of the
 * given extents fit the layout and 0 if not (a test can so see the check refuse).
 */
int dt8_selfcheck_table_extents(uint32_t *s_first, int *s_entries, uint32_t *u_first, int *u_entries);
int dt8_selfcheck_layout_fits(uint32_t s_first, int s_entries, uint32_t u_first, int u_entries);

/* Optional: upload the constant tables to the current device now (otherwise the first call does
 * it).  Blocking; call outside stream capture. */
int dt8_init(void);

/*
 * Block-wise quantization (Eq. quant1 + quant2).  For every block: absmax[b] = max |x_i|;
 * v_i = x_i / absmax[b] (0 for an all-zero block); codes_i = index of the table value nearest to
 * v_i, the lower index on an exact tie.  With the unsigned table negative inputs map to code 0.
 *   x       device, const float[n]         input
 *   codes   device, uint8_t[n]             output
 *   absmax  device, float[ceil(n/B)]       output
 */
int dt8_quantize_blockwise(const float *x, int64_t n, int block_size, int is_signed,
                           uint8_t *codes, float *absmax, void *stream);

/*
 * Block-wise dequantization (Eq. quant3): out_i = table[codes_i] * absmax[block of i].
 *   codes   device, const uint8_t[n];  absmax device, const float[ceil(n/B)];  out device, float[n]
 */
int dt8_dequantize_blockwise(const uint8_t *codes, const float *absmax, int64_t n, int block_size,
                             int is_signed, float *out, void *stream);

/*
 * One 8-bit SGD-with-momentum step, in place (Eq. sgd wrapped in Eq. quant3 / quant1 / quant2):
 *     m   = table_s[m_codes] * m_absmax[b]
 *     g'  = g + weight_decay * p                 (skipped when weight_decay == 0)
 *     m'  = momentum * m + g'                    (from the zero state this is m_0 = g_0)
 *     p  <- p - lr * m'
 *     (m_codes, m_absmax) <- quantize(m') with the signed table
 *   p         device, float[n]                   parameters, updated
 *   g         device, const float[n] or const bf16[n] per g_dtype (bf16 is widened exactly)
 *   m_codes   device, uint8_t[n];  m_absmax device, float[ceil(n/B)]    state, updated
 *   step      1-based index of this step (accepted for symmetry; the rule does not use it)
 */
int dt8_sgd_step(float *p, const void *g, int g_dtype, uint8_t *m_codes, float *m_absmax,
                 int64_t n, float lr, float momentum, float weight_decay, int64_t step,
                 int block_size, void *stream);

/*
 * One 8-bit Adam / AdamW step, in place (Eq. adam wrapped in Eq. quant3 / quant1 / quant2):
 *     m = table_s[m_codes]*m_absmax[b];  r = table_u[r_codes]*r_absmax[b]
 *     decoupled decay: p <- p*(1 - lr*weight_decay);  coupled: g <- g + weight_decay*p
 *     m' = beta1*m + (1-beta1)*g;   r' = beta2*r + (1-beta2)*(g*g)
 *     p <- p - lr * (m'/bc1) / (sqrt(r'/bc2) + eps),  bc_i = 1 - beta_i^step, or 1 without bias
 *          correction
 *     m' is re-quantized with the signed table, r' with the unsigned table.
 * The parameter update uses the 32-bit m', r' before they are quantized.  With decoupled decay, or
 * with weight_decay == 0, the parameter update is evaluated with a single-instruction reciprocal
 * and square root (relative error ~2e-7 of the update term; when eps*sqrt(bc2) < 1e-12 the forms
 * of these instructions that keep subnormal numbers are used, so that a tiny second moment is not
 * flushed to zero).  With coupled decay, where p feeds the states, and for a learning rate outside
 * 1e-20 .. 1e20, every written operation is one correctly rounded binary32 operation (the
 * divisions and the root by the IEEE instructions, or inside their tested ranges by corrected
 * approximations with the same results), so that the update is bit-reproducible against a plain
 * binary32 evaluation.
 */
int dt8_adam_step(float *p, const void *g, int g_dtype, uint8_t *m_codes, float *m_absmax,
                  uint8_t *r_codes, float *r_absmax, int64_t n, float lr, float beta1, float beta2,
                  float eps, float weight_decay, int64_t step, int block_size, uint32_t flags,
                  void *stream);

/*
 * The same two steps for parameters of either element type (p_dtype: DT8_F32 or DT8_BF16).
 * The paper keeps parameters in 32-bit floating point (Section II); bfloat16 parameters without a
 * 32-bit copy are a variant of this library: the stored parameter is widened exactly, the update
 * of Eq. sgd / Eq. adam is evaluated in binary32 exactly as for binary32 parameters, and the
 * result is rounded once, to nearest even, when it is stored.  States and their arithmetic do
 * not change.  bfloat16 parameters need 8-byte alignment.  dt8_sgd_step(p, ...) is
 * dt8_sgd_step_ex(p, DT8_F32, ...), and likewise for Adam.
 *   p   device, float[n] or bf16[n] per p_dtype, updated in place
 */
int dt8_sgd_step_ex(void *p, int p_dtype, const void *g, int g_dtype, uint8_t *m_codes,
                    float *m_absmax, int64_t n, float lr, float momentum, float weight_decay,
                    int64_t step, int block_size, void *stream);

int dt8_adam_step_ex(void *p, int p_dtype, const void *g, int g_dtype, uint8_t *m_codes,
                     float *m_absmax, uint8_t *r_codes, float *r_absmax, int64_t n, float lr,
                     float beta1, float beta2, float eps, float weight_decay, int64_t step,
                     int block_size, uint32_t flags, void *stream);

/*
 * Pointer-list forms: the same step applied to num_tensors tensors in one kernel launch per 256
 * tensors (the paper's networks hold hundreds of small convolution and batch-norm tensors,
 * Section III layer tables).  The arrays p, g, m_codes, m_absmax, r_codes, r_absmax and n are HOST
 * arrays of num_tensors entries, read before the call returns; their entries are device pointers
 * (sizes for n).  Every tensor is chunked on its own: tensor t has ceil(n[t]/B) blocks.  All
 * gradients share g_dtype.  Tensors with n[t] == 0 are skipped.  Results are identical to calling
 * the single-tensor form on each tensor.
 */
int dt8_sgd_step_multi(int num_tensors, float *const *p, const void *const *g, int g_dtype,
                       uint8_t *const *m_codes, float *const *m_absmax, const int64_t *n, float lr,
                       float momentum, float weight_decay, int64_t step, int block_size,
                       void *stream);

int dt8_adam_step_multi(int num_tensors, float *const *p, const void *const *g, int g_dtype,
                        uint8_t *const *m_codes, float *const *m_absmax, uint8_t *const *r_codes,
                        float *const *r_absmax, const int64_t *n, float lr, float beta1,
                        float beta2, float eps, float weight_decay, int64_t step, int block_size,
                        uint32_t flags, void *stream);

/* Pointer-list forms for parameters of either element type (all parameters of a call share
 * p_dtype); otherwise as above. */
int dt8_sgd_step_multi_ex(int num_tensors, void *const *p, int p_dtype, const void *const *g,
                          int g_dtype, uint8_t *const *m_codes, float *const *m_absmax,
                          const int64_t *n, float lr, float momentum, float weight_decay,
                          int64_t step, int block_size, void *stream);

int dt8_adam_step_multi_ex(int num_tensors, void *const *p, int p_dtype, const void *const *g,
                           int g_dtype, uint8_t *const *m_codes, float *const *m_absmax,
                           uint8_t *const *r_codes, float *const *r_absmax, const int64_t *n,
                           float lr, float beta1, float beta2, float eps, float weight_decay,
                           int64_t step, int block_size, uint32_t flags, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* DT8_H_ */
