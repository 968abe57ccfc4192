/*
 * luq.h - C ABI of the B200 (sm_100a) 4-bit training hot path.
 *
 * The library implements the quantize-then-multiply pipeline of "Accurate
 * Neural Training with 4-bit Matrix Multiplications at Standard Formats":
 * per-tensor max, INT4 round-to-nearest quantization of weights/activations,
 * LUQ (logarithmic unbiased quantization) of neural gradients to the FP4
 * [sign,exp,mantissa] = [1,3,0] grid, and the three training GEMMs.
 *
 * Conventions
 *   - Row-major tensors.  A layer has activations A[M x K], weights W[N x K],
 *     pre-activation gradient G[M x N].
 *       forward   Z  = A . W^T  [M x N]
 *       backward  dA = G . W    [M x K]
 *       update    dW = G^T . A  [N x K]
 *   - Packed codes: two 4-bit codes per byte along the contiguous dimension,
 *     element 2j in the low nibble, element 2j+1 in the high nibble.
 *       INT4 : two's-complement integer q in [-7, 7]; value q * scale.
 *       UINT4: (optional, non-negative tensors) integer q in [0, 15]; value q * scale.
 *       LUQ  : bit 3 = sign, bits 0..2 = c; c = 0 is zero (always nibble 0x0),
 *              c >= 1 is alpha * 2^(c-1).  With the compiled level count
 *              (luq_kmax() = 4) the codes 0..5 occur.
 *   - Every pointer named d_* is a DEVICE pointer owned by the caller and must
 *     be 16-byte aligned.  Scalars (max, scales) stay in device memory so a
 *     whole step needs no host synchronisation.
 *   - Every call is asynchronous on `stream` (a cudaStream_t passed as void*;
 *     NULL = the default stream) and returns 0 on success or a negative
 *     LUQ_ERR_* code.  Nothing throws, aborts or traps the device.
 *   - Conditions found on the device set bits in a status word read with
 *     luq_status(): outputs stay defined (zero codes and a zero scale for a
 *     non-finite or out-of-range max; unspecified values after a TIMEOUT).
 *   - A context serves one stream at a time; calls that overlap on the GPU
 *     through the same context race on its workspace.
 */
#ifndef LUQ_H_
#define LUQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* element types of the high-precision inputs */
#define LUQ_F32 0
#define LUQ_BF16 1

/* return codes */
#define LUQ_OK 0
#define LUQ_ERR_ARG (-1)         /* null/misaligned pointer, bad size, bad n_samples */
#define LUQ_ERR_CUDA (-2)        /* a CUDA runtime/driver call failed */
#define LUQ_ERR_UNSUPPORTED (-3) /* device is not sm_100, or option unknown */
#define LUQ_ERR_WORKSPACE (-4)   /* problem needs more split workspace than the context holds */

/* device status bits (luq_status) */
#define LUQ_STATUS_NONFINITE 1 /* a max / clip was Inf or NaN: zero codes, zero scale */
#define LUQ_STATUS_RANGE 2     /* a non-zero max / clip outside [2^-100, 2^100]: zero codes, zero scale */
#define LUQ_STATUS_TIMEOUT 4   /* a bounded wait inside a kernel expired; outputs unspecified */
#define LUQ_STATUS_BOUNDS 8    /* only from the checking build of the library (compiled with -DLUQ_DEBUG, see
                                  luq_debug_build): an address a kernel formed lay outside its region; that access
                                  was skipped (never a trap), outputs unspecified */

/* options for luq_set_option */
#define LUQ_OPT_MMA_KIND 1 /* 0: tcgen05 kind::f8f6f4 on e4m3 operands (operand bytes passed to a GEMM are then
                              ignored); 1: kind::i8 on int8 operands; 2 (default): int8, except e4m3 where an
                              int32 accumulator could wrap (contractions beyond about 2^18 terms) */
#define LUQ_OPT_SPLITS 2   /* 0: choose the contraction split automatically (default); n >= 1: force n */
#define LUQ_OPT_PAIRS 3    /* CTA pairs (tcgen05 cta_group::2: a 256-row tile on two SMs, each fetching half of B) for
                              unsplit products whose operands both arrive as operand bytes.  0: never; 1: wherever
                              possible; 2 (default): where measured faster - long contractions with B stored
                              contraction-major (the backward and update products of a wide layer).  Results are
                              bit-identical either way. */
#define LUQ_OPT_UNSIGNED_ACTIVATIONS 5 /* 1: the activation codes given to luq_gemm_fwd and luq_gemm_wgrad are
                              unsigned INT4 (from luq_quant_uint4).  Such an operand is always fetched as bytes:
                              pass the operand bytes luq_quant_uint4 wrote, or the GEMM expands a plane into the
                              context workspace (LUQ_ERR_WORKSPACE if it does not fit: 76 MiB). */
#define LUQ_OPT_OUTPUT_BF16 6 /* 1: luq_gemm_fwd / bwd / wgrad write bf16 outputs (the fp32 result rounded to
                              nearest even) instead of fp32: half the output traffic, which is what bounds the
                              backward product of a wide layer.  The output's row length must then be a
                              multiple of 8 elements.  Not available in luq_gemm_wgrad_static. */
#define LUQ_OPT_GRADIENT_INT4 7 /* 1: the gradient codes handed to luq_gemm_bwd / luq_gemm_wgrad are signed INT4
                              (from luq_quant_grad_ablation with LUQ_SCHEME_INT4_SR; d_alpha is then its
                              scale max/7).  Such an operand is fetched as bytes: the caller's operand bytes,
                              or a plane expanded into the context workspace (LUQ_ERR_WORKSPACE beyond 76 MiB).
                              Not available in luq_gemm_wgrad_static. */
#define LUQ_OPT_SM_LIMIT 8 /* n >= 1: the GEMMs of this context occupy at most n SMs (one persistent CTA each; the
                              contraction split is chosen for n SMs); 0 (default): all SMs.  Two products that do not
                              depend on one another - the backward product, which is bound by its output stream and
                              leaves the tensor cores idle, and the update product, which is bound by the tensor
                              cores and moves little memory - can then run side by side on two streams (two
                              contexts), each on its share of the SMs.  Results do not depend on the limit. */
#define LUQ_OPT_SUM_SAMPLES 9 /* 1: with n_samples >= 2 (SMP, Sec. 5.1) the operand bytes that luq_quant_grad,
                              luq_amax_quant_grad, luq_quant_grad_pw2 and luq_quant_grad_hindsight write are ONE
                              plane of rows * cols bytes: byte e = the sum over the samples of the int8 value
                              +-2^(c-1) of element e (the packed codes stay one plane per sample), and luq_gemm_bwd /
                              luq_gemm_wgrad given such bytes with that n_samples read one plane and divide by
                              n_samples.  The mean over samples of the products is, by linearity, the product with
                              the summed operand divided by n_samples, and both are exact in the int32
                              accumulator: results equal those of the per-sample planes bit for bit, at the cost
                              of one sample's product.  Needs n_samples * 2^kmax <= 127 (two samples at the
                              default level count, up to three at kmax = 5) and int8 operands, otherwise the
                              quantizer / the product returns LUQ_ERR_UNSUPPORTED; the ablation's quantizers
                              return it too.  Set it on the quantizing and on the multiplying context alike.
                              0 (default): one plane per sample.  The paper states SMP as repeated products;
                              it has no counterpart of this shortcut. */
#define LUQ_OPT_LEVELS 4   /* kmax of the gradient quantizers, 1..6 (default luq_kmax() = 4): levels
                              alpha * 2^0 .. alpha * 2^kmax with alpha = max / 2^kmax, codes 0..kmax+1.  The
                              other grids of the paper from the same kernels: kmax = 2 is the FP2 grid of
                              the ablation figure (Sec. 4), kmax = 6 uses the whole 3-bit exponent. */

#define LUQ_MAX_SAMPLES 8

/* Operand bytes ("d_*_operand" arguments, all optional: pass NULL to leave them out).
 * The 4-bit codes are the format of the paper (Sec. 3, Sec. 4) and what is stored;
 * the tensor cores of this GPU read 8-bit operands, so a GEMM has to widen every
 * code once per tile that reads it.  A quantizer can write the widened form next to
 * the codes in the same pass, and a GEMM given those bytes fetches them instead of
 * widening the codes again.  They carry the same integers as the codes, so every
 * result is bit-identical with or without them.  Layout: one int8 per element, in
 * the element order of the tensor (sample planes one after the other, rows*cols
 * bytes each).  INT4: 16 * q (the code nibble in the high half of the byte).  LUQ:
 * +-2^(c-1) for code c >= 1, 0 for c = 0.  16-byte aligned.  A GEMM uses them where
 * at least two of its tiles re-read the operand and the contraction is long, or
 * where the contraction is short (at most four 128-deep stages), the output fp32
 * and the bytes of BOTH operands are given (such a product is bound by its output
 * and then stores whole output rows); it reads the codes otherwise.  The codes
 * must always be passed. */

typedef struct luq_ctx luq_ctx;

/* Creates a context on `device`: a device status word, 48 KB of scratch words for grid-wide
 * maxima, and the workspace (96 MiB: partial tiles of split contractions and 8-bit operand
 * planes that a GEMM expands itself when the caller passes none).  Allocates device memory;
 * call outside stream capture.  Every other call of the library allocates nothing and does
 * not synchronise with the host (luq_status excepted), so a sequence of calls can be captured
 * in a CUDA graph.  Two streams that run calls concurrently need two contexts. */
int luq_create(luq_ctx** out, int device);
int luq_destroy(luq_ctx* ctx);
int luq_set_option(luq_ctx* ctx, int option, int value);

/* Default number of binades between the underflow threshold and the tensor maximum:
 * alpha = max|x| / 2^kmax.  The paper's Eq. (alpha) prints 2^(2^(b-1)) with
 * b = 3, i.e. kmax = 4.  LUQ_OPT_LEVELS changes it per context. */
int luq_kmax(void);

/* max_i |x_i| of a tensor of n elements (Sec. 4, "Above FP maximum": the top
 * level is the tensor maximum, Eq. alpha).  d_amax receives one float.  If any
 * element is Inf/NaN the result is Inf/NaN and LUQ_STATUS_NONFINITE is set. */
int luq_amax(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_amax, void* stream);

/* Q_INT, INT4 round-to-nearest (Sec. 3.3: RDN for weights and activations in
 * all phases; Appendix A.1: one high-precision scale per tensor).
 *   scale = clip / 7, q = clamp(rint(x * (7 / clip)), -7, 7), ties to even.
 * d_clip is usually the tensor max from luq_amax; any caller clip is allowed.
 * rows*cols must be even.  d_codes: rows*cols/2 bytes.  d_scale: one float. */
int luq_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols,
                   const float* d_clip, uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream);

/* luq_amax and luq_quant_int4 for several tensors of one element type in ONE launch each (the
 * forward pass of a layer quantizes its activations and its weights; a small tensor's launch and
 * reduction latency then hides behind the large one's stream).  count <= 4.  The arrays are HOST
 * arrays of `count` entries holding device pointers / element counts; results are exactly those
 * of the separate calls.  n[i] even for luq_quant_int4_multi; d_operand[i] may be NULL. */
int luq_amax_multi(luq_ctx* ctx, int count, const void* const* d_x, int dtype, const size_t* n,
                   float* const* d_amax, void* stream);
int luq_quant_int4_multi(luq_ctx* ctx, int count, const void* const* d_x, int dtype, const size_t* n,
                         const float* const* d_clip, uint8_t* const* d_codes, float* const* d_scale,
                         int8_t* const* d_operand, void* stream);

/* Unsigned INT4 for tensors that cannot be negative (post-ReLU activations).  Appendix
 * "Quantization formats": scale = Delta / (2^b - 1) with Delta the quantized range - for the
 * range [0, clip] all sixteen codes lie on one side of zero:
 *   scale = clip / 15, q = clamp(rint(x * (15 / clip)), 0, 15), ties to even; code nibble = q.
 * Half the step of luq_quant_int4 on the same range.  Operand bytes (optional): int8 q.
 * Use with LUQ_OPT_UNSIGNED_ACTIVATIONS = 1 on the context whose GEMMs read the codes. */
int luq_quant_uint4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols,
                    const float* d_clip, uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream);

/* luq_amax followed by luq_quant_int4 with that maximum as the clip, as ONE kernel (the paper's
 * forward quantization measures the tensor and then quantizes it, Sec. 3; two launches of
 * streaming kernels cost more than the second pass when the tensor is small).  Every block
 * first reduces its share of max|x|, the blocks meet at a grid barrier, then all quantize.
 * *d_amax receives the maximum; codes, scale, operand bytes and status bits are exactly those
 * of the two separate calls.  The launch is cooperative; the barrier's wait is bounded, and if
 * it expires LUQ_STATUS_TIMEOUT is raised and no codes are written. */
int luq_amax_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols,
                        float* d_amax, uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream);

/* INT4 with the in-hindsight range (Sec. 7 "Reducing the data movement", Appendix A.5.4, applied to
 * the forward tensors): the tensor is quantized in ONE pass with the clip estimate *d_chat made from
 * earlier steps (values beyond it saturate at +-7, as with any caller-supplied clip), its own max|x|
 * is measured on the way into *d_measured_max, and the estimate for the next step replaces *d_chat:
 *   c_hat <- (1 - eta) * measured + eta * c_hat     (binary32, one rounding per operation).
 * This removes the max pass over the tensor, i.e. one of the two reads of the activations.
 * *d_scale receives c_hat / 7 (the estimate used).  Initialise *d_chat before the first step, e.g.
 * with luq_amax.  0 <= eta <= 1.  Codes, operand bytes and status bits are those of
 * luq_quant_int4 called with d_clip = the estimate. */
int luq_quant_int4_hindsight(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols,
                             float* d_chat, float eta, uint8_t* d_codes, float* d_scale,
                             float* d_measured_max, int8_t* d_operand, void* stream);

/* Q_FP = LUQ (Sec. 4): alpha = max / 2^kmax (Eq. alpha); |x| < alpha becomes
 * sign*alpha with probability |x|/alpha, else 0 (Eq. StochasticPruning);
 * in-range values round stochastically between the two enclosing powers of two
 * (Eq. unbiasedFpQ).  t = |x|/alpha is an IEEE binary32 quotient; one 32-bit
 * Philox4x32-10 word per element and sample decides: key = seed + sample,
 * counter = index/4, word = index%4 (index = flat row-major element index).
 * SMP (Sec. 5.1): n_samples independent draws, written as n_samples planes of
 * rows*cols/2 bytes, sample-major.  d_amax usually comes from luq_amax; a
 * smaller value clips to the top level.  d_alpha receives alpha. */
int luq_quant_grad(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                   const float* d_amax, uint64_t seed, int n_samples,
                   uint8_t* d_codes, float* d_alpha, int8_t* d_operand, void* stream);

/* luq_amax followed by luq_quant_grad with that maximum, as ONE kernel (Sec. 4: the underflow
 * threshold follows the maximum of the tensor at hand, measured in every backward pass).
 * Same construction and guarantees as luq_amax_quant_int4; *d_amax receives the maximum. */
int luq_amax_quant_grad(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                        uint64_t seed, int n_samples, float* d_amax,
                        uint8_t* d_codes, float* d_alpha, int8_t* d_operand, void* stream);

/* Biased logarithmic quantization, the "FP4" baseline of the paper's ablation (Sec. 4, Eq. RC):
 * the grid, scale, code layout and clipping of luq_quant_grad, but deterministic.  In range, the
 * nearer level in LINEAR distance (round-to-nearest-power: up from 2^n alpha exactly when
 * |x| >= 3/2 * 2^n alpha, i.e. 2^floor(log2(4/3 * |x|/alpha))); below alpha, the nearer of 0 and alpha
 * (up when |x| >= alpha/2).  One plane, no seed.  Implemented as the LUQ decision at probability
 * 1/2: every random word is replaced by 2^31 - 1, no generator runs. */
int luq_quant_grad_nearest(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                           const float* d_amax, uint8_t* d_codes, float* d_alpha, int8_t* d_operand,
                           void* stream);

/* The other gradient quantizers of the paper's ablation (Sec. 4, ablation figure and caption; the
 * paper names and draws these arms, it does not print them - the readings are stated here).
 * `scheme` says which region of the LUQ grid is stochastic:
 *   LUQ_SCHEME_FP4      neither: the biased baseline, the same codes as luq_quant_grad_nearest
 *   LUQ_SCHEME_FP4_SR   stochastic rounding inside the range (Eq. unbiasedFpQ); below alpha the
 *                       nearer of 0 and alpha ("FP4 + SR": unbiased inside the range only)
 *   LUQ_SCHEME_FP4_SU   stochastic underflow below alpha (Eq. StochasticPruning); inside the range
 *                       round-to-nearest-power (Eq. RC)
 *   LUQ_SCHEME_LUQ      both: the codes of luq_quant_grad (with the scale of Eq. alpha this is
 *                       LUQ itself; the figure's "FP4 + SR + SU" arm must differ from it by a
 *                       range the paper does not give)
 *   LUQ_SCHEME_INT4_SR  "INT4 unbiased": the uniform grid -7..7 with step max/7 and stochastic
 *                       rounding (Sec. 3.1, Eq. SR) of the magnitude: y = |x| * fl(7/max), up from
 *                       floor(y) when word < trunc((y - floor(y)) * 2^32), sign applied afterwards.
 *                       Codes are INT4 nibbles (two's complement), operand bytes 16 * q, *d_scale
 *                       receives max/7; elements beyond a smaller caller-supplied maximum take +-7.
 * For the first four, grid, level count (LUQ_OPT_LEVELS), scale (*d_scale receives alpha), code
 * layout, sample planes and random words are those of luq_quant_grad.  To multiply with
 * LUQ_SCHEME_INT4_SR codes set LUQ_OPT_GRADIENT_INT4.  One plain streaming kernel per call. */
#define LUQ_SCHEME_FP4 0
#define LUQ_SCHEME_FP4_SR 1
#define LUQ_SCHEME_FP4_SU 2
#define LUQ_SCHEME_LUQ 3
#define LUQ_SCHEME_INT4_SR 4
int luq_quant_grad_ablation(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                            const float* d_amax, uint64_t seed, int n_samples, int scheme,
                            uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream);

/* LUQ with a power-of-two scale (Appendix A.7, LUQ_PW2): as luq_quant_grad, but
 * alpha = 2^ceil(log2 max) / 2^kmax - the maximum is rounded UP to a power of two,
 * so nothing is clipped, every level is a power of two and |x| / alpha is an exact
 * exponent shift.  d_alpha receives the power-of-two alpha. */
int luq_quant_grad_pw2(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                       const float* d_amax, uint64_t seed, int n_samples,
                       uint8_t* d_codes, float* d_alpha, int8_t* d_operand, void* stream);

/* LUQ with the in-hindsight maximum (Sec. 7 "Reducing the data movement", Appendix
 * A.5.4): the tensor is quantized in ONE pass with the estimate *d_mhat made from
 * earlier steps (values above it clip to the top level), its own max|x| is measured
 * on the way into *d_measured_max, and the estimate for the next step replaces
 * *d_mhat:   m_hat <- (1 - eta) * measured + eta * m_hat     (binary32, one
 * rounding per operation; the paper uses eta = 0.1).  pw2 = 1 additionally rounds
 * the estimate up to a power of two before use (LUQ_PW2 + Hindsight).  Initialise
 * *d_mhat before the first step, e.g. with luq_amax.  0 <= eta <= 1. */
int luq_quant_grad_hindsight(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols,
                             float* d_mhat, float eta, int pw2, uint64_t seed, int n_samples,
                             uint8_t* d_codes, float* d_alpha, float* d_measured_max, int8_t* d_operand,
                             void* stream);

/* Diagnostic for the division-free quotient inside luq_quant_grad (reading of
 * Eq. StochasticPruning / Eq. unbiasedFpQ: the probabilities are functions of
 * t = |x| / alpha): writes, for n fp32 elements, the value t the quantizer forms
 * with alpha = *d_amax / 2^kmax, before its clamp to the top level.  It must
 * equal the IEEE binary32 quotient wherever that quotient is a normal number. */
int luq_debug_quotient(luq_ctx* ctx, const float* d_x, size_t n, const float* d_amax, float* d_t, void* stream);

/* Diagnostic for the bounded waits (the paper has no counterpart): launches one thread that waits on a
 * barrier nothing ever arrives on, with a short limit.  The wait expires, the kernel raises
 * LUQ_STATUS_TIMEOUT the way the GEMM roles and the fused quantizers do, and returns normally; the
 * context stays usable and luq_status() reports and clears the bit. */
int luq_debug_expire_wait(luq_ctx* ctx, void* stream);

/* The three GEMMs write fp32 outputs (void* d_z / d_da / d_dw point to floats) unless
 * LUQ_OPT_OUTPUT_BF16 is set on the context, in which case they point to bf16 values.
 *
 * Forward GEMM (Eq. Forward; scale factoring of Appendix A.1):
 *   Z[m,n] = (sa*sw) * sum_k qA[m,k] * qW[n,k]        fp32 accumulate, fp32 out.
 * a_codes [M x K/2], w_codes [N x K/2].  K must be a multiple of 32. */
int luq_gemm_fwd(luq_ctx* ctx, const uint8_t* d_a_codes, const float* d_sa, const int8_t* d_a_operand,
                 const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                 void* d_z, int64_t M, int64_t N, int64_t K, void* stream);

/* luq_quant_int4 of the activations followed by luq_gemm_fwd, as ONE kernel (Eq. Forward on
 * Q_INT(A), Sec. 3.3; Sec. 7 "Reducing the data movement": the passes over the tensors, not the
 * MACs, are the cost).  For a layer with one column of output tiles (N <= 256) every row block
 * of A is read by exactly one tile, so the GEMM takes the HIGH-PRECISION activations d_a
 * [M x K, fp32 or bf16], quantizes them on the way in with the clip *d_clip (usually the max from
 * luq_amax), and writes their packed codes d_a_codes [M x K/2] and scale *d_sa as by-products
 * (the update GEMM reads them).  A is streamed once at memory speed and the tensor-core work
 * hides under that stream.  Codes, scale, status bits and Z are exactly those of the two
 * separate calls.  d_w_operand (optional): W's operand bytes from luq_quant_int4; without them
 * W's codes are widened once into the context workspace.  K must be a multiple of 32.  Where
 * the fusion does not apply (N > 256, bf16 output, unsigned activations, e4m3 operands forced)
 * the call runs the two separate kernels. */
int luq_quant_int4_gemm_fwd(luq_ctx* ctx, const void* d_a, int dtype, const float* d_clip,
                            uint8_t* d_a_codes, float* d_sa,
                            const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                            void* d_z, int64_t M, int64_t N, int64_t K, void* stream);

/* The same kernel with the in-hindsight maximum of Sec. 7 / App. A.5.4 (luq_quant_int4_hindsight followed by
 * luq_gemm_fwd, as ONE pass over the activations): A is quantized with the running estimate *d_chat, not
 * with its own maximum - values beyond it saturate at +-7 - while max|A| is measured on the way; *d_sa
 * receives chat / 7, *d_measured_max the measured maximum, and *d_chat is replaced by
 * (1 - eta) * measured + eta * chat for the next step (a non-finite measurement keeps the estimate and
 * raises LUQ_STATUS_NONFINITE; an unusable estimate gives zero codes, a zero scale and a zero Z, and is
 * replaced by the measurement).  No max pass over A at all.  Results are those of the two separate calls
 * bit for bit; where the fusion does not apply the call runs them.  0 <= eta <= 1. */
int luq_quant_int4_hindsight_gemm_fwd(luq_ctx* ctx, const void* d_a, int dtype, float* d_chat, float eta,
                                      uint8_t* d_a_codes, float* d_sa, float* d_measured_max,
                                      const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                                      void* d_z, int64_t M, int64_t N, int64_t K, void* stream);

/* Backward GEMM (Eq. Backward), SMP average fused (Sec. 5.1):
 *   dA[m,k] = (alpha*sw/n_samples) * sum_s sum_n qG_s[m,n] * qW[n,k].
 * g_codes: n_samples planes [M x N/2]; w_codes [N x K/2].
 * N and K must be multiples of 32. */
int luq_gemm_bwd(luq_ctx* ctx, const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                 const int8_t* d_g_operand, const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                 void* d_da, int64_t M, int64_t N, int64_t K, void* stream);

/* Update GEMM (Eq. Update), SMP average fused (Sec. 5.1):
 *   dW[n,k] = (alpha*sa/n_samples) * sum_s sum_m qG_s[m,n] * qA[m,k].
 * g_codes: n_samples planes [M x N/2]; a_codes [M x K/2].
 * N and K must be multiples of 32.  Uses the context's split workspace when
 * the output has few tiles (contraction over M is split across CTAs). */
int luq_gemm_wgrad(luq_ctx* ctx, const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                   const int8_t* d_g_operand, const uint8_t* d_a_codes, const float* d_sa, const int8_t* d_a_operand,
                   void* d_dw, int64_t M, int64_t N, int64_t K, void* stream);

/* Update GEMM without any allocation.  (The paper has no counterpart; this entry
 * point exists for the sake of callers.)
 *
 * Some callers cannot obtain device memory themselves: code that runs inside a
 * stream capture, inside another framework's allocator hooks or a memory-frozen
 * serving process, or under a memory budget that forbids cudaMalloc after start-up.
 * luq_create allocates the split workspace with cudaMalloc, so it is closed to
 * them.  This variant of luq_gemm_wgrad takes no context and keeps its split
 * workspace (the partial tiles of the contraction split) in a fixed 19 MiB array
 * inside the library image.  It calls no allocation routine of any kind.
 *
 *  - Same arguments and result as luq_gemm_wgrad, on the CURRENT device.
 *  - Limit: the output N x K may have at most 152 tiles of 128 x 256 elements
 *    (for example N = 256, K <= 19456); larger outputs return LUQ_ERR_WORKSPACE.
 *  - The first call on each device looks up the device address of the array
 *    (cudaGetSymbolAddress) and clears the variant's status word; make that first
 *    call outside any stream capture.  Later calls only launch kernels.
 *  - The array is shared by all calls on a device and keeps the previous call's
 *    partial tiles.  Every call rewrites all tiles it later reads, so nothing has
 *    to be cleared, but two calls that overlap on the GPU (different streams) race
 *    on it: serialise them.
 *  - A bounded wait that expires cannot be reported through luq_status here; it
 *    leaves the output unspecified, as in luq_gemm_wgrad. */
int luq_gemm_wgrad_static(const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                          const uint8_t* d_a_codes, const float* d_sa,
                          float* d_dw, int64_t M, int64_t N, int64_t K, void* stream);

/* 1 if this library was compiled with -DLUQ_DEBUG: every shared-memory, tensor-memory and global
 * address that the converters, epilogues and streaming loops form is checked against its region
 * before use; a violation raises LUQ_STATUS_BOUNDS and skips the access.  (The pool this library
 * was developed on offers no compute-sanitizer; this build stands in for it.)  0 otherwise. */
int luq_debug_build(void);

/* Diagnostic for the checking build (the paper has no counterpart): launches one thread that forms an
 * address just beyond a small shared-memory region and puts it to the check WITHOUT accessing it.  In
 * the checking build luq_status() then reports LUQ_STATUS_BOUNDS; in the normal build, nothing. */
int luq_debug_bounds_probe(luq_ctx* ctx, void* stream);

/* Synchronises `stream`, returns the device status bits in *host_flags and
 * clears them. */
int luq_status(luq_ctx* ctx, void* stream, int* host_flags);

/* Number of kernels this library has launched through `ctx` so far. */
int64_t luq_launch_count(luq_ctx* ctx);

const char* luq_strerror(int code);

#ifdef __cplusplus
}
#endif
#endif /* LUQ_H_ */
