// C ABI of the library (declared in luq.h): argument checks, context, launches.
#include <new>

#include "common.cuh"

namespace {

constexpr size_t kWorkspaceBytes = 96u << 20;  // 20 MiB of split partial tiles + 76 MiB of operand planes

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
cudaStream_t as_stream(void* s) { return reinterpret_cast<cudaStream_t>(s); }
int cuda_rc(int e) { return e == 0 ? LUQ_OK : (e < 0 ? e : LUQ_ERR_CUDA); }

struct DeviceGuard {
  int prev = -1;
  bool ok = true;
  explicit DeviceGuard(int dev) {
    if (cudaGetDevice(&prev) != cudaSuccess) { ok = false; return; }
    if (prev != dev && cudaSetDevice(dev) != cudaSuccess) ok = false;
  }
  ~DeviceGuard() { if (prev >= 0) cudaSetDevice(prev); }
};

}  // namespace

extern "C" {

int luq_kmax(void) { return LUQ_KMAX; }

int luq_debug_build(void) {
#ifdef LUQ_DEBUG
  return 1;
#else
  return 0;
#endif
}

const char* luq_strerror(int code) {
  switch (code) {
    case LUQ_OK: return "ok";
    case LUQ_ERR_ARG: return "invalid argument (null or misaligned pointer, bad size or sample count)";
    case LUQ_ERR_CUDA: return "a CUDA call failed";
    case LUQ_ERR_UNSUPPORTED: return "unsupported device or option";
    case LUQ_ERR_WORKSPACE: return "split workspace too small for this problem";
    default: return "unknown error";
  }
}

int luq_create(luq_ctx** out, int device) {
  if (!out) return LUQ_ERR_ARG;
  *out = nullptr;
  int count = 0;
  if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return LUQ_ERR_CUDA;
  cudaDeviceProp prop;
  if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return LUQ_ERR_CUDA;
  if (prop.major != 10) return LUQ_ERR_UNSUPPORTED;  // the kernels are sm_100a only
  DeviceGuard guard(device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  luq_ctx* c = new (std::nothrow) luq_ctx();
  if (!c) return LUQ_ERR_CUDA;
  c->device = device;
  c->sm_count = prop.multiProcessorCount;
  c->mma_kind = LUQ_DEFAULT_MMA_KIND;
  c->forced_splits = 0;
  c->use_pairs = 2;
  c->kmax = LUQ_KMAX;
  c->unsigned_act = 0;
  c->grad_int4 = 0;
  c->sm_limit = 0;
  c->out_bf16 = 0;
  c->launches = 0;
  c->workspace_bytes = kWorkspaceBytes;
  c->d_status = nullptr; c->d_scratch = nullptr; c->d_workspace = nullptr; c->encode_tiled = nullptr;
  // status word and the grid-maximum scratch share one small allocation
  const size_t small_bytes = (64 + static_cast<size_t>(LUQ_SCRATCH_WORDS)) * sizeof(unsigned int);
  bool ok = cudaMalloc(&c->d_status, small_bytes) == cudaSuccess &&
            cudaMalloc(&c->d_workspace, kWorkspaceBytes) == cudaSuccess;
  ok = ok && cudaMemset(c->d_status, 0, small_bytes) == cudaSuccess;
  if (ok) c->d_scratch = c->d_status + 64;
  if (ok) {
    cudaDriverEntryPointQueryResult q;
    ok = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &c->encode_tiled, cudaEnableDefault, &q) == cudaSuccess &&
         q == cudaDriverEntryPointSuccess && c->encode_tiled != nullptr;
  }
  if (!ok) { luq_destroy(c); return LUQ_ERR_CUDA; }
  *out = c;
  return LUQ_OK;
}

int luq_destroy(luq_ctx* ctx) {
  if (!ctx) return LUQ_OK;
  DeviceGuard guard(ctx->device);
  if (ctx->d_status) cudaFree(ctx->d_status);
  if (ctx->d_workspace) cudaFree(ctx->d_workspace);
  delete ctx;
  return LUQ_OK;
}

int luq_set_option(luq_ctx* ctx, int option, int value) {
  if (!ctx) return LUQ_ERR_ARG;
  switch (option) {
    case LUQ_OPT_MMA_KIND:
      if (value < 0 || value > 2) return LUQ_ERR_ARG;
      ctx->mma_kind = value;
      return LUQ_OK;
    case LUQ_OPT_SPLITS:
      if (value < 0 || value > 1024) return LUQ_ERR_ARG;
      ctx->forced_splits = value;
      return LUQ_OK;
    case LUQ_OPT_OUTPUT_BF16:
      if (value != 0 && value != 1) return LUQ_ERR_ARG;
      ctx->out_bf16 = value;
      return LUQ_OK;
    case LUQ_OPT_UNSIGNED_ACTIVATIONS:
      if (value != 0 && value != 1) return LUQ_ERR_ARG;
      ctx->unsigned_act = value;
      return LUQ_OK;
    case LUQ_OPT_GRADIENT_INT4:
      if (value != 0 && value != 1) return LUQ_ERR_ARG;
      ctx->grad_int4 = value;
      return LUQ_OK;
    case LUQ_OPT_LEVELS:
      if (value < 1 || value > 6) return LUQ_ERR_ARG;
      ctx->kmax = value;
      return LUQ_OK;
    case LUQ_OPT_SM_LIMIT:
      if (value < 0 || value > 4096) return LUQ_ERR_ARG;
      ctx->sm_limit = value;
      return LUQ_OK;
    case LUQ_OPT_SUM_SAMPLES:
      if (value != 0 && value != 1) return LUQ_ERR_ARG;
      ctx->sum_samples = value;
      return LUQ_OK;
    case LUQ_OPT_PAIRS:
      if (value < 0 || value > 2) return LUQ_ERR_ARG;
      ctx->use_pairs = value;
      return LUQ_OK;
    default:
      return LUQ_ERR_UNSUPPORTED;
  }
}

int64_t luq_launch_count(luq_ctx* ctx) { return ctx ? ctx->launches : 0; }

int luq_amax(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_amax, void* stream) {
  if (!ctx || !d_amax || (n && !d_x) || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  if (!aligned16(d_x) || (reinterpret_cast<uintptr_t>(d_amax) & 3u)) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_amax(ctx, d_x, dtype, n, d_amax, as_stream(stream)));
}

int luq_amax_multi(luq_ctx* ctx, int count, const void* const* d_x, int dtype, const size_t* n,
                   float* const* d_amax, void* stream) {
  if (!ctx || count < 1 || count > LUQ_SCRATCH_MULTI || !d_x || !n || !d_amax) return LUQ_ERR_ARG;
  if (dtype != LUQ_F32 && dtype != LUQ_BF16) return LUQ_ERR_ARG;
  for (int t = 0; t < count; ++t) {
    if (!d_amax[t] || (n[t] && !d_x[t]) || !aligned16(d_x[t]) || (reinterpret_cast<uintptr_t>(d_amax[t]) & 3u))
      return LUQ_ERR_ARG;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_amax_multi(ctx, count, d_x, n, d_amax, dtype, as_stream(stream)));
}

int luq_quant_int4_multi(luq_ctx* ctx, int count, const void* const* d_x, int dtype, const size_t* n,
                         const float* const* d_clip, uint8_t* const* d_codes, float* const* d_scale,
                         int8_t* const* d_operand, void* stream) {
  if (!ctx || count < 1 || count > LUQ_SCRATCH_MULTI || !d_x || !n || !d_clip || !d_codes || !d_scale || !d_operand)
    return LUQ_ERR_ARG;
  if (dtype != LUQ_F32 && dtype != LUQ_BF16) return LUQ_ERR_ARG;
  for (int t = 0; t < count; ++t) {
    if (!d_clip[t] || !d_scale[t] || (n[t] & 1u) || (n[t] && (!d_x[t] || !d_codes[t]))) return LUQ_ERR_ARG;
    if (!aligned16(d_x[t]) || !aligned16(d_codes[t]) || !aligned16(d_operand[t])) return LUQ_ERR_ARG;
  }
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_int4_multi(ctx, count, d_x, n, d_clip, d_codes, d_scale, d_operand, dtype,
                                             as_stream(stream)));
}

int luq_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols, const float* d_clip,
                   uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream) {
  if (!ctx || !d_clip || !d_scale || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  const size_t n = rows * cols;
  if (rows != 0 && n / rows != cols) return LUQ_ERR_ARG;
  if (n & 1u) return LUQ_ERR_ARG;
  if (n && (!d_x || !d_codes)) return LUQ_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_codes) || !aligned16(d_operand)) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_int4(ctx, d_x, dtype, n, d_clip, d_codes, n ? d_operand : nullptr, d_scale,
                                       nullptr, false, as_stream(stream)));
}

int luq_quant_uint4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols, const float* d_clip,
                    uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream) {
  if (!ctx || !d_clip || !d_scale || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  const size_t n = rows * cols;
  if (rows != 0 && n / rows != cols) return LUQ_ERR_ARG;
  if (n & 1u) return LUQ_ERR_ARG;
  if (n && (!d_x || !d_codes)) return LUQ_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_codes) || !aligned16(d_operand)) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_int4(ctx, d_x, dtype, n, d_clip, d_codes, n ? d_operand : nullptr, d_scale,
                                       nullptr, true, as_stream(stream)));
}

int luq_quant_int4_hindsight(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols, float* d_chat,
                             float eta, uint8_t* d_codes, float* d_scale, float* d_measured_max, int8_t* d_operand,
                             void* stream) {
  if (!ctx || !d_chat || !d_scale || !d_measured_max || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  if (!(eta >= 0.0f && eta <= 1.0f)) return LUQ_ERR_ARG;
  const size_t n = rows * cols;
  if (rows != 0 && n / rows != cols) return LUQ_ERR_ARG;
  if (n & 1u) return LUQ_ERR_ARG;
  if (n && (!d_x || !d_codes)) return LUQ_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_codes) || !aligned16(d_operand)) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_int4_hindsight(ctx, d_x, dtype, n, d_chat, eta, d_codes, n ? d_operand : nullptr,
                                                 d_scale, d_measured_max, as_stream(stream)));
}

int luq_amax_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t rows, size_t cols, float* d_amax,
                        uint8_t* d_codes, float* d_scale, int8_t* d_operand, void* stream) {
  if (!ctx || !d_amax || !d_scale || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  const size_t n = rows * cols;
  if (rows != 0 && n / rows != cols) return LUQ_ERR_ARG;
  if (n & 1u) return LUQ_ERR_ARG;
  if (n && (!d_x || !d_codes)) return LUQ_ERR_ARG;
  if (!aligned16(d_x) || !aligned16(d_codes) || !aligned16(d_operand)) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_int4(ctx, d_x, dtype, n, nullptr, d_codes, n ? d_operand : nullptr, d_scale,
                                       d_amax, false, as_stream(stream)));
}

static int quant_grad_args(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, const float* d_amax,
                           int n_samples, const uint8_t* d_codes, const float* d_alpha, const int8_t* d_operand,
                           size_t* n_out) {
  if (!ctx || !d_amax || !d_alpha || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  if (n_samples < 1 || n_samples > LUQ_MAX_SAMPLES) return LUQ_ERR_ARG;
  const size_t n = rows * cols;
  if (rows != 0 && n / rows != cols) return LUQ_ERR_ARG;
  if (n & 1u) return LUQ_ERR_ARG;
  if (n && (!d_g || !d_codes)) return LUQ_ERR_ARG;
  if (!aligned16(d_g) || !aligned16(d_codes) || !aligned16(d_operand)) return LUQ_ERR_ARG;
  *n_out = n;
  return LUQ_OK;
}

// LUQ_OPT_SUM_SAMPLES: flag bit for the LUQ launcher (0 when the option does not apply to this call), or
// LUQ_ERR_UNSUPPORTED when the sum of n_samples operand bytes of magnitude 2^kmax could leave int8
static int sum_flag(const luq_ctx* ctx, int n_samples, const int8_t* d_operand) {
  if (!ctx->sum_samples || !d_operand || n_samples < 2) return 0;
  return (n_samples << ctx->kmax) <= 127 ? 8 : LUQ_ERR_UNSUPPORTED;
}

int luq_quant_grad(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, const float* d_amax,
                   uint64_t seed, int n_samples, uint8_t* d_codes, float* d_alpha, int8_t* d_operand, void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_amax, n_samples, d_codes, d_alpha, d_operand, &n);
  if (rc) return rc;
  const int sum = sum_flag(ctx, n_samples, d_operand);
  if (sum < 0) return sum;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_grad_ex(ctx, d_g, dtype, n, d_amax, seed, n_samples, d_codes,
                                          n ? d_operand : nullptr, d_alpha, sum, nullptr, nullptr, 0.0f, nullptr,
                                          as_stream(stream)));
}

int luq_amax_quant_grad(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, uint64_t seed,
                        int n_samples, float* d_amax, uint8_t* d_codes, float* d_alpha, int8_t* d_operand,
                        void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_amax, n_samples, d_codes, d_alpha, d_operand, &n);
  if (rc) return rc;
  const int sum = sum_flag(ctx, n_samples, d_operand);
  if (sum < 0) return sum;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_grad_ex(ctx, d_g, dtype, n, nullptr, seed, n_samples, d_codes,
                                          n ? d_operand : nullptr, d_alpha, sum, nullptr, nullptr, 0.0f, d_amax,
                                          as_stream(stream)));
}

int luq_quant_grad_nearest(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, const float* d_amax,
                           uint8_t* d_codes, float* d_alpha, int8_t* d_operand, void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_amax, 1, d_codes, d_alpha, d_operand, &n);
  if (rc) return rc;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_grad_ex(ctx, d_g, dtype, n, d_amax, 0, 1, d_codes, n ? d_operand : nullptr,
                                          d_alpha, 4, nullptr, nullptr, 0.0f, nullptr, as_stream(stream)));
}

int luq_quant_grad_ablation(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, const float* d_amax,
                            uint64_t seed, int n_samples, int scheme, uint8_t* d_codes, float* d_scale,
                            int8_t* d_operand, void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_amax, n_samples, d_codes, d_scale, d_operand, &n);
  if (rc) return rc;
  if (scheme < 0 || scheme > LUQ_SCHEME_INT4_SR) return LUQ_ERR_ARG;
  if (ctx->sum_samples && d_operand && n_samples > 1) return LUQ_ERR_UNSUPPORTED;   // these kernels write one plane per sample
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_grad_ablation(ctx, d_g, dtype, n, d_amax, seed, n_samples, scheme, d_codes,
                                                n ? d_operand : nullptr, d_scale, as_stream(stream)));
}

int luq_quant_grad_pw2(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, const float* d_amax,
                       uint64_t seed, int n_samples, uint8_t* d_codes, float* d_alpha, int8_t* d_operand,
                       void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_amax, n_samples, d_codes, d_alpha, d_operand, &n);
  if (rc) return rc;
  const int sum = sum_flag(ctx, n_samples, d_operand);
  if (sum < 0) return sum;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_quant_grad_ex(ctx, d_g, dtype, n, d_amax, seed, n_samples, d_codes,
                                          n ? d_operand : nullptr, d_alpha, 1 | sum, nullptr, nullptr, 0.0f, nullptr,
                                          as_stream(stream)));
}

int luq_quant_grad_hindsight(luq_ctx* ctx, const void* d_g, int dtype, size_t rows, size_t cols, float* d_mhat,
                             float eta, int pw2, uint64_t seed, int n_samples, uint8_t* d_codes, float* d_alpha,
                             float* d_measured_max, int8_t* d_operand, void* stream) {
  size_t n = 0;
  const int rc = quant_grad_args(ctx, d_g, dtype, rows, cols, d_mhat, n_samples, d_codes, d_alpha, d_operand, &n);
  if (rc) return rc;
  if (!d_measured_max || !(eta >= 0.0f && eta <= 1.0f) || (pw2 != 0 && pw2 != 1)) return LUQ_ERR_ARG;
  const int sum = sum_flag(ctx, n_samples, d_operand);
  if (sum < 0) return sum;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  // one kernel: quantize with the estimate, measure, and let the last block replace the estimate
  return cuda_rc(luq_launch_quant_grad_ex(ctx, d_g, dtype, n, d_mhat, seed, n_samples, d_codes,
                                          n ? d_operand : nullptr, d_alpha, 2 | pw2 | sum, d_measured_max, d_mhat, eta,
                                          nullptr, as_stream(stream)));
}

int luq_debug_expire_wait(luq_ctx* ctx, void* stream) {
  if (!ctx) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_expire_wait(ctx, as_stream(stream)));
}

int luq_debug_bounds_probe(luq_ctx* ctx, void* stream) {
  if (!ctx) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_bounds_probe(ctx, as_stream(stream)));
}

int luq_debug_quotient(luq_ctx* ctx, const float* d_x, size_t n, const float* d_amax, float* d_t, void* stream) {
  if (!ctx || !d_amax || (n && (!d_x || !d_t))) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  return cuda_rc(luq_launch_debug_quotient(ctx, d_x, n, d_amax, d_t, as_stream(stream)));
}

static int gemm_common(luq_ctx* ctx, const uint8_t* x, const float* sx, const int8_t* xo, const uint8_t* y,
                       const float* sy, const int8_t* yo, const void* out, int64_t M, int64_t N, int64_t K,
                       int n_samples) {
  if (!ctx || !sx || !sy) return LUQ_ERR_ARG;
  if (M < 0 || N < 0 || K < 0 || M > (1ll << 31) || N > (1ll << 31) || K > (1ll << 31)) return LUQ_ERR_ARG;
  if (n_samples < 1 || n_samples > LUQ_MAX_SAMPLES) return LUQ_ERR_ARG;
  if (M && N && K && (!x || !y || !out)) return LUQ_ERR_ARG;
  if (!aligned16(x) || !aligned16(y) || !aligned16(out) || !aligned16(xo) || !aligned16(yo)) return LUQ_ERR_ARG;
  return LUQ_OK;
}

int luq_gemm_fwd(luq_ctx* ctx, const uint8_t* d_a_codes, const float* d_sa, const int8_t* d_a_operand,
                 const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand, void* d_z, int64_t M,
                 int64_t N, int64_t K, void* stream) {
  int rc = gemm_common(ctx, d_a_codes, d_sa, d_a_operand, d_w_codes, d_sw, d_w_operand, d_z, M, N, K, 1);
  if (rc) return rc;
  if (K % 32 || N % 4) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  luq_gemm_args a{};
  a.a_codes = d_a_codes; a.a_kind = ctx->unsigned_act ? 2 : 0; a.a_mn = 0; a.n_samples = 1;
  a.b_codes = d_w_codes; a.b_kind = 0; a.b_mn = 0;
  a.a_operand = d_a_operand; a.b_operand = d_w_operand;
  a.d_scale_a = d_sa; a.d_scale_b = d_sw; a.d_out = d_z; a.out_bf16 = ctx->out_bf16; a.Mo = M; a.No = N; a.Kc = K;
  a.d_workspace = ctx->d_workspace; a.workspace_bytes = ctx->workspace_bytes;
  a.allow_split = 1;
  return cuda_rc(luq_launch_gemm(ctx, a, as_stream(stream)));
}

int luq_quant_int4_gemm_fwd(luq_ctx* ctx, const void* d_a, int dtype, const float* d_clip, uint8_t* d_a_codes,
                            float* d_sa, const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                            void* d_z, int64_t M, int64_t N, int64_t K, void* stream) {
  if (!ctx || !d_clip || !d_sa || !d_sw || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  if (M < 0 || N < 0 || K < 0 || M > (1ll << 31) || N > (1ll << 31) || K > (1ll << 31)) return LUQ_ERR_ARG;
  if (K % 32 || N % 4) return LUQ_ERR_ARG;
  if (M && K && (!d_a || !d_a_codes)) return LUQ_ERR_ARG;
  if (M && N && K && (!d_w_codes || !d_z)) return LUQ_ERR_ARG;
  if (!aligned16(d_a) || !aligned16(d_a_codes) || !aligned16(d_w_codes) || !aligned16(d_w_operand) || !aligned16(d_z))
    return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  if (luq_quant_fwd_fusable(ctx, M, N, K, d_w_operand != nullptr))
    return cuda_rc(luq_launch_quant_fwd(ctx, d_a, dtype, d_clip, d_a_codes, d_sa, d_w_codes, d_sw, d_w_operand,
                                        static_cast<float*>(d_z), M, N, K, st));
  // the two separate kernels
  int rc = cuda_rc(luq_launch_quant_int4(ctx, d_a, dtype, static_cast<size_t>(M) * static_cast<size_t>(K), d_clip,
                                         d_a_codes, nullptr, d_sa, nullptr, false, st));
  if (rc) return rc;
  luq_gemm_args a{};
  a.a_codes = d_a_codes; a.a_kind = ctx->unsigned_act ? 2 : 0; a.a_mn = 0; a.n_samples = 1;
  a.b_codes = d_w_codes; a.b_kind = 0; a.b_mn = 0;
  a.a_operand = nullptr; a.b_operand = d_w_operand;
  a.d_scale_a = d_sa; a.d_scale_b = d_sw; a.d_out = d_z; a.out_bf16 = ctx->out_bf16; a.Mo = M; a.No = N; a.Kc = K;
  a.d_workspace = ctx->d_workspace; a.workspace_bytes = ctx->workspace_bytes;
  a.allow_split = 1;
  return cuda_rc(luq_launch_gemm(ctx, a, st));
}

int luq_quant_int4_hindsight_gemm_fwd(luq_ctx* ctx, const void* d_a, int dtype, float* d_chat, float eta,
                                      uint8_t* d_a_codes, float* d_sa, float* d_measured_max, const uint8_t* d_w_codes,
                                      const float* d_sw, const int8_t* d_w_operand, void* d_z, int64_t M, int64_t N,
                                      int64_t K, void* stream) {
  if (!ctx || !d_chat || !d_sa || !d_sw || !d_measured_max || (dtype != LUQ_F32 && dtype != LUQ_BF16)) return LUQ_ERR_ARG;
  if (!(eta >= 0.0f && eta <= 1.0f)) return LUQ_ERR_ARG;
  if (M < 0 || N < 0 || K < 0 || M > (1ll << 31) || N > (1ll << 31) || K > (1ll << 31)) return LUQ_ERR_ARG;
  if (K % 32 || N % 4) return LUQ_ERR_ARG;
  if (M && K && (!d_a || !d_a_codes)) return LUQ_ERR_ARG;
  if (M && N && K && (!d_w_codes || !d_z)) return LUQ_ERR_ARG;
  if (!aligned16(d_a) || !aligned16(d_a_codes) || !aligned16(d_w_codes) || !aligned16(d_w_operand) || !aligned16(d_z))
    return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  if (luq_quant_fwd_fusable(ctx, M, N, K, d_w_operand != nullptr))
    return cuda_rc(luq_launch_quant_fwd(ctx, d_a, dtype, nullptr, d_a_codes, d_sa, d_w_codes, d_sw, d_w_operand,
                                        static_cast<float*>(d_z), M, N, K, st, d_chat, eta, d_measured_max));
  // the two separate kernels
  int rc = cuda_rc(luq_launch_quant_int4_hindsight(ctx, d_a, dtype, static_cast<size_t>(M) * static_cast<size_t>(K),
                                                   d_chat, eta, d_a_codes, nullptr, d_sa, d_measured_max, st));
  if (rc) return rc;
  luq_gemm_args a{};
  a.a_codes = d_a_codes; a.a_kind = 0; a.a_mn = 0; a.n_samples = 1;
  a.b_codes = d_w_codes; a.b_kind = 0; a.b_mn = 0;
  a.a_operand = nullptr; a.b_operand = d_w_operand;
  a.d_scale_a = d_sa; a.d_scale_b = d_sw; a.d_out = d_z; a.out_bf16 = ctx->out_bf16; a.Mo = M; a.No = N; a.Kc = K;
  a.d_workspace = ctx->d_workspace; a.workspace_bytes = ctx->workspace_bytes;
  a.allow_split = 1;
  return cuda_rc(luq_launch_gemm(ctx, a, st));
}

int luq_gemm_bwd(luq_ctx* ctx, const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                 const int8_t* d_g_operand, const uint8_t* d_w_codes, const float* d_sw, const int8_t* d_w_operand,
                 void* d_da, int64_t M, int64_t N, int64_t K, void* stream) {
  int rc = gemm_common(ctx, d_g_codes, d_alpha, d_g_operand, d_w_codes, d_sw, d_w_operand, d_da, M, N, K, n_samples);
  if (rc) return rc;
  if (N % 32 || K % 32) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  luq_gemm_args a{};
  a.a_codes = d_g_codes; a.a_kind = ctx->grad_int4 ? 0 : 1; a.a_mn = 0; a.n_samples = n_samples;   // G[M x N]: contraction n contiguous
  a.b_codes = d_w_codes; a.b_kind = 0; a.b_mn = 1;                            // W[N x K]: rows are the contraction
  a.a_operand = d_g_operand; a.b_operand = d_w_operand;
  a.a_summed = (ctx->sum_samples && !ctx->grad_int4 && d_g_operand && n_samples > 1) ? n_samples : 0;
  a.d_scale_a = d_alpha; a.d_scale_b = d_sw; a.d_out = d_da; a.out_bf16 = ctx->out_bf16; a.Mo = M; a.No = K; a.Kc = N;
  a.d_workspace = ctx->d_workspace; a.workspace_bytes = ctx->workspace_bytes;
  a.allow_split = 1;
  return cuda_rc(luq_launch_gemm(ctx, a, as_stream(stream)));
}

int luq_gemm_wgrad(luq_ctx* ctx, const uint8_t* d_g_codes, const float* d_alpha, int n_samples,
                   const int8_t* d_g_operand, const uint8_t* d_a_codes, const float* d_sa, const int8_t* d_a_operand,
                   void* d_dw, int64_t M, int64_t N, int64_t K, void* stream) {
  int rc = gemm_common(ctx, d_g_codes, d_alpha, d_g_operand, d_a_codes, d_sa, d_a_operand, d_dw, M, N, K, n_samples);
  if (rc) return rc;
  if (N % 32 || K % 32) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  luq_gemm_args a{};
  a.a_codes = d_g_codes; a.a_kind = ctx->grad_int4 ? 0 : 1; a.a_mn = 1; a.n_samples = n_samples;   // G[M x N]: rows are the contraction
  a.b_codes = d_a_codes; a.b_kind = ctx->unsigned_act ? 2 : 0; a.b_mn = 1;    // A[M x K]: rows are the contraction
  a.a_operand = d_g_operand; a.b_operand = d_a_operand;
  a.a_summed = (ctx->sum_samples && !ctx->grad_int4 && d_g_operand && n_samples > 1) ? n_samples : 0;
  a.d_scale_a = d_alpha; a.d_scale_b = d_sa; a.d_out = d_dw; a.out_bf16 = ctx->out_bf16; a.Mo = N; a.No = K; a.Kc = M;
  a.d_workspace = ctx->d_workspace; a.workspace_bytes = ctx->workspace_bytes;
  a.allow_split = 1;
  return cuda_rc(luq_launch_gemm(ctx, a, as_stream(stream)));
}

int luq_status(luq_ctx* ctx, void* stream, int* host_flags) {
  if (!ctx || !host_flags) return LUQ_ERR_ARG;
  DeviceGuard guard(ctx->device);
  if (!guard.ok) return LUQ_ERR_CUDA;
  cudaStream_t st = as_stream(stream);
  unsigned int flags = 0;
  if (cudaMemcpyAsync(&flags, ctx->d_status, sizeof(flags), cudaMemcpyDeviceToHost, st) != cudaSuccess) return LUQ_ERR_CUDA;
  if (cudaStreamSynchronize(st) != cudaSuccess) return LUQ_ERR_CUDA;
  if (flags) {
    // a grid barrier that gave up leaves its counters behind: clear them with the status word
    if ((flags & LUQ_STATUS_TIMEOUT) &&
        cudaMemsetAsync(ctx->d_scratch, 0, 2 * sizeof(unsigned int), st) != cudaSuccess) return LUQ_ERR_CUDA;
    if (cudaMemsetAsync(ctx->d_status, 0, sizeof(unsigned int), st) != cudaSuccess) return LUQ_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return LUQ_ERR_CUDA;
  }
  *host_flags = static_cast<int>(flags);
  return LUQ_OK;
}

}  // extern "C"
