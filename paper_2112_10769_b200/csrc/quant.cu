// Memory-bound kernels of the path: tensor max, INT4 round-to-nearest
// quantize-and-pack, LUQ stochastic quantize-and-pack (Philox, n samples).
//
// All three stream the input once.  The unit of work is one 16-byte load
// (4 fp32 or 8 bf16 elements); consecutive lanes take consecutive 16-byte
// pieces, so every load instruction of a warp covers 512 contiguous bytes and
// the packed codes leave as contiguous 64- or 128-byte warp stores.  Grids are
// sized to the number of CTAs the GPU holds at once (SM count x occupancy) and
// walk the tensor with a grid-stride loop, several loads in flight per thread.
//
// Compile this file without FMA contraction and with IEEE division: code
// decisions must be bit-identical to a scalar IEEE implementation.
#include "common.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;  // independent 16-byte loads in flight per thread

// zero, non-finite or far-out-of-range max: every code is zero, the scale is zero
__device__ __forceinline__ bool scale_usable(float c, unsigned int* status) {
  const uint32_t b = __float_as_uint(c);
  if (c == 0.0f) return false;
  if ((b & 0x7FFFFFFFu) >= 0x7F800000u || (b >> 31)) {
    if (status) atomicOr(status, LUQ_STATUS_NONFINITE);
    return false;
  }
  if (c < 0x1p-100f || c > 0x1p100f) {
    if (status) atomicOr(status, LUQ_STATUS_RANGE);
    return false;
  }
  return true;
}

template <bool BF16> struct Item {
  static constexpr int kElems = BF16 ? 8 : 4;  // elements per 16-byte piece
  // widen one piece to fp32 (bf16 -> fp32 is exact: bits << 16)
  static __device__ __forceinline__ void widen(const uint4& u, float (&v)[kElems]) {
    if constexpr (BF16) {
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xFFFF0000u);
      }
    } else {
      v[0] = __uint_as_float(u.x); v[1] = __uint_as_float(u.y);
      v[2] = __uint_as_float(u.z); v[3] = __uint_as_float(u.w);
    }
  }
  static __device__ __forceinline__ float load1(const void* base, size_t i) {
    if constexpr (BF16)
      return __uint_as_float(static_cast<uint32_t>(reinterpret_cast<const uint16_t*>(base)[i]) << 16);
    else
      return reinterpret_cast<const float*>(base)[i];
  }
  // store the packed codes of one piece (2 bytes for fp32 input, 4 for bf16)
  static __device__ __forceinline__ void store(uint8_t* plane_base, size_t item, uint32_t word, bool aligned) {
    if (aligned) {
      if constexpr (BF16) reinterpret_cast<uint32_t*>(plane_base)[item] = word;
      else reinterpret_cast<uint16_t*>(plane_base)[item] = static_cast<uint16_t>(word);
    } else {
#pragma unroll
      for (int b = 0; b < kElems / 2; ++b) plane_base[item * (kElems / 2) + b] = static_cast<uint8_t>(word >> (8 * b));
    }
  }
};

// ------------------------------------------------------------------ amax ----
// |x| as an unsigned bit pattern is monotone in |x| for finite values, and every
// Inf/NaN pattern is larger than every finite one: one unsigned max does both
// the reduction and the non-finite detection.  Warp shuffle reduction (redux),
// then one shared-memory step per block, then one atomicMax per block.
template <bool BF16>
__global__ void __launch_bounds__(kThreads) amax_kernel(const void* __restrict__ x, size_t n,
                                                        unsigned int* __restrict__ out_bits,
                                                        unsigned int* __restrict__ status) {
  constexpr int kElems = Item<BF16>::kElems;
  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);
  uint32_t m = 0;
  auto fold = [&](const uint4& u) {
    if constexpr (BF16) {
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        m = max(m, (w[j] << 16) & 0x7FFFFFFFu);
        m = max(m, w[j] & 0x7FFF0000u);
      }
    } else {
      m = max(m, u.x & 0x7FFFFFFFu); m = max(m, u.y & 0x7FFFFFFFu);
      m = max(m, u.z & 0x7FFFFFFFu); m = max(m, u.w & 0x7FFFFFFFu);
    }
  };
  const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
  size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x;
  for (; i + (kUnroll - 1) * stride < items; i += kUnroll * stride) {
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) u[j] = __ldg(p + i + j * stride);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) fold(u[j]);
  }
  for (; i < items; i += stride) fold(__ldg(p + i));
  // ragged tail: fewer elements than one piece
  if (blockIdx.x == 0 && threadIdx.x < n - items * kElems)
    m = max(m, __float_as_uint(Item<BF16>::load1(x, items * kElems + threadIdx.x)) & 0x7FFFFFFFu);

  m = __reduce_max_sync(0xFFFFFFFFu, m);
  __shared__ uint32_t warp_max[kThreads / 32];
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (threadIdx.x == 0 && m != 0) {
      atomicMax(out_bits, m);
      if (m >= 0x7F800000u) atomicOr(status, LUQ_STATUS_NONFINITE);
    }
  }
}

// ------------------------------------------------------------------ INT4 ----
__device__ __forceinline__ uint32_t int4_code(float x, float inv) {
  const float y = x * inv;
  float r = rintf(y);                 // nearest, ties to even
  r = fminf(fmaxf(r, -7.0f), 7.0f);
  if (y != y) r = 0.0f;               // NaN element -> 0
  return static_cast<uint32_t>(static_cast<int>(r)) & 0xFu;
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads) quant_int4_kernel(const void* __restrict__ x, size_t n,
                                                              const float* __restrict__ d_clip,
                                                              uint8_t* __restrict__ codes,
                                                              float* __restrict__ d_scale,
                                                              unsigned int* __restrict__ status) {
  constexpr int kElems = Item<BF16>::kElems;
  const float clip = __ldg(d_clip);
  const bool first = blockIdx.x == 0 && threadIdx.x == 0;
  const bool ok = scale_usable(clip, first ? status : nullptr);
  const float inv = ok ? 7.0f / clip : 0.0f;
  if (first) *d_scale = ok ? clip / 7.0f : 0.0f;

  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);
  auto encode = [&](const uint4& u) -> uint32_t {
    if (!ok) return 0u;
    float v[kElems];
    Item<BF16>::widen(u, v);
    uint32_t word = 0;
#pragma unroll
    for (int j = 0; j < kElems; ++j) word |= int4_code(v[j], inv) << (4 * j);
    return word;
  };
  const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
  size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x;
  for (; i + (kUnroll - 1) * stride < items; i += kUnroll * stride) {
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) u[j] = __ldg(p + i + j * stride);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) Item<BF16>::store(codes, i + j * stride, encode(u[j]), true);
  }
  for (; i < items; i += stride) Item<BF16>::store(codes, i, encode(__ldg(p + i)), true);
  if (first) {  // tail: fewer elements than one piece, two per byte
    for (size_t e = items * kElems; e < n; e += 2) {
      const uint32_t lo = ok ? int4_code(Item<BF16>::load1(x, e), inv) : 0u;
      const uint32_t hi = (ok && e + 1 < n) ? int4_code(Item<BF16>::load1(x, e + 1), inv) : 0u;
      codes[e >> 1] = static_cast<uint8_t>(lo | (hi << 4));
    }
  }
}

// ------------------------------------------------------------------- LUQ ----
// Philox4x32-10: counter-based generator, ten rounds of two 32x32->64 multiplies
// with a Weyl key schedule.  The key is the same for the whole tensor, so the
// round keys are loop-invariant.
struct PhiloxKeys { uint32_t k0[10]; uint32_t k1[10]; };

__device__ __forceinline__ PhiloxKeys philox_keys(uint64_t key) {
  PhiloxKeys ks;
  uint32_t a = static_cast<uint32_t>(key), b = static_cast<uint32_t>(key >> 32);
#pragma unroll
  for (int r = 0; r < 10; ++r) { ks.k0[r] = a; ks.k1[r] = b; a += 0x9E3779B9u; b += 0xBB67AE85u; }
  return ks;
}

__device__ __forceinline__ uint4 philox_block(uint64_t block, const PhiloxKeys& ks) {
  uint32_t c0 = static_cast<uint32_t>(block), c1 = static_cast<uint32_t>(block >> 32), c2 = 0u, c3 = 0u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
    const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
    c0 = hi1 ^ c1 ^ ks.k0[r];
    c1 = lo1;
    c2 = hi0 ^ c3 ^ ks.k1[r];
    c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// Per element: lower code and the 32-bit threshold of the up-decision.
//   t = |x| / alpha (IEEE quotient).  t < 1: code 0, threshold trunc(t * 2^32)
//   (prune-up probability |x|/alpha).  t >= 1: code 1 + exponent(t), threshold
//   = mantissa field << 9 (up-probability (|x| - lo)/lo); at or above the top
//   level the code is kmax + 1 with no draw.
__device__ __forceinline__ void luq_bin(float x, float alpha, uint32_t& lo_code, uint32_t& thr) {
  const float t = __fdiv_rn(fabsf(x), alpha);
  const uint32_t u = __float_as_uint(t);
  if (t < 1.0f) {
    lo_code = 0;
    thr = __float2uint_rz(t * 4294967296.0f);
  } else {
    const int e = static_cast<int>((u >> 23) & 0xFFu) - 127;
    if (e >= LUQ_KMAX) { lo_code = LUQ_KMAX + 1; thr = 0; }
    else { lo_code = 1 + e; thr = (u & 0x7FFFFFu) << 9; }
  }
}

__device__ __forceinline__ uint32_t luq_nibble(uint32_t sign, uint32_t lo_code, uint32_t thr, uint32_t word) {
  const uint32_t c = lo_code + (word < thr ? 1u : 0u);
  return c ? ((sign << 3) | c) : 0u;
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads) quant_luq_kernel(const void* __restrict__ x, size_t n,
                                                             const float* __restrict__ d_amax,
                                                             uint64_t seed, int n_samples,
                                                             uint8_t* __restrict__ codes,
                                                             float* __restrict__ d_alpha,
                                                             unsigned int* __restrict__ status) {
  constexpr int kElems = Item<BF16>::kElems;
  const float mx = __ldg(d_amax);
  const bool first = blockIdx.x == 0 && threadIdx.x == 0;
  const bool ok = scale_usable(mx, first ? status : nullptr);
  const float alpha = ok ? mx * (1.0f / static_cast<float>(1 << LUQ_KMAX)) : 0.0f;  // exact scaling
  if (first) *d_alpha = alpha;

  const size_t plane = n / 2;
  const bool aligned = (plane % (kElems / 2)) == 0;  // planes start on a store boundary
  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);

  auto process = [&](size_t item, const uint4& u) {
    float v[kElems];
    uint32_t lo_code[kElems], thr[kElems], sign[kElems];
    Item<BF16>::widen(u, v);
#pragma unroll
    for (int j = 0; j < kElems; ++j) {
      luq_bin(v[j], alpha, lo_code[j], thr[j]);
      sign[j] = __float_as_uint(v[j]) >> 31;
    }
    for (int s = 0; s < n_samples; ++s) {
      const PhiloxKeys ks = philox_keys(seed + static_cast<uint64_t>(s));
      uint32_t word = 0;
#pragma unroll
      for (int b = 0; b < kElems / 4; ++b) {
        const uint4 r = philox_block(item * (kElems / 4) + b, ks);
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j)
          word |= luq_nibble(sign[4 * b + j], lo_code[4 * b + j], thr[4 * b + j], rw[j]) << (4 * (4 * b + j));
      }
      Item<BF16>::store(codes + plane * s, item, word, aligned || s == 0);
    }
  };

  const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
  size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x;
  if (ok) {
    for (; i + stride < items; i += 2 * stride) {
      const uint4 u0 = __ldg(p + i), u1 = __ldg(p + i + stride);
      process(i, u0);
      process(i + stride, u1);
    }
    for (; i < items; i += stride) process(i, __ldg(p + i));
  } else {
    for (; i < items; i += stride)
      for (int s = 0; s < n_samples; ++s) Item<BF16>::store(codes + plane * s, i, 0u, aligned || s == 0);
  }
  if (first) {  // tail: fewer elements than one piece, two per byte
    for (int s = 0; s < n_samples; ++s) {
      const PhiloxKeys ks = philox_keys(seed + static_cast<uint64_t>(s));
      for (size_t e = items * kElems; e < n; e += 2) {
        uint32_t nib[2] = {0u, 0u};
        for (int h = 0; h < 2; ++h) {
          const size_t idx = e + h;
          if (ok && idx < n) {
            const float xv = Item<BF16>::load1(x, idx);
            uint32_t lc, th;
            luq_bin(xv, alpha, lc, th);
            const uint4 r = philox_block(idx >> 2, ks);
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
            nib[h] = luq_nibble(__float_as_uint(xv) >> 31, lc, th, rw[idx & 3]);
          }
        }
        codes[plane * s + (e >> 1)] = static_cast<uint8_t>(nib[0] | (nib[1] << 4));
      }
    }
  }
}

// CTAs the GPU holds at once for `kernel`, capped by the work available
template <typename K>
int grid_for(const luq_ctx* ctx, K kernel, size_t thread_items) {
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  size_t want = (thread_items + kThreads - 1) / kThreads;
  const size_t cap = static_cast<size_t>(ctx->sm_count) * per_sm;
  if (want < 1) want = 1;
  return static_cast<int>(want < cap ? want : cap);
}

}  // namespace

int luq_launch_amax(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_amax, cudaStream_t st) {
  cudaError_t e = cudaMemsetAsync(d_amax, 0, sizeof(float), st);
  if (e != cudaSuccess) return static_cast<int>(e);
  if (n == 0) return 0;
  if (dtype == LUQ_BF16) {
    const int grid = grid_for(ctx, amax_kernel<true>, n / 8 / kUnroll + 1);
    amax_kernel<true><<<grid, kThreads, 0, st>>>(d_x, n, reinterpret_cast<unsigned int*>(d_amax), ctx->d_status);
  } else {
    const int grid = grid_for(ctx, amax_kernel<false>, n / 4 / kUnroll + 1);
    amax_kernel<false><<<grid, kThreads, 0, st>>>(d_x, n, reinterpret_cast<unsigned int*>(d_amax), ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(cudaGetLastError());
}

int luq_launch_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t n, const float* d_clip,
                          uint8_t* d_codes, float* d_scale, cudaStream_t st) {
  if (dtype == LUQ_BF16) {
    const int grid = grid_for(ctx, quant_int4_kernel<true>, n / 8 / kUnroll + 1);
    quant_int4_kernel<true><<<grid, kThreads, 0, st>>>(d_x, n, d_clip, d_codes, d_scale, ctx->d_status);
  } else {
    const int grid = grid_for(ctx, quant_int4_kernel<false>, n / 4 / kUnroll + 1);
    quant_int4_kernel<false><<<grid, kThreads, 0, st>>>(d_x, n, d_clip, d_codes, d_scale, ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(cudaGetLastError());
}

int luq_launch_quant_grad(luq_ctx* ctx, const void* d_g, int dtype, size_t n, const float* d_amax,
                          uint64_t seed, int n_samples, uint8_t* d_codes, float* d_alpha, cudaStream_t st) {
  if (dtype == LUQ_BF16) {
    const int grid = grid_for(ctx, quant_luq_kernel<true>, n / 8 / 2 + 1);
    quant_luq_kernel<true><<<grid, kThreads, 0, st>>>(d_g, n, d_amax, seed, n_samples, d_codes, d_alpha,
                                                      ctx->d_status);
  } else {
    const int grid = grid_for(ctx, quant_luq_kernel<false>, n / 4 / 2 + 1);
    quant_luq_kernel<false><<<grid, kThreads, 0, st>>>(d_g, n, d_amax, seed, n_samples, d_codes, d_alpha,
                                                       ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(cudaGetLastError());
}
