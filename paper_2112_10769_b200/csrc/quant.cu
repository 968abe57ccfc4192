// Memory-bound kernels of the path: tensor max, INT4 round-to-nearest
// quantize-and-pack (signed, and unsigned for non-negative tensors), LUQ stochastic
// quantize-and-pack (Philox, n samples) with its variants: power-of-two scale,
// in-hindsight maximum, other level counts, deterministic nearest power, and the
// ablation's other gradient quantizers (one region deterministic; uniform grid with
// stochastic rounding).
//
// All stream the input once.  The unit of work is one 16-byte load
// (4 fp32 or 8 bf16 elements); consecutive lanes take consecutive 16-byte
// pieces, so every load instruction of a warp covers 512 contiguous bytes and
// the packed codes leave as contiguous 64- or 128-byte warp stores.  Grids are
// sized to the number of CTAs the GPU holds at once (SM count x occupancy) and
// walk the tensor in contiguous 16 KB tiles, several loads in flight per thread.
// Every quantizer can also write the codes' 8-bit tensor-core form ("operand
// bytes") in the same pass, and can be launched "fused": it then reduces the
// tensor's maximum itself (first phase, grid barrier) instead of reading it.
//
// Compile this file without FMA contraction and with IEEE division: code
// decisions must be bit-identical to a scalar IEEE implementation.
#include "common.cuh"
#include "int4_math.cuh"

namespace {

constexpr int kThreads = 256;
constexpr int kUnroll = 4;  // independent 16-byte loads in flight per thread
// A block walks the tensor in contiguous tiles of kThreads * kUnroll pieces (16 KB):
// the loads a thread has in flight are 4 KB apart, inside one DRAM page neighbourhood.
constexpr int kTileItems = kThreads * kUnroll;

using luqdev::scale_usable;
using luqdev::int4_code;
using luqdev::uint4_code;
using luqdev::hindsight_next;

// checking build: is piece `idx` one of the tensor's `items` 16-byte pieces?  (a violation raises
// LUQ_STATUS_BOUNDS and the caller skips the access; always true, and free, in the normal build)
__device__ __forceinline__ bool piece_ok(size_t idx, size_t items, unsigned int* status) {
  (void)idx; (void)items; (void)status;
  return LUQ_IN_BOUNDS(idx < items, status);
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
  // store the operand bytes of one piece (4 bytes for fp32 input, 8 for bf16); w[j] holds elements 4j..4j+3
  static __device__ __forceinline__ void store_bytes(int8_t* bytes_base, size_t item, const uint32_t (&w)[kElems / 4],
                                                     bool aligned) {
    if (aligned) {
      if constexpr (BF16) reinterpret_cast<uint2*>(bytes_base)[item] = make_uint2(w[0], w[1]);
      else reinterpret_cast<uint32_t*>(bytes_base)[item] = w[0];
    } else {
#pragma unroll
      for (int b = 0; b < kElems; ++b) bytes_base[item * kElems + b] = static_cast<int8_t>(w[b / 4] >> (8 * (b % 4)));
    }
  }
};

// Grid-wide maximum without a pre-zeroed output: every block leaves its maximum in the
// context's scratch array and takes a ticket; the block that draws the last ticket reduces the
// array, resets the ticket counter and returns true in its thread 0 with the result in `m`.
// `rank` of `count` is the block's place among the blocks that work on this tensor (the whole grid,
// or a share of it in the kernels that take several tensors in one launch).
// scratch[0] is the ticket counter (zero between kernels), scratch[1] the departure counter of
// the fused kernels' grid barrier, scratch[2 + b] block b's maximum.
__device__ __forceinline__ bool grid_max_last_block(uint32_t& m, unsigned int* scratch, unsigned int rank,
                                                    unsigned int count) {
  __shared__ uint32_t warp_max[kThreads / 32];
  __shared__ bool last;
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (threadIdx.x == 0) {
      __stcg(scratch + 2 + rank, m);
      __threadfence();
      last = atomicAdd(scratch, 1u) == count - 1;
    }
  }
  __syncthreads();
  if (!last) return false;
  __threadfence();
  m = 0;
  for (unsigned int b = threadIdx.x; b < count; b += kThreads) m = max(m, __ldcg(scratch + 2 + b));
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  __syncthreads();            // warp_max is reused
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (threadIdx.x == 0) { *scratch = 0u; return true; }
  }
  return false;
}


// ------------------------------------------------------------------ amax ----
// |x| as an unsigned bit pattern is monotone in |x| for finite values, and every
// Inf/NaN pattern is larger than every finite one: one unsigned max does both
// the reduction and the non-finite detection.  Warp shuffle reduction (redux),
// then one shared-memory step per block, then the last block to finish reduces the
// block maxima (no pre-zeroed output, no atomics on it).
constexpr int kAmaxUnroll = 4;
constexpr int kAmaxCtasPerSm = 8;
template <bool BF16>
__device__ __forceinline__ void amax_body(const void* __restrict__ x, size_t n, unsigned int* __restrict__ out_bits,
                                          unsigned int* __restrict__ scratch, unsigned int* __restrict__ status,
                                          unsigned int rank, unsigned int count) {
  constexpr int kElems = Item<BF16>::kElems;
  constexpr int kUnroll = kAmaxUnroll;
  constexpr int kTileItems = kThreads * kUnroll;
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
  const size_t full_tiles = items / kTileItems;
  for (size_t t = rank; t < full_tiles; t += count) {
    const uint4* q = p + t * kTileItems + threadIdx.x;
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j)
      u[j] = piece_ok(t * kTileItems + threadIdx.x + j * kThreads, items, status) ? __ldg(q + j * kThreads) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) fold(u[j]);
  }
  if (rank == count - 1)   // pieces after the last full tile
    for (size_t i = full_tiles * kTileItems + threadIdx.x; i < items; i += kThreads) fold(__ldg(p + i));
  // ragged tail: fewer elements than one piece
  if (rank == 0 && threadIdx.x < n - items * kElems)
    m = max(m, __float_as_uint(Item<BF16>::load1(x, items * kElems + threadIdx.x)) & 0x7FFFFFFFu);

  if (grid_max_last_block(m, scratch, rank, count)) {
    *out_bits = m;
    if (m >= 0x7F800000u) atomicOr(status, LUQ_STATUS_NONFINITE);
  }
}

template <bool BF16>
__global__ void __launch_bounds__(kThreads) amax_kernel(const void* __restrict__ x, size_t n,
                                                        unsigned int* __restrict__ out_bits,
                                                        unsigned int* __restrict__ scratch,
                                                        unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  amax_body<BF16>(x, n, out_bits, scratch, status, blockIdx.x, gridDim.x);
}

// Several tensors in one launch (a layer's activations and weights, say): the blocks are dealt out
// to the tensors in proportion to their sizes, each tensor has its own 1024-word region of the
// scratch array.  A small tensor's launch and reduction latency hides behind the large one's stream.
constexpr int kMultiMax = LUQ_SCRATCH_MULTI;
struct MultiAmax {
  const void* x[kMultiMax]; size_t n[kMultiMax]; unsigned int* out[kMultiMax];
  unsigned int first_block[kMultiMax + 1]; int count;
};
template <bool BF16>
__global__ void __launch_bounds__(kThreads) amax_multi_kernel(const __grid_constant__ MultiAmax a,
                                                              unsigned int* __restrict__ scratch,
                                                              unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  int t = 0;
  while (t + 1 < a.count && blockIdx.x >= a.first_block[t + 1]) ++t;
  amax_body<BF16>(a.x[t], a.n[t], a.out[t], scratch + LUQ_SCRATCH_SINGLE + t * LUQ_SCRATCH_REGION, status,
                  blockIdx.x - a.first_block[t], a.first_block[t + 1] - a.first_block[t]);
}

// ------------------------------------------------- fused max (phase one) ----
// A quantizer launched "fused" first reduces max|x| itself: every block folds its share of the
// tensor, leaves its maximum in the scratch array and waits at a grid barrier; then every block
// reduces the array, so all of them hold the tensor's maximum without a second launch.  The
// launch is cooperative (one wave, all blocks resident).  The wait is bounded: when it expires
// the block raises LUQ_STATUS_TIMEOUT and the kernel returns without writing codes.
constexpr uint32_t kBarrierPolls = 4u << 20;   // x 200 ns of sleep: the better part of a second

template <bool BF16>
__device__ __forceinline__ bool fused_grid_max(const void* __restrict__ x, size_t n, unsigned int* scratch,
                                               unsigned int* status, uint32_t& result) {
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
  const size_t full_tiles = items / kTileItems;
  for (size_t t = blockIdx.x; t < full_tiles; t += gridDim.x) {   // front to back; phase two walks back to front
    const uint4* q = p + t * kTileItems + threadIdx.x;
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) u[j] = __ldg(q + j * kThreads);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) fold(u[j]);
  }
  if (blockIdx.x == gridDim.x - 1)
    for (size_t i = full_tiles * kTileItems + threadIdx.x; i < items; i += kThreads) fold(__ldg(p + i));
  if (blockIdx.x == 0 && threadIdx.x < n - items * kElems)
    m = max(m, __float_as_uint(Item<BF16>::load1(x, items * kElems + threadIdx.x)) & 0x7FFFFFFFu);

  __shared__ uint32_t warp_max[kThreads / 32];
  __shared__ uint32_t arrived;
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  if (threadIdx.x < 32) {
    m = threadIdx.x < kThreads / 32 ? warp_max[threadIdx.x] : 0u;
    m = __reduce_max_sync(0xFFFFFFFFu, m);
    if (threadIdx.x == 0) {
      __stcg(scratch + 2 + blockIdx.x, m);
      __threadfence();
      atomicAdd(scratch, 1u);
      uint32_t seen = 0, polls = 0;
      for (;;) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(scratch) : "memory");
        if (seen >= gridDim.x || ++polls > kBarrierPolls) break;
        __nanosleep(200);
      }
      arrived = seen;
    }
  }
  __syncthreads();
  if (arrived < gridDim.x) {                    // the barrier gave up: some block never arrived
    if (threadIdx.x == 0) atomicOr(status, LUQ_STATUS_TIMEOUT);
    return false;
  }
  __threadfence();
  m = 0;
  for (unsigned int b = threadIdx.x; b < gridDim.x; b += kThreads) m = max(m, __ldcg(scratch + 2 + b));
  m = __reduce_max_sync(0xFFFFFFFFu, m);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = m;
  __syncthreads();
  m = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) m = max(m, warp_max[w]);
  // the last block to leave the barrier resets both counters for the next kernel
  if (threadIdx.x == 0 && atomicAdd(scratch + 1, 1u) == gridDim.x - 1) { scratch[0] = 0u; scratch[1] = 0u; }
  result = m;
  return true;
}

// ------------------------------------------------------------------ INT4 ----
// PLANE: the tensor-core operand bytes (int8, 16 * q: the code nibble in the high half of the
// byte) are written next to the packed codes, one byte per element in element order.
// UNSIGNED: the grid 0..15 with scale clip / 15 (non-negative tensors); operand byte = q.
// TRACK: in-hindsight range - `clip` is an estimate from earlier steps (values beyond it saturate),
// the tensor's own max|x| is reduced on the way; the block that finishes last writes it to
// *measured_bits and replaces *d_estimate by (1 - eta) * measured + eta * estimate.
template <bool BF16, bool PLANE, bool UNSIGNED, bool TRACK = false>
__device__ __forceinline__ void quant_int4_body(const void* __restrict__ x, size_t n, float clip,
                                                uint8_t* __restrict__ codes, int8_t* __restrict__ operand,
                                                float* __restrict__ d_scale, unsigned int* __restrict__ status,
                                                unsigned int rank, unsigned int count,
                                                unsigned int* __restrict__ measured_bits = nullptr,
                                                float* d_estimate = nullptr, float eta = 0.0f,
                                                unsigned int* scratch = nullptr) {
  constexpr int kElems = Item<BF16>::kElems;
  const bool first = rank == 0 && threadIdx.x == 0;
  const bool ok = scale_usable(clip, first ? status : nullptr);
  constexpr float kTop = UNSIGNED ? 15.0f : 7.0f;
  constexpr int kByteShift = UNSIGNED ? 0 : 4;
  const float inv = ok ? kTop / clip : 0.0f;
  if (first) *d_scale = ok ? clip / kTop : 0.0f;
  auto code_of = [&](float v) { return UNSIGNED ? uint4_code(v, inv) : int4_code(v, inv); };
  uint32_t seen = 0;   // running max of |x| bit patterns (TRACK)

  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);
  auto emit = [&](size_t item, const uint4& u) {
    float v[kElems];
    Item<BF16>::widen(u, v);
    uint32_t word = 0;
    uint32_t bytes[kElems / 4] = {};
#pragma unroll
    for (int j = 0; j < kElems; ++j) {
      if constexpr (TRACK) seen = max(seen, __float_as_uint(v[j]) & 0x7FFFFFFFu);
      const uint32_t code = ok ? code_of(v[j]) : 0u;
      word |= code << (4 * j);
      if constexpr (PLANE) bytes[j / 4] |= code << (8 * (j % 4) + kByteShift);
    }
    Item<BF16>::store(codes, item, word, true);
    if constexpr (PLANE) Item<BF16>::store_bytes(operand, item, bytes, true);
  };
  // The tensor was just read front to back by the max reduction; its tail is what the
  // L2 still holds, so this pass walks the tiles from the back.
  const size_t full_tiles = items / kTileItems;
  for (size_t t = rank; t < full_tiles; t += count) {
    const size_t i0 = (full_tiles - 1 - t) * kTileItems + threadIdx.x;
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j)
      u[j] = piece_ok(i0 + j * kThreads, items, status) ? __ldg(p + i0 + j * kThreads) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j)
      if (piece_ok(i0 + j * kThreads, items, status)) emit(i0 + j * kThreads, u[j]);
  }
  if (rank == count - 1)
    for (size_t i = full_tiles * kTileItems + threadIdx.x; i < items; i += kThreads) emit(i, __ldg(p + i));
  if (first) {  // tail: fewer elements than one piece, two per byte
    for (size_t e = items * kElems; e < n; e += 2) {
      if constexpr (TRACK) {
        seen = max(seen, __float_as_uint(Item<BF16>::load1(x, e)) & 0x7FFFFFFFu);
        if (e + 1 < n) seen = max(seen, __float_as_uint(Item<BF16>::load1(x, e + 1)) & 0x7FFFFFFFu);
      }
      const uint32_t lo = ok ? code_of(Item<BF16>::load1(x, e)) : 0u;
      const uint32_t hi = (ok && e + 1 < n) ? code_of(Item<BF16>::load1(x, e + 1)) : 0u;
      codes[e >> 1] = static_cast<uint8_t>(lo | (hi << 4));
      if constexpr (PLANE) {
        operand[e] = static_cast<int8_t>(lo << kByteShift);
        if (e + 1 < n) operand[e + 1] = static_cast<int8_t>(hi << kByteShift);
      }
    }
  }
  if constexpr (TRACK) {   // Inf/NaN patterns win the maximum and raise the flag
    if (grid_max_last_block(seen, scratch, rank, count)) {
      *measured_bits = seen;
      if (seen >= 0x7F800000u) atomicOr(status, LUQ_STATUS_NONFINITE);
      *d_estimate = hindsight_next(seen, clip, eta);
    }
  }
}

// in-hindsight INT4: d_estimate is read as the clip by every block and replaced by the last one
template <bool BF16, bool PLANE>
__global__ void __launch_bounds__(kThreads) quant_int4_track_kernel(const void* __restrict__ x, size_t n,
                                                                    float* d_estimate, float eta,
                                                                    uint8_t* __restrict__ codes,
                                                                    int8_t* __restrict__ operand,
                                                                    float* __restrict__ d_scale,
                                                                    unsigned int* __restrict__ measured_bits,
                                                                    unsigned int* scratch,
                                                                    unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  const float clip = *d_estimate;
  quant_int4_body<BF16, PLANE, false, true>(x, n, clip, codes, operand, d_scale, status, blockIdx.x, gridDim.x,
                                            measured_bits, d_estimate, eta, scratch);
}

template <bool BF16, bool PLANE, bool UNSIGNED>
__global__ void __launch_bounds__(kThreads) quant_int4_kernel(const void* __restrict__ x, size_t n,
                                                              const float* d_clip,
                                                              uint8_t* __restrict__ codes,
                                                              int8_t* __restrict__ operand,
                                                              float* __restrict__ d_scale,
                                                              float* d_amax_out, unsigned int* scratch,
                                                              unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  float clip;
  if (d_amax_out != nullptr) {   // fused: the clip is this tensor's maximum, reduced here
    uint32_t bits;
    if (!fused_grid_max<BF16>(x, n, scratch, status, bits)) return;
    clip = __uint_as_float(bits);
    if (blockIdx.x == 0 && threadIdx.x == 0) *d_amax_out = clip;
  } else {
    clip = *d_clip;
  }
  quant_int4_body<BF16, PLANE, UNSIGNED>(x, n, clip, codes, operand, d_scale, status, blockIdx.x, gridDim.x);
}

// several tensors in one launch, see amax_multi_kernel; a tensor without operand bytes passes null
struct MultiInt4 {
  const void* x[kMultiMax]; size_t n[kMultiMax]; const float* clip[kMultiMax]; uint8_t* codes[kMultiMax];
  int8_t* operand[kMultiMax]; float* scale[kMultiMax];
  unsigned int first_block[kMultiMax + 1]; int count;
};
template <bool BF16>
__global__ void __launch_bounds__(kThreads) quant_int4_multi_kernel(const __grid_constant__ MultiInt4 a,
                                                                    unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  int t = 0;
  while (t + 1 < a.count && blockIdx.x >= a.first_block[t + 1]) ++t;
  const unsigned int rank = blockIdx.x - a.first_block[t], count = a.first_block[t + 1] - a.first_block[t];
  const float clip = *a.clip[t];
  if (a.operand[t] != nullptr)
    quant_int4_body<BF16, true, false>(a.x[t], a.n[t], clip, a.codes[t], a.operand[t], a.scale[t], status, rank, count);
  else
    quant_int4_body<BF16, false, false>(a.x[t], a.n[t], clip, a.codes[t], nullptr, a.scale[t], status, rank, count);
}

// ------------------------------------------------------------------- LUQ ----
// Philox4x32-10: counter-based generator, ten rounds of two 32x32->64 multiplies
// with a Weyl key schedule.  The key is the same for the whole tensor: the host
// expands it into the ten round keys of every sample and passes them as kernel
// parameters, so a round is two wide multiplies and two three-input XORs.
struct PhiloxKeys { uint32_t k0[10]; uint32_t k1[10]; };
// Per-launch constants of the LUQ kernel: the round keys of every sample, and the grid.
//   inv_levels = 2^-kmax (alpha = max * inv_levels), q_top = 2^(32 + kmax) (the top level on the
//   scale of Q).  fixed_word != 0 replaces every random word by that constant: with 0x7FFFFFFF
//   an element goes up exactly when its up-probability is at least 1/2, which is deterministic
//   round-to-nearest-power (Eq. RC), ties up.
struct PhiloxKeySet { PhiloxKeys s[LUQ_MAX_SAMPLES]; uint32_t fixed_word; float inv_levels; float q_top; };

__device__ __forceinline__ void mul_wide(uint32_t a, uint32_t b, uint32_t& lo, uint32_t& hi) {
  asm("{\n\t.reg .b64 t;\n\tmul.wide.u32 t, %2, %3;\n\tmov.b64 {%0, %1}, t;\n\t}" : "=r"(lo), "=r"(hi) : "r"(a), "r"(b));
}

__device__ __forceinline__ uint4 philox_block(uint64_t block, const PhiloxKeys& ks) {
  uint32_t c0 = static_cast<uint32_t>(block), c1 = static_cast<uint32_t>(block >> 32), c2 = 0u, c3 = 0u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint32_t lo0, hi0, lo1, hi1;
    mul_wide(0xD2511F53u, c0, lo0, hi0);
    mul_wide(0xCD9E8D57u, c2, lo1, hi1);
    c0 = hi1 ^ c1 ^ ks.k0[r];
    c1 = lo1;
    c2 = hi0 ^ c3 ^ ks.k1[r];
    c3 = lo0;
  }
  return make_uint4(c0, c1, c2, c3);
}

// The scale of one tensor, prepared once per thread.
//   alpha = max / 2^kmax (exact).  Every decision is a function of the IEEE round-to-nearest
//   quotient t = |x| / alpha, and is taken on Q = t * 2^32 = RN(|x| / beta) with
//   beta = alpha * 2^-32: scaling by a power of two commutes with the rounding, and the
//   32-bit threshold of an underflow element is simply trunc(Q).
//   With y = RN(1/beta) (correctly rounded) Q is obtained without a division: q0 = a*y is
//   within 1.5 ulp, one residual correction makes it faithful, a second one (residual now
//   exact) makes it correctly rounded (Markstein).  The residuals are exact as long as they
//   do not fall below the denormal grid, which holds for alpha >= 2^-71; for a smaller
//   alpha ("tiny") both operands are first scaled by 2^64 (exact).
struct LuqScale { float beta, recip, pre; bool tiny; };

__device__ __forceinline__ LuqScale luq_scale(float alpha) {
  LuqScale sc;
  sc.tiny = alpha < 0x1p-60f;
  sc.pre = sc.tiny ? 0x1p64f : 1.0f;
  sc.beta = alpha * sc.pre * 0x1p-32f;       // exact: alpha lies in [2^-104, 2^96]
  sc.recip = __frcp_rn(sc.beta);
  return sc;
}

// Q for a = |x| * pre (the caller applies pre; it is 1 unless the scale is tiny)
template <bool PW2 = false>
__device__ __forceinline__ float luq_scaled_quotient(float a, const LuqScale& sc) {
  if constexpr (PW2) return a * sc.recip;   // beta is a power of two: one exact scaling
  const float q0 = a * sc.recip;
  const float r0 = __fmaf_rn(-sc.beta, q0, a);
  const float q1 = __fmaf_rn(r0, sc.recip, q0);
  const float r1 = __fmaf_rn(-sc.beta, q1, a);
  return __fmaf_rn(r1, sc.recip, q1);
}
template <bool PW2 = false>
__device__ __forceinline__ float luq_quotient_clamped(float x, const LuqScale& sc, float q_top) {
  // an overflowing or non-finite quotient turns into NaN or Inf; both belong to the top level
  return fminf(luq_scaled_quotient<PW2>(fabsf(x) * sc.pre, sc), q_top);   // fminf(NaN, c) = c
}

// Per element: lower code and the 32-bit threshold of the up-decision, from the
// bit fields of Q = t * 2^32 (already clamped to 2^(kmax+32)).
//   t >= 1: code 1 + exponent(t), threshold = mantissa << 9 (up-probability
//           (|x| - lo)/lo); t = 2^kmax gives the top code with threshold 0.
//   t <  1: code 0, threshold trunc(Q) (prune-up probability |x|/alpha),
//           computed as (1.mantissa << 8) >> (158 - exponent field).
__device__ __forceinline__ void luq_bin(float q, uint32_t& lo_code, uint32_t& thr) {
  const uint32_t u = __float_as_uint(q);
  const int e = static_cast<int>(u >> 23);
  const uint32_t thr_in = u << 9;
  const uint32_t thr_under = __funnelshift_rc((u << 8) | 0x80000000u, 0u, static_cast<uint32_t>(158 - e));
  thr = u >= 0x4F800000u ? thr_in : thr_under;
  lo_code = static_cast<uint32_t>(max(e - 158, 0));
}

__device__ __forceinline__ uint32_t luq_nibble(uint32_t xbits, uint32_t lo_code, uint32_t thr, uint32_t word) {
  const uint32_t c = lo_code + (word < thr ? 1u : 0u);
  return c ? (((xbits >> 28) & 8u) | c) : 0u;
}
// the tensor-core operand byte of a LUQ nibble: int8 value +-2^(c-1), 0 for code 0
__device__ __forceinline__ uint32_t luq_operand_byte(uint32_t nibble) {
  const uint32_t mag = (1u << (nibble & 7u)) >> 1;
  return ((nibble & 8u) ? 0u - mag : mag) & 0xFFu;
}

// 2^ceil(log2 m) for a positive finite m (power-of-two LUQ: the maximum is rounded up, never down)
__device__ __forceinline__ float pw2_ceil(float m) {
  const uint32_t b = __float_as_uint(m);
  if (m > 0.0f && b < 0x7F800000u && (b & 0x007FFFFFu) != 0u) return __uint_as_float((b & 0x7F800000u) + 0x00800000u);
  return m;
}

// NS: number of samples known at compile time (1, 2) or 0 = read n_samples at run time.
// PW2: the scale is a power of two, the quotient an exact scaling (one multiply).
// TRACK: the tensor's own max|x| is reduced on the way (in-hindsight estimation: the scale
// in d_amax is an estimate from earlier steps, the measured maximum feeds the next one); the
// block that finishes last writes the measured maximum and replaces the estimate by
// (1 - eta) * measured + eta * estimate, every operation rounded once in binary32.
// PLANE: the tensor-core operand bytes (int8, +-2^(c-1)) of every sample are written next to
// the packed codes, one byte per element, sample s at offset s * n - or, with sum_planes, ONE plane
// whose byte is the sum of the samples' bytes (the host checks that n_samples * 2^kmax fits int8):
// the mean over samples of the products equals the product with the summed operand over n_samples.
template <bool BF16, int NS, bool PW2, bool TRACK, bool PLANE>
__global__ void __launch_bounds__(kThreads) quant_luq_kernel(const void* __restrict__ x, size_t n,
                                                             const float* d_amax,
                                                             const __grid_constant__ PhiloxKeySet keys,
                                                             int n_samples_rt, int sum_planes,
                                                             uint8_t* __restrict__ codes,
                                                             int8_t* __restrict__ operand,
                                                             float* __restrict__ d_alpha,
                                                             unsigned int* __restrict__ measured_bits,
                                                             float* d_estimate, float eta,
                                                             float* d_amax_out, unsigned int* scratch,
                                                             unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  const int n_samples = NS > 0 ? NS : n_samples_rt;
  const bool sum = PLANE && NS != 1 && sum_planes != 0;
  constexpr int kElems = Item<BF16>::kElems;
  float given;
  if (!TRACK && d_amax_out != nullptr) {   // fused: the maximum of this tensor, reduced here
    uint32_t bits;
    if (!fused_grid_max<BF16>(x, n, scratch, status, bits)) return;
    given = __uint_as_float(bits);
    if (blockIdx.x == 0 && threadIdx.x == 0) *d_amax_out = given;
  } else {
    given = *d_amax;   // with TRACK the last block overwrites it after every block has read it
  }
  const bool back_to_front = !TRACK && d_amax_out != nullptr;   // phase one ended at the tensor's tail
  const float mx = PW2 ? pw2_ceil(given) : given;
  const bool first = blockIdx.x == 0 && threadIdx.x == 0;
  const bool ok = scale_usable(mx, first ? status : nullptr);
  const float alpha = ok ? mx * keys.inv_levels : 0.0f;  // exact scaling
  const uint32_t fixed_word = keys.fixed_word;
  auto random_words = [&](uint64_t block, const PhiloxKeys& ks) {
    return fixed_word ? make_uint4(fixed_word, fixed_word, fixed_word, fixed_word) : philox_block(block, ks);
  };
  if (first) *d_alpha = alpha;
  const LuqScale sc = luq_scale(ok ? alpha : 1.0f);   // with a power-of-two alpha the reciprocal is exact
  uint32_t seen = 0;   // running max of |x| bit patterns (TRACK)

  const size_t plane = n / 2;
  const bool aligned = (plane % (kElems / 2)) == 0;  // planes start on a store boundary
  const bool aligned_op = (n % kElems) == 0;
  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);

  // Neural gradients are heavy-tailed: almost every element lies below alpha, in
  // the underflow bin, where the code is 0 or 1 and the threshold is trunc(t * 2^32).
  // A warp whose elements all do takes the short route; |x| < alpha is equivalent
  // to t < 1 (and false for NaN), so both routes give the same codes.
  auto process = [&](size_t item, const uint4& u, bool whole_warp) {
    float v[kElems];
    Item<BF16>::widen(u, v);
    bool in_range = false;
#pragma unroll
    for (int j = 0; j < kElems; ++j) in_range |= !(fabsf(v[j]) < alpha);
    if constexpr (TRACK) {
#pragma unroll
      for (int j = 0; j < kElems; ++j) seen = max(seen, __float_as_uint(v[j]) & 0x7FFFFFFFu);
    }
    // the vote needs every lane of the warp here: only the full-tile loop qualifies
    if (whole_warp && !sc.tiny && !__any_sync(0xFFFFFFFFu, in_range)) {
      // thr: the up-threshold trunc(Q) (Q < 2^32 here).  sn / ob: the element's non-zero nibble
      // (sign, code 1) and operand byte (-1 or +1), already shifted to their place in the word.
      uint32_t thr[kElems], sn[kElems], ob[kElems];
#pragma unroll
      for (int j = 0; j < kElems; ++j) {
        const uint32_t bits = __float_as_uint(v[j]);
        thr[j] = __float2uint_rz(luq_scaled_quotient<PW2>(fabsf(v[j]), sc));
        const int at = 4 * j;   // bit position of the nibble; the sign bit goes to at + 3
        sn[j] = ((bits >> (28 - at)) & (8u << at)) | (1u << at);
        if constexpr (PLANE) ob[j] = ((bits >> 31) ? 0xFFu : 0x01u) << (8 * (j % 4));
      }
      uint32_t total[kElems / 4] = {};   // per-byte sums over the samples (sum_planes)
#pragma unroll
      for (int s = 0; s < (NS > 0 ? NS : LUQ_MAX_SAMPLES); ++s) {
        if (NS == 0 && s >= n_samples) break;
        const PhiloxKeys& ks = keys.s[s];
        uint32_t word = 0;
        uint32_t bytes[kElems / 4] = {};
#pragma unroll
        for (int b = 0; b < kElems / 4; ++b) {
          const uint4 r = random_words(item * (kElems / 4) + b, ks);
          const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            if (rw[j] < thr[4 * b + j]) {
              word |= sn[4 * b + j];
              if constexpr (PLANE) bytes[b] |= ob[4 * b + j];
            }
          }
        }
        Item<BF16>::store(codes + plane * s, item, word, aligned || s == 0);
        if constexpr (PLANE) {
          if (sum) {
#pragma unroll
            for (int b = 0; b < kElems / 4; ++b) total[b] = __vadd4(total[b], bytes[b]);
          } else {
            Item<BF16>::store_bytes(operand + n * s, item, bytes, aligned_op || s == 0);
          }
        }
      }
      if constexpr (PLANE) if (sum) Item<BF16>::store_bytes(operand, item, total, true);
      return;
    }
    uint32_t lo_code[kElems], thr[kElems];
#pragma unroll
    for (int j = 0; j < kElems; ++j) luq_bin(luq_quotient_clamped<PW2>(v[j], sc, keys.q_top), lo_code[j], thr[j]);
    uint32_t total[kElems / 4] = {};
#pragma unroll
    for (int s = 0; s < (NS > 0 ? NS : LUQ_MAX_SAMPLES); ++s) {
      if (NS == 0 && s >= n_samples) break;
      const PhiloxKeys& ks = keys.s[s];
      uint32_t word = 0;
      uint32_t bytes[kElems / 4] = {};
#pragma unroll
      for (int b = 0; b < kElems / 4; ++b) {
        const uint4 r = random_words(item * (kElems / 4) + b, ks);
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const uint32_t nib = luq_nibble(__float_as_uint(v[4 * b + j]), lo_code[4 * b + j], thr[4 * b + j], rw[j]);
          word |= nib << (4 * (4 * b + j));
          if constexpr (PLANE) bytes[b] |= luq_operand_byte(nib) << (8 * j);
        }
      }
      Item<BF16>::store(codes + plane * s, item, word, aligned || s == 0);
      if constexpr (PLANE) {
        if (sum) {
#pragma unroll
          for (int b = 0; b < kElems / 4; ++b) total[b] = __vadd4(total[b], bytes[b]);
        } else {
          Item<BF16>::store_bytes(operand + n * s, item, bytes, aligned_op || s == 0);
        }
      }
    }
    if constexpr (PLANE) if (sum) Item<BF16>::store_bytes(operand, item, total, true);
  };

  const size_t full_tiles = items / kTileItems;
  if (ok) {
    for (size_t t = blockIdx.x; t < full_tiles; t += gridDim.x) {
      const size_t i0 = (back_to_front ? full_tiles - 1 - t : t) * kTileItems + threadIdx.x;
      uint4 u[kUnroll];
#pragma unroll
      for (int j = 0; j < kUnroll; ++j)
        u[j] = piece_ok(i0 + j * kThreads, items, status) ? __ldg(p + i0 + j * kThreads) : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
      for (int j = 0; j < kUnroll; ++j)
        if (piece_ok(i0 + j * kThreads, items, status)) process(i0 + j * kThreads, u[j], true);
    }
    if (blockIdx.x == gridDim.x - 1)
      for (size_t i = full_tiles * kTileItems + threadIdx.x; i < items; i += kThreads) process(i, __ldg(p + i), false);
  } else {
    const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
    for (size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x; i < items; i += stride) {
      for (int s = 0; s < n_samples; ++s) {
        Item<BF16>::store(codes + plane * s, i, 0u, aligned || s == 0);
        if constexpr (PLANE) {
          const uint32_t zero[kElems / 4] = {};
          if (!sum || s == 0) Item<BF16>::store_bytes(operand + n * s, i, zero, aligned_op || s == 0);
        }
      }
      if constexpr (TRACK) {   // an unusable estimate still needs this tensor's maximum for the next step
        float v[kElems];
        Item<BF16>::widen(__ldg(p + i), v);
#pragma unroll
        for (int j = 0; j < kElems; ++j) seen = max(seen, __float_as_uint(v[j]) & 0x7FFFFFFFu);
      }
    }
  }
  if (TRACK && first)
    for (size_t e = items * kElems; e < n; ++e) seen = max(seen, __float_as_uint(Item<BF16>::load1(x, e)) & 0x7FFFFFFFu);
  if (first) {  // tail: fewer elements than one piece, two per byte
    for (int s = 0; s < n_samples; ++s) {
      const PhiloxKeys& ks = keys.s[s];
      for (size_t e = items * kElems; e < n; e += 2) {
        uint32_t nib[2] = {0u, 0u};
        for (int h = 0; h < 2; ++h) {
          const size_t idx = e + h;
          if (ok && idx < n) {
            const float xv = Item<BF16>::load1(x, idx);
            uint32_t lc, th;
            luq_bin(luq_quotient_clamped<PW2>(xv, sc, keys.q_top), lc, th);
            const uint4 r = random_words(idx >> 2, ks);
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
            nib[h] = luq_nibble(__float_as_uint(xv), lc, th, rw[idx & 3]);
          }
        }
        codes[plane * s + (e >> 1)] = static_cast<uint8_t>(nib[0] | (nib[1] << 4));
        if constexpr (PLANE) {
          if (sum) {   // this thread wrote the earlier samples' sum itself
            const int8_t b0 = static_cast<int8_t>(luq_operand_byte(nib[0])), b1 = static_cast<int8_t>(luq_operand_byte(nib[1]));
            operand[e] = static_cast<int8_t>((s ? operand[e] : 0) + b0);
            if (e + 1 < n) operand[e + 1] = static_cast<int8_t>((s ? operand[e + 1] : 0) + b1);
          } else {
            operand[n * s + e] = static_cast<int8_t>(luq_operand_byte(nib[0]));
            if (e + 1 < n) operand[n * s + e + 1] = static_cast<int8_t>(luq_operand_byte(nib[1]));
          }
        }
      }
    }
  }
  if constexpr (TRACK) {   // Inf/NaN patterns win the maximum and raise the flag
    if (grid_max_last_block(seen, scratch, blockIdx.x, gridDim.x)) {
      *measured_bits = seen;
      if (seen >= 0x7F800000u) atomicOr(status, LUQ_STATUS_NONFINITE);
      *d_estimate = hindsight_next(seen, given, eta);
    }
  }
}

// The other gradient quantizers of the ablation (Sec. 4, ablation figure), one plain streaming
// kernel (no fused maximum, sample count read at run time): same pieces, stores, random words,
// sample planes and short route as the LUQ kernel.
//   UNIFORM = false: the LUQ grid with one region deterministic.  word_under / word_range replace
//     the random word of an element below alpha / inside the range when non-zero; 0x7FFFFFFF makes
//     that region round to the nearest level ("FP4 + SR": word_under set; stochastic underflow
//     alone: word_range set).
//   UNIFORM = true: "INT4 unbiased" - the grid -7..7 with step max/7 and stochastic rounding of
//     the magnitude: y = |x| * fl(7/max) clamped to 7, l = floor(y), up when word < trunc((y-l)*2^32);
//     two's-complement nibble, operand byte 16 * q (the INT4 operand form).
template <bool BF16, bool PLANE, bool UNIFORM>
__global__ void __launch_bounds__(kThreads) quant_ablation_kernel(const void* __restrict__ x, size_t n,
                                                                  const float* __restrict__ d_amax,
                                                                  const __grid_constant__ PhiloxKeySet keys,
                                                                  int n_samples, uint32_t word_under,
                                                                  uint32_t word_range,
                                                                  uint8_t* __restrict__ codes,
                                                                  int8_t* __restrict__ operand,
                                                                  float* __restrict__ d_scale,
                                                                  unsigned int* __restrict__ status) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  constexpr int kElems = Item<BF16>::kElems;
  const float given = *d_amax;
  const bool first = blockIdx.x == 0 && threadIdx.x == 0;
  const bool ok = scale_usable(given, first ? status : nullptr);
  const float scale = !ok ? 0.0f : UNIFORM ? given / 7.0f : given * keys.inv_levels;
  if (first) *d_scale = scale;
  const float inv = ok ? 7.0f / given : 0.0f;                         // uniform grid only
  const LuqScale sc = luq_scale(ok && !UNIFORM ? scale : 1.0f);

  // per element: the lower level, the 32-bit threshold of the up-decision, the constant that
  // replaces the random word (0: none)
  auto prepare = [&](float v, uint32_t& lo, uint32_t& thr, uint32_t& fixed) {
    if constexpr (UNIFORM) {
      const float y = fabsf(v) * inv;
      const float a = (y == y) ? fminf(y, 7.0f) : 0.0f;               // NaN element -> 0
      const float l = floorf(a);
      lo = __float2uint_rz(l);
      thr = __float2uint_rz((a - l) * 4294967296.0f);                 // a - l is exact
      fixed = 0u;
    } else {
      const float q = luq_quotient_clamped<false>(v, sc, keys.q_top);
      luq_bin(q, lo, thr);
      fixed = q < 4294967296.0f ? word_under : word_range;            // Q < 2^32 <=> |x| < alpha
    }
  };
  auto nibble_of = [&](uint32_t xbits, uint32_t lo, uint32_t thr, uint32_t fixed, uint32_t word) -> uint32_t {
    const uint32_t w = fixed ? fixed : word;
    if constexpr (UNIFORM) {
      const uint32_t m = lo + (w < thr ? 1u : 0u);
      return ((xbits >> 31) ? 0u - m : m) & 0xFu;
    } else {
      return luq_nibble(xbits, lo, thr, w);
    }
  };
  auto byte_of = [&](uint32_t nib) -> uint32_t { return UNIFORM ? (nib << 4) : luq_operand_byte(nib); };

  const size_t plane = n / 2;
  const bool aligned = (plane % (kElems / 2)) == 0;
  const bool aligned_op = (n % kElems) == 0;
  const size_t items = n / kElems;
  const uint4* p = reinterpret_cast<const uint4*>(x);

  auto process = [&](size_t item, const uint4& u, bool whole_warp) {
    float v[kElems];
    Item<BF16>::widen(u, v);
    if constexpr (!UNIFORM) {
      // the LUQ kernel's short route: a warp whose elements all lie below alpha only decides
      // between 0 and +-alpha; with a deterministic underflow region no generator runs at all
      bool in_range = false;
#pragma unroll
      for (int j = 0; j < kElems; ++j) in_range |= !(fabsf(v[j]) < scale);
      if (whole_warp && ok && !sc.tiny && !__any_sync(0xFFFFFFFFu, in_range)) {
        uint32_t thr[kElems], sn[kElems], ob[kElems];
#pragma unroll
        for (int j = 0; j < kElems; ++j) {
          const uint32_t bits = __float_as_uint(v[j]);
          thr[j] = __float2uint_rz(luq_scaled_quotient<false>(fabsf(v[j]), sc));
          const int at = 4 * j;
          sn[j] = ((bits >> (28 - at)) & (8u << at)) | (1u << at);
          if constexpr (PLANE) ob[j] = ((bits >> 31) ? 0xFFu : 0x01u) << (8 * (j % 4));
        }
        for (int s = 0; s < n_samples; ++s) {
          const PhiloxKeys& ks = keys.s[s];
          uint32_t word = 0;
          uint32_t bytes[kElems / 4] = {};
#pragma unroll
          for (int b = 0; b < kElems / 4; ++b) {
            uint4 r = make_uint4(word_under, word_under, word_under, word_under);
            if (word_under == 0u) r = philox_block(item * (kElems / 4) + b, ks);
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              if (rw[j] < thr[4 * b + j]) {
                word |= sn[4 * b + j];
                if constexpr (PLANE) bytes[b] |= ob[4 * b + j];
              }
            }
          }
          Item<BF16>::store(codes + plane * s, item, word, aligned || s == 0);
          if constexpr (PLANE) Item<BF16>::store_bytes(operand + n * s, item, bytes, aligned_op || s == 0);
        }
        return;
      }
    }
    uint32_t lo[kElems], thr[kElems], fixed[kElems];
#pragma unroll
    for (int j = 0; j < kElems; ++j) prepare(v[j], lo[j], thr[j], fixed[j]);
    for (int s = 0; s < n_samples; ++s) {
      const PhiloxKeys& ks = keys.s[s];
      uint32_t word = 0;
      uint32_t bytes[kElems / 4] = {};
#pragma unroll
      for (int b = 0; b < kElems / 4; ++b) {
        const uint4 r = philox_block(item * (kElems / 4) + b, ks);
        const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int e = 4 * b + j;
          const uint32_t nib = ok ? nibble_of(__float_as_uint(v[e]), lo[e], thr[e], fixed[e], rw[j]) : 0u;
          word |= nib << (4 * e);
          if constexpr (PLANE) bytes[b] |= byte_of(nib) << (8 * j);
        }
      }
      Item<BF16>::store(codes + plane * s, item, word, aligned || s == 0);
      if constexpr (PLANE) Item<BF16>::store_bytes(operand + n * s, item, bytes, aligned_op || s == 0);
    }
  };

  const size_t full_tiles = items / kTileItems;
  for (size_t t = blockIdx.x; t < full_tiles; t += gridDim.x) {
    const size_t i0 = t * kTileItems + threadIdx.x;
    uint4 u[kUnroll];
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) u[j] = __ldg(p + i0 + j * kThreads);
#pragma unroll
    for (int j = 0; j < kUnroll; ++j) process(i0 + j * kThreads, u[j], true);
  }
  if (blockIdx.x == gridDim.x - 1)
    for (size_t i = full_tiles * kTileItems + threadIdx.x; i < items; i += kThreads) process(i, __ldg(p + i), false);
  if (first) {  // tail: fewer elements than one piece, two per byte
    for (int s = 0; s < n_samples; ++s) {
      const PhiloxKeys& ks = keys.s[s];
      for (size_t e = items * kElems; e < n; e += 2) {
        uint32_t nib[2] = {0u, 0u};
        for (int h = 0; h < 2; ++h) {
          const size_t idx = e + h;
          if (ok && idx < n) {
            const float xv = Item<BF16>::load1(x, idx);
            uint32_t lo, thr, fixed;
            prepare(xv, lo, thr, fixed);
            const uint4 r = philox_block(idx >> 2, ks);
            const uint32_t rw[4] = {r.x, r.y, r.z, r.w};
            nib[h] = nibble_of(__float_as_uint(xv), lo, thr, fixed, rw[idx & 3]);
          }
        }
        codes[plane * s + (e >> 1)] = static_cast<uint8_t>(nib[0] | (nib[1] << 4));
        if constexpr (PLANE) {
          operand[n * s + e] = static_cast<int8_t>(byte_of(nib[0]));
          if (e + 1 < n) operand[n * s + e + 1] = static_cast<int8_t>(byte_of(nib[1]));
        }
      }
    }
  }
}

// Diagnostic: the quotient t = |x| / alpha exactly as the quantizer forms it
// (before the clamp to the top level), for comparison with an IEEE division.
__global__ void __launch_bounds__(kThreads) luq_quotient_kernel(const float* __restrict__ x, size_t n,
                                                                const float* __restrict__ d_amax,
                                                                float inv_levels, float* __restrict__ out) {
  luqdev::pdl_wait();
  luqdev::pdl_trigger();
  const float alpha = __ldg(d_amax) * inv_levels;
  const LuqScale sc = luq_scale(alpha);
  const size_t stride = static_cast<size_t>(gridDim.x) * kThreads;
  for (size_t i = static_cast<size_t>(blockIdx.x) * kThreads + threadIdx.x; i < n; i += stride)
    out[i] = luq_scaled_quotient<false>(fabsf(x[i]) * sc.pre, sc) * 0x1p-32f;   // t = Q * 2^-32
}

// Grid for a kernel that walks `tiles` tiles: at most the CTAs the GPU holds at once
// (optionally fewer per SM), a multiple of the SM count.
template <typename K>
int grid_for(const luq_ctx* ctx, K kernel, size_t tiles, int max_per_sm = 1 << 30) {
  int per_sm = 0;
  // These kernels are launched early (see luq_launch_kernel).  With a preference for the largest L1
  // their blocks do not become resident on an SM that is still carved for a GEMM block's shared
  // memory, where they would keep a small L1 for their whole life.
  cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxL1);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  if (per_sm > max_per_sm) per_sm = max_per_sm;
  size_t cap = static_cast<size_t>(ctx->sm_count) * per_sm;
  if (cap > LUQ_SCRATCH_REGION - 2) cap = LUQ_SCRATCH_REGION - 2;   // one scratch word per block of a reducing kernel
  if (tiles < 1) tiles = 1;
  if (tiles <= cap) return static_cast<int>(tiles);
  // More tiles than resident blocks: a whole number of blocks per SM, so that every SM carries the
  // same load (a grid of, say, 5.8 blocks per SM leaves the SMs with five blocks idle while those
  // with six finish); the tiles are dealt out round-robin and differ by at most one per block.
  const size_t whole = cap / static_cast<size_t>(ctx->sm_count) * static_cast<size_t>(ctx->sm_count);
  return static_cast<int>(whole > 0 ? whole : cap);
}

}  // namespace

int luq_launch_amax(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_amax, cudaStream_t st) {
  if (n == 0) return static_cast<int>(cudaMemsetAsync(d_amax, 0, sizeof(float), st));
  unsigned int* out = reinterpret_cast<unsigned int*>(d_amax);
  cudaError_t e;
  if (dtype == LUQ_BF16) {
    const int grid = grid_for(ctx, amax_kernel<true>, n / 8 / (kThreads * kAmaxUnroll) + 1, kAmaxCtasPerSm);
    e = luq_launch_kernel(amax_kernel<true>, grid, kThreads, 0, st, LUQ_LAUNCH_EARLY, 1, d_x, n, out, ctx->d_scratch, ctx->d_status);
  } else {
    const int grid = grid_for(ctx, amax_kernel<false>, n / 4 / (kThreads * kAmaxUnroll) + 1, kAmaxCtasPerSm);
    e = luq_launch_kernel(amax_kernel<false>, grid, kThreads, 0, st, LUQ_LAUNCH_EARLY, 1, d_x, n, out, ctx->d_scratch, ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(e);
}

namespace {
// Blocks of a several-tensor launch: one wave of the GPU, dealt out in proportion to the tensors'
// tile counts, at least one block each.
template <typename K>
void deal_blocks(const luq_ctx* ctx, K kernel, int count, const size_t* tiles, unsigned int* first_block) {
  int per_sm = 0;
  cudaFuncSetAttribute(kernel, cudaFuncAttributePreferredSharedMemoryCarveout, cudaSharedmemCarveoutMaxL1);
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kThreads, 0) != cudaSuccess || per_sm < 1)
    per_sm = 1;
  const size_t cap = static_cast<size_t>(ctx->sm_count) * per_sm;
  size_t total = 0;
  for (int t = 0; t < count; ++t) total += tiles[t];
  first_block[0] = 0;
  for (int t = 0; t < count; ++t) {
    size_t blocks = total <= cap ? tiles[t] : tiles[t] * cap / total;
    if (blocks < 1) blocks = 1;
    if (blocks > LUQ_SCRATCH_REGION - 2) blocks = LUQ_SCRATCH_REGION - 2;
    first_block[t + 1] = first_block[t] + static_cast<unsigned int>(blocks);
  }
}
}  // namespace

int luq_launch_amax_multi(luq_ctx* ctx, int count, const void* const* d_x, const size_t* n, float* const* d_amax,
                          int dtype, cudaStream_t st) {
  MultiAmax a{};
  size_t tiles[kMultiMax];
  const bool bf = dtype == LUQ_BF16;
  for (int t = 0; t < count; ++t) {
    a.x[t] = d_x[t]; a.n[t] = n[t]; a.out[t] = reinterpret_cast<unsigned int*>(d_amax[t]);
    tiles[t] = n[t] / (bf ? 8 : 4) / (kThreads * kAmaxUnroll) + 1;
  }
  a.count = count;
  cudaError_t e;
  if (bf) {
    deal_blocks(ctx, amax_multi_kernel<true>, count, tiles, a.first_block);
    e = luq_launch_kernel(amax_multi_kernel<true>, static_cast<int>(a.first_block[count]), kThreads, 0, st,
                          LUQ_LAUNCH_EARLY, 1, a, ctx->d_scratch, ctx->d_status);
  } else {
    deal_blocks(ctx, amax_multi_kernel<false>, count, tiles, a.first_block);
    e = luq_launch_kernel(amax_multi_kernel<false>, static_cast<int>(a.first_block[count]), kThreads, 0, st,
                          LUQ_LAUNCH_EARLY, 1, a, ctx->d_scratch, ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(e);
}

int luq_launch_quant_int4_multi(luq_ctx* ctx, int count, const void* const* d_x, const size_t* n,
                                const float* const* d_clip, uint8_t* const* d_codes, float* const* d_scale,
                                int8_t* const* d_operand, int dtype, cudaStream_t st) {
  MultiInt4 a{};
  size_t tiles[kMultiMax];
  const bool bf = dtype == LUQ_BF16;
  for (int t = 0; t < count; ++t) {
    a.x[t] = d_x[t]; a.n[t] = n[t]; a.clip[t] = d_clip[t]; a.codes[t] = d_codes[t]; a.scale[t] = d_scale[t];
    a.operand[t] = n[t] ? d_operand[t] : nullptr;
    tiles[t] = n[t] / (bf ? 8 : 4) / kTileItems + 1;
  }
  a.count = count;
  cudaError_t e;
  if (bf) {
    deal_blocks(ctx, quant_int4_multi_kernel<true>, count, tiles, a.first_block);
    e = luq_launch_kernel(quant_int4_multi_kernel<true>, static_cast<int>(a.first_block[count]), kThreads, 0, st,
                          LUQ_LAUNCH_EARLY, 1, a, ctx->d_status);
  } else {
    deal_blocks(ctx, quant_int4_multi_kernel<false>, count, tiles, a.first_block);
    e = luq_launch_kernel(quant_int4_multi_kernel<false>, static_cast<int>(a.first_block[count]), kThreads, 0, st,
                          LUQ_LAUNCH_EARLY, 1, a, ctx->d_status);
  }
  ctx->launches += 1;
  return static_cast<int>(e);
}

namespace {
template <bool BF16, bool PLANE, bool UNSIGNED>
int launch_int4(luq_ctx* ctx, const void* d_x, size_t n, const float* d_clip, uint8_t* d_codes, int8_t* d_operand,
                float* d_scale, float* d_amax_out, cudaStream_t st) {
  const int grid = grid_for(ctx, quant_int4_kernel<BF16, PLANE, UNSIGNED>, n / Item<BF16>::kElems / kTileItems + 1);
  const int mode = d_amax_out ? LUQ_LAUNCH_COOPERATIVE : LUQ_LAUNCH_EARLY;   // fused: grid barrier inside
  return static_cast<int>(luq_launch_kernel(quant_int4_kernel<BF16, PLANE, UNSIGNED>, grid, kThreads, 0, st, mode, 1, d_x, n,
                                            d_clip, d_codes, d_operand, d_scale, d_amax_out, ctx->d_scratch,
                                            ctx->d_status));
}
template <bool BF16, bool PLANE>
int launch_int4_grid(bool is_unsigned, luq_ctx* ctx, const void* d_x, size_t n, const float* d_clip, uint8_t* d_codes,
                     int8_t* d_operand, float* d_scale, float* d_amax_out, cudaStream_t st) {
  return is_unsigned ? launch_int4<BF16, PLANE, true>(ctx, d_x, n, d_clip, d_codes, d_operand, d_scale, d_amax_out, st)
                     : launch_int4<BF16, PLANE, false>(ctx, d_x, n, d_clip, d_codes, d_operand, d_scale, d_amax_out, st);
}
}  // namespace

int luq_launch_quant_int4_hindsight(luq_ctx* ctx, const void* d_x, int dtype, size_t n, float* d_estimate, float eta,
                                    uint8_t* d_codes, int8_t* d_operand, float* d_scale, float* d_measured,
                                    cudaStream_t st) {
  unsigned int* measured = reinterpret_cast<unsigned int*>(d_measured);
  const bool bf = dtype == LUQ_BF16;
  auto go = [&](auto kernel, int elems) {
    const int grid = grid_for(ctx, kernel, n / elems / kTileItems + 1);
    return static_cast<int>(luq_launch_kernel(kernel, grid, kThreads, 0, st, LUQ_LAUNCH_EARLY, 1, d_x, n, d_estimate, eta,
                                              d_codes, d_operand, d_scale, measured, ctx->d_scratch, ctx->d_status));
  };
  int rc;
  if (d_operand) rc = bf ? go(quant_int4_track_kernel<true, true>, 8) : go(quant_int4_track_kernel<false, true>, 4);
  else rc = bf ? go(quant_int4_track_kernel<true, false>, 8) : go(quant_int4_track_kernel<false, false>, 4);
  ctx->launches += 1;
  return rc;
}

// d_amax_out non-null: fused - the clip is the tensor's maximum, reduced by the same kernel and written there
int luq_launch_quant_int4(luq_ctx* ctx, const void* d_x, int dtype, size_t n, const float* d_clip,
                          uint8_t* d_codes, int8_t* d_operand, float* d_scale, float* d_amax_out, bool is_unsigned,
                          cudaStream_t st) {
  const bool bf = dtype == LUQ_BF16;
  int rc;
  if (d_operand) rc = bf ? launch_int4_grid<true, true>(is_unsigned, ctx, d_x, n, d_clip, d_codes, d_operand, d_scale, d_amax_out, st)
                         : launch_int4_grid<false, true>(is_unsigned, ctx, d_x, n, d_clip, d_codes, d_operand, d_scale, d_amax_out, st);
  else rc = bf ? launch_int4_grid<true, false>(is_unsigned, ctx, d_x, n, d_clip, d_codes, nullptr, d_scale, d_amax_out, st)
               : launch_int4_grid<false, false>(is_unsigned, ctx, d_x, n, d_clip, d_codes, nullptr, d_scale, d_amax_out, st);
  ctx->launches += 1;
  return rc;
}

namespace {
PhiloxKeySet expand_keys(uint64_t seed, int n_samples, int kmax, uint32_t fixed_word) {
  PhiloxKeySet keys{};
  keys.fixed_word = fixed_word;
  keys.inv_levels = 1.0f / static_cast<float>(1 << kmax);
  keys.q_top = 4294967296.0f * static_cast<float>(1 << kmax);
  for (int s = 0; s < n_samples; ++s) {   // sample s is keyed by seed + s
    const uint64_t key = seed + static_cast<uint64_t>(s);
    uint32_t a = static_cast<uint32_t>(key), b = static_cast<uint32_t>(key >> 32);
    for (int r = 0; r < 10; ++r) { keys.s[s].k0[r] = a; keys.s[s].k1[r] = b; a += 0x9E3779B9u; b += 0xBB67AE85u; }
  }
  return keys;
}

struct LuqLaunch {
  luq_ctx* ctx; const void* g; size_t n; const float* amax; PhiloxKeySet keys; int n_samples;
  uint8_t* codes; int8_t* operand; float* alpha; unsigned int* measured; float* estimate; float eta;
  float* amax_out;   // non-null: fused, the maximum is reduced by the same kernel (cooperative launch)
  cudaStream_t st;
  int sum_planes;    // one operand plane holding the sum over samples
};

template <bool BF16, int NS, bool PW2, bool TRACK, bool PLANE>
int launch_luq_ns(const LuqLaunch& a) {
  const size_t tiles = a.n / Item<BF16>::kElems / kTileItems + 1;
  const int grid = grid_for(a.ctx, quant_luq_kernel<BF16, NS, PW2, TRACK, PLANE>, tiles);
  const int mode = a.amax_out ? LUQ_LAUNCH_COOPERATIVE : LUQ_LAUNCH_EARLY;
  return static_cast<int>(luq_launch_kernel(quant_luq_kernel<BF16, NS, PW2, TRACK, PLANE>, grid, kThreads, 0, a.st, mode, 1,
                                            a.g, a.n, a.amax, a.keys, a.n_samples, a.sum_planes, a.codes, a.operand,
                                            a.alpha, a.measured, a.estimate, a.eta, a.amax_out, a.ctx->d_scratch,
                                            a.ctx->d_status));
}
template <bool BF16, bool PW2, bool TRACK, bool PLANE>
int launch_luq_plane(const LuqLaunch& a) {
  if (a.n_samples == 1) return launch_luq_ns<BF16, 1, PW2, TRACK, PLANE>(a);
  if (a.n_samples == 2) return launch_luq_ns<BF16, 2, PW2, TRACK, PLANE>(a);
  return launch_luq_ns<BF16, 0, PW2, TRACK, PLANE>(a);
}
template <bool BF16, bool PW2, bool TRACK>
int launch_luq(const LuqLaunch& a) {
  return a.operand ? launch_luq_plane<BF16, PW2, TRACK, true>(a) : launch_luq_plane<BF16, PW2, TRACK, false>(a);
}
}  // namespace

// flags: bit 0 = power-of-two scale; bit 1 = in-hindsight: d_amax is the running estimate, the
// tensor's own maximum goes to d_measured and the estimate is replaced (eta) by the same kernel;
// bit 2 = deterministic round-to-nearest-power instead of the random words;
// bit 3 = d_operand is ONE plane holding the sum of the samples' operand bytes
int luq_launch_quant_grad_ex(luq_ctx* ctx, const void* d_g, int dtype, size_t n, const float* d_amax, uint64_t seed,
                             int n_samples, uint8_t* d_codes, int8_t* d_operand, float* d_alpha, int flags,
                             float* d_measured, float* d_estimate, float eta, float* d_amax_out, cudaStream_t st) {
  const LuqLaunch a{ctx, d_g, n, d_amax, expand_keys(seed, n_samples, ctx->kmax, (flags & 4) ? 0x7FFFFFFFu : 0u),
                    n_samples, d_codes, d_operand, d_alpha,
                    reinterpret_cast<unsigned int*>(d_measured), d_estimate, eta, d_amax_out, st,
                    (flags & 8) && d_operand && n_samples > 1 ? 1 : 0};
  int rc;
  switch ((flags & 3) | (dtype == LUQ_BF16 ? 4 : 0)) {
    case 0: rc = launch_luq<false, false, false>(a); break;
    case 1: rc = launch_luq<false, true, false>(a); break;
    case 2: rc = launch_luq<false, false, true>(a); break;
    case 3: rc = launch_luq<false, true, true>(a); break;
    case 4: rc = launch_luq<true, false, false>(a); break;
    case 5: rc = launch_luq<true, true, false>(a); break;
    case 6: rc = launch_luq<true, false, true>(a); break;
    default: rc = launch_luq<true, true, true>(a); break;
  }
  ctx->launches += 1;
  return rc;
}

namespace {
template <bool BF16, bool PLANE, bool UNIFORM>
int launch_ablation(luq_ctx* ctx, const void* d_g, size_t n, const float* d_amax, const PhiloxKeySet& keys, int n_samples,
                    uint32_t word_under, uint32_t word_range, uint8_t* d_codes, int8_t* d_operand, float* d_scale,
                    cudaStream_t st) {
  const int grid = grid_for(ctx, quant_ablation_kernel<BF16, PLANE, UNIFORM>, n / Item<BF16>::kElems / kTileItems + 1);
  return static_cast<int>(luq_launch_kernel(quant_ablation_kernel<BF16, PLANE, UNIFORM>, grid, kThreads, 0, st,
                                            LUQ_LAUNCH_EARLY, 1, d_g, n, d_amax, keys, n_samples, word_under, word_range,
                                            d_codes, d_operand, d_scale, ctx->d_status));
}
template <bool BF16, bool PLANE>
int launch_ablation_grid(bool uniform, luq_ctx* ctx, const void* d_g, size_t n, const float* d_amax,
                         const PhiloxKeySet& keys, int n_samples, uint32_t word_under, uint32_t word_range,
                         uint8_t* d_codes, int8_t* d_operand, float* d_scale, cudaStream_t st) {
  return uniform ? launch_ablation<BF16, PLANE, true>(ctx, d_g, n, d_amax, keys, n_samples, 0u, 0u, d_codes, d_operand, d_scale, st)
                 : launch_ablation<BF16, PLANE, false>(ctx, d_g, n, d_amax, keys, n_samples, word_under, word_range, d_codes,
                                                       d_operand, d_scale, st);
}
}  // namespace

// scheme: bit 0 = stochastic rounding inside the range, bit 1 = stochastic underflow (the LUQ grid,
// the other region rounds to the nearest level); 4 = the uniform grid with stochastic rounding
int luq_launch_quant_grad_ablation(luq_ctx* ctx, const void* d_g, int dtype, size_t n, const float* d_amax,
                                   uint64_t seed, int n_samples, int scheme, uint8_t* d_codes, int8_t* d_operand,
                                   float* d_scale, cudaStream_t st) {
  const PhiloxKeySet keys = expand_keys(seed, n_samples, ctx->kmax, 0u);
  const bool uniform = scheme == 4;
  const uint32_t word_range = (scheme & 1) ? 0u : 0x7FFFFFFFu;
  const uint32_t word_under = (scheme & 2) ? 0u : 0x7FFFFFFFu;
  const bool bf = dtype == LUQ_BF16;
  int rc;
  if (d_operand) rc = bf ? launch_ablation_grid<true, true>(uniform, ctx, d_g, n, d_amax, keys, n_samples, word_under, word_range, d_codes, d_operand, d_scale, st)
                         : launch_ablation_grid<false, true>(uniform, ctx, d_g, n, d_amax, keys, n_samples, word_under, word_range, d_codes, d_operand, d_scale, st);
  else rc = bf ? launch_ablation_grid<true, false>(uniform, ctx, d_g, n, d_amax, keys, n_samples, word_under, word_range, d_codes, nullptr, d_scale, st)
               : launch_ablation_grid<false, false>(uniform, ctx, d_g, n, d_amax, keys, n_samples, word_under, word_range, d_codes, nullptr, d_scale, st);
  ctx->launches += 1;
  return rc;
}

int luq_launch_debug_quotient(luq_ctx* ctx, const float* d_x, size_t n, const float* d_amax, float* d_t,
                              cudaStream_t st) {
  if (n == 0) return 0;
  const int grid = grid_for(ctx, luq_quotient_kernel, n / kThreads + 1);
  const cudaError_t e = luq_launch_kernel(luq_quotient_kernel, grid, kThreads, 0, st, LUQ_LAUNCH_NORMAL, 1, d_x, n, d_amax,
                                          1.0f / static_cast<float>(1 << ctx->kmax), d_t);
  ctx->launches += 1;
  return static_cast<int>(e);
}
