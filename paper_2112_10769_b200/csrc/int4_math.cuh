// Arithmetic of the INT4 round-to-nearest quantizer (Sec. 3.3, App. A.1), shared by the streaming
// quantizer kernels and by the GEMM that quantizes its activations on the way in, so that both
// produce the same codes bit for bit.  Every operation is an explicitly rounded intrinsic: the
// result does not depend on the compiler's contraction setting.
#pragma once

#include "common.cuh"

#ifdef __CUDACC__
namespace luqdev {

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

// clamp, then add 1.5 * 2^23: the sum's low mantissa bits hold the integer rounded to
// nearest-even, already in two's complement (clamping before rounding equals clamping
// after it: the bounds are integers and rounding is monotone)
__device__ __forceinline__ uint32_t int4_code(float x, float inv) {
  const float y = __fmul_rn(x, inv);
  const float c = fminf(fmaxf(y, -7.0f), 7.0f);
  const uint32_t code = __float_as_uint(__fadd_rn(c, 12582912.0f)) & 0xFu;
  return (y == y) ? code : 0u;        // NaN element -> 0
}

// the same for the unsigned grid 0..15 (the clamp keeps negative inputs at 0)
__device__ __forceinline__ uint32_t uint4_code(float x, float inv) {
  const float y = __fmul_rn(x, inv);
  const float c = fminf(fmaxf(y, 0.0f), 15.0f);
  const uint32_t code = __float_as_uint(__fadd_rn(c, 12582912.0f)) & 0xFu;
  return (y == y) ? code : 0u;
}

}  // namespace luqdev
#endif
