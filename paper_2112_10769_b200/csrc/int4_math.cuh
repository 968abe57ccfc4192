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

// ---- four elements at a time (the GEMM that quantizes its activations on the way in) ----------
// int4_round_bits: the bit pattern of clamp(x * inv) + 1.5 * 2^23, whose low nibble is the code.
// The clamp propagates NaN (the sum is then a NaN pattern, bit 29 set; every valid sum is
// 0x4B3FFFF9 .. 0x4B400007, bit 29 clear): OR the results together and test bit 29 to find out
// whether any element needs int4_code()'s "NaN -> 0" rule.
__device__ __forceinline__ uint32_t int4_round_bits(float x, float inv) {
  const float y = __fmul_rn(x, inv);
  float c;
  asm("max.NaN.f32 %0, %1, %2;" : "=f"(c) : "f"(y), "f"(-7.0f));
  asm("min.NaN.f32 %0, %1, %2;" : "=f"(c) : "f"(c), "f"(7.0f));
  return __float_as_uint(__fadd_rn(c, 12582912.0f));
}
// the low bytes of four such sums, element 0 in byte 0 (the low nibble of a byte is the element's code)
__device__ __forceinline__ uint32_t int4_low_bytes(uint32_t t0, uint32_t t1, uint32_t t2, uint32_t t3) {
  return __byte_perm(__byte_perm(t0, t1, 0x0040), __byte_perm(t2, t3, 0x0040), 0x5410);
}
// those four bytes -> the four int8 operand bytes 16 * q
__device__ __forceinline__ uint32_t int4_operand_bytes(uint32_t low_bytes) { return (low_bytes << 4) & 0xF0F0F0F0u; }
// two such byte quadruples (elements 0-3 and 4-7) -> one word of eight packed codes
__device__ __forceinline__ uint32_t int4_pack8(uint32_t low_bytes_a, uint32_t low_bytes_b) {
  const uint32_t xa = low_bytes_a & 0x0F0F0F0Fu, xb = low_bytes_b & 0x0F0F0F0Fu;
  const uint32_t ya = xa | (xa >> 4), yb = xb | (xb >> 4);   // bytes 0 and 2 hold two codes each
  return __byte_perm(ya, yb, 0x6420);
}

// In-hindsight update of a running maximum (Sec. 7, App. A.5.4): (1 - eta) * measured + eta * estimate,
// one rounding per operation.  A measurement that is not finite (an Inf/NaN element) leaves the
// estimate as it was - one overflowed element must not turn every later estimate into Inf; an
// estimate that is not a positive finite number (0 before the first step) is replaced by the measurement.
__device__ __forceinline__ float hindsight_next(uint32_t measured_bits, float estimate, float eta) {
  if (measured_bits >= 0x7F800000u) return estimate;
  const uint32_t eb = __float_as_uint(estimate);
  if (eb == 0u || eb >= 0x7F800000u) return __uint_as_float(measured_bits);   // 0, negative, Inf, NaN
  const float keep = __fsub_rn(1.0f, eta);
  return __fadd_rn(__fmul_rn(keep, __uint_as_float(measured_bits)), __fmul_rn(eta, estimate));
}

}  // namespace luqdev
#endif
