// Shared host/device helpers of the AdaDim library (status codes, element loads, the
// group-parameter formula).  Internal header: the public interface is include/adadim.h.
#pragma once

#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/adadim.h"

namespace adadim {

constexpr int kTile = 128;          // quantizer tile edge; every supported group size divides it

#define ADADIM_CUDA_TRY(expr)                                   \
  do {                                                          \
    cudaError_t e__ = (expr);                                   \
    if (e__ != cudaSuccess) return ADADIM_ERR_CUDA;             \
  } while (0)

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t round_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Record a device-side condition: the first error wins.
__device__ __forceinline__ void report(int* status_dev, int code) {
  if (status_dev != nullptr) atomicCAS(status_dev, ADADIM_OK, code);
}

// ---- element access ---------------------------------------------------------------------
// load8: eight consecutive elements starting at a 16-byte (fp16) / 32-byte (fp32) aligned
// address, widened exactly to fp32.
__device__ __forceinline__ void load8(const __half* p, float (&v)[8]) {
  uint4 raw = *reinterpret_cast<const uint4*>(p);
  const __half2* h = reinterpret_cast<const __half2*>(&raw);
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    float2 f = __half22float2(h[k]);
    v[2 * k] = f.x;
    v[2 * k + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
  float4 a = *reinterpret_cast<const float4*>(p);
  float4 b = *reinterpret_cast<const float4*>(p + 4);
  v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
  v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// ---- the group-parameter formula (uniform asymmetric min-max; paper Section 4.1) ---------
// Evaluated in binary32 with round-to-nearest and true division, as the interface states.
struct GroupParams {
  float s;      // stored scale widened to fp32 (1 for a degenerate group)
  float z;      // integer zero point as a float
  float rcp;    // correctly rounded 1/s, or 0 for a degenerate group (forces code 0)
};

// The correctly rounded binary32 quotient w / s without a division instruction sequence:
// q0 = w * rcp is within an ulp of w / s, the residual w - s*q0 is exact in one FMA, and the
// corrected q0 + residual*rcp is the correctly rounded quotient because rcp is the correctly
// rounded reciprocal of s and the significand of s is not all ones (s is an fp16 value, or
// one of the constants 7, 15): Markstein's division step.  With rcp == 0 (degenerate group)
// the quotient is 0.
__device__ __forceinline__ float quotient(float w, float s, float rcp) {
  float q0 = __fmul_rn(w, rcp);
  float r = __fmaf_rn(-s, q0, w);
  return __fmaf_rn(r, rcp, q0);
}

// maxq is 2^bits - 1 and rcp_maxq the correctly rounded 1 / maxq (a compile-time constant at
// the call sites): both divisions of the formula go through quotient() above, which returns
// the correctly rounded binary32 quotient, so the result is that of true division.
__device__ __forceinline__ GroupParams group_params(float lo, float hi, float maxq, float rcp_maxq) {
  lo = fminf(lo, 0.0f);
  hi = fmaxf(hi, 0.0f);
  float s32 = quotient(__fsub_rn(hi, lo), maxq, rcp_maxq);
  float s = __half2float(__float2half_rn(s32));
  GroupParams g;
  if (s == 0.0f || !isfinite(s)) {
    g.s = 1.0f; g.z = 0.0f; g.rcp = 0.0f;
  } else {
    g.s = s;
    g.rcp = __frcp_rn(s);
    g.z = fminf(fmaxf(rintf(quotient(-lo, s, g.rcp)), 0.0f), maxq) + 0.0f;   // + 0: never store -0
  }
  return g;
}

// Adding 1.5 * 2^23 rounds a float of magnitude < 2^22 to an integer (ties to even) held in
// the low mantissa bits; larger magnitudes stay ordered, so a float clamp afterwards saturates
// them correctly.
constexpr float kRoundMagic = 12582912.0f;
constexpr int kRoundMagicBits = 0x4B400000;

// code = clamp(rint(q) + z, 0, maxq) as an integer.
__device__ __forceinline__ int code_of(float q, float z, float maxq) {
  float t = __fadd_rn(q, kRoundMagic);
  t = fminf(fmaxf(t, kRoundMagic - z), kRoundMagic + (maxq - z));
  return __float_as_int(t) - (kRoundMagicBits - static_cast<int>(z));
}

}  // namespace adadim
