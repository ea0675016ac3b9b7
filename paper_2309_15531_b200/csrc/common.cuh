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

// Argument rules shared by adadim_score_select and adadim_score_select_static (everything but
// the workspace).  Defined in api.cu.
int check_score_args(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits,
                     int group, const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, const double* err,
                     const int* chosen);

// The two helper streams of one factor / GPTQ call: a high-priority stream for the chain of small
// dependent kernels and a low-priority one for the bulk work that runs beside it, plus the events
// that order them.  open() makes the chain stream wait for everything already enqueued on the
// caller's stream.  The destructor runs on EVERY exit path, error returns included: it makes the
// caller's stream wait for whatever was enqueued on both helper streams (so the caller may free
// or reuse the workspace in stream order as usual) and releases streams and events; the runtime
// defers their destruction until the enqueued work has finished.
struct ForkedStreams {
  cudaStream_t caller = nullptr, chain = nullptr, side = nullptr, back = nullptr, back2 = nullptr;
  cudaEvent_t ev_a = nullptr, ev_b = nullptr, ev_c = nullptr, ev_join = nullptr;
  bool joined = false;
  // chain: highest priority; side: one step below it where the device has more than two levels;
  // back, back2 (only with `with_back`): lowest priority, for work that should fill idle SMs only
  int open(cudaStream_t st, bool with_back = false) {
    caller = st;
    int lo = 0, hi = 0;
    if (cudaDeviceGetStreamPriorityRange(&lo, &hi) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaStreamCreateWithPriority(&chain, cudaStreamNonBlocking, hi) != cudaSuccess) return ADADIM_ERR_CUDA;
    const int mid = with_back && hi + 1 < lo ? lo - 1 : lo;          // numerically lower = more urgent
    if (cudaStreamCreateWithPriority(&side, cudaStreamNonBlocking, mid) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (with_back && cudaStreamCreateWithPriority(&back, cudaStreamNonBlocking, lo) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (with_back && cudaStreamCreateWithPriority(&back2, cudaStreamNonBlocking, lo) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (with_back && cudaEventCreateWithFlags(&ev_c, cudaEventDisableTiming) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaEventCreateWithFlags(&ev_a, cudaEventDisableTiming) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaEventCreateWithFlags(&ev_b, cudaEventDisableTiming) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaEventCreateWithFlags(&ev_join, cudaEventDisableTiming) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaEventRecord(ev_join, caller) != cudaSuccess) return ADADIM_ERR_CUDA;
    if (cudaStreamWaitEvent(chain, ev_join, 0) != cudaSuccess) return ADADIM_ERR_CUDA;
    return ADADIM_OK;
  }
  // the caller's stream waits for everything enqueued so far on the helper streams
  int join() {
    if (ev_join == nullptr) return ADADIM_ERR_CUDA;
    bool ok = true;
    if (back2 != nullptr) ok = cudaEventRecord(ev_join, back2) == cudaSuccess && cudaStreamWaitEvent(caller, ev_join, 0) == cudaSuccess && ok;
    if (back != nullptr) ok = cudaEventRecord(ev_join, back) == cudaSuccess && cudaStreamWaitEvent(caller, ev_join, 0) == cudaSuccess && ok;
    if (side != nullptr) ok = cudaEventRecord(ev_join, side) == cudaSuccess && cudaStreamWaitEvent(caller, ev_join, 0) == cudaSuccess && ok;
    if (chain != nullptr) ok = cudaEventRecord(ev_join, chain) == cudaSuccess && cudaStreamWaitEvent(caller, ev_join, 0) == cudaSuccess && ok;
    joined = true;
    return ok ? ADADIM_OK : ADADIM_ERR_CUDA;
  }
  ~ForkedStreams() {
    if (!joined && ev_join != nullptr) join();
    if (ev_a != nullptr) cudaEventDestroy(ev_a);
    if (ev_b != nullptr) cudaEventDestroy(ev_b);
    if (ev_c != nullptr) cudaEventDestroy(ev_c);
    if (ev_join != nullptr) cudaEventDestroy(ev_join);
    if (chain != nullptr) cudaStreamDestroy(chain);
    if (side != nullptr) cudaStreamDestroy(side);
    if (back != nullptr) cudaStreamDestroy(back);
    if (back2 != nullptr) cudaStreamDestroy(back2);
  }
  ForkedStreams() = default;
  ForkedStreams(const ForkedStreams&) = delete;
  ForkedStreams& operator=(const ForkedStreams&) = delete;
};

// Layout of GPTQ's binary64 working weights (internal to one call's workspace): tiles of 32 rows
// x 16 columns, 4 KB each and contiguous, tile (R, C) at ((R * (in / 16)) + C) * 512 doubles.
// Inside a tile row r keeps its eight 16-byte column pairs at pair position p ^ (r & 7).  A tile
// is what one warp of the trailing update adds in one bulk operation and what the block kernel
// fetches in one bulk copy; the pair swizzle lets 32 threads that each own a row touch a tile
// without shared-memory bank conflicts.
constexpr int kWcTileRows = 32, kWcTileCols = 16, kWcTileElems = 512;
__host__ __device__ __forceinline__ int wc_in_tile(int r, int c) {          // r < 32, c < 16
  return r * 16 + ((((c >> 1) ^ (r & 7)) << 1) | (c & 1));
}
__host__ __device__ __forceinline__ int64_t wc_index(int64_t row, int64_t col, int64_t in) {
  return ((row >> 5) * (in >> 4) + (col >> 4)) * kWcTileElems + wc_in_tile(static_cast<int>(row & 31), static_cast<int>(col & 15));
}

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
