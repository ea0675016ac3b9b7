// Round-to-nearest group quantizer for both grouping dimensions in one pass over W
// (paper Section 3.3: the weights are quantized per-OC and per-IC independently; Section 4.1:
// uniform asymmetric, group size g).  A 128 x 128 tile of W holds whole per-OC groups (row
// segments) and whole per-IC groups (column segments) for every supported g, so one CTA reads
// its tile once, keeps it in registers and emits codes and parameters for both dimensions.
// The kernel is bound by HBM traffic: per weight it reads sizeof(T) bytes and writes, per
// dimension, bits/8 bytes of codes and 4/g bytes of parameters.
#include "common.cuh"

namespace adadim {
namespace {

constexpr int kThreads = 256;       // 16 threads across a tile row (8 columns each) x 16 rows
constexpr int kPasses = 8;          // 16 rows per pass

// Eight codes of one row segment from the correctly rounded quotients: adding 1.5 * 2^23 leaves
// rint(q) in the low mantissa bits; code = clamp(bits - bias, 0, maxq) with bias = magic - z is
// one integer add-min-relu; the codes are packed by multiply-add.  |q| stays far below 2^22
// here because every weight lies inside its own group's range.
// The eight codes come back as a 64-bit value in two words; only 8-bit codes use the second one.
template <int BITS>
__device__ __forceinline__ uint2 pack8(const float (&w)[8], const float (&s)[8], const float (&r)[8],
                                       const int (&nbias)[8]) {
  constexpr int maxq = (1 << BITS) - 1;
  uint32_t acc = 0, acc_hi = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const float t = __fadd_rn(quotient(w[k], s[k], r[k]), kRoundMagic);
    const int c = __viaddmin_s32_relu(__float_as_int(t), nbias[k], maxq);
    if (BITS * k < 32) acc = static_cast<uint32_t>(c) * (1u << ((BITS * k) & 31)) + acc;
    else acc_hi = static_cast<uint32_t>(c) * (1u << ((BITS * k) & 31)) + acc_hi;
  }
  return make_uint2(acc, acc_hi);
}

// Pack eight codes (column order) of `BITS` bits and hand back this thread's share of the
// row's bitstream.  acc arrives as sum_k(tbits_k << BITS*k) - bias, i.e. the packed value.
template <int BITS>
__device__ __forceinline__ void store_codes(uint2 packed2, uint32_t* row_words, int colvec, bool ok) {
  const uint32_t packed = packed2.x;
  if (BITS == 8) {          // 64 bits per thread: two whole words
    if (ok) *reinterpret_cast<uint2*>(row_words + colvec * 2) = packed2;
  } else if (BITS == 4) {
    if (ok) row_words[colvec] = packed;
  } else if (BITS == 2) {   // 16 bits per thread: two threads make a word
    const uint32_t up = __shfl_down_sync(0xffffffffu, packed, 1);
    if (ok && (colvec & 1) == 0) row_words[colvec >> 1] = packed | (up << 16);
  } else {  // BITS == 3: 24 bits per thread, four threads make three words
    uint32_t up = __shfl_down_sync(0xffffffffu, packed, 1);
    int k = colvec & 3;
    uint32_t word = (packed >> (8 * k)) | (up << (24 - 8 * k));
    if (ok && k < 3) row_words[(colvec >> 2) * 3 + k] = word;
  }
}
template <int BITS>
__device__ __forceinline__ void store_codes(uint32_t packed, uint32_t* row_words, int colvec, bool ok) {
  store_codes<BITS>(make_uint2(packed, 0u), row_words, colvec, ok);
}

template <typename T, int BITS, int G, bool DO_OC, bool DO_IC>
__global__ void __launch_bounds__(kThreads, 2)
rtn_tile_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw,
                adadim_qtensor qoc, adadim_qtensor qic) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;            // correctly rounded at compile time
  constexpr int NG = kTile / G;               // per-IC groups stacked in one tile
  constexpr int PPG = kPasses / NG;           // passes per such group
  constexpr int LANES_PER_OCG = G / 8;        // threads sharing one per-OC group

  __shared__ float s_mn[NG][8][kTile];
  __shared__ float s_mx[NG][8][kTile];
  __shared__ float s_s[NG][kTile];
  __shared__ float s_z[NG][kTile];

  const int tid = threadIdx.x;
  const int colvec = tid & 15, rowsub = tid >> 4;
  const int warp = tid >> 5, lane = tid & 31;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kTile;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * kTile;
  const int64_t col = c0 + colvec * 8;
  const bool col_ok = col < in;               // in % 32 == 0: a thread's 8 columns are all in or out
  const int64_t words_per_row = in * BITS / 32;

  float w[kPasses][8];
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    int64_t row = r0 + p * 16 + rowsub;
    if (col_ok && row < out) {
      load8(W + row * ldw + col, w[p]);
    } else {
#pragma unroll
      for (int k = 0; k < 8; ++k) w[p][k] = 0.0f;     // neutral: 0 always lies inside [lo, hi]
    }
  }

  // ---- per-IC statistics: column minima / maxima over each g-row group of the tile ---------
  if (DO_IC) {
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      float mn[8], mx[8];
#pragma unroll
      for (int k = 0; k < 8; ++k) { mn[k] = w[gi * PPG][k]; mx[k] = mn[k]; }
#pragma unroll
      for (int p = 1; p < PPG; ++p)
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          mn[k] = fminf(mn[k], w[gi * PPG + p][k]);
          mx[k] = fmaxf(mx[k], w[gi * PPG + p][k]);
        }
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        mn[k] = fminf(mn[k], __shfl_xor_sync(0xffffffffu, mn[k], 16));
        mx[k] = fmaxf(mx[k], __shfl_xor_sync(0xffffffffu, mx[k], 16));
      }
      if (lane < 16) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
          s_mn[gi][warp][colvec * 8 + k] = mn[k];
          s_mx[gi][warp][colvec * 8 + k] = mx[k];
        }
      }
    }
    __syncthreads();
    for (int t = tid; t < NG * kTile; t += kThreads) {
      int gi = t / kTile, c = t % kTile;
      float mn = s_mn[gi][0][c], mx = s_mx[gi][0][c];
#pragma unroll
      for (int wv = 1; wv < 8; ++wv) {
        mn = fminf(mn, s_mn[gi][wv][c]);
        mx = fmaxf(mx, s_mx[gi][wv][c]);
      }
      GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
      s_s[gi][c] = gp.rcp == 0.0f ? 0.0f : gp.s;      // 0 marks a degenerate group
      s_z[gi][c] = gp.z;
      int64_t grow = r0 / G + gi;
      if (c0 + c < in && grow * G < out) {
        qic.scales[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.s));
        qic.zeros[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.z));
      }
    }
    __syncthreads();
  }

  // ---- codes ------------------------------------------------------------------------------
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) {
    float ic_s[8], ic_r[8];
    int ic_nb[8];
    if (DO_IC) {
#pragma unroll
      for (int k = 0; k < 8; ++k) {
        float s = s_s[gi][colvec * 8 + k];
        ic_r[k] = s == 0.0f ? 0.0f : __frcp_rn(s);
        ic_s[k] = s == 0.0f ? 1.0f : s;
        ic_nb[k] = static_cast<int>(s_z[gi][colvec * 8 + k]) - kRoundMagicBits;
      }
    }
#pragma unroll
    for (int pp = 0; pp < PPG; ++pp) {
      const int p = gi * PPG + pp;
      const int64_t row = r0 + p * 16 + rowsub;
      const bool ok = col_ok && row < out;
      if (DO_OC) {
        float mn = w[p][0], mx = w[p][0];
#pragma unroll
        for (int k = 1; k < 8; ++k) { mn = fminf(mn, w[p][k]); mx = fmaxf(mx, w[p][k]); }
#pragma unroll
        for (int m = 1; m < LANES_PER_OCG; m <<= 1) {
          mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, m));
          mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, m));
        }
        GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
        if (ok && (colvec % LANES_PER_OCG) == 0) {
          int64_t idx = row * (in / G) + col / G;
          qoc.scales[idx] = __half_as_ushort(__float2half_rn(gp.s));
          qoc.zeros[idx] = __half_as_ushort(__float2half_rn(gp.z));
        }
        float s8[8], r8[8];
        int nb8[8];
#pragma unroll
        for (int k = 0; k < 8; ++k) { s8[k] = gp.s; r8[k] = gp.rcp; nb8[k] = static_cast<int>(gp.z) - kRoundMagicBits; }
        const uint2 acc = pack8<BITS>(w[p], s8, r8, nb8);
        store_codes<BITS>(acc, qoc.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, colvec, ok);
      }
      if (DO_IC) {
        const uint2 acc = pack8<BITS>(w[p], ic_s, ic_r, ic_nb);
        store_codes<BITS>(acc, qic.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, colvec, ok);
      }
    }
  }
}

// ---- fp16 weights --------------------------------------------------------------------------
// The same tile, kept in registers as it was loaded (f16x2 words) and widened to fp32 only where
// the codes are formed.  Differences from the general kernel above, all exact:
//  * minima and maxima are taken on f16x2 words (an fp16 minimum is exact);
//  * the per-OC statistics of the eight passes are reduced across the lanes of a group by a
//    reduce-scatter, so each lane ends up owning one (row, group), computes its parameters once
//    and hands reciprocal and zero point to the others by shuffle when the codes are formed;
//  * rint(w / s) for fp16 w and s needs no correctly rounded quotient.  Write w = a 2^x and
//    s = b 2^y with integers |a|, b < 2^11: w/s - (m + 1/2) is either 0 or at least 2^-13 in
//    magnitude for every integer m (its numerator is a non-zero integer over a denominator of
//    at most 2^13 whenever |w/s| >= 1/2).  p = w * rcp(s) is within 2^-20 of w/s for |w/s| <= 16.
//    fma(w, rcp, 192) rounds p to a multiple of 2^-16: an exact tie comes out as exactly m + 1/2,
//    everything else stays on its side of every m + 1/2.  Adding 1.5 * 2^23 - 192 then rounds
//    that to an integer, ties to even, which is rint of the correctly rounded quotient.
constexpr float kSnapMagic = 192.0f;                     // 1.5 * 2^7: ulp 2^-16 in [128, 256)
constexpr float kSnapToInt = 12582912.0f - 192.0f;       // exact in binary32

__device__ __forceinline__ uint32_t min_h2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("min.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t max_h2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ float lo_h2(uint32_t v) { return __half2float(__ushort_as_half(static_cast<unsigned short>(v & 0xffffu))); }
__device__ __forceinline__ float hi_h2(uint32_t v) { return __half2float(__ushort_as_half(static_cast<unsigned short>(v >> 16))); }

// volatile keeps the widening beside its use: only the packed tile stays live across the passes.
__device__ __forceinline__ void widen_h2(uint32_t v, float& a, float& b) {
  asm volatile("{\n\t.reg .b16 l, h;\n\tmov.b32 {l, h}, %2;\n\tcvt.f32.f16 %0, l;\n\tcvt.f32.f16 %1, h;\n\t}"
               : "=f"(a), "=f"(b) : "r"(v));
}

// One halving exchange of a reduce-scatter: the lanes whose `bit` is set keep the upper n words,
// the others the lower n, and each receives its partner's copy of the words it keeps.
template <int N>
__device__ __forceinline__ void halve_min(uint32_t (&v)[8], int lane, int bit) {
  const bool up = (lane & bit) != 0;
#pragma unroll
  for (int i = 0; i < N; ++i) {
    const uint32_t send = up ? v[i] : v[i + N], keep = up ? v[i + N] : v[i];
    v[i] = min_h2(keep, __shfl_xor_sync(0xffffffffu, send, bit));
  }
}

// v[0..7] hold one f16x2 word per pass; the minimum over the LANES consecutive lanes of a group is
// formed by halving exchanges.  Afterwards a lane holds the finished words of the passes
//   LANES == 16: (lane & 15) >> 1 in v[0]           (both lanes of a pair hold the same one)
//   LANES ==  8:  lane & 7        in v[0]
//   LANES ==  4:  2 * (lane & 1) + 4 * ((lane >> 1) & 1) + j  in v[j], j = 0, 1
template <int LANES>
__device__ __forceinline__ void reduce_scatter_min(uint32_t (&v)[8], int lane) {
  if (LANES == 16) {
    halve_min<4>(v, lane, 8);
    halve_min<2>(v, lane, 4);
    halve_min<1>(v, lane, 2);
    v[0] = min_h2(v[0], __shfl_xor_sync(0xffffffffu, v[0], 1));
  } else if (LANES == 8) {
    halve_min<4>(v, lane, 4);
    halve_min<2>(v, lane, 2);
    halve_min<1>(v, lane, 1);
  } else {  // LANES == 4
    halve_min<4>(v, lane, 2);
    halve_min<2>(v, lane, 1);
  }
}

// Eight codes of one row segment of fp16 weights (see the note above), packed by multiply-add.
// The two roundings run two weights at a time on the packed fp32x2 forms of fma and add; each
// half is the IEEE operation, so nothing changes numerically.
template <int BITS>
__device__ __forceinline__ uint32_t pack8_h(const float2 (&w)[4], const float2 (&r)[4], const int (&nbias)[8]) {
  constexpr int maxq = (1 << BITS) - 1;
  const float2 snap = make_float2(kSnapMagic, kSnapMagic), to_int = make_float2(kSnapToInt, kSnapToInt);
  uint32_t acc = 0;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const float2 t = __fadd2_rn(__ffma2_rn(w[k], r[k], snap), to_int);
    const int c0 = __viaddmin_s32_relu(__float_as_int(t.x), nbias[2 * k], maxq);
    const int c1 = __viaddmin_s32_relu(__float_as_int(t.y), nbias[2 * k + 1], maxq);
    acc = static_cast<uint32_t>(c0) * (1u << (BITS * 2 * k)) + acc;
    acc = static_cast<uint32_t>(c1) * (1u << (BITS * (2 * k + 1))) + acc;
  }
  return acc;
}

template <int BITS, int G, bool DO_OC, bool DO_IC>
__global__ void __launch_bounds__(kThreads, G == 32 ? 2 : 4)
rtn_half_kernel(const __half* __restrict__ W, int64_t out, int64_t in, int64_t ldw,
                adadim_qtensor qoc, adadim_qtensor qic) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;
  constexpr int NG = kTile / G;               // per-IC groups stacked in one tile
  constexpr int PPG = kPasses / NG;           // passes per such group
  constexpr int LANES = G / 8;                // lanes sharing one per-OC group
  constexpr int HELD = LANES == 4 ? 2 : 1;    // finished per-OC groups a lane owns

  __shared__ uint32_t s_mn[DO_IC ? NG : 1][8][kTile / 2];       // f16x2 column minima per warp
  __shared__ uint32_t s_mx[DO_IC ? NG : 1][8][kTile / 2];
  __shared__ __align__(16) float s_r[DO_IC ? NG : 1][kTile];    // reciprocal scale (0: degenerate group)
  __shared__ __align__(16) int s_nb[DO_IC ? NG : 1][kTile];     // zero point - bits of 1.5 * 2^23

  const int tid = threadIdx.x;
  const int colvec = tid & 15, rowsub = tid >> 4;
  const int warp = tid >> 5, lane = tid & 31;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kTile;
  const int64_t c0 = static_cast<int64_t>(blockIdx.x) * kTile;
  const int64_t col = c0 + colvec * 8;
  const bool col_ok = col < in;               // in % 32 == 0: a thread's 8 columns are all in or out
  const int64_t words_per_row = in * BITS / 32;

  uint4 x[kPasses];
  uint32_t oc[8];                             // per pass: (segment minimum, -segment maximum)
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    const int64_t row = r0 + p * 16 + rowsub;
    if (col_ok && row < out) x[p] = *reinterpret_cast<const uint4*>(W + row * ldw + col);
    else x[p] = make_uint4(0u, 0u, 0u, 0u);   // 0 is neutral: it lies inside every [lo, hi]
  }
#pragma unroll
  for (int p = 0; p < kPasses; ++p) {
    if (DO_OC) {
      const uint32_t mn = min_h2(min_h2(x[p].x, x[p].y), min_h2(x[p].z, x[p].w));
      const uint32_t nmx = max_h2(max_h2(x[p].x, x[p].y), max_h2(x[p].z, x[p].w)) ^ 0x80008000u;
      oc[p] = min_h2(__byte_perm(mn, nmx, 0x5410), __byte_perm(mn, nmx, 0x7632));
    } else {
      oc[p] = 0u;
    }
  }

  // ---- per-IC statistics: column minima / maxima over each g-row group of the tile ---------
  if (DO_IC) {
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
      uint32_t cmn[4] = {x[gi * PPG].x, x[gi * PPG].y, x[gi * PPG].z, x[gi * PPG].w};
      uint32_t cmx[4] = {cmn[0], cmn[1], cmn[2], cmn[3]};
#pragma unroll
      for (int pp = 1; pp < PPG; ++pp) {
        const uint4 v = x[gi * PPG + pp];
        cmn[0] = min_h2(cmn[0], v.x); cmn[1] = min_h2(cmn[1], v.y); cmn[2] = min_h2(cmn[2], v.z); cmn[3] = min_h2(cmn[3], v.w);
        cmx[0] = max_h2(cmx[0], v.x); cmx[1] = max_h2(cmx[1], v.y); cmx[2] = max_h2(cmx[2], v.z); cmx[3] = max_h2(cmx[3], v.w);
      }
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        cmn[k] = min_h2(cmn[k], __shfl_xor_sync(0xffffffffu, cmn[k], 16));
        cmx[k] = max_h2(cmx[k], __shfl_xor_sync(0xffffffffu, cmx[k], 16));
      }
      if (lane < 16) {
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          s_mn[gi][warp][colvec * 4 + k] = cmn[k];
          s_mx[gi][warp][colvec * 4 + k] = cmx[k];
        }
      }
    }
  }
  __syncthreads();

  // ---- group parameters: each group once --------------------------------------------------------
  float own_r[HELD];
  int own_nb[HELD];
#pragma unroll
  for (int j = 0; j < HELD; ++j) { own_r[j] = 0.0f; own_nb[j] = 0; }
  if (DO_OC) {
    reduce_scatter_min<LANES>(oc, lane);
#pragma unroll
    for (int j = 0; j < HELD; ++j) {
      const GroupParams gp = group_params(lo_h2(oc[j]), -hi_h2(oc[j]), maxq, rcp_maxq);
      own_r[j] = gp.rcp;
      own_nb[j] = static_cast<int>(gp.z) - kRoundMagicBits;
      const int p = LANES == 16 ? (lane & 15) >> 1 : LANES == 8 ? (lane & 7) : 2 * (lane & 1) + 4 * ((lane >> 1) & 1) + j;
      const int64_t row = r0 + p * 16 + rowsub;
      const bool writer = LANES == 16 ? (lane & 1) == 0 : true;
      if (writer && col_ok && row < out) {
        const int64_t idx = row * (in / G) + col / G;
        qoc.scales[idx] = __half_as_ushort(__float2half_rn(gp.s));
        qoc.zeros[idx] = __half_as_ushort(__float2half_rn(gp.z));
      }
    }
  }
  if (DO_IC) {
    for (int t = tid; t < NG * kTile; t += kThreads) {
      const int gi = t / kTile, c = t % kTile;
      uint32_t mn2 = s_mn[gi][0][c >> 1], mx2 = s_mx[gi][0][c >> 1];
#pragma unroll
      for (int wv = 1; wv < 8; ++wv) {
        mn2 = min_h2(mn2, s_mn[gi][wv][c >> 1]);
        mx2 = max_h2(mx2, s_mx[gi][wv][c >> 1]);
      }
      const float mn = (c & 1) ? hi_h2(mn2) : lo_h2(mn2), mx = (c & 1) ? hi_h2(mx2) : lo_h2(mx2);
      const GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
      s_r[gi][c] = gp.rcp;
      s_nb[gi][c] = static_cast<int>(gp.z) - kRoundMagicBits;
      const int64_t grow = r0 / G + gi;
      if (c0 + c < in && grow * G < out) {
        qic.scales[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.s));
        qic.zeros[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.z));
      }
    }
    __syncthreads();
  }

  // ---- codes ------------------------------------------------------------------------------
#pragma unroll
  for (int gi = 0; gi < NG; ++gi) {
    float2 ic_r[4];
    int ic_nb[8];
    if (DO_IC) {
#pragma unroll
      for (int k = 0; k < 4; ++k) ic_r[k] = make_float2(s_r[gi][colvec * 8 + 2 * k], s_r[gi][colvec * 8 + 2 * k + 1]);
#pragma unroll
      for (int k = 0; k < 8; ++k) ic_nb[k] = s_nb[gi][colvec * 8 + k];
    }
#pragma unroll
    for (int pp = 0; pp < PPG; ++pp) {
      const int p = gi * PPG + pp;
      const int64_t row = r0 + p * 16 + rowsub;
      const bool ok = col_ok && row < out;
      float2 w[4];
      widen_h2(x[p].x, w[0].x, w[0].y);
      widen_h2(x[p].y, w[1].x, w[1].y);
      widen_h2(x[p].z, w[2].x, w[2].y);
      widen_h2(x[p].w, w[3].x, w[3].y);
      if (DO_OC) {
        // the lane that owns (this row, this group) of pass p, and the slot it keeps it in
        const int base = lane & ~(LANES - 1);
        const int src = LANES == 16 ? base | (p << 1) : LANES == 8 ? base | p : base | (((p >> 2) & 1) << 1) | ((p >> 1) & 1);
        const int slot = LANES == 4 ? (p & 1) : 0;
        const float rr = __shfl_sync(0xffffffffu, own_r[slot], src);
        const int nbv = __shfl_sync(0xffffffffu, own_nb[slot], src);
        float2 r8[4];
        int nb8[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) r8[k] = make_float2(rr, rr);
#pragma unroll
        for (int k = 0; k < 8; ++k) nb8[k] = nbv;
        store_codes<BITS>(pack8_h<BITS>(w, r8, nb8), qoc.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, colvec, ok);
      }
      if (DO_IC) {
        store_codes<BITS>(pack8_h<BITS>(w, ic_r, ic_nb), qic.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, colvec, ok);
      }
    }
  }
}

template <int BITS, int G>
void launch_dims(const __half* W, int64_t out, int64_t in, int64_t ldw, int dim,
                 const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  dim3 grid(static_cast<unsigned>((in + kTile - 1) / kTile), static_cast<unsigned>((out + kTile - 1) / kTile));
  if (dim == ADADIM_DIM_BOTH)
    rtn_half_kernel<BITS, G, true, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else if (dim == ADADIM_DIM_OC)
    rtn_half_kernel<BITS, G, true, false><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else
    rtn_half_kernel<BITS, G, false, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
}

template <typename T, int BITS, int G>
void launch_dims(const T* W, int64_t out, int64_t in, int64_t ldw, int dim,
                 const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  dim3 grid(static_cast<unsigned>((in + kTile - 1) / kTile), static_cast<unsigned>((out + kTile - 1) / kTile));
  if (dim == ADADIM_DIM_BOTH)
    rtn_tile_kernel<T, BITS, G, true, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else if (dim == ADADIM_DIM_OC)
    rtn_tile_kernel<T, BITS, G, true, false><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else
    rtn_tile_kernel<T, BITS, G, false, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
}

template <typename T, int BITS>
void launch_group(const T* W, int64_t out, int64_t in, int64_t ldw, int group, int dim,
                  const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  if (group == 128) launch_dims<T, BITS, 128>(W, out, in, ldw, dim, qoc, qic, st);
  else if (group == 64) launch_dims<T, BITS, 64>(W, out, in, ldw, dim, qoc, qic, st);
  else launch_dims<T, BITS, 32>(W, out, in, ldw, dim, qoc, qic, st);
}

template <int BITS>
void launch_group_half(const __half* W, int64_t out, int64_t in, int64_t ldw, int group, int dim,
                       const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  if (group == 128) launch_dims<BITS, 128>(W, out, in, ldw, dim, qoc, qic, st);
  else if (group == 64) launch_dims<BITS, 64>(W, out, in, ldw, dim, qoc, qic, st);
  else launch_dims<BITS, 32>(W, out, in, ldw, dim, qoc, qic, st);
}

// ---- g = 256 (the largest group size of the paper's sweep, Section 4.4) ------------------------
// A 256 x 256 tile holds whole groups of both dimensions but not in registers, so the tile is read
// twice: once for the statistics, once (from L2, where it still is) for the codes.  A warp covers
// one row of the tile per pass (32 lanes x 8 columns), so a per-OC group is one warp-wide
// reduction; per-IC statistics are accumulated per thread over the 32 passes and combined across
// the eight warps through shared memory.  Exact formula throughout (the general quotient).
constexpr int kTile256 = 256;
template <typename T, int BITS, bool DO_OC, bool DO_IC>
__global__ void __launch_bounds__(kThreads, 2)
rtn_g256_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, adadim_qtensor qoc, adadim_qtensor qic) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;
  constexpr int kRowsPerPass = kThreads / 32;            // 8
  constexpr int kPasses256 = kTile256 / kRowsPerPass;    // 32
  __shared__ float s_cmn[kRowsPerPass][kTile256], s_cmx[kRowsPerPass][kTile256];
  __shared__ float s_ic_s[kTile256], s_ic_r[kTile256];
  __shared__ int s_ic_nb[kTile256];
  __shared__ float s_oc_s[kTile256], s_oc_r[kTile256];
  __shared__ int s_oc_nb[kTile256];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kTile256, c0 = static_cast<int64_t>(blockIdx.x) * kTile256;
  const int64_t col = c0 + lane * 8;
  const bool col_ok = col < in;
  const int64_t words_per_row = in * BITS / 32;

  // ---- statistics ----------------------------------------------------------------------------
  float cmn[8], cmx[8];
#pragma unroll
  for (int k = 0; k < 8; ++k) { cmn[k] = 0.0f; cmx[k] = 0.0f; }    // 0 always lies inside [lo, hi]
#pragma unroll 4
  for (int p = 0; p < kPasses256; ++p) {
    const int lr = p * kRowsPerPass + warp;
    const int64_t row = r0 + lr;
    float w[8];
    if (col_ok && row < out) load8(W + row * ldw + col, w);
    else {
#pragma unroll
      for (int k = 0; k < 8; ++k) w[k] = 0.0f;
    }
    if (DO_IC) {
#pragma unroll
      for (int k = 0; k < 8; ++k) { cmn[k] = fminf(cmn[k], w[k]); cmx[k] = fmaxf(cmx[k], w[k]); }
    }
    if (DO_OC) {
      float mn = w[0], mx = w[0];
#pragma unroll
      for (int k = 1; k < 8; ++k) { mn = fminf(mn, w[k]); mx = fmaxf(mx, w[k]); }
#pragma unroll
      for (int m = 16; m > 0; m >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, m));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, m));
      }
      if (lane == 0) {
        const GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
        s_oc_s[lr] = gp.s; s_oc_r[lr] = gp.rcp; s_oc_nb[lr] = static_cast<int>(gp.z) - kRoundMagicBits;
        if (row < out && c0 < in) {
          const int64_t idx = row * (in / kTile256) + c0 / kTile256;
          qoc.scales[idx] = __half_as_ushort(__float2half_rn(gp.s));
          qoc.zeros[idx] = __half_as_ushort(__float2half_rn(gp.z));
        }
      }
    }
  }
  if (DO_IC) {
#pragma unroll
    for (int k = 0; k < 8; ++k) { s_cmn[warp][lane * 8 + k] = cmn[k]; s_cmx[warp][lane * 8 + k] = cmx[k]; }
  }
  __syncthreads();
  if (DO_IC) {
    const int c = tid;                                   // one column per thread
    float mn = s_cmn[0][c], mx = s_cmx[0][c];
#pragma unroll
    for (int wv = 1; wv < kRowsPerPass; ++wv) { mn = fminf(mn, s_cmn[wv][c]); mx = fmaxf(mx, s_cmx[wv][c]); }
    const GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
    s_ic_s[c] = gp.s; s_ic_r[c] = gp.rcp; s_ic_nb[c] = static_cast<int>(gp.z) - kRoundMagicBits;
    const int64_t grow = r0 / kTile256;
    if (c0 + c < in && r0 < out) {
      qic.scales[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.s));
      qic.zeros[grow * in + c0 + c] = __half_as_ushort(__float2half_rn(gp.z));
    }
  }
  __syncthreads();

  // ---- codes ---------------------------------------------------------------------------------
  float ic_s[8], ic_r[8];
  int ic_nb[8];
  if (DO_IC) {
#pragma unroll
    for (int k = 0; k < 8; ++k) { ic_s[k] = s_ic_s[lane * 8 + k]; ic_r[k] = s_ic_r[lane * 8 + k]; ic_nb[k] = s_ic_nb[lane * 8 + k]; }
  }
#pragma unroll 2
  for (int p = 0; p < kPasses256; ++p) {
    const int lr = p * kRowsPerPass + warp;
    const int64_t row = r0 + lr;
    const bool ok = col_ok && row < out;
    float w[8];
    if (ok) load8(W + row * ldw + col, w);
    else {
#pragma unroll
      for (int k = 0; k < 8; ++k) w[k] = 0.0f;
    }
    if (DO_OC) {
      float s8[8], r8[8];
      int nb8[8];
      const float sv = s_oc_s[lr], rv = s_oc_r[lr];
      const int nbv = s_oc_nb[lr];
#pragma unroll
      for (int k = 0; k < 8; ++k) { s8[k] = sv; r8[k] = rv; nb8[k] = nbv; }
      store_codes<BITS>(pack8<BITS>(w, s8, r8, nb8), qoc.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, lane, ok);
    }
    if (DO_IC) {
      store_codes<BITS>(pack8<BITS>(w, ic_s, ic_r, ic_nb), qic.codes + (ok ? row : 0) * words_per_row + c0 * BITS / 32, lane, ok);
    }
  }
}

template <typename T, int BITS>
void launch_g256(const T* W, int64_t out, int64_t in, int64_t ldw, int dim,
                 const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  dim3 grid(static_cast<unsigned>((in + kTile256 - 1) / kTile256), static_cast<unsigned>((out + kTile256 - 1) / kTile256));
  if (dim == ADADIM_DIM_BOTH) rtn_g256_kernel<T, BITS, true, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else if (dim == ADADIM_DIM_OC) rtn_g256_kernel<T, BITS, true, false><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
  else rtn_g256_kernel<T, BITS, false, true><<<grid, kThreads, 0, st>>>(W, out, in, ldw, qoc, qic);
}

template <int BITS>
__global__ void unpack_kernel(const uint32_t* __restrict__ codes, int64_t out, int64_t in, uint8_t* __restrict__ dst) {
  // one thread per 32 codes (BITS words of input, 32 bytes of output)
  int64_t chunks_per_row = in / 32;
  int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= out * chunks_per_row) return;
  int64_t row = t / chunks_per_row, ch = t % chunks_per_row;
  const uint32_t* src = codes + row * (in * BITS / 32) + ch * BITS;
  uint32_t wds[BITS + 1];
#pragma unroll
  for (int k = 0; k < BITS; ++k) wds[k] = src[k];
  wds[BITS] = 0;
  uint32_t outw[8];
#pragma unroll
  for (int k = 0; k < 32; ++k) {
    int bit = k * BITS, wi = bit >> 5, sh = bit & 31;
    uint32_t v = wds[wi] >> sh;
    if (sh + BITS > 32) v |= wds[wi + 1] << (32 - sh);
    v &= (1u << BITS) - 1u;
    if ((k & 3) == 0) outw[k >> 2] = v; else outw[k >> 2] |= v << (8 * (k & 3));
  }
  uint4* d = reinterpret_cast<uint4*>(dst + row * in + ch * 32);
  d[0] = make_uint4(outw[0], outw[1], outw[2], outw[3]);
  d[1] = make_uint4(outw[4], outw[5], outw[6], outw[7]);
}

}  // namespace

template <typename T>
void launch_bits(const T* W, int64_t out, int64_t in, int64_t ldw, int bits, int group, int dim,
                 const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  if (group == 256) {
    if (bits == 2) launch_g256<T, 2>(W, out, in, ldw, dim, qoc, qic, st);
    else if (bits == 3) launch_g256<T, 3>(W, out, in, ldw, dim, qoc, qic, st);
    else if (bits == 4) launch_g256<T, 4>(W, out, in, ldw, dim, qoc, qic, st);
    else launch_g256<T, 8>(W, out, in, ldw, dim, qoc, qic, st);
  } else {
    if (bits == 2) launch_group<T, 2>(W, out, in, ldw, group, dim, qoc, qic, st);
    else if (bits == 3) launch_group<T, 3>(W, out, in, ldw, group, dim, qoc, qic, st);
    else if (bits == 4) launch_group<T, 4>(W, out, in, ldw, group, dim, qoc, qic, st);
    else launch_group<T, 8>(W, out, in, ldw, group, dim, qoc, qic, st);
  }
}

int rtn_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, int bits, int group, int dim,
               const adadim_qtensor& qoc, const adadim_qtensor& qic, cudaStream_t st) {
  if (wdtype == ADADIM_F16 && group != 256 && bits != 8) {
    // the register-resident f16x2 kernel; its division-free rounding is proven for |w / s| <= 16 (up to 4 bits)
    const __half* Wh = static_cast<const __half*>(W);
    if (bits == 2) launch_group_half<2>(Wh, out, in, ldw, group, dim, qoc, qic, st);
    else if (bits == 3) launch_group_half<3>(Wh, out, in, ldw, group, dim, qoc, qic, st);
    else launch_group_half<4>(Wh, out, in, ldw, group, dim, qoc, qic, st);
  } else if (wdtype == ADADIM_F16) {
    launch_bits(static_cast<const __half*>(W), out, in, ldw, bits, group, dim, qoc, qic, st);
  } else {
    launch_bits(static_cast<const float*>(W), out, in, ldw, bits, group, dim, qoc, qic, st);
  }
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

int unpack_launch(const uint32_t* codes, int64_t out, int64_t in, int bits, uint8_t* dst, cudaStream_t st) {
  int64_t n = out * (in / 32);
  if (n == 0) return ADADIM_OK;
  unsigned blocks = static_cast<unsigned>((n + 255) / 256);
  if (bits == 2) unpack_kernel<2><<<blocks, 256, 0, st>>>(codes, out, in, dst);
  else if (bits == 3) unpack_kernel<3><<<blocks, 256, 0, st>>>(codes, out, in, dst);
  else if (bits == 4) unpack_kernel<4><<<blocks, 256, 0, st>>>(codes, out, in, dst);
  else unpack_kernel<8><<<blocks, 256, 0, st>>>(codes, out, in, dst);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
