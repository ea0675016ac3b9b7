// GPTQ with lazily batched error compensation (paper Section 2.2; Section 3.3: the per-IC
// variant changes only the quantization step).  Columns are handled in blocks of 128:
//   block kernel    - one CTA per 128-row slab and grouping dimension walks the block's
//                     columns in order: group parameters from the current weights, code,
//                     error e = (w - q) / U[i,i], and the update of the block's remaining
//                     columns, w[j] -= e U[i,j].  The slab lives in shared memory; the 32
//                     columns being worked on live in registers.
//   trailing update - W[:, after the block] -= Err[out,128] * U[block rows, after the block]
//                     on the tensor cores with exactly sliced bf16 operands (gptq_tc.cu).
// Rows are independent under per-OC grouping; under per-IC grouping a group couples g
// consecutive rows of one column, which is why a CTA owns a whole 128-row slab.
#include <cuda.h>
#include <cuda_bf16.h>

#include "common.cuh"

namespace adadim {

struct TrailPlan {
  CUtensorMap e[3], u[3], w;
  float* Wc;
  int64_t rows_total, in;
  int sm_count;
};
int trail_split_u(const float* U, int64_t in, __nv_bfloat16* u0, __nv_bfloat16* u1, __nv_bfloat16* u2, cudaStream_t st);
int trail_plan(TrailPlan* plan, float* Wc, int64_t rows_total, int64_t in, const __nv_bfloat16* const e[3],
               const __nv_bfloat16* const u[3]);
int trail_launch(const TrailPlan& plan, int i1, int64_t c0, int ntiles, int tiles_per_cta, int* status_dev, cudaStream_t st);

size_t factor_workspace_bytes(int64_t n);
int factor_launch(const float* H, int64_t n, float percdamp, float* U, int* status_dev, void* workspace,
                  cudaStream_t st, const int* perm);

namespace {

constexpr int kBlk = 128;            // lazy-batch block width (columns) and slab height (rows)
constexpr int kSub = 32;             // columns held in registers at a time
constexpr int kPad = kBlk + 1;       // shared-memory row pitch (floats): conflict-free column access

template <typename T>
__global__ void __launch_bounds__(256)
init_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, const float* __restrict__ H, int ndim,
            float* __restrict__ Wc) {
  int64_t e = (static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x) * 8;
  if (e >= out * in) return;
  int64_t o = e / in, i = e % in;
  float v[8];
  load8(W + o * ldw + i, v);
#pragma unroll
  for (int k = 0; k < 8; ++k)
    if (H[(i + k) * in + (i + k)] == 0.0f) v[k] = 0.0f;        // dead column
  for (int d = 0; d < ndim; ++d) {
    float4* dst = reinterpret_cast<float4*>(Wc + static_cast<int64_t>(d) * out * in + e);
    dst[0] = make_float4(v[0], v[1], v[2], v[3]);
    dst[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

struct BlockArgs {
  float* Wc;                 // [ndim][out][in] working weights
  const float* U;            // [in][in]
  __nv_bfloat16* Ep[3];      // [ndim*out][128] errors as three fixed-point bf16 pieces
  double* loss_part;         // [ndim][out/128]
  adadim_qtensor q[2];       // outputs for the dimension(s) in flight
  int dim_of[2];             // grouping dimension of working copy d
  int64_t out, in;
  int i1;                    // first column of the block
  // activation reordering (null / unused in the natural order): column i of the working copy is
  // column perm[i] of W; per-OC parameters are fixed per original group beforehand
  const int* perm;
  const uint2* static_rec;   // [out][in/g]: {bits of 1/s (0: degenerate group), fp16 s | fp16 z << 16}
  uint32_t* codes[2];        // where the block kernel writes codes (in working-copy column order)
};

// ---- activation reordering (paper Section 2.2, Appendix A.1) ---------------------------------
// perm: input channels by descending diag(H) (a zero diagonal counts as 1, like the dead-column
// fix), equal values in their original order; rank is its inverse.  Every channel counts the
// channels that come before it: exact, deterministic, n^2 comparisons.
__global__ void __launch_bounds__(256)
order_kernel(const float* __restrict__ H, int64_t n, int* __restrict__ perm, int* __restrict__ rank) {
  __shared__ float tile[256];
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  float di = 0.0f;
  if (i < n) { di = H[i * n + i]; if (di == 0.0f) di = 1.0f; }
  int before = 0;
  for (int64_t j0 = 0; j0 < n; j0 += 256) {
    const int64_t j = j0 + threadIdx.x;
    float dj = 0.0f;
    if (j < n) { dj = H[j * n + j]; if (dj == 0.0f) dj = 1.0f; }
    __syncthreads();
    tile[threadIdx.x] = dj;
    __syncthreads();
    const int lim = static_cast<int>(n - j0 < 256 ? n - j0 : 256);
    for (int k = 0; k < lim; ++k) {
      const float d = tile[k];
      before += (d > di || (d == di && j0 + k < i)) ? 1 : 0;
    }
  }
  if (i < n) { rank[i] = before; perm[before] = static_cast<int>(i); }
}

// Working copies in the quantization order: Wc[d][o][i] = W[o][perm[i]] (0 for dead columns).
template <typename T>
__global__ void __launch_bounds__(256)
init_perm_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, const float* __restrict__ H,
                 const int* __restrict__ perm, int ndim, float* __restrict__ Wc) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= out * in) return;
  const int64_t o = e / in, c = perm[e % in];
  float v = static_cast<float>(W[o * ldw + c]);
  if (H[c * in + c] == 0.0f) v = 0.0f;
  for (int d = 0; d < ndim; ++d) Wc[static_cast<int64_t>(d) * out * in + e] = v;
}

// Static per-OC groups: parameters of every group of g consecutive original columns, from the
// original weights, before anything is reordered or updated.  One thread per (row, group).
template <typename T, int BITS>
__global__ void __launch_bounds__(256)
static_params_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, int group, adadim_qtensor q,
                     uint2* __restrict__ rec) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;
  const int64_t groups = in / group;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (t >= out * groups) return;
  const int64_t o = t / groups, g = t % groups;
  const T* src = W + o * ldw + g * group;
  float mn = 0.0f, mx = 0.0f;                     // 0 always lies inside [lo, hi]
  for (int k = 0; k < group; k += 8) {
    float v[8];
    load8(src + k, v);
#pragma unroll
    for (int m = 0; m < 8; ++m) { mn = fminf(mn, v[m]); mx = fmaxf(mx, v[m]); }
  }
  const GroupParams gp = group_params(mn, mx, maxq, rcp_maxq);
  const unsigned short sb = __half_as_ushort(__float2half_rn(gp.s)), zb = __half_as_ushort(__float2half_rn(gp.z));
  q.scales[t] = sb;
  q.zeros[t] = zb;
  rec[t] = make_uint2(__float_as_uint(gp.rcp), static_cast<uint32_t>(sb) | (static_cast<uint32_t>(zb) << 16));
}

// Codes from working-copy column order back to the original columns: out word by out word,
// code of original column c = code at position rank[c] of the row's temporary bitstream.
template <int BITS>
__global__ void __launch_bounds__(256)
unpermute_codes_kernel(const uint32_t* __restrict__ tmp, const int* __restrict__ rank, int64_t out, int64_t in,
                       uint32_t* __restrict__ codes) {
  const int64_t chunks = in / 32;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (t >= out * chunks) return;
  const int64_t o = t / chunks, ch = t % chunks;
  const uint32_t* row = tmp + o * (in * BITS / 32);
  uint32_t wds[BITS] = {};
#pragma unroll 4
  for (int k = 0; k < 32; ++k) {
    const int64_t bit = static_cast<int64_t>(rank[ch * 32 + k]) * BITS;
    const int64_t wi = bit >> 5;
    const int sh = static_cast<int>(bit & 31);
    uint32_t v = row[wi] >> sh;
    if (sh + BITS > 32) v |= row[wi + 1] << (32 - sh);
    v &= (1u << BITS) - 1u;
    const int ob = k * BITS, ow = ob >> 5, os = ob & 31;
#pragma unroll
    for (int m = 0; m < BITS; ++m) {
      if (m == ow) wds[m] |= v << os;
      if (m == ow + 1 && os + BITS > 32) wds[m] |= v >> (32 - os);
    }
  }
  uint32_t* dst = codes + o * (in * BITS / 32) + ch * BITS;
#pragma unroll
  for (int m = 0; m < BITS; ++m) dst[m] = wds[m];
}

__device__ __forceinline__ int ordered_key(float v) {
  const int b = __float_as_int(v);
  return b ^ ((b >> 31) & 0x7fffffff);
}
__device__ __forceinline__ float from_ordered_key(int k) { return __int_as_float(k ^ ((k >> 31) & 0x7fffffff)); }

// W[:, later columns] -= Err[:, this sub-block] * U[sub-block rows, later columns] for the whole
// 128-row slab in shared memory.  A row-per-thread loop needs one warp-uniform U value per
// multiply-add, all of it through the shared-memory return path, which bounds it at a quarter of
// the multiply-add rate; here a thread owns 8 rows x CW columns, so 8 + CW loads feed 8 CW
// multiply-adds.  Every element still receives its 32 updates in the same order as before.
template <int CW>
__device__ __forceinline__ void lazy_update(float* __restrict__ Ws, const float* __restrict__ Us,
                                            const float* __restrict__ Es, int cbase, int tid) {
  const int r0 = (tid >> 3) * 8;
  const int col0 = cbase + kSub + (tid & 7) * CW;
  float acc[8][CW];
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int n = 0; n < CW; ++n) acc[m][n] = Ws[(r0 + m) * kPad + col0 + n];
#pragma unroll 4
  for (int ii = 0; ii < kSub; ++ii) {
    float e[8], u[CW];
#pragma unroll
    for (int m = 0; m < 8; ++m) e[m] = Es[(r0 + m) * kPad + cbase + ii];
#pragma unroll
    for (int n4 = 0; n4 < CW / 4; ++n4) {
      const float4 t = *reinterpret_cast<const float4*>(Us + (cbase + ii) * kBlk + col0 + 4 * n4);
      u[4 * n4] = t.x; u[4 * n4 + 1] = t.y; u[4 * n4 + 2] = t.z; u[4 * n4 + 3] = t.w;
    }
#pragma unroll
    for (int m = 0; m < 8; ++m)
#pragma unroll
      for (int n = 0; n < CW; ++n) acc[m][n] = fmaf(-e[m], u[n], acc[m][n]);
  }
#pragma unroll
  for (int m = 0; m < 8; ++m)
#pragma unroll
    for (int n = 0; n < CW; ++n) Ws[(r0 + m) * kPad + col0 + n] = acc[m][n];
}

template <int BITS, int G>
__global__ void __launch_bounds__(kBlk, 1)
block_kernel(const BlockArgs a) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;            // correctly rounded at compile time
  constexpr int NG = kBlk / G;                       // per-IC groups in the slab
  extern __shared__ float sm[];
  float* Ws = sm;                                    // [128][129] slab of the working weights
  float* Us = Ws + kBlk * kPad;                      // [128][128] block of U (upper triangle used)
  float* Es = Us + kBlk * kBlk;                      // [128][129] errors
  float* invd = Es + kBlk * kPad;                    // [128] 1 / U[i,i]
  float* red = invd + kBlk;                          // [2][4][2] per-IC min / max exchange
  uint16_t* Ss = reinterpret_cast<uint16_t*>(red + 16);   // [NG][128] per-IC scales (fp16 bits)
  uint16_t* Zs = Ss + NG * kBlk;                          // [NG][128]

  const int d = blockIdx.y;
  const bool is_ic = a.dim_of[d] == ADADIM_DIM_IC;
  const adadim_qtensor q = a.q[d];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t row0 = static_cast<int64_t>(blockIdx.x) * kBlk;
  const int64_t row = row0 + tid;
  float* Wd = a.Wc + static_cast<int64_t>(d) * a.out * a.in;

  // Stage the U block and the slab (coalesced), then work row-per-thread; eight rows' worth of
  // loads are in flight before the first is stored, so each copy costs 4 memory latencies, not 32.
  // The kernel may have been scheduled while the launch before it in the stream (the update of this
  // block's columns) is still finishing: U does not depend on it and is staged first; everything
  // after the wait sees that launch's results.
#pragma unroll 1
  for (int e0 = 0; e0 < kBlk * kBlk / 4; e0 += 8 * kBlk) {
    float4 uv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * kBlk + tid, r = e >> 5, c4 = (e & 31) * 4;
      uv[u] = *reinterpret_cast<const float4*>(a.U + static_cast<int64_t>(a.i1 + r) * a.in + a.i1 + c4);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * kBlk + tid, r = e >> 5, c4 = (e & 31) * 4;
      *reinterpret_cast<float4*>(Us + r * kBlk + c4) = uv[u];
    }
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
#pragma unroll 1
  for (int e0 = 0; e0 < kBlk * kBlk / 4; e0 += 8 * kBlk) {
    float4 wv[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * kBlk + tid, r = e >> 5, c4 = (e & 31) * 4;
      wv[u] = *reinterpret_cast<const float4*>(Wd + (row0 + r) * a.in + a.i1 + c4);
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int e = e0 + u * kBlk + tid, r = e >> 5, c4 = (e & 31) * 4;
      Ws[r * kPad + c4 + 0] = wv[u].x; Ws[r * kPad + c4 + 1] = wv[u].y; Ws[r * kPad + c4 + 2] = wv[u].z; Ws[r * kPad + c4 + 3] = wv[u].w;
    }
  }
  __syncthreads();
  invd[tid] = 1.0f / Us[tid * kBlk + tid];
  __syncthreads();

  float* wrow = Ws + tid * kPad;
  float* erow = Es + tid * kPad;
  GroupParams gp = {1.0f, 0.0f, 0.0f};
  double loss = 0.0;

#pragma unroll 1
  for (int sb = 0; sb < kBlk / kSub; ++sb) {
    const int cbase = sb * kSub;
    float w[kSub], err[kSub];
    uint32_t cw[BITS] = {};
#pragma unroll
    for (int k = 0; k < kSub; ++k) w[k] = wrow[cbase + k];
    uint2 srec[kSub];                                // static per-OC records of these 32 columns
    if (!is_ic && a.static_rec != nullptr) {
#pragma unroll
      for (int k = 0; k < kSub; ++k)
        srec[k] = a.static_rec[row * (a.in / G) + a.perm[a.i1 + cbase + k] / G];
    }

#pragma unroll
    for (int ii = 0; ii < kSub; ++ii) {
      const int i = cbase + ii;                      // column inside the block
      if (!is_ic && a.static_rec != nullptr) {       // per-OC, static groups: parameters fixed beforehand
        const uint2 rec = srec[ii];
        gp.rcp = __uint_as_float(rec.x);
        gp.s = __half2float(__ushort_as_half(static_cast<unsigned short>(rec.y & 0xffffu)));
        gp.z = __half2float(__ushort_as_half(static_cast<unsigned short>(rec.y >> 16)));
      } else if (!is_ic) {
        if ((ii % G) == 0 && (cbase % G) == 0) {     // per-OC: parameters at the group's first column
          float mn = w[ii], mx = w[ii];
          if (G == kSub) {
#pragma unroll
            for (int k = 1; k < kSub; ++k) { mn = fminf(mn, w[k]); mx = fmaxf(mx, w[k]); }
          } else {
            for (int k = 1; k < G; ++k) { float v = wrow[i + k]; mn = fminf(mn, v); mx = fmaxf(mx, v); }
          }
          gp = group_params(mn, mx, maxq, rcp_maxq);
          int64_t idx = row * (a.in / G) + (a.i1 + i) / G;
          q.scales[idx] = __half_as_ushort(__float2half_rn(gp.s));
          q.zeros[idx] = __half_as_ushort(__float2half_rn(gp.z));
        }
      } else {                                       // per-IC: parameters of this column's g-row groups
        // warp minimum and maximum in one reduction instruction each, on a key that orders
        // floats as signed integers (negative values have their magnitude bits flipped)
        const int key = ordered_key(w[ii]);
        float mn = from_ordered_key(__reduce_min_sync(0xffffffffu, key));
        float mx = from_ordered_key(__reduce_max_sync(0xffffffffu, key));
        if (G > 32) {
          float* slot = red + (ii & 1) * 8;
          if (lane == 0) { slot[warp * 2] = mn; slot[warp * 2 + 1] = mx; }
          __syncthreads();
          constexpr int WPG = G / 32;                // warps per group
          const int w0 = (warp / WPG) * WPG;
          mn = slot[w0 * 2]; mx = slot[w0 * 2 + 1];
#pragma unroll
          for (int k = 1; k < WPG; ++k) { mn = fminf(mn, slot[(w0 + k) * 2]); mx = fmaxf(mx, slot[(w0 + k) * 2 + 1]); }
        }
        gp = group_params(mn, mx, maxq, rcp_maxq);
        if ((tid % G) == 0) {
          Ss[(tid / G) * kBlk + i] = __half_as_ushort(__float2half_rn(gp.s));
          Zs[(tid / G) * kBlk + i] = __half_as_ushort(__float2half_rn(gp.z));
        }
      }
      const int c = code_of(quotient(w[ii], gp.s, gp.rcp), gp.z, maxq);
      const float qv = __fmul_rn(gp.s, static_cast<float>(c) - gp.z);
      const float e = (w[ii] - qv) * invd[i];
      err[ii] = e;
      erow[i] = e;
      loss += static_cast<double>(e) * static_cast<double>(e);
      {
        const int bit = ii * BITS, wi = bit >> 5, sh = bit & 31;
        cw[wi] |= static_cast<uint32_t>(c) << sh;
        if (sh + BITS > 32) cw[wi + 1] |= static_cast<uint32_t>(c) >> (32 - sh);
      }
      const float* urow = Us + i * kBlk + cbase;
#pragma unroll
      for (int jj = ii + 1; jj < kSub; ++jj) w[jj] = fmaf(-e, urow[jj], w[jj]);
    }
    // codes of these 32 columns: BITS whole words of this row's bitstream
    uint32_t* cdst = a.codes[d] + row * (a.in * BITS / 32) + static_cast<int64_t>(a.i1 + cbase) * BITS / 32;
#pragma unroll
    for (int k = 0; k < BITS; ++k) cdst[k] = cw[k];
    // lazy update of the block's later columns with this sub-block's 32 errors, as a small
    // register-tiled product over the whole slab (see lazy_update)
    __syncthreads();
    const int later = kBlk - cbase - kSub;
    if (later == 96) lazy_update<12>(Ws, Us, Es, cbase, tid);
    else if (later == 64) lazy_update<8>(Ws, Us, Es, cbase, tid);
    else if (later == 32) lazy_update<4>(Ws, Us, Es, cbase, tid);
    __syncthreads();
  }

  // ---- outputs: errors (coalesced), per-IC parameters, loss ------------------------------
  __syncthreads();
  // errors as three fixed-point bf16 pieces on one grid per row (see gptq_tc.cu)
  {
    float m = 0.0f;
    for (int k = 0; k < kBlk; ++k) m = fmaxf(m, fabsf(erow[k]));
    int ex = (__float_as_int(m) >> 23) & 0xFF;
    ex = ex < 32 ? 32 : (ex > 250 ? 250 : ex);
    invd[tid] = __int_as_float((ex - 7) << 23);     // grid of this row (invd is free now)
  }
  __syncthreads();
  const int64_t ebase = (static_cast<int64_t>(d) * a.out + row0) * kBlk;
  // thread tid takes column tid of every row r (e = 128 r + tid): a warp stores 64 contiguous bytes
#pragma unroll 8
  for (int r = 0; r < kBlk; ++r) {
    const float v = Es[r * kPad + tid];
    const float g = invd[r];
    const float inv = __int_as_float(0x7F000000 - __float_as_int(g));   // 1 / g for a power of two, exact
    const float a0 = rintf(v * inv);
    const float r1 = fmaf(-a0, g, v);
    const float a1 = rintf(r1 * inv * 256.0f);
    const float r2 = fmaf(-a1, g * (1.0f / 256.0f), r1);
    const float a2 = rintf(r2 * inv * 65536.0f);
    const int64_t e = ebase + static_cast<int64_t>(r) * kBlk + tid;
    a.Ep[0][e] = __float2bfloat16_rn(a0 * g);
    a.Ep[1][e] = __float2bfloat16_rn(a1 * g * (1.0f / 256.0f));
    a.Ep[2][e] = __float2bfloat16_rn(a2 * g * (1.0f / 65536.0f));
  }
  if (is_ic) {
    for (int e = tid; e < NG * kBlk; e += kBlk) {
      const int wc = a.i1 + (e % kBlk);               // working-copy column -> original column
      int64_t idx = (row0 / G + e / kBlk) * a.in + (a.perm != nullptr ? a.perm[wc] : wc);
      q.scales[idx] = Ss[e];
      q.zeros[idx] = Zs[e];
    }
  }
  __shared__ double lred[kBlk / 32];
  for (int m = 16; m > 0; m >>= 1) loss += __shfl_xor_sync(0xffffffffu, loss, m);
  if (lane == 0) lred[warp] = loss;
  __syncthreads();
  if (tid == 0) a.loss_part[static_cast<int64_t>(d) * (a.out / kBlk) + blockIdx.x] += (lred[0] + lred[1]) + (lred[2] + lred[3]);
}

__global__ void loss_kernel(const double* __restrict__ part, int ndim, int slabs, BlockArgs a, double* loss_out) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    loss_out[0] = 0.0; loss_out[1] = 0.0;
    for (int d = 0; d < ndim; ++d) {
      double s = 0.0;
      for (int k = 0; k < slabs; ++k) s += part[d * slabs + k];
      loss_out[a.dim_of[d]] = 0.5 * s;
    }
  }
}

constexpr size_t block_smem_bytes() {
  return (kBlk * kPad * 2 + kBlk * kBlk + kBlk + 16) * sizeof(float) + 2 * 4 * kBlk * sizeof(uint16_t);
}

template <int BITS, int G>
int block_launch(const BlockArgs& a, int slabs, int ndim, cudaStream_t st) {
  ADADIM_CUDA_TRY(cudaFuncSetAttribute(block_kernel<BITS, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(block_smem_bytes())));
  // launched so that it may be scheduled while the kernel before it in the stream finishes
  // (it waits for that kernel itself, after staging what does not depend on it)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(slabs, ndim);
  cfg.blockDim = dim3(kBlk);
  cfg.dynamicSmemBytes = block_smem_bytes();
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  ADADIM_CUDA_TRY(cudaLaunchKernelEx(&cfg, block_kernel<BITS, G>, a));
  return ADADIM_OK;
}

struct GptqLayout {
  size_t wc_off, err_off, err_piece, loss_off, up_off, up_piece, u_off, factor_off;
  size_t perm_off, rank_off, rec_off, tmp_off, tmp_piece, total;     // used by the reordered variant only
};
GptqLayout gptq_layout(int64_t out, int64_t in) {
  GptqLayout L;
  size_t off = 0;
  L.wc_off = off;     off += round_up(static_cast<size_t>(2) * out * in * 4, 256);
  L.err_piece = round_up(static_cast<size_t>(2) * 2 * out * kBlk * 2, 1024);      // two alternating sets
  L.err_off = off;    off += 3 * L.err_piece;
  L.up_piece = round_up(static_cast<size_t>(in) * in * 2, 1024);
  L.up_off = off;     off += 3 * L.up_piece;
  L.loss_off = off;   off += round_up(static_cast<size_t>(2) * (out / kBlk + 1) * 8, 256);
  L.u_off = off;      off += round_up(static_cast<size_t>(in) * in * 4, 256);
  L.factor_off = off; off += factor_workspace_bytes(in);
  L.perm_off = off;   off += round_up(static_cast<size_t>(in) * 4, 256);
  L.rank_off = off;   off += round_up(static_cast<size_t>(in) * 4, 256);
  L.rec_off = off;    off += round_up(static_cast<size_t>(out) * (in / 32) * 8, 256);     // g >= 32
  L.tmp_piece = round_up(static_cast<size_t>(out) * in / 2, 256);                          // bits <= 4
  L.tmp_off = off;    off += 2 * L.tmp_piece;
  L.total = off;
  return L;
}

}  // namespace

size_t gptq_workspace_bytes(int64_t out, int64_t in) { return gptq_layout(out, in).total; }

int gptq_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, const float* U_in,
                int bits, int group, int dim, float percdamp, const adadim_qtensor* q_oc, const adadim_qtensor* q_ic,
                double* gptq_loss, int* status_dev, void* workspace, cudaStream_t st, bool reorder, int* perm_out) {
  GptqLayout L = gptq_layout(out, in);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  BlockArgs a = {};
  a.Wc = reinterpret_cast<float*>(ws + L.wc_off);
  const __nv_bfloat16* ep[3];
  const __nv_bfloat16* up[3];
  for (int k = 0; k < 3; ++k) {
    a.Ep[k] = reinterpret_cast<__nv_bfloat16*>(ws + L.err_off + k * L.err_piece);
    ep[k] = a.Ep[k];
    up[k] = reinterpret_cast<__nv_bfloat16*>(ws + L.up_off + k * L.up_piece);
  }
  a.loss_part = reinterpret_cast<double*>(ws + L.loss_off);
  a.out = out;
  a.in = in;
  int ndim = 0;
  if (dim == ADADIM_DIM_OC || dim == ADADIM_DIM_BOTH) { a.q[ndim] = *q_oc; a.dim_of[ndim] = ADADIM_DIM_OC; ++ndim; }
  if (dim == ADADIM_DIM_IC || dim == ADADIM_DIM_BOTH) { a.q[ndim] = *q_ic; a.dim_of[ndim] = ADADIM_DIM_IC; ++ndim; }

  int* perm = nullptr;
  int* rank = nullptr;
  for (int d = 0; d < ndim; ++d) a.codes[d] = a.q[d].codes;
  if (reorder) {
    perm = reinterpret_cast<int*>(ws + L.perm_off);
    rank = reinterpret_cast<int*>(ws + L.rank_off);
    order_kernel<<<static_cast<unsigned>((in + 255) / 256), 256, 0, st>>>(H, in, perm, rank);
    if (perm_out != nullptr)
      ADADIM_CUDA_TRY(cudaMemcpyAsync(perm_out, perm, static_cast<size_t>(in) * 4, cudaMemcpyDeviceToDevice, st));
    a.perm = perm;
    for (int d = 0; d < ndim; ++d) a.codes[d] = reinterpret_cast<uint32_t*>(ws + L.tmp_off + d * L.tmp_piece);
    if (a.dim_of[0] == ADADIM_DIM_OC) {              // static groups for the per-OC copy (always copy 0)
      uint2* rec = reinterpret_cast<uint2*>(ws + L.rec_off);
      const unsigned sb = static_cast<unsigned>((out * (in / group) + 255) / 256);
      if (wdtype == ADADIM_F16) {
        if (bits == 3) static_params_kernel<__half, 3><<<sb, 256, 0, st>>>(static_cast<const __half*>(W), out, in, ldw, group, a.q[0], rec);
        else static_params_kernel<__half, 4><<<sb, 256, 0, st>>>(static_cast<const __half*>(W), out, in, ldw, group, a.q[0], rec);
      } else {
        if (bits == 3) static_params_kernel<float, 3><<<sb, 256, 0, st>>>(static_cast<const float*>(W), out, in, ldw, group, a.q[0], rec);
        else static_params_kernel<float, 4><<<sb, 256, 0, st>>>(static_cast<const float*>(W), out, in, ldw, group, a.q[0], rec);
      }
      a.static_rec = rec;
    }
  }

  const float* U = U_in;
  if (U == nullptr || reorder) {                     // a caller's factor belongs to the natural order
    float* Uw = reinterpret_cast<float*>(ws + L.u_off);
    int rc = factor_launch(H, in, percdamp, Uw, status_dev, ws + L.factor_off, st, perm);
    if (rc != ADADIM_OK) return rc;
    U = Uw;
  }
  a.U = U;
  int rc0 = trail_split_u(U, in, const_cast<__nv_bfloat16*>(up[0]), const_cast<__nv_bfloat16*>(up[1]),
                          const_cast<__nv_bfloat16*>(up[2]), st);
  if (rc0 != ADADIM_OK) return rc0;

  if (reorder) {
    const unsigned pb = static_cast<unsigned>((out * in + 255) / 256);
    if (wdtype == ADADIM_F16) init_perm_kernel<<<pb, 256, 0, st>>>(static_cast<const __half*>(W), out, in, ldw, H, perm, ndim, a.Wc);
    else init_perm_kernel<<<pb, 256, 0, st>>>(static_cast<const float*>(W), out, in, ldw, H, perm, ndim, a.Wc);
  } else {
    const unsigned ib = static_cast<unsigned>((out * in / 8 + 255) / 256);
    if (wdtype == ADADIM_F16) init_kernel<<<ib, 256, 0, st>>>(static_cast<const __half*>(W), out, in, ldw, H, ndim, a.Wc);
    else init_kernel<<<ib, 256, 0, st>>>(static_cast<const float*>(W), out, in, ldw, H, ndim, a.Wc);
  }
  ADADIM_CUDA_TRY(cudaMemsetAsync(a.loss_part, 0, static_cast<size_t>(2) * (out / kBlk + 1) * 8, st));

  const int slabs = static_cast<int>(out / kBlk);
  TrailPlan plan;
  rc0 = trail_plan(&plan, a.Wc, static_cast<int64_t>(ndim) * out, in, ep, up);
  if (rc0 != ADADIM_OK) return rc0;
  // Block b+1 only needs its own 128 columns from block b's trailing update.  That part runs on a
  // high-priority stream together with the block kernels; the rest of each trailing update runs
  // beside the next block kernel on a second stream, on the SMs the block kernel leaves free.  The
  // error pieces alternate between two sets, so a block kernel never overwrites what the other
  // stream still reads.
  cudaStream_t chain = nullptr, side = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_block = nullptr, ev_rest = nullptr, ev_join = nullptr;
  int prio_least = 0, prio_greatest = 0;
  ADADIM_CUDA_TRY(cudaDeviceGetStreamPriorityRange(&prio_least, &prio_greatest));
  ADADIM_CUDA_TRY(cudaStreamCreateWithPriority(&chain, cudaStreamNonBlocking, prio_greatest));
  ADADIM_CUDA_TRY(cudaStreamCreateWithPriority(&side, cudaStreamNonBlocking, prio_least));
  ADADIM_CUDA_TRY(cudaEventCreateWithFlags(&ev_fork, cudaEventDisableTiming));
  ADADIM_CUDA_TRY(cudaEventCreateWithFlags(&ev_block, cudaEventDisableTiming));
  ADADIM_CUDA_TRY(cudaEventCreateWithFlags(&ev_rest, cudaEventDisableTiming));
  ADADIM_CUDA_TRY(cudaEventCreateWithFlags(&ev_join, cudaEventDisableTiming));
  ADADIM_CUDA_TRY(cudaEventRecord(ev_fork, st));
  ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_fork, 0));
  const int64_t rows_total = static_cast<int64_t>(ndim) * out;
  // the side-stream launches get the SMs that the block kernel leaves free (finer CTAs were
  // measured slower: every CTA reloads its 96 KB of error pieces and refills the pipeline)
  const int free_sms = plan.sm_count - slabs * ndim;
  const int64_t mblocks = rows_total / kBlk;
  const int rest_split = free_sms >= mblocks ? static_cast<int>(free_sms / mblocks) : 1;
  __nv_bfloat16* ep_base[3] = {a.Ep[0], a.Ep[1], a.Ep[2]};
  bool rest_pending = false;
  for (int i1 = 0; i1 < in; i1 += kBlk) {
    a.i1 = i1;
    for (int k = 0; k < 3; ++k) a.Ep[k] = ep_base[k] + static_cast<int64_t>((i1 / kBlk) & 1) * rows_total * kBlk;
    int rc;
    if (bits == 3) {
      rc = group == 128 ? block_launch<3, 128>(a, slabs, ndim, chain) : group == 64 ? block_launch<3, 64>(a, slabs, ndim, chain)
                                                                                    : block_launch<3, 32>(a, slabs, ndim, chain);
    } else {
      rc = group == 128 ? block_launch<4, 128>(a, slabs, ndim, chain) : group == 64 ? block_launch<4, 64>(a, slabs, ndim, chain)
                                                                                    : block_launch<4, 32>(a, slabs, ndim, chain);
    }
    if (rc != ADADIM_OK) return rc;
    const int tiles_after = static_cast<int>((in - i1 - kBlk) / kBlk);
    if (tiles_after > 0) {
      if (tiles_after > 1) ADADIM_CUDA_TRY(cudaEventRecord(ev_block, chain));
      // the next block's columns were last written by the previous block's side-stream launch
      if (rest_pending) ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_rest, 0));
      rest_pending = false;
      rc = trail_launch(plan, i1, static_cast<int64_t>(i1) + kBlk, 1, 1, status_dev, chain);
      if (rc != ADADIM_OK) return rc;
      if (tiles_after > 1) {
        ADADIM_CUDA_TRY(cudaStreamWaitEvent(side, ev_block, 0));
        rc = trail_launch(plan, i1, static_cast<int64_t>(i1) + 2 * kBlk, tiles_after - 1,
                          (tiles_after - 1 + rest_split - 1) / rest_split, status_dev, side);
        if (rc != ADADIM_OK) return rc;
        ADADIM_CUDA_TRY(cudaEventRecord(ev_rest, side));
        rest_pending = true;
      }
    }
  }
  if (rest_pending) ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_rest, 0));
  ADADIM_CUDA_TRY(cudaEventRecord(ev_join, chain));
  ADADIM_CUDA_TRY(cudaStreamWaitEvent(st, ev_join, 0));
  // destruction is deferred by the runtime until the work already enqueued has finished
  cudaEventDestroy(ev_fork);
  cudaEventDestroy(ev_block);
  cudaEventDestroy(ev_rest);
  cudaEventDestroy(ev_join);
  cudaStreamDestroy(chain);
  cudaStreamDestroy(side);
  for (int k = 0; k < 3; ++k) a.Ep[k] = ep_base[k];
  if (reorder) {
    const unsigned ub = static_cast<unsigned>((out * (in / 32) + 255) / 256);
    for (int d = 0; d < ndim; ++d) {
      if (bits == 3) unpermute_codes_kernel<3><<<ub, 256, 0, st>>>(a.codes[d], rank, out, in, a.q[d].codes);
      else unpermute_codes_kernel<4><<<ub, 256, 0, st>>>(a.codes[d], rank, out, in, a.q[d].codes);
    }
  }
  if (gptq_loss != nullptr) loss_kernel<<<1, 32, 0, st>>>(a.loss_part, ndim, slabs, a, gptq_loss);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
