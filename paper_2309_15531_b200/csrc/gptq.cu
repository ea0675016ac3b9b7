// GPTQ with lazily batched error compensation (paper Section 2.2; Section 3.3: the per-IC
// variant changes only the quantization step).  Columns are handled in blocks of 128:
//   block kernel    - one CTA per 128-row slab and grouping dimension walks the block's
//                     columns in order: group parameters from the current weights, code,
//                     error e = (w - q) / U[i,i], and the update of the block's remaining
//                     columns, w[j] -= e U[i,j].  The slab lives in shared memory; the 32
//                     columns being worked on live in registers.
//   trailing update - W[:, after the block] -= Err[out,128] * U[block rows, after the block]
//                     on the tensor cores with exactly sliced bf16 operands (gptq_tc.cu).
// The working weights, the factor and every update inside a block are binary64: a weight is
// rounded thousands of columns after the first error was folded into it, and a binary32 copy
// re-rounded at every update drifts far enough (a few 1e-6 of a quantization step) to move
// individual rounding decisions, each of which then changes everything after it.  Only the
// decision itself (group parameters and the code of the weight as it stands, rounded once to
// binary32) is binary32 arithmetic, as the quantizer's definition says.
// Rows are independent under per-OC grouping; under per-IC grouping a group couples g
// consecutive rows of one column, which is why a CTA owns a whole 128-row slab.
#include <cuda.h>
#include <cuda_bf16.h>

#include "umma.cuh"

namespace adadim {

struct TrailPlan {
  CUtensorMap e[3], u[3];
  double* Wc;
  int64_t rows_total, in;
  int sm_count;
};
int trail_split_u(const double* U, int64_t in, __nv_bfloat16* u0, __nv_bfloat16* u1, __nv_bfloat16* u2, cudaStream_t st);
int trail_plan(TrailPlan* plan, double* Wc, int64_t rows_total, int64_t in, const __nv_bfloat16* const e[3],
               const __nv_bfloat16* const u[3]);
int trail_launch(const TrailPlan& plan, int i1, int64_t c0, int ntiles, int max_ctas, int* status_dev, cudaStream_t st);

size_t factor_workspace_bytes(int64_t n);
int factor_launch(const float* H, int64_t n, double percdamp, double* U, int* status_dev, void* workspace,
                  cudaStream_t st, const int* perm);

namespace {

constexpr int kBlk = 128;            // lazy-batch block width (columns) and slab height (rows)
constexpr int kSub = 32;             // columns held in registers at a time
constexpr int kLater = kBlk - kSub;  // columns of a block that are not in registers during its first sub-block
constexpr int kEP = kSub + 1;        // row pitch (doubles) of the current sub-block's errors
constexpr int kLaterTiles = (kBlk / kWcTileRows) * (kLater / kWcTileCols);       // 24 tiles of the working-weight layout
constexpr int kFirstTiles = (kBlk / kWcTileRows) * (kSub / kWcTileCols);         // 8 tiles

// The U block is upper triangular: row tile t (rows 32 t .. 32 t + 31) keeps columns 32 t .. 127
// only, with row pitch 128 - 32 t.
__host__ __device__ constexpr int u_tile_off(int t) { return 32 * (128 * t - 16 * t * (t - 1)); }
__host__ __device__ constexpr int u_tile_pitch(int t) { return kBlk - 32 * t; }
constexpr int kUPacked = u_tile_off(4);              // 10240 doubles

// A CTA fills a strip of 256 columns x kInitRows rows of every copy: lane = 8-column vector of the
// strip, warp = row lane.  The eight diagonal entries of H that tell dead columns are read once per
// thread and serve all its rows (they sit in eight different cache lines).
constexpr int kInitRows = 64;
template <typename T>
__global__ void __launch_bounds__(256)
init_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, const float* __restrict__ H, int ndim,
            double* __restrict__ Wc /* first of ndim consecutive copies of this layer */) {
  const int lane = threadIdx.x & 31, rl = threadIdx.x >> 5;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * 256 + lane * 8;
  if (i >= in) return;
  unsigned dead = 0;
#pragma unroll
  for (int k = 0; k < 8; ++k)
    if (H[(i + k) * in + (i + k)] == 0.0f) dead |= 1u << k;     // dead column
  const int64_t r0 = static_cast<int64_t>(blockIdx.y) * kInitRows;
#pragma unroll 2
  for (int t = rl; t < kInitRows; t += 8) {
    const int64_t o = r0 + t;
    if (o >= out) break;
    float v[8];
    load8(W + o * ldw + i, v);
#pragma unroll
    for (int k = 0; k < 8; ++k)
      if ((dead >> k) & 1u) v[k] = 0.0f;
    for (int d = 0; d < ndim; ++d) {
      double* dst = Wc + static_cast<int64_t>(d) * out * in;
#pragma unroll
      for (int k = 0; k < 4; ++k)          // four column pairs of one row of one tile
        *reinterpret_cast<double2*>(dst + wc_index(o, i + 2 * k, in)) =
            make_double2(static_cast<double>(v[2 * k]), static_cast<double>(v[2 * k + 1]));
    }
  }
}

// One working copy: one layer under one grouping dimension.  The copies of a call (several layers
// that share the Hessian, each in one or both dimensions) are stacked along the rows, so that one
// chain of block kernels and one chain of trailing updates serves them all.
constexpr int kMaxCopies = 16;
struct Copy {
  int64_t slab0;             // first 128-row slab of this copy in the stacked working weights
  int64_t out;               // rows of the layer
  adadim_qtensor q[2];       // the layer's per-OC and per-IC outputs (only the one in use is written)
  uint32_t* codes;           // where codes go instead of q[dim].codes (reordered variant: a temporary stream), or null
  const int* chosen;         // dim < 0: the grouping dimension is read from this device word
  double* loss;              // optional device double[2] of the layer: element [dim] receives 1/2 sum e^2
  const uint2* static_rec;   // per-OC static groups (reordered variant): [out][in/g] records
                             // {bits of 1/s (0: degenerate group), fp16 s | fp16 z << 16}, else null
  int dim;                   // ADADIM_DIM_OC, ADADIM_DIM_IC, or -1
};
struct BlockArgs {
  double* Wc;                // stacked working weights [rows][in] in the tiled layout of wc_index()
  const double* U;           // [in][in]
  int* status_dev;
  __nv_bfloat16* Ep[3];      // [rows][128] errors as three fixed-point bf16 pieces
  double* loss_part;         // [rows / 128]
  float* oc_rcp;             // [rows] g = 256 only: 1 / s of the row's current per-OC group, handed from the group's first block to its second
  int64_t in;
  int i1;                    // first column of the block
  // activation reordering (null in the natural order): column i of the working copy is column perm[i] of W
  const int* perm;
  int ncopies;
  Copy c[kMaxCopies];
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

// Working copies in the quantization order: element (o, i) of copy d = W[o][perm[i]] (0 for dead columns).
template <typename T>
__global__ void __launch_bounds__(256)
init_perm_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, const float* __restrict__ H,
                 const int* __restrict__ perm, int ndim, double* __restrict__ Wc) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= out * in) return;
  const int64_t o = e / in, c = perm[e % in];
  float v = static_cast<float>(W[o * ldw + c]);
  if (H[c * in + c] == 0.0f) v = 0.0f;
  for (int d = 0; d < ndim; ++d) Wc[static_cast<int64_t>(d) * out * in + wc_index(o, e % in, in)] = static_cast<double>(v);
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

// Position (in doubles) of element (r, lc) of the slab's later columns in shared memory: the 24
// tiles are kept as fetched, tile (r / 32, lc / 16) at slot (r / 32) * 6 + lc / 16.
__device__ __forceinline__ int later_at(int r, int lc) {
  return ((r >> 5) * (kLater / kWcTileCols) + (lc >> 4)) * kWcTileElems + wc_in_tile(r & 31, lc & 15);
}

// W[:, later columns] -= Err[:, this sub-block] * U[sub-block rows, later columns] for the whole
// 128-row slab in shared memory, in binary64.  A row-per-thread loop needs one warp-uniform U
// value per multiply-add, all of it through the shared-memory return path; here a thread owns
// 8 rows x CH columns at a time (two such column pieces), so 8 + CH loads feed 8 CH
// multiply-adds.  Every element receives its 32 updates in column order.
//   Wt  later columns of the slab (tiles, see later_at)
//   Ut  row tile of the packed U block that holds the sub-block's rows (pitch up)
//   Es  the sub-block's errors, Es[r * kEP + ii]
template <int CH>
__device__ __forceinline__ void lazy_update(double* __restrict__ Wt, const double* __restrict__ Ut, int up,
                                            const double* __restrict__ Es, int cbase, int tid) {
  const int r0 = (tid >> 3) * 8;
#pragma unroll 1
  for (int piece = 0; piece < 2; ++piece) {
    const int lc = ((tid & 7) * 2 + piece) * CH;     // first of this thread's columns among the later ones (even)
    double acc[8][CH];
    int at[CH / 2];                                  // position of row r0's column pairs; row r0 + m differs by a swizzle
#pragma unroll
    for (int n2 = 0; n2 < CH / 2; ++n2) at[n2] = later_at(r0, cbase + lc + 2 * n2);
#pragma unroll
    for (int m = 0; m < 8; ++m)
#pragma unroll
      for (int n2 = 0; n2 < CH / 2; ++n2) {
        // r0 is a multiple of 8, so row r0 + m has swizzle m: pair position p ^ m, 16 doubles further per row
        const double2 t = *reinterpret_cast<const double2*>(Wt + (at[n2] ^ (m << 1)) + m * 16);
        acc[m][2 * n2] = t.x; acc[m][2 * n2 + 1] = t.y;
      }
#pragma unroll 2
    for (int ii = 0; ii < kSub; ++ii) {
      double e[8], u[CH];
#pragma unroll
      for (int m = 0; m < 8; ++m) e[m] = Es[(r0 + m) * kEP + ii];
#pragma unroll
      for (int n2 = 0; n2 < CH / 2; ++n2) {
        const double2 t = *reinterpret_cast<const double2*>(Ut + ii * up + kSub + lc + 2 * n2);
        u[2 * n2] = t.x; u[2 * n2 + 1] = t.y;
      }
#pragma unroll
      for (int m = 0; m < 8; ++m)
#pragma unroll
        for (int n = 0; n < CH; ++n) acc[m][n] = fma(-e[m], u[n], acc[m][n]);
    }
#pragma unroll
    for (int m = 0; m < 8; ++m)
#pragma unroll
      for (int n2 = 0; n2 < CH / 2; ++n2)
        *reinterpret_cast<double2*>(Wt + (at[n2] ^ (m << 1)) + m * 16) = make_double2(acc[m][2 * n2], acc[m][2 * n2 + 1]);
  }
}

template <int BITS, int G>
__global__ void __launch_bounds__(kBlk, 1)
block_kernel(const BlockArgs a) {
  constexpr float maxq = static_cast<float>((1 << BITS) - 1);
  constexpr float rcp_maxq = 1.0f / maxq;            // correctly rounded at compile time
  constexpr int NG = G >= kBlk ? 1 : kBlk / G;       // per-IC groups in the slab (g = 256: half a group)
  extern __shared__ __align__(128) double smd[];
  double* Wt = smd;                                  // 24 tiles: columns 32..127 of the slab (later_at)
  double* Us = Wt + kLaterTiles * kWcTileElems;      // packed upper block-triangle of the U block
  double* Es = Us + kUPacked;                        // [128][33] errors of the current sub-block; first the
                                                     // landing zone of the 8 tiles of columns 0..31
  double* invd = Es + kBlk * kEP;                    // [128] 1 / U[i,i]
  float* gridr = reinterpret_cast<float*>(invd + kBlk);   // [128] slicing grid of every row's errors
  float* red = gridr + kBlk;                         // [2][4][2] per-IC min / max exchange
  uint16_t* Ss = reinterpret_cast<uint16_t*>(red + 16);   // [NG][128] per-IC scales (fp16 bits)
  uint16_t* Zs = Ss + NG * kBlk;                          // [NG][128]
  __shared__ uint64_t bar[2];
  __shared__ int dead_flag;
  __shared__ float xch[4];                           // g = 256: the neighbouring slab's per-IC minimum and maximum, two slots

  int ci = 0;                                        // the copy this slab belongs to
  while (ci + 1 < a.ncopies && static_cast<int64_t>(blockIdx.x) >= a.c[ci + 1].slab0) ++ci;
  const Copy& cp = a.c[ci];
  const int dim = cp.dim >= 0 ? cp.dim : *cp.chosen;
  const bool is_ic = dim == ADADIM_DIM_IC;
  const adadim_qtensor q = cp.q[is_ic ? 1 : 0];
  uint32_t* const codes = cp.codes != nullptr ? cp.codes : q.codes;
  const uint2* const static_rec = is_ic ? nullptr : cp.static_rec;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int64_t srow0 = static_cast<int64_t>(blockIdx.x) * kBlk;                 // in the stacked working weights
  const int64_t row0 = (static_cast<int64_t>(blockIdx.x) - cp.slab0) * kBlk;     // in the layer
  const int64_t row = row0 + tid;
  const double* Wd = a.Wc;

  // Staging by bulk copies: one memory latency for the U block and one for the slab.  The kernel
  // may have been scheduled while the launch before it in the stream (the update of this block's
  // columns) is still finishing: U does not depend on it and is fetched first; everything after
  // the wait sees that launch's results.
  if (tid == 0) {
    ptx::mbar_init(&bar[0], 1);
    ptx::mbar_init(&bar[1], 1);
    dead_flag = 0;
    ptx::fence_mbar_init();
    ptx::mbar_arrive_expect_tx(&bar[0], kUPacked * sizeof(double));
    ptx::mbar_arrive_expect_tx(&bar[1], (kLaterTiles + kFirstTiles) * kWcTileElems * sizeof(double));
  }
  __syncthreads();
  {
    // row tid of the U block: columns from the start of its 32-row tile to the end of the block
    const int t = tid >> 5, up = u_tile_pitch(t);
    ptx::bulk_load(Us + u_tile_off(t) + (tid & 31) * up, a.U + static_cast<int64_t>(a.i1 + tid) * a.in + a.i1 + 32 * t,
                   static_cast<uint32_t>(up * sizeof(double)), &bar[0]);
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid < kLaterTiles + kFirstTiles) {
    // tile tid of the slab: 4 tile rows x 8 tile columns; the first two tile columns land in Es
    const int tr = tid >> 3, tc = tid & 7;
    const double* src = Wd + ((srow0 / kWcTileRows + tr) * (a.in / kWcTileCols) + a.i1 / kWcTileCols + tc) * kWcTileElems;
    double* dst = tc < 2 ? Es + (tr * 2 + tc) * kWcTileElems : Wt + (tr * (kLater / kWcTileCols) + tc - 2) * kWcTileElems;
    ptx::bulk_load(dst, src, kWcTileElems * sizeof(double), &bar[1]);
  }
  const bool staged = ptx::mbar_wait(&bar[0], 0, &dead_flag, a.status_dev) &
                      ptx::mbar_wait(&bar[1], 0, &dead_flag, a.status_dev);
  bool go = __syncthreads_and(staged) != 0;
  if (G > kBlk) {
    // g = 256: the two CTAs of a pair meet at a cluster barrier in every per-IC column, so they go on
    // or stop together: each tells the other whether its copies arrived
    if (tid == 0) ptx::st_cluster_f32(ptx::map_to_cta(ptx::smem_addr(&xch[3]), ptx::cluster_ctarank() ^ 1u), go ? 1.0f : 0.0f);
    ptx::cluster_sync();
    go = go && xch[3] != 0.0f;
    ptx::cluster_sync();                             // both have read the word before a column's exchange could reuse the array
  }
  if (!go) {
    // a copy did not arrive in time (reported as ADADIM_ERR_TIMEOUT): give what is in flight one more
    // bounded wait so that nothing lands in shared memory after the CTA has gone, then stop
    const long long c0 = clock64();
    while (!(ptx::mbar_try_wait(&bar[0], 0) && ptx::mbar_try_wait(&bar[1], 0)) && clock64() - c0 < ptx::kWaitLimit) {}
    return;
  }
  invd[tid] = 1.0 / Us[u_tile_off(tid >> 5) + (tid & 31) * u_tile_pitch(tid >> 5) + (tid & 31)];

  double* erow = Es + tid * kEP;
  GroupParams gp = {1.0f, 0.0f, 0.0f};
  double loss = 0.0;
  float emax = 0.0f;

#pragma unroll 1
  for (int sb = 0; sb < kBlk / kSub; ++sb) {
    const int cbase = sb * kSub;
    const int up = u_tile_pitch(sb);
    const double* Ut = Us + u_tile_off(sb);
    double w[kSub];
    uint32_t cw[BITS] = {};
    if (sb == 0) {
      // this row's first 32 weights from the landing zone, which then becomes the error array
#pragma unroll
      for (int k2 = 0; k2 < kSub / 2; ++k2) {
        const double2 t = *reinterpret_cast<const double2*>(
            Es + ((tid >> 5) * 2 + (k2 >> 3)) * kWcTileElems + wc_in_tile(lane, 2 * (k2 & 7)));
        w[2 * k2] = t.x; w[2 * k2 + 1] = t.y;
      }
      __syncthreads();                               // every row has been read before the first error is written
    } else {
      // columns cbase .. cbase + 31 are later columns cbase - 32 ..; their slots are free from here
      // on and take the previous sub-block's errors, rounded to binary32, for the slicing at the end:
      // errors of sub-block j at later columns 32 j .. 32 j + 15 (two floats per slot)
      float4 ef[kSub / 4];
#pragma unroll
      for (int k = 0; k < kSub / 4; ++k)
        ef[k] = make_float4(static_cast<float>(erow[4 * k]), static_cast<float>(erow[4 * k + 1]),
                            static_cast<float>(erow[4 * k + 2]), static_cast<float>(erow[4 * k + 3]));
#pragma unroll
      for (int k2 = 0; k2 < kSub / 2; ++k2) {
        const double2 t = *reinterpret_cast<const double2*>(Wt + later_at(tid, cbase - kSub + 2 * k2));
        w[2 * k2] = t.x; w[2 * k2 + 1] = t.y;
      }
#pragma unroll
      for (int k = 0; k < kSub / 4; ++k)
        *reinterpret_cast<float4*>(Wt + later_at(tid, cbase - kSub + 2 * k)) = ef[k];
    }
    uint2 srec[kSub];                                // static per-OC records of these 32 columns
    if (static_rec != nullptr) {
#pragma unroll
      for (int k = 0; k < kSub; ++k)
        srec[k] = static_rec[row * (a.in / G) + a.perm[a.i1 + cbase + k] / G];
    }

#pragma unroll
    for (int ii = 0; ii < kSub; ++ii) {
      const int i = cbase + ii;                      // column inside the block
      const float w32 = static_cast<float>(w[ii]);   // the weight as it stands, rounded once: what is quantized
      if (static_rec != nullptr) {                   // per-OC, static groups: parameters fixed beforehand
        const uint2 rec = srec[ii];
        gp.rcp = __uint_as_float(rec.x);
        gp.s = __half2float(__ushort_as_half(static_cast<unsigned short>(rec.y & 0xffffu)));
        gp.z = __half2float(__ushort_as_half(static_cast<unsigned short>(rec.y >> 16)));
      } else if (!is_ic) {
        if ((ii % G) == 0 && ((a.i1 + cbase) % G) == 0) {     // per-OC: parameters at the group's first column
          float mn = w32, mx = w32;
#pragma unroll
          for (int k = 1; k < (G < kSub ? G : kSub); ++k) {
            const float v = static_cast<float>(w[ii + k < kSub ? ii + k : kSub - 1]);
            mn = fminf(mn, v); mx = fmaxf(mx, v);
          }
          for (int k = kSub; k < (G < kBlk ? G : kBlk); ++k) {    // the group's columns beyond the ones in registers
            const float v = static_cast<float>(Wt[later_at(tid, cbase + k - kSub)]);
            mn = fminf(mn, v); mx = fmaxf(mx, v);
          }
          if (G > kBlk) {
            // g = 256: the group's other 128 columns are the next block's, read where they stand in the
            // working weights (every update of earlier blocks has reached them: the host orders this
            // block kernel behind the side stream's launch at a group's first block)
            const double* nxt = a.Wc + ((srow0 + tid) >> 5) * (a.in >> 4) * kWcTileElems + ((a.i1 + kBlk) >> 4) * kWcTileElems;
#pragma unroll 4
            for (int k2 = 0; k2 < kBlk / 2; ++k2) {
              const double2 t = *reinterpret_cast<const double2*>(nxt + (k2 >> 3) * kWcTileElems + wc_in_tile(lane, 2 * (k2 & 7)));
              const float v0 = static_cast<float>(t.x), v1 = static_cast<float>(t.y);
              mn = fminf(mn, fminf(v0, v1)); mx = fmaxf(mx, fmaxf(v0, v1));
            }
          }
          gp = group_params(mn, mx, maxq, rcp_maxq);
          int64_t idx = row * (a.in / G) + (a.i1 + i) / G;
          q.scales[idx] = __half_as_ushort(__float2half_rn(gp.s));
          q.zeros[idx] = __half_as_ushort(__float2half_rn(gp.z));
          if (G > kBlk) a.oc_rcp[srow0 + tid] = gp.rcp;
        } else if (G > kBlk && i == 0) {
          // g = 256, the group's second block: the parameters its first block took
          const int64_t idx = row * (a.in / G) + a.i1 / G;
          gp.s = __half2float(__ushort_as_half(q.scales[idx]));
          gp.z = __half2float(__ushort_as_half(q.zeros[idx]));
          gp.rcp = a.oc_rcp[srow0 + tid];
        }
      } else {                                       // per-IC: parameters of this column's g-row groups
        // warp minimum and maximum in one reduction instruction each, on a key that orders
        // floats as signed integers (negative values have their magnitude bits flipped)
        const int key = ordered_key(w32);
        float mn = from_ordered_key(__reduce_min_sync(0xffffffffu, key));
        float mx = from_ordered_key(__reduce_max_sync(0xffffffffu, key));
        if (G > 32) {
          float* slot = red + (ii & 1) * 8;
          if (lane == 0) { slot[warp * 2] = mn; slot[warp * 2 + 1] = mx; }
          __syncthreads();
          constexpr int WPG = (G < kBlk ? G : kBlk) / 32;     // warps per group (g = 256: all four, half a group)
          const int w0 = (warp / WPG) * WPG;
          mn = slot[w0 * 2]; mx = slot[w0 * 2 + 1];
#pragma unroll
          for (int k = 1; k < WPG; ++k) { mn = fminf(mn, slot[(w0 + k) * 2]); mx = fmaxf(mx, slot[(w0 + k) * 2 + 1]); }
        }
        if (G > kBlk) {
          // g = 256: a group spans this slab and its neighbour, which the other CTA of the pair (a
          // cluster of two) holds.  Each writes its minimum and maximum into the other's shared memory;
          // the cluster barrier orders the writes before the reads.  Slots alternate with the column: a
          // CTA can reach its write for column ii + 2 only after the other has passed the barrier of
          // column ii + 1, i.e. after it has read the slot of column ii.
          float* mine = xch + (ii & 1) * 2;
          if (tid == 0) {
            const uint32_t remote = ptx::map_to_cta(ptx::smem_addr(mine), ptx::cluster_ctarank() ^ 1u);
            ptx::st_cluster_f32(remote, mn);
            ptx::st_cluster_f32(remote + 4, mx);
          }
          ptx::cluster_sync();
          mn = fminf(mn, mine[0]);
          mx = fmaxf(mx, mine[1]);
        }
        gp = group_params(mn, mx, maxq, rcp_maxq);
        if ((tid % G) == 0) {
          Ss[(tid / G) * kBlk + i] = __half_as_ushort(__float2half_rn(gp.s));
          Zs[(tid / G) * kBlk + i] = __half_as_ushort(__float2half_rn(gp.z));
        }
      }
      const int c = code_of(quotient(w32, gp.s, gp.rcp), gp.z, maxq);
      const float qv = __fmul_rn(gp.s, static_cast<float>(c) - gp.z);
      const double e = (w[ii] - static_cast<double>(qv)) * invd[i];
      erow[ii] = e;
      emax = fmaxf(emax, fabsf(static_cast<float>(e)));
      loss = fma(e, e, loss);
      {
        const int bit = ii * BITS, wi = bit >> 5, sh = bit & 31;
        cw[wi] |= static_cast<uint32_t>(c) << sh;
        if (sh + BITS > 32) cw[wi + 1] |= static_cast<uint32_t>(c) >> (32 - sh);
      }
      const double* urow = Ut + ii * up;
#pragma unroll
      for (int jj = ii + 1; jj < kSub; ++jj) w[jj] = fma(-e, urow[jj], w[jj]);
    }
    // codes of these 32 columns: BITS whole words of this row's bitstream
    uint32_t* cdst = codes + row * (a.in * BITS / 32) + static_cast<int64_t>(a.i1 + cbase) * BITS / 32;
#pragma unroll
    for (int k = 0; k < BITS; ++k) cdst[k] = cw[k];
    // lazy update of the block's later columns with this sub-block's 32 errors, as a small
    // register-tiled product over the whole slab (see lazy_update)
    __syncthreads();
    if (sb == 0) lazy_update<6>(Wt, Ut, up, Es, cbase, tid);
    else if (sb == 1) lazy_update<4>(Wt, Ut, up, Es, cbase, tid);
    else if (sb == 2) lazy_update<2>(Wt, Ut, up, Es, cbase, tid);
    __syncthreads();
  }

  // ---- outputs: errors (coalesced), per-IC parameters, loss ------------------------------
  // errors as three fixed-point bf16 pieces on one grid per row (see gptq_tc.cu).  The binary32
  // errors of sub-blocks 0..2 already sit in the slab's free slots; those of the last one follow.
#pragma unroll
  for (int k = 0; k < kSub / 4; ++k)
    *reinterpret_cast<float4*>(Wt + later_at(tid, kLater - kSub / 2 + 2 * k)) =
        make_float4(static_cast<float>(erow[4 * k]), static_cast<float>(erow[4 * k + 1]),
                    static_cast<float>(erow[4 * k + 2]), static_cast<float>(erow[4 * k + 3]));
  {
    int ex = (__float_as_int(emax) >> 23) & 0xFF;
    ex = ex < 32 ? 32 : (ex > 250 ? 250 : ex);
    gridr[tid] = __int_as_float((ex - 7) << 23);     // grid of this row
  }
  __syncthreads();
  const int64_t ebase = srow0 * kBlk;
  // thread tid takes column tid of every row r (e = 128 r + tid): a warp stores 64 contiguous bytes.
  // Column tid = 32 j + k: float k of the 16 slots that hold sub-block j's errors.
  const int eslot = (warp < 3 ? kSub * warp : kLater - kSub / 2) + (lane >> 1);
#pragma unroll 8
  for (int r = 0; r < kBlk; ++r) {
    const float v = reinterpret_cast<const float*>(Wt + later_at(r, eslot))[lane & 1];
    const float g = gridr[r];
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
  if (tid == 0) a.loss_part[blockIdx.x] += (lred[0] + lred[1]) + (lred[2] + lred[3]);
}

// 1/2 sum e^2 of every copy into its layer's loss[dim], the slabs' partial sums in a fixed order.
__global__ void loss_kernel(const BlockArgs a) {
  const int ci = threadIdx.x;
  if (ci >= a.ncopies || a.c[ci].loss == nullptr) return;
  const Copy& cp = a.c[ci];
  const int dim = cp.dim >= 0 ? cp.dim : *cp.chosen;
  double s = 0.0;
  for (int64_t k = 0; k < cp.out / kBlk; ++k) s += a.loss_part[cp.slab0 + k];
  cp.loss[dim == ADADIM_DIM_IC ? 1 : 0] = 0.5 * s;
}

constexpr size_t block_smem_bytes() {
  return (kLaterTiles * kWcTileElems + kUPacked + kBlk * kEP + kBlk) * sizeof(double) + (kBlk + 16) * sizeof(float) +
         2 * 4 * kBlk * sizeof(uint16_t);
}

template <int BITS, int G>
int block_launch(const BlockArgs& a, int slabs, cudaStream_t st) {
  ADADIM_CUDA_TRY(cudaFuncSetAttribute(block_kernel<BITS, G>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(block_smem_bytes())));
  // launched so that it may be scheduled while the kernel before it in the stream finishes
  // (it waits for that kernel itself, after staging what does not depend on it)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(slabs);
  cfg.blockDim = dim3(kBlk);
  cfg.dynamicSmemBytes = block_smem_bytes();
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  if (G > kBlk) {                                    // pairs of slabs exchange per-IC statistics: clusters of two CTAs
    attr[1].id = cudaLaunchAttributeClusterDimension;
    attr[1].val.clusterDim.x = 2;
    attr[1].val.clusterDim.y = 1;
    attr[1].val.clusterDim.z = 1;
    cfg.numAttrs = 2;
  }
  ADADIM_CUDA_TRY(cudaLaunchKernelEx(&cfg, block_kernel<BITS, G>, a));
  return ADADIM_OK;
}

struct GptqLayout {
  size_t wc_off, err_off, err_piece, loss_off, rcp_off, up_off, up_piece, u_off, factor_off;
  size_t perm_off, rank_off, rec_off, tmp_off, total;      // the last four: the reordered variant only
};
// rows: all working copies stacked (a layer quantized in both dimensions counts twice)
GptqLayout gptq_layout(int64_t rows, int64_t in) {
  GptqLayout L;
  size_t off = 0;
  L.wc_off = off;     off += round_up(static_cast<size_t>(rows) * in * 8, 256);
  L.err_piece = round_up(static_cast<size_t>(2) * rows * kBlk * 2, 1024);         // two alternating sets
  L.err_off = off;    off += 3 * L.err_piece;
  L.up_piece = round_up(static_cast<size_t>(in) * in * 2, 1024);
  L.up_off = off;     off += 3 * L.up_piece;
  L.loss_off = off;   off += round_up(static_cast<size_t>(rows / kBlk + 2) * 8, 256);
  L.rcp_off = off;    off += round_up(static_cast<size_t>(rows) * 4, 256);
  L.u_off = off;      off += round_up(static_cast<size_t>(in) * in * 8, 256);
  L.factor_off = off; off += factor_workspace_bytes(in);
  L.perm_off = off;   off += round_up(static_cast<size_t>(in) * 4, 256);
  L.rank_off = off;   off += round_up(static_cast<size_t>(in) * 4, 256);
  L.rec_off = off;    off += round_up(static_cast<size_t>(rows) * (in / 32) * 8, 256);    // g >= 32
  L.tmp_off = off;    off += round_up(static_cast<size_t>(rows) * in, 256);               // bits <= 8
  L.total = off;
  return L;
}

template <typename T>
void static_params_launch(const T* W, int64_t out, int64_t in, int64_t ldw, int bits, int group, adadim_qtensor q, uint2* rec,
                          unsigned blocks, cudaStream_t st) {
  if (bits == 2) static_params_kernel<T, 2><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, q, rec);
  else if (bits == 3) static_params_kernel<T, 3><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, q, rec);
  else if (bits == 4) static_params_kernel<T, 4><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, q, rec);
  else static_params_kernel<T, 8><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, q, rec);
}

template <int BITS>
int block_launch_g(const BlockArgs& a, int group, int slabs, cudaStream_t st) {
  return group == 256 ? block_launch<BITS, 256>(a, slabs, st)
       : group == 128 ? block_launch<BITS, 128>(a, slabs, st)
       : group == 64  ? block_launch<BITS, 64>(a, slabs, st)
                      : block_launch<BITS, 32>(a, slabs, st);
}

}  // namespace

size_t gptq_workspace_bytes(int64_t rows, int64_t in) { return gptq_layout(rows, in).total; }

// One layer of a call, as the launcher sees it.
struct GptqLayer {
  const void* W;
  int64_t out, ldw;
  const adadim_qtensor* q_oc;
  const adadim_qtensor* q_ic;
  int dim;                   // ADADIM_DIM_OC / IC / BOTH / CHOSEN
  const int* chosen;         // device word, for ADADIM_DIM_CHOSEN
  double* loss;              // optional device double[2]
};

int gptq_launch(const GptqLayer* layers, int n_layers, int wdtype, int64_t in, const float* H, const double* U_in,
                int bits, int group, double percdamp, int* status_dev, void* workspace, cudaStream_t st, bool reorder,
                int* perm_out) {
  // the working copies, stacked in layer order
  BlockArgs a = {};
  int64_t rows = 0;
  for (int l = 0; l < n_layers; ++l) {
    const GptqLayer& y = layers[l];
    const int dims[2] = {y.dim == ADADIM_DIM_BOTH ? ADADIM_DIM_OC : y.dim == ADADIM_DIM_CHOSEN ? -1 : y.dim,
                         ADADIM_DIM_IC};
    const int nd = y.dim == ADADIM_DIM_BOTH ? 2 : 1;
    for (int d = 0; d < nd; ++d) {
      if (a.ncopies == kMaxCopies) return ADADIM_ERR_PARAM;
      Copy& c = a.c[a.ncopies++];
      c.slab0 = rows / kBlk;
      c.out = y.out;
      if (y.q_oc != nullptr) c.q[0] = *y.q_oc;
      if (y.q_ic != nullptr) c.q[1] = *y.q_ic;
      c.dim = dims[d];
      c.chosen = y.chosen;
      c.loss = y.loss;
      rows += y.out;
    }
  }
  GptqLayout L = gptq_layout(rows, in);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  a.Wc = reinterpret_cast<double*>(ws + L.wc_off);
  a.status_dev = status_dev;
  const __nv_bfloat16* ep[3];
  const __nv_bfloat16* up[3];
  for (int k = 0; k < 3; ++k) {
    a.Ep[k] = reinterpret_cast<__nv_bfloat16*>(ws + L.err_off + k * L.err_piece);
    ep[k] = a.Ep[k];
    up[k] = reinterpret_cast<__nv_bfloat16*>(ws + L.up_off + k * L.up_piece);
  }
  a.loss_part = reinterpret_cast<double*>(ws + L.loss_off);
  a.oc_rcp = reinterpret_cast<float*>(ws + L.rcp_off);
  a.in = in;

  int* perm = nullptr;
  int* rank = nullptr;
  if (reorder) {                                     // one layer, checked by the caller
    const GptqLayer& y = layers[0];
    perm = reinterpret_cast<int*>(ws + L.perm_off);
    rank = reinterpret_cast<int*>(ws + L.rank_off);
    order_kernel<<<static_cast<unsigned>((in + 255) / 256), 256, 0, st>>>(H, in, perm, rank);
    if (perm_out != nullptr)
      ADADIM_CUDA_TRY(cudaMemcpyAsync(perm_out, perm, static_cast<size_t>(in) * 4, cudaMemcpyDeviceToDevice, st));
    a.perm = perm;
    for (int d = 0; d < a.ncopies; ++d)
      a.c[d].codes = reinterpret_cast<uint32_t*>(ws + L.tmp_off + static_cast<size_t>(d) * round_up(static_cast<size_t>(y.out) * in, 256));
    if (a.c[0].dim == ADADIM_DIM_OC) {               // static groups for the per-OC copy (always copy 0)
      uint2* rec = reinterpret_cast<uint2*>(ws + L.rec_off);
      const unsigned sb = static_cast<unsigned>((y.out * (in / group) + 255) / 256);
      if (wdtype == ADADIM_F16) static_params_launch(static_cast<const __half*>(y.W), y.out, in, y.ldw, bits, group, a.c[0].q[0], rec, sb, st);
      else static_params_launch(static_cast<const float*>(y.W), y.out, in, y.ldw, bits, group, a.c[0].q[0], rec, sb, st);
      a.c[0].static_rec = rec;
    }
  }

  const double* U = U_in;
  if (U == nullptr || reorder) {                     // a caller's factor belongs to the natural order
    double* Uw = reinterpret_cast<double*>(ws + L.u_off);
    int rc = factor_launch(H, in, percdamp, Uw, status_dev, ws + L.factor_off, st, perm);
    if (rc != ADADIM_OK) return rc;
    U = Uw;
  }
  a.U = U;
  int rc0 = trail_split_u(U, in, const_cast<__nv_bfloat16*>(up[0]), const_cast<__nv_bfloat16*>(up[1]),
                          const_cast<__nv_bfloat16*>(up[2]), st);
  if (rc0 != ADADIM_OK) return rc0;

  {
    int ci = 0;
    for (int l = 0; l < n_layers; ++l) {
      const GptqLayer& y = layers[l];
      const int nd = y.dim == ADADIM_DIM_BOTH ? 2 : 1;
      double* dst = a.Wc + a.c[ci].slab0 * kBlk * in;
      if (reorder) {
        const unsigned pb = static_cast<unsigned>((y.out * in + 255) / 256);
        if (wdtype == ADADIM_F16) init_perm_kernel<<<pb, 256, 0, st>>>(static_cast<const __half*>(y.W), y.out, in, y.ldw, H, perm, nd, dst);
        else init_perm_kernel<<<pb, 256, 0, st>>>(static_cast<const float*>(y.W), y.out, in, y.ldw, H, perm, nd, dst);
      } else {
        const dim3 ib(static_cast<unsigned>((in + 255) / 256), static_cast<unsigned>((y.out + kInitRows - 1) / kInitRows));
        if (wdtype == ADADIM_F16) init_kernel<<<ib, 256, 0, st>>>(static_cast<const __half*>(y.W), y.out, in, y.ldw, H, nd, dst);
        else init_kernel<<<ib, 256, 0, st>>>(static_cast<const float*>(y.W), y.out, in, y.ldw, H, nd, dst);
      }
      ci += nd;
    }
  }
  const int slabs = static_cast<int>(rows / kBlk);
  ADADIM_CUDA_TRY(cudaMemsetAsync(a.loss_part, 0, static_cast<size_t>(slabs + 2) * 8, st));

  TrailPlan plan;
  rc0 = trail_plan(&plan, a.Wc, rows, in, ep, up);
  if (rc0 != ADADIM_OK) return rc0;
  // Block b+1 only needs its own 128 columns from block b's trailing update.  That part runs on a
  // high-priority stream together with the block kernels; the rest of each trailing update runs
  // beside the next block kernel on a second stream, on the SMs the block kernel leaves free.  The
  // error pieces alternate between two sets, so a block kernel never overwrites what the other
  // stream still reads.
  {
    ForkedStreams fs;                                // joins and releases on every way out of this scope
    rc0 = fs.open(st);
    if (rc0 != ADADIM_OK) return rc0;
    cudaStream_t chain = fs.chain, side = fs.side;
    cudaEvent_t ev_block = fs.ev_a, ev_rest = fs.ev_b;
    // the side-stream launches get the SMs that the block kernel leaves free: one CTA on each, the
    // launch's tiles dealt out evenly among them; the chain's launch gets the SMs the block kernel
    // has just left
    const int free_sms = plan.sm_count - slabs % plan.sm_count;
    const int chain_sms = slabs < plan.sm_count ? slabs : plan.sm_count;
    __nv_bfloat16* ep_base[3] = {a.Ep[0], a.Ep[1], a.Ep[2]};
    bool rest_pending = false;
    for (int i1 = 0; i1 < in; i1 += kBlk) {
      a.i1 = i1;
      for (int k = 0; k < 3; ++k) a.Ep[k] = ep_base[k] + static_cast<int64_t>((i1 / kBlk) & 1) * rows * kBlk;
      if (group > kBlk && i1 % group == 0 && rest_pending) {
        // g = 256: per-OC statistics at a group's first block also read the NEXT block's columns, which
        // the side stream's launch of the block before last wrote
        ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_rest, 0));
        rest_pending = false;
      }
      int rc = bits == 2 ? block_launch_g<2>(a, group, slabs, chain) : bits == 3 ? block_launch_g<3>(a, group, slabs, chain)
             : bits == 4 ? block_launch_g<4>(a, group, slabs, chain) : block_launch_g<8>(a, group, slabs, chain);
      if (rc != ADADIM_OK) return rc;
      const int tiles_after = static_cast<int>((in - i1 - kBlk) / kBlk);
      if (tiles_after > 0) {
        if (tiles_after > 1) ADADIM_CUDA_TRY(cudaEventRecord(ev_block, chain));
        // the next block's columns were last written by the previous block's side-stream launch
        if (rest_pending) ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_rest, 0));
        rest_pending = false;
        rc = trail_launch(plan, i1, static_cast<int64_t>(i1) + kBlk, 1, chain_sms, status_dev, chain);
        if (rc != ADADIM_OK) return rc;
        if (tiles_after > 1) {
          ADADIM_CUDA_TRY(cudaStreamWaitEvent(side, ev_block, 0));
          // On the free SMs alone the launch runs beside the next block kernel.  Where the block kernel
          // leaves fewer than half of the SMs (128 slabs on 148 SMs: 20), the launch gets all of them
          // instead and the two alternate (8192 x 28672 in both dimensions: 748 ms on the 20 free SMs,
          // 187 ms on all; 64 slabs x 11008 columns: 15.3 ms on the 84 free SMs, 16.1 ms on all).
          const bool all = 2 * free_sms < plan.sm_count;
          rc = trail_launch(plan, i1, static_cast<int64_t>(i1) + 2 * kBlk, tiles_after - 1, all ? plan.sm_count : free_sms, status_dev, side);
          if (rc != ADADIM_OK) return rc;
          ADADIM_CUDA_TRY(cudaEventRecord(ev_rest, side));
          rest_pending = true;
        }
      }
    }
    for (int k = 0; k < 3; ++k) a.Ep[k] = ep_base[k];
    rc0 = fs.join();
    if (rc0 != ADADIM_OK) return rc0;
  }
  if (reorder) {
    const int64_t out = layers[0].out;
    const unsigned ub = static_cast<unsigned>((out * (in / 32) + 255) / 256);
    for (int d = 0; d < a.ncopies; ++d) {
      const adadim_qtensor& q = a.c[d].q[a.c[d].dim == ADADIM_DIM_IC ? 1 : 0];
      if (bits == 2) unpermute_codes_kernel<2><<<ub, 256, 0, st>>>(a.c[d].codes, rank, out, in, q.codes);
      else if (bits == 3) unpermute_codes_kernel<3><<<ub, 256, 0, st>>>(a.c[d].codes, rank, out, in, q.codes);
      else if (bits == 4) unpermute_codes_kernel<4><<<ub, 256, 0, st>>>(a.c[d].codes, rank, out, in, q.codes);
      else unpermute_codes_kernel<8><<<ub, 256, 0, st>>>(a.c[d].codes, rank, out, in, q.codes);
    }
  }
  loss_kernel<<<1, 32, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
