// Damped Cholesky-inverse factor for GPTQ (paper Section 2.2 cites the algorithm; the damping
// and the factor are the published algorithm's):  Hd = H + lambda I,  Hd^-1 = U^T U,  U upper.
//
// Route: with P the index reversal, factor A = P Hd P = L L^T (L lower) and invert the
// triangle; then U = P L^-1 P, because Hd = (P L P)(P L P)^T with P L P upper triangular and
// Hd^-1 = (P L^-1 P)^T (P L^-1 P).  This needs one factorization and one triangular inverse
// instead of a factorization, a full inverse and a second factorization.  All arithmetic is
// binary64, the large products on the fp64 matrix instruction (the factor decides GPTQ's rounding, so it is kept well inside
// the fp32 precision of U); U is returned in binary64 as well.
//
//   factorization : 64-column panels (diagonal block on one CTA, then the panel below it
//                   multiplied by the inverted diagonal block).  Panels are grouped four at a
//                   time: inside a group only the group's own columns are updated after each
//                   panel; the rest of the matrix gets one rank-256 update per group, on
//                   128 x 64 tiles.
//   inverse       : recursive doubling.  inv([[A,0],[C,B]]) = [[A^-1,0],[-B^-1 C A^-1,B^-1]]:
//                   level by level, adjacent inverted diagonal blocks are merged with two
//                   batched triangular-aware matrix products, log2(n/64) levels in all.
// The strict upper triangle of the work matrix is kept at zero outside 64-blocks on the
// diagonal, so whole diagonal tiles can be used as triangular operands.
#include "common.cuh"

namespace adadim {
namespace {

constexpr int kNB = 64;     // panel width and small tile edge
constexpr int kGroup = 4;   // panels per rank-256 update

__host__ __device__ __forceinline__ int64_t mn64(int64_t a, int64_t b) { return a < b ? a : b; }
__host__ __device__ __forceinline__ int64_t mx64(int64_t a, int64_t b) { return a > b ? a : b; }

// Programmatic dependent launch for the chain of small kernels: a kernel launched with the
// attribute below may be scheduled while its predecessor in the stream is still finishing; it then
// waits here until that predecessor has completed and its writes are visible.  dep_release() lets
// the successor of the calling kernel be scheduled early in the same way.  Both are no-ops for a
// kernel launched the ordinary way.
__device__ __forceinline__ void dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void dep_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
cudaError_t launch_chained(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// D += A B on 8 x 8 x 4 fp64 fragments: lane l holds A[l/4][l%4], B[l%4][l/4] and the two
// outputs D[l/4][2 (l%4)], D[l/4][2 (l%4) + 1].
__device__ __forceinline__ void mma_f64(double (&c)[2], double a, double b) {
  asm volatile("mma.sync.aligned.m8n8k4.row.col.f64.f64.f64.f64 {%0,%1}, {%2}, {%3}, {%0,%1};"
               : "+d"(c[0]), "+d"(c[1]) : "d"(a), "d"(b));
}

// ---- 64 x 64 output tile product (K = 64) on the fp64 matrix instruction, 256 threads ---------
// acc += A[64 x 64] * B, A row-major with leading dimension lda;
// B_T: B is given as [64 cols][64] row-major (product with the transpose), else as [64][64 cols].
// Each of the eight warps owns 32 rows x 16 columns as 4 x 2 fragments.  These tiles sit on the
// factorization's critical chain, so every global load of both operands is issued before the
// first one is used (one memory latency per tile), and the operands are staged in two K-halves.
// The row pitch is 4 mod 16 doubles: 64-bit shared-memory accesses are served a half-warp at a
// time, and a half-warp's fragment load (4 k-rows x 4 columns) then falls on 16 distinct banks;
// the loaders put consecutive lanes on consecutive rows, so their transposing stores do too.
constexpr int kHalfK = kNB / 2;
#define TILE_SMEM                           \
  __shared__ double sa[kHalfK][kNB + 4];    \
  __shared__ double sb[kHalfK][kNB + 4];

template <bool B_T>
__device__ __forceinline__ void tile_product(const double* __restrict__ A, int64_t lda, const double* __restrict__ B,
                                             int64_t ldb, double (&acc)[4][2][2], double (*sa)[kNB + 4],
                                             double (*sb)[kNB + 4]) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 1) * 32, wn = (warp >> 1) * 16;
  const int fk = lane & 3, fr = lane >> 2;
  const int r = tid & 63, kq = (tid >> 6) * 8;           // loader: row (or column of B^T), first k of eight
  const int kk = tid >> 3, nc = tid & 7;                 // loader of a non-transposed B: k row, 16-byte chunks nc + 8 t
  double2 av[2][4], bv[2][4];
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    const double2* asrc = reinterpret_cast<const double2*>(A + static_cast<int64_t>(r) * lda + h * kHalfK + kq);
    const double2* bsrc = B_T ? reinterpret_cast<const double2*>(B + static_cast<int64_t>(r) * ldb + h * kHalfK + kq)
                              : reinterpret_cast<const double2*>(B + static_cast<int64_t>(h * kHalfK + kk) * ldb) + nc;
#pragma unroll
    for (int t = 0; t < 4; ++t) { av[h][t] = asrc[t]; bv[h][t] = bsrc[B_T ? t : 8 * t]; }
  }
#pragma unroll
  for (int h = 0; h < 2; ++h) {
    if (h > 0) __syncthreads();                          // the first half has been consumed
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      sa[kq + 2 * t][r] = av[h][t].x; sa[kq + 2 * t + 1][r] = av[h][t].y;
      if (B_T) { sb[kq + 2 * t][r] = bv[h][t].x; sb[kq + 2 * t + 1][r] = bv[h][t].y; }
      else *reinterpret_cast<double2*>(&sb[kk][2 * (nc + 8 * t)]) = bv[h][t];
    }
    __syncthreads();
#pragma unroll
    for (int ks = 0; ks < kHalfK; ks += 4) {
      double af[4], bf[2];
#pragma unroll
      for (int i = 0; i < 4; ++i) af[i] = sa[ks + fk][wm + 8 * i + fr];
#pragma unroll
      for (int j = 0; j < 2; ++j) bf[j] = sb[ks + fk][wn + 8 * j + fr];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) mma_f64(acc[i][j], af[i], bf[j]);
    }
  }
}

// Applies f(row, first column, values of 2 consecutive columns) to a thread's outputs of the tile.
template <typename F>
__device__ __forceinline__ void for_each_pair64(double (&acc)[4][2][2], F f) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wm = (warp & 1) * 32, wn = (warp >> 1) * 16;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 2; ++j) f(wm + 8 * i + (lane >> 2), wn + 8 * j + 2 * (lane & 3), acc[i][j]);
}

// ---- 128 x 64 output tile product on the fp64 tensor-core path, 256 threads ----------------
// Each of the eight warps owns a 32 x 32 piece of the tile as 4 x 4 fragments of the 8 x 8 x 4
// fp64 matrix instruction (full fp64 multiply-add rate with an eighth of the instruction issue and
// a fraction of the shared-memory traffic of scalar multiply-adds, which were bound by shared-memory
// bandwidth here).  Rows >= a_rows (64 or 128) of A are not read (treated as zero).  K is a
// multiple of 8.  Shared-memory slabs are double-buffered; the slab after the next one is already
// on its way from global memory into registers while the current one is multiplied, and two CTAs
// share an SM, so global latency is covered.  The row pitches are 4 mod 16 doubles and the
// loaders put consecutive lanes on consecutive rows (see tile_product): no bank conflicts.
constexpr int kT = 128, kTN = 64, kBK = 8;
struct TileSmem {
  double a[2][kBK][kT + 4];
  double b[2][kBK][kTN + 4];
};

// acc[i][j] is the fragment at rows 8 i, columns 8 j of the warp's piece: this lane holds row
// lane / 4 and columns 2 (lane % 4), 2 (lane % 4) + 1 of it.
template <bool B_T>
__device__ __forceinline__ void product_tile(const double* __restrict__ A, int64_t lda, int a_rows,
                                             const double* __restrict__ B, int64_t ldb, int K,
                                             double (&acc)[4][4][2], TileSmem& sm) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 3) * 32, wn = (warp >> 2) * 32;
  const int fk = lane & 3, fr = lane >> 2;                      // fragment coordinates of this lane
  const int ar = tid & 127, akq = (tid >> 7) * 4;               // A loader: row, first k of four
  const int br = tid & 63, bkq = (tid >> 6) * 2;                // B loader (transposed): column, first k of two
  const int bkk = tid >> 5, bnq = (tid & 31) * 2;               // B loader (not transposed): k row, first col of two
  const bool a_ok = ar < a_rows;
  const double* ap = A + static_cast<int64_t>(ar) * lda + akq;
  const double* bp = B_T ? B + static_cast<int64_t>(br) * ldb + bkq : B + static_cast<int64_t>(bkk) * ldb + bnq;
  const int64_t bstep = B_T ? kBK : static_cast<int64_t>(kBK) * ldb;
  const double2 zero2 = make_double2(0.0, 0.0);
  struct Slab { double2 a0, a1, b; };                           // one thread's share of a slab
  Slab s0, s1;                                                  // two slabs in flight

  auto fetch = [&](Slab& r, int k0) {
    if (a_ok) { const double2* g = reinterpret_cast<const double2*>(ap + k0); r.a0 = g[0]; r.a1 = g[1]; }
    else { r.a0 = zero2; r.a1 = zero2; }
    r.b = *reinterpret_cast<const double2*>(bp + (k0 / kBK) * bstep);
  };
  auto stash = [&](const Slab& r, int buf) {
    sm.a[buf][akq + 0][ar] = r.a0.x; sm.a[buf][akq + 1][ar] = r.a0.y;
    sm.a[buf][akq + 2][ar] = r.a1.x; sm.a[buf][akq + 3][ar] = r.a1.y;
    if (B_T) { sm.b[buf][bkq][br] = r.b.x; sm.b[buf][bkq + 1][br] = r.b.y; }
    else *reinterpret_cast<double2*>(&sm.b[buf][bkk][bnq]) = r.b;
  };
  auto multiply = [&](int buf) {
#pragma unroll
    for (int ks = 0; ks < kBK; ks += 4) {
      double af[4], bf[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        af[i] = sm.a[buf][ks + fk][wm + 8 * i + fr];
        bf[i] = sm.b[buf][ks + fk][wn + 8 * i + fr];
      }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) mma_f64(acc[i][j], af[i], bf[j]);
    }
  };

  // slab i is multiplied from buffer i & 1 while slab i+1 moves from registers to the other
  // buffer and slab i+2 starts its trip from global memory
  const int nslab = K / kBK;
  fetch(s0, 0);
  if (nslab > 1) fetch(s1, kBK);
  stash(s0, 0);
  __syncthreads();
  for (int i = 0; i < nslab; i += 2) {
    if (i + 1 < nslab) stash(s1, 1);
    if (i + 2 < nslab) fetch(s0, (i + 2) * kBK);
    multiply(0);
    __syncthreads();
    if (i + 1 < nslab) {
      if (i + 2 < nslab) stash(s0, 0);
      if (i + 3 < nslab) fetch(s1, (i + 3) * kBK);
      multiply(1);
      __syncthreads();
    }
  }
}

// Applies f(row, first column, values of 2 consecutive columns) to a thread's outputs.
template <typename F>
__device__ __forceinline__ void for_each_pair(double (&acc)[4][4][2], F f) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int wm = (warp & 3) * 32, wn = (warp >> 2) * 32;
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) f(wm + 8 * i + (lane >> 2), wn + 8 * j + 2 * (lane & 3), acc[i][j]);
}

// ---- 64 x 64 output tile product with any K (a multiple of 8), same scheme as the 128 x 64 one --
// Used where a launch has few tiles or long reductions (the rank update of the next group's own
// columns; the merges, whose longest reductions decide the kernel's length): half the work per
// CTA, twice the CTAs.  Warps own 32 x 16 pieces (4 x 2 fragments) as in tile_product.
struct TileSmem64 {
  double a[2][kBK][kNB + 4];
  double b[2][kBK][kNB + 4];
};

template <bool B_T>
__device__ __forceinline__ void product_tile64(const double* __restrict__ A, int64_t lda,
                                               const double* __restrict__ B, int64_t ldb, int K,
                                               double (&acc)[4][2][2], TileSmem64& sm) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int wm = (warp & 1) * 32, wn = (warp >> 1) * 16;
  const int fk = lane & 3, fr = lane >> 2;
  const int ar = tid & 63, akq = (tid >> 6) * 2;                // A / B^T loader: row, first k of two
  const int bkk = tid >> 5, bnq = (tid & 31) * 2;               // B loader (not transposed): k row, first col of two
  const double* ap = A + static_cast<int64_t>(ar) * lda + akq;
  const double* bp = B_T ? B + static_cast<int64_t>(ar) * ldb + akq : B + static_cast<int64_t>(bkk) * ldb + bnq;
  const int64_t bstep = B_T ? kBK : static_cast<int64_t>(kBK) * ldb;
  struct Slab { double2 a, b; };
  Slab s0, s1;

  auto fetch = [&](Slab& r, int k0) {
    r.a = *reinterpret_cast<const double2*>(ap + k0);
    r.b = *reinterpret_cast<const double2*>(bp + (k0 / kBK) * bstep);
  };
  auto stash = [&](const Slab& r, int buf) {
    sm.a[buf][akq][ar] = r.a.x; sm.a[buf][akq + 1][ar] = r.a.y;
    if (B_T) { sm.b[buf][akq][ar] = r.b.x; sm.b[buf][akq + 1][ar] = r.b.y; }
    else *reinterpret_cast<double2*>(&sm.b[buf][bkk][bnq]) = r.b;
  };
  auto multiply = [&](int buf) {
#pragma unroll
    for (int ks = 0; ks < kBK; ks += 4) {
      double af[4], bf[2];
#pragma unroll
      for (int i = 0; i < 4; ++i) af[i] = sm.a[buf][ks + fk][wm + 8 * i + fr];
#pragma unroll
      for (int j = 0; j < 2; ++j) bf[j] = sm.b[buf][ks + fk][wn + 8 * j + fr];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 2; ++j) mma_f64(acc[i][j], af[i], bf[j]);
    }
  };

  const int nslab = K / kBK;
  fetch(s0, 0);
  if (nslab > 1) fetch(s1, kBK);
  stash(s0, 0);
  __syncthreads();
  for (int i = 0; i < nslab; i += 2) {
    if (i + 1 < nslab) stash(s1, 1);
    if (i + 2 < nslab) fetch(s0, (i + 2) * kBK);
    multiply(0);
    __syncthreads();
    if (i + 1 < nslab) {
      if (i + 2 < nslab) stash(s0, 0);
      if (i + 3 < nslab) fetch(s1, (i + 3) * kBK);
      multiply(1);
      __syncthreads();
    }
  }
}

// ---- set-up --------------------------------------------------------------------------------
// stats[0] = lambda = percdamp * mean_i diag(H) after the dead-column fix (fixed summation order).
__global__ void __launch_bounds__(256)
damp_kernel(const float* __restrict__ H, int64_t n, double percdamp, double* stats) {
  __shared__ double red[256];
  double s = 0.0;
  for (int64_t i = threadIdx.x; i < n; i += 256) {
    float d = H[i * n + i];
    s += d == 0.0f ? 1.0 : static_cast<double>(d);
  }
  red[threadIdx.x] = s;
  __syncthreads();
  for (int m = 128; m > 0; m >>= 1) {
    if (threadIdx.x < m) red[threadIdx.x] += red[threadIdx.x + m];
    __syncthreads();
  }
  if (threadIdx.x == 0) stats[0] = percdamp * (red[0] / static_cast<double>(n));
}

// A[r][c] = Hd[p(n-1-r)][p(n-1-c)] on and below the diagonal, 0 above it; p is the column order
// the caller quantizes in (identity when perm is null)
__global__ void __launch_bounds__(256)
build_kernel(const float* __restrict__ H, int64_t n, const double* __restrict__ stats, const int* __restrict__ perm,
             double* __restrict__ A) {
  int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= n * n) return;
  int64_t r = e / n, c = e % n;
  double v = 0.0;
  if (r >= c) {
    int64_t i = n - 1 - r, j = n - 1 - c;
    if (perm != nullptr) { i = perm[i]; j = perm[j]; }
    v = static_cast<double>(H[i * n + j]);
    if (i == j) {
      if (v == 0.0) v = 1.0;
      v += stats[0];
    }
  }
  A[e] = v;
}

// ---- diagonal block: Cholesky factor and its inverse, one CTA of 256 threads -------------------
// Shared memory of the block factorization.  The row pitches are 4 mod 16 doubles, which keeps the
// fragment loads of the fp64 matrix instruction (8 rows x 4 columns per half-warp) on distinct banks.
struct PotrfSmem {
  double M[kNB][kNB + 4];
  double T[kNB / 2][kNB / 2 + 4];
  double rdiag[kNB];                       // 1 / L[j][j]
};

// One merge level of the in-block inverse: for every pair of adjacent SZ x SZ inverted diagonal
// blocks XA, XB with the block C of the factor between them,  T = C XA,  C <- -XB T.
// M is zero above the diagonal.  Scalar version (SZ = 8): a thread owns SZ/8 elements.
template <int SZ>
__device__ __forceinline__ void merge_level(double (*M)[kNB + 4], double (*T)[kNB / 2 + 4], int tid) {
  constexpr int PER = SZ / 8;
  int gi[PER], jj[PER], a0[PER];
  double acc[PER];
#pragma unroll
  for (int u = 0; u < PER; ++u) {
    const int e = tid + 256 * u;
    gi[u] = e / SZ;
    jj[u] = e % SZ;
    a0[u] = (gi[u] / SZ) * 2 * SZ;
    acc[u] = 0.0;
  }
#pragma unroll
  for (int m = 0; m < SZ; ++m)
#pragma unroll
    for (int u = 0; u < PER; ++u)
      acc[u] = fma(M[a0[u] + SZ + gi[u] % SZ][a0[u] + m], M[a0[u] + m][a0[u] + jj[u]], acc[u]);
#pragma unroll
  for (int u = 0; u < PER; ++u) { T[gi[u]][jj[u]] = acc[u]; acc[u] = 0.0; }
  __syncthreads();
#pragma unroll
  for (int m = 0; m < SZ; ++m)
#pragma unroll
    for (int u = 0; u < PER; ++u)
      acc[u] = fma(M[a0[u] + SZ + gi[u] % SZ][a0[u] + SZ + m], T[(gi[u] / SZ) * SZ + m][jj[u]], acc[u]);
#pragma unroll
  for (int u = 0; u < PER; ++u) M[a0[u] + SZ + gi[u] % SZ][a0[u] + jj[u]] = -acc[u];
  __syncthreads();
}
// The same level on the fp64 matrix instruction (SZ = 16, 32): 8 x 8 output tiles, warp w takes
// tiles w, w + 8, ...; the sums skip the k-steps that lie wholly above the diagonal of XA / XB.
template <int SZ>
__device__ __forceinline__ void merge_level_mma(double (*M)[kNB + 4], double (*T)[kNB / 2 + 4], int tid) {
  constexpr int TS = SZ / 8;                       // tiles per side of a pair's block
  constexpr int NT = (kNB / (2 * SZ)) * TS * TS;   // tiles of the level
  const int warp = tid >> 5, lane = tid & 31, fr = lane >> 2, fk = lane & 3;
  for (int t = warp; t < NT; t += 8) {
    const int p = t / (TS * TS), ti = (t / TS) % TS, tj = t % TS, a0 = p * 2 * SZ;
    double acc[2] = {0.0, 0.0};
#pragma unroll
    for (int k0 = 0; k0 < SZ; k0 += 4)
      if (k0 + 4 > tj * 8) mma_f64(acc, M[a0 + SZ + ti * 8 + fr][a0 + k0 + fk], M[a0 + k0 + fk][a0 + tj * 8 + fr]);
    T[p * SZ + ti * 8 + fr][tj * 8 + 2 * fk] = acc[0];
    T[p * SZ + ti * 8 + fr][tj * 8 + 2 * fk + 1] = acc[1];
  }
  __syncthreads();
  for (int t = warp; t < NT; t += 8) {
    const int p = t / (TS * TS), ti = (t / TS) % TS, tj = t % TS, a0 = p * 2 * SZ;
    double acc[2] = {0.0, 0.0};
#pragma unroll
    for (int k0 = 0; k0 < SZ; k0 += 4)
      if (k0 < (ti + 1) * 8) mma_f64(acc, M[a0 + SZ + ti * 8 + fr][a0 + SZ + k0 + fk], T[p * SZ + k0 + fk][tj * 8 + fr]);
    M[a0 + SZ + ti * 8 + fr][a0 + tj * 8 + 2 * fk] = -acc[0];
    M[a0 + SZ + ti * 8 + fr][a0 + tj * 8 + 2 * fk + 1] = -acc[1];
  }
  __syncthreads();
}

// In-place Cholesky of the 64 x 64 block held in s.M (its lower triangle; what is above the
// diagonal is ignored) and the triangular inverse of the factor.  On return the factor is in
// blk (row pitch n, zeros above the diagonal) and the inverse in dk (64 x 64, pitch 64).  Every
// thread of the CTA calls it, after a barrier that follows the writes to s.M.
// The block is worked in eight sub-panels of eight columns, right-looking inside shared memory:
//   (a) warps 0 and 1: every thread factors the 8 x 8 diagonal piece redundantly in registers (the
//       sequential chain of eight reciprocal square roots then needs no exchange between threads)
//       and solves the row it owns below the piece by substitution, step by step with the chain;
//   (b) rank-8 update of what follows on the fp64 matrix instruction in 8 x 8 tiles: the next
//       eight columns first (one tile per warp), then, while (a) already runs on them, the rest
//       on the other six warps.
// The inverse is built in place by recursive doubling: 8 x 8 diagonal pieces by substitution
// (one warp each, one column per lane), then three merge levels
//   inv([[A,0],[C,B]]) = [[A^-1,0],[-B^-1 C A^-1,B^-1]].
__device__ __forceinline__ void potrf_block(PotrfSmem& s, double* __restrict__ blk, int64_t n,
                                            double* __restrict__ dk, int* status_dev) {
  constexpr int kSub = 8;
  double (*M)[kNB + 4] = s.M;
  double (*T)[kNB / 2 + 4] = s.T;
  double* rdiag = s.rdiag;
  const int tid = threadIdx.x;
  double d[kSub][kSub], x[kSub];
  bool bad = false;
  auto factor_and_solve = [&](int j0) {
    const int row = j0 + kSub + tid;
#pragma unroll
    for (int r = 0; r < kSub; ++r)
#pragma unroll
      for (int c = 0; c <= r; ++c) d[r][c] = M[j0 + r][j0 + c];
#pragma unroll
    for (int c = 0; c < kSub; ++c) x[c] = row < kNB ? M[row][j0 + c] : 0.0;
#pragma unroll
    for (int c = 0; c < kSub; ++c) {
      double piv = d[c][c];
      if (!(piv > 0.0)) { bad = true; piv = 1.0; }
      const double r = rsqrt(piv);
      if (tid == 63) rdiag[j0 + c] = r;
      d[c][c] = piv * r;
      x[c] *= r;
#pragma unroll
      for (int r2 = c + 1; r2 < kSub; ++r2) d[r2][c] *= r;
#pragma unroll
      for (int c2 = c + 1; c2 < kSub; ++c2) {
#pragma unroll
        for (int r2 = c2; r2 < kSub; ++r2) d[r2][c2] = fma(-d[r2][c], d[c2][c], d[r2][c2]);
        x[c2] = fma(-x[c], d[c2][c], x[c2]);
      }
    }
  };
  auto store_results = [&](int j0) {                   // of factor_and_solve(j0), by the threads that ran it
    const int row = j0 + kSub + tid;
    if (row < kNB) {
#pragma unroll
      for (int c = 0; c < kSub; ++c) M[row][j0 + c] = x[c];
    } else if (tid == 63) {                            // never owns a row: j0 + 8 + 63 > 63
#pragma unroll
      for (int r = 0; r < kSub; ++r)
#pragma unroll
        for (int c = 0; c <= r; ++c) M[j0 + r][j0 + c] = d[r][c];
      if (bad) report(status_dev, ADADIM_ERR_NOT_PD);
    }
  };
  // M[r0 .. r0+8)[c0 .. c0+8) -= M[r0 ..][j0 .. j0+8) M[c0 ..][j0 .. j0+8)^T, one warp
  auto update_tile = [&](int j0, int r0, int c0) {
    const int lane = tid & 31, fr = lane >> 2, fk = lane & 3;
    const double a0 = M[r0 + fr][j0 + fk], a1 = M[r0 + fr][j0 + 4 + fk];
    const double b0 = M[c0 + fr][j0 + fk], b1 = M[c0 + fr][j0 + 4 + fk];
    double2* o = reinterpret_cast<double2*>(&M[r0 + fr][c0 + 2 * fk]);
    const double2 ov = *o;
    double p[2] = {0.0, 0.0}, q[2] = {0.0, 0.0};
    mma_f64(p, a0, b0);
    mma_f64(q, a1, b1);
    *o = make_double2(ov.x - (p[0] + q[0]), ov.y - (p[1] + q[1]));
  };

  if (tid < 64) { factor_and_solve(0); store_results(0); }
  __syncthreads();
#pragma unroll 1
  for (int j0 = 0; j0 + kSub < kNB; j0 += kSub) {
    const int lim = j0 + kSub, warp = tid >> 5;
    const int m = (kNB - lim) / kSub;                  // 8 x 8 tiles per side of what is left
    if (warp < m) update_tile(j0, lim + warp * kSub, lim);
    __syncthreads();
    if (tid < 64) {
      factor_and_solve(lim);
      store_results(lim);                              // columns lim .. lim+7: no tile of the branch below touches them
    } else {
      // tile t = ti (ti - 1) / 2 + (tj - 1), 1 <= tj <= ti < m, on warps 2..7
      for (int t = warp - 2; t < m * (m - 1) / 2; t += 6) {
        int ti = 1;
        while (t >= ti * (ti + 1) / 2) ++ti;
        const int tj = t - ti * (ti - 1) / 2 + 1;
        update_tile(j0, lim + ti * kSub, lim + tj * kSub);
      }
    }
    __syncthreads();
  }

  // the factor goes back to the matrix; above the diagonal it is zero there and, from here on, in
  // M too (the updates that produced this block left symmetric leftovers there, and the merges
  // below sum over whole rows and columns)
  for (int e = tid; e < kNB * kNB; e += 256) {
    const int r = e >> 6, c = e & 63;
    if (r < c) M[r][c] = 0.0;
    blk[static_cast<int64_t>(r) * n + c] = r >= c ? M[r][c] : 0.0;
  }
  __syncthreads();

  // ---- inverse, in place ----------------------------------------------------------------------
  {
    const int wv = tid >> 5, c = tid & 31;             // warp wv inverts piece wv, lane c its column c
    const int o = wv * kSub;
    double xx[kSub];
    if (c < kSub) {
      // column c by forward substitution, finished entries pushed forward
#pragma unroll
      for (int r = 0; r < kSub; ++r) xx[r] = r == c ? 1.0 : 0.0;
#pragma unroll
      for (int r = 0; r < kSub; ++r) {
        xx[r] *= rdiag[o + r];
#pragma unroll
        for (int r2 = r + 1; r2 < kSub; ++r2) xx[r2] = fma(-M[o + r2][o + r], xx[r], xx[r2]);
      }
    }
    __syncwarp();
    if (c < kSub) {
#pragma unroll
      for (int r = 0; r < kSub; ++r) M[o + r][o + c] = xx[r];                    // zeros above the diagonal
    }
  }
  __syncthreads();
  merge_level<8>(M, T, tid);
  merge_level_mma<16>(M, T, tid);
  merge_level_mma<32>(M, T, tid);
  for (int e = tid; e < kNB * kNB; e += 256) {
    const int r = e >> 6, c = e & 63;
    dk[e] = r >= c ? M[r][c] : 0.0;
  }
}

// Diagonal block k as a launch of its own (block 0; every later one is factored by the CTA that
// finishes its last update, see group_update_kernel and rank_update_first_kernel).
__global__ void __launch_bounds__(256, 2)
potrf_kernel(double* __restrict__ A, int64_t n, int k, double* __restrict__ dinv, int* status_dev) {
  __shared__ PotrfSmem s;
  const int tid = threadIdx.x;
  double* blk = A + (static_cast<int64_t>(k) * kNB) * n + static_cast<int64_t>(k) * kNB;
  dep_release();
  dep_wait();
  {
    double v[kNB * kNB / 256];                         // all loads in flight before the first store
#pragma unroll
    for (int u = 0; u < kNB * kNB / 256; ++u) {
      const int e = tid + 256 * u;
      v[u] = blk[static_cast<int64_t>(e >> 6) * n + (e & 63)];
    }
#pragma unroll
    for (int u = 0; u < kNB * kNB / 256; ++u) {
      const int e = tid + 256 * u;
      s.M[e >> 6][e & 63] = v[u];
    }
  }
  __syncthreads();
  potrf_block(s, blk, n, dinv + static_cast<int64_t>(k) * kNB * kNB, status_dev);
}

// Panel below diagonal block k:  A[i][k] <- A[i][k] * inv(L_kk)^T   (one 64-row tile per CTA)
// The kernels of the chain start before their predecessor has finished (programmatic dependent
// launch) and wait for it inside, so what the predecessor writes is not read-only for the kernel's
// lifetime: `dinv` must not be `const __restrict__`, which would let its loads be treated as
// invariant and moved above the wait.
__global__ void __launch_bounds__(256)
panel_kernel(double* __restrict__ A, int64_t n, int k, const double* dinv) {
  TILE_SMEM
  const int64_t row0 = (static_cast<int64_t>(k) + 1 + blockIdx.x) * kNB;
  double* tile = A + row0 * n + static_cast<int64_t>(k) * kNB;
  dep_release();
  dep_wait();
  double acc[4][2][2] = {};
  tile_product<true>(tile, n, dinv + static_cast<int64_t>(k) * kNB * kNB, kNB, acc, sa, sb);
  for_each_pair64(acc, [&](int r, int c, const double* v) {
    *reinterpret_cast<double2*>(tile + static_cast<int64_t>(r) * n + c) = make_double2(v[0], v[1]);
  });
}

// Update inside the current group of panels after panel k:  A[i][j] -= L[i][k] L[j][k]^T for the
// column tiles j of the group that follow k and all row tiles i >= j.  blockIdx.x = i - (k+1),
// blockIdx.y = j - (k+1).
// The CTA of tile (k+1, k+1) then holds the next diagonal block in its final state: it does not
// store it but factors it on the spot (potrf_block), so that the chain goes on without a launch
// and a round trip through memory in between, while the other CTAs finish their tiles.
__global__ void __launch_bounds__(256, 2)
group_update_kernel(double* __restrict__ A, int64_t n, int k, double* __restrict__ dinv, int* status_dev) {
  __shared__ __align__(16) unsigned char raw[sizeof(PotrfSmem)];
  static_assert(sizeof(PotrfSmem) >= 2 * kHalfK * (kNB + 4) * sizeof(double), "tile staging fits");
  double (*sa)[kNB + 4] = reinterpret_cast<double (*)[kNB + 4]>(raw);
  double (*sb)[kNB + 4] = sa + kHalfK;
  dep_release();
  dep_wait();
  if (blockIdx.y > blockIdx.x) return;
  const int64_t ri = (static_cast<int64_t>(k) + 1 + blockIdx.x) * kNB, rj = (static_cast<int64_t>(k) + 1 + blockIdx.y) * kNB;
  const int64_t ck = static_cast<int64_t>(k) * kNB;
  double acc[4][2][2] = {};
  tile_product<true>(A + ri * n + ck, n, A + rj * n + ck, n, acc, sa, sb);
  double* c0 = A + ri * n + rj;
  if (blockIdx.x == 0 && blockIdx.y == 0) {
    PotrfSmem& s = *reinterpret_cast<PotrfSmem*>(raw);
    __syncthreads();                                   // the staged operands have been read by every warp
    for_each_pair64(acc, [&](int r, int c, const double* v) {
      const double2 u = *reinterpret_cast<const double2*>(c0 + static_cast<int64_t>(r) * n + c);
      *reinterpret_cast<double2*>(&s.M[r][c]) = make_double2(u.x - v[0], u.y - v[1]);
    });
    __syncthreads();
    potrf_block(s, c0, n, dinv + (static_cast<int64_t>(k) + 1) * kNB * kNB, status_dev);
    return;
  }
  for_each_pair64(acc, [&](int r, int c, const double* v) {
    double2* p = reinterpret_cast<double2*>(c0 + static_cast<int64_t>(r) * n + c);
    double2 u = *p;
    u.x -= v[0]; u.y -= v[1];
    *p = u;
  });
}

// Rank-`kw` update of everything right of a finished group, for the region starting at row/column e:
//   A[i][j] -= L[i][j0 .. j0+kw) L[j][j0 .. j0+kw)^T   on and below the diagonal.
// The update is issued in two parts so that the next group's factorization can start early:
//  * the next group's own columns [e, e + 256): rank_update_first_kernel, 64 x 64 tiles, one wave
//    of short CTAs on the high-priority chain; the CTA of the first diagonal tile goes straight on
//    to factor it (as in group_update_kernel);
//  * the rest: rank_update_kernel, 128 x 64 tiles over the whole triangle, skipping those columns.
// In the second kernel row block ti meets column blocks 0 .. 2*ti+1; the tile right of the diagonal
// 64-block (column block 2*ti+1) only stores its lower 64 rows: the block above them must stay zero.
constexpr int kLook = kGroup * kNB / kTN;
__global__ void __launch_bounds__(256, 2)
rank_update_first_kernel(double* __restrict__ A, int64_t n, int64_t e, int64_t j0, int kw,
                         double* __restrict__ dinv, int* status_dev) {
  __shared__ __align__(16) unsigned char raw[sizeof(PotrfSmem)];
  static_assert(sizeof(PotrfSmem) >= sizeof(TileSmem64), "tile staging fits");
  TileSmem64& sm = *reinterpret_cast<TileSmem64*>(raw);
  const int ti = blockIdx.y, cj = blockIdx.x;               // 64-row block, 64-column block of the region
  dep_release();
  dep_wait();
  if (cj > ti) return;
  const int64_t ri = e + static_cast<int64_t>(ti) * kNB, rj = e + static_cast<int64_t>(cj) * kNB;
  if (rj >= n) return;
  double acc[4][2][2] = {};
  product_tile64<true>(A + ri * n + j0, n, A + rj * n + j0, n, kw, acc, sm);
  if (ti == 0 && cj == 0) {
    // the next group's first diagonal block is final with this update: factor it here
    PotrfSmem& s = *reinterpret_cast<PotrfSmem*>(raw);
    double* blk = A + ri * n + rj;
    __syncthreads();                                   // the staged slabs have been read by every warp
    for_each_pair64(acc, [&](int r, int c2, const double* v) {
      const double2 u = *reinterpret_cast<const double2*>(blk + static_cast<int64_t>(r) * n + c2);
      *reinterpret_cast<double2*>(&s.M[r][c2]) = make_double2(u.x - v[0], u.y - v[1]);
    });
    __syncthreads();
    potrf_block(s, blk, n, dinv + (e / kNB) * kNB * kNB, status_dev);
    return;
  }
  for_each_pair64(acc, [&](int r, int c2, const double* v) {
    double2* p = reinterpret_cast<double2*>(A + (ri + r) * n + rj + c2);
    double2 u = *p;
    u.x -= v[0]; u.y -= v[1];
    *p = u;
  });
}

__global__ void __launch_bounds__(256, 2)
rank_update_kernel(double* __restrict__ A, int64_t n, int64_t e, int64_t j0, int kw) {
  __shared__ TileSmem sm;
  const int t = blockIdx.x;
  int ti = static_cast<int>((sqrt(4.0 * t + 1.0) - 1.0) * 0.5);
  while (ti * (ti + 1) > t) --ti;
  while ((ti + 1) * (ti + 2) <= t) ++ti;
  const int cj = t - ti * (ti + 1);
  if (cj < kLook) return;
  const int64_t ri = e + static_cast<int64_t>(ti) * kT, rj = e + static_cast<int64_t>(cj) * kTN;
  if (rj >= n) return;
  const int vr = static_cast<int>(mn64(kT, n - ri));
  double acc[4][4][2] = {};
  product_tile<true>(A + ri * n + j0, n, vr, A + rj * n + j0, n, kw, acc, sm);
  const int skip_rows = cj == 2 * ti + 1 ? 64 : 0;
  for_each_pair(acc, [&](int r, int c2, const double* v) {
    if (r >= vr || r < skip_rows) return;
    double2* p = reinterpret_cast<double2*>(A + (ri + r) * n + rj + c2);
    double2 u = *p;
    u.x -= v[0]; u.y -= v[1];
    *p = u;
  });
}

// ---- inverse by recursive doubling -----------------------------------------------------------
__global__ void __launch_bounds__(256)
seed_kernel(double* __restrict__ A, int64_t n, const double* __restrict__ dinv, int k0) {
  // diagonal 64-blocks k0 + blockIdx.x of A <- their inverses
  const int k = k0 + blockIdx.x;
  double* blk = A + (static_cast<int64_t>(k) * kNB) * n + static_cast<int64_t>(k) * kNB;
  const double* dk = dinv + static_cast<int64_t>(k) * kNB * kNB;
  for (int e = threadIdx.x; e < kNB * kNB; e += 256) blk[static_cast<int64_t>(e >> 6) * n + (e & 63)] = dk[e];
}

// Level with half-size s (elements): pair p covers [p*2s, p*2s+2s); its A part is the first s
// rows/cols (already inverted: XA), its B part the rest (XB, sB <= s rows), C the block below A.
// T is packed pair after pair (every earlier pair has s B-rows), rows local to the B part, pitch s.
// step 1:  T = C * XA      (T tile (r,c): reduction over XA rows m >= c only, XA is lower)
// step 2:  C <- -XB * T    (C tile (r,c): reduction over XB columns m <= r only)
// A launch covers the pairs p0 + blockIdx.{x,y} of one level; the pair's T is slot blockIdx.{x,y}
// of the level's region (pitch s, s rows per slot).
__global__ void __launch_bounds__(256)
merge1_64_kernel(const double* __restrict__ A, int64_t n, double* __restrict__ T, int p0) {      // s == 64
  TILE_SMEM
  const int64_t s = kNB, a0 = static_cast<int64_t>(p0 + blockIdx.x) * 2 * s, b0 = a0 + s;
  if (b0 >= n) return;
  double acc[4][2][2] = {};
  tile_product<false>(A + b0 * n + a0, n, A + a0 * n + a0, n, acc, sa, sb);
  double* t = T + static_cast<int64_t>(blockIdx.x) * s * s;
  for_each_pair64(acc, [&](int r, int c, const double* v) {
    *reinterpret_cast<double2*>(t + r * s + c) = make_double2(v[0], v[1]);
  });
}
__global__ void __launch_bounds__(256)
merge2_64_kernel(double* __restrict__ A, int64_t n, const double* __restrict__ T, int p0) {      // s == 64
  TILE_SMEM
  const int64_t s = kNB, a0 = static_cast<int64_t>(p0 + blockIdx.x) * 2 * s, b0 = a0 + s;
  if (b0 >= n) return;
  double acc[4][2][2] = {};
  tile_product<false>(A + b0 * n + b0, n, T + static_cast<int64_t>(blockIdx.x) * s * s, s, acc, sa, sb);
  double* dst = A + b0 * n + a0;
  for_each_pair64(acc, [&](int r, int c, const double* v) {
    *reinterpret_cast<double2*>(dst + static_cast<int64_t>(r) * n + c) = make_double2(-v[0], -v[1]);
  });
}

__global__ void __launch_bounds__(256, 2)
merge1_kernel(const double* __restrict__ A, int64_t n, int64_t s, double* __restrict__ T, int p0) {      // s >= 128
  __shared__ TileSmem64 sm;
  const int64_t a0 = static_cast<int64_t>(p0 + blockIdx.y) * 2 * s, b0 = a0 + s;
  // 64-row block r, 64-column block c; the reduction length s - 64 c falls with c, so tiles are
  // handed out column block by column block: the longest ones start first
  const int rtiles = static_cast<int>(s / kNB);
  const int64_t sB = mn64(s, n - b0);
  const int r = blockIdx.x % rtiles, c = blockIdx.x / rtiles;
  if (static_cast<int64_t>(r) * kNB >= sB) return;
  const int64_t m0 = static_cast<int64_t>(c) * kNB;
  double acc[4][2][2] = {};
  product_tile64<false>(A + (b0 + static_cast<int64_t>(r) * kNB) * n + a0 + m0, n, A + (a0 + m0) * n + a0 + m0, n,
                        static_cast<int>(s - m0), acc, sm);
  double* tp = T + static_cast<int64_t>(blockIdx.y) * s * s + static_cast<int64_t>(r) * kNB * s + m0;
  for_each_pair64(acc, [&](int rr, int c2, const double* v) {
    *reinterpret_cast<double2*>(tp + static_cast<int64_t>(rr) * s + c2) = make_double2(v[0], v[1]);
  });
}
// Rows [64 r_lo, 64 r_hi) of the pair's lower-left block only: row block r of the result needs rows
// <= r of XB, which are final as soon as the factorization has passed them.
__global__ void __launch_bounds__(256, 2)
merge2_kernel(double* __restrict__ A, int64_t n, int64_t s, const double* __restrict__ T, int p0, int r_lo, int r_hi) {      // s >= 128
  __shared__ TileSmem64 sm;
  const int ctiles = static_cast<int>(s / kNB);
  const int64_t a0 = static_cast<int64_t>(p0 + blockIdx.y) * 2 * s, b0 = a0 + s;
  // the reduction length 64 (r + 1) grows with the row block: the last row blocks start first
  const int r = r_hi - 1 - static_cast<int>(blockIdx.x) / ctiles, c = blockIdx.x % ctiles;
  const int64_t sB = mn64(s, n - b0);
  if (r < r_lo || static_cast<int64_t>(r) * kNB >= sB) return;
  const int64_t row0 = b0 + static_cast<int64_t>(r) * kNB;
  const int K = static_cast<int>(mn64(static_cast<int64_t>(r + 1) * kNB, sB));
  double acc[4][2][2] = {};
  product_tile64<false>(A + row0 * n + b0, n, T + static_cast<int64_t>(blockIdx.y) * s * s + static_cast<int64_t>(c) * kNB,
                        s, K, acc, sm);
  double* dst = A + row0 * n + a0 + static_cast<int64_t>(c) * kNB;
  for_each_pair64(acc, [&](int rr, int c2, const double* v) {
    *reinterpret_cast<double2*>(dst + static_cast<int64_t>(rr) * n + c2) = make_double2(-v[0], -v[1]);
  });
}

// U[i][j] = Linv[n-1-i][n-1-j] for i <= j, else 0
__global__ void __launch_bounds__(256)
emit_kernel(const double* __restrict__ A, int64_t n, double* __restrict__ U) {
  int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= n * n) return;
  int64_t i = e / n, j = e % n;
  U[e] = i <= j ? A[(n - 1 - i) * n + (n - 1 - j)] : 0.0;
}

// ---- the inverse's schedule ---------------------------------------------------------------------
// Level l merges with half-size s = 64 << l; pair p of a level covers [p 2s, p 2s + 2s) and exists
// when its second half starts inside the matrix.  A pair's first step (T = C XA) needs columns
// [0, p 2s + s) of L final and its first half inverted; its second step needs the whole pair.  The
// factorization finishes L's columns from the left, so most steps can be issued while it is still
// running: InverseSchedule::advance(done) issues, level by level, every step that has become
// possible once columns [0, done) are final.  None of them writes a row or column >= done, and the
// factorization from there on only reads rows >= done of those columns (its rank updates), so the
// two never meet; what is left after the last diagonal block is the last pair of every level.
//
// Above half-size 256 a pair's second step is itself issued in slices of rows: row block r of
// -XB T needs rows <= r of XB only, and those are final once the factorization has passed them (the
// lower levels, issued first, have completed them up to the same point).
//
// A level keeps T for the pairs of ONE first-step launch (`slots` of them, s x s each, s x (n - s)
// when the matrix is shorter): a new first step is issued only after the second steps of the
// previous launch, all on one stream.
constexpr int kMaxLevels = 40;
struct LevelPlan { int64_t s; int npairs, slots; size_t t_off; };
struct InversePlan { int nlev; LevelPlan lev[kMaxLevels]; size_t t_doubles; };
InversePlan inverse_plan(int64_t n) {
  InversePlan P;
  P.nlev = 0;
  size_t off = 0;
  for (int64_t s = kNB; s < n && P.nlev < kMaxLevels; s *= 2) {
    LevelPlan& L = P.lev[P.nlev++];
    L.s = s;
    L.npairs = static_cast<int>((n - s + 2 * s - 1) / (2 * s));
    L.slots = static_cast<int>(mx64(1, static_cast<int64_t>(kGroup) * kNB / (2 * s)));
    L.t_off = off;
    off += static_cast<size_t>(L.slots > 1 ? L.slots * s * s : s * mn64(s, n - s));
  }
  P.t_doubles = off;
  return P;
}

struct FactorLayout { size_t a_off, t_off, dinv_off, stats_off, total; };
FactorLayout factor_layout(int64_t n) {
  FactorLayout L;
  size_t off = 0;
  L.a_off = off;     off += round_up(static_cast<size_t>(n) * n * 8, 256);
  L.t_off = off;     off += round_up(inverse_plan(n).t_doubles * 8 + 256, 256);
  L.dinv_off = off;  off += round_up(static_cast<size_t>(n) * kNB * 8, 256);
  L.stats_off = off; off += 256;
  L.total = off;
  return L;
}

struct InverseSchedule {
  InversePlan P;
  double* A;
  double* T;
  const double* dinv;
  int64_t n;
  int seeded = 0;                                   // diagonal blocks already replaced by their inverses
  int m1[kMaxLevels] = {}, m2[kMaxLevels] = {}, base[kMaxLevels] = {};   // pairs with step 1 / step 2 issued; first pair of the latest step-1 launch
  int rows2[kMaxLevels] = {};                       // 64-row blocks of pair m2's second step already issued (levels above kSmallLevel)
  InverseSchedule(double* A_, double* T_, const double* dinv_, int64_t n_) : P(inverse_plan(n_)), A(A_), T(T_), dinv(dinv_), n(n_) {}

  // The levels up to half-size kSmallLevel are short launches of a few CTAs, bound by their
  // latency; the levels above them are long and bound by throughput.  They go to two streams
  // (`st`, `st_big`) so that the second kind runs beside the first; `ev` carries the dependency
  // of a level on the ones below it across the two.
  static constexpr int64_t kSmallLevel = 256;
  int advance(int64_t done, cudaStream_t st_small, cudaStream_t st_big, cudaEvent_t ev) {
    const int nbk = static_cast<int>(done / kNB);
    if (nbk > seeded) {
      seed_kernel<<<nbk - seeded, 256, 0, st_small>>>(A, n, dinv, seeded);
      seeded = nbk;
    }
    bool crossed = false;
    for (int l = 0; l < P.nlev; ++l) {
      const LevelPlan& L = P.lev[l];
      const int64_t s = L.s;
      cudaStream_t st = s <= kSmallLevel ? st_small : st_big;
      if (s > kSmallLevel && !crossed) {
        crossed = true;
        ADADIM_CUDA_TRY(cudaEventRecord(ev, st_small));
        ADADIM_CUDA_TRY(cudaStreamWaitEvent(st_big, ev, 0));
      }
      double* t = T + L.t_off;
      const unsigned tiles = static_cast<unsigned>((s / kNB) * (s / kNB));
      for (;;) {
        if (s > kSmallLevel) {
          // one pair at a time, its second step in row slices as the factorization passes them
          if (m2[l] < m1[l]) {
            const int q = m2[l];
            const int64_t b0 = static_cast<int64_t>(q) * 2 * s + s, sB = mn64(s, n - b0);
            int avail = static_cast<int>((mn64(done, b0 + sB) - b0) / kNB);
            const int half = static_cast<int>(s / (2 * kNB));                  // slices of half the block: short slices fill the machine badly
            if (static_cast<int64_t>(avail) * kNB < sB) avail = avail / half * half;
            if (avail > rows2[l]) {
              const unsigned gx = static_cast<unsigned>((avail - rows2[l]) * (s / kNB));
              merge2_kernel<<<dim3(gx, 1), 256, 0, st>>>(A, n, s, t, q, rows2[l], avail);
              rows2[l] = avail;
            }
            if (static_cast<int64_t>(rows2[l]) * kNB >= sB) { ++m2[l]; rows2[l] = 0; }
          }
        } else {
          int q2 = m2[l];
          while (q2 < m1[l] && mn64(static_cast<int64_t>(q2 + 1) * 2 * s, n) <= done) ++q2;
          if (q2 > m2[l]) {
            const unsigned cnt = static_cast<unsigned>(q2 - m2[l]);
            double* ts = t + static_cast<size_t>(m2[l] - base[l]) * s * s;
            if (s == kNB) merge2_64_kernel<<<cnt, 256, 0, st>>>(A, n, ts, m2[l]);
            else merge2_kernel<<<dim3(tiles, cnt), 256, 0, st>>>(A, n, s, ts, m2[l], 0, static_cast<int>(s / kNB));
            m2[l] = q2;
          }
        }
        if (m2[l] < m1[l]) break;                       // a pair still waits for its second half
        int q1 = m1[l];
        while (q1 < L.npairs && q1 - m1[l] < L.slots && static_cast<int64_t>(q1) * 2 * s + s <= done) ++q1;
        if (q1 == m1[l]) break;
        const unsigned cnt = static_cast<unsigned>(q1 - m1[l]);
        if (s == kNB) merge1_64_kernel<<<cnt, 256, 0, st>>>(A, n, t, m1[l]);
        else merge1_kernel<<<dim3(tiles, cnt), 256, 0, st>>>(A, n, s, t, m1[l]);
        base[l] = m1[l];
        m1[l] = q1;
      }
    }
    return ADADIM_OK;
  }
};

}  // namespace

size_t factor_workspace_bytes(int64_t n) { return factor_layout(n).total; }

int factor_launch(const float* H, int64_t n, double percdamp, double* U, int* status_dev, void* workspace,
                  cudaStream_t st, const int* perm) {
  FactorLayout Lo = factor_layout(n);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  double* A = reinterpret_cast<double*>(ws + Lo.a_off);
  double* T = reinterpret_cast<double*>(ws + Lo.t_off);
  double* dinv = reinterpret_cast<double*>(ws + Lo.dinv_off);
  double* stats = reinterpret_cast<double*>(ws + Lo.stats_off);
  const int nb = static_cast<int>(n / kNB);
  const unsigned eb = static_cast<unsigned>((n * n + 255) / 256);

  // The factorization's chain of small kernels (diagonal blocks, panels, in-group updates and the
  // rank update of the next group's own columns) runs on a high-priority stream; the rest of each
  // group's rank update runs beside it on a second stream.  Every kernel of the chain fits on an
  // SM next to one CTA of the rank update, so the chain is scheduled as soon as any CTA retires.
  // The inverse's merges run behind both on a third, lowest-priority stream as soon as the columns
  // they need are final (InverseSchedule); only the last pair of each level is left when the chain
  // ends.
  ForkedStreams fs;                                  // joins and releases on every way out of this function
  bool rest_pending = false;

  damp_kernel<<<1, 256, 0, st>>>(H, n, percdamp, stats);
  build_kernel<<<eb, 256, 0, st>>>(H, n, stats, perm, A);
  {
    const int rc = fs.open(st, true);
    if (rc != ADADIM_OK) return rc;
  }
  cudaStream_t chain = fs.chain, side = fs.side, back = fs.back;
  cudaEvent_t ev_panels = fs.ev_a, ev_rest = fs.ev_b;
  InverseSchedule inv(A, T, dinv, n);
  for (int g0 = 0; g0 < nb; g0 += kGroup) {
    const int g1 = g0 + kGroup < nb ? g0 + kGroup : nb;
    for (int k = g0; k < g1; ++k) {
      // diagonal block k > 0 was factored by the launch that completed it
      if (k == 0) ADADIM_CUDA_TRY(launch_chained(potrf_kernel, dim3(1), dim3(256), chain, A, n, k, dinv, status_dev));
      const int below = nb - k - 1;
      if (below > 0) ADADIM_CUDA_TRY(launch_chained(panel_kernel, dim3(below), dim3(256), chain, A, n, k, static_cast<const double*>(dinv)));
      const int inner = g1 - k - 1;
      if (below > 0 && inner > 0) ADADIM_CUDA_TRY(launch_chained(group_update_kernel, dim3(below, inner), dim3(256), chain, A, n, k, dinv, status_dev));
    }
    const int64_t e = static_cast<int64_t>(g1) * kNB;
    ADADIM_CUDA_TRY(cudaEventRecord(ev_panels, chain));          // columns [0, e) of L are final
    if (e < n) {
      const int nt = static_cast<int>((n - e + kT - 1) / kT);
      const int64_t j0 = static_cast<int64_t>(g0) * kNB;
      const int kw = (g1 - g0) * kNB;
      const bool has_rest = e + kLook * kTN < n;
      // the columns updated next were last written by the previous group's side-stream launch
      if (rest_pending) ADADIM_CUDA_TRY(cudaStreamWaitEvent(chain, ev_rest, 0));
      ADADIM_CUDA_TRY(launch_chained(rank_update_first_kernel, dim3(kLook, static_cast<unsigned>((n - e) / kNB)), dim3(256), chain, A, n, e, j0, kw, dinv, status_dev));
      rest_pending = false;
      if (has_rest) {
        ADADIM_CUDA_TRY(cudaStreamWaitEvent(side, ev_panels, 0));
        rank_update_kernel<<<nt * (nt + 1), 256, 0, side>>>(A, n, e, j0, kw);
        ADADIM_CUDA_TRY(cudaEventRecord(ev_rest, side));
        rest_pending = true;
      }
    }
    ADADIM_CUDA_TRY(cudaStreamWaitEvent(back, ev_panels, 0));
    {
      const int rc = inv.advance(e < n ? e : n, back, fs.back2, fs.ev_c);
      if (rc != ADADIM_OK) return rc;
    }
  }
  {
    const int rc = fs.join();
    if (rc != ADADIM_OK) return rc;
  }
  emit_kernel<<<eb, 256, 0, st>>>(A, n, U);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
