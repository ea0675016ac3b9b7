// Damped Cholesky-inverse factor for GPTQ (paper Section 2.2 cites the algorithm; the damping
// and the factor are the published algorithm's):  Hd = H + lambda I,  Hd^-1 = U^T U,  U upper.
//
// Route: with P the index reversal, factor A = P Hd P = L L^T (L lower) and invert the
// triangle; then U = P L^-1 P, because Hd = (P L P)(P L P)^T with P L P upper triangular and
// Hd^-1 = (P L^-1 P)^T (P L^-1 P).  This needs one factorization and one triangular inverse
// instead of a factorization, a full inverse and a second factorization.  All arithmetic is
// binary64 on the CUDA cores (the factor decides GPTQ's rounding, so it is kept well inside
// the fp32 precision of U); U is rounded to fp32 on output.
//
//   factorization : right-looking, 64-column panels (diagonal block on one CTA, then a panel
//                   multiply by the inverted diagonal block, then the trailing update)
//   inverse       : recursive doubling.  inv([[A,0],[C,B]]) = [[A^-1,0],[-B^-1 C A^-1,B^-1]]:
//                   level by level, adjacent inverted diagonal blocks are merged with two
//                   batched triangular-aware matrix products, log2(n/64) levels in all.
#include "common.cuh"

namespace adadim {
namespace {

constexpr int kNB = 64;     // panel width and tile edge

// ---- 64 x 64 output tile product, 256 threads, 4 x 4 outputs per thread --------------------
// acc += A[64 x K] * B, A row-major with leading dimension lda;
// B_T: B is given as [64 cols][K] row-major (product with the transpose), else as [K][64 cols].
template <bool B_T>
__device__ __forceinline__ void tile_product(const double* __restrict__ A, int64_t lda, const double* __restrict__ B,
                                             int64_t ldb, int K, double (&acc)[4][4], double (*sa)[kNB + 2],
                                             double (*sb)[kNB + 2]) {
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  for (int k0 = 0; k0 < K; k0 += 16) {
    {
      const int r = threadIdx.x >> 2, kq = (threadIdx.x & 3) * 4;
      const double2* src = reinterpret_cast<const double2*>(A + static_cast<int64_t>(r) * lda + k0 + kq);
      double2 v0 = src[0], v1 = src[1];
      sa[kq + 0][r] = v0.x; sa[kq + 1][r] = v0.y; sa[kq + 2][r] = v1.x; sa[kq + 3][r] = v1.y;
    }
    if (B_T) {
      const int r = threadIdx.x >> 2, kq = (threadIdx.x & 3) * 4;
      const double2* src = reinterpret_cast<const double2*>(B + static_cast<int64_t>(r) * ldb + k0 + kq);
      double2 v0 = src[0], v1 = src[1];
      sb[kq + 0][r] = v0.x; sb[kq + 1][r] = v0.y; sb[kq + 2][r] = v1.x; sb[kq + 3][r] = v1.y;
    } else {
      const int kk = threadIdx.x >> 4, nq = (threadIdx.x & 15) * 4;
      const double2* src = reinterpret_cast<const double2*>(B + static_cast<int64_t>(k0 + kk) * ldb + nq);
      double2 v0 = src[0], v1 = src[1];
      sb[kk][nq + 0] = v0.x; sb[kk][nq + 1] = v0.y; sb[kk][nq + 2] = v1.x; sb[kk][nq + 3] = v1.y;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      double a[4], b[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) { a[m] = sa[kk][ty * 4 + m]; b[m] = sb[kk][tx * 4 + m]; }
#pragma unroll
      for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int n = 0; n < 4; ++n) acc[m][n] = fma(a[m], b[n], acc[m][n]);
    }
    __syncthreads();
  }
}

#define TILE_SMEM                      \
  __shared__ double sa[16][kNB + 2];   \
  __shared__ double sb[16][kNB + 2];

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
  if (threadIdx.x == 0) stats[0] = percdamp * red[0] / static_cast<double>(n);
}

// A[r][c] = Hd[n-1-r][n-1-c]
__global__ void __launch_bounds__(256)
build_kernel(const float* __restrict__ H, int64_t n, const double* __restrict__ stats, double* __restrict__ A) {
  int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= n * n) return;
  int64_t r = e / n, c = e % n;
  int64_t i = n - 1 - r, j = n - 1 - c;
  double v = static_cast<double>(H[i * n + j]);
  if (i == j) {
    if (v == 0.0) v = 1.0;
    v += stats[0];
  }
  A[e] = v;
}

// ---- factorization -------------------------------------------------------------------------
// Diagonal block k: in-place Cholesky of the 64 x 64 block and its triangular inverse -> dinv[k].
__global__ void __launch_bounds__(256)
potrf_kernel(double* __restrict__ A, int64_t n, int k, double* __restrict__ dinv, int* status_dev) {
  __shared__ double L[kNB][kNB + 1];
  double* blk = A + (static_cast<int64_t>(k) * kNB) * n + static_cast<int64_t>(k) * kNB;
  for (int e = threadIdx.x; e < kNB * kNB; e += 256) L[e >> 6][e & 63] = blk[static_cast<int64_t>(e >> 6) * n + (e & 63)];
  __syncthreads();
  for (int j = 0; j < kNB; ++j) {
    double piv = L[j][j];
    __syncthreads();
    if (!(piv > 0.0)) {
      if (threadIdx.x == 0) report(status_dev, ADADIM_ERR_NOT_PD);
      piv = 1.0;
    }
    const double d = sqrt(piv);
    if (threadIdx.x == 0) L[j][j] = d;
    if (threadIdx.x > j && threadIdx.x < kNB) L[threadIdx.x][j] /= d;
    __syncthreads();
    // trailing rank-one update of the lower triangle
    for (int e = threadIdx.x; e < kNB * kNB; e += 256) {
      int r = e >> 6, c = e & 63;
      if (c > j && r >= c) L[r][c] -= L[r][j] * L[c][j];
    }
    __syncthreads();
  }
  // X = L^-1 by forward substitution, one column per thread, the column held in registers.
  // Entries above the diagonal come out as exact zeros (their right-hand side is zero).
  double* dk = dinv + static_cast<int64_t>(k) * kNB * kNB;
  if (threadIdx.x < kNB) {
    const int c = threadIdx.x;
    double x[kNB];
#pragma unroll
    for (int r = 0; r < kNB; ++r) {
      double s = (r == c) ? 1.0 : 0.0;
#pragma unroll
      for (int m = 0; m < r; ++m) s = fma(-L[r][m], x[m], s);
      x[r] = s / L[r][r];
      dk[r * kNB + c] = x[r];
    }
  }
  for (int e = threadIdx.x; e < kNB * kNB; e += 256) {
    int r = e >> 6, c = e & 63;
    blk[static_cast<int64_t>(r) * n + c] = r >= c ? L[r][c] : 0.0;
  }
}

// Panel below diagonal block k:  A[i][k] <- A[i][k] * inv(L_kk)^T   (one 64-row tile per CTA)
__global__ void __launch_bounds__(256)
panel_kernel(double* __restrict__ A, int64_t n, int k, const double* __restrict__ dinv) {
  TILE_SMEM
  const int64_t row0 = (static_cast<int64_t>(k) + 1 + blockIdx.x) * kNB;
  double* tile = A + row0 * n + static_cast<int64_t>(k) * kNB;
  double acc[4][4] = {};
  tile_product<true>(tile, n, dinv + static_cast<int64_t>(k) * kNB * kNB, kNB, kNB, acc, sa, sb);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int c = 0; c < 4; ++c) tile[static_cast<int64_t>(ty * 4 + m) * n + tx * 4 + c] = acc[m][c];
}

// Trailing update after panel k:  A[i][j] -= L[i][k] L[j][k]^T  for k < j <= i (tiles of 64).
__global__ void __launch_bounds__(256)
trailing_kernel(double* __restrict__ A, int64_t n, int k) {
  TILE_SMEM
  // blockIdx.x enumerates the lower triangle (ti >= tj) of the trailing tile grid
  int t = blockIdx.x;
  int ti = static_cast<int>((sqrt(8.0 * t + 1.0) - 1.0) * 0.5);
  while (ti * (ti + 1) / 2 > t) --ti;
  while ((ti + 1) * (ti + 2) / 2 <= t) ++ti;
  const int tj = t - ti * (ti + 1) / 2;
  const int64_t ri = (static_cast<int64_t>(k) + 1 + ti) * kNB, rj = (static_cast<int64_t>(k) + 1 + tj) * kNB;
  const int64_t ck = static_cast<int64_t>(k) * kNB;
  double acc[4][4] = {};
  tile_product<true>(A + ri * n + ck, n, A + rj * n + ck, n, kNB, acc, sa, sb);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  double* c = A + ri * n + rj;
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int q = 0; q < 4; ++q) c[static_cast<int64_t>(ty * 4 + m) * n + tx * 4 + q] -= acc[m][q];
}

// ---- inverse by recursive doubling -----------------------------------------------------------
__global__ void __launch_bounds__(256)
seed_kernel(double* __restrict__ A, int64_t n, const double* __restrict__ dinv) {
  // diagonal 64-blocks of A <- their inverses
  const int k = blockIdx.x;
  double* blk = A + (static_cast<int64_t>(k) * kNB) * n + static_cast<int64_t>(k) * kNB;
  const double* dk = dinv + static_cast<int64_t>(k) * kNB * kNB;
  for (int e = threadIdx.x; e < kNB * kNB; e += 256) blk[static_cast<int64_t>(e >> 6) * n + (e & 63)] = dk[e];
}

// Level with half-size s (elements): pair p covers [p*2s, p*2s+2s); its A part is the first s
// rows/cols (already inverted: XA), its B part the rest (XB, sB <= s rows), C the block below A.
// step 1:  T = C * XA      (T tile (r,c): reduction over XA rows m >= c only, XA is lower)
__global__ void __launch_bounds__(256)
merge1_kernel(const double* __restrict__ A, int64_t n, int64_t s, double* __restrict__ T) {
  TILE_SMEM
  const int tiles = static_cast<int>(s / kNB);
  const int64_t a0 = static_cast<int64_t>(blockIdx.y) * 2 * s, b0 = a0 + s;
  const int r = blockIdx.x / tiles, c = blockIdx.x % tiles;
  if (b0 + static_cast<int64_t>(r) * kNB >= n) return;
  double acc[4][4] = {};
  const int64_t m0 = static_cast<int64_t>(c) * kNB;
  tile_product<false>(A + (b0 + static_cast<int64_t>(r) * kNB) * n + a0 + m0, n, A + (a0 + m0) * n + a0 + m0, n,
                      static_cast<int>(s - m0), acc, sa, sb);
  // T is packed pair after pair (every earlier pair has s B-rows), rows local to the B part
  double* t = T + static_cast<int64_t>(blockIdx.y) * s * s + static_cast<int64_t>(r) * kNB * s + m0;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int q = 0; q < 4; ++q) t[static_cast<int64_t>(ty * 4 + m) * s + tx * 4 + q] = acc[m][q];
}
// step 2:  C <- -XB * T    (C tile (r,c): reduction over XB columns m <= r only)
__global__ void __launch_bounds__(256)
merge2_kernel(double* __restrict__ A, int64_t n, int64_t s, const double* __restrict__ T) {
  TILE_SMEM
  const int tiles = static_cast<int>(s / kNB);
  const int64_t a0 = static_cast<int64_t>(blockIdx.y) * 2 * s, b0 = a0 + s;
  const int r = blockIdx.x / tiles, c = blockIdx.x % tiles;
  const int64_t row0 = b0 + static_cast<int64_t>(r) * kNB;
  if (row0 >= n) return;
  double acc[4][4] = {};
  tile_product<false>(A + row0 * n + b0, n, T + static_cast<int64_t>(blockIdx.y) * s * s + static_cast<int64_t>(c) * kNB, s,
                      (r + 1) * kNB, acc, sa, sb);
  double* dst = A + row0 * n + a0 + static_cast<int64_t>(c) * kNB;
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int q = 0; q < 4; ++q) dst[static_cast<int64_t>(ty * 4 + m) * n + tx * 4 + q] = -acc[m][q];
}

// U[i][j] = Linv[n-1-i][n-1-j] for i <= j, else 0
__global__ void __launch_bounds__(256)
emit_kernel(const double* __restrict__ A, int64_t n, float* __restrict__ U) {
  int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= n * n) return;
  int64_t i = e / n, j = e % n;
  U[e] = i <= j ? static_cast<float>(A[(n - 1 - i) * n + (n - 1 - j)]) : 0.0f;
}

struct FactorLayout { size_t a_off, t_off, dinv_off, stats_off, total; };
FactorLayout factor_layout(int64_t n) {
  FactorLayout L;
  size_t off = 0;
  L.a_off = off;     off += round_up(static_cast<size_t>(n) * n * 8, 256);
  L.t_off = off;     off += round_up(static_cast<size_t>(n) * (n / 2 + kNB) * 8, 256);
  L.dinv_off = off;  off += round_up(static_cast<size_t>(n) * kNB * 8, 256);
  L.stats_off = off; off += 256;
  L.total = off;
  return L;
}

}  // namespace

size_t factor_workspace_bytes(int64_t n) { return factor_layout(n).total; }

int factor_launch(const float* H, int64_t n, float percdamp, float* U, int* status_dev, void* workspace,
                  cudaStream_t st) {
  FactorLayout Lo = factor_layout(n);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  double* A = reinterpret_cast<double*>(ws + Lo.a_off);
  double* T = reinterpret_cast<double*>(ws + Lo.t_off);
  double* dinv = reinterpret_cast<double*>(ws + Lo.dinv_off);
  double* stats = reinterpret_cast<double*>(ws + Lo.stats_off);
  const int nb = static_cast<int>(n / kNB);
  const unsigned eb = static_cast<unsigned>((n * n + 255) / 256);

  damp_kernel<<<1, 256, 0, st>>>(H, n, static_cast<double>(percdamp), stats);
  build_kernel<<<eb, 256, 0, st>>>(H, n, stats, A);
  for (int k = 0; k < nb; ++k) {
    potrf_kernel<<<1, 256, 0, st>>>(A, n, k, dinv, status_dev);
    const int m = nb - k - 1;
    if (m > 0) {
      panel_kernel<<<m, 256, 0, st>>>(A, n, k, dinv);
      trailing_kernel<<<m * (m + 1) / 2, 256, 0, st>>>(A, n, k);
    }
  }
  seed_kernel<<<nb, 256, 0, st>>>(A, n, dinv);
  for (int64_t s = kNB; s < n; s *= 2) {
    const unsigned pairs = static_cast<unsigned>((n + 2 * s - 1) / (2 * s));
    const unsigned tiles = static_cast<unsigned>((s / kNB) * (s / kNB));
    merge1_kernel<<<dim3(tiles, pairs), 256, 0, st>>>(A, n, s, T);
    merge2_kernel<<<dim3(tiles, pairs), 256, 0, st>>>(A, n, s, T);
  }
  emit_kernel<<<eb, 256, 0, st>>>(A, n, U);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
