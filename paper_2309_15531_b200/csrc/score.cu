// Reconstruction-error scorer and selection (paper Section 3.3, Eq. 1; Appendix B):
//   E_dim = || X (W - Q_dim)^T ||_F^2 = 1/2 trace(D_dim H D_dim^T),  D_dim = W - Q_dim,
//   chosen = IC iff E_ic < E_oc.
// Steps: (1) D for each dimension, rounded to bf16;
// (2) tensor-core symmetric product D^T D on lower-triangle tiles with sum(H .* D^T D) taken per
//     tile against the fp32 H (tc_gemm.cu): half the multiplications of D H, and H stays exact;
// (3) fixed-order reduction of the per-tile partials and the comparison.
#include <cuda_bf16.h>

#include "common.cuh"

namespace adadim {

int gram_launch(const __nv_bfloat16* D0, const __nv_bfloat16* D1, int64_t rows, int64_t in, const float* H,
                double* partial, int* status_dev, cudaStream_t st);
int gram_tiles(int64_t in);

namespace {

// One thread dequantizes 32 consecutive codes of one row (BITS words) and writes W - Q as bf16.
template <typename T, int BITS>
__global__ void __launch_bounds__(256)
diff_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, int group, bool is_ic,
            adadim_qtensor q, __nv_bfloat16* __restrict__ D) {
  const int64_t chunks = in / 32;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= out * chunks) return;
  const int64_t row = t / chunks, col0 = (t % chunks) * 32;
  const uint32_t* src = q.codes + row * (in * BITS / 32) + col0 * BITS / 32;
  uint32_t wds[BITS + 1];
#pragma unroll
  for (int k = 0; k < BITS; ++k) wds[k] = src[k];
  wds[BITS] = 0;
  float s_oc = 0.f, z_oc = 0.f;
  if (!is_ic) {
    int64_t idx = row * (in / group) + col0 / group;        // group >= 32: one group per chunk
    s_oc = __half2float(__ushort_as_half(q.scales[idx]));
    z_oc = __half2float(__ushort_as_half(q.zeros[idx]));
  }
  const uint16_t* sc = q.scales + (row / group) * in + col0;
  const uint16_t* zr = q.zeros + (row / group) * in + col0;
#pragma unroll
  for (int v8 = 0; v8 < 4; ++v8) {
    float w[8];
    load8(W + row * ldw + col0 + v8 * 8, w);
    __nv_bfloat162 o[4];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const int kk = v8 * 8 + k;
      const int bit = kk * BITS, wi = bit >> 5, sh = bit & 31;
      uint32_t c = wds[wi] >> sh;
      if (sh + BITS > 32) c |= wds[wi + 1] << (32 - sh);
      c &= (1u << BITS) - 1u;
      float s = s_oc, z = z_oc;
      if (is_ic) {
        s = __half2float(__ushort_as_half(sc[kk]));
        z = __half2float(__ushort_as_half(zr[kk]));
      }
      float qv = __fmul_rn(s, static_cast<float>(c) - z);   // exact: 11-bit scale times a small integer
      float d = __fsub_rn(w[k], qv);
      if (k & 1) o[k >> 1].y = __float2bfloat16_rn(d); else o[k >> 1].x = __float2bfloat16_rn(d);
    }
    *reinterpret_cast<uint4*>(D + row * in + col0 + v8 * 8) = *reinterpret_cast<uint4*>(o);
  }
}

// partial is [tiles][2 halves][4]; tiles below `tiles_first` belong to the first scored
// dimension.  Sums are taken in a fixed order.
__global__ void __launch_bounds__(256)
finalize_kernel(const double* __restrict__ partial, int num_tiles, int tiles_first,
                int first_dim, bool have_second, double* err, int* chosen, int* status_dev) {
  __shared__ double red[2][256];
  double acc[2] = {0.0, 0.0};
  for (int e = threadIdx.x; e < num_tiles * 2; e += 256) {
    const int tile = e >> 1;
    const double* pp = partial + static_cast<int64_t>(e) * 4;
    double s = (pp[0] + pp[1]) + (pp[2] + pp[3]);
    acc[tile < tiles_first ? 0 : 1] += s;
  }
  red[0][threadIdx.x] = acc[0];
  red[1][threadIdx.x] = acc[1];
  __syncthreads();
  for (int m = 128; m > 0; m >>= 1) {
    if (threadIdx.x < m) {
      red[0][threadIdx.x] += red[0][threadIdx.x + m];
      red[1][threadIdx.x] += red[1][threadIdx.x + m];
    }
    __syncthreads();
  }
  if (threadIdx.x == 0) {
    const double inf = __longlong_as_double(0x7ff0000000000000LL);
    double e[2] = {inf, inf};
    e[first_dim] = 0.5 * red[0][0];
    if (have_second) e[1 - first_dim] = 0.5 * red[1][0];
    err[0] = e[0];
    err[1] = e[1];
    int pick = ADADIM_DIM_OC;
    if (e[0] != e[0] || e[1] != e[1]) report(status_dev, ADADIM_ERR_NUMERIC);
    else if (e[1] < e[0]) pick = ADADIM_DIM_IC;
    *chosen = pick;
  }
}

template <typename T>
void diff_launch(const T* W, int64_t out, int64_t in, int64_t ldw, int bits, int group, bool is_ic,
                 const adadim_qtensor& q, __nv_bfloat16* D, cudaStream_t st) {
  int64_t n = out * (in / 32);
  unsigned blocks = static_cast<unsigned>((n + 255) / 256);
  if (bits == 3) diff_kernel<T, 3><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, is_ic, q, D);
  else diff_kernel<T, 4><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, is_ic, q, D);
}

struct ScoreLayout {
  size_t d_off, part_off, total;
};
ScoreLayout score_layout(int64_t out, int64_t in) {
  ScoreLayout L;
  size_t off = 0;
  L.d_off = off;    off += round_up(static_cast<size_t>(2 * out) * in * 2, 256);
  L.part_off = off; off += round_up(static_cast<size_t>(2 * gram_tiles(in)) * 8 * sizeof(double), 256);
  L.total = off;
  return L;
}

}  // namespace

size_t score_workspace_bytes(int64_t out, int64_t in) { return score_layout(out, in).total; }

int score_launch(const void* W, int wdtype, int64_t out, int64_t in, int64_t ldw, const float* H, int bits, int group,
                 const adadim_qtensor* q_oc, const adadim_qtensor* q_ic, double* err, int* chosen, int* status_dev,
                 void* workspace, cudaStream_t st) {
  ScoreLayout L = score_layout(out, in);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  __nv_bfloat16* D = reinterpret_cast<__nv_bfloat16*>(ws + L.d_off);
  double* partial = reinterpret_cast<double*>(ws + L.part_off);

  const adadim_qtensor* qs[2] = {q_oc, q_ic};
  const int first_dim = q_oc != nullptr ? ADADIM_DIM_OC : ADADIM_DIM_IC;
  const bool have_second = q_oc != nullptr && q_ic != nullptr;
  int64_t rows = 0;
  for (int d = 0; d < 2; ++d) {
    if (qs[d] == nullptr) continue;
    __nv_bfloat16* dst = D + rows * in;
    if (wdtype == ADADIM_F16) diff_launch(static_cast<const __half*>(W), out, in, ldw, bits, group, d == 1, *qs[d], dst, st);
    else diff_launch(static_cast<const float*>(W), out, in, ldw, bits, group, d == 1, *qs[d], dst, st);
    rows += out;
  }
  if (cudaGetLastError() != cudaSuccess) return ADADIM_ERR_CUDA;
  int rc = gram_launch(D, have_second ? D + out * in : nullptr, out, in, H, partial, status_dev, st);
  if (rc != ADADIM_OK) return rc;
  const int tiles = gram_tiles(in);
  finalize_kernel<<<1, 256, 0, st>>>(partial, tiles * (have_second ? 2 : 1), tiles, first_dim, have_second, err, chosen,
                                     status_dev);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
