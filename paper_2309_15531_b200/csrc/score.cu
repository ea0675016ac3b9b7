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

// W - Q as bf16 for one or both quantized tensors, from one read of W.  One thread handles
// eight consecutive weights of a row (one 16-byte load and one 16-byte store per output), so
// neighbouring threads touch neighbouring memory.  qa/Da are the per-OC tensor and its output,
// qb/Db the per-IC ones; a null codes pointer skips that side.
template <typename T, int BITS>
__global__ void __launch_bounds__(256)
diff_kernel(const T* __restrict__ W, int64_t out, int64_t in, int64_t ldw, int group,
            adadim_qtensor qa, __nv_bfloat16* __restrict__ Da, adadim_qtensor qb, __nv_bfloat16* __restrict__ Db) {
  const int64_t vecs = in / 8;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  // the product kernel behind this one may be scheduled already: its set-up overlaps this kernel's tail
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (t >= out * vecs) return;
  const int64_t row = t / vecs, col0 = (t % vecs) * 8;
  float w[8];
  load8(W + row * ldw + col0, w);
  // the eight codes start at bit col0*BITS of the row's stream: at most two words
  const int64_t bit0 = col0 * BITS;
  const int64_t word0 = row * (in * BITS / 32) + (bit0 >> 5);
  const int sh0 = static_cast<int>(bit0 & 31);
  const bool two = sh0 + 8 * BITS > 32;
#pragma unroll
  for (int side = 0; side < 2; ++side) {
    const adadim_qtensor& q = side == 0 ? qa : qb;
    if (q.codes == nullptr) continue;
    uint64_t bitsv = q.codes[word0];
    if (two) bitsv |= static_cast<uint64_t>(q.codes[word0 + 1]) << 32;
    bitsv >>= sh0;
    float s[8], z[8];
    if (side == 0) {
      const int64_t idx = row * (in / group) + col0 / group;      // group >= 32: one group per vector
      const float s0 = __half2float(__ushort_as_half(q.scales[idx]));
      const float z0 = __half2float(__ushort_as_half(q.zeros[idx]));
#pragma unroll
      for (int k = 0; k < 8; ++k) { s[k] = s0; z[k] = z0; }
    } else {
      const uint4 sv = *reinterpret_cast<const uint4*>(q.scales + (row / group) * in + col0);
      const uint4 zv = *reinterpret_cast<const uint4*>(q.zeros + (row / group) * in + col0);
      const __half2* sh = reinterpret_cast<const __half2*>(&sv);
      const __half2* zh = reinterpret_cast<const __half2*>(&zv);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        float2 a = __half22float2(sh[k]), b = __half22float2(zh[k]);
        s[2 * k] = a.x; s[2 * k + 1] = a.y; z[2 * k] = b.x; z[2 * k + 1] = b.y;
      }
    }
    __align__(16) __nv_bfloat162 o[4];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
      const uint32_t c = static_cast<uint32_t>(bitsv >> (k * BITS)) & ((1u << BITS) - 1u);
      const float qv = __fmul_rn(s[k], static_cast<float>(c) - z[k]);   // exact: 11-bit scale times a small integer
      const float d = __fsub_rn(w[k], qv);
      if (k & 1) o[k >> 1].y = __float2bfloat16_rn(d); else o[k >> 1].x = __float2bfloat16_rn(d);
    }
    *reinterpret_cast<uint4*>((side == 0 ? Da : Db) + row * in + col0) = *reinterpret_cast<uint4*>(o);
  }
}

// partial is [tiles][2 halves][4]; tiles below `tiles_first` belong to the first scored
// dimension.  Sums are taken in a fixed order.
__global__ void __launch_bounds__(256)
finalize_kernel(const double* partial, int num_tiles, int tiles_first,
                int first_dim, bool have_second, double* err, int* chosen, int* status_dev) {
  __shared__ double red[2][256];
  // launched with programmatic serialization behind the product kernel: wait for its completion here.
  // (`partial` is written by that kernel while this one is already alive, so it is not declared
  // `const __restrict__`: loads through such a pointer may be moved above the wait.)
  asm volatile("griddepcontrol.wait;" ::: "memory");
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
void diff_launch(const T* W, int64_t out, int64_t in, int64_t ldw, int bits, int group, const adadim_qtensor& qa,
                 __nv_bfloat16* Da, const adadim_qtensor& qb, __nv_bfloat16* Db, cudaStream_t st) {
  const int64_t n = out * (in / 8);
  const unsigned blocks = static_cast<unsigned>((n + 255) / 256);
  if (bits == 2) diff_kernel<T, 2><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, qa, Da, qb, Db);
  else if (bits == 3) diff_kernel<T, 3><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, qa, Da, qb, Db);
  else if (bits == 4) diff_kernel<T, 4><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, qa, Da, qb, Db);
  else diff_kernel<T, 8><<<blocks, 256, 0, st>>>(W, out, in, ldw, group, qa, Da, qb, Db);
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

  const int first_dim = q_oc != nullptr ? ADADIM_DIM_OC : ADADIM_DIM_IC;
  const bool have_second = q_oc != nullptr && q_ic != nullptr;
  const adadim_qtensor none = {nullptr, nullptr, nullptr};
  const adadim_qtensor qa = q_oc != nullptr ? *q_oc : none, qb = q_ic != nullptr ? *q_ic : none;
  __nv_bfloat16* Da = D;                                        // first scored dimension first
  __nv_bfloat16* Db = q_oc != nullptr ? D + out * in : D;
  if (wdtype == ADADIM_F16) diff_launch(static_cast<const __half*>(W), out, in, ldw, bits, group, qa, Da, qb, Db, st);
  else diff_launch(static_cast<const float*>(W), out, in, ldw, bits, group, qa, Da, qb, Db, st);
  if (cudaGetLastError() != cudaSuccess) return ADADIM_ERR_CUDA;
  int rc = gram_launch(D, have_second ? D + out * in : nullptr, out, in, H, partial, status_dev, st);
  if (rc != ADADIM_OK) return rc;
  const int tiles = gram_tiles(in);
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(1);
    cfg.blockDim = dim3(256);
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (cudaLaunchKernelEx(&cfg, finalize_kernel, static_cast<const double*>(partial), tiles * (have_second ? 2 : 1), tiles,
                           first_dim, have_second, err, chosen, status_dev) != cudaSuccess)
      return ADADIM_ERR_CUDA;
  }
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
