// Tensor-core kernels (tcgen05 MMA, TMEM accumulators, TMA-fed shared-memory ring):
//   * calibration Hessian  H += 2 X^T X  (paper Section 4.4; Section 2.2) as a symmetric
//     rank-k update over the tokens, lower-triangle 256 x 256 output tiles only (a copy kernel
//     mirrors them into the upper triangle afterwards);
//   * the reconstruction-error contraction of  1/2 trace(D H D^T) = 1/2 sum(H .* D^T D)
//     (Section 3.3, Eq. 1): D^T D is the same kind of symmetric product, over the rows of D, and
//     the sum against the fp32 H is taken in the epilogue, so H is never rounded.
// One CTA owns a 256 x 256 output tile as two 128 x 256 fp32 accumulators filling all 512
// TMEM columns.  Warp 0 feeds the ring with TMA, one thread of warp 1 issues the MMAs, warps
// 2..5 drain the accumulators.  All CTAs sweep the reduction dimension from the start at the
// same rate, so the operand window they share stays resident in L2.
#include <cuda_bf16.h>

#include "umma.cuh"

namespace adadim {

// ---------------------------------------------------------------------------------------------
// host: tensor maps
// ---------------------------------------------------------------------------------------------
namespace {
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = []() -> EncodeTiledFn {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return nullptr;
    if (q != cudaDriverEntryPointSuccess) return nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}
}  // namespace

int make_tmap_bf16(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                   uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return ADADIM_ERR_CUDA;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {64, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ADADIM_OK : ADADIM_ERR_CUDA;
}

int make_tmap_f32(CUtensorMap* map, const void* base, uint64_t inner, uint64_t rows, uint64_t pitch_bytes,
                  uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr) return ADADIM_ERR_CUDA;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {32, box_rows};
  cuuint32_t estr[2] = {1, 1};
  CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? ADADIM_OK : ADADIM_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// device
// ---------------------------------------------------------------------------------------------
namespace {

enum class Mode { kHessian, kGram };

struct TcParams {
  int num_tiles;            // output tiles (256 x 256) to process
  int num_k;                // 64-deep reduction steps per tile
  int k_chunk;              // steps accumulated in TMEM before the accumulators are drained
  int* status_dev;
  // Hessian
  float* H;
  int64_t in;               // H is [in][in]; also the column count of D
  // Gram (scorer): tiles [0, tiles_per_dim) belong to the first D, the rest to the second
  int tiles_per_dim;
  double* partial;          // [num_tiles][2 halves][4 warps]
};

constexpr int kKT = 64;                       // reduction depth of one ring stage
constexpr int kTcThreads = 192;
constexpr uint32_t kOperandBytes = 256 * kKT * 2;   // one 256-wide bf16 operand slab per stage
constexpr uint32_t kOutChunk = 32 * 32 * 4;          // one epilogue warp's staging tile: 32 rows x 32 fp32 columns

template <Mode MODE> struct TcCfg;
template <> struct TcCfg<Mode::kHessian> { static constexpr int NB = 1, STAGES = 3; static constexpr bool MN = true; };
template <> struct TcCfg<Mode::kGram>    { static constexpr int NB = 1, STAGES = 3; static constexpr bool MN = true; };

template <Mode MODE>
constexpr size_t tc_smem_bytes() {
  return static_cast<size_t>(TcCfg<MODE>::STAGES) * (1 + TcCfg<MODE>::NB) * kOperandBytes + 4 * kOutChunk + 1024 + 256;
}

__device__ __forceinline__ void tri_coords(int t, int& rb, int& cb) {
  int r = static_cast<int>((sqrt(8.0 * t + 1.0) - 1.0) * 0.5);
  while (r * (r + 1) / 2 > t) --r;
  while ((r + 1) * (r + 2) / 2 <= t) ++r;
  rb = r;
  cb = t - r * (r + 1) / 2;
}

template <Mode MODE>
__global__ void __launch_bounds__(kTcThreads, 1)
tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
          const __grid_constant__ CUtensorMap tmB1, const TcParams p) {
  using Cfg = TcCfg<MODE>;
  constexpr int NB = Cfg::NB, STAGES = Cfg::STAGES;
  constexpr uint32_t STAGE_BYTES = (1 + NB) * kOperandBytes;

  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* out_smem = smem + STAGES * STAGE_BYTES;     // [4 warps][32 rows][128 B], 128-byte swizzle (Hessian drains)
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_smem + 4 * kOutChunk);
  uint64_t* full = bars;                   // [STAGES] TMA -> MMA
  uint64_t* empty = bars + STAGES;         // [STAGES] MMA -> TMA
  uint64_t* acc_full = bars + 2 * STAGES;  // MMA -> epilogue
  uint64_t* acc_empty = acc_full + 1;      // epilogue -> MMA
  uint64_t* drain = acc_full + 2;          // used only when a wait ran out
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_full + 3);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // a kernel launched behind this one with programmatic serialization may be scheduled from now on
  // (it waits for this grid's completion itself before it reads what this grid writes)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    ptx::mbar_init(acc_full, 1);
    ptx::mbar_init(acc_empty, 4);
    ptx::mbar_init(drain, 1);
    *dead = 0;
    ptx::fence_mbar_init();
    ptx::tma_prefetch_desc(&tmA);
    ptx::tma_prefetch_desc(&tmB0);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_slot, 512);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before_sync();
  __syncthreads();
  ptx::tc_fence_after_sync();
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      int stage = 0;
      uint32_t phase = 0;
      int last_phase[STAGES];
      for (int s = 0; s < STAGES; ++s) last_phase[s] = -1;
      // The scorer's launch is scheduled while the kernel that writes its operands is finishing
      // (the set-up above overlaps that kernel's tail); the operands are read only from here on.
      // The H read by the epilogue and everything else this grid touches is older than that kernel.
      asm volatile("griddepcontrol.wait;" ::: "memory");
      for (int t = blockIdx.x; t < p.num_tiles && !*dead; t += gridDim.x) {
        int rb, cb;
        const int which = MODE == Mode::kGram ? t / p.tiles_per_dim : 0;     // which stacked matrix
        tri_coords(MODE == Mode::kGram ? t % p.tiles_per_dim : t, rb, cb);
        const CUtensorMap* tm = which == 0 ? &tmA : &tmB0;
        const bool shared_operand = rb == cb;                              // B is A on the diagonal
        for (int k = 0; k < p.num_k; ++k) {
          if (!ptx::mbar_wait(&empty[stage], phase ^ 1u, dead, p.status_dev)) break;
          uint8_t* a_dst = smem + stage * STAGE_BYTES;
          uint8_t* b_dst = a_dst + kOperandBytes;
          ptx::mbar_arrive_expect_tx(&full[stage], shared_operand ? kOperandBytes : STAGE_BYTES);
          last_phase[stage] = static_cast<int>(phase);
          // the matrix is [tokens][in]: boxes of 64 channels x 64 tokens, channels contiguous (MN-major)
#pragma unroll
          for (int j = 0; j < 4; ++j)
            ptx::tma_load_2d(a_dst + j * (kKT * 128), tm, rb * 256 + j * 64, k * kKT, &full[stage]);
          if (!shared_operand) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
              ptx::tma_load_2d(b_dst + j * (kKT * 128), tm, cb * 256 + j * 64, k * kKT, &full[stage]);
          }
          if (++stage == STAGES) { stage = 0; phase ^= 1u; }
        }
      }
      if (*dead) {
        // a wait ran out somewhere: let the copies already issued land before shared memory goes away
        for (int s = 0; s < STAGES; ++s) {
          if (last_phase[s] < 0) continue;
          const long long t0 = clock64();
          while (!ptx::mbar_try_wait(&full[s], static_cast<uint32_t>(last_phase[s])) && clock64() - t0 < ptx::kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      constexpr uint32_t idesc = ptx::idesc_bf16(128, 256, Cfg::MN, Cfg::MN);
      // MN-major: 64-channel blocks are kKT*128 bytes apart (LBO), 8-token groups 1024 bytes (SBO).
      // K-major: 8-row groups are 1024 bytes apart (SBO); LBO is not used with a 128-byte swizzle.
      constexpr uint64_t desc = Cfg::MN ? ptx::smem_desc_sw128(kKT * 128, 1024) : ptx::smem_desc_sw128(16, 1024);
      constexpr uint32_t a_half = Cfg::MN ? 2 * kKT * 128 : 128 * 128;   // bytes between the two 128-row halves of A
      constexpr uint32_t k16_step = Cfg::MN ? 16 * 128 : 32;             // bytes per 16 reduction elements
      int stage = 0;
      uint32_t phase = 0, acc_phase = 0;
      for (int t = blockIdx.x; t < p.num_tiles && !*dead; t += gridDim.x) {
        int rb, cb;
        tri_coords(MODE == Mode::kGram ? t % p.tiles_per_dim : t, rb, cb);
        const bool shared_operand = rb == cb;
        bool ok = true;
        for (int kc = 0; kc < p.num_k && ok; kc += p.k_chunk) {
          if (!ptx::mbar_wait(acc_empty, acc_phase ^ 1u, dead, p.status_dev)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const int kend = min(kc + p.k_chunk, p.num_k);
          for (int k = kc; k < kend; ++k) {
            if (!ptx::mbar_wait(&full[stage], phase, dead, p.status_dev)) { ok = false; break; }
            ptx::tc_fence_after_sync();
            const uint32_t a_addr = ptx::smem_addr(smem + stage * STAGE_BYTES);
            const uint32_t b_addr = shared_operand ? a_addr : a_addr + kOperandBytes;
#pragma unroll
            for (int k16 = 0; k16 < kKT / 16; ++k16) {
#pragma unroll
              for (int a = 0; a < 2; ++a) {
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                  ptx::mma_f16(tmem_base + a * 256,
                               ptx::with_start(desc, a_addr + a * a_half + k16 * k16_step),
                               ptx::with_start(desc, b_addr + b * kOperandBytes + k16 * k16_step),
                               idesc, ((k - kc) | k16 | b) != 0);
                }
              }
            }
            ptx::mma_commit(&empty[stage]);
            if (++stage == STAGES) { stage = 0; phase ^= 1u; }
          }
          if (!ok) break;
          ptx::mma_commit(acc_full);
          acc_phase ^= 1u;
        }
        if (!ok) break;
      }
      if (*dead) {
        ptx::mma_commit(drain);
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(drain, 0) && clock64() - t0 < ptx::kWaitLimit) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ epilogue (warps 2..5)
    const int q = warp & 3;                       // TMEM lane quadrant this warp may read
    uint32_t acc_phase = 0;
    uint8_t* stage_tile = out_smem + q * kOutChunk;
    uint8_t* my_row = stage_tile + lane * 128;    // this lane's row of the staging tile
    for (int t = blockIdx.x; t < p.num_tiles; t += gridDim.x) {
      int rb, cb;
      tri_coords(MODE == Mode::kGram ? t % p.tiles_per_dim : t, rb, cb);
      bool live = true;
      for (int kc = 0; kc < p.num_k; kc += p.k_chunk) {
      // Scorer: the H values of the first 32-column chunk are fetched BEFORE the accumulators are
      // waited for, and every later chunk's while the one before it is being used, so the tensor
      // pipe (which idles while its only accumulator set is drained) waits for one TMEM read and
      // 32 multiply-adds per chunk instead of a round trip to L2 each time.
      float4 h0[8], h1[8];
      auto load_h = [&](int idx, float4 (&h)[8]) {
        const int64_t i = static_cast<int64_t>(rb) * 256 + (idx >> 3) * 128 + q * 32 + lane;
        const int64_t j0 = static_cast<int64_t>(cb) * 256 + (idx & 7) * 32;
        const float* hrow = p.H + i * p.in + j0;
#pragma unroll
        for (int k4 = 0; k4 < 8; ++k4)
          h[k4] = i < p.in && j0 + k4 * 4 < p.in ? *reinterpret_cast<const float4*>(hrow + k4 * 4) : make_float4(0.f, 0.f, 0.f, 0.f);
      };
      if (MODE == Mode::kGram) load_h(0, h0);
      live = ptx::mbar_wait(acc_full, acc_phase, dead, p.status_dev);
      if (!live) break;
      ptx::tc_fence_after_sync();
      // The adds of the previous drain went to the same elements of H: they must be complete
      // before this drain's are issued, or the order of the two roundings would not be fixed.
      if (MODE == Mode::kHessian) {
        if (lane == 0) ptx::bulk_wait_all();
        __syncwarp();
      }
      double part[2] = {0.0, 0.0};
      if (MODE == Mode::kGram) {
        // sum of H .* (D^T D) over this warp's rows of the tile; tiles below the diagonal stand for
        // their mirror image too (accumulator entries outside the matrix are zero)
        auto use_h = [&](int idx, const float4 (&h)[8]) {
          float v[32];
          ptx::tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + (idx >> 3) * 256 + (idx & 7) * 32, v);
          float acc = 0.0f;
#pragma unroll
          for (int k4 = 0; k4 < 8; ++k4) {
            acc = fmaf(h[k4].x, v[k4 * 4 + 0], acc); acc = fmaf(h[k4].y, v[k4 * 4 + 1], acc);
            acc = fmaf(h[k4].z, v[k4 * 4 + 2], acc); acc = fmaf(h[k4].w, v[k4 * 4 + 3], acc);
          }
          part[idx >> 3] += static_cast<double>(acc) * (rb == cb ? 1.0 : 2.0);
        };
#pragma unroll 1
        for (int idx = 0; idx < 16; idx += 2) {
          load_h(idx + 1, h1);
          use_h(idx, h0);
          if (idx + 2 < 16) load_h(idx + 2, h0);
          use_h(idx + 1, h1);
        }
      }
#pragma unroll 1
      for (int a = 0; a < (MODE == Mode::kGram ? 0 : 2); ++a) {
        const int64_t i = static_cast<int64_t>(rb) * 256 + a * 128 + q * 32 + lane;
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
          float v[32];
          ptx::tmem_ld32(tmem_base + (static_cast<uint32_t>(q * 32) << 16) + a * 256 + c * 32, v);
          const int64_t j0 = static_cast<int64_t>(cb) * 256 + c * 32;
          if (MODE == Mode::kHessian) {
            // H += 2 acc as an element-wise add done by the memory system: the doubled values go
            // to a swizzled staging tile and from there into H, 32 rows x 32 columns at a time
            // (the part of a tile outside the matrix is not written).  H is never read here.
            const int64_t i0 = static_cast<int64_t>(rb) * 256 + a * 128 + q * 32;
            if (i0 < p.in && j0 < p.in) {
              if (lane == 0) ptx::bulk_wait_read();   // the previous add has finished reading the staging tile
              __syncwarp();
#pragma unroll
              for (int k4 = 0; k4 < 8; ++k4) {        // 16-byte chunk k4 of the row sits at chunk k4 ^ (row % 8)
                float4 x;
                x.x = 2.0f * v[k4 * 4 + 0]; x.y = 2.0f * v[k4 * 4 + 1];
                x.z = 2.0f * v[k4 * 4 + 2]; x.w = 2.0f * v[k4 * 4 + 3];
                *reinterpret_cast<float4*>(my_row + ((k4 ^ (lane & 7)) << 4)) = x;
              }
              ptx::fence_proxy_async();
              __syncwarp();
              if (lane == 0) {
                ptx::tma_reduce_add_2d(&tmB1, static_cast<int>(j0), static_cast<int>(i0), stage_tile);
                ptx::bulk_commit();
              }
            }
          }
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(acc_empty);
      if (MODE == Mode::kGram) {
        // one partial per (tile, 128-row half, warp): no cross-warp synchronisation needed
#pragma unroll
        for (int a = 0; a < 2; ++a) {
          double s = part[a];
          for (int m = 16; m > 0; m >>= 1) s += __shfl_xor_sync(0xffffffffu, s, m);
          if (lane == 0) p.partial[(static_cast<int64_t>(t) * 2 + a) * 4 + q] = s;
        }
      }
      acc_phase ^= 1u;
      }
      if (!live) break;
    }
    if (MODE == Mode::kHessian && lane == 0) ptx::bulk_wait_all();   // every add is complete before the CTA ends
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Copies the strictly-lower 256-blocks of H into the upper triangle: H[j][i] = H[i][j] wherever
// i / 256 > j / 256 (diagonal 256-blocks are computed in full by the tile kernel).
__global__ void __launch_bounds__(256)
mirror_kernel(float* __restrict__ H, int64_t n) {
  __shared__ float tile[32][33];
  const int bi = blockIdx.y, bj = blockIdx.x;               // 32 x 32 tiles; source tile (bi, bj)
  if ((bi >> 3) <= (bj >> 3)) return;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;   // 32 x 8
  for (int r = ty; r < 32; r += 8) {
    int64_t i = static_cast<int64_t>(bi) * 32 + r, j = static_cast<int64_t>(bj) * 32 + tx;
    tile[r][tx] = (i < n && j < n) ? H[i * n + j] : 0.0f;
  }
  __syncthreads();
  for (int r = ty; r < 32; r += 8) {
    int64_t j = static_cast<int64_t>(bj) * 32 + r, i = static_cast<int64_t>(bi) * 32 + tx;
    if (i < n && j < n) H[j * n + i] = tile[tx][r];
  }
}

// ---- fp32 activations: plain FFMA kernel (small calibration sets; keeps full fp32 products) ----
__global__ void __launch_bounds__(256)
hessian_f32_kernel(const float* __restrict__ X, int64_t n_tokens, int64_t in, int64_t ldx, float* __restrict__ H) {
  // one 64 x 64 lower-triangle tile of H per CTA, 4 x 4 outputs per thread
  __shared__ float sa[16][64 + 4];
  __shared__ float sb[16][64 + 4];
  int rb, cb;
  tri_coords(blockIdx.x, rb, cb);
  const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
  float acc[4][4] = {};
  for (int64_t t0 = 0; t0 < n_tokens; t0 += 16) {
    for (int e = threadIdx.x; e < 16 * 64; e += 256) {
      int tt = e >> 6, c = e & 63;
      int64_t tok = t0 + tt;
      int64_t ia = static_cast<int64_t>(rb) * 64 + c, ib = static_cast<int64_t>(cb) * 64 + c;
      sa[tt][c] = (tok < n_tokens && ia < in) ? X[tok * ldx + ia] : 0.0f;
      sb[tt][c] = (tok < n_tokens && ib < in) ? X[tok * ldx + ib] : 0.0f;
    }
    __syncthreads();
#pragma unroll
    for (int tt = 0; tt < 16; ++tt) {
      float a[4], b[4];
#pragma unroll
      for (int m = 0; m < 4; ++m) { a[m] = sa[tt][ty * 4 + m]; b[m] = sb[tt][tx * 4 + m]; }
#pragma unroll
      for (int m = 0; m < 4; ++m)
#pragma unroll
        for (int n = 0; n < 4; ++n) acc[m][n] = fmaf(a[m], b[n], acc[m][n]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int m = 0; m < 4; ++m)
#pragma unroll
    for (int n = 0; n < 4; ++n) {
      int64_t i = static_cast<int64_t>(rb) * 64 + ty * 4 + m, j = static_cast<int64_t>(cb) * 64 + tx * 4 + n;
      if (i < in && j < in) {
        if (rb != cb) {
          H[i * in + j] += 2.0f * acc[m][n];
          H[j * in + i] += 2.0f * acc[m][n];
        } else {
          H[i * in + j] += 2.0f * acc[m][n];     // the diagonal tile computes its full square
        }
      }
    }
}

template <Mode MODE>
int tc_launch(const CUtensorMap& a, const CUtensorMap& b0, const CUtensorMap& b1, const TcParams& p, cudaStream_t st,
              bool chained = false) {
  static int sm_count = 0;
  if (sm_count == 0) {
    int dev = 0;
    ADADIM_CUDA_TRY(cudaGetDevice(&dev));
    ADADIM_CUDA_TRY(cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, dev));
  }
  ADADIM_CUDA_TRY(cudaFuncSetAttribute(tc_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(tc_smem_bytes<MODE>())));
  int grid = p.num_tiles < sm_count ? p.num_tiles : sm_count;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(static_cast<unsigned>(grid));
  cfg.blockDim = dim3(kTcThreads);
  cfg.dynamicSmemBytes = tc_smem_bytes<MODE>();
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = chained ? 1 : 0;                      // chained: may start while the launch before it in the stream finishes
  ADADIM_CUDA_TRY(cudaLaunchKernelEx(&cfg, tc_kernel<MODE>, a, b0, b1, p));
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace

int hessian_bf16_launch(const void* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, int* status_dev,
                        cudaStream_t st) {
  CUtensorMap tm;
  int rc = make_tmap_bf16(&tm, X, static_cast<uint64_t>(in), static_cast<uint64_t>(n_tokens),
                          static_cast<uint64_t>(ldx) * 2, kKT);
  if (rc != ADADIM_OK) return rc;
  TcParams p = {};
  const int nblk = static_cast<int>((in + 255) / 256);
  p.num_tiles = nblk * (nblk + 1) / 2;
  p.num_k = static_cast<int>((n_tokens + kKT - 1) / kKT);
  // The tensor core adds each 16-token product into the fp32 accumulator with truncation, a
  // bias that grows with the number of additions (about 5e-8 relative per addition, measured);
  // draining the accumulators into H every 8192 tokens keeps it near 3e-5.
  p.k_chunk = 8192 / kKT;
  p.status_dev = status_dev;
  p.H = H;
  p.in = in;
  CUtensorMap th;                                      // H itself, for the element-wise adds of the drains
  rc = make_tmap_f32(&th, H, static_cast<uint64_t>(in), static_cast<uint64_t>(in), static_cast<uint64_t>(in) * 4, 32);
  if (rc != ADADIM_OK) return rc;
  rc = tc_launch<Mode::kHessian>(tm, tm, th, p, st);
  if (rc != ADADIM_OK) return rc;
  const unsigned nt = static_cast<unsigned>((in + 31) / 32);
  if (nblk > 1) mirror_kernel<<<dim3(nt, nt), 256, 0, st>>>(H, in);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

// ---- fp32 activations on the tensor cores ---------------------------------------------------------
// A binary32 number is the exact sum of three bf16 numbers (8 significant bits each).  With
// Z = [X_hi | X_mid | X_lo] (the channel axis three times as wide) the bf16 kernel above forms
// 2 Z^T Z, whose nine in x in blocks are the products 2 X_p^T X_q of the pieces; H gets the six
// blocks that matter (p + q <= 2; the other three are below 2^-24 of the result), smallest first.
// Every product of two pieces is exact in the tensor core; what is rounded is the fp32 accumulation,
// as for bf16 activations.
namespace {
__global__ void __launch_bounds__(256)
split3_kernel(const float* __restrict__ X, int64_t n_tokens, int64_t in, int64_t ldx, __nv_bfloat16* __restrict__ Z) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= n_tokens * in) return;
  const int64_t t = e / in, i = e % in;
  const float x = X[t * ldx + i];
  const __nv_bfloat16 h = __float2bfloat16_rn(x);
  const float r1 = x - __bfloat162float(h);                  // exact
  const __nv_bfloat16 m = __float2bfloat16_rn(r1);
  const float r2 = r1 - __bfloat162float(m);                 // exact
  __nv_bfloat16* z = Z + t * 3 * in + i;
  z[0] = h;
  z[in] = m;
  z[2 * in] = __float2bfloat16_rn(r2);
}
__global__ void __launch_bounds__(256)
combine3_kernel(const float* __restrict__ Hp, int64_t in, float* __restrict__ H) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (e >= in * in) return;
  const int64_t i = e / in, j = e % in, n3 = 3 * in;
  auto blk = [&](int p, int q) { return Hp[(p * in + i) * n3 + q * in + j]; };
  const float small = (blk(0, 2) + blk(2, 0)) + blk(1, 1);
  const float mid = blk(0, 1) + blk(1, 0);
  H[e] += (small + mid) + blk(0, 0);
}
}  // namespace

size_t hessian_f32_tc_workspace_bytes(int64_t n_tokens, int64_t in) {
  return round_up(static_cast<size_t>(n_tokens) * 3 * in * 2, 256) + round_up(static_cast<size_t>(9) * in * in * 4, 256);
}

int hessian_f32_tc_launch(const float* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, int* status_dev,
                          void* workspace, cudaStream_t st) {
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  __nv_bfloat16* Z = reinterpret_cast<__nv_bfloat16*>(ws);
  float* Hp = reinterpret_cast<float*>(ws + round_up(static_cast<size_t>(n_tokens) * 3 * in * 2, 256));
  ADADIM_CUDA_TRY(cudaMemsetAsync(Hp, 0, static_cast<size_t>(9) * in * in * 4, st));
  split3_kernel<<<static_cast<unsigned>((n_tokens * in + 255) / 256), 256, 0, st>>>(X, n_tokens, in, ldx, Z);
  const int rc = hessian_bf16_launch(Z, n_tokens, 3 * in, 3 * in, Hp, status_dev, st);
  if (rc != ADADIM_OK) return rc;
  combine3_kernel<<<static_cast<unsigned>((in * in + 255) / 256), 256, 0, st>>>(Hp, in, H);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

int hessian_f32_launch(const float* X, int64_t n_tokens, int64_t in, int64_t ldx, float* H, cudaStream_t st) {
  const int nblk = static_cast<int>((in + 63) / 64);
  hessian_f32_kernel<<<nblk * (nblk + 1) / 2, 256, 0, st>>>(X, n_tokens, in, ldx, H);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

// Scorer contraction: for each stacked D (bf16 [rows][in]) the lower-triangle tiles of D^T D are
// formed like the Hessian's and dotted with the fp32 H in the epilogue;
// partial[tile][half][warp] holds each epilogue warp's share of sum(H .* D^T D).
int gram_launch(const __nv_bfloat16* D0, const __nv_bfloat16* D1, int64_t rows, int64_t in, const float* H,
                double* partial, int* status_dev, cudaStream_t st) {
  CUtensorMap t0, t1;
  int rc = make_tmap_bf16(&t0, D0, static_cast<uint64_t>(in), static_cast<uint64_t>(rows), static_cast<uint64_t>(in) * 2, kKT);
  if (rc != ADADIM_OK) return rc;
  rc = make_tmap_bf16(&t1, D1 != nullptr ? D1 : D0, static_cast<uint64_t>(in), static_cast<uint64_t>(rows),
                      static_cast<uint64_t>(in) * 2, kKT);
  if (rc != ADADIM_OK) return rc;
  TcParams p = {};
  const int nblk = static_cast<int>((in + 255) / 256);
  p.tiles_per_dim = nblk * (nblk + 1) / 2;
  p.num_tiles = p.tiles_per_dim * (D1 != nullptr ? 2 : 1);
  p.num_k = static_cast<int>((rows + kKT - 1) / kKT);
  p.k_chunk = p.num_k;
  p.status_dev = status_dev;
  p.H = const_cast<float*>(H);        // read only in this mode
  p.in = in;
  p.partial = partial;
  return tc_launch<Mode::kGram>(t0, t1, t0, p, st, true);   // behind the kernel that writes D0, D1
}

int gram_tiles(int64_t in) {
  const int nblk = static_cast<int>((in + 255) / 256);
  return nblk * (nblk + 1) / 2;
}

}  // namespace adadim
