// GPTQ lazy-batch trailing update on the tensor cores (paper Section 2.2: the rounding error of
// a block of columns is propagated to the columns not yet quantized):
//     W[:, c0:] -= Err[rows,128] * U[i1:i1+128, c0:]
// The update feeds later rounding decisions, so it needs fp32-grade accuracy, and the tensor
// core's fp32 accumulation truncates (a bias of about half an ulp per addition, measured), which
// summed over thousands of columns moved per-IC scales far more than an FFMA chain does.  The
// operands are therefore sliced into three 8-bit fixed-point pieces on a common grid per Err row
// and per U column of the block (x = p0 + p1 + p2, piece k a multiple of grid * 2^-8k).  Every
// bf16 product of two leading pieces is then an integer multiple of one unit with at most 16
// bits, a sum of 128 of them has at most 23 bits, and the accumulation is exact: nothing is
// left to truncate.  The leading products go to one TMEM accumulator, the eight smaller
// products (2^-8 ... 2^-32 of the result) to a second one, and the two are added in binary64 in
// the epilogue.  All nine products are formed: leaving out the three smallest (2^-24 of the
// largest term) was measured to flip a rounding decision now and then on long layers.  The working weights themselves are binary64 (gptq.cu says why): the
// epilogue widens the negated product and hands it to the memory system as an element-wise
// binary64 add, so the SM never reads W.
//
// The 128 x 128 tiles of a launch (128-row blocks of the stacked working weights x 128-column
// tiles) are numbered row block by row block and dealt out in equal contiguous ranges, one per
// CTA, so that a launch fills exactly the SMs it is given; a range may run from one row block
// into the next.  The Err pieces of the current row block (K = 128) stay in shared memory and are
// reloaded when the range crosses into another block; U pieces stream through a ring of 32-row
// slabs; two pairs of TMEM accumulators alternate so the read-modify-write of W of one tile
// overlaps the MMAs of the next.
#include <cuda_bf16.h>

#include "umma.cuh"

namespace adadim {
namespace {

constexpr int kThreads = 320;                      // TMA warp, MMA warp, eight epilogue warps
constexpr uint32_t kAPiece = 128 * 64 * 2;          // one Err piece, one 64-deep half of K: 16 KB
constexpr uint32_t kABytes = 6 * kAPiece;           // 3 pieces x 2 halves
constexpr int kTileN = 128;
constexpr uint32_t kBPiece = kTileN * 32 * 2;       // one U piece, 32 k-rows x 128 columns: 8 KB
constexpr uint32_t kBStage = 3 * kBPiece;           // 24 KB
constexpr int kBStages = 4;
constexpr uint32_t kOutChunk = 32 * 16 * 8;          // one epilogue warp's staging tile: 32 rows x 16 fp64 columns
constexpr size_t kSmemBytes = kABytes + kBStages * kBStage + 8 * kOutChunk + 1024 + 256;

struct TrailParams {
  double* Wc;           // stacked working weights, rows_total x in, in the tiled layout of wc_index()
  int64_t in;
  int64_t c0;           // first column to update
  int i1;               // first row of U's block
  int ntiles;           // 128-column tiles from c0
  int mblocks;          // 128-row blocks of the stacked working weights
  int e_row0;           // first row of this block's error pieces (the pieces are kept in two alternating sets)
  int* status_dev;
};

__global__ void __launch_bounds__(kThreads, 1)
trail_kernel(const __grid_constant__ CUtensorMap tmE0, const __grid_constant__ CUtensorMap tmE1,
             const __grid_constant__ CUtensorMap tmE2, const __grid_constant__ CUtensorMap tmU0,
             const __grid_constant__ CUtensorMap tmU1, const __grid_constant__ CUtensorMap tmU2,
             const TrailParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* a_smem = smem;
  uint8_t* b_smem = smem + kABytes;
  uint8_t* out_smem = b_smem + kBStages * kBStage;  // [8 warps][32 rows][128 B]
  uint64_t* bars = reinterpret_cast<uint64_t*>(out_smem + 8 * kOutChunk);
  uint64_t* a_full = bars;
  uint64_t* a_empty = bars + 15;                    // MMA -> TMA: the Err pieces of a finished row block may be overwritten
  uint64_t* b_full = bars + 1;                      // [kBStages]
  uint64_t* b_empty = b_full + kBStages;            // [kBStages]
  uint64_t* acc_full = b_empty + kBStages;          // [2]
  uint64_t* acc_empty = acc_full + 2;               // [2]
  uint64_t* drain = acc_empty + 2;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* dead = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  // a kernel launched behind this one with programmatic serialization may be scheduled from now
  // on; it still waits for this grid's completion before it reads anything this grid writes
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  // this CTA's tiles: an even share of [0, mblocks * ntiles), tile g = row block g / ntiles, column tile g % ntiles
  const int64_t total = static_cast<int64_t>(p.mblocks) * p.ntiles;
  const int t0 = static_cast<int>(total * blockIdx.x / gridDim.x);
  const int t1 = static_cast<int>(total * (blockIdx.x + 1) / gridDim.x);

  if (threadIdx.x == 0) {
    ptx::mbar_init(a_full, 1);
    ptx::mbar_init(a_empty, 1);
    for (int s = 0; s < kBStages; ++s) { ptx::mbar_init(&b_full[s], 1); ptx::mbar_init(&b_empty[s], 1); }
    for (int s = 0; s < 2; ++s) { ptx::mbar_init(&acc_full[s], 1); ptx::mbar_init(&acc_empty[s], 8); }
    ptx::mbar_init(drain, 1);
    *dead = 0;
    ptx::fence_mbar_init();
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
    if (lane == 0 && t0 < t1) {
      const CUtensorMap* tmE[3] = {&tmE0, &tmE1, &tmE2};
      const CUtensorMap* tmU[3] = {&tmU0, &tmU1, &tmU2};
      int stage = 0;
      uint32_t phase = 0;
      int last_phase[kBStages];
      for (int s = 0; s < kBStages; ++s) last_phase[s] = -1;
      int rb_now = -1, a_loads = 0;
      for (int g = t0; g < t1 && !*dead; ++g) {
        const int rb = g / p.ntiles, t = g % p.ntiles;
        if (rb != rb_now) {
          // Err pieces of the next row block, once the MMAs that read the previous ones are done
          if (a_loads > 0 && !ptx::mbar_wait(a_empty, static_cast<uint32_t>((a_loads - 1) & 1), dead, p.status_dev)) break;
          ptx::mbar_arrive_expect_tx(a_full, kABytes);
          for (int pc = 0; pc < 3; ++pc)
            for (int kh = 0; kh < 2; ++kh)
              ptx::tma_load_2d(a_smem + (pc * 2 + kh) * kAPiece, tmE[pc], kh * 64, p.e_row0 + rb * 128, a_full);
          rb_now = rb;
          ++a_loads;
        }
        const int col = static_cast<int>(p.c0) + t * kTileN;
        for (int kc = 0; kc < 4; ++kc) {
          if (!ptx::mbar_wait(&b_empty[stage], phase ^ 1u, dead, p.status_dev)) break;
          ptx::mbar_arrive_expect_tx(&b_full[stage], kBStage);
          last_phase[stage] = static_cast<int>(phase);
          uint8_t* dst = b_smem + stage * kBStage;
          for (int pc = 0; pc < 3; ++pc)
            for (int j = 0; j < kTileN / 64; ++j)
              ptx::tma_load_2d(dst + pc * kBPiece + j * (32 * 128), tmU[pc], col + j * 64, p.i1 + kc * 32, &b_full[stage]);
          if (++stage == kBStages) { stage = 0; phase ^= 1u; }
        }
      }
      if (*dead) {
        // a wait ran out somewhere: let the copies already issued land before shared memory goes away
        const long long c0 = clock64();
        while (a_loads > 0 && !ptx::mbar_try_wait(a_full, static_cast<uint32_t>((a_loads - 1) & 1)) && clock64() - c0 < ptx::kWaitLimit) {}
        for (int s = 0; s < kBStages; ++s) {
          if (last_phase[s] < 0) continue;
          const long long c1 = clock64();
          while (!ptx::mbar_try_wait(&b_full[s], static_cast<uint32_t>(last_phase[s])) && clock64() - c1 < ptx::kWaitLimit) {}
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0 && t0 < t1) {
      constexpr uint32_t idesc = ptx::idesc_bf16(128, kTileN, false, true);
      constexpr uint64_t adesc = ptx::smem_desc_sw128(16, 1024);          // K-major, 8-row groups 1024 B apart
      constexpr uint64_t bdesc = ptx::smem_desc_sw128(32 * 128, 1024);    // MN-major, 64-column blocks 4 KB apart
      bool ok = true;
      int stage = 0, rb_now = -1, a_seen = 0;
      uint32_t phase = 0, acc_phase[2] = {0, 0};
      for (int g = t0; g < t1 && ok; ++g) {
        const int rb = g / p.ntiles;
        if (rb != rb_now) {
          if (!ptx::mbar_wait(a_full, static_cast<uint32_t>(a_seen & 1), dead, p.status_dev)) break;
          rb_now = rb;
          ++a_seen;
        }
        const int buf = (g - t0) & 1;
        if (!ptx::mbar_wait(&acc_empty[buf], acc_phase[buf] ^ 1u, dead, p.status_dev)) break;
        ptx::tc_fence_after_sync();
        for (int kc = 0; kc < 4; ++kc) {
          if (!ptx::mbar_wait(&b_full[stage], phase, dead, p.status_dev)) { ok = false; break; }
          ptx::tc_fence_after_sync();
          const uint32_t a_addr = ptx::smem_addr(a_smem) + (kc >> 1) * kAPiece + (kc & 1) * 64;
          const uint32_t b_addr = ptx::smem_addr(b_smem + stage * kBStage);
#pragma unroll
          for (int k16 = 0; k16 < 2; ++k16) {
#pragma unroll
            for (int pr = 0; pr < 9; ++pr) {
              // all nine (Err piece, U piece) products, by falling magnitude: piece index sums 0, 1, 1, 2, 2, 2, 3, 3, 4
              const int pa = pr == 0 ? 0 : pr == 1 ? 0 : pr == 2 ? 1 : pr == 3 ? 0 : pr == 4 ? 1 : pr == 5 ? 2 : pr == 6 ? 1 : 2;
              const int pb = pr == 0 ? 0 : pr == 1 ? 1 : pr == 2 ? 0 : pr == 3 ? 2 : pr == 4 ? 1 : pr == 5 ? 0 : pr == 6 ? 2 : pr == 7 ? 1 : 2;
              // leading product -> exact accumulator; the rest -> the second one
              const uint32_t acc = tmem_base + buf * 256 + (pr == 0 ? 0 : kTileN);
              const bool first = (kc | k16) == 0 && pr <= 1;
              ptx::mma_f16(acc, ptx::with_start(adesc, a_addr + pa * 2 * kAPiece + k16 * 32),
                           ptx::with_start(bdesc, b_addr + pb * kBPiece + k16 * (16 * 128)), idesc, !first);
            }
          }
          ptx::mma_commit(&b_empty[stage]);
          if (++stage == kBStages) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        ptx::mma_commit(&acc_full[buf]);
        acc_phase[buf] ^= 1u;
        if (g + 1 < t1 && (g + 1) / p.ntiles != rb) ptx::mma_commit(a_empty);    // this row block's Err pieces are free once these MMAs are done
      }
      if (*dead) {
        ptx::mma_commit(drain);
        const long long c0 = clock64();
        while (!ptx::mbar_try_wait(drain, 0) && clock64() - c0 < ptx::kWaitLimit) {}
      }
    }
  } else {
    // Two warps per TMEM lane quadrant, each taking one 64-column half of every tile.  W is never
    // read here: 32 rows x 16 columns of the negated product, widened to binary64, are laid out in
    // a staging tile exactly as a tile of the working weights is laid out in memory (wc_index) and
    // handed to the memory system as one 4 KB element-wise add into that tile (W + (-p) is the same
    // operation as W - p), so the epilogue only issues writes.
    const int q = warp & 3, half = (warp - 2) >> 2;
    uint32_t acc_phase[2] = {0, 0};
    uint8_t* stage_tile = out_smem + (warp - 2) * kOutChunk;
    uint8_t* my_row = stage_tile + lane * 128;        // this lane's row of the staging tile
    for (int g = t0; g < t1; ++g) {
      const int rb = g / p.ntiles, t = g % p.ntiles;
      const int buf = (g - t0) & 1;
      // first tile of this warp's rows of the row block and of the launch's first column
      double* wtile = p.Wc + (static_cast<int64_t>((rb * 128 + q * 32) / kWcTileRows) * (p.in / kWcTileCols) +
                              (p.c0 + half * 64) / kWcTileCols) * kWcTileElems;
      if (!ptx::mbar_wait(&acc_full[buf], acc_phase[buf], dead, p.status_dev)) break;
      ptx::tc_fence_after_sync();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float v[16], v2[16];
        const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + buf * 256 + half * 64 + c * 16;
        ptx::tmem_ld16_nowait(taddr, v);
        ptx::tmem_ld16_nowait(taddr + kTileN, v2);
        ptx::tmem_ld_wait();
        if (lane == 0) ptx::bulk_wait_read();         // the previous add has finished reading the staging tile
        __syncwarp();
#pragma unroll
        for (int k = 0; k < 8; ++k) {                  // column pair k of the row sits at pair position k ^ (row % 8)
          double2 x;
          x.x = -(static_cast<double>(v[2 * k]) + static_cast<double>(v2[2 * k]));
          x.y = -(static_cast<double>(v[2 * k + 1]) + static_cast<double>(v2[2 * k + 1]));
          *reinterpret_cast<double2*>(my_row + ((k ^ (lane & 7)) << 4)) = x;
        }
        ptx::fence_proxy_async();
        __syncwarp();
        if (lane == 0) {
          ptx::bulk_reduce_add_f64(wtile + (static_cast<int64_t>(t) * (kTileN / kWcTileCols) + c) * kWcTileElems, stage_tile,
                                   kOutChunk);
          ptx::bulk_commit();
        }
      }
      ptx::tc_fence_before_sync();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&acc_empty[buf]);
      acc_phase[buf] ^= 1u;
    }
    if (lane == 0) ptx::bulk_wait_all();               // every add of this warp is complete before the CTA ends
  }

  ptx::tc_fence_before_sync();
  __syncthreads();
  if (warp == 1) {
    ptx::tc_fence_after_sync();
    ptx::tmem_dealloc(tmem_base, 512);
  }
}

// Fixed-point slicing shared by both operands: with ex the biased exponent of the largest
// magnitude of a slice group (clamped so that all three grids are normal numbers),
// grid = 2^(ex - 134), and x = a0*grid + a1*grid/256 + a2*grid/65536 with integers |a0| <= 256,
// |a1|, |a2| <= 128 (each product a*grid is exact in bf16).
struct SliceGrid { float g, inv; };
__device__ __forceinline__ SliceGrid slice_grid(float maxabs) {
  int ex = (__float_as_int(maxabs) >> 23) & 0xFF;
  ex = ex < 32 ? 32 : (ex > 250 ? 250 : ex);
  SliceGrid s;
  s.g = __int_as_float((ex - 7) << 23);             // 2^(ex - 127 - 7)
  s.inv = __int_as_float((254 - (ex - 7)) << 23);   // 1 / g
  return s;
}
__device__ __forceinline__ void slice3(float x, SliceGrid s, __nv_bfloat16& p0, __nv_bfloat16& p1, __nv_bfloat16& p2) {
  const float a0 = rintf(x * s.inv);
  const float r1 = fmaf(-a0, s.g, x);                       // exact
  const float a1 = rintf(r1 * s.inv * 256.0f);
  const float r2 = fmaf(-a1, s.g * (1.0f / 256.0f), r1);    // exact
  const float a2 = rintf(r2 * s.inv * 65536.0f);
  p0 = __float2bfloat16_rn(a0 * s.g);
  p1 = __float2bfloat16_rn(a1 * s.g * (1.0f / 256.0f));
  p2 = __float2bfloat16_rn(a2 * s.g * (1.0f / 65536.0f));
}

// U pieces: one grid per (128-row block b, column c).  Only columns right of the block are
// ever read by the trailing update, so only those are written.
__global__ void __launch_bounds__(128)
slice_u_kernel(const double* __restrict__ U, int64_t in, __nv_bfloat16* __restrict__ p0, __nv_bfloat16* __restrict__ p1,
               __nv_bfloat16* __restrict__ p2) {
  const int b = blockIdx.y;
  if (static_cast<int>(blockIdx.x) <= b) return;
  const int64_t c = static_cast<int64_t>(blockIdx.x) * 128 + threadIdx.x;
  const double* src = U + static_cast<int64_t>(b) * 128 * in + c;
  float v[128];
  float m = 0.0f;
#pragma unroll
  for (int i = 0; i < 128; ++i) { v[i] = static_cast<float>(src[static_cast<int64_t>(i) * in]); m = fmaxf(m, fabsf(v[i])); }
  const SliceGrid sg = slice_grid(m);
#pragma unroll
  for (int i = 0; i < 128; ++i) {
    __nv_bfloat16 a, bb, cc;
    slice3(v[i], sg, a, bb, cc);
    const int64_t idx = (static_cast<int64_t>(b) * 128 + i) * in + c;
    p0[idx] = a; p1[idx] = bb; p2[idx] = cc;
  }
}

}  // namespace

// Host-side state of one GPTQ call's trailing updates: the six tensor maps never change
// between blocks, only the coordinates do.
struct TrailPlan {
  CUtensorMap e[3], u[3];
  double* Wc;
  int64_t rows_total, in;
  int sm_count;
};

int trail_split_u(const double* U, int64_t in, __nv_bfloat16* u0, __nv_bfloat16* u1, __nv_bfloat16* u2, cudaStream_t st) {
  const unsigned nb = static_cast<unsigned>(in / 128);
  if (nb > 1) slice_u_kernel<<<dim3(nb, nb - 1), 128, 0, st>>>(U, in, u0, u1, u2);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

int trail_plan(TrailPlan* plan, double* Wc, int64_t rows_total, int64_t in, const __nv_bfloat16* const e[3],
               const __nv_bfloat16* const u[3]) {
  plan->Wc = Wc;
  plan->rows_total = rows_total;
  plan->in = in;
  for (int k = 0; k < 3; ++k) {
    int rc = make_tmap_bf16(&plan->e[k], e[k], 128, static_cast<uint64_t>(2 * rows_total), 256, 128);   // two sets
    if (rc != ADADIM_OK) return rc;
    rc = make_tmap_bf16(&plan->u[k], u[k], static_cast<uint64_t>(in), static_cast<uint64_t>(in),
                        static_cast<uint64_t>(in) * 2, 32);
    if (rc != ADADIM_OK) return rc;
  }
  int dev = 0;
  ADADIM_CUDA_TRY(cudaGetDevice(&dev));
  ADADIM_CUDA_TRY(cudaDeviceGetAttribute(&plan->sm_count, cudaDevAttrMultiProcessorCount, dev));
  ADADIM_CUDA_TRY(cudaFuncSetAttribute(trail_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                       static_cast<int>(kSmemBytes)));
  return ADADIM_OK;
}

// Updates `ntiles` 128-column tiles starting at column c0, in every 128-row block, with the errors of
// the block whose first column is i1 (error set i1/128 & 1), on at most `max_ctas` CTAs (one per SM:
// the count of SMs the caller leaves to this launch).
int trail_launch(const TrailPlan& plan, int i1, int64_t c0, int ntiles, int max_ctas, int* status_dev, cudaStream_t st) {
  TrailParams p;
  p.Wc = plan.Wc;
  p.in = plan.in;
  p.c0 = c0;
  p.i1 = i1;
  p.ntiles = ntiles;
  p.mblocks = static_cast<int>(plan.rows_total / 128);
  p.e_row0 = static_cast<int>(((i1 / 128) & 1) * plan.rows_total);
  p.status_dev = status_dev;
  if (p.ntiles <= 0) return ADADIM_OK;
  const int64_t total = static_cast<int64_t>(p.mblocks) * ntiles;
  const int ctas = static_cast<int>(total < max_ctas ? total : max_ctas);
  trail_kernel<<<dim3(static_cast<unsigned>(ctas < 1 ? 1 : ctas)), kThreads, kSmemBytes, st>>>(plan.e[0], plan.e[1], plan.e[2], plan.u[0],
                                                                                                plan.u[1], plan.u[2], p);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
