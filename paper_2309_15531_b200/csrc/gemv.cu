// Matrix-vector product with the quantized weights, y = Q x (paper Section 4.5 and Appendix D:
// the latency of one decoder-layer product with per-IC quantized weights, fp16 vector in and out).
//
// Per-IC grouping gives every column i of a g-row group k its own scale and zero point, so
//     y[o] = sum_i a_k[i] * code[o,i]  -  b_k,     a_k[i] = s[k,i] x[i],   b_k = sum_i s[k,i] z[k,i] x[i]
// for the rows o of group k: the scale is folded into the vector once per group (Section 4.5 says
// the same of its lookup tables) and what remains per weight is an integer code times a number.
// The product is bound by the bytes of the codes, so the work per code has to stay near one
// instruction.  Two kernels:
//   prepare  a_k in binary32, cut into three signed 7-bit fixed-point pieces on one power-of-two grid
//            per group and 128-column block (a = grid * (p0 + p1/128 + p2/16384), |p| <= 64: 21 bits
//            below the block's largest |a|), stored as bytes in the order the main kernel consumes;
//            the block's grid and its share of b_k beside them.  One warp per (group, block).
//   product  a warp owns 16 rows and walks over the columns 128 at a time: codes are spread to bytes
//            (two to six logic instructions per word) and multiplied against the three pieces by the
//            integer matrix instruction (16 rows x 32 columns x 8 vectors per issue, three of the
//            eight vectors in use); a block's exact integer sums are scaled by the block's grid and
//            added in binary32 in column order; one fp16 rounding at the end.
// The instruction is the register-operand integer MMA: the operands are produced in registers by
// the unpacking and there is nothing to gain from staging 8-bit copies of a 3- or 4-bit stream in
// shared memory for the tensor-memory path.
#include "common.cuh"

namespace adadim {
namespace {

constexpr int kRowsPerWarp = 16;
constexpr int kWarps = 4;                      // 64 rows per CTA
constexpr int kColBlock = 128;                 // columns per warp step (four matrix instructions)

// ---- prepare ------------------------------------------------------------------------------
// pieces: [groups][3][in] bytes.  Within every 128-column block the bytes are ordered as the main
// kernel's lanes read them: lane quad position t takes bytes 32 t .. 32 t + 31 as eight words, word
// 2 j + h feeding matrix instruction j (h = 0: its first 16 reduction slots, h = 1: the other 16).
// For 3-bit codes the unpacking yields the columns in natural order; for 4-bit codes a word of
// eight codes splits into its even codes (h = 0) and its odd codes (h = 1).
template <int BITS>
__device__ __forceinline__ int piece_position(int w /* column within its 128-block */) {
  if (BITS == 3) return w;
  const int t = w >> 5, j = (w >> 3) & 3, e = w & 7;
  return t * 32 + j * 8 + (e & 1) * 4 + (e >> 1);
}

struct BlockMeta { float grid; float bsum; };       // per (group, 128-column block)

__device__ __forceinline__ void load8h(const uint16_t* p, float (&v)[8]) {
  load8(reinterpret_cast<const __half*>(p), v);
}

// One warp per (group k, 128-column block): lanes 0..15 take eight columns each.
template <int BITS>
__global__ void __launch_bounds__(256)
gemv_prepare_kernel(const uint16_t* __restrict__ scales, const uint16_t* __restrict__ zeros, const __half* __restrict__ x,
                    int64_t in, int64_t groups, int8_t* __restrict__ pieces, BlockMeta* __restrict__ meta) {
  const int nblocks = static_cast<int>(in / kColBlock);
  const int64_t wid = static_cast<int64_t>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (wid >= groups * nblocks) return;
  const int64_t k = wid / nblocks;
  const int blk = static_cast<int>(wid % nblocks);
  const int lane = threadIdx.x & 31;
  const int64_t i0 = static_cast<int64_t>(blk) * kColBlock + (lane & 15) * 8;
  float sv[8], zv[8], xv[8], a[8];
  load8h(scales + k * in + i0, sv);
  load8h(zeros + k * in + i0, zv);
  load8(x + i0, xv);
  float amax = 0.0f;
#pragma unroll
  for (int e = 0; e < 8; ++e) { a[e] = sv[e] * xv[e]; amax = fmaxf(amax, fabsf(a[e])); }
  for (int m = 8; m > 0; m >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xffffffffu, amax, m));
  // grid = 2^(e - 6) with 2^e > amax >= 2^(e-1): |a / grid| < 64.  Clamped so that all three grids are normal.
  int ex = ((__float_as_int(amax) >> 23) & 0xFF) + 1;
  ex = ex < 32 ? 32 : (ex > 250 ? 250 : ex);
  const float grid = __int_as_float((ex - 6) << 23);
  const float inv = __int_as_float((254 - (ex - 6)) << 23);
  float bsum = 0.0f;
  uint32_t pk[3][2] = {};
#pragma unroll
  for (int e = 0; e < 8; ++e) {
    bsum = fmaf(a[e], zv[e], bsum);
    const float p0 = rintf(a[e] * inv);
    const float r1 = fmaf(-p0, grid, a[e]);                       // exact
    const float p1 = rintf(r1 * inv * 128.0f);
    const float r2 = fmaf(-p1, grid * (1.0f / 128.0f), r1);       // exact
    const float p2 = rintf(r2 * inv * 16384.0f);
    // byte of column e inside this lane's eight: natural order (3-bit) or even codes first (4-bit);
    // eight consecutive columns keep their place as a unit in both orders (see piece_position)
    const int pos = BITS == 3 ? e : (e & 1) * 4 + (e >> 1);
    pk[0][pos >> 2] |= (static_cast<uint32_t>(static_cast<int>(p0)) & 0xFFu) << (8 * (pos & 3));
    pk[1][pos >> 2] |= (static_cast<uint32_t>(static_cast<int>(p1)) & 0xFFu) << (8 * (pos & 3));
    pk[2][pos >> 2] |= (static_cast<uint32_t>(static_cast<int>(p2)) & 0xFFu) << (8 * (pos & 3));
  }
  if (lane < 16) {
    int8_t* dst = pieces + k * 3 * in + i0;
#pragma unroll
    for (int p = 0; p < 3; ++p) *reinterpret_cast<uint2*>(dst + p * in) = make_uint2(pk[p][0], pk[p][1]);
  } else {
    bsum = 0.0f;                                     // lanes 16..31 mirror lanes 0..15
  }
  for (int m = 16; m > 0; m >>= 1) bsum += __shfl_xor_sync(0xffffffffu, bsum, m);      // a fixed tree
  if (lane == 0) { meta[wid].grid = grid; meta[wid].bsum = bsum; }
}

// ---- product --------------------------------------------------------------------------------
// D (16 x 8, s32) += A (16 x 32, s8, row) * B (32 x 8, s8, col).  Lane l = 4 g + t holds
//   a0: row g, slots 4t..4t+3    a1: row g+8, same slots    a2, a3: the same rows, slots 16+4t..16+4t+3
//   b0: slots 4t..4t+3 of vector g    b1: slots 16+4t.. of vector g
//   d0, d1: row g, vectors 2t, 2t+1    d2, d3: row g+8, vectors 2t, 2t+1
__device__ __forceinline__ void imma(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                     uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.s8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
               : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// This lane's 32 codes of one row in one 128-column block, as loaded: four words (4-bit) or three (3-bit).
template <int BITS>
struct RawCodes { uint32_t w[BITS]; };

template <int BITS>
__device__ __forceinline__ RawCodes<BITS> load_raw(const uint32_t* __restrict__ rowp, int cb, int t) {
  RawCodes<BITS> r;
  if (BITS == 4) {
    const uint4 v = __ldcs(reinterpret_cast<const uint4*>(rowp + cb * 16 + t * 4));     // streamed once: evict first
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[3] = v.w;
  } else {
    const uint32_t* p = rowp + cb * 12 + t * 3;
#pragma unroll
    for (int k = 0; k < BITS; ++k) r.w[k] = __ldcs(p + k);
  }
  return r;
}

// Eight byte-words (four instructions x two halves), one code per byte.
template <int BITS>
__device__ __forceinline__ void spread(const RawCodes<BITS>& r, uint32_t (&u)[8]) {
  if (BITS == 4) {
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      u[2 * j] = r.w[j] & 0x0F0F0F0Fu;                 // codes 0, 2, 4, 6 of the word
      u[2 * j + 1] = (r.w[j] >> 4) & 0x0F0F0F0Fu;      // codes 1, 3, 5, 7
    }
  } else {
#pragma unroll
    for (int m = 0; m < 8; ++m) {
      // codes 4m .. 4m+3: 12 bits at bit 12 m of the lane's 96, spread to one code per byte
      const int bit = 12 * m, idx = bit >> 5, sh = bit & 31;
      uint32_t v = sh + 12 <= 32 ? r.w[idx] >> sh : __funnelshift_r(r.w[idx], r.w[idx + 1 < BITS ? idx + 1 : idx], sh);
      v &= 0xFFFu;
      const uint32_t t1 = (v | (v << 10)) & 0x003F003Fu;
      u[m] = (t1 | (t1 << 5)) & 0x07070707u;
    }
  }
}

constexpr int kUnroll = 4;                     // column blocks per step of the main loop

template <int BITS>
__global__ void __launch_bounds__(kWarps * 32)
gemv_product_kernel(const uint32_t* __restrict__ codes, const int8_t* __restrict__ pieces,
                    const BlockMeta* __restrict__ meta, int64_t out, int64_t in, int group, int blocks_per_split,
                    float* __restrict__ partial, __half* __restrict__ y /* non-null: one column range, write the result */) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t r0 = (static_cast<int64_t>(blockIdx.x) * kWarps + warp) * kRowsPerWarp;
  if (r0 >= out) return;
  const int64_t k = r0 / group;
  const int nblocks = static_cast<int>(in / kColBlock);
  const int cb0 = blockIdx.y * blocks_per_split;
  const int cb1 = min(cb0 + blocks_per_split, nblocks);
  const int64_t words_per_row = in * BITS / 32;
  const uint32_t* rowa = codes + (r0 + g) * words_per_row;
  const uint32_t* rowb = rowa + 8 * words_per_row;
  // vector g of the instruction is piece g (g < 3); the other five vectors are zero
  const int8_t* pz = pieces + (k * 3 + (g < 3 ? g : 0)) * in + t * 32;
  const BlockMeta* bm = meta + k * nblocks;
  // this lane's weights for its two result columns of the instruction: pieces 0 and 1 (t = 0), piece 2 (t = 1)
  const float w0 = t == 0 ? 1.0f : t == 1 ? 1.0f / 16384.0f : 0.0f, w1 = t == 0 ? 1.0f / 128.0f : 0.0f;
  float acc_a = 0.0f, acc_b = 0.0f, bsum = 0.0f;
  // a block's four instructions, then its exact integer sums scaled by the block's grid
  auto finish_block = [&](const int (&d)[4], int blk) {
    const BlockMeta m = bm[blk];
    acc_a = fmaf(m.grid, fmaf(static_cast<float>(d[1]), w1, static_cast<float>(d[0]) * w0), acc_a);
    acc_b = fmaf(m.grid, fmaf(static_cast<float>(d[3]), w1, static_cast<float>(d[2]) * w0), acc_b);
    bsum += m.bsum;
  };
  int cb = cb0;
#pragma unroll 1
  for (; cb + kUnroll <= cb1; cb += kUnroll) {
    RawCodes<BITS> ra[kUnroll], rb[kUnroll];
    uint4 b01[kUnroll], b23[kUnroll];
#pragma unroll
    for (int q = 0; q < kUnroll; ++q) {
      ra[q] = load_raw<BITS>(rowa, cb + q, t);
      rb[q] = load_raw<BITS>(rowb, cb + q, t);
    }
#pragma unroll
    for (int q = 0; q < kUnroll; ++q) {
      b01[q] = make_uint4(0u, 0u, 0u, 0u);
      b23[q] = b01[q];
      if (g < 3) {
        const uint4* bp = reinterpret_cast<const uint4*>(pz + static_cast<int64_t>(cb + q) * kColBlock);
        b01[q] = bp[0];
        b23[q] = bp[1];
      }
    }
#pragma unroll
    for (int q = 0; q < kUnroll; ++q) {
      uint32_t ua[8], ub[8];
      int d[4] = {0, 0, 0, 0};
      spread<BITS>(ra[q], ua);
      spread<BITS>(rb[q], ub);
      imma(d, ua[0], ub[0], ua[1], ub[1], b01[q].x, b01[q].y);
      imma(d, ua[2], ub[2], ua[3], ub[3], b01[q].z, b01[q].w);
      imma(d, ua[4], ub[4], ua[5], ub[5], b23[q].x, b23[q].y);
      imma(d, ua[6], ub[6], ua[7], ub[7], b23[q].z, b23[q].w);
      finish_block(d, cb + q);
    }
  }
#pragma unroll 1
  for (; cb < cb1; ++cb) {
    uint32_t ua[8], ub[8];
    spread<BITS>(load_raw<BITS>(rowa, cb, t), ua);
    spread<BITS>(load_raw<BITS>(rowb, cb, t), ub);
    uint4 b01 = make_uint4(0u, 0u, 0u, 0u), b23 = b01;
    if (g < 3) {
      const uint4* bp = reinterpret_cast<const uint4*>(pz + static_cast<int64_t>(cb) * kColBlock);
      b01 = bp[0];
      b23 = bp[1];
    }
    int d[4] = {0, 0, 0, 0};
    imma(d, ua[0], ub[0], ua[1], ub[1], b01.x, b01.y);
    imma(d, ua[2], ub[2], ua[3], ub[3], b01.z, b01.w);
    imma(d, ua[4], ub[4], ua[5], ub[5], b23.x, b23.y);
    imma(d, ua[6], ub[6], ua[7], ub[7], b23.z, b23.w);
    finish_block(d, cb);
  }
  // row sums over the three pieces: lane t = 0 holds pieces 0 and 1, lane t = 1 piece 2
  acc_a += __shfl_xor_sync(0xffffffffu, acc_a, 1);
  acc_b += __shfl_xor_sync(0xffffffffu, acc_b, 1);
  if (t == 0) {
    if (y != nullptr) {
      y[r0 + g] = __float2half_rn(acc_a - bsum);
      y[r0 + g + 8] = __float2half_rn(acc_b - bsum);
    } else {
      float* dst = partial + static_cast<int64_t>(blockIdx.y) * out;
      dst[r0 + g] = acc_a - bsum;
      dst[r0 + g + 8] = acc_b - bsum;
    }
  }
}

__global__ void __launch_bounds__(256)
gemv_finish_kernel(const float* __restrict__ partial, int64_t out, int splits, __half* __restrict__ y) {
  const int64_t o = static_cast<int64_t>(blockIdx.x) * 256 + threadIdx.x;
  if (o >= out) return;
  float acc = 0.0f;
  for (int s = 0; s < splits; ++s) acc += partial[static_cast<int64_t>(s) * out + o];     // fixed order
  y[o] = __float2half_rn(acc);
}

struct GemvLayout { size_t pieces_off, meta_off, partial_off, total; int splits, blocks_per_split; };
GemvLayout gemv_layout(int64_t out, int64_t in, int group) {
  GemvLayout L;
  const int64_t groups = group > 0 ? out / group : 0;
  const int nblocks = static_cast<int>(in / kColBlock);
  const int64_t ctas_x = (out + kWarps * kRowsPerWarp - 1) / (kWarps * kRowsPerWarp);
  // enough warps to cover the memory latency: about 48 per SM (148 SMs), four per CTA; the column range is
  // split when the rows alone do not provide them
  int splits = static_cast<int>((148 * 12 + ctas_x - 1) / (ctas_x > 0 ? ctas_x : 1));
  if (splits > nblocks) splits = nblocks;
  if (splits < 1) splits = 1;
  L.blocks_per_split = (nblocks + splits - 1) / splits;
  L.splits = L.blocks_per_split > 0 ? (nblocks + L.blocks_per_split - 1) / L.blocks_per_split : 1;
  size_t off = 0;
  L.pieces_off = off;  off += round_up(static_cast<size_t>(groups) * 3 * in, 256);
  L.meta_off = off;    off += round_up(static_cast<size_t>(groups) * nblocks * sizeof(BlockMeta), 256);
  L.partial_off = off; off += round_up(static_cast<size_t>(L.splits) * out * 4, 256);
  L.total = off;
  return L;
}

}  // namespace

size_t gemv_workspace_bytes(int64_t out, int64_t in, int group) { return gemv_layout(out, in, group).total; }

int gemv_launch(const adadim_qtensor& q, int64_t out, int64_t in, int bits, int group, const void* x, void* y,
                void* workspace, cudaStream_t st) {
  const GemvLayout L = gemv_layout(out, in, group);
  uint8_t* ws = static_cast<uint8_t*>(workspace);
  int8_t* pieces = reinterpret_cast<int8_t*>(ws + L.pieces_off);
  BlockMeta* meta = reinterpret_cast<BlockMeta*>(ws + L.meta_off);
  float* partial = reinterpret_cast<float*>(ws + L.partial_off);
  const int64_t groups = out / group;
  const __half* xh = static_cast<const __half*>(x);
  __half* yh = static_cast<__half*>(y);
  const unsigned pgrid = static_cast<unsigned>((groups * (in / kColBlock) + 7) / 8);
  if (bits == 3) gemv_prepare_kernel<3><<<pgrid, 256, 0, st>>>(q.scales, q.zeros, xh, in, groups, pieces, meta);
  else gemv_prepare_kernel<4><<<pgrid, 256, 0, st>>>(q.scales, q.zeros, xh, in, groups, pieces, meta);
  const dim3 grid(static_cast<unsigned>((out + kWarps * kRowsPerWarp - 1) / (kWarps * kRowsPerWarp)), L.splits);
  __half* direct = L.splits == 1 ? yh : nullptr;
  if (bits == 3) gemv_product_kernel<3><<<grid, kWarps * 32, 0, st>>>(q.codes, pieces, meta, out, in, group, L.blocks_per_split, partial, direct);
  else gemv_product_kernel<4><<<grid, kWarps * 32, 0, st>>>(q.codes, pieces, meta, out, in, group, L.blocks_per_split, partial, direct);
  if (L.splits > 1)
    gemv_finish_kernel<<<static_cast<unsigned>((out + 255) / 256), 256, 0, st>>>(partial, out, L.splits, yh);
  return cudaGetLastError() == cudaSuccess ? ADADIM_OK : ADADIM_ERR_CUDA;
}

}  // namespace adadim
