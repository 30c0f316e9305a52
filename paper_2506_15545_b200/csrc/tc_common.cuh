// Pieces shared by the tensor-core kernels (forward and backward): the shared-memory tile
// layout a 128-byte-swizzled TMA load produces, the tcgen05 operand descriptors for it, the
// 128 x 128 x 128 MMA chains, the in-place feature map and the host-side tensor maps.
#pragma once

#include <cuda_fp16.h>

#include "rattn_internal.h"
#include "tc_ptx.cuh"

namespace rattn {
namespace tc {

using namespace ptx;

constexpr int TILE = 128;
constexpr int HALF_BYTES = TILE * 64 * 2;   // one [128 x 64] bf16 sub-tile, 128-byte rows
constexpr int TILE_BYTES = 2 * HALF_BYTES;

// Operand descriptors.  The descriptor of a tile is built once from its base address; the
// eight (or four) reduction steps of a product then only add a constant to its start-address
// field (bytes / 16; shared-memory addresses stay below 2^18, so the field never carries).
//   K-major operand: [128 rows x 128 reduction] as two 64-wide halves; 16 reduction elements
//   per MMA = 32 bytes along the 128-byte row.
//   MN-major operand: rows are the reduction index (128-byte rows of 64 columns, two column
//   halves 16 KB apart); 16 reduction rows per MMA = 2048 bytes.
__device__ __forceinline__ uint64_t kmajor_base(uint32_t base) { return smem_desc(base, 16, 1024); }
__device__ __forceinline__ uint64_t mnmajor_base(uint32_t base) { return smem_desc(base, HALF_BYTES, 1024); }
__host__ __device__ constexpr uint32_t kstep_k(int k, int half_bytes) { return (uint32_t)(((k >> 2) * half_bytes + (k & 3) * 32) >> 4); }
__host__ __device__ constexpr uint32_t kstep_mn(int k) { return (uint32_t)((k * 2048) >> 4); }
__device__ __forceinline__ uint64_t kmajor_desc(uint32_t base, int kstep) { return kmajor_base(base) + kstep_k(kstep, HALF_BYTES); }
__device__ __forceinline__ uint64_t mnmajor_desc(uint32_t base, int kstep) { return mnmajor_base(base) + kstep_mn(kstep); }

// D[128x128] (+)= A B^T-style products over a reduction of 128, 8 MMAs of K = 16.  (Unrolled on
// purpose: with rolled issue loops the MMA warps, which sit on the critical path, measured 6-25 % slower.)
__device__ __forceinline__ void mma_kk(uint32_t d, uint32_t a_base, uint32_t b_base, bool acc) {
  constexpr uint32_t idesc = instr_desc(128, 128, 0, 0);
  const uint64_t a0 = kmajor_base(a_base), b0 = kmajor_base(b_base);
#pragma unroll
  for (int k = 0; k < 8; ++k)
    mma_bf16(d, a0 + kstep_k(k, HALF_BYTES), b0 + kstep_k(k, HALF_BYTES), idesc, (acc || k > 0) ? 1u : 0u);
}
template <int AB_BF16>
__device__ __forceinline__ void mma_kmn(uint32_t d, uint32_t a_base, uint32_t b_base, bool acc) {
  constexpr uint32_t idesc = instr_desc(128, 128, 0, 1, AB_BF16);
  const uint64_t a0 = kmajor_base(a_base), b0 = mnmajor_base(b_base);
#pragma unroll
  for (int k = 0; k < 8; ++k) mma_bf16(d, a0 + kstep_k(k, HALF_BYTES), b0 + kstep_mn(k), idesc, (acc || k > 0) ? 1u : 0u);
}
__device__ __forceinline__ void mma_mnmn(uint32_t d, uint32_t a_base, uint32_t b_base, bool acc) {
  constexpr uint32_t idesc = instr_desc(128, 128, 1, 1);
  const uint64_t a0 = mnmajor_base(a_base), b0 = mnmajor_base(b_base);
#pragma unroll
  for (int k = 0; k < 8; ++k) mma_bf16(d, a0 + kstep_mn(k), b0 + kstep_mn(k), idesc, (acc || k > 0) ? 1u : 0u);
}

// ---- half tiles: [64 rows x 128 columns] bf16 as two [64 x 64] boxes of 8 KB ------------
constexpr int HT_HALF = 64 * 64 * 2;
constexpr int HT_BYTES = 2 * HT_HALF;
// B operand, K-major: the half tile's 64 rows are N, its 128 columns the reduction (8 steps)
__device__ __forceinline__ uint64_t kmajor_base_h(uint32_t base) { return smem_desc(base, 16, 1024); }
// B operand, MN-major: the half tile's 128 columns are N, its 64 rows the reduction (4 steps)
__device__ __forceinline__ uint64_t mnmajor_base_h(uint32_t base) { return smem_desc(base, HT_HALF, 1024); }
// D[128 x 64] = A[128 x 128] (K-major full tile) . B[64 x 128]^T (K-major half tile)
__device__ __forceinline__ void mma_k_kh(uint32_t d, uint32_t a_base, uint32_t b_base) {
  constexpr uint32_t idesc = instr_desc(128, 64, 0, 0);
  const uint64_t a0 = kmajor_base(a_base), b0 = kmajor_base_h(b_base);
#pragma unroll
  for (int k = 0; k < 8; ++k)
    mma_bf16(d, a0 + kstep_k(k, HALF_BYTES), b0 + kstep_k(k, HT_HALF), idesc, k > 0 ? 1u : 0u);
}
// D[128 x 128] (+)= A[128 x 64] (bf16 in TMEM) . B[64 x 128] (MN-major half tile).  A sits where
// the row groups left it: reduction elements 0..31 in columns 0..15 and 32..63 in columns
// 32..47 of the slot (each group packs its 32 fp32 columns into the first 16 of them).
__device__ __forceinline__ void mma_ts_h(uint32_t d, uint32_t a_tmem, uint32_t b_base, bool acc) {
  constexpr uint32_t idesc = instr_desc(128, 128, 0, 1);
  const uint64_t b0 = mnmajor_base_h(b_base);
#pragma unroll
  for (int k = 0; k < 4; ++k)
    mma_bf16_ts(d, a_tmem + (k < 2 ? 8 * k : 32 + 8 * (k - 2)), b0 + kstep_mn(k), idesc, (acc || k > 0) ? 1u : 0u);
}
// A caller's tensor (q, k, v, out and the gradients): its heads may be dense ([B, H, T, d]) or interleaved
// ([B, T, H, d]), so its map has four dimensions (d, T, H, B) and a matrix index z = b * H + h is split.
struct alignas(64) UMap {
  CUtensorMap m;
  int H;
};
__device__ __forceinline__ void prefetch_map(const UMap* tm) { prefetch_tensormap(&tm->m); }
__device__ __forceinline__ void load_tile(unsigned char* dst, const UMap* tm, uint64_t* bar, int row, int z) {
  const int b = z / tm->H, h = z - b * tm->H;
  tma_load_4d(dst, &tm->m, bar, 0, row, h, b);
  tma_load_4d(dst + HALF_BYTES, &tm->m, bar, 64, row, h, b);
}
// `tm` must have a [64 columns x 64 rows] box
__device__ __forceinline__ void load_half_tile(unsigned char* dst, const UMap* tm, uint64_t* bar, int row, int z) {
  const int b = z / tm->H, h = z - b * tm->H;
  tma_load_4d(dst, &tm->m, bar, 0, row, h, b);
  tma_load_4d(dst + HT_HALF, &tm->m, bar, 64, row, h, b);
}
__device__ __forceinline__ void load_tile(unsigned char* dst, const CUtensorMap* tm, uint64_t* bar, int row, int z) {
  tma_load_3d(dst, tm, bar, 0, row, z);
  tma_load_3d(dst + HALF_BYTES, tm, bar, 64, row, z);
}
// `tm` must have a [64 columns x 64 rows] box
__device__ __forceinline__ void load_half_tile(unsigned char* dst, const CUtensorMap* tm, uint64_t* bar, int row, int z) {
  tma_load_3d(dst, tm, bar, 0, row, z);
  tma_load_3d(dst + HT_HALF, tm, bar, 64, row, z);
}

// The same for bf16 output: 32 values of row r become one 64-byte row of an 8 KB region
// (16-byte chunks XOR-swizzled by row pair), flushed in 64-byte segments, eight rows per
// instruction.  dst points at column 32*c of the tile's first row (row pitch 128 bf16).
__device__ __forceinline__ void stage_bf16_block(unsigned char* stage, int r, const float (&x)[32]) {
#pragma unroll
  for (int e = 0; e < 4; ++e)
    *reinterpret_cast<uint4*>(stage + r * 64 + ((e ^ ((r >> 1) & 3)) << 4)) =
        make_uint4(pack_bf16(x[8 * e], x[8 * e + 1]), pack_bf16(x[8 * e + 2], x[8 * e + 3]),
                   pack_bf16(x[8 * e + 4], x[8 * e + 5]), pack_bf16(x[8 * e + 6], x[8 * e + 7]));
}
__device__ __forceinline__ void flush_bf16_block(const unsigned char* stage, int r, __nv_bfloat16* dst, int n_rows) {
  const int sub = r & 3;
#pragma unroll
  for (int k = 0; k < 4; ++k) {
    const int row = (r >> 5) * 32 + 8 * k + ((r & 31) >> 2);
    const uint4 v = *reinterpret_cast<const uint4*>(stage + row * 64 + ((sub ^ ((row >> 1) & 3)) << 4));
    if (row < n_rows) *reinterpret_cast<uint4*>(dst + (size_t)row * 128 + 8 * sub) = v;
  }
}

// phi over the 128 features of one row by a pair of adjacent lanes: this lane owns the 64
// columns of column half `half` (eight 16-byte chunks at src + row * 128 within that half's box).
// src_half / dst_half point at the [rows x 64] box of this lane's column half.
__device__ __forceinline__ void feature_map_pair(const unsigned char* src_half, unsigned char* dst_half, int row) {
  float x[64];
  float m = -INFINITY;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const uint4 u = *reinterpret_cast<const uint4*>(src_half + row * 128 + ((c ^ (row & 7)) << 4));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(h[e]);
      x[c * 8 + 2 * e] = f.x;
      x[c * 8 + 2 * e + 1] = f.y;
      m = fmaxf(m, fmaxf(f.x, f.y));
    }
  }
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  const float ml = m * 1.4426950408889634f;
  float sum = 0.f;
#pragma unroll
  for (int i = 0; i < 64; ++i) {
    x[i] = ex2(x[i] * 1.4426950408889634f - ml);
    sum += x[i];
  }
  sum += __shfl_xor_sync(0xffffffffu, sum, 1);
  const float inv = 1.f / sum;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    uint4 u;
    u.x = pack_bf16(x[c * 8 + 0] * inv, x[c * 8 + 1] * inv);
    u.y = pack_bf16(x[c * 8 + 2] * inv, x[c * 8 + 3] * inv);
    u.z = pack_bf16(x[c * 8 + 4] * inv, x[c * 8 + 5] * inv);
    u.w = pack_bf16(x[c * 8 + 6] * inv, x[c * 8 + 7] * inv);
    *reinterpret_cast<uint4*>(dst_half + row * 128 + ((c ^ (row & 7)) << 4)) = u;
  }
}

// The element-wise maps of the paper's ablation (Table 6) on packed bf16 pairs: ReLU; the
// identity needs no arithmetic at all.
__device__ __forceinline__ uint4 relu_bf16x8(uint4 u) {
  __nv_bfloat162* h = reinterpret_cast<__nv_bfloat162*>(&u);
  const __nv_bfloat162 z = __floats2bfloat162_rn(0.f, 0.f);
#pragma unroll
  for (int e = 0; e < 4; ++e) h[e] = __hmax2(h[e], z);
  return u;
}
// feature_map_pair for any map: softmax as above; ReLU / identity element-wise (src may differ from dst)
__device__ __forceinline__ void feature_map_pair_any(const unsigned char* src_half, unsigned char* dst_half, int row, int phi) {
  if (phi == RATTN_PHI_SOFTMAX) {
    feature_map_pair(src_half, dst_half, row);
    return;
  }
  if (phi == RATTN_PHI_IDENTITY && src_half == dst_half) return;
#pragma unroll
  for (int c = 0; c < 8; ++c) {
    const int off = row * 128 + ((c ^ (row & 7)) << 4);
    const uint4 u = *reinterpret_cast<const uint4*>(src_half + off);
    *reinterpret_cast<uint4*>(dst_half + off) = phi == RATTN_PHI_RELU ? relu_bf16x8(u) : u;
  }
}

// byte offset of 16-byte chunk c (0..15) of row r inside a swizzled [128 x 128] bf16 tile
__device__ __forceinline__ uint32_t swz(int r, int c) {
  return (uint32_t)((c >> 3) * HALF_BYTES + r * 128 + (((c & 7) ^ (r & 7)) << 4));
}

// One [128 x 128] bf16 tile staged in shared memory (swizzled like a loaded tile) goes to
// rows row0.. of matrix z of a tensor map: two 64-column boxes; rows past the end are clipped.
__device__ __forceinline__ void store_tile(const UMap* tm, const unsigned char* tile, int row0, int z) {
  const int b = z / tm->H, h = z - b * tm->H;
  tma_store_4d(&tm->m, tile, 0, row0, h, b);
  tma_store_4d(&tm->m, tile + HALF_BYTES, 64, row0, h, b);
}
// one 64-column half of a staged tile
__device__ __forceinline__ void store_half(const UMap* tm, const unsigned char* half, int x, int row0, int z) {
  const int b = z / tm->H, h = z - b * tm->H;
  tma_store_4d(&tm->m, half, x, row0, h, b);
}
__device__ __forceinline__ void store_tile(const CUtensorMap* tm, const unsigned char* tile, int row0, int z) {
  tma_store_3d(tm, tile, 0, row0, z);
  tma_store_3d(tm, tile + HALF_BYTES, 64, row0, z);
}

// Row-owner r holds 32 fp32 values (columns 32*c .. 32*c+31 of its row).  Stages them in a
// 16 KB region ([128 rows x 128 bytes], 16-byte chunks XOR-swizzled by row) so that the 128
// row owners can then write the [128 x 32] block to global memory with full 128-byte segments.
__device__ __forceinline__ void stage_f32_block(unsigned char* stage, int r, const float (&x)[32]) {
#pragma unroll
  for (int e = 0; e < 8; ++e)
    *reinterpret_cast<float4*>(stage + r * 128 + ((e ^ (r & 7)) << 4)) =
        make_float4(x[4 * e], x[4 * e + 1], x[4 * e + 2], x[4 * e + 3]);
}
// dst points at column 32*c of the tile's first row (row pitch 128 floats); rows >= n_rows are skipped.
__device__ __forceinline__ void flush_f32_block(const unsigned char* stage, int r, float* dst, int n_rows) {
  const int sub = r & 7;
#pragma unroll
  for (int k = 0; k < 8; ++k) {
    const int row = (r >> 5) * 32 + 4 * k + ((r & 31) >> 3);
    const float4 v = *reinterpret_cast<const float4*>(stage + row * 128 + ((sub ^ (row & 7)) << 4));
    if (row < n_rows) *reinterpret_cast<float4*>(dst + (size_t)row * 128 + 4 * sub) = v;
  }
}

// Bit e of the result says whether column 32*c + e of a [128 x 128] score tile is kept for row
// r: on the diagonal tile the keys j <= r, on the oldest tile of the band the keys j >= r.
__device__ __forceinline__ uint32_t keep_bits(int r, int c, bool diag, bool bound) {
  const int rd = r - 32 * c;                      // column of the row's own position in this chunk
  uint32_t m = 0xffffffffu;
  if (diag) m &= rd >= 31 ? 0xffffffffu : (rd < 0 ? 0u : ((2u << rd) - 1u));
  if (bound) m &= rd <= 0 ? 0xffffffffu : (rd > 31 ? 0u : ~((1u << rd) - 1u));
  return m;
}

// bits e >= rd, e > rd, e <= rd of a 32-bit chunk mask (any integer rd)
__device__ __forceinline__ uint32_t bits_ge(int rd) { return rd <= 0 ? 0xffffffffu : (rd > 31 ? 0u : ~((1u << rd) - 1u)); }
__device__ __forceinline__ uint32_t bits_gt(int rd) { return bits_ge(rd + 1); }
__device__ __forceinline__ uint32_t bits_le(int rd) { return ~bits_gt(rd); }
__device__ __forceinline__ uint32_t bits_lt(int rd) { return ~bits_ge(rd); }

// Maximum of 32 registers as four independent chains (the row threads run two or three warps per
// scheduler, so a 32-long dependent chain would sit exposed at full latency).
__device__ __forceinline__ float max32(const float (&x)[32]) {
  float m0 = x[0], m1 = x[1], m2 = x[2], m3 = x[3];
#pragma unroll
  for (int e = 4; e < 32; e += 4) {
    m0 = fmaxf(m0, x[e]);
    m1 = fmaxf(m1, x[e + 1]);
    m2 = fmaxf(m2, x[e + 2]);
    m3 = fmaxf(m3, x[e + 3]);
  }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}
// columns whose keep bit is clear become -inf: no part in the maximum, weight exactly zero
__device__ __forceinline__ void mask32(float (&x)[32], uint32_t keep) {
#pragma unroll
  for (int e = 0; e < 32; ++e) x[e] = (keep >> e) & 1u ? x[e] : -INFINITY;
}
__device__ __forceinline__ float max32_masked(const float (&x)[32], uint32_t keep) {
  float m0 = -INFINITY, m1 = -INFINITY, m2 = -INFINITY, m3 = -INFINITY;
#pragma unroll
  for (int e = 0; e < 32; e += 4) {
    m0 = fmaxf(m0, (keep >> e) & 1u ? x[e] : -INFINITY);
    m1 = fmaxf(m1, (keep >> (e + 1)) & 1u ? x[e + 1] : -INFINITY);
    m2 = fmaxf(m2, (keep >> (e + 2)) & 1u ? x[e + 2] : -INFINITY);
    m3 = fmaxf(m3, (keep >> (e + 3)) & 1u ? x[e + 3] : -INFINITY);
  }
  return fmaxf(fmaxf(m0, m1), fmaxf(m2, m3));
}

// The helpers below walk a row in sixteen 16-byte steps with a rolled loop: compact code
// matters more than loop overhead here (large unrolled kernels are instruction-fetch bound).
// Row maximum of row r of a swizzled bf16 tile.
__device__ __forceinline__ float row_max_bf16(const unsigned char* tile, int r) {
  // packed bf16 maxima (two values per instruction), four independent chains
  __nv_bfloat162 m[4];
  {
    const uint4 u = *reinterpret_cast<const uint4*>(tile + swz(r, 0));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) m[e] = h[e];
  }
#pragma unroll 3
  for (int c = 1; c < 16; ++c) {
    const uint4 u = *reinterpret_cast<const uint4*>(tile + swz(r, c));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) m[e] = __hmax2(m[e], h[e]);
  }
  const float2 f = __bfloat1622float2(__hmax2(__hmax2(m[0], m[1]), __hmax2(m[2], m[3])));
  return fmaxf(f.x, f.y);
}
// x -> exp(x - max) over row r, in place, as fp16 (FP16 = true) or bf16; returns the row sum.
template <bool FP16>
__device__ __forceinline__ float row_exp_inplace(unsigned char* tile, int r, float ml) {
  float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
#pragma unroll 2
  for (int c = 0; c < 16; ++c) {
    uint4 u = *reinterpret_cast<const uint4*>(tile + swz(r, c));
    uint32_t* w = reinterpret_cast<uint32_t*>(&u);
    float ex[8];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[e]));
      ex[2 * e] = ex2(f.x * 1.4426950408889634f - ml);
      ex[2 * e + 1] = ex2(f.y * 1.4426950408889634f - ml);
      w[e] = FP16 ? pack_f16(ex[2 * e], ex[2 * e + 1]) : pack_bf16(ex[2 * e], ex[2 * e + 1]);
    }
    s0 += ex[0] + ex[4];
    s1 += ex[1] + ex[5];
    s2 += ex[2] + ex[6];
    s3 += ex[3] + ex[7];
    *reinterpret_cast<uint4*>(tile + swz(r, c)) = u;
  }
  return (s0 + s1) + (s2 + s3);
}
// Un-normalised feature map of row r, in place: x -> exp(x - max) (bf16); returns 1 / sum so
// that the caller can scale whatever is linear in this row afterwards.
__device__ __forceinline__ float feature_map_row_unnorm_inplace(unsigned char* tile, int r) {
  const float ml = row_max_bf16(tile, r) * 1.4426950408889634f;
  return 1.f / row_exp_inplace<false>(tile, r, ml);
}
// phi of row r, in place, with few live registers: the exponentials are parked in the tile
// itself as fp16 between the summation and the normalisation (one bf16 rounding in the end).
__device__ __forceinline__ void feature_map_row_inplace_lr(unsigned char* tile, int r) {
  const float ml = row_max_bf16(tile, r) * 1.4426950408889634f;
  const float inv = 1.f / row_exp_inplace<true>(tile, r, ml);
#pragma unroll 1
  for (int c = 0; c < 16; ++c) {
    uint4 u = *reinterpret_cast<const uint4*>(tile + swz(r, c));
    uint32_t* w = reinterpret_cast<uint32_t*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&w[e]));
      w[e] = pack_bf16(f.x * inv, f.y * inv);
    }
    *reinterpret_cast<uint4*>(tile + swz(r, c)) = u;
  }
}

// phi (softmax over the 128 features) of row r of a swizzled bf16 tile, in place.
// NORMALISE = false leaves exp(x - max) (bf16) and returns 1 / sum, for callers that scale
// whatever is linear in this row afterwards.  The row lives in 128 registers in between: one
// read and one write of shared memory.
template <bool NORMALISE = true>
__device__ __forceinline__ float feature_map_row_inplace(unsigned char* tile, int r) {
  float x[128];
  float m = -INFINITY;
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    uint4 u = *reinterpret_cast<const uint4*>(tile + swz(r, c));
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      float2 f = __bfloat1622float2(h[e]);
      x[c * 8 + 2 * e] = f.x;
      x[c * 8 + 2 * e + 1] = f.y;
      m = fmaxf(m, fmaxf(f.x, f.y));
    }
  }
  float sum = 0.f;
  const float ml = m * 1.4426950408889634f;
#pragma unroll
  for (int i = 0; i < 128; ++i) {
    x[i] = ex2(x[i] * 1.4426950408889634f - ml);
    sum += x[i];
  }
  const float inv = 1.f / sum, sc = NORMALISE ? inv : 1.f;
#pragma unroll
  for (int c = 0; c < 16; ++c) {
    uint4 u;
    u.x = pack_bf16(x[c * 8 + 0] * sc, x[c * 8 + 1] * sc);
    u.y = pack_bf16(x[c * 8 + 2] * sc, x[c * 8 + 3] * sc);
    u.z = pack_bf16(x[c * 8 + 4] * sc, x[c * 8 + 5] * sc);
    u.w = pack_bf16(x[c * 8 + 6] * sc, x[c * 8 + 7] * sc);
    *reinterpret_cast<uint4*>(tile + swz(r, c)) = u;
  }
  return inv;
}

// phi of row r of a swizzled bf16 tile, in place, for any map.  NORMALISE = false: the softmax
// map leaves exp(x - max) and returns 1 / sum (see feature_map_row_inplace); the element-wise
// maps have no normalisation and return 1.
// The softmax map comes in two forms: fully unrolled with the row in 128 registers (one read and one
// write of shared memory, but 16 KB of code per call site) and compact (rolled loops, two or three
// passes over the row in shared memory, twice the cycles).  The kernels that call this are larger
// than the instruction cache; a caller whose launch executes much other code (the training-mode
// forward) is faster with the compact form, the others with the unrolled one.
template <bool NORMALISE>
__device__ __forceinline__ float feature_map_row_any(unsigned char* tile, int r, int phi, bool compact = false) {
  if (phi == RATTN_PHI_SOFTMAX) {
    if (!compact) return feature_map_row_inplace<NORMALISE>(tile, r);
    if (NORMALISE) {
      feature_map_row_inplace_lr(tile, r);
      return 1.f;
    }
    return feature_map_row_unnorm_inplace(tile, r);
  }
  if (phi == RATTN_PHI_RELU) {
#pragma unroll 4
    for (int c = 0; c < 16; ++c) {
      uint4* p = reinterpret_cast<uint4*>(tile + swz(r, c));
      *p = relu_bf16x8(*p);
    }
  }
  return 1.f;
}

// ------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess) return (EncodeTiledFn) nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// [n_mats, rows, 128] bf16, box = 64 columns x 128 rows x 1, 128-byte swizzle, zero fill.
inline bool make_map(CUtensorMap* m, const void* base, uint64_t rows, uint64_t n_mats, uint32_t box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[3] = {128, rows, n_mats};
  const cuuint64_t strides[2] = {128 * 2, rows * 128 * 2};
  const cuuint32_t box[3] = {64, box_rows, 1};
  const cuuint32_t estr[3] = {1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// A caller's tensor with T rows per head, H heads, B batch entries: [B, H, T, 128] (layout 0) or
// [B, T, H, 128] (layout 1), bf16; box = 64 columns x box_rows rows of one head.
inline bool make_user_map(UMap* u, const void* base, uint64_t T, uint64_t H, uint64_t B, int layout,
                          uint32_t box_rows = 128) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  u->H = (int)H;
  const cuuint64_t dims[4] = {128, T, H, B};
  const cuuint64_t row = 128 * 2;
  const cuuint64_t strides[3] = {layout ? H * row : row, layout ? row : T * row, T * H * row};
  const cuuint32_t box[4] = {64, box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(&u->m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// The same tensor read as whole rows: box = 128 columns x box_rows rows of one head, no swizzle.
inline bool make_row_map(CUtensorMap* m, const void* base, uint64_t T, uint64_t H, uint64_t B, int layout,
                         uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[4] = {128, T, H, B};
  const cuuint64_t row = 128 * 2;
  const cuuint64_t strides[3] = {layout ? H * row : row, layout ? row : T * row, T * H * row};
  const cuuint32_t box[4] = {128, box_rows, 1, 1};
  const cuuint32_t estr[4] = {1, 1, 1, 1};
  return fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// [n_mats, 128, 128] bf16 chunk states.  Modes without a linear branch keep none: the kernels
// then never use the map, which is encoded over one matrix of `any` (some valid bf16 buffer of
// at least 128 x 128 elements) so that it is well formed.
inline bool make_state_map(CUtensorMap* m, const void* states, const void* any, uint64_t n_mats) {
  return states ? make_map(m, states, 128, n_mats) : make_map(m, any, 128, 1);
}

}  // namespace tc
}  // namespace rattn
