// Building blocks of the portable fp32-FMA kernels: padded shared-memory tiles, the
// softmax feature map of Section 3.1 on a tile, and register-tiled products
// (16x16 thread grid, strided micro-tiles so float4 shared-memory reads are conflict-free).
#pragma once
#include "rattn_internal.h"

namespace rattn {
namespace generic {

constexpr int NT = 256;       // threads per CTA
constexpr int PAD = 4;        // fp32 padding per smem row (keeps float4 reads conflict-free)

template <typename T> __device__ __forceinline__ float4 load4(const T* p);
template <> __device__ __forceinline__ float4 load4<float>(const float* p) {
  return *reinterpret_cast<const float4*>(p);
}
template <> __device__ __forceinline__ float4 load4<__nv_bfloat16>(const __nv_bfloat16* p) {
  uint2 u = *reinterpret_cast<const uint2*>(p);
  __nv_bfloat162 a = *reinterpret_cast<__nv_bfloat162*>(&u.x);
  __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&u.y);
  float2 fa = __bfloat1622float2(a), fb = __bfloat1622float2(b);
  return make_float4(fa.x, fa.y, fb.x, fb.y);
}
template <typename T> __device__ __forceinline__ void store4(T* p, float4 v);
template <> __device__ __forceinline__ void store4<float>(float* p, float4 v) {
  *reinterpret_cast<float4*>(p) = v;
}
template <> __device__ __forceinline__ void store4<__nv_bfloat16>(__nv_bfloat16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y);
  __nv_bfloat162 b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<uint32_t*>(&a);
  u.y = *reinterpret_cast<uint32_t*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// Where head (b, h) of a caller's tensor with H heads and T rows per head starts, and the distance
// between its rows, in elements: [B, H, T, D] (layout 0) or [B, T, H, D] (layout 1).
template <int D>
__device__ __forceinline__ size_t head_base(int b, int h, int H, int T, int layout) {
  return layout ? ((size_t)b * T * H + h) * D : ((size_t)b * H + h) * (size_t)T * D;
}
template <int D>
__device__ __forceinline__ size_t row_pitch(int H, int layout) { return layout ? (size_t)H * D : (size_t)D; }

// Copy a [ROWS, D] tile (rows row0.., zero beyond n_rows; `pitch` elements between rows) into padded fp32
// shared memory.
template <typename TIO, int D, int ROWS>
__device__ __forceinline__ void load_tile(float* dst, const TIO* src, int row0, int n_rows, int tid, size_t pitch = D) {
  constexpr int LD = D + PAD;
  constexpr int V4 = D / 4;
  for (int i = tid; i < ROWS * V4; i += NT) {
    int r = i / V4, c = (i % V4) * 4;
    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < n_rows) x = load4<TIO>(src + (size_t)(row0 + r) * pitch + c);
    *reinterpret_cast<float4*>(dst + r * LD + c) = x;
  }
}

// phi of each of the ROWS (<= 64) rows of src, written to dst (Section 3.1): softmax over the
// D features, or one of the element-wise maps of the paper's ablation.  Four threads per row.
template <int D, int ROWS>
__device__ __forceinline__ void feature_map_tile(float* dst, const float* src, int tid, int phi) {
  constexpr int LD = D + PAD;
  int r = tid >> 2, part = tid & 3;
  if (r >= ROWS) return;            // whole warps drop out (ROWS is a multiple of 8)
  const float* s = src + r * LD;
  if (phi != RATTN_PHI_SOFTMAX) {
    float* o = dst + r * LD;
    for (int a = part; a < D; a += 4) o[a] = phi == RATTN_PHI_RELU ? fmaxf(s[a], 0.f) : s[a];
    return;
  }
  float m = -INFINITY;
  for (int a = part; a < D; a += 4) m = fmaxf(m, s[a]);
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 1));
  m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 2));
  float sum = 0.f;
  float* o = dst + r * LD;
  for (int a = part; a < D; a += 4) {
    float e = __expf(s[a] - m);
    o[a] = e;
    sum += e;
  }
  sum += __shfl_xor_sync(0xffffffffu, sum, 1);
  sum += __shfl_xor_sync(0xffffffffu, sum, 2);
  float inv = 1.f / sum;
  for (int a = part; a < D; a += 4) o[a] *= inv;
}

// Gradient through the feature map for one element: f = phi(x), df = dL/df, dot = <df, f> over
// the row (used by the softmax map only).
__device__ __forceinline__ float feature_map_grad(int phi, float f, float df, float dot) {
  if (phi == RATTN_PHI_SOFTMAX) return f * (df - dot);
  if (phi == RATTN_PHI_RELU) return f > 0.f ? df : 0.f;       // relu(x) > 0 exactly where x > 0
  return df;
}

__device__ __forceinline__ float group16_max(float x) {
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 1));
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 2));
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 4));
  x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, 8));
  return x;
}
__device__ __forceinline__ float group16_sum(float x) {
  x += __shfl_xor_sync(0xffffffffu, x, 1);
  x += __shfl_xor_sync(0xffffffffu, x, 2);
  x += __shfl_xor_sync(0xffffffffu, x, 4);
  x += __shfl_xor_sync(0xffffffffu, x, 8);
  return x;
}

// scores[i][j] = sum_a A[ty+16i][a] * Bt[tx+16j][a]   (A has 16*NA rows, Bt has 16*NB rows)
template <int D, int NA, int NB>
__device__ __forceinline__ void tile_scores(float (&s)[NA][NB], const float* A, const float* Bt,
                                            int ty, int tx) {
  constexpr int LD = D + PAD;
#pragma unroll
  for (int i = 0; i < NA; ++i)
#pragma unroll
    for (int j = 0; j < NB; ++j) s[i][j] = 0.f;
#pragma unroll 4
  for (int a = 0; a < D; a += 4) {
    float4 av[NA], bv[NB];
#pragma unroll
    for (int i = 0; i < NA; ++i) av[i] = *reinterpret_cast<const float4*>(A + (ty + 16 * i) * LD + a);
#pragma unroll
    for (int j = 0; j < NB; ++j) bv[j] = *reinterpret_cast<const float4*>(Bt + (tx + 16 * j) * LD + a);
#pragma unroll
    for (int i = 0; i < NA; ++i)
#pragma unroll
      for (int j = 0; j < NB; ++j)
        s[i][j] += av[i].x * bv[j].x + av[i].y * bv[j].y + av[i].z * bv[j].z + av[i].w * bv[j].w;
  }
}

// acc[i][c] += sum_{j<NJ} P[ty+16i][j] * V[j][tx*4 + 64c .. +3]   (P has 16*NA rows of NJ+PAD)
template <int D, int NA, int NJ>
__device__ __forceinline__ void tile_pv(float4 (&acc)[NA][D / 64], const float* P, const float* V,
                                        int ty, int tx) {
  constexpr int LD = D + PAD;
  constexpr int LP = NJ + PAD;
#pragma unroll 2
  for (int j = 0; j < NJ; j += 4) {
    float4 p[NA];
#pragma unroll
    for (int i = 0; i < NA; ++i) p[i] = *reinterpret_cast<const float4*>(P + (ty + 16 * i) * LP + j);
#pragma unroll
    for (int jj = 0; jj < 4; ++jj) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        float4 v = *reinterpret_cast<const float4*>(V + (j + jj) * LD + tx * 4 + 64 * c);
#pragma unroll
        for (int i = 0; i < NA; ++i) {
          float pv = jj == 0 ? p[i].x : jj == 1 ? p[i].y : jj == 2 ? p[i].z : p[i].w;
          acc[i][c].x += pv * v.x;
          acc[i][c].y += pv * v.y;
          acc[i][c].z += pv * v.z;
          acc[i][c].w += pv * v.w;
        }
      }
    }
  }
}

}  // namespace generic
}  // namespace rattn
