// qk-norm and rotary embedding of q and k in one pass (Table 1 "qk-norm"; Section 4 "Model Setup":
// local layers rotate with theta = 5e5, global layers do not), and the gradient of that pass.
//
// Streaming kernels: every element is read once and written once, so the bound is HBM bandwidth.
// A head vector of d features is held by d/16 neighbouring lanes, each with features
// [8l, 8l+8) and [d/2 + 8l, d/2 + 8l + 8): the two halves of its 8 rotation pairs, one 16-byte
// (bf16) or two 16-byte (fp32) loads per half.  A thread keeps one sequence position and walks
// over the heads of a batch entry, so the 8 sines and cosines it needs are computed once and
// used for every head; four heads are loaded before the first is stored, which keeps enough
// loads in flight with inputs and outputs allowed to alias.
#include <cmath>
#include <cstdint>

#include "rattn_internal.h"

namespace rattn {
namespace {

constexpr int QK_THREADS = 256;
constexpr int QK_MAX_CTAS = 2048;     // bounds the partial sums of the gain gradients
constexpr int QK_FWD_BATCH = 4;       // heads in flight per thread, forward
constexpr int QK_BWD_BATCH = 2;       // backward (two tensors per head)

struct Freqs {
  double inv[64];                     // theta^(-2i/d), i < d/2
};

struct QkArgs {
  const void* x[2];                   // q, k
  void* y[2];                         // forward: q_out, k_out; backward: dq, dk
  const void* dy[2];                  // backward: dq_out, dk_out
  const float* gain[2];
  float* partial;                     // backward: [2][n_cta][d] or null
  int H[2];
  int B, T, S, nblk_t;
  float eps;
  int rotate;
  long long pos0;
  const int* pos;
};

struct Geometry {
  int rpb, nblk_t, S, gx, gy;
  int n_cta() const { return gx * gy; }
};

Geometry geometry(int B, int H_q, int H_kv, int T, int d) {
  Geometry g;
  g.rpb = QK_THREADS / (d / 16);
  g.nblk_t = (T + g.rpb - 1) / g.rpb;
  const int heads = H_q + H_kv;
  g.S = heads / 8 < 1 ? 1 : heads / 8 > 8 ? 8 : heads / 8;
  g.gy = B * g.S;
  const int cap = QK_MAX_CTAS / g.gy < 1 ? 1 : QK_MAX_CTAS / g.gy;
  g.gx = g.nblk_t < cap ? g.nblk_t : cap;
  return g;
}

template <typename T> struct Io;
template <> struct Io<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const void* base, size_t elem, float (&x)[8]) {
    const uint4 u = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(base) + elem);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[2 * i] = __uint_as_float(w[i] << 16);
      x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
  static __device__ __forceinline__ void store(void* base, size_t elem, const float (&x)[8]) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(x[2 * i], x[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(base) + elem) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <> struct Io<float> {
  static __device__ __forceinline__ void load(const void* base, size_t elem, float (&x)[8]) {
    const float4* p = reinterpret_cast<const float4*>(static_cast<const float*>(base) + elem);
    const float4 a = p[0], b = p[1];
    x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
  }
  static __device__ __forceinline__ void store(void* base, size_t elem, const float (&x)[8]) {
    float4* p = reinterpret_cast<float4*>(static_cast<float*>(base) + elem);
    p[0] = make_float4(x[0], x[1], x[2], x[3]);
    p[1] = make_float4(x[4], x[5], x[6], x[7]);
  }
};

__device__ __forceinline__ void zero8(float (&x)[8]) {
#pragma unroll
  for (int i = 0; i < 8; ++i) x[i] = 0.f;
}

// Sum over the d/16 lanes that hold one head vector (they are neighbours inside a warp).
template <int LPR>
__device__ __forceinline__ float row_sum(float v) {
#pragma unroll
  for (int o = 1; o < LPR; o <<= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// cos and sin of position * inv_freq for this lane's 8 pairs.  The angle is formed and reduced
// to [-pi, pi] in fp64: an fp32 product would be off by up to 0.01 rad at position 1e5.
__device__ __forceinline__ void rotation(const Freqs& f, int first_pair, long long position, int rotate,
                                         float (&c)[8], float (&s)[8]) {
  constexpr double kTwoPi = 6.283185307179586476925286766559;
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    if (rotate) {
      double ang = (double)position * f.inv[first_pair + j];
      ang -= kTwoPi * rint(ang * (1.0 / kTwoPi));
      sincosf((float)ang, &s[j], &c[j]);
    } else {
      c[j] = 1.f;
      s[j] = 0.f;
    }
  }
}

__device__ __forceinline__ void load_gain(const float* gain, int lo_first, int half, float (&g_lo)[8],
                                          float (&g_hi)[8]) {
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    g_lo[j] = gain ? gain[lo_first + j] : 1.f;
    g_hi[j] = gain ? gain[half + lo_first + j] : 1.f;
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(QK_THREADS, 2) qk_prologue_kernel(const __grid_constant__ QkArgs a, const __grid_constant__ Freqs f) {
  constexpr int LPR = D / 16, RPB = QK_THREADS / LPR, U = QK_FWD_BATCH;
  const int l = threadIdx.x % LPR, row = threadIdx.x / LPR;
  const int b = blockIdx.y / a.S, slice = blockIdx.y % a.S;
  const long long p0 = a.pos ? (long long)a.pos[b] : a.pos0;

  for (int tb = blockIdx.x; tb < a.nblk_t; tb += gridDim.x) {
    const int t = tb * RPB + row;
    const bool live = t < a.T;
    float c[8], s[8];
    rotation(f, 8 * l, p0 + t, a.rotate, c, s);

#pragma unroll 1
    for (int which = 0; which < 2; ++which) {
      const int H = a.H[which];
      if (H == 0) continue;
      float g_lo[8], g_hi[8];
      load_gain(a.gain[which], 8 * l, D / 2, g_lo, g_hi);
      const void* x = a.x[which];
      void* y = a.y[which];
#pragma unroll 1
      for (int h0 = slice; h0 < H; h0 += U * a.S) {
        float lo[U][8], hi[U][8];
        size_t at[U];
        bool on[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * a.S;
          on[u] = live && h < H;
          at[u] = (((size_t)b * H + (on[u] ? h : 0)) * a.T + (live ? t : 0)) * D + 8 * l;
          if (on[u]) {
            Io<T>::load(x, at[u], lo[u]);
            Io<T>::load(x, at[u] + D / 2, hi[u]);
          } else {
            zero8(lo[u]);
            zero8(hi[u]);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          float ss = 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) ss += lo[u][j] * lo[u][j] + hi[u][j] * hi[u][j];
          ss = row_sum<LPR>(ss);
          const float r = rsqrtf(ss * (1.f / D) + a.eps);
          float o_lo[8], o_hi[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float n_lo = lo[u][j] * r * g_lo[j], n_hi = hi[u][j] * r * g_hi[j];
            o_lo[j] = n_lo * c[j] - n_hi * s[j];
            o_hi[j] = n_hi * c[j] + n_lo * s[j];
          }
          if (on[u]) {
            Io<T>::store(y, at[u], o_lo);
            Io<T>::store(y, at[u] + D / 2, o_hi);
          }
        }
      }
    }
  }
}

template <typename T, int D>
__global__ void __launch_bounds__(QK_THREADS, 2) qk_prologue_bwd_kernel(const __grid_constant__ QkArgs a, const __grid_constant__ Freqs f) {
  constexpr int LPR = D / 16, RPB = QK_THREADS / LPR, U = QK_BWD_BATCH;
  __shared__ float red[RPB][D];
  __shared__ __align__(16) float gain_s[D];       // read at each use: the registers go to the loads in flight
  const int l = threadIdx.x % LPR, row = threadIdx.x / LPR;
  const int b = blockIdx.y / a.S, slice = blockIdx.y % a.S;
  const long long p0 = a.pos ? (long long)a.pos[b] : a.pos0;
  const int cta = blockIdx.y * gridDim.x + blockIdx.x, n_cta = gridDim.x * gridDim.y;

  // q, then k: one set of gain-gradient accumulators alive at a time
#pragma unroll 1
  for (int which = 0; which < 2; ++which) {
    const int H = a.H[which];
    float acc[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) acc[i] = 0.f;
    __syncthreads();
    if (threadIdx.x < D) gain_s[threadIdx.x] = a.gain[which] ? a.gain[which][threadIdx.x] : 1.f;
    __syncthreads();
    const float* g_lo = gain_s + 8 * l;
    const float* g_hi = gain_s + D / 2 + 8 * l;
    const void* x = a.x[which];
    const void* dy = a.dy[which];
    void* dx = a.y[which];

    for (int tb = blockIdx.x; tb < a.nblk_t && H > 0; tb += gridDim.x) {
      const int t = tb * RPB + row;
      const bool live = t < a.T;
      float c[8], s[8];
      rotation(f, 8 * l, p0 + t, a.rotate, c, s);
#pragma unroll 1
      for (int h0 = slice; h0 < H; h0 += U * a.S) {
        float lo[U][8], hi[U][8], e_lo[U][8], e_hi[U][8];
        size_t at[U];
        bool on[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
          const int h = h0 + u * a.S;
          on[u] = live && h < H;
          at[u] = (((size_t)b * H + (on[u] ? h : 0)) * a.T + (live ? t : 0)) * D + 8 * l;
          if (on[u]) {
            Io<T>::load(x, at[u], lo[u]);
            Io<T>::load(x, at[u] + D / 2, hi[u]);
            Io<T>::load(dy, at[u], e_lo[u]);
            Io<T>::load(dy, at[u] + D / 2, e_hi[u]);
          } else {
            zero8(lo[u]); zero8(hi[u]); zero8(e_lo[u]); zero8(e_hi[u]);
          }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
          // the rotation is orthogonal: its transpose turns by the opposite angle
          float du_lo[8], du_hi[8];
          float ss = 0.f, dot = 0.f;
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            du_lo[j] = e_lo[u][j] * c[j] + e_hi[u][j] * s[j];
            du_hi[j] = e_hi[u][j] * c[j] - e_lo[u][j] * s[j];
            ss += lo[u][j] * lo[u][j] + hi[u][j] * hi[u][j];
            dot += du_lo[j] * g_lo[j] * lo[u][j] + du_hi[j] * g_hi[j] * hi[u][j];
          }
          ss = row_sum<LPR>(ss);
          dot = row_sum<LPR>(dot);
          const float r = rsqrtf(ss * (1.f / D) + a.eps);
          const float back = r * r * r * dot * (1.f / D);
          float o_lo[8], o_hi[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            acc[j] += du_lo[j] * lo[u][j] * r;
            acc[8 + j] += du_hi[j] * hi[u][j] * r;
            o_lo[j] = r * du_lo[j] * g_lo[j] - lo[u][j] * back;
            o_hi[j] = r * du_hi[j] * g_hi[j] - hi[u][j] * back;
          }
          if (on[u]) {
            Io<T>::store(dx, at[u], o_lo);
            Io<T>::store(dx, at[u] + D / 2, o_hi);
          }
        }
      }
    }

    if (a.partial != nullptr) {
      // per-CTA sum over its rows in row order, then one partial row per CTA
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        red[row][8 * l + j] = acc[j];
        red[row][D / 2 + 8 * l + j] = acc[8 + j];
      }
      __syncthreads();
      if (threadIdx.x < D) {
        float sum = 0.f;
        for (int r = 0; r < RPB; ++r) sum += red[r][threadIdx.x];
        a.partial[((size_t)which * n_cta + cta) * D + threadIdx.x] = sum;
      }
      __syncthreads();
    }
  }
}

// gain gradient = sum of the per-CTA partial sums, added in an order fixed by the sizes alone
template <int D>
__global__ void __launch_bounds__(1024) qk_gain_reduce_kernel(const float* partial, int n_cta, float* dq_gain,
                                                              float* dk_gain) {
  constexpr int SL = 1024 / D;
  __shared__ float part[SL][D];
  float* out = blockIdx.x == 0 ? dq_gain : dk_gain;
  if (out == nullptr) return;
  const int fi = threadIdx.x % D, sl = threadIdx.x / D;
  const float* p = partial + (size_t)blockIdx.x * n_cta * D;
  float sum = 0.f;
  for (int i = sl; i < n_cta; i += SL) sum += p[(size_t)i * D + fi];
  part[sl][fi] = sum;
  __syncthreads();
  if (sl == 0) {
    float tot = 0.f;
    for (int i = 0; i < SL; ++i) tot += part[i][fi];
    out[fi] = tot;
  }
}

bool misaligned16(const void* p) { return ((uintptr_t)p & 15u) != 0; }

int check(const rattn_qk_params* p) {
  if (!p) return RATTN_ERR_NULL_PTR;
  if (p->B < 1 || p->H_q < 1 || p->H_kv < 0 || p->T < 1) return RATTN_ERR_BAD_ARG;
  if (!(p->eps >= 0.f) || std::isinf(p->eps) || std::isnan(p->theta) || std::isinf(p->theta)) return RATTN_ERR_BAD_ARG;
  if (p->pos == nullptr && p->pos0 < 0) return RATTN_ERR_BAD_ARG;
  if (p->d != 64 && p->d != 128) return RATTN_ERR_UNSUPPORTED;
  if (p->dtype != RATTN_BF16 && p->dtype != RATTN_F32) return RATTN_ERR_UNSUPPORTED;
  if (!p->q) return RATTN_ERR_NULL_PTR;
  if (p->H_kv > 0 && !p->k) return RATTN_ERR_NULL_PTR;
  if (misaligned16(p->q) || misaligned16(p->k) || misaligned16(p->q_gain) || misaligned16(p->k_gain))
    return RATTN_ERR_MISALIGNED;
  if (((uintptr_t)p->pos & 3u) != 0) return RATTN_ERR_MISALIGNED;
  if ((long long)p->B * geometry(p->B, p->H_q, p->H_kv, p->T, p->d).S > 65535) return RATTN_ERR_BAD_ARG;
  return RATTN_OK;
}

void fill(const rattn_qk_params* p, const Geometry& g, QkArgs* a, Freqs* f) {
  a->x[0] = p->q; a->x[1] = p->k;
  a->gain[0] = p->q_gain; a->gain[1] = p->k_gain;
  a->H[0] = p->H_q; a->H[1] = p->H_kv;
  a->B = p->B; a->T = p->T; a->S = g.S; a->nblk_t = g.nblk_t;
  a->eps = p->eps;
  a->rotate = p->theta > 0.f;
  a->pos0 = p->pos0;
  a->pos = p->pos;
  a->partial = nullptr;
  a->dy[0] = a->dy[1] = nullptr;
  for (int i = 0; i < 64; ++i)
    f->inv[i] = a->rotate && i < p->d / 2 ? std::pow((double)p->theta, -2.0 * i / p->d) : 0.0;
}

template <typename T>
cudaError_t launch_fwd(const QkArgs& a, const Freqs& f, const Geometry& g, int d, cudaStream_t s) {
  KernelTimer kt("qk_prologue", s);
  const dim3 grid(g.gx, g.gy);
  if (d == 128) qk_prologue_kernel<T, 128><<<grid, QK_THREADS, 0, s>>>(a, f);
  else qk_prologue_kernel<T, 64><<<grid, QK_THREADS, 0, s>>>(a, f);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T>
cudaError_t launch_bwd(const QkArgs& a, const Freqs& f, const Geometry& g, int d, float* dq_gain, float* dk_gain,
                       cudaStream_t s) {
  const dim3 grid(g.gx, g.gy);
  {
    KernelTimer kt("qk_prologue_bwd", s);
    if (d == 128) qk_prologue_bwd_kernel<T, 128><<<grid, QK_THREADS, 0, s>>>(a, f);
    else qk_prologue_bwd_kernel<T, 64><<<grid, QK_THREADS, 0, s>>>(a, f);
    count_launches(1);
  }
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess || a.partial == nullptr) return e;
  KernelTimer kt("qk_gain_reduce", s);
  if (d == 128) qk_gain_reduce_kernel<128><<<2, 1024, 0, s>>>(a.partial, g.n_cta(), dq_gain, dk_gain);
  else qk_gain_reduce_kernel<64><<<2, 1024, 0, s>>>(a.partial, g.n_cta(), dq_gain, dk_gain);
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace
}  // namespace rattn

using namespace rattn;

extern "C" {

size_t rattn_qk_prologue_workspace_bytes(int B, int H_q, int H_kv, int T, int d) {
  if (B < 1 || H_q < 1 || H_kv < 0 || T < 1 || (d != 64 && d != 128)) return 0;
  const Geometry g = geometry(B, H_q, H_kv, T, d);
  return ((size_t)2 * g.n_cta() * d * sizeof(float) + 255) / 256 * 256;
}

int rattn_qk_prologue(const rattn_qk_params* p, void* stream) {
  int rc = check(p);
  if (rc != RATTN_OK) return rc;
  if (!p->q_out || (p->H_kv > 0 && !p->k_out)) return RATTN_ERR_NULL_PTR;
  if (misaligned16(p->q_out) || misaligned16(p->k_out)) return RATTN_ERR_MISALIGNED;
  const Geometry g = geometry(p->B, p->H_q, p->H_kv, p->T, p->d);
  QkArgs a;
  Freqs f;
  fill(p, g, &a, &f);
  a.y[0] = p->q_out; a.y[1] = p->k_out;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const cudaError_t e = p->dtype == RATTN_BF16 ? launch_fwd<__nv_bfloat16>(a, f, g, p->d, s)
                                               : launch_fwd<float>(a, f, g, p->d, s);
  if (e != cudaSuccess) { set_last_cuda_error((int)e); return RATTN_ERR_CUDA; }
  return RATTN_OK;
}

int rattn_qk_prologue_backward(const rattn_qk_params* p, const void* dq_out, const void* dk_out, void* dq, void* dk,
                               float* dq_gain, float* dk_gain, void* workspace, size_t workspace_bytes,
                               void* stream) {
  int rc = check(p);
  if (rc != RATTN_OK) return rc;
  if (!dq_out || !dq || (p->H_kv > 0 && (!dk_out || !dk))) return RATTN_ERR_NULL_PTR;
  if (p->H_kv == 0 && dk_gain) return RATTN_ERR_BAD_ARG;
  if (misaligned16(dq_out) || misaligned16(dk_out) || misaligned16(dq) || misaligned16(dk) ||
      misaligned16(dq_gain) || misaligned16(dk_gain))
    return RATTN_ERR_MISALIGNED;
  const Geometry g = geometry(p->B, p->H_q, p->H_kv, p->T, p->d);
  QkArgs a;
  Freqs f;
  fill(p, g, &a, &f);
  a.y[0] = dq; a.y[1] = dk;
  a.dy[0] = dq_out; a.dy[1] = dk_out;
  if (dq_gain || dk_gain) {
    if (!workspace || workspace_bytes < rattn_qk_prologue_workspace_bytes(p->B, p->H_q, p->H_kv, p->T, p->d) ||
        ((uintptr_t)workspace & 255u) != 0)
      return RATTN_ERR_WORKSPACE;
    a.partial = static_cast<float*>(workspace);
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  const cudaError_t e = p->dtype == RATTN_BF16
                            ? launch_bwd<__nv_bfloat16>(a, f, g, p->d, dq_gain, dk_gain, s)
                            : launch_bwd<float>(a, f, g, p->d, dq_gain, dk_gain, s);
  if (e != cudaSuccess) { set_last_cuda_error((int)e); return RATTN_ERR_CUDA; }
  return RATTN_OK;
}

}  // extern "C"
