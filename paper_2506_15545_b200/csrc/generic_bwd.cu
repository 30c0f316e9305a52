// Portable backward kernels (fp32 FMA arithmetic, any window, any T, d in {64,128}).
//
// The paper prints no backward formulas; these follow from its definitions by the chain
// rule.  With o_s, o_r the un-normalised branch outputs saved by the forward:
//   norm (Section 3.2):  r = sqrt(mean(o^2)+eps), n = o/r, gh = dy*gamma,
//                        do = (gh - n*mean(gh*n))/r,   dgamma += dy*n
//   SWA (Section 2.1):   p_tj = exp(scale q_t.k_j - lse_t);  D_t = do_s_t . o_s_t
//                        ds_tj = p_tj (do_s_t.v_j - D_t)
//                        dq_t += scale ds k_j; dk_j += scale ds q_t; dv_j += p do_s_t
//   RLA (Eq. 4 unrolled, j < t-w):  a_tj = phi(q_t).phi(k_j);  da_tj = do_r_t.v_j
//                        dphi_q_t += da phi(k_j); dphi_k_j += da phi(q_t); dv_j += a do_r_t
//   feature map (Section 3.1):  dx = phi * (dphi - <dphi, phi>)
//   GQA: dk, dv of a K/V head sum over the query heads of its group.
// Three launches: a per-row preprocess, a dq kernel (one CTA per query tile) and a dk/dv
// kernel (one CTA per key tile that loops over the group's heads), so no atomics are
// needed for dq/dk/dv and the result is deterministic.
#include "generic_common.cuh"

namespace rattn {
namespace {

using namespace generic;

__device__ __forceinline__ float warp_sum32(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// One warp per (b,h,t) row: do_s, do_r, D_t and the gain gradients.
template <typename TIO, int D>
__global__ void __launch_bounds__(256) bwd_preprocess_kernel(Args a, float* __restrict__ do_s,
                                                             float* __restrict__ do_r,
                                                             float* __restrict__ delta) {
  const int lane = threadIdx.x & 31;
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  const size_t n_rows = (size_t)a.B * a.H_q * a.T;
  if (row >= n_rows) return;
  const int h = (int)((row / a.T) % a.H_q);
  constexpr int E = D / 32;
  const int bq_ = (int)(row / a.T), t_ = (int)(row - (size_t)bq_ * a.T);
  const TIO* dy = reinterpret_cast<const TIO*>(a.dout) + head_base<D>(bq_ / a.H_q, bq_ % a.H_q, a.H_q, a.T, a.layout) +
                  (size_t)t_ * row_pitch<D>(a.H_q, a.layout);
  float xs[E], xr[E], g[E];
  float ss = 0.f, sr = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int c = lane + 32 * e;
    xs[e] = a.o_swa[row * D + c];
    xr[e] = a.o_rla[row * D + c];
    g[e] = (float)dy[c];
    ss += xs[e] * xs[e];
    sr += xr[e] * xr[e];
  }
  ss = warp_sum32(ss);
  sr = warp_sum32(sr);
  const float is = rsqrtf(ss / D + a.eps), ir = rsqrtf(sr / D + a.eps);
  float ms = 0.f, mr = 0.f;
  float ghs[E], ghr[E];
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int c = lane + 32 * e;
    const float gs = a.gamma_swa ? a.gamma_swa[(size_t)h * D + c] : 1.f;
    const float gr = a.gamma_rla ? a.gamma_rla[(size_t)h * D + c] : 1.f;
    ghs[e] = g[e] * gs;
    ghr[e] = g[e] * gr;
    ms += ghs[e] * xs[e] * is;
    mr += ghr[e] * xr[e] * ir;
    if (a.dgamma_swa) atomicAdd(a.dgamma_swa + (size_t)h * D + c, g[e] * xs[e] * is);
    if (a.dgamma_rla && a.mode == RATTN_MODE_RATTN)
      atomicAdd(a.dgamma_rla + (size_t)h * D + c, g[e] * xr[e] * ir);
  }
  ms = warp_sum32(ms) / D;
  mr = warp_sum32(mr) / D;
  float dl = 0.f;
#pragma unroll
  for (int e = 0; e < E; ++e) {
    const int c = lane + 32 * e;
    const float ds = (ghs[e] - xs[e] * is * ms) * is;
    const float dr = (ghr[e] - xr[e] * ir * mr) * ir;
    do_s[row * D + c] = ds;
    do_r[row * D + c] = dr;
    dl += ds * xs[e];
  }
  dl = warp_sum32(dl);
  if (lane == 0) delta[row] = dl;
}

// ---------------------------------------------------------------------------------- dq
template <typename TIO, int D>
__global__ void __launch_bounds__(NT) bwd_dq_kernel(Args a, const float* __restrict__ do_s,
                                                    const float* __restrict__ do_r,
                                                    const float* __restrict__ delta) {
  constexpr int BQ = 32, BK = 64, LD = D + PAD, LP = BK + PAD;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;                  // [BQ][LD]
  float* Fq = Qs + BQ * LD;
  float* Gs = Fq + BQ * LD;          // do_s tile
  float* Gr = Gs + BQ * LD;          // do_r tile
  float* Ks = Gr + BQ * LD;          // [BK][LD]
  float* Vs = Ks + BK * LD;
  float* Fk = Vs + BK * LD;
  float* Ps = Fk + BK * LD;          // [BQ][LP]
  float* lse_s = Ps + BQ * LP;       // [BQ]
  float* del_s = lse_s + BQ;

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int n_qt = (a.T + BQ - 1) / BQ;
  const int qt = n_qt - 1 - blockIdx.x;
  const int bh = blockIdx.y, b = bh / a.H_q, h = bh % a.H_q, hk = h / a.group;
  const int q0 = qt * BQ, T = a.T, w = a.w;
  const bool rla_on = (a.mode == RATTN_MODE_RATTN);
  const size_t row_base = ((size_t)b * a.H_q + h) * T;
  const size_t q_pitch = row_pitch<D>(a.H_q, a.layout), kv_pitch = row_pitch<D>(a.H_kv, a.layout);
  const TIO* qg = reinterpret_cast<const TIO*>(a.q) + head_base<D>(b, h, a.H_q, T, a.layout);
  const TIO* kg = reinterpret_cast<const TIO*>(a.k) + head_base<D>(b, hk, a.H_kv, T, a.layout);
  const TIO* vg = reinterpret_cast<const TIO*>(a.v) + head_base<D>(b, hk, a.H_kv, T, a.layout);

  load_tile<TIO, D, BQ>(Qs, qg, q0, T, tid, q_pitch);
  load_tile<float, D, BQ>(Gs, do_s + row_base * D, q0, T, tid);
  load_tile<float, D, BQ>(Gr, do_r + row_base * D, q0, T, tid);
  if (tid < BQ) {
    const int t = q0 + tid;
    lse_s[tid] = t < T ? a.lse[row_base + t] : 0.f;
    del_s[tid] = t < T ? delta[row_base + t] : 0.f;
  }
  __syncthreads();
  if (rla_on) feature_map_tile<D, BQ>(Fq, Qs, tid, a.phi);

  float4 dq[2][D / 64], dfq[2][D / 64];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
      dq[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
      dfq[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }

  const int q_last = min(q0 + BQ, T) - 1;
  const int n_kt = q_last / BK + 1;
  for (int kt = 0; kt < n_kt; ++kt) {
    const int j0 = kt * BK;
    const bool need_swa = (j0 + BK - 1 >= q0 - w);
    const bool need_rla = rla_on && (j0 < q_last - w);
    if (!need_swa && !need_rla) continue;
    __syncthreads();
    load_tile<TIO, D, BK>(Ks, kg, j0, T, tid, kv_pitch);
    load_tile<TIO, D, BK>(Vs, vg, j0, T, tid, kv_pitch);
    __syncthreads();
    if (need_rla) feature_map_tile<D, BK>(Fk, Ks, tid, a.phi);
    if (need_swa) {
      float s[2][4], dp[2][4];
      tile_scores<D, 2, 4>(s, Qs, Ks, ty, tx);
      tile_scores<D, 2, 4>(dp, Gs, Vs, ty, tx);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int r = ty + 16 * i, t = q0 + r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int jj = j0 + tx + 16 * j;
          const bool ok = (jj <= t) && (jj >= t - w) && (t < T);
          const float p = ok ? __expf(s[i][j] * a.scale - lse_s[r]) : 0.f;
          Ps[r * LP + tx + 16 * j] = p * (dp[i][j] - del_s[r]) * a.scale;
        }
      }
      __syncthreads();
      tile_pv<D, 2, BK>(dq, Ps, Ks, ty, tx);
    }
    if (need_rla) {
      __syncthreads();
      float da[2][4];
      tile_scores<D, 2, 4>(da, Gr, Vs, ty, tx);
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int r = ty + 16 * i, t = q0 + r;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int jj = j0 + tx + 16 * j;
          Ps[r * LP + tx + 16 * j] = (jj < t - w && t < T) ? da[i][j] : 0.f;
        }
      }
      __syncthreads();
      tile_pv<D, 2, BK>(dfq, Ps, Fk, ty, tx);
    }
  }
  // dq += gradient through phi: phi(q) * (dphi_q - <dphi_q, phi(q)>) for the softmax map
  TIO* dqg = reinterpret_cast<TIO*>(a.dq) + head_base<D>(b, h, a.H_q, T, a.layout);
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int r = ty + 16 * i, t = q0 + r;
    float dot = 0.f;
    float4 f[D / 64];
    if (rla_on) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        f[c] = *reinterpret_cast<const float4*>(Fq + r * LD + tx * 4 + 64 * c);
        dot += f[c].x * dfq[i][c].x + f[c].y * dfq[i][c].y + f[c].z * dfq[i][c].z + f[c].w * dfq[i][c].w;
      }
      dot = group16_sum(dot);
    }
    if (t < T) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        float4 o = dq[i][c];
        if (rla_on) {
          o.x += feature_map_grad(a.phi, f[c].x, dfq[i][c].x, dot);
          o.y += feature_map_grad(a.phi, f[c].y, dfq[i][c].y, dot);
          o.z += feature_map_grad(a.phi, f[c].z, dfq[i][c].z, dot);
          o.w += feature_map_grad(a.phi, f[c].w, dfq[i][c].w, dot);
        }
        store4<TIO>(dqg + (size_t)t * q_pitch + tx * 4 + 64 * c, o);
      }
    }
  }
}

// ------------------------------------------------------------------------------ dk, dv
template <typename TIO, int D>
__global__ void __launch_bounds__(NT) bwd_dkv_kernel(Args a, const float* __restrict__ do_s,
                                                     const float* __restrict__ do_r,
                                                     const float* __restrict__ delta) {
  constexpr int BQ = 32, BK = 64, LD = D + PAD, LP = BQ + PAD;
  extern __shared__ __align__(16) float smem[];
  float* Ks = smem;                  // [BK][LD]
  float* Vs = Ks + BK * LD;
  float* Fk = Vs + BK * LD;
  float* Qs = Fk + BK * LD;          // [BQ][LD]
  float* Fq = Qs + BQ * LD;
  float* Gs = Fq + BQ * LD;
  float* Gr = Gs + BQ * LD;
  float* Ps = Gr + BQ * LD;          // [BK][LP]  (key rows, query columns)
  float* lse_s = Ps + BK * LP;
  float* del_s = lse_s + BQ;

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int kt = blockIdx.x;
  const int bhk = blockIdx.y, b = bhk / a.H_kv, hk = bhk % a.H_kv;
  const int j0 = kt * BK, T = a.T, w = a.w;
  const bool rla_on = (a.mode == RATTN_MODE_RATTN);
  const size_t q_pitch = row_pitch<D>(a.H_q, a.layout), kv_pitch = row_pitch<D>(a.H_kv, a.layout);
  const size_t kv_head = head_base<D>(b, hk, a.H_kv, T, a.layout);
  const TIO* kg = reinterpret_cast<const TIO*>(a.k) + kv_head;
  const TIO* vg = reinterpret_cast<const TIO*>(a.v) + kv_head;

  load_tile<TIO, D, BK>(Ks, kg, j0, T, tid, kv_pitch);
  load_tile<TIO, D, BK>(Vs, vg, j0, T, tid, kv_pitch);
  __syncthreads();
  if (rla_on) feature_map_tile<D, BK>(Fk, Ks, tid, a.phi);

  float4 dk[4][D / 64], dv[4][D / 64], dfk[4][D / 64];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
      dk[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
      dv[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
      dfk[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }

  const int n_qt = (T + BQ - 1) / BQ;
  for (int hh = 0; hh < a.group; ++hh) {
    const int h = hk * a.group + hh;
    const size_t row_base = ((size_t)b * a.H_q + h) * T;
    const TIO* qg = reinterpret_cast<const TIO*>(a.q) + head_base<D>(b, h, a.H_q, T, a.layout);
    for (int qt = j0 / BQ; qt < n_qt; ++qt) {
      const int q0 = qt * BQ, q_last = min(q0 + BQ, T) - 1;
      const bool need_swa = (j0 <= q_last) && (j0 + BK - 1 >= q0 - w);
      const bool need_rla = rla_on && (j0 < q_last - w);
      if (!need_swa && !need_rla) continue;
      __syncthreads();
      load_tile<TIO, D, BQ>(Qs, qg, q0, T, tid, q_pitch);
      load_tile<float, D, BQ>(Gs, do_s + row_base * D, q0, T, tid);
      if (need_rla) load_tile<float, D, BQ>(Gr, do_r + row_base * D, q0, T, tid);
      if (tid < BQ) {
        const int t = q0 + tid;
        lse_s[tid] = t < T ? a.lse[row_base + t] : 0.f;
        del_s[tid] = t < T ? delta[row_base + t] : 0.f;
      }
      __syncthreads();
      if (need_rla) feature_map_tile<D, BQ>(Fq, Qs, tid, a.phi);
      if (need_swa) {
        float s[4][2], dp[4][2];
        tile_scores<D, 4, 2>(s, Ks, Qs, ty, tx);
        tile_scores<D, 4, 2>(dp, Vs, Gs, ty, tx);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int jj = j0 + ty + 16 * i;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = tx + 16 * j, t = q0 + c;
            const bool ok = (jj <= t) && (jj >= t - w) && (t < T);
            s[i][j] = ok ? __expf(s[i][j] * a.scale - lse_s[c]) : 0.f;
            Ps[(ty + 16 * i) * LP + c] = s[i][j];
          }
        }
        __syncthreads();
        tile_pv<D, 4, BQ>(dv, Ps, Gs, ty, tx);
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = tx + 16 * j;
            Ps[(ty + 16 * i) * LP + c] = s[i][j] * (dp[i][j] - del_s[c]) * a.scale;
          }
        __syncthreads();
        tile_pv<D, 4, BQ>(dk, Ps, Qs, ty, tx);
      }
      if (need_rla) {
        __syncthreads();
        float at[4][2], da[4][2];
        tile_scores<D, 4, 2>(at, Fk, Fq, ty, tx);
        tile_scores<D, 4, 2>(da, Vs, Gr, ty, tx);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int jj = j0 + ty + 16 * i;
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const int c = tx + 16 * j, t = q0 + c;
            const bool ok = (jj < t - w) && (t < T);
            da[i][j] = ok ? da[i][j] : 0.f;
            Ps[(ty + 16 * i) * LP + c] = ok ? at[i][j] : 0.f;
          }
        }
        __syncthreads();
        tile_pv<D, 4, BQ>(dv, Ps, Gr, ty, tx);
        __syncthreads();
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 2; ++j) Ps[(ty + 16 * i) * LP + tx + 16 * j] = da[i][j];
        __syncthreads();
        tile_pv<D, 4, BQ>(dfk, Ps, Fq, ty, tx);
      }
    }
  }
  TIO* dkg = reinterpret_cast<TIO*>(a.dk) + kv_head;
  TIO* dvg = reinterpret_cast<TIO*>(a.dv) + kv_head;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = ty + 16 * i, jj = j0 + r;
    float dot = 0.f;
    float4 f[D / 64];
    if (rla_on) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        f[c] = *reinterpret_cast<const float4*>(Fk + r * LD + tx * 4 + 64 * c);
        dot += f[c].x * dfk[i][c].x + f[c].y * dfk[i][c].y + f[c].z * dfk[i][c].z + f[c].w * dfk[i][c].w;
      }
      dot = group16_sum(dot);
    }
    if (jj < T) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        float4 o = dk[i][c];
        if (rla_on) {
          o.x += feature_map_grad(a.phi, f[c].x, dfk[i][c].x, dot);
          o.y += feature_map_grad(a.phi, f[c].y, dfk[i][c].y, dot);
          o.z += feature_map_grad(a.phi, f[c].z, dfk[i][c].z, dot);
          o.w += feature_map_grad(a.phi, f[c].w, dfk[i][c].w, dot);
        }
        store4<TIO>(dkg + (size_t)jj * kv_pitch + tx * 4 + 64 * c, o);
        store4<TIO>(dvg + (size_t)jj * kv_pitch + tx * 4 + 64 * c, dv[i][c]);
      }
    }
  }
}

template <typename TIO, int D>
cudaError_t launch_bwd(const Args& a, cudaStream_t s) {
  const size_t n_rows = (size_t)a.B * a.H_q * a.T;
  float* do_s = a.do_swa;
  float* do_r = a.do_rla;
  float* delta = a.delta;
  cudaError_t e;
  if (a.dgamma_swa) {
    e = cudaMemsetAsync(a.dgamma_swa, 0, sizeof(float) * a.H_q * D, s);
    if (e != cudaSuccess) return e;
  }
  if (a.dgamma_rla) {
    e = cudaMemsetAsync(a.dgamma_rla, 0, sizeof(float) * a.H_q * D, s);
    if (e != cudaSuccess) return e;
  }
  { KernelTimer kt("generic_bwd_preprocess", s);
    bwd_preprocess_kernel<TIO, D><<<(unsigned)((n_rows + 7) / 8), 256, 0, s>>>(a, do_s, do_r, delta); }
  constexpr int LD = D + PAD;
  constexpr size_t smem_dq = (size_t)(4 * 32 * LD + 3 * 64 * LD + 32 * (64 + PAD) + 64) * sizeof(float);
  constexpr size_t smem_dkv = (size_t)(4 * 32 * LD + 3 * 64 * LD + 64 * (32 + PAD) + 64) * sizeof(float);
  e = cudaFuncSetAttribute(bwd_dq_kernel<TIO, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dq);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(bwd_dkv_kernel<TIO, D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_dkv);
  if (e != cudaSuccess) return e;
  dim3 gq((a.T + 31) / 32, a.B * a.H_q);
  { KernelTimer kt("generic_bwd_dq", s); bwd_dq_kernel<TIO, D><<<gq, NT, smem_dq, s>>>(a, do_s, do_r, delta); }
  dim3 gk((a.T + 63) / 64, a.B * a.H_kv);
  { KernelTimer kt("generic_bwd_dkv", s); bwd_dkv_kernel<TIO, D><<<gk, NT, smem_dkv, s>>>(a, do_s, do_r, delta); }
  count_launches(3);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_generic_backward(const Args& a, cudaStream_t s) {
  if (a.dtype == RATTN_F32)
    return a.d == 64 ? launch_bwd<float, 64>(a, s) : launch_bwd<float, 128>(a, s);
  return a.d == 64 ? launch_bwd<__nv_bfloat16, 64>(a, s) : launch_bwd<__nv_bfloat16, 128>(a, s);
}

}  // namespace rattn
