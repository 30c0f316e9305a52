// Portable forward kernel: fp32 FMA arithmetic, any window, any T, d in {64,128},
// fp32 or bf16 I/O.  It evaluates both branches tile by tile in their quadratic form:
//   SWA (Section 2.1): online softmax over the key tiles that intersect the band,
//   RLA (Eq. 4 unrolled): sum over residual keys of (phi(q).phi(k)) v,
// then applies the two RMS norms of Section 3.2.  It is the path for the fp32
// configuration and for shapes the tensor-core kernels do not take.
#include "generic_common.cuh"

namespace rattn {
namespace {

using namespace generic;
constexpr int BM = 64;        // query rows per CTA
constexpr int BN = 64;        // keys per tile

template <typename TIO, int D>
__global__ void __launch_bounds__(NT) generic_fwd_kernel(Args a) {
  constexpr int LD = D + PAD;
  constexpr int LP = BN + PAD;
  extern __shared__ __align__(16) float smem[];
  float* Qs = smem;
  float* Fq = Qs + BM * LD;
  float* Ks = Fq + BM * LD;
  float* Fk = Ks + BN * LD;
  float* Vs = Fk + BN * LD;
  float* Ps = Vs + BN * LD;

  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int n_qt = (a.T + BM - 1) / BM;
  const int qt = n_qt - 1 - blockIdx.x;          // long rows first
  const int bh = blockIdx.y;
  const int b = bh / a.H_q, h = bh % a.H_q, hk = h / a.group;
  const int q0 = qt * BM;
  // T: this entry's valid query rows (variable-length batches); Tk, off: key rows and the key
  // position of query row 0 (a resumed sequence carries its history in front of the chunk)
  const int T = a.seq_lens ? min(a.T, a.seq_lens[b]) : a.T, w = a.w;
  const int off = a.q_off, Tk = a.seq_lens ? T : a.Tk;
  const bool rla_on = (a.mode == RATTN_MODE_RATTN);
  if (q0 >= T) return;

  const size_t q_pitch = row_pitch<D>(a.H_q, a.layout), kv_pitch = row_pitch<D>(a.H_kv, a.kv_layout);
  const TIO* qg = reinterpret_cast<const TIO*>(a.q) + head_base<D>(b, h, a.H_q, a.T, a.layout);
  const TIO* kg = reinterpret_cast<const TIO*>(a.k) + head_base<D>(b, hk, a.H_kv, a.Tk, a.kv_layout);
  const TIO* vg = reinterpret_cast<const TIO*>(a.v) + head_base<D>(b, hk, a.H_kv, a.Tk, a.kv_layout);

  load_tile<TIO, D, 64>(Qs, qg, q0, T, tid, q_pitch);
  __syncthreads();
  if (rla_on) feature_map_tile<D, 64>(Fq, Qs, tid, a.phi);

  float m_run[4], l_run[4];
  float4 acc_s[4][D / 64], acc_r[4][D / 64];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    m_run[i] = -INFINITY;
    l_run[i] = 0.f;
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
      acc_s[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
      acc_r[i][c] = make_float4(0.f, 0.f, 0.f, 0.f);
    }
  }

  const int q_last = min(q0 + BM, T) - 1;
  const int n_kt = (q_last + off) / BN + 1;
  for (int kt = 0; kt < n_kt; ++kt) {
    const int j0 = kt * BN;
    // some row t in [q0, q_last] has this tile's keys inside its window / residual set
    const bool need_swa = (j0 + BN - 1 >= q0 + off - w);
    const bool need_rla = rla_on && (j0 < q_last + off - w);
    if (!need_swa && !need_rla) continue;
    __syncthreads();                              // previous tile fully consumed
    load_tile<TIO, D, 64>(Ks, kg, j0, Tk, tid, kv_pitch);
    load_tile<TIO, D, 64>(Vs, vg, j0, Tk, tid, kv_pitch);
    __syncthreads();
    if (need_rla) feature_map_tile<D, 64>(Fk, Ks, tid, a.phi);

    if (need_swa) {
      float s[4][4];
      tile_scores<D, 4, 4>(s, Qs, Ks, ty, tx);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = q0 + ty + 16 * i, tk = t + off;
        float mx = -INFINITY;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int jj = j0 + tx + 16 * j;
          const bool ok = (jj <= tk) && (jj >= tk - w) && (t < T);
          s[i][j] = ok ? s[i][j] * a.scale : -INFINITY;
          mx = fmaxf(mx, s[i][j]);
        }
        mx = group16_max(mx);
        const float m_new = fmaxf(m_run[i], mx);
        const float corr = (m_new == -INFINITY) ? 1.f : __expf(m_run[i] - m_new);
        float rs = 0.f;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const float p = (s[i][j] == -INFINITY) ? 0.f : __expf(s[i][j] - m_new);
          rs += p;
          Ps[(ty + 16 * i) * LP + tx + 16 * j] = p;
        }
        rs = group16_sum(rs);
        l_run[i] = l_run[i] * corr + rs;
        m_run[i] = m_new;
#pragma unroll
        for (int c = 0; c < D / 64; ++c) {
          acc_s[i][c].x *= corr; acc_s[i][c].y *= corr; acc_s[i][c].z *= corr; acc_s[i][c].w *= corr;
        }
      }
      __syncthreads();
      tile_pv<D, 4, 64>(acc_s, Ps, Vs, ty, tx);
    }
    if (need_rla) {
      __syncthreads();                            // Fk written, Ps free again
      float s[4][4];
      tile_scores<D, 4, 4>(s, Fq, Fk, ty, tx);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const int t = q0 + ty + 16 * i;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          const int jj = j0 + tx + 16 * j;
          Ps[(ty + 16 * i) * LP + tx + 16 * j] = (jj < t + off - w && t < T) ? s[i][j] : 0.f;
        }
      }
      __syncthreads();
      tile_pv<D, 4, 64>(acc_r, Ps, Vs, ty, tx);
    }
  }

  // A resumed sequence: the tokens before the history reach every row through the incoming state,
  // o_rla += phi(q) S_in (Eq. 4), 64 feature rows of S_in at a time.
  if (rla_on && a.state_in) {
    const float* Sg = a.state_in + ((size_t)b * a.H_kv + hk) * D * D;
    for (int f0 = 0; f0 < D; f0 += 64) {
      __syncthreads();
      for (int i = tid; i < 64 * (D / 4); i += NT) {
        const int r = i / (D / 4), c = (i % (D / 4)) * 4;
        *reinterpret_cast<float4*>(Vs + r * LD + c) = *reinterpret_cast<const float4*>(Sg + (size_t)(f0 + r) * D + c);
      }
      for (int i = tid; i < 64 * 64; i += NT) {
        const int r = i >> 6, c = i & 63;
        Ps[r * LP + c] = Fq[r * LD + f0 + c];
      }
      __syncthreads();
      tile_pv<D, 4, 64>(acc_r, Ps, Vs, ty, tx);
    }
  }

  // Section 3.2: two separate RMS norms, then the sum.
  TIO* og = reinterpret_cast<TIO*>(a.out) + head_base<D>(b, h, a.H_q, a.T, a.layout);
  const size_t row_base = ((size_t)b * a.H_q + h) * a.T;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int t = q0 + ty + 16 * i;
    const float inv_l = (l_run[i] > 0.f) ? 1.f / l_run[i] : 0.f;
    float ss = 0.f, sr = 0.f;
#pragma unroll
    for (int c = 0; c < D / 64; ++c) {
      acc_s[i][c].x *= inv_l; acc_s[i][c].y *= inv_l; acc_s[i][c].z *= inv_l; acc_s[i][c].w *= inv_l;
      ss += acc_s[i][c].x * acc_s[i][c].x + acc_s[i][c].y * acc_s[i][c].y +
            acc_s[i][c].z * acc_s[i][c].z + acc_s[i][c].w * acc_s[i][c].w;
      sr += acc_r[i][c].x * acc_r[i][c].x + acc_r[i][c].y * acc_r[i][c].y +
            acc_r[i][c].z * acc_r[i][c].z + acc_r[i][c].w * acc_r[i][c].w;
    }
    ss = group16_sum(ss);
    sr = group16_sum(sr);
    const float rinv_s = rsqrtf(ss / D + a.eps);
    const float rinv_r = rsqrtf(sr / D + a.eps);
    if (t < T) {
#pragma unroll
      for (int c = 0; c < D / 64; ++c) {
        const int col = tx * 4 + 64 * c;
        float4 gs = make_float4(1.f, 1.f, 1.f, 1.f), gr = gs;
        if (a.gamma_swa) gs = *reinterpret_cast<const float4*>(a.gamma_swa + (size_t)h * D + col);
        if (a.gamma_rla) gr = *reinterpret_cast<const float4*>(a.gamma_rla + (size_t)h * D + col);
        float4 y;
        y.x = gs.x * acc_s[i][c].x * rinv_s;
        y.y = gs.y * acc_s[i][c].y * rinv_s;
        y.z = gs.z * acc_s[i][c].z * rinv_s;
        y.w = gs.w * acc_s[i][c].w * rinv_s;
        if (rla_on) {
          y.x += gr.x * acc_r[i][c].x * rinv_r;
          y.y += gr.y * acc_r[i][c].y * rinv_r;
          y.z += gr.z * acc_r[i][c].z * rinv_r;
          y.w += gr.w * acc_r[i][c].w * rinv_r;
        }
        store4<TIO>(og + (size_t)t * q_pitch + col, y);
        if (a.o_swa) *reinterpret_cast<float4*>(a.o_swa + (row_base + t) * D + col) = acc_s[i][c];
        if (a.o_rla) *reinterpret_cast<float4*>(a.o_rla + (row_base + t) * D + col) = acc_r[i][c];
      }
      if (a.lse && tx == 0) a.lse[row_base + t] = m_run[i] + __logf(l_run[i]);
    }
  }
}

template <typename TIO, int D>
cudaError_t launch_fwd(const Args& a, cudaStream_t s) {
  constexpr size_t smem = (size_t)(5 * BM * (D + PAD) + BM * (BN + PAD)) * sizeof(float);
  cudaError_t e = cudaFuncSetAttribute(generic_fwd_kernel<TIO, D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  dim3 grid((a.T + BM - 1) / BM, a.B * a.H_q);
  { KernelTimer kt("generic_fwd", s); generic_fwd_kernel<TIO, D><<<grid, NT, smem, s>>>(a); }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_generic_forward(const Args& a, cudaStream_t s) {
  if (a.dtype == RATTN_F32) {
    return a.d == 64 ? launch_fwd<float, 64>(a, s) : launch_fwd<float, 128>(a, s);
  }
  return a.d == 64 ? launch_fwd<__nv_bfloat16, 64>(a, s) : launch_fwd<__nv_bfloat16, 128>(a, s);
}

}  // namespace rattn
