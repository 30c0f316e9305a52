// Single-token decode step and the prefill -> decode hand-off.
//
// Decode keeps, per K/V head, a ring of the last w keys/values (Section 2.1: the SWA
// cache is at most w+1 tokens, the newest being the incoming one) and the fixed-size
// fp32 state S of Eq. 4.  One step streams the ring once, reads S once and writes it
// back with the evicted token folded in: the step is bound by HBM traffic, so all
// global accesses are 16-byte vectors and every CTA keeps several loads in flight.
#include "rattn_internal.h"

namespace rattn {
namespace {

constexpr int DEC_THREADS = 512;
constexpr int DEC_WARPS = DEC_THREADS / 32;
constexpr int GH = 4;                       // query heads processed per pass over the ring

template <typename T> struct Vec16;        // a 16-byte vector of I/O elements
template <> struct Vec16<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
    unpack(*reinterpret_cast<const uint4*>(p), f);
  }
  static __device__ __forceinline__ void unpack(uint4 u, float (&f)[8]) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      float2 x = __bfloat1622float2(h[i]);
      f[2 * i] = x.x;
      f[2 * i + 1] = x.y;
    }
  }
};
template <> struct Vec16<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float (&f)[4]) {
    float4 u = *reinterpret_cast<const float4*>(p);
    f[0] = u.x; f[1] = u.y; f[2] = u.z; f[3] = u.w;
  }
  static __device__ __forceinline__ void unpack(uint4 u, float (&f)[4]) {
    f[0] = __uint_as_float(u.x); f[1] = __uint_as_float(u.y); f[2] = __uint_as_float(u.z); f[3] = __uint_as_float(u.w);
  }
};

__device__ __forceinline__ float to_f(float x) { return x; }
__device__ __forceinline__ float to_f(__nv_bfloat16 x) { return __bfloat162float(x); }
template <typename T> __device__ __forceinline__ T from_f(float x);
template <> __device__ __forceinline__ float from_f<float>(float x) { return x; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float x) {
  return __float2bfloat16_rn(x);
}

__device__ __forceinline__ float warp_max(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x = fmaxf(x, __shfl_xor_sync(0xffffffffu, x, o));
  return x;
}
__device__ __forceinline__ float warp_sum(float x) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
  return x;
}

// phi over D features by one warp: dst[a] = phi(src)[a] (softmax, or an element-wise map)
template <int D>
__device__ __forceinline__ void warp_feature_map(float* dst, const float* src, int lane, int phi) {
  if (phi != RATTN_PHI_SOFTMAX) {
    for (int a = lane; a < D; a += 32) dst[a] = phi == RATTN_PHI_RELU ? fmaxf(src[a], 0.f) : src[a];
    return;
  }
  float m = -INFINITY;
  for (int a = lane; a < D; a += 32) m = fmaxf(m, src[a]);
  m = warp_max(m);
  float s = 0.f;
  for (int a = lane; a < D; a += 32) {
    float e = __expf(src[a] - m);
    dst[a] = e;
    s += e;
  }
  s = warp_sum(s);
  const float inv = 1.f / s;
  for (int a = lane; a < D; a += 32) dst[a] *= inv;
}

struct DecodeArgs {
  const void* q; const void* k; const void* v;
  void* k_ring; void* v_ring; float* state; void* out;
  const float* gamma_swa; const float* gamma_rla;
  const int* pos_dev;                       // optional [B]: one position per batch entry
  int B, H_q, H_kv, w, pos, group, phi;
  float scale, eps;
};

// One CTA per (batch entry, K/V head); the g query heads of the group are served GH at a time.
//   scores   thread = ring slot: the slot's whole key row is read with 16-byte loads and dotted
//            with the GH query vectors held in shared memory (no cross-lane reduction at all)
//   softmax  one warp per head over the w + 1 logits in shared memory
//   P V      16 lanes x 16 bytes cover a value row; a thread keeps GH x 8 partial sums over its
//            share of the slots; partial sums are merged through shared memory
//   state    read-out phi(q) S and the update S += phi(k_old)^T v_old in one pass, float4
template <typename TIO, int D>
__global__ void __launch_bounds__(DEC_THREADS, 2) decode_kernel(DecodeArgs a) {
  constexpr int EPL = Vec16<TIO>::N;        // elements per 16-byte load
  constexpr int LPR = D / EPL;              // lanes (loads) that cover one row
  constexpr int RPP = DEC_THREADS / LPR;    // value rows in flight per pass of the P V phase
  constexpr int C4 = D / 4;                 // float4 columns of a state row
  constexpr int RP = DEC_THREADS / C4;      // state rows per pass

  extern __shared__ __align__(16) float sm[];
  const int g = a.group;
  const int w = a.w;
  float* q_s = sm;                          // [g][D] raw q, pre-multiplied by the logit scale
  float* fq_s = q_s + g * D;                // [g][D] phi(q)
  float* k_new = fq_s + g * D;              // [D]
  float* v_new = k_new + D;
  float* k_old = v_new + D;
  float* v_old = k_old + D;
  float* fk_old = v_old + D;
  float* p_s = fk_old + D;                  // [GH][w + 1] logits, then weights (slot w = the incoming token)
  float* red = p_s + GH * (w + 1) + ((GH * (w + 1)) & 1 ? 3 : 0) + 2;   // padded to 16 bytes below
  red = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(red) + 15) & ~uintptr_t(15));
  float* o_swa = red;                       // [GH][D]
  float* o_rla = o_swa + GH * D;            // [GH][D]
  float* stat = o_rla + GH * D;             // [GH] 1 / sum of weights
  float* part = stat + 4 * GH;              // [max(DEC_WARPS, RP)][GH][D] partial sums

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int b = blockIdx.x / a.H_kv, hk = blockIdx.x % a.H_kv;
  const int pos = a.pos_dev ? a.pos_dev[b] : a.pos;
  const bool evict = pos - w >= 0;
  const int slot = pos % w;
  const int n_valid = pos < w ? pos : w;

  const TIO* qg = reinterpret_cast<const TIO*>(a.q) + ((size_t)b * a.H_q + (size_t)hk * g) * D;
  const TIO* kg = reinterpret_cast<const TIO*>(a.k) + ((size_t)b * a.H_kv + hk) * D;
  const TIO* vg = reinterpret_cast<const TIO*>(a.v) + ((size_t)b * a.H_kv + hk) * D;
  TIO* kr = reinterpret_cast<TIO*>(a.k_ring) + ((size_t)b * a.H_kv + hk) * (size_t)w * D;
  TIO* vr = reinterpret_cast<TIO*>(a.v_ring) + ((size_t)b * a.H_kv + hk) * (size_t)w * D;
  float* S = a.state + ((size_t)b * a.H_kv + hk) * (size_t)D * D;
  TIO* og = reinterpret_cast<TIO*>(a.out) + ((size_t)b * a.H_q + (size_t)hk * g) * D;

  // The value ring and the state are needed only after the logits: ask L2 for them now (one request
  // per 128-byte line), so that their HBM latency runs under the key phase.
  {
    const char* kb = reinterpret_cast<const char*>(kr);
    const char* vb = reinterpret_cast<const char*>(vr);
    const size_t v_bytes = (size_t)n_valid * D * sizeof(TIO);
    for (size_t off = (size_t)tid * 128; off < v_bytes; off += (size_t)DEC_THREADS * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(kb + off));
    for (size_t off = (size_t)tid * 128; off < v_bytes; off += (size_t)DEC_THREADS * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(vb + off));
    const char* sb = reinterpret_cast<const char*>(S);
    for (size_t off = (size_t)tid * 128; off < (size_t)D * D * sizeof(float); off += (size_t)DEC_THREADS * 128)
      asm volatile("prefetch.global.L2 [%0];" ::"l"(sb + off));
  }
  for (int i = tid; i < g * D; i += DEC_THREADS) q_s[i] = to_f(qg[i]);
  if (tid < D) {
    k_new[tid] = to_f(kg[tid]);
    v_new[tid] = to_f(vg[tid]);
    if (evict) {
      k_old[tid] = to_f(kr[(size_t)slot * D + tid]);
      v_old[tid] = to_f(vr[(size_t)slot * D + tid]);
    }
  }
  __syncthreads();
  for (int r = warp; r <= g; r += DEC_WARPS) {
    if (r < g) warp_feature_map<D>(fq_s + r * D, q_s + r * D, lane, a.phi);
    else if (evict) warp_feature_map<D>(fk_old, k_old, lane, a.phi);
  }
  __syncthreads();
  for (int i = tid; i < g * D; i += DEC_THREADS) q_s[i] *= a.scale;     // phi has seen the raw q
  __syncthreads();

  for (int h0 = 0; h0 < g; h0 += GH) {
    const int nh = (g - h0) < GH ? (g - h0) : GH;
    // ---- SWA logits (Section 2.1): one ring slot per thread.  The slot's whole key row is read by
    // its thread (16-byte loads, eight in flight) and dotted with the GH query vectors, which every
    // lane reads from the same shared-memory address (a broadcast): no cross-lane reduction at all.
    // (Eight lanes per row with coalesced 32-byte pieces and three shuffle rounds measured 60 % slower.)
    for (int s = tid; s < n_valid; s += DEC_THREADS) {
      float dot[GH];
#pragma unroll
      for (int hh = 0; hh < GH; ++hh) dot[hh] = 0.f;
      const TIO* row = kr + (size_t)s * D;
#pragma unroll 8
      for (int c = 0; c < LPR; ++c) {
        float kx[EPL];
        Vec16<TIO>::load(row + c * EPL, kx);
#pragma unroll
        for (int hh = 0; hh < GH; ++hh) {
          if (hh < nh) {
            const float* qh = q_s + (h0 + hh) * D + c * EPL;
#pragma unroll
            for (int e = 0; e < EPL; ++e) dot[hh] += qh[e] * kx[e];
          }
        }
      }
#pragma unroll
      for (int hh = 0; hh < GH; ++hh) p_s[hh * (w + 1) + s] = dot[hh];
    }
    if (warp == DEC_WARPS - 1) {                                 // the incoming token, one warp
#pragma unroll
      for (int hh = 0; hh < GH; ++hh) {
        float x = 0.f;
        if (hh < nh)
          for (int c = lane; c < D; c += 32) x += q_s[(h0 + hh) * D + c] * k_new[c];
        x = warp_sum(x);
        if (lane == 0) p_s[hh * (w + 1) + w] = x;
      }
    }
    __syncthreads();
    // ---- softmax over the window, one warp per head ----------------------------------------
    if (warp < nh) {
      float* ph = p_s + warp * (w + 1);
      float m = ph[w];
      for (int s = lane; s < n_valid; s += 32) m = fmaxf(m, ph[s]);
      m = warp_max(m);
      float l = 0.f;
      for (int s = lane; s < n_valid; s += 32) {
        const float e = __expf(ph[s] - m);
        ph[s] = e;
        l += e;
      }
      l = warp_sum(l);
      const float en = __expf(ph[w] - m);
      if (lane == 0) {
        ph[w] = en;
        stat[warp] = 1.f / (l + en);
      }
    }
    __syncthreads();
    // ---- P V: LPR lanes cover a value row, RPP rows in flight -------------------------------
    {
      const int chunk = tid % LPR, r0 = tid / LPR;
      float acc[GH][EPL];
#pragma unroll
      for (int hh = 0; hh < GH; ++hh)
#pragma unroll
        for (int e = 0; e < EPL; ++e) acc[hh][e] = 0.f;
#pragma unroll 4
      for (int s = r0; s < n_valid; s += RPP) {
        float vx[EPL];
        Vec16<TIO>::load(vr + (size_t)s * D + chunk * EPL, vx);
#pragma unroll
        for (int hh = 0; hh < GH; ++hh) {
          const float p = p_s[hh * (w + 1) + s];
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[hh][e] += p * vx[e];
        }
      }
      // merge the rows held by the lanes of a warp that share `chunk`, then the warps
#pragma unroll
      for (int o = LPR; o < 32; o <<= 1)
#pragma unroll
        for (int hh = 0; hh < GH; ++hh)
#pragma unroll
          for (int e = 0; e < EPL; ++e) acc[hh][e] += __shfl_xor_sync(0xffffffffu, acc[hh][e], o);
      if (lane < LPR) {
#pragma unroll
        for (int hh = 0; hh < GH; ++hh)
#pragma unroll
          for (int e = 0; e < EPL; ++e) part[(warp * GH + hh) * D + chunk * EPL + e] = acc[hh][e];
      }
    }
    __syncthreads();
    for (int i = tid; i < nh * D; i += DEC_THREADS) {
      const int hh = i / D, c = i % D;
      float O = p_s[hh * (w + 1) + w] * v_new[c];
      for (int wv = 0; wv < DEC_WARPS; ++wv) O += part[(wv * GH + hh) * D + c];
      o_swa[hh * D + c] = O * stat[hh];
    }
    __syncthreads();

    // ---- RLA read-out phi(q) S and, once, the state update S += phi(k_old)^T v_old (Eq. 4)
    {
      const int c4 = tid % C4, rl = tid / C4;
      float4 ar[GH];
#pragma unroll
      for (int hh = 0; hh < GH; ++hh) ar[hh] = make_float4(0.f, 0.f, 0.f, 0.f);
      const bool update = evict && (h0 + GH >= g);   // fold the evicted token in on the last pass
      float4 vo = make_float4(0.f, 0.f, 0.f, 0.f);
      if (update) vo = *reinterpret_cast<const float4*>(v_old + c4 * 4);
#pragma unroll 4
      for (int r = rl; r < D; r += RP) {
        float4 s4 = *reinterpret_cast<const float4*>(S + (size_t)r * D + c4 * 4);
#pragma unroll
        for (int hh = 0; hh < GH; ++hh) {
          const float f = hh < nh ? fq_s[(h0 + hh) * D + r] : 0.f;
          ar[hh].x += f * s4.x; ar[hh].y += f * s4.y; ar[hh].z += f * s4.z; ar[hh].w += f * s4.w;
        }
        if (update) {
          const float fk = fk_old[r];
          s4.x += fk * vo.x; s4.y += fk * vo.y; s4.z += fk * vo.z; s4.w += fk * vo.w;
          *reinterpret_cast<float4*>(S + (size_t)r * D + c4 * 4) = s4;
        }
      }
#pragma unroll
      for (int hh = 0; hh < GH; ++hh)
        *reinterpret_cast<float4*>(part + ((size_t)(rl * GH + hh)) * D + c4 * 4) = ar[hh];
    }
    __syncthreads();
    for (int i = tid; i < nh * D; i += DEC_THREADS) {
      const int hh = i / D, c = i % D;
      float O = 0.f;
      for (int r = 0; r < RP; ++r) O += part[(r * GH + hh) * D + c];
      o_rla[hh * D + c] = O;
    }
    __syncthreads();

    // ---- Section 3.2: two RMS norms and the sum --------------------------------------
    if (warp < nh) {
      const int h = hk * g + h0 + warp;
      float ss = 0.f, sr = 0.f;
      for (int c = lane; c < D; c += 32) {
        const float x = o_swa[warp * D + c], y = o_rla[warp * D + c];
        ss += x * x;
        sr += y * y;
      }
      ss = warp_sum(ss);
      sr = warp_sum(sr);
      const float is = rsqrtf(ss / D + a.eps), ir = rsqrtf(sr / D + a.eps);
      for (int c = lane; c < D; c += 32) {
        const float gs = a.gamma_swa ? a.gamma_swa[(size_t)h * D + c] : 1.f;
        const float gr = a.gamma_rla ? a.gamma_rla[(size_t)h * D + c] : 1.f;
        og[(size_t)(h0 + warp) * D + c] =
            from_f<TIO>(gs * o_swa[warp * D + c] * is + gr * o_rla[warp * D + c] * ir);
      }
    }
    __syncthreads();
  }
  // the incoming token takes the evicted token's slot
  if (tid < D) {
    kr[(size_t)slot * D + tid] = kg[tid];
    vr[(size_t)slot * D + tid] = vg[tid];
  }
}

template <int D> size_t decode_smem_floats(int g, int w) {
  constexpr int RP = DEC_THREADS / (D / 4);
  constexpr int PR = RP > DEC_WARPS ? RP : DEC_WARPS;
  return (size_t)2 * g * D + 5 * D + (size_t)GH * (w + 1) + 16 + 2 * GH * D + 4 * GH + (size_t)PR * GH * D;
}

template <typename TIO, int D>
cudaError_t launch_dec(const DecodeArgs& a, cudaStream_t s) {
  const size_t smem = decode_smem_floats<D>(a.group, a.w) * sizeof(float);
  if (smem > 227 * 1024) return cudaErrorInvalidValue;
  cudaError_t e = cudaFuncSetAttribute(decode_kernel<TIO, D>,
                                       cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  { KernelTimer kt("decode_step", s); decode_kernel<TIO, D><<<a.B * a.H_kv, DEC_THREADS, smem, s>>>(a); }
  count_launches(1);
  return cudaGetLastError();
}

// ---------------------------------------------------------------- prefill -> decode hand-off
// state_out[b,hk] = sum_{j < T-w} phi(k_j)^T v_j  (Eq. 4), one CTA per 8 feature rows.
// T: key rows per head in memory; len[b] (optional): valid rows of entry b; state_in (optional):
// the sum over the tokens before row 0.
template <typename TIO, int D>
__global__ void __launch_bounds__(256) handoff_state_kernel(const TIO* __restrict__ k,
                                                            const TIO* __restrict__ v,
                                                            float* __restrict__ state, int T, int w, int phi,
                                                            const int* __restrict__ len, int H_kv,
                                                            const float* __restrict__ state_in, int layout) {
  constexpr int ROWS = 8, TOK = 32;
  __shared__ float fk[TOK][ROWS];
  __shared__ float vs[TOK][D];
  const int bh = blockIdx.y, r0 = blockIdx.x * ROWS;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  // head (b, hk) of [B, H_kv, T, D] (layout 0) or [B, T, H_kv, D] (layout 1): first row and row pitch
  const size_t head0 = layout ? ((size_t)(bh / H_kv) * T * H_kv + bh % H_kv) * D : (size_t)bh * T * D;
  const size_t pitch = layout ? (size_t)H_kv * D : (size_t)D;
  const TIO* kg = k + head0;
  const TIO* vg = v + head0;
  const int n = (len ? min(T, len[bh / H_kv]) : T) - w;   // tokens 0..n-1 have left every window
  // thread -> (row, column group): 8 rows x 32 column lanes, D/32 columns each
  const int row = tid / 32, cl = tid % 32;
  float acc[D / 32];
#pragma unroll
  for (int c = 0; c < D / 32; ++c)
    acc[c] = state_in ? state_in[((size_t)bh * D + r0 + row) * D + cl + 32 * c] : 0.f;
  for (int j0 = 0; j0 < n; j0 += TOK) {
    __syncthreads();
    for (int jj = warp; jj < TOK; jj += 8) {   // warp-level softmax of k_j, keep rows r0..r0+7
      const int j = j0 + jj;
      float x[D / 32];
      float m = -INFINITY;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        x[c] = j < n ? to_f(kg[(size_t)j * pitch + lane + 32 * c]) : 0.f;
        m = fmaxf(m, x[c]);
      }
      m = warp_max(m);
      float s = 0.f;
      if (phi == RATTN_PHI_SOFTMAX) {
#pragma unroll
        for (int c = 0; c < D / 32; ++c) { x[c] = __expf(x[c] - m); s += x[c]; }
        s = warp_sum(s);
      } else {
        s = 1.f;
        if (phi == RATTN_PHI_RELU) {
#pragma unroll
          for (int c = 0; c < D / 32; ++c) x[c] = fmaxf(x[c], 0.f);
        }
      }
      const float inv = j < n ? 1.f / s : 0.f;
#pragma unroll
      for (int c = 0; c < D / 32; ++c) {
        const int col = lane + 32 * c;
        if (col >= r0 && col < r0 + ROWS) fk[jj][col - r0] = x[c] * inv;
        vs[jj][col] = j < n ? to_f(vg[(size_t)j * pitch + col]) : 0.f;
      }
    }
    __syncthreads();
#pragma unroll 8
    for (int jj = 0; jj < TOK; ++jj) {
      const float f = fk[jj][row];
#pragma unroll
      for (int c = 0; c < D / 32; ++c) acc[c] += f * vs[jj][cl + 32 * c];
    }
  }
#pragma unroll
  for (int c = 0; c < D / 32; ++c) state[((size_t)bh * D + r0 + row) * D + cl + 32 * c] = acc[c];
}

// ring[b,hk, j % w] = x[b,hk, j] for the last min(w,T) tokens; other slots zero.
template <typename TIO>
__global__ void handoff_ring_kernel(const TIO* __restrict__ k, const TIO* __restrict__ v,
                                    TIO* __restrict__ kr, TIO* __restrict__ vr, int T, int w, int D,
                                    const int* __restrict__ len, int H_kv, int pos_shift, int layout) {
  const int bh = blockIdx.y;
  const size_t head0 = layout ? ((size_t)(bh / H_kv) * T * H_kv + bh % H_kv) * D : (size_t)bh * T * D;
  const size_t pitch = layout ? (size_t)H_kv * D : (size_t)D;
  const int slot = blockIdx.x;
  // Row j of k, v is the token at sequence position j + pos_shift (a resumed sequence's rows start
  // before the chunk); the ring keeps position p at slot p % w.  The newest row that maps to this slot:
  const int Tb = len ? min(T, len[bh / H_kv]) : T;
  const int last = Tb - 1;
  const int j = last - ((last + pos_shift - slot) % w + w) % w;
  const bool valid = j >= 0 && j >= Tb - w;
  for (int c = threadIdx.x; c < D; c += blockDim.x) {
    const size_t dst = ((size_t)bh * w + slot) * D + c;
    if (valid) {
      kr[dst] = k[head0 + (size_t)j * pitch + c];
      vr[dst] = v[head0 + (size_t)j * pitch + c];
    } else {
      kr[dst] = from_f<TIO>(0.f);
      vr[dst] = from_f<TIO>(0.f);
    }
  }
}

template <typename TIO, int D>
cudaError_t launch_handoff_t(const Args& a, cudaStream_t s, bool state_too) {
  const int BH = a.B * a.H_kv;
  if (a.state_out && state_too) {
    dim3 grid(D / 8, BH);
    KernelTimer kt("handoff_state", s);
    handoff_state_kernel<TIO, D><<<grid, 256, 0, s>>>(reinterpret_cast<const TIO*>(a.k),
                                                      reinterpret_cast<const TIO*>(a.v),
                                                      a.state_out, a.Tk, a.w, a.phi, a.seq_lens, a.H_kv, a.state_in, a.kv_layout);
    count_launches(1);
  }
  if (a.k_ring_out && a.v_ring_out) {
    dim3 grid(a.w, BH);
    KernelTimer kt("handoff_ring", s);
    handoff_ring_kernel<TIO><<<grid, 64, 0, s>>>(reinterpret_cast<const TIO*>(a.k),
                                                 reinterpret_cast<const TIO*>(a.v),
                                                 reinterpret_cast<TIO*>(a.k_ring_out),
                                                 reinterpret_cast<TIO*>(a.v_ring_out), a.Tk, a.w, D, a.seq_lens,
                                                 a.H_kv, a.pos_shift, a.kv_layout);
    count_launches(1);
  }
  return cudaGetLastError();
}

// k_ext[bh, e] = e < w ? ring[bh, (pos0 - w + e) % w] : chunk[bh, e - w]   (16-byte vectors)
__global__ void gather_history_kernel(const uint4* __restrict__ k_chunk, const uint4* __restrict__ v_chunk,
                                      const uint4* __restrict__ k_ring, const uint4* __restrict__ v_ring,
                                      uint4* __restrict__ k_ext, uint4* __restrict__ v_ext, int T, int w, int pos0,
                                      int vec_per_row, int H_kv, int layout) {
  const int bh = blockIdx.y;
  // the chunk is the caller's tensor: [B, H_kv, T, d] (layout 0) or [B, T, H_kv, d] (layout 1), in 16-byte vectors
  const size_t head0 = layout ? ((size_t)(bh / H_kv) * T * H_kv + bh % H_kv) * vec_per_row : (size_t)bh * T * vec_per_row;
  const size_t pitch = layout ? (size_t)H_kv * vec_per_row : (size_t)vec_per_row;
  const size_t n_ext = (size_t)(w + T) * vec_per_row;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n_ext; i += (size_t)gridDim.x * blockDim.x) {
    const int e = (int)(i / vec_per_row), c = (int)(i % vec_per_row);
    uint4 kk, vv;
    if (e < w) {
      const int slot = (pos0 - w + e) % w;
      kk = k_ring[((size_t)bh * w + slot) * vec_per_row + c];
      vv = v_ring[((size_t)bh * w + slot) * vec_per_row + c];
    } else {
      kk = k_chunk[head0 + (size_t)(e - w) * pitch + c];
      vv = v_chunk[head0 + (size_t)(e - w) * pitch + c];
    }
    k_ext[(size_t)bh * n_ext + i] = kk;
    v_ext[(size_t)bh * n_ext + i] = vv;
  }
}

}  // namespace

cudaError_t launch_gather_history(const Args& a, const void* k_chunk, const void* v_chunk, const void* k_ring,
                                  const void* v_ring, void* k_ext, void* v_ext, int pos0, cudaStream_t s) {
  const int elem = a.dtype == RATTN_F32 ? 4 : 2;
  const int vec_per_row = a.d * elem / 16;
  const size_t n_ext = (size_t)(a.w + a.T) * vec_per_row;
  dim3 grid((unsigned)((n_ext + 255) / 256 < 1024 ? (n_ext + 255) / 256 : 1024), a.B * a.H_kv);
  KernelTimer kt("gather_history", s);
  gather_history_kernel<<<grid, 256, 0, s>>>(
      reinterpret_cast<const uint4*>(k_chunk), reinterpret_cast<const uint4*>(v_chunk),
      reinterpret_cast<const uint4*>(k_ring), reinterpret_cast<const uint4*>(v_ring),
      reinterpret_cast<uint4*>(k_ext), reinterpret_cast<uint4*>(v_ext), a.T, a.w, pos0, vec_per_row, a.H_kv, a.layout);
  count_launches(1);
  return cudaGetLastError();
}

cudaError_t launch_decode(const Args& p, void* k_ring, void* v_ring, float* state, int pos, const int* pos_dev,
                          cudaStream_t s) {
  if (!(p.flags & RATTN_FLAG_FORCE_GENERIC) && decode_tc_applies(p, p.w))
    return launch_decode_tc(p, k_ring, v_ring, state, pos, pos_dev, s);
  DecodeArgs a;
  a.pos_dev = pos_dev;
  a.q = p.q; a.k = p.k; a.v = p.v; a.k_ring = k_ring; a.v_ring = v_ring; a.state = state;
  a.out = p.out; a.gamma_swa = p.gamma_swa; a.gamma_rla = p.gamma_rla;
  a.B = p.B; a.H_q = p.H_q; a.H_kv = p.H_kv; a.w = p.w; a.pos = pos; a.group = p.group; a.phi = p.phi;
  a.scale = p.scale; a.eps = p.eps;
  if (p.dtype == RATTN_F32)
    return p.d == 64 ? launch_dec<float, 64>(a, s) : launch_dec<float, 128>(a, s);
  return p.d == 64 ? launch_dec<__nv_bfloat16, 64>(a, s) : launch_dec<__nv_bfloat16, 128>(a, s);
}

cudaError_t launch_handoff(const Args& a, cudaStream_t s, bool state_too) {
  if (a.dtype == RATTN_F32)
    return a.d == 64 ? launch_handoff_t<float, 64>(a, s, state_too) : launch_handoff_t<float, 128>(a, s, state_too);
  return a.d == 64 ? launch_handoff_t<__nv_bfloat16, 64>(a, s, state_too)
                   : launch_handoff_t<__nv_bfloat16, 128>(a, s, state_too);
}

}  // namespace rattn
