// qk-norm and rotary embedding of q and k in one pass (Table 1 "qk-norm"; Section 4 "Model Setup":
// local layers rotate with theta = 5e5, global layers do not), and the gradient of that pass.
//
// Streaming kernels: every element is read once and written once, so the bound is HBM bandwidth.
// The unit of work is a chunk: the rows of one head that one CTA's threads cover (256 / (d/16)
// consecutive positions, 8 KB of bf16), contiguous in memory.  Chunks travel global -> shared
// -> global as bulk asynchronous copies through a ring of stages, so the bytes in flight do not
// depend on registers or on where the warps are in their arithmetic; the threads transform a
// chunk in place in shared memory.  A head vector of d features is held by d/16 neighbouring
// lanes, each with features [8l, 8l+8) and [d/2 + 8l, d/2 + 8l + 8): the two halves of its 8
// rotation pairs.  Chunks are ordered tensor, row block, head, and every CTA takes an equal
// contiguous share of them: consecutive chunks share their positions, so a thread computes its
// 8 sines and cosines once per row block.
#include <cmath>
#include <cstdint>

#include "rattn_internal.h"
#include "tc_ptx.cuh"

namespace rattn {
namespace {

constexpr int QK_THREADS = 256;
constexpr int QK_MAX_CTAS = 1024;     // bounds the partial sums of the gain gradients
constexpr int QK_CTAS_PER_SM = 3;

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
  float inv_H[2];                     // 1 / H
  int n_chunks[2];                    // chunks of q, of k
  int tbl_tokens;                     // [B,T,H,d]: positions a rotation table holds
  int layout;                         // rattn_layout of x, y, dy
  int B, T, nblk_t;
  float eps;
  int rotate;
  long long pos0;
  const int* pos;
};

__device__ int g_qk_status;           // RATTN_ERR_TIMEOUT once a bounded wait has expired

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

// single-thread forms of the bulk copies (one issuing thread per CTA, once per chunk)
__device__ __forceinline__ void expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(ptx::smem_u32(bar)), "r"(bytes)
               : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(ptx::smem_u32(dst)), "l"(src), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}
__device__ __forceinline__ void bulk_store(void* dst, const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
               ::"l"(dst), "r"(ptx::smem_u32(src)), "r"(bytes)
               : "memory");
}
// all but the newest of this thread's store groups have finished reading shared memory
__device__ __forceinline__ void store_wait_read_but_one() {
  asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
}

template <typename T, bool BWD> struct Ring {
  static constexpr int kChunk = 4096 * (int)sizeof(T);           // rows per CTA x row bytes, any d
  static constexpr int kBufs = BWD ? 2 : 1;                      // backward: the input and its output gradient
  static constexpr int kStages = BWD ? (sizeof(T) == 2 ? 4 : 3) : (sizeof(T) == 2 ? 8 : 4);
  static constexpr int kRed = BWD ? 4096 * 4 : 0;                // backward: block reduction of the gain gradients
  static constexpr int kBytes = kStages * kBufs * kChunk + kRed + 128;
};

// Chunks and their order.
//   [B, H, T, d]: a chunk = RPB consecutive positions of one head; chunks are numbered tensor, batch entry,
//                 row block, head, so consecutive chunks share their positions and a thread forms its 8
//                 sines and cosines once per row block.
//   [B, T, H, d]: memory is a sequence of head vectors in (b, t, h) order; a chunk = RPB consecutive ones
//                 (a few positions' worth).  The sines and cosines of a chunk's positions are formed once
//                 per CTA, one chunk ahead, in a small shared-memory table.
// A cursor is set once and then stepped.
struct Cursor {
  int which;            // 0: q, 1: k
  int b, tb, h;         // [B, H, T, d]
  int c;                // [B, T, H, d]: chunk inside the tensor; its first head vector is head h0 of
  int h0, t0, b0;       //               position t0 of batch entry b0
};
// x / H for 0 <= x < 8192 without an integer division ((x + 0.5) / H is at least 0.5 / H away from an integer)
__device__ __forceinline__ int small_div(int x, float inv_H) { return __float2int_rd(((float)x + 0.5f) * inv_H); }
template <int RPB>
__device__ __forceinline__ Cursor cursor_at(const QkArgs& a, int i) {
  Cursor c;
  c.which = i >= a.n_chunks[0];
  if (c.which) i -= a.n_chunks[0];
  c.c = i;
  const int H = a.H[c.which];
  {
    const long long bt = (long long)i * RPB / H;
    c.h0 = (int)((long long)i * RPB - bt * H);
    c.b0 = (int)(bt / a.T);
    c.t0 = (int)(bt - (long long)c.b0 * a.T);
  }
  const int rb = i / H;
  c.h = i - rb * H;
  c.b = rb / a.nblk_t;
  c.tb = rb - c.b * a.nblk_t;
  return c;
}
template <bool BTHD, int RPB>
__device__ __forceinline__ void step(const QkArgs& a, Cursor& c) {
  if (BTHD) {
    if (++c.c >= a.n_chunks[c.which]) {
      c.c = c.h0 = c.t0 = c.b0 = 0;
      ++c.which;
      return;
    }
    c.h0 += RPB;                                   // the next run of RPB head vectors
    const int carry = small_div(c.h0, a.inv_H[c.which]);
    c.h0 -= carry * a.H[c.which];
    c.t0 += carry;
    while (c.t0 >= a.T) { c.t0 -= a.T; ++c.b0; }
    return;
  }
  if (++c.h < a.H[c.which]) return;
  c.h = 0;
  if (++c.tb < a.nblk_t) return;
  c.tb = 0;
  if (++c.b < a.B) return;
  c.b = 0;
  ++c.which;
}
// byte offset of the cursor's chunk in its tensor and the rows of it that exist
template <int RPB, int ROW, bool BTHD>
__device__ __forceinline__ void where(const QkArgs& a, const Cursor& c, size_t* at, int* rows) {
  const int H = a.H[c.which];
  if (!BTHD) {
    *rows = a.T - c.tb * RPB < RPB ? a.T - c.tb * RPB : RPB;
    *at = (((size_t)c.b * H + c.h) * a.T + (size_t)c.tb * RPB) * ROW;
  } else {
    const int n_vec = a.B * a.T * H, v0 = c.c * RPB;          // < 2^31, checked on the host
    *rows = n_vec - v0 < RPB ? n_vec - v0 : RPB;
    *at = (size_t)v0 * ROW;
  }
}

template <typename T, int D, bool BWD, bool BTHD>
__global__ void __launch_bounds__(QK_THREADS, BWD ? 2 : QK_CTAS_PER_SM)
qk_prologue_kernel(const __grid_constant__ QkArgs a, const __grid_constant__ Freqs f) {
  using R = Ring<T, BWD>;
  constexpr int LPR = D / 16, RPB = QK_THREADS / LPR, ROW = D * (int)sizeof(T), S = R::kStages;
  extern __shared__ __align__(128) unsigned char smem[];
  unsigned char* stage = smem;                                                    // [S][kBufs][kChunk]
  float* red = reinterpret_cast<float*>(smem + S * R::kBufs * R::kChunk);         // [RPB][D] (backward)
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + S * R::kBufs * R::kChunk + R::kRed);
  volatile int* abort = reinterpret_cast<volatile int*>(full + S);
  float2* tbl = reinterpret_cast<float2*>(smem + R::kBytes);                      // [2][tbl_tokens][D/2] (cos, sin)

  const int tid = threadIdx.x, l = tid % LPR, row = tid / LPR;
  const long long n_all = (long long)a.n_chunks[0] + a.n_chunks[1];           // < 2^31, checked on the host
  const int lo = (int)(n_all * blockIdx.x / gridDim.x), hi = (int)(n_all * (blockIdx.x + 1) / gridDim.x);

  if (tid == 0) {
    for (int i = 0; i < S; ++i) ptx::mbar_init(&full[i], 1);
    *abort = 0;
    ptx::fence_mbar_init();
  }
  if (BWD && a.partial != nullptr && tid < D) {
    a.partial[((size_t)0 * gridDim.x + blockIdx.x) * D + tid] = 0.f;
    a.partial[((size_t)1 * gridDim.x + blockIdx.x) * D + tid] = 0.f;
  }
  __syncthreads();

  Cursor ahead = cursor_at<RPB>(a, lo);                    // thread 0's cursor: the next chunk to load
  auto issue = [&](int i) {                           // thread 0 only; i must be the cursor's chunk
    const Cursor c = ahead;
    step<BTHD, RPB>(a, ahead);
    size_t at;
    int rows;
    where<RPB, ROW, BTHD>(a, c, &at, &rows);
    const int slot = (i - lo) % S;
    unsigned char* dst = stage + (size_t)slot * R::kBufs * R::kChunk;
    expect_tx(&full[slot], (uint32_t)(rows * ROW * R::kBufs));
    bulk_load(dst, static_cast<const unsigned char*>(a.x[c.which]) + at, (uint32_t)(rows * ROW), &full[slot]);
    if (BWD)
      bulk_load(dst + R::kChunk, static_cast<const unsigned char*>(a.dy[c.which]) + at, (uint32_t)(rows * ROW),
                &full[slot]);
  };
  if (tid == 0)
    for (int i = lo; i < hi && i < lo + S - 1; ++i) issue(i);

  float c[8], s[8], g_lo[8], g_hi[8], acc[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) acc[j] = 0.f;
  int cur_which = -1, cur_rb = -1;

  // per-CTA sum of the gain-gradient terms over its rows, in row order, to this CTA's partial row
  auto flush = [&](int which) {
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      red[row * D + 8 * l + j] = acc[j];
      red[row * D + D / 2 + 8 * l + j] = acc[8 + j];
      acc[j] = acc[8 + j] = 0.f;
    }
    __syncthreads();
    if (tid < D) {
      float sum = 0.f;
      for (int r = 0; r < RPB; ++r) sum += red[r * D + tid];
      a.partial[((size_t)which * gridDim.x + blockIdx.x) * D + tid] = sum;
    }
    __syncthreads();
  };

  // [B, T, H, d]: cos and sin of every (position, pair) of the cursor's chunk into table `buf`, one entry per
  // thread and round (a chunk of RPB head vectors spans RPB / H positions, plus one when it straddles)
  const bool tabled = BTHD && a.rotate;
  auto fill_table = [&](const Cursor& cx, int buf) {
    constexpr double kTwoPi = 6.283185307179586476925286766559;
    size_t at_;
    int rows_;
    where<RPB, ROW, BTHD>(a, cx, &at_, &rows_);
    const int n_tok = small_div(cx.h0 + rows_ - 1, a.inv_H[cx.which]) + 1;
    for (int e = tid; e < n_tok * (D / 2); e += QK_THREADS) {
      const int tok = e / (D / 2), pair = e % (D / 2);
      int t = cx.t0 + tok, b = cx.b0;
      while (t >= a.T) { t -= a.T; ++b; }
      const long long position = (a.pos ? (long long)a.pos[b] : a.pos0) + t;
      double ang = (double)position * f.inv[pair];
      ang -= kTwoPi * rint(ang * (1.0 / kTwoPi));
      float sn, cs;
      sincosf((float)ang, &sn, &cs);
      tbl[((size_t)buf * a.tbl_tokens + tok) * (D / 2) + pair] = make_float2(cs, sn);
    }
  };
  Cursor ch = cursor_at<RPB>(a, lo);
  if (tabled && lo < hi) fill_table(ch, 0);
  if (!a.rotate) {
#pragma unroll
    for (int j = 0; j < 8; ++j) { c[j] = 1.f; s[j] = 0.f; }
  }
  __syncthreads();

  int i = lo;
  bool ok = true;
  for (; i < hi; ++i, step<BTHD, RPB>(a, ch)) {
    const int n = i - lo, slot = n % S;
    if (ch.which != cur_which) {
      if (BWD && a.partial != nullptr && cur_which >= 0) flush(cur_which);
      load_gain(a.gain[ch.which], 8 * l, D / 2, g_lo, g_hi);
      cur_which = ch.which;
      cur_rb = -1;
    }
    size_t ch_at;
    int ch_rows;
    where<RPB, ROW, BTHD>(a, ch, &ch_at, &ch_rows);
    if (!BTHD) {
      const int rb = ch.b * a.nblk_t + ch.tb;
      if (rb != cur_rb && a.rotate) {
        const long long p0 = a.pos ? (long long)a.pos[ch.b] : a.pos0;
        rotation(f, 8 * l, p0 + ch.tb * RPB + row, a.rotate, c, s);
        cur_rb = rb;
      }
    } else if (tabled) {
      // the next chunk's table while this chunk's data is on its way; this chunk's was written one
      // iteration ago (or before the loop) and the barrier in between made it visible
      if (i + 1 < hi) {
        Cursor nx = ch;
        step<BTHD, RPB>(a, nx);
        fill_table(nx, (n + 1) & 1);
      }
      const int tok = small_div(ch.h0 + row, a.inv_H[ch.which]);
      const float2* e = tbl + ((size_t)(n & 1) * a.tbl_tokens + (row < ch_rows ? tok : 0)) * (D / 2) + 8 * l;
#pragma unroll
      for (int j = 0; j < 8; ++j) { c[j] = e[j].x; s[j] = e[j].y; }
    }
    const bool live = row < ch_rows;
    unsigned char* buf = stage + (size_t)slot * R::kBufs * R::kChunk + (size_t)row * ROW;
    const bool got = ptx::mbar_wait_warp(&full[slot], (uint32_t)(n / S) & 1u, abort);
    if (got) {
      float x_lo[8], x_hi[8];
      if (live) {
        Io<T>::load(buf, 8 * l, x_lo);
        Io<T>::load(buf, D / 2 + 8 * l, x_hi);
      } else {
        zero8(x_lo);
        zero8(x_hi);
      }
      float ss = 0.f;
#pragma unroll
      for (int j = 0; j < 8; ++j) ss += x_lo[j] * x_lo[j] + x_hi[j] * x_hi[j];
      if (!BWD) {
        ss = row_sum<LPR>(ss);
        const float r = rsqrtf(ss * (1.f / D) + a.eps);
        float o_lo[8], o_hi[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float n_lo = x_lo[j] * r * g_lo[j], n_hi = x_hi[j] * r * g_hi[j];
          o_lo[j] = n_lo * c[j] - n_hi * s[j];
          o_hi[j] = n_hi * c[j] + n_lo * s[j];
        }
        if (live) {
          Io<T>::store(buf, 8 * l, o_lo);
          Io<T>::store(buf, D / 2 + 8 * l, o_hi);
        }
      } else {
        float e_lo[8], e_hi[8];
        if (live) {
          Io<T>::load(buf + R::kChunk, 8 * l, e_lo);
          Io<T>::load(buf + R::kChunk, D / 2 + 8 * l, e_hi);
        } else {
          zero8(e_lo);
          zero8(e_hi);
        }
        // the rotation is orthogonal: its transpose turns by the opposite angle
        float du_lo[8], du_hi[8], dot = 0.f;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          du_lo[j] = e_lo[j] * c[j] + e_hi[j] * s[j];
          du_hi[j] = e_hi[j] * c[j] - e_lo[j] * s[j];
          dot += du_lo[j] * g_lo[j] * x_lo[j] + du_hi[j] * g_hi[j] * x_hi[j];
        }
        ss = row_sum<LPR>(ss);
        dot = row_sum<LPR>(dot);
        const float r = rsqrtf(ss * (1.f / D) + a.eps);
        const float back = r * r * r * dot * (1.f / D);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          acc[j] += du_lo[j] * x_lo[j] * r;
          acc[8 + j] += du_hi[j] * x_hi[j] * r;
          e_lo[j] = r * du_lo[j] * g_lo[j] - x_lo[j] * back;
          e_hi[j] = r * du_hi[j] * g_hi[j] - x_hi[j] * back;
        }
        if (live) {
          Io<T>::store(buf + R::kChunk, 8 * l, e_lo);
          Io<T>::store(buf + R::kChunk, D / 2 + 8 * l, e_hi);
        }
      }
      ptx::fence_proxy_async_smem();
    }
    ok = __syncthreads_and(got) != 0;
    if (!ok) break;
    if (tid == 0) {
      const int rows = ch_rows;
      const size_t at = ch_at;
      unsigned char* src = stage + (size_t)slot * R::kBufs * R::kChunk + (BWD ? R::kChunk : 0);
      bulk_store(static_cast<unsigned char*>(a.y[ch.which]) + at, src, (uint32_t)(rows * ROW));
      ptx::tma_store_commit();
      const int next = i + S - 1;
      if (next < hi) {
        store_wait_read_but_one();          // the slot of chunk i - 1 has been read out
        issue(next);
      }
    }
  }

  if (tid == 0) {
    ptx::tma_store_wait();
    if (!ok) {
      // give the loads still in flight a bounded time to land before the CTA's memory goes away
      const int issued = i + S - 1 < hi ? i + S - 1 : hi;
      for (int j = i; j < issued; ++j) {
        const int n = j - lo;
        for (int it = 0; it < ptx::kWaitPolls && !ptx::mbar_try_wait(&full[n % S], (uint32_t)(n / S) & 1u); ++it) {}
      }
      g_qk_status = RATTN_ERR_TIMEOUT;
    }
  }
  if (BWD && ok && a.partial != nullptr && cur_which >= 0) flush(cur_which);
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
  if (p->layout != RATTN_LAYOUT_BHTD && p->layout != RATTN_LAYOUT_BTHD) return RATTN_ERR_UNSUPPORTED;
  const int rpb = QK_THREADS / (p->d / 16);
  if ((long long)p->B * ((p->T + rpb - 1) / rpb) * ((long long)p->H_q + p->H_kv) >= (1ll << 31)) return RATTN_ERR_BAD_ARG;
  if (p->layout == RATTN_LAYOUT_BTHD && ((long long)p->B * p->T * (p->H_q > p->H_kv ? p->H_q : p->H_kv) >= (1ll << 31) ||
                                         p->H_q > 4096 || p->H_kv > 4096))
    return RATTN_ERR_BAD_ARG;
  return RATTN_OK;
}

void fill(const rattn_qk_params* p, QkArgs* a, Freqs* f) {
  a->x[0] = p->q; a->x[1] = p->k;
  a->gain[0] = p->q_gain; a->gain[1] = p->k_gain;
  a->H[0] = p->H_q; a->H[1] = p->H_kv;
  a->inv_H[0] = 1.f / (float)p->H_q; a->inv_H[1] = p->H_kv > 0 ? 1.f / (float)p->H_kv : 0.f;
  const int rpb = QK_THREADS / (p->d / 16);
  a->B = p->B; a->T = p->T; a->nblk_t = (p->T + rpb - 1) / rpb;
  a->layout = p->layout;
  a->tbl_tokens = 0;
  for (int w = 0; w < 2; ++w) {     // [B,H,T,d]: row blocks x heads; [B,T,H,d]: runs of rpb head vectors
    a->n_chunks[w] = p->layout == RATTN_LAYOUT_BHTD ? p->B * a->nblk_t * a->H[w]
                                                    : (int)(((long long)p->B * p->T * a->H[w] + rpb - 1) / rpb);
    if (p->layout != RATTN_LAYOUT_BHTD && a->H[w] > 0 && p->theta > 0.f) {
      const int tokens = (rpb + a->H[w] - 1) / a->H[w] + 1;      // positions a chunk can touch
      if (tokens > a->tbl_tokens) a->tbl_tokens = tokens;
    }
  }
  a->eps = p->eps;
  a->rotate = p->theta > 0.f;
  a->pos0 = p->pos0;
  a->pos = p->pos;
  a->partial = nullptr;
  a->dy[0] = a->dy[1] = nullptr;
  a->y[0] = a->y[1] = nullptr;
  for (int i = 0; i < 64; ++i)
    f->inv[i] = a->rotate && i < p->d / 2 ? std::pow((double)p->theta, -2.0 * i / p->d) : 0.0;
}

// CTAs of a launch: every resident slot of the device, fewer when there are fewer chunks
cudaError_t grid_size(const QkArgs& a, int per_sm, int* n_cta) {
  int dev = 0, n_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  long long n = (long long)a.n_chunks[0] + a.n_chunks[1];
  if (n > (long long)n_sm * per_sm) n = (long long)n_sm * per_sm;
  if (n > QK_MAX_CTAS) n = QK_MAX_CTAS;
  *n_cta = (int)n;
  return cudaSuccess;
}

template <typename T, int D, bool BWD, bool BTHD>
cudaError_t launch_layout(const QkArgs& a, const Freqs& f, int n_cta, cudaStream_t s) {
  const int smem = Ring<T, BWD>::kBytes + 2 * a.tbl_tokens * (D / 2) * (int)sizeof(float2);
  cudaError_t e = cudaFuncSetAttribute(qk_prologue_kernel<T, D, BWD, BTHD>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  KernelTimer kt(BWD ? "qk_prologue_bwd" : "qk_prologue", s);
  qk_prologue_kernel<T, D, BWD, BTHD><<<n_cta, QK_THREADS, smem, s>>>(a, f);
  count_launches(1);
  return cudaGetLastError();
}

template <typename T, int D, bool BWD>
cudaError_t launch_one(const QkArgs& a, const Freqs& f, int n_cta, cudaStream_t s) {
  return a.layout == RATTN_LAYOUT_BHTD ? launch_layout<T, D, BWD, false>(a, f, n_cta, s)
                                       : launch_layout<T, D, BWD, true>(a, f, n_cta, s);
}

template <bool BWD>
cudaError_t launch(const QkArgs& a, const Freqs& f, int d, int dtype, int n_cta, cudaStream_t s) {
  if (dtype == RATTN_BF16)
    return d == 128 ? launch_one<__nv_bfloat16, 128, BWD>(a, f, n_cta, s) : launch_one<__nv_bfloat16, 64, BWD>(a, f, n_cta, s);
  return d == 128 ? launch_one<float, 128, BWD>(a, f, n_cta, s) : launch_one<float, 64, BWD>(a, f, n_cta, s);
}

int fail(cudaError_t e) {
  set_last_cuda_error((int)e);
  return RATTN_ERR_CUDA;
}

}  // namespace
}  // namespace rattn

using namespace rattn;

extern "C" {

size_t rattn_qk_prologue_workspace_bytes(int B, int H_q, int H_kv, int T, int d) {
  if (B < 1 || H_q < 1 || H_kv < 0 || T < 1 || (d != 64 && d != 128)) return 0;
  return (size_t)2 * QK_MAX_CTAS * d * sizeof(float);
}

int rattn_qk_prologue(const rattn_qk_params* p, void* stream) {
  int rc = check(p);
  if (rc != RATTN_OK) return rc;
  if (!p->q_out || (p->H_kv > 0 && !p->k_out)) return RATTN_ERR_NULL_PTR;
  if (misaligned16(p->q_out) || misaligned16(p->k_out)) return RATTN_ERR_MISALIGNED;
  QkArgs a;
  Freqs f;
  fill(p, &a, &f);
  a.y[0] = p->q_out; a.y[1] = p->k_out;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int n_cta = 0;
  cudaError_t e = grid_size(a, QK_CTAS_PER_SM, &n_cta);
  if (e == cudaSuccess) e = launch<false>(a, f, p->d, p->dtype, n_cta, s);
  return e == cudaSuccess ? RATTN_OK : fail(e);
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
  QkArgs a;
  Freqs f;
  fill(p, &a, &f);
  a.y[0] = dq; a.y[1] = dk;
  a.dy[0] = dq_out; a.dy[1] = dk_out;
  if (dq_gain || dk_gain) {
    if (!workspace || workspace_bytes < rattn_qk_prologue_workspace_bytes(p->B, p->H_q, p->H_kv, p->T, p->d) ||
        ((uintptr_t)workspace & 255u) != 0)
      return RATTN_ERR_WORKSPACE;
    a.partial = static_cast<float*>(workspace);
  }
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int n_cta = 0;
  cudaError_t e = grid_size(a, 2, &n_cta);
  if (e == cudaSuccess) e = launch<true>(a, f, p->d, p->dtype, n_cta, s);
  if (e == cudaSuccess && a.partial != nullptr) {
    KernelTimer kt("qk_gain_reduce", s);
    if (p->d == 128) qk_gain_reduce_kernel<128><<<2, 1024, 0, s>>>(a.partial, n_cta, dq_gain, dk_gain);
    else qk_gain_reduce_kernel<64><<<2, 1024, 0, s>>>(a.partial, n_cta, dq_gain, dk_gain);
    count_launches(1);
    e = cudaGetLastError();
  }
  return e == cudaSuccess ? RATTN_OK : fail(e);
}

int rattn_qk_prologue_status(void* stream) {
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int word = 0;
  cudaError_t e = cudaMemcpyFromSymbolAsync(&word, g_qk_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && word != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbolAsync(g_qk_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  if (e != cudaSuccess) return fail(e);
  return word == 0 ? RATTN_OK : RATTN_ERR_TIMEOUT;
}

}  // extern "C"
