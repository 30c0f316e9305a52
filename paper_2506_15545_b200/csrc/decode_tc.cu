// Single-token decode step for bf16, d = 128, windows that are a multiple of 64 and groups of up
// to 8 query heads: the ring and the state stream through shared memory by TMA.
//
// The step reads the K ring, the V ring and the fp32 state of a K/V head once and writes the
// state back (Section 2.1: a cache of at most w+1 tokens; Eq. 4: the state), so it is bound by
// HBM traffic.  One CTA per (batch entry, K/V head), two CTAs per SM.  Everything it will read
// is requested up front as 16 KB pieces (64 ring slots, or 32 state rows) that pass through a
// ring of stages (as many as let two CTAs share an SM, five at w = 512 with four heads), so the memory system always has the next pieces in flight, whatever the
// warps are doing.  The two ring products are small matrix products with the group's query heads
// as rows (q K^T, then P V), issued as warp-level mma on the pieces in shared memory (the K and V
// pieces arrive 128-byte swizzled, so the fragment loads are conflict-free); with at most 8 rows
// they are far too small for tcgen05's 64-row minimum.  The attention weights enter P V as a
// bf16 pair (value + remainder), which keeps 16 bits of them.  The state is read out and updated
// in fp32 on the CUDA cores.
#include "rattn_internal.h"
#include "tc_common.cuh"
#include "tc_ptx.cuh"

namespace rattn {
namespace {

using namespace ptx;

constexpr int DT_THREADS = 256;
constexpr int DT_WARPS = DT_THREADS / 32;
constexpr int DT_MAX_STAGES = 8;
constexpr int DT_PIECE = 16384;            // 64 ring slots x 128 bf16, or 32 state rows x 128 fp32
constexpr int D = 128;
constexpr int QB_STRIDE = D + 8;           // bf16 elements; 272 bytes: rows fall 16 bytes apart modulo 128

__device__ int g_decode_status;            // RATTN_ERR_TIMEOUT once a bounded wait has expired

struct DecodeTcArgs {
  const __nv_bfloat16* q; const __nv_bfloat16* k; const __nv_bfloat16* v;
  __nv_bfloat16* k_ring; __nv_bfloat16* v_ring; float* state; __nv_bfloat16* out;
  const float* gamma_swa; const float* gamma_rla;
  const int* pos_dev;
  int B, H_q, H_kv, w, pos, group, phi, stages;
  float scale, eps;
};

struct DecodeTcMaps {
  CUtensorMap k, v;                        // [B*H_kv, w, 128] bf16, box 64 columns x 64 slots
};

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

// phi over the 128 features by one warp (softmax, or one of the element-wise maps)
__device__ __forceinline__ void warp_feature_map(float* dst, const float* src, int lane, int phi) {
  float x[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) x[i] = src[lane + 32 * i];
  if (phi == RATTN_PHI_SOFTMAX) {
    const float m = warp_max(fmaxf(fmaxf(x[0], x[1]), fmaxf(x[2], x[3])));
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[i] = __expf(x[i] - m);
      s += x[i];
    }
    const float inv = 1.f / warp_sum(s);
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] *= inv;
  } else if (phi == RATTN_PHI_RELU) {
#pragma unroll
    for (int i = 0; i < 4; ++i) x[i] = fmaxf(x[i], 0.f);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) dst[lane + 32 * i] = x[i];
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
// c[16 x 8] += a[16 x 16] b[16 x 8], bf16 in, fp32 accumulate
__device__ __forceinline__ void mma_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// A fragment register holds the values of slots s (low half) and s + 1 (high half): zero those
// at or beyond `live`.
__device__ __forceinline__ uint32_t keep_valid(uint32_t pair, int s, int live) {
  return pair & (s < live ? 0x0000ffffu : 0u) | pair & (s + 1 < live ? 0xffff0000u : 0u);
}

// Shared-memory plan (bytes, after the 1024-byte aligned stages).
struct Plan {
  int stages, q_b, zero, p_hi, p_lo, logit, q_f, fq, vec, o_swa, o_rla, stat, red, bars, total;
};
__host__ __device__ inline Plan plan_with(int g, int w, int stages) {
  Plan p;
  p.stages = stages;
  int off = stages * DT_PIECE;
  auto take = [&](int bytes) { const int at = off; off += (bytes + 15) & ~15; return at; };
  p.q_b = take(8 * QB_STRIDE * 2);         // bf16 [8][136]: the group's queries, rows >= g zero
  p.zero = take(16);                       // what the fragment rows 8..15 point at
  p.p_hi = take(g * (w + 8) * 2);          // bf16 [g][w + 8]: attention weights, leading part
  p.p_lo = take(g * (w + 8) * 2);          //                  remainder
  p.logit = take(g * (w + 4) * 4);         // fp32 [g][w + 4]: scaled logits, then un-normalised weights
  p.q_f = take(g * D * 4);                 // fp32 raw q
  p.fq = take(g * D * 4);                  // phi(q)
  p.vec = take(5 * D * 4);                 // k_new, v_new, k_old, v_old, phi(k_old)
  p.o_swa = take(g * D * 4);
  p.o_rla = take(g * D * 4);
  p.stat = take(4 * 8 * 4);                // per head: 1 / sum, weight of the incoming token, incoming logit
  p.red = take(2 * DT_WARPS * 8 * 4);       // per warp and head: maximum, then sum, of its share of the logits
  p.bars = take(8 * DT_MAX_STAGES + 16);
  p.total = off + 1024;                    // room to align the stages
  return p;
}
// As many stages as let two CTAs share an SM (each may use (227 KB - 2 KB) / 2), at least three.
__host__ __device__ inline Plan plan(int g, int w, int forced = 0) {
  if (forced >= 3 && forced <= DT_MAX_STAGES && plan_with(g, w, forced).total <= 227 * 1024) return plan_with(g, w, forced);
  int stages = 6;
  while (stages > 3 && plan_with(g, w, stages).total > (227 * 1024 - 2048) / 2) --stages;
  return plan_with(g, w, stages);
}

template <int G>
__global__ void __launch_bounds__(DT_THREADS, 2)
decode_tc_kernel(const __grid_constant__ DecodeTcArgs a, const __grid_constant__ DecodeTcMaps maps) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int g = a.group, w = a.w;
  const Plan P = plan(g, w, a.stages);
  const int NS = P.stages;
  __nv_bfloat16* q_b = reinterpret_cast<__nv_bfloat16*>(sm + P.q_b);
  __nv_bfloat16* p_hi = reinterpret_cast<__nv_bfloat16*>(sm + P.p_hi);
  __nv_bfloat16* p_lo = reinterpret_cast<__nv_bfloat16*>(sm + P.p_lo);
  float* logit = reinterpret_cast<float*>(sm + P.logit);
  float* q_f = reinterpret_cast<float*>(sm + P.q_f);
  float* fq_s = reinterpret_cast<float*>(sm + P.fq);
  float* k_new = reinterpret_cast<float*>(sm + P.vec);
  float* v_new = k_new + D;
  float* k_old = v_new + D;
  float* v_old = k_old + D;
  float* fk_old = v_old + D;
  float* o_swa = reinterpret_cast<float*>(sm + P.o_swa);
  float* o_rla = reinterpret_cast<float*>(sm + P.o_rla);
  float* inv_sum = reinterpret_cast<float*>(sm + P.stat);      // [8]
  float* p_new = inv_sum + 8;                                  // [8] un-normalised weight of the incoming token
  float* l_new = p_new + 8;                                    // [8] its scaled logit
  float* w_max = reinterpret_cast<float*>(sm + P.red);         // [8 warps][8 heads]
  float* w_sum = w_max + DT_WARPS * 8;
  uint64_t* full = reinterpret_cast<uint64_t*>(sm + P.bars);
  volatile int* abort = reinterpret_cast<volatile int*>(full + DT_MAX_STAGES);
  const int LS = w + 4, PS = w + 8;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int z = blockIdx.x, b = z / a.H_kv, hk = z % a.H_kv;
  const int pos = a.pos_dev ? a.pos_dev[b] : a.pos;
  const bool evict = pos - w >= 0;
  const int slot = pos % w;
  const int n_valid = pos < w ? pos : w;
  const int np = (n_valid + 63) >> 6;                          // K (and V) pieces that hold valid slots
  const int n_pieces = 2 * np + 4;

  const __nv_bfloat16* qg = a.q + ((size_t)b * a.H_q + (size_t)hk * g) * D;
  const __nv_bfloat16* kg = a.k + (size_t)z * D;
  const __nv_bfloat16* vg = a.v + (size_t)z * D;
  __nv_bfloat16* kr = a.k_ring + (size_t)z * w * D;
  __nv_bfloat16* vr = a.v_ring + (size_t)z * w * D;
  float* S = a.state + (size_t)z * D * D;
  __nv_bfloat16* og = a.out + ((size_t)b * a.H_q + (size_t)hk * g) * D;

  // The step's small operands are requested before any bulk traffic: behind 20 MB of ring pieces
  // they would wait microseconds.  They go to registers here and to shared memory once the pieces
  // have been asked for.
  if (tid == 0) {
    prefetch_tensormap(&maps.k);
    prefetch_tensormap(&maps.v);
  }
  uint4 q_reg = make_uint4(0u, 0u, 0u, 0u);                      // thread (row, 16-byte chunk) of the group's queries
  if (tid < g * 16) q_reg = reinterpret_cast<const uint4*>(qg)[tid];
  __nv_bfloat16 kn = __float2bfloat16_rn(0.f), vn = kn, ko = kn, vo_ = kn;
  if (tid < D) {
    kn = kg[tid];
    vn = vg[tid];
    if (evict) {
      ko = kr[(size_t)slot * D + tid];
      vo_ = vr[(size_t)slot * D + tid];
    }
  }
  if (tid == 0) {
    for (int i = 0; i < NS; ++i) mbar_init(&full[i], 1);
    *abort = 0;
    fence_mbar_init();
  }
  __syncthreads();

  // piece p of the step's stream into stage p % NS (warp 0, all lanes)
  auto issue = [&](int p) {
    unsigned char* dst = sm + (p % NS) * DT_PIECE;
    uint64_t* bar = &full[p % NS];
    mbar_arrive_expect_tx(bar, DT_PIECE);
    if (p < 2 * np) {
      const CUtensorMap* m = p < np ? &maps.k : &maps.v;
      const int row = (p < np ? p : p - np) * 64;
      tma_load_3d(dst, m, bar, 0, row, z);
      tma_load_3d(dst + DT_PIECE / 2, m, bar, 64, row, z);
    } else {
      bulk_load_1d(dst, S + (size_t)(p - 2 * np) * 32 * D, DT_PIECE, bar);
    }
  };
  if (warp == 0)
    for (int p = 0; p < NS && p < n_pieces; ++p) issue(p);

  // queries: bf16 rows for the fragments (rows beyond the group zero), fp32 for phi and the new logit
  if (tid < 128) {
    const int r = tid >> 4, c = tid & 15;
    *reinterpret_cast<uint4*>(q_b + r * QB_STRIDE + c * 8) = q_reg;
    if (r < g) {
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&q_reg);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 x = __bfloat1622float2(h2[i]);
        q_f[r * D + c * 8 + 2 * i] = x.x;
        q_f[r * D + c * 8 + 2 * i + 1] = x.y;
      }
    }
  }
  if (tid < 4) reinterpret_cast<uint32_t*>(sm + P.zero)[tid] = 0u;
  if (tid < D) {
    k_new[tid] = __bfloat162float(kn);
    v_new[tid] = __bfloat162float(vn);
    k_old[tid] = __bfloat162float(ko);
    v_old[tid] = __bfloat162float(vo_);
  }
  // weights of slots that hold no token yet
  for (int r = 0; r < g; ++r)
    for (int c = n_valid + tid; c < PS; c += DT_THREADS) p_hi[r * PS + c] = p_lo[r * PS + c] = __float2bfloat16_rn(0.f);
  __syncthreads();

  // query fragments: rows 0..7 from q_b, rows 8..15 are zero
  const uint32_t zero_addr = smem_u32(sm + P.zero);
  uint32_t qa[8][4];
  {
    const bool upper = (lane >> 3) & 1;
#pragma unroll
    for (int kk = 0; kk < 8; ++kk) {
      const uint32_t addr = upper ? zero_addr : smem_u32(q_b + (lane & 7) * QB_STRIDE + (kk * 2 + (lane >> 4)) * 8);
      ldmatrix_x4(addr, qa[kk]);
    }
  }

  // phi(q), phi(k_old) and the incoming token's logit (Section 2.1), while the first pieces are on their way
  for (int r = warp; r <= g; r += DT_WARPS) {
    if (r < g) warp_feature_map(fq_s + r * D, q_f + r * D, lane, a.phi);
    else warp_feature_map(fk_old, k_old, lane, a.phi);
  }
  if (warp == DT_WARPS - 1) {
    for (int hh = 0; hh < g; ++hh) {
      float x = 0.f;
#pragma unroll
      for (int i = 0; i < 4; ++i) x += q_f[hh * D + lane + 32 * i] * k_new[lane + 32 * i];
      x = warp_sum(x);
      if (lane == 0) l_new[hh] = x * a.scale;
    }
  }

  int pc = 0;                                                    // pieces consumed so far
  bool ok = true;
  // ---- q K^T over the ring: piece = 64 slots, warp = 8 of them --------------------------------
  float my_max = -INFINITY;                                      // over this thread's logits (head lane / 4)
  for (int j = 0; j < np && ok; ++j, ++pc) {
    const bool got = mbar_wait_warp(&full[pc % NS], (uint32_t)(pc / NS) & 1u, abort);
    if (got) {
      const uint32_t base = smem_u32(sm + (pc % NS) * DT_PIECE);
      const int row = 8 * warp + (lane & 7);
      float c[4] = {0.f, 0.f, 0.f, 0.f}, c2[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int kk0 = 0; kk0 < 8; kk0 += 2) {
        const int chunk = (kk0 + (lane >> 4)) * 2 + ((lane >> 3) & 1);
        uint32_t kb[4];
        ldmatrix_x4(base + (chunk >> 3) * (DT_PIECE / 2) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4), kb);
        mma_16816(c, qa[kk0], kb[0], kb[1]);
        mma_16816(c2, qa[kk0 + 1], kb[2], kb[3]);
      }
      const int hh = lane >> 2, s = j * 64 + 8 * warp + 2 * (lane & 3);
      if (hh < g) {
        const float l0 = (c[0] + c2[0]) * a.scale, l1 = (c[1] + c2[1]) * a.scale;
        logit[hh * LS + s] = l0;
        logit[hh * LS + s + 1] = l1;
        if (s < n_valid) my_max = fmaxf(my_max, l0);             // a slot without a token may hold anything
        if (s + 1 < n_valid) my_max = fmaxf(my_max, l1);
      }
    }
    ok = __syncthreads_and(got) != 0;
    if (ok && warp == 0 && pc + NS < n_pieces) issue(pc + NS);
  }
  my_max = fmaxf(my_max, __shfl_xor_sync(0xffffffffu, my_max, 1));
  my_max = fmaxf(my_max, __shfl_xor_sync(0xffffffffu, my_max, 2));
  if ((lane & 3) == 0) w_max[warp * 8 + (lane >> 2)] = my_max;
  __syncthreads();

  // ---- softmax over the window: thread = slot, all heads; weights as a bf16 pair ------------------
  {
    float m[G], l[G];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      l[hh] = 0.f;
      m[hh] = hh < g ? l_new[hh] : 0.f;
#pragma unroll
      for (int wv = 0; wv < DT_WARPS; ++wv) m[hh] = fmaxf(m[hh], w_max[wv * 8 + hh]);
    }
    for (int s = tid; s < n_valid; s += DT_THREADS) {
#pragma unroll
      for (int hh = 0; hh < G; ++hh) {
        if (hh < g) {
          const float e = __expf(logit[hh * LS + s] - m[hh]);
          l[hh] += e;
          const __nv_bfloat16 hi = __float2bfloat16_rn(e);
          p_hi[hh * PS + s] = hi;
          p_lo[hh * PS + s] = __float2bfloat16_rn(e - __bfloat162float(hi));
        }
      }
    }
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
      l[hh] = warp_sum(l[hh]);
      if (lane == 0) w_sum[warp * 8 + hh] = l[hh];
    }
    __syncthreads();
    if (tid < g) {
      float tot = 0.f;
#pragma unroll
      for (int wv = 0; wv < DT_WARPS; ++wv) tot += w_sum[wv * 8 + tid];
      float mm = l_new[tid];
#pragma unroll
      for (int wv = 0; wv < DT_WARPS; ++wv) mm = fmaxf(mm, w_max[wv * 8 + tid]);
      const float en = __expf(l_new[tid] - mm);
      p_new[tid] = en;
      inv_sum[tid] = 1.f / (tot + en);
    }
    __syncthreads();
  }

  // ---- P V: piece = 64 slots of V, warp = 16 of the 128 value features.  Rows 0..7 of the weight
  // fragment carry the leading parts, rows 8..15 the remainders: one product gives both.
  float o[2][2][4];                                              // [slot-step parity][feature tile][fragment]
#pragma unroll
  for (int i = 0; i < 16; ++i) o[i >> 3][(i >> 2) & 1][i & 3] = 0.f;
  for (int j = 0; j < np && ok; ++j, ++pc) {
    const bool got = mbar_wait_warp(&full[pc % NS], (uint32_t)(pc / NS) & 1u, abort);
    if (got) {
      unsigned char* piece = sm + (pc % NS) * DT_PIECE;
      const uint32_t base = smem_u32(piece);
      const bool upper = (lane >> 3) & 1;
      const int chunk = 2 * warp + (lane >> 4);
      const int live = n_valid - j * 64;                         // slots of this piece that hold a token
      const __nv_bfloat16* p_part = (upper ? p_lo : p_hi) + (lane & 7) * PS + j * 64 + (lane >> 4) * 8;
#pragma unroll
      for (int ks = 0; ks < 4; ++ks) {
        if (ks * 16 >= live) break;                              // nothing but zero weights from here on
        const int row = ks * 16 + (lane & 7) + (upper ? 8 : 0);
        uint32_t vb[4], pa[4];
        ldmatrix_x4_trans(base + (chunk >> 3) * (DT_PIECE / 2) + row * 128 + (((chunk & 7) ^ (row & 7)) << 4), vb);
        if (live < 64) {
          // a slot without a token may hold anything; its weight is zero, but 0 * NaN is not
          const int s0 = ks * 16 + 2 * (lane & 3);
          vb[0] = keep_valid(vb[0], s0, live);
          vb[2] = keep_valid(vb[2], s0, live);
          vb[1] = keep_valid(vb[1], s0 + 8, live);
          vb[3] = keep_valid(vb[3], s0 + 8, live);
        }
        ldmatrix_x4((lane & 7) >= g ? zero_addr : smem_u32(p_part + ks * 16), pa);
        mma_16816(o[ks & 1][0], pa, vb[0], vb[1]);
        mma_16816(o[ks & 1][1], pa, vb[2], vb[3]);
      }
    }
    ok = __syncthreads_and(got) != 0;
    if (ok && warp == 0 && pc + NS < n_pieces) issue(pc + NS);
  }
  if (ok) {
    const int hh = lane >> 2;
    if (hh < g) {
#pragma unroll
      for (int nt = 0; nt < 2; ++nt) {
        const int c = 16 * warp + 8 * nt + 2 * (lane & 3);
        const float x0 = o[0][nt][0] + o[0][nt][2] + o[1][nt][0] + o[1][nt][2];
        const float x1 = o[0][nt][1] + o[0][nt][3] + o[1][nt][1] + o[1][nt][3];
        o_swa[hh * D + c] = (x0 + p_new[hh] * v_new[c]) * inv_sum[hh];
        o_swa[hh * D + c + 1] = (x1 + p_new[hh] * v_new[c + 1]) * inv_sum[hh];
      }
    }
    // the incoming token takes the evicted token's slot: every piece of the ring has been consumed
    if (tid < D) {
      kr[(size_t)slot * D + tid] = kn;
      vr[(size_t)slot * D + tid] = vn;
    }
  }

  // ---- the state: read-out phi(q) S and the update S += phi(k_old)^T v_old (Eq. 4), fp32 -----------
  // thread = one float4 column group (c4) and one of 8 row lanes (rl) that sit in the same warp
  {
    const int rl = (lane >> 2) & 7, c4 = (lane & 3) | (warp << 2);
    float4 ar[G];
#pragma unroll
    for (int hh = 0; hh < G; ++hh) ar[hh] = make_float4(0.f, 0.f, 0.f, 0.f);
    const float4 vo = *reinterpret_cast<const float4*>(v_old + c4 * 4);
    for (int i = 0; i < 4 && ok; ++i, ++pc) {
      const bool got = mbar_wait_warp(&full[pc % NS], (uint32_t)(pc / NS) & 1u, abort);
      if (got) {
        const float* piece = reinterpret_cast<const float*>(sm + (pc % NS) * DT_PIECE);
#pragma unroll
        for (int m = 0; m < 4; ++m) {
          const int rp = rl + 8 * m, r = 32 * i + rp;
          float4 s4 = *reinterpret_cast<const float4*>(piece + rp * D + c4 * 4);
#pragma unroll
          for (int hh = 0; hh < G; ++hh) {
            const float f = hh < g ? fq_s[hh * D + r] : 0.f;
            ar[hh].x += f * s4.x; ar[hh].y += f * s4.y; ar[hh].z += f * s4.z; ar[hh].w += f * s4.w;
          }
          if (evict) {
            const float fk = fk_old[r];
            s4.x += fk * vo.x; s4.y += fk * vo.y; s4.z += fk * vo.z; s4.w += fk * vo.w;
            *reinterpret_cast<float4*>(S + (size_t)r * D + c4 * 4) = s4;
          }
        }
      }
      ok = __syncthreads_and(got) != 0;
      if (ok && warp == 0 && pc + NS < n_pieces) issue(pc + NS);
    }
#pragma unroll
    for (int hh = 0; hh < G; ++hh) {
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        ar[hh].x += __shfl_xor_sync(0xffffffffu, ar[hh].x, off);
        ar[hh].y += __shfl_xor_sync(0xffffffffu, ar[hh].y, off);
        ar[hh].z += __shfl_xor_sync(0xffffffffu, ar[hh].z, off);
        ar[hh].w += __shfl_xor_sync(0xffffffffu, ar[hh].w, off);
      }
      if (rl == 0 && hh < g) *reinterpret_cast<float4*>(o_rla + hh * D + c4 * 4) = ar[hh];
    }
  }
  __syncthreads();

  if (!ok) {
    // a wait ran out: give what is still in flight a bounded time to land, report, leave the caches alone
    if (tid == 0) {
      for (int p = pc; p < n_pieces && p < pc + NS; ++p)
        for (int it = 0; it < kWaitPolls && !mbar_try_wait(&full[p % NS], (uint32_t)(p / NS) & 1u); ++it) {}
      g_decode_status = RATTN_ERR_TIMEOUT;
    }
    return;
  }

  // ---- Section 3.2: two RMS norms and the sum -----------------------------------------------------
  if (warp < g) {
    const int h = hk * g + warp;
    float x[4], y[4], ss = 0.f, sr = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      x[i] = o_swa[warp * D + lane + 32 * i];
      y[i] = o_rla[warp * D + lane + 32 * i];
      ss += x[i] * x[i];
      sr += y[i] * y[i];
    }
    ss = warp_sum(ss);
    sr = warp_sum(sr);
    const float is = rsqrtf(ss / D + a.eps), ir = rsqrtf(sr / D + a.eps);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int c = lane + 32 * i;
      const float gs = a.gamma_swa ? a.gamma_swa[(size_t)h * D + c] : 1.f;
      const float gr = a.gamma_rla ? a.gamma_rla[(size_t)h * D + c] : 1.f;
      og[(size_t)warp * D + c] = __float2bfloat16_rn(gs * x[i] * is + gr * y[i] * ir);
    }
  }
}

template <int G>
cudaError_t launch_g(const DecodeTcArgs& a, const DecodeTcMaps& m, int smem, cudaStream_t s) {
  cudaError_t e = cudaFuncSetAttribute(decode_tc_kernel<G>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
  if (e != cudaSuccess) return e;
  { KernelTimer kt("decode_step", s); decode_tc_kernel<G><<<a.B * a.H_kv, DT_THREADS, smem, s>>>(a, m); }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace

bool decode_tc_applies(const Args& p, int w) {
  return p.dtype == RATTN_BF16 && p.d == 128 && w % 64 == 0 && p.group <= 8 && plan(p.group, w).total <= 227 * 1024;
}

cudaError_t launch_decode_tc(const Args& p, void* k_ring, void* v_ring, float* state, int pos, const int* pos_dev,
                             cudaStream_t s) {
  DecodeTcArgs a;
  a.q = static_cast<const __nv_bfloat16*>(p.q);
  a.k = static_cast<const __nv_bfloat16*>(p.k);
  a.v = static_cast<const __nv_bfloat16*>(p.v);
  a.k_ring = static_cast<__nv_bfloat16*>(k_ring);
  a.v_ring = static_cast<__nv_bfloat16*>(v_ring);
  a.state = state;
  a.out = static_cast<__nv_bfloat16*>(p.out);
  a.gamma_swa = p.gamma_swa; a.gamma_rla = p.gamma_rla;
  a.pos_dev = pos_dev;
  a.B = p.B; a.H_q = p.H_q; a.H_kv = p.H_kv; a.w = p.w; a.pos = pos; a.group = p.group; a.phi = p.phi;
  a.scale = p.scale; a.eps = p.eps;
  DecodeTcMaps m;
  if (!tc::make_map(&m.k, k_ring, (uint64_t)p.w, (uint64_t)p.B * p.H_kv, 64) ||
      !tc::make_map(&m.v, v_ring, (uint64_t)p.w, (uint64_t)p.B * p.H_kv, 64))
    return cudaErrorInvalidValue;
  a.stages = tuning(RATTN_TUNE_DECODE_STAGES);
  const int smem = plan(p.group, p.w, a.stages).total;
  if (p.group == 1) return launch_g<1>(a, m, smem, s);
  if (p.group == 2) return launch_g<2>(a, m, smem, s);
  if (p.group <= 4) return launch_g<4>(a, m, smem, s);
  return launch_g<8>(a, m, smem, s);
}

int decode_tc_status(cudaStream_t s, cudaError_t* err) {
  int word = 0;
  cudaError_t e = cudaMemcpyFromSymbolAsync(&word, g_decode_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && word != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbolAsync(g_decode_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  *err = e;
  return word;
}

}  // namespace rattn
