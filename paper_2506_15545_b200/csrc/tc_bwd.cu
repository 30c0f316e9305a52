// Tensor-core backward for bf16, d = 128, window a multiple of 128 (sm_100a: TMA + tcgen05 + TMEM).
//
// The paper prints no backward formulas; these follow from its definitions by the chain rule
// (Section 2.1 for the window branch, Eq. 4 in the chunkwise form of Eq. 2-3 for the residual
// branch, Section 3.1 for the feature map, Section 3.2 for the two norms).  With 128-token
// tiles, chunk c = key tile c, lag wt = w / 128, and for query tile i the "boundary" chunk
// cb = i - wt (the chunk the residual branch reads in intra form, masked to j < t - w):
//
//   prep      per row: gradients g_s, g_r of the two un-normalised branch outputs (through the
//             RMS norms and gains), D_t = g_s . o_swa, all from the forward's residuals.
//   window    P = exp(scale q.k - lse),  dP = g_s V^T,  dS = P * (dP - D) * scale,
//             dQ += dS K,   dK += dS^T Q,   dV += P^T g_s.
//   residual  forward states S_c = sum_{c' < c} phi(K_c')^T V_c' (saved by the forward) and
//             reverse states R_c = sum_{i > c + wt} phi(Q_i)^T g_r,i (summed over the query
//             heads of the group; computed here by an outer-product kernel and a suffix scan):
//               dphi_q = g_r S_cb^T + ((g_r V_cb^T) masked) phi(K_cb)
//               dphi_k = V_c R_c^T  + ((V_c g_r^T) masked) phi(Q_{c+wt})
//               dV    += phi(K_c) R_c + ((phi(K_c) phi(Q_{c+wt})^T) masked) g_r
//   feature   dq += phi(q) * (dphi_q - <dphi_q, phi(q)>), the same for k.
//
// Two main kernels, so that every output tile has one owner and nothing is accumulated with
// atomics (results are deterministic):
//   tc_bwd_dq_kernel   a (query head, query tile) item loops over the key tiles of its band;
//   tc_bwd_dkv_kernel  a (K/V head, key tile) item loops over the group's query heads and, for
//                      each, over the query half tiles whose band contains the key tile.
// Both are persistent (one CTA per SM walks its items, the next item's loads in flight while
// the current one's epilogue drains) and warp-specialised: row groups of 128 threads own one
// accumulator row each (row = TMEM lane), a loader warp issues the TMA loads, an MMA warp the
// tcgen05 products; all accumulation is fp32 in TMEM, and the weight matrices of each tile
// pair (P, dS) are rounded to bf16 and handed to the tensor core through TMEM.
#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

constexpr float LOG2E = 1.4426950408889634f;

struct BwdArgs {
  __nv_bfloat16* dq;
  __nv_bfloat16* dk;
  __nv_bfloat16* dv;
  const float* lse;     // [B,H_q,T]  natural-log log-sum-exp of the window logits
  const float* delta;   // [B,H_q,T]  D_t
  const float* lse2p;   // [B*H_q, t_pad]  lse * log2(e), +inf beyond T   (t_pad = T rounded up to 128)
  const float* dscp;    // [B*H_q, t_pad]  D_t * scale, 0 beyond T
  int t_pad;
  int* status;
  int T, w, H_q, group, mode, n_chunks;
  int phi;              // rattn_feature_map
  float scale, scale_log2;
};

#define WAIT_OR_RETURN(bar, parity) \
  do { if (!mbar_wait(&(bar), (parity), &bars->abort)) return false; } while (0)
// for roles run by a whole converged warp
#define WAIT_OR_RETURN_W(bar, parity) \
  do { if (!mbar_wait_warp(&(bar), (parity), &bars->abort)) return false; } while (0)

// ------------------------------------------------------------------------------ prep
// A pure stream: dO and the two un-normalised branch outputs in, g_s and g_r out (bf16), plus the
// per-row statistics; bound by HBM.  The unit is a chunk of 32 rows of one head (8 KB per tensor,
// contiguous), which travels global -> shared -> global as bulk asynchronous copies through a ring
// of stages, so the bytes in flight do not depend on where the warps are; the rows are transformed
// in place in shared memory (g_s over o_swa, g_r over o_rla).  Eight neighbouring lanes hold a row:
// lane l has features [8l, 8l+8) and [64+8l, 64+8l+8).  Every CTA takes an equal contiguous share of
// the chunks (head-major), so it meets few heads and keeps its gain-gradient sums in registers.
// With n = o / r (r the rms incl. eps), gh = dy * gain, A = gh . o:
//   g = (gh - n * (A / (128 r))) / r,   D = g . o = (A - A ss / (128 r^2)) / r,
// so each branch needs two row sums (ss = o . o and A).
constexpr int PREP_THREADS = 256;
constexpr int PREP_ROWS = 32;                       // rows of a chunk
constexpr int PREP_CHUNK = PREP_ROWS * 256;         // bytes of a chunk of one tensor
constexpr int PREP_STAGES = 4;
constexpr int PREP_SMEM = PREP_STAGES * 3 * PREP_CHUNK + 128;

struct PrepArgs {
  const __nv_bfloat16* o_s; const __nv_bfloat16* o_r;
  const float* gamma_s; const float* gamma_r;
  __nv_bfloat16* g_s; __nv_bfloat16* g_r;
  float* delta; float* dgamma_s; float* dgamma_r;
  const float* lse; float* lse2p; float* dscp;
  int* status;
  int n_heads, T, t_pad, H_q, rla_on;
  float eps, scale;
};

__device__ __forceinline__ void unpack8(const unsigned char* p, float (&x)[8]) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    x[2 * i] = __uint_as_float(w[i] << 16);
    x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
  }
}

__global__ void __launch_bounds__(PREP_THREADS, 2)
tc_bwd_prep_kernel(const __grid_constant__ PrepArgs a, const __grid_constant__ CUtensorMap dy_map) {
  extern __shared__ __align__(128) unsigned char psm[];
  uint64_t* full = reinterpret_cast<uint64_t*>(psm + PREP_STAGES * 3 * PREP_CHUNK);
  volatile int* abort = reinterpret_cast<volatile int*>(full + PREP_STAGES);
  const int tid = threadIdx.x, l = tid & 7, row = tid >> 3;
  const int cph = a.t_pad / PREP_ROWS;                              // chunks per head
  const long long n_all = (long long)a.n_heads * cph;
  const int lo = (int)(n_all * blockIdx.x / gridDim.x), hi = (int)(n_all * (blockIdx.x + 1) / gridDim.x);
  const int n_in = a.rla_on ? 3 : 2;                                // tensors read per chunk

  if (tid == 0) {
    prefetch_tensormap(&dy_map);
    for (int i = 0; i < PREP_STAGES; ++i) mbar_init(&full[i], 1);
    *abort = 0;
    fence_mbar_init();
  }
  __syncthreads();

  // chunk i: head i / cph, rows t0 .. t0 + 31 of it; rows at or beyond T are padding (nothing is copied)
  auto rows_of = [&](int i) { const int t0 = (i % cph) * PREP_ROWS; return a.T - t0 < 0 ? 0 : a.T - t0 < PREP_ROWS ? a.T - t0 : PREP_ROWS; };
  // Thread 0 keeps the ring fed: the next chunk with data goes into stage (chunks issued so far) % stages.
  int cursor = lo, n_issued = 0;
  auto issue_next = [&]() {
    while (cursor < hi && rows_of(cursor) == 0) ++cursor;
    if (cursor >= hi) return;
    const int i = cursor++, rows = rows_of(i);
    const size_t at = ((size_t)(i / cph) * a.T + (size_t)(i % cph) * PREP_ROWS) * 128;
    unsigned char* dst = psm + (size_t)(n_issued % PREP_STAGES) * 3 * PREP_CHUNK;
    uint64_t* bar = &full[n_issued % PREP_STAGES];
    ++n_issued;
    const uint32_t bytes = (uint32_t)rows * 256;
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;"
                 ::"r"(smem_u32(bar)), "r"((uint32_t)PREP_CHUNK + bytes * (n_in - 1)) : "memory");
    // dO is the caller's tensor (either head layout): a tiled copy of 32 whole rows, rows beyond T read as zero
    const int bq_ = i / cph, b_ = bq_ / a.H_q, h_ = bq_ - b_ * a.H_q;
    asm volatile("cp.async.bulk.tensor.4d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5, %6}], [%2];"
                 ::"r"(smem_u32(dst)), "l"(&dy_map), "r"(smem_u32(bar)), "r"(0), "r"((i % cph) * PREP_ROWS), "r"(h_), "r"(b_)
                 : "memory");
    const __nv_bfloat16* src[3] = {nullptr, a.o_s, a.o_r};
    for (int k = 1; k < n_in; ++k)
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(dst + k * PREP_CHUNK)), "l"(src[k] + at), "r"(bytes), "r"(smem_u32(bar)) : "memory");
  };
  if (tid == 0)
    for (int k = 0; k < PREP_STAGES - 1; ++k) issue_next();

  float gs_lo[8], gs_hi[8], gr_lo[8], gr_hi[8], acc_s[16], acc_r[16];
#pragma unroll
  for (int e = 0; e < 16; ++e) acc_s[e] = acc_r[e] = 0.f;
  int cur_h = -1;
  auto flush = [&]() {                                              // this CTA's sums for head cur_h
    if (cur_h < 0) return;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      if (a.dgamma_s) {
        atomicAdd(a.dgamma_s + (size_t)cur_h * 128 + 8 * l + e, acc_s[e]);
        atomicAdd(a.dgamma_s + (size_t)cur_h * 128 + 64 + 8 * l + e, acc_s[8 + e]);
      }
      if (a.dgamma_r && a.rla_on) {
        atomicAdd(a.dgamma_r + (size_t)cur_h * 128 + 8 * l + e, acc_r[e]);
        atomicAdd(a.dgamma_r + (size_t)cur_h * 128 + 64 + 8 * l + e, acc_r[8 + e]);
      }
      acc_s[e] = acc_s[8 + e] = acc_r[e] = acc_r[8 + e] = 0.f;
    }
  };

  int i = lo, n_cons = 0;                                           // n_cons: chunks with data consumed so far
  bool ok = true;
  for (; i < hi; ++i) {
    const int bq = i / cph, t0 = (i % cph) * PREP_ROWS, rows = rows_of(i);
    const int t = t0 + row;
    const size_t prow = (size_t)bq * a.t_pad + t;
    if (rows == 0) {                                                // padding only: statistics that make every weight zero
      if (l == 0) { a.lse2p[prow] = INFINITY; a.dscp[prow] = 0.f; }
      continue;
    }
    const int h = bq % a.H_q;
    if (h != cur_h) {
      if (a.dgamma_s || a.dgamma_r) flush();
      cur_h = h;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        gs_lo[e] = a.gamma_s ? __ldg(a.gamma_s + (size_t)h * 128 + 8 * l + e) : 1.f;
        gs_hi[e] = a.gamma_s ? __ldg(a.gamma_s + (size_t)h * 128 + 64 + 8 * l + e) : 1.f;
        gr_lo[e] = a.gamma_r ? __ldg(a.gamma_r + (size_t)h * 128 + 8 * l + e) : 1.f;
        gr_hi[e] = a.gamma_r ? __ldg(a.gamma_r + (size_t)h * 128 + 64 + 8 * l + e) : 1.f;
      }
    }
    const int slot = n_cons % PREP_STAGES;
    unsigned char* buf = psm + (size_t)slot * 3 * PREP_CHUNK + row * 256 + 16 * l;
    const bool live = row < rows;
    // the row's log-sum-exp is asked for before the wait, so that its latency passes under it
    const float lse_row = (live && l == 0) ? __ldg(a.lse + (size_t)bq * a.T + t) : 0.f;
    const bool got = mbar_wait_warp(&full[slot], (uint32_t)(n_cons / PREP_STAGES) & 1u, abort);
    if (got) {
      float g_lo[8], g_hi[8], s_lo[8], s_hi[8], r_lo[8], r_hi[8];
      if (live) {
        unpack8(buf, g_lo); unpack8(buf + 128, g_hi);
        unpack8(buf + PREP_CHUNK, s_lo); unpack8(buf + PREP_CHUNK + 128, s_hi);
      }
      if (live && a.rla_on) { unpack8(buf + 2 * PREP_CHUNK, r_lo); unpack8(buf + 2 * PREP_CHUNK + 128, r_hi); }
      if (!live || !a.rla_on) {
#pragma unroll
        for (int e = 0; e < 8; ++e) r_lo[e] = r_hi[e] = 0.f;
      }
      if (!live) {
#pragma unroll
        for (int e = 0; e < 8; ++e) g_lo[e] = g_hi[e] = s_lo[e] = s_hi[e] = 0.f;
      }
      float ss = 0.f, sr = 0.f, As = 0.f, Ar = 0.f;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        ss += s_lo[e] * s_lo[e] + s_hi[e] * s_hi[e];
        sr += r_lo[e] * r_lo[e] + r_hi[e] * r_hi[e];
        As += g_lo[e] * gs_lo[e] * s_lo[e] + g_hi[e] * gs_hi[e] * s_hi[e];
        Ar += g_lo[e] * gr_lo[e] * r_lo[e] + g_hi[e] * gr_hi[e] * r_hi[e];
      }
#pragma unroll
      for (int o = 1; o < 8; o <<= 1) {
        ss += __shfl_xor_sync(0xffffffffu, ss, o);
        sr += __shfl_xor_sync(0xffffffffu, sr, o);
        As += __shfl_xor_sync(0xffffffffu, As, o);
        Ar += __shfl_xor_sync(0xffffffffu, Ar, o);
      }
      const float is = rsqrtf(ss * (1.f / 128.f) + a.eps), ir = rsqrtf(sr * (1.f / 128.f) + a.eps);
      const float cs = As * is * is * (1.f / 128.f), cr = Ar * ir * ir * (1.f / 128.f);   // mean(gh n) / r
      if (live) {
        uint32_t w_lo[4], w_hi[4];
#pragma unroll
        for (int e = 0; e < 8; e += 2) {
          w_lo[e >> 1] = pack_bf16((g_lo[e] * gs_lo[e] - s_lo[e] * cs) * is, (g_lo[e + 1] * gs_lo[e + 1] - s_lo[e + 1] * cs) * is);
          w_hi[e >> 1] = pack_bf16((g_hi[e] * gs_hi[e] - s_hi[e] * cs) * is, (g_hi[e + 1] * gs_hi[e + 1] - s_hi[e + 1] * cs) * is);
        }
        *reinterpret_cast<uint4*>(buf + PREP_CHUNK) = make_uint4(w_lo[0], w_lo[1], w_lo[2], w_lo[3]);
        *reinterpret_cast<uint4*>(buf + PREP_CHUNK + 128) = make_uint4(w_hi[0], w_hi[1], w_hi[2], w_hi[3]);
        if (a.rla_on) {
#pragma unroll
          for (int e = 0; e < 8; e += 2) {
            w_lo[e >> 1] = pack_bf16((g_lo[e] * gr_lo[e] - r_lo[e] * cr) * ir, (g_lo[e + 1] * gr_lo[e + 1] - r_lo[e + 1] * cr) * ir);
            w_hi[e >> 1] = pack_bf16((g_hi[e] * gr_hi[e] - r_hi[e] * cr) * ir, (g_hi[e + 1] * gr_hi[e + 1] - r_hi[e + 1] * cr) * ir);
          }
          *reinterpret_cast<uint4*>(buf + 2 * PREP_CHUNK) = make_uint4(w_lo[0], w_lo[1], w_lo[2], w_lo[3]);
          *reinterpret_cast<uint4*>(buf + 2 * PREP_CHUNK + 128) = make_uint4(w_hi[0], w_hi[1], w_hi[2], w_hi[3]);
        }
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          acc_s[e] += g_lo[e] * s_lo[e] * is;
          acc_s[8 + e] += g_hi[e] * s_hi[e] * is;
          acc_r[e] += g_lo[e] * r_lo[e] * ir;
          acc_r[8 + e] += g_hi[e] * r_hi[e] * ir;
        }
      }
      if (l == 0) {
        if (live) {
          const size_t grow = (size_t)bq * a.T + t;
          const float dl = (As - cs * ss) * is;                     // D_t = g_s . o_swa
          a.delta[grow] = dl;
          a.lse2p[prow] = lse_row * LOG2E;
          a.dscp[prow] = dl * a.scale;
        } else {
          a.lse2p[prow] = INFINITY;
          a.dscp[prow] = 0.f;
        }
      }
      fence_proxy_async_smem();
    }
    ok = __syncthreads_and(got) != 0;
    if (!ok) break;
    if (tid == 0) {
      const size_t at = ((size_t)bq * a.T + t0) * 128;
      unsigned char* src = psm + (size_t)slot * 3 * PREP_CHUNK;
      const uint32_t bytes = (uint32_t)rows * 256;
      asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(a.g_s + at), "r"(smem_u32(src + PREP_CHUNK)), "r"(bytes) : "memory");
      if (a.rla_on)
        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(a.g_r + at), "r"(smem_u32(src + 2 * PREP_CHUNK)), "r"(bytes) : "memory");
      tma_store_commit();
      asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");   // the stage of the chunk before this one has been read out
      issue_next();
    }
    ++n_cons;
  }
  if (tid == 0) {
    tma_store_wait();
    if (!ok) {
      // give the copies still in flight a bounded time to land before the CTA's memory goes away
      for (int n = n_cons; n < n_issued; ++n)
        for (int it = 0; it < kWaitPolls && !mbar_try_wait(&full[n % PREP_STAGES], (uint32_t)(n / PREP_STAGES) & 1u); ++it) {}
      atomicExch(a.status, RATTN_ERR_TIMEOUT);
    }
  }
  if (ok && (a.dgamma_s || a.dgamma_r)) flush();
}

// ================================================================================ dq
// Persistent: one CTA per SM walks a list of (query head, query tile) items, so that an item's
// first loads are in flight while the previous item's epilogue drains (at w = 512 the fixed
// cost per tile -- first TMA touch, output staging -- is larger than the band itself).
//   loader warp   Q (two buffers, alternating), g_s, K/V tiles through a ring of two stages;
//                 the residual operands (g_r, stored state) take one more slot of that ring
//   MMA warp      per key tile S = Q K^T, dP = g_s V^T; after the row groups have overwritten S
//                 with dS (bf16, in TMEM): dQ += dS K.  Then the residual part.
//   row groups    two groups of 128 threads (thread = query row = TMEM lane), group g takes the
//                 key columns 64g .. 64g+63 of every tile; group 0 runs the epilogue
// All barriers run on with phase counters that every role advances in the same way.
constexpr int DQ_OFF_Q = 0;                 // Q buffer 0
constexpr int DQ_OFF_G = 1 * TILE_BYTES;
constexpr int DQ_OFF_K = 2 * TILE_BYTES;   // 2 stages
constexpr int DQ_OFF_V = 4 * TILE_BYTES;   // 2 stages
constexpr int DQ_OFF_Q1 = 6 * TILE_BYTES;  // Q buffer 1
constexpr int DQ_OFF_BAR = 7 * TILE_BYTES;
constexpr int DQ_SMEM = DQ_OFF_BAR + 256;
constexpr int DQ_THREADS = 320;            // 2 row groups, MMA warp, loader warp

struct DqBars {
  uint64_t qg_full, kv_full[2], kv_free[2], s_full, ds_full, phik_ready, o_done, acc_free, q_read, drain;
  uint32_t tmem_base;
  int abort;
};

struct DqItem {
  int q0, bh_q, bh_kv, n_kt, st_index;
  bool has_boundary, has_rla, has_state;
};

__device__ __forceinline__ DqItem dq_item(const BwdArgs& a, int idx, int n_qt) {
  DqItem it;
  it.bh_q = idx / n_qt;
  const int qt = n_qt - 1 - idx % n_qt;                    // long bands first within a head
  it.q0 = qt * TILE;
  const int b = it.bh_q / a.H_q, h = it.bh_q % a.H_q;
  it.bh_kv = b * (a.H_q / a.group) + h / a.group;
  const int wt = a.w / TILE;
  it.has_boundary = (a.mode != RATTN_MODE_FULL_CAUSAL) && (qt - wt >= 0);
  it.n_kt = (it.has_boundary ? wt : qt) + 1;
  it.has_rla = it.has_boundary && (a.mode == RATTN_MODE_RATTN);
  const int cb = qt - wt;
  it.has_state = it.has_rla && cb > 0;
  it.st_index = it.bh_kv * a.n_chunks + (cb > 0 ? cb : 0);
  return it;
}

struct DqMaps {
  UMap q, k, v, dq;             // the caller's tensors (either head layout)
  CUtensorMap gs, gr, st;
};

__device__ bool dq_loader(const DqMaps& tm, const BwdArgs& a, unsigned char* smem, DqBars* bars, int n_items, int n_qt) {
  int kc = 0, n = 0, co = 0;                               // ring uses, items, o_done completions so far
  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++n) {
    const DqItem it = dq_item(a, idx, n_qt);
    auto ring_wait = [&]() -> bool {                       // the slot's previous user has been consumed
      const int st = kc & 1, use = kc >> 1;
      if (use >= 1) WAIT_OR_RETURN_W(bars->kv_free[st], (use - 1) & 1);
      return true;
    };
    // The barrier's previous phase must be over before this item arrives on it: after a short
    // item the loader gets here while that item's Q and g_s are still in flight.
    if (n >= 1) WAIT_OR_RETURN_W(bars->qg_full, (n - 1) & 1);
    mbar_arrive_expect_tx(&bars->qg_full, 2 * TILE_BYTES);
    // Q into the buffer last used two items ago: free once that item's epilogue has left it
    if (n >= 2) {
      WAIT_OR_RETURN_W(bars->acc_free, (n - 2) & 1);
      WAIT_OR_RETURN_W(bars->q_read, (n - 2) & 1);      // and its dQ, staged there, has left
    }
    load_tile(smem + ((n & 1) ? DQ_OFF_Q1 : DQ_OFF_Q), &tm.q, &bars->qg_full, it.q0, it.bh_q);
    // g_s: its one buffer is free once every product of the previous item has completed
    // (o_done completes twice for an item with a residual part, once otherwise)
    if (n >= 1) WAIT_OR_RETURN_W(bars->o_done, (co - 1) & 1);
    co += it.has_rla ? 2 : 1;
    load_tile(smem + DQ_OFF_G, &tm.gs, &bars->qg_full, it.q0, it.bh_q);
    for (int i = 0; i < it.n_kt; ++i, ++kc) {
      if (!ring_wait()) return false;
      const int st = kc & 1;
      mbar_arrive_expect_tx(&bars->kv_full[st], 2 * TILE_BYTES);
      load_tile(smem + DQ_OFF_K + st * TILE_BYTES, &tm.k, &bars->kv_full[st], it.q0 - i * TILE, it.bh_kv);
      load_tile(smem + DQ_OFF_V + st * TILE_BYTES, &tm.v, &bars->kv_full[st], it.q0 - i * TILE, it.bh_kv);
    }
    if (it.has_rla) {                                      // g_r in the V half of the slot, the state in the K half
      if (!ring_wait()) return false;
      const int st = kc & 1;
      mbar_arrive_expect_tx(&bars->kv_full[st], (it.has_state ? 2 : 1) * TILE_BYTES);
      load_tile(smem + DQ_OFF_V + st * TILE_BYTES, &tm.gr, &bars->kv_full[st], it.q0, it.bh_q);
      if (it.has_state) load_tile(smem + DQ_OFF_K + st * TILE_BYTES, &tm.st, &bars->kv_full[st], 0, it.st_index);
      ++kc;
    }
  }
  return true;
}

__device__ bool dq_mma(const BwdArgs& a, unsigned char* smem, DqBars* bars, uint32_t tmem, int n_items, int n_qt) {
  const uint32_t sG = smem_u32(smem + DQ_OFF_G), sK = smem_u32(smem + DQ_OFF_K), sV = smem_u32(smem + DQ_OFF_V);
  const uint32_t tS = tmem, tP = tmem + 128, tQ = tmem + 256, tF = tmem + 384;
  constexpr uint32_t idesc_ts = instr_desc(128, 128, 0, 1);
  int kc = 0, n = 0, cs = 0, cr = 0;                       // ring uses, items, score hand-overs, residual items
  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++n) {
    const DqItem it = dq_item(a, idx, n_qt);
    const uint32_t sQ = smem_u32(smem + ((n & 1) ? DQ_OFF_Q1 : DQ_OFF_Q));
    WAIT_OR_RETURN_W(bars->qg_full, n & 1);
    int last_st = 0;
    for (int i = 0; i < it.n_kt; ++i, ++kc, ++cs) {
      const int st = kc & 1;
      last_st = st;
      WAIT_OR_RETURN_W(bars->kv_full[st], (kc >> 1) & 1);
      tc_fence_after();
      mma_kk(tS, sQ, sK + st * TILE_BYTES, false);         // S  = Q K^T
      mma_kk(tP, sG, sV + st * TILE_BYTES, false);         // dP = g_s V^T
      mma_commit(&bars->s_full);
      WAIT_OR_RETURN_W(bars->ds_full, cs & 1);
      if (i == 0 && n >= 1) WAIT_OR_RETURN_W(bars->acc_free, (n - 1) & 1);   // the previous item's epilogue has read dQ
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 8; ++k)                          // dQ += dS K, dS read from TMEM
        mma_bf16_ts(tQ, tS + (k < 4 ? 8 * k : 64 + 8 * (k - 4)), mnmajor_desc(sK + st * TILE_BYTES, k), idesc_ts, (i > 0 || k > 0) ? 1u : 0u);
      // the last tile's K turns into phi(K) for the residual part: its slot is released there
      if (!(it.has_rla && i == it.n_kt - 1)) mma_commit(&bars->kv_free[st]);
      // the next tile's scores follow these products in the tensor pipe, which runs in issue order
    }
    if (it.has_rla) {
      const int xs = kc & 1;                               // slot of g_r and the stored state
      const uint32_t sG2 = sV + xs * TILE_BYTES, sSt = sK + xs * TILE_BYTES;
      mma_commit(&bars->o_done);                           // (interim) every window product done: K_cb may be rewritten
      WAIT_OR_RETURN_W(bars->kv_full[xs], (kc >> 1) & 1);
      tc_fence_after();
      mma_kk(tS, sG2, sV + last_st * TILE_BYTES, false);   // dA = g_r V_cb^T
      if (it.has_state) mma_kk(tF, sG2, sSt, false);       // g_r S_cb^T
      mma_commit(&bars->s_full);
      WAIT_OR_RETURN_W(bars->phik_ready, cr & 1);
      WAIT_OR_RETURN_W(bars->ds_full, cs & 1);
      tc_fence_after();
#pragma unroll
      for (int k = 0; k < 8; ++k)                          // (dA masked) phi(K_cb)
        mma_bf16_ts(tF, tS + (k < 4 ? 8 * k : 64 + 8 * (k - 4)), mnmajor_desc(sK + last_st * TILE_BYTES, k), idesc_ts, (it.has_state || k > 0) ? 1u : 0u);
      mma_commit(&bars->kv_free[last_st]);
      mma_commit(&bars->kv_free[xs]);
      ++kc; ++cs; ++cr;
    }
    mma_commit(&bars->o_done);
  }
  return true;
}

__device__ bool dq_rows(const DqMaps& tm, const BwdArgs& a, unsigned char* smem, DqBars* bars, uint32_t tmem, int g, int r,
                        int n_items, int n_qt) {
  const uint32_t lane_off = (uint32_t)((r & ~31) << 16);
  const uint32_t tS = tmem + lane_off, tP = tmem + 128 + lane_off, tQ = tmem + 256 + lane_off,
                 tF = tmem + 384 + lane_off;
  int kc = 0, n = 0, cs = 0, co = 0;                       // ring uses, items, score hand-overs, o_done completions
  bool store_pending = false;                              // this thread issued a dQ store whose read-out it has not confirmed
  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++n) {
    const DqItem it = dq_item(a, idx, n_qt);
    const int n_kt = it.n_kt;
    unsigned char* sQ = smem + ((n & 1) ? DQ_OFF_Q1 : DQ_OFF_Q);
    const int t = it.q0 + r;
    const bool live = t < a.T;
    const size_t row = (size_t)it.bh_q * a.T + t;
    const float l2 = live ? a.lse[row] * LOG2E : INFINITY;
    const float Drs = live ? a.delta[row] * a.scale : 0.f;

    for (int i = 0; i < n_kt; ++i, ++cs) {
      WAIT_OR_RETURN(bars->s_full, cs & 1);
      tc_fence_after();
      const bool diag = (i == 0), bound = it.has_boundary && (i == n_kt - 1);
#pragma unroll 1
      for (int c = 2 * g; c < 2 * g + 2; ++c) {                 // rolled: compact code
        float s[32], dp[32];
        tmem_ld32(tS + 32 * c, s);
        tmem_ld32(tP + 32 * c, dp);
        tmem_wait_ld();
        uint32_t pk[16];
        if (diag || bound) {                       // only the two edge tiles of the band need a mask
          const uint32_t keep = keep_bits(r, c, diag, bound);
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float p0 = ex2(s[e] * a.scale_log2 - l2), p1 = ex2(s[e + 1] * a.scale_log2 - l2);
            const float d0 = (keep >> e) & 1u ? p0 * (dp[e] * a.scale - Drs) : 0.f;
            const float d1 = (keep >> (e + 1)) & 1u ? p1 * (dp[e + 1] * a.scale - Drs) : 0.f;
            pk[e >> 1] = pack_bf16(d0, d1);
          }
        } else {
#pragma unroll
          for (int e = 0; e < 32; e += 2) {
            const float p0 = ex2(s[e] * a.scale_log2 - l2), p1 = ex2(s[e + 1] * a.scale_log2 - l2);
            pk[e >> 1] = pack_bf16(p0 * (dp[e] * a.scale - Drs), p1 * (dp[e + 1] * a.scale - Drs));
          }
        }
        // dS (bf16, two per column) overwrites this group's own S columns already consumed
        tmem_st16(tS + 64 * g + 16 * (c - 2 * g), pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->ds_full);
      if (i == 0 && store_pending) {                         // the previous item's dQ has left its Q buffer by now
        tma_store_wait_read();
        mbar_arrive(&bars->q_read);
        store_pending = false;
      }
    }
    kc += n_kt;

    if (it.has_rla) {
      const int last = (kc - 1) & 1;
      WAIT_OR_RETURN(bars->o_done, co & 1);                    // every window product done: K_cb is no longer read raw
      ++co;
      {
        const int t2 = g * 128 + r;                              // two threads per key row
        unsigned char* kh = smem + DQ_OFF_K + last * TILE_BYTES + (t2 & 1) * HALF_BYTES;
        feature_map_pair_any(kh, kh, t2 >> 1, a.phi);
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->phik_ready);
      WAIT_OR_RETURN(bars->s_full, cs & 1);
      tc_fence_after();
#pragma unroll 1
      for (int c = 2 * g; c < 2 * g + 2; ++c) {
        float x[32];
        tmem_ld32(tS + 32 * c, x);
        tmem_wait_ld();
        const uint32_t keep = bits_lt(r - 32 * c);               // residual keys of row r in this chunk: j < r
        uint32_t pk[16];
#pragma unroll
        for (int e = 0; e < 32; e += 2)
          pk[e >> 1] = pack_bf16((keep >> e) & 1u ? x[e] : 0.f, (keep >> (e + 1)) & 1u ? x[e + 1] : 0.f);
        tmem_st16(tS + 64 * g + 16 * (c - 2 * g), pk);
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->ds_full);
      ++cs;
      ++kc;
    }

    // ---- dq = dQ + phi(q) * (dphi_q - <dphi_q, phi(q)>) -----------------------------------
    const int co_final = co++;
    if (g != 0) continue;                                      // group 0 alone runs the epilogue
    WAIT_OR_RETURN(bars->o_done, co_final & 1);
    tc_fence_after();
    float m = 0.f, inv = 0.f, dot = 0.f;
    const bool soft = (a.phi == RATTN_PHI_SOFTMAX);
    if (it.has_rla && soft) {
      m = -INFINITY;
#pragma unroll
      for (int c = 0; c < 16; ++c) {
        const uint4 u = *reinterpret_cast<const uint4*>(sQ + swz(r, c));
        const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(h[e]);
          m = fmaxf(m, fmaxf(f.x, f.y));
        }
      }
      const float ml = m * LOG2E;
      float sum = 0.f, du = 0.f;
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float df[32];
        tmem_ld32(tF + 32 * c, df);
        tmem_wait_ld();
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const uint4 u = *reinterpret_cast<const uint4*>(sQ + swz(r, 4 * c + cc));
          const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            const float e0 = ex2(f.x * LOG2E - ml), e1 = ex2(f.y * LOG2E - ml);
            sum += e0 + e1;
            du += e0 * df[8 * cc + 2 * e] + e1 * df[8 * cc + 2 * e + 1];
          }
        }
      }
      inv = 1.f / sum;
      dot = du * inv;
      m = ml;
    }
    // every product has completed: this item's Q buffer stages the output, each thread
    // rewriting its own row in place, for one TMA store
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      float x[32], df[32];
      tmem_ld32(tQ + 32 * c, x);
      if (it.has_rla) tmem_ld32(tF + 32 * c, df);
      tmem_wait_ld();
      if (it.has_rla) {
#pragma unroll
        for (int cc = 0; cc < 4; ++cc) {
          const uint4 u = *reinterpret_cast<const uint4*>(sQ + swz(r, 4 * c + cc));
          const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 f = __bfloat1622float2(h[e]);
            if (soft) {
              const float e0 = ex2(f.x * LOG2E - m) * inv, e1 = ex2(f.y * LOG2E - m) * inv;
              x[8 * cc + 2 * e] += e0 * (df[8 * cc + 2 * e] - dot);
              x[8 * cc + 2 * e + 1] += e1 * (df[8 * cc + 2 * e + 1] - dot);
            } else {
              // element-wise maps: ReLU passes the gradient where q > 0, the identity everywhere
              const bool relu = (a.phi == RATTN_PHI_RELU);
              x[8 * cc + 2 * e] += (relu && !(f.x > 0.f)) ? 0.f : df[8 * cc + 2 * e];
              x[8 * cc + 2 * e + 1] += (relu && !(f.y > 0.f)) ? 0.f : df[8 * cc + 2 * e + 1];
            }
          }
        }
      }
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        uint4 u;
        u.x = pack_bf16(x[8 * e + 0], x[8 * e + 1]);
        u.y = pack_bf16(x[8 * e + 2], x[8 * e + 3]);
        u.z = pack_bf16(x[8 * e + 4], x[8 * e + 5]);
        u.w = pack_bf16(x[8 * e + 6], x[8 * e + 7]);
        *reinterpret_cast<uint4*>(sQ + swz(r, 4 * c + e)) = u;
      }
    }
    tc_fence_before();
    mbar_arrive(&bars->acc_free);          // the dQ / dphi_q columns have been read
    fence_proxy_async_smem();
    rows_sync();
    if (r == 0) {
      // nobody waits for the store to read the Q buffer out: the loader refills that buffer two items
      // on, after q_read, which this thread confirms once the next item's first key tile is behind it
      store_tile(&tm.dq, sQ, it.q0, it.bh_q);
      tma_store_commit();
      store_pending = true;
    }
  }
  if (store_pending) tma_store_wait();     // the last store has completed before the CTA may go
  return true;
}

__global__ void __launch_bounds__(DQ_THREADS, 1)
tc_bwd_dq_kernel(const __grid_constant__ DqMaps tm, BwdArgs a, int n_items, int n_qt) {
  extern __shared__ __align__(1024) unsigned char smem[];
  DqBars* bars = reinterpret_cast<DqBars*>(smem + DQ_OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0 && a.status) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    mbar_init(&bars->qg_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->kv_full[i], 1);
      mbar_init(&bars->kv_free[i], 1);
    }
    mbar_init(&bars->s_full, 1);
    mbar_init(&bars->ds_full, 256);
    mbar_init(&bars->phik_ready, 256);
    mbar_init(&bars->o_done, 1);
    mbar_init(&bars->acc_free, 128);
    mbar_init(&bars->q_read, 1);
    mbar_init(&bars->drain, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  if (tid == 288) {
    prefetch_map(&tm.q);
    prefetch_map(&tm.k);
    prefetch_map(&tm.v);
    prefetch_tensormap(&tm.gs);
    prefetch_tensormap(&tm.gr);
    prefetch_tensormap(&tm.st);
    prefetch_map(&tm.dq);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  bool ok = true;
  if (warp < 8) {
    ok = dq_rows(tm, a, smem, bars, tmem, warp >> 2, tid & 127, n_items, n_qt);
  } else if (warp == 8) {
    ok = dq_mma(a, smem, bars, tmem, n_items, n_qt);
    if (!ok) {
      mma_commit(&bars->drain);
      for (int it = 0; it < (1 << 16) && !mbar_try_wait(&bars->drain, 0); ++it) {}
    }
  } else {
    ok = dq_loader(tm, a, smem, bars, n_items, n_qt);
  }
  if (!ok && a.status) atomicExch(a.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// =============================================================================== dkv
// One CTA per (key tile j, K/V head).  K_j, V_j (and phi(K_j)) stay in shared memory, the dV
// and dK accumulators in TMEM.  The work is a list of items, one per (query head of the
// group, query half tile of 64 rows): first the residual-branch items (query tile j + wt),
// then the window items (query tiles j .. j + wt).  Two row groups of 128 threads (thread =
// key row = TMEM lane) take the items alternately, each with its own TMEM slot, so that one
// group's exponentials overlap the other group's products:
//   loader thread   TMA: K, V, [R_j], then per item Q_h, g_h and the query-side row statistics
//   MMA thread      per item: S^T = K Q_h^T and dP^T = V g_h^T into the slot (128 x 64 each);
//                   after the row group has overwritten them with bf16 P^T and dS^T:
//                   dV += P^T g_h, dK += dS^T Q_h with the A operand read from TMEM
//   row group       P^T = exp2(S^T * scale_log2 - lse2[q]), dS^T = P^T (dP^T scale - D[q] scale)
// The residual items run first and leave dphi_k in the dK accumulator; row group 0 then folds
// the feature-map Jacobian into it (dK := phi(k) (dphi_k - <dphi_k, phi(k)>)) and the window
// items accumulate on top.
constexpr int KV_NS = 3;                                   // item stages
constexpr int KV_OFF_K = 0;
constexpr int KV_OFF_V = 1 * TILE_BYTES;
constexpr int KV_OFF_KPHI = 2 * TILE_BYTES;                // phi(K_j); stages dK at the end of an item
constexpr int KV_OFF_OUT = 3 * TILE_BYTES;                 // stages dV at the end of an item
constexpr int KV_OFF_STAGE = 4 * TILE_BYTES;               // KV_NS x [Q_h 16 KB | g_h 16 KB]
constexpr int KV_OFF_STAT = KV_OFF_STAGE + KV_NS * TILE_BYTES;   // KV_NS x (lse2[64], D*scale[64]) fp32
constexpr int KV_OFF_BAR = KV_OFF_STAT + KV_NS * 512;
constexpr int KV_SMEM = KV_OFF_BAR + 256;
constexpr int KV_THREADS = 352;                            // 2 row groups, score warp, loader warp, accumulate warp

struct KvBars {
  uint64_t kv_full, kphi_ready, full[KV_NS], acc_done[KV_NS], s_full[2], p_ready[2], phiq_ready[2],
      r_acc_done, fold_done, all_done, acc_free, out_read, drain, drain2;
  uint32_t tmem_base;
  int abort;
};

struct KvMaps {
  UMap k, v, qh, dk, dv;        // the caller's tensors (either head layout)
  CUtensorMap rs, gsh, grh;
};

// One key tile (j, K/V head) of the persistent CTA's work list, and how its half-tile items
// are numbered.  Counters that run on across key tiles (ring slots, TMEM slots, barrier
// phases) are kept by every role in the same way.
struct KvPlan {
  int j, bh_kv, rs_index, n_qt, wt, group, n_R, n_s_tiles, N;
  bool windowed, has_inter;
  __device__ bool is_r(int n) const { return n < n_R; }
  __device__ int head(int n) const { return n < n_R ? (n >> 1) : (n - n_R) / (2 * n_s_tiles); }
  __device__ int qtile(int n) const { return n < n_R ? j + wt : j + (((n - n_R) % (2 * n_s_tiles)) >> 1); }
  __device__ int half(int n) const { return n < n_R ? (n & 1) : ((n - n_R) & 1); }
};

__device__ __forceinline__ KvPlan kv_plan(const BwdArgs& a, int idx) {
  KvPlan pl;
  pl.n_qt = (a.T + TILE - 1) / TILE;
  pl.bh_kv = idx / pl.n_qt;
  pl.j = idx % pl.n_qt;
  pl.rs_index = pl.bh_kv * a.n_chunks + pl.j;
  pl.wt = a.w / TILE;
  pl.group = a.group;
  pl.windowed = (a.mode != RATTN_MODE_FULL_CAUSAL);
  const int i_hi = (pl.windowed && pl.j + pl.wt < pl.n_qt - 1) ? pl.j + pl.wt : pl.n_qt - 1;
  pl.n_s_tiles = i_hi - pl.j + 1;
  const bool r_tile = pl.windowed && (a.mode == RATTN_MODE_RATTN) && (pl.j + pl.wt <= pl.n_qt - 1);
  pl.n_R = r_tile ? 2 * a.group : 0;
  pl.has_inter = r_tile && (pl.j + pl.wt + 1 <= pl.n_qt - 1);
  pl.N = pl.n_R + 2 * a.group * pl.n_s_tiles;
  return pl;
}

// running counters shared by the three roles: key tiles done, ring slots used, half-tile items
// done, key tiles with residual items done
struct KvCount {
  int it, seq, gi, cr;
};

__device__ bool kv_loader(const KvMaps& tm, const BwdArgs& a, unsigned char* smem, KvBars* bars, int n_items) {
  KvCount c = {0, 0, 0, 0};
  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++c.it) {
    const KvPlan pl = kv_plan(a, idx);
    const int j0 = pl.j * TILE;
    // K_j, V_j replace the previous key tile's once every product that read them has completed
    if (c.it >= 1) WAIT_OR_RETURN_W(bars->all_done, (c.it - 1) & 1);
    mbar_arrive_expect_tx(&bars->kv_full, 2 * TILE_BYTES);
    load_tile(smem + KV_OFF_K, &tm.k, &bars->kv_full, j0, pl.bh_kv);
    load_tile(smem + KV_OFF_V, &tm.v, &bars->kv_full, j0, pl.bh_kv);
    // dK of the previous key tile left through the ring slot this tile uses third: its store must
    // have read the slot out first
    const int gate_seq = c.seq + 2;
    auto ring = [&](int& st) -> bool {                     // next ring slot, once its previous user is consumed
      st = c.seq % KV_NS;
      const int use = c.seq / KV_NS;
      if (use >= 1) WAIT_OR_RETURN_W(bars->acc_done[st], (use - 1) & 1);
      if (c.it >= 1 && c.seq == gate_seq) WAIT_OR_RETURN_W(bars->out_read, (c.it - 1) & 1);
      ++c.seq;
      return true;
    };
    if (pl.has_inter) {
      int st;
      if (!ring(st)) return false;
      mbar_arrive_expect_tx(&bars->full[st], TILE_BYTES);
      load_tile(smem + KV_OFF_STAGE + st * TILE_BYTES, &tm.rs, &bars->full[st], 0, pl.rs_index);
    }
    for (int n = 0; n < pl.N; ++n) {
      int st;
      if (!ring(st)) return false;
      unsigned char* dst = smem + KV_OFF_STAGE + st * TILE_BYTES;
      const int z = pl.bh_kv * pl.group + pl.head(n);
      const int row = pl.qtile(n) * TILE + 64 * pl.half(n);
      if (pl.is_r(n)) {
        mbar_arrive_expect_tx(&bars->full[st], 2 * HT_BYTES);
        load_half_tile(dst, &tm.qh, &bars->full[st], row, z);
        load_half_tile(dst + HT_BYTES, &tm.grh, &bars->full[st], row, z);
      } else {
        mbar_arrive_expect_tx(&bars->full[st], 2 * HT_BYTES + 512);
        load_half_tile(dst, &tm.qh, &bars->full[st], row, z);
        load_half_tile(dst + HT_BYTES, &tm.gsh, &bars->full[st], row, z);
        float* stat = reinterpret_cast<float*>(smem + KV_OFF_STAT + st * 512);
        bulk_load_1d(stat, a.lse2p + (size_t)z * a.t_pad + row, 256, &bars->full[st]);
        bulk_load_1d(stat + 64, a.dscp + (size_t)z * a.t_pad + row, 256, &bars->full[st]);
      }
    }
  }
  return true;
}

// The products are issued by two warps: the score warp issues S^T and dP^T of every item, the accumulate
// warp everything that writes the dV / dK accumulators, so that the waits of one (a wait that is already
// satisfied still costs an issuing warp some 300 cycles) pass under the products of the other.  A third
// issuer (S^T and dP^T apart) measured no faster: what then limits an item is the chain scores -> row
// group -> accumulate on its TMEM slot, of which there are two.  Order between the two warps:
//   scores(n) -> row group -> p_ready -> accumulate(n)        (existing barriers)
//   accumulate(n - 2) complete -> scores(n) may overwrite the TMEM slot they share   (acc_done of n - 2's stage)
__device__ bool kv_mma_scores(const BwdArgs& a, unsigned char* smem, KvBars* bars, uint32_t tmem, int n_items) {
  const uint32_t sK = smem_u32(smem + KV_OFF_K), sV = smem_u32(smem + KV_OFF_V), sKphi = smem_u32(smem + KV_OFF_KPHI);
  const uint32_t sStage = smem_u32(smem + KV_OFF_STAGE);
  // slot s: [S^T | dP^T] at columns 256 + 128 s and 320 + 128 s (computed, not looked up: an array
  // indexed by the slot would live in local memory)
  const uint32_t tS0 = tmem + 256, tP0 = tmem + 320;
  KvCount c = {0, 0, 0, 0};
  int cq0 = 0, cq1 = 0;                                    // phi(Q_h) hand-overs per TMEM slot

  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++c.it) {
    const KvPlan pl = kv_plan(a, idx);
    // K_j, V_j have landed (which also means every product of the previous key tile has completed)
    WAIT_OR_RETURN_W(bars->kv_full, c.it & 1);
    if (pl.n_R > 0) WAIT_OR_RETURN_W(bars->kphi_ready, c.cr & 1);
    if (pl.has_inter) ++c.seq;                             // the reverse state's ring slot (accumulate warp)
    const int seq0 = c.seq, gi0 = c.gi;
    for (int n = 0; n < pl.N; ++n) {
      const int st = (seq0 + n) % KV_NS, use = (seq0 + n) / KV_NS, slot = (gi0 + n) & 1;
      const uint32_t sQh = sStage + st * TILE_BYTES, sGh = sQh + HT_BYTES;
      WAIT_OR_RETURN_W(bars->full[st], use & 1);
      if (pl.is_r(n)) {
        WAIT_OR_RETURN_W(bars->phiq_ready[slot], (slot ? cq1 : cq0) & 1);
        if (slot) ++cq1; else ++cq0;
      }
      if (n >= 2) {                                        // the slot's previous item has been accumulated
        const int st2 = (seq0 + n - 2) % KV_NS, use2 = (seq0 + n - 2) / KV_NS;
        WAIT_OR_RETURN_W(bars->acc_done[st2], use2 & 1);
      }
      tc_fence_after();
      mma_k_kh(tS0 + 128 * slot, pl.is_r(n) ? sKphi : sK, sQh);   // S^T  = K Q_h^T   (phi(K) phi(Q_h)^T)
      mma_k_kh(tP0 + 128 * slot, sV, sGh);                         // dP^T = V g_h^T
      mma_commit(&bars->s_full[slot]);
    }
    c.seq += pl.N;
    c.gi += pl.N;
    if (pl.n_R > 0) ++c.cr;
  }
  return true;
}

__device__ bool kv_mma_accum(const BwdArgs& a, unsigned char* smem, KvBars* bars, uint32_t tmem, int n_items) {
  const uint32_t sV = smem_u32(smem + KV_OFF_V), sKphi = smem_u32(smem + KV_OFF_KPHI);
  const uint32_t sStage = smem_u32(smem + KV_OFF_STAGE);
  const uint32_t tV = tmem, tK = tmem + 128;
  const uint32_t tS0 = tmem + 256, tP0 = tmem + 320;
  KvCount c = {0, 0, 0, 0};

  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x, ++c.it) {
    const KvPlan pl = kv_plan(a, idx);
    bool accV = false, accK = false;
    // the previous key tile's epilogue has read the two accumulators
    bool acc_ok = (c.it == 0);
    if (pl.has_inter) {
      const int st = c.seq % KV_NS, use = c.seq / KV_NS;
      ++c.seq;
      WAIT_OR_RETURN_W(bars->kv_full, c.it & 1);
      WAIT_OR_RETURN_W(bars->kphi_ready, c.cr & 1);
      WAIT_OR_RETURN_W(bars->full[st], use & 1);
      if (!acc_ok) { WAIT_OR_RETURN_W(bars->acc_free, (c.it - 1) & 1); acc_ok = true; }
      tc_fence_after();
      mma_kk(tK, sV, sStage + st * TILE_BYTES, false);     // dphi_k = V_j R_j^T
      mma_kmn<1>(tV, sKphi, sStage + st * TILE_BYTES, false);   // dV     = phi(K_j) R_j
      mma_commit(&bars->acc_done[st]);
      accV = accK = true;
    }
    const int seq0 = c.seq, gi0 = c.gi;
    for (int m = 0; m < pl.N; ++m) {
      const int st = (seq0 + m) % KV_NS, slot = (gi0 + m) & 1;
      const uint32_t sQh = sStage + st * TILE_BYTES, sGh = sQh + HT_BYTES;
      WAIT_OR_RETURN_W(bars->p_ready[slot], ((gi0 + m) >> 1) & 1);
      if (m == pl.n_R && pl.n_R > 0) WAIT_OR_RETURN_W(bars->fold_done, c.cr & 1);
      if (!acc_ok) { WAIT_OR_RETURN_W(bars->acc_free, (c.it - 1) & 1); acc_ok = true; }
      tc_fence_after();
      mma_ts_h(tV, tS0 + 128 * slot, sGh, accV);           // dV += P^T g_h
      mma_ts_h(tK, tP0 + 128 * slot, sQh, accK);           // dK += dS^T Q_h   (dphi_k += dA^T phi(Q_h))
      accV = accK = true;
      mma_commit(&bars->acc_done[st]);
      if (m == pl.n_R - 1) mma_commit(&bars->r_acc_done);
    }
    c.seq += pl.N;
    c.gi += pl.N;
    if (pl.n_R > 0) ++c.cr;
    mma_commit(&bars->all_done);
  }
  return true;
}

__device__ bool kv_rows(const KvMaps& tm, const BwdArgs& a, unsigned char* smem, KvBars* bars, uint32_t tmem, int gg,
                        int r, int n_items) {
  // two groups of 128 threads (thread = key row = TMEM lane), one per TMEM slot; a thread takes
  // all 64 query columns of its item, 32 at a time (more row groups per slot measured no faster
  // and cost registers)
  const int g = gg;
  const uint32_t lane_off = (uint32_t)((r & ~31) << 16);
  const uint32_t tV = tmem + lane_off, tK = tmem + 128 + lane_off;
  const uint32_t tS = tmem + 256 + 128 * g + lane_off, tP = tS + 64;
  const unsigned char* sKphi = smem + KV_OFF_KPHI;
  KvCount cnt = {0, 0, 0, 0};

  for (int idx = blockIdx.x; idx < n_items; idx += gridDim.x) {
  const KvPlan pl = kv_plan(a, idx);
  const int bh_kv = pl.bh_kv;
  if (gg < 2) {
    WAIT_OR_RETURN(bars->kv_full, cnt.it & 1);
    if (pl.n_R > 0) {
      // phi(K_j) into its own tile: 256 threads, two per row
      const int t2 = gg * 128 + r, row = t2 >> 1, hf = t2 & 1;
      feature_map_pair_any(smem + KV_OFF_K + hf * HALF_BYTES, smem + KV_OFF_KPHI + hf * HALF_BYTES, row, a.phi);
      fence_proxy_async_smem();
      mbar_arrive(&bars->kphi_ready);
    }
    // the previous key tile's dK has long left its ring slot by now: tell the loader
    if (gg == 0 && r == 0 && cnt.it >= 1) {
      tma_store_wait_read();
      mbar_arrive(&bars->out_read);
    }
  }
  const int seq0 = cnt.seq + (pl.has_inter ? 1 : 0), gi0 = cnt.gi;

  for (int n = 0; n < pl.N; ++n) {
    if (((gi0 + n) & 1) != g) continue;                       // the other TMEM slot's item
    const int st = (seq0 + n) % KV_NS, use = (seq0 + n) / KV_NS;
    const bool is_r = pl.is_r(n);
    const int i = pl.qtile(n), hf = pl.half(n);
    unsigned char* sQh = smem + KV_OFF_STAGE + st * TILE_BYTES;
    WAIT_OR_RETURN(bars->full[st], use & 1);
    if (is_r) {
      // phi(Q_h) in place: 64 rows, two threads per row
      const int row = r >> 1, ch = r & 1;
      feature_map_pair_any(sQh + ch * HT_HALF, sQh + ch * HT_HALF, row, a.phi);
      fence_proxy_async_smem();
      mbar_arrive(&bars->phiq_ready[g]);
    }
    WAIT_OR_RETURN(bars->s_full[g], ((gi0 + n) >> 1) & 1);
    tc_fence_after();
    const bool diag = !is_r && (i == pl.j), bound = !is_r && pl.windowed && (i == pl.j + pl.wt);
    const float* l2 = reinterpret_cast<const float*>(smem + KV_OFF_STAT + st * 512);
    const float* Ds = l2 + 64;
#pragma unroll 1
    for (int c = 0; c < 2; ++c) {                              // rolled: compact code
      float s[32], dp[32];
      tmem_ld32(tS + 32 * c, s);
      tmem_ld32(tP + 32 * c, dp);
      tmem_wait_ld();
      const int rd = r - (64 * hf + 32 * c);                   // key row relative to this chunk's first query
      uint32_t pk1[16], pk2[16];
      if (is_r) {
        const uint32_t keep = bits_gt(rd);                     // keep key r < query q
#pragma unroll
        for (int e = 0; e < 32; e += 2) {
          const bool k0 = (keep >> e) & 1u, k1 = (keep >> (e + 1)) & 1u;
          pk1[e >> 1] = pack_bf16(k0 ? s[e] : 0.f, k1 ? s[e + 1] : 0.f);
          pk2[e >> 1] = pack_bf16(k0 ? dp[e] : 0.f, k1 ? dp[e + 1] : 0.f);
        }
      } else {
        // diagonal tile: queries q >= r; oldest tile of the band: queries q <= r
        const uint32_t keep = (diag ? bits_ge(rd) : 0xffffffffu) & (bound ? bits_le(rd) : 0xffffffffu);
        if (!diag && !bound) {                     // interior tiles of the band: no mask
#pragma unroll
          for (int e4 = 0; e4 < 32; e4 += 4) {
            const float4 lv = *reinterpret_cast<const float4*>(l2 + 32 * c + e4);
            const float4 dv = *reinterpret_cast<const float4*>(Ds + 32 * c + e4);
            const float lq[4] = {lv.x, lv.y, lv.z, lv.w}, dq4[4] = {dv.x, dv.y, dv.z, dv.w};
            float p[4], d[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
              p[u] = ex2(s[e4 + u] * a.scale_log2 - lq[u]);
              d[u] = p[u] * (dp[e4 + u] * a.scale - dq4[u]);
            }
            pk1[e4 >> 1] = pack_bf16(p[0], p[1]);
            pk1[(e4 >> 1) + 1] = pack_bf16(p[2], p[3]);
            pk2[e4 >> 1] = pack_bf16(d[0], d[1]);
            pk2[(e4 >> 1) + 1] = pack_bf16(d[2], d[3]);
          }
        } else
#pragma unroll
        for (int e4 = 0; e4 < 32; e4 += 4) {
          const float4 lv = *reinterpret_cast<const float4*>(l2 + 32 * c + e4);
          const float4 dv = *reinterpret_cast<const float4*>(Ds + 32 * c + e4);
          const float lq[4] = {lv.x, lv.y, lv.z, lv.w}, dq4[4] = {dv.x, dv.y, dv.z, dv.w};
          float p[4], d[4];
#pragma unroll
          for (int u = 0; u < 4; ++u) {
            const bool ok = (keep >> (e4 + u)) & 1u;
            const float pv = ex2(s[e4 + u] * a.scale_log2 - lq[u]);
            p[u] = ok ? pv : 0.f;
            d[u] = ok ? pv * (dp[e4 + u] * a.scale - dq4[u]) : 0.f;
          }
          pk1[e4 >> 1] = pack_bf16(p[0], p[1]);
          pk1[(e4 >> 1) + 1] = pack_bf16(p[2], p[3]);
          pk2[e4 >> 1] = pack_bf16(d[0], d[1]);
          pk2[(e4 >> 1) + 1] = pack_bf16(d[2], d[3]);
        }
      }
      // bf16 results (two per column) overwrite the first half of the chunk just consumed
      tmem_st16(tS + 32 * c, pk1);
      tmem_st16(tP + 32 * c, pk2);
    }
    tmem_wait_st();
    tc_fence_before();
    mbar_arrive(&bars->p_ready[g]);

    if (gg == 0 && is_r && n + 2 >= pl.n_R) {                   // group 0's last residual item of this key tile
      // end of the residual items: dK := dphi_k through the feature map's gradient
      // (softmax map: phi(k) (dphi_k - <dphi_k, phi(k)>))
      WAIT_OR_RETURN(bars->r_acc_done, cnt.cr & 1);
      tc_fence_after();
      const bool soft = (a.phi == RATTN_PHI_SOFTMAX);
      float dot = 0.f;
      if (soft) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float df[32];
          tmem_ld32(tK + 32 * c, df);
          tmem_wait_ld();
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            const uint4 u = *reinterpret_cast<const uint4*>(sKphi + swz(r, 4 * c + cc));
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 f = __bfloat1622float2(h2[e]);
              dot += f.x * df[8 * cc + 2 * e] + f.y * df[8 * cc + 2 * e + 1];
            }
          }
        }
      }
      // the identity map leaves dphi_k as it is
      if (a.phi != RATTN_PHI_IDENTITY) {
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float df[32];
          tmem_ld32(tK + 32 * c, df);
          tmem_wait_ld();
#pragma unroll
          for (int cc = 0; cc < 4; ++cc) {
            const uint4 u = *reinterpret_cast<const uint4*>(sKphi + swz(r, 4 * c + cc));
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const float2 f = __bfloat1622float2(h2[e]);
              if (soft) {
                df[8 * cc + 2 * e] = f.x * (df[8 * cc + 2 * e] - dot);
                df[8 * cc + 2 * e + 1] = f.y * (df[8 * cc + 2 * e + 1] - dot);
              } else {                                   // ReLU: relu(k) > 0 exactly where k > 0
                df[8 * cc + 2 * e] = f.x > 0.f ? df[8 * cc + 2 * e] : 0.f;
                df[8 * cc + 2 * e + 1] = f.y > 0.f ? df[8 * cc + 2 * e + 1] : 0.f;
              }
            }
          }
          tmem_st32(tK + 32 * c, df);
        }
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(&bars->fold_done);
    }
  }

  // every product has completed: group 1 stores dV, staged in its own tile; group 0 stores dK, staged
  // in the ring slot that the next key tile uses third (its last user was this tile's last item), so
  // that nobody has to wait for a store to read its source out: phi(K) of the next tile goes to its
  // own tile at once, and the loader waits for out_read before it refills that slot
  if (gg < 2) {
    WAIT_OR_RETURN(bars->all_done, cnt.it & 1);
    tc_fence_after();
    if (gg == 1 && r == 0) tma_store_wait_read();            // the previous dV has left the staging tile
    if (gg == 1) group_sync(1);
    unsigned char* sOut = gg == 0 ? smem + KV_OFF_STAGE + ((seq0 + pl.N + 2) % KV_NS) * TILE_BYTES : smem + KV_OFF_OUT;
    const uint32_t tOut = gg == 0 ? tK : tV;
#pragma unroll 1
    for (int cc = 0; cc < 4; cc += 2) {                        // two loads in flight
      float x[2][32];
      tmem_ld32(tOut + 32 * cc, x[0]);
      tmem_ld32(tOut + 32 * (cc + 1), x[1]);
      tmem_wait_ld();
#pragma unroll
      for (int h2 = 0; h2 < 2; ++h2)
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          uint4 u;
          u.x = pack_bf16(x[h2][8 * e + 0], x[h2][8 * e + 1]);
          u.y = pack_bf16(x[h2][8 * e + 2], x[h2][8 * e + 3]);
          u.z = pack_bf16(x[h2][8 * e + 4], x[h2][8 * e + 5]);
          u.w = pack_bf16(x[h2][8 * e + 6], x[h2][8 * e + 7]);
          *reinterpret_cast<uint4*>(sOut + swz(r, 4 * (cc + h2) + e)) = u;
        }
    }
    tc_fence_before();
    mbar_arrive(&bars->acc_free);                              // the accumulators have been read
    fence_proxy_async_smem();
    group_sync(gg);
    if (r == 0) {
      store_tile(gg == 0 ? &tm.dk : &tm.dv, sOut, pl.j * TILE, bh_kv);
      tma_store_commit();
    }
  }
  cnt.seq = seq0 + pl.N;
  cnt.gi += pl.N;
  if (pl.n_R > 0) ++cnt.cr;
  ++cnt.it;
  }
  if (r == 0) tma_store_wait();                               // this thread's last store has completed
  return true;
}

__global__ void __launch_bounds__(KV_THREADS, 1)
tc_bwd_dkv_kernel(const __grid_constant__ KvMaps tm, BwdArgs a, int n_items) {
  extern __shared__ __align__(1024) unsigned char smem[];
  KvBars* bars = reinterpret_cast<KvBars*>(smem + KV_OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0 && a.status) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    mbar_init(&bars->kv_full, 1);
    mbar_init(&bars->kphi_ready, 256);
    for (int i = 0; i < KV_NS; ++i) {
      mbar_init(&bars->full[i], 1);
      mbar_init(&bars->acc_done[i], 1);
    }
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_ready[i], 128);
      mbar_init(&bars->phiq_ready[i], 128);
    }
    mbar_init(&bars->r_acc_done, 1);
    mbar_init(&bars->fold_done, 128);
    mbar_init(&bars->all_done, 1);
    mbar_init(&bars->acc_free, 256);
    mbar_init(&bars->out_read, 1);
    mbar_init(&bars->drain, 1);
    mbar_init(&bars->drain2, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
  }
  if (tid == 288) {
    prefetch_map(&tm.k);
    prefetch_map(&tm.v);
    prefetch_tensormap(&tm.rs);
    prefetch_map(&tm.qh);
    prefetch_tensormap(&tm.gsh);
    prefetch_tensormap(&tm.grh);
    prefetch_map(&tm.dk);
    prefetch_map(&tm.dv);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  bool ok = true;
  if (warp < 8) {
    ok = kv_rows(tm, a, smem, bars, tmem, warp >> 2, tid & 127, n_items);
  } else if (warp == 8 || warp == 10) {
    ok = warp == 8 ? kv_mma_scores(a, smem, bars, tmem, n_items) : kv_mma_accum(a, smem, bars, tmem, n_items);
    if (!ok) {                                             // let this warp's products in flight finish
      uint64_t* drain = warp == 8 ? &bars->drain : &bars->drain2;
      mma_commit(drain);
      for (int it = 0; it < (1 << 16) && !mbar_try_wait(drain, 0); ++it) {}
    }
  } else if (warp == 9) {
    ok = kv_loader(tm, a, smem, bars, n_items);
  }
  if (!ok && a.status) atomicExch(a.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

}  // namespace

cudaError_t launch_tc_backward(const Args& a, cudaStream_t s) {
  __nv_bfloat16* g_s = reinterpret_cast<__nv_bfloat16*>(a.do_swa);
  __nv_bfloat16* g_r = reinterpret_cast<__nv_bfloat16*>(a.do_rla);
  const bool rla_on = (a.mode == RATTN_MODE_RATTN);
  const int n_qt = (a.T + TILE - 1) / TILE;
  const int wt = a.w / TILE;
  cudaError_t e;
  if (a.dgamma_swa) {
    e = cudaMemsetAsync(a.dgamma_swa, 0, sizeof(float) * a.H_q * 128, s);
    if (e != cudaSuccess) return e;
  }
  if (a.dgamma_rla) {
    e = cudaMemsetAsync(a.dgamma_rla, 0, sizeof(float) * a.H_q * 128, s);
    if (e != cudaSuccess) return e;
  }
  const int t_pad = a.n_chunks * TILE;
  {
    PrepArgs pa;
    pa.o_s = reinterpret_cast<const __nv_bfloat16*>(a.o_swa);
    pa.o_r = reinterpret_cast<const __nv_bfloat16*>(a.o_rla);
    pa.gamma_s = a.gamma_swa; pa.gamma_r = a.gamma_rla;
    pa.g_s = g_s; pa.g_r = g_r;
    pa.delta = a.delta; pa.dgamma_s = a.dgamma_swa; pa.dgamma_r = a.dgamma_rla;
    pa.lse = a.lse; pa.lse2p = a.lse2p; pa.dscp = a.dscp;
    pa.status = a.status;
    pa.n_heads = a.B * a.H_q; pa.T = a.T; pa.t_pad = t_pad; pa.H_q = a.H_q; pa.rla_on = rla_on ? 1 : 0;
    pa.eps = a.eps; pa.scale = a.scale;
    int dev = 0, n_sm = 0;
    e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tc_bwd_prep_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, PREP_SMEM);
    if (e != cudaSuccess) return e;
    const long long n_chunks_all = (long long)pa.n_heads * (t_pad / PREP_ROWS);
    const int grid = (int)(n_chunks_all < 2ll * n_sm ? n_chunks_all : 2ll * n_sm);
    CUtensorMap dy_map;
    if (!make_row_map(&dy_map, a.dout, a.T, a.H_q, a.B, a.layout, PREP_ROWS)) return cudaErrorInvalidValue;
    KernelTimer kt("tc_bwd_prep", s);
    tc_bwd_prep_kernel<<<grid, PREP_THREADS, PREP_SMEM, s>>>(pa, dy_map);
  }
  count_launches(1);

  UMap tm_q, tm_k, tm_v, tm_dq, tm_dk, tm_dv;
  CUtensorMap tm_gs, tm_gr, tm_st, tm_rs;
  const uint64_t nq = (uint64_t)a.B * a.H_q, nkv = (uint64_t)a.B * a.H_kv;
  if (!make_user_map(&tm_q, a.q, a.T, a.H_q, a.B, a.layout) || !make_user_map(&tm_k, a.k, a.T, a.H_kv, a.B, a.layout) ||
      !make_user_map(&tm_v, a.v, a.T, a.H_kv, a.B, a.layout) ||
      !make_map(&tm_gs, g_s, a.T, nq) || !make_map(&tm_gr, g_r, a.T, nq) ||
      !make_user_map(&tm_dq, a.dq, a.T, a.H_q, a.B, a.layout) || !make_user_map(&tm_dk, a.dk, a.T, a.H_kv, a.B, a.layout) ||
      !make_user_map(&tm_dv, a.dv, a.T, a.H_kv, a.B, a.layout) ||
      !make_state_map(&tm_st, a.chunk_state, a.k, nkv * a.n_chunks) || !make_state_map(&tm_rs, a.rstate, a.k, nkv * a.n_chunks))
    return cudaErrorInvalidValue;

  // reverse states of the residual branch: chunks c with a query tile beyond c + wt
  const int n_r = rla_on && a.mode != RATTN_MODE_FULL_CAUSAL ? n_qt - wt - 1 : 0;
  // R_c for c = 0 .. n_r-1: walk the query tiles from the last one down to wt+1
  {
    StateLaunch L;
    L.ready = nullptr;
    L.x = a.q; L.y = g_r; L.out = a.rstate;
    L.x_heads = a.H_q; L.x_layout = a.layout; L.y_heads = 0; L.y_layout = 0;
    L.T = a.T; L.n_kv = (int)nkv; L.group = a.group; L.n_chunks = a.n_chunks;
    L.n_steps = n_r; L.first = n_qt - 1; L.dir = -1; L.out_first = n_qt - wt - 2;
    L.store_every = 1; L.store_phase = 0; L.handoff = 0; L.w = a.w; L.final_out = nullptr;
    L.state_in = nullptr; L.seq_lens = nullptr; L.kv_per_batch = 1;
    L.phi = a.phi;
    L.status = a.status; L.name = "tc_state_bwd";
    e = launch_tc_states(L, s);
  }
  if (e != cudaSuccess) return e;

  BwdArgs t;
  t.dq = reinterpret_cast<__nv_bfloat16*>(a.dq);
  t.dk = reinterpret_cast<__nv_bfloat16*>(a.dk);
  t.dv = reinterpret_cast<__nv_bfloat16*>(a.dv);
  t.lse = a.lse; t.delta = a.delta; t.status = a.status;
  t.lse2p = a.lse2p; t.dscp = a.dscp; t.t_pad = t_pad;
  t.T = a.T; t.w = a.w; t.H_q = a.H_q; t.group = a.group; t.mode = a.mode; t.n_chunks = a.n_chunks;
  t.scale = a.scale; t.scale_log2 = a.scale * LOG2E;
  t.phi = a.phi;
  e = cudaFuncSetAttribute(tc_bwd_dq_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, DQ_SMEM);
  if (e != cudaSuccess) return e;
  e = cudaFuncSetAttribute(tc_bwd_dkv_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, KV_SMEM);
  if (e != cudaSuccess) return e;
  {
    DqMaps dm;
    dm.q = tm_q; dm.k = tm_k; dm.v = tm_v; dm.gs = tm_gs; dm.gr = tm_gr; dm.st = tm_st; dm.dq = tm_dq;
    int dev = 0, n_sm = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int n_items = n_qt * (int)nq;
    KernelTimer kt("tc_bwd_dq", s);
    tc_bwd_dq_kernel<<<n_items < n_sm ? n_items : n_sm, DQ_THREADS, DQ_SMEM, s>>>(dm, t, n_items, n_qt);
  }
  KvMaps km;
  km.k = tm_k; km.v = tm_v; km.rs = tm_rs; km.dk = tm_dk; km.dv = tm_dv;
  if (!make_user_map(&km.qh, a.q, a.T, a.H_q, a.B, a.layout, 64) || !make_map(&km.gsh, g_s, a.T, nq, 64) ||
      !make_map(&km.grh, g_r, a.T, nq, 64))
    return cudaErrorInvalidValue;
  {
    int dev = 0, n_sm = 0;
    e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
    if (e != cudaSuccess) return e;
    const int n_items = n_qt * (int)nkv;
    KernelTimer kt("tc_bwd_dkv", s);
    tc_bwd_dkv_kernel<<<n_items < n_sm ? n_items : n_sm, KV_THREADS, KV_SMEM, s>>>(km, t, n_items);
  }
  count_launches(2);
  return cudaGetLastError();
}

}  // namespace rattn
