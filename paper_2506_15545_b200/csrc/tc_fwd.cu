// Tensor-core forward for bf16, d = 128, window a multiple of 128 (sm_100a: TMA + tcgen05 + TMEM).
//
// Per query tile of 128 rows (one CTA) the work is, with key tiles of 128 and chunk C = 128:
//   SWA (Section 2.1): for the w/128 + 1 key tiles of the band, S = Q K^T (tcgen05.mma into
//       TMEM), online softmax by one thread per row straight out of TMEM, P (fp16) staged in
//       shared memory, O_swa += P V (tcgen05.mma, accumulator resident in TMEM).  The
//       diagonal tile keeps j <= t, the oldest tile of the band keeps j >= t - w.
//   RLA (Eq. 4 in the chunkwise form of Eq. 2-3 with the window lag): the oldest tile of the
//       band is also the chunk the residual branch reads in its "intra" form,
//           O_rla = phi(Q) S_[c] + ((phi(Q) phi(K_c)^T) masked to j < t - w) V_c,
//       where S_[c] = sum over the chunks before c of phi(K)^T V.  phi (softmax over the head
//       features, Section 3.1) is applied to the Q and K tiles in shared memory, in place, so
//       it never goes to HBM (the paper's fused feature map).
//   Precision of the two weight matrices: P and the masked phi(Q) phi(K)^T are rounded to
//       fp16 (11-bit significand), not bf16 -- the branch outputs are small sums of
//       independent value rows that the RMS norm rescales to unit size, so the weights'
//       rounding error passes straight into y; with bf16 weights it alone is as large as the
//       final bf16 rounding of y.  tcgen05.mma needs A and B of one type, so a helper warp
//       group re-encodes each V tile from bf16 to fp16 in shared memory (exact for
//       2^-14 <= |v| <= 65504; larger magnitudes saturate).
//   Section 3.2: both accumulators are read from TMEM once, normalised by their RMS, scaled
//       by the per-head gains and summed.
// The chunk states S_[c] come from two small kernels that run first: per-chunk phi(K)^T V on
// the tensor cores, then an exclusive prefix over the chunks of each K/V head (the paper's
// stored chunk states, here stored for every chunk and in bf16, the MMA operand type).
#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

// ---------------------------------------------------------------- shared-memory map
constexpr int OFF_Q = 0;
constexpr int OFF_K = OFF_Q + TILE_BYTES;          // 2 stages
constexpr int OFF_V = OFF_K + 2 * TILE_BYTES;      // 2 stages
constexpr int OFF_P = OFF_V + 2 * TILE_BYTES;
constexpr int OFF_ST = OFF_P + TILE_BYTES;
constexpr int OFF_BAR = OFF_ST + TILE_BYTES;
constexpr int FWD_SMEM = OFF_BAR + 256 + 1024;     // + slack to align the base to 1024

struct FwdBars {
  uint64_t q_full, st_full, k_full[2], v_full[2], v_ready[2], s_full[2], s_empty[2], p_full, pv_done,
      phi_ready, o_done, drain;
  uint32_t tmem_base;
  int abort;
};

struct TcArgs {
  __nv_bfloat16* out;
  float* lse;
  float* o_swa;
  float* o_rla;
  const float* gamma_swa;
  const float* gamma_rla;
  int* status;
  int T, w, H_q, group, mode, n_chunks;
  float scale_log2, eps;
};

#define WAIT_OR_RETURN(bar, parity) \
  do { if (!mbar_wait(&(bar), (parity), &bars->abort)) return false; } while (0)
// for roles run by a whole converged warp
#define WAIT_OR_RETURN_W(bar, parity) \
  do { if (!mbar_wait_warp(&(bar), (parity), &bars->abort)) return false; } while (0)

// ------------------------------------------------------------------ control warp (all 32 lanes)
__device__ bool control_role(const CUtensorMap* tm_q, const CUtensorMap* tm_k, const CUtensorMap* tm_v,
                             const CUtensorMap* tm_st, unsigned char* smem, FwdBars* bars, uint32_t tmem,
                             int q0, int bh_q, int bh_kv, int n_kt, bool has_rla, bool has_state, int st_index) {
  const uint32_t sQ = smem_u32(smem + OFF_Q), sK = smem_u32(smem + OFF_K), sV = smem_u32(smem + OFF_V);
  const uint32_t sP = smem_u32(smem + OFF_P), sST = smem_u32(smem + OFF_ST);
  const uint32_t tS[2] = {tmem, tmem + 128}, tOs = tmem + 256, tOr = tmem + 384;

  auto load_tile = [&](const CUtensorMap* tm, int off, uint64_t* bar, int row, int z) {
    mbar_arrive_expect_tx(bar, TILE_BYTES);
    tma_load_3d(smem + off, tm, bar, 0, row, z);
    tma_load_3d(smem + off + HALF_BYTES, tm, bar, 64, row, z);
  };
  load_tile(tm_q, OFF_Q, &bars->q_full, q0, bh_q);
  const int n_pre = n_kt < 2 ? n_kt : 2;
  for (int i = 0; i < n_pre; ++i) {
    load_tile(tm_k, OFF_K + i * TILE_BYTES, &bars->k_full[i], q0 - i * TILE, bh_kv);
    load_tile(tm_v, OFF_V + i * TILE_BYTES, &bars->v_full[i], q0 - i * TILE, bh_kv);
  }
  if (has_state) load_tile(tm_st, OFF_ST, &bars->st_full, 0, st_index);

  WAIT_OR_RETURN_W(bars->q_full, 0);
  WAIT_OR_RETURN_W(bars->k_full[0], 0);
  tc_fence_after();
  mma_kk(tS[0], sQ, sK, false);
  mma_commit(&bars->s_full[0]);

  for (int i = 0; i < n_kt; ++i) {
    if (i + 1 < n_kt) {                       // scores of the next tile into the other buffer
      const int b = (i + 1) & 1;
      WAIT_OR_RETURN_W(bars->k_full[b], ((i + 1) >> 1) & 1);
      if (i + 1 >= 2) WAIT_OR_RETURN_W(bars->s_empty[b], (((i + 1) >> 1) - 1) & 1);
      tc_fence_after();
      mma_kk(tS[b], sQ, sK + b * TILE_BYTES, false);
      mma_commit(&bars->s_full[b]);
    }
    if (i >= 1 && i + 1 < n_kt) {             // V of tile i+1 replaces V of tile i-1
      WAIT_OR_RETURN_W(bars->pv_done, (i - 1) & 1);
      load_tile(tm_v, OFF_V + ((i + 1) & 1) * TILE_BYTES, &bars->v_full[(i + 1) & 1], q0 - (i + 1) * TILE, bh_kv);
    }
    if (i + 2 < n_kt) {                       // K of tile i+2 replaces K of tile i
      WAIT_OR_RETURN_W(bars->s_full[i & 1], (i >> 1) & 1);
      load_tile(tm_k, OFF_K + (i & 1) * TILE_BYTES, &bars->k_full[i & 1], q0 - (i + 2) * TILE, bh_kv);
    }
    WAIT_OR_RETURN_W(bars->p_full, i & 1);
    WAIT_OR_RETURN_W(bars->v_ready[i & 1], (i >> 1) & 1);
    tc_fence_after();
    mma_kmn<0>(tOs, sP, sV + (i & 1) * TILE_BYTES, i > 0);
    mma_commit(&bars->pv_done);
  }

  if (has_rla) {
    const int last = (n_kt - 1) & 1;          // stage of the oldest tile of the band
    const int ba = n_kt & 1;                  // score buffer for phi(Q) phi(K)^T
    const int uses = (n_kt - ba + 1) >> 1;    // earlier uses of that buffer
    WAIT_OR_RETURN_W(bars->phi_ready, 0);
    if (uses > 0) WAIT_OR_RETURN_W(bars->s_empty[ba], (uses - 1) & 1);
    tc_fence_after();
    mma_kk(tS[ba], sQ, sK + last * TILE_BYTES, false);
    mma_commit(&bars->s_full[ba]);
    if (has_state) {
      WAIT_OR_RETURN_W(bars->st_full, 0);
      tc_fence_after();
      mma_kmn<1>(tOr, sQ, sST, false);
    }
    WAIT_OR_RETURN_W(bars->p_full, n_kt & 1);
    tc_fence_after();
    mma_kmn<0>(tOr, sP, sV + last * TILE_BYTES, has_state);
  }
  mma_commit(&bars->o_done);
  return true;
}

// ------------------------------------------------------------------ softmax / epilogue
__device__ bool softmax_role(const TcArgs& a, const CUtensorMap* tm_out, unsigned char* smem, FwdBars* bars, uint32_t tmem, int r,
                             int q0, int bh_q, int h, int n_kt, bool has_boundary, bool has_rla) {
  const uint32_t lane_off = (uint32_t)((r & ~31) << 16);   // this warp's 32 TMEM lanes
  const uint32_t tS[2] = {tmem + lane_off, tmem + 128 + lane_off};
  const uint32_t tOs = tmem + 256 + lane_off, tOr = tmem + 384 + lane_off;
  unsigned char* sP = smem + OFF_P;

  float m_ref = -INFINITY, l = 0.f;
  for (int i = 0; i < n_kt; ++i) {
    const int b = i & 1;
    WAIT_OR_RETURN(bars->s_full[b], (i >> 1) & 1);
    tc_fence_after();
    float s[128];
#pragma unroll
    for (int c = 0; c < 4; ++c) tmem_ld32(tS[b] + 32 * c, *reinterpret_cast<float(*)[32]>(&s[32 * c]));
    tmem_wait_ld();
    tc_fence_before();
    mbar_arrive(&bars->s_empty[b]);

    const bool diag = (i == 0), bound = has_boundary && (i == n_kt - 1);
    float mx = -INFINITY;
#pragma unroll
    for (int j = 0; j < 128; ++j) {
      const bool ok = !((diag && j > r) || (bound && j < r));
      s[j] = ok ? s[j] * a.scale_log2 : -INFINITY;
      mx = fmaxf(mx, s[j]);
    }
    // lazy rescale: the reference maximum only moves when the row maximum grew by more than 2^8
    const float m_new = fmaxf(m_ref, mx);
    bool rescale = false;
    if (i == 0) {
      m_ref = m_new;
    } else {
      rescale = __any_sync(0xffffffffu, m_new > m_ref + 8.f);
    }
    const float m_use = rescale ? m_new : m_ref;
    uint32_t pk[64];
    float psum = 0.f;
#pragma unroll
    for (int j = 0; j < 64; ++j) {
      const float p0 = ex2(s[2 * j] - m_use), p1 = ex2(s[2 * j + 1] - m_use);
      psum += p0 + p1;
      pk[j] = pack_f16(p0, p1);
    }
    if (i > 0) WAIT_OR_RETURN(bars->pv_done, (i - 1) & 1);   // P buffer free, O_swa settled
    if (rescale) {
      const float f = ex2(m_ref - m_new);
      tc_fence_after();
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        float o[32];
        tmem_ld32(tOs + 32 * c, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) o[e] *= f;
        tmem_st32(tOs + 32 * c, o);
      }
      tmem_wait_st();
      l *= f;
      m_ref = m_new;
    }
    l += psum;
#pragma unroll
    for (int c = 0; c < 16; ++c)
      *reinterpret_cast<uint4*>(sP + swz(r, c)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
    fence_proxy_async_smem();
    tc_fence_before();
    mbar_arrive(&bars->p_full);
  }

  if (has_rla) {
    // every Q K^T product has completed (the last s_full was observed): phi in place
    const int last = (n_kt - 1) & 1;
    feature_map_row_inplace(smem + OFF_Q, r);
    feature_map_row_inplace(smem + OFF_K + last * TILE_BYTES, r);
    fence_proxy_async_smem();
    mbar_arrive(&bars->phi_ready);
    const int ba = n_kt & 1, uses = (n_kt - ba + 1) >> 1;
    WAIT_OR_RETURN(bars->s_full[ba], uses & 1);
    tc_fence_after();
    uint32_t pk[64];
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float x[32];
      tmem_ld32(tS[ba] + 32 * c, x);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) {
        const int j = 32 * c + 2 * e;        // residual keys of row r inside this chunk: j < r
        pk[16 * c + e] = pack_f16(j < r ? x[2 * e] : 0.f, j + 1 < r ? x[2 * e + 1] : 0.f);
      }
    }
    WAIT_OR_RETURN(bars->pv_done, (n_kt - 1) & 1);
#pragma unroll
    for (int c = 0; c < 16; ++c)
      *reinterpret_cast<uint4*>(sP + swz(r, c)) = make_uint4(pk[4 * c], pk[4 * c + 1], pk[4 * c + 2], pk[4 * c + 3]);
    fence_proxy_async_smem();
    tc_fence_before();
    mbar_arrive(&bars->p_full);
  }

  // ---- Section 3.2: two RMS norms, gains, sum --------------------------------------
  WAIT_OR_RETURN(bars->o_done, 0);
  tc_fence_after();
  const float inv_l = 1.f / l;
  float ss = 0.f, sr = 0.f;
#pragma unroll
  for (int c = 0; c < 4; ++c) {
    float o[32];
    tmem_ld32(tOs + 32 * c, o);
    tmem_wait_ld();
#pragma unroll
    for (int e = 0; e < 32; ++e) ss += o[e] * o[e];
    if (has_rla) {
      tmem_ld32(tOr + 32 * c, o);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) sr += o[e] * o[e];
    }
  }
  const float rs = inv_l * rsqrtf(ss * inv_l * inv_l * (1.f / 128.f) + a.eps);
  const float rr = rsqrtf(sr * (1.f / 128.f) + a.eps);
  const int t = q0 + r;
  const bool live = t < a.T;
  const size_t row = (size_t)bh_q * a.T + t;
  // Every product has completed, so the operand tiles are free: y is staged in the P tile
  // (bf16, swizzled) for one TMA store, the fp32 residuals in the K stages, 32 columns at a
  // time, so that each warp writes whole 128-byte segments of its own 32 rows.
  unsigned char* sY = smem + OFF_P;
  unsigned char* stage_s = smem + OFF_K;
  unsigned char* stage_r = smem + OFF_K + 16384;
  const size_t tile_row0 = (size_t)bh_q * a.T + q0;
#pragma unroll 1
  for (int c = 0; c < 4; ++c) {
    float os[32], orl[32];
    tmem_ld32(tOs + 32 * c, os);
    if (has_rla) tmem_ld32(tOr + 32 * c, orl);
    tmem_wait_ld();
    float y[32];
#pragma unroll
    for (int e = 0; e < 32; ++e) {
      const float gs = a.gamma_swa ? __ldg(a.gamma_swa + (size_t)h * 128 + 32 * c + e) : 1.f;
      y[e] = gs * os[e] * rs;
      if (has_rla) {
        const float gr = a.gamma_rla ? __ldg(a.gamma_rla + (size_t)h * 128 + 32 * c + e) : 1.f;
        y[e] += gr * orl[e] * rr;
      }
    }
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      uint4 u;
      u.x = pack_bf16(y[8 * e + 0], y[8 * e + 1]);
      u.y = pack_bf16(y[8 * e + 2], y[8 * e + 3]);
      u.z = pack_bf16(y[8 * e + 4], y[8 * e + 5]);
      u.w = pack_bf16(y[8 * e + 6], y[8 * e + 7]);
      *reinterpret_cast<uint4*>(sY + swz(r, 4 * c + e)) = u;
    }
    if (a.o_swa) {
#pragma unroll
      for (int e = 0; e < 32; ++e) {
        os[e] *= inv_l;
        if (!has_rla) orl[e] = 0.f;
      }
      __syncwarp();
      stage_f32_block(stage_s, r, os);
      stage_f32_block(stage_r, r, orl);
      __syncwarp();
      flush_f32_block(stage_s, r, a.o_swa + tile_row0 * 128 + 32 * c, a.T - q0);
      flush_f32_block(stage_r, r, a.o_rla + tile_row0 * 128 + 32 * c, a.T - q0);
    }
  }
  fence_proxy_async_smem();
  rows_sync();
  if (r == 0) {
    store_tile(tm_out, sY, q0, bh_q);
    tma_store_commit();
    tma_store_wait_read();
  }
  if (live && a.lse) a.lse[row] = (m_ref + log2f(l)) * 0.6931471805599453f;
  tc_fence_before();
  return true;
}

// ------------------------------------------------------------------ V re-encoding
__device__ bool convert_role(unsigned char* smem, FwdBars* bars, int cid, int n_kt) {
  for (int i = 0; i < n_kt; ++i) {
    WAIT_OR_RETURN(bars->v_full[i & 1], (i >> 1) & 1);
    unsigned char* tile = smem + OFF_V + (i & 1) * TILE_BYTES;
#pragma unroll 4
    for (int c = cid; c < TILE_BYTES / 16; c += 96) {
      uint4 u = *reinterpret_cast<uint4*>(tile + c * 16);
      u.x = bf16x2_to_f16x2(u.x);
      u.y = bf16x2_to_f16x2(u.y);
      u.z = bf16x2_to_f16x2(u.z);
      u.w = bf16x2_to_f16x2(u.w);
      *reinterpret_cast<uint4*>(tile + c * 16) = u;
    }
    fence_proxy_async_smem();
    mbar_arrive(&bars->v_ready[i & 1]);
  }
  return true;
}

__global__ void __launch_bounds__(256, 1)
tc_fwd_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_k,
              const __grid_constant__ CUtensorMap tm_v, const __grid_constant__ CUtensorMap tm_st,
              const __grid_constant__ CUtensorMap tm_out, TcArgs a) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  FwdBars* bars = reinterpret_cast<FwdBars*>(smem + OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;

  const int n_qt = (a.T + TILE - 1) / TILE;
  const int qt = n_qt - 1 - (int)blockIdx.x;
  const int q0 = qt * TILE;
  const int bh_q = blockIdx.y;
  const int b = bh_q / a.H_q, h = bh_q % a.H_q;
  const int bh_kv = b * (a.H_q / a.group) + h / a.group;
  const int wt = a.w / TILE;                               // window in tiles (w = T for full causal)
  const bool has_boundary = (a.mode != RATTN_MODE_FULL_CAUSAL) && (qt - wt >= 0);
  const int n_kt = (has_boundary ? wt : qt) + 1;
  const bool has_rla = has_boundary && (a.mode == RATTN_MODE_RATTN);
  const int cb = qt - wt;                                  // chunk the residual branch reads intra
  const bool has_state = has_rla && cb > 0;
  const int st_index = bh_kv * a.n_chunks + (cb > 0 ? cb : 0);

  if (tid == 0) {
    mbar_init(&bars->q_full, 1);
    mbar_init(&bars->st_full, 1);
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->k_full[i], 1);
      mbar_init(&bars->v_full[i], 1);
      mbar_init(&bars->v_ready[i], 96);
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->s_empty[i], 128);
    }
    mbar_init(&bars->p_full, 128);
    mbar_init(&bars->pv_done, 1);
    mbar_init(&bars->phi_ready, 128);
    mbar_init(&bars->o_done, 1);
    mbar_init(&bars->drain, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 4) {
    tmem_alloc(&bars->tmem_base, 512);
    tmem_relinquish();
    if (tid == 128) {   // one lane is enough for the prefetches
      prefetch_tensormap(&tm_q);
      prefetch_tensormap(&tm_k);
      prefetch_tensormap(&tm_v);
      prefetch_tensormap(&tm_st);
      prefetch_tensormap(&tm_out);
    }
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  bool ok = true;
  if (warp < 4) {
    ok = softmax_role(a, &tm_out, smem, bars, tmem, tid, q0, bh_q, h, n_kt, has_boundary, has_rla);
  } else if (warp == 4) {
    ok = control_role(&tm_q, &tm_k, &tm_v, &tm_st, smem, bars, tmem, q0, bh_q, bh_kv, n_kt, has_rla,
                      has_state, st_index);
    if (!ok) {
      // give the MMAs already issued a bounded time to finish before TMEM is released
      mma_commit(&bars->drain);
      for (int it = 0; it < (1 << 16) && !mbar_try_wait(&bars->drain, 0); ++it) {}
    }
  } else if (warp > 4) {
    ok = convert_role(smem, bars, tid - 160, n_kt);
  }
  if (!ok && a.status) atomicExch(a.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 4) {
    tc_fence_after();
    tmem_dealloc(tmem, 512);
  }
}

// ------------------------------------------------------------ per-chunk state kernel
constexpr int CS_SMEM = 2 * TILE_BYTES + 64 + 1024;

__global__ void __launch_bounds__(128)
tc_chunk_delta_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                      float* __restrict__ delta, int n_chunks, int* status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = reinterpret_cast<unsigned char*>(((uintptr_t)smem_raw + 1023) & ~(uintptr_t)1023);
  struct Bars { uint64_t full, done; uint32_t tmem_base; int abort; };
  Bars* bars = reinterpret_cast<Bars*>(smem + 2 * TILE_BYTES);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int c = blockIdx.x, kv = blockIdx.y;
  if (tid == 0) {
    mbar_init(&bars->full, 1);
    mbar_init(&bars->done, 1);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 0) {
    tmem_alloc(&bars->tmem_base, 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  if (warp == 0) {
    mbar_arrive_expect_tx(&bars->full, 2 * TILE_BYTES);
    tma_load_3d(smem, &tm_k, &bars->full, 0, c * TILE, kv);
    tma_load_3d(smem + HALF_BYTES, &tm_k, &bars->full, 64, c * TILE, kv);
    tma_load_3d(smem + TILE_BYTES, &tm_v, &bars->full, 0, c * TILE, kv);
    tma_load_3d(smem + TILE_BYTES + HALF_BYTES, &tm_v, &bars->full, 64, c * TILE, kv);
  }
  bool ok = mbar_wait(&bars->full, 0, &bars->abort);
  if (ok) {
    feature_map_row_inplace(smem, tid);        // phi(k_j) for token j = tid of the chunk
    fence_proxy_async_smem();
  }
  __syncthreads();
  if (warp == 0 && !__any_sync(0xffffffffu, bars->abort != 0)) {
    tc_fence_after();
    mma_mnmn(tmem, smem_u32(smem), smem_u32(smem + TILE_BYTES), false);   // phi(K)^T V  (Eq. 2)
    mma_commit(&bars->done);
  }
  ok = ok && mbar_wait(&bars->done, 0, &bars->abort);
  if (ok) {
    tc_fence_after();
    float* dst = delta + (((size_t)kv * n_chunks + c) * 128 + tid) * 128;   // row = feature index
#pragma unroll
    for (int cc = 0; cc < 4; ++cc) {
      float x[32];
      tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + 32 * cc, x);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 8; ++e)
        *reinterpret_cast<float4*>(dst + 32 * cc + 4 * e) = make_float4(x[4 * e], x[4 * e + 1], x[4 * e + 2], x[4 * e + 3]);
    }
  } else if (status) {
    atomicExch(status, 1);
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

// state[kv][c+1] = sum_{c' <= c} delta[kv][c']   (bf16), c = 0..n_delta-1.  (Eq. 2)
__global__ void __launch_bounds__(256)
tc_chunk_scan_kernel(const float* __restrict__ delta, __nv_bfloat16* __restrict__ state, int n_chunks,
                     int n_delta) {
  const int kv = blockIdx.x;
  const int idx = blockIdx.y * 256 + threadIdx.x;          // float4 index inside a 128x128 matrix
  const float4* src = reinterpret_cast<const float4*>(delta) + (size_t)kv * n_chunks * 4096 + idx;
  uint2* dst = reinterpret_cast<uint2*>(state) + (size_t)kv * n_chunks * 4096 + idx;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int c = 0; c < n_delta; ++c) {
    const float4 x = src[(size_t)c * 4096];
    acc.x += x.x; acc.y += x.y; acc.z += x.z; acc.w += x.w;
    dst[(size_t)(c + 1) * 4096] = make_uint2(pack_bf16(acc.x, acc.y), pack_bf16(acc.z, acc.w));
  }
}

}  // namespace

cudaError_t launch_tc_forward(const Args& a, cudaStream_t s) {
  CUtensorMap tm_q, tm_k, tm_v, tm_st, tm_out;
  if (!make_map(&tm_q, a.q, a.T, (uint64_t)a.B * a.H_q)) return cudaErrorInvalidValue;
  if (!make_map(&tm_k, a.k, a.T, (uint64_t)a.B * a.H_kv)) return cudaErrorInvalidValue;
  if (!make_map(&tm_v, a.v, a.T, (uint64_t)a.B * a.H_kv)) return cudaErrorInvalidValue;
  if (!make_map(&tm_out, a.out, a.T, (uint64_t)a.B * a.H_q)) return cudaErrorInvalidValue;
  if (!make_map(&tm_st, a.chunk_state, 128, (uint64_t)a.B * a.H_kv * a.n_chunks)) return cudaErrorInvalidValue;

  const int n_qt = (a.T + TILE - 1) / TILE;
  const int n_delta = (a.mode == RATTN_MODE_RATTN) ? n_qt - 1 - a.w / TILE : 0;
  cudaError_t e;
  if (n_delta > 0) {
    e = cudaFuncSetAttribute(tc_chunk_delta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CS_SMEM);
    if (e != cudaSuccess) return e;
    {
      KernelTimer kt("tc_chunk_delta", s);
      tc_chunk_delta_kernel<<<dim3(n_delta, a.B * a.H_kv), 128, CS_SMEM, s>>>(tm_k, tm_v, a.chunk_delta, a.n_chunks, a.status);
    }
    {
      KernelTimer kt("tc_chunk_scan", s);
      tc_chunk_scan_kernel<<<dim3(a.B * a.H_kv, 16), 256, 0, s>>>(a.chunk_delta, a.chunk_state, a.n_chunks, n_delta);
    }
    count_launches(2);
  }
  TcArgs t;
  t.out = reinterpret_cast<__nv_bfloat16*>(a.out);
  t.lse = a.lse; t.o_swa = a.o_swa; t.o_rla = a.o_rla;
  t.gamma_swa = a.gamma_swa; t.gamma_rla = a.gamma_rla; t.status = a.status;
  t.T = a.T; t.w = a.w; t.H_q = a.H_q; t.group = a.group; t.mode = a.mode; t.n_chunks = a.n_chunks;
  t.scale_log2 = a.scale * 1.4426950408889634f; t.eps = a.eps;
  e = cudaFuncSetAttribute(tc_fwd_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, FWD_SMEM);
  if (e != cudaSuccess) return e;
  {
    KernelTimer kt("tc_fwd", s);
    tc_fwd_kernel<<<dim3(n_qt, a.B * a.H_q), 256, FWD_SMEM, s>>>(tm_q, tm_k, tm_v, tm_st, tm_out, t);
  }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace rattn
