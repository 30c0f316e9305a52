// Tensor-core forward for bf16, d = 128, window a multiple of 128 (sm_100a: TMA + tcgen05 + TMEM).
//
// Persistent kernel, one CTA per SM.  A work unit is a pair of adjacent query tiles (A = 2p,
// B = 2p+1, 128 rows each) of one query head; the two tiles share one descending stream of
// key tiles (2p+1 down to 2p - w/128), so every K/V tile is fetched once for both.
//
//   row group A / B (4 warps each, thread = query row = TMEM lane)
//       SWA (Section 2.1): online softmax straight out of TMEM; P (fp16) is written back over
//       the score columns and read from there by the P V product, so it never touches shared
//       memory.  While one group exponentiates, the tensor pipe works for the other group.
//   MMA warp      S = Q K^T, O += P V (A operand from TMEM), the residual-branch products
//   loader warp   TMA: Q tiles, K/V stages, the stored chunk state
//   2 helper warps re-encode each V tile bf16 -> fp16 in place (tcgen05 needs A and B of one type)
//
//   RLA (Eq. 4 in the chunkwise form of Eq. 2-3 with the window lag): when a tile's window loop
//   ends, its normalised window output is parked in registers (fp16) and the same accumulator
//   is reused.  With cA = 2p - w/128 the chunk tile A reads in "intra" form and S_[cA] the stored
//   state (sum over the chunks before cA of phi(K)^T V):
//       O_rla(A) = phi(Q_A) S_[cA] + ((phi(Q_A) phi(K_cA)^T) masked to j < t - w) V_cA
//       O_rla(B) = phi(Q_B) S_[cA] +  (phi(Q_B) phi(K_cA)^T) V_cA                       (chunk cA whole)
//                                  + ((phi(Q_B) phi(K_cB)^T) masked) V_cB,   cB = cA + 1
//   so one stored state serves both tiles.  phi (softmax over the head features, Section 3.1)
//   is applied to the Q and K tiles in shared memory, in place: it never goes to HBM.
//   Section 3.2: y = g_s * o_swa / rms(o_swa) + g_r * o_rla / rms(o_rla), staged in the tile's Q
//   buffer and written by one TMA store.
#include <type_traits>

#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

constexpr int F_OFF_Q = 0;                       // Q_A, Q_B
constexpr int F_OFF_KV = 2 * TILE_BYTES;         // 2 stages x [K | V]
constexpr int F_OFF_X = 6 * TILE_BYTES;          // stored chunk state
constexpr int F_OFF_BAR = 7 * TILE_BYTES;
constexpr int F_SMEM = F_OFF_BAR + 512;
constexpr int F_THREADS = 384;
constexpr float LOG2E = 1.4426950408889634f;

constexpr int SCHED_SLOTS = 4;
constexpr int SCHED_READERS = 256 + 1 + 64;      // row threads, the MMA warp's lane 0, the converter threads

struct FBars {
  uint64_t q_full[2], q_free[2], k_full[2], v_full[2], v_ready[2], k_free[2], v_free[2], x_full, x_free;
  uint64_t s_full[2], p_ready[2], o_ready[2], stash_done[2], phiq_ready[2], phik_ready[2], o_free[2], y_done[2], drain;
  uint64_t sched_full[SCHED_SLOTS], sched_free[SCHED_SLOTS];
  int sched_unit[SCHED_SLOTS];
  uint32_t tmem_base;
  int abort;
};

struct FArgs {
  float* lse;
  __nv_bfloat16* o_swa;   // training mode: un-normalised branch outputs [B*H_q, T, 128] as bf16
  __nv_bfloat16* o_rla;   // (the tensor-core backward reads them in that form)
  const float* gamma_swa;
  const float* gamma_rla;
  int* status;
  int* work_counter;      // next unit to hand out (device memory, zero at launch); null: static round-robin
  int T, w, H_q, group, mode, n_chunks, n_qt, n_pairs, n_units, n_bh;
  int phi;                // rattn_feature_map
  int off;                // key tile of query tile 0 (a resumed sequence carries w/128 history tiles in front)
  int first_state;        // smallest chunk index whose state is stored: 1 (S_[0] = 0), or 0 with an incoming state
  const int* seq_lens;    // optional [B]: valid query rows per batch entry
  int n_stateless;        // pairs whose tiles read no stored state; their units come first
  int wait_for_states;    // a chunk-state kernel runs ahead of this one: wait for it before the first state load
  const int* state_ready; // ... or, per K/V head, for the number of states it has published so far (null: the former)
  int ascending;          // units in sequence order, the order in which their states appear
  int debug_skip_arrive;  // debug build only: tile A's row group withholds its first hand-over (a wait then runs out)
  float scale_log2, eps;
};

struct FMaps {
  UMap q, k, v, out;          // the caller's tensors (either head layout)
  CUtensorMap st;
  CUtensorMap o_swa, o_rla;   // training mode: the un-normalised branch outputs, [B*H_q, T, 128] bf16
};

// What one unit consists of; every role derives the same plan from the unit index.
struct Unit {
  int bh_q, bh_kv, h;
  int t[2];                 // tile index of A, B (B: -1 when the sequence ends after A)
  int kt_hi, n;             // key tiles kt_hi, kt_hi-1, ..., kt_hi-n+1
  int i0[2], i1[2];         // stream positions each tile is active on (inclusive)
  bool rla[2];
  bool has_state;           // cA > 0: a stored state exists
  int cA;
  bool windowed;
  int wt;
};

__device__ __forceinline__ Unit make_unit(const FArgs& a, int u) {
  Unit un;
  // Order: first the pairs that read no stored state (they can run while the chunk-state kernel
  // is still at work), then the others, heaviest first.
  const int pr = u / a.n_bh;
  un.bh_q = u % a.n_bh;
  const int p = (a.ascending || pr < a.n_stateless) ? pr : a.n_pairs - 1 - (pr - a.n_stateless);
  const int b = un.bh_q / a.H_q;
  un.h = un.bh_q % a.H_q;
  un.bh_kv = b * (a.H_q / a.group) + un.h / a.group;
  un.wt = a.w / TILE;
  un.windowed = (a.mode != RATTN_MODE_FULL_CAUSAL);
  // tile indices are key-space positions: query tile i of the call sits at key tile i + off
  const int n_qt = a.seq_lens ? (min(a.T, a.seq_lens[b]) + TILE - 1) / TILE : a.n_qt;
  un.t[0] = (2 * p < n_qt) ? a.off + 2 * p : -1;             // a unit without tile A is empty
  un.t[1] = (2 * p + 1 < n_qt) ? a.off + 2 * p + 1 : -1;
  un.kt_hi = un.t[1] >= 0 ? un.t[1] : un.t[0];
  const int loA = un.windowed ? max(0, un.t[0] - un.wt) : 0;
  un.n = un.kt_hi - loA + 1;
  un.i0[0] = un.kt_hi - un.t[0];
  un.i1[0] = un.n - 1;
  un.i0[1] = 0;
  un.i1[1] = un.t[1] >= 0 ? un.kt_hi - (un.windowed ? max(0, un.t[1] - un.wt) : 0) : -1;
  const bool rla_mode = un.windowed && a.mode == RATTN_MODE_RATTN;
  un.rla[0] = rla_mode && un.t[0] - un.wt >= 0;
  un.rla[1] = rla_mode && un.t[1] >= 0 && un.t[1] - un.wt >= 0;
  un.cA = un.t[0] - un.wt;
  un.has_state = un.rla[0] && un.cA >= a.first_state;
  return un;
}

__device__ __forceinline__ bool active(const Unit& un, int X, int i) { return un.t[X] >= 0 && i >= un.i0[X] && i <= un.i1[X]; }

// Optional timeline for tuning (compiled in only with -DRATTN_TIMELINE): one CTA records
// (event id, clock) pairs per role.
#ifdef RATTN_TIMELINE
__device__ unsigned long long g_timeline[4][2048];
__device__ int g_timeline_n[4];
#define TL_DECL(on_expr) const bool tl_on = (on_expr); int tl_i = 0; (void)tl_on; (void)tl_i
#define TL(role, id) do { if (tl_on && tl_i < 1000) { unsigned long long c_; asm volatile("mov.u64 %0, %%clock64;" : "=l"(c_) :: "memory"); \
    g_timeline[role][2 * tl_i] = (unsigned long long)(id); g_timeline[role][2 * tl_i + 1] = c_; ++tl_i; g_timeline_n[role] = tl_i; } } while (0)
#else
#define TL_DECL(on_expr) do { } while (0)
#define TL(role, id) do { } while (0)
#endif

// the MMA warp's own events cost it issue slots: they are a second switch (-DRATTN_TIMELINE_MMA)
#ifdef RATTN_TIMELINE_MMA
#define TLM(role, id) TL(role, id)
#else
#define TLM(role, id) do { } while (0)
#endif

#define WAIT_OR_RETURN(bar, parity) \
  do { if (!mbar_wait(&(bar), (parity), &bars->abort)) return false; } while (0)
#define WAIT_OR_RETURN_W(bar, parity) \
  do { if (!mbar_wait_warp(&(bar), (parity), &bars->abort)) return false; } while (0)

// D[128x128] (+)= P[128 x 128 keys] (fp16 in TMEM, 64 columns) . V[128 keys x 128] (fp16, MN-major)
__device__ __forceinline__ void mma_pv(uint32_t d, uint32_t p_tmem, uint32_t v_base, bool acc) {
  constexpr uint32_t idesc = instr_desc(128, 128, 0, 1, 0);
  const uint64_t b0 = mnmajor_base(v_base);
#pragma unroll
  for (int k = 0; k < 8; ++k) mma_bf16_ts(d, p_tmem + 8 * k, b0 + kstep_mn(k), idesc, (acc || k > 0) ? 1u : 0u);
}

// ------------------------------------------------------------------------------ work units
// The loader warp draws the CTA's next unit (from a device-wide counter, so that CTAs that start
// late -- their SM was still running the chunk-state kernel -- simply take fewer units) and
// publishes it in a small ring; the other roles read the ring in order.  A slot is rewritten
// only after every reader has read it.
__device__ __forceinline__ bool sched_next_producer(const FArgs& a, FBars* bars, int n, int* u_out) {
  const int slot = n % SCHED_SLOTS, use = n / SCHED_SLOTS;
  if (use >= 1) { if (!mbar_wait_warp(&bars->sched_free[slot], (use - 1) & 1, &bars->abort)) return false; }
  int u = 0;
  if (a.work_counter) {
    if ((threadIdx.x & 31) == 0) u = atomicAdd(a.work_counter, 1);
    u = __shfl_sync(0xffffffffu, u, 0);
  } else {
    u = blockIdx.x + n * gridDim.x;
  }
  if (u >= a.n_units) u = -1;
  if ((threadIdx.x & 31) == 0) {
    bars->sched_unit[slot] = u;
    mbar_arrive(&bars->sched_full[slot]);
  }
  __syncwarp();
  *u_out = u;
  return true;
}
// every reading thread calls this; `arrives` says whether this thread is one of the counted readers
__device__ __forceinline__ bool sched_next(FBars* bars, int n, bool arrives, int* u_out) {
  const int slot = n % SCHED_SLOTS, use = n / SCHED_SLOTS;
  if (!mbar_wait(&bars->sched_full[slot], use & 1, &bars->abort)) return false;
  *u_out = bars->sched_unit[slot];
  if (arrives) mbar_arrive(&bars->sched_free[slot]);
  return true;
}

// ----------------------------------------------------------------------------- loader
// Bounded wait (whole warp) until a progress word of another kernel reaches `need`; the TMA loads
// that follow are ordered behind the acquiring read.
__device__ __forceinline__ bool wait_published(const int* word, int need, volatile int* abort) {
#pragma unroll 1
  for (int it = 0; it < (1 << 20); ++it) {
    if (ld_acquire_gpu(word) >= need) {
      fence_proxy_async_all();
      return true;
    }
    if ((it & 15) == 15 && *abort) return false;
    __nanosleep(200);
  }
  *abort = 1;
  return false;
}
__device__ bool fwd_loader(const FMaps& tm, const FArgs& a, unsigned char* smem, FBars* bars) {
  int kv_count = 0, cntU[2] = {0, 0}, cntX = 0;
  bool states_ready = (a.wait_for_states == 0);
  for (int n = 0;; ++n) {
    int u;
    if (!sched_next_producer(a, bars, n, &u)) return false;
    if (u < 0) break;
    const Unit un = make_unit(a, u);
    if (un.t[0] < 0) continue;                    // beyond this batch entry's length
#pragma unroll
    for (int X = 0; X < 2; ++X) {
      if (un.t[X] < 0) continue;
      if (cntU[X] >= 1) WAIT_OR_RETURN_W(bars->q_free[X], (cntU[X] - 1) & 1);
      mbar_arrive_expect_tx(&bars->q_full[X], TILE_BYTES);
      load_tile(smem + F_OFF_Q + X * TILE_BYTES, &tm.q, &bars->q_full[X], (un.t[X] - a.off) * TILE, un.bh_q);
      ++cntU[X];
    }
    for (int i = 0; i < un.n; ++i, ++kv_count) {
      const int st = kv_count & 1, use = kv_count >> 1;
      // K and V of a stage are released separately: a K tile has served its last scores one
      // stream position before its V tile has served its last product, and the next K load
      // needs that head start to arrive in time
      unsigned char* dst = smem + F_OFF_KV + st * 2 * TILE_BYTES;
      if (use >= 1) WAIT_OR_RETURN_W(bars->k_free[st], (use - 1) & 1);
      mbar_arrive_expect_tx(&bars->k_full[st], TILE_BYTES);
      load_tile(dst, &tm.k, &bars->k_full[st], (un.kt_hi - i) * TILE, un.bh_kv);
      if (use >= 1) WAIT_OR_RETURN_W(bars->v_free[st], (use - 1) & 1);
      mbar_arrive_expect_tx(&bars->v_full[st], TILE_BYTES);
      load_tile(dst + TILE_BYTES, &tm.v, &bars->v_full[st], (un.kt_hi - i) * TILE, un.bh_kv);
    }
    if (un.has_state) {
      if (cntX >= 1) WAIT_OR_RETURN_W(bars->x_free, (cntX - 1) & 1);
      // the same buffer stages the outputs: every tile of the units before has left it
#pragma unroll
      for (int X = 0; X < 2; ++X) {
        const int done_before = cntU[X] - (un.t[X] >= 0 ? 1 : 0);      // epilogues of tile X before this unit
        if (done_before >= 1) WAIT_OR_RETURN_W(bars->y_done[X], (done_before - 1) & 1);
      }
      if (a.state_ready) {
        // the chunk-state kernel, still running beside this one, has stored and published S_[cA]
        if (!wait_published(a.state_ready + un.bh_kv, un.cA + 1, &bars->abort)) return false;
      } else if (!states_ready) {
        // the chunk-state kernel launched ahead of this one has completed and its stores are visible
        asm volatile("griddepcontrol.wait;" ::: "memory");
        states_ready = true;
      }
      mbar_arrive_expect_tx(&bars->x_full, TILE_BYTES);
      load_tile(smem + F_OFF_X, &tm.st, &bars->x_full, 0, un.bh_kv * a.n_chunks + un.cA);
      ++cntX;
    }
  }
  // not to end before the kernel whose states were taken as they appeared
  if (a.state_ready && a.wait_for_states) asm volatile("griddepcontrol.wait;" ::: "memory");
  return true;
}

// -------------------------------------------------------------------------- V re-encoding
__device__ bool fwd_convert(const FArgs& a, unsigned char* smem, FBars* bars, int cid) {
  int kv_count = 0;
  for (int n = 0;; ++n) {
    int u;
    if (!sched_next(bars, n, true, &u)) return false;
    if (u < 0) break;
    const Unit un = make_unit(a, u);
    if (un.t[0] < 0) continue;
    for (int i = 0; i < un.n; ++i, ++kv_count) {
      const int st = kv_count & 1, use = kv_count >> 1;
      WAIT_OR_RETURN(bars->v_full[st], use & 1);
      unsigned char* tile = smem + F_OFF_KV + st * 2 * TILE_BYTES + TILE_BYTES;
#pragma unroll 4
      for (int c = cid; c < TILE_BYTES / 16; c += 64) {
        uint4 x = *reinterpret_cast<uint4*>(tile + c * 16);
        x.x = bf16x2_to_f16x2(x.x);
        x.y = bf16x2_to_f16x2(x.y);
        x.z = bf16x2_to_f16x2(x.z);
        x.w = bf16x2_to_f16x2(x.w);
        *reinterpret_cast<uint4*>(tile + c * 16) = x;
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->v_ready[st]);
    }
  }
  return true;
}

// ----------------------------------------------------------------------------- MMA warp
__device__ bool fwd_mma(const FArgs& a, unsigned char* smem, FBars* bars, uint32_t tmem) {
  const uint32_t sQ[2] = {smem_u32(smem + F_OFF_Q), smem_u32(smem + F_OFF_Q + TILE_BYTES)};
  const uint32_t sKV = smem_u32(smem + F_OFF_KV), sX = smem_u32(smem + F_OFF_X);
  const uint32_t tS[2] = {tmem, tmem + 128}, tO[2] = {tmem + 256, tmem + 384};
  int kv_count = 0, cntU[2] = {0, 0}, cntX = 0, cntP[2] = {0, 0}, cntR[2] = {0, 0}, cntK[2] = {0, 0};
  TL_DECL(blockIdx.x == 7 && (threadIdx.x & 31) == 0);

  for (int n = 0;; ++n) {
    int u;
    if (!sched_next(bars, n, (threadIdx.x & 31) == 0, &u)) return false;
    u = __shfl_sync(0xffffffffu, u, 0);
    if (u < 0) break;
    const Unit un = make_unit(a, u);
    if (un.t[0] < 0) continue;
    const int kv0 = kv_count;
    auto stage_of = [&](int i) { return (kv0 + i) & 1; };
    auto use_of = [&](int i) { return (kv0 + i) >> 1; };
    auto sK = [&](int i) { return sKV + stage_of(i) * 2 * TILE_BYTES; };
    auto sV = [&](int i) { return sKV + stage_of(i) * 2 * TILE_BYTES + TILE_BYTES; };
#pragma unroll
    for (int X = 0; X < 2; ++X) {
      if (un.t[X] < 0) continue;
      if (cntU[X] >= 1) WAIT_OR_RETURN_W(bars->o_free[X], (cntU[X] - 1) & 1);   // previous unit has read O_X
      WAIT_OR_RETURN_W(bars->q_full[X], cntU[X] & 1);
      ++cntU[X];
    }
    // first scores of each tile
    // stream positions whose stage the residual branch still reads (chunks cA, cB)
    auto kept = [&](int i) { return (un.rla[0] && i == un.n - 1) || (un.rla[1] && i == un.i1[1]); };
    WAIT_OR_RETURN_W(bars->k_full[stage_of(0)], use_of(0) & 1);
    tc_fence_after();
#pragma unroll
    for (int X = 1; X >= 0; --X) {
      if (active(un, X, 0)) {
        mma_kk(tS[X], sQ[X], sK(0), false);
        mma_commit(&bars->s_full[X]);
      }
    }
    if (!kept(0)) mma_commit(&bars->k_free[stage_of(0)]);
    for (int i = 0; i < un.n; ++i) {
      // The operands of this position are awaited once and ahead of the weights, so that the
      // products and the next scores go out the moment a row group hands its weights over
      // (a wait costs this warp a few hundred cycles even when it is already satisfied).
      WAIT_OR_RETURN_W(bars->v_ready[stage_of(i)], use_of(i) & 1);
      if (i + 1 < un.n) WAIT_OR_RETURN_W(bars->k_full[stage_of(i + 1)], use_of(i + 1) & 1);
#pragma unroll
      for (int X = 0; X < 2; ++X) {
        if (active(un, X, i)) {
          TLM(2, 10 * i + X);
          WAIT_OR_RETURN_W(bars->p_ready[X], cntP[X] & 1);
          ++cntP[X];
          TLM(2, 200 + 10 * i + X);
          tc_fence_after();
          mma_pv(tO[X], tS[X], sV(i), i > un.i0[X]);                             // O_X += P V
          if (i == un.i1[X]) mma_commit(&bars->o_ready[X]);
          TLM(2, 300 + 10 * i + X);
        }
        if (i + 1 < un.n && active(un, X, i + 1)) {
          tc_fence_after();
          mma_kk(tS[X], sQ[X], sK(i + 1), false);                                // S_X = Q_X K^T (after P V in pipe order)
          mma_commit(&bars->s_full[X]);
          TLM(2, 500 + 10 * i + X);
        }
      }
      // K of the next position has served all its scores, V of this one all its products
      if (i + 1 < un.n && !kept(i + 1)) mma_commit(&bars->k_free[stage_of(i + 1)]);
      if (!kept(i)) mma_commit(&bars->v_free[stage_of(i)]);
    }
    // ---- residual branch ---------------------------------------------------------------
    const int iA = un.n - 1, iB = un.i1[1];          // stream positions of chunks cA, cB
    if (un.rla[0] || un.rla[1]) {
      if (un.has_state) {
        WAIT_OR_RETURN_W(bars->x_full, cntX & 1);
        ++cntX;
      }
      // scores first (they only need the feature maps), the products into the accumulators once
      // the row groups have parked the window outputs
      if (un.rla[0]) {
        WAIT_OR_RETURN_W(bars->phiq_ready[0], cntR[0] & 1);
        WAIT_OR_RETURN_W(bars->phik_ready[0], cntK[0] & 1);
        tc_fence_after();
        mma_kk(tS[0], sQ[0], sK(iA), false);                                     // phi(Q_A) phi(K_cA)^T
        mma_commit(&bars->s_full[0]);
      }
      if (un.rla[1] && un.rla[0]) {
        WAIT_OR_RETURN_W(bars->phiq_ready[1], cntR[1] & 1);
        tc_fence_after();
        mma_kk(tS[1], sQ[1], sK(iA), false);                                     // phi(Q_B) phi(K_cA)^T, whole chunk
        mma_commit(&bars->s_full[1]);
      }
      if (un.rla[0] && un.has_state) {
        WAIT_OR_RETURN_W(bars->stash_done[0], cntR[0] & 1);
        tc_fence_after();
        mma_kmn<1>(tO[0], sQ[0], sX, false);                                     // phi(Q_A) S_[cA]
      }
      if (un.rla[1]) {
        if (!un.rla[0]) WAIT_OR_RETURN_W(bars->phiq_ready[1], cntR[1] & 1);
        if (un.rla[0] && un.has_state) {
          WAIT_OR_RETURN_W(bars->stash_done[1], cntR[1] & 1);
          tc_fence_after();
          mma_kmn<1>(tO[1], sQ[1], sX, false);                                   // phi(Q_B) S_[cA]
        }
      }
      if (un.rla[0]) {
        if (!un.has_state) WAIT_OR_RETURN_W(bars->stash_done[0], cntR[0] & 1);   // O_A is free
        WAIT_OR_RETURN_W(bars->p_ready[0], cntP[0] & 1);
        ++cntP[0];
        tc_fence_after();
        mma_pv(tO[0], tS[0], sV(iA), un.has_state);
        mma_commit(&bars->o_ready[0]);
      }
      if (un.rla[1]) {
        if (!(un.rla[0] && un.has_state)) WAIT_OR_RETURN_W(bars->stash_done[1], cntR[1] & 1);   // O_B is free
        if (un.rla[0]) {
          WAIT_OR_RETURN_W(bars->p_ready[1], cntP[1] & 1);
          ++cntP[1];
          tc_fence_after();
          mma_pv(tO[1], tS[1], sV(iA), un.has_state);
        }
        WAIT_OR_RETURN_W(bars->phik_ready[1], cntK[1] & 1);
        tc_fence_after();
        mma_kk(tS[1], sQ[1], sK(iB), false);                                     // phi(Q_B) phi(K_cB)^T
        mma_commit(&bars->s_full[1]);
        WAIT_OR_RETURN_W(bars->p_ready[1], cntP[1] & 1);
        ++cntP[1];
        tc_fence_after();
        mma_pv(tO[1], tS[1], sV(iB), un.rla[0]);
        mma_commit(&bars->o_ready[1]);
      }
      if (un.has_state) mma_commit(&bars->x_free);
      if (un.rla[0]) { ++cntR[0]; ++cntK[0]; }
      if (un.rla[1]) { ++cntR[1]; ++cntK[1]; }
      // the chunk stages
      if (un.rla[0]) {
        mma_commit(&bars->k_free[stage_of(iA)]);
        mma_commit(&bars->v_free[stage_of(iA)]);
      }
      if (un.rla[1] && !(un.rla[0] && iB == iA)) {
        mma_commit(&bars->k_free[stage_of(iB)]);
        mma_commit(&bars->v_free[stage_of(iB)]);
      }
    }
    kv_count += un.n;
    TLM(2, 1000 + u);
  }
  return true;
}

// ------------------------------------------------------------------------------ row groups
__device__ __forceinline__ uint32_t lane_base(int r) { return (uint32_t)((r & ~31) << 16); }

// The per-tile loops below are rolled over 32-column chunks on purpose: with everything
// unrolled the kernel was ~390 KB of code and ran instruction-fetch bound.
__device__ bool fwd_rows(const FMaps& tm, const FArgs& a, unsigned char* smem, FBars* bars, uint32_t tmem, int X,
                         int r) {
  const uint32_t tS = tmem + 128 * X + lane_base(r), tO = tmem + 256 + 128 * X + lane_base(r);
  unsigned char* sQ = smem + F_OFF_Q + X * TILE_BYTES;
  int kv_count = 0, cntS = 0, cntO = 0;
  TL_DECL(blockIdx.x == 7 && r == 0);

  for (int n = 0;; ++n) {
    int u;
    if (!sched_next(bars, n, true, &u)) return false;
    if (u < 0) break;
    const Unit un = make_unit(a, u);
    if (un.t[0] < 0) continue;
    TL(X, 1000 + u);
    const int kv0 = kv_count;
    kv_count += un.n;
    const int tX = X ? un.t[1] : un.t[0], i0 = X ? un.i0[1] : un.i0[0], i1 = X ? un.i1[1] : un.i1[0];
    const bool rlaX = X ? un.rla[1] : un.rla[0];
    if (tX < 0) continue;
    const int q0 = (tX - a.off) * TILE;          // first query row of the tile (tX is its key-space index)
    const int t = q0 + r;

    // ---- window branch: online softmax over the key tiles of the band -------------------
    // On the two edge tiles of the band a warp's 32 rows keep whole 32-column chunks, drop whole
    // chunks (no score reads, no exponentials: zero weights) and mask exactly one chunk, the one
    // their own positions fall into: diagonal tile -> chunks 0 .. wq, oldest tile -> chunks wq .. 3.
    float m_ref = -INFINITY, l = 0.f;
    const int wq = r >> 5;                         // this warp's quarter of the tile's rows
#pragma unroll 1
    for (int i = i0; i <= i1; ++i) {
      const int kt = un.kt_hi - i;
      TL(X, 100 + i);
      WAIT_OR_RETURN(bars->s_full[X], cntS & 1);
      TL(X, 200 + i);
      ++cntS;
      tc_fence_after();
      const bool diag = (kt == tX), bound = un.windowed && (kt == tX - un.wt);
      const int c_lo = bound ? wq : 0, c_hi = diag ? wq : 3;     // chunks with kept columns
      // The whole score row is read once (128 registers; the row groups run with a raised
      // register allowance, see the kernel body) and kept for both the maximum and the weights.
      float x[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(tS + 32 * c, x[c]);      // dropped chunks too: four loads in flight
      tmem_wait_ld();
      if (diag || bound) {
        // the one chunk this warp keeps partly: dropped columns become -inf (weight zero)
        const uint32_t keep = keep_bits(r, wq, diag, bound);
#pragma unroll
        for (int c = 0; c < 4; ++c)
          if (c == wq) mask32(x[c], keep);
      }
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < 4; ++c)
        if (c >= c_lo && c <= c_hi) mx = fmaxf(mx, max32(x[c]));
      mx *= a.scale_log2;                                              // scale > 0
      // lazy rescale: the reference maximum only moves when the row maximum grew by more than 2^8
      const float m_new = fmaxf(m_ref, mx);
      bool rescale = false;
      if (i == i0) m_ref = m_new;
      else rescale = __any_sync(0xffffffffu, m_new > m_ref + 8.f);
      if (rescale) {
        // P V of the previous tile has completed (the commit behind these scores covers it)
        const float f = ex2(m_ref - m_new);
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float o[32];
          tmem_ld32(tO + 32 * c, o);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) o[e] *= f;
          tmem_st32(tO + 32 * c, o);
        }
        l *= f;
        m_ref = m_new;
      }
      TL(X, 300 + i);
      // weights, written back (fp16, two per column) over the score columns
      const float2 sc2 = make_float2(a.scale_log2, a.scale_log2), nm2 = make_float2(-m_ref, -m_ref);
      float2 ps0 = make_float2(0.f, 0.f), ps1 = make_float2(0.f, 0.f);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
        uint32_t pk[16];
        if (c < c_lo || c > c_hi) {
#pragma unroll
          for (int e = 0; e < 16; ++e) pk[e] = 0u;
        } else {
#pragma unroll
          for (int e = 0; e < 16; ++e) {
            const float2 y = __ffma2_rn(make_float2(x[c][2 * e], x[c][2 * e + 1]), sc2, nm2);
            const float2 pp = make_float2(ex2(y.x), ex2(y.y));
            if (e & 1) ps1 = __fadd2_rn(ps1, pp);
            else ps0 = __fadd2_rn(ps0, pp);
            pk[e] = pack_f16(pp.x, pp.y);
          }
        }
        tmem_st16(tS + 16 * c, pk);
      }
      const float psum = (ps0.x + ps0.y) + (ps1.x + ps1.y);
      l += psum;
      tmem_wait_st();
      tc_fence_before();
#ifdef RATTN_DEBUG_KNOBS
      // failure injection for the time-out test: an arrival that nothing else depends on is left
      // out, so the MMA warp's bounded wait expires and every role takes the abort path
      if (!(a.debug_skip_arrive && X == 0 && n == 0 && i == i0))
#endif
      mbar_arrive(&bars->p_ready[X]);
      TL(X, 400 + i);
    }

    // ---- residual branch, first part: feature maps ------------------------------------------
    // Done right here, while the last P V of the window loop is still running and before the
    // parked output takes 64 registers: the row fits in registers, so phi is one read and one
    // write of shared memory.  Every Q_X K^T and every product reading the raw chunk K has
    // completed (the commit behind this tile's last scores covers them).
    float rr = 0.f, sr = 0.f, inv_q = 1.f;
    if (rlaX) {
      // phi(Q_X) without its normalisation: everything that follows is linear in this row,
      // so 1/sum is applied to the accumulator row at the end
      inv_q = feature_map_row_any<false>(sQ, r, a.phi, a.o_swa != nullptr);
      fence_proxy_async_smem();
      mbar_arrive(&bars->phiq_ready[X]);
      TL(X, 503);
      // this tile's own chunk: A -> last stream position, B -> its last active position
      const int ic = (X == 0) ? un.n - 1 : un.i1[1];
      feature_map_row_any<true>(smem + F_OFF_KV + ((kv0 + ic) & 1) * 2 * TILE_BYTES, r, a.phi, a.o_swa != nullptr);
      fence_proxy_async_smem();
      mbar_arrive(&bars->phik_ready[X]);
      TL(X, 504);
    }

    // ---- park the normalised window output (Section 3.2, first norm) in registers ---------
    TL(X, 500);
    WAIT_OR_RETURN(bars->o_ready[X], cntO & 1);
    TL(X, 501);
    ++cntO;
    tc_fence_after();
    const float inv_l = 1.f / l;
    uint32_t stash[64];
    float ss = 0.f;
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
      float o[32];
      tmem_ld32(tO + 32 * c, o);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 32; ++e) ss += o[e] * o[e];
    }
    const float ms = ss * inv_l * inv_l * (1.f / 128.f) + a.eps;     // mean square of o_swa, plus eps
    const float rs = rsqrtf(ms);
#pragma unroll
    for (int c = 0; c < 4; ++c) {
      float o[32];
      tmem_ld32(tO + 32 * c, o);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 16; ++e) stash[16 * c + e] = pack_f16(o[2 * e] * inv_l * rs, o[2 * e + 1] * inv_l * rs);
    }

    // ---- residual branch, second part -------------------------------------------------------
    TL(X, 502);
    if (rlaX) {
      tc_fence_before();
      mbar_arrive(&bars->stash_done[X]);
      const int n_terms = (X == 1 && un.rla[0]) ? 2 : 1;
#pragma unroll 1
      for (int term = 0; term < n_terms; ++term) {
        const bool masked = (term == n_terms - 1);                     // B's first term takes chunk cA whole
        WAIT_OR_RETURN(bars->s_full[X], cntS & 1);
        ++cntS;
        tc_fence_after();
#pragma unroll 1
        for (int c = 0; c < 4; ++c) {
          float x[32];
          tmem_ld32(tS + 32 * c, x);
          tmem_wait_ld();
          // residual keys of row r in its chunk: j < r
          const int rd = r - 32 * c;
          const uint32_t keep = !masked ? 0xffffffffu : (rd >= 32 ? 0xffffffffu : (rd <= 0 ? 0u : ((1u << rd) - 1u)));
          uint32_t pk[16];
#pragma unroll
          for (int e = 0; e < 16; ++e)
            pk[e] = pack_f16((keep >> (2 * e)) & 1u ? x[2 * e] : 0.f, (keep >> (2 * e + 1)) & 1u ? x[2 * e + 1] : 0.f);
          tmem_st16(tS + 16 * c, pk);                                  // columns already consumed
        }
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->p_ready[X]);
      }
      WAIT_OR_RETURN(bars->o_ready[X], cntO & 1);
      ++cntO;
      tc_fence_after();
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float o[32];
        tmem_ld32(tO + 32 * c, o);
        tmem_wait_ld();
#pragma unroll
        for (int e = 0; e < 32; ++e) sr += o[e] * o[e];
      }
      rr = inv_q * rsqrtf(sr * inv_q * inv_q * (1.f / 128.f) + a.eps);     // o_rla = inv_q * accumulator
    }

    // ---- Section 3.2: gains, sum; outputs leave through the tile's Q buffer ---------------
    TL(X, 530);
    const float rms_s = ms * rs;                                       // sqrt(mean square + eps)
    if (a.o_swa) {
      // training mode: the un-normalised branch outputs (bf16) for the backward.  Each leaves as one
      // whole tile: every thread writes its row into the tile's Q buffer (phi(Q_X) has been consumed),
      // swizzled like a loaded tile, and one TMA store sends it off -- plain 16-byte global stores
      // from 128 threads kept the load/store unit busy under the other group's feature maps.
      unsigned char* stage = sQ;
      if (rlaX) group_sync(X);
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          uint32_t wv[4];
#pragma unroll
          for (int k2 = 0; k2 < 4; ++k2) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&stash[16 * c + 4 * e + k2]));
            wv[k2] = pack_bf16(f.x * rms_s, f.y * rms_s);
          }
          *reinterpret_cast<uint4*>(stage + swz(r, 4 * c + e)) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
        }
      }
      fence_proxy_async_smem();
      group_sync(X);
      if (r == 0) {
        store_tile(&tm.o_swa, stage, q0, un.bh_q);
        tma_store_commit();
        tma_store_wait_read();
      }
      group_sync(X);
#pragma unroll 1
      for (int c = 0; c < 4; ++c) {
        float x[32];
        if (rlaX) {
          tmem_ld32(tO + 32 * c, x);
          tmem_wait_ld();
#pragma unroll
          for (int e = 0; e < 32; ++e) x[e] *= inv_q;
        } else {
#pragma unroll
          for (int e = 0; e < 32; ++e) x[e] = 0.f;
        }
#pragma unroll
        for (int e = 0; e < 4; ++e)
          *reinterpret_cast<uint4*>(stage + swz(r, 4 * c + e)) =
              make_uint4(pack_bf16(x[8 * e], x[8 * e + 1]), pack_bf16(x[8 * e + 2], x[8 * e + 3]),
                         pack_bf16(x[8 * e + 4], x[8 * e + 5]), pack_bf16(x[8 * e + 6], x[8 * e + 7]));
      }
      fence_proxy_async_smem();
      group_sync(X);
      if (r == 0) {
        store_tile(&tm.o_rla, stage, q0, un.bh_q);
        tma_store_commit();
        tma_store_wait_read();
      }
      group_sync(X);
    }
    TL(X, 535);
    const float* gs = a.gamma_swa ? a.gamma_swa + (size_t)un.h * 128 : nullptr;
    const float* gr = a.gamma_rla ? a.gamma_rla + (size_t)un.h * 128 : nullptr;
    // y leaves through the state tile's buffer (free once this unit's residual products are done;
    // 16 KB per row group), one 64-column half at a time, so that the tile's Q buffer and the
    // K/V stages can take the next unit's loads while the epilogue runs.  The branches on "gains
    // given" and "tile has a residual branch" are taken once, outside the loops.
    unsigned char* sY = smem + F_OFF_X + X * HALF_BYTES;
    auto emit_y = [&](auto has_gains_t, auto has_rla_t) {
      constexpr bool has_gains = decltype(has_gains_t)::value, has_rla = decltype(has_rla_t)::value;
#pragma unroll
      for (int hf = 0; hf < 2; ++hf) {
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4) {                               // 16 columns at a time
          const int c = 4 * hf + c4;
          float orl[16];
          if constexpr (has_rla) {
            tmem_ld16(tO + 16 * c, orl);
            tmem_wait_ld();
          }
          uint32_t yk[8];
#pragma unroll
          for (int e = 0; e < 8; ++e) {
            const float2 f = __half22float2(*reinterpret_cast<const __half2*>(&stash[8 * c + e]));
            const int col = 16 * c + 2 * e;
            float y0 = f.x, y1 = f.y;
            if constexpr (has_gains) {
              y0 *= gs ? __ldg(gs + col) : 1.f;
              y1 *= gs ? __ldg(gs + col + 1) : 1.f;
            }
            if constexpr (has_rla) {
              float r0 = orl[2 * e] * rr, r1 = orl[2 * e + 1] * rr;
              if constexpr (has_gains) {
                r0 *= gr ? __ldg(gr + col) : 1.f;
                r1 *= gr ? __ldg(gr + col + 1) : 1.f;
              }
              y0 += r0;
              y1 += r1;
            }
            yk[e] = pack_bf16(y0, y1);
          }
          *reinterpret_cast<uint4*>(sY + swz(r, 2 * c4)) = make_uint4(yk[0], yk[1], yk[2], yk[3]);
          *reinterpret_cast<uint4*>(sY + swz(r, 2 * c4 + 1)) = make_uint4(yk[4], yk[5], yk[6], yk[7]);
        }
        if (hf == 1) {
          tc_fence_before();
          mbar_arrive(&bars->o_free[X]);   // last read of the accumulator: scores and output columns may be overwritten
        }
        fence_proxy_async_smem();
        group_sync(X);
        if (r == 0) {
          store_half(&tm.out, sY, 64 * hf, q0, un.bh_q);
          tma_store_commit();
        }
        // The Q buffer (phi(Q_X) has long been consumed) is released only once the last store is
        // in the TMA queue: the next unit's loads, issued the moment it is released, would
        // otherwise sit in front of the stores and hold the staging buffer for thousands of cycles.
        if (hf == 1) mbar_arrive(&bars->q_free[X]);
        if (r == 0) tma_store_wait_read();
        group_sync(X);
      }
    };
    const bool gains = gs != nullptr || gr != nullptr;
    if (gains) {
      if (rlaX) emit_y(std::true_type{}, std::true_type{});
      else emit_y(std::true_type{}, std::false_type{});
    } else {
      if (rlaX) emit_y(std::false_type{}, std::true_type{});
      else emit_y(std::false_type{}, std::false_type{});
    }
    if (t < a.T && a.lse) a.lse[(size_t)un.bh_q * a.T + t] = (m_ref + log2f(l)) * 0.6931471805599453f;
    mbar_arrive(&bars->y_done[X]);         // the staging buffer may take the next state tile
    TL(X, 540);
  }
  return true;
}

__global__ void __launch_bounds__(F_THREADS, 1)
tc_fwd2_kernel(const __grid_constant__ FMaps tm, FArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  FBars* bars = reinterpret_cast<FBars*>(smem + F_OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0 && a.status) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->q_full[i], 1);
      mbar_init(&bars->q_free[i], 128);
      mbar_init(&bars->k_full[i], 1);
      mbar_init(&bars->v_full[i], 1);
      mbar_init(&bars->v_ready[i], 64);
      mbar_init(&bars->k_free[i], 1);
      mbar_init(&bars->v_free[i], 1);
      mbar_init(&bars->s_full[i], 1);
      mbar_init(&bars->p_ready[i], 128);
      mbar_init(&bars->o_ready[i], 1);
      mbar_init(&bars->stash_done[i], 128);
      mbar_init(&bars->phiq_ready[i], 128);
      mbar_init(&bars->phik_ready[i], 128);
      mbar_init(&bars->o_free[i], 128);
      mbar_init(&bars->y_done[i], 128);
    }
    mbar_init(&bars->x_full, 1);
    mbar_init(&bars->x_free, 1);
    mbar_init(&bars->drain, 1);
    for (int i = 0; i < SCHED_SLOTS; ++i) {
      mbar_init(&bars->sched_full[i], 1);
      mbar_init(&bars->sched_free[i], SCHED_READERS);
    }
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
    prefetch_tensormap(&tm.st);
    prefetch_map(&tm.out);
    prefetch_tensormap(&tm.o_swa);
    prefetch_tensormap(&tm.o_rla);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;

  // Registers follow the work: the row groups keep a whole score row (128 values) live, the
  // other four warps need few.  2 x 128 x 192 + 128 x 120 = 384 x 168, the CTA's allocation; with this split neither side spills.
  bool ok = true;
  if (warp < 8) setmaxnreg_inc<192>();
  else setmaxnreg_dec<120>();
  if (warp < 8) {
    ok = fwd_rows(tm, a, smem, bars, tmem, warp >> 2, tid & 127);
  } else if (warp == 8) {
    ok = fwd_mma(a, smem, bars, tmem);
    if (!ok) {
      mma_commit(&bars->drain);
      for (int it = 0; it < (1 << 16) && !mbar_try_wait(&bars->drain, 0); ++it) {}
    }
  } else if (warp == 9) {
    ok = fwd_loader(tm, a, smem, bars);
  } else {
    ok = fwd_convert(a, smem, bars, tid - 320);
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

#ifdef RATTN_TIMELINE
extern "C" int rattn_timeline_read(unsigned long long* out, int* n) {
  cudaMemcpyFromSymbol(out, g_timeline, sizeof(g_timeline));
  cudaMemcpyFromSymbol(n, g_timeline_n, sizeof(g_timeline_n));
  int z[4] = {0, 0, 0, 0};
  cudaMemcpyToSymbol(g_timeline_n, z, sizeof(z));
  return 0;
}
#endif

cudaError_t launch_tc_forward_main(const Args& a, cudaStream_t s, bool after_states) {
  FMaps tm;
  if (!make_user_map(&tm.q, a.q, a.T, a.H_q, a.B, a.layout) || !make_user_map(&tm.k, a.k, a.Tk, a.H_kv, a.B, a.kv_layout) ||
      !make_user_map(&tm.v, a.v, a.Tk, a.H_kv, a.B, a.kv_layout) || !make_user_map(&tm.out, a.out, a.T, a.H_q, a.B, a.layout) ||
      !make_state_map(&tm.st, a.chunk_state, a.k, (uint64_t)a.B * a.H_kv * a.n_chunks) ||
      !make_map(&tm.o_swa, a.o_swa ? (const void*)a.o_swa : a.out, a.T, (uint64_t)a.B * a.H_q) ||
      !make_map(&tm.o_rla, a.o_rla ? (const void*)a.o_rla : a.out, a.T, (uint64_t)a.B * a.H_q))
    return cudaErrorInvalidValue;
  int dev = 0, n_sm = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  e = cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return e;
  FArgs t;
  t.lse = a.lse;
  t.o_swa = reinterpret_cast<__nv_bfloat16*>(a.o_swa);   // the fp32-sized regions of the workspace hold bf16 here
  t.o_rla = reinterpret_cast<__nv_bfloat16*>(a.o_rla);
  t.gamma_swa = a.gamma_swa; t.gamma_rla = a.gamma_rla; t.status = a.status;
  t.T = a.T; t.w = a.w; t.H_q = a.H_q; t.group = a.group; t.mode = a.mode; t.n_chunks = a.n_chunks;
  t.n_qt = (a.T + TILE - 1) / TILE;
  t.n_pairs = (t.n_qt + 1) / 2;
  t.n_bh = a.B * a.H_q;
  t.n_units = t.n_pairs * t.n_bh;
  t.scale_log2 = a.scale * LOG2E; t.eps = a.eps;
  t.phi = a.phi;
  t.off = a.q_off / TILE;
  t.first_state = a.state_in ? 0 : 1;
  t.seq_lens = a.seq_lens;
  // pairs p with 2p - w/128 <= 0 read no stored state (a resumed sequence has none: every tile reads one)
  t.n_stateless = 0;
  // ... which pays when the chunk-state kernel leaves many SMs free for them (it runs one CTA per K/V head)
  const int order = tuning(RATTN_TUNE_UNIT_ORDER);
  const bool stateless_first = order == 1 || (order == 0 && 2 * a.B * a.H_kv <= n_sm);
  if (a.mode == RATTN_MODE_RATTN && after_states && !a.state_in && stateless_first) {
    t.n_stateless = (a.w / TILE) / 2 + 1;
    if (t.n_stateless > t.n_pairs) t.n_stateless = t.n_pairs;
  }
  t.wait_for_states = after_states ? 1 : 0;
  t.state_ready = (after_states && a.mode == RATTN_MODE_RATTN) ? a.state_ready : nullptr;
  // with per-head progress words the units can follow the chain; worth it where the order above would
  // have put the units without a state first anyway (few K/V heads, many SMs free beside the chain)
  t.ascending = (t.state_ready && t.n_stateless > 0) ? 1 : 0;
  t.debug_skip_arrive = debug_skip_arrive();
  t.work_counter = (a.status && order != 3) ? a.status + 2 : nullptr;
  e = cudaFuncSetAttribute(tc_fwd2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, F_SMEM);
  if (e != cudaSuccess) return e;
  if (tuning(RATTN_TUNE_GRID) > 0 && tuning(RATTN_TUNE_GRID) < n_sm) n_sm = tuning(RATTN_TUNE_GRID);
  const int grid = t.n_units < n_sm ? t.n_units : n_sm;
  {
    KernelTimer kt("tc_fwd", s);
    // Programmatic dependent launch: when a chunk-state kernel precedes it on the stream, this
    // kernel may begin while that one is still running; its loader waits (griddepcontrol.wait)
    // before the first state load.  Without a preceding state kernel the attribute changes nothing.
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(F_THREADS);
    cfg.dynamicSmemBytes = F_SMEM;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = (after_states && tuning(RATTN_TUNE_OVERLAP)) ? 1 : 0;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, tc_fwd2_kernel, tm, t);
    if (e != cudaSuccess) return e;
  }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace rattn
