// Chunk states of the linear branch, one pass (sm_100a: TMA + tcgen05 + TMEM).
//
// Forward (Eq. 2 of the paper, chunk C = 128):  S_[c+1] = S_[c] + phi(K_c)^T V_c,  S_[0] = 0.
// Backward, the mirror image over query tiles:   R_c = sum_{i > c + w/128} sum_heads phi(Q_i)^T g_r,i.
// Both are running sums of 128 x 128 outer-product blocks along the sequence, so one kernel
// serves both: a CTA owns one K/V head, walks the chunks in order and keeps the running sum in
// TMEM (fp32).  The sum leaves as bf16 (the operand type of the products that read it) after
// every `store_every`-th chunk -- the paper's "states stored every m chunks" -- and, when the
// caller wants the decode state, once more in fp32 at the end.  phi (softmax over the head
// features, Section 3.1) is applied to the loaded tile in shared memory.
//
// The chain is a pipeline of four roles, so that a step costs little more than its slowest
// stage (the feature map, bound by the exponential unit):
//   loader warp    TMA: X and Y tiles of the next chunks into a ring of three stages
//   8 phi warps    feature map of the X tile in place, two lanes per row
//   MMA warp       acc += phi(X)^T Y as soon as the tile is mapped
//   4 flush warps  after a stored step: accumulator -> registers (the MMA warp goes on as soon as
//                  the TMEM loads have landed) -> bf16 -> staging tile -> TMA store
#include <climits>

#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

constexpr int ST_NS = 3;                                   // ring stages
constexpr int ST_STAGE = 2 * TILE_BYTES;                   // X tile + Y tile
constexpr int ST_OFF_OUT = ST_NS * ST_STAGE;               // staging for one [128 x 128] bf16 matrix
constexpr int ST_OFF_BAR = ST_OFF_OUT + TILE_BYTES;
constexpr int ST_SMEM = ST_OFF_BAR + 128;
constexpr int ST_THREADS = 448;                            // 8 phi warps, MMA warp, loader warp, 4 flush warps

struct StateArgs {
  int n_steps;      // chunks to walk
  int first, dir;   // chunk index of step s: first + dir * s
  int group;        // heads summed per chunk (X/Y matrix index = kv * group + head)
  int out_first;    // output matrix of step s: kv * n_chunks + out_first + dir * s
  int n_chunks;
  int store_every;  // the sum after step s is stored iff (out_first + dir * s) % store_every == store_phase
  int store_phase;
  int handoff;      // forward chain that also yields the decode state (see StateLaunch)
  int T, w;         // rows per head in memory, window
  float* final_out; // optional fp32 [n_kv, 128, 128]: the sum after the last step
  const float* state_in;   // optional fp32 [n_kv, 128, 128]: the sum starts from it; matrix out_first - dir holds it
  const int* seq_lens;     // optional: valid rows per batch entry
  int kv_per_batch;
  int phi;          // rattn_feature_map
  int* status;
  int* ready;       // optional [n_kv]: number of leading output matrices stored so far (forward chain)
};

struct StBars {
  uint64_t full[ST_NS], phi_ready[ST_NS], free_[ST_NS], done, acc_free;
  uint32_t tmem_base;
  int abort;
};

__device__ __forceinline__ bool stored_step(const StateArgs& a, int s) {
  const int o = a.out_first + a.dir * s;
  return o >= 0 && (o % a.store_every) == a.store_phase;
}
__device__ __forceinline__ bool flushed_step(const StateArgs& a, int s, int n_steps) {
  return stored_step(a, s) || (a.final_out != nullptr && s == n_steps - 1);
}

__global__ void __launch_bounds__(ST_THREADS, 1)
tc_state_scan_kernel(const __grid_constant__ UMap tm_x, const __grid_constant__ UMap tm_y,
                     const __grid_constant__ CUtensorMap tm_out, StateArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  StBars* bars = reinterpret_cast<StBars*>(smem + ST_OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int kv = blockIdx.x;
  // the kernel that follows may start its own prologue (and whatever does not read the states)
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0 && a.status) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < ST_NS; ++i) {
      mbar_init(&bars->full[i], 1);
      mbar_init(&bars->phi_ready[i], 256);
      mbar_init(&bars->free_[i], 1);
    }
    mbar_init(&bars->done, 1);
    mbar_init(&bars->acc_free, 128);
    bars->abort = 0;
    fence_mbar_init();
  }
  if (warp == 8) {
    tmem_alloc(&bars->tmem_base, 128);
    tmem_relinquish();
  }
  if (tid == 288) {
    prefetch_map(&tm_x);
    prefetch_map(&tm_y);
    prefetch_tensormap(&tm_out);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = bars->tmem_base;
  // this head's chain: the caller's step count, or -- variable-length batches -- what the entry's own
  // length asks for; with the hand-off the tokens from len - w on are still inside the window
  int n_steps = a.n_steps, row_limit = INT_MAX;
  {
    const int len = a.seq_lens ? min(a.T, a.seq_lens[kv / a.kv_per_batch]) : a.T;
    if (a.seq_lens) {
      const int nd = max(0, (len + TILE - 1) / TILE - 1 - a.w / TILE);
      n_steps = (a.handoff && len > a.w) ? nd + 1 : nd;
    }
    if (a.handoff) row_limit = len - a.w;
  }
  const bool has_init = (a.state_in != nullptr);
  const int n_items = n_steps * a.group;
  bool ok = true;

  if (warp < 8) {
    // ---- feature map of the X tile, in place: two adjacent lanes per row ------------------
    for (int it = 0; it < n_items && ok; ++it) {
      const int st = it % ST_NS, use = it / ST_NS;
      ok = mbar_wait(&bars->full[st], use & 1, &bars->abort);
      if (!ok) break;
      unsigned char* xh = smem + st * ST_STAGE + (tid & 1) * HALF_BYTES;
      const int row = tid >> 1;
      const int token = (a.first + a.dir * (it / a.group)) * TILE + row;
      // every lane maps its row (the softmax map exchanges partial results between the two lanes
      // of a row with full-warp shuffles, so no lane may skip it); rows past the limit are then cleared
      feature_map_pair_any(xh, xh, row, a.phi);
      if (token >= row_limit) {
#pragma unroll
        for (int c = 0; c < 8; ++c) *reinterpret_cast<uint4*>(xh + row * 128 + (c << 4)) = make_uint4(0, 0, 0, 0);
      }
      fence_proxy_async_smem();
      mbar_arrive(&bars->phi_ready[st]);
    }
  } else if (warp == 8) {
    // ---- acc[128 features x 128] += phi(X)^T Y   (both operands MN-major: rows are the tokens)
    int n_wait = 0;                                          // hand-backs of the accumulator so far
    for (int it = 0; it < n_items && ok; ++it) {
      const int st = it % ST_NS, use = it / ST_NS;
      const int s = it / a.group, hh = it - s * a.group;
      ok = mbar_wait_warp(&bars->phi_ready[st], use & 1, &bars->abort);
      // the flush warps hold the previous sum, or are still writing the incoming state into the accumulator
      if (ok && hh == 0 && ((s > 0 && flushed_step(a, s - 1, n_steps)) || (s == 0 && has_init))) {
        ok = mbar_wait_warp(&bars->acc_free, n_wait & 1, &bars->abort);
        ++n_wait;
      }
      if (!ok) break;
      tc_fence_after();
      mma_mnmn(tmem, smem_u32(smem + st * ST_STAGE), smem_u32(smem + st * ST_STAGE + TILE_BYTES), it > 0 || has_init);
      mma_commit(&bars->free_[st]);
      if (hh == a.group - 1 && flushed_step(a, s, n_steps)) mma_commit(&bars->done);
    }
  } else if (warp == 9) {
    // ---- loader ---------------------------------------------------------------------------
    for (int it = 0; it < n_items && ok; ++it) {
      const int st = it % ST_NS, use = it / ST_NS;
      const int s = it / a.group, hh = it - s * a.group;
      if (use >= 1) ok = mbar_wait_warp(&bars->free_[st], (use - 1) & 1, &bars->abort);
      if (!ok) break;
      const int row = (a.first + a.dir * s) * TILE, z = kv * a.group + hh;
      unsigned char* dst = smem + st * ST_STAGE;
      mbar_arrive_expect_tx(&bars->full[st], ST_STAGE);
      load_tile(dst, &tm_x, &bars->full[st], row, z);
      load_tile(dst + TILE_BYTES, &tm_y, &bars->full[st], row, z);
    }
  } else {
    // ---- flush: thread = accumulator row (its warp's TMEM lane quarter) --------------------
    const int r = (warp & 3) * 32 + (tid & 31);
    const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    unsigned char* s_out = smem + ST_OFF_OUT;
    const bool issuer = (tid == 320);
    int n_flush = 0;
    // bf16 copy of this thread's row of the sum -> staging -> matrix `mat` of the head, one TMA store
    int pending = 0;                                         // matrices stored, not yet published
    auto publish = [&]() {
      tma_store_wait();
      fence_proxy_async_all();
      __threadfence();
      st_release_gpu(a.ready + kv, pending);
      pending = 0;
    };
    auto store_row = [&](const float (&x)[4][32], int mat) {
      if (issuer) {
        // The kernel that reads the states runs beside this one and takes them as they appear.  The
        // matrix stored last is published here, one flush later, when its store has long completed
        // (it must be in memory, not merely read out of the staging tile, before its index is shown).
        if (a.ready && pending) publish();
        else tma_store_wait_read();                          // the staging tile has left
      }
      asm volatile("bar.sync 4, 128;" ::: "memory");
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          uint4 u;
          u.x = pack_bf16(x[c][8 * e + 0], x[c][8 * e + 1]);
          u.y = pack_bf16(x[c][8 * e + 2], x[c][8 * e + 3]);
          u.z = pack_bf16(x[c][8 * e + 4], x[c][8 * e + 5]);
          u.w = pack_bf16(x[c][8 * e + 6], x[c][8 * e + 7]);
          *reinterpret_cast<uint4*>(s_out + swz(r, 4 * c + e)) = u;
        }
      }
      fence_proxy_async_smem();
      asm volatile("bar.sync 4, 128;" ::: "memory");
      if (issuer) {
        store_tile(&tm_out, s_out, 0, kv * a.n_chunks + mat);
        tma_store_commit();
        pending = mat + 1;
      }
    };
    auto write_final = [&](const float (&x)[4][32]) {
      float* dst = a.final_out + ((size_t)kv * 128 + r) * 128;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 8; ++e)
          *reinterpret_cast<float4*>(dst + 32 * c + 4 * e) =
              make_float4(x[c][4 * e], x[c][4 * e + 1], x[c][4 * e + 2], x[c][4 * e + 3]);
      }
    };
    if (has_init || (a.final_out != nullptr && n_steps == 0)) {
      // the chain starts from the incoming state (zero without one): into the accumulator, into the
      // matrix in front of the first step's, and -- when no token leaves the window -- straight out
      float x[4][32];
      const float* src = has_init ? a.state_in + ((size_t)kv * 128 + r) * 128 : nullptr;
#pragma unroll
      for (int c = 0; c < 4; ++c) {
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const float4 f = src ? *reinterpret_cast<const float4*>(src + 32 * c + 4 * e) : make_float4(0.f, 0.f, 0.f, 0.f);
          x[c][4 * e] = f.x; x[c][4 * e + 1] = f.y; x[c][4 * e + 2] = f.z; x[c][4 * e + 3] = f.w;
        }
      }
      if (has_init) {
#pragma unroll
        for (int c = 0; c < 4; ++c) tmem_st32(t_row + 32 * c, x[c]);
        tmem_wait_st();
        tc_fence_before();
        mbar_arrive(&bars->acc_free);
        if (stored_step(a, -1)) store_row(x, a.out_first - a.dir);
      }
      if (a.final_out != nullptr && n_steps == 0) write_final(x);
    }
    for (int s = 0; s < n_steps && ok; ++s) {
      if (!flushed_step(a, s, n_steps)) continue;
      ok = mbar_wait(&bars->done, n_flush & 1, &bars->abort);
      ++n_flush;
      if (!ok) break;
      tc_fence_after();
      float x[4][32];
#pragma unroll
      for (int c = 0; c < 4; ++c) tmem_ld32(t_row + 32 * c, x[c]);
      tmem_wait_ld();
      tc_fence_before();
      mbar_arrive(&bars->acc_free);                            // the next step may accumulate
      if (stored_step(a, s)) store_row(x, a.out_first + a.dir * s);
      if (a.final_out != nullptr && s == n_steps - 1) write_final(x);
    }
    if (issuer) {
      if (a.ready && pending) publish();
      else tma_store_wait();
    }
  }
  if (!ok && a.status) atomicExch(a.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 8) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

}  // namespace

// x, y: [n_kv * group, T, 128] bf16; out: [n_kv * n_chunks, 128, 128] bf16.
cudaError_t launch_tc_states(const StateLaunch& L, cudaStream_t s) {
  if (L.n_steps <= 0 && !L.state_in && !(L.seq_lens && L.final_out)) return cudaSuccess;
  UMap tm_x, tm_y;
  CUtensorMap tm_out;
  const uint64_t n_mats = (uint64_t)L.n_kv * L.group;
  auto user = [&](UMap* m, const void* base, int heads, int layout) {
    return heads > 0 ? make_user_map(m, base, L.T, heads, n_mats / heads, layout) : make_user_map(m, base, L.T, n_mats, 1, 0);
  };
  if (!user(&tm_x, L.x, L.x_heads, L.x_layout) || !user(&tm_y, L.y, L.y_heads, L.y_layout) ||
      !make_map(&tm_out, L.out, 128, (uint64_t)L.n_kv * L.n_chunks))
    return cudaErrorInvalidValue;
  StateArgs a;
  a.n_steps = L.n_steps; a.first = L.first; a.dir = L.dir; a.group = L.group; a.out_first = L.out_first;
  a.n_chunks = L.n_chunks; a.status = L.status;
  a.store_every = L.store_every > 0 ? L.store_every : 1;
  a.store_phase = L.store_phase;
  a.handoff = L.handoff; a.T = L.T; a.w = L.w;
  a.final_out = L.final_out;
  a.state_in = L.state_in;
  a.seq_lens = L.seq_lens; a.kv_per_batch = L.kv_per_batch > 0 ? L.kv_per_batch : 1;
  a.phi = L.phi;
  a.ready = (L.dir > 0 && L.group == 1) ? L.ready : nullptr;
  cudaError_t e = cudaFuncSetAttribute(tc_state_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM);
  if (e != cudaSuccess) return e;
  {
    KernelTimer kt(L.name, s);
    tc_state_scan_kernel<<<L.n_kv, ST_THREADS, ST_SMEM, s>>>(tm_x, tm_y, tm_out, a);
  }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace rattn
