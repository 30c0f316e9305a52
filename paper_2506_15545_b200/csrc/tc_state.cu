// Chunk states of the linear branch, one pass (sm_100a: TMA + tcgen05 + TMEM).
//
// Forward (Eq. 2 of the paper, chunk C = 128):  S_[c+1] = S_[c] + phi(K_c)^T V_c,  S_[0] = 0.
// Backward, the mirror image over query tiles:   R_c = sum_{i > c + w/128} sum_heads phi(Q_i)^T g_r,i.
// Both are running sums of 128 x 128 outer-product blocks along the sequence, so one kernel
// serves both: a CTA (256 threads) owns one K/V head, walks the chunks in order, keeps the
// running sum in TMEM (fp32) and writes it out after every chunk in bf16, the operand type of
// the products that read it.  Compared with "one block
// per chunk, then a prefix-sum kernel" this never writes the fp32 blocks to HBM.  phi (softmax
// over the head features, Section 3.1) is applied to the loaded tile in shared memory.
#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

constexpr int ST_STAGE = 2 * TILE_BYTES;                   // X tile + Y tile
constexpr int ST_OFF_OUT = 2 * ST_STAGE;                   // staging for one [128 x 128] bf16 matrix
constexpr int ST_OFF_BAR = ST_OFF_OUT + TILE_BYTES;
constexpr int ST_SMEM = ST_OFF_BAR + 64;

struct StateArgs {
  int n_steps;      // chunks to walk
  int first, dir;   // chunk index of step s: first + dir * s
  int group;        // heads summed per chunk (X/Y matrix index = kv * group + head)
  int out_first;    // output matrix of step s: kv * n_chunks + out_first + dir * s
  int n_chunks;
  int* status;
};

struct StBars {
  uint64_t full[2], free_[2], done;
  uint32_t tmem_base;
  int abort;
};

__global__ void __launch_bounds__(256)
tc_state_scan_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_y,
                     const __grid_constant__ CUtensorMap tm_out, StateArgs a) {
  extern __shared__ __align__(1024) unsigned char smem[];
  StBars* bars = reinterpret_cast<StBars*>(smem + ST_OFF_BAR);
  const int tid = threadIdx.x, warp = tid >> 5;
  const int kv = blockIdx.x;
  if ((smem_u32(smem) & 1023u) != 0) {
    if (tid == 0 && a.status) atomicExch(a.status, 2);
    return;
  }
  if (tid == 0) {
    for (int i = 0; i < 2; ++i) {
      mbar_init(&bars->full[i], 1);
      mbar_init(&bars->free_[i], 1);
    }
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
  const int r = tid & 127, ch = tid >> 7;                   // accumulator row and column half of this thread
  const uint32_t t_row = tmem + ((uint32_t)((warp & 3) * 32) << 16) + 64 * ch;
  unsigned char* s_out = smem + ST_OFF_OUT;
  const int n_items = a.n_steps * a.group;

  auto load_item = [&](int it) {                           // warp 0, converged
    const int s = it / a.group, hh = it - s * a.group, st = it & 1;
    const int row = (a.first + a.dir * s) * TILE, z = kv * a.group + hh;
    unsigned char* dst = smem + st * ST_STAGE;
    mbar_arrive_expect_tx(&bars->full[st], ST_STAGE);
    load_tile(dst, &tm_x, &bars->full[st], row, z);
    load_tile(dst + TILE_BYTES, &tm_y, &bars->full[st], row, z);
  };
  // running sum after step s -> bf16 -> staging (every thread its row)
  auto stage_sum = [&]() {
#pragma unroll
    for (int c = 0; c < 2; ++c) {
      float x[32];
      tmem_ld32(t_row + 32 * c, x);
      tmem_wait_ld();
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        uint4 u;
        u.x = pack_bf16(x[8 * e + 0], x[8 * e + 1]);
        u.y = pack_bf16(x[8 * e + 2], x[8 * e + 3]);
        u.z = pack_bf16(x[8 * e + 4], x[8 * e + 5]);
        u.w = pack_bf16(x[8 * e + 6], x[8 * e + 7]);
        *reinterpret_cast<uint4*>(s_out + swz(r, 8 * ch + 4 * c + e)) = u;
      }
    }
    fence_proxy_async_smem();
    tc_fence_before();
  };

  if (warp == 0 && n_items > 0) load_item(0);
  bool ok = true;
  for (int it = 0; it < n_items; ++it) {
    const int s = it / a.group, hh = it - s * a.group, st = it & 1;
    if (warp == 0 && it + 1 < n_items) {
      // the other stage is free once the product of item it-1 has completed
      if (it >= 1) ok = mbar_wait_warp(&bars->free_[(it + 1) & 1], ((it - 1) >> 1) & 1, &bars->abort) && ok;
      load_item(it + 1);
    }
    ok = mbar_wait(&bars->full[st], (it >> 1) & 1, &bars->abort) && ok;
    // phi of the chunk's tokens: two adjacent lanes per row, each one column half
    feature_map_pair(smem + st * ST_STAGE + (tid & 1) * HALF_BYTES, smem + st * ST_STAGE + (tid & 1) * HALF_BYTES, tid >> 1);
    fence_proxy_async_smem();
    const bool flush = (hh == 0 && s > 0);
    if (flush) {
      // the sum after step s-1 leaves before this step's first product touches the accumulator
      if (tid == 0) tma_store_wait_read();                       // staging free again
      ok = mbar_wait(&bars->done, (s - 1) & 1, &bars->abort) && ok;
      __syncthreads();
      tc_fence_after();
      stage_sum();
    }
    __syncthreads();
    if (warp == 0) {
      if (flush && tid == 0) {
        store_tile(&tm_out, s_out, 0, kv * a.n_chunks + a.out_first + a.dir * (s - 1));
        tma_store_commit();
      }
      __syncwarp();
      tc_fence_after();
      // acc[128 features x 128] += phi(X)^T Y   (both operands MN-major: rows are the tokens)
      mma_mnmn(tmem, smem_u32(smem + st * ST_STAGE), smem_u32(smem + st * ST_STAGE + TILE_BYTES), it > 0);
      mma_commit(&bars->free_[st]);
      if (hh == a.group - 1) mma_commit(&bars->done);
    }
  }
  if (n_items > 0) {
    if (tid == 0) tma_store_wait_read();
    ok = mbar_wait(&bars->done, (a.n_steps - 1) & 1, &bars->abort) && ok;
    __syncthreads();
    tc_fence_after();
    stage_sum();
    __syncthreads();
    if (tid == 0) {
      store_tile(&tm_out, s_out, 0, kv * a.n_chunks + a.out_first + a.dir * (a.n_steps - 1));
      tma_store_commit();
      tma_store_wait_read();
    }
  }
  if (!ok && a.status) atomicExch(a.status, 1);
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

}  // namespace

// x, y: [n_kv * group, T, 128] bf16; out: [n_kv * n_chunks, 128, 128] bf16.
cudaError_t launch_tc_states(const void* x, const void* y, void* out, int T, int n_kv, int group, int n_chunks,
                             int n_steps, int first, int dir, int out_first, int* status, const char* name,
                             cudaStream_t s) {
  if (n_steps <= 0) return cudaSuccess;
  CUtensorMap tm_x, tm_y, tm_out;
  if (!make_map(&tm_x, x, T, (uint64_t)n_kv * group) || !make_map(&tm_y, y, T, (uint64_t)n_kv * group) ||
      !make_map(&tm_out, out, 128, (uint64_t)n_kv * n_chunks))
    return cudaErrorInvalidValue;
  StateArgs a;
  a.n_steps = n_steps; a.first = first; a.dir = dir; a.group = group; a.out_first = out_first;
  a.n_chunks = n_chunks; a.status = status;
  cudaError_t e = cudaFuncSetAttribute(tc_state_scan_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ST_SMEM);
  if (e != cudaSuccess) return e;
  {
    KernelTimer kt(name, s);
    tc_state_scan_kernel<<<n_kv, 256, ST_SMEM, s>>>(tm_x, tm_y, tm_out, a);
  }
  count_launches(1);
  return cudaGetLastError();
}

}  // namespace rattn
