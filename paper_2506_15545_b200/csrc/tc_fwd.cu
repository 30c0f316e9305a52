// Tensor-core forward for bf16, d = 128, window a multiple of 128: the chunk states of the linear
// branch first, then the main kernel (tc_fwd2.cu).
//
// Chunk states S_[c] = sum_{c' < c} phi(K_c')^T V_c' (Eq. 2), two ways:
//   many K/V heads   one CTA per head walks the chunks with the sum in TMEM (tc_state.cu): no
//                    fp32 blocks in HBM, but a serial chain as long as the sequence;
//   few K/V heads    one CTA per (chunk, head) computes phi(K_c)^T V_c in parallel (fp32 to HBM),
//                    then a prefix-sum kernel: more traffic, a much shorter critical path.
#include "tc_common.cuh"

namespace rattn {
namespace {

using namespace ptx;
using namespace tc;

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
  const int n_qt = (a.T + TILE - 1) / TILE;
  // S_[c] for c = 1 .. n_delta: the states some query tile reads (S_[0] = 0 is never read)
  const int n_delta = (a.mode == RATTN_MODE_RATTN) ? n_qt - 1 - a.w / TILE : 0;
  const int n_kv = a.B * a.H_kv;
  cudaError_t e = cudaSuccess;
  if (n_delta > 0 && n_kv < 64 && a.chunk_delta) {
    CUtensorMap tm_k, tm_v;
    if (!make_map(&tm_k, a.k, a.T, (uint64_t)n_kv)) return cudaErrorInvalidValue;
    if (!make_map(&tm_v, a.v, a.T, (uint64_t)n_kv)) return cudaErrorInvalidValue;
    e = cudaFuncSetAttribute(tc_chunk_delta_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, CS_SMEM);
    if (e != cudaSuccess) return e;
    {
      KernelTimer kt("tc_chunk_delta", s);
      tc_chunk_delta_kernel<<<dim3(n_delta, n_kv), 128, CS_SMEM, s>>>(tm_k, tm_v, a.chunk_delta, a.n_chunks, a.status);
    }
    {
      KernelTimer kt("tc_chunk_scan", s);
      tc_chunk_scan_kernel<<<dim3(n_kv, 16), 256, 0, s>>>(a.chunk_delta, a.chunk_state, a.n_chunks, n_delta);
    }
    count_launches(2);
    e = cudaGetLastError();
  } else {
    e = launch_tc_states(a.k, a.v, a.chunk_state, a.T, n_kv, 1, a.n_chunks, n_delta, 0, +1, 1, a.status,
                         "tc_state_fwd", s);
  }
  if (e != cudaSuccess) return e;
  return launch_tc_forward_main(a, s);
}

}  // namespace rattn
