// Tensor-core forward for bf16, d = 128, window a multiple of 128: the chunk states of the linear
// branch first (tc_state.cu), then the main kernel (tc_fwd2.cu).
#include "tc_common.cuh"

namespace rattn {

cudaError_t launch_tc_forward(const Args& a, cudaStream_t s) {
  const int n_qt = (a.T + tc::TILE - 1) / tc::TILE;
  // S_[c] for c = 1 .. n_delta: the states some query tile reads (Eq. 2; S_[0] = 0 is never read)
  const int n_delta = (a.mode == RATTN_MODE_RATTN) ? n_qt - 1 - a.w / tc::TILE : 0;
  cudaError_t e = launch_tc_states(a.k, a.v, a.chunk_state, a.T, a.B * a.H_kv, 1, a.n_chunks, n_delta, 0, +1, 1,
                                   a.status, "tc_state_fwd", s);
  if (e != cudaSuccess) return e;
  return launch_tc_forward_main(a, s);
}

}  // namespace rattn
