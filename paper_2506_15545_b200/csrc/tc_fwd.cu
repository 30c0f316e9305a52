// Tensor-core forward for bf16, d = 128, window a multiple of 128: the chunk states of the linear
// branch first (tc_state.cu), then the main kernel (tc_fwd2.cu).
//
// Chunk states S_[c] = sum_{c' < c} phi(K_c')^T V_c' (Eq. 2): one CTA per K/V head walks the chunks
// with the sum in TMEM.  The main kernel reads S_[c] only for c = 2p - w/128 (one stored state serves
// a pair of query tiles), so an inference forward stores every second state -- the paper's "states
// stored every m chunks" with m = 2; a training forward stores all of them, because the backward
// reads one per query tile.  When the caller asks for the decode state, the chain runs one chunk
// further (tokens up to T - w, the rest of that chunk masked) and leaves its fp32 sum there.
// The main kernel is launched so that it may start while the chain still runs (programmatic
// dependent launch): its window loops need no state, and it waits for the chain only before its
// first state load.
#include "tc_common.cuh"

namespace rattn {

cudaError_t launch_tc_forward(const Args& a, cudaStream_t s) {
  // key-space tiles: a resumed sequence carries its w-token history in front of the chunk
  const int n_kt = (a.Tk + tc::TILE - 1) / tc::TILE;
  const int wt = a.w / tc::TILE, off = a.q_off / tc::TILE;
  const bool rla = (a.mode == RATTN_MODE_RATTN);
  // S_[c] for c = 1 .. n_delta: the states some query tile reads (S_[0] is the incoming state, zero
  // for a fresh sequence, where it is never read)
  const int n_delta = rla ? n_kt - 1 - wt : 0;
  const int n_kv = a.B * a.H_kv;
  const bool want_state = rla && a.state_out != nullptr;
  bool chained = false;
  // The main kernel can take the chunk states as the chain publishes them instead of waiting for the whole
  // chain.  That pays where the chain is long and leaves most SMs to the main kernel, which otherwise runs out
  // of work that needs no state (config 3: 16 chains of 64 chunks); elsewhere publishing only slows the chain.
  // With wide windows the units without a state are many and heavy already, and taking the units in sequence
  // order (light ones first) costs more at the tail than the earlier start gains (measured from w = 1024 on).
  bool progress = a.state_ready != nullptr;
  if (progress) {
    const int knob = tuning(RATTN_TUNE_STATE_PROGRESS);
    int dev = 0, n_sm = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
      n_sm = 0;
    progress = knob == 1 || (knob == 0 && 4 * n_kv <= n_sm && n_kt >= 48 && wt <= 4);
  }
  if (want_state && a.Tk <= a.w && !a.seq_lens) {
    // nothing has left the window yet
    cudaError_t e = cudaMemsetAsync(a.state_out, 0, sizeof(float) * (size_t)n_kv * 128 * 128, s);
    if (e != cudaSuccess) return e;
  }
  const int n_steps = (want_state && (a.Tk > a.w || a.seq_lens)) ? n_delta + 1 : n_delta;
  if (n_steps > 0 || (a.state_in && rla) || (a.seq_lens && want_state)) {
    StateLaunch L;
    L.x = a.k; L.y = a.v; L.out = a.chunk_state;
    L.x_heads = L.y_heads = a.H_kv; L.x_layout = L.y_layout = a.kv_layout;
    L.T = a.Tk; L.n_kv = n_kv; L.group = 1; L.n_chunks = a.n_chunks;
    L.n_steps = n_steps > 0 ? n_steps : 0; L.first = 0; L.dir = +1; L.out_first = 1;
    // the main kernel reads S_[c] for c = off + 2p - wt only
    const int m = tuning(RATTN_TUNE_STATE_STRIDE);
    const bool every = a.training || m == 1;
    L.store_every = every ? 1 : 2;
    L.store_phase = every ? 0 : ((off + wt) & 1);
    L.handoff = want_state ? 1 : 0;
    L.w = a.w;
    L.final_out = want_state ? a.state_out : nullptr;
    L.state_in = a.state_in;
    L.seq_lens = a.seq_lens; L.kv_per_batch = a.H_kv;
    L.phi = a.phi;
    L.status = a.status; L.name = "tc_state_fwd";
    L.ready = progress ? a.state_ready : nullptr;
    cudaError_t e = launch_tc_states(L, s);
    if (e != cudaSuccess) return e;
    chained = true;
  }
  Args m = a;
  if (!progress) m.state_ready = nullptr;            // the main kernel waits for the whole chain instead
  return launch_tc_forward_main(m, s, chained);
}

}  // namespace rattn
