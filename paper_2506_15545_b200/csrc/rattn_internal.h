// Internal declarations shared by the translation units of librattn.so.
// Nothing here is part of the public ABI (include/rattn.h).
#pragma once

#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stddef.h>
#include <stdint.h>

#include "rattn.h"

namespace rattn {

// Byte offsets inside the caller's workspace.  Every region is 256-byte aligned; a region the
// call's mode and flags do not need has offset kAbsent and takes no room.
struct WorkspaceLayout {
  size_t status;        // 256 bytes; word 0 = device status, word 1 = detail code; behind it, on the tensor-core
                        // path with a linear branch, one progress word per K/V head (status_bytes in all)
  size_t status_bytes;  // what a forward clears before its kernels
  size_t lse;           // fp32 [B,H_q,T]      log-sum-exp of the SWA logits (natural log)
  size_t o_swa;         // fp32 [B,H_q,T,d]    un-normalised SWA branch output (bf16 on the tensor-core path)
  size_t o_rla;         // fp32 [B,H_q,T,d]    un-normalised RLA branch output (likewise)
  size_t do_swa;        // fp32 [B,H_q,T,d]    backward scratch (the tensor-core path keeps bf16 there)
  size_t do_rla;        // fp32 [B,H_q,T,d]    backward scratch (likewise)
  size_t delta;         // fp32 [B,H_q,T]      backward scratch
  size_t chunk_state;   // bf16 [B,H_kv,n_chunks,d,d]  exclusive prefix over chunks
  size_t rstate;        // bf16 [B,H_kv,n_chunks,d,d]  backward: suffix sums of phi(Q)^T g_r
  size_t lse2p;         // fp32 [B*H_q, n_chunks*128]  backward: lse * log2(e), +inf in the padding
  size_t dscp;          // fp32 [B*H_q, n_chunks*128]  backward: D_t * scale, 0 in the padding
  size_t k_ext;         // I/O type [B,H_kv,w+T,d]  chunked prefill: history + chunk keys, in time order
  size_t v_ext;         //                          ... values
  size_t total;
  int n_chunks;         // ceil(T / 128)
};

// Offset of a region the call does not use.
constexpr size_t kAbsent = ~(size_t)0;

// T: query rows of the call; history: 1 when the call resumes a sequence (chunked prefill)
WorkspaceLayout workspace_layout(int B, int H_q, int H_kv, int T, int d, int w, int dtype, int mode,
                                 unsigned flags, int history = 0);

// Resolved arguments handed to the kernel launchers (all device pointers).
struct Args {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int B, H_q, H_kv, T, d, w;   // w already replaced by T for FULL_CAUSAL
  // Chunked prefill: k, v then point at the history (the w tokens before the chunk, in time
  // order) followed by the chunk, Tk = w + T rows per head, and query row t sits at key
  // position t + q_off (q_off = w); state_in holds the sum over the tokens before the history.
  // A fresh sequence has Tk = T, q_off = 0, state_in = null.
  int Tk, q_off;
  const float* state_in;
  const int* seq_lens;         // optional device [B]: valid tokens of each batch entry (fresh sequences only)
  int pos_shift;               // sequence position of key row 0 (pos0 - w for a resumed sequence, else 0)
  int group;                   // H_q / H_kv
  int dtype, mode;
  unsigned flags;              // rattn_params.flags
  int layout;                  // rattn_layout of q, out, dout, dq (and of k, v, dk, dv unless kv_layout says otherwise)
  int kv_layout;               // layout of the k, v the kernels read: dense when they are the gathered history + chunk
  int phi;                     // rattn_feature_map
  float scale, eps;
  const float* gamma_swa;
  const float* gamma_rla;
  // residuals (may be null in inference mode)
  float* lse;
  float* o_swa;
  float* o_rla;
  // tensor-path scratch
  __nv_bfloat16* chunk_state;
  __nv_bfloat16* rstate;
  float* lse2p;
  float* dscp;
  int n_chunks;
  int* status;                 // device status block (may be null when no workspace): word 0 status,
                               // word 1 detail, word 2 the forward's work counter
  int* state_ready;            // [B*H_kv], zero at launch: chunk states the chunk-state kernel has stored so far
                               // (null: the main kernel waits for that whole kernel instead)
  bool training;               // the backward will read every chunk state
  // hand-off
  float* state_out;
  void* k_ring_out;
  void* v_ring_out;
  // backward
  const void* dout;
  void* dq;
  void* dk;
  void* dv;
  float* dgamma_swa;
  float* dgamma_rla;
  float* do_swa;               // fp32 [B,H_q,T,d]  gradient w.r.t. the SWA branch output
  float* do_rla;               // fp32 [B,H_q,T,d]  gradient w.r.t. the RLA branch output
  float* delta;                // fp32 [B,H_q,T]    do_swa . o_swa per row
};

// Launchers; each returns the cudaError_t of its launches (cudaGetLastError).
cudaError_t launch_generic_forward(const Args& a, cudaStream_t s);
cudaError_t launch_generic_backward(const Args& a, cudaStream_t s);
cudaError_t launch_decode(const Args& a, void* k_ring, void* v_ring, float* state, int pos, const int* pos_dev,
                          cudaStream_t s);
// The TMA-staged decode step (bf16, d = 128, w a multiple of 64, groups of up to 8 heads) and
// its status word (RATTN_ERR_TIMEOUT once a bounded wait has expired; reading clears it).
bool decode_tc_applies(const Args& a, int w);
cudaError_t launch_decode_tc(const Args& a, void* k_ring, void* v_ring, float* state, int pos, const int* pos_dev,
                             cudaStream_t s);
int decode_tc_status(cudaStream_t s, cudaError_t* err);
// prefill -> decode hand-off: the rings, and (state_too) the state by the portable kernel
cudaError_t launch_handoff(const Args& a, cudaStream_t s, bool state_too);
cudaError_t launch_tc_forward(const Args& a, cudaStream_t s);        // chunk states, then the main kernel
// after_states: a chunk-state kernel was launched just before on the same stream
cudaError_t launch_tc_forward_main(const Args& a, cudaStream_t s, bool after_states);
// Running sums of phi(X_c)^T Y_c over the chunks first, first+dir, ... (n_steps of them) for every
// K/V head (tc_state.cu).  The sum after step s goes, as bf16, to matrix out_first + dir*s of the
// head when that index is congruent to store_phase modulo store_every.  With `handoff` the chain
// is the forward's and also yields the decode state: per head it walks ceil((len - w) / 128) chunks
// (len = T, or the batch entry's own length), tokens at positions >= len - w contribute nothing,
// and the final sum goes to final_out in fp32.
struct StateLaunch {
  const void* x;            // [n_kv * group, T, 128] bf16, mapped through phi
  const void* y;            // [n_kv * group, T, 128] bf16
  // x and y as the caller's tensors: heads per batch entry and head layout (rattn_layout); 0 heads = a dense
  // internal tensor of n_kv * group matrices
  int x_heads, x_layout, y_heads, y_layout;
  void* out;                // [n_kv * n_chunks, 128, 128] bf16
  int T, n_kv, group, n_chunks;
  int n_steps, first, dir, out_first;
  int store_every, store_phase;
  int handoff;              // 1: the chain ends with the decode state (tokens before len - w, len = T or the
  int w;                    //    entry's own length), left in final_out; the step count follows the length
  float* final_out;
  const float* state_in;    // optional fp32 [n_kv,128,128]: the sum starts from it and matrix 0 holds it
  const int* seq_lens;      // optional [n_kv / kv_per_batch]: valid rows of each batch entry
  int kv_per_batch;
  int phi;                  // rattn_feature_map applied to x
  int* status;
  int* ready;               // optional [n_kv] (forward chain): matrices stored so far, published after each store
  const char* name;         // label of the timing record
};
cudaError_t launch_tc_states(const StateLaunch& L, cudaStream_t s);
cudaError_t launch_tc_backward(const Args& a, cudaStream_t s);
// chunked prefill: k_ext/v_ext[b,hk] = the ring's tokens pos0-w .. pos0-1 in time order, then the chunk
cudaError_t launch_gather_history(const Args& a, const void* k_chunk, const void* v_chunk, const void* k_ring,
                                  const void* v_ring, void* k_ext, void* v_ext, int pos0, cudaStream_t s);

int debug_skip_arrive();                    // always 0 outside the debug build
int tuning(int knob);                       // current value of a rattn_knob
void count_launches(int n);
void set_last_cuda_error(int cuda_error);   // what rattn_last_cuda_error() reports for this thread

// Records a CUDA event pair around one kernel launch on its stream while per-kernel
// timing is enabled (rattn_timing_enable); free otherwise.
class KernelTimer {
 public:
  KernelTimer(const char* name, cudaStream_t s);
  ~KernelTimer();
 private:
  cudaStream_t stream_;
  int slot_;
};

}  // namespace rattn
