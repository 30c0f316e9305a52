/*
 * rattn.h -- C ABI of the RAttention operator for NVIDIA B200 (sm_100a).
 *
 * The operator is one attention layer's token mixing (Section 3.2 of the paper):
 *
 *     y_t = rmsnorm(o_swa_t; g_swa) + rmsnorm(o_rla_t; g_rla)
 *
 *   o_swa_t = softmax attention of q_t over the keys max(0,t-w) <= j <= t   (Section 2.1)
 *   o_rla_t = phi(q_t) S_{t-w-1},  S_n = sum_{j<=n} phi(k_j)^T v_j          (Eq. 4)
 *   phi     = softmax over the d head features, d' = d                      (Section 3.1)
 *
 * with K/V (and the state S) shared by the H_q/H_kv query heads of a group
 * (Section 3.1, "Group-Query Variant": query head h reads K/V head h / (H_q/H_kv)).
 *
 * Conventions for every entry point
 *   - Positions are 0-indexed.  The window holds w+1 keys including the current one.
 *   - Tensors are dense, row-major, innermost dimension d:
 *       q, out, dout, dq : [B, H_q,  T, d]      k, v, dk, dv : [B, H_kv, T, d]
 *     (or, with rattn_params.layout = RATTN_LAYOUT_BTHD, [B, T, H_q, d] and [B, T, H_kv, d])
 *   - All data pointers are DEVICE pointers unless a parameter says "host".
 *     They must be 16-byte aligned.  The caller owns every buffer; the library
 *     keeps no reference after the call returns, allocates no device memory
 *     (one documented exception: rattn_forward), and never synchronises
 *     (exception: rattn_read_status): all work is enqueued on `stream` (a
 *     cudaStream_t passed as void*; NULL is the legacy default stream).
 *   - Return value: RATTN_OK (0) or a negative rattn_status.  Nothing is launched
 *     when an argument check fails.  No C++ exception crosses this boundary.
 *   - Device-side waits are bounded: if one expires the kernel stops early and
 *     records RATTN_ERR_TIMEOUT in the status word inside the workspace
 *     (see rattn_read_status).
 */
#ifndef RATTN_H_
#define RATTN_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum rattn_status {
  RATTN_OK = 0,
  RATTN_ERR_BAD_ARG = -1,        /* a size is out of range (B,H,T < 1, w < 1, H_q % H_kv != 0, ...) */
  RATTN_ERR_NULL_PTR = -2,       /* a required pointer is NULL */
  RATTN_ERR_MISALIGNED = -3,     /* a data pointer is not 16-byte aligned */
  RATTN_ERR_UNSUPPORTED = -4,    /* d not in {64,128}, unknown dtype / mode */
  RATTN_ERR_WORKSPACE = -5,      /* workspace missing or smaller than rattn_workspace_bytes() */
  RATTN_ERR_CUDA = -6,           /* a CUDA call failed; see rattn_last_cuda_error() */
  RATTN_ERR_TIMEOUT = -7,        /* a bounded device-side wait expired (status word) */
  RATTN_ERR_STATIC_LIMIT = -8    /* rattn_forward_static: sizes exceed its fixed scratch */
} rattn_status;

typedef enum rattn_dtype { RATTN_BF16 = 0, RATTN_F32 = 1 } rattn_dtype;

typedef enum rattn_mode {
  RATTN_MODE_RATTN = 0,          /* SWA + RLA, the operator above */
  RATTN_MODE_SWA_ONLY = 1,       /* y = rmsnorm(o_swa); the RLA branch is skipped */
  RATTN_MODE_FULL_CAUSAL = 2     /* w := T: y = rmsnorm(causal softmax attention) */
} rattn_mode;

/* The feature map phi of the linear branch (Section 3.1, "Parameterization").  The paper's
 * models use the softmax map; its ablation (Table 6) also tries ReLU and the identity. */
typedef enum rattn_feature_map {
  RATTN_PHI_SOFTMAX = 0,         /* softmax over the d head features */
  RATTN_PHI_RELU = 1,            /* max(x, 0), element-wise */
  RATTN_PHI_IDENTITY = 2         /* x */
} rattn_feature_map;

/* Memory layout of the operator's tensors (rattn_params.layout).  The projections of a transformer
 * layer produce [B, T, H * d]; RATTN_LAYOUT_BTHD reads and writes that directly (through the strides of
 * the TMA tensor maps on the tensor-core path), so no transposing copy is needed around the operator.
 * Applies to q, out, dout, dq (H = H_q) and k, v, dk, dv (H = H_kv) of rattn_forward_ex and
 * rattn_backward_ex; decode tokens, rings, states and gains keep their layouts. */
typedef enum rattn_layout {
  RATTN_LAYOUT_BHTD = 0,         /* [B, H, T, d], the default */
  RATTN_LAYOUT_BTHD = 1          /* [B, T, H, d] */
} rattn_layout;

/* Path selection for rattn_params.flags. */
#define RATTN_FLAG_FORCE_GENERIC 1u  /* use the portable fp32-FMA kernels even where the
                                        tensor-core path applies (debugging / comparison) */
#define RATTN_FLAG_SAVE_RESIDUALS 2u /* training mode: the forward also writes what the
                                        backward needs (log-sum-exp and the two un-normalised
                                        branch outputs) into the workspace */

/*
 * Parameter block of the *_ex entry points.  Zero-initialise it, then fill in.
 *   dtype      I/O element type of q,k,v,out,dout,dq,dk,dv and the decode ring.
 *              Accumulation, softmax, feature map, norms and the state are fp32.
 *              Value range on the bf16 tensor-core path: the attention weights and v enter
 *              the tensor cores as fp16, so |v| above 65504 saturates to 65504, |v| below
 *              6.1e-5 (2^-14) keeps fewer than 11 bits and |v| below 6e-8 reads as zero.
 *              Nothing detects this.  Both norms cancel a common factor of v, so a caller
 *              whose values sit outside roughly [1e-3, 1e4] rescales v (and eps by the
 *              square of the factor) or sets RATTN_FLAG_FORCE_GENERIC.
 *   scale      multiplies the SWA logits q.k only (the paper writes none: 1.0).  The
 *              tensor-core kernels need scale > 0 and return RATTN_ERR_UNSUPPORTED
 *              otherwise; the portable kernels (RATTN_FLAG_FORCE_GENERIC) take any finite
 *              value.
 *   eps        added to mean(x^2) inside the RMS-norm square root.
 *   gamma_swa, gamma_rla   fp32 [H_q, d] gains of the two norms, or NULL for ones.
 *   workspace  scratch + saved residuals, rattn_workspace_bytes_ex() bytes for this
 *              call's sizes, mode and flags, 256-byte aligned.  May be NULL where that
 *              size is 256 (nothing but the status word would live there).
 *              rattn_forward_ex writes it; rattn_backward_ex reads the
 *              residuals the forward left there, so pass the same buffer, untouched,
 *              with the same sizes, mode and flags (the tensor-core and the portable
 *              kernels keep their residuals in different forms).
 *   state_out, k_ring_out, v_ring_out   optional prefill -> decode hand-off written by
 *              rattn_forward_ex: state [B,H_kv,d,d] fp32 = sum over tokens j < T-w of
 *              phi(k_j)^T v_j; rings [B,H_kv,w,d] (I/O dtype) holding token j at slot
 *              j % w for the last min(w,T) tokens (other slots zero).
 *   dgamma_swa, dgamma_rla   optional fp32 [H_q,d] outputs of rattn_backward_ex.
 *   feature_map   phi of the linear branch (forward, backward and decode must agree).
 *   state_in, k_ring_in, v_ring_in, pos0   chunked prefill: this call's q, k, v are the tokens
 *              pos0 .. pos0+T-1 of a longer sequence; the rings and the state are what an
 *              earlier rattn_forward_ex call on the tokens before them handed out (state_out,
 *              k_ring_out, v_ring_out -- the same buffers may be passed as both in and out).
 *              out holds the T rows of this chunk, identical to rows pos0.. of one call on
 *              the whole sequence.  Needs pos0 >= w (a first chunk of at least w tokens) and a
 *              workspace (rattn_workspace_bytes_chunked); forward only.
 *   seq_lens   variable-length batches: entry b has seq_lens[b] valid tokens.  Its valid rows
 *              are what a call on that entry alone would give (the operator is causal, so
 *              nothing behind an entry's end reaches them); tiles that lie wholly beyond an
 *              entry's end are skipped, the other rows of out beyond it hold unspecified
 *              values, and the hand-off (state_out, rings) is taken at each entry's own length.
 */
typedef struct rattn_params {
  const void* q;
  const void* k;
  const void* v;
  void* out;
  int32_t B, H_q, H_kv, T, d, w;
  int32_t dtype;                 /* rattn_dtype */
  int32_t mode;                  /* rattn_mode */
  float scale;
  float eps;
  const float* gamma_swa;
  const float* gamma_rla;
  void* workspace;
  size_t workspace_bytes;
  float* state_out;
  void* k_ring_out;
  void* v_ring_out;
  /* backward only */
  const void* dout;
  void* dq;
  void* dk;
  void* dv;
  float* dgamma_swa;
  float* dgamma_rla;
  uint32_t flags;                /* RATTN_FLAG_* */
  int32_t feature_map;           /* rattn_feature_map; 0 = the paper's softmax map */
  /* chunked prefill (forward only): resume a sequence whose first pos0 tokens were processed
   * by earlier calls.  pos0 = 0 with the three pointers NULL is a fresh sequence. */
  const float* state_in;         /* [B,H_kv,d,d] fp32: state over the tokens j < pos0 - w */
  const void* k_ring_in;         /* [B,H_kv,w,d]: tokens pos0-w .. pos0-1 at slot j % w */
  const void* v_ring_in;
  int32_t pos0;                  /* tokens that precede this call's T tokens; 0 or >= w */
  int32_t layout;                /* rattn_layout of q, k, v, out, dout, dq, dk, dv */
  const int32_t* seq_lens;       /* optional device [B]: valid tokens of each batch entry, 1 <= len <= T
                                    (fresh sequences only); NULL: all T */
  const int32_t* pos;            /* decode only: optional device [B] positions, one per batch entry
                                    (overrides the pos argument) */
} rattn_params;

/*
 * Forward, Section 3.2 (SWA of Section 2.1 + RLA of Eq. 4 + two RMS norms).
 * bf16 I/O, scale = 1, unit gains, eps = 1e-6, mode RATTN, inference (no residuals).
 * T need not be a multiple of any tile.  This is the one entry point that may take
 * device memory on its own: where the tensor-core path applies (d = 128, w % 128 == 0)
 * it needs scratch for the chunk states of the linear branch
 * (rattn_workspace_bytes_ex(..., RATTN_MODE_RATTN, 0) bytes) and obtains it with
 * cudaMallocAsync / cudaFreeAsync on `stream` (the device's stream-ordered pool; no
 * synchronisation).  Callers that must control every allocation use rattn_forward_ex
 * with their own workspace.  That scratch, and the status word in it, are gone when the call
 * returns, so the word is latched into the library before the scratch is freed:
 * rattn_forward_status (synchronises the stream) returns RATTN_ERR_TIMEOUT if a bounded
 * device-side wait has expired in any rattn_forward call on the current device since it was
 * last asked, else RATTN_OK.
 */
int rattn_forward(const void* q, const void* k, const void* v,
                  int B, int H_q, int H_kv, int T, int d, int w,
                  void* out, void* stream);

/*
 * Forward that allocates nothing (the paper has no counterpart; this exists for the sake
 * of callers, not of the method).  Same operator and conventions as rattn_forward (bf16,
 * unit gains, eps = 1e-6, inference) with an explicit logit `scale`.
 *
 * Who needs it: code that is not in a position to obtain device memory at call time and
 * has no workspace to pass -- a server whose own cache manager already owns all of the
 * GPU's memory, an operator plugged into another framework that cannot reach that
 * framework's allocator, a latency-bound loop that must stay clear of the driver's
 * allocation lock.  Where the tensor-core path applies (d = 128, w % 128 == 0) its chunk
 * states go into a fixed array inside the library instead: RATTN_STATIC_MAX_CHUNK_STATES
 * matrices of 128 x 128 bf16 (2 MiB in all, plus 512 bytes of status and progress words, held by every GPU that loads the library until
 * the process exits).  The call is refused with RATTN_ERR_STATIC_LIMIT when
 * B * H_kv * ceil(T / 128) exceeds that number; other shapes run the portable kernel,
 * which needs no scratch, so they are never refused for size.
 *
 * The call itself makes no cudaMalloc / cudaFree / pool allocation.  The first call on
 * each device looks up the array's device address (a one-time set-up step; make that
 * first call outside any stream capture).  All calls on a device share the one array and
 * it keeps the previous call's contents (the library clears the part that must start at
 * zero): two calls whose kernels may overlap on the GPU -- different streams, no ordering
 * between them -- race on it, so serialise them.
 */
#define RATTN_STATIC_MAX_CHUNK_STATES 64
int rattn_forward_static(const void* q, const void* k, const void* v,
                         int B, int H_q, int H_kv, int T, int d, int w, float scale,
                         void* out, void* stream);

/* The device status word of rattn_forward_static's calls on the current device (it sits at
 * the head of the fixed array, which the caller cannot name): synchronises `stream`, then
 * returns RATTN_OK, RATTN_ERR_TIMEOUT (a bounded device-side wait of the last call expired)
 * or RATTN_ERR_CUDA.  Allocates nothing. */
int rattn_static_status(void* stream);

/* Forward with the full parameter block (dtype, scale, gains, mode, workspace,
 * residuals for the backward, prefill -> decode hand-off). */
int rattn_forward_status(void* stream);
int rattn_forward_ex(const rattn_params* p, void* stream);

/*
 * Backward of the same operator: given dout = dL/dy, writes dq, dk, dv (I/O dtype;
 * dk, dv summed over the query heads of each group).  The paper prints no backward
 * formulas; these are the chain rule through Section 2.1, Eq. 4, the softmax feature
 * map and the two RMS norms, using per-chunk states as the paper's kernel-design
 * paragraph describes (states saved at chunk boundaries, intra-chunk terms recomputed).
 * bf16, scale = 1, unit gains, eps = 1e-6.  `ws` must be the workspace a preceding
 * rattn_forward_ex call with the same sizes filled.
 */
int rattn_backward(const void* q, const void* k, const void* v, const void* dout,
                   void* ws, size_t ws_bytes,
                   int B, int H_q, int H_kv, int T, int d, int w,
                   void* dq, void* dk, void* dv, void* stream);

int rattn_backward_ex(const rattn_params* p, void* stream);

/*
 * One decode step (Section 2.1: at most w+1 cached tokens; Eq. 4: constant-size state).
 * For every batch entry, at position pos (the same for the whole batch):
 *   SWA over the ring's tokens pos-w..pos-1 (those >= 0) plus the incoming token,
 *   RLA read-out phi(q) . state  (state holds tokens j < pos-w),
 *   y = rmsnorm(o_swa) + rmsnorm(o_rla) -> out [B,H_q,d];
 * then the token leaving the window (pos-w, if >= 0) is folded into the state,
 * state += phi(k_old)^T v_old, and the incoming k,v overwrite ring slot pos % w.
 *   q [B,H_q,d]; k, v [B,H_kv,d]; k_ring, v_ring [B,H_kv,w,d] (same dtype as q);
 *   state [B,H_kv,d,d] fp32 (rows: feature index of phi(k), columns: value index).
 * Ring and state are updated in place.  bf16, scale = 1, unit gains, eps = 1e-6.
 */
int rattn_decode_step(const void* q, const void* k, const void* v,
                      void* k_ring, void* v_ring, float* state, int pos,
                      int B, int H_q, int H_kv, int d, int w,
                      void* out, void* stream);

/* Decode step with dtype / scale / eps / gains taken from `p` (p->q,k,v,out are the
 * step's tensors; p->T is ignored).  k_ring, v_ring, state, pos as above. */
int rattn_decode_step_ex(const rattn_params* p, void* k_ring, void* v_ring, float* state,
                         int pos, void* stream);

/* For bf16, d = 128, w a multiple of 64 and H_q / H_kv <= 8 (unless RATTN_FLAG_FORCE_GENERIC) the
 * decode step stages the ring and the state through shared memory with asynchronous copies and
 * waits for them with a bound.  rattn_decode_status (synchronises the stream) returns
 * RATTN_ERR_TIMEOUT if such a wait has expired in any decode step on the current device since it
 * was last asked (the step then left its outputs, ring and state in an unspecified state), else
 * RATTN_OK. */
int rattn_decode_status(void* stream);

/*
 * Bytes of workspace a call with these sizes, mode (rattn_mode) and flags (RATTN_FLAG_*)
 * needs; dtype is a rattn_dtype.  Returns 0 for invalid arguments.  The first 256 bytes hold
 * the device status word (on the tensor-core kernels in mode RATTN one progress word per K/V
 * head follows it, rounded up to 256 bytes).  What the rest holds depends on the call:
 *   inference, portable kernels        nothing more (256 bytes in all);
 *   inference, tensor-core kernels     the chunk states of the linear branch (Eq. 2; the
 *                                      paper's stored states): bf16 [B,H_kv,ceil(T/128),d,d],
 *                                      mode RATTN only;
 *   RATTN_FLAG_SAVE_RESIDUALS          in addition the residuals of Section 3.2's two branches
 *                                      (log-sum-exp, un-normalised o_swa and o_rla: bf16 on the
 *                                      tensor-core path, fp32 on the portable one) and the
 *                                      backward's scratch of the same shapes.
 * The backward needs the size of its forward (same sizes, mode, flags with
 * RATTN_FLAG_SAVE_RESIDUALS set).  A larger buffer is always accepted.
 */
size_t rattn_workspace_bytes_ex(int B, int H_q, int H_kv, int T, int d, int w, int dtype,
                                int mode, unsigned flags);

/* The same for a forward that resumes a sequence (rattn_params.pos0 > 0): in addition the
 * history + chunk keys and values in time order, 2 x [B,H_kv,w+T,d] elements. */
size_t rattn_workspace_bytes_chunked(int B, int H_q, int H_kv, int T, int d, int w, int dtype,
                                     unsigned flags);

/* An upper bound of rattn_workspace_bytes_ex over every mode and every flag combination for
 * these sizes (the training layout of the larger kernel family). */
size_t rattn_workspace_bytes(int B, int H_q, int H_kv, int T, int d, int w, int dtype);

/* Reads the status word of a workspace (synchronises `stream` first, copies 4 bytes
 * device -> host).  Returns RATTN_OK, RATTN_ERR_TIMEOUT, or RATTN_ERR_CUDA. */
int rattn_read_status(const void* workspace, void* stream);

/* Static string for a status code.  Host memory owned by the library. */
const char* rattn_strerror(int status);

/* The cudaError_t (as int) behind the calling thread's last RATTN_ERR_CUDA. */
int rattn_last_cuda_error(void);

/* Number of kernel launches this process has enqueued through the library so far
 * (host counter; used by the benchmark to report its launch count). */
uint64_t rattn_launch_count(void);

/*
 * Optional per-kernel device timing for benchmarks.  While enabled, every kernel the
 * library launches is bracketed by a CUDA event pair on its stream.  Enabling or
 * disabling clears the records.  rattn_timing_read waits for the recorded events, then
 * writes one text line per kernel name, "name launches total_ms\n", NUL-terminated,
 * into the HOST buffer `buf` (truncated to buf_bytes) and returns the bytes needed.
 */
int rattn_timing_enable(int on);
size_t rattn_timing_read(char* buf, size_t buf_bytes);

/*
 * Tuning parameters of the tensor-core forward, process-wide (the counterpart of the paper's
 * search over the stored-state stride m and the chunk size C, Section 3.2 "Kernel Design"; here
 * the chunk is the 128-token MMA tile and is fixed).  rattn_tune returns the previous value,
 * or RATTN_ERR_BAD_ARG for an unknown knob or a value out of range.  Defaults are what the
 * sweep in profiles/ found best on B200.
 */
typedef enum rattn_knob {
  RATTN_TUNE_STATE_STRIDE = 0,   /* m: 0 = automatic (2 for an inference forward, whose query-tile pairs read every
                                    second chunk state; 1 when the backward will read them all), 1, 2 */
  RATTN_TUNE_OVERLAP = 1,        /* 1 (default): the main kernel starts under the chunk-state kernel
                                    (programmatic dependent launch); 0: strictly one after the other */
  RATTN_TUNE_UNIT_ORDER = 2,     /* order in which the persistent forward kernel hands out its work units:
                                    0 (default) automatic; 1 units that read no stored state first (they can run
                                    under the chunk-state kernel), then heaviest first; 2 heaviest first
                                    throughout; 3 the same, dealt round-robin instead of drawn from a counter.
                                    Automatic = 1 when the state kernel leaves at least half of the SMs free. */
  RATTN_TUNE_GRID = 3,           /* CTAs of the persistent forward kernel: 0 (default) = one per SM */
  RATTN_TUNE_DECODE_STAGES = 4,  /* 16 KB stages of the staged decode step: 0 (default) = as many as let two
                                    CTAs share an SM; 3..8 (ignored where that many do not fit) */
  RATTN_TUNE_STATE_PROGRESS = 5  /* the main kernel takes the chunk states as the chunk-state kernel publishes them
                                    (one progress word per K/V head, work units in sequence order) instead of
                                    waiting for that whole kernel: 0 (default) automatic = on for long chains on
                                    few K/V heads with windows up to 512 (T >= 6144, 4 B H_kv <= SMs); 1 on; 2 off */
} rattn_knob;
int rattn_tune(int knob, int value);

/* 1 when the tensor-core (tcgen05) forward would be chosen for these sizes. */
int rattn_uses_tensor_path(int d, int w, int dtype, int mode, unsigned flags);

/*
 * What the paper's models apply to q and k between the projections and the operator, as one
 * pass over both tensors (one read and one write of each element instead of two of each for a
 * norm kernel followed by a rotation kernel):
 *
 *   qk-norm (Table 1, "qk-norm: yes"):  n = x / sqrt(mean(x^2) + eps) * gain   per head vector,
 *           gain fp32 [d], one for the queries and one for the keys (NULL = ones);
 *   rotary embedding (Section 4, "Model Setup": local layers, theta = 5e5; global layers none):
 *           features i and i + d/2 (i < d/2) of the token at sequence position p are rotated by
 *           the angle p * theta^(-2i/d):
 *               y_i       = n_i cos - n_{i+d/2} sin,     y_{i+d/2} = n_{i+d/2} cos + n_i sin.
 *
 *   q, k           inputs, [B,H_q,T,d] and [B,H_kv,T,d], element type dtype.  k (and k_out) may be
 *                  NULL with H_kv = 0 to transform one tensor only.
 *   q_out, k_out   results, same shapes and type; each may be the same pointer as its input.
 *   theta          rotation base; theta <= 0 skips the rotation (global layers).
 *   pos0, pos      row t of batch entry b sits at position (pos ? pos[b] : pos0) + t; pos is an
 *                  optional device int32 [B] (decoding a batch whose entries have different lengths).
 *                  Angles are formed in fp64 and reduced before the fp32 sine and cosine, so
 *                  positions up to 2^31 keep full fp32 accuracy.
 *   layout         RATTN_LAYOUT_BHTD (default) or RATTN_LAYOUT_BTHD: q as [B,T,H_q,d], k as [B,T,H_kv,d],
 *                  the layout the projections write; the results and gradients have the same layout.
 *   d              64 or 128.  Arithmetic is fp32; sums over a row are taken in a fixed order.
 *
 * rattn_qk_prologue_backward: given the same inputs (the tensors as they were BEFORE the forward
 * pass, so not after an in-place call) and the gradients dq_out, dk_out with respect to the
 * results, writes the gradients dq, dk with respect to q, k (each may alias its dq_out / dk_out)
 * and, where the pointers are not NULL, the gain gradients dq_gain, dk_gain (fp32 [d],
 * overwritten).  Gain gradients need a workspace of rattn_qk_prologue_workspace_bytes() bytes
 * (256-byte aligned) for per-CTA partial sums, which a second kernel adds in a fixed order: the
 * result does not depend on scheduling.
 *
 * Errors as for the other entry points; nothing is launched when a check fails.  The kernels
 * stage their data through shared memory with asynchronous copies and wait for them with a
 * bound; rattn_qk_prologue_status (synchronises the stream) returns RATTN_ERR_TIMEOUT if such a
 * wait has expired in any prologue call on the current device since it was last asked, else RATTN_OK.
 */
typedef struct rattn_qk_params {
  const void* q;
  const void* k;
  void* q_out;
  void* k_out;
  const float* q_gain;
  const float* k_gain;
  int32_t B, H_q, H_kv, T, d;
  int32_t dtype;                 /* rattn_dtype */
  float eps;
  float theta;
  int32_t pos0;
  int32_t layout;                /* rattn_layout of q, k, their outputs and gradients */
  const int32_t* pos;
} rattn_qk_params;

int rattn_qk_prologue(const rattn_qk_params* p, void* stream);
int rattn_qk_prologue_backward(const rattn_qk_params* p, const void* dq_out, const void* dk_out,
                               void* dq, void* dk, float* dq_gain, float* dk_gain,
                               void* workspace, size_t workspace_bytes, void* stream);
size_t rattn_qk_prologue_workspace_bytes(int B, int H_q, int H_kv, int T, int d);
int rattn_qk_prologue_status(void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RATTN_H_ */
