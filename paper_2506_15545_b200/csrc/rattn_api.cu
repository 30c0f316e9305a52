// C ABI of librattn.so: argument checks, workspace carving, path selection.
// See include/rattn.h for the contract of every entry point.
#include <atomic>
#include <cstdio>
#include <cstring>
#include <map>
#include <mutex>
#include <string>
#include <vector>

#include "rattn_internal.h"
#ifdef RATTN_DEBUG_KNOBS
#include "rattn_debug.h"
#endif

namespace rattn {

static std::atomic<uint64_t> g_launches{0};
static thread_local int g_last_cuda_error = 0;

static std::atomic<int> g_debug_skip_arrive{0};
int debug_skip_arrive() {
#ifdef RATTN_DEBUG_KNOBS
  return g_debug_skip_arrive.load(std::memory_order_relaxed);
#else
  return 0;
#endif
}

static std::atomic<int> g_tuning[6] = {{0}, {1}, {0}, {0}, {0}, {0}};
int tuning(int knob) { return g_tuning[knob].load(std::memory_order_relaxed); }

void count_launches(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
void set_last_cuda_error(int cuda_error) { g_last_cuda_error = cuda_error; }

// ---- optional per-kernel timing ------------------------------------------------------
struct TimingRecord { const char* name; cudaEvent_t begin, end; };
static std::mutex g_timing_mu;
static std::vector<TimingRecord> g_timing;
static std::atomic<int> g_timing_on{0};
constexpr size_t kMaxTimingRecords = 1 << 16;

KernelTimer::KernelTimer(const char* name, cudaStream_t s) : stream_(s), slot_(-1) {
  if (!g_timing_on.load(std::memory_order_relaxed)) return;
  std::lock_guard<std::mutex> lk(g_timing_mu);
  if (g_timing.size() >= kMaxTimingRecords) return;
  TimingRecord r{name, nullptr, nullptr};
  if (cudaEventCreate(&r.begin) != cudaSuccess) return;
  if (cudaEventCreate(&r.end) != cudaSuccess) { cudaEventDestroy(r.begin); return; }
  cudaEventRecord(r.begin, s);
  g_timing.push_back(r);
  slot_ = (int)g_timing.size() - 1;
}

KernelTimer::~KernelTimer() {
  if (slot_ < 0) return;
  std::lock_guard<std::mutex> lk(g_timing_mu);
  if (slot_ < (int)g_timing.size()) cudaEventRecord(g_timing[slot_].end, stream_);
}

static void timing_clear_locked() {
  for (auto& r : g_timing) { cudaEventDestroy(r.begin); cudaEventDestroy(r.end); }
  g_timing.clear();
}

static inline size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

static bool tensor_path(int d, int w, int dtype, int mode, unsigned flags) {
#ifdef RATTN_HAVE_TC
  if (flags & RATTN_FLAG_FORCE_GENERIC) return false;
  if (dtype != RATTN_BF16 || d != 128) return false;
  if (mode != RATTN_MODE_FULL_CAUSAL && (w % 128) != 0) return false;
  return true;
#else
  (void)d; (void)w; (void)dtype; (void)mode; (void)flags;
  return false;
#endif
}

// What a call with these sizes, mode and flags keeps in its workspace.  Inference on the
// portable kernels: the status block only.  Inference on the tensor-core kernels: the status
// block and the chunk states of the linear branch.  Training (RATTN_FLAG_SAVE_RESIDUALS) adds the
// residuals the backward reads and the backward's own scratch, in the element type the chosen
// kernels keep them in (bf16 on the tensor-core path, fp32 on the portable one).
WorkspaceLayout workspace_layout(int B, int H_q, int H_kv, int T, int d, int w, int dtype, int mode,
                                 unsigned flags, int history) {
  WorkspaceLayout L;
  const bool tc = tensor_path(d, mode == RATTN_MODE_FULL_CAUSAL ? T : w, dtype, mode, flags);
  const bool train = (flags & RATTN_FLAG_SAVE_RESIDUALS) != 0;
  const bool rla = (mode == RATTN_MODE_RATTN);
  const size_t rows = (size_t)B * H_q * T;
  const size_t branch_elem = tc ? sizeof(__nv_bfloat16) : sizeof(float);
  size_t off = 0;
  auto take = [&](bool present, size_t bytes) -> size_t {
    if (!present) return kAbsent;
    const size_t at = off;
    off += align256(bytes);
    return at;
  };
  const int Tk = history ? w + T : T;           // key rows per head: the history precedes the chunk
  L.n_chunks = (Tk + 127) / 128;
  const size_t states = (size_t)B * H_kv * L.n_chunks * d * d;
  const size_t rows_pad = (size_t)B * H_q * L.n_chunks * 128;
  L.status_bytes = 256 + ((tc && rla) ? align256(sizeof(int) * (size_t)B * H_kv) : 0);
  L.status = take(true, L.status_bytes);
  L.lse = take(train, rows * sizeof(float));
  L.o_swa = take(train, rows * d * branch_elem);
  L.o_rla = take(train, rows * d * branch_elem);
  L.do_swa = take(train, rows * d * branch_elem);
  L.do_rla = take(train, rows * d * branch_elem);
  L.delta = take(train, rows * sizeof(float));
  L.chunk_state = take(tc && rla, states * sizeof(__nv_bfloat16));
  L.rstate = take(tc && rla && train, states * sizeof(__nv_bfloat16));
  L.lse2p = take(tc && train, rows_pad * sizeof(float));
  L.dscp = take(tc && train, rows_pad * sizeof(float));
  const size_t io_elem = dtype == RATTN_F32 ? sizeof(float) : sizeof(__nv_bfloat16);
  L.k_ext = take(history != 0, (size_t)B * H_kv * Tk * d * io_elem);
  L.v_ext = take(history != 0, (size_t)B * H_kv * Tk * d * io_elem);
  L.total = off;
  return L;
}

static int fail_cuda(cudaError_t e) {
  g_last_cuda_error = (int)e;
  return RATTN_ERR_CUDA;
}

static bool misaligned(const void* p) { return ((uintptr_t)p & 15u) != 0; }

// Common checks of the size fields; fills the resolved Args.
static int resolve(const rattn_params* p, Args* a, bool need_T) {
  if (!p) return RATTN_ERR_NULL_PTR;
  if (p->B < 1 || p->H_q < 1 || p->H_kv < 1 || p->w < 1 || (need_T && p->T < 1)) return RATTN_ERR_BAD_ARG;
  if (p->H_q % p->H_kv != 0) return RATTN_ERR_BAD_ARG;
  if (p->d != 64 && p->d != 128) return RATTN_ERR_UNSUPPORTED;
  if (p->dtype != RATTN_BF16 && p->dtype != RATTN_F32) return RATTN_ERR_UNSUPPORTED;
  if (p->mode < RATTN_MODE_RATTN || p->mode > RATTN_MODE_FULL_CAUSAL) return RATTN_ERR_UNSUPPORTED;
  if (p->feature_map < RATTN_PHI_SOFTMAX || p->feature_map > RATTN_PHI_IDENTITY) return RATTN_ERR_UNSUPPORTED;
  if (p->layout != RATTN_LAYOUT_BHTD && p->layout != RATTN_LAYOUT_BTHD) return RATTN_ERR_UNSUPPORTED;
  if (!(p->eps > 0.f) || !(p->scale == p->scale)) return RATTN_ERR_BAD_ARG;
  if (!p->q || !p->k || !p->v || !p->out) return RATTN_ERR_NULL_PTR;
  if (misaligned(p->q) || misaligned(p->k) || misaligned(p->v) || misaligned(p->out) ||
      misaligned(p->gamma_swa) || misaligned(p->gamma_rla))
    return RATTN_ERR_MISALIGNED;
  std::memset(a, 0, sizeof(*a));
  a->q = p->q; a->k = p->k; a->v = p->v; a->out = p->out;
  a->B = p->B; a->H_q = p->H_q; a->H_kv = p->H_kv; a->T = p->T; a->d = p->d;
  a->Tk = p->T;
  a->w = (p->mode == RATTN_MODE_FULL_CAUSAL && need_T) ? p->T : p->w;
  a->group = p->H_q / p->H_kv;
  a->dtype = p->dtype; a->mode = p->mode;
  a->flags = p->flags;
  a->layout = a->kv_layout = p->layout;
  a->phi = p->feature_map;
  a->scale = p->scale; a->eps = p->eps;
  a->gamma_swa = p->gamma_swa; a->gamma_rla = p->gamma_rla;
  return RATTN_OK;
}

static int bind_workspace(const rattn_params* p, Args* a, bool required, unsigned flags, int history = 0,
                          WorkspaceLayout* layout = nullptr) {
  if (!p->workspace) return required ? RATTN_ERR_WORKSPACE : RATTN_OK;
  if (((uintptr_t)p->workspace & 255u) != 0) return RATTN_ERR_MISALIGNED;
  const WorkspaceLayout L = workspace_layout(p->B, p->H_q, p->H_kv, p->T, p->d, p->w, p->dtype, p->mode, flags, history);
  if (layout) *layout = L;
  if (p->workspace_bytes < L.total) return RATTN_ERR_WORKSPACE;
  char* base = reinterpret_cast<char*>(p->workspace);
  auto at = [&](size_t off) -> char* { return off == kAbsent ? nullptr : base + off; };
  a->status = reinterpret_cast<int*>(at(L.status));
  a->state_ready = L.status_bytes > 256 ? a->status + 64 : nullptr;
  a->lse = reinterpret_cast<float*>(at(L.lse));
  a->o_swa = reinterpret_cast<float*>(at(L.o_swa));
  a->o_rla = reinterpret_cast<float*>(at(L.o_rla));
  a->do_swa = reinterpret_cast<float*>(at(L.do_swa));
  a->do_rla = reinterpret_cast<float*>(at(L.do_rla));
  a->delta = reinterpret_cast<float*>(at(L.delta));
  a->chunk_state = reinterpret_cast<__nv_bfloat16*>(at(L.chunk_state));
  a->rstate = reinterpret_cast<__nv_bfloat16*>(at(L.rstate));
  a->lse2p = reinterpret_cast<float*>(at(L.lse2p));
  a->dscp = reinterpret_cast<float*>(at(L.dscp));
  a->n_chunks = L.n_chunks;
  return RATTN_OK;
}

static int forward_impl(const rattn_params* p, cudaStream_t s) {
  Args a;
  int rc = resolve(p, &a, true);
  if (rc != RATTN_OK) return rc;
  const bool want_handoff = p->state_out || p->k_ring_out || p->v_ring_out;
  if (want_handoff) {
    if ((p->k_ring_out == nullptr) != (p->v_ring_out == nullptr)) return RATTN_ERR_NULL_PTR;
    if (misaligned(p->state_out) || misaligned(p->k_ring_out) || misaligned(p->v_ring_out))
      return RATTN_ERR_MISALIGNED;
    if (p->mode != RATTN_MODE_RATTN) return RATTN_ERR_UNSUPPORTED;
  }
  const bool tc = tensor_path(p->d, a.w, p->dtype, p->mode, p->flags);
  // the tensor-core kernels take the row maximum before multiplying by the scale
  if (tc && !(p->scale > 0.f)) return RATTN_ERR_UNSUPPORTED;
  const bool train = (p->flags & RATTN_FLAG_SAVE_RESIDUALS) != 0;
  // chunked prefill: the chunk continues a sequence whose last w tokens and state come with it
  const bool resume = p->pos0 != 0 || p->state_in || p->k_ring_in || p->v_ring_in;
  if (resume) {
    if (p->pos0 < p->w) return RATTN_ERR_BAD_ARG;
    if (!p->state_in || !p->k_ring_in || !p->v_ring_in) return RATTN_ERR_NULL_PTR;
    if (misaligned(p->state_in) || misaligned(p->k_ring_in) || misaligned(p->v_ring_in)) return RATTN_ERR_MISALIGNED;
    if (p->mode != RATTN_MODE_RATTN || train || p->seq_lens) return RATTN_ERR_UNSUPPORTED;
  }
  if (p->seq_lens && (((uintptr_t)p->seq_lens & 3u) != 0)) return RATTN_ERR_MISALIGNED;
  if (p->seq_lens && train) return RATTN_ERR_UNSUPPORTED;
  // a workspace is needed for the residuals, for the chunk states of the tensor-core path and for
  // the history + chunk keys and values of a resumed sequence
  WorkspaceLayout L;
  rc = bind_workspace(p, &a, train || resume || (tc && p->mode == RATTN_MODE_RATTN), p->flags, resume ? 1 : 0, &L);
  if (rc != RATTN_OK) return rc;
  a.seq_lens = p->seq_lens;
  a.state_out = p->state_out; a.k_ring_out = p->k_ring_out; a.v_ring_out = p->v_ring_out;
  a.training = train;
  cudaError_t e;
  if (a.status) {
    e = cudaMemsetAsync(a.status, 0, L.status_bytes, s);
    if (e != cudaSuccess) return fail_cuda(e);
  }
  if (resume) {
    char* base = reinterpret_cast<char*>(p->workspace);
    void* k_ext = base + L.k_ext;
    void* v_ext = base + L.v_ext;
    e = launch_gather_history(a, p->k, p->v, p->k_ring_in, p->v_ring_in, k_ext, v_ext, p->pos0, s);
    if (e != cudaSuccess) return fail_cuda(e);
    a.k = k_ext; a.v = v_ext;
    a.kv_layout = RATTN_LAYOUT_BHTD;                       // the gathered history + chunk is dense per head
    a.Tk = p->w + p->T; a.q_off = p->w; a.state_in = p->state_in; a.pos_shift = p->pos0 - p->w;
  }
#ifdef RATTN_HAVE_TC
  if (tc) e = launch_tc_forward(a, s);
  else
#endif
    e = launch_generic_forward(a, s);
  if (e != cudaSuccess) return fail_cuda(e);
  if (want_handoff) {
    e = launch_handoff(a, s, !tc);      // the tensor-core forward has left the state itself
    if (e != cudaSuccess) return fail_cuda(e);
  }
  return RATTN_OK;
}

static int backward_impl(const rattn_params* p, cudaStream_t s) {
  Args a;
  int rc = resolve(p, &a, true);
  if (rc != RATTN_OK) return rc;
  if (!p->dout || !p->dq || !p->dk || !p->dv) return RATTN_ERR_NULL_PTR;
  if (p->pos0 != 0 || p->state_in || p->seq_lens) return RATTN_ERR_UNSUPPORTED;   // training runs on whole, fresh sequences
  if (misaligned(p->dout) || misaligned(p->dq) || misaligned(p->dk) || misaligned(p->dv) ||
      misaligned(p->dgamma_swa) || misaligned(p->dgamma_rla))
    return RATTN_ERR_MISALIGNED;
  const bool tc = tensor_path(p->d, a.w, p->dtype, p->mode, p->flags);
  if (tc && !(p->scale > 0.f)) return RATTN_ERR_UNSUPPORTED;
  rc = bind_workspace(p, &a, true, p->flags | RATTN_FLAG_SAVE_RESIDUALS);
  if (rc != RATTN_OK) return rc;
  a.dout = p->dout; a.dq = p->dq; a.dk = p->dk; a.dv = p->dv;
  a.dgamma_swa = p->dgamma_swa; a.dgamma_rla = p->dgamma_rla;
  cudaError_t e;
#ifdef RATTN_HAVE_TC
  // The tensor-core backward reads the chunk states the tensor-core forward left in the
  // workspace: both calls must take the same path (same sizes, mode and flags).
  if (tc) e = launch_tc_backward(a, s);
  else
#endif
    e = launch_generic_backward(a, s);
  if (e != cudaSuccess) return fail_cuda(e);
  return RATTN_OK;
}

}  // namespace rattn

using namespace rattn;

namespace {
// rattn_forward's scratch, status word included, is freed before the call returns: a one-thread
// kernel copies a non-zero word into this one first (sticky until rattn_forward_status reads it).
__device__ int g_forward_status;
__global__ void latch_status_kernel(const int* word) {
  if (*word != 0) g_forward_status = *word;
}

}  // namespace

extern "C" {

int rattn_forward_ex(const rattn_params* p, void* stream) {
  return forward_impl(p, reinterpret_cast<cudaStream_t>(stream));
}

int rattn_forward_status(void* stream) {
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int word = 0;
  cudaError_t e = cudaMemcpyFromSymbolAsync(&word, g_forward_status, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e == cudaSuccess && word != 0) {
    const int zero = 0;
    e = cudaMemcpyToSymbolAsync(g_forward_status, &zero, sizeof(int), 0, cudaMemcpyHostToDevice, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  }
  if (e != cudaSuccess) return fail_cuda(e);
  return word == 0 ? RATTN_OK : RATTN_ERR_TIMEOUT;
}

int rattn_forward(const void* q, const void* k, const void* v, int B, int H_q, int H_kv, int T,
                  int d, int w, void* out, void* stream) {
  rattn_params p;
  std::memset(&p, 0, sizeof(p));
  p.q = q; p.k = k; p.v = v; p.out = out;
  p.B = B; p.H_q = H_q; p.H_kv = H_kv; p.T = T; p.d = d; p.w = w;
  p.dtype = RATTN_BF16; p.mode = RATTN_MODE_RATTN; p.scale = 1.f; p.eps = 1e-6f;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  if (!tensor_path(d, w, RATTN_BF16, RATTN_MODE_RATTN, 0)) return forward_impl(&p, s);
  // The tensor-core path needs scratch for the chunk states of the linear branch: take it
  // from the device's stream-ordered pool for the duration of this call's work.
  Args chk;
  int rc = resolve(&p, &chk, true);
  if (rc != RATTN_OK) return rc;
  const size_t bytes = rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, RATTN_BF16, RATTN_MODE_RATTN, 0);
  void* ws = nullptr;
  cudaError_t e = cudaMallocAsync(&ws, bytes, s);
  if (e != cudaSuccess) return fail_cuda(e);
  p.workspace = ws;
  p.workspace_bytes = bytes;
  rc = forward_impl(&p, s);
  if (rc == RATTN_OK) {
    latch_status_kernel<<<1, 1, 0, s>>>(static_cast<const int*>(ws));
    count_launches(1);
  }
  e = cudaFreeAsync(ws, s);
  if (rc == RATTN_OK && e != cudaSuccess) return fail_cuda(e);
  return rc;
}

int rattn_backward_ex(const rattn_params* p, void* stream) {
  return backward_impl(p, reinterpret_cast<cudaStream_t>(stream));
}

int rattn_backward(const void* q, const void* k, const void* v, const void* dout, void* ws,
                   size_t ws_bytes, int B, int H_q, int H_kv, int T, int d, int w, void* dq,
                   void* dk, void* dv, void* stream) {
  rattn_params p;
  std::memset(&p, 0, sizeof(p));
  p.q = q; p.k = k; p.v = v; p.out = dq;   /* `out` is not written by the backward */
  p.B = B; p.H_q = H_q; p.H_kv = H_kv; p.T = T; p.d = d; p.w = w;
  p.dtype = RATTN_BF16; p.mode = RATTN_MODE_RATTN; p.scale = 1.f; p.eps = 1e-6f;
  p.workspace = ws; p.workspace_bytes = ws_bytes;
  p.dout = dout; p.dq = dq; p.dk = dk; p.dv = dv;
  return backward_impl(&p, reinterpret_cast<cudaStream_t>(stream));
}

int rattn_decode_step_ex(const rattn_params* p, void* k_ring, void* v_ring, float* state, int pos,
                         void* stream) {
  Args a;
  int rc = resolve(p, &a, false);
  if (rc != RATTN_OK) return rc;
  if (!k_ring || !v_ring || !state) return RATTN_ERR_NULL_PTR;
  if (misaligned(k_ring) || misaligned(v_ring) || misaligned(state)) return RATTN_ERR_MISALIGNED;
  if (pos < 0) return RATTN_ERR_BAD_ARG;
  if (p->mode != RATTN_MODE_RATTN) return RATTN_ERR_UNSUPPORTED;
  if (a.group > 64) return RATTN_ERR_UNSUPPORTED;
  if (p->pos && (((uintptr_t)p->pos & 3u) != 0)) return RATTN_ERR_MISALIGNED;
  a.w = p->w;
  cudaError_t e = launch_decode(a, k_ring, v_ring, state, pos, p->pos, reinterpret_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return fail_cuda(e);
  return RATTN_OK;
}

int rattn_decode_status(void* stream) {
  cudaError_t e = cudaSuccess;
  const int word = decode_tc_status(reinterpret_cast<cudaStream_t>(stream), &e);
  if (e != cudaSuccess) return fail_cuda(e);
  return word == 0 ? RATTN_OK : RATTN_ERR_TIMEOUT;
}

int rattn_decode_step(const void* q, const void* k, const void* v, void* k_ring, void* v_ring,
                      float* state, int pos, int B, int H_q, int H_kv, int d, int w, void* out,
                      void* stream) {
  rattn_params p;
  std::memset(&p, 0, sizeof(p));
  p.q = q; p.k = k; p.v = v; p.out = out;
  p.B = B; p.H_q = H_q; p.H_kv = H_kv; p.T = 1; p.d = d; p.w = w;
  p.dtype = RATTN_BF16; p.mode = RATTN_MODE_RATTN; p.scale = 1.f; p.eps = 1e-6f;
  return rattn_decode_step_ex(&p, k_ring, v_ring, state, pos, stream);
}

size_t rattn_workspace_bytes_ex(int B, int H_q, int H_kv, int T, int d, int w, int dtype, int mode,
                                unsigned flags) {
  if (B < 1 || H_q < 1 || H_kv < 1 || T < 1 || w < 1 || (d != 64 && d != 128)) return 0;
  if (H_q % H_kv != 0) return 0;
  if (dtype != RATTN_BF16 && dtype != RATTN_F32) return 0;
  if (mode < RATTN_MODE_RATTN || mode > RATTN_MODE_FULL_CAUSAL) return 0;
  return workspace_layout(B, H_q, H_kv, T, d, w, dtype, mode, flags).total;
}

size_t rattn_workspace_bytes_chunked(int B, int H_q, int H_kv, int T, int d, int w, int dtype, unsigned flags) {
  if (B < 1 || H_q < 1 || H_kv < 1 || T < 1 || w < 1 || (d != 64 && d != 128)) return 0;
  if (H_q % H_kv != 0) return 0;
  if (dtype != RATTN_BF16 && dtype != RATTN_F32) return 0;
  return workspace_layout(B, H_q, H_kv, T, d, w, dtype, RATTN_MODE_RATTN, flags & ~RATTN_FLAG_SAVE_RESIDUALS, 1).total;
}

size_t rattn_workspace_bytes(int B, int H_q, int H_kv, int T, int d, int w, int dtype) {
  // enough for any mode and any flags: the training layout of either kernel family
  const unsigned train = RATTN_FLAG_SAVE_RESIDUALS;
  const size_t a = rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, dtype, RATTN_MODE_RATTN, train);
  const size_t b = rattn_workspace_bytes_ex(B, H_q, H_kv, T, d, w, dtype, RATTN_MODE_RATTN,
                                            train | RATTN_FLAG_FORCE_GENERIC);
  return a > b ? a : b;
}

int rattn_read_status(const void* workspace, void* stream) {
  if (!workspace) return RATTN_ERR_NULL_PTR;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);
  int word = 0;
  cudaError_t e = cudaMemcpyAsync(&word, workspace, sizeof(int), cudaMemcpyDeviceToHost, s);
  if (e == cudaSuccess) e = cudaStreamSynchronize(s);
  if (e != cudaSuccess) return fail_cuda(e);
  return word == 0 ? RATTN_OK : RATTN_ERR_TIMEOUT;
}

const char* rattn_strerror(int status) {
  switch (status) {
    case RATTN_OK: return "ok";
    case RATTN_ERR_BAD_ARG: return "size argument out of range";
    case RATTN_ERR_NULL_PTR: return "required pointer is NULL";
    case RATTN_ERR_MISALIGNED: return "pointer is not sufficiently aligned";
    case RATTN_ERR_UNSUPPORTED: return "unsupported head size, dtype or mode";
    case RATTN_ERR_WORKSPACE: return "workspace missing or too small";
    case RATTN_ERR_CUDA: return "CUDA call failed (see rattn_last_cuda_error)";
    case RATTN_ERR_TIMEOUT: return "a bounded device-side wait expired";
    case RATTN_ERR_STATIC_LIMIT: return "problem needs more chunk states than rattn_forward_static's fixed scratch holds";
    default: return "unknown status";
  }
}

int rattn_last_cuda_error(void) { return g_last_cuda_error; }

uint64_t rattn_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

int rattn_timing_enable(int on) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  timing_clear_locked();
  g_timing_on.store(on ? 1 : 0, std::memory_order_relaxed);
  return RATTN_OK;
}

size_t rattn_timing_read(char* buf, size_t buf_bytes) {
  std::lock_guard<std::mutex> lk(g_timing_mu);
  std::map<std::string, std::pair<long, double>> acc;
  for (auto& r : g_timing) {
    float ms = 0.f;
    if (cudaEventSynchronize(r.end) != cudaSuccess) continue;
    if (cudaEventElapsedTime(&ms, r.begin, r.end) != cudaSuccess) continue;
    auto& e = acc[r.name];
    e.first += 1;
    e.second += ms;
  }
  std::string out;
  char line[256];
  for (auto& kv : acc) {
    std::snprintf(line, sizeof(line), "%s %ld %.6f\n", kv.first.c_str(), kv.second.first, kv.second.second);
    out += line;
  }
  if (buf && buf_bytes > 0) {
    const size_t n = out.size() < buf_bytes - 1 ? out.size() : buf_bytes - 1;
    std::memcpy(buf, out.data(), n);
    buf[n] = 0;
  }
  return out.size() + 1;
}

#ifdef RATTN_DEBUG_KNOBS
int rattn_debug_withhold_arrival(int on) {
  g_debug_skip_arrive.store(on ? 1 : 0, std::memory_order_relaxed);
  return RATTN_OK;
}
#endif

int rattn_tune(int knob, int value) {
  static const int lo[6] = {0, 0, 0, 0, 0, 0}, hi[6] = {2, 1, 3, 1 << 16, 8, 2};
  if (knob < 0 || knob > 5 || value < lo[knob] || value > hi[knob]) return RATTN_ERR_BAD_ARG;
  return g_tuning[knob].exchange(value, std::memory_order_relaxed);
}

int rattn_uses_tensor_path(int d, int w, int dtype, int mode, unsigned flags) {
  return tensor_path(d, w, dtype, mode, flags) ? 1 : 0;
}

}  // extern "C"
