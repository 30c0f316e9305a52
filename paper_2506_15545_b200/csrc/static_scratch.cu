// rattn_forward_static: the forward for callers that cannot allocate device memory.
//
// The tensor-core forward keeps the per-chunk states of the linear branch in scratch
// memory.  Every other entry point gets that scratch from the caller's workspace (or,
// for rattn_forward, from the stream-ordered pool).  Some callers can do neither: a
// serving process that has already handed all of the GPU's memory to its own cache
// manager, a plug-in that runs inside another framework's step and has no handle on that
// framework's allocator, or a latency-critical loop that must not take the driver's
// allocation lock.  For them the scratch lives in the fixed array below.  It is part of
// the library image, so every GPU that loads the library holds it until the process ends.
#include <cstring>
#include <mutex>

#include "rattn_internal.h"

namespace rattn {
namespace {

constexpr size_t kMatrices = RATTN_STATIC_MAX_CHUNK_STATES;
constexpr size_t kStatusBytes = 512;                       // status block + one progress word per K/V head (at most kMatrices)
constexpr size_t kStateBytes = kMatrices * 128 * 128 * sizeof(__nv_bfloat16);

// [status block, 256 B | progress words, 256 B | chunk states, bf16]
static __device__ __align__(256) unsigned char g_static_scratch[kStatusBytes + kStateBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
unsigned char* g_scratch_addr[kMaxDevices] = {};

// In host code the name `g_static_scratch` is only a handle for the symbol, not a device
// address; a kernel handed it would read the wrong memory.  The address is asked for once
// per device, with that device current, and remembered.
cudaError_t scratch_address(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_addr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    g_scratch_addr[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

int cuda_failure(cudaError_t e) {
  set_last_cuda_error(static_cast<int>(e));
  return RATTN_ERR_CUDA;
}

}  // namespace
}  // namespace rattn

using namespace rattn;

extern "C" int rattn_forward_static(const void* q, const void* k, const void* v, int B, int H_q, int H_kv,
                                    int T, int d, int w, float scale, void* out, void* stream) {
  if (!q || !k || !v || !out) return RATTN_ERR_NULL_PTR;
  if (B < 1 || H_q < 1 || H_kv < 1 || T < 1 || w < 1 || H_q % H_kv != 0 || !(scale == scale))
    return RATTN_ERR_BAD_ARG;
  if (d != 64 && d != 128) return RATTN_ERR_UNSUPPORTED;
  if ((((uintptr_t)q | (uintptr_t)k | (uintptr_t)v | (uintptr_t)out) & 15u) != 0) return RATTN_ERR_MISALIGNED;
  cudaStream_t s = reinterpret_cast<cudaStream_t>(stream);

  Args a;
  std::memset(&a, 0, sizeof(a));
  a.q = q; a.k = k; a.v = v; a.out = out;
  a.B = B; a.H_q = H_q; a.H_kv = H_kv; a.T = T; a.Tk = T; a.d = d; a.w = w;
  a.group = H_q / H_kv;
  a.dtype = RATTN_BF16; a.mode = RATTN_MODE_RATTN;
  a.scale = scale; a.eps = 1e-6f;

  cudaError_t e;
  if (!rattn_uses_tensor_path(d, w, RATTN_BF16, RATTN_MODE_RATTN, 0)) {
    // the portable kernel keeps everything on chip: no scratch involved
    e = launch_generic_forward(a, s);
    return e == cudaSuccess ? RATTN_OK : cuda_failure(e);
  }
  const int n_chunks = (T + 127) / 128;
  if ((size_t)B * H_kv * n_chunks > kMatrices) return RATTN_ERR_STATIC_LIMIT;
  unsigned char* base = nullptr;
  e = scratch_address(&base);
  if (e != cudaSuccess) return cuda_failure(e);
  a.status = reinterpret_cast<int*>(base);
  a.state_ready = reinterpret_cast<int*>(base + 256);
  a.chunk_state = reinterpret_cast<__nv_bfloat16*>(base + kStatusBytes);
  a.n_chunks = n_chunks;
  // The array keeps whatever the previous call left.  Only the status block (status word and
  // the forward's work counter) has to start at zero: every state the forward reads is rewritten
  // by this call's own pre-pass first.
  e = cudaMemsetAsync(base, 0, kStatusBytes, s);
  if (e != cudaSuccess) return cuda_failure(e);
  e = launch_tc_forward(a, s);
  return e == cudaSuccess ? RATTN_OK : cuda_failure(e);
}

extern "C" int rattn_static_status(void* stream) {
  unsigned char* base = nullptr;
  cudaError_t e = scratch_address(&base);
  if (e != cudaSuccess) return cuda_failure(e);
  return rattn_read_status(base, stream);
}
