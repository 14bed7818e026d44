// lrsa_score_select_static: the scoring/selection call for callers that cannot hand the library
// any device memory of their own for scratch and cannot let it allocate either.
//
// Who that is: code that runs where every byte of HBM is already spoken for or where the CUDA
// allocator must not be entered - for example a plugin inside a training or serving process whose
// caching allocator has reserved the whole device (a raw cudaMalloc there fails or steals from the
// pool), or a latency-critical loop that cannot afford the device-wide synchronisation cudaMalloc
// and cudaFree imply.  Such a caller still owns its inputs and outputs, but has nowhere to put the
// few megabytes of counters, per-window statistics and per-token spreads the kernel needs.
//
// The scratch therefore lives in a fixed array in this library's device image.  Every GPU that
// loads the library carries those LRSA_STATIC_SCRATCH_BYTES until the process exits, used or not.
#include <mutex>

#include "lrsa_internal.h"

namespace {

// The scratch itself.  In host code this name is only a handle for the runtime's symbol table; the
// device address is looked up below and that pointer is what the kernel receives.
static __device__ __align__(256) unsigned char g_static_scratch[LRSA_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

// Device address of the array on the CURRENT device, resolved once per device.
int static_scratch(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return LRSA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return LRSA_ERR_CUDA;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return LRSA_OK;
}

}  // namespace

extern "C" int lrsa_score_select_static(const lrsa_params_t* params, const void* K, const void* V,
                                        int32_t* idx, float* score, void* cuda_stream) {
  using namespace lrsa;
  NvtxRange nvtx_range("lrsa_score_select_static");
  launch_counter().n = 0;
  Geom g;
  const int rc = make_geom(params, &g);
  if (rc != LRSA_OK) return rc;
  if (!K || !V) return LRSA_ERR_INVALID_ARG;
  if (g.Wtot > 0 && !idx) return LRSA_ERR_INVALID_ARG;
  auto misaligned = [](const void* p, size_t a) { return reinterpret_cast<uintptr_t>(p) % a != 0; };
  if (misaligned(K, 16) || misaligned(V, 16) || misaligned(idx, 4) || misaligned(score, 4))
    return LRSA_ERR_INVALID_ARG;
  // the problem must fit the fixed array: nothing larger is attempted
  if (score_select_ws_bytes(g) > (size_t)LRSA_STATIC_SCRATCH_BYTES) return LRSA_ERR_WORKSPACE_TOO_SMALL;
  void* scratch = nullptr;
  const int sc = static_scratch(&scratch);
  if (sc != LRSA_OK) return sc;
  // The status word, counters and statistics that must start at zero are cleared on the stream before the
  // kernel; whatever else the previous call left in the array is overwritten before it is read.
  return run_score_select(params, g, static_cast<const __nv_bfloat16*>(K), static_cast<const __nv_bfloat16*>(V),
                          idx, score, scratch, static_cast<cudaStream_t>(cuda_stream));
}

// Status word of the last lrsa_score_select_static call on the current device (the first word of the
// fixed array).  Waits for `cuda_stream`, copies four bytes, allocates nothing.
extern "C" int lrsa_score_select_static_status(void* cuda_stream) {
  void* scratch = nullptr;
  const int sc = static_scratch(&scratch);
  if (sc != LRSA_OK) return sc;
  return lrsa_workspace_status(scratch, cuda_stream);
}
