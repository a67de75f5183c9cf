// la_fwd_noalloc: the forward pass for callers that cannot provide scratch memory.
//
// la_fwd cuts a long sequence into segments and needs device scratch for the per-segment
// states (its `workspace` argument), which the caller normally allocates.  Some callers
// cannot allocate at the time they call: a serving process that handed every byte of device
// memory to its own pool at start-up and treats any later cudaMalloc as a bug, a
// latency-critical loop that cannot afford the device-wide synchronisation an allocation
// implies, or a plug-in that only receives tensor pointers and a stream and has no allocator
// to ask.  For them the scratch lives here, in a fixed array in the library's own device image.
//
// Cost and limits: every GPU that loads the library holds LA_NOALLOC_SCRATCH_BYTES (32 MiB)
// until the process exits.  With lazy module loading the array may only come into being when
// its address is first asked for, so the first call on a device is the warm-up that can fail
// for lack of room: make it before a pool takes the remaining device memory (and before any
// stream capture).  A shape whose la_workspace_bytes(LA_OP_FWD, ..) exceeds that is
// rejected with LA_ERR_SCRATCH_LIMIT before anything is launched.  All calls on a device share
// the one array, so two calls that may overlap on the GPU (different streams) race on it; calls
// on one stream are safe.  The array keeps whatever the previous call left, which is harmless:
// the forward pass writes every scratch element it later reads (the pre-pass fills all
// segment-local states before the scan reads them), so nothing has to start at zero.
//
// This file makes no cudaMalloc / cudaFree call and calls no allocating library routine.
#include <cuda_runtime.h>

#include <mutex>

#include "../../include/la.h"

namespace {

// The name `g_noalloc_scratch` is only a host-side handle here: passing it to a kernel would hand
// the kernel a host address.  The device address is asked for once per device (below).
static __device__ __align__(256) unsigned char g_noalloc_scratch[LA_NOALLOC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {nullptr};

// Device address of the scratch array on the current device; resolved on the first call per
// device, with that device current, and remembered.
la_status scratch_for_current_device(void** out) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return LA_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return LA_ERR_UNSUPPORTED;
  std::lock_guard<std::mutex> lock(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_noalloc_scratch) != cudaSuccess || !p) {
      cudaGetLastError();  // leave no stale error behind in the runtime for the caller's next call
      return LA_ERR_CUDA;
    }
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return LA_OK;
}

}  // namespace

extern "C" la_status la_fwd_noalloc(const la_shape* shape, const void* q, const void* k, const void* v,
                                    const float* lambda_host, void* o, const float* kv_in, float* kv_out,
                                    void* stream) {
  const size_t need = la_workspace_bytes(LA_OP_FWD, shape);
  if (need == (size_t)-1) {
    // let la_fwd produce the precise argument error (it fails before launching anything)
    return la_fwd(shape, q, k, v, lambda_host, o, kv_in, kv_out, nullptr, 0, stream);
  }
  if (need > (size_t)LA_NOALLOC_SCRATCH_BYTES) return LA_ERR_SCRATCH_LIMIT;
  void* scratch = nullptr;
  if (need > 0) {
    const la_status st = scratch_for_current_device(&scratch);
    if (st != LA_OK) return st;
  }
  return la_fwd(shape, q, k, v, lambda_host, o, kv_in, kv_out, scratch, need > 0 ? (size_t)LA_NOALLOC_SCRATCH_BYTES : 0,
                stream);
}
