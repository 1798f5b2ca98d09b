// us_linear_fwd_static_ws: the forward linear op for callers that cannot provide a workspace.
//
// The linear kernels need a few bytes of global scratch (the status word a kernel raises when
// one of its bounded waits gives up).  Normally the caller allocates that workspace.  Some
// callers cannot: a plug-in that is handed nothing but its input and output buffers by the
// runtime that hosts it, a serving loop that forbids allocation after start-up because
// cudaMalloc stalls the whole device, or a process whose framework has already reserved all
// device memory for its own pool.  For them the scratch lives here, in a fixed array inside the
// library image; nothing is allocated or freed, by this code or through any library.
#include <cuda_runtime.h>

#include "../../include/unitscale.h"

namespace {

// Capacity of the built-in scratch.  Every GPU that loads the library holds these bytes until
// the process exits.
constexpr size_t kStaticWsBytes = 1024;

__device__ __align__(256) unsigned char g_static_ws[kStaticWsBytes];

constexpr int kMaxDevices = 64;
// Device address of g_static_ws on each device, 0 = not set up.  Written without a lock: threads that race
// on the first call of a device all store the same value.
void* g_ws_addr[kMaxDevices];

// In host code `g_static_ws` names a host-side shadow of the symbol, not device memory, so it
// must never be handed to a kernel.  Ask the runtime for the real address, once per device,
// with that device current.
us_status static_ws_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return US_ERR_CUDA;
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return US_ERR_CUDA;
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
  return US_OK;
}

}  // namespace

extern "C" us_status us_linear_fwd_static_ws(const us_mat* X, const us_mat* W, float alpha, const us_epilogue* ep,
                                             const us_mat* Y, void** ws_out, void* stream) {
  // The scratch the kernel needs does not grow with the problem; should a later version need
  // more than the built-in array holds, refuse instead of overrunning it.
  if (us_workspace_bytes() > kStaticWsBytes) return US_ERR_WORKSPACE;
  void* ws = nullptr;
  us_status s = static_ws_address(&ws);
  if (s != US_OK) return s;
  // Every host-side check of us_linear_fwd first, so that a call with bad arguments enqueues nothing
  // (no clearing of the status word either) and leaves the previous call's status readable.
  s = us_linear_fwd_check(X, W, ep, Y, ws, kStaticWsBytes);
  if (s != US_OK) return s;
  // The array keeps whatever the previous call left in it: the status word has to start at zero.
  if (cudaMemsetAsync(ws, 0, us_workspace_bytes(), static_cast<cudaStream_t>(stream)) != cudaSuccess)
    return US_ERR_CUDA;
  if (ws_out) *ws_out = ws;
  return us_linear_fwd(X, W, alpha, ep, Y, ws, kStaticWsBytes, stream);
}
