// Backward pass for callers that cannot hand the library a workspace: the scratch that nsp_attn_bwd normally
// takes from the caller (the fp32 dQ accumulator and the delta vector) lives in a fixed array inside the
// library image instead.
//
// Who needs this: a training executor that has given every byte of device memory to its own planner or
// caching pool before the first iteration, so that neither it nor the library may call cudaMalloc later
// (a raw allocation synchronises the whole device, can fail when the pool already owns the memory, and is
// forbidden outright inside some schedulers' critical sections). Such a caller still owns its inputs and
// outputs, which its planner sized up front, but has nowhere to put a transient q-sized fp32 buffer.
//
// Cost: every GPU on which the module of this file is loaded carries NSP_STATIC_WS_BYTES of global memory until
// the process exits. With lazy module loading (the CUDA default) the module is loaded, and the memory reserved, by
// the first cudaGetSymbolAddress on that device, i.e. inside the first call of the entry point: that call belongs at
// start-up, before the caller's pool has taken the rest of the memory. All calls share the one array. It keeps whatever the previous call left in it; the part
// that has to start at zero (the dQ accumulator) is cleared on the stream at the start of every call. Two calls
// whose device work overlaps in time (different streams, or different host threads) race on the array.
#include <mutex>
#include <cuda_runtime.h>
#include "../../include/nsp.h"

namespace {

// The array's name is only a handle on the host side; the device address comes from cudaGetSymbolAddress.
static __device__ __align__(256) unsigned char g_static_ws[NSP_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_ws_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device, resolved once per device.
int static_ws_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return NSP_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) {
      cudaGetLastError();
      return NSP_ERR_CUDA;
    }
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
  return NSP_OK;
}

}  // namespace

extern "C" int nsp_attn_bwd_static(const nsp_plan_t* plan, const void* q, const void* k, const void* v, const void* o,
                                   const void* d_o, const float* lse, void* dq, void* dk, void* dv, int dq_dtype,
                                   int dkv_dtype, float softmax_scale, void* stream) {
  if (!plan) return NSP_ERR_INVALID_ARG;
  size_t need = 0;
  const int rc = nsp_plan_sizes(plan, nullptr, nullptr, nullptr, nullptr, &need);
  if (rc != NSP_OK) return rc;
  if (need > static_cast<size_t>(NSP_STATIC_WS_BYTES)) return NSP_ERR_WORKSPACE;  // batch too large for the fixed array
  void* ws = nullptr;
  const int rs = static_ws_address(&ws);
  if (rs != NSP_OK) return rs;
  // Same kernels as nsp_attn_bwd; it clears the accumulator part of the scratch on `stream` before using it.
  return nsp_attn_bwd(plan, q, k, v, o, d_o, lse, dq, dk, dv, dq_dtype, dkv_dtype, softmax_scale, ws,
                      static_cast<size_t>(NSP_STATIC_WS_BYTES), stream);
}
