// metis_linear_fwd_static_ws: the forward layer for callers that cannot hand the library a workspace.
//
// Who needs this: code that runs after a process has committed all of its device memory up front
// (a serving process whose framework pool owns every free byte, so a late cudaMalloc fails), and
// plug-in style callers that are handed tensors but are not allowed to call an allocator at all.
// Such a caller has inputs and outputs but nowhere to put the layer's intermediate operands.  This
// entry point keeps those intermediates in a fixed array that is part of the library image itself.
#include <mutex>

#include "common.cuh"

namespace {

constexpr size_t STATIC_WS_BYTES = METIS_STATIC_WS_BYTES;

// Part of the module image: every GPU that loads the library holds these 4 MiB until the process exits.
static __device__ __align__(256) unsigned char g_static_ws[STATIC_WS_BYTES];

constexpr int MAX_DEVICES = 64;
void* g_ws_addr[MAX_DEVICES] = {};     // device address of g_static_ws on each device, filled at first use
std::mutex g_ws_mutex;

// In host code the name g_static_ws is only a handle for the runtime, not a device address: the address a
// kernel can use has to be asked for, once per device, while that device is current.
metis_status_t static_ws_address(int device, void** out) {
  if (device < 0 || device >= MAX_DEVICES) return METIS_ERR_INVALID_ARG;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  if (g_ws_addr[device] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || p == nullptr) return METIS_ERR_CUDA;
    g_ws_addr[device] = p;
  }
  *out = g_ws_addr[device];
  return METIS_OK;
}

}  // namespace

extern "C" metis_status_t metis_linear_fwd_static_ws(metis_handle_t h, const metis_operand_t* x, const metis_operand_t* w,
                                                     void* y, int32_t y_dtype, int64_t ldy, metis_stream_t stream) {
  METIS_NVTX("metis_linear_fwd_static_ws");
  if (!h || !x || !w || !y) return METIS_ERR_INVALID_ARG;
  int current = -1;
  if (cudaGetDevice(&current) != cudaSuccess) return METIS_ERR_CUDA;
  if (current != h->device) return METIS_ERR_INVALID_ARG;          // the handle's device must be the current one
  void* ws = nullptr;
  METIS_TRY(static_ws_address(current, &ws));
  // Nothing in the array has to start at zero: every intermediate the layer reads back is written earlier in
  // the same call, so the previous call's contents are simply overwritten.  metis_linear_fwd lays its
  // intermediates out inside the bytes it is given and refuses, before it enqueues anything, a layer whose
  // intermediates do not fit (METIS_ERR_WORKSPACE); argument and shape errors are reported as usual.
  return metis_linear_fwd(h, x, w, y, y_dtype, ldy, ws, STATIC_WS_BYTES, stream);
}
