// hswa_decode_attn_static_ws: decode attention whose split-K scratch lives in a fixed device array that is
// part of this library's image, for callers that must not allocate device memory.
//
// Who needs it: code that runs where an allocation is off limits -- a serving loop that was handed a fixed
// memory budget and has none left to carve a workspace from, a plugin that may only touch the buffers it was
// given, or a latency-critical section in which cudaMalloc's implicit device synchronisation is not
// acceptable.  Such callers still pass q, k_new, v_new, out and lse; only the scratch comes from here.
#include <mutex>

#include "hswa_internal.cuh"

namespace {

// The scratch itself.  Every GPU that loads this library holds these bytes until the process exits.
static __device__ __align__(256) unsigned char g_static_ws[HSWA_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_ws_addr[kMaxDevices] = {};  // device address of g_static_ws on each device, resolved on first use

// In host code the name g_static_ws is only a stand-in for the symbol, not an address a kernel can use:
// the device address must be asked for, once per device, with that device current.
hswa_status static_ws_address(int device, void** out) {
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_ws_addr[device] == nullptr) {
    void* ptr = nullptr;
    if (cudaGetSymbolAddress(&ptr, g_static_ws) != cudaSuccess || ptr == nullptr) return HSWA_ERR_CUDA;
    g_ws_addr[device] = ptr;
  }
  *out = g_ws_addr[device];
  return HSWA_OK;
}

}  // namespace

extern "C" hswa_status hswa_decode_attn_static_ws(hswa_handle* h, const hswa_layer* layer, const hswa_batch* batch,
                                                  const void* q, const void* k_new, const void* v_new, void* out,
                                                  float* lse, void* stream) {
  if (!h) return HSWA_ERR_INVALID_ARG;
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess) return HSWA_ERR_CUDA;
  if (dev != h->device || dev < 0 || dev >= kMaxDevices) return HSWA_ERR_INVALID_ARG;
  void* ws = nullptr;
  const hswa_status st = static_ws_address(dev, &ws);
  if (st != HSWA_OK) return st;
  // hswa_decode_attn computes the exact scratch need of this batch and answers HSWA_ERR_WORKSPACE, launching
  // nothing, when it exceeds the bytes offered: that is the size limit of this entry point.
  return hswa_decode_attn(h, layer, batch, q, k_new, v_new, out, lse, ws, (size_t)HSWA_STATIC_WS_BYTES, stream);
}
