// ahakv_score_static: the eviction score with its scratch memory inside the library.
//
// Some callers cannot hand ahakv_score a workspace because they cannot allocate device memory at the
// point of the call: a serving loop whose memory pool was sized once and is closed to new requests,
// a plug-in that is given tensors but no allocator, code that runs where cudaMalloc is not allowed
// (it synchronises the device and may fail late under memory pressure).  For them the scratch lives
// here, in a fixed device array that every GPU holds from the moment the library is loaded until the
// process exits, and the entry point makes no allocation of any kind.
#include <mutex>

#include "ahakv_internal.cuh"

namespace {

// The scratch itself.  In host code this name stands for the symbol, not for a device address: the
// address the kernels need comes from cudaGetSymbolAddress, asked once per device (below).
static __device__ __align__(256) unsigned char g_static_ws[AHAKV_STATIC_WS_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void* g_ws_addr[kMaxDevices];   // device address of g_static_ws on each device, nullptr until asked

// Address of the array on the current device.  The first call on a device asks the runtime (with that
// device current, as the caller has it); later calls read the table.
ahakv_status static_ws_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return AHAKV_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_ws_addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_static_ws) != cudaSuccess || !p) return AHAKV_ERR_CUDA;
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
  return AHAKV_OK;
}

}  // namespace

extern "C" {

size_t ahakv_static_workspace_bytes(void) { return (size_t)AHAKV_STATIC_WS_BYTES; }

ahakv_status ahakv_score_static(const ahakv_params* p, const void* q_obs, const void* k, const void* v,
                                const float* score_prev, float* score, ahakv_stream_t stream) {
  ahakv::Plan pl;
  ahakv_status rc = ahakv::make_plan(p, &pl);                     // the same verdict on the parameters as ahakv_score's
  if (rc != AHAKV_OK) return rc;
  if (pl.ws_total > (size_t)AHAKV_STATIC_WS_BYTES) return AHAKV_ERR_WORKSPACE;   // too large for the built-in scratch
  void* ws = nullptr;
  rc = static_ws_address(&ws);
  if (rc != AHAKV_OK) return rc;
  // Same kernels, same order as ahakv_score; it clears the words of the scratch that must start at
  // zero (and marks the run partials "not published") itself, so what the last call left is harmless.
  return ahakv_score(p, q_obs, k, v, score_prev, score, ws, (size_t)AHAKV_STATIC_WS_BYTES, stream);
}

// The status word the kernels of the last ahakv_score_static call on this device left at the head of the
// array: AHAKV_OK, or AHAKV_ERR_TIMEOUT if a bounded device-side wait gave up.  Synchronises `stream`.
ahakv_status ahakv_static_last_device_status(ahakv_stream_t stream) {
  void* ws = nullptr;
  const ahakv_status rc = static_ws_address(&ws);
  if (rc != AHAKV_OK) return rc;
  return ahakv_last_device_status(ws, stream);
}

}  // extern "C"
