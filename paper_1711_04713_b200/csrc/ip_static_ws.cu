// adaption_lp_ip_fwd_static_ws: LPInnerProduct forward for callers that cannot allocate device
// memory.  The split-K scratch (the int64 partial-sum matrix that adaption_lp_ip_fwd takes as a
// caller-owned workspace) lives in a fixed array inside the library image instead.
#include <mutex>

#include "common.cuh"

namespace {

// The scratch itself: part of the library image, present on every GPU that loads the library
// until the process exits.  Its name is only meaningful to device code; host code must ask the
// runtime for the device address (see scratch_address below).
static __device__ __align__(256) unsigned char g_ip_static_ws[ADAPTION_STATIC_WORKSPACE_BYTES];

constexpr int kMaxDevices = 64;
void* g_ws_addr[kMaxDevices] = {};
std::mutex g_ws_mutex;

// Device address of the scratch array on the current device, looked up once per device.  (The
// cached address belongs to the device's current primary context: after a cudaDeviceReset the
// process must not call this entry point on that device again.)
int scratch_address(void** out) {
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return ADAPTION_ERR_CUDA;
  std::lock_guard<std::mutex> lock(g_ws_mutex);
  if (g_ws_addr[dev] == nullptr) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_ip_static_ws) != cudaSuccess || p == nullptr) {
      (void)cudaGetLastError();
      return ADAPTION_ERR_CUDA;
    }
    g_ws_addr[dev] = p;
  }
  *out = g_ws_addr[dev];
  return ADAPTION_OK;
}

}  // namespace

extern "C" int adaption_lp_ip_fwd_static_ws(int64_t B, int64_t K, int64_t O, adaption_qtensor x,
                                            adaption_qtensor w, const int16_t* d_bias_q,
                                            int32_t bias_frac_bits, int32_t relu, int32_t mode, int32_t algo,
                                            adaption_qtensor y, adaption_stats* d_stats, void* stream) {
  const size_t need = adaption_lp_ip_workspace_bytes(B, K, O, x.fmt, w.fmt, algo);
  if (need > (size_t)ADAPTION_STATIC_WORKSPACE_BYTES) return ADAPTION_ERR_WORKSPACE;
  void* ws = nullptr;
  if (need > 0) {
    const int rc = scratch_address(&ws);
    if (rc != ADAPTION_OK) return rc;
  }
  // The regular entry point zeroes the part of the workspace it uses before accumulating into
  // it, so whatever an earlier call left in the array does not matter.
  return adaption_lp_ip_fwd(B, K, O, x, w, d_bias_q, bias_frac_bits, relu, mode, algo, y, d_stats, ws,
                            need > 0 ? (size_t)ADAPTION_STATIC_WORKSPACE_BYTES : 0, stream);
}
