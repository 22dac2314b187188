// heart_drift_static: the drift / refresh decision for callers that cannot hand the library a
// scratch buffer.  Its scratch lives in a fixed array inside the loaded library image instead.
#include <mutex>

#include "common.cuh"

using namespace heart;

namespace {

// The scratch itself: part of the module, so every GPU that loads the library carries these bytes
// until the process exits.  On the host this name is only a handle for cudaGetSymbolAddress -- it is
// not a device address and must never be passed to a kernel as one.
static __device__ __align__(256) unsigned char g_static_scratch[HEART_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_addr[kMaxDevices] = {};  // device address of g_static_scratch, per device ordinal

// Looks up (once per device, with that device current) where the array lives on the current device.
cudaError_t scratch_for_current_device(void **out) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_mu);
  if (g_scratch_addr[dev] == nullptr) {
    void *p = nullptr;
    e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr || (reinterpret_cast<uintptr_t>(p) & 255u)) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

}  // namespace

extern "C" {

int heart_drift_static(const heart_config *cfg, const void *Q, const void *K, const double *delta,
                       heart_state *st, double *drift_out, uint8_t *refresh_out, heart_stream_t stream) {
  if (cfg == nullptr) return HEART_ERR_INVALID;
  // Size check first, from the same accounting the caller-allocated path uses (the part of the
  // workspace that the drift kernels touch: the pooled-score area of the mask predictor lies behind it).
  Geom geom;
  const int shape_rc = make_geom(cfg, &geom);
  if (shape_rc != HEART_OK) return shape_rc;  // the code heart_drift gives for this cfg
  const size_t need = heart_drift_workspace_bytes(cfg);
  if (need > (size_t)HEART_STATIC_SCRATCH_BYTES) return HEART_ERR_TOO_LARGE;
  if (!Q || !K || !delta || !st || !st->anchor_q || !st->anchor_k || !st->has_anchor) return HEART_ERR_INVALID;
  if ((reinterpret_cast<uintptr_t>(Q) & 15u) || (reinterpret_cast<uintptr_t>(K) & 15u)) return HEART_ERR_INVALID;
  void *scratch = nullptr;
  cudaError_t e = scratch_for_current_device(&scratch);
  if (e != cudaSuccess) return HEART_ERR_CUDA;
  // From here on this is heart_drift with the library's own scratch in place of the caller's.
  heart_state full = *st;
  // heart_drift insists on a complete state; this entry point never touches the mask fields, so give
  // placeholders that satisfy the null checks without being dereferenced by the drift kernels.
  if (!full.mask_bits) full.mask_bits = reinterpret_cast<uint32_t *>(scratch);
  if (!full.kv_idx) full.kv_idx = reinterpret_cast<int32_t *>(scratch);
  if (!full.kv_cnt) full.kv_cnt = reinterpret_cast<int32_t *>(scratch);
  // The one word the kernels expect at zero (the gate's ticket counter): an earlier pair of calls that
  // overlapped on the GPU may have left it anywhere, and the caller has no handle on this array.
  e = cudaMemsetAsync(static_cast<int32_t *>(scratch) + kStatusTicketWord, 0, sizeof(int32_t),
                      static_cast<cudaStream_t>(stream));
  if (e != cudaSuccess) return HEART_ERR_CUDA;
  return heart_drift(cfg, Q, K, delta, &full, drift_out, refresh_out, scratch, stream);
}

}  // extern "C"
