// Host-side entry points that launch nothing heavy: status word, strings, anchor count, workspace size.
#include <cfenv>
#include <cmath>

#include "common.cuh"

namespace relaxkv {

__device__ DeviceStatus g_status_word;

DeviceStatus* status_word() {
  // One lookup per device; the address of a __device__ variable differs between devices.
  static std::atomic<DeviceStatus*> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  DeviceStatus* p = cached[dev].load(std::memory_order_acquire);
  if (!p) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_status_word) != cudaSuccess) return nullptr;
    p = static_cast<DeviceStatus*>(q);
    cached[dev].store(p, std::memory_order_release);
  }
  return p;
}

int sm_count_of_current_device() {
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 0;
  int n = cached[dev].load(std::memory_order_acquire);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n < 1) return 0;
    cached[dev].store(n, std::memory_order_release);
  }
  return n;
}

static std::atomic<int> g_chained_launch{1};
bool chained_launch_enabled() { return g_chained_launch.load(std::memory_order_relaxed) != 0; }

}  // namespace relaxkv

using namespace relaxkv;

extern "C" int32_t relaxkv_set_chained_launch(int32_t on) {
  return g_chained_launch.exchange(on ? 1 : 0, std::memory_order_relaxed);
}

extern "C" const char* relaxkv_status_string(int32_t status) {
  switch (status) {
    case RELAXKV_OK: return "ok";
    case RELAXKV_ERR_INVALID_ARG: return "invalid argument";
    case RELAXKV_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case RELAXKV_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case RELAXKV_ERR_CUDA: return "CUDA error";
    case RELAXKV_ERR_BAD_INDEX: return "bad index seen on the device";
    case RELAXKV_ERR_TIMEOUT: return "bounded device wait expired";
    default: return "unknown status";
  }
}

extern "C" int32_t relaxkv_anchor_count(int32_t ctx_len, double ratio) {
  if (ctx_len < 1) return 0;
  const int old = std::fegetround();
  std::fesetround(FE_TONEAREST);
  double x = std::nearbyint(ratio * static_cast<double>(ctx_len));
  std::fesetround(old);
  long long k = static_cast<long long>(x);
  if (k < 1) k = 1;
  if (k > ctx_len) k = ctx_len;
  return static_cast<int32_t>(k);
}

extern "C" size_t relaxkv_workspace_bytes(const relaxkv_shape* shape, int32_t n_layers, const int32_t* /*h_k*/) {
  if (check_shape(shape) != RELAXKV_OK || n_layers < 1) return 0;
  return ws_layout(shape, n_layers).total;
}

extern "C" relaxkv_status relaxkv_read_device_status(int32_t* h_status_out, int32_t* h_detail_out,
                                                     relaxkv_stream stream) {
  RELAXKV_RANGE("relaxkv_read_device_status");
  if (!h_status_out) return RELAXKV_ERR_INVALID_ARG;
  DeviceStatus* st = status_word();
  if (!st) return RELAXKV_ERR_CUDA;
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  DeviceStatus h{};
  if (cudaMemcpyAsync(&h, st, sizeof(h), cudaMemcpyDeviceToHost, s) != cudaSuccess) return RELAXKV_ERR_CUDA;
  if (cudaMemsetAsync(st, 0, sizeof(h), s) != cudaSuccess) return RELAXKV_ERR_CUDA;
  if (cudaStreamSynchronize(s) != cudaSuccess) return RELAXKV_ERR_CUDA;
  *h_status_out = h.status;
  if (h_detail_out) {
    h_detail_out[0] = h.kernel; h_detail_out[1] = h.block; h_detail_out[2] = h.v0; h_detail_out[3] = h.v1;
  }
  return RELAXKV_OK;
}
