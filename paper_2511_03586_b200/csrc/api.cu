// Status handling, device checks and the device status word of the pd library.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstdlib>

#include "pd_common.cuh"

namespace pd {
namespace {

thread_local int tl_last_cuda_error = 0;
constexpr int kMaxDevices = 64;

// Written by the bounded waits of the tensor-core kernels when they give up.
__device__ int g_device_status;

}  // namespace

namespace {
std::atomic<uint64_t> g_wait_limit_ns{2000000000ull};
std::atomic<int> g_withhold_loads{0};
}  // namespace
uint64_t debug_wait_limit_ns() { return g_wait_limit_ns.load(std::memory_order_relaxed); }
int debug_withhold_loads() { return g_withhold_loads.load(std::memory_order_relaxed); }

bool log_enabled() {
  static const bool on = [] {
    const char* v = std::getenv("PD_LOG");
    return v != nullptr && v[0] != '\0' && v[0] != '0';
  }();
  return on;
}
void logf(const char* fmt, ...) {
  if (!log_enabled()) return;
  va_list ap;
  va_start(ap, fmt);
  std::fputs("pd: ", stderr);
  std::vfprintf(stderr, fmt, ap);
  std::fputc('\n', stderr);
  va_end(ap);
}

pd_status record_cuda_error(cudaError_t e) {
  if (e == cudaSuccess) return PD_OK;
  tl_last_cuda_error = (int)e;
  return PD_ERR_CUDA;
}

pd_status require_sm100() {
  // The per-device caches of this file are atomics: concurrent first calls from several host threads each
  // query the device and store the same value.
  static std::atomic<int> cached_major[kMaxDevices];  // 0 = not queried yet
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return record_cuda_error(e);
  if (dev < 0 || dev >= kMaxDevices) return PD_ERR_UNSUPPORTED;
  int major = cached_major[dev].load(std::memory_order_relaxed);
  if (major == 0) {
    e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
    if (e != cudaSuccess) return record_cuda_error(e);
    major = major > 0 ? major : -1;
    cached_major[dev].store(major, std::memory_order_relaxed);
  }
  return major == 10 ? PD_OK : PD_ERR_UNSUPPORTED;
}

int sm_count() {
  static std::atomic<int> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return 148;
  int n = cached[dev].load(std::memory_order_relaxed);
  if (n == 0) {
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
    cached[dev].store(n, std::memory_order_relaxed);
  }
  return n;
}

int* device_status_ptr() {
  static std::atomic<int*> cached[kMaxDevices];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
  int* q = cached[dev].load(std::memory_order_acquire);
  if (!q) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_device_status) != cudaSuccess) return nullptr;
    q = static_cast<int*>(p);
    cached[dev].store(q, std::memory_order_release);
  }
  return q;
}

}  // namespace pd

extern "C" const char* pd_status_string(pd_status status) {
  switch (status) {
    case PD_OK: return "PD_OK";
    case PD_ERR_NULL_POINTER: return "PD_ERR_NULL_POINTER";
    case PD_ERR_BAD_SHAPE: return "PD_ERR_BAD_SHAPE";
    case PD_ERR_UNSUPPORTED: return "PD_ERR_UNSUPPORTED";
    case PD_ERR_ALIGNMENT: return "PD_ERR_ALIGNMENT";
    case PD_ERR_WORKSPACE_TOO_SMALL: return "PD_ERR_WORKSPACE_TOO_SMALL";
    case PD_ERR_CUDA: return "PD_ERR_CUDA";
    case PD_ERR_DEVICE_TIMEOUT: return "PD_ERR_DEVICE_TIMEOUT";
  }
  return "PD_ERR_UNKNOWN";
}

extern "C" int pd_last_cuda_error(void) { return pd::tl_last_cuda_error; }

extern "C" pd_status pd_get_device_status(int* code) {
  if (!code) return PD_ERR_NULL_POINTER;
  int* p = pd::device_status_ptr();
  if (!p) return PD_ERR_CUDA;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemcpy(code, p, sizeof(int), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return pd::record_cuda_error(e);
  return *code == 0 ? PD_OK : PD_ERR_DEVICE_TIMEOUT;
}

extern "C" pd_status pd_clear_device_status(void) {
  int* p = pd::device_status_ptr();
  if (!p) return PD_ERR_CUDA;
  cudaError_t e = cudaDeviceSynchronize();
  if (e == cudaSuccess) e = cudaMemset(p, 0, sizeof(int));
  return pd::record_cuda_error(e);
}

extern "C" pd_status pd_debug_set_wait_limit_ns(uint64_t limit_ns) {
  if (limit_ns < 1000ull || limit_ns > 10000000000ull) return PD_ERR_BAD_SHAPE;
  pd::g_wait_limit_ns.store(limit_ns, std::memory_order_relaxed);
  return PD_OK;
}

extern "C" pd_status pd_debug_withhold_loads(int on) {
  if (on < 0 || on > 1) return PD_ERR_BAD_SHAPE;
  pd::g_withhold_loads.store(on, std::memory_order_relaxed);
  return PD_OK;
}
