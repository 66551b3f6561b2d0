// Status strings, thread-local error text and the device status word.
#include <atomic>
#include <mutex>

#include "common.cuh"

namespace szo {

thread_local int64_t g_launch_count = 0;

// Bumped whenever szo_device_status reads a non-zero status word: a kernel that gave up may have left
// the self-resetting K-split tickets of its plan non-zero; plans compare their own copy of this
// counter before a launch and clear their tickets when it has moved (gemm_tc.cu).
std::atomic<uint64_t> g_abort_epoch{0};

char* last_error_buffer() {
  static thread_local char buf[512] = {0};
  return buf;
}

szo_status fail(szo_status code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(last_error_buffer(), 512, fmt, ap);
  va_end(ap);
  return code;
}

uint64_t abort_epoch() { return g_abort_epoch.load(); }

int32_t* device_status_word() {
  static int32_t* words[64] = {nullptr};
  static std::mutex mu;
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(mu);
  if (!words[dev]) {
    int32_t* p = nullptr;
    if (cudaMalloc(&p, sizeof(int32_t)) != cudaSuccess) return nullptr;
    cudaMemset(p, 0, sizeof(int32_t));
    words[dev] = p;
  }
  return words[dev];
}

}  // namespace szo

extern "C" {

const char* szo_status_string(szo_status s) {
  switch (s) {
    case SZO_OK: return "SZO_OK";
    case SZO_ERR_INVALID_ARG: return "SZO_ERR_INVALID_ARG";
    case SZO_ERR_SHAPE: return "SZO_ERR_SHAPE";
    case SZO_ERR_ALIGNMENT: return "SZO_ERR_ALIGNMENT";
    case SZO_ERR_UNSUPPORTED: return "SZO_ERR_UNSUPPORTED";
    case SZO_ERR_WORKSPACE: return "SZO_ERR_WORKSPACE";
    case SZO_ERR_CUDA: return "SZO_ERR_CUDA";
    case SZO_ERR_NONFINITE: return "SZO_ERR_NONFINITE";
    case SZO_ERR_TIMEOUT: return "SZO_ERR_TIMEOUT";
    default: return "SZO_ERR_UNKNOWN";
  }
}

const char* szo_last_error(void) { return szo::last_error_buffer(); }

int szo_version(void) { return 100; }

szo_status szo_device_status(int32_t* status_host) {
  SZO_REQUIRE(status_host != nullptr, SZO_ERR_INVALID_ARG, "status_host is NULL");
  int32_t* w = szo::device_status_word();
  SZO_REQUIRE(w != nullptr, SZO_ERR_CUDA, "no device status word (no CUDA device?)");
  SZO_CHECK_CUDA(cudaDeviceSynchronize());
  SZO_CHECK_CUDA(cudaMemcpy(status_host, w, sizeof(int32_t), cudaMemcpyDeviceToHost));
  SZO_CHECK_CUDA(cudaMemset(w, 0, sizeof(int32_t)));
  if (*status_host != 0) szo::g_abort_epoch.fetch_add(1);
  return SZO_OK;
}

}  // extern "C"
