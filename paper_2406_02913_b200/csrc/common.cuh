// Shared host-side helpers of the szo library: error reporting, argument checks, and the
// declarations of the internal launchers that the model driver calls directly.
#pragma once
#include <cstdlib>
#include <cuda_bf16.h>
#include <cuda_fp16.h>
#include <cuda_runtime.h>

#include <cstdarg>
#include <cstdint>
#include <cstdio>

#include "../../include/szo.h"

namespace szo {

// Thread-local detail string behind szo_last_error().
char* last_error_buffer();
szo_status fail(szo_status code, const char* fmt, ...);

// Device status word (one per device, allocated on first use on the current device).
int32_t* device_status_word();
// Host-side count of non-zero status reads (see status.cu).
uint64_t abort_epoch();

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline size_t dtype_size(int dt) { return dt == SZO_F32 ? 4 : 2; }
inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
inline size_t round_up(size_t a, size_t b) { return (a + b - 1) / b * b; }

#define SZO_CHECK_CUDA(expr)                                                              \
  do {                                                                                    \
    cudaError_t e__ = (expr);                                                             \
    if (e__ != cudaSuccess)                                                               \
      return ::szo::fail(SZO_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__));  \
  } while (0)

#define SZO_CHECK_LAUNCH(name)                                                            \
  do {                                                                                    \
    cudaError_t e__ = cudaGetLastError();                                                 \
    if (e__ != cudaSuccess)                                                               \
      return ::szo::fail(SZO_ERR_CUDA, "launch of %s failed: %s", name,                   \
                         cudaGetErrorString(e__));                                        \
  } while (0)

#define SZO_REQUIRE(cond, code, ...)                    \
  do {                                                  \
    if (!(cond)) return ::szo::fail(code, __VA_ARGS__); \
  } while (0)

#define SZO_TRY(expr)                    \
  do {                                   \
    szo_status s__ = (expr);             \
    if (s__ != SZO_OK) return s__;       \
  } while (0)

// Chained launches (programmatic dependent launch).  A token step is a chain of short kernels, each
// reading what the one before wrote; launched `chained`, a kernel may be placed on the SMs while its
// predecessor drains and do there whatever does not depend on it (the weight-streaming kernels start
// reading their weights).  Rules for a kernel that may be launched this way: chain_release() first
// (lets ITS successor be placed early), chain_wait() before the first access to anything an earlier
// kernel of the stream wrote or still reads.  chain_wait returns only when the predecessor grid has
// completed and its writes are visible, so the kernels of a chain still run their dependent parts in
// order.  Both are no-ops in a kernel launched the ordinary way.
#ifdef __CUDACC__
__device__ __forceinline__ void chain_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void chain_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
#endif
template <typename... KArgs, typename... Args>
inline cudaError_t launch_maybe_chained(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                        bool chained, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = chained ? attr : nullptr;
  cfg.numAttrs = chained ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// The kernels of a training step that follow one another on a stream are launched as a chain too (each starts
// with chain_release(); chain_wait();, so only its placement on the SMs overlaps the predecessor's last
// blocks).  SZO_STEP_CHAIN=0: ordinary launches (A/B measurement).
inline bool step_chained() {
  static const bool v = [] {
    const char* e = getenv("SZO_STEP_CHAIN");
    return !(e != nullptr && e[0] == '0');
  }();
  return v;
}

// Launch counter used by the model to report how many kernels one step enqueued.
extern thread_local int64_t g_launch_count;
inline void count_launch(int n = 1) { g_launch_count += n; }

// Scale of a sparse axpy pass: a host value, or -(float)(lr * (f+ - f-) / (2 eps)) formed on
// the device from the two losses (when f_plus != nullptr).
struct ScaleArg {
  float scale;
  float lr, eps;
  const double* f_plus;
  const double* f_minus;
};
// z_out != nullptr: also keep z_j in z_out[j]
szo_status launch_sparse_axpy(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                              int64_t idx_base, uint64_t seed, uint64_t step, ScaleArg sa,
                              cudaStream_t st, float* z_out = nullptr);
// The +eps, -2 eps, +eps passes of one (seed, step) in one launch, z kept in z_out: S_out takes the value the
// three passes leave (same roundings); S_plus / S_minus, where not NULL, the values after the first / second
szo_status launch_sparse_axpy_three(const float* S_in, float* S_out, const int64_t* idx, int64_t k, int64_t idx_base,
                                    uint64_t seed, uint64_t step, float eps, cudaStream_t st, float* z_out,
                                    float* S_plus, float* S_minus);
// S_out[j] = fma(scale, z[j], S_in[j]) with kept z
szo_status launch_sparse_axpy_kept(const float* S_in, float* S_out, const float* z, int64_t k, ScaleArg sa,
                                   cudaStream_t st);

// Causal attention for bf16 activations (attention.cu); q, k, v, o are [B*S, heads*hd] row-major.
szo_status launch_flash_attention_bf16(const void* q, const void* k, const void* v, void* o, int B, int S, int H,
                                       int Hkv, int hd, cudaStream_t st);

// The same for the paired form of a ZO step's two forwards: centre rows first, half-difference rows
// from row `row0` on in every buffer.
szo_status launch_flash_attention_pair_bf16(const void* q, const void* k, const void* v, void* o, int64_t row0, int B,
                                            int S, int H, int Hkv, int hd, cudaStream_t st);

}  // namespace szo
