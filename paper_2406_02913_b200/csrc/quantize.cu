// Group-wise asymmetric int4 quantizer for the frozen dense part w_dense (Section 3.5,
// "Integration with quantization").  One warp per (row, group): min/max by shuffles, then
// scale = round16((max-min)/15), zero = round16(min), code = clamp(rint((w-zero)/scale), 0, 15),
// in IEEE fp32 with explicit round-to-nearest intrinsics so that no contraction changes a bit.
#include "common.cuh"

namespace szo {

template <typename T> __device__ __forceinline__ float load_f32(const T* p, int64_t i);
template <> __device__ __forceinline__ float load_f32<float>(const float* p, int64_t i) { return p[i]; }
template <> __device__ __forceinline__ float load_f32<__nv_bfloat16>(const __nv_bfloat16* p, int64_t i) {
  return __bfloat162float(p[i]);
}

template <typename SZ> __device__ __forceinline__ SZ round16(float v);
template <> __device__ __forceinline__ __nv_bfloat16 round16<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }
template <> __device__ __forceinline__ __half round16<__half>(float v) { return __float2half_rn(v); }
__device__ __forceinline__ float widen(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ float widen(__half v) { return __half2float(v); }

template <typename WT, typename SZ>
__global__ void __launch_bounds__(256)
quantize_kernel(const WT* __restrict__ W, int64_t N, int64_t K, int G, uint8_t* __restrict__ codes,
                SZ* __restrict__ scales, SZ* __restrict__ zeros) {
  const int lane = threadIdx.x & 31;
  const int64_t groups_per_row = K / G;
  const int64_t total = N * groups_per_row;
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  for (int64_t g = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; g < total; g += warps) {
    const int64_t row = g / groups_per_row, grp = g % groups_per_row;
    const int64_t base = row * K + grp * G;
    float mn = INFINITY, mx = -INFINITY;
    for (int c = lane; c < G; c += 32) {
      const float w = load_f32(W, base + c);
      mn = fminf(mn, w);
      mx = fmaxf(mx, w);
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const SZ s16 = round16<SZ>(__fdiv_rn(__fsub_rn(mx, mn), 15.0f));
    const SZ z16 = round16<SZ>(mn);
    const float s = widen(s16), z0 = widen(z16);
    if (lane == 0) {
      scales[g] = s16;
      zeros[g] = z16;
    }
    for (int c = lane * 2; c < G; c += 64) {
      int q[2];
#pragma unroll
      for (int t = 0; t < 2; ++t) {
        const float w = load_f32(W, base + c + t);
        float r = (s == 0.0f) ? 0.0f : rintf(__fdiv_rn(__fsub_rn(w, z0), s));
        r = fminf(fmaxf(r, 0.0f), 15.0f);
        q[t] = static_cast<int>(r);
      }
      codes[(base + c) >> 1] = static_cast<uint8_t>(q[0] | (q[1] << 4));
    }
  }
}

// G in {32, 64, 128} with fp32 weights: a warp takes 128 consecutive elements of a row (one 16-byte
// load per lane, kept in registers for the second step), i.e. 128 / G groups of G / 4 lanes each; the
// min/max shuffles stay inside a group's lanes, a lane writes its four codes as one 16-bit store.
// Same arithmetic, instruction by instruction, as the general kernel: the same bits.
template <typename SZ>
__global__ void __launch_bounds__(256)
quantize_f32_vec_kernel(const float* __restrict__ W, int64_t N, int64_t K, int G, uint8_t* __restrict__ codes,
                        SZ* __restrict__ scales, SZ* __restrict__ zeros) {
  const int lane = threadIdx.x & 31;
  const int lanes_per_group = G >> 2;
  const int64_t chunks = N * K / 128;          // K % G == 0 and G | 128, K % 128 == 0 (checked by the caller)
  const int64_t warps = (static_cast<int64_t>(gridDim.x) * blockDim.x) >> 5;
  for (int64_t ch = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) >> 5; ch < chunks; ch += warps) {
    const int64_t e0 = ch * 128 + lane * 4;    // flat element index of this lane's first weight
    const float4 w4 = *reinterpret_cast<const float4*>(W + e0);
    const float w[4] = {w4.x, w4.y, w4.z, w4.w};
    float mn = fminf(fminf(w[0], w[1]), fminf(w[2], w[3]));
    float mx = fmaxf(fmaxf(w[0], w[1]), fmaxf(w[2], w[3]));
    for (int o = lanes_per_group >> 1; o; o >>= 1) {
      mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    }
    const SZ s16 = round16<SZ>(__fdiv_rn(__fsub_rn(mx, mn), 15.0f));
    const SZ z16 = round16<SZ>(mn);
    const float s = widen(s16), z0 = widen(z16);
    if ((lane & (lanes_per_group - 1)) == 0) {
      const int64_t g = e0 / G;                // groups are numbered row-major, like the elements
      scales[g] = s16;
      zeros[g] = z16;
    }
    uint32_t packed = 0;
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      float r = (s == 0.0f) ? 0.0f : rintf(__fdiv_rn(__fsub_rn(w[t], z0), s));
      r = fminf(fmaxf(r, 0.0f), 15.0f);
      packed |= static_cast<uint32_t>(static_cast<int>(r)) << (4 * t);
    }
    *reinterpret_cast<uint16_t*>(codes + (e0 >> 1)) = static_cast<uint16_t>(packed);
  }
}

template <typename WT, typename SZ>
szo_status launch_quantize(const void* W, int64_t N, int64_t K, int G, uint8_t* codes, void* scales,
                           void* zeros, cudaStream_t st) {
  if constexpr (sizeof(WT) == 4) {
    if ((G == 32 || G == 64 || G == 128) && K % 128 == 0) {
      int64_t blocks = ceil_div(N * K / 128, 8);
      if (blocks > 148 * 32) blocks = 148 * 32;
      quantize_f32_vec_kernel<SZ><<<static_cast<unsigned>(blocks), 256, 0, st>>>(
          static_cast<const float*>(W), N, K, G, codes, static_cast<SZ*>(scales), static_cast<SZ*>(zeros));
      count_launch();
      SZO_CHECK_LAUNCH("quantize_f32_vec_kernel");
      return SZO_OK;
    }
  }
  const int64_t total_warps = N * (K / G);
  int64_t blocks = ceil_div(total_warps, 8);
  if (blocks > 148 * 16) blocks = 148 * 16;
  quantize_kernel<WT, SZ><<<static_cast<unsigned>(blocks), 256, 0, st>>>(
      static_cast<const WT*>(W), N, K, G, codes, static_cast<SZ*>(scales), static_cast<SZ*>(zeros));
  count_launch();
  SZO_CHECK_LAUNCH("quantize_kernel");
  return SZO_OK;
}

}  // namespace szo

extern "C" szo_status szo_quantize(const void* W, szo_dtype w_dtype, int64_t N, int64_t K, int32_t G,
                                   szo_dtype sz_dtype, uint8_t* codes, void* scales, void* zeros,
                                   void* stream) {
  using namespace szo;
  SZO_REQUIRE(N >= 0 && K >= 0, SZO_ERR_SHAPE, "negative shape");
  SZO_REQUIRE(G > 0 && G % 2 == 0, SZO_ERR_SHAPE, "G must be positive and even (got %d)", G);
  SZO_REQUIRE(K % G == 0, SZO_ERR_SHAPE, "K (%lld) must be a multiple of G (%d)", (long long)K, G);
  SZO_REQUIRE(w_dtype == SZO_F32 || w_dtype == SZO_BF16, SZO_ERR_UNSUPPORTED, "w_dtype must be f32 or bf16");
  SZO_REQUIRE(sz_dtype == SZO_BF16 || sz_dtype == SZO_F16, SZO_ERR_UNSUPPORTED, "sz_dtype must be bf16 or f16");
  if (N == 0 || K == 0) return SZO_OK;
  SZO_REQUIRE(W && codes && scales && zeros, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(aligned16(W) && aligned16(codes) && aligned16(scales) && aligned16(zeros), SZO_ERR_ALIGNMENT,
              "buffers must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (w_dtype == SZO_F32) {
    return sz_dtype == SZO_BF16 ? launch_quantize<float, __nv_bfloat16>(W, N, K, G, codes, scales, zeros, st)
                                : launch_quantize<float, __half>(W, N, K, G, codes, scales, zeros, st);
  }
  return sz_dtype == SZO_BF16
             ? launch_quantize<__nv_bfloat16, __nv_bfloat16>(W, N, K, G, codes, scales, zeros, st)
             : launch_quantize<__nv_bfloat16, __half>(W, N, K, G, codes, scales, zeros, st);
}
