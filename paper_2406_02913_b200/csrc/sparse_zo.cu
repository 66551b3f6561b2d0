// Sparse perturb / restore / update passes of the ZO step and the projected gradient.
//
// Definition 4 (sensitive sparse ZO-SGD) perturbs and updates only the k masked coordinates; the
// Section 3.4 decomposition makes them a contiguous fp32 vector S.  z is regenerated from a
// counter-based generator (Section 2.1 seed trick) keyed by (seed, step, global parameter index):
// Philox4x32-10 (Salmon et al., SC'11) followed by the Box-Muller cosine branch.
#include <type_traits>

#include "common.cuh"

namespace szo {

constexpr uint32_t kPhiloxM0 = 0xD2511F53u;
constexpr uint32_t kPhiloxM1 = 0xCD9E8D57u;
constexpr uint32_t kPhiloxW0 = 0x9E3779B9u;
constexpr uint32_t kPhiloxW1 = 0xBB67AE85u;

// The ten round keys (key + r * Weyl constant) are the same for every entry of a pass: the host
// computes them once and passes them by value, so that each round is two wide multiplies and two
// three-input XORs.
struct PhiloxKeys {
  uint32_t k0[10], k1[10];
};

// Ten Philox rounds; only output words 0 and 1 are consumed by the Gaussian draw.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              const PhiloxKeys& K, uint32_t& r0, uint32_t& r1) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const unsigned long long p0 = static_cast<unsigned long long>(kPhiloxM0) * c0;   // (hi0, lo0)
    const unsigned long long p1 = static_cast<unsigned long long>(kPhiloxM1) * c2;   // (hi1, lo1)
    const uint32_t n0 = static_cast<uint32_t>(p1 >> 32) ^ c1 ^ K.k0[r];
    const uint32_t n2 = static_cast<uint32_t>(p0 >> 32) ^ c3 ^ K.k1[r];
    c1 = static_cast<uint32_t>(p1);
    c3 = static_cast<uint32_t>(p0);
    c0 = n0;
    c2 = n2;
  }
  r0 = c0;
  r1 = c1;
}

// z = sqrt(-2 ln u1) cos(2 pi u2), u1 = ((r0 >> 8) + 1) 2^-24 in (0,1], u2 = (r1 >> 8) 2^-24 in [0,1).
// The pass is bound by instruction issue as much as by memory, so ln and cos are evaluated by short
// polynomials without the special-case handling of the library routines (u1 is a normal number in
// (0,1], the cosine argument is exactly reduced):
//   ln u1:  u1 = f 2^e with f in [sqrt(1/2), sqrt(2)), s = f - 1, ln(1+s) = s - s^2/2 + s^3 P(s)
//   cos(2 pi u2) = -cos(pi y), y = 2 u2 - 1; with a = |y| and b = min(a, 1 - a) in [0, 1/2]:
//                  cos(pi a) = +-cos(pi b) = +-C(b^2)
// P (degree 7) and C (degree 6) are least-squares fits on Chebyshev nodes; tests/test_gauss_polynomials.py
// reads the coefficients below, refits them and checks |z - z_fp64| <= 5e-7 max(1,|z|) for this arithmetic.
__device__ __forceinline__ float gaussian_from_words(uint32_t r0, uint32_t r1) {
  const float u1 = static_cast<float>((r0 >> 8) + 1u) * 5.9604644775390625e-8f;
  const int bits = __float_as_int(u1);
  const int e = (bits - 0x3F3504F3) >> 23;
  const float s = __int_as_float(bits - (e << 23)) - 1.0f;
  float p = -8.102270427e-02f;
  p = fmaf(p, s, 1.271267889e-01f);
  p = fmaf(p, s, -1.297214522e-01f);
  p = fmaf(p, s, 1.420211430e-01f);
  p = fmaf(p, s, -1.664225085e-01f);
  p = fmaf(p, s, 2.000147135e-01f);
  p = fmaf(p, s, -2.500029652e-01f);
  p = fmaf(p, s, 3.333332856e-01f);
  const float s2 = s * s;
  const float lg = fmaf(s2 * s, p, fmaf(-0.5f, s2, s));
  const float L = fmaf(static_cast<float>(e), 0.6931471805599453f, lg);
  float rad;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rad) : "f"(-2.0f * L));

  const float x = static_cast<float>(r1 >> 8) * 1.1920928955078125e-7f;   // 2 u2 in [0, 2), exact
  const float a = fabsf(x - 1.0f);
  const float b = fminf(a, 1.0f - a);
  const float t = b * b;
  float c = 1.840005517e-03f;
  c = fmaf(c, t, -2.577632849e-02f);
  c = fmaf(c, t, 2.353254400e-01f);
  c = fmaf(c, t, -1.335262316e+00f);
  c = fmaf(c, t, 4.058712108e+00f);
  c = fmaf(c, t, -4.934802200e+00f);
  c = fmaf(c, t, 1.0f);
  return (a > 0.5f) ? rad * c : -(rad * c);
}

__device__ __forceinline__ float z_of(uint64_t gidx, uint32_t step_lo, uint32_t step_hi, const PhiloxKeys& K) {
  uint32_t r0, r1;
  philox4x32_10(static_cast<uint32_t>(gidx), static_cast<uint32_t>(gidx >> 32), step_lo, step_hi, K, r0, r1);
  return gaussian_from_words(r0, r1);
}

__device__ __forceinline__ float resolve_scale(const ScaleArg& a) {
  if (a.f_plus == nullptr) return a.scale;
  const double g = (*a.f_plus - *a.f_minus) / (2.0 * static_cast<double>(a.eps));
  return -static_cast<float>(static_cast<double>(a.lr) * g);
}

// Eight entries per thread and iteration (four 16-byte index loads, two 16-byte value loads and
// stores): eight independent Philox / Box-Muller chains in flight hide the latency of the serial
// ten-round chain.  The next iteration's loads are issued before the current values are computed.
constexpr int kAxpyPer = 8;

// kKeepZ: also store z_j to z_out[j], for the later passes of the same (seed, step).
// kThree: the +eps, -2 eps, +eps passes of the seed trick in one (scale = eps): with sp = fma(eps, z, S),
// sm = fma(-2 eps, z, sp), s0 = fma(eps, z, sm) (the roundings of the three separate passes), S_out = s0
// and, where given, S_plus = sp and S_minus = sm.  The pass is bound by drawing z, so the two extra fused
// multiply-adds and stores cost nothing measurable.
template <bool kKeepZ, bool kThree>
__global__ void __launch_bounds__(256)
sparse_axpy_kernel(const float* S_in, float* S_out,      // may alias (in-place passes): no __restrict__
                   const int64_t* __restrict__ idx, int64_t k, int64_t idx_base, const PhiloxKeys K,
                   uint32_t step_lo, uint32_t step_hi, ScaleArg sa, float* __restrict__ z_out,
                   float* __restrict__ S_plus, float* __restrict__ S_minus) {
  const float scale = resolve_scale(sa);
  auto apply = [&](float z, float s, float& sp, float& sm) -> float {
    if constexpr (kThree) {
      sp = fmaf(scale, z, s);
      sm = fmaf(-2.0f * scale, z, sp);
      return fmaf(scale, z, sm);
    } else {
      sp = sm = 0.f;
      return fmaf(scale, z, s);
    }
  };
  const int64_t octs = k / kAxpyPer;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  for (int64_t p = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x; p < octs; p += stride) {
    longlong2 id[4];
    float4 s[2];
#pragma unroll
    for (int j = 0; j < 4; ++j) id[j] = reinterpret_cast<const longlong2*>(idx)[4 * p + j];
#pragma unroll
    for (int j = 0; j < 2; ++j) s[j] = reinterpret_cast<const float4*>(S_in)[2 * p + j];
    float z[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      z[2 * j] = z_of(static_cast<uint64_t>(idx_base + id[j].x), step_lo, step_hi, K);
      z[2 * j + 1] = z_of(static_cast<uint64_t>(idx_base + id[j].y), step_lo, step_hi, K);
    }
#pragma unroll
    for (int j = 0; j < 2; ++j) {
      float4 o, op, om;
      o.x = apply(z[4 * j], s[j].x, op.x, om.x);
      o.y = apply(z[4 * j + 1], s[j].y, op.y, om.y);
      o.z = apply(z[4 * j + 2], s[j].z, op.z, om.z);
      o.w = apply(z[4 * j + 3], s[j].w, op.w, om.w);
      reinterpret_cast<float4*>(S_out)[2 * p + j] = o;
      if constexpr (kThree) {
        if (S_plus != nullptr) reinterpret_cast<float4*>(S_plus)[2 * p + j] = op;
        if (S_minus != nullptr) reinterpret_cast<float4*>(S_minus)[2 * p + j] = om;
      }
      if constexpr (kKeepZ)
        reinterpret_cast<float4*>(z_out)[2 * p + j] = make_float4(z[4 * j], z[4 * j + 1], z[4 * j + 2], z[4 * j + 3]);
    }
  }
  // up to seven trailing entries
  const int64_t j = octs * kAxpyPer + threadIdx.x;
  if (blockIdx.x == 0 && threadIdx.x < kAxpyPer && j < k) {
    const float z = z_of(static_cast<uint64_t>(idx_base + idx[j]), step_lo, step_hi, K);
    float sp, sm;
    S_out[j] = apply(z, S_in[j], sp, sm);
    if constexpr (kThree) {
      if (S_plus != nullptr) S_plus[j] = sp;
      if (S_minus != nullptr) S_minus[j] = sm;
    }
    if constexpr (kKeepZ) z_out[j] = z;
  }
}

// The later passes of a step with z kept by the first one: S_out[j] = fma(scale, z[j], S_in[j]),
// 12 bytes per entry and one fma: a plain stream.  Sixteen entries per thread and iteration, all
// eight 16-byte loads issued before the first use (a pass over a few million entries lasts ~15 us:
// memory-level parallelism per thread is what fills the pipe that quickly).
constexpr int kKeptUnroll = 4;
__global__ void __launch_bounds__(256)
sparse_axpy_kept_kernel(const float* S_in, float* S_out /* may alias S_in */, const float* __restrict__ z,
                        int64_t k, ScaleArg sa) {
  const float scale = resolve_scale(sa);
  const int64_t quads = k / 4;
  const int64_t stride = static_cast<int64_t>(gridDim.x) * blockDim.x;
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  for (int64_t p0 = t; p0 < quads; p0 += stride * kKeptUnroll) {
    float4 s[kKeptUnroll], zz[kKeptUnroll];
#pragma unroll
    for (int u = 0; u < kKeptUnroll; ++u) {
      const int64_t p = p0 + u * stride;
      if (p < quads) {
        s[u] = reinterpret_cast<const float4*>(S_in)[p];
        zz[u] = reinterpret_cast<const float4*>(z)[p];
      }
    }
#pragma unroll
    for (int u = 0; u < kKeptUnroll; ++u) {
      const int64_t p = p0 + u * stride;
      if (p < quads) {
        float4 o;
        o.x = fmaf(scale, zz[u].x, s[u].x);
        o.y = fmaf(scale, zz[u].y, s[u].y);
        o.z = fmaf(scale, zz[u].z, s[u].z);
        o.w = fmaf(scale, zz[u].w, s[u].w);
        reinterpret_cast<float4*>(S_out)[p] = o;
      }
    }
  }
  const int64_t j = quads * 4 + threadIdx.x;
  if (blockIdx.x == 0 && threadIdx.x < 4 && j < k) S_out[j] = fmaf(scale, z[j], S_in[j]);
}

__global__ void projected_gradient_kernel(const double* f_plus, const double* f_minus, float eps,
                                          double* g) {
  *g = (*f_plus - *f_minus) / (2.0 * static_cast<double>(eps));
}

szo_status launch_sparse_axpy_kept(const float* S_in, float* S_out, const float* z, int64_t k, ScaleArg sa,
                                   cudaStream_t st) {
  if (k == 0) return SZO_OK;
  int64_t blocks = ceil_div(ceil_div(k, 4 * kKeptUnroll), 256);
  const int64_t wave = 148 * 8;
  if (blocks > wave) blocks = wave;
  sparse_axpy_kept_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(S_in, S_out, z, k, sa);
  count_launch();
  SZO_CHECK_LAUNCH("sparse_axpy_kept_kernel");
  return SZO_OK;
}

static szo_status launch_sparse_axpy_any(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                                         int64_t idx_base, uint64_t seed, uint64_t step, ScaleArg sa,
                                         cudaStream_t st, float* z_out, bool three, float* S_plus, float* S_minus) {
  if (k == 0) return SZO_OK;
  PhiloxKeys K;
  uint32_t k0 = static_cast<uint32_t>(seed), k1 = static_cast<uint32_t>(seed >> 32);
  for (int r = 0; r < 10; ++r) {
    K.k0[r] = k0;
    K.k1[r] = k1;
    k0 += kPhiloxW0;
    k1 += kPhiloxW1;
  }
  // grid: whole waves of 148 x 8 blocks when there is enough work, so that every SM gets the same share
  const int64_t quads = (k + kAxpyPer - 1) / kAxpyPer;     // work items (groups of kAxpyPer entries)
  int64_t blocks = ceil_div(quads, 256);
  const int64_t wave = 148 * 8;
  if (blocks > wave) {
    const int64_t sweeps = ceil_div(blocks, wave);          // iterations of the grid-stride loop
    blocks = ceil_div(ceil_div(quads, sweeps), 256);        // just enough threads for that many sweeps
    if (blocks > wave) blocks = wave;
  }
  const uint32_t lo = static_cast<uint32_t>(step), hi = static_cast<uint32_t>(step >> 32);
  const unsigned nb = static_cast<unsigned>(blocks);
  if (three)
    sparse_axpy_kernel<true, true><<<nb, 256, 0, st>>>(S_in, S_out, idx, k, idx_base, K, lo, hi, sa, z_out, S_plus, S_minus);
  else if (z_out != nullptr)
    sparse_axpy_kernel<true, false><<<nb, 256, 0, st>>>(S_in, S_out, idx, k, idx_base, K, lo, hi, sa, z_out, nullptr, nullptr);
  else
    sparse_axpy_kernel<false, false><<<nb, 256, 0, st>>>(S_in, S_out, idx, k, idx_base, K, lo, hi, sa, nullptr, nullptr, nullptr);
  count_launch();
  SZO_CHECK_LAUNCH("sparse_axpy_kernel");
  return SZO_OK;
}

szo_status launch_sparse_axpy(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                              int64_t idx_base, uint64_t seed, uint64_t step, ScaleArg sa,
                              cudaStream_t st, float* z_out) {
  return launch_sparse_axpy_any(S_in, S_out, idx, k, idx_base, seed, step, sa, st, z_out, false, nullptr, nullptr);
}

szo_status launch_sparse_axpy_three(const float* S_in, float* S_out, const int64_t* idx, int64_t k, int64_t idx_base,
                                    uint64_t seed, uint64_t step, float eps, cudaStream_t st, float* z_out,
                                    float* S_plus, float* S_minus) {
  if (z_out == nullptr) return fail(SZO_ERR_INVALID_ARG, "the three-pass form keeps z");
  ScaleArg sa{eps, 0.f, 0.f, nullptr, nullptr};
  return launch_sparse_axpy_any(S_in, S_out, idx, k, idx_base, seed, step, sa, st, z_out, true, S_plus, S_minus);
}

}  // namespace szo

namespace szo {
// Sparse values stored in 16 bits (Section 3.5): S[j] = widen(RN_T16(S[j])), optionally the stored form too
template <typename T16>
__global__ void round_sparse16_kernel(float* __restrict__ S, int64_t k, T16* __restrict__ out) {
  const int64_t j = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (j >= k) return;
  T16 h;
  if constexpr (sizeof(T16) == sizeof(__half) && !std::is_same<T16, __nv_bfloat16>::value) h = __float2half_rn(S[j]);
  else h = __float2bfloat16_rn(S[j]);
  if (out != nullptr) out[j] = h;
  if constexpr (std::is_same<T16, __nv_bfloat16>::value) S[j] = __bfloat162float(h);
  else S[j] = __half2float(h);
}
}  // namespace szo

extern "C" {

szo_status szo_perturb(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                       int64_t idx_base, uint64_t seed, uint64_t step, float scale, void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S_in && S_out && idx, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(idx_base >= 0, SZO_ERR_INVALID_ARG, "idx_base < 0");
  SZO_REQUIRE(szo::aligned16(S_in) && szo::aligned16(S_out) && szo::aligned16(idx), SZO_ERR_ALIGNMENT,
              "S_in, S_out and idx must be 16-byte aligned");
  szo::ScaleArg sa{scale, 0.f, 0.f, nullptr, nullptr};
  return szo::launch_sparse_axpy(S_in, S_out, idx, k, idx_base, seed, step, sa,
                                 static_cast<cudaStream_t>(stream));
}

szo_status szo_perturb_keep_z(const float* S_in, float* S_out, const int64_t* idx, int64_t k, int64_t idx_base,
                              uint64_t seed, uint64_t step, float scale, float* z_out, void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S_in && S_out && idx && z_out, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(idx_base >= 0, SZO_ERR_INVALID_ARG, "idx_base < 0");
  SZO_REQUIRE(szo::aligned16(S_in) && szo::aligned16(S_out) && szo::aligned16(idx) && szo::aligned16(z_out),
              SZO_ERR_ALIGNMENT, "S_in, S_out, idx and z_out must be 16-byte aligned");
  szo::ScaleArg sa{scale, 0.f, 0.f, nullptr, nullptr};
  return szo::launch_sparse_axpy(S_in, S_out, idx, k, idx_base, seed, step, sa, static_cast<cudaStream_t>(stream),
                                 z_out);
}

szo_status szo_perturb3_keep_z(const float* S_in, float* S_out, const int64_t* idx, int64_t k, int64_t idx_base,
                               uint64_t seed, uint64_t step, float eps, float* z_out, float* S_plus, float* S_minus,
                               void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S_in && S_out && idx && z_out, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(idx_base >= 0, SZO_ERR_INVALID_ARG, "idx_base < 0");
  SZO_REQUIRE(szo::aligned16(S_in) && szo::aligned16(S_out) && szo::aligned16(idx) && szo::aligned16(z_out) &&
                  szo::aligned16(S_plus) && szo::aligned16(S_minus),
              SZO_ERR_ALIGNMENT, "S_in, S_out, idx, z_out, S_plus and S_minus must be 16-byte aligned");
  return szo::launch_sparse_axpy_three(S_in, S_out, idx, k, idx_base, seed, step, eps, static_cast<cudaStream_t>(stream),
                                       z_out, S_plus, S_minus);
}

szo_status szo_perturb_kept_z(const float* S_in, float* S_out, const float* z, int64_t k, float scale, void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S_in && S_out && z, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(szo::aligned16(S_in) && szo::aligned16(S_out) && szo::aligned16(z), SZO_ERR_ALIGNMENT,
              "S_in, S_out and z must be 16-byte aligned");
  szo::ScaleArg sa{scale, 0.f, 0.f, nullptr, nullptr};
  return szo::launch_sparse_axpy_kept(S_in, S_out, z, k, sa, static_cast<cudaStream_t>(stream));
}

szo_status szo_update_kept_z(float* S, const float* z, int64_t k, float lr, const double* f_plus_dev,
                             const double* f_minus_dev, float eps, void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  SZO_REQUIRE(f_plus_dev && f_minus_dev, SZO_ERR_INVALID_ARG, "NULL loss pointer");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S && z, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(szo::aligned16(S) && szo::aligned16(z), SZO_ERR_ALIGNMENT, "S and z must be 16-byte aligned");
  szo::ScaleArg sa{0.f, lr, eps, f_plus_dev, f_minus_dev};
  return szo::launch_sparse_axpy_kept(S, S, z, k, sa, static_cast<cudaStream_t>(stream));
}

szo_status szo_update(float* S, const int64_t* idx, int64_t k, int64_t idx_base, uint64_t seed,
                      uint64_t step, float lr, const double* f_plus_dev, const double* f_minus_dev,
                      float eps, void* stream) {
  SZO_REQUIRE(k >= 0, SZO_ERR_INVALID_ARG, "k < 0");
  SZO_REQUIRE(f_plus_dev && f_minus_dev, SZO_ERR_INVALID_ARG, "NULL loss pointer");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  if (k == 0) return SZO_OK;
  SZO_REQUIRE(S && idx, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(idx_base >= 0, SZO_ERR_INVALID_ARG, "idx_base < 0");
  SZO_REQUIRE(szo::aligned16(S) && szo::aligned16(idx), SZO_ERR_ALIGNMENT,
              "S and idx must be 16-byte aligned");
  szo::ScaleArg sa{0.f, lr, eps, f_plus_dev, f_minus_dev};
  return szo::launch_sparse_axpy(S, S, idx, k, idx_base, seed, step, sa,
                                 static_cast<cudaStream_t>(stream));
}

szo_status szo_replay(float* S, const int64_t* idx, int64_t k, int64_t idx_base, uint64_t seed,
                      const uint64_t* steps_host, const double* g_host, int64_t n, float eps, float lr, void* stream) {
  SZO_REQUIRE(k >= 0 && n >= 0, SZO_ERR_INVALID_ARG, "k < 0 or n < 0");
  if (k == 0 || n == 0) return SZO_OK;
  SZO_REQUIRE(S && idx && steps_host && g_host, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(idx_base >= 0, SZO_ERR_INVALID_ARG, "idx_base < 0");
  SZO_REQUIRE(szo::aligned16(S) && szo::aligned16(idx), SZO_ERR_ALIGNMENT, "S and idx must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  for (int64_t t = 0; t < n; ++t) {
    if (eps != 0.f) {     // the roundings of the original step's +eps, -2 eps, +eps passes
      const float sc[3] = {eps, -2.0f * eps, eps};
      for (int i = 0; i < 3; ++i) {
        szo::ScaleArg sa{sc[i], 0.f, 0.f, nullptr, nullptr};
        SZO_TRY(szo::launch_sparse_axpy(S, S, idx, k, idx_base, seed, steps_host[t], sa, st));
      }
    }
    szo::ScaleArg su{-static_cast<float>(static_cast<double>(lr) * g_host[t]), 0.f, 0.f, nullptr, nullptr};
    SZO_TRY(szo::launch_sparse_axpy(S, S, idx, k, idx_base, seed, steps_host[t], su, st));
  }
  return SZO_OK;
}

szo_status szo_round_sparse16(float* S, int64_t k, szo_dtype dt, void* S16_out, void* stream) {
  SZO_REQUIRE(k >= 0 && (k == 0 || S != nullptr), SZO_ERR_INVALID_ARG, "NULL S or k < 0");
  SZO_REQUIRE(dt == SZO_BF16 || dt == SZO_F16, SZO_ERR_INVALID_ARG, "the storage format must be SZO_BF16 or SZO_F16");
  if (k == 0) return SZO_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const unsigned blocks = static_cast<unsigned>(szo::ceil_div(k, 256));
  if (dt == SZO_BF16) szo::round_sparse16_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(S, k, static_cast<__nv_bfloat16*>(S16_out));
  else szo::round_sparse16_kernel<__half><<<blocks, 256, 0, st>>>(S, k, static_cast<__half*>(S16_out));
  szo::count_launch();
  SZO_CHECK_LAUNCH("round_sparse16_kernel");
  return SZO_OK;
}

szo_status szo_projected_gradient(const double* f_plus_dev, const double* f_minus_dev, float eps,
                                  double* g_dev, void* stream) {
  SZO_REQUIRE(f_plus_dev && f_minus_dev && g_dev, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  szo::projected_gradient_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(f_plus_dev, f_minus_dev,
                                                                              eps, g_dev);
  szo::count_launch();
  SZO_CHECK_LAUNCH("projected_gradient_kernel");
  return SZO_OK;
}

}  // extern "C"
