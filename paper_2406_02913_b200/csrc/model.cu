// Loss path of a decoder-only language model and the whole ZO-SGD step on one GPU.
//
// Definition 1 (SPSA) evaluates the loss at w + eps z and w - eps z; Definitions 2 and 4 update the
// k sensitive values.  Everything between the linear layers (embedding, RMSNorm/LayerNorm, rotary
// positions, causal attention, SiLU-gated or ReLU MLP, residuals, cross-entropy) is plain CUDA
// here.  The residual stream is fp32; activations fed to the linears are T = bf16 (tensor-core
// path) or fp32 (validation path); per-token losses are summed in fp64 in a fixed order so that
// f+ and f- are produced by the identical, deterministic kernel sequence.
#include <vector>

#include "linear.cuh"

namespace szo {

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// Block-wide sum with a fixed reduction tree (blockDim.x a multiple of 32, <= 1024).
__device__ __forceinline__ float block_sum(float v, float* scratch) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[w] = v;
  __syncthreads();
  float t = 0.f;
  for (int i = 0; i < nw; ++i) t += scratch[i];
  return t;
}

// h[m, :] = embed[tok[m], :] (+ pos[pos0 + m % S, :]); pos0 > 0 when the rows continue a cached prefix
__global__ void embed_kernel(const int32_t* __restrict__ tok, const __nv_bfloat16* __restrict__ embed,
                             const __nv_bfloat16* __restrict__ pos, int S, int d, int vocab,
                             float* __restrict__ h, int pos0 = 0, const int32_t* __restrict__ pos_dev = nullptr) {
  if (pos_dev != nullptr) pos0 = *pos_dev;
  const int64_t m = blockIdx.x;
  int32_t t = tok[m];
  t = t < 0 ? 0 : (t >= vocab ? vocab - 1 : t);
  const __nv_bfloat16* e = embed + static_cast<int64_t>(t) * d;
  const __nv_bfloat16* p = pos ? pos + static_cast<int64_t>(pos0 + m % S) * d : nullptr;
  for (int c = threadIdx.x; c < d; c += blockDim.x)
    h[m * d + c] = __bfloat162float(e[c]) + (p ? __bfloat162float(p[c]) : 0.f);
}

// Residual add fused with the norm that follows it: h[m] += y[m] (when y != nullptr; written back
// unless the rows are a strided selection), then RMSNorm (x / sqrt(mean x^2 + eps) * gamma) or
// LayerNorm of the row.  One block per row; the row (d <= 8192 floats) lives in registers, so global
// memory is read once.  row_stride/row_offset select which rows are normalised (all rows, or the
// last token of each sequence when only that one feeds the loss).
// kMaxV: float4 per thread a row may need (d <= 1024 kMaxV); with 4 the kernel keeps half the registers and twice
// the blocks per SM (their load and reduction phases overlap: 86 -> 63 us per call at 8192 rows of 4096).
template <typename T, typename TO = T, int kMaxV = 8>
__global__ void __launch_bounds__(256)
add_norm_kernel(float* __restrict__ h, const T* __restrict__ y, const float* __restrict__ gamma,
                const float* __restrict__ beta, int d, float eps, bool layer_norm, int64_t row_stride,
                int64_t row_offset, TO* __restrict__ out) {
  __shared__ float scratch[32];
  chain_release();
  chain_wait();
  const int64_t m = static_cast<int64_t>(blockIdx.x) * row_stride + row_offset;
  float* x = h + m * d;
  TO* o = out + static_cast<int64_t>(blockIdx.x) * d;
  const int nv = d >> 2;                         // float4 units in a row
  float4 v[kMaxV];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    const int c = threadIdx.x + i * 256;
    v[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < nv) {
      v[i] = reinterpret_cast<const float4*>(x)[c];
      if (y != nullptr) {
        const T* yp = y + m * d + c * 4;
        if constexpr (sizeof(T) == 2) {              // four bf16 in one 8-byte load (rows are 8-byte aligned: d % 4 == 0)
          const uint2 raw = *reinterpret_cast<const uint2*>(yp);
          v[i].x += __uint_as_float(raw.x << 16);
          v[i].y += __uint_as_float(raw.x & 0xFFFF0000u);
          v[i].z += __uint_as_float(raw.y << 16);
          v[i].w += __uint_as_float(raw.y & 0xFFFF0000u);
        } else {
          v[i].x += to_f32<T>(yp[0]);
          v[i].y += to_f32<T>(yp[1]);
          v[i].z += to_f32<T>(yp[2]);
          v[i].w += to_f32<T>(yp[3]);
        }
        if (row_stride == 1) reinterpret_cast<float4*>(x)[c] = v[i];
      }
      s += (v[i].x + v[i].y) + (v[i].z + v[i].w);
    }
  }
  const float mu = layer_norm ? block_sum(s, scratch) / d : 0.f;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    if (threadIdx.x + i * 256 < nv) {
      const float a0 = v[i].x - mu, a1 = v[i].y - mu, a2 = v[i].z - mu, a3 = v[i].w - mu;
      q += (a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3);
    }
  }
  const float var = block_sum(q, scratch) / d;
  const float r = 1.0f / sqrtf(var + eps);
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    const int c = threadIdx.x + i * 256;
    if (c < nv) {
      const float4 g = reinterpret_cast<const float4*>(gamma)[c];
      float4 bt = make_float4(0.f, 0.f, 0.f, 0.f);
      if (beta) bt = reinterpret_cast<const float4*>(beta)[c];
      TO* op = o + c * 4;
      const float o0 = (v[i].x - mu) * r * g.x + bt.x, o1 = (v[i].y - mu) * r * g.y + bt.y;
      const float o2 = (v[i].z - mu) * r * g.z + bt.z, o3 = (v[i].w - mu) * r * g.w + bt.w;
      if constexpr (sizeof(TO) == 2) {
        const __nv_bfloat162 lo = __floats2bfloat162_rn(o0, o1), hi = __floats2bfloat162_rn(o2, o3);
        uint2 pk;
        pk.x = *reinterpret_cast<const uint32_t*>(&lo);
        pk.y = *reinterpret_cast<const uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(op) = pk;
      } else {
        *reinterpret_cast<float4*>(op) = make_float4(o0, o1, o2, o3);
      }
    }
  }
}

// cos/sin table [max_seq, hd/2] from fp64 math: angle = p * base^(-2i/hd).
__global__ void rope_table_kernel(int max_seq, int half, double base, float2* __restrict__ tab) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= max_seq * half) return;
  const int p = i / half, j = i % half;
  const double ang = static_cast<double>(p) * pow(base, -2.0 * j / (2.0 * half));
  tab[i] = make_float2(static_cast<float>(cos(ang)), static_cast<float>(sin(ang)));
}

// In-place rotation of the pairs (i, i + hd/2) of every head of q [M, H*hd] and k [M, Hkv*hd] in one
// launch.  A thread rotates kN consecutive pairs (one 16-byte vector from each half of a head).
template <typename T>
__global__ void rope_kernel(T* __restrict__ q, T* __restrict__ k, const float2* __restrict__ tab, int64_t M, int S,
                            int H, int Hkv, int hd, int pos0 = 0, const int32_t* __restrict__ pos_dev = nullptr) {
  chain_release();
  chain_wait();
  if (pos_dev != nullptr) pos0 = *pos_dev;
  constexpr int kN = 16 / sizeof(T);
  const int half = hd >> 1, vec_per_head = half / kN;
  const int64_t per_token = static_cast<int64_t>(H + Hkv) * vec_per_head;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= M * per_token) return;
  const int64_t m = i / per_token;
  int r = static_cast<int>(i % per_token);
  const int head = r / vec_per_head, j0 = (r % vec_per_head) * kN;
  T* p = (head < H) ? q + (m * H + head) * hd : k + (m * Hkv + (head - H)) * hd;
  const float2* cs = tab + static_cast<int64_t>(pos0 + m % S) * half + j0;
  T lo[kN], hi[kN];
  *reinterpret_cast<uint4*>(lo) = *reinterpret_cast<const uint4*>(p + j0);
  *reinterpret_cast<uint4*>(hi) = *reinterpret_cast<const uint4*>(p + half + j0);
#pragma unroll
  for (int j = 0; j < kN; ++j) {
    const float a = to_f32<T>(lo[j]), b = to_f32<T>(hi[j]);
    const float2 t = cs[j];
    lo[j] = from_f32<T>(a * t.x - b * t.y);
    hi[j] = from_f32<T>(b * t.x + a * t.y);
  }
  *reinterpret_cast<uint4*>(p + j0) = *reinterpret_cast<const uint4*>(lo);
  *reinterpret_cast<uint4*>(p + half + j0) = *reinterpret_cast<const uint4*>(hi);
}

// Causal softmax attention, one warp per query; lanes split the head dimension.
template <typename T, int HD>
__global__ void __launch_bounds__(128)
attn_warp_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v, T* __restrict__ o,
                 int S, int H, int Hkv, float scale) {
  constexpr int E = HD / 32;
  const int lane = threadIdx.x & 31;
  const int s = blockIdx.x * 4 + (threadIdx.x >> 5);
  const int hq = blockIdx.y, b = blockIdx.z;
  if (s >= S) return;
  const int hk = hq / (H / Hkv);
  const int64_t dq = static_cast<int64_t>(H) * HD, dk = static_cast<int64_t>(Hkv) * HD;
  const T* qp = q + (static_cast<int64_t>(b) * S + s) * dq + hq * HD;
  float qr[E], acc[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    qr[j] = to_f32<T>(qp[lane + 32 * j]) * scale;
    acc[j] = 0.f;
  }
  float mx = -INFINITY, l = 0.f;
  for (int t = 0; t <= s; ++t) {
    const T* kp = k + (static_cast<int64_t>(b) * S + t) * dk + hk * HD;
    const T* vp = v + (static_cast<int64_t>(b) * S + t) * dk + hk * HD;
    float dot = 0.f;
#pragma unroll
    for (int j = 0; j < E; ++j) dot = fmaf(qr[j], to_f32<T>(kp[lane + 32 * j]), dot);
#pragma unroll
    for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    const float mn = fmaxf(mx, dot);
    const float corr = expf(mx - mn), p = expf(dot - mn);
    l = l * corr + p;
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = fmaf(p, to_f32<T>(vp[lane + 32 * j]), acc[j] * corr);
    mx = mn;
  }
  T* op = o + (static_cast<int64_t>(b) * S + s) * dq + hq * HD;
  const float inv = 1.0f / l;
#pragma unroll
  for (int j = 0; j < E; ++j) op[lane + 32 * j] = from_f32<T>(acc[j] * inv);
}

// Elementwise kernels work on 16-byte vectors (8 bf16 or 4 fp32 per thread); every tensor they
// touch has a multiple of 8 elements per row and 16-byte aligned rows.
template <typename T> struct Vec16 {
  static constexpr int kN = 16 / sizeof(T);
  T v[16 / sizeof(T)];
};
template <typename T> __device__ __forceinline__ Vec16<T> load16(const T* p) {
  Vec16<T> r;
  *reinterpret_cast<uint4*>(r.v) = *reinterpret_cast<const uint4*>(p);
  return r;
}
template <typename T> __device__ __forceinline__ void store16(T* p, const Vec16<T>& r) {
  *reinterpret_cast<uint4*>(p) = *reinterpret_cast<const uint4*>(r.v);
}

template <typename T>
__global__ void silu_mul_kernel(const T* __restrict__ gate, const T* __restrict__ up, int64_t n, T* __restrict__ out) {
  constexpr int kN = Vec16<T>::kN;
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * kN;
  if (i >= n) return;
  const Vec16<T> g = load16(gate + i), u = load16(up + i);
  Vec16<T> r;
#pragma unroll
  for (int j = 0; j < kN; ++j) {
    const float x = to_f32<T>(g.v[j]);
    r.v[j] = from_f32<T>(x / (1.0f + expf(-x)) * to_f32<T>(u.v[j]));
  }
  store16(out + i, r);
}

template <typename T>
__global__ void relu_kernel(T* __restrict__ x, int64_t n) {
  constexpr int kN = Vec16<T>::kN;
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * kN;
  if (i >= n) return;
  Vec16<T> r = load16(x + i);
#pragma unroll
  for (int j = 0; j < kN; ++j) r.v[j] = from_f32<T>(fmaxf(to_f32<T>(r.v[j]), 0.f));
  store16(x + i, r);
}

template <typename T>
__global__ void residual_add_kernel(float* __restrict__ h, const T* __restrict__ y, int64_t n) {
  constexpr int kN = Vec16<T>::kN;
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * kN;
  if (i >= n) return;
  const Vec16<T> r = load16(y + i);
#pragma unroll
  for (int j = 0; j < kN; j += 4) {
    float4 a = *reinterpret_cast<float4*>(h + i + j);
    a.x += to_f32<T>(r.v[j]);
    a.y += to_f32<T>(r.v[j + 1]);
    a.z += to_f32<T>(r.v[j + 2]);
    a.w += to_f32<T>(r.v[j + 3]);
    *reinterpret_cast<float4*>(h + i + j) = a;
  }
}

// Next-token cross-entropy of row m (position s < S-1 predicts tok[m+1]); 0 for the last position.
// One pass over the row: every thread keeps a running maximum and the sum of exp(x - maximum) of its
// elements (16-byte loads when the row allows it), the block then brings the partial sums to the
// common maximum.
__global__ void __launch_bounds__(256)
ce_rows_kernel(const float* __restrict__ logits, const int32_t* __restrict__ tok, int S, int V,
               double* __restrict__ tok_loss) {
  __shared__ float scratch[32];
  const int64_t m = blockIdx.x;
  if ((m % S) == S - 1) {
    if (threadIdx.x == 0) tok_loss[m] = 0.0;
    return;
  }
  const float* row = logits + m * V;
  float mx = -INFINITY, s = 0.f;
  auto fold = [&](float cmax, float csum_at_cmax) {      // merge a chunk given at its own maximum
    if (cmax > mx) {
      s = s * __expf(mx - cmax) + csum_at_cmax;
      mx = cmax;
    } else {
      s += csum_at_cmax * __expf(cmax - mx);
    }
  };
  if ((V & 3) == 0) {
    const float4* row4 = reinterpret_cast<const float4*>(row);
    for (int c = threadIdx.x; c < (V >> 2); c += blockDim.x) {
      const float4 x = row4[c];
      const float cm = fmaxf(fmaxf(x.x, x.y), fmaxf(x.z, x.w));
      fold(cm, __expf(x.x - cm) + __expf(x.y - cm) + __expf(x.z - cm) + __expf(x.w - cm));
    }
  } else {
    for (int c = threadIdx.x; c < V; c += blockDim.x) fold(row[c], 1.f);
  }
  // block maximum, then every partial sum rescaled to it
  float bm = mx;
#pragma unroll
  for (int o = 16; o; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = bm;
  __syncthreads();
  for (int i = 0; i < (blockDim.x >> 5); ++i) bm = fmaxf(bm, scratch[i]);
  s = (mx == -INFINITY) ? 0.f : s * __expf(mx - bm);
  s = block_sum(s, scratch);
  if (threadIdx.x == 0) {
    int32_t t = tok[m + 1];
    t = t < 0 ? 0 : (t >= V ? V - 1 : t);
    tok_loss[m] = (static_cast<double>(bm) + log(static_cast<double>(s))) - static_cast<double>(row[t]);
  }
}

// 2-way cross-entropy over the logits of two candidate ids for the normalised last-token state.
template <typename T>
__global__ void __launch_bounds__(256)
cls2_kernel(const T* __restrict__ a_last, const __nv_bfloat16* __restrict__ lm_head, const int32_t* __restrict__ cand,
            const int32_t* __restrict__ labels, int d, int V, double* __restrict__ seq_loss) {
  __shared__ float scratch[32];
  const int b = blockIdx.x;
  const T* a = a_last + static_cast<int64_t>(b) * d;
  int32_t c0 = cand[0], c1 = cand[1];
  c0 = c0 < 0 ? 0 : (c0 >= V ? V - 1 : c0);
  c1 = c1 < 0 ? 0 : (c1 >= V ? V - 1 : c1);
  const __nv_bfloat16* e0 = lm_head + static_cast<int64_t>(c0) * d;
  const __nv_bfloat16* e1 = lm_head + static_cast<int64_t>(c1) * d;
  float s0 = 0.f, s1 = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float x = to_f32<T>(a[c]);
    s0 = fmaf(x, __bfloat162float(e0[c]), s0);
    s1 = fmaf(x, __bfloat162float(e1[c]), s1);
  }
  s0 = block_sum(s0, scratch);
  s1 = block_sum(s1, scratch);
  if (threadIdx.x == 0) {
    const double l0 = s0, l1 = s1, mx = l0 > l1 ? l0 : l1;
    const double lse = mx + log(exp(l0 - mx) + exp(l1 - mx));
    seq_loss[b] = lse - (labels[b] ? l1 : l0);
  }
}



// ------------------------------------------------------------------------------ token generation
// cache[b][pos0 + t][:] = new[b * T + t][:] for the keys AND the values of T new tokens per sequence
// (cache layout [B][Smax][width]); 16-byte vectors; the first n_vec threads copy keys, the others values.
template <typename T>
__global__ void kv_append_kernel(const T* __restrict__ k_new, const T* __restrict__ v_new, T* __restrict__ k_cache,
                                 T* __restrict__ v_cache, int Tn, const int32_t* __restrict__ pos_dev, int64_t Smax,
                                 int64_t width, int64_t n_vec) {
  constexpr int kN = Vec16<T>::kN;
  const int pos0 = *pos_dev;
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= 2 * n_vec) return;
  const bool is_v = i >= n_vec;
  if (is_v) i -= n_vec;
  const T* src = is_v ? v_new : k_new;
  T* dst = is_v ? v_cache : k_cache;
  const int64_t per_row = width / kN;
  const int64_t row = i / per_row, c = (i - row * per_row) * kN;
  const int64_t b = row / Tn, t = row - b * Tn;
  store16(dst + (b * Smax + pos0 + t) * width + c, load16(src + row * width + c));
}

// Attention of T new tokens per sequence against the cache: query (b, t) attends to the cached
// positions 0 .. pos0 + t (its own key included: the cache already holds the new keys).  One block of
// four warps per (query, head): warp w takes the keys n = w, w + 4, ... (lanes split the head
// dimension, online softmax per warp), then the four partial (maximum, sum, output) triples are merged
// in warp order.  q, o: [B * T, H * HD]; kc, vc: [B][Smax][Hkv * HD].  The number of cached positions is
// read from device memory, so that one captured graph of a token step serves every position.
template <typename T, int HD>
__global__ void __launch_bounds__(128)
attn_decode_kernel(const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc, T* __restrict__ o,
                   int Tn, const int32_t* __restrict__ pos_dev, int64_t Smax, int H, int Hkv, float scale) {
  constexpr int E = HD / 32;
  __shared__ float part_acc[4][HD];
  __shared__ float part_m[4], part_l[4];
  const int pos0 = *pos_dev;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int t = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int hk = hq / (H / Hkv);
  const int64_t dq = static_cast<int64_t>(H) * HD, dk = static_cast<int64_t>(Hkv) * HD;
  const T* qp = q + (static_cast<int64_t>(b) * Tn + t) * dq + hq * HD;
  float qr[E], acc[E];
#pragma unroll
  for (int j = 0; j < E; ++j) {
    qr[j] = to_f32<T>(qp[lane + 32 * j]) * scale;
    acc[j] = 0.f;
  }
  float mx = -INFINITY, l = 0.f;
  const T* kb = kc + static_cast<int64_t>(b) * Smax * dk + hk * HD;
  const T* vb = vc + static_cast<int64_t>(b) * Smax * dk + hk * HD;
  for (int n = w; n <= pos0 + t; n += 4) {
    const T* kp = kb + n * dk;
    const T* vp = vb + n * dk;
    float kv[E], vv[E];
#pragma unroll
    for (int j = 0; j < E; ++j) {
      kv[j] = to_f32<T>(kp[lane + 32 * j]);
      vv[j] = to_f32<T>(vp[lane + 32 * j]);
    }
    float dot = 0.f;
#pragma unroll
    for (int j = 0; j < E; ++j) dot = fmaf(qr[j], kv[j], dot);
#pragma unroll
    for (int off = 16; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    const float mn = fmaxf(mx, dot);
    const float corr = expf(mx - mn), p = expf(dot - mn);
    l = l * corr + p;
#pragma unroll
    for (int j = 0; j < E; ++j) acc[j] = fmaf(p, vv[j], acc[j] * corr);
    mx = mn;
  }
#pragma unroll
  for (int j = 0; j < E; ++j) part_acc[w][lane + 32 * j] = acc[j];
  if (lane == 0) {
    part_m[w] = mx;
    part_l[w] = l;
  }
  __syncthreads();
  if (w == 0) {
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) M = fmaxf(M, part_m[i]);
    float L = 0.f, out[E];
#pragma unroll
    for (int j = 0; j < E; ++j) out[j] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float f = part_m[i] == -INFINITY ? 0.f : expf(part_m[i] - M);     // a warp without keys contributes nothing
      L += part_l[i] * f;
#pragma unroll
      for (int j = 0; j < E; ++j) out[j] = fmaf(part_acc[i][lane + 32 * j], f, out[j]);
    }
    T* op = o + (static_cast<int64_t>(b) * Tn + t) * dq + hq * HD;
    const float inv = 1.0f / L;
#pragma unroll
    for (int j = 0; j < E; ++j) op[lane + 32 * j] = from_f32<T>(out[j] * inv);
  }
}

// The same attention with the two kernels before it folded in, for a handful of new tokens (a token
// step is a chain of short dependent launches: two fewer per layer).  q and k_new arrive unrotated.
// Block (t, hq, b) rotates its query at position pos0 + t, reads the keys and values of the new
// tokens 0 .. t from k_new / v_new (rotating each key at its position) and the older ones from the
// cache; the first query head of every key/value head also stores the rotated key and the value of
// token t in the cache.  No block reads a cache row that this launch writes.  Rotated values are
// rounded to T exactly where rope_kernel and the cache would round them.
// Sixteen key streams per block: a quarter warp (8 lanes) takes the keys n = s, s + 16, ... of stream
// s; a lane holds HD / 8 contiguous elements (16- or 32-byte loads), so a key costs three shuffles
// for the dot product, and four keys are in flight per warp.  Every stream keeps its own online
// softmax state; the streams are merged at the end in a fixed order (quarters of a warp by two
// shuffle steps, then the four warps through shared memory).
template <typename T, int HD>
__global__ void __launch_bounds__(128)
attn_decode_fused_kernel(const T* __restrict__ q, const T* __restrict__ k_new, const T* __restrict__ v_new,
                         T* __restrict__ kc, T* __restrict__ vc, T* __restrict__ o, const float2* __restrict__ rope_tab,
                         int Tn, const int32_t* __restrict__ pos_dev, int64_t Smax, int H, int Hkv, float scale) {
  constexpr int E = HD / 8, half = HD / 2;            // elements per lane; a lane's rotation partner is lane ^ 4
  __shared__ float part_acc[4][HD];
  __shared__ float part_m[4], part_l[4];
  chain_release();
  chain_wait();
  const int pos0 = *pos_dev;
  const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
  const int ql = lane & 7, stream = w * 4 + (lane >> 3);
  const int t = blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int hk = hq / (H / Hkv);
  const int64_t dq = static_cast<int64_t>(H) * HD, dk = static_cast<int64_t>(Hkv) * HD;
  const int e0 = ql * E;                              // first element of this lane
  auto load = [&](const T* p, float (&x)[E]) {        // E contiguous elements from p + e0
    constexpr int kN = 16 / static_cast<int>(sizeof(T));
#pragma unroll
    for (int i = 0; i < E; i += kN) {
      const Vec16<T> v = load16(p + e0 + i);
#pragma unroll
      for (int j = 0; j < kN; ++j) x[i + j] = to_f32<T>(v.v[j]);
    }
  };
  auto store = [&](T* p, const float (&x)[E]) {
    constexpr int kN = 16 / static_cast<int>(sizeof(T));
#pragma unroll
    for (int i = 0; i < E; i += kN) {
      Vec16<T> v;
#pragma unroll
      for (int j = 0; j < kN; ++j) v.v[j] = from_f32<T>(x[i + j]);
      store16(p + e0 + i, v);
    }
  };
  // element e < half pairs with e + half, held by lane ^ 4 at the same index
  auto rotate = [&](float (&x)[E], int pos) {
    if (rope_tab == nullptr) return;
    const bool low = ql < 4;
    const float2* cs = rope_tab + static_cast<int64_t>(pos) * half + (low ? e0 : e0 - half);
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float other = __shfl_xor_sync(0xffffffffu, x[i], 4);
      const float2 c = cs[i];
      // low half: a cos - b sin with (a, b) = (x, other); high half: b cos + a sin with (a, b) = (other, x)
      x[i] = to_f32<T>(from_f32<T>(low ? x[i] * c.x - other * c.y : x[i] * c.x + other * c.y));
    }
  };
  float qr[E], acc[E];
  load(q + (static_cast<int64_t>(b) * Tn + t) * dq + hq * HD, qr);
  rotate(qr, pos0 + t);
#pragma unroll
  for (int i = 0; i < E; ++i) {
    qr[i] *= scale;
    acc[i] = 0.f;
  }
  const T* knb = k_new + static_cast<int64_t>(b) * Tn * dk + hk * HD;
  const T* vnb = v_new + static_cast<int64_t>(b) * Tn * dk + hk * HD;
  T* kb = kc + static_cast<int64_t>(b) * Smax * dk + hk * HD;
  T* vb = vc + static_cast<int64_t>(b) * Smax * dk + hk * HD;
  if (w == 3 && hq % (H / Hkv) == 0) {                // (the warp with the fewest keys when few are cached)
    float kv[E], vv[E];
    load(knb + t * dk, kv);
    load(vnb + t * dk, vv);
    rotate(kv, pos0 + t);
    if (lane < 8) {
      store(kb + (pos0 + t) * dk, kv);
      store(vb + (pos0 + t) * dk, vv);
    }
  }
  float mx = -INFINITY, l = 0.f;
  const int last = pos0 + t;
  for (int n0 = 0; n0 <= last; n0 += 16) {            // (uniform trip count: the rotation shuffles need whole warps)
    const int n = n0 + stream;
    const bool live = n <= last;
    const int nn = live ? n : last;
    const bool fresh = nn >= pos0;
    float kv[E], vv[E];
    load(fresh ? knb + (nn - pos0) * dk : kb + nn * dk, kv);
    load(fresh ? vnb + (nn - pos0) * dk : vb + nn * dk, vv);
    if (__any_sync(0xffffffffu, fresh)) {
      float kr[E];
#pragma unroll
      for (int i = 0; i < E; ++i) kr[i] = kv[i];
      rotate(kr, nn);
      if (fresh) {
#pragma unroll
        for (int i = 0; i < E; ++i) kv[i] = kr[i];
      }
    }
    float dot = 0.f;
#pragma unroll
    for (int i = 0; i < E; ++i) dot = fmaf(qr[i], kv[i], dot);
#pragma unroll
    for (int off = 4; off; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
    if (live) {
      const float mn = fmaxf(mx, dot);
      const float corr = expf(mx - mn), p = expf(dot - mn);
      l = l * corr + p;
#pragma unroll
      for (int i = 0; i < E; ++i) acc[i] = fmaf(p, vv[i], acc[i] * corr);
      mx = mn;
    }
  }
  // merge the four streams of a warp (quarters 0+1 and 2+3, then the two halves), lower stream first
#pragma unroll
  for (int off = 8; off <= 16; off <<= 1) {
    const float om = __shfl_xor_sync(0xffffffffu, mx, off), ol = __shfl_xor_sync(0xffffffffu, l, off);
    const float M2 = fmaxf(mx, om);
    const float fs = mx == -INFINITY ? 0.f : expf(mx - M2), fo = om == -INFINITY ? 0.f : expf(om - M2);
    const bool first = (lane & off) == 0;             // this lane's state is the lower stream's
#pragma unroll
    for (int i = 0; i < E; ++i) {
      const float oa = __shfl_xor_sync(0xffffffffu, acc[i], off);
      acc[i] = first ? fmaf(oa, fo, acc[i] * fs) : fmaf(acc[i], fs, oa * fo);
    }
    l = first ? fmaf(ol, fo, l * fs) : fmaf(l, fs, ol * fo);
    mx = M2;
  }
  if (lane < 8) {
#pragma unroll
    for (int i = 0; i < E; ++i) part_acc[w][e0 + i] = acc[i];
    if (lane == 0) {
      part_m[w] = mx;
      part_l[w] = l;
    }
  }
  __syncthreads();
  if (w == 0 && lane < 8) {
    float M = -INFINITY;
#pragma unroll
    for (int i = 0; i < 4; ++i) M = fmaxf(M, part_m[i]);
    float L = 0.f, out[E];
#pragma unroll
    for (int j = 0; j < E; ++j) out[j] = 0.f;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float f = part_m[i] == -INFINITY ? 0.f : expf(part_m[i] - M);     // a warp without keys contributes nothing
      L += part_l[i] * f;
#pragma unroll
      for (int j = 0; j < E; ++j) out[j] = fmaf(part_acc[i][e0 + j], f, out[j]);
    }
    const float inv = 1.0f / L;
#pragma unroll
    for (int j = 0; j < E; ++j) out[j] *= inv;
    store(o + (static_cast<int64_t>(b) * Tn + t) * dq + hq * HD, out);
  }
}

// ------------------------------------------------------------------------------ paired form
// The two forwards of a ZO step (Definition 1: the loss at w + eps zbar and at w - eps zbar, same
// batch) carried through the network as centre c = (x+ + x-)/2 and half-difference d = (x+ - x-)/2
// instead of x+ and x-.  The perturbation changes an activation by less than a bf16 ulp; stored as
// x+ and x-, each rounded on its own, the difference f+ - f- (all that the projected gradient uses)
// drowns in rounding, whereas d has its own exponent and keeps 8 significant bits whatever its size.
// Every kernel below evaluates its function at c + d and c - d in fp32 and returns centre and
// half-difference of the two results, with the half-difference formed from expressions that do not
// cancel.  Buffers hold the centre rows first and the half-difference rows from row `row0` on.

// sinh(a) without cancellation for small |a|
__device__ __forceinline__ float sinh_stable(float a) {
  const float a2 = a * a;
  if (a2 < 0.25f) return a * (1.0f + a2 * (1.0f / 6.0f + a2 * (1.0f / 120.0f + a2 * (1.0f / 5040.0f + a2 * (1.0f / 362880.0f)))));
  const float u = __expf(a);
  return 0.5f * (u - __fdividef(1.0f, u));
}

// Block-wide sums of two values at once (same tree as block_sum).
__device__ __forceinline__ float2 block_sum2(float a, float b, float2* scratch) {
#pragma unroll
  for (int o = 16; o; o >>= 1) {
    a += __shfl_xor_sync(0xffffffffu, a, o);
    b += __shfl_xor_sync(0xffffffffu, b, o);
  }
  const int w = threadIdx.x >> 5, nw = blockDim.x >> 5;
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[w] = make_float2(a, b);
  __syncthreads();
  float2 t = make_float2(0.f, 0.f);
  for (int i = 0; i < nw; ++i) {
    t.x += scratch[i].x;
    t.y += scratch[i].y;
  }
  return t;
}

// add_norm_kernel in the paired form.  Residual add of both parts (linear), then with
// x+- = c +- d:  mean(x+-^2) = mean(c^2 + d^2) +- 2 mean(c d) = sc +- sx, a+- = sqrt(sc +- sx + eps),
// r+- = 1/a+-:  rc = (r+ + r-)/2,  rd = (r+ - r-)/2 = -sx / ((a+ + a-) a+ a-);
// out_c = (c rc + d rd) gamma (+ beta),  out_d = (c rd + d rc) gamma.  LayerNorm: the same on c - mean(c),
// d - mean(d).  One block per token; h_d = h + row0 * d_model etc.
// kMaxV: float4 per thread a row may need (d <= 1024 kMaxV): the smaller instantiation keeps half the registers
// and so twice the blocks per SM, whose load and reduction phases then overlap.
template <typename T, typename TO = T, int kMaxV = 8>
__global__ void __launch_bounds__(256)
add_norm_pair_kernel(float* __restrict__ h, const T* __restrict__ y, int64_t row0, const float* __restrict__ gamma,
                     const float* __restrict__ beta, int d, float eps, bool layer_norm, int64_t row_stride,
                     int64_t row_offset, TO* __restrict__ out, int64_t out_row0) {
  __shared__ float2 scratch[32];
  chain_release();
  chain_wait();
  const int64_t m = static_cast<int64_t>(blockIdx.x) * row_stride + row_offset;
  float* xc = h + m * d;
  float* xd = h + (row0 + m) * d;
  const int nv = d >> 2;
  float4 vc[kMaxV], vd[kMaxV];
  float s1 = 0.f, s2 = 0.f;
  auto add4 = [](float4& v, const T* yp) {
    if constexpr (sizeof(T) == 2) {
      const uint2 raw = *reinterpret_cast<const uint2*>(yp);
      v.x += __uint_as_float(raw.x << 16);
      v.y += __uint_as_float(raw.x & 0xFFFF0000u);
      v.z += __uint_as_float(raw.y << 16);
      v.w += __uint_as_float(raw.y & 0xFFFF0000u);
    } else {
      v.x += to_f32<T>(yp[0]);
      v.y += to_f32<T>(yp[1]);
      v.z += to_f32<T>(yp[2]);
      v.w += to_f32<T>(yp[3]);
    }
  };
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    const int c = threadIdx.x + i * 256;
    vc[i] = vd[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (c < nv) {
      vc[i] = reinterpret_cast<const float4*>(xc)[c];
      vd[i] = reinterpret_cast<const float4*>(xd)[c];
      if (y != nullptr) {
        add4(vc[i], y + m * d + c * 4);
        add4(vd[i], y + (row0 + m) * d + c * 4);
        if (row_stride == 1) {
          reinterpret_cast<float4*>(xc)[c] = vc[i];
          reinterpret_cast<float4*>(xd)[c] = vd[i];
        }
      }
      s1 += (vc[i].x + vc[i].y) + (vc[i].z + vc[i].w);
      s2 += (vd[i].x + vd[i].y) + (vd[i].z + vd[i].w);
    }
  }
  float mc = 0.f, md = 0.f;
  if (layer_norm) {
    const float2 mu = block_sum2(s1, s2, scratch);
    mc = mu.x / d;
    md = mu.y / d;
  }
  float qc = 0.f, qx = 0.f;
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    if (threadIdx.x + i * 256 < nv) {
      const float c0 = vc[i].x - mc, c1 = vc[i].y - mc, c2 = vc[i].z - mc, c3 = vc[i].w - mc;
      const float d0 = vd[i].x - md, d1 = vd[i].y - md, d2 = vd[i].z - md, d3 = vd[i].w - md;
      qc += ((c0 * c0 + d0 * d0) + (c1 * c1 + d1 * d1)) + ((c2 * c2 + d2 * d2) + (c3 * c3 + d3 * d3));
      qx += (c0 * d0 + c1 * d1) + (c2 * d2 + c3 * d3);
    }
  }
  const float2 q = block_sum2(qc, qx, scratch);
  const float sc = q.x / d, sx = 2.0f * q.y / d;
  const float ap = sqrtf(sc + sx + eps), am = sqrtf(sc - sx + eps);
  const float rc = 0.5f * (1.0f / ap + 1.0f / am);
  const float rd = -sx / ((ap + am) * ap * am);
  TO* oc = out + static_cast<int64_t>(blockIdx.x) * d;
  TO* od = out + (out_row0 + static_cast<int64_t>(blockIdx.x)) * d;
  auto put4 = [](TO* op, float o0, float o1, float o2, float o3) {
    if constexpr (sizeof(TO) == 2) {
      const __nv_bfloat162 lo = __floats2bfloat162_rn(o0, o1), hi = __floats2bfloat162_rn(o2, o3);
      uint2 pk;
      pk.x = *reinterpret_cast<const uint32_t*>(&lo);
      pk.y = *reinterpret_cast<const uint32_t*>(&hi);
      *reinterpret_cast<uint2*>(op) = pk;
    } else {
      *reinterpret_cast<float4*>(op) = make_float4(o0, o1, o2, o3);
    }
  };
#pragma unroll
  for (int i = 0; i < kMaxV; ++i) {
    const int c = threadIdx.x + i * 256;
    if (c < nv) {
      const float4 g = reinterpret_cast<const float4*>(gamma)[c];
      float4 bt = make_float4(0.f, 0.f, 0.f, 0.f);
      if (beta) bt = reinterpret_cast<const float4*>(beta)[c];
      const float c0 = vc[i].x - mc, c1 = vc[i].y - mc, c2 = vc[i].z - mc, c3 = vc[i].w - mc;
      const float d0 = vd[i].x - md, d1 = vd[i].y - md, d2 = vd[i].z - md, d3 = vd[i].w - md;
      put4(oc + c * 4, (c0 * rc + d0 * rd) * g.x + bt.x, (c1 * rc + d1 * rd) * g.y + bt.y,
           (c2 * rc + d2 * rd) * g.z + bt.z, (c3 * rc + d3 * rd) * g.w + bt.w);
      put4(od + c * 4, (c0 * rd + d0 * rc) * g.x, (c1 * rd + d1 * rc) * g.y, (c2 * rd + d2 * rc) * g.z,
           (c3 * rd + d3 * rc) * g.w);
    }
  }
}

// silu(g) * u in the paired form, in place on gate.  With g+- = gc +- gd and s(x) = 1/(1+exp(-x)):
// s+ - s- = 2 exp(-gc) sinh(gd) s+ s-  (for gc < 0 written with 1 - s, so that nothing overflows);
// silu: tc = gc sc + gd sd, td = gc sd + gd sc;  out_c = tc uc + td ud,  out_d = tc ud + td uc.
template <typename T>
__global__ void silu_mul_pair_kernel(T* __restrict__ gate, const T* __restrict__ up, int64_t n, int64_t off_d) {
  chain_release();
  chain_wait();
  constexpr int kN = Vec16<T>::kN;
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * kN;
  if (i >= n) return;
  const Vec16<T> gc = load16(gate + i), gd = load16(gate + off_d + i), uc = load16(up + i), ud = load16(up + off_d + i);
  Vec16<T> rc, rd;
#pragma unroll
  for (int j = 0; j < kN; ++j) {
    const float c = to_f32<T>(gc.v[j]), d = to_f32<T>(gd.v[j]);
    // (fast reciprocals: 2 ulp, against a result rounded to bf16; with the exact division the kernel was bound by
    // instruction issue, not by its 540 MB)
    const float sp = __fdividef(1.0f, 1.0f + __expf(-(c + d))), sm = __fdividef(1.0f, 1.0f + __expf(-(c - d)));
    const float q = __expf(-fabsf(c)) * sinh_stable(d);
    const float sd = c >= 0.f ? q * sp * sm : q * (1.0f - sp) * (1.0f - sm);
    const float sc = 0.5f * (sp + sm);
    const float tc = c * sc + d * sd, td = c * sd + d * sc;
    const float a = to_f32<T>(uc.v[j]), b = to_f32<T>(ud.v[j]);
    rc.v[j] = from_f32<T>(tc * a + td * b);
    rd.v[j] = from_f32<T>(tc * b + td * a);
  }
  store16(gate + i, rc);
  store16(gate + off_d + i, rd);
}

// max(x, 0) in the paired form, in place.
template <typename T>
__global__ void relu_pair_kernel(T* __restrict__ x, int64_t n, int64_t off_d) {
  constexpr int kN = Vec16<T>::kN;
  const int64_t i = (static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x) * kN;
  if (i >= n) return;
  Vec16<T> c = load16(x + i), d = load16(x + off_d + i);
#pragma unroll
  for (int j = 0; j < kN; ++j) {
    const float a = to_f32<T>(c.v[j]), b = to_f32<T>(d.v[j]);
    const float p = a + b, q = a - b;
    if (p > 0.f && q > 0.f) continue;                   // both sides pass: (a, b) unchanged
    const float rp = fmaxf(p, 0.f), rq = fmaxf(q, 0.f); // at least one side is clamped: no cancellation to fear
    c.v[j] = from_f32<T>(0.5f * (rp + rq));
    d.v[j] = from_f32<T>(0.5f * (rp - rq));
  }
  store16(x + i, c);
  store16(x + off_d + i, d);
}

// ce_rows_kernel in the paired form: logits lc (row m) and ld (row row0 + m).  With reference value R >=
// every lc + |ld|:  P = sum exp(lc - R) cosh(ld),  D = sum exp(lc - R) sinh(ld), so that
// logsumexp(lc +- ld) = R + log(P +- D).  Centre and half-difference of the two cross-entropies:
//   cc = R + (log(P + D) + log(P - D)) / 2 - lc[t],   cd = log1p(2 D / (P - D)) / 2 - ld[t];
// loss_plus[m] = cc + cd, loss_minus[m] = cc - cd in fp64.
__global__ void __launch_bounds__(256)
ce_rows_pair_kernel(const float* __restrict__ logits, int64_t row0, const int32_t* __restrict__ tok, int S, int V,
                    double* __restrict__ loss_plus, double* __restrict__ loss_minus) {
  __shared__ float2 scratch2[32];
  __shared__ float scratch[32];
  const int64_t m = blockIdx.x;
  if ((m % S) == S - 1) {
    if (threadIdx.x == 0) {
      loss_plus[m] = 0.0;
      loss_minus[m] = 0.0;
    }
    return;
  }
  const float* lc = logits + m * V;
  const float* ld = logits + (row0 + m) * V;
  float R = -INFINITY, Ps = 0.f, Ds = 0.f;
  for (int c = threadIdx.x; c < V; c += blockDim.x) {
    const float a = lc[c], b = ld[c];
    const float ref = a + fabsf(b);
    if (ref > R) {
      const float sc = __expf(R - ref);     // exp(-inf) = 0 on the first element
      Ps *= sc;
      Ds *= sc;
      R = ref;
    }
    const float e = __expf(a - R), u = __expf(b);
    Ps += e * 0.5f * (u + 1.0f / u);
    Ds += e * sinh_stable(b);
  }
  float bm = R;
#pragma unroll
  for (int o = 16; o; o >>= 1) bm = fmaxf(bm, __shfl_xor_sync(0xffffffffu, bm, o));
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = bm;
  __syncthreads();
  for (int i = 0; i < (blockDim.x >> 5); ++i) bm = fmaxf(bm, scratch[i]);
  const float sc = (R == -INFINITY) ? 0.f : __expf(R - bm);
  const float2 t = block_sum2(Ps * sc, Ds * sc, scratch2);
  if (threadIdx.x == 0) {
    int32_t tg = tok[m + 1];
    tg = tg < 0 ? 0 : (tg >= V ? V - 1 : tg);
    const double P = t.x, D = t.y;
    const double cc = static_cast<double>(bm) + 0.5 * (log(P + D) + log(P - D)) - static_cast<double>(lc[tg]);
    const double cd = 0.5 * log1p(2.0 * D / (P - D)) - static_cast<double>(ld[tg]);
    loss_plus[m] = cc + cd;
    loss_minus[m] = cc - cd;
  }
}

// cls2_kernel in the paired form: a_last holds the B centre states, then the B half-differences.
__global__ void __launch_bounds__(256)
cls2_pair_kernel(const float* __restrict__ a_last, int B, const __nv_bfloat16* __restrict__ lm_head,
                 const int32_t* __restrict__ cand, const int32_t* __restrict__ labels, int d, int V,
                 double* __restrict__ loss_plus, double* __restrict__ loss_minus) {
  __shared__ float2 scratch[32];
  const int b = blockIdx.x;
  const float* ac = a_last + static_cast<int64_t>(b) * d;
  const float* ad = a_last + static_cast<int64_t>(B + b) * d;
  int32_t c0 = cand[0], c1 = cand[1];
  c0 = c0 < 0 ? 0 : (c0 >= V ? V - 1 : c0);
  c1 = c1 < 0 ? 0 : (c1 >= V ? V - 1 : c1);
  const __nv_bfloat16* e0 = lm_head + static_cast<int64_t>(c0) * d;
  const __nv_bfloat16* e1 = lm_head + static_cast<int64_t>(c1) * d;
  float s0c = 0.f, s1c = 0.f, s0d = 0.f, s1d = 0.f;
  for (int c = threadIdx.x; c < d; c += blockDim.x) {
    const float w0 = __bfloat162float(e0[c]), w1 = __bfloat162float(e1[c]);
    s0c = fmaf(ac[c], w0, s0c);
    s1c = fmaf(ac[c], w1, s1c);
    s0d = fmaf(ad[c], w0, s0d);
    s1d = fmaf(ad[c], w1, s1d);
  }
  const float2 tc = block_sum2(s0c, s1c, scratch);
  const float2 td = block_sum2(s0d, s1d, scratch);
  if (threadIdx.x == 0) {
    for (int sgn = 0; sgn < 2; ++sgn) {
      const double f = sgn ? -1.0 : 1.0;
      const double l0 = tc.x + f * td.x, l1 = tc.y + f * td.y, mx = l0 > l1 ? l0 : l1;
      const double lse = mx + log(exp(l0 - mx) + exp(l1 - mx));
      (sgn ? loss_minus : loss_plus)[b] = lse - (labels[b] ? l1 : l0);
    }
  }
}

__global__ void set_i32_kernel(int32_t* p, int32_t v) { *p = v; }

// *out = (sum of v[0..n)) / denom, fixed order, fp64.
__global__ void __launch_bounds__(1024) mean_f64_kernel(const double* __restrict__ v, int64_t n, double denom,
                                                        double* __restrict__ out) {
  __shared__ double s[1024];
  double t = 0.0;
  for (int64_t i = threadIdx.x; i < n; i += 1024) t += v[i];
  s[threadIdx.x] = t;
  __syncthreads();
  for (int o = 512; o; o >>= 1) {
    if (threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) *out = s[0] / denom;
}

// sums = (f+ * count, f- * count, count): what data-parallel replicas add up
__global__ void loss_sums_kernel(const double* __restrict__ fp, const double* __restrict__ fm, double count,
                                 double* __restrict__ sums) {
  sums[0] = *fp * count;
  sums[1] = *fm * count;
  sums[2] = count;
}
// (f+, f-) = (sums[0], sums[1]) / sums[2]
__global__ void loss_means_kernel(const double* __restrict__ sums, double* __restrict__ fp, double* __restrict__ fm) {
  *fp = sums[0] / sums[2];
  *fm = sums[1] / sums[2];
}

__global__ void offset_eid_kernel(const int32_t* __restrict__ eid, int64_t n, int32_t off, int32_t* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) out[i] = eid[i] + off;
}

__global__ void gidx_kernel(const int64_t* __restrict__ idx, int64_t nnz, int64_t base, int64_t* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < nnz) out[i] = base + idx[i];
}

}  // namespace szo

using namespace szo;

struct szo_model {
  szo_model_config cfg;
  szo_model_weights top;
  std::vector<szo_layer_weights> layers;
  std::vector<szo_linear_t*> plans;      // n_layers * n_lin
  std::vector<int64_t> offsets;          // start of each linear's entries in S_all (+ total)
  szo_linear_t* lm_head_plan = nullptr;
  int n_lin = 0;
  float* S_all = nullptr;
  int64_t k_total = 0;
  int64_t* gidx = nullptr;
  // paired form, sparse product: linear t's record slots are [offsets[t], offsets[t + 1]) of these arrays
  uint32_t* colk = nullptr;              // per slot: column | width of the column field << 24
  int32_t* csrc = nullptr;               // per slot: the entry (index into S_all / z) it holds
  uint32_t* crecs = nullptr;             // per slot: the record of the current step
  int32_t* geid = nullptr;      // [k_total] entry id in S_all of each bucket-ordered record
  uint16_t* gpos = nullptr;     // [k_total] in-tile position of each bucket-ordered record
  uint2* recs = nullptr;        // [k_total] (position, value) records of the current forward
  float* zkept = nullptr;       // [k_total] z of the current step, kept by the first perturb pass
  float *Splus = nullptr, *Sminus = nullptr;   // [k_total] the two perturbed copies of S (two forwards side by side)
  bool dual_rows = false;       // the activation buffers hold 2 * Mmax rows
  bool paired = false;          // SZO_MODE_PAIRED: a step's two forwards as centre and half-difference
  // dense bf16 weights (group == 0) with many tokens: every launch group keeps its effective weight
  // resident (a private copy of the frozen matrices, masked entries rewritten per forward)
  bool resident = false;
  std::vector<__nv_bfloat16*> res_W, res_saved;   // indexed by the first linear of a group; else nullptr
  int64_t Mmax = 0;
  // activations
  float* h = nullptr;
  void *a = nullptr, *q = nullptr, *k = nullptr, *v = nullptr, *o = nullptr, *y = nullptr, *gate = nullptr,
       *up = nullptr;
  float* logits = nullptr;
  double* tok_loss = nullptr;
  float2* rope_tab = nullptr;
  void* ws = nullptr;
  size_t ws_bytes = 0;
  int32_t *d_tokens = nullptr, *d_labels = nullptr, *d_cand = nullptr;
  double* d_scalars = nullptr;
  int64_t last_launches = 0;
  void *kcache = nullptr, *vcache = nullptr;     // [n_layers][max_batch][max_seq][n_kv_heads * head_dim], act dtype
  float* h2 = nullptr;                           // [2][d_model]: second copy of the residual stream of a one- or two-row token step
  int sparse_dt = SZO_F32;                       // storage format of the sparse values (szo_model_set_sparse_storage)
  void* S16_out = nullptr;                       // caller-owned mirror of the stored form, or NULL
  szo_linear_t* decode_head = nullptr;           // LM head plan of the decode path when the loss path has none
  int32_t* d_pos = nullptr;                      // cached positions before the current decode call
  int32_t* dec_tokens = nullptr;                 // the call's tokens, at an address that a captured graph can keep
  float* dec_logits = nullptr;                   // [max_batch][vocab]
  struct DecodeGraph {
    int B, T;
    const float* Sv;
    cudaGraphExec_t exec;
  };
  std::vector<DecodeGraph> dec_graphs;           // one captured token step per (B, T, sparse values)
  bool dec_use_graph = true;
  bool z_valid = false;         // zkept holds the z of the last szo_model_zo_losses, not yet consumed
  std::vector<void*> owned;
  // measurement aid: CUDA events around every decoder-block linear launch
  bool timing = false;
  std::vector<cudaEvent_t> events;
  size_t events_used = 0;
};

namespace {

template <typename P> szo_status dev_alloc(szo_model* m, P** p, size_t bytes) {
  void* q = nullptr;
  SZO_CHECK_CUDA(cudaMalloc(&q, bytes ? bytes : 16));
  m->owned.push_back(q);
  *p = static_cast<P*>(q);
  return SZO_OK;
}

void linear_shape(const szo_model_config& c, int j, int64_t* N, int64_t* K) {
  const int64_t d = c.d_model, kv = static_cast<int64_t>(c.n_kv_heads) * (c.d_model / c.n_heads), ff = c.d_ff;
  if (c.arch == 0) {
    const int64_t n[7] = {d, kv, kv, d, ff, ff, d}, k[7] = {d, d, d, d, d, d, ff};
    *N = n[j]; *K = k[j];
  } else {
    const int64_t n[6] = {d, kv, kv, d, ff, d}, k[6] = {d, d, d, d, d, ff};
    *N = n[j]; *K = k[j];
  }
}

unsigned blocks_for(int64_t n, int t) { return static_cast<unsigned>(ceil_div(n, t)); }

// One forward, or (Sv2 != nullptr) the two forwards of a ZO step side by side: the same tokens with
// two sets of sparse values.  Every activation buffer then holds 2 M rows (set 0 first), the
// elementwise, norm and attention kernels run once over both sets, and each linear group makes one
// weight pass for both (materialised form only).
template <typename T>
szo_status run_loss_t(szo_model* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand, int B,
                      int S, const float* Sv, double* loss_dev, cudaStream_t st, const float* Sv2 = nullptr,
                      double* loss_dev2 = nullptr) {
  const szo_model_config& c = m->cfg;
  const int64_t M = static_cast<int64_t>(B) * S;
  const int nsets = Sv2 != nullptr ? 2 : 1;
  const int64_t Mr = nsets * M;                 // rows of the activation buffers
  const int Br = nsets * B;                     // sequences
  const int d = c.d_model, H = c.n_heads, Hkv = c.n_kv_heads, hd = d / H, ff = c.d_ff;
  const int act = c.act_dtype;
  const bool opt = c.arch == 1;
  auto add_norm = d <= 4096 ? add_norm_kernel<T, T, 4> : add_norm_kernel<T, T, 8>;
  T *a = static_cast<T*>(m->a), *q = static_cast<T*>(m->q), *k = static_cast<T*>(m->k), *v = static_cast<T*>(m->v),
    *o = static_cast<T*>(m->o), *y = static_cast<T*>(m->y), *gate = static_cast<T*>(m->gate),
    *up = static_cast<T*>(m->up);
  // a lone forward of a model in the paired mode (szo_model_loss) is a SparseAdd forward
  const int32_t lmode = c.linear_mode == SZO_MODE_PAIRED ? SZO_MODE_SPARSE_ADD : c.linear_mode;
  const bool pregather = lmode != SZO_MODE_FP32_VALIDATE && lmode != SZO_MODE_SPMM && m->k_total > 0;
  auto lin_single = [&](int layer, int j, const void* x, void* out) -> szo_status {
    const int t = layer * m->n_lin + j;
    if (m->timing) {
      while (m->events.size() < m->events_used + 2) {
        cudaEvent_t e;
        SZO_CHECK_CUDA(cudaEventCreate(&e));
        m->events.push_back(e);
      }
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used], st));
    }
    const szo_status rc = linear_fwd_impl(m->plans[t], x, act, M, Sv + m->offsets[t],
                                          pregather ? m->recs + m->offsets[t] : nullptr, out, act, lmode,
                                          m->ws, m->ws_bytes, st);
    if (m->timing) {
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used + 1], st));
      m->events_used += 2;
    }
    return rc;
  };
  // layers j0 .. j0 + n - 1 read the same x: one fused launch when the tensor-core path allows it
  // relu_applied (n == 1 only): asks for y = max(y, 0); set when the launch applied it in its epilogue
  auto lin_group = [&](int layer, int j0, int n, const void* x, void* const* outs,
                       bool* relu_applied = nullptr) -> szo_status {
    const int t0 = layer * m->n_lin + j0;
    const szo_linear* plans[3];
    const uint2* recs[3];
    for (int i = 0; i < n; ++i) {
      plans[i] = m->plans[t0 + i];
      recs[i] = m->recs + m->offsets[t0 + i];
    }
    const bool res = m->resident && sizeof(T) == 2;
    if (!res && nsets == 1 && !(pregather && sizeof(T) == 2 && (n == 1 || tc_can_fuse(plans, n, M)))) {
      for (int i = 0; i < n; ++i) SZO_TRY(lin_single(layer, j0 + i, x, outs[i]));
      return SZO_OK;
    }
    if (!res && nsets == 1 && n == 1) return lin_single(layer, j0, x, outs[0]);
    const bool mat = res || nsets == 2 || tc_use_materialised(plans[0], M);
    const float* spert[3];
    const float* spert2[3];
    for (int i = 0; i < n; ++i) {
      spert[i] = Sv + m->offsets[t0 + i];
      spert2[i] = nsets == 2 ? Sv2 + m->offsets[t0 + i] : nullptr;
    }
    if (m->timing) {
      while (m->events.size() < m->events_used + 2) {
        cudaEvent_t e;
        SZO_CHECK_CUDA(cudaEventCreate(&e));
        m->events.push_back(e);
      }
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used], st));
    }
    const szo_status rc = mat ? linear_fwd_tc_materialised(plans, n, x, M, spert, outs, act, m->ws, m->ws_bytes, st,
                                                           nsets == 2 ? spert2 : nullptr, res ? m->res_W[t0] : nullptr,
                                                           res ? m->res_saved[t0] : nullptr, relu_applied != nullptr)
                              : linear_fwd_tc_group(plans, n, x, M, recs, outs, act, m->ws, m->ws_bytes, st);
    if (mat && relu_applied != nullptr) *relu_applied = true;
    if (m->timing) {
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used + 1], st));
      m->events_used += 2;
    }
    return rc;
  };
  auto lin = [&](int layer, int j, const void* x, void* out) -> szo_status {
    void* const outs[1] = {out};
    return lin_group(layer, j, 1, x, outs);
  };
  for (int set = 0; set < nsets; ++set) {
    embed_kernel<<<static_cast<unsigned>(M), 128, 0, st>>>(tokens, static_cast<const __nv_bfloat16*>(m->top.embed),
                                                          static_cast<const __nv_bfloat16*>(m->top.pos), S, d,
                                                          c.vocab, m->h + set * M * d);
    count_launch();
  }
  // One gather of all sparse values into the bucket order of every linear (SparseAdd mode)
  if (nsets == 1 && pregather && !m->resident && !(m->plans.size() > 0 && tc_use_materialised(m->plans[0], M)))
    SZO_TRY(gather_values(Sv, m->geid, m->gpos, m->k_total, m->recs, st));
  const T* pending = nullptr;     // projection output still to be added to the residual stream
  for (int l = 0; l < c.n_layers; ++l) {
    const szo_layer_weights& L = m->layers[l];
    add_norm<<<static_cast<unsigned>(Mr), 256, 0, st>>>(m->h, pending, L.attn_norm_g, L.attn_norm_b, d,
                                                                 c.norm_eps, opt, 1, 0, a);
    count_launch();
    {
      void* const qkv[3] = {q, k, v};
      SZO_TRY(lin_group(l, 0, 3, a, qkv));
    }
    if (!opt) {
      const int64_t n_vec = Mr * (H + Hkv) * ((hd / 2) / Vec16<T>::kN);
      rope_kernel<T><<<blocks_for(n_vec, 256), 256, 0, st>>>(q, k, m->rope_tab, Mr, S, H, Hkv, hd);
      count_launch();
    }
    if constexpr (sizeof(T) == 2) {
      SZO_TRY(launch_flash_attention_bf16(q, k, v, o, Br, S, H, Hkv, hd, st));
    } else {
      dim3 grid(static_cast<unsigned>(ceil_div(S, 4)), H, Br);
      const float scale = 1.0f / sqrtf(static_cast<float>(hd));
      if (hd == 64) attn_warp_kernel<T, 64><<<grid, 128, 0, st>>>(q, k, v, o, S, H, Hkv, scale);
      else attn_warp_kernel<T, 128><<<grid, 128, 0, st>>>(q, k, v, o, S, H, Hkv, scale);
      count_launch();
    }
    SZO_TRY(lin(l, 3, o, y));
    add_norm<<<static_cast<unsigned>(Mr), 256, 0, st>>>(m->h, y, L.mlp_norm_g, L.mlp_norm_b, d, c.norm_eps,
                                                                 opt, 1, 0, a);
    count_launch();
    if (!opt) {
      void* const gu[2] = {gate, up};
      SZO_TRY(lin_group(l, 4, 2, a, gu));
      silu_mul_kernel<T><<<blocks_for(Mr * ff / Vec16<T>::kN, 256), 256, 0, st>>>(gate, up, Mr * ff, gate);
      count_launch();
      SZO_TRY(lin(l, 6, gate, y));
    } else {
      bool relu_applied = false;
      {
        void* const fc1_out[1] = {gate};
        SZO_TRY(lin_group(l, 4, 1, a, fc1_out, &relu_applied));
      }
      if (!relu_applied) {
        relu_kernel<T><<<blocks_for(Mr * ff / Vec16<T>::kN, 256), 256, 0, st>>>(gate, Mr * ff);
        count_launch();
      }
      SZO_TRY(lin(l, 5, gate, y));
    }
    pending = y;                  // added by the next norm (next layer's, or the final one)
  }
  double* const loss_out[2] = {loss_dev, loss_dev2};
  if (c.loss_kind == 0) {
    add_norm<<<static_cast<unsigned>(Mr), 256, 0, st>>>(m->h, pending, m->top.final_norm_g,
                                                                 m->top.final_norm_b, d, c.norm_eps, opt, 1, 0, a);
    count_launch();
    const int mode = lmode == SZO_MODE_FP32_VALIDATE ? SZO_MODE_FP32_VALIDATE : SZO_MODE_SPARSE_ADD;
    SZO_TRY(szo_linear_fwd(m->lm_head_plan, a, static_cast<szo_dtype>(act), Mr, nullptr, m->logits, SZO_F32, mode,
                           m->ws, m->ws_bytes, st));
    for (int set = 0; set < nsets; ++set) {
      ce_rows_kernel<<<static_cast<unsigned>(M), 256, 0, st>>>(m->logits + set * M * c.vocab, tokens, S, c.vocab,
                                                              m->tok_loss + set * M);
      mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss + set * M, M, static_cast<double>(B) * (S - 1), loss_out[set]);
      count_launch(2);
    }
  } else {
    // only B rows per set feed this loss: keep their normalised states in fp32 (the q buffer is free here)
    float* a_last = reinterpret_cast<float*>(m->q);
    add_norm_kernel<T, float><<<static_cast<unsigned>(Br), 256, 0, st>>>(
        m->h, pending, m->top.final_norm_g, m->top.final_norm_b, d, c.norm_eps, opt, S, S - 1, a_last);
    count_launch();
    for (int set = 0; set < nsets; ++set) {
      cls2_kernel<float><<<static_cast<unsigned>(B), 256, 0, st>>>(
          a_last + static_cast<int64_t>(set) * B * d, static_cast<const __nv_bfloat16*>(m->top.lm_head), cand, labels, d,
          c.vocab, m->tok_loss + set * B);
      mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss + set * B, B, static_cast<double>(B), loss_out[set]);
      count_launch(2);
    }
  }
  SZO_CHECK_LAUNCH("model kernels");
  return SZO_OK;
}


// Both forwards of a ZO step in the paired form (see the kernels above): bf16 activations, dense
// mode of the tensor-core kernel on W = RN_bf16(Dequantize(Q) + S) (written per launch group, or
// resident for dense bf16 weights), eps * xc Zbar^T added to the half-difference rows in the
// epilogue.  Rows [0, M) of every activation buffer are the centre, rows [Mp, Mp + M) the
// half-difference, Mp = M rounded up to 256 (rows in between are never read as results).
szo_status run_loss_paired(szo_model* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand, int B, int S,
                           const float* Sv, const float* z, float eps, double* loss_plus_dev, double* loss_minus_dev,
                           cudaStream_t st) {
  using T = __nv_bfloat16;
  const szo_model_config& c = m->cfg;
  const int64_t M = static_cast<int64_t>(B) * S;
  const int64_t Mp = static_cast<int64_t>(round_up(static_cast<size_t>(M), 256));
  const int64_t Mr = Mp + M;
  const int d = c.d_model, H = c.n_heads, Hkv = c.n_kv_heads, hd = d / H, ff = c.d_ff;
  const int64_t dkv = static_cast<int64_t>(Hkv) * hd;
  const bool opt = c.arch == 1;
  auto add_norm_pair = d <= 4096 ? add_norm_pair_kernel<T, T, 4> : add_norm_pair_kernel<T, T, 8>;
  T *a = static_cast<T*>(m->a), *q = static_cast<T*>(m->q), *k = static_cast<T*>(m->k), *v = static_cast<T*>(m->v),
    *o = static_cast<T*>(m->o), *y = static_cast<T*>(m->y), *gate = static_cast<T*>(m->gate), *up = static_cast<T*>(m->up);
  auto lin_group = [&](int layer, int j0, int n, const void* x, void* const* outs) -> szo_status {
    const int t0 = layer * m->n_lin + j0;
    const szo_linear* plans[3];
    const float* sv[3];
    const uint32_t* crec[3];
    const float* zz[3];
    for (int i = 0; i < n; ++i) {
      plans[i] = m->plans[t0 + i];
      sv[i] = Sv + m->offsets[t0 + i];
      crec[i] = m->crecs + m->offsets[t0 + i];
      zz[i] = z + m->offsets[t0 + i];
    }
    if (m->timing) {
      while (m->events.size() < m->events_used + 2) {
        cudaEvent_t e;
        SZO_CHECK_CUDA(cudaEventCreate(&e));
        m->events.push_back(e);
      }
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used], st));
    }
    const PairedArgs pa{crec, zz, eps, tc_paired_dense_cross(plans, n)};
    const bool res = m->resident;
    const szo_status rc = linear_fwd_tc_materialised(plans, n, x, M, sv, outs, SZO_BF16, m->ws, m->ws_bytes, st, nullptr,
                                                     res ? m->res_W[t0] : nullptr, res ? m->res_saved[t0] : nullptr,
                                                     false, &pa);
    if (m->timing) {
      SZO_CHECK_CUDA(cudaEventRecord(m->events[m->events_used + 1], st));
      m->events_used += 2;
    }
    return rc;
  };
  auto lin = [&](int layer, int j, const void* x, void* out) -> szo_status {
    void* const outs[1] = {out};
    return lin_group(layer, j, 1, x, outs);
  };
  // (column, eps * z) of every record slot, once for all linears of the step, in one launch (the
  // record layout depends on K: the width of the column field travels with the column)
  SZO_TRY(pack_cross_records_all(m->colk, m->csrc, z, eps, m->k_total, m->crecs, st));
  embed_kernel<<<static_cast<unsigned>(M), 128, 0, st>>>(tokens, static_cast<const __nv_bfloat16*>(m->top.embed),
                                                        static_cast<const __nv_bfloat16*>(m->top.pos), S, d, c.vocab, m->h);
  SZO_CHECK_CUDA(cudaMemsetAsync(m->h + Mp * d, 0, static_cast<size_t>(M) * d * sizeof(float), st));   // both forwards embed alike
  count_launch();
  const T* pending = nullptr;
  for (int l = 0; l < c.n_layers; ++l) {
    const szo_layer_weights& L = m->layers[l];
    SZO_CHECK_CUDA(launch_maybe_chained(add_norm_pair, dim3(static_cast<unsigned>(M)), dim3(256), 0, st, step_chained(), m->h, pending,
                                        Mp, L.attn_norm_g, L.attn_norm_b, d, c.norm_eps, opt, 1, 0, a, Mp));
    count_launch();
    {
      void* const qkv[3] = {q, k, v};
      SZO_TRY(lin_group(l, 0, 3, a, qkv));
    }
    if (!opt) {        // the rotation is linear: the same kernel on both parts
      const int64_t n_vec = M * (H + Hkv) * ((hd / 2) / Vec16<T>::kN);
      if (Mp == M) {   // no gap between the two kinds of rows: one launch (a row's position is its index modulo S)
        SZO_CHECK_CUDA(launch_maybe_chained(rope_kernel<T>, dim3(blocks_for(2 * n_vec, 256)), dim3(256), 0, st, step_chained(), q, k,
                                            m->rope_tab, 2 * M, S, H, Hkv, hd, 0, nullptr));
        count_launch();
      } else {
        rope_kernel<T><<<blocks_for(n_vec, 256), 256, 0, st>>>(q, k, m->rope_tab, M, S, H, Hkv, hd);
        rope_kernel<T><<<blocks_for(n_vec, 256), 256, 0, st>>>(q + Mp * d, k + Mp * dkv, m->rope_tab, M, S, H, Hkv, hd);
        count_launch(2);
      }
    }
    SZO_TRY(launch_flash_attention_pair_bf16(q, k, v, o, Mp, B, S, H, Hkv, hd, st));
    SZO_TRY(lin(l, 3, o, y));
    SZO_CHECK_CUDA(launch_maybe_chained(add_norm_pair, dim3(static_cast<unsigned>(M)), dim3(256), 0, st, step_chained(), m->h, y, Mp,
                                        L.mlp_norm_g, L.mlp_norm_b, d, c.norm_eps, opt, 1, 0, a, Mp));
    count_launch();
    if (!opt) {
      void* const gu[2] = {gate, up};
      SZO_TRY(lin_group(l, 4, 2, a, gu));
      SZO_CHECK_CUDA(launch_maybe_chained(silu_mul_pair_kernel<T>, dim3(blocks_for(M * ff / Vec16<T>::kN, 256)), dim3(256), 0, st,
                                          step_chained(), gate, up, M * ff, Mp * ff));
      count_launch();
      SZO_TRY(lin(l, 6, gate, y));
    } else {
      SZO_TRY(lin(l, 4, a, gate));
      relu_pair_kernel<T><<<blocks_for(M * ff / Vec16<T>::kN, 256), 256, 0, st>>>(gate, M * ff, Mp * ff);
      count_launch();
      SZO_TRY(lin(l, 5, gate, y));
    }
    pending = y;
  }
  if (c.loss_kind == 0) {
    add_norm_pair<<<static_cast<unsigned>(M), 256, 0, st>>>(m->h, pending, Mp, m->top.final_norm_g,
                                                                     m->top.final_norm_b, d, c.norm_eps, opt, 1, 0, a, Mp);
    count_launch();
    SZO_TRY(szo_linear_fwd(m->lm_head_plan, a, SZO_BF16, Mr, nullptr, m->logits, SZO_F32, SZO_MODE_SPARSE_ADD, m->ws,
                           m->ws_bytes, st));
    ce_rows_pair_kernel<<<static_cast<unsigned>(M), 256, 0, st>>>(m->logits, Mp, tokens, S, c.vocab, m->tok_loss,
                                                                 m->tok_loss + M);
    mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss, M, static_cast<double>(B) * (S - 1), loss_plus_dev);
    mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss + M, M, static_cast<double>(B) * (S - 1), loss_minus_dev);
    count_launch(3);
  } else {
    float* a_last = reinterpret_cast<float*>(m->q);       // B centre states, then B half-differences, fp32
    add_norm_pair_kernel<T, float><<<static_cast<unsigned>(B), 256, 0, st>>>(
        m->h, pending, Mp, m->top.final_norm_g, m->top.final_norm_b, d, c.norm_eps, opt, S, S - 1, a_last, B);
    cls2_pair_kernel<<<static_cast<unsigned>(B), 256, 0, st>>>(a_last, B, static_cast<const __nv_bfloat16*>(m->top.lm_head),
                                                              cand, labels, d, c.vocab, m->tok_loss, m->tok_loss + B);
    mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss, B, static_cast<double>(B), loss_plus_dev);
    mean_f64_kernel<<<1, 1024, 0, st>>>(m->tok_loss + B, B, static_cast<double>(B), loss_minus_dev);
    count_launch(4);
  }
  SZO_CHECK_LAUNCH("model kernels (paired form)");
  return SZO_OK;
}


// T new tokens per sequence after pos0 cached positions (see szo_model_decode_step).
template <typename T>
szo_status run_decode_t(szo_model* m, const int32_t* tokens, int B, int Tn, const float* Sv, float* logits,
                        cudaStream_t st) {
  const int32_t* pos_dev = m->d_pos;                 // cached positions before this call, set by the caller
  const szo_model_config& c = m->cfg;
  const int64_t M = static_cast<int64_t>(B) * Tn;
  const int d = c.d_model, H = c.n_heads, Hkv = c.n_kv_heads, hd = d / H, ff = c.d_ff;
  const int64_t dkv = static_cast<int64_t>(Hkv) * hd, Smax = c.max_seq;
  const int act = c.act_dtype;
  const bool opt = c.arch == 1;
  // few tokens: SZO_MODE_AUTO takes the weight-streaming kernel where it applies (the appendix's
  // SparseAddMM order, the faster one for token generation)
  const int32_t lmode = c.linear_mode == SZO_MODE_FP32_VALIDATE ? SZO_MODE_FP32_VALIDATE : SZO_MODE_AUTO;
  T *a = static_cast<T*>(m->a), *q = static_cast<T*>(m->q), *k = static_cast<T*>(m->k), *v = static_cast<T*>(m->v),
    *o = static_cast<T*>(m->o), *y = static_cast<T*>(m->y), *gate = static_cast<T*>(m->gate), *up = static_cast<T*>(m->up);
  auto lin = [&](int layer, int j, const void* x, void* out) -> szo_status {
    const int t = layer * m->n_lin + j;
    return linear_fwd_impl(m->plans[t], x, act, M, Sv + m->offsets[t], nullptr, out, act, lmode, m->ws, m->ws_bytes, st);
  };
  // n matrices that read the same activations: one launch of the weight-streaming kernel where it
  // takes the group, else one call each
  const bool streaming = lmode == SZO_MODE_AUTO && act == SZO_BF16;
  // The layer kernels of a few-token step are launched as a chain (common.cuh): each may be placed while
  // the one before drains.  SZO_DECODE_CHAIN=0 launches them the ordinary way (A/B measurement).
  static const bool chain_on = [] {
    const char* e = getenv("SZO_DECODE_CHAIN");
    return e == nullptr || e[0] != '0';
  }();
  const bool chained = streaming && chain_on && M <= 16;
  auto lin_group = [&](int layer, int j0, int n, const void* x, void* const* outs) -> szo_status {
    const int t0 = layer * m->n_lin + j0;
    const szo_linear* plans[3];
    const float* sv[3];
    for (int i = 0; i < n; ++i) {
      plans[i] = m->plans[t0 + i];
      sv[i] = Sv + m->offsets[t0 + i];
    }
    if (streaming && few_token_applies(plans, n, M))
      return linear_fwd_skinny_group(plans, n, x, nullptr, M, sv, outs, act, st, chained);
    for (int i = 0; i < n; ++i) SZO_TRY(lin(layer, j0 + i, x, outs[i]));
    return SZO_OK;
  };
  // One or two rows: residual add and norm are formed inside the projection that reads them (the
  // residual stream alternates between m->h and m->h2: a layer reads h, writes h2 in its q/k/v launch,
  // and h again in its gate/up launch).  SZO_DECODE_FUSED_NORM=0 keeps the separate kernel (A/B).
  static const bool fuse_norm_on = [] {
    const char* e = getenv("SZO_DECODE_FUSED_NORM");
    return e == nullptr || e[0] != '0';
  }();
  bool fused_norms = false;                          // decided once: the shapes are those of every layer
  if constexpr (sizeof(T) == 2) {
    const szo_linear* const* p0 = m->plans.data();
    fused_norms = streaming && fuse_norm_on && d <= 8192 && gemv_applies(p0, 3, M) && gemv_applies(p0 + 4, opt ? 1 : 2, M);
  }
  auto norm_lin_group = [&](int layer, int j0, int n, const float* h_in, const T* y_add, float* h_out, const float* gamma,
                            const float* beta, void* const* outs) -> szo_status {
    const int t0 = layer * m->n_lin + j0;
    const szo_linear* plans[3];
    const float* sv[3];
    for (int i = 0; i < n; ++i) {
      plans[i] = m->plans[t0 + i];
      sv[i] = Sv + m->offsets[t0 + i];
    }
    const FusedNorm fn{h_in, reinterpret_cast<const __nv_bfloat16*>(y_add), h_out, gamma, beta, c.norm_eps, opt};
    return linear_fwd_gemv(plans, n, nullptr, nullptr, M, sv, outs, act, st, chained, &fn);
  };
  embed_kernel<<<static_cast<unsigned>(M), 128, 0, st>>>(tokens, static_cast<const __nv_bfloat16*>(m->top.embed),
                                                        static_cast<const __nv_bfloat16*>(m->top.pos), Tn, d, c.vocab, m->h, 0, pos_dev);
  count_launch();
  const T* pending = nullptr;
  const int64_t layer_cache = static_cast<int64_t>(c.max_batch) * Smax * dkv;
  for (int l = 0; l < c.n_layers; ++l) {
    const szo_layer_weights& L = m->layers[l];
    {
      void* const qkv[3] = {q, k, v};
      if (fused_norms) {
        SZO_TRY(norm_lin_group(l, 0, 3, m->h, pending, m->h2, L.attn_norm_g, L.attn_norm_b, qkv));
      } else {
        SZO_CHECK_CUDA(launch_maybe_chained(add_norm_kernel<T, T>, dim3(static_cast<unsigned>(M)), dim3(256), 0, st, chained, m->h,
                                            pending, L.attn_norm_g, L.attn_norm_b, d, c.norm_eps, opt, int64_t(1), int64_t(0), a));
        count_launch();
        SZO_TRY(lin_group(l, 0, 3, a, qkv));
      }
    }
    T* kc = static_cast<T*>(m->kcache) + l * layer_cache;
    T* vc = static_cast<T*>(m->vcache) + l * layer_cache;
    dim3 grid(static_cast<unsigned>(Tn), H, B);
    const float scale = 1.0f / sqrtf(static_cast<float>(hd));
    if (Tn <= 16) {
      // rotation, cache append and attention in one launch
      const float2* tab = opt ? nullptr : m->rope_tab;
      auto attn = hd == 64 ? attn_decode_fused_kernel<T, 64> : attn_decode_fused_kernel<T, 128>;
      SZO_CHECK_CUDA(launch_maybe_chained(attn, grid, dim3(128), 0, st, chained, q, k, v, kc, vc, o, tab, Tn, pos_dev, Smax, H, Hkv,
                                          scale));
      count_launch();
    } else {
      if (!opt) {
        const int64_t n_rot = M * (H + Hkv) * ((hd / 2) / Vec16<T>::kN);
        rope_kernel<T><<<blocks_for(n_rot, 256), 256, 0, st>>>(q, k, m->rope_tab, M, Tn, H, Hkv, hd, 0, pos_dev);
        count_launch();
      }
      const int64_t n_vec = M * dkv / Vec16<T>::kN;
      kv_append_kernel<T><<<blocks_for(2 * n_vec, 256), 256, 0, st>>>(k, v, kc, vc, Tn, pos_dev, Smax, dkv, n_vec);
      if (hd == 64) attn_decode_kernel<T, 64><<<grid, 128, 0, st>>>(q, kc, vc, o, Tn, pos_dev, Smax, H, Hkv, scale);
      else attn_decode_kernel<T, 128><<<grid, 128, 0, st>>>(q, kc, vc, o, Tn, pos_dev, Smax, H, Hkv, scale);
      count_launch(2);
    }
    {
      void* const out[1] = {y};
      SZO_TRY(lin_group(l, 3, 1, o, out));
    }
    {
      void* const gu[2] = {gate, up};
      if (fused_norms) {
        SZO_TRY(norm_lin_group(l, 4, opt ? 1 : 2, m->h2, y, m->h, L.mlp_norm_g, L.mlp_norm_b, gu));
      } else {
        SZO_CHECK_CUDA(launch_maybe_chained(add_norm_kernel<T, T>, dim3(static_cast<unsigned>(M)), dim3(256), 0, st, chained, m->h,
                                            static_cast<const T*>(y), L.mlp_norm_g, L.mlp_norm_b, d, c.norm_eps, opt, int64_t(1),
                                            int64_t(0), a));
        count_launch();
        if (opt) SZO_TRY(lin(l, 4, a, gate));
        else SZO_TRY(lin_group(l, 4, 2, a, gu));
      }
    }
    if (!opt) {
      const szo_linear* down = m->plans[l * m->n_lin + 6];
      if (streaming && few_token_applies(&down, 1, M)) {
        // silu(gate) * up is formed while the down projection stages its activations
        const float* sv = Sv + m->offsets[l * m->n_lin + 6];
        void* const out[1] = {y};
        SZO_TRY(linear_fwd_skinny_group(&down, 1, gate, up, M, &sv, out, act, st, chained));
      } else {
        silu_mul_kernel<T><<<blocks_for(M * ff / Vec16<T>::kN, 256), 256, 0, st>>>(gate, up, M * ff, gate);
        count_launch();
        SZO_TRY(lin(l, 6, gate, y));
      }
    } else {
      relu_kernel<T><<<blocks_for(M * ff / Vec16<T>::kN, 256), 256, 0, st>>>(gate, M * ff);
      count_launch();
      SZO_TRY(lin(l, 5, gate, y));
    }
    pending = y;
  }
  // the last new token of every sequence: final norm, LM head
  add_norm_kernel<T><<<static_cast<unsigned>(B), 256, 0, st>>>(m->h, pending, m->top.final_norm_g, m->top.final_norm_b, d,
                                                              c.norm_eps, opt, Tn, Tn - 1, a);
  count_launch();
  szo_linear_t* head = m->lm_head_plan != nullptr ? m->lm_head_plan : m->decode_head;
  const int hmode = lmode == SZO_MODE_FP32_VALIDATE ? SZO_MODE_FP32_VALIDATE : SZO_MODE_SPARSE_ADD;
  SZO_TRY(szo_linear_fwd(head, a, static_cast<szo_dtype>(act), B, nullptr, logits, SZO_F32, hmode, m->ws, m->ws_bytes, st));
  SZO_CHECK_LAUNCH("decode kernels");
  return SZO_OK;
}

szo_status run_loss(szo_model* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand, int B, int S,
                    const float* Sv, double* loss_dev, cudaStream_t st) {
  if (m->cfg.act_dtype == SZO_F32) return run_loss_t<float>(m, tokens, labels, cand, B, S, Sv, loss_dev, st);
  return run_loss_t<__nv_bfloat16>(m, tokens, labels, cand, B, S, Sv, loss_dev, st);
}

// Both perturbed forwards of a step side by side (see run_loss_t); bf16 tensor-core path with the
// materialised form only: the caller checks dual_forward_applies().
bool dual_forward_applies(const szo_model* m, int64_t M) {
  return m->dual_rows && !m->paired && m->cfg.act_dtype != SZO_F32 && m->cfg.linear_mode != SZO_MODE_FP32_VALIDATE &&
         m->cfg.linear_mode != SZO_MODE_SPMM && !m->plans.empty() && m->k_total > 0 &&
         (m->resident || tc_use_materialised(m->plans[0], M, true));
}

szo_status check_batch(const szo_model* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand, int B,
                       int S) {
  SZO_REQUIRE(m != nullptr, SZO_ERR_INVALID_ARG, "model is NULL");
  SZO_REQUIRE(tokens != nullptr, SZO_ERR_INVALID_ARG, "tokens is NULL");
  SZO_REQUIRE(B >= 1 && B <= m->cfg.max_batch && S >= 2 && S <= m->cfg.max_seq, SZO_ERR_SHAPE,
              "need 1 <= B <= %d and 2 <= S <= %d (got B=%d, S=%d)", m->cfg.max_batch, m->cfg.max_seq, B, S);
  SZO_REQUIRE(m->cfg.loss_kind == 0 || (labels && cand), SZO_ERR_INVALID_ARG,
              "labels and cand are required for the 2-candidate loss");
  SZO_REQUIRE(m->cfg.arch == 0 || S <= m->cfg.max_pos, SZO_ERR_SHAPE, "S exceeds the position table");
  return SZO_OK;
}

}  // namespace

extern "C" {

szo_status szo_model_create(szo_model_t** out, const szo_model_config* cfg, const szo_model_weights* top,
                            const szo_layer_weights* layers_host, float* S_all, void* stream) {
  SZO_REQUIRE(out && cfg && top && layers_host, SZO_ERR_INVALID_ARG, "NULL argument");
  *out = nullptr;
  const szo_model_config& c = *cfg;
  SZO_REQUIRE(c.arch == 0 || c.arch == 1, SZO_ERR_INVALID_ARG, "arch must be 0 or 1");
  SZO_REQUIRE(c.n_layers > 0 && c.d_model > 0 && c.n_heads > 0 && c.n_kv_heads > 0 && c.d_ff > 0 && c.vocab > 1,
              SZO_ERR_SHAPE, "non-positive model dimension");
  SZO_REQUIRE(c.d_model % c.n_heads == 0 && c.n_heads % c.n_kv_heads == 0, SZO_ERR_SHAPE,
              "d_model %% n_heads and n_heads %% n_kv_heads must be 0");
  const int hd = c.d_model / c.n_heads;
  SZO_REQUIRE(hd == 64 || hd == 128, SZO_ERR_UNSUPPORTED, "head dimension must be 64 or 128 (got %d)", hd);
  SZO_REQUIRE(c.d_model % 8 == 0 && c.d_ff % 8 == 0, SZO_ERR_SHAPE, "d_model and d_ff must be multiples of 8");
  SZO_REQUIRE(c.d_model <= 8192, SZO_ERR_UNSUPPORTED, "d_model above 8192 is not supported by the norm kernel");
  SZO_REQUIRE(c.act_dtype == SZO_BF16 || c.act_dtype == SZO_F32, SZO_ERR_UNSUPPORTED, "act_dtype must be bf16 or f32");
  SZO_REQUIRE(c.act_dtype == SZO_BF16 || c.linear_mode == SZO_MODE_FP32_VALIDATE, SZO_ERR_UNSUPPORTED,
              "fp32 activations need the fp32 validation mode");
  SZO_REQUIRE(c.linear_mode >= SZO_MODE_AUTO && c.linear_mode <= SZO_MODE_PAIRED, SZO_ERR_INVALID_ARG,
              "unknown linear_mode %d", c.linear_mode);
  SZO_REQUIRE(c.loss_kind == 0 || c.loss_kind == 1, SZO_ERR_INVALID_ARG, "loss_kind must be 0 or 1");
  SZO_REQUIRE(c.max_batch > 0 && c.max_seq > 1, SZO_ERR_SHAPE, "max_batch/max_seq");
  SZO_REQUIRE(c.arch == 0 || (top->pos && c.max_pos >= c.max_seq), SZO_ERR_INVALID_ARG, "position table missing/short");
  SZO_REQUIRE(top->embed && top->lm_head && top->final_norm_g, SZO_ERR_INVALID_ARG, "missing top-level weights");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  szo_model* m = new szo_model();
  m->cfg = c;
  m->top = *top;
  m->n_lin = c.arch == 0 ? 7 : 6;
  m->layers.assign(layers_host, layers_host + c.n_layers);
  m->S_all = S_all;
  m->Mmax = static_cast<int64_t>(c.max_batch) * c.max_seq;
  m->paired = c.linear_mode == SZO_MODE_PAIRED;
  const int32_t lmode = m->paired ? SZO_MODE_SPARSE_ADD : c.linear_mode;   // mode of a lone forward
  auto bail = [&](szo_status s) {
    szo_model_destroy(m);
    return s;
  };
#define SZO_M_TRY(expr)                    \
  do {                                     \
    szo_status s__ = (expr);               \
    if (s__ != SZO_OK) return bail(s__);   \
  } while (0)
  // plans and offsets
  size_t ws_need = 0;
  m->offsets.push_back(0);
  for (int l = 0; l < c.n_layers; ++l) {
    for (int j = 0; j < m->n_lin; ++j) {
      int64_t N, K;
      linear_shape(c, j, &N, &K);
      const szo_linear_weights& w = m->layers[l].lin[j];
      szo_linear_t* p = nullptr;
      if (c.group == -1)   // non-uniform 4-bit format: `scales` is the per-row table [N,16]
        SZO_M_TRY(szo_linear_create_lut(&p, N, K, static_cast<const uint8_t*>(w.codes), w.scales,
                                        static_cast<szo_dtype>(c.sz_dtype), w.idx, w.nnz, w.bias, st));
      else
        SZO_M_TRY(szo_linear_create(&p, N, K, c.group, w.codes, w.scales, w.zeros, static_cast<szo_dtype>(c.sz_dtype),
                                    w.idx, w.nnz, w.bias, st));
      m->plans.push_back(p);
      m->offsets.push_back(m->offsets.back() + w.nnz);
      const size_t need = szo_linear_workspace_bytes(p, m->Mmax, lmode);
      if (need > ws_need) ws_need = need;
    }
  }
  if (!m->plans.empty() && c.linear_mode != SZO_MODE_FP32_VALIDATE) {
    // K-split scratch of the pair-tile kernel: at most one 256 x 256 fp32 tile per cluster
    const size_t need = tc_tail_ws_bound();
    if (need > ws_need) ws_need = need;
    // scratch of the materialised form: the largest group of layers that share their input
    if (tc_use_materialised(m->plans[0], m->Mmax, true) || (m->paired && c.group != 0)) {
      for (int l = 0; l < c.n_layers; ++l) {
        const szo_linear* const* pl = m->plans.data() + static_cast<size_t>(l) * m->n_lin;
        const bool px = m->paired;
        const size_t g0 = tc_materialised_ws_bytes(pl, 3, m->Mmax, px && tc_paired_dense_cross(pl, 3));   // q, k, v
        const size_t g1 = c.arch == 0 ? tc_materialised_ws_bytes(pl + 4, 2, m->Mmax, px && tc_paired_dense_cross(pl + 4, 2)) : 0;  // gate, up
        size_t g2 = 0;
        for (int j = 0; j < m->n_lin; ++j) {
          const size_t one = tc_materialised_ws_bytes(pl + j, 1, m->Mmax, px && tc_paired_dense_cross(pl + j, 1));
          if (one > g2) g2 = one;
        }
        const size_t mx = g0 > g1 ? (g0 > g2 ? g0 : g2) : (g1 > g2 ? g1 : g2);
        if (mx > ws_need) ws_need = mx;
      }
    }
  }
  m->k_total = m->offsets.back();
  if (m->k_total > 0 && S_all == nullptr) return bail(fail(SZO_ERR_INVALID_ARG, "S_all is NULL"));
  // resident effective weights of the launch groups (dense bf16 weights, many tokens)
  // (SZO_MODEL_RESIDENT=0 at creation keeps the fused form, for A/B and for tests that compare the two)
  const char* res_env = getenv("SZO_MODEL_RESIDENT");
  m->resident = !(res_env != nullptr && res_env[0] == '0') && c.group == 0 && c.act_dtype == SZO_BF16 &&
                c.linear_mode != SZO_MODE_FP32_VALIDATE && c.linear_mode != SZO_MODE_SPMM && !m->plans.empty() &&
                tc_use_resident(m->plans[0], m->Mmax);
  if (m->resident) {
    m->res_W.assign(m->plans.size(), nullptr);
    m->res_saved.assign(m->plans.size(), nullptr);
    const int n_groups = 4;
    const int g_first[4] = {0, 3, 4, c.arch == 0 ? 6 : 5};
    const int g_count[4] = {3, 1, c.arch == 0 ? 2 : 1, 1};
    for (int l = 0; l < c.n_layers; ++l) {
      for (int g = 0; g < n_groups; ++g) {
        const size_t t0 = static_cast<size_t>(l) * m->n_lin + g_first[g];
        const szo_linear* const* pl = m->plans.data() + t0;
        if (!tc_can_stack(pl, g_count[g])) return bail(fail(SZO_ERR_UNSUPPORTED, "resident form: group cannot be stacked"));
        size_t wb = 0, sb = 0;
        const bool ext = m->paired && tc_paired_dense_cross(pl, g_count[g]);
        tc_resident_bytes(pl, g_count[g], &wb, &sb, ext);
        SZO_M_TRY(dev_alloc(m, &m->res_W[t0], wb));
        SZO_M_TRY(dev_alloc(m, &m->res_saved[t0], sb));
        SZO_M_TRY(tc_resident_init(pl, g_count[g], m->res_W[t0], m->res_saved[t0], st, ext));
      }
    }
  }
  if (c.loss_kind == 0) {
    SZO_M_TRY(szo_linear_create(&m->lm_head_plan, c.vocab, c.d_model, 0, top->lm_head, nullptr, nullptr, SZO_BF16,
                                nullptr, 0, nullptr, st));
    const size_t need = szo_linear_workspace_bytes(m->lm_head_plan, 2 * m->Mmax + 256, lmode);
    if (need > ws_need) ws_need = need;
  }
  // buffers
  const size_t e = c.act_dtype == SZO_F32 ? 4 : 2;
  // When the step can run its two forwards side by side (bf16 tensor-core path in the materialised
  // form; SZO_DUAL_FORWARD=0 at creation switches it off for A/B), every activation buffer holds
  // two sets of Mmax rows.
  {
    const char* env = getenv("SZO_DUAL_FORWARD");
    m->dual_rows = !(env != nullptr && env[0] == '0') && !m->paired && c.act_dtype != SZO_F32 &&
                   c.linear_mode != SZO_MODE_FP32_VALIDATE && c.linear_mode != SZO_MODE_SPMM && !m->plans.empty() &&
                   m->k_total > 0 && (m->resident || tc_use_materialised(m->plans[0], m->Mmax, true));
  }
  // paired form: centre rows, then the half-difference rows from a multiple of 256 on
  const int64_t Mpmax = static_cast<int64_t>(round_up(static_cast<size_t>(m->Mmax), 256));
  const int64_t Mx = m->paired ? Mpmax + m->Mmax : m->Mmax * (m->dual_rows ? 2 : 1), d = c.d_model,
                dkv = static_cast<int64_t>(c.n_kv_heads) * hd, ff = c.d_ff;
  if (m->dual_rows) {
    SZO_M_TRY(dev_alloc(m, &m->Splus, m->k_total * sizeof(float)));
    SZO_M_TRY(dev_alloc(m, &m->Sminus, m->k_total * sizeof(float)));
  }
  SZO_M_TRY(dev_alloc(m, &m->gidx, m->k_total * sizeof(int64_t)));
  SZO_M_TRY(dev_alloc(m, &m->h, Mx * d * sizeof(float)));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->a), Mx * d * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->q), Mx * d * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->k), Mx * dkv * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->v), Mx * dkv * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->o), Mx * d * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->y), Mx * d * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->gate), Mx * ff * e));
  SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->up), Mx * ff * e));
  if (c.loss_kind == 0) SZO_M_TRY(dev_alloc(m, &m->logits, Mx * c.vocab * sizeof(float)));
  SZO_M_TRY(dev_alloc(m, &m->tok_loss, Mx * sizeof(double)));
  SZO_M_TRY(dev_alloc(m, &m->rope_tab, static_cast<size_t>(c.max_seq) * (hd / 2) * sizeof(float2)));
  if (ws_need) SZO_M_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->ws), ws_need));
  m->ws_bytes = ws_need;
  SZO_M_TRY(dev_alloc(m, &m->d_tokens, m->Mmax * sizeof(int32_t)));
  SZO_M_TRY(dev_alloc(m, &m->d_labels, c.max_batch * sizeof(int32_t)));
  SZO_M_TRY(dev_alloc(m, &m->d_cand, 16));
  SZO_M_TRY(dev_alloc(m, &m->d_scalars, 4 * sizeof(double)));
  // global indices and the rotary table
  int64_t base = 0;
  for (int l = 0, t = 0; l < c.n_layers; ++l) {
    for (int j = 0; j < m->n_lin; ++j, ++t) {
      int64_t N, K;
      linear_shape(c, j, &N, &K);
      const szo_linear_weights& w = m->layers[l].lin[j];
      if (w.nnz)
        gidx_kernel<<<blocks_for(w.nnz, 256), 256, 0, st>>>(w.idx, w.nnz, base, m->gidx + m->offsets[t]);
      base += N * K;
    }
  }
  // model-wide bucket order: linear t's records occupy [offsets[t], offsets[t+1]) and refer to S_all
  SZO_M_TRY(dev_alloc(m, &m->geid, m->k_total * sizeof(int32_t)));
  SZO_M_TRY(dev_alloc(m, &m->gpos, m->k_total * sizeof(uint16_t)));
  SZO_M_TRY(dev_alloc(m, &m->recs, m->k_total * sizeof(uint2)));
  SZO_M_TRY(dev_alloc(m, &m->zkept, m->k_total * sizeof(float)));
  SZO_M_TRY(dev_alloc(m, &m->colk, m->k_total * sizeof(uint32_t)));
  SZO_M_TRY(dev_alloc(m, &m->csrc, m->k_total * sizeof(int32_t)));
  SZO_M_TRY(dev_alloc(m, &m->crecs, m->k_total * sizeof(uint32_t)));
  if (m->k_total >= (int64_t(1) << 31)) return bail(fail(SZO_ERR_SHAPE, "more than 2^31 sparse entries"));
  for (size_t t = 0; t < m->plans.size(); ++t) {
    const szo_linear* p = m->plans[t];
    if (p->nnz) {
      const szo_status cs = cross_copy_slots(p, static_cast<int32_t>(m->offsets[t]), m->colk + m->offsets[t],
                                             m->csrc + m->offsets[t], st);
      if (cs != SZO_OK) return bail(cs);
      offset_eid_kernel<<<blocks_for(p->nnz, 256), 256, 0, st>>>(p->bucket_eid, p->nnz, static_cast<int32_t>(m->offsets[t]),
                                                               m->geid + m->offsets[t]);
      cudaMemcpyAsync(m->gpos + m->offsets[t], p->bucket_pos, p->nnz * sizeof(uint16_t), cudaMemcpyDeviceToDevice, st);
    }
  }
  rope_table_kernel<<<blocks_for(static_cast<int64_t>(c.max_seq) * (hd / 2), 256), 256, 0, st>>>(
      c.max_seq, hd / 2, static_cast<double>(c.rope_base), m->rope_tab);
  if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return bail(fail(SZO_ERR_CUDA, "model set-up kernels failed"));
#undef SZO_M_TRY
  *out = m;
  return SZO_OK;
}

szo_status szo_attention(const void* q, const void* k, const void* v, void* o, szo_dtype dtype, int32_t B, int32_t S,
                         int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream) {
  SZO_REQUIRE(q && k && v && o, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(B > 0 && S > 0 && n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0, SZO_ERR_SHAPE, "bad shape");
  SZO_REQUIRE(head_dim == 64 || head_dim == 128, SZO_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  SZO_REQUIRE(dtype == SZO_BF16 || dtype == SZO_F32, SZO_ERR_UNSUPPORTED, "dtype must be bf16 or f32");
  SZO_REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(o), SZO_ERR_ALIGNMENT, "buffers must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (dtype == SZO_BF16) return launch_flash_attention_bf16(q, k, v, o, B, S, n_heads, n_kv_heads, head_dim, st);
  dim3 grid(static_cast<unsigned>(ceil_div(S, 4)), n_heads, B);
  const float scale = 1.0f / sqrtf(static_cast<float>(head_dim));
  auto *qf = static_cast<const float*>(q), *kf = static_cast<const float*>(k), *vf = static_cast<const float*>(v);
  if (head_dim == 64) attn_warp_kernel<float, 64><<<grid, 128, 0, st>>>(qf, kf, vf, static_cast<float*>(o), S, n_heads, n_kv_heads, scale);
  else attn_warp_kernel<float, 128><<<grid, 128, 0, st>>>(qf, kf, vf, static_cast<float*>(o), S, n_heads, n_kv_heads, scale);
  count_launch();
  SZO_CHECK_LAUNCH("attn_warp_kernel");
  return SZO_OK;
}

szo_status szo_attention_paired(const void* q, const void* k, const void* v, void* o, int64_t row0, int32_t B,
                                int32_t S, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream) {
  SZO_REQUIRE(q && k && v && o, SZO_ERR_INVALID_ARG, "NULL pointer");
  SZO_REQUIRE(B > 0 && S > 0 && n_heads > 0 && n_kv_heads > 0 && n_heads % n_kv_heads == 0, SZO_ERR_SHAPE, "bad shape");
  SZO_REQUIRE(row0 >= static_cast<int64_t>(B) * S, SZO_ERR_SHAPE, "row0 must leave room for the B*S centre rows");
  SZO_REQUIRE(head_dim == 64 || head_dim == 128, SZO_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
  SZO_REQUIRE(aligned16(q) && aligned16(k) && aligned16(v) && aligned16(o), SZO_ERR_ALIGNMENT, "buffers must be 16-byte aligned");
  return launch_flash_attention_pair_bf16(q, k, v, o, row0, B, S, n_heads, n_kv_heads, head_dim,
                                          static_cast<cudaStream_t>(stream));
}

int64_t szo_model_k_total(const szo_model_t* m) { return m ? m->k_total : 0; }
const int64_t* szo_model_gidx(const szo_model_t* m) { return m ? m->gidx : nullptr; }
int64_t szo_model_last_launches(const szo_model_t* m) { return m ? m->last_launches : 0; }

szo_status szo_model_loss(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                          int32_t B, int32_t S, const float* S_vals, double* loss_dev, void* stream) {
  SZO_TRY(check_batch(m, tokens, labels, cand, B, S));
  SZO_REQUIRE(loss_dev != nullptr, SZO_ERR_INVALID_ARG, "loss_dev is NULL");
  return run_loss(m, tokens, labels, cand, B, S, S_vals ? S_vals : m->S_all, loss_dev, static_cast<cudaStream_t>(stream));
}

// First half of a step: z is drawn (and kept), both perturbed losses are evaluated, S is back where the
// in-place +eps, -2 eps, +eps sequence leaves it.
static szo_status zo_losses_impl(szo_model* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                                 int32_t B, int32_t S, uint64_t seed, uint64_t step, float eps, double* f_plus_dev,
                                 double* f_minus_dev, cudaStream_t st) {
  const int64_t k = m->k_total;
  float* Sv = m->S_all;
  ScaleArg sa{eps, 0.f, 0.f, nullptr, nullptr};
  if (m->paired) {
    // S goes through the seed trick's +eps, -2 eps, +eps sequence (so that it ends where the
    // in-place order leaves it) while z is kept; the two forwards then run in the paired form on the
    // restored S, with +-eps z applied inside the linears in fp32
    // (one launch: the pass is bound by drawing z, the other two are its fused multiply-adds)
    SZO_TRY(launch_sparse_axpy_three(Sv, Sv, m->gidx, k, 0, seed, step, eps, st, m->zkept, nullptr, nullptr));
    return run_loss_paired(m, tokens, labels, cand, B, S, Sv, m->zkept, eps, f_plus_dev, f_minus_dev, st);
  }
  if (dual_forward_applies(m, static_cast<int64_t>(B) * S)) {
    // both forwards side by side: the same arithmetic on S as the in-place sequence below
    // (+eps, -2 eps, +eps), written to two copies, so that every linear makes one weight pass
    // S+ = S + eps z, S- = S+ - 2 eps z, S = S- + eps z in one launch
    SZO_TRY(launch_sparse_axpy_three(Sv, Sv, m->gidx, k, 0, seed, step, eps, st, m->zkept, m->Splus, m->Sminus));
    return run_loss_t<__nv_bfloat16>(m, tokens, labels, cand, B, S, m->Splus, f_plus_dev, st, m->Sminus, f_minus_dev);
  }
  // z is generated once per step (first pass) and kept: the other passes stream it
  SZO_TRY(launch_sparse_axpy(Sv, Sv, m->gidx, k, 0, seed, step, sa, st, m->zkept));       // S += eps z
  SZO_TRY(run_loss(m, tokens, labels, cand, B, S, Sv, f_plus_dev, st));                   // f+
  sa.scale = -2.0f * eps;
  SZO_TRY(launch_sparse_axpy_kept(Sv, Sv, m->zkept, k, sa, st));                          // S -= 2 eps z
  SZO_TRY(run_loss(m, tokens, labels, cand, B, S, Sv, f_minus_dev, st));                  // f-
  sa.scale = eps;
  return launch_sparse_axpy_kept(Sv, Sv, m->zkept, k, sa, st);                            // S += eps z
}

// Second half: g from the two losses, then S -= lr g z with the kept z.
// Sparse values kept in 16 bits (Section 3.5): one rounding to the storage format after a step's update
static szo_status store_sparse(szo_model* m, cudaStream_t st) {
  if (m->sparse_dt == SZO_F32) return SZO_OK;
  return szo_round_sparse16(m->S_all, m->k_total, static_cast<szo_dtype>(m->sparse_dt), m->S16_out, st);
}

static szo_status zo_apply_impl(szo_model* m, float eps, float lr, const double* f_plus_dev, const double* f_minus_dev,
                                double* g_dev, cudaStream_t st) {
  SZO_TRY(szo_projected_gradient(f_plus_dev, f_minus_dev, eps, g_dev, st));
  ScaleArg su{0.f, lr, eps, f_plus_dev, f_minus_dev};
  SZO_TRY(launch_sparse_axpy_kept(m->S_all, m->S_all, m->zkept, m->k_total, su, st));
  return store_sparse(m, st);
}

szo_status szo_model_zo_step(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                             int32_t B, int32_t S, uint64_t seed, uint64_t step, float eps, float lr,
                             double* f_plus_dev, double* f_minus_dev, double* g_dev, void* stream) {
  SZO_TRY(check_batch(m, tokens, labels, cand, B, S));
  SZO_REQUIRE(f_plus_dev && f_minus_dev && g_dev, SZO_ERR_INVALID_ARG, "NULL output scalar");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t before = g_launch_count;
  SZO_TRY(zo_losses_impl(m, tokens, labels, cand, B, S, seed, step, eps, f_plus_dev, f_minus_dev, st));
  SZO_TRY(zo_apply_impl(m, eps, lr, f_plus_dev, f_minus_dev, g_dev, st));
  m->z_valid = false;
  m->last_launches = g_launch_count - before;
  return SZO_OK;
}

szo_status szo_model_zo_step_n(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                               int32_t B, int32_t S, uint64_t seed, uint64_t step, int32_t n, float eps, float lr,
                               double* f_plus_dev, double* f_minus_dev, double* g_dev, void* stream) {
  SZO_TRY(check_batch(m, tokens, labels, cand, B, S));
  SZO_REQUIRE(f_plus_dev && f_minus_dev && g_dev, SZO_ERR_INVALID_ARG, "NULL output array");
  SZO_REQUIRE(eps != 0.f && n >= 1 && n <= 1024, SZO_ERR_INVALID_ARG, "need eps != 0 and 1 <= n <= 1024");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t before = g_launch_count;
  // every sample's losses around the same S (each call returns S to where the +eps, -2 eps, +eps order leaves it)
  for (int32_t i = 0; i < n; ++i) {
    const uint64_t c = step * static_cast<uint64_t>(n) + static_cast<uint64_t>(i);
    SZO_TRY(zo_losses_impl(m, tokens, labels, cand, B, S, seed, c, eps, f_plus_dev + i, f_minus_dev + i, st));
    SZO_TRY(szo_projected_gradient(f_plus_dev + i, f_minus_dev + i, eps, g_dev + i, st));
  }
  // S -= (lr / n) g_i z_i, i in turn; z_i is regenerated (only the last sample's z is still kept)
  const float lr_n = static_cast<float>(static_cast<double>(lr) / n);
  for (int32_t i = 0; i < n; ++i) {
    const uint64_t c = step * static_cast<uint64_t>(n) + static_cast<uint64_t>(i);
    ScaleArg su{0.f, lr_n, eps, f_plus_dev + i, f_minus_dev + i};
    SZO_TRY(launch_sparse_axpy(m->S_all, m->S_all, m->gidx, m->k_total, 0, seed, c, su, st));
  }
  SZO_TRY(store_sparse(m, st));
  m->z_valid = false;
  m->last_launches = g_launch_count - before;
  return SZO_OK;
}

szo_status szo_model_set_sparse_storage(szo_model_t* m, szo_dtype dt, void* S16_out, void* stream) {
  SZO_REQUIRE(m != nullptr, SZO_ERR_INVALID_ARG, "model is NULL");
  SZO_REQUIRE(dt == SZO_F32 || dt == SZO_BF16 || dt == SZO_F16, SZO_ERR_INVALID_ARG, "unknown storage format");
  m->sparse_dt = dt;
  m->S16_out = dt == SZO_F32 ? nullptr : S16_out;
  return store_sparse(m, static_cast<cudaStream_t>(stream));
}

szo_status szo_model_zo_losses(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                               int32_t B, int32_t S, uint64_t seed, uint64_t step, float eps, double* sums_dev,
                               void* stream) {
  SZO_TRY(check_batch(m, tokens, labels, cand, B, S));
  SZO_REQUIRE(sums_dev != nullptr, SZO_ERR_INVALID_ARG, "sums_dev is NULL");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int64_t before = g_launch_count;
  SZO_TRY(zo_losses_impl(m, tokens, labels, cand, B, S, seed, step, eps, m->d_scalars, m->d_scalars + 1, st));
  const double count = m->cfg.loss_kind == 0 ? static_cast<double>(B) * (S - 1) : static_cast<double>(B);
  loss_sums_kernel<<<1, 1, 0, st>>>(m->d_scalars, m->d_scalars + 1, count, sums_dev);
  count_launch();
  SZO_CHECK_LAUNCH("loss_sums_kernel");
  m->z_valid = true;
  m->last_launches = g_launch_count - before;
  return SZO_OK;
}

szo_status szo_model_zo_apply(szo_model_t* m, float eps, float lr, const double* sums_dev, double* f_plus_dev,
                              double* f_minus_dev, double* g_dev, void* stream) {
  SZO_REQUIRE(m != nullptr, SZO_ERR_INVALID_ARG, "model is NULL");
  SZO_REQUIRE(sums_dev && f_plus_dev && f_minus_dev && g_dev, SZO_ERR_INVALID_ARG, "NULL scalar pointer");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  SZO_REQUIRE(m->z_valid, SZO_ERR_INVALID_ARG, "szo_model_zo_apply needs the z kept by a preceding szo_model_zo_losses");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  loss_means_kernel<<<1, 1, 0, st>>>(sums_dev, f_plus_dev, f_minus_dev);
  count_launch();
  SZO_CHECK_LAUNCH("loss_means_kernel");
  SZO_TRY(zo_apply_impl(m, eps, lr, f_plus_dev, f_minus_dev, g_dev, st));
  m->z_valid = false;
  return SZO_OK;
}

szo_status szo_model_zo_step_host(szo_model_t* m, const int32_t* tokens_host, const int32_t* labels_host,
                                  const int32_t* cand_host, int32_t B, int32_t S, uint64_t seed, uint64_t step,
                                  float eps, float lr, double* out3_host, void* stream) {
  SZO_TRY(check_batch(m, tokens_host, labels_host, cand_host, B, S));
  SZO_REQUIRE(out3_host != nullptr, SZO_ERR_INVALID_ARG, "out3_host is NULL");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  SZO_CHECK_CUDA(cudaMemcpyAsync(m->d_tokens, tokens_host, static_cast<size_t>(B) * S * sizeof(int32_t),
                                 cudaMemcpyHostToDevice, st));
  if (m->cfg.loss_kind == 1) {
    SZO_CHECK_CUDA(cudaMemcpyAsync(m->d_labels, labels_host, B * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SZO_CHECK_CUDA(cudaMemcpyAsync(m->d_cand, cand_host, 2 * sizeof(int32_t), cudaMemcpyHostToDevice, st));
  }
  SZO_TRY(szo_model_zo_step(m, m->d_tokens, m->d_labels, m->d_cand, B, S, seed, step, eps, lr, m->d_scalars,
                            m->d_scalars + 1, m->d_scalars + 2, stream));
  SZO_CHECK_CUDA(cudaMemcpyAsync(out3_host, m->d_scalars, 3 * sizeof(double), cudaMemcpyDeviceToHost, st));
  SZO_CHECK_CUDA(cudaStreamSynchronize(st));
  return SZO_OK;
}

szo_status szo_model_enable_decode(szo_model_t* m, void* stream) {
  SZO_REQUIRE(m != nullptr, SZO_ERR_INVALID_ARG, "model is NULL");
  if (m->kcache != nullptr) return SZO_OK;
  const szo_model_config& c = m->cfg;
  const size_t e = c.act_dtype == SZO_F32 ? 4 : 2;
  const size_t bytes = static_cast<size_t>(c.n_layers) * c.max_batch * c.max_seq * c.n_kv_heads * (c.d_model / c.n_heads) * e;
  SZO_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->kcache), bytes));
  SZO_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->vcache), bytes));
  SZO_TRY(dev_alloc(m, &m->d_pos, sizeof(int32_t)));
  SZO_TRY(dev_alloc(m, &m->h2, 2 * static_cast<size_t>(c.d_model) * sizeof(float)));
  SZO_TRY(dev_alloc(m, &m->dec_tokens, static_cast<size_t>(m->Mmax) * sizeof(int32_t)));
  SZO_TRY(dev_alloc(m, &m->dec_logits, static_cast<size_t>(c.max_batch) * c.vocab * sizeof(float)));
  SZO_REQUIRE(device_status_word() != nullptr, SZO_ERR_CUDA, "no device status word");    // allocated outside any capture
  {
    const char* env = getenv("SZO_DECODE_GRAPH");
    m->dec_use_graph = !(env != nullptr && env[0] == '0');
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (m->lm_head_plan == nullptr) {
    SZO_TRY(szo_linear_create(&m->decode_head, c.vocab, c.d_model, 0, m->top.lm_head, nullptr, nullptr, SZO_BF16, nullptr,
                              0, nullptr, st));
    const int32_t hmode = c.linear_mode == SZO_MODE_FP32_VALIDATE ? SZO_MODE_FP32_VALIDATE : SZO_MODE_SPARSE_ADD;
    const size_t need = szo_linear_workspace_bytes(m->decode_head, c.max_batch, hmode);
    if (need > m->ws_bytes) {
      SZO_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->ws), need));      // the earlier workspace stays owned and is freed with the model
      m->ws_bytes = need;
    }
  }
  // the few-token linears of the decode path (SZO_MODE_AUTO) may want more workspace than the loss path's mode
  if (c.linear_mode != SZO_MODE_FP32_VALIDATE) {
    size_t need = m->ws_bytes;
    for (szo_linear_t* p : m->plans) {
      const size_t w = szo_linear_workspace_bytes(p, m->Mmax, SZO_MODE_AUTO);
      if (w > need) need = w;
    }
    if (need > m->ws_bytes) {
      SZO_TRY(dev_alloc(m, reinterpret_cast<char**>(&m->ws), need));
      m->ws_bytes = need;
    }
  }
  return SZO_OK;
}

szo_status szo_model_decode_step(szo_model_t* m, const int32_t* tokens, int32_t B, int32_t T, int32_t pos0,
                                 const float* S_vals, float* logits_dev, void* stream) {
  SZO_REQUIRE(m != nullptr && tokens != nullptr && logits_dev != nullptr, SZO_ERR_INVALID_ARG, "NULL argument");
  SZO_REQUIRE(m->kcache != nullptr, SZO_ERR_INVALID_ARG, "call szo_model_enable_decode first");
  SZO_REQUIRE(B >= 1 && B <= m->cfg.max_batch && T >= 1 && pos0 >= 0 && pos0 + T <= m->cfg.max_seq, SZO_ERR_SHAPE,
              "need 1 <= B <= %d, T >= 1 and pos0 + T <= %d (got B=%d, T=%d, pos0=%d)", m->cfg.max_batch, m->cfg.max_seq, B,
              T, pos0);
  SZO_REQUIRE(static_cast<int64_t>(B) * T <= m->Mmax, SZO_ERR_SHAPE, "B * T exceeds max_batch * max_seq");
  SZO_REQUIRE(m->cfg.arch == 0 || pos0 + T <= m->cfg.max_pos, SZO_ERR_SHAPE, "position beyond the position table");
  const float* Sv = S_vals ? S_vals : m->S_all;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  auto run = [&](const int32_t* toks, float* out) -> szo_status {
    if (m->cfg.act_dtype == SZO_F32) return run_decode_t<float>(m, toks, B, T, Sv, out, st);
    return run_decode_t<__nv_bfloat16>(m, toks, B, T, Sv, out, st);
  };
  set_i32_kernel<<<1, 1, 0, st>>>(m->d_pos, pos0);
  count_launch();
  // A token step is several hundred short launches: on a stream that can be captured it is recorded once
  // per (B, T, sparse values) as a CUDA graph and replayed (the position comes from device memory, the
  // tokens and logits pass through buffers of the model); the legacy default stream runs it launch by launch.
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  const bool capturable = m->dec_use_graph && st != nullptr && st != cudaStreamLegacy &&
                          cudaStreamIsCapturing(st, &cap) == cudaSuccess && cap == cudaStreamCaptureStatusNone;
  if (!capturable) return run(tokens, logits_dev);
  SZO_CHECK_CUDA(cudaMemcpyAsync(m->dec_tokens, tokens, static_cast<size_t>(B) * T * sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
  cudaGraphExec_t exec = nullptr;
  for (const auto& g : m->dec_graphs)
    if (g.B == B && g.T == T && g.Sv == Sv) exec = g.exec;
  if (exec == nullptr) {
    SZO_CHECK_CUDA(cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal));
    const szo_status rc = run(m->dec_tokens, m->dec_logits);
    cudaGraph_t graph = nullptr;
    const cudaError_t ce = cudaStreamEndCapture(st, &graph);
    if (rc != SZO_OK) {
      if (graph) cudaGraphDestroy(graph);
      return rc;
    }
    SZO_REQUIRE(ce == cudaSuccess && graph != nullptr, SZO_ERR_CUDA, "capture of the token step failed: %s", cudaGetErrorString(ce));
    const cudaError_t ie = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    SZO_REQUIRE(ie == cudaSuccess, SZO_ERR_CUDA, "cudaGraphInstantiate failed: %s", cudaGetErrorString(ie));
    if (m->dec_graphs.size() >= 8) {            // a small cache: drop the oldest
      cudaGraphExecDestroy(m->dec_graphs.front().exec);
      m->dec_graphs.erase(m->dec_graphs.begin());
    }
    m->dec_graphs.push_back({B, T, Sv, exec});
  }
  SZO_CHECK_CUDA(cudaGraphLaunch(exec, st));
  SZO_CHECK_CUDA(cudaMemcpyAsync(logits_dev, m->dec_logits, static_cast<size_t>(B) * m->cfg.vocab * sizeof(float),
                                 cudaMemcpyDeviceToDevice, st));
  return SZO_OK;
}

szo_status szo_model_enable_timing(szo_model_t* m, int32_t on) {
  SZO_REQUIRE(m != nullptr, SZO_ERR_INVALID_ARG, "model is NULL");
  m->timing = on != 0;
  m->events_used = 0;
  return SZO_OK;
}

szo_status szo_model_linear_time(szo_model_t* m, double* ms_total_host, int64_t* launches_host) {
  SZO_REQUIRE(m && ms_total_host && launches_host, SZO_ERR_INVALID_ARG, "NULL argument");
  SZO_CHECK_CUDA(cudaDeviceSynchronize());
  double total = 0.0;
  for (size_t i = 0; i + 1 < m->events_used; i += 2) {
    float ms = 0.f;
    SZO_CHECK_CUDA(cudaEventElapsedTime(&ms, m->events[i], m->events[i + 1]));
    total += ms;
  }
  *ms_total_host = total;
  *launches_host = static_cast<int64_t>(m->events_used / 2);
  m->events_used = 0;
  return SZO_OK;
}

void szo_model_destroy(szo_model_t* m) {
  if (!m) return;
  for (cudaEvent_t e : m->events) cudaEventDestroy(e);
  for (szo_linear_t* p : m->plans) szo_linear_destroy(p);
  szo_linear_destroy(m->lm_head_plan);
  szo_linear_destroy(m->decode_head);
  for (auto& g : m->dec_graphs) cudaGraphExecDestroy(g.exec);
  for (void* p : m->owned) cudaFree(p);
  delete m;
}

}  // extern "C"
