// Decomposed linear layer y = x Dequantize(Q(w_dense))^T + x w_sparse^T (Section 3.4 and the
// appendix "Implementation of Sparse Operations in Linear Layers"): plan construction, the fp32
// validation path (SparseAdd at full precision: dequantise to fp32, add the sparse values, plain
// fp32 GEMM), the CSR SpMM used by the SparseAddMM order, and the mode dispatch.
#include "linear.cuh"

namespace szo {

// ------------------------------------------------------------------------------ plan kernels
// Kernel-ready (scale, zero) table, transposed to [K/G][Npad] so that the 128 rows of a tile are
// contiguous for one group (one bulk copy per tile and k-block).  fp16 inputs are widened to fp32
// pairs; bf16 inputs are stored as the bit patterns of the packed pairs (scale,scale), (zero,zero)
// that the packed-bf16 conversion consumes directly.
__device__ __forceinline__ float2 sz_entry(__half s, __half z) { return make_float2(__half2float(s), __half2float(z)); }
__device__ __forceinline__ float2 sz_entry(__nv_bfloat16 s, __nv_bfloat16 z) {
  const uint32_t sb = *reinterpret_cast<const uint16_t*>(&s), zb = *reinterpret_cast<const uint16_t*>(&z);
  return make_float2(__uint_as_float(sb | (sb << 16)), __uint_as_float(zb | (zb << 16)));
}
template <typename SZ>
__global__ void widen_sz_kernel(const SZ* __restrict__ scales, const SZ* __restrict__ zeros, int64_t N,
                                int64_t groups, int64_t Npad, float2* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= N * groups) return;
  const int64_t n = i / groups, g = i % groups;
  out[g * Npad + n] = sz_entry(scales[i], zeros[i]);
}

// Copy of the packed codes in tile order: block (t, kb) holds rows [128 t, 128 t + 128) x bytes
// [32 kb, 32 kb + 32) of the caller's [N, K/2] array, 4 KiB contiguous, rows beyond N zero.  Inside
// each 32-bit word (eight consecutive columns c .. c+7) the nibbles are re-ordered so that nibble i
// holds column c + 2 i and nibble 4 + i column c + 2 i + 1: the pair (c + 2 i, c + 2 i + 1) is then
// (w >> 4 i) & 0x000F000F, one code per 16-bit half, which is what the bf16 conversion wants.  One
// thread moves 16 bytes.
__device__ __forceinline__ uint32_t pair_order(uint32_t w) {
  uint32_t o = 0;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    o |= ((w >> (8 * i)) & 0xFu) << (4 * i);             // column 2 i: low nibble of byte i
    o |= ((w >> (8 * i + 4)) & 0xFu) << (16 + 4 * i);    // column 2 i + 1: high nibble of byte i
  }
  return o;
}
__global__ void tile_codes_kernel(const uint8_t* __restrict__ codes, int64_t N, int64_t K, int64_t n_tiles,
                                  uint8_t* __restrict__ out) {
  const int64_t nkb = K / 64;
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;     // 16-byte unit
  if (i >= n_tiles * nkb * 256) return;
  const int64_t half = i & 1, r = (i >> 1) & 127, blk = i >> 8;
  const int64_t t = blk / nkb, kb = blk % nkb;
  const int64_t row = t * 128 + r;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (row < N) v = *reinterpret_cast<const uint4*>(codes + row * (K / 2) + kb * 32 + half * 16);
  v = make_uint4(pair_order(v.x), pair_order(v.y), pair_order(v.z), pair_order(v.w));
  *reinterpret_cast<uint4*>(out + i * 16) = v;
}

// Per entry: column, validity (strictly ascending, in range) and the size of its (128-row, 64-col)
// bucket, counted into bucket_ptr[b + 1].
__global__ void entry_kernel(const int64_t* __restrict__ idx, int64_t nnz, int64_t N, int64_t K,
                             int64_t nkb, int32_t* __restrict__ ent_col, int32_t* __restrict__ bucket_ptr,
                             int32_t* __restrict__ bad) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= nnz) return;
  const int64_t v = idx[e];
  if (v < 0 || v >= N * K || (e > 0 && idx[e - 1] >= v)) {
    *bad = 1;
    ent_col[e] = 0;
    return;
  }
  const int64_t row = v / K, col = v % K;
  ent_col[e] = static_cast<int32_t>(col);
  atomicAdd(&bucket_ptr[(row >> 7) * nkb + (col >> 6) + 1], 1);
}

// In-place inclusive scan of a[0..n) by one block (chunks of 1024, carried sequentially).
__global__ void __launch_bounds__(1024) scan_i32_kernel(int32_t* __restrict__ a, int64_t n) {
  __shared__ int32_t s[1024];
  __shared__ int32_t carry;
  if (threadIdx.x == 0) carry = 0;
  __syncthreads();
  for (int64_t base = 0; base < n; base += 1024) {
    const int64_t i = base + threadIdx.x;
    s[threadIdx.x] = i < n ? a[i] : 0;
    __syncthreads();
    for (int o = 1; o < 1024; o <<= 1) {
      const int32_t t = threadIdx.x >= o ? s[threadIdx.x - o] : 0;
      __syncthreads();
      s[threadIdx.x] += t;
      __syncthreads();
    }
    if (i < n) a[i] = carry + s[threadIdx.x];
    __syncthreads();
    if (threadIdx.x == 1023) carry += s[1023];
    __syncthreads();
  }
}

__global__ void row_ptr_kernel(const int64_t* __restrict__ idx, int64_t nnz, int64_t N, int64_t K,
                               int32_t* __restrict__ row_ptr) {
  const int64_t r = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (r > N) return;
  const int64_t key = r * K;
  int64_t lo = 0, hi = nnz;
  while (lo < hi) {
    const int64_t mid = (lo + hi) >> 1;
    if (idx[mid] < key) lo = mid + 1; else hi = mid;
  }
  row_ptr[r] = static_cast<int32_t>(lo);
}

// One thread per 128-row tile walks its entries in index order and appends them to their buckets.
__global__ void bucket_fill_kernel(const int64_t* __restrict__ idx, const int32_t* __restrict__ row_ptr,
                                   const int32_t* __restrict__ ent_col, int64_t N, int64_t K, int64_t nkb,
                                   int64_t n_rowgroups, const int32_t* __restrict__ bucket_ptr,
                                   int32_t* __restrict__ cursor, int32_t* __restrict__ bucket_eid,
                                   uint16_t* __restrict__ bucket_pos) {
  const int64_t g = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (g >= n_rowgroups) return;
  const int64_t r0 = g * 128, r1 = (r0 + 128 < N) ? r0 + 128 : N;
  for (int32_t e = row_ptr[r0]; e < row_ptr[r1]; ++e) {
    const int32_t col = ent_col[e];
    const int64_t row = idx[e] / K;
    const int64_t b = g * nkb + (col >> 6);
    const int32_t pos = bucket_ptr[b] + cursor[b]++;
    bucket_eid[pos] = e;
    // byte offset of the element in the tile's shared-memory image: [128 rows x 64 bf16], rows of 128
    // bytes whose 16-byte chunks are XOR-swizzled by (row & 7) (the layout the MMA descriptor reads)
    const int rl = static_cast<int>(row - r0), cl = static_cast<int>(col & 63);
    bucket_pos[pos] = static_cast<uint16_t>(rl * 128 + (((cl >> 3) ^ (rl & 7)) << 4) + (cl & 7) * 2);
  }
}

// ------------------------------------------------------------------------------ fp32 path
// W_eff[n, c] = fma(q, scale, zero) in fp32 (two elements per thread), from the caller's tables.
template <typename SZ>
__global__ void dequant_f32_kernel(const uint8_t* __restrict__ codes, const SZ* __restrict__ scales,
                                   const SZ* __restrict__ zeros, int64_t N, int64_t K, int G, float* __restrict__ W) {
  const int64_t t = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (t >= N * K / 2) return;
  const int64_t n = (2 * t) / K, c = (2 * t) % K;
  const int64_t gi = n * (K / G) + c / G;
  const float s = static_cast<float>(scales[gi]), z = static_cast<float>(zeros[gi]);
  const uint8_t b = codes[t];
  W[2 * t] = fmaf(static_cast<float>(b & 15), s, z);
  W[2 * t + 1] = fmaf(static_cast<float>(b >> 4), s, z);
}

__global__ void widen_bf16_kernel(const __nv_bfloat16* __restrict__ in, int64_t n, float* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __bfloat162float(in[i]);
}

__global__ void scatter_add_f32_kernel(float* __restrict__ W, const int64_t* __restrict__ idx,
                                       const float* __restrict__ S, int64_t nnz) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e < nnz) W[idx[e]] += S[e];
}

template <typename T> __device__ __forceinline__ void load4(const T* p, float (&v)[4]);
template <> __device__ __forceinline__ void load4<float>(const float* p, float (&v)[4]) {
  const float4 t = *reinterpret_cast<const float4*>(p);
  v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
}
template <> __device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&v)[4]) {
  const uint2 t = *reinterpret_cast<const uint2*>(p);
  v[0] = __uint_as_float(t.x << 16); v[1] = __uint_as_float(t.x & 0xFFFF0000u);
  v[2] = __uint_as_float(t.y << 16); v[3] = __uint_as_float(t.y & 0xFFFF0000u);
}
__device__ __forceinline__ void store1(float* p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// C[m,n] = sum_k A[m,k] B[n,k] + bias[n]; 64x64x16 tiles, 256 threads, 4x4 outputs per thread,
// fp32 accumulation in ascending k.
template <typename TA, typename TC>
__global__ void __launch_bounds__(256)
sgemm_nt_kernel(const TA* __restrict__ A, const float* __restrict__ B, const float* __restrict__ bias,
                TC* __restrict__ C, int64_t M, int64_t N, int64_t K) {
  __shared__ float As[16][68];
  __shared__ float Bs[16][68];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  const int64_t m0 = static_cast<int64_t>(blockIdx.y) * 64, n0 = static_cast<int64_t>(blockIdx.x) * 64;
  const int lr = tid >> 2, lk = (tid & 3) * 4;
  float acc[4][4] = {};
  for (int64_t k0 = 0; k0 < K; k0 += 16) {
    float a[4] = {0.f, 0.f, 0.f, 0.f}, b[4] = {0.f, 0.f, 0.f, 0.f};
    if (m0 + lr < M) load4<TA>(A + (m0 + lr) * K + k0 + lk, a);
    if (n0 + lr < N) load4<float>(B + (n0 + lr) * K + k0 + lk, b);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lr] = a[i];
      Bs[lk + i][lr] = b[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float ar[4] = {av.x, av.y, av.z, av.w}, br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int64_t m = m0 + ty * 4 + i;
    if (m >= M) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int64_t n = n0 + tx * 4 + j;
      if (n < N) store1(C + m * N + n, acc[i][j] + (bias ? bias[n] : 0.f));
    }
  }
}

// Non-uniform 4-bit format: W[n, c] = lut[n][q[n, c]] (fp32 holds a 16-bit float exactly).
template <typename T>
__global__ void dequant_lut_f32_kernel(const uint8_t* __restrict__ codes, const T* __restrict__ lut, int64_t N,
                                       int64_t K, float* __restrict__ W) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;   // one byte: two columns
  if (i >= N * (K / 2)) return;
  const int64_t n = i / (K / 2);
  const uint8_t b = codes[i];
  W[2 * i] = static_cast<float>(lut[n * 16 + (b & 0xF)]);
  W[2 * i + 1] = static_cast<float>(lut[n * 16 + (b >> 4)]);
}

template <typename T>
__global__ void lut_to_bf16_kernel(const T* __restrict__ lut, int64_t n, __nv_bfloat16* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) out[i] = __float2bfloat16_rn(static_cast<float>(lut[i]));
}

size_t linear_ws_fp32(const szo_linear* p, int64_t) {
  return round_up(static_cast<size_t>(p->N) * p->K * sizeof(float), 256);
}

szo_status linear_fwd_fp32(const szo_linear* p, const void* x, int x_dtype, int64_t M, const float* S,
                           void* y, int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st) {
  SZO_REQUIRE(ws && ws_bytes >= linear_ws_fp32(p, M), SZO_ERR_WORKSPACE,
              "fp32 path needs a workspace of %zu bytes", linear_ws_fp32(p, M));
  float* W = static_cast<float*>(ws);
  const int64_t NK = p->N * p->K;
  if (p->G < 0) {
    if (p->sz_dtype == SZO_BF16)
      dequant_lut_f32_kernel<__nv_bfloat16><<<static_cast<unsigned>(ceil_div(NK / 2, 256)), 256, 0, st>>>(
          static_cast<const uint8_t*>(p->codes), static_cast<const __nv_bfloat16*>(p->lut), p->N, p->K, W);
    else
      dequant_lut_f32_kernel<__half><<<static_cast<unsigned>(ceil_div(NK / 2, 256)), 256, 0, st>>>(
          static_cast<const uint8_t*>(p->codes), static_cast<const __half*>(p->lut), p->N, p->K, W);
  } else if (p->G > 0) {
    if (p->sz_dtype == SZO_BF16)
      dequant_f32_kernel<__nv_bfloat16><<<static_cast<unsigned>(ceil_div(NK / 2, 256)), 256, 0, st>>>(
          static_cast<const uint8_t*>(p->codes), static_cast<const __nv_bfloat16*>(p->scales),
          static_cast<const __nv_bfloat16*>(p->zeros), p->N, p->K, p->G, W);
    else
      dequant_f32_kernel<__half><<<static_cast<unsigned>(ceil_div(NK / 2, 256)), 256, 0, st>>>(
          static_cast<const uint8_t*>(p->codes), static_cast<const __half*>(p->scales),
          static_cast<const __half*>(p->zeros), p->N, p->K, p->G, W);
  } else {
    widen_bf16_kernel<<<static_cast<unsigned>(ceil_div(NK, 256)), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(p->codes), NK, W);
  }
  count_launch();
  if (p->nnz) {
    scatter_add_f32_kernel<<<static_cast<unsigned>(ceil_div(p->nnz, 256)), 256, 0, st>>>(W, p->idx, S, p->nnz);
    count_launch();
  }
  dim3 grid(static_cast<unsigned>(ceil_div(p->N, 64)), static_cast<unsigned>(ceil_div(M, 64)));
  if (x_dtype == SZO_F32 && y_dtype == SZO_F32)
    sgemm_nt_kernel<float, float><<<grid, 256, 0, st>>>(static_cast<const float*>(x), W, p->bias,
                                                       static_cast<float*>(y), M, p->N, p->K);
  else if (x_dtype == SZO_F32)
    sgemm_nt_kernel<float, __nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const float*>(x), W, p->bias,
                                                               static_cast<__nv_bfloat16*>(y), M, p->N, p->K);
  else if (y_dtype == SZO_F32)
    sgemm_nt_kernel<__nv_bfloat16, float><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), W, p->bias,
                                                               static_cast<float*>(y), M, p->N, p->K);
  else
    sgemm_nt_kernel<__nv_bfloat16, __nv_bfloat16><<<grid, 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(x), W, p->bias, static_cast<__nv_bfloat16*>(y), M, p->N, p->K);
  count_launch();
  SZO_CHECK_LAUNCH("fp32 linear kernels");
  return SZO_OK;
}

// ------------------------------------------------------------------------------ CSR SpMM
// y[m, r] += sum_{e in row r} S[e] x[m, c_e].  A block stages a slab of TM tokens of x in shared
// memory as xs[c][TM]; its threads walk the rows r (coalesced along r in y), each gathering the
// TM values of column c_e with one vector read.  Rows are independent: deterministic.
template <int TM, typename TY>
__global__ void __launch_bounds__(256)
spmm_slab_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ row_ptr,
                 const int32_t* __restrict__ ent_col, const float* __restrict__ S, TY* __restrict__ y,
                 int64_t M, int64_t N, int64_t K) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);   // [K][TM]
  const int64_t m0 = static_cast<int64_t>(blockIdx.x) * TM;
  for (int64_t i = threadIdx.x; i < K * TM; i += blockDim.x) {
    const int64_t t = i / K, c = i % K;              // coalesced along c
    xs[c * TM + t] = (m0 + t < M) ? x[(m0 + t) * K + c] : __float2bfloat16_rn(0.f);
  }
  __syncthreads();
  for (int64_t r = threadIdx.x; r < N; r += blockDim.x) {
    const int32_t e0 = row_ptr[r], e1 = row_ptr[r + 1];
    if (e0 == e1) continue;
    float acc[TM];
#pragma unroll
    for (int t = 0; t < TM; ++t) acc[t] = 0.f;
    for (int32_t e = e0; e < e1; ++e) {
      const float s = S[e];
      const __nv_bfloat16* col = xs + static_cast<int64_t>(ent_col[e]) * TM;
#pragma unroll
      for (int t = 0; t < TM; ++t) acc[t] = fmaf(s, __bfloat162float(col[t]), acc[t]);
    }
#pragma unroll
    for (int t = 0; t < TM; ++t) {
      if (m0 + t < M) {
        TY* dst = y + (m0 + t) * N + r;
        store1(dst, static_cast<float>(*dst) + acc[t]);
      }
    }
  }
}

szo_status linear_spmm(const szo_linear* p, const void* x, int64_t M, const float* S, void* y,
                       int y_dtype, cudaStream_t st) {
  if (p->nnz == 0 || M == 0) return SZO_OK;
  const int TM = (p->K * 8 * 2 <= 200 * 1024) ? 8 : 4;
  const size_t smem = static_cast<size_t>(p->K) * TM * 2;
  SZO_REQUIRE(smem <= 220 * 1024, SZO_ERR_UNSUPPORTED, "K = %lld too large for the SpMM slab", (long long)p->K);
  const unsigned grid = static_cast<unsigned>(ceil_div(M, TM));
  const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
#define SZO_SPMM(TMV, TYV)                                                                          \
  do {                                                                                              \
    cudaFuncSetAttribute(spmm_slab_kernel<TMV, TYV>, cudaFuncAttributeMaxDynamicSharedMemorySize,   \
                         static_cast<int>(smem));                                                   \
    spmm_slab_kernel<TMV, TYV><<<grid, 256, smem, st>>>(xb, p->row_ptr, p->ent_col, S,             \
                                                        static_cast<TYV*>(y), M, p->N, p->K);       \
  } while (0)
  if (TM == 8) {
    if (y_dtype == SZO_F32) SZO_SPMM(8, float); else SZO_SPMM(8, __nv_bfloat16);
  } else {
    if (y_dtype == SZO_F32) SZO_SPMM(4, float); else SZO_SPMM(4, __nv_bfloat16);
  }
#undef SZO_SPMM
  count_launch();
  SZO_CHECK_LAUNCH("spmm_slab_kernel");
  return SZO_OK;
}

// rec[p] = (position of bucket entry p inside its tile, bits of S[eid[p]])
__global__ void gather_values_kernel(const float* __restrict__ S, const int32_t* __restrict__ eid,
                                     const uint16_t* __restrict__ pos, int64_t n, uint2* __restrict__ out) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i < n) out[i] = make_uint2(pos[i], __float_as_uint(S[eid[i]]));
}

szo_status gather_values(const float* S, const int32_t* eid, const uint16_t* pos, int64_t n, uint2* out,
                         cudaStream_t st) {
  if (n == 0) return SZO_OK;
  gather_values_kernel<<<static_cast<unsigned>(ceil_div(n, 256)), 256, 0, st>>>(S, eid, pos, n, out);
  count_launch();
  SZO_CHECK_LAUNCH("gather_values_kernel");
  return SZO_OK;
}

szo_status linear_fwd_impl(const szo_linear* p, const void* x, int x_dtype, int64_t M, const float* S_pert,
                           const uint2* S_bucket, void* y, int y_dtype, int32_t mode, void* workspace,
                           size_t workspace_bytes, cudaStream_t st) {
  if (mode == SZO_MODE_FP32_VALIDATE)
    return linear_fwd_fp32(p, x, x_dtype, M, S_pert, y, y_dtype, workspace, workspace_bytes, st);
  SZO_REQUIRE(!(p->G < 0 && mode == SZO_MODE_SPMM), SZO_ERR_UNSUPPORTED,
              "table-coded weights take the SparseAdd order only (SZO_MODE_AUTO or SZO_MODE_SPARSE_ADD)");
  if (mode == SZO_MODE_SPMM) {
    SZO_TRY(linear_fwd_tc(p, x, M, nullptr, y, y_dtype, workspace, workspace_bytes, st));
    return linear_spmm(p, x, M, S_pert, y, y_dtype, st);
  }
  if (mode == SZO_MODE_AUTO && few_token_applies(&p, 1, M)) return linear_fwd_skinny(p, x, M, S_pert, y, y_dtype, st);
  if (tc_use_materialised(p, M))
    return linear_fwd_tc_materialised(&p, 1, x, M, &S_pert, &y, y_dtype, workspace, workspace_bytes, st);
  unsigned char* ws = static_cast<unsigned char*>(workspace);
  if (p->nnz > 0 && S_bucket == nullptr) {
    const size_t need = round_up(static_cast<size_t>(p->nnz) * sizeof(uint2), 256);
    SZO_REQUIRE(workspace && workspace_bytes >= need, SZO_ERR_WORKSPACE,
                "SparseAdd needs a workspace of %zu bytes for the bucket-ordered values", need);
    SZO_TRY(gather_values(S_pert, p->bucket_eid, p->bucket_pos, p->nnz, static_cast<uint2*>(workspace), st));
    S_bucket = static_cast<const uint2*>(workspace);
    ws += need;
    workspace_bytes -= need;
  }
  return linear_fwd_tc(p, x, M, S_bucket, y, y_dtype, workspace ? ws : nullptr, workspace ? workspace_bytes : 0, st);
}

static void free_plan(szo_linear* p) {
  if (!p) return;
  tc_plan_destroy(p);
  cudaFree(p->sz);
  cudaFree(p->lut_bf16);
  cudaFree(p->codes_tiled);
  cudaFree(p->ent_col);
  cudaFree(p->row_ptr);
  cudaFree(p->bucket_ptr);
  cudaFree(p->bucket_eid);
  cudaFree(p->bucket_pos);
  delete p;
}

}  // namespace szo

using namespace szo;

// G == -1: codes into the per-row table `lut` (type sz_dtype), scales/zeros unused.
static szo_status create_plan(szo_linear_t** out, int64_t N, int64_t K, int32_t G,
                              const void* codes_or_bf16_W, const void* scales, const void* zeros,
                              const void* lut, szo_dtype sz_dtype, const int64_t* idx, int64_t nnz,
                              const float* bias, void* stream) {
  SZO_REQUIRE(out != nullptr, SZO_ERR_INVALID_ARG, "out is NULL");
  *out = nullptr;
  SZO_REQUIRE(N > 0 && K > 0, SZO_ERR_SHAPE, "N and K must be positive");
  SZO_REQUIRE(K % 64 == 0, SZO_ERR_SHAPE, "K (%lld) must be a multiple of 64", (long long)K);
  SZO_REQUIRE(G >= -1 && (G <= 0 || ((G == 32 || G % 64 == 0) && K % G == 0)), SZO_ERR_SHAPE,
              "G (%d) must be 0, 32 or a multiple of 64, and divide K", G);
  SZO_REQUIRE(G != -1 || lut != nullptr, SZO_ERR_INVALID_ARG, "lut is NULL");
  SZO_REQUIRE(aligned16(lut), SZO_ERR_ALIGNMENT, "lut must be 16-byte aligned");
  SZO_REQUIRE(N * K < (int64_t(1) << 40), SZO_ERR_SHAPE, "tensor too large");
  SZO_REQUIRE(nnz >= 0 && nnz <= N * K && nnz < (int64_t(1) << 31), SZO_ERR_INVALID_ARG, "bad nnz");
  SZO_REQUIRE(codes_or_bf16_W != nullptr, SZO_ERR_INVALID_ARG, "weight pointer is NULL");
  SZO_REQUIRE(G <= 0 || (scales && zeros), SZO_ERR_INVALID_ARG, "scales/zeros are NULL");
  SZO_REQUIRE(G == 0 || sz_dtype == SZO_BF16 || sz_dtype == SZO_F16, SZO_ERR_UNSUPPORTED,
              "the 16-bit table type must be bf16 or f16");
  SZO_REQUIRE(nnz == 0 || idx != nullptr, SZO_ERR_INVALID_ARG, "idx is NULL");
  SZO_REQUIRE(aligned16(codes_or_bf16_W) && aligned16(scales) && aligned16(zeros) && aligned16(idx) &&
                  aligned16(bias),
              SZO_ERR_ALIGNMENT, "buffers must be 16-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  szo_linear* p = new szo_linear();
  *p = szo_linear{};
  p->N = N; p->K = K; p->G = G; p->sz_dtype = sz_dtype; p->nnz = nnz;
  p->codes = codes_or_bf16_W; p->scales = scales; p->zeros = zeros; p->idx = idx; p->bias = bias;
  p->lut = lut;
  p->n_rowgroups = ceil_div(N, 128);
  p->Npad = ceil_div(N, 256) * 256;   // the pair-tile kernel copies 128-row strips up to this bound
  p->n_kblocks = K / 64;
  const int64_t nb = p->n_rowgroups * p->n_kblocks;
  int32_t* cursor = nullptr;
  int32_t* bad = nullptr;
  szo_status rc = SZO_OK;
  auto cleanup = [&](szo_status s) {
    cudaFree(cursor);
    cudaFree(bad);
    if (s != SZO_OK) free_plan(p);
    return s;
  };
#define SZO_PLAN_CUDA(expr)                                                                  \
  do {                                                                                       \
    cudaError_t e__ = (expr);                                                                \
    if (e__ != cudaSuccess)                                                                  \
      return cleanup(fail(SZO_ERR_CUDA, "%s failed: %s", #expr, cudaGetErrorString(e__)));   \
  } while (0)
  if (G > 0) {
    const int64_t ng = N * (K / G);
    SZO_PLAN_CUDA(cudaMalloc(&p->sz, p->Npad * (K / G) * sizeof(float2)));
    SZO_PLAN_CUDA(cudaMemsetAsync(p->sz, 0, p->Npad * (K / G) * sizeof(float2), st));
    if (sz_dtype == SZO_BF16)
      widen_sz_kernel<__nv_bfloat16><<<static_cast<unsigned>(ceil_div(ng, 256)), 256, 0, st>>>(
          static_cast<const __nv_bfloat16*>(scales), static_cast<const __nv_bfloat16*>(zeros), N, K / G, p->Npad, p->sz);
    else
      widen_sz_kernel<__half><<<static_cast<unsigned>(ceil_div(ng, 256)), 256, 0, st>>>(
          static_cast<const __half*>(scales), static_cast<const __half*>(zeros), N, K / G, p->Npad, p->sz);
  }
  if (G < 0) {
    SZO_PLAN_CUDA(cudaMalloc(&p->lut_bf16, p->Npad * 16 * sizeof(__nv_bfloat16)));
    SZO_PLAN_CUDA(cudaMemsetAsync(p->lut_bf16, 0, p->Npad * 16 * sizeof(__nv_bfloat16), st));
    if (sz_dtype == SZO_BF16)
      lut_to_bf16_kernel<__nv_bfloat16><<<static_cast<unsigned>(ceil_div(N * 16, 256)), 256, 0, st>>>(
          static_cast<const __nv_bfloat16*>(lut), N * 16, p->lut_bf16);
    else
      lut_to_bf16_kernel<__half><<<static_cast<unsigned>(ceil_div(N * 16, 256)), 256, 0, st>>>(
          static_cast<const __half*>(lut), N * 16, p->lut_bf16);
  }
  if (G != 0) {
    const int64_t n_code_tiles = p->Npad / 128;      // padded to an even count for the pair-tile kernel
    const int64_t units = n_code_tiles * (K / 64) * 256;
    SZO_PLAN_CUDA(cudaMalloc(&p->codes_tiled, units * 16));
    tile_codes_kernel<<<static_cast<unsigned>(ceil_div(units, 256)), 256, 0, st>>>(
        static_cast<const uint8_t*>(codes_or_bf16_W), N, K, n_code_tiles, p->codes_tiled);
  }
  SZO_PLAN_CUDA(cudaMalloc(&p->row_ptr, (N + 1) * sizeof(int32_t)));
  SZO_PLAN_CUDA(cudaMalloc(&p->bucket_ptr, (nb + 1) * sizeof(int32_t)));
  SZO_PLAN_CUDA(cudaMemsetAsync(p->bucket_ptr, 0, (nb + 1) * sizeof(int32_t), st));
  SZO_PLAN_CUDA(cudaMalloc(&bad, sizeof(int32_t)));
  SZO_PLAN_CUDA(cudaMemsetAsync(bad, 0, sizeof(int32_t), st));
  if (nnz > 0) {
    SZO_PLAN_CUDA(cudaMalloc(&p->ent_col, nnz * sizeof(int32_t)));
    SZO_PLAN_CUDA(cudaMalloc(&p->bucket_eid, nnz * sizeof(int32_t)));
    SZO_PLAN_CUDA(cudaMalloc(&p->bucket_pos, nnz * sizeof(uint16_t)));
    SZO_PLAN_CUDA(cudaMalloc(&cursor, nb * sizeof(int32_t)));
    SZO_PLAN_CUDA(cudaMemsetAsync(cursor, 0, nb * sizeof(int32_t), st));
    entry_kernel<<<static_cast<unsigned>(ceil_div(nnz, 256)), 256, 0, st>>>(idx, nnz, N, K, p->n_kblocks,
                                                                           p->ent_col, p->bucket_ptr, bad);
    scan_i32_kernel<<<1, 1024, 0, st>>>(p->bucket_ptr, nb + 1);
  }
  row_ptr_kernel<<<static_cast<unsigned>(ceil_div(N + 1, 256)), 256, 0, st>>>(idx, nnz, N, K, p->row_ptr);
  if (nnz > 0) {
    bucket_fill_kernel<<<static_cast<unsigned>(ceil_div(p->n_rowgroups, 128)), 128, 0, st>>>(
        idx, p->row_ptr, p->ent_col, N, K, p->n_kblocks, p->n_rowgroups, p->bucket_ptr, cursor,
        p->bucket_eid, p->bucket_pos);
  }
  SZO_PLAN_CUDA(cudaGetLastError());
  int32_t bad_h = 0;
  SZO_PLAN_CUDA(cudaMemcpyAsync(&bad_h, bad, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
  SZO_PLAN_CUDA(cudaStreamSynchronize(st));
  if (bad_h) return cleanup(fail(SZO_ERR_INVALID_ARG, "idx must be strictly ascending and inside [0, N*K)"));
  rc = tc_plan_create(p, st);
  if (rc != SZO_OK) return cleanup(rc);
#undef SZO_PLAN_CUDA
  cleanup(SZO_OK);
  *out = p;
  return SZO_OK;
}

extern "C" {

szo_status szo_linear_create(szo_linear_t** out, int64_t N, int64_t K, int32_t G,
                             const void* codes_or_bf16_W, const void* scales, const void* zeros,
                             szo_dtype sz_dtype, const int64_t* idx, int64_t nnz, const float* bias,
                             void* stream) {
  SZO_REQUIRE(G >= 0, SZO_ERR_SHAPE, "G (%d) must be 0, 32 or a multiple of 64, and divide K", G);
  return create_plan(out, N, K, G, codes_or_bf16_W, scales, zeros, nullptr, sz_dtype, idx, nnz, bias, stream);
}

szo_status szo_linear_create_lut(szo_linear_t** out, int64_t N, int64_t K, const uint8_t* codes,
                                 const void* lut, szo_dtype lut_dtype, const int64_t* idx, int64_t nnz,
                                 const float* bias, void* stream) {
  return create_plan(out, N, K, -1, codes, nullptr, nullptr, lut, lut_dtype, idx, nnz, bias, stream);
}

size_t szo_linear_workspace_bytes(const szo_linear_t* p, int64_t M, int32_t mode) {
  if (!p) return 0;
  if (mode == SZO_MODE_FP32_VALIDATE) return linear_ws_fp32(p, M);
  const szo_linear* self = p;
  if (mode == SZO_MODE_AUTO && few_token_applies(&self, 1, M)) return 0;
  const szo_linear* pp = p;
  const size_t tail = tc_tail_ws_bytes(&pp, 1, M);                     // K-split tiles of the last round
  if (mode == SZO_MODE_SPMM) return tail;
  if (tc_use_materialised(p, M)) return tc_materialised_ws_bytes(&pp, 1, M);
  return round_up(static_cast<size_t>(p->nnz) * sizeof(uint2), 256) + tail;   // + bucket-ordered sparse records
}

szo_status szo_linear_fwd(const szo_linear_t* p, const void* x, szo_dtype x_dtype, int64_t M,
                          const float* S_pert, void* y, szo_dtype y_dtype, int32_t mode, void* workspace,
                          size_t workspace_bytes, void* stream) {
  SZO_REQUIRE(p != nullptr, SZO_ERR_INVALID_ARG, "plan is NULL");
  SZO_REQUIRE(M >= 0, SZO_ERR_SHAPE, "M < 0");
  SZO_REQUIRE(mode >= SZO_MODE_AUTO && mode <= SZO_MODE_FP32_VALIDATE, SZO_ERR_INVALID_ARG, "unknown mode %d", mode);
  SZO_REQUIRE(y_dtype == SZO_BF16 || y_dtype == SZO_F32, SZO_ERR_UNSUPPORTED, "y must be bf16 or f32");
  SZO_REQUIRE(x_dtype == SZO_BF16 || (x_dtype == SZO_F32 && mode == SZO_MODE_FP32_VALIDATE), SZO_ERR_UNSUPPORTED,
              "x must be bf16 (f32 only in the validation mode)");
  if (M == 0) return SZO_OK;
  SZO_REQUIRE(x && y, SZO_ERR_INVALID_ARG, "x or y is NULL");
  SZO_REQUIRE(p->nnz == 0 || S_pert, SZO_ERR_INVALID_ARG, "S_pert is NULL");
  SZO_REQUIRE(aligned16(x) && aligned16(y) && aligned16(workspace), SZO_ERR_ALIGNMENT,
              "x, y and workspace must be 16-byte aligned");
  SZO_REQUIRE((reinterpret_cast<uintptr_t>(S_pert) & 3u) == 0, SZO_ERR_ALIGNMENT, "S_pert must be 4-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  return linear_fwd_impl(p, x, x_dtype, M, S_pert, nullptr, y, y_dtype, mode, workspace, workspace_bytes, st);
}

size_t szo_linear_paired_workspace_bytes(const szo_linear_t* p, int64_t M) {
  if (!p || M <= 0 || p->tc == nullptr) return 0;
  const szo_linear* pp = p;
  return tc_materialised_ws_bytes(&pp, 1, M, tc_paired_dense_cross(&pp, 1)) + cross_rec_bytes(&pp, 1);
}

szo_status szo_linear_fwd_paired(const szo_linear_t* p, const void* x, int64_t M, const float* S, const float* z,
                                 float eps, void* y, szo_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                 void* stream) {
  SZO_REQUIRE(p != nullptr, SZO_ERR_INVALID_ARG, "plan is NULL");
  SZO_REQUIRE(M >= 0 && M < (int64_t(1) << 30), SZO_ERR_SHAPE, "bad M");
  SZO_REQUIRE(y_dtype == SZO_BF16 || y_dtype == SZO_F32, SZO_ERR_UNSUPPORTED, "y must be bf16 or f32");
  SZO_REQUIRE(eps != 0.f, SZO_ERR_INVALID_ARG, "eps == 0");
  if (M == 0) return SZO_OK;
  SZO_REQUIRE(x && y, SZO_ERR_INVALID_ARG, "x or y is NULL");
  SZO_REQUIRE(p->nnz == 0 || (S && z), SZO_ERR_INVALID_ARG, "S or z is NULL");
  SZO_REQUIRE(aligned16(x) && aligned16(y) && aligned16(workspace), SZO_ERR_ALIGNMENT,
              "x, y and workspace must be 16-byte aligned");
  SZO_REQUIRE(((reinterpret_cast<uintptr_t>(S) | reinterpret_cast<uintptr_t>(z)) & 3u) == 0, SZO_ERR_ALIGNMENT,
              "S and z must be 4-byte aligned");
  const size_t need = szo_linear_paired_workspace_bytes(p, M);
  SZO_REQUIRE(workspace != nullptr && workspace_bytes >= need, SZO_ERR_WORKSPACE,
              "the paired form needs a workspace of %zu bytes", need);
  const szo_linear* pp = p;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t rec_bytes = cross_rec_bytes(&pp, 1);
  uint32_t* rec = reinterpret_cast<uint32_t*>(static_cast<unsigned char*>(workspace) + (need - rec_bytes));
  const bool dense = tc_paired_dense_cross(&pp, 1);
  SZO_TRY(pack_cross_records(p, z, eps, rec, st));
  const uint32_t* recs[1] = {rec};
  const PairedArgs pa{recs, &z, eps, dense};
  return linear_fwd_tc_materialised(&pp, 1, x, M, &S, &y, y_dtype, workspace, need - rec_bytes,
                                    static_cast<cudaStream_t>(stream), nullptr, nullptr, nullptr, false, &pa);
}

void szo_linear_destroy(szo_linear_t* p) { free_plan(p); }

}  // extern "C"
