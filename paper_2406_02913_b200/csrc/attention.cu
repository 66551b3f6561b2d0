// Causal softmax attention for the bf16 activation path: a flash-style kernel on warp-level tensor
// core MMAs (mma.sync m16n8k16, bf16 inputs, fp32 accumulation and softmax statistics).
//
// The loss path needs attention only as one block of the black-box loss f (Definition 1); it is a
// few percent of a step's flops, so the legacy warp-level MMA is enough here and the tcgen05
// machinery is kept for the linears.  One CTA = 64 queries of one (batch, head); 4 warps x 16 rows;
// K/V tiles of 64 keys double-buffered in padded shared memory (cp.async); online softmax; grouped-query attention by
// mapping query head h to KV head h / (H / Hkv).  q, k, v, o are [B*S, heads*HD] bf16 row-major.
#include "common.cuh"

namespace szo {

namespace {

constexpr int kQT = 64, kKT = 64;

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
               : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

// Copies a [rows x HD] bf16 tile (row stride `ld` elements in global memory) into padded shared
// memory (row stride HD + 8), zero-filling rows at or beyond `valid`.
template <int HD>
__device__ __forceinline__ void load_tile(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int valid) {
  constexpr int kChunks = HD / 8;                 // 16-byte chunks per row
  for (int i = threadIdx.x; i < 64 * kChunks; i += 128) {
    const int r = i / kChunks, c = i % kChunks;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (r < valid) v = *reinterpret_cast<const uint4*>(src + r * ld + c * 8);
    *reinterpret_cast<uint4*>(dst + r * (HD + 8) + c * 8) = v;
  }
}

// Same copy with cp.async (16 bytes per request, bypassing L1), for the double-buffered K/V tiles.
template <int HD>
__device__ __forceinline__ void load_tile_async(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int valid) {
  constexpr int kChunks = HD / 8;
  for (int i = threadIdx.x; i < 64 * kChunks; i += 128) {
    const int r = i / kChunks, c = i % kChunks;
    __nv_bfloat16* d = dst + r * (HD + 8) + c * 8;
    if (r < valid) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(d))),
                   "l"(src + r * ld + c * 8)
                   : "memory");
    } else {
      *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

template <int HD>
__global__ void __launch_bounds__(128, 3)
flash_attn_bf16_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                       const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, int S, int H, int Hkv,
                       float scale_log2e) {
  constexpr int LDS = HD + 8;
  extern __shared__ __align__(16) unsigned char smem_attn[];
  // two stages of (K tile, V tile); the query tile first sits in stage 1's K slot and is moved to
  // registers before that stage is filled (4 tiles of shared memory: three CTAs per SM)
  __nv_bfloat16* sKV = reinterpret_cast<__nv_bfloat16*>(smem_attn);
  __nv_bfloat16* sQ = sKV + 2 * kKT * LDS;

  // heavy query tiles (many key tiles) are scheduled first
  const int qt = gridDim.x - 1 - blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int hk = hq / (H / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t ldq = static_cast<int64_t>(H) * HD, ldk = static_cast<int64_t>(Hkv) * HD;
  const int q0 = qt * kQT;
  const __nv_bfloat16* qbase = q + (static_cast<int64_t>(b) * S + q0) * ldq + hq * HD;
  auto issue_kv = [&](int kt) {                 // K and V tile kt into stage kt & 1
    const int k0 = kt * kKT;
    const int valid = S - k0 < kKT ? S - k0 : kKT;
    __nv_bfloat16* dK = sKV + (kt & 1) * 2 * kKT * LDS;
    load_tile_async<HD>(dK, k + (static_cast<int64_t>(b) * S + k0) * ldk + hk * HD, ldk, valid);
    load_tile_async<HD>(dK + kKT * LDS, v + (static_cast<int64_t>(b) * S + k0) * ldk + hk * HD, ldk, valid);
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  // the query tile and the first K/V tile travel together: one global-memory latency for both
  load_tile_async<HD>(sQ, qbase, ldq, S - q0 < kQT ? S - q0 : kQT);
  asm volatile("cp.async.commit_group;" ::: "memory");
  issue_kv(0);
  asm volatile("cp.async.wait_group 1;" ::: "memory");          // the query tile has landed
  __syncthreads();

  // this warp's 16 query rows as A fragments, kept in registers
  uint32_t qa[HD / 16][4];
#pragma unroll
  for (int ks = 0; ks < HD / 16; ++ks) {
    const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(
        sQ + (warp * 16 + (lane & 15)) * LDS + ks * 16 + (lane >> 4) * 8));
    ldsm_x4(addr, qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
  }

  float oacc[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) oacc[i][0] = oacc[i][1] = oacc[i][2] = oacc[i][3] = 0.f;
  float mrow[2] = {-INFINITY, -INFINITY}, lrow[2] = {0.f, 0.f};
  const int row_a = q0 + warp * 16 + g, row_b = row_a + 8;     // the two query rows of this thread

  __syncthreads();                              // every warp holds its query fragments: stage 1 is free
  for (int kt = 0; kt <= qt; ++kt) {
    const int k0 = kt * kKT;
    const int valid = S - k0 < kKT ? S - k0 : kKT;
    if (kt + 1 <= qt) {
      issue_kv(kt + 1);                                         // overlaps with the math on tile kt
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();                                            // tile kt is visible to every warp
    const __nv_bfloat16* sK = sKV + (kt & 1) * 2 * kKT * LDS;
    const __nv_bfloat16* sV = sK + kKT * LDS;

    // scores: 16 rows x 64 keys per warp
    float sacc[kKT / 8][4];
#pragma unroll
    for (int i = 0; i < kKT / 8; ++i) sacc[i][0] = sacc[i][1] = sacc[i][2] = sacc[i][3] = 0.f;
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
#pragma unroll
      for (int np = 0; np < kKT / 16; ++np) {                   // two key tiles of 8 per ldmatrix.x4
        uint32_t b0, b1, b2, b3;
        const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(
            sK + (np * 16 + (lane & 7) + (lane >> 4) * 8) * LDS + ks * 16 + ((lane >> 3) & 1) * 8));
        ldsm_x4(addr, b0, b1, b2, b3);
        mma_bf16(sacc[2 * np], qa[ks], b0, b1);
        mma_bf16(sacc[2 * np + 1], qa[ks], b2, b3);
      }
    }
    // causal mask (diagonal tile) and keys beyond the sequence
    if (kt == qt || valid < kKT) {
#pragma unroll
      for (int i = 0; i < kKT / 8; ++i) {
        const int c = k0 + i * 8 + 2 * t;
        if (c > row_a || c >= S) sacc[i][0] = -INFINITY;
        if (c + 1 > row_a || c + 1 >= S) sacc[i][1] = -INFINITY;
        if (c > row_b || c >= S) sacc[i][2] = -INFINITY;
        if (c + 1 > row_b || c + 1 >= S) sacc[i][3] = -INFINITY;
      }
    }
    // online softmax, rows g and g+8
    float mx[2] = {mrow[0], mrow[1]};
#pragma unroll
    for (int i = 0; i < kKT / 8; ++i) {
      mx[0] = fmaxf(mx[0], fmaxf(sacc[i][0], sacc[i][1]));
      mx[1] = fmaxf(mx[1], fmaxf(sacc[i][2], sacc[i][3]));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    float corr[2], msc[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      // a row always has at least its own key in the first tile, so mx is finite from then on
      msc[r] = (mx[r] == -INFINITY) ? 0.f : mx[r] * scale_log2e;
      corr[r] = (mrow[r] == -INFINITY) ? 0.f : exp2f(mrow[r] * scale_log2e - msc[r]);
      mrow[r] = mx[r];
      lrow[r] *= corr[r];
    }
    uint32_t pa[kKT / 16][4];
    float psum[2] = {0.f, 0.f};
#pragma unroll
    for (int i = 0; i < kKT / 8; ++i) {
      const float p0 = exp2f(sacc[i][0] * scale_log2e - msc[0]), p1 = exp2f(sacc[i][1] * scale_log2e - msc[0]);
      const float p2 = exp2f(sacc[i][2] * scale_log2e - msc[1]), p3 = exp2f(sacc[i][3] * scale_log2e - msc[1]);
      psum[0] += p0 + p1;
      psum[1] += p2 + p3;
      // accumulator layout of two adjacent 8-key tiles = A fragment of one 16-key step
      pa[i >> 1][(i & 1) * 2 + 0] = pack2(p0, p1);
      pa[i >> 1][(i & 1) * 2 + 1] = pack2(p2, p3);
    }
    lrow[0] += psum[0];
    lrow[1] += psum[1];
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      oacc[i][0] *= corr[0];
      oacc[i][1] *= corr[0];
      oacc[i][2] *= corr[1];
      oacc[i][3] *= corr[1];
    }
    // O += P V
#pragma unroll
    for (int ks = 0; ks < kKT / 16; ++ks) {
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {                    // two 8-wide d tiles per ldmatrix.x4.trans
        uint32_t b0, b1, b2, b3;
        const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(
            sV + (ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + dp * 16 + (lane >> 4) * 8));
        ldsm_x4_trans(addr, b0, b1, b2, b3);
        mma_bf16(oacc[2 * dp], pa[ks], b0, b1);
        mma_bf16(oacc[2 * dp + 1], pa[ks], b2, b3);
      }
    }
    __syncthreads();                                            // stage kt & 1 may be refilled now
  }
  // row sums across the quad, normalise, store
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 1);
    lrow[r] += __shfl_xor_sync(0xffffffffu, lrow[r], 2);
  }
  const float inv_a = 1.0f / lrow[0], inv_b = 1.0f / lrow[1];
  __nv_bfloat16* obase = o + static_cast<int64_t>(b) * S * ldq + hq * HD;
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    const int c = i * 8 + 2 * t;
    if (row_a < S) *reinterpret_cast<uint32_t*>(obase + row_a * ldq + c) = pack2(oacc[i][0] * inv_a, oacc[i][1] * inv_a);
    if (row_b < S) *reinterpret_cast<uint32_t*>(obase + row_b * ldq + c) = pack2(oacc[i][2] * inv_b, oacc[i][3] * inv_b);
  }
}

// ------------------------------------------------------------------------------ paired form
// Causal attention of the two forwards of a ZO step given as centre and half-difference (see
// model.cu): inputs qc, qd, kc, kd, vc, vd; with s+- = (qc +- qd)(kc +- kd)^T = sc +- sd,
//   sc = qc kc^T + qd kd^T,  sd = qc kd^T + qd kc^T,
//   p+- = exp(sc - m) exp(+-sd):  pc = exp(sc - m) cosh(sd),  pd = exp(sc - m) sinh(sd)   (m >= sc + |sd|),
//   Oc = pc vc + pd vd,  Od = pc vd + pd vc,  lc = sum pc,  ld = sum pd,
//   o+- = (Oc +- Od) / (lc +- ld):  oc = (Oc lc - Od ld) / (lc^2 - ld^2),  od = (Od lc - Oc ld) / (lc^2 - ld^2).
// Nothing is dropped: the result is the exact centre and half-difference of the two attentions, up
// to the rounding of pc, pd to bf16 and the fp32 accumulation.  Same tiling as above with 32-key
// tiles (twice the accumulators); the query tiles stay in shared memory.
constexpr int kKT2 = 32;

// 2^x by the hardware approximation alone (two units in the last place; exp2f adds a rescaling for results
// below 2^-126, which a probability that is rounded to bf16 does not need)
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// cosh(a) and sinh(a).  The half-difference of a score is small against one (it is of the order of eps
// times the score), so both come from their series, good to 1e-7 below |a| = 0.5; beyond that from e^a.
__device__ __forceinline__ void cosh_sinh(float a, float* ch, float* sh) {
  const float a2 = a * a;
  if (a2 < 0.25f) {
    *ch = 1.0f + a2 * (0.5f + a2 * (1.0f / 24.0f + a2 * (1.0f / 720.0f + a2 * (1.0f / 40320.0f))));
    *sh = a * (1.0f + a2 * (1.0f / 6.0f + a2 * (1.0f / 120.0f + a2 * (1.0f / 5040.0f + a2 * (1.0f / 362880.0f)))));
  } else {
    const float u = __expf(a), r = __fdividef(1.0f, u);
    *ch = 0.5f * (u + r);
    *sh = 0.5f * (u - r);
  }
}

template <int HD>
__device__ __forceinline__ void load_tile_async_rows(__nv_bfloat16* dst, const __nv_bfloat16* src, int64_t ld, int rows,
                                                     int valid) {
  constexpr int kChunks = HD / 8;
  for (int i = threadIdx.x; i < rows * kChunks; i += 128) {
    const int r = i / kChunks, c = i % kChunks;
    __nv_bfloat16* d = dst + r * (HD + 8) + c * 8;
    if (r < valid) {
      asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(static_cast<uint32_t>(__cvta_generic_to_shared(d))),
                   "l"(src + r * ld + c * 8)
                   : "memory");
    } else {
      *reinterpret_cast<uint4*>(d) = make_uint4(0u, 0u, 0u, 0u);
    }
  }
}

template <int HD>
__global__ void __launch_bounds__(128, 2)
flash_attn_pair_bf16_kernel(const __nv_bfloat16* __restrict__ q, const __nv_bfloat16* __restrict__ k,
                            const __nv_bfloat16* __restrict__ v, __nv_bfloat16* __restrict__ o, int64_t row0, int S,
                            int H, int Hkv, float scale, float scale_log2e) {
  constexpr int LDS = HD + 8;
  extern __shared__ __align__(16) unsigned char smem_attn[];
  chain_release();
  chain_wait();
  __nv_bfloat16* sQc = reinterpret_cast<__nv_bfloat16*>(smem_attn);
  __nv_bfloat16* sQd = sQc + kQT * LDS;
  __nv_bfloat16* sKV = sQd + kQT * LDS;          // two stages of (Kc, Kd, Vc, Vd), kKT2 rows each

  const int qt = gridDim.x - 1 - blockIdx.x, hq = blockIdx.y, b = blockIdx.z;
  const int hk = hq / (H / Hkv);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int64_t ldq = static_cast<int64_t>(H) * HD, ldk = static_cast<int64_t>(Hkv) * HD;
  const int q0 = qt * kQT;
  const int64_t offq = row0 * ldq, offk = row0 * ldk;           // the half-difference rows
  const __nv_bfloat16* qbase = q + (static_cast<int64_t>(b) * S + q0) * ldq + hq * HD;
  const int n_kt = (((q0 + kQT < S) ? q0 + kQT : S) + kKT2 - 1) / kKT2;
  auto issue_kv = [&](int kt) {
    const int k0 = kt * kKT2;
    const int valid = S - k0 < kKT2 ? S - k0 : kKT2;
    __nv_bfloat16* st = sKV + (kt & 1) * 4 * kKT2 * LDS;
    const __nv_bfloat16* kp = k + (static_cast<int64_t>(b) * S + k0) * ldk + hk * HD;
    const __nv_bfloat16* vp = v + (static_cast<int64_t>(b) * S + k0) * ldk + hk * HD;
    load_tile_async_rows<HD>(st, kp, ldk, kKT2, valid);
    load_tile_async_rows<HD>(st + kKT2 * LDS, kp + offk, ldk, kKT2, valid);
    load_tile_async_rows<HD>(st + 2 * kKT2 * LDS, vp, ldk, kKT2, valid);
    load_tile_async_rows<HD>(st + 3 * kKT2 * LDS, vp + offk, ldk, kKT2, valid);
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  {
    const int valid = S - q0 < kQT ? S - q0 : kQT;
    load_tile_async_rows<HD>(sQc, qbase, ldq, kQT, valid);
    load_tile_async_rows<HD>(sQd, qbase + offq, ldq, kQT, valid);
    asm volatile("cp.async.commit_group;" ::: "memory");
  }
  issue_kv(0);

  float oc[HD / 8][4], od[HD / 8][4];
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    oc[i][0] = oc[i][1] = oc[i][2] = oc[i][3] = 0.f;
    od[i][0] = od[i][1] = od[i][2] = od[i][3] = 0.f;
  }
  float mrow[2] = {-INFINITY, -INFINITY}, lc[2] = {0.f, 0.f}, ldr[2] = {0.f, 0.f};
  const int row_a = q0 + warp * 16 + g, row_b = row_a + 8;

  for (int kt = 0; kt < n_kt; ++kt) {
    const int k0 = kt * kKT2;
    if (kt + 1 < n_kt) {
      issue_kv(kt + 1);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
    const __nv_bfloat16* sKc = sKV + (kt & 1) * 4 * kKT2 * LDS;
    const __nv_bfloat16* sKd = sKc + kKT2 * LDS;
    const __nv_bfloat16* sVc = sKd + kKT2 * LDS;
    const __nv_bfloat16* sVd = sVc + kKT2 * LDS;

    float sc[kKT2 / 8][4], sd[kKT2 / 8][4];
#pragma unroll
    for (int i = 0; i < kKT2 / 8; ++i) {
      sc[i][0] = sc[i][1] = sc[i][2] = sc[i][3] = 0.f;
      sd[i][0] = sd[i][1] = sd[i][2] = sd[i][3] = 0.f;
    }
#pragma unroll
    for (int ks = 0; ks < HD / 16; ++ks) {
      uint32_t ac[4], ad[4];
      const int qoff = (warp * 16 + (lane & 15)) * LDS + ks * 16 + (lane >> 4) * 8;
      ldsm_x4(static_cast<uint32_t>(__cvta_generic_to_shared(sQc + qoff)), ac[0], ac[1], ac[2], ac[3]);
      ldsm_x4(static_cast<uint32_t>(__cvta_generic_to_shared(sQd + qoff)), ad[0], ad[1], ad[2], ad[3]);
#pragma unroll
      for (int np = 0; np < kKT2 / 16; ++np) {
        const int koff = (np * 16 + (lane & 7) + (lane >> 4) * 8) * LDS + ks * 16 + ((lane >> 3) & 1) * 8;
        uint32_t b0, b1, b2, b3, d0, d1, d2, d3;
        ldsm_x4(static_cast<uint32_t>(__cvta_generic_to_shared(sKc + koff)), b0, b1, b2, b3);
        ldsm_x4(static_cast<uint32_t>(__cvta_generic_to_shared(sKd + koff)), d0, d1, d2, d3);
        mma_bf16(sc[2 * np], ac, b0, b1);
        mma_bf16(sc[2 * np + 1], ac, b2, b3);
        mma_bf16(sc[2 * np], ad, d0, d1);
        mma_bf16(sc[2 * np + 1], ad, d2, d3);
        mma_bf16(sd[2 * np], ac, d0, d1);
        mma_bf16(sd[2 * np + 1], ac, d2, d3);
        mma_bf16(sd[2 * np], ad, b0, b1);
        mma_bf16(sd[2 * np + 1], ad, b2, b3);
      }
    }
    // causal mask and keys beyond the sequence
    if (k0 + kKT2 > q0 || k0 + kKT2 > S) {
#pragma unroll
      for (int i = 0; i < kKT2 / 8; ++i) {
        const int c = k0 + i * 8 + 2 * t;
        if (c > row_a || c >= S) { sc[i][0] = -INFINITY; sd[i][0] = 0.f; }
        if (c + 1 > row_a || c + 1 >= S) { sc[i][1] = -INFINITY; sd[i][1] = 0.f; }
        if (c > row_b || c >= S) { sc[i][2] = -INFINITY; sd[i][2] = 0.f; }
        if (c + 1 > row_b || c + 1 >= S) { sc[i][3] = -INFINITY; sd[i][3] = 0.f; }
      }
    }
    // reference value per row: >= sc + |sd| of every key seen so far (raw score units)
    float mx[2] = {mrow[0], mrow[1]};
#pragma unroll
    for (int i = 0; i < kKT2 / 8; ++i) {
      mx[0] = fmaxf(mx[0], fmaxf(sc[i][0] + fabsf(sd[i][0]), sc[i][1] + fabsf(sd[i][1])));
      mx[1] = fmaxf(mx[1], fmaxf(sc[i][2] + fabsf(sd[i][2]), sc[i][3] + fabsf(sd[i][3])));
    }
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 1));
      mx[r] = fmaxf(mx[r], __shfl_xor_sync(0xffffffffu, mx[r], 2));
    }
    float corr[2], msc[2];
#pragma unroll
    for (int r = 0; r < 2; ++r) {
      msc[r] = (mx[r] == -INFINITY) ? 0.f : mx[r] * scale_log2e;
      corr[r] = (mrow[r] == -INFINITY) ? 0.f : exp2f(mrow[r] * scale_log2e - msc[r]);
      mrow[r] = mx[r];
      lc[r] *= corr[r];
      ldr[r] *= corr[r];
    }
    uint32_t pac[kKT2 / 16][4], pad[kKT2 / 16][4];
#pragma unroll
    for (int i = 0; i < kKT2 / 8; ++i) {
      float pc4[4], pd4[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float e = ex2_approx(sc[i][j] * scale_log2e - msc[j >> 1]);
        float ch, sh;
        cosh_sinh(sd[i][j] * scale, &ch, &sh);
        pc4[j] = e * ch;
        pd4[j] = e * sh;
      }
      lc[0] += pc4[0] + pc4[1];
      lc[1] += pc4[2] + pc4[3];
      ldr[0] += pd4[0] + pd4[1];
      ldr[1] += pd4[2] + pd4[3];
      pac[i >> 1][(i & 1) * 2 + 0] = pack2(pc4[0], pc4[1]);
      pac[i >> 1][(i & 1) * 2 + 1] = pack2(pc4[2], pc4[3]);
      pad[i >> 1][(i & 1) * 2 + 0] = pack2(pd4[0], pd4[1]);
      pad[i >> 1][(i & 1) * 2 + 1] = pack2(pd4[2], pd4[3]);
    }
#pragma unroll
    for (int i = 0; i < HD / 8; ++i) {
      oc[i][0] *= corr[0]; oc[i][1] *= corr[0]; oc[i][2] *= corr[1]; oc[i][3] *= corr[1];
      od[i][0] *= corr[0]; od[i][1] *= corr[0]; od[i][2] *= corr[1]; od[i][3] *= corr[1];
    }
#pragma unroll
    for (int ks = 0; ks < kKT2 / 16; ++ks) {
#pragma unroll
      for (int dp = 0; dp < HD / 16; ++dp) {
        const int voff = (ks * 16 + (lane & 7) + ((lane >> 3) & 1) * 8) * LDS + dp * 16 + (lane >> 4) * 8;
        uint32_t b0, b1, b2, b3, d0, d1, d2, d3;
        ldsm_x4_trans(static_cast<uint32_t>(__cvta_generic_to_shared(sVc + voff)), b0, b1, b2, b3);
        ldsm_x4_trans(static_cast<uint32_t>(__cvta_generic_to_shared(sVd + voff)), d0, d1, d2, d3);
        mma_bf16(oc[2 * dp], pac[ks], b0, b1);
        mma_bf16(oc[2 * dp + 1], pac[ks], b2, b3);
        mma_bf16(oc[2 * dp], pad[ks], d0, d1);
        mma_bf16(oc[2 * dp + 1], pad[ks], d2, d3);
        mma_bf16(od[2 * dp], pac[ks], d0, d1);
        mma_bf16(od[2 * dp + 1], pac[ks], d2, d3);
        mma_bf16(od[2 * dp], pad[ks], b0, b1);
        mma_bf16(od[2 * dp + 1], pad[ks], b2, b3);
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int r = 0; r < 2; ++r) {
    lc[r] += __shfl_xor_sync(0xffffffffu, lc[r], 1);
    lc[r] += __shfl_xor_sync(0xffffffffu, lc[r], 2);
    ldr[r] += __shfl_xor_sync(0xffffffffu, ldr[r], 1);
    ldr[r] += __shfl_xor_sync(0xffffffffu, ldr[r], 2);
  }
  const float inv_a = 1.0f / (lc[0] * lc[0] - ldr[0] * ldr[0]), inv_b = 1.0f / (lc[1] * lc[1] - ldr[1] * ldr[1]);
  __nv_bfloat16* obase = o + static_cast<int64_t>(b) * S * ldq + hq * HD;
#pragma unroll
  for (int i = 0; i < HD / 8; ++i) {
    const int c = i * 8 + 2 * t;
    if (row_a < S) {
      __nv_bfloat16* p = obase + row_a * ldq + c;
      *reinterpret_cast<uint32_t*>(p) = pack2((oc[i][0] * lc[0] - od[i][0] * ldr[0]) * inv_a, (oc[i][1] * lc[0] - od[i][1] * ldr[0]) * inv_a);
      *reinterpret_cast<uint32_t*>(p + offq) = pack2((od[i][0] * lc[0] - oc[i][0] * ldr[0]) * inv_a, (od[i][1] * lc[0] - oc[i][1] * ldr[0]) * inv_a);
    }
    if (row_b < S) {
      __nv_bfloat16* p = obase + row_b * ldq + c;
      *reinterpret_cast<uint32_t*>(p) = pack2((oc[i][2] * lc[1] - od[i][2] * ldr[1]) * inv_b, (oc[i][3] * lc[1] - od[i][3] * ldr[1]) * inv_b);
      *reinterpret_cast<uint32_t*>(p + offq) = pack2((od[i][2] * lc[1] - oc[i][2] * ldr[1]) * inv_b, (od[i][3] * lc[1] - oc[i][3] * ldr[1]) * inv_b);
    }
  }
}

}  // namespace

szo_status launch_flash_attention_bf16(const void* q, const void* k, const void* v, void* o, int B, int S, int H,
                                       int Hkv, int hd, cudaStream_t st) {
  SZO_REQUIRE(hd == 64 || hd == 128, SZO_ERR_UNSUPPORTED, "head dimension must be 64 or 128");
  const float scale_log2e = 1.4426950408889634f / sqrtf(static_cast<float>(hd));
  dim3 grid(static_cast<unsigned>(ceil_div(S, kQT)), H, B);
  const size_t smem = static_cast<size_t>(4) * 64 * (hd + 8) * 2;      // two (K, V) stages; Q borrows one slot
  auto* qb = static_cast<const __nv_bfloat16*>(q);
  auto* kb = static_cast<const __nv_bfloat16*>(k);
  auto* vb = static_cast<const __nv_bfloat16*>(v);
  auto* ob = static_cast<__nv_bfloat16*>(o);
  if (hd == 64) {
    static bool configured64 = false;
    if (!configured64) {
      SZO_CHECK_CUDA(cudaFuncSetAttribute(flash_attn_bf16_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem)));
      configured64 = true;
    }
    flash_attn_bf16_kernel<64><<<grid, 128, smem, st>>>(qb, kb, vb, ob, S, H, Hkv, scale_log2e);
  } else {
    static bool configured = false;
    if (!configured) {
      SZO_CHECK_CUDA(cudaFuncSetAttribute(flash_attn_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          static_cast<int>(smem)));
      configured = true;
    }
    flash_attn_bf16_kernel<128><<<grid, 128, smem, st>>>(qb, kb, vb, ob, S, H, Hkv, scale_log2e);
  }
  count_launch();
  SZO_CHECK_LAUNCH("flash_attn_bf16_kernel");
  return SZO_OK;
}

}  // namespace szo

namespace szo {

// Paired form: every buffer holds the B*S centre rows first and the half-difference rows from row
// `row0` on.
szo_status launch_flash_attention_pair_bf16(const void* q, const void* k, const void* v, void* o, int64_t row0, int B,
                                            int S, int H, int Hkv, int hd, cudaStream_t st) {
  SZO_REQUIRE(hd == 64 || hd == 128, SZO_ERR_UNSUPPORTED, "head dimension must be 64 or 128");
  const float scale = 1.0f / sqrtf(static_cast<float>(hd));
  const float scale_log2e = 1.4426950408889634f * scale;
  dim3 grid(static_cast<unsigned>(ceil_div(S, kQT)), H, B);
  const size_t smem = static_cast<size_t>(2 * kQT + 8 * kKT2) * (hd + 8) * 2;
  auto* qb = static_cast<const __nv_bfloat16*>(q);
  auto* kb = static_cast<const __nv_bfloat16*>(k);
  auto* vb = static_cast<const __nv_bfloat16*>(v);
  auto* ob = static_cast<__nv_bfloat16*>(o);
  // (the attribute is per device; setting it before every launch costs a host call, no device work)
  if (hd == 64) {
    SZO_CHECK_CUDA(cudaFuncSetAttribute(flash_attn_pair_bf16_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)));
    SZO_CHECK_CUDA(launch_maybe_chained(flash_attn_pair_bf16_kernel<64>, grid, dim3(128), smem, st, step_chained(), qb, kb, vb, ob, row0,
                                        S, H, Hkv, scale, scale_log2e));
  } else {
    SZO_CHECK_CUDA(cudaFuncSetAttribute(flash_attn_pair_bf16_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        static_cast<int>(smem)));
    SZO_CHECK_CUDA(launch_maybe_chained(flash_attn_pair_bf16_kernel<128>, grid, dim3(128), smem, st, step_chained(), qb, kb, vb, ob, row0,
                                        S, H, Hkv, scale, scale_log2e));
  }
  count_launch();
  SZO_CHECK_LAUNCH("flash_attn_pair_bf16_kernel");
  return SZO_OK;
}

}  // namespace szo
