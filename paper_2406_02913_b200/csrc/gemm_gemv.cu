// Weight-streaming form of the decomposed linear for one or two tokens (a token-generation step):
//   y[m, n] = sum_k x[m,k] * Dequantize(Q)[n,k] + sum_{(n,c) in mask} x[m,c] * S[n,c] + bias[n]
// (appendix "Implementation of Sparse Operations in Linear Layers": the SparseAddMM order, which the
// paper finds the faster one for token generation).  With so few tokens all activations of a row of
// x fit the shared memory of every CTA, so nothing has to be split along K between CTAs and no CTA
// waits for another (the 16-token kernel of gemm_skinny.cu meets in a cluster once per 128 weight
// rows; at one token that rendezvous and the start-up before it are most of its time):
//   * persistent CTAs take 16 weight rows (one MMA row block) of one matrix and all of K at a time; the
//     activations are staged once per CTA; seven weight warps split K in runs of 128-column steps;
//   * every lane reads its own 16 bytes of codes per weight row and step straight from global memory
//     in the fragment layout (the 16 rows of a k-block are 512 contiguous bytes of the tiled codes: one
//     coalesced 128-bit load per warp), four steps ahead in registers, across row groups (the stream
//     never drains) and from the first instruction on, before the activations are even staged.
//     (Bulk copies of 512 bytes into a ring in shared memory were tried first: the copy engine took
//     about 36 ns per copy whatever its size, 16 us for the 66 000 copies of an 11008 x 4096 matrix.)
//   * the product is the group form of the 16-token kernel: m16n8k16 MMAs of (128 + code) as bf16
//     against the tokens, scale and zero applied once per 128-column step to the fp32 sums,
//     sum_k x_k (q_k s + z) = s sum_k x_k (128 + q_k) + (z - 128 s) sum_k x_k;
//   * the eighth warp forms the sparse term of the 16 rows in fp32 (row pointers two row groups
//     ahead, entries and values one ahead, activations from shared memory), then adds the weight
//     warps' partial sums in warp order, the sparse term and the bias, and stores y; the partial
//     sums are double-buffered, so the weight warps never wait for it.
// One launch serves up to three matrices that read the same activations (q/k/v, gate/up).  The
// activations may be formed while they are staged: silu(x) * x_mul (the gated MLP's product), or the
// normalised residual stream (FusedNorm in linear.cuh: residual add, RMSNorm or LayerNorm).
// Quantization groups must be multiples of 128 columns.
// Codes into a per-row table of 16 values (the non-uniform 4-bit format) take the same kernel: the
// tables of the 16 rows (512 bytes as bf16) travel with every step in the registers that otherwise
// carry (scale, zero), are put into the warp's own shared memory when a row group begins, and every
// code is looked up there (one 2-byte read of shared memory per code instead of half an AND-OR).
// The kernel waits on nothing but its own block barriers.
#include <cstdlib>
#include <mutex>

#include "tc_common.cuh"

namespace szo {

namespace {

constexpr int kGvRows = 16;          // weight rows per CTA
constexpr int kGvWarps = 7;          // weight warps; the eighth forms the sparse term and the final sums
                                     // (eight warps: two per scheduler and CTA, 128 registers each with two CTAs per SM)
constexpr int kGvThreads = (kGvWarps + 1) * 32;
constexpr int kGvStepK = 128;        // columns per step
constexpr int kGvDepth = 4;          // steps in flight per warp (registers)
constexpr int kGvMaxTok = 2;         // more tokens: the 16-token kernel (staging four rows of x per CTA costs more than its rendezvous)
constexpr int kGvPad = 32;           // elements added to a token row in shared memory
constexpr int kGvTabStride = 48;     // bytes per row of a warp's table block in shared memory (32 used)

struct GemvSub {
  const uint8_t* codes_tiled;
  const float2* sz;
  const __nv_bfloat16* lut; // [Npad][16] (table-coded weights), else NULL
  int64_t Npad;
  const int32_t* row_ptr;   // NULL: no sparse entries
  const int32_t* ent_col;
  const float* S;
  const float* bias;
  void* y;
  int64_t N;
  int cta_begin;            // number of this matrix's first CTA
};
struct GemvArgs {
  GemvSub sub[3];
  int n;
  const __nv_bfloat16* x;
  const __nv_bfloat16* x_mul;   // not NULL: the activations are silu(x) * x_mul
  FusedNorm norm;               // h_in not NULL: the activations are the normalised residual stream (linear.cuh)
  int M;
  int64_t K;
  int G;
};

// Position of the 16-byte chunk c (columns 8c .. 8c+7) of a token row: inside a 128-column step lane
// t of the MMA works on chunks 4t .. 4t+3, one per turn; chunk 4t+w sits at 4w+t, so that the four
// lanes' chunks of a turn are side by side.
__device__ __forceinline__ int gv_chunk_pos(int c) { return (c & ~15) | ((c & 3) << 2) | ((c >> 2) & 3); }

// (a & b) | c in one instruction (written out: the compiler makes three of the C++ expression)
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// D = A B
__device__ __forceinline__ void gv_mma_new(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}
// D = A B + D
__device__ __forceinline__ void gv_mma_acc(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <bool kBf16Tables>
__device__ __forceinline__ float2 gv_sz_f32(float2 p) {
  if constexpr (kBf16Tables)
    return make_float2(__uint_as_float(__float_as_uint(p.x) & 0xFFFF0000u), __uint_as_float(__float_as_uint(p.y) & 0xFFFF0000u));
  else
    return p;
}

// silu(g) * u of eight bf16 pairs, each product rounded to bf16.  Every CTA forms all K products, so
// the fast exponential and division are used (relative error near 2^-21, far below the bf16 rounding
// of the result; the model's own SiLU-gating kernel uses the exact ones)
__device__ __forceinline__ uint4 gv_silu_mul(uint4 g, uint4 u) {
  const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float g0 = __uint_as_float(gw[i] << 16), g1 = __uint_as_float(gw[i] & 0xFFFF0000u);
    const float u0 = __uint_as_float(uw[i] << 16), u1 = __uint_as_float(uw[i] & 0xFFFF0000u);
    const __nv_bfloat162 r = __floats2bfloat162_rn(__fdividef(g0, 1.0f + __expf(-g0)) * u0, __fdividef(g1, 1.0f + __expf(-g1)) * u1);
    o[i] = *reinterpret_cast<const uint32_t*>(&r);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

// Block-wide sum of 256 threads with the fixed tree of the model's norm kernel: shuffles inside a warp,
// then the eight warps' values in warp order
__device__ __forceinline__ float gv_block_sum(float v, float* scratch) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if ((threadIdx.x & 31) == 0) scratch[threadIdx.x >> 5] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int i = 0; i < kGvThreads / 32; ++i) t += scratch[i];
  return t;
}

// streaming 128-bit load: the weights are read once
__device__ __forceinline__ uint4 gv_ld_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}

// Named barriers: 1 = everybody (staging); 2 + buf = "the partial sums of buffer buf are written" (the
// weight warps arrive, the eighth warp waits); 4 + buf = "buffer buf has been read" (the other way round).
__device__ __forceinline__ void gv_bar_sync(int id) { asm volatile("bar.sync %0, %1;" ::"r"(id), "n"(kGvThreads) : "memory"); }
__device__ __forceinline__ void gv_bar_arrive(int id) {
  __threadfence_block();
  asm volatile("bar.arrive %0, %1;" ::"r"(id), "n"(kGvThreads) : "memory");
}

// Grid: persistent CTAs; CTA b takes the 16-row groups b, b + gridDim.x, ... of the `total` groups of
// all matrices (numbered in matrix order).
template <bool kLut, bool kBf16Tables, typename TY>
__global__ void __launch_bounds__(kGvThreads, 2) szo_linear_gemv_kernel(const __grid_constant__ GemvArgs a, int total) {
  extern __shared__ __align__(128) unsigned char smem_gv[];
  __shared__ float part[2][kGvWarps][kGvRows * 8];        // [buffer][warp][row][token]
  __shared__ __align__(16) unsigned char wtab_s[kLut ? kGvWarps * kGvRows * kGvTabStride : 16];   // per warp: the 16 rows' tables

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int M = a.M, G = a.G;
  const int64_t K = a.K;
  const int n_steps = static_cast<int>(K / kGvStepK);
  const int ld = static_cast<int>(K) + kGvPad;
  const int stride = static_cast<int>(gridDim.x);
  __nv_bfloat16* sx = reinterpret_cast<__nv_bfloat16*>(smem_gv);                                       // [M][ld]
  float* xsum = reinterpret_cast<float*>(sx + static_cast<size_t>(M) * ld);                            // [n_steps][8]
  auto sub_of = [&](int grp) -> const GemvSub& {
    return a.sub[(a.n > 1 && grp >= a.sub[1].cta_begin) + (a.n > 2 && grp >= a.sub[2].cta_begin)];
  };

  chain_release();
  // ---------------------------------------------------------------- weight warps: start the stream
  const int s_begin = warp < kGvWarps ? warp * n_steps / kGvWarps : 0;
  const int n_my = warp < kGvWarps ? (warp + 1) * n_steps / kGvWarps - s_begin : 0;
  // fetch cursor: step fj of group fg, with running pointers to this lane's 16 bytes of row g in k-block
  // (t >> 1) of that step (row g + 8 is 256 bytes further) and to its (scale, zero) entry (rows g, g + 8)
  const int steps_per_qgroup = kLut ? 1 : G / kGvStepK; // steps that share one (scale, zero) entry
  int fg = static_cast<int>(blockIdx.x), fj = 0, fzc = 0;
  const uint8_t* fc = nullptr;
  const float2* fz = nullptr;
  int64_t fNpad = 0;
  auto set_fetch_group = [&]() {
    const GemvSub& sb = sub_of(fg);
    const int r16 = fg - sb.cta_begin;
    fc = sb.codes_tiled + (static_cast<int64_t>(r16 >> 3) * (K / 64) + 2 * s_begin + (t >> 1)) * 4096 + (r16 & 7) * 512 +
         g * 32 + (t & 1) * 16;
    fNpad = sb.Npad;
    if constexpr (kLut) {
      // lane l carries half l & 1 of the table of row l >> 1 (16 bytes)
      fz = reinterpret_cast<const float2*>(sb.lut + (static_cast<int64_t>(r16) * kGvRows + (lane >> 1)) * 16 + (lane & 1) * 8);
    } else {
      fz = sb.sz + static_cast<int64_t>(r16) * kGvRows + g + static_cast<int64_t>(s_begin / steps_per_qgroup) * fNpad;
      fzc = s_begin % steps_per_qgroup;
    }
  };
  const bool one_step_groups = steps_per_qgroup == 1;     // G = 128: a new (scale, zero) entry every step
  auto fetch = [&](uint4& wa, uint4& wb, float2& pa, float2& pb) {     // the step under the cursor, then advance it
    if (fg < total) {
      // (addresses from the step counter: a wide multiply-add each on the FMA pipe, where running pointers and
      // their counters are four or five instructions on the ALU pipe, the busy one)
      const uint8_t* src = fc + static_cast<int64_t>(fj) * (2 * 4096);
      wa = gv_ld_stream(src);
      wb = gv_ld_stream(src + 8 * 32);
      if constexpr (kLut) {
        const float4 tb = __ldg(reinterpret_cast<const float4*>(fz));     // (L2 after the group's first step)
        pa = make_float2(tb.x, tb.y);
        pb = make_float2(tb.z, tb.w);
      } else {
        const float2* z = fz + static_cast<int64_t>(one_step_groups ? fj : (fzc + fj) / steps_per_qgroup) * fNpad;
        pa = __ldg(z);
        pb = __ldg(z + 8);
      }
      if (++fj == n_my) {
        fj = 0;
        fg += stride;
        if (fg < total) set_fetch_group();
      }
    }
  };
  uint4 rwa[kGvDepth], rwb[kGvDepth];
  float2 rpa[kGvDepth], rpb[kGvDepth];
  if (warp < kGvWarps && n_my > 0) {
    if (fg < total) set_fetch_group();
#pragma unroll
    for (int d = 0; d < kGvDepth; ++d) {
      rwa[d] = rwb[d] = make_uint4(0u, 0u, 0u, 0u);
      rpa[d] = rpb[d] = make_float2(0.f, 0.f);
      fetch(rwa[d], rwb[d], rpa[d], rpb[d]);
    }
  }
  // ---------------------------------------------------------------- eighth warp: row pointers and entries ahead
  // lane = (row, token parity): tokens sp_mh and sp_mh + 2.  Row pointers are fetched two groups ahead,
  // the first kPre entries of a row one group ahead.
  constexpr int kPre = 8;
  const int sp_row = lane & 15, sp_mh = lane >> 4;
  const bool sp_tok = sp_mh < M;
  auto load_rp = [&](int grp, int32_t& rb, int32_t& re) {
    rb = re = 0;
    if (grp < total && sp_tok) {
      const GemvSub& sb = sub_of(grp);
      if (sb.row_ptr != nullptr) {
        const int64_t n = static_cast<int64_t>(grp - sb.cta_begin) * kGvRows + sp_row, N = sb.N;
        rb = sb.row_ptr[(n < N) ? n : N];                   // rows beyond N: empty
        re = sb.row_ptr[(n + 1 < N) ? n + 1 : N];
      }
    }
  };
  auto load_entries = [&](int grp, int32_t e, int32_t re, int (&col)[kPre], float (&val)[kPre]) {
    const GemvSub& sb = sub_of(grp < total ? grp : 0);
#pragma unroll
    for (int q = 0; q < kPre; ++q) {
      col[q] = (e + q < re) ? sb.ent_col[e + q] : -1;
      val[q] = (e + q < re) ? sb.S[e + q] : 0.f;
    }
  };
  // ---------------------------------------------------------------- everybody: stage the activations, once
  chain_wait();          // the weights above are nobody's output; the activations are the predecessor's
  if (a.norm.h_in != nullptr) {
    // residual add and norm (add_norm_kernel's arithmetic and reduction tree, 256 threads): v goes
    // through shared memory as fp32, since the thread that normalises a 16-byte chunk is not the
    // one that summed it
    float* vs = xsum + n_steps * 8;                       // [M][K]
    float* scratch = &part[0][0][0];
    const int nv = static_cast<int>(K / 4);
    for (int m = 0; m < M; ++m) {
      const float4* hp = reinterpret_cast<const float4*>(a.norm.h_in + static_cast<int64_t>(m) * K);
      float sum = 0.f;
      for (int c = threadIdx.x; c < nv; c += kGvThreads) {
        float4 v = hp[c];
        if (a.norm.y_add != nullptr) {
          const uint2 raw = *reinterpret_cast<const uint2*>(a.norm.y_add + static_cast<int64_t>(m) * K + c * 4);
          v.x += __uint_as_float(raw.x << 16);
          v.y += __uint_as_float(raw.x & 0xFFFF0000u);
          v.z += __uint_as_float(raw.y << 16);
          v.w += __uint_as_float(raw.y & 0xFFFF0000u);
        }
        reinterpret_cast<float4*>(vs + static_cast<size_t>(m) * K)[c] = v;
        if (blockIdx.x == 0) reinterpret_cast<float4*>(a.norm.h_out + static_cast<int64_t>(m) * K)[c] = v;
        sum += (v.x + v.y) + (v.z + v.w);
      }
      const float mu = a.norm.layer_norm ? gv_block_sum(sum, scratch) / static_cast<float>(K) : 0.f;
      float q = 0.f;
      for (int c = threadIdx.x; c < nv; c += kGvThreads) {
        const float4 v = reinterpret_cast<const float4*>(vs + static_cast<size_t>(m) * K)[c];
        const float a0 = v.x - mu, a1 = v.y - mu, a2 = v.z - mu, a3 = v.w - mu;
        q += (a0 * a0 + a1 * a1) + (a2 * a2 + a3 * a3);
      }
      const float var = gv_block_sum(q, scratch) / static_cast<float>(K);
      const float r = 1.0f / sqrtf(var + a.norm.eps);
      for (int c8 = threadIdx.x; c8 < nv / 2; c8 += kGvThreads) {        // one 16-byte chunk of bf16
        uint32_t o[4];
#pragma unroll
        for (int hx = 0; hx < 2; ++hx) {
          const int c = c8 * 2 + hx;
          const float4 v = reinterpret_cast<const float4*>(vs + static_cast<size_t>(m) * K)[c];
          const float4 gm = reinterpret_cast<const float4*>(a.norm.gamma)[c];
          float4 bt = make_float4(0.f, 0.f, 0.f, 0.f);
          if (a.norm.beta != nullptr) bt = reinterpret_cast<const float4*>(a.norm.beta)[c];
          const __nv_bfloat162 lo = __floats2bfloat162_rn((v.x - mu) * r * gm.x + bt.x, (v.y - mu) * r * gm.y + bt.y);
          const __nv_bfloat162 hi = __floats2bfloat162_rn((v.z - mu) * r * gm.z + bt.z, (v.w - mu) * r * gm.w + bt.w);
          o[2 * hx] = *reinterpret_cast<const uint32_t*>(&lo);
          o[2 * hx + 1] = *reinterpret_cast<const uint32_t*>(&hi);
        }
        *reinterpret_cast<uint4*>(sx + static_cast<size_t>(m) * ld + gv_chunk_pos(c8) * 8) = make_uint4(o[0], o[1], o[2], o[3]);
      }
    }
  } else {
    // (all loads of a batch first: a chunk is one round trip to L2, and there are one to five batches)
    const int chunks = static_cast<int>(K / 8), total_chunks = chunks * M;
    constexpr int kBatch = 4;
    for (int base = threadIdx.x; base < total_chunks; base += kGvThreads * kBatch) {
      uint4 v[kBatch], u[kBatch];
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int idx = base + q * kGvThreads;
        if (idx < total_chunks) {
          v[q] = __ldg(reinterpret_cast<const uint4*>(a.x) + idx);            // row m = idx / chunks starts at m * chunks
          if (a.x_mul != nullptr) u[q] = __ldg(reinterpret_cast<const uint4*>(a.x_mul) + idx);
        }
      }
#pragma unroll
      for (int q = 0; q < kBatch; ++q) {
        const int idx = base + q * kGvThreads;
        if (idx < total_chunks) {
          const int m = idx / chunks, c = idx - m * chunks;
          if (a.x_mul != nullptr) v[q] = gv_silu_mul(v[q], u[q]);
          *reinterpret_cast<uint4*>(sx + static_cast<size_t>(m) * ld + gv_chunk_pos(c) * 8) = v[q];
        }
      }
    }
  }
  {
    for (int i = threadIdx.x; i < n_steps * 8; i += kGvThreads)
      if ((i & 7) >= M) xsum[i] = 0.f;
    gv_bar_sync(1);
    // sum of a token's activations over each step: half a warp per (step, token), a fixed shuffle tree
    for (int i0 = warp * 2; i0 < n_steps * M; i0 += (kGvThreads / 32) * 2) {
      const int i = i0 + (lane >> 4);
      float acc = 0.f;
      if (i < n_steps * M) {
        const int st = i / M, m = i % M;
        const uint4 v = *reinterpret_cast<const uint4*>(sx + static_cast<size_t>(m) * ld + st * kGvStepK + (lane & 15) * 8);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) acc += __uint_as_float(w[e] << 16) + __uint_as_float(w[e] & 0xFFFF0000u);
      }
#pragma unroll
      for (int o = 8; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
      if (i < n_steps * M && (lane & 15) == 0) xsum[(i / M) * 8 + (i % M)] = acc;
    }
    gv_bar_sync(1);
  }

  if (warp < kGvWarps) {
    // -------------------------------------------------------------- weight warps
    // The steps of all of this CTA's row groups form one sequence; step q of it sits in register slot
    // q % kGvDepth (the loop is unrolled over the slots, a row group may end in any of them).
    int it = 0, cj = 0, grp = static_cast<int>(blockIdx.x);
    float tot[4] = {0.f, 0.f, 0.f, 0.f};
    // token g of the MMA's eight; where there is none, token 0 again: those columns of the result are never read
    const __nv_bfloat16* xs0 = sx + static_cast<size_t>(g < M ? g : 0) * ld + s_begin * kGvStepK + t * 8;
    const float* xsum0 = xsum + s_begin * 8 + 2 * t;                                              // tokens 2t, 2t+1
    while (grp < total) {
#pragma unroll
      for (int d = 0; d < kGvDepth; ++d) {
        if (grp < total) {
          const uint4 wa = rwa[d], wb = rwb[d];
          const float2 pa = rpa[d], pb = rpb[d];
          const uint32_t qa[4] = {wa.x, wa.y, wa.z, wa.w}, qb[4] = {wb.x, wb.y, wb.z, wb.w};
          const __nv_bfloat16* xs = xs0 + cj * kGvStepK;
          float accq[2][4];                                 // even and odd words: two shorter chains
          if constexpr (kLut) {
            unsigned char* wtab = wtab_s + warp * (kGvRows * kGvTabStride);
            if (cj == 0) {                                  // a new row group: its tables into the warp's block
              __syncwarp();
              *reinterpret_cast<float4*>(wtab + (lane >> 1) * kGvTabStride + (lane & 1) * 16) = make_float4(pa.x, pa.y, pb.x, pb.y);
              __syncwarp();
            }
            const unsigned char* ta = wtab + g * kGvTabStride;          // row g; row g + 8 is 8 strides further
            auto look = [&](const unsigned char* tab, uint32_t q, int lo_shift) -> uint32_t {
              // bf16 pair (table[nibble at lo_shift], table[nibble at lo_shift + 16]); byte offset = 2 * nibble
              const uint32_t o0 = lo_shift == 0 ? (q << 1) & 0x1Eu : (q >> (lo_shift - 1)) & 0x1Eu;
              const uint32_t o1 = (q >> (lo_shift + 15)) & 0x1Eu;
              const uint32_t v0 = *reinterpret_cast<const unsigned short*>(tab + o0);
              const uint32_t v1 = *reinterpret_cast<const unsigned short*>(tab + o1);
              return v0 | (v1 << 16);
            };
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {
              uint32_t a0[4], a1[4];
              a0[0] = look(ta, qa[wd], 0);
              a0[1] = look(ta + 8 * kGvTabStride, qb[wd], 0);
              a0[2] = look(ta, qa[wd], 4);
              a0[3] = look(ta + 8 * kGvTabStride, qb[wd], 4);
              a1[0] = look(ta, qa[wd], 8);
              a1[1] = look(ta + 8 * kGvTabStride, qb[wd], 8);
              a1[2] = look(ta, qa[wd], 12);
              a1[3] = look(ta + 8 * kGvTabStride, qb[wd], 12);
              const uint4 xv = *reinterpret_cast<const uint4*>(xs + wd * 32);
              if (wd < 2) gv_mma_new(accq[wd & 1], a0, xv.x, xv.y);
              else gv_mma_acc(accq[wd & 1], a0, xv.x, xv.y);
              gv_mma_acc(accq[wd & 1], a1, xv.z, xv.w);
            }
            tot[0] += accq[0][0] + accq[1][0];
            tot[1] += accq[0][1] + accq[1][1];
            tot[2] += accq[0][2] + accq[1][2];
            tot[3] += accq[0][3] + accq[1][3];
          } else {
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {                // one 32-bit word = 8 columns = two k16 MMAs
              uint32_t a0[4], a1[4];
              a0[0] = and_or(qa[wd], 0x000F000Fu, 0x43004300u);
              a0[1] = and_or(qb[wd], 0x000F000Fu, 0x43004300u);
              a0[2] = and_or(qa[wd] >> 4, 0x000F000Fu, 0x43004300u);
              a0[3] = and_or(qb[wd] >> 4, 0x000F000Fu, 0x43004300u);
              a1[0] = and_or(qa[wd] >> 8, 0x000F000Fu, 0x43004300u);
              a1[1] = and_or(qb[wd] >> 8, 0x000F000Fu, 0x43004300u);
              a1[2] = and_or(qa[wd] >> 12, 0x000F000Fu, 0x43004300u);
              a1[3] = and_or(qb[wd] >> 12, 0x000F000Fu, 0x43004300u);
              const uint4 xv = *reinterpret_cast<const uint4*>(xs + wd * 32);
              if (wd < 2) gv_mma_new(accq[wd & 1], a0, xv.x, xv.y);
              else gv_mma_acc(accq[wd & 1], a0, xv.x, xv.y);
              gv_mma_acc(accq[wd & 1], a1, xv.z, xv.w);
            }
            const float2 fa = gv_sz_f32<kBf16Tables>(pa), fb = gv_sz_f32<kBf16Tables>(pb);
            const float za = fmaf(-128.f, fa.x, fa.y), zb = fmaf(-128.f, fb.x, fb.y);
            const float2 xs2 = *reinterpret_cast<const float2*>(xsum0 + cj * 8);
            tot[0] = fmaf(fa.x, accq[0][0] + accq[1][0], fmaf(za, xs2.x, tot[0]));
            tot[1] = fmaf(fa.x, accq[0][1] + accq[1][1], fmaf(za, xs2.y, tot[1]));
            tot[2] = fmaf(fb.x, accq[0][2] + accq[1][2], fmaf(zb, xs2.x, tot[2]));
            tot[3] = fmaf(fb.x, accq[0][3] + accq[1][3], fmaf(zb, xs2.y, tot[3]));
          }
          fetch(rwa[d], rwb[d], rpa[d], rpb[d]);            // (after the slot's last use: no copies of its registers)
          if (++cj == n_my) {                               // the row group is complete
            const int buf = it & 1;
            if (it >= 2) gv_bar_sync(4 + buf);              // the sums of two groups ago have been read
            // accumulator layout: [0], [1] = (row g, tokens 2t, 2t+1); [2], [3] = (row g+8, same tokens)
            float* mine = part[buf][warp] + g * 8 + 2 * t;
            mine[0] = tot[0];
            mine[1] = tot[1];
            mine[8 * 8] = tot[2];
            mine[8 * 8 + 1] = tot[3];
            gv_bar_arrive(2 + buf);
            tot[0] = tot[1] = tot[2] = tot[3] = 0.f;
            cj = 0;
            grp += stride;
            ++it;
          }
        }
      }
    }
  } else {
    // -------------------------------------------------------------- sparse term, sum over the warps, store
    int32_t rb0, re0, rb1, re1;
    int col0[kPre], col1[kPre];
    float val0[kPre], val1[kPre];
    load_rp(static_cast<int>(blockIdx.x), rb0, re0);
    load_rp(static_cast<int>(blockIdx.x) + stride, rb1, re1);
    load_entries(static_cast<int>(blockIdx.x), rb0, re0, col0, val0);
    int it = 0;
    for (int grp = static_cast<int>(blockIdx.x); grp < total; grp += stride, ++it) {
      int32_t rb2, re2;
      load_rp(grp + 2 * stride, rb2, re2);
      load_entries(grp + stride, rb1, re1, col1, val1);
      float sp[2] = {0.f, 0.f};
      for (int32_t e = rb0; e < re0; e += kPre) {
        if (e > rb0) load_entries(grp, e, re0, col0, val0);   // rows with more entries: another round trip
#pragma unroll
        for (int q = 0; q < kPre; ++q) {
          if (col0[q] >= 0) {
            const int pos = gv_chunk_pos(col0[q] >> 3) * 8 + (col0[q] & 7);
            sp[0] = fmaf(__bfloat162float(sx[static_cast<size_t>(sp_mh) * ld + pos]), val0[q], sp[0]);
            if (sp_mh + 2 < M) sp[1] = fmaf(__bfloat162float(sx[static_cast<size_t>(sp_mh + 2) * ld + pos]), val0[q], sp[1]);
          }
        }
      }
      const int buf = it & 1;
      gv_bar_sync(2 + buf);
      const GemvSub& sb = sub_of(grp);
      const int64_t N = sb.N, n = static_cast<int64_t>(grp - sb.cta_begin) * kGvRows + sp_row;
      if (n < N) {
        const float bv = sb.bias != nullptr ? sb.bias[n] : 0.f;
        TY* __restrict__ y = static_cast<TY*>(sb.y);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int m = sp_mh + 2 * h;
          if (m < M) {
            float v = part[buf][0][sp_row * 8 + m];
#pragma unroll
            for (int w = 1; w < kGvWarps; ++w) v += part[buf][w][sp_row * 8 + m];
            v += sp[h] + bv;
            if constexpr (sizeof(TY) == 2) y[static_cast<int64_t>(m) * N + n] = __float2bfloat16_rn(v);
            else y[static_cast<int64_t>(m) * N + n] = v;
          }
        }
      }
      if (grp + 2 * stride < total) gv_bar_arrive(4 + buf);   // (only if the buffer will be written again)
      rb0 = rb1; re0 = re1; rb1 = rb2; re1 = re2;
#pragma unroll
      for (int q = 0; q < kPre; ++q) {
        col0[q] = col1[q];
        val0[q] = val1[q];
      }
    }
  }
}

size_t gemv_dyn_smem(int64_t K, int64_t M, bool norm = false) {
  return static_cast<size_t>(M) * (K + kGvPad) * 2 + static_cast<size_t>(K / kGvStepK) * 8 * sizeof(float) +
         (norm ? static_cast<size_t>(M) * K * sizeof(float) : 0);
}
constexpr size_t kGvMaxDynSmem = 200 * 1024;

template <bool kLut, bool kBf16Tables, typename TY>
szo_status launch_gemv(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                       const float* const* S, void* const* y, cudaStream_t st, bool chained, const FusedNorm* norm) {
  auto kern = szo_linear_gemv_kernel<kLut, kBf16Tables, TY>;
  static bool configured[64] = {false};
  static std::mutex mu;
  int dev = 0;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_REQUIRE(dev >= 0 && dev < 64, SZO_ERR_UNSUPPORTED, "device ordinal %d", dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
      SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kGvMaxDynSmem)));
      configured[dev] = true;
    }
  }
  const szo_linear* p = plans[0];
  GemvArgs a{};
  a.n = n;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.x_mul = static_cast<const __nv_bfloat16*>(x_mul);
  if (norm != nullptr) {
    SZO_REQUIRE(norm->h_in != nullptr && norm->h_out != nullptr && norm->h_in != norm->h_out && norm->gamma != nullptr &&
                    x_mul == nullptr && plans[0]->K <= 8192,
                SZO_ERR_INVALID_ARG, "fused norm: h_in, h_out (different buffers) and gamma are needed, K at most 8192");
    a.norm = *norm;
  }
  a.M = static_cast<int>(M);
  a.K = p->K;
  a.G = p->G;
  int ctas = 0;
  for (int i = 0; i < n; ++i) {
    const szo_linear* q = plans[i];
    a.sub[i] = GemvSub{q->codes_tiled, q->sz, q->lut_bf16, q->Npad, q->nnz > 0 ? q->row_ptr : nullptr, q->ent_col, S[i],
                       q->bias, y[i], q->N, ctas};
    ctas += static_cast<int>(ceil_div(q->N, kGvRows));
  }
  // persistent CTAs: as many as are resident at once (two per SM while the activations leave room)
  const size_t smem = gemv_dyn_smem(p->K, M, norm != nullptr);
  int sms = 148;
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int per_sm = (2 * (smem + 9 * 1024) <= 227 * 1024) ? 2 : 1;
  const int grid = ctas < per_sm * sms ? ctas : per_sm * sms;
  SZO_CHECK_CUDA(launch_maybe_chained(kern, dim3(static_cast<unsigned>(grid)), dim3(kGvThreads), smem, st, chained, a, ctas));
  count_launch();
  SZO_CHECK_LAUNCH("szo_linear_gemv_kernel");
  return SZO_OK;
}

}  // namespace

// int4 plans with groups of a multiple of 128 columns or with per-row tables, at most two tokens, up to
// three matrices with the same K, group size and table type.  SZO_GEMV=0 switches the kernel off (A/B measurement).
bool gemv_applies(const szo_linear* const* plans, int n, int64_t M) {
  static const bool off = [] {
    const char* e = getenv("SZO_GEMV");
    return e != nullptr && e[0] == '0';
  }();
  if (off || n < 1 || n > 3 || M < 1 || M > kGvMaxTok) return false;
  const szo_linear* p = plans[0];
  const bool lut = p->G == -1 && p->lut_bf16 != nullptr;
  if (!(lut || (p->G > 0 && p->G % kGvStepK == 0)) || p->K % kGvStepK != 0 || p->K / kGvStepK < kGvWarps ||
      gemv_dyn_smem(p->K, M) > kGvMaxDynSmem)
    return false;
  for (int i = 0; i < n; ++i)
    if (plans[i]->K != p->K || plans[i]->G != p->G || plans[i]->sz_dtype != p->sz_dtype || plans[i]->codes_tiled == nullptr ||
        (lut && plans[i]->lut_bf16 == nullptr))
      return false;
  return true;
}

szo_status linear_fwd_gemv(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                           const float* const* S_pert, void* const* y, int y_dtype, cudaStream_t st, bool chained,
                           const FusedNorm* norm) {
  SZO_REQUIRE(gemv_applies(plans, n, M), SZO_ERR_UNSUPPORTED, "shapes not covered by the few-token kernel");
  const bool bf = plans[0]->sz_dtype == SZO_BF16;
  if (plans[0]->G == -1) {                    // (the plan's bf16 copy of the tables is read: the tables' own type does not matter)
    if (y_dtype == SZO_F32) return launch_gemv<true, false, float>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
    return launch_gemv<true, false, __nv_bfloat16>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
  }
  if (y_dtype == SZO_F32) {
    if (bf) return launch_gemv<false, true, float>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
    return launch_gemv<false, false, float>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
  }
  if (bf) return launch_gemv<false, true, __nv_bfloat16>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
  return launch_gemv<false, false, __nv_bfloat16>(plans, n, x, x_mul, M, S_pert, y, st, chained, norm);
}

}  // namespace szo
