// Building blocks of the tensor-core kernel and its host side: tile constants, kernel parameters,
// the PTX wrappers (mbarrier, TMA, tcgen05 / TMEM), descriptor encoders and the int4 -> bf16
// conversion of one 32-bit word of codes.
#pragma once
#include <cuda.h>

#include "linear.cuh"

namespace szo {
namespace tc {

constexpr int kBM = 128;           // weight rows per tile (UMMA M)
constexpr int kBK = 64;            // K per stage: 64 bf16 = one 128-byte swizzle row
constexpr int kUmmaK = 16;
constexpr int kATileBytes = kBM * kBK * 2;   // 16 KiB
constexpr int kCodesBytes = kBM * kBK / 2;   // 4 KiB of packed codes per stage
constexpr int kSzBytes = 2048;               // (scale, zero) fp32 pairs: 128 rows x up to 2 groups
constexpr int kRecCap = 128;                 // sparse records of a k-block kept in the shared-memory ring
constexpr long long kWaitLimitCycles = 4000000000ll;   // about 2 s of SM cycles

// One weight matrix of a launch: several linear layers that read the same activations (q/k/v,
// gate/up) are concatenated along their output rows.
struct TcSub {
  const uint8_t* codes;    // tile order: block (128-row tile t, k-block kb) = 4 KiB at (t * nkb + kb) * 4096
  const float2* sz;        // [K/G][Npad]; fp32 (scale, zero), or packed bf16 pairs when kFast
  const int32_t* bucket_ptr;
  const uint2* Sb;         // sparse records (byte offset in the tile, value bits) in bucket order; nullptr: none
  const float* bias;
  void* y;
  int64_t N, Npad;
  int n_rowtiles;          // 128-row tiles that have buckets
  int n_tiles;             // 256-row pair tiles
};

struct TcParams {
  int64_t M, K;
  int G;
  int nkb;                 // K / 64
  int64_t m_tiles, n_tiles;   // 256-token tiles; 256-row pair tiles of all matrices together
  // Tile order.  0: weight tile slowest, token tile fastest (a weight tile meets every token tile while it
  // is hot).  m_band > 0: the token tiles are taken in bands of m_band; inside a band the order is as before.
  // The tokens of a band (m_band x 256 x K bf16) then stay in L2 across the rounds of tiles, at the
  // price of one more pass over the weights per band: with 8192 token rows of K = 4096 the whole token
  // matrix (67 MB) was re-read from DRAM by most rounds (1.6 GB per launch against 0.6 GB algorithmic).
  int m_band;
  int y_f32;
  int relu;                // y = max(y, 0) in the epilogue (the ReLU of an OPT-style MLP after its first matrix)
  int32_t* status;
  int nsub;
  TcSub sub[3];
  // Work units of pair p: full tiles p + lt * n_pairs for lt < full_rounds, then (p < tail_tiles *
  // tail_parts) one unit of the tail: tile full_rounds * n_pairs + p % tail_tiles, k-blocks
  // [tail_kb[part], tail_kb[part + 1]) with part = p / tail_tiles.  With tail_parts > 1 the parts of
  // a tile meet in `partial` (fp32 [tail_tiles][tail_parts][2 ranks][256 tokens][128 rows]); when all
  // are parked (tickets; every cluster of the launch is resident, so the wait is for running code,
  // and it is bounded) each part's CTA adds up, in part order, its share of the tile's tokens and
  // stores y; the last one to finish resets the counters.
  int full_rounds, tail_tiles, tail_parts;
  int tail_kb[5];
  float* partial;
  int32_t* tickets;        // [tail_tiles][2 ranks]: parts of the tile parked so far
  int32_t* tickets_done;   // [tail_tiles][2 ranks]: parts that have finished their share of the sum
  // Paired form of the two forwards of a ZO step (dense mode only).  The token rows hold the centre
  // xc = (x+ + x-)/2 in rows [0, M_c) and the half-difference xd = (x+ - x-)/2 from row pair_row0 (a
  // multiple of 256) on.  With W = RN_bf16(Dequantize(Q) + S) unperturbed,
  //   centre rows:           y = xc W^T + bias
  //   half-difference rows:  y = xd W^T + eps * xc Zbar^T          (Zbar: z at the sensitive entries)
  // so x+- (W +- eps Zbar)^T = (centre) +- (half-difference) up to the term eps xd Zbar^T, which is of
  // relative order eps^2.  This kernel computes the dense products of both kinds of rows in one launch
  // and leaves the bias out of the half-difference rows; the sparse product is added to those rows by
  // pair_cross_kernel after it.
  int64_t pair_row0;       // first half-difference row (0: not a paired launch)
  // pair_ext != 0: the sparse product runs on the tensor cores too.  The weight buffer is [rows][2 K]:
  // W in columns [0, K), eps * Zbar as a dense bf16 matrix in columns [K, 2 K).  A half-difference
  // token tile then runs 2 K / 64 k-blocks: the first K / 64 multiply xd by W, the others multiply the
  // CENTRE rows of the same tokens (token row - pair_row0) by eps * Zbar, into the same accumulator.
  int pair_ext;
};

// Position in a ring of n slots: slot index and the parity of the current pass over the ring.
// Every role keeps running cursors instead of deriving them from the iteration number: the
// producer and MMA roles are single threads, where an integer division per k-block would be a
// large part of the loop.
struct RingPos {
  int idx;
  uint32_t phase;
  __device__ __forceinline__ void advance(int n) {
    if (++idx == n) {
      idx = 0;
      phase ^= 1u;
    }
  }
  // steps <= n slots forward in one go
  __device__ __forceinline__ void advance_by(int steps, int n) {
    idx += steps;
    if (idx >= n) {
      idx -= n;
      phase ^= 1u;
    }
  }
};

// ------------------------------------------------------------------------------ PTX wrappers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// Bounded wait: false when the limit expired or another role already gave up.  Between polls the
// warp sleeps for `backoff_ns` so that waiting roles do not take issue slots from the few threads
// that feed the tensor core; the SM cycle counter bounds the wait (kWaitLimitCycles is about two
// seconds at 2 GHz).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, int32_t* status,
                                          unsigned backoff_ns = 32, long long limit_cycles = kWaitLimitCycles) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  int polls = 0;
  while (true) {
    if (backoff_ns) __nanosleep(backoff_ns);
    if (mbar_try_wait(bar, parity)) return true;
    if ((++polls & 1023) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > limit_cycles) {
        *abort_flag = 1;
        atomicExch(status, static_cast<int32_t>(SZO_ERR_TIMEOUT));
        return false;
      }
    }
  }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}
// L2 eviction priorities: the token matrix is re-read by every round of tiles and should stay, the output
// is written once and should not push it out.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_2d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar,
                                                 uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void st_bf16_hint(__nv_bfloat16* p, __nv_bfloat16 v, uint64_t policy) {
  asm volatile("st.global.L2::cache_hint.b16 [%0], %1, %2;" ::"l"(p), "h"(*reinterpret_cast<const unsigned short*>(&v)), "l"(policy)
               : "memory");
}
__device__ __forceinline__ void bulk_load_1d(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
               "l"(reinterpret_cast<uint64_t>(src)), "r"(bytes), "r"(bar)
               : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&v)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
        "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]),
        "=r"(v[16]), "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]),
        "=r"(v[24]), "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Shared-memory matrix descriptor: K-major tile whose rows are 128 bytes, 128-byte swizzle,
// 8-row groups 1024 bytes apart (SBO), descriptor version 1, layout type 2 (SWIZZLE_128B).
__device__ __forceinline__ uint64_t make_desc_sw128(uint32_t smem_addr) {
  return static_cast<uint64_t>((smem_addr & 0x3FFFFu) >> 4) | (1ull << 16) | (static_cast<uint64_t>(1024 >> 4) << 32) |
         (1ull << 46) | (2ull << 61);
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 x bf16, both operands K-major.
__host__ __device__ constexpr uint32_t make_idesc(int M, int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(N >> 3) << 17) | (static_cast<uint32_t>(M >> 4) << 24);
}

__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}

__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// Eight codes of one 32-bit word of the plan's tile-ordered copy -> eight bf16 values q*scale+zero
// (one rounding each).  The word holds the codes of columns c .. c+7 in pair order: nibble i is
// column c + 2 i, nibble 4 + i is column c + 2 i + 1.
// kFast (bf16 scales/zeros): p carries the bit patterns of the packed pairs (scale,scale) and
// (zero,zero); the arithmetic is exact packed bf16: (128+q) as bf16 is 0x4300|q, minus 128, then
// one fused multiply-add.  Otherwise p = (scale, zero) in fp32: fp32 fma, then one conversion.
template <bool kFast>
__device__ __forceinline__ uint4 dequant_word(uint32_t w, float2 p) {
  uint32_t o[4];
  if constexpr (kFast) {
    const uint32_t sb = __float_as_uint(p.x), zb = __float_as_uint(p.y);
    const __nv_bfloat162 s2 = *reinterpret_cast<const __nv_bfloat162*>(&sb);
    const __nv_bfloat162 z2 = *reinterpret_cast<const __nv_bfloat162*>(&zb);
    const uint32_t magic = 0x43004300u;
    const __nv_bfloat162 m2 = *reinterpret_cast<const __nv_bfloat162*>(&magic);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      uint32_t t;                                                    // ((w >> 4 i) & 0x000F000F) | magic: one shift and ONE logic op
      asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(t) : "r"(w >> (4 * i)), "r"(0x000F000Fu), "r"(magic));   // (written out: the compiler makes two of it)
      const __nv_bfloat162 q2 = __hsub2(*reinterpret_cast<const __nv_bfloat162*>(&t), m2);
      const __nv_bfloat162 r = __hfma2(q2, s2, z2);
      o[i] = *reinterpret_cast<const uint32_t*>(&r);
    }
  } else {
    float f[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
      const int nib = (e >> 1) + 4 * (e & 1);
      const float q = __uint_as_float(0x4B000000u | ((w >> (4 * nib)) & 0xFu)) - 8388608.0f;
      f[e] = fmaf(q, p.x, p.y);
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) o[i] = pack_bf16x2(f[2 * i], f[2 * i + 1]);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}

}  // namespace tc

// Two-CTA pair-tile kernel (gemm_tc2.cu): tmap_x has a [128 x 64] box; P.m_tiles counts
// 256-token tiles, P.n_tiles the 256-row tiles of all P.nsub matrices; n_pairs clusters are launched.
// dequant == false: dense bf16 weight through mw (one matrix only).
szo_status launch_pair_kernel(bool dequant, bool bf16_tables, const CUtensorMap& mx, const CUtensorMap& mw,
                              const tc::TcParams& P, int n_pairs, cudaStream_t st);

// Self-test of the bounded waits (gemm_tc2.cu): *gave_up_dev = 1 when the wait expired.
szo_status launch_wait_timeout_selftest(long long limit_cycles, int32_t* gave_up_dev, cudaStream_t st);

}  // namespace szo
