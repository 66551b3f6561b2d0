// The fused linear on the tensor cores: persistent, warp-specialised tcgen05 kernel on two-CTA
// clusters (cta_group::2).
//
// A cluster of two CTAs on neighbouring SMs computes one 256 (weight rows) x 256 (tokens) tile:
// each CTA owns 128 weight rows (its half of the MMA's M dimension: dequantised and SparseAdd-ed in
// its own shared memory, accumulated in its own TMEM) and loads only 128 of the 256 tokens (its half
// of the N dimension); the tensor cores of both SMs read both halves.  Against a one-CTA form a
// k-block moves 16 KiB instead of 32 KiB of tokens through each SM's shared memory, which is what
// bounds that form (it measured 1.39 against 1.53 PFLOP/s on dense weights).  Small token counts use
// the same kernel (the token tile is zero-filled by TMA) with the tiles split along K.
//
// Three rings in shared memory, each with its own life time: X token tiles (TMA -> MMA), C packed
// codes + scale/zero strip (bulk copy -> conversion), A dequantised weight tiles in the swizzled
// K-major layout (conversion -> MMA).  Roles per CTA:
//   warp 0       X producer: TMA of the CTA's own token half (and its bf16 weight tile in dense mode)
//   warp 4       C producer: bulk copies of the CTA's code tile and scale/zero strip
//   warp 8       TMEM allocation; in the leader CTA (cluster rank 0) one thread issues the
//                tcgen05.mma.cta_group::2 instructions and commits, multicast, to the barriers of
//                both CTAs
//   warp 12      sparse-record prefetch (register-pipelined loads into a ring in shared memory)
//   12 warps     weight producers (w < 16, w % 4 != 0; three groups of four take k-blocks in turn): int4 -> bf16 conversion and SparseAdd of the CTA's own rows; when
//                the tile is final and the CTA's token half has landed they arrive, with cluster
//                scope, on the leader's aready barrier (8 arrivals: one group of each CTA).  In dense
//                mode the same warps add the sparse values to the TMA-loaded tile and relay.
//   warps 16-19  epilogue of the CTA's own 128 rows x 256 tokens (tcgen05.ld, bias, store)
// Work units: a launch covers up to three weight matrices that share the activations (their pair
// tiles are numbered consecutively), and the last, partial round of tiles is split along K into
// up to four parts so that every cluster stays busy; the parts of a tile meet in an fp32 workspace
// and the last one to finish adds them in part order (deterministic) and stores y.
// All waits are bounded; no TMA load uses cluster multicast.
#include <mutex>

#include "tc_common.cuh"

namespace szo {

namespace {

using namespace tc;

constexpr int kMaxDevices = 64;
constexpr int kPairBT = 256;                 // tokens per pair tile (UMMA N)
constexpr int kXHalfBytes = 128 * kBK * 2;   // this CTA's half of the token tile: 16 KiB
constexpr int kCStages2 = 8;
constexpr int kASlots2 = 6;
// 20 warps: four single-thread roles, three groups of four conversion warps, four epilogue warps.
// Warp w issues on scheduler w % 4.  The single-thread roles (warps 0, 4, 8, 12) share scheduler 0
// with one epilogue warp only, so the thread that issues the MMAs never competes with conversion
// warps for issue slots; the twelve conversion warps are the warps < 16 with w % 4 != 0; the
// epilogue warps 16-19 cover the four TMEM lane quarters.
constexpr int kGroups2 = 3, kWarpsPerGroup2 = 4;
constexpr int kWarpX = 0, kWarpC = 4, kWarpMma = 8, kWarpRec = 12;
constexpr int kEpiWarp02 = 16;
constexpr int kNumWarps2 = kEpiWarp02 + 4;
// sparse records: ring of per-k-block slots, filled a chunk of four k-blocks at a time
constexpr int kRecChunk = 4, kRecChunks = 3, kRecSlots2 = kRecChunk * kRecChunks;

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive on the barrier at the same shared-memory offset in CTA `target`.  The data the arrival
// publishes sits in this CTA's shared memory and is read by the tensor cores (async proxy), for
// which the preceding fence.proxy.async orders the writes; a cluster-scope release on top of that
// measured about a thousand cycles per arrival.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t local_bar, uint32_t target) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(target));
  asm volatile("mbarrier.arrive.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ void tmem_alloc2(uint32_t result_smem, uint32_t ncols) {
  asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(result_smem), "r"(ncols)
               : "memory");
  asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc2(uint32_t taddr, uint32_t ncols) {
  asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma2_bf16(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                           uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Commit: when the MMAs issued so far retire, arrive once on the barrier at this offset in both CTAs.
__device__ __forceinline__ void umma2_commit_both(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile(
      "tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::"r"(bar),
      "h"(mask)
      : "memory");
}

// One work unit of a cluster: k-blocks [kb0, kb1) of the pair tile (matrix s, this CTA's 128-row
// tile n_tile of that matrix, token tile m_tile).
struct Unit {
  int s, n_tile, m_tile, kb0, kb1, part, parts, slot;
  int g_tile;      // 128-row tile counted over all matrices of the launch (rows of a shared dense weight buffer)
};
__device__ __forceinline__ int tail_kb_at(const TcParams& P, int i) {
  return i == 0 ? P.tail_kb[0] : i == 1 ? P.tail_kb[1] : i == 2 ? P.tail_kb[2] : i == 3 ? P.tail_kb[3] : P.tail_kb[4];
}
__device__ __forceinline__ Unit decode_unit(const TcParams& P, int pair, int n_pairs, int rank, int lt) {
  Unit u;
  int tile;
  if (lt < P.full_rounds) {
    tile = lt * n_pairs + pair;
    u.kb0 = 0;
    u.kb1 = P.nkb;
    u.part = 0;
    u.parts = 1;
    u.slot = 0;
  } else {
    u.part = pair / P.tail_tiles;
    u.slot = pair - u.part * P.tail_tiles;
    u.parts = P.tail_parts;
    tile = P.full_rounds * n_pairs + u.slot;
    u.kb0 = tail_kb_at(P, u.part);
    u.kb1 = tail_kb_at(P, u.part + 1);
  }
  const int m_tiles = static_cast<int>(P.m_tiles);
  int np;
  if (P.m_band > 0) {
    const int per_band = static_cast<int>(P.n_tiles) * P.m_band;
    const int band = tile / per_band;
    const int r = tile - band * per_band;
    const int m_first = band * P.m_band;
    const int width = (m_tiles - m_first < P.m_band) ? m_tiles - m_first : P.m_band;      // the last band may be narrower
    np = r / width;
    u.m_tile = m_first + (r - np * width);
  } else {
    np = tile / m_tiles;
    u.m_tile = tile - np * m_tiles;
  }
  if (P.pair_ext && static_cast<int64_t>(u.m_tile) * 256 >= P.pair_row0) {
    u.kb0 *= 2;          // half-difference token tile: twice the k-blocks (xd W^T, then xc (eps Zbar)^T)
    u.kb1 *= 2;
  }
  u.g_tile = np * 2 + rank;
  u.s = 0;
  if (P.nsub > 1 && np >= P.sub[0].n_tiles) {
    np -= P.sub[0].n_tiles;
    u.s = 1;
    if (P.nsub > 2 && np >= P.sub[1].n_tiles) {
      np -= P.sub[1].n_tiles;
      u.s = 2;
    }
  }
  u.n_tile = np * 2 + rank;
  return u;
}
// Fields of matrix s, selected without indexing the parameter block dynamically.
#define SZO_SUB(P, s, f) ((s) == 0 ? (P).sub[0].f : ((s) == 1 ? (P).sub[1].f : (P).sub[2].f))

// Sum of the K-split parts of one CTA's 128 rows, tokens [t_begin, mlimit) of the tile, + bias, stored to
// y; run by every thread of the CTA after its roles have finished.  A part is [token][128 rows] fp32, parts are
// 2 * 256 * 128 floats apart; the sum runs in part order, so the result does not depend on which
// part finished last.  Thread -> one float4 (4 rows of one token) per step of nthreads, seven in
// flight per part.  Kept out of line: its registers would otherwise add to every role's.
__device__ __noinline__ void reduce_parts(const float* part0, int parts, int64_t n0, int64_t N, const float* bias_p,
                                          void* y, int y_f32, int relu, int64_t m0, int t_begin, int mlimit, int tid,
                                          int nthreads) {
  constexpr int64_t kPartFloats = static_cast<int64_t>(kPairBT) * kBM;
  constexpr int kBatch = 7;
  const int total = mlimit * (kBM / 4);          // float4s up to the last token of this share
  for (int base = t_begin * (kBM / 4) + tid; base < total; base += nthreads * kBatch) {
    float4 acc[kBatch];
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int f = base + i * nthreads;
      if (f < total) acc[i] = __ldcg(reinterpret_cast<const float4*>(part0) + f);
    }
    for (int q = 1; q < parts; ++q) {
      const float4* pq = reinterpret_cast<const float4*>(part0 + q * 2 * kPartFloats);
      float4 tt[kBatch];
#pragma unroll
      for (int i = 0; i < kBatch; ++i) {
        const int f = base + i * nthreads;
        if (f < total) tt[i] = __ldcg(pq + f);
      }
#pragma unroll
      for (int i = 0; i < kBatch; ++i) {
        acc[i].x += tt[i].x;
        acc[i].y += tt[i].y;
        acc[i].z += tt[i].z;
        acc[i].w += tt[i].w;
      }
    }
#pragma unroll
    for (int i = 0; i < kBatch; ++i) {
      const int f = base + i * nthreads;
      if (f >= total) continue;
      const int mm = f >> 5;
      const int64_t n4 = n0 + ((f & 31) << 2);
      if (n4 >= N) continue;
      float o[4] = {acc[i].x, acc[i].y, acc[i].z, acc[i].w};
      if (bias_p != nullptr) {
#pragma unroll
        for (int e = 0; e < 4; ++e)
          if (n4 + e < N) o[e] += __ldg(bias_p + n4 + e);
      }
      if (relu) {
#pragma unroll
        for (int e = 0; e < 4; ++e) o[e] = fmaxf(o[e], 0.f);
      }
      const bool vec_ok = (N % 4 == 0) && (n4 + 3 < N);
      const int64_t off = (m0 + mm) * N + n4;
      if (y_f32) {
        float* yp = static_cast<float*>(y) + off;
        if (vec_ok) {
          *reinterpret_cast<float4*>(yp) = make_float4(o[0], o[1], o[2], o[3]);
        } else {
          for (int e = 0; e < 4; ++e)
            if (n4 + e < N) yp[e] = o[e];
        }
      } else {
        __nv_bfloat16* yp = static_cast<__nv_bfloat16*>(y) + off;
        if (vec_ok) {
          const __nv_bfloat162 lo = __floats2bfloat162_rn(o[0], o[1]), hi = __floats2bfloat162_rn(o[2], o[3]);
          uint2 pk;
          pk.x = *reinterpret_cast<const uint32_t*>(&lo);
          pk.y = *reinterpret_cast<const uint32_t*>(&hi);
          *reinterpret_cast<uint2*>(yp) = pk;
        } else {
          for (int e = 0; e < 4; ++e)
            if (n4 + e < N) yp[e] = __float2bfloat16_rn(o[e]);
        }
      }
    }
  }
}

// kRelu: y = max(y, 0) in the epilogue (dense mode only: its own instantiation, so that the other
// launches' store loops stay as they are)
// kPaired: the paired form of a ZO step's two forwards (dense mode only, see TcParams): bias on the
// centre rows only
template <int kXS, bool kDequant, bool kFast, bool kRelu = false, bool kPaired = false>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumWarps2 * 32, 1)
szo_linear_tc2_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                      const TcParams P) {
  constexpr int kXStageBytes = kXHalfBytes + (kDequant ? 0 : kATileBytes);
  constexpr int kCStageBytes = kCodesBytes + kSzBytes;
  constexpr int kCS = kDequant ? kCStages2 : 1;
  constexpr int kAS = kDequant ? kASlots2 : kXS;            // dense: the weight tile lives in the X stage
  constexpr int kGroups = kGroups2, kWarpsPerGroup = kWarpsPerGroup2;
  constexpr uint32_t kTmemCols = 512;                       // two accumulators of 256 columns
  constexpr uint32_t kIdesc = make_idesc(256, kPairBT);
  constexpr uint32_t kCBase = kXS * kXStageBytes, kABase = kCBase + (kDequant ? kCS * kCStageBytes : 0);

  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kXS + 2 * kCS + 2 * kAS + 4 + 2 * kRecSlots2];
  __shared__ __align__(16) uint2 rec_ring[kRecSlots2][kRecCap];
  __shared__ __align__(16) int32_t bound_ring[kRecSlots2][4];   // e0, e1, matrix index
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;
  __shared__ int epi_count_s, reduce_flag_s;   // K-split tail: epilogue warps done, this CTA sums the parts

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_ctarank());
  const bool leader = rank == 0;
  volatile int* abort_flag = &abort_flag_s;

  auto xfull_bar = [&](int s) { return smem_u32(&bars[s]); };                  // own X stage landed (TMA)
  auto xempty_bar = [&](int s) { return smem_u32(&bars[kXS + s]); };           // its MMAs retired (commit to both)
  auto cfull_bar = [&](int c) { return smem_u32(&bars[2 * kXS + c]); };
  auto cempty_bar = [&](int c) { return smem_u32(&bars[2 * kXS + kCS + c]); };
  auto aready_bar = [&](int t) { return smem_u32(&bars[2 * kXS + 2 * kCS + t]); };          // leader: both CTAs' tiles final
  auto aempty_bar = [&](int t) { return smem_u32(&bars[2 * kXS + 2 * kCS + kAS + t]); };    // MMAs retired (commit to both)
  auto accfull_bar = [&](int a) { return smem_u32(&bars[2 * kXS + 2 * kCS + 2 * kAS + a]); };
  auto accempty_bar = [&](int a) { return smem_u32(&bars[2 * kXS + 2 * kCS + 2 * kAS + 2 + a]); };   // leader
  auto recready_bar = [&](int r) { return smem_u32(&bars[2 * kXS + 2 * kCS + 2 * kAS + 4 + r]); };
  auto recfree_bar = [&](int r) { return smem_u32(&bars[2 * kXS + 2 * kCS + 2 * kAS + 4 + kRecSlots2 + r]); };
  auto b_off = [&](int s) { return static_cast<uint32_t>(s) * kXStageBytes; };
  auto c_off = [&](int c) { return kCBase + static_cast<uint32_t>(c) * kCStageBytes; };
  auto a_off = [&](int s, int t) {
    return kDequant ? kABase + static_cast<uint32_t>(t) * kATileBytes : b_off(s) + kXHalfBytes;
  };

  const bool sparse = P.sub[0].Sb != nullptr || (P.nsub > 1 && P.sub[1].Sb != nullptr) || (P.nsub > 2 && P.sub[2].Sb != nullptr);
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    epi_count_s = 0;
    reduce_flag_s = 0;
    for (int s = 0; s < kXS; ++s) {
      mbar_init(xfull_bar(s), 1);
      mbar_init(xempty_bar(s), 1);
    }
    for (int c = 0; c < kCS; ++c) {
      mbar_init(cfull_bar(c), 1);
      mbar_init(cempty_bar(c), kWarpsPerGroup);
    }
    for (int t = 0; t < kAS; ++t) {
      mbar_init(aready_bar(t), 2 * kWarpsPerGroup);
      mbar_init(aempty_bar(t), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accfull_bar(a), 1);
      mbar_init(accempty_bar(a), 8);
    }
    for (int r = 0; r < kRecSlots2; ++r) {
      mbar_init(recready_bar(r), 1);
      mbar_init(recfree_bar(r), kWarpsPerGroup);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) tmem_alloc2(smem_u32(&tmem_base_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers exist before anyone arrives on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  // work units of this cluster (see TcParams): full tiles first, then at most one unit of the tail
  const int pair = static_cast<int>(blockIdx.x >> 1), n_pairs = static_cast<int>(gridDim.x >> 1);
  const int nkb = P.nkb;
  const bool has_tail = pair < P.tail_tiles * P.tail_parts;
  const int my_units = P.full_rounds + (has_tail ? 1 : 0);
  const int full_iters = P.full_rounds * nkb;
  const int tail_part = has_tail ? pair / P.tail_tiles : 0;
  const int tail_kb0 = has_tail ? tail_kb_at(P, tail_part) : 0;
  int my_iters = full_iters + (has_tail ? tail_kb_at(P, tail_part + 1) - tail_kb0 : 0);
  if constexpr (kPaired) {
    if (P.pair_ext) {      // units differ in length: add them up
      my_iters = 0;
      for (int lt = 0; lt < my_units; ++lt) {
        const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
        my_iters += u.kb1 - u.kb0;
      }
    }
  }

  if (warp == kWarpX) {
    // ---------------------------------------------------------------- X producer (own token half)
    if (lane == 0) {
      RingPos x{0, 0};
      bool ok = true;
      const uint64_t keep = l2_policy_evict_last();
      for (int lt = 0; lt < my_units && ok; ++lt) {
        const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
        const int tok0 = u.m_tile * kPairBT + rank * 128;
        const int row0 = u.g_tile * kBM;   // dense weights of a launch are one buffer, each matrix padded to 256 rows
        for (int kb = u.kb0; kb < u.kb1; ++kb) {
          if (!mbar_wait(xempty_bar(x.idx), x.phase ^ 1u, abort_flag, P.status)) { ok = false; break; }
          mbar_expect_tx(xfull_bar(x.idx), kXStageBytes);
          int xk = kb * kBK, xt = tok0;
          if constexpr (kPaired) {
            if (kb >= nkb) {            // second half of a half-difference tile: the centre rows of the same tokens
              xk -= nkb * kBK;
              xt -= static_cast<int>(P.pair_row0);
            }
          }
          tma_load_2d_hint(tiles_base + b_off(x.idx), &tmap_x, xk, xt, xfull_bar(x.idx), keep);
          if constexpr (!kDequant) tma_load_2d(tiles_base + a_off(x.idx, 0), &tmap_w, kb * kBK, row0, xfull_bar(x.idx));
          x.advance(kXS);
        }
      }
    }
  } else if (warp == kWarpC) {
    // ---------------------------------------------------------------- C producer (codes, scale/zero)
    if constexpr (kDequant) {
      if (lane == 0) {
        // Everything the loop needs advances by addition: this is one thread, and every dependent
        // instruction of its loop body is several cycles of the k-block period.
        const int groups_kb = (P.G < kBK) ? kBK / P.G : 1;     // scale groups per k-block
        const int kb_per_group = (P.G > kBK) ? P.G / kBK : 1;  // k-blocks per scale group
        const uint32_t tx_bytes = static_cast<uint32_t>(kCodesBytes + groups_kb * 1024);
        int cidx = 0;
        uint32_t cphase = 0, dst = tiles_base + kCBase;
        bool ok = true;
        for (int lt = 0; lt < my_units && ok; ++lt) {
          const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
          const int64_t Npad = SZO_SUB(P, u.s, Npad);
          const int64_t sz_step = static_cast<int64_t>(groups_kb) * Npad;
          // a unit starts on a scale-group boundary (the host aligns the K split)
          const uint8_t* codes = SZO_SUB(P, u.s, codes) + (static_cast<int64_t>(u.n_tile) * nkb + u.kb0) * kCodesBytes;
          const float2* sz = SZO_SUB(P, u.s, sz) + static_cast<int64_t>(u.n_tile) * kBM + (u.kb0 / kb_per_group) * sz_step;
          int kbg = 0;
          for (int kb = u.kb0; kb < u.kb1; ++kb) {
            if (!mbar_wait(cempty_bar(cidx), cphase ^ 1u, abort_flag, P.status)) { ok = false; break; }
            const uint32_t bar = cfull_bar(cidx);
            mbar_expect_tx(bar, tx_bytes);
            bulk_load_1d(dst, codes, kCodesBytes, bar);
            bulk_load_1d(dst + kCodesBytes, sz, 1024, bar);
            for (int g = 1; g < groups_kb; ++g) bulk_load_1d(dst + kCodesBytes + g * 1024, sz + g * Npad, 1024, bar);
            codes += kCodesBytes;
            if (++kbg == kb_per_group) {
              kbg = 0;
              sz += sz_step;
            }
            dst += kCStageBytes;
            if (++cidx == kCS) {
              cidx = 0;
              cphase ^= 1u;
              dst = tiles_base + kCBase;
            }
          }
        }
      }
    }
  } else if (warp == kWarpMma) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      RingPos x{0, 0}, a{0, 0};
      bool ok = true;
      for (int lt = 0; lt < my_units && ok; ++lt) {
        const int as = lt & 1;
        const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
        int n_kb = (lt < P.full_rounds) ? nkb : my_iters - full_iters;
        if constexpr (kPaired) {
          if (P.pair_ext) {
            const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
            n_kb = u.kb1 - u.kb0;
          }
        }
        if (!mbar_wait(accempty_bar(as), aph ^ 1u, abort_flag, P.status, 0)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kPairBT);
        for (int kb = 0; kb < n_kb; ++kb) {
          // both CTAs' weight tiles final and both token halves landed
          if (!mbar_wait(aready_bar(a.idx), a.phase, abort_flag, P.status, 0)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = make_desc_sw128(tiles_base + a_off(x.idx, a.idx));
          const uint64_t bdesc = make_desc_sw128(tiles_base + b_off(x.idx));
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) umma2_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc, (kb | k) ? 1u : 0u);
          umma2_commit_both(xempty_bar(x.idx));
          if constexpr (kDequant) umma2_commit_both(aempty_bar(a.idx));
          x.advance(kXS);
          a.advance(kAS);
        }
        if (ok) umma2_commit_both(accfull_bar(as));
      }
    }
  } else if (warp == kWarpRec) {
    // ---------------------------------------------------------------- sparse-record warp
    // Brings the bucket bounds and the sparse records (position in tile, fp32 value) of every
    // k-block of this CTA into a ring of per-k-block slots in shared memory, a chunk of four
    // k-blocks per loop iteration (lane j < 4 owns the bounds of k-block it0 + j), up to three chunks
    // ahead of their use.  The bounds of the next chunk are fetched while this chunk's records are
    // in flight, so one global-load latency is exposed per four k-blocks.
    if (sparse && my_units > 0) {
      auto load_bounds = [&](int it0, int32_t& e0, int32_t& e1, int& sm) {
        const int itl = it0 + (lane & (kRecChunk - 1));
        e0 = 0;
        e1 = 0;
        sm = 0;
        if (itl < my_iters) {
          int lt, kb;
          if (itl < full_iters) {
            lt = itl / nkb;
            kb = itl - lt * nkb;
          } else {
            lt = P.full_rounds;
            kb = tail_kb0 + (itl - full_iters);
          }
          const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
          sm = u.s;
          if (u.n_tile < SZO_SUB(P, u.s, n_rowtiles) && SZO_SUB(P, u.s, Sb) != nullptr) {
            const int32_t* bp = SZO_SUB(P, u.s, bucket_ptr) + static_cast<int64_t>(u.n_tile) * nkb + kb;
            e0 = __ldg(bp);
            e1 = __ldg(bp + 1);
          }
        }
      };
      int32_t e0, e1;
      int sm;
      load_bounds(0, e0, e1, sm);
      int cs = 0;                       // chunk slot: ring slots cs * 4 .. cs * 4 + 3
      uint32_t cphase = 0;
      bool first_pass = true;
      bool ok = true;
      for (int it0 = 0; it0 < my_iters && ok; it0 += kRecChunk) {
        int32_t ne0, ne1;
        int nsm;
        load_bounds(it0 + kRecChunk, ne0, ne1, nsm);
        if (!first_pass) {              // the slots' previous k-blocks must have been consumed
#pragma unroll
          for (int j = 0; j < kRecChunk; ++j)
            if (it0 + j < my_iters && !mbar_wait(recfree_bar(cs * kRecChunk + j), cphase ^ 1u, abort_flag, P.status)) ok = false;
          if (!ok) break;
        }
        uint2 r[kRecChunk][kRecCap / 32];
        int32_t n[kRecChunk];
#pragma unroll
        for (int j = 0; j < kRecChunk; ++j) {
          const int32_t b0 = __shfl_sync(0xFFFFFFFFu, e0, j), b1 = __shfl_sync(0xFFFFFFFFu, e1, j);
          const int sj = __shfl_sync(0xFFFFFFFFu, sm, j);
          const uint2* Sb = SZO_SUB(P, sj, Sb);
          n[j] = (b1 - b0 < kRecCap) ? b1 - b0 : kRecCap;
#pragma unroll
          for (int q = 0; q < kRecCap / 32; ++q)
            if (lane + 32 * q < n[j]) r[j][q] = __ldg(Sb + b0 + lane + 32 * q);
        }
        // (slots past the end of the stream still belong to k-blocks that may not have been consumed)
        if (lane < kRecChunk && it0 + lane < my_iters)
          *reinterpret_cast<int4*>(bound_ring[cs * kRecChunk + lane]) = make_int4(e0, e1, sm, 0);
#pragma unroll
        for (int j = 0; j < kRecChunk; ++j) {
#pragma unroll
          for (int q = 0; q < kRecCap / 32; ++q)
            if (lane + 32 * q < n[j]) rec_ring[cs * kRecChunk + j][lane + 32 * q] = r[j][q];
        }
        __syncwarp();
        if (lane < kRecChunk && it0 + lane < my_iters) mbar_arrive(recready_bar(cs * kRecChunk + lane));
        e0 = ne0;
        e1 = ne1;
        sm = nsm;
        if (++cs == kRecChunks) {
          cs = 0;
          cphase ^= 1u;
          first_pass = false;
        }
      }
    }
  } else if ((warp & 3) != 0 && warp < kEpiWarp02) {
    // ---------------------------------------------------------------- weight producers
    const int dw = (warp >> 2) * 3 + (warp & 3) - 1;
    const int gq = dw / kWarpsPerGroup, wq = dw % kWarpsPerGroup;
    constexpr int kRowsPerWarp = kBM / kWarpsPerGroup;
    auto add_record = [&](unsigned char* A, uint2 rc) {
      // rc.x: byte offset of the element in the swizzled tile (row = offset / 128)
      if (static_cast<int>(rc.x >> 7) / kRowsPerWarp == wq) {
        __nv_bfloat16* el = reinterpret_cast<__nv_bfloat16*>(A + rc.x);
        *el = __float2bfloat16_rn(__bfloat162float(*el) + __uint_as_float(rc.y));
      }
    };
    if constexpr (kDequant) {
      constexpr int kPasses = kRowsPerWarp / 4;
      const int sub = lane >> 3, chunk = lane & 7;
      const int gsel = (P.G < kBK) ? (chunk * 8) / P.G : 0;
      RingPos c{0, 0}, a{0, 0}, x{0, 0}, rr{0, 0};
      for (int j = 0; j < gq; ++j) {
        c.advance(kCS);
        a.advance(kAS);
        x.advance(kXS);
        rr.advance(kRecSlots2);
      }
      for (int it = gq; it < my_iters; it += kGroups) {
        unsigned char* A = tiles_ptr + a_off(0, a.idx);
        const unsigned char* C = tiles_ptr + c_off(c.idx);
        const float2* SZ = reinterpret_cast<const float2*>(C + kCodesBytes) + gsel * kBM;
        if (!mbar_wait(cfull_bar(c.idx), c.phase, abort_flag, P.status)) break;
        uint32_t w[kPasses];
        float2 zs[kPasses];
#pragma unroll
        for (int i = 0; i < kPasses; ++i) {
          const int r = wq * kRowsPerWarp + i * 4 + sub;
          w[i] = *reinterpret_cast<const uint32_t*>(C + r * 32 + chunk * 4);
          zs[i] = SZ[r];
        }
        int32_t e0 = 0, e1 = 0;
        uint2 rec = make_uint2(0xFFFFFFFFu, 0u);
        if (sparse) {
          if (!mbar_wait(recready_bar(rr.idx), rr.phase, abort_flag, P.status)) break;
          const int2 be = *reinterpret_cast<const int2*>(bound_ring[rr.idx]);
          e0 = be.x;
          e1 = be.y;
          if (lane < e1 - e0) rec = rec_ring[rr.idx][lane];
        }
        if (!mbar_wait(aempty_bar(a.idx), a.phase ^ 1u, abort_flag, P.status)) break;
#pragma unroll
        for (int i = 0; i < kPasses; ++i) {
          const int r = wq * kRowsPerWarp + i * 4 + sub;
          const uint4 v = dequant_word<kFast>(w[i], zs[i]);
          *reinterpret_cast<uint4*>(A + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
        }
        if (e1 > e0) {
          __syncwarp();
          if (lane < e1 - e0) add_record(A, rec);
          for (int32_t j = lane + 32; j < e1 - e0; j += 32)
            add_record(A, (j < kRecCap) ? rec_ring[rr.idx][j] : __ldg(SZO_SUB(P, bound_ring[rr.idx][2], Sb) + e0 + j));
        }
        fence_async_smem();
        __syncwarp();
        // the leader's MMA of this k-block also reads this CTA's token half: it has long landed
        if (!mbar_wait(xfull_bar(x.idx), x.phase, abort_flag, P.status)) break;
        if (lane == 0) {
          mbar_arrive_cluster(aready_bar(a.idx), 0);
          mbar_arrive(cempty_bar(c.idx));
          if (sparse) mbar_arrive(recfree_bar(rr.idx));
        }
        static_assert(kGroups <= kCS && kGroups <= kAS && kGroups <= kXS && kGroups <= kRecSlots2, "ring shorter than a stride");
        c.advance_by(kGroups, kCS);
        a.advance_by(kGroups, kAS);
        x.advance_by(kGroups, kXS);
        rr.advance_by(kGroups, kRecSlots2);
      }
    } else {
      // dense bf16 weight tile delivered by TMA: add the bucket's sparse values (if any) and relay
      // "this CTA's stage is final" to the leader
      RingPos x{0, 0}, rr{0, 0};
      for (int j = 0; j < gq; ++j) {
        x.advance(kXS);
        rr.advance(kRecSlots2);
      }
      for (int it = gq; it < my_iters; it += kGroups) {
        int32_t e0 = 0, e1 = 0;
        if (sparse) {
          if (!mbar_wait(recready_bar(rr.idx), rr.phase, abort_flag, P.status)) break;
          e0 = bound_ring[rr.idx][0];
          e1 = bound_ring[rr.idx][1];
        }
        if (!mbar_wait(xfull_bar(x.idx), x.phase, abort_flag, P.status)) break;
        if (e1 > e0) {
          unsigned char* A = tiles_ptr + a_off(x.idx, x.idx);
          for (int32_t j = lane; j < e1 - e0; j += 32)
            add_record(A, (j < kRecCap) ? rec_ring[rr.idx][j] : __ldg(SZO_SUB(P, bound_ring[rr.idx][2], Sb) + e0 + j));
          fence_async_smem();
        }
        __syncwarp();
        if (lane == 0) {
          mbar_arrive_cluster(aready_bar(x.idx), 0);
          if (sparse) mbar_arrive(recfree_bar(rr.idx));
        }
        x.advance_by(kGroups, kXS);
        rr.advance_by(kGroups, kRecSlots2);
      }
    }
  } else if (warp >= kEpiWarp02) {
    // ---------------------------------------------------------------- epilogue (own 128 rows)
    const int qd = warp & 3;
    const uint64_t stream_out = l2_policy_evict_first();
    for (int lt = 0; lt < my_units; ++lt) {
      const Unit u = decode_unit(P, pair, n_pairs, rank, lt);
      const int as = lt & 1;
      const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
      if (!mbar_wait(accfull_bar(as), aph, abort_flag, P.status, 256)) break;
      tc_fence_after();
      const int64_t N = SZO_SUB(P, u.s, N);
      const int64_t m0 = static_cast<int64_t>(u.m_tile) * kPairBT;
      const float* bias_p = SZO_SUB(P, u.s, bias);
      if constexpr (kPaired) {
        if (m0 >= P.pair_row0) bias_p = nullptr;        // the half-difference of a constant is zero
      }
      void* y = SZO_SUB(P, u.s, y);
      const int64_t n = static_cast<int64_t>(u.n_tile) * kBM + qd * 32 + lane;
      const float bias = (bias_p != nullptr && n < N) ? bias_p[n] : 0.f;
      const int mlimit = static_cast<int>((P.M - m0 < kPairBT) ? P.M - m0 : kPairBT);
      // y[m0 + c0 + j, n] = v[j] + bias for the valid tokens of a 32-token chunk
      auto act = [&](float t) {
        if constexpr (kRelu) return fmaxf(t, 0.f);
        else return t;
      };
      auto store_chunk = [&](int c0, const uint32_t (&v)[32]) {
        if (n < N && c0 < mlimit) {
          const int cnt = mlimit - c0;
          if (P.y_f32) {
            float* yp = static_cast<float*>(y) + (m0 + c0) * N + n;
            if (cnt >= 32) {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                *yp = act(__uint_as_float(v[j]) + bias);
                yp += N;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (j < cnt) *yp = act(__uint_as_float(v[j]) + bias);
                yp += N;
              }
            }
          } else {
            __nv_bfloat16* yp = static_cast<__nv_bfloat16*>(y) + (m0 + c0) * N + n;
            if (cnt >= 32 && bias_p == nullptr) {
              // a full chunk: no per-token predicate, two tokens per conversion (and nothing to add)
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(act(__uint_as_float(v[j])), act(__uint_as_float(v[j + 1])));
                st_bf16_hint(yp, pr.x, stream_out);
                st_bf16_hint(yp + N, pr.y, stream_out);
                yp += 2 * N;
              }
            } else if (cnt >= 32) {
#pragma unroll
              for (int j = 0; j < 32; j += 2) {
                const __nv_bfloat162 pr = __floats2bfloat162_rn(act(__uint_as_float(v[j]) + bias),
                                                                act(__uint_as_float(v[j + 1]) + bias));
                st_bf16_hint(yp, pr.x, stream_out);
                st_bf16_hint(yp + N, pr.y, stream_out);
                yp += 2 * N;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 32; ++j) {
                if (j < cnt) *yp = __float2bfloat16_rn(act(__uint_as_float(v[j]) + bias));
                yp += N;
              }
            }
          }
        }
      };
      const uint32_t t_acc = tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + static_cast<uint32_t>(as * kPairBT);
      if (u.parts == 1) {
        for (int c0 = 0; c0 < kPairBT; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(t_acc + static_cast<uint32_t>(c0), v);
          store_chunk(c0, v);
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(accempty_bar(as), 0);
      } else {
        // K-split tile (always this CTA's last unit): park this part's fp32 accumulator
        // ([token][row], rows contiguous).  The last of the four epilogue warps takes the tile's
        // ticket; the CTA holding the last part's ticket sums the parts after its roles are done.
        constexpr int64_t kPartFloats = static_cast<int64_t>(kPairBT) * kBM;
        float* mine = P.partial + (static_cast<int64_t>(u.slot * u.parts + u.part) * 2 + rank) * kPartFloats + qd * 32 + lane;
        for (int c0 = 0; c0 < kPairBT; c0 += 32) {
          uint32_t v[32];
          tmem_ld32(t_acc + static_cast<uint32_t>(c0), v);
#pragma unroll
          for (int j = 0; j < 32; ++j) __stcg(mine + (c0 + j) * kBM, __uint_as_float(v[j]));
        }
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive_cluster(accempty_bar(as), 0);
        __threadfence();
        __syncwarp();
        if (lane == 0 && atomicAdd_block(&epi_count_s, 1) == 3) {
          __threadfence();
          atomicAdd(P.tickets + u.slot * 2 + rank, 1);      // this part is parked
          reduce_flag_s = 1;                                 // this CTA sums a share of the tile's tokens
        }
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  if (reduce_flag_s && !*abort_flag) {
    constexpr int64_t kPartFloats = static_cast<int64_t>(kPairBT) * kBM;
    const Unit u = decode_unit(P, pair, n_pairs, rank, my_units - 1);
    int32_t* ticket = P.tickets + u.slot * 2 + rank;
    int32_t* done = P.tickets_done + u.slot * 2 + rank;
    if (threadIdx.x == 0) {
      // all parts of the tile parked?  Their clusters are resident and running: a bounded wait
      const long long t0 = clock64();
      while (*reinterpret_cast<volatile int32_t*>(ticket) < u.parts) {
        __nanosleep(64);
        if (clock64() - t0 > kWaitLimitCycles) {
          *abort_flag = 1;
          atomicExch(P.status, static_cast<int32_t>(SZO_ERR_TIMEOUT));
          break;
        }
      }
      __threadfence();               // the other parts' tiles are read after this point (from L2, ld.cg)
    }
    __syncthreads();
    if (!*abort_flag) {
      const int64_t m0 = static_cast<int64_t>(u.m_tile) * kPairBT;
      const int mlimit = static_cast<int>((P.M - m0 < kPairBT) ? P.M - m0 : kPairBT);
      const int t_begin = (kPairBT * u.part) / u.parts, t_end = (kPairBT * (u.part + 1)) / u.parts;
      const float* bias_p = SZO_SUB(P, u.s, bias);
      if constexpr (kPaired) {
        if (m0 >= P.pair_row0) bias_p = nullptr;
      }
      if (t_begin < mlimit)
        reduce_parts(P.partial + (static_cast<int64_t>(u.slot * u.parts) * 2 + rank) * kPartFloats, u.parts,
                     static_cast<int64_t>(u.n_tile) * kBM, SZO_SUB(P, u.s, N), bias_p, SZO_SUB(P, u.s, y), P.y_f32,
                     kRelu ? 1 : 0, m0, t_begin, t_end < mlimit ? t_end : mlimit, static_cast<int>(threadIdx.x),
                     kNumWarps2 * 32);
      __syncthreads();
      if (threadIdx.x == 0 && atomicAdd(done, 1) == u.parts - 1) {      // the last share: ready for the next launch
        *ticket = 0;
        *done = 0;
      }
    }
  }
  cluster_sync_all();          // no CTA leaves while its peer may still signal it or read its tiles
  tc_fence_after();
  if (warp == kWarpMma) tmem_dealloc2(tmem_base, kTmemCols);
}

template <int kXS, bool kDequant, bool kFast, bool kRelu = false, bool kPaired = false>
szo_status launch_tc2(const CUtensorMap& mx, const CUtensorMap& mw, const TcParams& P, int n_pairs, cudaStream_t st) {
  constexpr size_t smem = static_cast<size_t>(kXS) * (kXHalfBytes + (kDequant ? 0 : kATileBytes)) +
                          (kDequant ? kCStages2 * (kCodesBytes + kSzBytes) + kASlots2 * kATileBytes : 0) + 1024;
  auto kern = szo_linear_tc2_kernel<kXS, kDequant, kFast, kRelu, kPaired>;
  // the attribute belongs to the (function, device) pair: one flag per device, set under a lock
  static std::mutex mu;
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_REQUIRE(dev >= 0 && dev < kMaxDevices, SZO_ERR_UNSUPPORTED, "device ordinal %d out of range", dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (!configured[dev]) {
      SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
      configured[dev] = true;
    }
  }
  kern<<<static_cast<unsigned>(2 * n_pairs), kNumWarps2 * 32, smem, st>>>(mx, mw, P);
  count_launch();
  SZO_CHECK_LAUNCH("szo_linear_tc2_kernel");
  return SZO_OK;
}

}  // namespace

namespace {
// One thread waits, with a limit of `limit_cycles` SM cycles, on an mbarrier that nothing ever arrives
// on: the wait must give up, record SZO_ERR_TIMEOUT in the status word and let the kernel return.
__global__ void wait_timeout_selftest_kernel(long long limit_cycles, int32_t* status, int32_t* gave_up) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag_s;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    tc::mbar_init(tc::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    volatile int* abort_flag = &abort_flag_s;
    const bool ok = tc::mbar_wait(tc::smem_u32(&bar), 0u, abort_flag, status, 32, limit_cycles);
    *gave_up = ok ? 0 : 1;
  }
}
}  // namespace

szo_status launch_wait_timeout_selftest(long long limit_cycles, int32_t* gave_up_dev, cudaStream_t st) {
  int32_t* status = device_status_word();
  SZO_REQUIRE(status != nullptr, SZO_ERR_CUDA, "no device status word");
  wait_timeout_selftest_kernel<<<1, 32, 0, st>>>(limit_cycles, status, gave_up_dev);
  count_launch();
  SZO_CHECK_LAUNCH("wait_timeout_selftest_kernel");
  return SZO_OK;
}

szo_status launch_pair_kernel(bool dequant, bool bf16_tables, const CUtensorMap& mx, const CUtensorMap& mw,
                              const tc::TcParams& P, int n_pairs, cudaStream_t st) {
  if (P.pair_row0 > 0) {
    SZO_REQUIRE(!dequant && !P.relu, SZO_ERR_UNSUPPORTED, "the paired form exists in the dense mode without ReLU only");
    return launch_tc2<6, false, false, false, true>(mx, mw, P, n_pairs, st);
  }
  if (!dequant && P.relu) return launch_tc2<6, false, false, true>(mx, mw, P, n_pairs, st);
  if (!dequant) return launch_tc2<6, false, false>(mx, mw, P, n_pairs, st);
  SZO_REQUIRE(!P.relu, SZO_ERR_UNSUPPORTED, "the ReLU epilogue exists in the dense mode only");
  if (bf16_tables) return launch_tc2<4, true, true>(mx, mw, P, n_pairs, st);
  return launch_tc2<4, true, false>(mx, mw, P, n_pairs, st);
}

}  // namespace szo
