// Two-CTA (cta_group::2) version of the fused linear for M > 128 tokens.
//
// A cluster of two CTAs on neighbouring SMs computes one 256 (weight rows) x 256 (tokens) tile:
// each CTA owns 128 weight rows (its half of the MMA's M dimension, dequantised and SparseAdd-ed in
// its own shared memory, accumulated in its own TMEM) and loads only 128 of the 256 tokens (its half
// of the N dimension); the tensor cores of both SMs read both halves.  Against the one-CTA kernel
// this halves the activation bytes fetched from L2 per flop and shrinks a pipeline stage, so seven
// raw stages (token tile + codes + scale/zero strip) and three dequantised weight slots fit.
//
//   warp 0       TMA producer (own token half, own codes / scale-zero strip, or own bf16 weight tile)
//   warp 1       TMEM allocation; in the leader CTA (cluster rank 0) one thread issues the
//                tcgen05.mma.cta_group::2 instructions and commits, multicast, to the stage and
//                accumulator barriers of both CTAs
//   warp 2       stage finisher: waits for the dequantised (or TMA-loaded) weight tile, adds the
//                bucket's sparse values in shared memory (records prefetched with cp.async), fences
//                and arrives, with cluster scope, on the leader's ready[s] barrier (2 arrivals)
//   warps 4-11   int4 -> bf16 conversion, shared -> shared, into the swizzled K-major layout
//   warps 12-15  epilogue of the CTA's own 128 rows x 256 tokens (tcgen05.ld, bias, store)
// All waits are bounded; no TMA load uses cluster multicast.
#include "tc_common.cuh"

namespace szo {

namespace {

using namespace tc;

constexpr int kBT2 = 256;                    // tokens per pair tile (UMMA N)
constexpr int kBHalfBytes = 128 * kBK * 2;   // this CTA's half of the token tile: 16 KiB
constexpr int kARing = 3;                    // dequantised weight slots

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// Arrive (release, cluster scope) on the barrier at the same shared-memory offset in CTA `target`.
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t local_bar, uint32_t target) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local_bar), "r"(target));
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, volatile int* abort_flag,
                                                  int32_t* status) {
  for (int i = 0; i < 256; ++i)
    if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  while (true) {
    for (int i = 0; i < 256; ++i)
      if (mbar_try_wait_cluster(bar, parity)) return true;
    if (*abort_flag) return false;
    if (clock64() - t0 > kWaitLimitCycles) {
      *abort_flag = 1;
      atomicExch(status, static_cast<int32_t>(SZO_ERR_TIMEOUT));
      return false;
    }
  }
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

template <int kRaw, bool kDequant, bool kFast>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumWarps * 32, 1)
szo_linear_tc2_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                      const TcParams P) {
  constexpr int kRawBytes = kBHalfBytes + (kDequant ? kCodesBytes + kSzBytes : kATileBytes);
  constexpr uint32_t kTmemCols = 512;
  constexpr uint32_t kIdesc = make_idesc(256, kBT2);

  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[3 * kRaw + 2 * kARing + 4];
  __shared__ __align__(16) uint2 rec_ring[kRecSlots][kRecCap];
  __shared__ __align__(8) int32_t bound_ring[kBoundSlots][2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  volatile int* abort_flag = &abort_flag_s;

  auto full_bar = [&](int s) { return smem_u32(&bars[s]); };                    // local TMA bytes landed
  auto ready_bar = [&](int s) { return smem_u32(&bars[kRaw + s]); };            // leader: both CTAs' tiles final
  auto empty_bar = [&](int s) { return smem_u32(&bars[2 * kRaw + s]); };        // MMAs of the raw stage retired
  auto deq_bar = [&](int t) { return smem_u32(&bars[3 * kRaw + t]); };          // weight slot t converted
  auto aempty_bar = [&](int t) { return smem_u32(&bars[3 * kRaw + kARing + t]); };  // weight slot t consumed
  auto accfull_bar = [&](int a) { return smem_u32(&bars[3 * kRaw + 2 * kARing + a]); };
  auto accempty_bar = [&](int a) { return smem_u32(&bars[3 * kRaw + 2 * kARing + 2 + a]); };  // leader
  // shared-memory carve-up: kRaw raw stages, then (dequant mode) kARing weight slots
  auto raw_off = [&](int s) { return static_cast<uint32_t>(s) * kRawBytes; };
  auto b_tile = [&](int s) { return tiles_base + raw_off(s); };
  auto c_tile = [&](int s) { return tiles_base + raw_off(s) + kBHalfBytes; };   // codes (+ sz) or bf16 weight tile
  auto a_off = [&](int s, int t) {
    return kDequant ? static_cast<uint32_t>(kRaw) * kRawBytes + static_cast<uint32_t>(t) * kATileBytes
                    : raw_off(s) + kBHalfBytes;
  };

  const bool sparse = P.Sb != nullptr;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < kRaw; ++s) {
      mbar_init(full_bar(s), 1);
      mbar_init(ready_bar(s), 2);
      mbar_init(empty_bar(s), 1);
    }
    for (int t = 0; t < kARing; ++t) {
      mbar_init(deq_bar(t), kNumDeqWarps);
      mbar_init(aempty_bar(t), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accfull_bar(a), 1);
      mbar_init(accempty_bar(a), 8);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc2(smem_u32(&tmem_base_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // the peer's barriers exist before anyone arrives on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  const int64_t pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int64_t total_tiles = P.m_tiles * P.n_tiles;
  const int64_t my_tiles = (total_tiles > pair) ? (total_tiles - pair + n_pairs - 1) / n_pairs : 0;
  const int64_t my_iters = my_tiles * P.nkb;
  auto tile_of = [&](int64_t it) { return pair + (it / P.nkb) * n_pairs; };

  if (warp == 0) {
    // ---------------------------------------------------------------- TMA producer
    if (lane == 0) {
      const int groups_kb = (kDequant && P.G < kBK) ? kBK / P.G : 1;
      for (int64_t it = 0; it < my_iters; ++it) {
        const int64_t tile = tile_of(it);
        const int kb = static_cast<int>(it % P.nkb);
        const int64_t row0 = (tile / P.m_tiles) * 256 + rank * 128;       // this CTA's weight rows
        const int64_t tok0 = (tile % P.m_tiles) * kBT2 + rank * 128;      // this CTA's half of the tokens
        const int s = static_cast<int>(it % kRaw);
        const uint32_t ph = static_cast<uint32_t>((it / kRaw) & 1);
        if (!mbar_wait(empty_bar(s), ph ^ 1u, abort_flag, P.status)) break;
        if constexpr (kDequant) {
          mbar_expect_tx(full_bar(s), kBHalfBytes + kCodesBytes + groups_kb * 1024);
          bulk_load_1d(c_tile(s), P.codes + ((row0 / kBM) * P.nkb + kb) * static_cast<int64_t>(kCodesBytes), kCodesBytes,
                       full_bar(s));
          const int64_t g0 = (static_cast<int64_t>(kb) * kBK) / P.G;
          for (int g = 0; g < groups_kb; ++g)
            bulk_load_1d(c_tile(s) + kCodesBytes + g * 1024, P.sz + (g0 + g) * P.Npad + row0, 1024, full_bar(s));
        } else {
          mbar_expect_tx(full_bar(s), kBHalfBytes + kATileBytes);
          tma_load_2d(c_tile(s), &tmap_w, kb * kBK, static_cast<int>(row0), full_bar(s));
        }
        tma_load_2d(b_tile(s), &tmap_x, kb * kBK, static_cast<int>(tok0), full_bar(s));
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer (leader CTA only)
    if (leader && lane == 0) {
      bool ok = true;
      for (int64_t lt = 0; lt < my_tiles && ok; ++lt) {
        const int as = static_cast<int>(lt & 1);
        const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
        if (!mbar_wait_cluster(accempty_bar(as), aph ^ 1u, abort_flag, P.status)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kBT2);
        for (int kb = 0; kb < P.nkb; ++kb) {
          const int64_t it = lt * P.nkb + kb;
          const int s = static_cast<int>(it % kRaw), t = static_cast<int>(it % kARing);
          const uint32_t ph = static_cast<uint32_t>((it / kRaw) & 1);
          if (!mbar_wait_cluster(ready_bar(s), ph, abort_flag, P.status)) { ok = false; break; }
          tc_fence_after();
          const uint64_t adesc = make_desc_sw128(tiles_base + a_off(s, t)), bdesc = make_desc_sw128(b_tile(s));
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) umma2_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc, (kb | k) ? 1u : 0u);
          umma2_commit_both(empty_bar(s));
          if constexpr (kDequant) umma2_commit_both(aempty_bar(t));
        }
        if (ok) umma2_commit_both(accfull_bar(as));
      }
    }
  } else if (warp == 2) {
    // ---------------------------------------------------------------- stage finisher / SparseAdd
    if (my_iters > 0) {
      auto bucket_of = [&](int64_t it) { return ((tile_of(it) / P.m_tiles) * 2 + rank) * P.n_kblocks + (it % P.nkb); };
      auto has_bucket = [&](int64_t it) { return (tile_of(it) / P.m_tiles) * 2 + rank < P.n_rowtiles; };
      auto issue_bounds = [&](int64_t it) {
        if (sparse && it < my_iters && lane < 2) {
          if (has_bucket(it)) cp_async_4(smem_u32(&bound_ring[it % kBoundSlots][lane]), P.bucket_ptr + bucket_of(it) + lane);
          else bound_ring[it % kBoundSlots][lane] = 0;
        }
      };
      auto issue_records = [&](int64_t it) {
        if (sparse && it < my_iters) {
          const int32_t e0 = bound_ring[it % kBoundSlots][0], e1 = bound_ring[it % kBoundSlots][1];
          const int32_t n = (e1 - e0 < kRecCap) ? e1 - e0 : kRecCap;
          for (int32_t j = lane; j < n; j += 32) cp_async_8(smem_u32(&rec_ring[it % kRecSlots][j]), P.Sb + e0 + j);
        }
      };
      for (int64_t j = 0; j < 2 * kLook; ++j) issue_bounds(j);
      cp_async_commit();
      cp_async_wait_all();
      __syncwarp();
      for (int64_t j = 0; j < kLook; ++j) {
        issue_records(j);
        cp_async_commit();
      }
      for (int64_t it = 0; it < my_iters; ++it) {
        const int s = static_cast<int>(it % kRaw), t = static_cast<int>(it % kARing);
        const uint32_t ph = static_cast<uint32_t>((it / kRaw) & 1), pht = static_cast<uint32_t>((it / kARing) & 1);
        // group(j) = { bounds(j + 2 kLook), records(j + kLook) }: with at most kLook - 1 groups pending,
        // group(it - kLook) has landed, i.e. records(it) and bounds(it + kLook)
        cp_async_wait_group<kLook - 1>();
        __syncwarp();
        issue_bounds(it + 2 * kLook);
        issue_records(it + kLook);
        cp_async_commit();
        if (!mbar_wait(kDequant ? deq_bar(t) : full_bar(s), kDequant ? pht : ph, abort_flag, P.status)) break;
        if (sparse) {
          const int32_t e0 = bound_ring[it % kBoundSlots][0], e1 = bound_ring[it % kBoundSlots][1];
          unsigned char* A = tiles_ptr + a_off(s, t);
          for (int32_t j = lane; j < e1 - e0; j += 32) {
            const uint2 rec = (j < kRecCap) ? rec_ring[it % kRecSlots][j] : __ldg(P.Sb + e0 + j);
            const int r = static_cast<int>(rec.x >> 6), c = static_cast<int>(rec.x & 63);
            __nv_bfloat16* el = reinterpret_cast<__nv_bfloat16*>(A + r * 128 + (((c >> 3) ^ (r & 7)) << 4) + (c & 7) * 2);
            *el = __float2bfloat16_rn(__bfloat162float(*el) + __uint_as_float(rec.y));
          }
          fence_async_smem();
          __syncwarp();
        }
        if (lane == 0) mbar_arrive_cluster(ready_bar(s), 0);
      }
      cp_async_wait_all();
    }
  } else if (warp >= kDeqWarp0 && warp < kDeqWarp0 + kNumDeqWarps) {
    // ---------------------------------------------------------------- dequantisation warps
    if constexpr (kDequant) {
      const int dw = warp - kDeqWarp0;
      const int sub = lane >> 3, chunk = lane & 7;
      const int gsel = (P.G < kBK) ? (chunk * 8) / P.G : 0;
      for (int64_t it = 0; it < my_iters; ++it) {
        const int s = static_cast<int>(it % kRaw), t = static_cast<int>(it % kARing);
        const uint32_t ph = static_cast<uint32_t>((it / kRaw) & 1), pht = static_cast<uint32_t>((it / kARing) & 1);
        unsigned char* A = tiles_ptr + a_off(s, t);
        const unsigned char* C = tiles_ptr + raw_off(s) + kBHalfBytes;
        const float2* SZ = reinterpret_cast<const float2*>(C + kCodesBytes) + gsel * kBM;
        if (!mbar_wait(full_bar(s), ph, abort_flag, P.status)) break;
        if (!mbar_wait(aempty_bar(t), pht ^ 1u, abort_flag, P.status)) break;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const int r = dw * 16 + i * 4 + sub;
          const uint32_t w = *reinterpret_cast<const uint32_t*>(C + r * 32 + chunk * 4);
          const uint4 v = dequant_word<kFast>(w, SZ[r]);
          *reinterpret_cast<uint4*>(A + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) mbar_arrive(deq_bar(t));
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ---------------------------------------------------------------- epilogue (own 128 rows)
    const int qd = warp & 3;
    for (int64_t lt = 0; lt < my_tiles; ++lt) {
      const int64_t tile = pair + lt * n_pairs;
      const int64_t n_tile = tile / P.m_tiles, m_tile = tile % P.m_tiles;
      const int as = static_cast<int>(lt & 1);
      const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
      if (!mbar_wait(accfull_bar(as), aph, abort_flag, P.status)) break;
      tc_fence_after();
      const int64_t n = n_tile * 256 + rank * 128 + qd * 32 + lane;
      const float bias = (P.bias != nullptr && n < P.N) ? P.bias[n] : 0.f;
      const int64_t m0 = m_tile * kBT2;
      const int mlimit = static_cast<int>((P.M - m0 < kBT2) ? P.M - m0 : kBT2);
      for (int c0 = 0; c0 < kBT2; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + static_cast<uint32_t>(as * kBT2 + c0), v);
        if (n < P.N && c0 < mlimit) {
          const int cnt = mlimit - c0;
          if (P.y_f32) {
            float* yp = static_cast<float*>(P.y) + (m0 + c0) * P.N + n;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < cnt) *yp = __uint_as_float(v[j]) + bias;
              yp += P.N;
            }
          } else {
            __nv_bfloat16* yp = static_cast<__nv_bfloat16*>(P.y) + (m0 + c0) * P.N + n;
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              if (j < cnt) *yp = __float2bfloat16_rn(__uint_as_float(v[j]) + bias);
              yp += P.N;
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(accempty_bar(as), 0);
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();          // no CTA leaves while its peer may still signal it or read its tiles
  tc_fence_after();
  if (warp == 1) tmem_dealloc2(tmem_base, kTmemCols);
}

template <int kRaw, bool kDequant, bool kFast>
szo_status launch_tc2(const CUtensorMap& mx, const CUtensorMap& mw, const TcParams& P, int sms, cudaStream_t st) {
  constexpr size_t raw = kBHalfBytes + (kDequant ? kCodesBytes + kSzBytes : kATileBytes);
  constexpr size_t smem = kRaw * raw + (kDequant ? kARing * kATileBytes : 0) + 1024;
  auto kern = szo_linear_tc2_kernel<kRaw, kDequant, kFast>;
  static bool configured = false;
  if (!configured) {
    SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    configured = true;
  }
  const int64_t tiles = P.m_tiles * P.n_tiles;
  const int64_t max_pairs = sms / 2;
  const unsigned grid = static_cast<unsigned>(2 * (tiles < max_pairs ? tiles : max_pairs));
  kern<<<grid, kNumWarps * 32, smem, st>>>(mx, mw, P);
  count_launch();
  SZO_CHECK_LAUNCH("szo_linear_tc2_kernel");
  return SZO_OK;
}

}  // namespace

// Pair-tile launch: tmap_x must have a [128 x 64] box; P.m_tiles / P.n_tiles count 256-wide tiles.
szo_status linear_fwd_tc2(const szo_linear* p, const CUtensorMap& mx, const CUtensorMap& mw, const tc::TcParams& P,
                          int sms, cudaStream_t st) {
  if (p->G == 0) return launch_tc2<6, false, false>(mx, mw, P, sms, st);
  if (p->sz_dtype == SZO_BF16) return launch_tc2<7, true, true>(mx, mw, P, sms, st);
  return launch_tc2<7, true, false>(mx, mw, P, sms, st);
}

}  // namespace szo
