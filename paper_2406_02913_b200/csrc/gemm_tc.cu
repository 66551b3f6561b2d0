// Tensor-core path of the decomposed linear layer for sm_100a:
//   y[m, n] = sum_k x[m,k] * (Dequantize(Q)[n,k] + S[n,k]) + bias[n]
// as one persistent, warp-specialised tcgen05 kernel (appendix "Implementation of Sparse Operations
// in Linear Layers": DenseMM(SparseAdd(w_sparse, Dequantize(Q(w_dense))), x)).
//
// Orientation: the WEIGHT is the MMA's A operand (128 rows of W per tile = UMMA M), the tokens are
// the N dimension (BT <= 256 per tile).  A weight element is therefore dequantised once per
// 2*BT flops, and the accumulator D[n, m] sits in TMEM with one output feature per lane.
//
// Per CTA (one per SM, static round-robin over tiles):
//   warp 0       TMA producer: x tile [BT x 64] bf16 (and the bf16 weight tile in dense mode) with
//                the 128-byte swizzle, completion on full[s]
//   warp 1       allocates TMEM, issues tcgen05.mma (one thread), commits to empty[s] / acc_full
//   warps 4-11   weight producers: int4 codes -> bf16 (q*scale+zero) written in the swizzled K-major
//                layout the MMA descriptor expects, then the tile's sparse values are added in shared
//                memory (SparseAdd), fence.proxy.async, arrive on a_ready[s]
//   warps 12-15  epilogue: tcgen05.ld of the fp32 accumulator, + bias, store y; double-buffered
//                accumulator so the next tile's main loop overlaps
// Every mbarrier wait is bounded; on expiry the kernel records SZO_ERR_TIMEOUT in the device status
// word, lets in-flight copies land, frees its TMEM and returns.
#include <cstdlib>

#include "tc_common.cuh"

namespace szo {

namespace {

using namespace tc;

constexpr int kCStages = 4;   // code-tile stages (cover the TMA latency)
constexpr int kASlots = 4;    // dequantised weight slots (cover conversion + SparseAdd)

// ------------------------------------------------------------------------------ the kernel
// Three rings in shared memory, each with its own life time:
//   X ring  token tile [BT x 64] bf16 (+ the bf16 weight tile in dense mode): TMA -> MMA
//   C ring  packed codes [128 x 32 B] + (scale, zero) strip of the k-block:      TMA -> conversion
//   A ring  dequantised weight tile [128 x 64] bf16, swizzled K-major:           conversion -> MMA
// so that the small code tiles can be fetched far ahead while the large token tiles are held only
// for the TMA latency.  The eight conversion warps form kGroups groups that take alternate
// k-blocks, which keeps several stages in conversion at once.
// kDequant: A tile produced from int4 codes (else loaded as bf16 by TMA).  kFast: bf16 scales/zeros.
template <int BT, int kXS, bool kDequant, bool kFast>
__global__ void __launch_bounds__(kNumWarps * 32, 1)
szo_linear_tc_kernel(const __grid_constant__ CUtensorMap tmap_x, const __grid_constant__ CUtensorMap tmap_w,
                     const TcParams P) {
  constexpr int kBTileBytes = BT * kBK * 2;
  constexpr int kXStageBytes = kBTileBytes + (kDequant ? 0 : kATileBytes);
  constexpr int kCStageBytes = kCodesBytes + kSzBytes;
  constexpr int kCS = kDequant ? kCStages : 1;               // C ring stages
  constexpr int kAS = kDequant ? kASlots : kXS;                    // A ring slots (dense: the X stage itself)
  constexpr int kGroups = 2, kWarpsPerGroup = kNumDeqWarps / kGroups;
  constexpr int kAccStride = BT < 32 ? 32 : BT;             // TMEM columns per accumulator buffer
  constexpr uint32_t kTmemCols = static_cast<uint32_t>(2 * kAccStride);
  constexpr uint32_t kIdesc = make_idesc(kBM, BT);
  constexpr uint32_t kXBase = 0, kCBase = kXS * kXStageBytes, kABase = kCBase + (kDequant ? kCS * kCStageBytes : 0);

  extern __shared__ unsigned char smem_raw[];
  __shared__ __align__(8) unsigned long long bars[2 * kXS + 2 * kCS + 3 * kAS + 4 + 2 * kRecSlots];
  __shared__ __align__(16) uint2 rec_ring[kRecSlots][kRecCap];      // sparse records, per k-block
  __shared__ __align__(8) int32_t bound_ring[kBoundSlots][2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag_s;

  const uint32_t tiles_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
  unsigned char* tiles_ptr = smem_raw + (tiles_base - smem_u32(smem_raw));
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &abort_flag_s;

  auto xfull_bar = [&](int s) { return smem_u32(&bars[s]); };                  // X stage landed (TMA)
  auto xempty_bar = [&](int s) { return smem_u32(&bars[kXS + s]); };           // its MMAs retired
  auto cfull_bar = [&](int c) { return smem_u32(&bars[2 * kXS + c]); };        // C stage landed (TMA)
  auto cempty_bar = [&](int c) { return smem_u32(&bars[2 * kXS + kCS + c]); }; // converted by its group
  auto adone_bar = [&](int t) { return smem_u32(&bars[2 * kXS + 2 * kCS + t]); };            // A slot written
  auto aready_bar = [&](int t) { return smem_u32(&bars[2 * kXS + 2 * kCS + kAS + t]); };     // sparse values added
  auto aempty_bar = [&](int t) { return smem_u32(&bars[2 * kXS + 2 * kCS + 2 * kAS + t]); }; // its MMAs retired
  auto accfull_bar = [&](int a) { return smem_u32(&bars[2 * kXS + 2 * kCS + 3 * kAS + a]); };
  auto accempty_bar = [&](int a) { return smem_u32(&bars[2 * kXS + 2 * kCS + 3 * kAS + 2 + a]); };
  auto recready_bar = [&](int r) { return smem_u32(&bars[2 * kXS + 2 * kCS + 3 * kAS + 4 + r]); };  // records of a k-block landed
  auto recfree_bar = [&](int r) { return smem_u32(&bars[2 * kXS + 2 * kCS + 3 * kAS + 4 + kRecSlots + r]); };  // ... and consumed
  auto b_off = [&](int s) { return kXBase + static_cast<uint32_t>(s) * kXStageBytes; };
  auto c_off = [&](int c) { return kCBase + static_cast<uint32_t>(c) * kCStageBytes; };
  auto a_off = [&](int s, int t) {     // weight tile of iteration (X stage s, A slot t)
    return kDequant ? kABase + static_cast<uint32_t>(t) * kATileBytes : b_off(s) + kBTileBytes;
  };

  const bool sparse = P.Sb != nullptr;
  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int s = 0; s < kXS; ++s) {
      mbar_init(xfull_bar(s), 1);
      mbar_init(xempty_bar(s), 1);
    }
    for (int c = 0; c < kCS; ++c) {
      mbar_init(cfull_bar(c), 1);
      mbar_init(cempty_bar(c), kWarpsPerGroup);
    }
    for (int t = 0; t < kAS; ++t) {
      mbar_init(adone_bar(t), kWarpsPerGroup);
      mbar_init(aready_bar(t), kWarpsPerGroup);
      mbar_init(aempty_bar(t), 1);
    }
    for (int a = 0; a < 2; ++a) {
      mbar_init(accfull_bar(a), 1);
      mbar_init(accempty_bar(a), 4);
    }
    for (int r = 0; r < kRecSlots; ++r) {
      mbar_init(recready_bar(r), 1);
      mbar_init(recfree_bar(r), kWarpsPerGroup);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) tmem_alloc(smem_u32(&tmem_base_slot), kTmemCols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  // tiles of this CTA: tile(lt) = blockIdx.x + lt * gridDim.x, tile = n_tile * m_tiles + m_tile
  const int total_tiles = static_cast<int>(P.m_tiles * P.n_tiles), m_tiles = static_cast<int>(P.m_tiles);
  const int my_tiles = (total_tiles > static_cast<int>(blockIdx.x))
                           ? (total_tiles - static_cast<int>(blockIdx.x) + static_cast<int>(gridDim.x) - 1) / static_cast<int>(gridDim.x)
                           : 0;
  const int nkb = P.nkb;

  if (warp == 0) {
    // ---------------------------------------------------------------- X producer (token tiles)
    if (lane == 0) {
      RingPos x{0, 0};
      bool ok = true;
      for (int lt = 0; lt < my_tiles && ok; ++lt) {
        const int tile = blockIdx.x + lt * gridDim.x;
        const int m0 = (tile % m_tiles) * BT, n0 = (tile / m_tiles) * kBM;
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(xempty_bar(x.idx), x.phase ^ 1u, abort_flag, P.status)) { ok = false; break; }
          mbar_expect_tx(xfull_bar(x.idx), kXStageBytes);
          tma_load_2d(tiles_base + b_off(x.idx), &tmap_x, kb * kBK, m0, xfull_bar(x.idx));
          if constexpr (!kDequant) tma_load_2d(tiles_base + a_off(x.idx, 0), &tmap_w, kb * kBK, n0, xfull_bar(x.idx));
          x.advance(kXS);
        }
      }
    }
  } else if (warp == 3) {
    // ---------------------------------------------------------------- C producer (codes, scale/zero)
    if constexpr (kDequant) {
      if (lane == 0) {
        const int groups_kb = (P.G < kBK) ? kBK / P.G : 1;     // scale groups per k-block
        RingPos c{0, 0};
        bool ok = true;
        for (int lt = 0; lt < my_tiles && ok; ++lt) {
          const int n_tile = (blockIdx.x + lt * gridDim.x) / m_tiles;
          const uint8_t* codes = P.codes + static_cast<int64_t>(n_tile) * nkb * kCodesBytes;
          const float2* sz = P.sz + static_cast<int64_t>(n_tile) * kBM;
          for (int kb = 0; kb < nkb; ++kb) {
            if (!mbar_wait(cempty_bar(c.idx), c.phase ^ 1u, abort_flag, P.status)) { ok = false; break; }
            mbar_expect_tx(cfull_bar(c.idx), kCodesBytes + groups_kb * 1024);
            bulk_load_1d(tiles_base + c_off(c.idx), codes + static_cast<int64_t>(kb) * kCodesBytes, kCodesBytes,
                         cfull_bar(c.idx));
            const int g0 = (kb * kBK) / P.G;
            for (int g = 0; g < groups_kb; ++g)
              bulk_load_1d(tiles_base + c_off(c.idx) + kCodesBytes + g * 1024, sz + static_cast<int64_t>(g0 + g) * P.Npad,
                           1024, cfull_bar(c.idx));
            c.advance(kCS);
          }
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------------------------------------- MMA issuer
    if (lane == 0) {
      RingPos x{0, 0}, a{0, 0};
      bool ok = true;
      for (int lt = 0; lt < my_tiles && ok; ++lt) {
        const int as = lt & 1;
        const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
        if (!mbar_wait(accempty_bar(as), aph ^ 1u, abort_flag, P.status, 0)) break;
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + static_cast<uint32_t>(as * kAccStride);
        for (int kb = 0; kb < nkb; ++kb) {
          if (!mbar_wait(xfull_bar(x.idx), x.phase, abort_flag, P.status, 0)) { ok = false; break; }
          if constexpr (kDequant) {     // converted (and, with sparse entries, already SparseAdd-ed) by the conversion warps
            if (!mbar_wait(adone_bar(a.idx), a.phase, abort_flag, P.status, 0)) { ok = false; break; }
          } else if (sparse) {          // dense weight tile: SparseAdd-ed by warp 2
            if (!mbar_wait(aready_bar(a.idx), a.phase, abort_flag, P.status, 0)) { ok = false; break; }
          }
          tc_fence_after();
          const uint64_t adesc = make_desc_sw128(tiles_base + a_off(x.idx, a.idx));
          const uint64_t bdesc = make_desc_sw128(tiles_base + b_off(x.idx));
#pragma unroll
          for (int k = 0; k < kBK / kUmmaK; ++k) {
            // advance both descriptors by 16 elements = 32 bytes (>> 4 = 2) inside the swizzle row
            umma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, kIdesc, (kb | k) ? 1u : 0u);
          }
          umma_commit(xempty_bar(x.idx));
          if constexpr (kDequant) umma_commit(aempty_bar(a.idx));
          x.advance(kXS);
          a.advance(kAS);
        }
        if (ok) umma_commit(accfull_bar(as));
      }
    }
  } else if (warp == 2) {
    // ---------------------------------------------------------------- sparse-record warp
    // Brings the bucket bounds and the sparse records (position in tile, fp32 value) of every
    // (tile, k-block) into two small rings in shared memory, a few k-blocks ahead of their use.
    // Plain global loads into registers, stored to shared memory two iterations later (two register
    // sets in flight), so that no load latency sits on this warp's loop.  Warps 4-11 add the values to
    // the weight tile (after converting it, or after TMA delivered a dense bf16 tile).
    //   iteration it:  store {bounds(it+6), records(it+3)} loaded at it-2, signal recready(it+3),
    //                  load  {bounds(it+8), records(it+5)}    (records(it+5) are addressed by
    //                  bounds(it+5), stored at it-1)
    if (sparse && my_tiles > 0) {
      const int n_kblocks = static_cast<int>(P.n_kblocks);
      const int my_iters = my_tiles * nkb;
      struct Cursor {
        int it, lt, kb, bucket0;     // bucket0 = n_tile * n_kblocks of the cursor's tile
      };
      auto make_cursor = [&]() { return Cursor{0, 0, 0, static_cast<int>(blockIdx.x / m_tiles) * n_kblocks}; };
      auto step = [&](Cursor& c) {
        ++c.it;
        if (++c.kb == nkb) {
          c.kb = 0;
          ++c.lt;
          c.bucket0 = ((blockIdx.x + c.lt * gridDim.x) / m_tiles) * n_kblocks;
        }
      };
      struct Loaded {
        int32_t bound;               // lanes 0,1: bucket_ptr[b], bucket_ptr[b+1]
        uint2 rec[kRecCap / 32];     // records lane, lane + 32, ... of the bucket
        int32_t n;                   // records of the bucket held in the ring (<= kRecCap)
      };
      Cursor cb = make_cursor(), cr = make_cursor();       // bounds stream, records stream
      auto load_set = [&](Loaded& L) {                     // bounds(cb.it), records(cr.it)
        L.bound = 0;
        L.n = 0;
        if (cb.it < my_iters) {
          if (lane < 2) L.bound = __ldg(P.bucket_ptr + cb.bucket0 + cb.kb + lane);
        }
        if (cr.it < my_iters) {
          const int32_t e0 = bound_ring[cr.it & (kBoundSlots - 1)][0], e1 = bound_ring[cr.it & (kBoundSlots - 1)][1];
          L.n = (e1 - e0 < kRecCap) ? e1 - e0 : kRecCap;
#pragma unroll
          for (int q = 0; q < kRecCap / 32; ++q)
            if (lane + 32 * q < L.n) L.rec[q] = __ldg(P.Sb + e0 + lane + 32 * q);
        }
      };
      auto store_set = [&](const Loaded& L) {              // then advance both streams
        if (cb.it < my_iters) {
          if (lane < 2) bound_ring[cb.it & (kBoundSlots - 1)][lane] = L.bound;
          step(cb);
        }
        if (cr.it < my_iters) {
#pragma unroll
          for (int q = 0; q < kRecCap / 32; ++q)
            if (lane + 32 * q < L.n) rec_ring[cr.it & (kRecSlots - 1)][lane + 32 * q] = L.rec[q];
          step(cr);
        }
      };
      static_assert(kRecSlots == 8 && kBoundSlots == 16, "ring sizes are part of the schedule");
      // prologue: bounds 0..5 and records 0..2 directly, then prime the two register sets
      Loaded set0, set1;
      for (int j = 0; j < 6; ++j) {                        // bounds only (the records stream idles)
        Loaded L;
        L.bound = 0;
        L.n = 0;
        if (cb.it < my_iters && lane < 2) L.bound = __ldg(P.bucket_ptr + cb.bucket0 + cb.kb + lane);
        if (cb.it < my_iters) {
          if (lane < 2) bound_ring[cb.it & (kBoundSlots - 1)][lane] = L.bound;
          step(cb);
        }
      }
      __syncwarp();
      for (int j = 0; j < 3; ++j) {                        // records 0..2 (bounds stream idles)
        if (cr.it < my_iters) {
          const int32_t e0 = bound_ring[cr.it & (kBoundSlots - 1)][0], e1 = bound_ring[cr.it & (kBoundSlots - 1)][1];
          const int32_t n = (e1 - e0 < kRecCap) ? e1 - e0 : kRecCap;
          for (int32_t q = lane; q < n; q += 32) rec_ring[cr.it & (kRecSlots - 1)][q] = __ldg(P.Sb + e0 + q);
          __syncwarp();
          if (lane == 0) mbar_arrive(recready_bar(cr.it & (kRecSlots - 1)));
          step(cr);
        }
      }
      // the two sets in flight: {bounds(6), records(3)} and {bounds(7), records(4)}
      {
        Cursor sb = cb, sr = cr;
        load_set(set0);
        step(cb);
        step(cr);
        load_set(set1);
        cb = sb;
        cr = sr;
      }
      // one iteration, on the register set that was loaded two iterations ago
      auto iteration = [&](int it, Loaded& L) -> bool {
        // records(it+3) reuse the ring slot of k-block it-5: wait until the warps that add them have
        // read it (that slot's previous phase, so the parity wait cannot alias)
        if (it >= 5) {
          const int prev = it - 5;
          if (!mbar_wait(recfree_bar(prev & (kRecSlots - 1)), static_cast<uint32_t>((prev / kRecSlots) & 1), abort_flag, P.status))
            return false;
        }
        const int rec_it = cr.it;
        store_set(L);                                      // {bounds(it+6), records(it+3)}
        __syncwarp();
        if (lane == 0 && rec_it < my_iters) mbar_arrive(recready_bar(rec_it & (kRecSlots - 1)));
        {                                                  // {bounds(it+8), records(it+5)}
          Cursor sb = cb, sr = cr;
          step(cb);
          step(cr);
          load_set(L);
          cb = sb;
          cr = sr;
        }
        return true;
      };
      for (int it = 0; it < my_iters; it += 2) {
        if (!iteration(it, set0)) break;
        if (it + 1 < my_iters && !iteration(it + 1, set1)) break;
      }
    }
  } else if (warp >= kDeqWarp0 && warp < kDeqWarp0 + kNumDeqWarps) {
    // ---------------------------------------------------------------- conversion warps
    // Group gq converts the k-blocks it = gq (mod kGroups); inside a group each warp converts 32 rows
    // in eight passes of 4 rows x 8 sixteen-byte chunks (conflict-free loads and stores).
    if constexpr (kDequant) {
      const int dw = warp - kDeqWarp0;
      const int gq = dw / kWarpsPerGroup, wq = dw % kWarpsPerGroup;
      constexpr int kRowsPerWarp = kBM / kWarpsPerGroup, kPasses = kRowsPerWarp / 4;
      const int sub = lane >> 3, chunk = lane & 7;
      const int gsel = (P.G < kBK) ? (chunk * 8) / P.G : 0;
      RingPos c{0, 0}, a{0, 0};
      for (int j = 0; j < gq; ++j) {
        c.advance(kCS);
        a.advance(kAS);
      }
      const int my_iters = my_tiles * nkb;
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
        // the bucket's sparse records (usually fewer than 32): one per lane, fetched before the conversion
        int32_t e0 = 0, e1 = 0;
        uint2 rec = make_uint2(0xFFFFFFFFu, 0u);
        if (sparse) {
          if (!mbar_wait(recready_bar(it & (kRecSlots - 1)), static_cast<uint32_t>((it / kRecSlots) & 1), abort_flag, P.status)) break;
          e0 = bound_ring[it & (kBoundSlots - 1)][0];
          e1 = bound_ring[it & (kBoundSlots - 1)][1];
          if (lane < e1 - e0) rec = rec_ring[it & (kRecSlots - 1)][lane];
        }
        if (!mbar_wait(aempty_bar(a.idx), a.phase ^ 1u, abort_flag, P.status)) break;
#pragma unroll
        for (int i = 0; i < kPasses; ++i) {
          const int r = wq * kRowsPerWarp + i * 4 + sub;
          const uint4 v = dequant_word<kFast>(w[i], zs[i]);
          *reinterpret_cast<uint4*>(A + r * 128 + ((chunk ^ (r & 7)) << 4)) = v;
        }
        if (e1 > e0) {
          // SparseAdd: add the bucket's fp32 values to this warp's rows of the bf16 tile
          __syncwarp();
          auto apply = [&](uint2 rc) {
            if (static_cast<int>(rc.x >> 7) / kRowsPerWarp == wq) {     // rc.x: byte offset in the swizzled tile
              __nv_bfloat16* el = reinterpret_cast<__nv_bfloat16*>(A + rc.x);
              *el = __float2bfloat16_rn(__bfloat162float(*el) + __uint_as_float(rc.y));
            }
          };
          if (lane < e1 - e0) apply(rec);
          for (int32_t j = lane + 32; j < e1 - e0; j += 32)
            apply((j < kRecCap) ? rec_ring[it & (kRecSlots - 1)][j] : __ldg(P.Sb + e0 + j));
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(adone_bar(a.idx));
          mbar_arrive(cempty_bar(c.idx));
          if (sparse) mbar_arrive(recfree_bar(it & (kRecSlots - 1)));
        }
#pragma unroll
        for (int j = 0; j < kGroups; ++j) {
          c.advance(kCS);
          a.advance(kAS);
        }
      }
    } else if (sparse) {
      // dense bf16 weight tile delivered by TMA: the same warps add the bucket's sparse values
      const int dw = warp - kDeqWarp0;
      const int gq = dw / kWarpsPerGroup, wq = dw % kWarpsPerGroup;
      constexpr int kRowsPerWarp = kBM / kWarpsPerGroup;
      RingPos x{0, 0};
      for (int j = 0; j < gq; ++j) x.advance(kXS);
      const int my_iters = my_tiles * nkb;
      for (int it = gq; it < my_iters; it += kGroups) {
        if (!mbar_wait(recready_bar(it & (kRecSlots - 1)), static_cast<uint32_t>((it / kRecSlots) & 1), abort_flag, P.status)) break;
        const int32_t e0 = bound_ring[it & (kBoundSlots - 1)][0], e1 = bound_ring[it & (kBoundSlots - 1)][1];
        if (!mbar_wait(xfull_bar(x.idx), x.phase, abort_flag, P.status)) break;
        unsigned char* A = tiles_ptr + a_off(x.idx, x.idx);
        for (int32_t j = lane; j < e1 - e0; j += 32) {
          const uint2 rc = (j < kRecCap) ? rec_ring[it & (kRecSlots - 1)][j] : __ldg(P.Sb + e0 + j);
          if (static_cast<int>(rc.x >> 7) / kRowsPerWarp == wq) {
            __nv_bfloat16* el = reinterpret_cast<__nv_bfloat16*>(A + rc.x);
            *el = __float2bfloat16_rn(__bfloat162float(*el) + __uint_as_float(rc.y));
          }
        }
        fence_async_smem();
        __syncwarp();
        if (lane == 0) {
          mbar_arrive(aready_bar(x.idx));
          mbar_arrive(recfree_bar(it & (kRecSlots - 1)));
        }
#pragma unroll
        for (int j = 0; j < kGroups; ++j) x.advance(kXS);
      }
    }
  } else if (warp >= kEpiWarp0) {
    // ---------------------------------------------------------------- epilogue
    const int qd = warp & 3;                        // TMEM lane quarter this warp may read
    for (int lt = 0; lt < my_tiles; ++lt) {
      const int tile = blockIdx.x + lt * gridDim.x;
      const int64_t n_tile = tile / m_tiles, m_tile = tile % m_tiles;
      const int as = lt & 1;
      const uint32_t aph = static_cast<uint32_t>((lt >> 1) & 1);
      if (!mbar_wait(accfull_bar(as), aph, abort_flag, P.status, 256)) break;
      tc_fence_after();
      const int64_t n = n_tile * kBM + qd * 32 + lane;
      const float bias = (P.bias != nullptr && n < P.N) ? P.bias[n] : 0.f;
      const int64_t m0 = m_tile * BT;
      const int mlimit = static_cast<int>((P.M - m0 < BT) ? P.M - m0 : BT);   // valid tokens in this tile
      for (int c0 = 0; c0 < BT; c0 += 32) {
        uint32_t v[32];
        tmem_ld32(tmem_base + (static_cast<uint32_t>(qd * 32) << 16) + static_cast<uint32_t>(as * kAccStride + c0), v);
        if (n < P.N && c0 < mlimit) {
          const int cnt = mlimit - c0;                 // tokens c0 .. c0+cnt-1 are valid (cnt may exceed 32)
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
      if (lane == 0) mbar_arrive(accempty_bar(as));
    }
  }

  // ------------------------------------------------------------------ teardown
  if (*abort_flag) {
    // a wait expired somewhere: give copies and MMAs in flight time to land before the CTA exits
    for (int i = 0; i < 200; ++i) __nanosleep(1000);
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (warp == 1) tmem_dealloc(tmem_base, kTmemCols);
}

// ------------------------------------------------------------------------------ host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// bf16 matrix [rows, cols] row-major, box [box_rows x 64 cols], 128-byte swizzle, zero fill.
szo_status make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  SZO_REQUIRE(fn != nullptr, SZO_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols) * 2};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK), static_cast<cuuint32_t>(box_rows)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  SZO_REQUIRE(r == CUDA_SUCCESS, SZO_ERR_CUDA, "cuTensorMapEncodeTiled failed (%d)", static_cast<int>(r));
  return SZO_OK;
}

struct TcPlan {
  CUtensorMap w_map;    // dense bf16 weight (G == 0) or the packed codes as bytes (G > 0)
  int sms;
  int32_t* tickets;     // device, [sms / 2][2][4], zero between launches (K-split tiles of the pair kernel)
};

// Work schedule of the pair-tile kernel over `tiles` pair tiles (see TcParams).  The last, partial
// round of tiles (all of them when there are fewer tiles than clusters) is split along K into up to
// four parts of whole scale groups, at least eight k-blocks each, when a workspace is available.
struct PairSchedule {
  int n_pairs, full_rounds, tail_tiles, tail_parts;
  int tail_kb[5];
  size_t ws_bytes;
};
PairSchedule pair_schedule(int64_t tiles, int nkb, int G, int sms, bool allow_split) {
  PairSchedule sc{};
  const int max_pairs = sms / 2;
  sc.full_rounds = static_cast<int>(tiles / max_pairs);
  sc.tail_tiles = static_cast<int>(tiles % max_pairs);
  sc.tail_parts = 1;
  const int kb_per_group = (G > kBK) ? G / kBK : 1;
  const int groups = nkb / kb_per_group;
  if (allow_split && sc.tail_tiles > 0) {
    int parts = max_pairs / sc.tail_tiles;
    if (parts > 4) parts = 4;
    while (parts > 1 && (groups / parts) * kb_per_group < 8) --parts;
    // parking and summing the parts costs about as much as 30 k-blocks of a tile
    if (parts > 1 && nkb - nkb / parts < 40) parts = 1;
    sc.tail_parts = parts;
  }
  for (int i = 0; i <= 4; ++i) {
    const int ii = i < sc.tail_parts ? i : sc.tail_parts;
    sc.tail_kb[i] = static_cast<int>((static_cast<int64_t>(groups) * ii) / sc.tail_parts) * kb_per_group;
  }
  sc.tail_kb[sc.tail_parts] = nkb;
  sc.n_pairs = sc.full_rounds > 0 ? max_pairs : sc.tail_tiles * sc.tail_parts;
  sc.ws_bytes = sc.tail_parts > 1 ? static_cast<size_t>(sc.tail_tiles) * sc.tail_parts * 2 * 256 * kBM * sizeof(float) : 0;
  return sc;
}

// uint8 matrix [rows, cols_bytes] row-major, box [128 rows x 32 bytes], no swizzle.
szo_status make_codes_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols_bytes) {
  EncodeTiledFn fn = encode_fn();
  SZO_REQUIRE(fn != nullptr, SZO_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
  const cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols_bytes), static_cast<cuuint64_t>(rows)};
  const cuuint64_t strides[1] = {static_cast<cuuint64_t>(cols_bytes)};
  const cuuint32_t box[2] = {static_cast<cuuint32_t>(kBK / 2), static_cast<cuuint32_t>(kBM)};
  const cuuint32_t estr[2] = {1, 1};
  const CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<void*>(base), dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  SZO_REQUIRE(r == CUDA_SUCCESS, SZO_ERR_CUDA, "cuTensorMapEncodeTiled (codes) failed (%d)", static_cast<int>(r));
  return SZO_OK;
}

template <int BT, int kXS, bool kDequant, bool kFast>
szo_status launch_tc(const CUtensorMap& mx, const CUtensorMap& mw, const TcParams& P, int sms, cudaStream_t st) {
  constexpr size_t smem = static_cast<size_t>(kXS) * (BT * kBK * 2 + (kDequant ? 0 : kATileBytes)) +
                          (kDequant ? kCStages * (kCodesBytes + kSzBytes) + kASlots * kATileBytes : 0) + 1024;
  auto kern = szo_linear_tc_kernel<BT, kXS, kDequant, kFast>;
  static bool configured = false;
  if (!configured) {
    SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
    configured = true;
  }
  const int64_t tiles = P.m_tiles * P.n_tiles;
  const unsigned grid = static_cast<unsigned>(tiles < sms ? tiles : sms);
  kern<<<grid, kNumWarps * 32, smem, st>>>(mx, mw, P);
  count_launch();
  SZO_CHECK_LAUNCH("szo_linear_tc_kernel");
  return SZO_OK;
}

// kXD / kXQ: token-tile stages in dense and in dequantising mode (the latter also holds the C and A rings)
template <int BT, int kXD, int kXQ>
szo_status dispatch_kind(const szo_linear* p, const CUtensorMap& mx, const CUtensorMap& mw, const TcParams& P, int sms,
                         cudaStream_t st) {
  if (p->G == 0) return launch_tc<BT, kXD, false, false>(mx, mw, P, sms, st);
  if (p->sz_dtype == SZO_BF16) return launch_tc<BT, kXQ, true, true>(mx, mw, P, sms, st);
  return launch_tc<BT, kXQ, true, false>(mx, mw, P, sms, st);
}

}  // namespace

szo_status tc_plan_create(szo_linear* p, cudaStream_t) {
  TcPlan* t = new TcPlan();
  int dev = 0;
  t->sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&t->sms, cudaDevAttrMultiProcessorCount, dev);
  // the dense bf16 weight is fetched by TMA; packed codes are fetched with plain bulk copies from the
  // plan's tile-ordered copy, so that map only has to be valid (it is never used)
  const szo_status s = (p->G == 0) ? make_map(&t->w_map, p->codes, p->N, p->K, kBM)
                                   : make_codes_map(&t->w_map, p->codes, p->N, p->K / 2);
  if (s != SZO_OK) {
    delete t;
    return s;
  }
  const size_t tk = static_cast<size_t>(t->sms / 2) * 8 * sizeof(int32_t);
  if (cudaMalloc(&t->tickets, tk) != cudaSuccess || cudaMemset(t->tickets, 0, tk) != cudaSuccess) {
    cudaFree(t->tickets);
    delete t;
    return fail(SZO_ERR_CUDA, "cannot allocate the K-split tickets");
  }
  p->tc = t;
  return SZO_OK;
}

void tc_plan_destroy(szo_linear* p) {
  TcPlan* t = static_cast<TcPlan*>(p->tc);
  if (t) cudaFree(t->tickets);
  delete t;
  p->tc = nullptr;
}

static bool force_one_cta() {
  // SZO_LINEAR_KERNEL=1cta keeps the one-CTA kernel for every M (A/B measurement)
  static const bool v = [] {
    const char* e = getenv("SZO_LINEAR_KERNEL");
    return e != nullptr && e[0] == '1';
  }();
  return v;
}

static int64_t pair_tiles(const szo_linear* const* plans, int n, int64_t M) {
  int64_t nt = 0;
  for (int i = 0; i < n; ++i) nt += ceil_div(plans[i]->N, 256);
  return nt * ceil_div(M, 256);
}

size_t tc_tail_ws_bytes(const szo_linear* const* plans, int n, int64_t M) {
  if (n < 1 || M <= 128 || force_one_cta() || plans[0]->tc == nullptr) return 0;
  const TcPlan* t = static_cast<const TcPlan*>(plans[0]->tc);
  return pair_schedule(pair_tiles(plans, n, M), static_cast<int>(plans[0]->K / kBK), plans[0]->G, t->sms, true).ws_bytes;
}

size_t tc_tail_ws_bound() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return static_cast<size_t>(sms / 2) * 2 * 256 * kBM * sizeof(float);
}

bool tc_can_fuse(const szo_linear* const* plans, int n, int64_t M) {
  if (n < 2 || n > 3 || M <= 128 || force_one_cta()) return false;
  for (int i = 0; i < n; ++i)
    if (plans[i]->G == 0 || plans[i]->tc == nullptr || plans[i]->K != plans[0]->K || plans[i]->G != plans[0]->G ||
        plans[i]->sz_dtype != plans[0]->sz_dtype)
      return false;
  return true;
}

// Pair-tile launch of n matrices that share x (n == 1, or tc_can_fuse).
szo_status linear_fwd_tc_group(const szo_linear* const* plans, int n, const void* x, int64_t M,
                               const uint2* const* S_bucket, void* const* y, int y_dtype, void* ws, size_t ws_bytes,
                               cudaStream_t st) {
  const szo_linear* p0 = plans[0];
  const TcPlan* t = static_cast<const TcPlan*>(p0->tc);
  SZO_REQUIRE(t != nullptr, SZO_ERR_INVALID_ARG, "plan has no tensor-core data");
  SZO_REQUIRE(M < (int64_t(1) << 31), SZO_ERR_SHAPE, "M too large");
  CUtensorMap mx;
  SZO_TRY(make_map(&mx, x, M, p0->K, 128));
  TcParams P{};
  P.M = M; P.K = p0->K; P.G = p0->G; P.nkb = static_cast<int>(p0->K / kBK);
  P.m_tiles = ceil_div(M, 256);
  P.nsub = n;
  int64_t n_tiles = 0;
  for (int i = 0; i < n; ++i) {
    const szo_linear* p = plans[i];
    SZO_REQUIRE(p->N < (int64_t(1) << 31), SZO_ERR_SHAPE, "N too large");
    TcSub& sb = P.sub[i];
    sb.codes = p->codes_tiled;
    sb.sz = p->sz;
    sb.bucket_ptr = p->bucket_ptr;
    sb.Sb = (p->nnz > 0) ? S_bucket[i] : nullptr;
    sb.bias = p->bias;
    sb.y = y[i];
    sb.N = p->N;
    sb.Npad = p->Npad;
    sb.n_rowtiles = static_cast<int>(p->n_rowgroups);
    sb.n_tiles = static_cast<int>(ceil_div(p->N, 256));
    n_tiles += sb.n_tiles;
  }
  P.n_tiles = n_tiles;
  P.y_f32 = (y_dtype == SZO_F32) ? 1 : 0;
  P.status = device_status_word();
  SZO_REQUIRE(P.status != nullptr, SZO_ERR_CUDA, "no device status word");
  const int64_t tiles = P.m_tiles * P.n_tiles;
  SZO_REQUIRE(tiles < (int64_t(1) << 30), SZO_ERR_SHAPE, "too many tiles");
  PairSchedule sc = pair_schedule(tiles, P.nkb, P.G, t->sms, ws != nullptr);
  if (sc.ws_bytes > ws_bytes) sc = pair_schedule(tiles, P.nkb, P.G, t->sms, false);
  P.full_rounds = sc.full_rounds;
  P.tail_tiles = sc.tail_tiles;
  P.tail_parts = sc.tail_parts;
  for (int i = 0; i < 5; ++i) P.tail_kb[i] = sc.tail_kb[i];
  P.partial = static_cast<float*>(ws);
  P.tickets = t->tickets;
  return launch_pair_kernel(p0->G != 0, p0->sz_dtype == SZO_BF16, mx, t->w_map, P, sc.n_pairs, st);
}

szo_status linear_fwd_tc(const szo_linear* p, const void* x, int64_t M, const uint2* S_bucket, void* y,
                         int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st) {
  if (M > 128 && !force_one_cta()) return linear_fwd_tc_group(&p, 1, x, M, &S_bucket, &y, y_dtype, ws, ws_bytes, st);
  const TcPlan* t = static_cast<const TcPlan*>(p->tc);
  SZO_REQUIRE(t != nullptr, SZO_ERR_INVALID_ARG, "plan has no tensor-core data");
  SZO_REQUIRE(M < (int64_t(1) << 31) && p->N < (int64_t(1) << 31), SZO_ERR_SHAPE, "M or N too large");
  int BT = 256;
  if (M <= 16) BT = 16; else if (M <= 32) BT = 32; else if (M <= 64) BT = 64; else if (M <= 128) BT = 128;
  CUtensorMap mx;
  SZO_TRY(make_map(&mx, x, M, p->K, BT));
  TcParams P{};
  P.M = M; P.N = p->N; P.K = p->K; P.G = p->G; P.nkb = static_cast<int>(p->K / kBK);
  P.m_tiles = ceil_div(M, BT); P.n_tiles = ceil_div(p->N, kBM);
  P.codes = p->codes_tiled;
  P.sz = p->sz;
  P.bucket_ptr = p->bucket_ptr;
  P.n_kblocks = p->n_kblocks;
  P.n_rowtiles = p->n_rowgroups;
  P.Npad = p->Npad;
  P.Sb = (p->nnz > 0) ? S_bucket : nullptr;
  P.bias = p->bias;
  P.y = y; P.y_f32 = (y_dtype == SZO_F32) ? 1 : 0;
  P.status = device_status_word();
  SZO_REQUIRE(P.status != nullptr, SZO_ERR_CUDA, "no device status word");
  const CUtensorMap& mw = t->w_map;
  switch (BT) {
    case 16: return dispatch_kind<16, 8, 8>(p, mx, mw, P, t->sms, st);
    case 32: return dispatch_kind<32, 8, 8>(p, mx, mw, P, t->sms, st);
    case 64: return dispatch_kind<64, 8, 8>(p, mx, mw, P, t->sms, st);
    case 128: return dispatch_kind<128, 6, 6>(p, mx, mw, P, t->sms, st);
    default: return dispatch_kind<256, 4, 4>(p, mx, mw, P, t->sms, st);
  }
}

}  // namespace szo
