// Weight-streaming form of the decomposed linear for a handful of tokens (M <= 16):
//   y[m, n] = sum_k x[m,k] * Dequantize(Q)[n,k] + sum_{(n,c) in mask} x[m,c] * S[n,c] + bias[n]
// (appendix "Implementation of Sparse Operations in Linear Layers": the SparseAddMM form, which
// the paper finds the faster one when few tokens are processed).  With so few tokens the layer is
// bound by reading the int4 weights once from HBM, so the kernel is built around that stream, not
// around the tensor cores' peak:
//   * persistent clusters of 8 CTAs: a cluster takes 128-row tiles of the weight in turn and splits
//     K between its CTAs, so that a CTA always works on the same columns and keeps its slice of the
//     activations (8 or 16 tokens) in shared memory for the whole launch, 16-byte chunks permuted
//     so that the lanes' 128-bit reads are free of bank conflicts;
//   * one producer thread per CTA streams the CTA's part of the tiled codes (8 KB per 128-column
//     step, contiguous) and the (scale, zero) entries of the step through an 8-stage ring of bulk
//     copies that complete on mbarriers; it runs ahead across tile boundaries, so the stream never
//     drains;
//   * 8 weight warps own 16 rows each; per step a lane takes 16 bytes (32 codes) of each of its two
//     rows from the stage.  The product runs on warp-level MMAs (m16n8k16: 16 weight rows x 8
//     tokens, the weight as the A operand).  A dot product does not care about the order of k, so
//     lane t uses its own four consecutive columns where the fragment layout names columns
//     (2t, 2t+1, 2t+8, 2t+9), for the weights and the tokens alike;
//   * when the quantization group covers whole steps (G a multiple of 128) the codes are not
//     dequantised one by one: with q the codes of a group, scale s and zero z,
//         sum_k x_k (q_k s + z) = s * sum_k x_k (128 + q_k) + (z - 128 s) * sum_k x_k,
//     where 128 + q_k as bf16 is the code OR-ed into a constant (two instructions per pair of codes),
//     the first sum is the MMA of the codes, the second is formed once per CTA when the activations
//     are staged; scale and zero are applied once per step to the fp32 accumulators.  This is the
//     exact (unrounded) Dequantize(Q).  Smaller groups (32, 64) take the packed-bf16 conversion of
//     the large-M kernel instead;
//   * a ninth warp forms the sparse term of 16 rows of the tile in fp32: its loads from global
//     memory are pipelined over tiles, and the activations at the entries' columns come from the
//     shared memory of the CTA that staged them (distributed shared memory, no trip through L2);
//   * the K-split partial sums meet through distributed shared memory too: a tenth warp of CTA c
//     adds the eight partials of rows 16c .. 16c+15 in CTA order (deterministic), then the sparse
//     term and the bias, and stores y.  Partials and sparse terms are double-buffered and everyone
//     waits only for the barrier of the tile before, so nobody stands still for the sum.
// Codes into a per-row table of 16 values (the non-uniform 4-bit format) take the kernel too: the
// tile's tables (128 rows x 32 bytes as bf16) travel with every step where the (scale, zero) entries
// otherwise are, and every code is looked up there.
// One launch may serve up to three matrices that read the same activations (q/k/v, gate/up of a decoder
// layer): their 128-row tiles are numbered one after the other, and a tile's number names its matrix.
// The activations may be formed while they are staged: silu(x) * x_mul, rounded to bf16 (the
// gated MLP's product, which then never goes through device memory).
// Waits on mbarriers are bounded (status SZO_ERR_TIMEOUT); after a failed wait a thread keeps the
// control flow, and with it the cluster barriers, but skips waiting and copying.
#include <mutex>

#include "tc_common.cuh"

namespace szo {

namespace {

constexpr int kRowsWarp = 16;    // weight rows per warp (MMA M)
constexpr int kWarps = 8;        // weight warps; then one warp each: sparse term, sum over the K-parts, producer
constexpr int kWarpSparse = kWarps, kWarpSum = kWarps + 1, kWarpProducer = kWarps + 2;
constexpr int kRowsCta = kRowsWarp * kWarps;   // 128: one tile of the plan's tiled codes
constexpr int kSplit = 8;        // CTAs per cluster = parts K is split in
constexpr int kTok = 8;          // tokens per token tile (MMA N)
constexpr int kStepK = 128;      // columns per step: 4 lanes x 32 codes per row
constexpr int kStages = 8;       // most steps in flight per CTA (the launch may ask for fewer: n_stages)
constexpr int kSpChunk = 128;    // sparse entries the sparse warp takes at a time
constexpr int kPad = 32;         // elements added to a token row in shared memory: row stride = 16 words mod 32
constexpr int kThreads = (kWarps + 3) * 32;
constexpr int kWorkers = (kWarps + 2) * 32;    // all but the producer warp
constexpr int kBlk1 = 4096 + 64; // offset of the step's second k-block in a stage: 16 banks away from the first
constexpr int kSzOff = kBlk1 + 4096;           // (scale, zero) entries of the step: 1 KB per group
constexpr size_t kMaxDynSmem = 190 * 1024;

// Where the 16-byte chunk c (columns 8c .. 8c+7 of the CTA's slice) of a token row sits in shared
// memory.  Inside a 128-column step, lane t works on chunks 4t .. 4t+3, one per turn; storing chunk
// 4t+w at position 4w+t puts the four lanes' chunks of one turn side by side (64 contiguous bytes
// per token), and with the row stride above the eight lanes of a quarter warp touch every bank once.
__device__ __forceinline__ int chunk_pos(int c) { return (c & ~15) | ((c & 3) << 2) | ((c >> 2) & 3); }

// (a & b) | c in one instruction (written out: the compiler makes three of the C++ expression)
__device__ __forceinline__ uint32_t and_or(uint32_t a, uint32_t b, uint32_t c) {
  uint32_t d;
  asm("lop3.b32 %0, %1, %2, %3, 0xEA;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
  return d;
}

// D = A B + C, C given
__device__ __forceinline__ void mma_acc(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// D = A B
__device__ __forceinline__ void mma_new(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%10,%10,%10};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(0.f));
}

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// Address of `local` (a pointer into this CTA's shared memory) in CTA `cta` of the cluster
__device__ __forceinline__ uint32_t cluster_addr(const void* local, uint32_t cta) {
  const uint32_t a = static_cast<uint32_t>(__cvta_generic_to_shared(local));
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(cta));
  return ra;
}
// Loads from the cluster's shared memory.  (volatile keeps them after the cluster barrier's wait,
// which is volatile too; no memory clobber, so that the compiler may keep several in flight.)
__device__ __forceinline__ uint4 ld_cluster_v4(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared::cluster.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
  return v;
}
__device__ __forceinline__ float ld_cluster_f32(uint32_t addr) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
  return v;
}

// (scale, zero) of one table entry as fp32; bf16 tables are stored as packed pairs (s,s), (z,z)
template <bool kBf16Tables>
__device__ __forceinline__ float2 sz_f32(float2 p) {
  if constexpr (kBf16Tables)
    return make_float2(__uint_as_float(__float_as_uint(p.x) & 0xFFFF0000u), __uint_as_float(__float_as_uint(p.y) & 0xFFFF0000u));
  else
    return p;
}

// A release at cluster scope measured about a microsecond per use here, so exactly one warp per CTA
// (the summing warp) arrives with release, after a CTA-level barrier with the warps whose writes it
// publishes; everybody else arrives relaxed.
__device__ __forceinline__ void cluster_arrive_release() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_arrive_relaxed() { asm volatile("barrier.cluster.arrive.relaxed.aligned;" ::: "memory"); }
// CTA-level barrier 2: the weight warps and the sparse warp arrive, the summing warp waits
__device__ __forceinline__ void tile_written_arrive() { asm volatile("bar.arrive 2, %0;" ::"n"((kWarps + 2) * 32) : "memory"); }
__device__ __forceinline__ void tile_written_sync() { asm volatile("bar.sync 2, %0;" ::"n"((kWarps + 2) * 32) : "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void workers_sync() { asm volatile("bar.sync 1, %0;" ::"n"(kWorkers) : "memory"); }

struct SkinnySub {
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
  int tile_begin;           // number of this matrix's first tile
};
struct SkinnyArgs {
  SkinnySub sub[3];
  int n;
  const __nv_bfloat16* x;
  const __nv_bfloat16* x_mul;   // not NULL: the activations are silu(x) * x_mul
  int M;
  int64_t K;
  int G, n_tiles, n_stages;
  int32_t* status;
};
// silu(g) * u of eight bf16 pairs, each product rounded to bf16 (the arithmetic of the model's own
// SiLU-gating kernel, so that either route gives the same bits)
__device__ __forceinline__ uint4 silu_mul_bf16x8(uint4 g, uint4 u) {
  const uint32_t gw[4] = {g.x, g.y, g.z, g.w}, uw[4] = {u.x, u.y, u.z, u.w};
  uint32_t o[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float g0 = __uint_as_float(gw[i] << 16), g1 = __uint_as_float(gw[i] & 0xFFFF0000u);
    const float u0 = __uint_as_float(uw[i] << 16), u1 = __uint_as_float(uw[i] & 0xFFFF0000u);
    const __nv_bfloat162 r = __floats2bfloat162_rn(g0 / (1.0f + expf(-g0)) * u0, g1 / (1.0f + expf(-g1)) * u1);
    o[i] = *reinterpret_cast<const uint32_t*>(&r);
  }
  return make_uint4(o[0], o[1], o[2], o[3]);
}
__device__ __forceinline__ int sub_of_tile(const SkinnyArgs& a, int tile) {
  return (a.n > 1 && tile >= a.sub[1].tile_begin) + (a.n > 2 && tile >= a.sub[2].tile_begin);
}

// kNT: token tiles per CTA (1: up to 8 tokens, 2: up to 16).  kDeq: how a code becomes a weight: kDeqGroup: G is a
// multiple of 128 (scale and zero applied to the sums of a step); kDeqSmall: groups of 32 or 64 (packed bf16
// conversion per code); kDeqLut: per-row tables.
constexpr int kDeqSmall = 0, kDeqGroup = 1, kDeqLut = 2;
// Grid: kSplit * n_clusters CTAs, clusters of kSplit along x; cluster c takes tiles c, c + n_clusters, ...
// Cluster barriers, the same sequence for every thread (no early exit): number 0 says that every
// CTA has staged its activations, number it + 1 that part and sparse term of the cluster's tile it
// are written, the last one that nobody reads a peer any more.  A thread arrives at number k + 1
// only after it is done with what number k - 1 published (the buffers alternate).
template <bool kBf16Tables, int kDeq, typename TY, int kNT>
__global__ void __cluster_dims__(kSplit, 1, 1) __launch_bounds__(kThreads, 2)
szo_linear_skinny_kernel(const __grid_constant__ SkinnyArgs a) {
  constexpr int kT = kTok * kNT;                       // tokens per CTA
  const int M = a.M, G = a.G, n_tiles = a.n_tiles, n_stages = a.n_stages;
  const int64_t K = a.K;
  int32_t* const status = a.status;
  const __nv_bfloat16* __restrict__ x = a.x;
  extern __shared__ __align__(128) unsigned char smem_sk[];
  __shared__ float part[2][kRowsCta * kT];             // this CTA's K-part of a 128-row tile: [row][token]
  __shared__ float spart[2][kRowsWarp * kT];           // sparse term of the 16 rows this CTA sums: [row][token]
  __shared__ float sp_x[kT * kSpChunk];                // sparse warp: activations at the chunk's columns, [token][entry]
  __shared__ float sp_val[kSpChunk];                   //              values of the chunk's entries
  __shared__ __align__(8) uint64_t bars[2 * kStages];  // full[kStages], empty[kStages]
  __shared__ int abort_flag_s;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, t = lane & 3;
  const int rank = static_cast<int>(cluster_rank());
  const int cid = static_cast<int>(blockIdx.x / kSplit), n_clusters = static_cast<int>(gridDim.x / kSplit);
  const int n_steps = static_cast<int>(K / kStepK);
  const int s_begin = rank * n_steps / kSplit, my_steps = (rank + 1) * n_steps / kSplit - s_begin;
  const int ld = ((n_steps + kSplit - 1) / kSplit) * kStepK + kPad;    // the same in every CTA: peers index each other's rows
  const int64_t nkb = K / 64;
  const int ngs = kDeq == kDeqLut ? 4 : ((G >= kStepK) ? 1 : kStepK / G);   // KB per step beside the codes: (scale, zero) groups, or the tables
  const uint32_t stage_bytes = (static_cast<uint32_t>(kSzOff + ngs * 1024) + 127u) & ~127u;
  unsigned char* ring = smem_sk;
  __nv_bfloat16* sx = reinterpret_cast<__nv_bfloat16*>(smem_sk + n_stages * stage_bytes);   // [kT][ld]: the CTA's columns of x
  float* xsum = reinterpret_cast<float*>(sx + kT * ld);                                    // [my_steps][kT]
  __nv_bfloat16* xt = reinterpret_cast<__nv_bfloat16*>(xsum + (ld - kPad) / kStepK * kT);  // [column of the slice][kT]: for the sparse warps
  auto full_bar = [&](int i) { return tc::smem_u32(&bars[i]); };
  auto empty_bar = [&](int i) { return tc::smem_u32(&bars[kStages + i]); };
  volatile int* abort_flag = &abort_flag_s;

  if (threadIdx.x == 0) {
    abort_flag_s = 0;
    for (int i = 0; i < kStages; ++i) {
      tc::mbar_init(full_bar(i), 1);
      tc::mbar_init(empty_bar(i), kWarps);
    }
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  bool failed = false;
  chain_release();

  if (warp == kWarpProducer) {
    // ---------------------------------------------------------------- producer
    tc::RingPos p{0, 0};
    int it = 0;
    const uint32_t tx_bytes = 8192u + static_cast<uint32_t>(ngs) * 1024u;
    const uint32_t steps_per_group = (kDeq != kDeqLut && G >= kStepK) ? static_cast<uint32_t>(G / kStepK) : 0u;   // 0: several groups per step
    cluster_arrive_relaxed();                           // number 0 (it stages nothing)
    // It takes its turn at barrier number it only after tile it + 1 is issued (as far as the ring lets
    // it), so that the stream does not stop while the cluster meets.
    auto issue_tile = [&](int tile) {
      if (lane == 0) {
        // (a lone thread runs a dependent instruction every few cycles: no 64-bit division in here)
        const SkinnySub& sb = a.sub[sub_of_tile(a, tile)];
        const int64_t Npad = sb.Npad;
        const int ltile = tile - sb.tile_begin;
        const uint8_t* src = sb.codes_tiled + (static_cast<int64_t>(ltile) * nkb + 2 * s_begin) * 4096;
        const float2* zsrc = sb.sz + static_cast<int64_t>(ltile) * kRowsCta;
        for (int i = 0; i < my_steps; ++i) {
          if (!failed && !tc::mbar_wait(empty_bar(p.idx), p.phase ^ 1u, abort_flag, status)) failed = true;
          if (!failed) {
            const uint32_t dst = tc::smem_u32(ring + p.idx * stage_bytes);
            const uint32_t bar = full_bar(p.idx);
            tc::mbar_expect_tx(bar, tx_bytes);
            tc::bulk_load_1d(dst, src, 4096, bar);
            tc::bulk_load_1d(dst + kBlk1, src + 4096, 4096, bar);
            if constexpr (kDeq == kDeqLut) {
              tc::bulk_load_1d(dst + kSzOff, sb.lut + static_cast<int64_t>(ltile) * kRowsCta * 16, 4096, bar);
            } else {
              const uint32_t grp0 = (steps_per_group > 0) ? static_cast<uint32_t>(s_begin + i) / steps_per_group
                                                          : static_cast<uint32_t>(s_begin + i) * static_cast<uint32_t>(ngs);
              const float2* z = zsrc + static_cast<int64_t>(grp0) * Npad;
              for (int q = 0; q < ngs; ++q, z += Npad) tc::bulk_load_1d(dst + kSzOff + q * 1024, z, 1024, bar);
            }
          }
          src += 8192;
          p.advance(n_stages);
        }
      }
      __syncwarp();
    };
    issue_tile(cid);
    for (int tile = cid; tile < n_tiles; tile += n_clusters, ++it) {
      if (tile + n_clusters < n_tiles) issue_tile(tile + n_clusters);
      cluster_wait();
      cluster_arrive_relaxed();
    }
    cluster_wait();
    if (lane == 0 && (failed || *abort_flag)) {
      for (int i = 0; i < 200; ++i) __nanosleep(1000);      // copies in flight land before the CTA leaves
    }
  } else {
    // the sparse warp's first row pointers (tiles it, it + 1) are on their way while the activations are staged
    const int sp_r = lane >> 1;
    const int64_t sp_row = rank * kRowsWarp + sp_r;                       // its lane's row inside a tile
    auto load_rp = [&](int tile, int32_t& rb, int32_t& re) {
      rb = re = 0;
      if (tile < n_tiles) {
        const SkinnySub& sb = a.sub[sub_of_tile(a, tile)];
        if (sb.row_ptr != nullptr) {
          const int64_t n = static_cast<int64_t>(tile - sb.tile_begin) * kRowsCta + sp_row, N = sb.N;
          rb = sb.row_ptr[(n < N) ? n : N];                              // rows beyond N: empty
          re = sb.row_ptr[(n + 1 < N) ? n + 1 : N];
        }
      }
    };
    int32_t b0 = 0, e0 = 0, b1 = 0, e1 = 0;
    if (warp == kWarpSparse) {
      load_rp(cid, b0, e0);
      load_rp(cid + n_clusters, b1, e1);
    }
    // ---------------------------------------------------------------- workers: stage the activations
    chain_wait();        // (launched in a chain: the activations are the predecessor's output; weights and entries are nobody's)
    {
      // a thread takes one 16-byte chunk (8 columns) of the 8 tokens of a token tile: 8 loads, the same chunks into the
      // [token][column] tile, and their 8 x 8 transpose into the [column][token] copy
      const int chunks = my_steps * (kStepK / 8);
      const __nv_bfloat16* xsrc = x + static_cast<int64_t>(s_begin) * kStepK;
      for (int cj = threadIdx.x; cj < chunks * kNT; cj += kWorkers) {
        const int c = cj / kNT, j = cj % kNT;               // chunk, token tile
        uint4 v[kTok];
#pragma unroll
        for (int r = 0; r < kTok; ++r)
          v[r] = (8 * j + r < M) ? __ldg(reinterpret_cast<const uint4*>(xsrc + static_cast<int64_t>(8 * j + r) * K + c * 8))
                                 : make_uint4(0u, 0u, 0u, 0u);
        if (a.x_mul != nullptr) {
          const __nv_bfloat16* usrc = a.x_mul + static_cast<int64_t>(s_begin) * kStepK;
#pragma unroll
          for (int r = 0; r < kTok; ++r)
            if (8 * j + r < M)
              v[r] = silu_mul_bf16x8(v[r], __ldg(reinterpret_cast<const uint4*>(usrc + static_cast<int64_t>(8 * j + r) * K + c * 8)));
        }
#pragma unroll
        for (int r = 0; r < kTok; ++r) *reinterpret_cast<uint4*>(sx + (8 * j + r) * ld + chunk_pos(c) * 8) = v[r];
#pragma unroll
        for (int e = 0; e < 8; ++e) {                     // column c * 8 + e: tokens (2p, 2p + 1) share a word
          const uint32_t sel = (e & 1) ? 0x7632u : 0x5410u;
          uint32_t o[4];
#pragma unroll
          for (int p2 = 0; p2 < 4; ++p2) {
            const uint4& lo = v[2 * p2];
            const uint4& hi = v[2 * p2 + 1];
            const uint32_t wl = (e >> 1) == 0 ? lo.x : (e >> 1) == 1 ? lo.y : (e >> 1) == 2 ? lo.z : lo.w;
            const uint32_t wh = (e >> 1) == 0 ? hi.x : (e >> 1) == 1 ? hi.y : (e >> 1) == 2 ? hi.z : hi.w;
            o[p2] = tc::prmt(wl, wh, sel);
          }
          *reinterpret_cast<uint4*>(xt + (c * 8 + e) * kT + 8 * j) = make_uint4(o[0], o[1], o[2], o[3]);
        }
      }
      workers_sync();
      if (warp == kWarpSum) cluster_arrive_release();   // number 0: the CTA's activations are staged
      else cluster_arrive_relaxed();
      // sum of a token's activations over each step (the chunk permutation stays inside a step)
      // half a warp per (step, token): a lane adds the eight values of one chunk, a fixed shuffle tree the rest
      for (int i0 = warp * 2; i0 < my_steps * kT; i0 += (kWorkers / 32) * 2) {
        const int i = i0 + (lane >> 4);
        float acc = 0.f;
        if (i < my_steps * kT) {
          const int st = i / kT, m = i % kT;
          const uint4 v = *reinterpret_cast<const uint4*>(sx + m * ld + st * kStepK + (lane & 15) * 8);
          const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int e = 0; e < 4; ++e) acc += __uint_as_float(w[e] << 16) + __uint_as_float(w[e] & 0xFFFF0000u);
        }
#pragma unroll
        for (int o = 8; o >= 1; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (i < my_steps * kT && (lane & 15) == 0) xsum[i] = acc;
      }
      workers_sync();
    }

    if (warp == kWarpSparse) {
      // -------------------------------------------------------------- sparse warp
      // Sparse term of rows 16 rank .. 16 rank + 15 of each tile.  The entries of the 16 rows are one
      // contiguous CSR range, taken in chunks of kSpChunk: every lane fetches (column, value) of its
      // entries, then the tokens' activations at those columns from the shared memory of the CTA
      // that staged them, all loads independent; then lane = (row, token parity) adds its row's
      // entries in ascending order, one fma each, from shared memory.  The dependent loads from
      // global memory (row pointers, then entries) are software-pipelined over tiles: the row
      // pointers of tile it + 2 and the first chunk of entries of tile it + 1 are in flight while
      // tile it is summed.
      constexpr int kGatherQ = kSpChunk / 32 / kNT;                      // entries per lane whose activations are fetched at once
      const int r = sp_r, h = lane & 1;
      // entries [base, end) of the matrix that tile `tile` belongs to (an empty range for a tile past the last)
      auto load_entries = [&](int tile, int32_t base, int32_t end, int (&col)[kSpChunk / 32], float (&val)[kSpChunk / 32]) {
        const SkinnySub& sb = a.sub[tile < n_tiles ? sub_of_tile(a, tile) : 0];
#pragma unroll
        for (int q = 0; q < kSpChunk / 32; ++q) {
          const int32_t e = base + lane + 32 * q;
          col[q] = (e < end) ? sb.ent_col[e] : -1;
          val[q] = (e < end) ? sb.S[e] : 0.f;
        }
      };
      int32_t b2, e2;                                                    // row pointers of tile it + 2
      int col0[kSpChunk / 32], col1[kSpChunk / 32];
      float val0[kSpChunk / 32], val1[kSpChunk / 32];
      load_entries(cid, __shfl_sync(0xffffffffu, b0, 0), __shfl_sync(0xffffffffu, e0, 31), col0, val0);
      int it = 0;
      for (int tile = cid; tile < n_tiles; tile += n_clusters, ++it) {
        load_rp(tile + 2 * n_clusters, b2, e2);
        load_entries(tile + n_clusters, __shfl_sync(0xffffffffu, b1, 0), __shfl_sync(0xffffffffu, e1, 31), col1, val1);
        const int32_t tile_b = __shfl_sync(0xffffffffu, b0, 0), tile_e = __shfl_sync(0xffffffffu, e0, 31);
        if (it == 0) cluster_wait();         // number 0: the peers' activations are staged
        float sp[kT / 2];
#pragma unroll
        for (int j = 0; j < kT / 2; ++j) sp[j] = 0.f;
        for (int32_t base = tile_b; base < tile_e; base += kSpChunk) {
          if (base > tile_b) load_entries(tile, base, tile_e, col0, val0);     // rows with more entries than one chunk
          // (all loads of a pass first, then the stores: a store to shared memory between two loads
          // from the cluster's shared memory would keep the second load waiting for the first)
#pragma unroll
          for (int q0 = 0; q0 < kSpChunk / 32; q0 += kGatherQ) {
            uint4 xv[kGatherQ][kNT];
#pragma unroll
            for (int q = 0; q < kGatherQ; ++q) {
              // column -> the CTA whose K-part holds it, and the position inside that CTA's slice
              const int colq = col0[q0 + q] >= 0 ? col0[q0 + q] : 0;
              const int step = colq >> 7;
              const int owner = (kSplit * (step + 1) - 1) / n_steps;
              const int lc = colq - (owner * n_steps / kSplit) * kStepK;
              const uint32_t src = cluster_addr(xt + lc * kT, static_cast<uint32_t>(owner));
#pragma unroll
              for (int j = 0; j < kNT; ++j) xv[q][j] = ld_cluster_v4(src + 16u * j);     // 8 tokens per load
            }
#pragma unroll
            for (int q = 0; q < kGatherQ; ++q) {
              const bool live = col0[q0 + q] >= 0;       // (rows of x beyond M are staged as zeros)
              sp_val[lane + 32 * (q0 + q)] = val0[q0 + q];
#pragma unroll
              for (int j = 0; j < kNT; ++j) {
                const uint32_t w[4] = {xv[q][j].x, xv[q][j].y, xv[q][j].z, xv[q][j].w};
#pragma unroll
                for (int e = 0; e < 8; ++e)
                  sp_x[(8 * j + e) * kSpChunk + lane + 32 * (q0 + q)] =
                      live ? __uint_as_float((e & 1) ? (w[e >> 1] & 0xFFFF0000u) : (w[e >> 1] << 16)) : 0.f;
              }
            }
          }
          __syncwarp();
          const int lo = ((b0 > base) ? b0 : base) - base;
          const int hi = ((e0 < base + kSpChunk) ? e0 : base + kSpChunk) - base;
#pragma unroll 4
          for (int i = lo; i < hi; ++i) {
            const float sv = sp_val[i];
#pragma unroll
            for (int j = 0; j < kT / 2; ++j) sp[j] = fmaf(sp_x[(2 * j + h) * kSpChunk + i], sv, sp[j]);
          }
          __syncwarp();
        }
        if (it > 0) cluster_wait();          // number it: the tile of two turns ago is summed, its buffer free
#pragma unroll
        for (int j = 0; j < kT / 2; ++j) spart[it & 1][r * kT + 2 * j + h] = sp[j];
        tile_written_arrive();
        cluster_arrive_relaxed();            // number it + 1
        b0 = b1; e0 = e1; b1 = b2; e1 = e2;
#pragma unroll
        for (int q = 0; q < kSpChunk / 32; ++q) {
          col0[q] = col1[q];
          val0[q] = val1[q];
        }
      }
      cluster_wait();
    } else if (warp == kWarpSum) {
      // -------------------------------------------------------------- sum over the cluster's K-parts
      // Rows 16 rank .. 16 rank + 15 of each tile: the eight CTAs' parts in CTA order, then the
      // sparse term and the bias.  lane = (row, token parity) as in the sparse warp.
      const int r = lane >> 1, h = lane & 1;
      cluster_wait();                        // number 0
      int it = 0;
      for (int tile = cid; tile < n_tiles; tile += n_clusters, ++it) {
        tile_written_sync();                 // this CTA's part and sparse term of the tile are written
        cluster_arrive_release();            // number it + 1 (and: the tile before is summed and stored)
        cluster_wait();
        const SkinnySub& sb = a.sub[sub_of_tile(a, tile)];
        const int64_t N = sb.N;
        const int64_t n = static_cast<int64_t>(tile - sb.tile_begin) * kRowsCta + rank * kRowsWarp + r;
        const float bv = (sb.bias != nullptr && n < N) ? sb.bias[n] : 0.f;
        TY* __restrict__ y = static_cast<TY*>(sb.y);
        float v[kT / 2];
#pragma unroll
        for (int j0 = 0; j0 < kT / 2; j0 += 4) {                       // four tokens at a time
          float pv[kSplit][4];
#pragma unroll
          for (int cta = 0; cta < kSplit; ++cta) {                     // all loads first, then the sums in CTA order
            const uint32_t src = cluster_addr(part[it & 1] + (rank * kRowsWarp + r) * kT + h, static_cast<uint32_t>(cta));
#pragma unroll
            for (int j = 0; j < 4; ++j) pv[cta][j] = ld_cluster_f32(src + 8u * (j0 + j));
          }
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            v[j0 + j] = pv[0][j];
#pragma unroll
            for (int cta = 1; cta < kSplit; ++cta) v[j0 + j] += pv[cta][j];
          }
        }
#pragma unroll
        for (int j = 0; j < kT / 2; ++j) {
          const int m = 2 * j + h;
          const float out = v[j] + spart[it & 1][r * kT + m] + bv;
          if (n < N && m < M) {
            if constexpr (sizeof(TY) == 2) y[static_cast<int64_t>(m) * N + n] = __float2bfloat16_rn(out);
            else y[static_cast<int64_t>(m) * N + n] = out;
          }
        }
      }
    } else {
      // -------------------------------------------------------------- weight warps
      tc::RingPos c{0, 0};
      const uint32_t w_off = static_cast<uint32_t>((t >> 1) * kBlk1 + (warp * kRowsWarp + g) * 32 + (t & 1) * 16);
      const uint32_t z_off = kDeq == kDeqLut ? static_cast<uint32_t>(kSzOff + (warp * kRowsWarp + g) * 32)     // the row's table
                                             : static_cast<uint32_t>(kSzOff + ((G >= kStepK) ? 0 : (t * 32 / G)) * 1024 + (warp * kRowsWarp + g) * 8);
      int it = 0;
      for (int tile = cid; tile < n_tiles; tile += n_clusters, ++it) {
        float tot[kNT][4];
#pragma unroll
        for (int j = 0; j < kNT; ++j) tot[j][0] = tot[j][1] = tot[j][2] = tot[j][3] = 0.f;
        // one step: 16 rows x 128 columns of this warp against the staged tokens
        auto step_body = [&](int i, const unsigned char* stg) {
          const uint4 wa = *reinterpret_cast<const uint4*>(stg + w_off);
          const uint4 wb = *reinterpret_cast<const uint4*>(stg + w_off + 8 * 32);
          float2 pa = make_float2(0.f, 0.f), pb = pa;
          if constexpr (kDeq != kDeqLut) {
            pa = *reinterpret_cast<const float2*>(stg + z_off);
            pb = *reinterpret_cast<const float2*>(stg + z_off + 8 * 8);
          }
          const uint32_t qa[4] = {wa.x, wa.y, wa.z, wa.w}, qb[4] = {wb.x, wb.y, wb.z, wb.w};
          const __nv_bfloat16* xs = sx + g * ld + i * kStepK + t * 8;      // token g; word wd of this lane: + wd * 32
          if constexpr (kDeq == kDeqLut) {
            const unsigned char* ta = stg + z_off;                         // table of row g; row g + 8: 8 * 32 bytes further
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
              const uint32_t a0[4] = {look(ta, qa[wd], 0), look(ta + 8 * 32, qb[wd], 0), look(ta, qa[wd], 4), look(ta + 8 * 32, qb[wd], 4)};
              const uint32_t a1[4] = {look(ta, qa[wd], 8), look(ta + 8 * 32, qb[wd], 8), look(ta, qa[wd], 12), look(ta + 8 * 32, qb[wd], 12)};
#pragma unroll
              for (int j = 0; j < kNT; ++j) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + j * kTok * ld + wd * 32);
                mma_acc(tot[j], a0, xv.x, xv.y);
                mma_acc(tot[j], a1, xv.z, xv.w);
              }
            }
          } else if constexpr (kDeq == kDeqGroup) {
            float accq[kNT][2][4];                                         // even and odd words: two shorter chains
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {                                // one 32-bit word = 8 columns = two k16 MMAs
              uint32_t a0[4], a1[4];
              a0[0] = and_or(qa[wd], 0x000F000Fu, 0x43004300u);
              a0[1] = and_or(qb[wd], 0x000F000Fu, 0x43004300u);
              a0[2] = and_or(qa[wd] >> 4, 0x000F000Fu, 0x43004300u);
              a0[3] = and_or(qb[wd] >> 4, 0x000F000Fu, 0x43004300u);
              a1[0] = and_or(qa[wd] >> 8, 0x000F000Fu, 0x43004300u);
              a1[1] = and_or(qb[wd] >> 8, 0x000F000Fu, 0x43004300u);
              a1[2] = and_or(qa[wd] >> 12, 0x000F000Fu, 0x43004300u);
              a1[3] = and_or(qb[wd] >> 12, 0x000F000Fu, 0x43004300u);
#pragma unroll
              for (int j = 0; j < kNT; ++j) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + j * kTok * ld + wd * 32);
                if (wd < 2) mma_new(accq[j][wd & 1], a0, xv.x, xv.y);
                else mma_acc(accq[j][wd & 1], a0, xv.x, xv.y);
                mma_acc(accq[j][wd & 1], a1, xv.z, xv.w);
              }
            }
            const float2 fa = sz_f32<kBf16Tables>(pa), fb = sz_f32<kBf16Tables>(pb);
            const float za = fmaf(-128.f, fa.x, fa.y), zb = fmaf(-128.f, fb.x, fb.y);
#pragma unroll
            for (int j = 0; j < kNT; ++j) {
              const float2 xs2 = *reinterpret_cast<const float2*>(xsum + i * kT + kTok * j + 2 * t);   // tokens 2t, 2t+1
              tot[j][0] = fmaf(fa.x, accq[j][0][0] + accq[j][1][0], fmaf(za, xs2.x, tot[j][0]));
              tot[j][1] = fmaf(fa.x, accq[j][0][1] + accq[j][1][1], fmaf(za, xs2.y, tot[j][1]));
              tot[j][2] = fmaf(fb.x, accq[j][0][2] + accq[j][1][2], fmaf(zb, xs2.x, tot[j][2]));
              tot[j][3] = fmaf(fb.x, accq[j][0][3] + accq[j][1][3], fmaf(zb, xs2.y, tot[j][3]));
            }
          } else {
#pragma unroll
            for (int wd = 0; wd < 4; ++wd) {
              const uint4 da = tc::dequant_word<kBf16Tables>(qa[wd], pa);
              const uint4 db = tc::dequant_word<kBf16Tables>(qb[wd], pb);
              const uint32_t a0[4] = {da.x, db.x, da.y, db.y};
              const uint32_t a1[4] = {da.z, db.z, da.w, db.w};
#pragma unroll
              for (int j = 0; j < kNT; ++j) {
                const uint4 xv = *reinterpret_cast<const uint4*>(xs + j * kTok * ld + wd * 32);
                mma_acc(tot[j], a0, xv.x, xv.y);
                mma_acc(tot[j], a1, xv.z, xv.w);
              }
            }
          }
        };
        // two steps at a time: their instruction streams are independent and interleave
        for (int i = 0; i < my_steps; i += 2) {
          const bool two = i + 1 < my_steps;
          tc::RingPos c1 = c;
          c1.advance(n_stages);
          if (!failed && !tc::mbar_wait(full_bar(c.idx), c.phase, abort_flag, status)) failed = true;
          if (two && !failed && !tc::mbar_wait(full_bar(c1.idx), c1.phase, abort_flag, status)) failed = true;
          step_body(i, ring + c.idx * stage_bytes);
          if (two) step_body(i + 1, ring + c1.idx * stage_bytes);
          __syncwarp();
          if (lane == 0 && !failed) {                      // the stages' data are in registers and used
            tc::mbar_arrive(empty_bar(c.idx));
            if (two) tc::mbar_arrive(empty_bar(c1.idx));
          }
          c = c1;
          if (two) c.advance(n_stages);
        }
        // accumulator layout: [0], [1] = (row g, tokens 2t, 2t+1); [2], [3] = (row g+8, same tokens)
        cluster_wait();                                   // number it: the tile of two turns ago is summed, its buffer free
#pragma unroll
        for (int j = 0; j < kNT; ++j) {
          float* mine = part[it & 1] + (warp * kRowsWarp + g) * kT + kTok * j + 2 * t;
          mine[0] = tot[j][0];
          mine[1] = tot[j][1];
          mine[8 * kT] = tot[j][2];
          mine[8 * kT + 1] = tot[j][3];
        }
        tile_written_arrive();
        cluster_arrive_relaxed();                         // number it + 1
      }
      cluster_wait();
    }
  }
  cluster_arrive_relaxed();                             // nobody leaves while its shared memory may still be read
  cluster_wait();
}

size_t skinny_dyn_smem(int64_t K, int G, int kT, int n_stages = kStages) {
  const int64_t n_steps = K / kStepK, max_steps = ceil_div(n_steps, kSplit);
  const size_t ngs = G < 0 ? 4 : ((G >= kStepK) ? 1 : kStepK / G);     // G < 0: per-row tables, 4 KB per step
  const size_t stage = (static_cast<size_t>(kSzOff) + ngs * 1024 + 127) & ~static_cast<size_t>(127);
  return n_stages * stage + static_cast<size_t>(kT) * (max_steps * kStepK + kPad) * 2 + static_cast<size_t>(max_steps) * kT * 4 +
         static_cast<size_t>(max_steps) * kStepK * kT * 2;     // ring, x [token][column], step sums, x [column][token]
}

template <bool kBf16Tables, int kDeq, typename TY, int kNT>
szo_status launch_skinny(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                         const float* const* S, void* const* y, cudaStream_t st, bool chained) {
  auto kern = szo_linear_skinny_kernel<kBf16Tables, kDeq, TY, kNT>;
  const szo_linear* p = plans[0];
  // A ring of 8 steps when two CTAs of that size still share an SM (or when 4 would not change that
  // either), else 4: two CTAs with 4 steps in flight each hide more than one with 8.
  constexpr size_t kStaticSmem = (kNT == 1) ? 14 * 1024 : 28 * 1024;            // upper bounds of the kernel's static arrays
  constexpr size_t kTwoPerSm = (227 * 1024) / 2 - 1024;                         // per CTA, 1 KB reserved by the driver each
  int n_stages = kStages;
  if (skinny_dyn_smem(p->K, p->G, kTok * kNT, kStages) + kStaticSmem > kTwoPerSm &&
      skinny_dyn_smem(p->K, p->G, kTok * kNT, kStages / 2) + kStaticSmem <= kTwoPerSm)
    n_stages = kStages / 2;
  const size_t smem = skinny_dyn_smem(p->K, p->G, kTok * kNT, n_stages);
  // per device: the attribute, and how many clusters fit at once with this much shared memory
  struct PerDevice {
    bool configured = false;
    size_t asked_smem = ~static_cast<size_t>(0);
    int max_clusters = 0;
  };
  static PerDevice per_device[64];
  static std::mutex mu;
  int dev = 0;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_REQUIRE(dev >= 0 && dev < 64, SZO_ERR_UNSUPPORTED, "device ordinal %d", dev);
  int max_clusters = 0;
  {
    std::lock_guard<std::mutex> lock(mu);
    PerDevice& pd = per_device[dev];
    if (!pd.configured) {
      SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(kMaxDynSmem)));
      pd.configured = true;
    }
    if (smem != pd.asked_smem) {
      cudaLaunchConfig_t cfg = {};
      cfg.gridDim = dim3(static_cast<unsigned>(kSplit * 64));
      cfg.blockDim = dim3(kThreads);
      cfg.dynamicSmemBytes = smem;
      SZO_CHECK_CUDA(cudaOccupancyMaxActiveClusters(&pd.max_clusters, kern, &cfg));
      if (pd.max_clusters < 1) pd.max_clusters = 1;
      pd.asked_smem = smem;
    }
    max_clusters = pd.max_clusters;
  }
  SkinnyArgs a{};
  a.n = n;
  a.x = static_cast<const __nv_bfloat16*>(x);
  a.x_mul = static_cast<const __nv_bfloat16*>(x_mul);
  a.M = static_cast<int>(M);
  a.K = p->K;
  a.G = p->G;
  a.n_stages = n_stages;
  a.status = device_status_word();
  SZO_REQUIRE(a.status != nullptr, SZO_ERR_CUDA, "no device status word");
  int n_tiles = 0;
  for (int i = 0; i < n; ++i) {
    const szo_linear* q = plans[i];
    a.sub[i] = SkinnySub{q->codes_tiled, q->sz, q->lut_bf16, q->Npad, q->nnz > 0 ? q->row_ptr : nullptr, q->ent_col, S[i],
                         q->bias, y[i], q->N, n_tiles};
    n_tiles += static_cast<int>(ceil_div(q->N, kRowsCta));
  }
  a.n_tiles = n_tiles;
  const int n_clusters = n_tiles < max_clusters ? n_tiles : max_clusters;
  // (with two token tiles per CTA an early-placed successor costs more than it hides: 4.8 -> 5.4 ms per 16-token step)
  SZO_CHECK_CUDA(launch_maybe_chained(kern, dim3(static_cast<unsigned>(kSplit * n_clusters)), dim3(kThreads), smem, st,
                                      chained && kNT == 1, a));
  count_launch();
  SZO_CHECK_LAUNCH("szo_linear_skinny_kernel");
  return SZO_OK;
}

template <bool kBf16Tables, typename TY>
szo_status launch_skinny_nt(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                            const float* const* S, void* const* y, cudaStream_t st, bool chained) {
  if (plans[0]->G < 0) {                       // per-row tables (the plan's bf16 copy: the tables' own type does not matter)
    if constexpr (!kBf16Tables) {
      if (M <= kTok) return launch_skinny<false, kDeqLut, TY, 1>(plans, n, x, x_mul, M, S, y, st, chained);
      return launch_skinny<false, kDeqLut, TY, 2>(plans, n, x, x_mul, M, S, y, st, chained);
    } else {
      return fail(SZO_ERR_UNSUPPORTED, "table-coded plans take the f16-table instantiation");
    }
  }
  const bool group = plans[0]->G % kStepK == 0;
  if (M <= kTok) {
    if (group) return launch_skinny<kBf16Tables, kDeqGroup, TY, 1>(plans, n, x, x_mul, M, S, y, st, chained);
    return launch_skinny<kBf16Tables, kDeqSmall, TY, 1>(plans, n, x, x_mul, M, S, y, st, chained);
  }
  if (group) return launch_skinny<kBf16Tables, kDeqGroup, TY, 2>(plans, n, x, x_mul, M, S, y, st, chained);
  return launch_skinny<kBf16Tables, kDeqSmall, TY, 2>(plans, n, x, x_mul, M, S, y, st, chained);
}

}  // namespace

// The shapes the weight-streaming kernel takes: int4 plans with groups of 32, 64 or a multiple of
// 128 columns or with per-row tables, at most 16 tokens, K a multiple of 128 whose per-CTA slice of the tokens fits shared
// memory (K up to about 25 000 for 8 tokens, 14 000 for 16).
bool skinny_applies(const szo_linear* p, int64_t M) {
  const bool lut = p->G == -1 && p->lut_bf16 != nullptr;
  return (lut || (p->G > 0 && (p->G == 32 || p->G == 64 || p->G % kStepK == 0))) && p->codes_tiled != nullptr && M >= 1 &&
         M <= 2 * kTok && p->K % kStepK == 0 && skinny_dyn_smem(p->K, p->G, M <= kTok ? kTok : 2 * kTok) <= kMaxDynSmem;
}

// Up to three matrices with the same K, group size and table type in one launch
bool skinny_group_applies(const szo_linear* const* plans, int n, int64_t M) {
  if (n < 1 || n > 3) return false;
  for (int i = 0; i < n; ++i)
    if (!skinny_applies(plans[i], M) || plans[i]->K != plans[0]->K || plans[i]->G != plans[0]->G ||
        plans[i]->sz_dtype != plans[0]->sz_dtype)
      return false;
  return true;
}

bool few_token_applies(const szo_linear* const* plans, int n, int64_t M) {
  return gemv_applies(plans, n, M) || skinny_group_applies(plans, n, M);
}

szo_status linear_fwd_skinny_group(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                                   const float* const* S_pert, void* const* y, int y_dtype, cudaStream_t st, bool chained) {
  if (gemv_applies(plans, n, M)) return linear_fwd_gemv(plans, n, x, x_mul, M, S_pert, y, y_dtype, st, chained);
  SZO_REQUIRE(skinny_group_applies(plans, n, M), SZO_ERR_UNSUPPORTED, "shapes not covered by the weight-streaming kernel");
  const bool bf = plans[0]->sz_dtype == SZO_BF16 && plans[0]->G > 0;
  if (y_dtype == SZO_F32) {
    if (bf) return launch_skinny_nt<true, float>(plans, n, x, x_mul, M, S_pert, y, st, chained);
    return launch_skinny_nt<false, float>(plans, n, x, x_mul, M, S_pert, y, st, chained);
  }
  if (bf) return launch_skinny_nt<true, __nv_bfloat16>(plans, n, x, x_mul, M, S_pert, y, st, chained);
  return launch_skinny_nt<false, __nv_bfloat16>(plans, n, x, x_mul, M, S_pert, y, st, chained);
}

szo_status linear_fwd_skinny(const szo_linear* p, const void* x, int64_t M, const float* S_pert, void* y, int y_dtype,
                             cudaStream_t st) {
  return linear_fwd_skinny_group(&p, 1, x, nullptr, M, &S_pert, &y, y_dtype, st);
}

}  // namespace szo
