// Sparse product of the paired form of a ZO step's two forwards:
//   yd[t][n] += eps * sum_e z_e * xc[t][col_e]   over the sensitive entries e of weight row n
// (Zbar of Definition 4 times the centre activations, the term that the perturbation of the sparse part
// adds to the half-difference rows), for the M half-difference rows of up to three matrices that share x.
// It runs after the tensor-core launch that wrote xd W^T into those rows.  The sum is formed in fp32 and
// added to the stored value (the half-difference has its own exponent, so a bf16 rounding costs 2^-9 of
// ITS size, not of the centre's): for fp32 y by a read-modify-write, for bf16 y by a reduction in L2.
//
// A block stages xc[TM tokens][all K columns] transposed in shared memory, then each thread walks weight rows.
// Tried before this form: columns of a transposed copy of xc read from L2 per entry (8 KB per entry, 2.6 TB/s:
// 20 ms of a Llama-2-7B-shaped step), the slab copied from that transposed copy (16 bytes every 8 KB: the
// strided reads camp on a few L2 slices, 25 ms), and the sum inside the epilogue of the tensor-core kernel
// (that epilogue is on the kernel's critical path: the decoder-block linears became 45 % slower).
// Tried after it: the product as mma.sync m16n8k16 instructions (records in chunks of 16 grouped by eight
// weight rows, the A operand gathered from the slab by ldmatrix .trans, B = RN_bf16(eps z) placed by the
// record's row, the records of a warp's next 32 rows copied into a shared-memory ring by cp.async).  At
// N = 22016, K = 4096, M = 4096: 80 M warp instructions against 98 M, but 30.8 M load/store wavefronts against
// 26.0 M (an 8 x 16-byte ldmatrix phase meets the same bank conflicts as a quarter warp of 16-byte loads, and
// the records pass through shared memory once more): 157 us against 163 us, and at K = 11008, where only eight
// tokens fit and half of every mma is empty, 169 us against 146 us.  Not kept: 3 % for eps z rounded to bf16.
// Nor was fma.rn.f32.bf16 (fp32 += bf16 * bf16 in one instruction, no unpacking of x, eps z as bf16): 78 M
// instructions against 98 M, 151 us against 161 us alone (ncu) and 6 to 10 us per paired linear in a call that
// alternated the two libraries (0.9 ms of a 113 ms step): the kernel waits on its record loads (long scoreboard
// 6.1 cycles per issue) more than on issue slots, and eps z would lose three to five bits.
#include <algorithm>
#include <cstdlib>
#include <vector>

#include "linear.cuh"

namespace szo {

namespace {

// Per-plan data of the product (device memory, owned): record slot s holds entry src[s] of the plan and
// colk[s] = its column | (width of the column field << 24).  Slot order = CSR order with the entries of each
// row permuted (build_layout); the column field has as many bits as K - 1 needs.
struct CrossPlan {
  int64_t slots;
  uint32_t* colk;
  int32_t* src;
};

uint32_t col_bits_of(int64_t K) {
  uint32_t bits = 1;
  while ((int64_t(1) << bits) < K) ++bits;
  return bits;
}

struct HostLayout {
  std::vector<uint32_t> colk;
  std::vector<int32_t> src;
};

// The kernel gives lane l of a warp the rows 2 l and 2 l + 1 of a 64-row span and walks the even rows
// first, then the odd ones: the lanes of a quarter warp thus read, in trip i, entry slot i of eight rows two
// apart.  For each such set of eight rows and each trip, every row in turn takes one of its remaining entries
// whose bank group (column mod 8) no earlier row of the trip has taken, or, failing that, its first remaining
// one.  (Bank conflicts of a gate/up launch at K = 4096: 8.8 M -> 5.7 M, 197 -> 193 us.)
void build_layout(int64_t N, int64_t K, const std::vector<int32_t>& rp, const std::vector<int32_t>& col, HostLayout* out) {
  const size_t nnz = col.size();
  out->src.resize(nnz);
  out->colk.resize(nnz);
  for (size_t s = 0; s < nnz; ++s) out->src[s] = static_cast<int32_t>(s);
  // (dense masks keep the entry order: the search below is quadratic in a row's entries, and those masks take the
  // tensor-core form of the product)
  const bool ordered = static_cast<double>(nnz) < 0.002 * static_cast<double>(N) * static_cast<double>(K);
  std::vector<char> taken;
  for (int64_t n0 = 0; ordered && n0 < N; n0 += 16) {
    for (int parity = 0; parity < 2; ++parity) {
      int32_t maxlen = 0;
      for (int l = 0; l < 8; ++l) {
        const int64_t n = n0 + 2 * l + parity;
        if (n < N && rp[n + 1] - rp[n] > maxlen) maxlen = rp[n + 1] - rp[n];
      }
      taken.assign(static_cast<size_t>(maxlen) * 8, 0);              // [lane][entry of the row]
      for (int32_t i = 0; i < maxlen; ++i) {
        unsigned used = 0;
        for (int l = 0; l < 8; ++l) {
          const int64_t n = n0 + 2 * l + parity;
          if (n >= N) continue;
          const int32_t b = rp[n], len = rp[n + 1] - b;
          if (i >= len) continue;
          int32_t pick = -1, first = -1;
          for (int32_t j = 0; j < len; ++j) {
            if (taken[static_cast<size_t>(l) * maxlen + j]) continue;
            if (first < 0) first = j;
            if (!(used >> (col[b + j] & 7) & 1u)) {
              pick = j;
              break;
            }
          }
          if (pick < 0) pick = first;
          taken[static_cast<size_t>(l) * maxlen + pick] = 1;
          used |= 1u << (col[b + pick] & 7);
          out->src[b + i] = b + pick;
        }
      }
    }
  }
  const uint32_t bits = col_bits_of(K);
  for (size_t s = 0; s < nnz; ++s) out->colk[s] = static_cast<uint32_t>(col[out->src[s]]) | (bits << 24);
}

template <typename T>
bool to_device(const std::vector<T>& v, T** out) {
  *out = nullptr;
  if (v.empty()) return true;
  return cudaMalloc(out, v.size() * sizeof(T)) == cudaSuccess &&
         cudaMemcpy(*out, v.data(), v.size() * sizeof(T), cudaMemcpyHostToDevice) == cudaSuccess;
}

}  // namespace

// Host side, at plan creation (which has synchronised; not on a step's path).
szo_status cross_plan_create(szo_linear* p) {
  p->cross = nullptr;
  if (p->nnz == 0 || p->K > (int64_t(1) << 18)) return SZO_OK;
  const int64_t N = p->N;
  std::vector<int32_t> rp(static_cast<size_t>(N) + 1), col(static_cast<size_t>(p->nnz));
  SZO_CHECK_CUDA(cudaMemcpy(rp.data(), p->row_ptr, rp.size() * sizeof(int32_t), cudaMemcpyDeviceToHost));
  SZO_CHECK_CUDA(cudaMemcpy(col.data(), p->ent_col, col.size() * sizeof(int32_t), cudaMemcpyDeviceToHost));
  HostLayout h;
  CrossPlan* c = new CrossPlan();
  build_layout(N, p->K, rp, col, &h);
  c->slots = static_cast<int64_t>(h.src.size());
  if (!to_device(h.colk, &c->colk) || !to_device(h.src, &c->src)) {
    cudaFree(c->colk);
    cudaFree(c->src);
    delete c;
    return fail(SZO_ERR_CUDA, "cannot store the record layout of the sparse product");
  }
  p->cross = c;
  return SZO_OK;
}

void cross_plan_destroy(szo_linear* p) {
  CrossPlan* c = static_cast<CrossPlan*>(p->cross);
  if (c) {
    cudaFree(c->colk);
    cudaFree(c->src);
  }
  delete c;
  p->cross = nullptr;
}

size_t cross_rec_bytes(const szo_linear* const* plans, int n) {
  size_t nnz = 0;
  for (int i = 0; i < n; ++i) nnz += static_cast<size_t>(plans[i]->nnz);
  return round_up(nnz * sizeof(uint32_t), 256);
}

// ------------------------------------------------------------------------------ records
namespace {

// rec[s] = colk[s]'s column field and, above it, fp32(eps * z[src[s]]) rounded to the nearest value with
// 32 - bits bits (ties to even): sign, exponent and at least 9 bits of mantissa for K up to 16384 (5 at the
// largest K, 2^18).
__global__ void pack_cross_records_kernel(const uint32_t* __restrict__ colk, const int32_t* __restrict__ src,
                                          const float* __restrict__ z, float eps, int64_t n, uint32_t* __restrict__ rec) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  const uint32_t ck = colk[i];
  const uint32_t bits = ck >> 24, low_mask = (1u << bits) - 1u;
  uint32_t b = __float_as_uint(eps * z[src[i]]);
  b += (low_mask >> 1) + ((b >> bits) & 1u);
  rec[i] = (b & ~low_mask) | (ck & 0x00FFFFFFu);
}

__global__ void offset_slots_kernel(const uint32_t* __restrict__ colk_in, const int32_t* __restrict__ src_in, int64_t n,
                                    int32_t base, uint32_t* __restrict__ colk, int32_t* __restrict__ src) {
  const int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= n) return;
  colk[i] = colk_in[i];
  src[i] = base + src_in[i];
}

}  // namespace

szo_status cross_copy_slots(const szo_linear* p, int32_t base, uint32_t* colk, int32_t* src, cudaStream_t st) {
  const CrossPlan* c = static_cast<const CrossPlan*>(p->cross);
  if (c == nullptr || c->slots == 0) return SZO_OK;
  offset_slots_kernel<<<static_cast<unsigned>(ceil_div(c->slots, 256)), 256, 0, st>>>(c->colk, c->src, c->slots, base, colk, src);
  SZO_CHECK_LAUNCH("offset_slots_kernel");
  return SZO_OK;
}

szo_status pack_cross_records_all(const uint32_t* colk, const int32_t* src, const float* z, float eps, int64_t n, uint32_t* rec,
                                  cudaStream_t st) {
  if (n == 0) return SZO_OK;
  pack_cross_records_kernel<<<static_cast<unsigned>(ceil_div(n, 256)), 256, 0, st>>>(colk, src, z, eps, n, rec);
  count_launch();
  SZO_CHECK_LAUNCH("pack_cross_records_kernel");
  return SZO_OK;
}

szo_status pack_cross_records(const szo_linear* p, const float* z, float eps, uint32_t* rec, cudaStream_t st) {
  const CrossPlan* c = static_cast<const CrossPlan*>(p->cross);
  if (p->nnz == 0) return SZO_OK;
  SZO_REQUIRE(c != nullptr, SZO_ERR_UNSUPPORTED, "K = %lld too large for the paired form", (long long)p->K);
  return pack_cross_records_all(c->colk, c->src, z, eps, c->slots, rec, st);
}

// ------------------------------------------------------------------------------ kernels
namespace {

struct CrossSub {
  const int32_t* ptr;    // row_ptr [N + 1]
  const uint32_t* rec;   // the plan's packed records
  void* yd;              // first half-difference row of this matrix's y
  int64_t N;
};
struct CrossArgs {
  CrossSub sub[3];
  int n;
  const __nv_bfloat16* x;   // centre rows [M][K]
  int64_t M, K;
  uint32_t col_mask;        // (1 << col_bits) - 1, col_bits = bits needed for K - 1
  int64_t unit_end[3];      // running count of units (R adjacent weight rows) through the matrices
};

__device__ __forceinline__ uint32_t prmt_b32(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t d;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(sel));
  return d;
}

// y (bf16) += the fp32 sums, as reductions performed by L2: each element of the half-difference rows gets
// exactly one addend per launch, so the result does not depend on the order of the blocks.  The addend is
// rounded to bf16 first (2^-9 of the sum's own size), the result once more, as a bf16 store would.
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
  const __nv_bfloat162 q = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&q);
}
__device__ __forceinline__ void red_add_bf16x2(void* addr, uint32_t v) {
  asm volatile("red.global.add.noftz.bf16x2 [%0], %1;" ::"l"(addr), "r"(v) : "memory");
}
__device__ __forceinline__ void red_add_bf16x2_v4(void* addr, uint32_t v0, uint32_t v1, uint32_t v2, uint32_t v3) {
  asm volatile("red.global.v4.bf16x2.add.noftz [%0], {%1, %2, %3, %4};" ::"l"(addr), "r"(v0), "r"(v1), "r"(v2), "r"(v3) : "memory");
}

template <int TM> struct SlabVec;
template <> struct SlabVec<16> { using type = uint4; };   // two per column
template <> struct SlabVec<8> { using type = uint4; };
template <> struct SlabVec<4> { using type = uint2; };
template <> struct SlabVec<2> { using type = uint32_t; };

// Tokens m0 .. m0 + TM - 1 of x into the slab.  The slab is kept in kVecs planes, plane q holding tokens
// q * kTokPlane .. of every column ([plane][K][kTokPlane]): a 16-byte read of column c then falls into bank
// group c mod 8 (eight classes for the eight lanes of a quarter warp; with the two vectors of a column side
// by side there were four).  A plane is followed by 64
// bytes, so that the staging stores of the two planes use different banks.
// lane = (column group, token t): one 16-byte load of 8 columns of token t.  The lanes of tokens 2p and
// 2p + 1 then swap halves (the even one sends columns 2, 3, 6, 7 and gets the odd one's 0, 1, 4, 5), so
// that each holds both tokens of four columns and stores four 4-byte words xs[c][2p .. 2p + 1]: a
// quarter of the instructions of eight 2-byte stores with their selects.
template <int TM>
__device__ __forceinline__ void stage_slab(const CrossArgs& a, int64_t m0, unsigned char* slab, size_t plane_bytes) {
  using V = typename SlabVec<TM>::type;
  constexpr int kVecs = TM * 2 / static_cast<int>(sizeof(V));
  constexpr int kTokPlane = TM / kVecs;
  constexpr int kLaneTok = TM < 32 ? TM : 32;
  static_assert(kLaneTok % 2 == 0, "token pairs");
  const int t = threadIdx.x % kLaneTok;
  const bool odd = (t & 1) != 0;
  const int64_t per_pass = static_cast<int64_t>(blockDim.x / kLaneTok) * 8;       // columns per pass of the block
  const bool valid = m0 + t < a.M;
  const __nv_bfloat16* row = a.x + (m0 + t) * a.K;
  const int64_t c_first = static_cast<int64_t>(threadIdx.x / kLaneTok) * 8;
  for (int64_t base = 0; base < a.K; base += per_pass) {             // (uniform trip count: the swap needs both lanes)
    const int64_t c8 = base + c_first;
    uint4 v = make_uint4(0u, 0u, 0u, 0u);
    if (valid && c8 < a.K) v = *reinterpret_cast<const uint4*>(row + c8);
    const uint32_t r0 = __shfl_xor_sync(0xffffffffu, odd ? v.x : v.y, 1);
    const uint32_t r1 = __shfl_xor_sync(0xffffffffu, odd ? v.z : v.w, 1);
    const uint32_t k0 = odd ? v.y : v.x, k1 = odd ? v.w : v.z;       // columns (2, 3), (6, 7) or (0, 1), (4, 5) of this token
    const uint32_t lo0 = odd ? r0 : k0, hi0 = odd ? k0 : r0;         // the even token goes to the low half of a word
    const uint32_t lo1 = odd ? r1 : k1, hi1 = odd ? k1 : r1;
    if (c8 < a.K) {
      constexpr int kWp = kTokPlane / 2;                             // words per column and plane
      uint32_t* dst = reinterpret_cast<uint32_t*>(slab + (t / kTokPlane) * plane_bytes) + (c8 + (odd ? 2 : 0)) * kWp +
                      ((t % kTokPlane) >> 1);
      dst[0] = prmt_b32(lo0, hi0, 0x5410u);
      dst[kWp] = prmt_b32(lo0, hi0, 0x7632u);
      dst[4 * kWp] = prmt_b32(lo1, hi1, 0x5410u);
      dst[5 * kWp] = prmt_b32(lo1, hi1, 0x7632u);
    }
  }
}

// R weight rows per thread (2 when N is even: y is then read and written four bytes per lane).  The rows of
// a lane are walked one after the other, and a warp runs each walk as long as its longest row: at 4
// entries per row that is about twice the mean.  Giving lane l the l-th longest and the l-th shortest
// row of a 64-row group instead (so that lanes finish together) measured 16 % slower: the walks are
// still separate loops, and the two rows of a lane are then no longer adjacent (two-byte accesses to y).
// A sorted-slice layout (rows of a 256-row window ordered by entry count, 32 equally long rows per warp,
// records of a trip side by side, sums passed through a shared-memory tile and added to y eight bytes at
// a time by four independent thread groups per block) removed the idle lanes (119 M instructions
// against 140 M) but tripled the shared-memory wavefronts (37 M, 22 M of them bank conflicts: all
// 32 lanes now read random columns, and the tile is written at random rows): 265 us against 211 at
// K = 4096, 3 % ahead at K = 11008; not kept.
// Work = (token group, unit), a unit being R adjacent weight rows of one of the matrices; the units of a token
// group are numbered through the matrices (unit_end).  The grid is as many blocks as the device holds at once,
// and block b takes the b-th of gridDim.x equal, contiguous shares of that list: a share covers the end of one
// token group, whole groups and the start of another, and the block stages the slab of each group it touches
// (about 2.7 at M = 4096).  Before, a block was one token group and one of two row shares: 512 equal blocks,
// 3.46 waves, 15 % of the SM cycles idle in the last one.  Measured in one call, the libraries alternating:
// gate/up 1211 -> 1199 us per paired linear, q/k/v 693 -> 686, o 267 -> 265, down (K = 11008) unchanged.
// (A last quarter of the token groups in blocks a quarter the size, to fill the last wave, did not help.)
// Wide K (a slab of 16 tokens does not fit beyond K = 6400, of 8 beyond 12800): staging the columns in ranges,
// 16 tokens each, was 6 % faster for a whole paired linear at K = 20480 and 1.5 % at K = 11008, but then an
// element of y receives one addend per range from blocks that run at the same time: the sum of roundings
// depends on their order.  Not done: every element gets exactly one addend per launch.
template <int TM, int R, typename TY>
__global__ void __launch_bounds__(TM >= 8 ? 1024 : 512) pair_cross_kernel(const CrossArgs a) {
  using V = typename SlabVec<TM>::type;
  constexpr int kVecs = TM * 2 / static_cast<int>(sizeof(V));    // vectors per column
  constexpr int kTokPlane = TM / kVecs;
  extern __shared__ __align__(16) unsigned char cross_smem[];
  chain_release();
  chain_wait();
  const size_t plane_bytes = static_cast<size_t>(a.K) * kTokPlane * sizeof(__nv_bfloat16) + 64;
  const unsigned char* xs = cross_smem;
  const int64_t U = a.unit_end[a.n - 1];                 // units per token group
  const int64_t T = ((a.M + TM - 1) / TM) * U;
  int64_t lo = T / gridDim.x * blockIdx.x + T % gridDim.x * blockIdx.x / gridDim.x;
  const int64_t hi = T / gridDim.x * (blockIdx.x + 1) + T % gridDim.x * (blockIdx.x + 1) / gridDim.x;
  bool first = true;
  while (lo < hi) {
    const int64_t group = lo / U, u0 = lo - group * U;
    const int64_t u1 = hi - lo < U - u0 ? u0 + (hi - lo) : U;
    lo += u1 - u0;
    const int64_t m0 = group * TM;
    if (!first) __syncthreads();                 // every thread is done with the previous group's slab
    first = false;
    stage_slab<TM>(a, m0, cross_smem, plane_bytes);
    __syncthreads();
    const int cnt = static_cast<int>(a.M - m0 < TM ? a.M - m0 : TM);
    for (int s = 0; s < a.n; ++s) {
      const int32_t* row_ptr = s == 0 ? a.sub[0].ptr : (s == 1 ? a.sub[1].ptr : a.sub[2].ptr);
      if (row_ptr == nullptr) continue;
      const int64_t ub = s == 0 ? 0 : a.unit_end[s - 1], ue = a.unit_end[s];
      const int64_t s0 = (u0 > ub ? u0 : ub) - ub, s1 = (u1 < ue ? u1 : ue) - ub;   // this matrix's units in the share
      if (s0 >= s1) continue;
      const uint32_t* rec = s == 0 ? a.sub[0].rec : (s == 1 ? a.sub[1].rec : a.sub[2].rec);
      TY* yd = static_cast<TY*>(s == 0 ? a.sub[0].yd : (s == 1 ? a.sub[1].yd : a.sub[2].yd));
      const int64_t N = s == 0 ? a.sub[0].N : (s == 1 ? a.sub[1].N : a.sub[2].N);
      for (int64_t n = (s0 + threadIdx.x) * R; n < s1 * R; n += static_cast<int64_t>(blockDim.x) * R) {
        int32_t eb[R + 1];
#pragma unroll
        for (int r = 0; r <= R; ++r) eb[r] = __ldg(row_ptr + (n + r <= N ? n + r : N));
        if (eb[0] == eb[R]) continue;
        float acc[R][TM];
#pragma unroll
        for (int r = 0; r < R; ++r) {
#pragma unroll
          for (int j = 0; j < TM; ++j) acc[r][j] = 0.f;
          for (int32_t e = eb[r]; e < eb[r + 1]; ++e) {
            const uint32_t rc = __ldg(rec + e);
            const float zz = __uint_as_float(rc & ~a.col_mask);
            const uint32_t col = rc & a.col_mask;
#pragma unroll
            for (int q = 0; q < kVecs; ++q) {
              const V v = *reinterpret_cast<const V*>(xs + q * plane_bytes + col * sizeof(V));
              const uint32_t* w = reinterpret_cast<const uint32_t*>(&v);
              constexpr int kW = static_cast<int>(sizeof(V)) / 4;
#pragma unroll
              for (int h = 0; h < kW; ++h) {
                acc[r][q * kW * 2 + 2 * h] = fmaf(zz, __uint_as_float(w[h] << 16), acc[r][q * kW * 2 + 2 * h]);
                acc[r][q * kW * 2 + 2 * h + 1] = fmaf(zz, __uint_as_float(w[h] & 0xFFFF0000u), acc[r][q * kW * 2 + 2 * h + 1]);
              }
            }
          }
        }
        TY* yp = yd + m0 * N + n;
        if constexpr (R == 2 && sizeof(TY) == 2) {
#pragma unroll
          for (int j = 0; j < TM; ++j)
            if (j < cnt) red_add_bf16x2(yp + j * N, pack_bf16x2(acc[0][j], acc[1][j]));
        } else {
#pragma unroll
          for (int r = 0; r < R; ++r) {
            if (n + r >= N) continue;
            float old[TM];
#pragma unroll
            for (int j = 0; j < TM; ++j) old[j] = (j < cnt) ? static_cast<float>(yp[j * N + r]) : 0.f;
#pragma unroll
            for (int j = 0; j < TM; ++j) {
              if (j < cnt) {
                if constexpr (sizeof(TY) == 2) yp[j * N + r] = __float2bfloat16_rn(old[j] + acc[r][j]);
                else yp[j * N + r] = old[j] + acc[r][j];
              }
            }
          }
        }
      }
    }
  }
}

template <typename Kern>
szo_status launch_cross(Kern kern, const char* name, CrossArgs ca, int TM, int R, int threads, size_t smem, cudaStream_t st) {
  SZO_CHECK_CUDA(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem)));
  int64_t units = 0;
  for (int i = 0; i < ca.n; ++i) {
    units += ceil_div(ca.sub[i].N, R);
    ca.unit_end[i] = units;
  }
  int dev = 0, sms = 148, per_sm = 1;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_CHECK_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  SZO_CHECK_CUDA(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, threads, smem));
  if (per_sm < 1) per_sm = 1;
  // as many blocks as the device holds at once; fewer when there is less than one unit per thread
  const int64_t total = ceil_div(ca.M, TM) * units;
  int64_t blocks = ceil_div(total, threads);
  if (blocks > static_cast<int64_t>(sms) * per_sm) blocks = static_cast<int64_t>(sms) * per_sm;
  if (blocks < 1) blocks = 1;
  SZO_CHECK_CUDA(launch_maybe_chained(kern, dim3(static_cast<unsigned>(blocks)), dim3(threads), smem, st, step_chained(), ca));
  count_launch();
  SZO_CHECK_LAUNCH(name);
  return SZO_OK;
}

template <int TM>
szo_status launch_cross_tm(const CrossArgs& ca, bool even, bool f32, cudaStream_t st) {
  constexpr int kThreads = TM >= 8 ? 1024 : 512;
  const size_t smem = static_cast<size_t>(ca.K) * TM * sizeof(__nv_bfloat16) + 128;       // (+ 64 per plane)
  if (f32) return launch_cross(pair_cross_kernel<TM, 1, float>, "pair_cross_kernel", ca, TM, 1, kThreads, smem, st);
  if (even) return launch_cross(pair_cross_kernel<TM, 2, __nv_bfloat16>, "pair_cross_kernel", ca, TM, 2, kThreads, smem, st);
  return launch_cross(pair_cross_kernel<TM, 1, __nv_bfloat16>, "pair_cross_kernel", ca, TM, 1, kThreads, smem, st);
}

}  // namespace

// rec[i]: the packed records of plans[i] (pack_cross_records / pack_cross_records_all); yd[i]: the first
// half-difference row of its y.  The plans share K, hence the kernel.
szo_status launch_paired_cross(const szo_linear* const* plans, int n, const void* x, int64_t M, const uint32_t* const* rec,
                               void* const* yd, int y_dtype, cudaStream_t st) {
  const szo_linear* p0 = plans[0];
  CrossArgs ca{};
  ca.n = n; ca.x = static_cast<const __nv_bfloat16*>(x); ca.M = M; ca.K = p0->K;
  ca.col_mask = (1u << col_bits_of(p0->K)) - 1u;
  bool even = true, any = false;
  for (int i = 0; i < n; ++i) {
    const szo_linear* p = plans[i];
    const CrossPlan* c = static_cast<const CrossPlan*>(p->cross);
    SZO_REQUIRE(p->nnz == 0 || c != nullptr, SZO_ERR_UNSUPPORTED, "K = %lld too large for the paired form", (long long)p->K);
    if (p->N & 1) even = false;
    if (c != nullptr) any = true;
    ca.sub[i] = CrossSub{c == nullptr ? nullptr : p->row_ptr, rec[i], yd[i], p->N};
  }
  if (!any) return SZO_OK;
  const size_t per_token = static_cast<size_t>(p0->K) * sizeof(__nv_bfloat16);
  const bool f32 = y_dtype == SZO_F32;
  static const int tm_env = [] {
    const char* e = getenv("SZO_CROSS_TM");
    return e == nullptr ? 0 : atoi(e);
  }();
  if (tm_env == 8 && 8 * per_token <= 200 * 1024) return launch_cross_tm<8>(ca, even, f32, st);
  // (16 tokens per slab pay from about 1300 tokens on: 0.493 -> 0.485 ms per paired gate/up linear at M = 1536, equal at
  // 1024, 0.223 -> 0.227 ms at 512)
  if (16 * per_token <= 200 * 1024 && ((M >= 1280 && tm_env != 8) || tm_env == 16)) return launch_cross_tm<16>(ca, even, f32, st);
  if (8 * per_token <= 200 * 1024) return launch_cross_tm<8>(ca, even, f32, st);
  if (4 * per_token <= 200 * 1024) return launch_cross_tm<4>(ca, even, f32, st);
  SZO_REQUIRE(2 * per_token <= 200 * 1024, SZO_ERR_UNSUPPORTED, "K = %lld too large for the paired form", (long long)p0->K);
  return launch_cross_tm<2>(ca, even, f32, st);
}

}  // namespace szo
