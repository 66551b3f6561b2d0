// Host side of the tensor-core path of the decomposed linear layer
//   y[m, n] = sum_k x[m,k] * (Dequantize(Q)[n,k] + S[n,k]) + bias[n]
// (appendix "Implementation of Sparse Operations in Linear Layers":
// DenseMM(SparseAdd(w_sparse, Dequantize(Q(w_dense))), x)): tensor maps, the per-plan data, the work
// schedule of the pair-tile kernel (gemm_tc2.cu) and its launch for one layer or for several layers
// that read the same activations.
#include <cstdlib>
#include <vector>

#include "tc_common.cuh"

namespace szo {

namespace {

using namespace tc;

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
  uint64_t clean_epoch; // abort_epoch() when the tickets were last known to be zero
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

}  // namespace

// A kernel that gave up on a bounded wait leaves the tickets of its K-split tiles non-zero (only the
// part that finishes last resets them).  Once the host has seen that status (szo_device_status), every
// plan clears its tickets before its next launch.
static szo_status refresh_tickets(const TcPlan* tc, cudaStream_t st) {
  TcPlan* t = const_cast<TcPlan*>(tc);
  const uint64_t now = abort_epoch();
  if (t->clean_epoch != now) {
    SZO_CHECK_CUDA(cudaMemsetAsync(t->tickets, 0, static_cast<size_t>(t->sms / 2) * 8 * sizeof(int32_t), st));
    t->clean_epoch = now;
  }
  return SZO_OK;
}

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
  t->clean_epoch = abort_epoch();
  p->tc = t;
  const szo_status bs = cross_plan_create(p);
  if (bs != SZO_OK) {
    tc_plan_destroy(p);
    return bs;
  }
  return SZO_OK;
}

void tc_plan_destroy(szo_linear* p) {
  TcPlan* t = static_cast<TcPlan*>(p->tc);
  if (t) cudaFree(t->tickets);
  delete t;
  cross_plan_destroy(p);
  p->tc = nullptr;
}

static int64_t pair_tiles(const szo_linear* const* plans, int n, int64_t M) {
  int64_t nt = 0;
  for (int i = 0; i < n; ++i) nt += ceil_div(plans[i]->N, 256);
  return nt * ceil_div(M, 256);
}

size_t tc_tail_ws_bytes(const szo_linear* const* plans, int n, int64_t M) {
  if (n < 1 || plans[0]->tc == nullptr) return 0;
  const TcPlan* t = static_cast<const TcPlan*>(plans[0]->tc);
  return pair_schedule(pair_tiles(plans, n, M), static_cast<int>(plans[0]->K / kBK), plans[0]->G, t->sms, true).ws_bytes;
}

size_t tc_tail_ws_bound() {
  int dev = 0, sms = 148;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  return static_cast<size_t>(sms / 2) * 2 * 256 * kBM * sizeof(float);
}

bool tc_can_fuse(const szo_linear* const* plans, int n, int64_t M) {
  if (n < 2 || n > 3) return false;
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
  P.tickets_done = t->tickets + (t->sms / 2) * 4;
  SZO_TRY(refresh_tickets(t, st));
  return launch_pair_kernel(p0->G != 0, p0->sz_dtype == SZO_BF16, mx, t->w_map, P, sc.n_pairs, st);
}

// ------------------------------------------------------------------------------ materialised form
// For many tokens the appendix's DenseMM(SparseAdd(w_sparse, Dequantize(Q(w_dense))), x) is cheaper
// taken literally: one pass writes the effective weight RN_bf16(q*scale+zero), RN_bf16(. + S) at the
// masked positions, as a bf16 matrix into scratch (2.5 bytes per weight of HBM traffic), and the
// tensor-core kernel runs in its dense mode, where no conversion competes with the MMAs for issue
// slots.  The values are bit-identical to what the fused mode builds in shared memory.
namespace {

// Up to three matrices (the layers of one launch) per kernel call.
struct MatSub {
  const uint8_t* codes_tiled;
  const float2* sz;
  int64_t Npad;
  __nv_bfloat16* out;         // [Npad, K] row-major
  const int64_t* idx;         // sparse entries: flat indices n * K + c, values S
  const float* S;
  int64_t words_end, nnz_end; // running totals over the matrices: work items of this and the earlier ones
  __nv_bfloat16* saved;       // [nnz] dense values at the masked positions (two-set form)
  const __nv_bfloat16* lut;   // [Npad][16] per-row table of the non-uniform 4-bit format (G == -1), else nullptr
};
struct MatArgs {
  MatSub sub[3];
  int n, nkb, G;
  int64_t K;
  int64_t ld;                 // row stride of the output buffers in elements (K, or 2 K when eps * Zbar sits beside W)
  int scatter_mode;           // 0: w += S; 1: saved = w, w += S; 2: w = saved + S (second set of sparse values)
};

// thread -> four 32-bit words of the tile-ordered codes (8 weights each, rows r, r + 32, r + 64, r + 96
// of one tile) -> four 16-byte pieces of the row-major output; the four loads are issued before the
// first use.  A warp covers four k-blocks of one row at a time: 32-byte reads from four code
// blocks, one 512-byte contiguous write.  Work items per matrix: (Npad / 128) * ceil(nkb / 4) * 1024.
// kKind 0: fp32 (scale, zero) pairs; 1: packed bf16 pairs (exact bf16 arithmetic); 2: the non-uniform
// format, where the code selects one of the 16 bf16 values of its row (a warp works on one row per
// load, so the 32 look-ups of an instruction hit one 32-byte line).
template <int kKind>
__global__ void materialise_kernel(const MatArgs a) {
  chain_release();
  chain_wait();          // (the scratch it overwrites is what the previous tensor-core launch read)
  int64_t i = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (i >= a.sub[a.n - 1].words_end) return;
  int s = 0;
  if (i >= a.sub[0].words_end) s = (a.n > 2 && i >= a.sub[1].words_end) ? 2 : 1;
  if (s > 0) i -= a.sub[s - 1].words_end;
  const uint8_t* codes_tiled = s == 0 ? a.sub[0].codes_tiled : (s == 1 ? a.sub[1].codes_tiled : a.sub[2].codes_tiled);
  const float2* sz = s == 0 ? a.sub[0].sz : (s == 1 ? a.sub[1].sz : a.sub[2].sz);
  const int64_t Npad = s == 0 ? a.sub[0].Npad : (s == 1 ? a.sub[1].Npad : a.sub[2].Npad);
  __nv_bfloat16* out = s == 0 ? a.sub[0].out : (s == 1 ? a.sub[1].out : a.sub[2].out);
  const int chunk = static_cast<int>(i & 7), kbo = static_cast<int>((i >> 3) & 3), r0 = static_cast<int>((i >> 5) & 31);
  const int nkb4 = (a.nkb + 3) >> 2;
  const int64_t grp = i >> 10;
  const int64_t t = grp / nkb4;
  const int kb = static_cast<int>(grp - t * nkb4) * 4 + kbo;
  if (kb >= a.nkb) return;
  const uint8_t* src = codes_tiled + (t * a.nkb + kb) * kCodesBytes + r0 * 32 + chunk * 4;
  __nv_bfloat16* dst = out + (t * kBM + r0) * a.ld + kb * kBK + chunk * 8;
  uint32_t w[4];
  if constexpr (kKind == 2) {
    const __nv_bfloat16* lut = s == 0 ? a.sub[0].lut : (s == 1 ? a.sub[1].lut : a.sub[2].lut);
    const unsigned short* row = reinterpret_cast<const unsigned short*>(lut) + (t * kBM + r0) * 16;
#pragma unroll
    for (int j = 0; j < 4; ++j) w[j] = *reinterpret_cast<const uint32_t*>(src + j * 32 * 32);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const unsigned short* rj = row + j * 32 * 16;
      uint32_t o[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {       // nibble i is column 2 i, nibble 4 + i column 2 i + 1 (pair order)
        const uint32_t lo = __ldg(rj + ((w[j] >> (4 * i)) & 0xFu));
        const uint32_t hi = __ldg(rj + ((w[j] >> (16 + 4 * i)) & 0xFu));
        o[i] = lo | (hi << 16);
      }
      *reinterpret_cast<uint4*>(dst + static_cast<int64_t>(j) * 32 * a.ld) = make_uint4(o[0], o[1], o[2], o[3]);
    }
  } else {
    const int g = (kb * kBK + chunk * 8) / a.G;
    const float2* szp = sz + static_cast<int64_t>(g) * Npad + t * kBM + r0;
    float2 p[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      w[j] = *reinterpret_cast<const uint32_t*>(src + j * 32 * 32);
      p[j] = szp[j * 32];
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      *reinterpret_cast<uint4*>(dst + static_cast<int64_t>(j) * 32 * a.ld) = dequant_word<kKind == 1>(w[j], p[j]);
  }
}

// SparseAdd on the materialised matrices: indices are unique, so no two threads touch one element.
// With two sets of sparse values for one weight pass (the two perturbed forwards of a ZO step) the
// dense values at the masked positions are kept aside by the first scatter and reused by the second.
__global__ void scatter_add_bf16_kernel(const MatArgs a) {
  chain_release();
  chain_wait();
  int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= a.sub[a.n - 1].nnz_end) return;
  int s = 0;
  if (e >= a.sub[0].nnz_end) s = (a.n > 2 && e >= a.sub[1].nnz_end) ? 2 : 1;
  if (s > 0) e -= a.sub[s - 1].nnz_end;
  const int64_t* idx = s == 0 ? a.sub[0].idx : (s == 1 ? a.sub[1].idx : a.sub[2].idx);
  const float* S = s == 0 ? a.sub[0].S : (s == 1 ? a.sub[1].S : a.sub[2].S);
  __nv_bfloat16* saved = s == 0 ? a.sub[0].saved : (s == 1 ? a.sub[1].saved : a.sub[2].saved);
  const int64_t flat = idx[e];
  const int64_t row = flat / a.K;
  __nv_bfloat16* el = (s == 0 ? a.sub[0].out : (s == 1 ? a.sub[1].out : a.sub[2].out)) + row * a.ld + (flat - row * a.K);
  __nv_bfloat16 base;
  if (a.scatter_mode == 2) {
    base = saved[e];              // the element itself is not read: it holds the other set's value
  } else {
    base = *el;
    if (a.scatter_mode == 1) saved[e] = base;
  }
  *el = __float2bfloat16_rn(__bfloat162float(base) + S[e]);
}

}  // namespace

namespace {

// Dense form of the sparse product (TcParams::pair_ext): eps * z written as bf16 into the second half
// [K, 2 K) of the weight rows, which is zero elsewhere.
__global__ void scatter_z_bf16_kernel(const MatArgs a, float eps) {
  int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e >= a.sub[a.n - 1].nnz_end) return;
  int s = 0;
  if (e >= a.sub[0].nnz_end) s = (a.n > 2 && e >= a.sub[1].nnz_end) ? 2 : 1;
  if (s > 0) e -= a.sub[s - 1].nnz_end;
  const int64_t* idx = s == 0 ? a.sub[0].idx : (s == 1 ? a.sub[1].idx : a.sub[2].idx);
  const float* z = s == 0 ? a.sub[0].S : (s == 1 ? a.sub[1].S : a.sub[2].S);     // the S slot carries z here
  const int64_t flat = idx[e];
  const int64_t row = flat / a.K;
  __nv_bfloat16* el = (s == 0 ? a.sub[0].out : (s == 1 ? a.sub[1].out : a.sub[2].out)) + row * a.ld + a.K + (flat - row * a.K);
  *el = __float2bfloat16_rn(eps * z[e]);
}

// SZO_LINEAR_MATERIALISE=0 / 1 switches the form off / on for every M (A/B measurement)
int materialise_override() {
  static const int v = [] {
    const char* e = getenv("SZO_LINEAR_MATERIALISE");
    return e == nullptr ? -1 : (e[0] == '0' ? 0 : 1);
  }();
  return v;
}

}  // namespace

bool tc_use_materialised(const szo_linear* p, int64_t M, bool two_sets) {
  if (p->G == 0 || p->tc == nullptr) return false;
  if (p->G < 0) return true;      // table-coded weights have this form only
  const int o = materialise_override();
  if (o >= 0) return o == 1;
  // the extra pass costs about 2.5 N K bytes of traffic, the fused conversion 5-10 % of 2 M N K flop at
  // the kernel's rate: measured break-even near M = 2048 (4096^2: 73 vs 75 us), 7 % ahead at M = 4096.
  // When one weight pass serves the two perturbed forwards of a step, the break-even halves
  // (Llama-2-7B-shaped step: 54.2 vs 57.5 ms at 2048 tokens, 31.3 vs 31.6 at 1024, 21.1 vs 20.8 at 512).
  return M >= (two_sets ? 2048 : 4096);
}

size_t tc_materialised_ws_bytes(const szo_linear* const* plans, int n, int64_t M, bool ext) {
  size_t rows = 0;
  for (int i = 0; i < n; ++i) rows += static_cast<size_t>(plans[i]->Npad);
  size_t nnz = 0;
  for (int i = 0; i < n; ++i) nnz += static_cast<size_t>(plans[i]->nnz);
  return round_up(rows * static_cast<size_t>(plans[0]->K) * (ext ? 2 : 1) * sizeof(__nv_bfloat16), 256) +
         round_up(nnz * sizeof(__nv_bfloat16), 256) + tc_tail_ws_bound();
}

// Paired form: where does eps * xc Zbar^T run?  On the CUDA cores (pair_cross_kernel) its cost grows
// with the number of entries (18.8 ms of a Llama-2-7B-shaped step at 0.1 %, 200 ms of a Mistral-7B-shaped
// one at 1 %); on the tensor cores it is half the dense flops again whatever the mask.  The break-even
// is near a density of 0.2 %.  SZO_PAIRED_CROSS=sparse|dense forces either (A/B, tests).
bool tc_paired_dense_cross(const szo_linear* const* plans, int n) {
  static const int forced = [] {
    const char* e = getenv("SZO_PAIRED_CROSS");
    return e == nullptr ? -1 : (e[0] == 'd' ? 1 : 0);
  }();
  double nnz = 0, elems = 0;
  for (int i = 0; i < n; ++i) {
    nnz += static_cast<double>(plans[i]->nnz);
    elems += static_cast<double>(plans[i]->N) * static_cast<double>(plans[i]->K);
  }
  if (nnz == 0) return false;
  if (forced >= 0) return forced == 1;
  return nnz >= 0.002 * elems;
}

// Resident form (dense bf16 plans, G == 0).  With nothing to dequantise, the effective weight of a
// launch group can stay in device memory across calls: a private copy [sum Npad, K] of the group's
// frozen weights, made once, plus the frozen values at the masked positions.  A forward then only
// rewrites the masked entries (RN_bf16(frozen + S), the SparseAdd of the appendix on sparse
// operations) and runs the dense mode of the kernel; no entry needs restoring afterwards, because the
// next scatter writes every masked position again from the saved frozen value.
// Measured on the Mistral-7B shape (1 % mask) it is ahead of the fused form at every token count tried
// (step at 4096 / 2048 / 1024 / 512 tokens: 115 / 60 / 35 / 23 ms against 132 / 72 / 42 / 31), so it is
// taken for every M; SZO_LINEAR_MATERIALISE=0 switches it off.
bool tc_use_resident(const szo_linear* p, int64_t) {
  if (p->G != 0 || p->tc == nullptr) return false;
  return materialise_override() != 0;
}

bool tc_can_stack(const szo_linear* const* plans, int n) {
  if (n < 1 || n > 3) return false;
  for (int i = 0; i < n; ++i)
    if (plans[i]->G != 0 || plans[i]->tc == nullptr || plans[i]->K != plans[0]->K) return false;
  return true;
}

void tc_resident_bytes(const szo_linear* const* plans, int n, size_t* w_bytes, size_t* saved_bytes, bool ext) {
  size_t rows = 0, nnz = 0;
  for (int i = 0; i < n; ++i) {
    rows += static_cast<size_t>(plans[i]->Npad);
    nnz += static_cast<size_t>(plans[i]->nnz);
  }
  *w_bytes = round_up(rows * static_cast<size_t>(plans[0]->K) * (ext ? 2 : 1) * sizeof(__nv_bfloat16), 256);
  *saved_bytes = round_up(nnz * sizeof(__nv_bfloat16), 256);
}

namespace {
__global__ void gather_bf16_kernel(const __nv_bfloat16* __restrict__ W, const int64_t* __restrict__ idx, int64_t nnz,
                                   __nv_bfloat16* __restrict__ out) {
  const int64_t e = static_cast<int64_t>(blockIdx.x) * blockDim.x + threadIdx.x;
  if (e < nnz) out[e] = W[idx[e]];
}
}  // namespace

// Fills the resident buffers of one launch group: rows [0, N) of every matrix copied from the frozen
// weight, the padding rows zero, saved[e] = the frozen value at masked position e.
szo_status tc_resident_init(const szo_linear* const* plans, int n, __nv_bfloat16* W, __nv_bfloat16* saved,
                            cudaStream_t st, bool ext) {
  SZO_REQUIRE(tc_can_stack(plans, n), SZO_ERR_INVALID_ARG, "resident form: dense bf16 plans with one K only");
  int64_t row0 = 0, nnz = 0;
  const int64_t ld = plans[0]->K * (ext ? 2 : 1);       // ext: columns [K, 2 K) hold eps * Zbar, zero outside the mask
  for (int i = 0; i < n; ++i) {
    const szo_linear* p = plans[i];
    __nv_bfloat16* dst = W + row0 * ld;
    if (ext || p->Npad > p->N)
      SZO_CHECK_CUDA(cudaMemsetAsync(dst, 0, static_cast<size_t>(p->Npad) * ld * sizeof(__nv_bfloat16), st));
    SZO_CHECK_CUDA(cudaMemcpy2DAsync(dst, ld * sizeof(__nv_bfloat16), p->codes, p->K * sizeof(__nv_bfloat16),
                                     p->K * sizeof(__nv_bfloat16), p->N, cudaMemcpyDeviceToDevice, st));
    if (p->nnz > 0) {
      gather_bf16_kernel<<<static_cast<unsigned>(ceil_div(p->nnz, 256)), 256, 0, st>>>(
          static_cast<const __nv_bfloat16*>(p->codes), p->idx, p->nnz, saved + nnz);
      count_launch();
    }
    nnz += p->nnz;
    row0 += p->Npad;
  }
  SZO_CHECK_LAUNCH("gather_bf16_kernel");
  return SZO_OK;
}

// n matrices that share x (n == 1 or tc_can_fuse): materialise, SparseAdd, dense launch.  With
// S_second != nullptr the weight pass serves two sets of sparse values (S_pert and S_second) and two
// sets of M tokens each: x and every y[i] then hold 2 M rows, set 0 first.
szo_status linear_fwd_tc_materialised(const szo_linear* const* plans, int n, const void* x, int64_t M,
                                      const float* const* S_pert, void* const* y, int y_dtype, void* ws,
                                      size_t ws_bytes, cudaStream_t st, const float* const* S_second,
                                      __nv_bfloat16* W_resident, __nv_bfloat16* saved_resident, bool relu,
                                      const PairedArgs* paired) {
  const szo_linear* p0 = plans[0];
  const bool resident = W_resident != nullptr;
  SZO_REQUIRE(paired == nullptr || (S_second == nullptr && !relu), SZO_ERR_INVALID_ARG,
              "the paired form takes one set of sparse values and no ReLU epilogue");
  // paired form: M centre rows, then M half-difference rows from row Mp (a multiple of 256) on
  const int64_t Mp = paired != nullptr ? static_cast<int64_t>(round_up(static_cast<size_t>(M), 256)) : 0;
  const int64_t M_rows = paired != nullptr ? Mp + M : M;
  const TcPlan* t = static_cast<const TcPlan*>(p0->tc);
  SZO_REQUIRE(t != nullptr, SZO_ERR_INVALID_ARG, "plan has no tensor-core data");
  SZO_REQUIRE(M < (int64_t(1) << 31), SZO_ERR_SHAPE, "M too large");
  int64_t rows = 0;
  size_t nnz_all = 0;
  for (int i = 0; i < n; ++i) {
    rows += plans[i]->Npad;
    nnz_all += static_cast<size_t>(plans[i]->nnz);
  }
  // dense form of the paired sparse product: eps * Zbar beside W, rows 2 K wide
  const bool ext = paired != nullptr && paired->dense && nnz_all > 0;
  const int64_t ld = p0->K * (ext ? 2 : 1);
  // resident form: the weight and the dense values at the masked positions live in the caller's buffers
  const size_t w_bytes = resident ? 0 : round_up(static_cast<size_t>(rows) * ld * sizeof(__nv_bfloat16), 256);
  const size_t saved_bytes = resident ? 0 : round_up(nnz_all * sizeof(__nv_bfloat16), 256);
  SZO_REQUIRE(resident || (ws != nullptr && ws_bytes >= w_bytes + saved_bytes), SZO_ERR_WORKSPACE,
              "the materialised form needs a workspace of at least %zu bytes", w_bytes + saved_bytes);
  SZO_REQUIRE(!resident || nnz_all == 0 || saved_resident != nullptr, SZO_ERR_INVALID_ARG,
              "resident form without the saved dense values");
  SZO_REQUIRE(rows < (int64_t(1) << 31), SZO_ERR_SHAPE, "too many weight rows in one launch");
  __nv_bfloat16* W = resident ? W_resident : static_cast<__nv_bfloat16*>(ws);
  __nv_bfloat16* saved = resident ? saved_resident
                                  : reinterpret_cast<__nv_bfloat16*>(static_cast<unsigned char*>(ws) + w_bytes);
  const int nkb = static_cast<int>(p0->K / kBK);
  MatArgs a{};
  a.n = n; a.nkb = nkb; a.G = p0->G; a.K = p0->K; a.ld = ld;
  int64_t row0 = 0, words = 0, nnz = 0;
  for (int i = 0; i < n; ++i) {
    const szo_linear* p = plans[i];
    words += (p->Npad / kBM) * ((nkb + 3) / 4) * 1024;
    SZO_REQUIRE(p->G == p0->G && p->K == p0->K, SZO_ERR_INVALID_ARG, "matrices of one launch must share K and format");
    a.sub[i] = MatSub{p->codes_tiled, p->sz, p->Npad, W + row0 * ld, p->idx, S_pert[i], words, nnz + p->nnz, saved + nnz,
                      p->lut_bf16};
    nnz += p->nnz;
    row0 += p->Npad;
  }
  if (!resident && p0->G == 0) {
    // dense bf16 plans outside a model (which keeps them resident): copy the frozen weight
    int64_t r0 = 0;
    for (int i = 0; i < n; ++i) {
      const szo_linear* p = plans[i];
      SZO_CHECK_CUDA(cudaMemcpy2DAsync(W + r0 * ld, ld * sizeof(__nv_bfloat16), p->codes, p->K * sizeof(__nv_bfloat16),
                                       p->K * sizeof(__nv_bfloat16), p->N, cudaMemcpyDeviceToDevice, st));
      if (p->Npad > p->N)
        SZO_CHECK_CUDA(cudaMemsetAsync(W + (r0 + p->N) * ld, 0, static_cast<size_t>(p->Npad - p->N) * ld * sizeof(__nv_bfloat16), st));
      r0 += p->Npad;
    }
  } else if (!resident) {
    const unsigned blocks = static_cast<unsigned>(ceil_div(words, 256));
    auto mk = p0->G < 0 ? materialise_kernel<2> : (p0->sz_dtype == SZO_BF16 ? materialise_kernel<1> : materialise_kernel<0>);
    SZO_CHECK_CUDA(launch_maybe_chained(mk, dim3(blocks), dim3(256), 0, st, step_chained(), a));
    count_launch();
    SZO_CHECK_LAUNCH("materialise_kernel");
  }
  if (ext && !resident)        // the eps * Zbar half starts from zero (the resident buffer keeps its zeros: the
                               // entries sit at the same positions every step)
    SZO_CHECK_CUDA(cudaMemset2DAsync(W + p0->K, ld * sizeof(__nv_bfloat16), 0, p0->K * sizeof(__nv_bfloat16), rows, st));
  CUtensorMap mw;
  SZO_TRY(make_map(&mw, W, rows, ld, kBM));
  TcParams P{};
  P.M = M_rows; P.K = p0->K; P.G = 0; P.nkb = nkb;
  P.relu = relu ? 1 : 0;
  P.m_tiles = ceil_div(M_rows, 256);
  P.nsub = n;
  if (paired != nullptr) {
    P.pair_row0 = Mp;
    P.pair_ext = ext ? 1 : 0;
  }
  int64_t n_tiles = 0;
  for (int i = 0; i < n; ++i) {
    const szo_linear* p = plans[i];
    TcSub& sb = P.sub[i];
    sb.codes = nullptr;
    sb.sz = nullptr;
    sb.bucket_ptr = nullptr;
    sb.Sb = nullptr;
    sb.bias = p->bias;
    sb.N = p->N;
    sb.Npad = p->Npad;
    sb.n_rowtiles = 0;
    sb.n_tiles = static_cast<int>(p->Npad / 256);     // the buffer pads every matrix to whole pair tiles
    n_tiles += sb.n_tiles;
  }
  P.n_tiles = n_tiles;
  // bands of token tiles that fit L2 with room to spare: at most 48 MB of tokens per band, and bands of equal
  // height (32 token tiles: two bands of 16 at K = 4096, four of 8 at K = 11008; measured per paired linear,
  // 8192 rows: K = 4096, N = 22016: 8 / 12 / 16 / 24 tiles per band 1.265 / 1.240 / 1.226 / 1.251 ms, no bands
  // 1.31 ms; K = 11008, N = 4096: 4 / 5 / 8 / 16 tiles 0.665 / 0.669 / 0.653 / 0.655 ms, no bands 0.689 ms)
  {
    static const int band_env = [] {
      const char* e = getenv("SZO_TILE_BAND");
      return e == nullptr ? -1 : atoi(e);
    }();
    const int64_t band_max = (48ll << 20) / (256 * p0->K * 2);
    int band = 0;
    if (band_max >= 1 && P.m_tiles > band_max) band = static_cast<int>(ceil_div(P.m_tiles, ceil_div(P.m_tiles, band_max)));
    if (band_env >= 0) band = band_env;
    P.m_band = (band > 0 && P.m_tiles > band) ? band : 0;
  }
  P.y_f32 = (y_dtype == SZO_F32) ? 1 : 0;
  P.status = device_status_word();
  SZO_REQUIRE(P.status != nullptr, SZO_ERR_CUDA, "no device status word");
  const int64_t tiles = P.m_tiles * P.n_tiles;
  SZO_REQUIRE(tiles < (int64_t(1) << 30), SZO_ERR_SHAPE, "too many tiles");
  void* tail = ws == nullptr ? nullptr : static_cast<unsigned char*>(ws) + w_bytes + saved_bytes;
  const size_t tail_bytes = ws == nullptr ? 0 : ws_bytes - w_bytes - saved_bytes;
  PairSchedule sc = pair_schedule(tiles, P.nkb, 0, t->sms, tail != nullptr);
  if (sc.ws_bytes > tail_bytes) sc = pair_schedule(tiles, P.nkb, 0, t->sms, false);
  P.full_rounds = sc.full_rounds;
  P.tail_tiles = sc.tail_tiles;
  P.tail_parts = sc.tail_parts;
  for (int i = 0; i < 5; ++i) P.tail_kb[i] = sc.tail_kb[i];
  P.partial = static_cast<float*>(tail);
  P.tickets = t->tickets;
  P.tickets_done = t->tickets + (t->sms / 2) * 4;
  SZO_TRY(refresh_tickets(t, st));
  const size_t y_elt = (y_dtype == SZO_F32) ? 4 : 2;
  const int n_sets = S_second != nullptr ? 2 : 1;
  if (ext) {
    MatArgs az = a;
    for (int i = 0; i < n; ++i) az.sub[i].S = paired->z[i];
    scatter_z_bf16_kernel<<<static_cast<unsigned>(ceil_div(nnz, 256)), 256, 0, st>>>(az, paired->eps);
    count_launch();
    SZO_CHECK_LAUNCH("scatter_z_bf16_kernel");
  }
  for (int set = 0; set < n_sets; ++set) {
    if (nnz > 0) {
      a.scatter_mode = resident ? 2 : (n_sets == 1 ? 0 : set + 1);
      if (set == 1)
        for (int i = 0; i < n; ++i) a.sub[i].S = S_second[i];
      SZO_CHECK_CUDA(launch_maybe_chained(scatter_add_bf16_kernel, dim3(static_cast<unsigned>(ceil_div(nnz, 256))), dim3(256), 0, st,
                                          step_chained(), a));
      count_launch();
    }
    CUtensorMap mx;
    SZO_TRY(make_map(&mx, static_cast<const __nv_bfloat16*>(x) + static_cast<int64_t>(set) * M * p0->K, M_rows, p0->K, 128));
    for (int i = 0; i < n; ++i)
      P.sub[i].y = static_cast<unsigned char*>(y[i]) + static_cast<size_t>(set) * M * plans[i]->N * y_elt;
    SZO_TRY(launch_pair_kernel(false, false, mx, mw, P, sc.n_pairs, st));
  }
  if (paired != nullptr && nnz_all > 0 && !ext) {
    void* yd[3];
    for (int i = 0; i < n; ++i) yd[i] = static_cast<unsigned char*>(y[i]) + static_cast<size_t>(Mp) * plans[i]->N * y_elt;
    SZO_TRY(launch_paired_cross(plans, n, x, M, paired->rec, yd, y_dtype, st));
  }
  return SZO_OK;
}

szo_status linear_fwd_tc(const szo_linear* p, const void* x, int64_t M, const uint2* S_bucket, void* y,
                         int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st) {
  return linear_fwd_tc_group(&p, 1, x, M, &S_bucket, &y, y_dtype, ws, ws_bytes, st);
}

}  // namespace szo

extern "C" szo_status szo_selftest_wait_timeout(double limit_ms, int32_t* gave_up_host, void* stream) {
  using namespace szo;
  SZO_REQUIRE(gave_up_host != nullptr, SZO_ERR_INVALID_ARG, "gave_up_host is NULL");
  SZO_REQUIRE(limit_ms > 0.0 && limit_ms <= 100.0, SZO_ERR_INVALID_ARG, "limit_ms must be in (0, 100]");
  int dev = 0, khz = 0;
  SZO_CHECK_CUDA(cudaGetDevice(&dev));
  SZO_CHECK_CUDA(cudaDeviceGetAttribute(&khz, cudaDevAttrClockRate, dev));
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  int32_t* flag = nullptr;
  SZO_CHECK_CUDA(cudaMalloc(&flag, sizeof(int32_t)));
  cudaMemsetAsync(flag, 0, sizeof(int32_t), st);
  szo_status rc = launch_wait_timeout_selftest(static_cast<long long>(limit_ms * khz), flag, st);
  if (rc == SZO_OK && (cudaMemcpyAsync(gave_up_host, flag, sizeof(int32_t), cudaMemcpyDeviceToHost, st) != cudaSuccess ||
                       cudaStreamSynchronize(st) != cudaSuccess))
    rc = fail(SZO_ERR_CUDA, "self-test read-back failed");
  cudaFree(flag);
  return rc;
}
