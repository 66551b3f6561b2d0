// Host side of the tensor-core path of the decomposed linear layer
//   y[m, n] = sum_k x[m,k] * (Dequantize(Q)[n,k] + S[n,k]) + bias[n]
// (appendix "Implementation of Sparse Operations in Linear Layers":
// DenseMM(SparseAdd(w_sparse, Dequantize(Q(w_dense))), x)): tensor maps, the per-plan data, the work
// schedule of the pair-tile kernel (gemm_tc2.cu) and its launch for one layer or for several layers
// that read the same activations.
#include <cstdlib>

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
  return launch_pair_kernel(p0->G != 0, p0->sz_dtype == SZO_BF16, mx, t->w_map, P, sc.n_pairs, st);
}

szo_status linear_fwd_tc(const szo_linear* p, const void* x, int64_t M, const uint2* S_bucket, void* y,
                         int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st) {
  return linear_fwd_tc_group(&p, 1, x, M, &S_bucket, &y, y_dtype, ws, ws_bytes, st);
}

}  // namespace szo
