// Plan of one decomposed linear layer and the internal launchers around it.
#pragma once
#include "common.cuh"

struct szo_linear {
  int64_t N, K;
  int32_t G;          // 0: dense bf16 weight; -1: 4-bit codes into a per-row table of 16 values (lut)
  int32_t sz_dtype;
  int64_t nnz;
  // caller-owned
  const void* codes;  // uint8 [N,K/2] or bf16 [N,K]
  const void* scales;
  const void* zeros;
  const int64_t* idx;
  const float* bias;
  // derived, owned by the plan (device memory)
  uint8_t* codes_tiled;  // [Npad/128][K/64][128 rows][32 B]: the codes of one (128-row tile, k-block) contiguous,
                         // nibbles of each 32-bit word in pair order (see tile_codes_kernel)
  float2* sz;            // [K/G][Npad] (scale, zero) widened to fp32, group-major (G > 0)
  int64_t Npad;          // N rounded up to a multiple of 256
  int32_t* ent_col;      // [nnz] column of entry e
  int32_t* row_ptr;      // [N+1] entries of row r are [row_ptr[r], row_ptr[r+1])
  int32_t* bucket_ptr;   // [n_rowgroups * n_kblocks + 1]; bucket = (row/128, col/64)
  int32_t* bucket_eid;   // [nnz] entry id (index into S) in bucket order
  uint16_t* bucket_pos;  // [nnz] byte offset of the element inside its swizzled [128 x 64] bf16 tile, bucket order
  int64_t n_rowgroups, n_kblocks;
  void* tc;              // tensor-core side data (tensor maps), owned; see gemm_tc.cu
  void* cross;           // record layout of the paired form's sparse product, owned; see cross.cu (NULL: no entries)
  const void* lut;           // caller-owned table [N][16] (G == -1), 16-bit floats of type sz_dtype
  __nv_bfloat16* lut_bf16;   // owned: [Npad][16], RN_bf16 of the table, padding rows zero
};

namespace szo {

// fp32 reference path (linear.cu)
szo_status linear_fwd_fp32(const szo_linear* p, const void* x, int x_dtype, int64_t M, const float* S,
                           void* y, int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st);
size_t linear_ws_fp32(const szo_linear* p, int64_t M);

// CSR SpMM y[m, r] += sum_e S[e] x[m, c_e] (linear.cu); x bf16, y bf16 or fp32
szo_status linear_spmm(const szo_linear* p, const void* x, int64_t M, const float* S, void* y,
                       int y_dtype, cudaStream_t st);

// Weight-streaming kernel for at most 16 tokens (gemm_skinny.cu): int4 plans, K a multiple of 128;
// the sparse term is added in fp32 from the CSR rows (SparseAddMM).  Needs no workspace.
bool skinny_applies(const szo_linear* p, int64_t M);
// One to four tokens (gemm_gemv.cu): a CTA per 16 weight rows, no K-split between CTAs; same
// arguments as linear_fwd_skinny_group, which hands such calls over.
bool gemv_applies(const szo_linear* const* plans, int n, int64_t M);
// chained: launched as part of a chain of dependent kernels (common.cuh); x, x_mul and the norm's inputs must
// then be the only arguments that an earlier kernel of the stream writes.
// norm != NULL (x is then unused): the activations are the normalised residual stream, formed while they are
// staged, row m: v = h_in[m] + y_add[m] (y_add may be NULL), x[m] = RMSNorm or LayerNorm of v times gamma
// (plus beta) rounded to bf16, the arithmetic of the model's add_norm_kernel; the first CTA also writes v to
// h_out[m] (h_out must not be h_in: the other CTAs still read it).  K at most 8192.
struct FusedNorm {
  const float* h_in;
  const __nv_bfloat16* y_add;
  float* h_out;
  const float* gamma;
  const float* beta;
  float eps;
  bool layer_norm;
};
szo_status linear_fwd_gemv(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                           const float* const* S_pert, void* const* y, int y_dtype, cudaStream_t st, bool chained = false,
                           const FusedNorm* norm = nullptr);
// Up to three matrices that read the same activations in one launch (same K, G and table type);
// x_mul != NULL: the activations are silu(x) * x_mul rounded to bf16, formed while they are staged.
bool skinny_group_applies(const szo_linear* const* plans, int n, int64_t M);
bool few_token_applies(const szo_linear* const* plans, int n, int64_t M);     // either few-token kernel takes the group
szo_status linear_fwd_skinny_group(const szo_linear* const* plans, int n, const void* x, const void* x_mul, int64_t M,
                                   const float* const* S_pert, void* const* y, int y_dtype, cudaStream_t st,
                                   bool chained = false);
szo_status linear_fwd_skinny(const szo_linear* p, const void* x, int64_t M, const float* S_pert, void* y, int y_dtype,
                             cudaStream_t st);

// tensor-core path (gemm_tc.cu)
szo_status tc_plan_create(szo_linear* p, cudaStream_t st);
void tc_plan_destroy(szo_linear* p);
// S_bucket: the sparse entries gathered into bucket order as records
// (bucket_pos[p], bits of S[bucket_eid[p]]), or nullptr to leave the sparse term out (it is then
// applied by linear_spmm).
// ws: scratch of tc_tail_ws_bytes() bytes for the K-split tiles of the last round (may be nullptr:
// no split).
szo_status linear_fwd_tc(const szo_linear* p, const void* x, int64_t M, const uint2* S_bucket, void* y,
                         int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st);
// Several layers that read the same x in one launch (q/k/v, gate/up): same K, G and table dtype,
// G > 0, M > 128 (tc_can_fuse).  S_bucket[i] / y[i] belong to plans[i].
bool tc_can_fuse(const szo_linear* const* plans, int n, int64_t M);
szo_status linear_fwd_tc_group(const szo_linear* const* plans, int n, const void* x, int64_t M,
                               const uint2* const* S_bucket, void* const* y, int y_dtype, void* ws, size_t ws_bytes,
                               cudaStream_t st);
size_t tc_tail_ws_bytes(const szo_linear* const* plans, int n, int64_t M);
size_t tc_tail_ws_bound();   // enough for any M and any group
// Materialised form (gemm_tc.cu): the effective bf16 weight is written to scratch, then the dense
// mode of the kernel runs.  Chosen for int4 plans when M is large (tc_use_materialised).
bool tc_use_materialised(const szo_linear* p, int64_t M, bool two_sets = false);   // two_sets: one weight pass for two forwards
size_t tc_materialised_ws_bytes(const szo_linear* const* plans, int n, int64_t M, bool ext = false);   // ext: rows 2 K wide
// Paired form of a ZO step's two forwards (see tc::TcParams): x and every y[i] hold the M centre rows
// first and the M half-difference rows from row round_up(M, 256) on; S_pert are the unperturbed sparse
// values; rec[i] = the packed records of plans[i] (cross.cu).
// dense: the product runs on the tensor cores instead (eps * z written as a bf16 matrix beside W; z, eps
// are used, rec is not).
struct PairedArgs {
  const uint32_t* const* rec;
  const float* const* z;
  float eps;
  bool dense;
};
bool tc_paired_dense_cross(const szo_linear* const* plans, int n);
// Sparse product of the paired form (cross.cu).  A plan has one record slot per entry (the entries of a weight
// row in the order the kernel walks them); a record is one word, column and eps * z.
szo_status cross_plan_create(szo_linear* p);     // called by tc_plan_create; needs row_ptr and ent_col
void cross_plan_destroy(szo_linear* p);
size_t cross_rec_bytes(const szo_linear* const* plans, int n);
// rec[s] for the slots of one plan; z: the plan's entries
szo_status pack_cross_records(const szo_linear* p, const float* z, float eps, uint32_t* rec, cudaStream_t st);
// The records of many matrices in one launch: cross_copy_slots writes, once, a plan's slot descriptions into
// its part of model-wide arrays (src offset by base, where the plan's entries start in the model's z);
// pack_cross_records_all then packs all n slots.
szo_status cross_copy_slots(const szo_linear* p, int32_t base, uint32_t* colk, int32_t* src, cudaStream_t st);
szo_status pack_cross_records_all(const uint32_t* colk, const int32_t* src, const float* z, float eps, int64_t n, uint32_t* rec,
                                  cudaStream_t st);
// yd[i]: first half-difference row of plans[i]'s y; x: the centre rows
szo_status launch_paired_cross(const szo_linear* const* plans, int n, const void* x, int64_t M, const uint32_t* const* rec,
                               void* const* yd, int y_dtype, cudaStream_t st);
szo_status linear_fwd_tc_materialised(const szo_linear* const* plans, int n, const void* x, int64_t M,
                                      const float* const* S_pert, void* const* y, int y_dtype, void* ws,
                                      size_t ws_bytes, cudaStream_t st, const float* const* S_second = nullptr,
                                      __nv_bfloat16* W_resident = nullptr, __nv_bfloat16* saved_resident = nullptr,
                                      bool relu = false,    // relu: y = max(y, 0) applied in the epilogue
                                      const PairedArgs* paired = nullptr);
// Resident form for dense bf16 plans (G == 0): W_resident [sum Npad, K] and saved_resident [sum nnz]
// are filled once by tc_resident_init and passed to linear_fwd_tc_materialised, which then skips the
// weight pass and writes every masked entry as RN_bf16(saved + S); ws is only the K-split scratch.
bool tc_use_resident(const szo_linear* p, int64_t M);
bool tc_can_stack(const szo_linear* const* plans, int n);
void tc_resident_bytes(const szo_linear* const* plans, int n, size_t* w_bytes, size_t* saved_bytes, bool ext = false);
szo_status tc_resident_init(const szo_linear* const* plans, int n, __nv_bfloat16* W, __nv_bfloat16* saved,
                            cudaStream_t st, bool ext = false);
// S_second: a second set of sparse values and of M tokens served by the same weight pass (x and
// y[i] hold 2 M rows).
// out[p] = (pos[p], bits of S[eid[p]]) for p in [0, n)
szo_status gather_values(const float* S, const int32_t* eid, const uint16_t* pos, int64_t n, uint2* out,
                         cudaStream_t st);
// Forward with every option: S_bucket may be given (pre-gathered, SparseAdd mode) to skip the
// per-call gather into the workspace.
szo_status linear_fwd_impl(const szo_linear* p, const void* x, int x_dtype, int64_t M, const float* S_pert,
                           const uint2* S_bucket, void* y, int y_dtype, int32_t mode, void* workspace,
                           size_t workspace_bytes, cudaStream_t st);

}  // namespace szo
