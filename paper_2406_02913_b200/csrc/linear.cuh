// Plan of one decomposed linear layer and the internal launchers around it.
#pragma once
#include "common.cuh"

struct szo_linear {
  int64_t N, K;
  int32_t G;          // 0: dense bf16 weight
  int32_t sz_dtype;
  int64_t nnz;
  // caller-owned
  const void* codes;  // uint8 [N,K/2] or bf16 [N,K]
  const void* scales;
  const void* zeros;
  const int64_t* idx;
  const float* bias;
  // derived, owned by the plan (device memory)
  float2* sz;            // [N, K/G] (scale, zero) widened to fp32 (G > 0)
  int32_t* ent_col;      // [nnz] column of entry e
  int32_t* row_ptr;      // [N+1] entries of row r are [row_ptr[r], row_ptr[r+1])
  int32_t* bucket_ptr;   // [n_rowgroups * n_kblocks + 1]; bucket = (row/32, col/64)
  int32_t* bucket_eid;   // [nnz] entry id (index into S) in bucket order
  uint16_t* bucket_pos;  // [nnz] (local_row << 6) | local_col in bucket order
  int64_t n_rowgroups, n_kblocks;
  void* tc;              // tensor-core side data (tensor maps), owned; see gemm_tc.cu
};

namespace szo {

// fp32 reference path (linear.cu)
szo_status linear_fwd_fp32(const szo_linear* p, const void* x, int x_dtype, int64_t M, const float* S,
                           void* y, int y_dtype, void* ws, size_t ws_bytes, cudaStream_t st);
size_t linear_ws_fp32(const szo_linear* p, int64_t M);

// CSR SpMM y[m, r] += sum_e S[e] x[m, c_e] (linear.cu); x bf16, y bf16 or fp32
szo_status linear_spmm(const szo_linear* p, const void* x, int64_t M, const float* S, void* y,
                       int y_dtype, cudaStream_t st);

// tensor-core path (gemm_tc.cu)
szo_status tc_plan_create(szo_linear* p, cudaStream_t st);
void tc_plan_destroy(szo_linear* p);
szo_status linear_fwd_tc(const szo_linear* p, const void* x, int64_t M, const float* S, void* y,
                         int y_dtype, bool sparse_add, cudaStream_t st);

}  // namespace szo
