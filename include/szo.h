/* szo.h - C ABI of the sensitive-sparse zeroth-order (ZO) fine-tuning step for sm_100a.
 *
 * The library implements the hot path of "Zeroth-Order Fine-Tuning of LLMs with Extreme
 * Sparsity": the SPSA / ZO-SGD step restricted to k "sensitive" parameters, on linear layers
 * whose weight is a frozen 4-bit quantized dense part plus k fp32 sparse values.
 *
 * Conventions (all entry points)
 *   pointers   Device pointers unless the name ends in _host.  The caller owns every buffer it
 *              passes; the library allocates inside *_create (freed by *_destroy) and, once per
 *              device, a 4-byte status word on the first call that may report a device-side problem.
 *              Buffers must be 16-byte aligned (SZO_ERR_ALIGNMENT otherwise).
 *   stream     `void* stream` is a cudaStream_t (NULL = default stream).  Calls enqueue work and
 *              return; none synchronises unless its comment says so.
 *   errors     Arguments are validated on the host before any launch.  Return value 0 = SZO_OK,
 *              negative = error; szo_last_error() gives a thread-local detail string.  Kernels
 *              never trap: a bounded wait that expires inside a kernel is recorded in a device
 *              status word readable with szo_device_status().
 *   layouts    Matrices are row-major.  A linear has weight W[N,K] (out, in), input x[M,K],
 *              output y[M,N].  int4 codes: uint8 [N,K/2], two codes per byte, even column in the
 *              low nibble.  scales/zeros: 16-bit floats [N,K/G], G = group size along K.
 *   determinism Same inputs give bitwise-same outputs (no floating-point atomics).
 */
#ifndef SZO_H_
#define SZO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t szo_status;
enum {
  SZO_OK = 0,
  SZO_ERR_INVALID_ARG = -1,
  SZO_ERR_SHAPE = -2,
  SZO_ERR_ALIGNMENT = -3,
  SZO_ERR_UNSUPPORTED = -4,
  SZO_ERR_WORKSPACE = -5,
  SZO_ERR_CUDA = -6,
  SZO_ERR_NONFINITE = -7,
  SZO_ERR_TIMEOUT = -8
};

typedef enum { SZO_F32 = 0, SZO_BF16 = 1, SZO_F16 = 2 } szo_dtype;

/* How szo_linear_fwd evaluates y = x Dequantize(Q)^T + x S^T (the paper's appendix
 * "Implementation of Sparse Operations in Linear Layers" gives the two orders). */
typedef enum {
  SZO_MODE_AUTO = 0,          /* SPARSE_ADD, except for an int4 plan with M <= 16 tokens and K % 128 == 0:
                                 there the layer is bound by reading the codes once, and a
                                 weight-streaming kernel evaluates SparseAddMM(Dequantize(Q) x, S, x)
                                 with the sparse term in fp32 (the order the appendix finds faster
                                 for few tokens); it needs no workspace */
  SZO_MODE_SPARSE_ADD = 1,    /* DenseMM(SparseAdd(S, Dequantize(Q)), x): S is added to the
                                 dequantised bf16 tile in shared memory before the tensor-core MMA */
  SZO_MODE_SPMM = 2,          /* SparseAddMM(Dequantize(Q) x, S, x): tensor-core GEMM on the dense
                                 part, then a row-bucketed CSR SpMM with fp32 values */
  SZO_MODE_FP32_VALIDATE = 3, /* fp32 CUDA-core evaluation of the same expression (exact fp32
                                 sparse term); slow, for checking losses and projected gradients */
  SZO_MODE_PAIRED = 4         /* szo_model_config.linear_mode only: the two forwards of a ZO step run as
                                 ONE pass that carries the centre (x+ + x-)/2 and the half-difference
                                 (x+ - x-)/2 of every activation (see szo_linear_fwd_paired); lone
                                 forwards (szo_model_loss) run as SZO_MODE_SPARSE_ADD */
} szo_linear_mode;

const char* szo_status_string(szo_status s);   /* static storage */
const char* szo_last_error(void);              /* thread-local; valid until the next call */
int szo_version(void);

/* Reads and clears the device status word (0 = no kernel reported a problem, else a negative
 * szo_status).  Synchronises the device.  After a non-zero status every plan clears the tickets of
 * its K-split tiles before its next launch (a kernel that gave up may have left them set). */
szo_status szo_device_status(int32_t* status_host);

/* Self-test of the bounded waits inside the kernels (no counterpart in the paper): launches one tiny
 * kernel whose only wait, limited to limit_ms milliseconds of SM clock, is on a barrier that nothing
 * ever signals.  The wait must give up: *gave_up_host = 1, the kernel returns, and the next
 * szo_device_status reports SZO_ERR_TIMEOUT.  Synchronises the stream. */
szo_status szo_selftest_wait_timeout(double limit_ms, int32_t* gave_up_host, void* stream);

/* ---- Quantizer Q for w_dense (Section 3.5, "Integration with quantization": the dense part is
 * stored in 4 bits; the paper leaves the choice of quantizer open).  Uniform asymmetric,
 * group-wise: for each row and each group of G consecutive columns, scale =
 * round16((max-min)/15), zero = round16(min), code = clamp(rint((w-zero)/scale), 0, 15) (0 when
 * scale == 0), IEEE fp32, ties to even.
 *   W        w_dtype [N,K] (SZO_F32 or SZO_BF16)      codes   uint8 [N,K/2]
 *   scales, zeros  sz_dtype [N,K/G] (SZO_BF16 or SZO_F16)
 * Requires K % G == 0, G % 2 == 0.  Non-finite weights are not detected. */
szo_status szo_quantize(const void* W, szo_dtype w_dtype, int64_t N, int64_t K, int32_t G,
                        szo_dtype sz_dtype, uint8_t* codes, void* scales, void* zeros, void* stream);

/* ---- Sensitive parameter mask (Definition 3: the mask with k nonzeros that maximises
 * ||m (.) grad f||^2, i.e. the k largest squared-gradient scores).  Ties go to the lowest index;
 * idx_out[k] is ascending.  Two-phase: call with workspace == NULL to obtain *workspace_bytes,
 * then again with a workspace of at least that size.  Cold path: the second call synchronises the
 * stream and returns SZO_ERR_NONFINITE if any score is NaN (idx_out is then unspecified).
 *   scores  fp32 [n]      idx_out  int64 [k]      0 <= k <= n */
szo_status szo_select_mask(const float* scores, int64_t n, int64_t k, int64_t* idx_out,
                           void* workspace, size_t* workspace_bytes, void* stream);

/* ---- Sensitive parameter mask without any allocation.  The paper has no counterpart: this is a
 * packaging variant of szo_select_mask for callers that cannot obtain device memory themselves,
 * for example a plug-in running inside a host application that owns the allocator and hands out only
 * the input and output buffers, or a process whose memory budget is fixed before it starts.  The
 * scratch that szo_select_mask takes as a workspace lives here in a fixed array inside the library
 * (196 864 bytes = 192.25 KiB of device memory on every GPU that loads the library, until the process
 * exits), so the call performs no cudaMalloc/cudaFree and needs no workspace query.
 *   limit     n <= 67 108 864 (2^26) scores; larger n returns SZO_ERR_WORKSPACE and touches nothing.
 *   set-up    the first call on each device looks up the array's device address (the device must be
 *             current, as for every call) and keeps it for the life of the process; it belongs to the
 *             device's primary context, so a cudaDeviceReset in the same process invalidates it.
 *   capture   like szo_select_mask the call ends in a stream synchronisation (it reads the NaN flag
 *             back), so it cannot be issued on a stream that is being captured.
 *   sharing   every call on a device uses the same array and finds the previous call's contents in
 *             it; the function clears what it needs.  Two calls that overlap on the GPU (different
 *             streams or threads) race on it: serialise them.
 * Results, tie rule, NaN handling and the final stream synchronisation are those of
 * szo_select_mask. */
szo_status szo_select_mask_static(const float* scores, int64_t n, int64_t k, int64_t* idx_out,
                                  void* stream);

/* ---- Sparse perturbation (Definition 4, zbar = z (.) m_k; Section 3.4 update rule on w_sparse;
 * Section 2.1 seed trick: z is regenerated, never stored).
 *   S_out[j] = fma(scale, z_j, S_in[j]),  z_j = Gaussian(Philox4x32-10(key = seed,
 *   counter = (idx_base + idx[j], step))): Box-Muller on the top 24 bits of words 0 and 1.
 * idx[k] int64, tensor-local flat indices; idx_base makes them global over all linear
 * parameters.  S_out may alias S_in.  Entries outside idx are never touched. */
szo_status szo_perturb(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                       int64_t idx_base, uint64_t seed, uint64_t step, float scale, void* stream);

/* ---- The same passes with z kept in device memory.  Section 2.1's seed trick regenerates z so that
 * no copy of a model-sized vector is held; with the Definition 4 mask only k values are needed
 * (26 MB at the 7B shape), so the first pass of a step can keep them and the -2 eps pass, the
 * restore and the update become plain 12-byte-per-entry streams with bit-identical results.
 *   szo_perturb_keep_z : szo_perturb, and z_out[j] = z_j (fp32[k], 16-byte aligned, caller-owned)
 *   szo_perturb_kept_z : S_out[j] = fma(scale, z[j], S_in[j])
 *   szo_update_kept_z  : szo_update with z read from z[] */
szo_status szo_perturb_keep_z(const float* S_in, float* S_out, const int64_t* idx, int64_t k,
                              int64_t idx_base, uint64_t seed, uint64_t step, float scale, float* z_out,
                              void* stream);
szo_status szo_perturb_kept_z(const float* S_in, float* S_out, const float* z, int64_t k, float scale,
                              void* stream);
/* The +eps, -2 eps, +eps passes of the seed trick for one (seed, step) in ONE launch (a step that evaluates both
 * losses from copies of S, or inside the linears, makes the three passes back to back; the pass is bound by
 * drawing z, so the other two cost their two fused multiply-adds):
 *   sp = fma(eps, z_j, S_in[j]), sm = fma(-2 eps, z_j, sp), S_out[j] = fma(eps, z_j, sm), z_out[j] = z_j,
 *   and S_plus[j] = sp, S_minus[j] = sm where those pointers are not NULL (fp32[k], 16-byte aligned).
 * The same bits as szo_perturb_keep_z(eps), szo_perturb_kept_z(-2 eps), szo_perturb_kept_z(eps) in turn. */
szo_status szo_perturb3_keep_z(const float* S_in, float* S_out, const int64_t* idx, int64_t k, int64_t idx_base,
                               uint64_t seed, uint64_t step, float eps, float* z_out, float* S_plus, float* S_minus,
                               void* stream);
szo_status szo_update_kept_z(float* S, const float* z, int64_t k, float lr, const double* f_plus_dev,
                             const double* f_minus_dev, float eps, void* stream);

/* ---- Projected gradient (Definition 1, SPSA): *g_dev = (*f_plus_dev - *f_minus_dev) / (2 eps),
 * fp64, all on the device. */
szo_status szo_projected_gradient(const double* f_plus_dev, const double* f_minus_dev, float eps,
                                  double* g_dev, void* stream);

/* ---- ZO-SGD update (Definition 2 with Definition 4): S[j] = fma(-(float)(lr*g), z_j, S[j]) with
 * g as above and the same z as szo_perturb for (seed, step).  The losses are read on the device. */
szo_status szo_update(float* S, const int64_t* idx, int64_t k, int64_t idx_base, uint64_t seed,
                      uint64_t step, float lr, const double* f_plus_dev, const double* f_minus_dev,
                      float eps, void* stream);

/* ---- Sparse values stored in 16 bits (Section 3.5: w_sparse is kept in 16 bits).  The paper does not say
 * where a step's arithmetic happens for such storage; this library widens the stored values to fp32
 * (exact), runs the step in fp32 (perturbations are never rounded to 16 bits) and rounds the updated
 * values to the storage format once, to nearest even.
 * szo_round_sparse16: S[j] = widen(RN_dt(S[j])) in place for j in [0, k), and S16_out[j] = RN_dt(S[j]) when
 * S16_out != NULL (device, k 16-bit values, caller-owned).  dt: SZO_BF16 or SZO_F16.  Call it after
 * szo_update to keep S representable in the storage format; values beyond the format's range become
 * infinities as IEEE rounding says.  Errors: NULL S with k > 0, dt == SZO_F32 -> SZO_ERR_INVALID_ARG. */
szo_status szo_round_sparse16(float* S, int64_t k, szo_dtype dt, void* S16_out, void* stream);

/* ---- Replay of a run from its log (Section 2.1, the seed trick: z_t is a function of (seed, step_t), so
 * the scalars g_t are a complete record of what a run did to the sparse values:
 * S_T = S_0 - sum_t lr g_t z_t; a checkpoint is S at some step plus the (step, g) pairs since).
 * For every logged step, in order: when eps != 0, the +eps, -2 eps, +eps passes of the in-place order
 * (so that S takes exactly the roundings of the original step; eps == 0 skips them), then
 * S[j] = fma(-(float)(lr * g_t), z_j, S[j]).  steps_host, g_host: HOST arrays of n entries.
 * Reproduces the S of szo_model_zo_step / szo_update runs bit for bit. */
szo_status szo_replay(float* S, const int64_t* idx, int64_t k, int64_t idx_base, uint64_t seed,
                      const uint64_t* steps_host, const double* g_host, int64_t n, float eps, float lr, void* stream);

/* ---- Decomposed linear layer (Section 3.4: w = w_sparse + w_dense; appendix on sparse
 * operations: y = x Dequantize(Q(w_dense))^T + x w_sparse^T).
 * A plan owns only derived, immutable data (kernel-layout scale/zero table, tile buckets and
 * row pointers of idx, tensor maps); the caller's codes, scales, zeros, idx and bias must
 * outlive it.  G == 0 means a dense bf16 weight [N,K] instead of codes (scales/zeros NULL).
 * Requires K % 64 == 0 and, for G > 0, G == 32 or G % 64 == 0.  idx[nnz] ascending flat indices n*K + c.
 * bias fp32 [N] or NULL.  szo_linear_create synchronises the stream. */
typedef struct szo_linear szo_linear_t;
szo_status szo_linear_create(szo_linear_t** out, int64_t N, int64_t K, int32_t G,
                             const void* codes_or_bf16_W, const void* scales, const void* zeros,
                             szo_dtype sz_dtype, const int64_t* idx, int64_t nnz, const float* bias,
                             void* stream);
/* Non-uniform 4-bit format (Section 4 and the hyperparameter appendix: the 4-bit experiments use
 * SqueezeLLM, whose codes index a table of 16 values per output channel instead of a scale and a
 * zero): Dequantize(Q(w_dense))[n,c] = lut[n][q[n,c]].  codes uint8 [N,K/2] as for szo_quantize
 * (low nibble = even column); lut lut_dtype (SZO_F16 or SZO_BF16) [N,16], caller-owned like the
 * codes; everything else as szo_linear_create.  How the table and the codes are fitted is the
 * quantizer's business (the paper takes any post-training quantizer) and not part of this library.
 * Such a plan runs in SZO_MODE_AUTO / SZO_MODE_SPARSE_ADD (for every M the effective bf16 weight
 * RN_bf16(lut[n][q]) , RN_bf16(. + S) at the masked positions, is written to the workspace and then
 * multiplied) and in SZO_MODE_FP32_VALIDATE; SZO_MODE_SPMM returns SZO_ERR_UNSUPPORTED. */
szo_status szo_linear_create_lut(szo_linear_t** out, int64_t N, int64_t K, const uint8_t* codes,
                                 const void* lut, szo_dtype lut_dtype, const int64_t* idx, int64_t nnz,
                                 const float* bias, void* stream);
/* x: x_dtype [M,K] (SZO_BF16; SZO_F32 also accepted in SZO_MODE_FP32_VALIDATE);
 * S_pert: fp32 [nnz] current (already perturbed) sparse values; y: y_dtype [M,N] (SZO_BF16 or
 * SZO_F32).  workspace: at least szo_linear_workspace_bytes(plan, M, mode) bytes (may be NULL
 * when that is 0), device memory, contents irrelevant on entry and undefined on return.  In the
 * tensor-core modes it holds the bucket-ordered sparse records and the fp32 scratch of tiles that
 * are split along K; for an int4 plan and M >= 4096 tokens it holds instead the effective bf16
 * weight Dequantize(Q) + w_sparse of this layer (2 N K bytes, rows padded to 256), which is written
 * first and then multiplied: the appendix's DenseMM(SparseAdd(w_sparse, Dequantize(Q)), x) literally.
 * Both forms give the same bits.  A plan must not run on two streams at once (its K-split
 * tickets are shared). */
szo_status szo_linear_fwd(const szo_linear_t* plan, const void* x, szo_dtype x_dtype, int64_t M,
                          const float* S_pert, void* y, szo_dtype y_dtype, int32_t mode,
                          void* workspace, size_t workspace_bytes, void* stream);
size_t szo_linear_workspace_bytes(const szo_linear_t* plan, int64_t M, int32_t mode);

/* ---- The same layer for BOTH forwards of a ZO step at once, in the paired form.  Definition 1 (SPSA)
 * needs the loss at w + eps zbar and at w - eps zbar on the same batch; only the difference of the
 * two enters the projected gradient.  The perturbation moves an activation by less than one bf16 ulp,
 * so two forwards whose activations are each rounded to bf16 lose that difference in rounding.  Here
 * the pair (x+, x-) travels as centre xc = (x+ + x-)/2 and half-difference xd = (x+ - x-)/2, each
 * in bf16 with its own exponent.  With W = RN_bf16(Dequantize(Q(w_dense)) + S) (Section 3.4's
 * decomposition, S unperturbed; the appendix's SparseAdd order) and Zbar = z at the sensitive
 * entries (Definition 4):
 *     yc = xc W^T (+ bias)            yd = xd W^T + eps * xc Zbar^T
 * which are centre and half-difference of x+ (W + eps Zbar)^T and x- (W - eps Zbar)^T except for the
 * term eps * xd Zbar^T in yc, of relative order eps^2 and left out.  The dense products run on the
 * tensor cores; eps * xc Zbar^T is accumulated in fp32 onto the fp32 accumulator before the one
 * rounding of the store (the appendix's SparseAddMM order, for the perturbation only).
 *   x   bf16 [M0 + M, K]: rows [0, M) = xc, rows [M0, M0 + M) = xd, M0 = M rounded up to a multiple of
 *       256 (rows in between are ignored)            y   y_dtype [M0 + M, N], same row layout
 *   S   fp32 [nnz] current sparse values             z   fp32 [nnz] z of this step at the entries of idx
 *   workspace  szo_linear_paired_workspace_bytes(plan, M) bytes (effective weight, K-split scratch)
 * Every plan format is accepted (int4 groups, per-row tables, dense bf16). */
size_t szo_linear_paired_workspace_bytes(const szo_linear_t* plan, int64_t M);
szo_status szo_linear_fwd_paired(const szo_linear_t* plan, const void* x, int64_t M, const float* S, const float* z,
                                 float eps, void* y, szo_dtype y_dtype, void* workspace, size_t workspace_bytes,
                                 void* stream);
void szo_linear_destroy(szo_linear_t* plan);

/* ---- Whole loss path and ZO step on one GPU (Definition 1 evaluates the loss twice per step;
 * Section 4 names the decoder families).  arch 0: RMSNorm, rotary positions, SiLU-gated MLP
 * (Llama/Mistral; grouped-query attention when n_kv_heads < n_heads); arch 1: LayerNorm, learned
 * positions, biases, ReLU MLP (OPT).  Linear order within a layer: arch 0: q,k,v,o,gate,up,down;
 * arch 1: q,k,v,o,fc1,fc2.  The flat parameter index that keys z runs over the linears in model
 * order, row-major inside each. */
typedef struct {
  int32_t arch;
  int32_t n_layers, d_model, n_heads, n_kv_heads, d_ff, vocab, max_pos;
  float norm_eps, rope_base;
  int32_t group;       /* int4 group size; 0 = dense bf16 linears; -1 = non-uniform 4-bit format
                          (szo_linear_create_lut) */
  int32_t sz_dtype;    /* szo_dtype of scales/zeros (of the tables when group == -1) */
  int32_t act_dtype;   /* SZO_BF16 (tensor-core path) or SZO_F32 (validation path) */
  int32_t linear_mode; /* szo_linear_mode used by every linear */
  int32_t loss_kind;   /* 0: mean next-token cross-entropy over B*(S-1) positions;
                          1: 2-way cross-entropy over two candidate ids at the last position */
  int32_t max_batch, max_seq;
} szo_model_config;

typedef struct {
  const void* codes;     /* uint8 [N,K/2], or bf16 [N,K] when group == 0 */
  const void* scales;    /* sz_dtype [N,K/G] or NULL; when group == -1 the table [N,16] */
  const void* zeros;
  const int64_t* idx;    /* [nnz] ascending tensor-local flat indices */
  int64_t nnz;
  const float* bias;     /* fp32 [N] or NULL */
} szo_linear_weights;

typedef struct {
  const float* attn_norm_g; const float* attn_norm_b;   /* fp32 [d]; *_b NULL for arch 0 */
  const float* mlp_norm_g;  const float* mlp_norm_b;
  szo_linear_weights lin[7];
} szo_layer_weights;

typedef struct {
  const void* embed;     /* bf16 [vocab, d] */
  const void* pos;       /* bf16 [max_pos, d] (arch 1) or NULL */
  const void* lm_head;   /* bf16 [vocab, d] */
  const float* final_norm_g; const float* final_norm_b;
} szo_model_weights;

/* Causal softmax attention, one block of the loss f that Definition 1 evaluates (scale 1/sqrt(head_dim),
 * grouped-query attention when n_kv_heads < n_heads).  q, o: dtype [B*S, n_heads*head_dim]; k, v: dtype
 * [B*S, n_kv_heads*head_dim]; token b*S+s is position s of sequence b.  dtype SZO_BF16 (tensor-core
 * flash kernel) or SZO_F32; head_dim 64 or 128. */
szo_status szo_attention(const void* q, const void* k, const void* v, void* o, szo_dtype dtype, int32_t B, int32_t S,
                         int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream);

/* The same attention in the paired form of szo_linear_fwd_paired: every buffer holds the B*S centre rows
 * first and the half-difference rows from row `row0` (>= B*S) on; the outputs are the exact centre and
 * half-difference of attention(q+, k+, v+) and attention(q-, k-, v-) (nothing of higher order is left
 * out), bf16 only. */
szo_status szo_attention_paired(const void* q, const void* k, const void* v, void* o, int64_t row0, int32_t B,
                                int32_t S, int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, void* stream);

typedef struct szo_model szo_model_t;
/* layers_host: host array of n_layers entries holding device pointers.  S_all: fp32 [k_total],
 * the trainable sparse values of all linears concatenated in model order (the only mutable
 * state; caller-owned, updated in place by szo_model_zo_step).  Synchronises the stream.
 * The weights are frozen by the method (Section 3.4: only w_sparse is trained) and must not change
 * after this call: with dense bf16 linears (group == 0) the model keeps its own copy of them
 * (2 bytes per weight more device memory), in which it rewrites the masked entries per forward. */
szo_status szo_model_create(szo_model_t** out, const szo_model_config* cfg,
                            const szo_model_weights* top, const szo_layer_weights* layers_host,
                            float* S_all, void* stream);
int64_t szo_model_k_total(const szo_model_t* m);
/* Global flat indices int64 [k_total] of the sparse entries (device pointer owned by the model). */
const int64_t* szo_model_gidx(const szo_model_t* m);
/* tokens int32 [B,S]; labels int32 [B] in {0,1} and cand int32 [2] for loss_kind 1 (else NULL);
 * S_vals fp32 [k_total] values to evaluate at (NULL = the model's S_all); *loss_dev fp64. */
szo_status szo_model_loss(szo_model_t* m, const int32_t* tokens, const int32_t* labels,
                          const int32_t* cand, int32_t B, int32_t S, const float* S_vals,
                          double* loss_dev, void* stream);
/* One step in the seed trick's in-place order: S += eps z; f+; S -= 2 eps z; f-; S += eps z;
 * g = (f+ - f-)/(2 eps); S -= lr g z.  Outputs are device scalars (fp64); no host read-back.
 * With linear_mode SZO_MODE_PAIRED, S goes through the same three passes first and both losses are then
 * evaluated in one pass in the paired form (z kept in device memory, +- eps z applied inside the linears
 * in fp32): f+ and f- are the same two function values, with their difference resolved far below the
 * bf16 rounding of the activations. */
szo_status szo_model_zo_step(szo_model_t* m, const int32_t* tokens, const int32_t* labels,
                             const int32_t* cand, int32_t B, int32_t S, uint64_t seed,
                             uint64_t step, float eps, float lr, double* f_plus_dev,
                             double* f_minus_dev, double* g_dev, void* stream);
/* n-sample SPSA (Definition 1 averaged over n independent perturbations; the paper's runs use n = 1, for
 * which this is szo_model_zo_step): for i = 0 .. n-1, z_i is drawn for the counter step * n + i and both
 * losses are evaluated around the same S; then S -= (lr / n) g_i z_i for i = 0 .. n-1 in turn.
 * f_plus_dev, f_minus_dev, g_dev: fp64 device arrays of n entries. */
szo_status szo_model_zo_step_n(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                               int32_t B, int32_t S, uint64_t seed, uint64_t step, int32_t n, float eps, float lr,
                               double* f_plus_dev, double* f_minus_dev, double* g_dev, void* stream);
/* The step in two halves, for data-parallel replicas (Definition 1 evaluates f on a batch: replicas that
 * hold the same weights, mask and S and use the same (seed, step) draw the same z, evaluate f+ and f-
 * on their own share of the batch and need to exchange only sums of losses before each applies the
 * identical update of Definition 2).
 *   szo_model_zo_losses: draws and keeps z, evaluates both losses on this replica's B sequences, leaves S
 *     where the +eps, -2 eps, +eps sequence leaves it, and writes sums_dev[3] (fp64, device) =
 *     (sum of the per-position losses of f+, the same for f-, number of positions).
 *   szo_model_zo_apply: takes sums_dev[3] ADDED UP OVER ALL REPLICAS (the caller's all-reduce: 24 bytes;
 *     with one replica, its own sums), forms f+- = sum / count, g = (f+ - f-)/(2 eps) and
 *     S -= lr g z with the kept z.  It must follow a szo_model_zo_losses on the same model.
 * szo_model_zo_step is the first followed by the second on one replica. */
szo_status szo_model_zo_losses(szo_model_t* m, const int32_t* tokens, const int32_t* labels, const int32_t* cand,
                               int32_t B, int32_t S, uint64_t seed, uint64_t step, float eps, double* sums_dev,
                               void* stream);
szo_status szo_model_zo_apply(szo_model_t* m, float eps, float lr, const double* sums_dev, double* f_plus_dev,
                              double* f_minus_dev, double* g_dev, void* stream);
/* Storage format of the model's sparse values (see szo_round_sparse16): with dt = SZO_BF16 or SZO_F16 every
 * update of szo_model_zo_step, szo_model_zo_step_n, szo_model_zo_apply and szo_model_zo_step_host is followed
 * by one rounding of S to that format (S stays an fp32 array holding representable values; S16_out, when not
 * NULL, is a caller-owned device array of k_total 16-bit values that receives the stored form after every
 * update).  The call itself rounds the current S once.  dt = SZO_F32 (the default) switches it off. */
szo_status szo_model_set_sparse_storage(szo_model_t* m, szo_dtype dt, void* S16_out, void* stream);
/* Same step through HOST buffers: copies tokens (and labels, cand) to the device, runs the step
 * and copies (f+, f-, g) back into out3_host[3]; synchronises the stream. */
szo_status szo_model_zo_step_host(szo_model_t* m, const int32_t* tokens_host,
                                  const int32_t* labels_host, const int32_t* cand_host, int32_t B,
                                  int32_t S, uint64_t seed, uint64_t step, float eps, float lr,
                                  double* out3_host, void* stream);
/* ---- Token generation with a KV cache (the regime of the paper's inference measurements: the speed
 * figure of Section 1, 128 generated tokens; the appendix on sparse operations finds the SparseAddMM
 * order the faster one there).
 *   szo_model_enable_decode: allocates the cache, act_dtype [n_layers][max_batch][max_seq][n_kv_heads *
 *     head_dim] for keys and for values (and an LM-head plan when the model's loss does not use one); once.
 *   szo_model_decode_step: T new tokens per sequence (tokens int32 [B, T]) that follow the pos0 positions
 *     already cached: their keys and values are appended at positions pos0 .. pos0 + T - 1, every new
 *     position attends to the cached ones and to the new ones up to itself, and logits_dev receives the
 *     fp32 logits [B, vocab] of the LAST new token.  A prompt is one call with pos0 = 0; generation is
 *     one call per token with T = 1.  The caller keeps pos0 (the cache is not cleared: positions at or
 *     beyond pos0 + T are simply not read).  Linears run in SZO_MODE_AUTO (the weight-streaming kernel
 *     with the sparse term in fp32 for at most 16 rows), or in the validation mode for an fp32 model.
 *     S_vals: fp32 [k_total] or NULL for the model's S.  On a stream other than the default one the
 *     several hundred launches of a step are captured once per (B, T, S_vals) into a CUDA graph and
 *     replayed (SZO_DECODE_GRAPH=0 at szo_model_enable_decode keeps the launch-by-launch form); the
 *     call itself must not be issued inside a capture of the caller's. */
szo_status szo_model_enable_decode(szo_model_t* m, void* stream);
szo_status szo_model_decode_step(szo_model_t* m, const int32_t* tokens, int32_t B, int32_t T, int32_t pos0,
                                 const float* S_vals, float* logits_dev, void* stream);
/* Number of kernel launches the last szo_model_zo_step on this model enqueued. */
int64_t szo_model_last_launches(const szo_model_t* m);
/* Measurement aid (no counterpart in the paper): when enabled, the model brackets every
 * decoder-block linear launch with CUDA events on the launching stream.  szo_model_linear_time
 * synchronises the device, returns the summed elapsed milliseconds and the number of launches
 * since the last call (or since enabling), and resets the counters. */
szo_status szo_model_enable_timing(szo_model_t* m, int32_t on);
szo_status szo_model_linear_time(szo_model_t* m, double* ms_total_host, int64_t* launches_host);
void szo_model_destroy(szo_model_t* m);

#ifdef __cplusplus
}
#endif
#endif /* SZO_H_ */
