// Internal launch interfaces shared by the translation units of the library.
#pragma once

#include "common.cuh"

namespace sgcn {

// ---- SpMM -------------------------------------------------------------------------------------
// Optional fused epilogue of the aggregation (used by transform-first layers):
//   y = dinv_i * acc + bias[col];  if relu: mask = (y > 0), y = max(y, 0);  if accumulate: y += Y_old
struct SpmmEpilogue {
    const float* bias = nullptr;
    int relu = 0;
    uint8_t* mask = nullptr;
    int64_t mask_ld = 0;
    int accumulate = 0;
};
int64_t spmm_partial_bytes(const slicegcn_graph* g, int width);
slicegcn_status_t spmm_run(const slicegcn_graph* g, bool transpose, int in_dtype, int out_dtype, const void* X,
                           int64_t ldx, void* Y, int64_t ldy, int width, const SpmmEpilogue* epi, void* ws,
                           int64_t ws_bytes, cudaStream_t st, bool instrument = true);

// ---- grouped row-panel GEMM  C_g = epilogue(A_g * B_g) ----------------------------------------
// Group g (one slice) reads K columns of A starting at a_start[g], multiplies by its own K x N
// block of B and writes N columns of C starting at c_start[g].  Epilogue, in this order:
//   x = acc + bias[g][n];  if relu: (mask_out = x > 0), x = max(x, 0);  x += post1[g][n] + post2[g][n];
//   if mul_pos: x *= (P[r, c] > 0);  if accumulate: x += C_old;  C = x
constexpr int kGateBytes = 2;   // GemmArgs::mul_pos_dtype: one byte per element (a ReLU mask)

struct GemmArgs {
    int64_t M = 0;
    int groups = 1, K = 0, N = 0;
    const void* A = nullptr;
    int64_t lda = 0;
    int a_dtype = SLICEGCN_F32;
    int a_start[SLICEGCN_MAX_SLICES] = {0};
    int a_pad_zero = 0;                // columns a_start+K .. next multiple of 8 exist (< lda) and hold zeros
    const uint8_t* a_mask = nullptr;   // A element (r, col) is multiplied by a_mask[r*a_mask_ld + col]
    int64_t a_mask_ld = 0;
    const float* B = nullptr;          // group g: B + g*b_gstride; element (k, n) at k*ldb + n, or n*ldb + k if b_trans
    int64_t b_gstride = 0;
    int ldb = 0;
    int b_trans = 0;
    // K index stacked over several weight blocks (groups == 1 only): k = q*b_kstack + j reads element j of block q at
    // B + q*b_gstride -- the sum over slices of dM_i W_i^T as ONE product over the concatenated dM (0: plain B)
    int b_kstack = 0;
    void* C = nullptr;
    int64_t ldc = 0;
    int c_dtype = SLICEGCN_F32;
    int reverse = 0;                   // visit the row tiles from the last one down (L2 reuse across consecutive kernels)
    int c_start[SLICEGCN_MAX_SLICES] = {0};
    const float* bias = nullptr;       // [groups][N] (stride N), added before the activation
    const float* post1 = nullptr;      // [groups][N], added after the activation
    const float* post2 = nullptr;
    int relu = 0;
    uint8_t* mask_out = nullptr;       // mask_out[r*mask_ld + c] = pre-activation > 0 (c = column of C)
    int64_t mask_ld = 0;
    const void* mul_pos = nullptr;     // tensor P indexed like C (own dtype / leading dimension): x *= (P > 0);
                                       // mul_pos_dtype kGateBytes: P is a byte mask (non-zero lets x pass)
    int64_t mul_pos_ld = 0;
    int mul_pos_dtype = SLICEGCN_F32;
    int accumulate = 0;
    // N is not a multiple of 4 but C has room up to the next one and those padding columns may be written (with zeros:
    // the weight image has none there); only without bias / post / ReLU.  Lets the aligned kernels take odd widths.
    int c_pad_write = 0;
    // tensor-core path: device status word (set when a bounded wait runs out) and scratch for the
    // prepared weight image (tc_image_bytes()); without both the CUDA-core kernel runs
    int* fault = nullptr;
    void* b_image = nullptr;
    int64_t b_image_bytes = 0;
    // optional second product added after the activation:  C = epilogue(A B) + A2 B2  (the self term of
    // Eq. 6 next to the aggregation term).  Same dtype, group count, N and b_trans as the first product.
    // Only the warp-specialised tensor-core kernel takes it; gemm_run() reports UNSUPPORTED otherwise.
    const void* A2 = nullptr;
    int64_t lda2 = 0;
    int a2_start[SLICEGCN_MAX_SLICES] = {0};
    int a2_pad_zero = 0;
    const float* B2 = nullptr;
    int64_t b2_gstride = 0;
    int K2 = 0;
};
slicegcn_status_t gemm_run(const GemmArgs& a, cudaStream_t st);
slicegcn_status_t tc_gemm_run(const GemmArgs& a, cudaStream_t st);
int64_t tc_image_bytes(int groups, int K, int N);
// Weight images kept across the GEMMs and epochs of a training run (see tc.cu).  Between begin and end the
// tensor-core GEMMs of the calling thread take their images from the cache region; begin converts every image
// recorded by earlier epochs in one launch.
struct TcImageCache;
TcImageCache* tc_image_cache_create();
void tc_image_cache_destroy(TcImageCache* c);
slicegcn_status_t tc_image_cache_begin(TcImageCache* c, void* region, int64_t bytes, const float* params, int64_t param_elems,
                                       cudaStream_t st);
void tc_image_cache_end();
// true when the tensor-core kernel that takes this product applies a.a_mask in its producer at no extra pass
// (otherwise multiplying the operand once up front is cheaper than the masked fallback kernels)
bool tc_gemm_masks_in_producer(const GemmArgs& a);

// ---- grouped weight gradient  dW_g = A_g^T * B_g  (reduction over all rows) -------------------
// A_g: K columns of A from a_start[g]; B_g: N columns of the fp32 matrix B from b_start[g], each
// element optionally multiplied by b_mask (same column indexing as B).  dW [groups][K][N] and,
// if dbias != NULL, dbias[groups][N] = column sums of (masked) B_g.  K may be 0 (bias only).
// Two-stage deterministic reduction through `scratch`.
struct WgradArgs {
    int64_t M = 0;
    int groups = 1, K = 0, N = 0;
    const void* A = nullptr;
    int64_t lda = 0;
    int a_dtype = SLICEGCN_F32;
    int a_start[SLICEGCN_MAX_SLICES] = {0};
    const float* B = nullptr;
    int64_t ldb = 0;
    int b_start[SLICEGCN_MAX_SLICES] = {0};
    const uint8_t* b_mask = nullptr;
    int64_t b_mask_ld = 0;
    int a_pad_zero = 0;        // A / B columns up to the next multiple of 4 past the last group exist and hold zeros
    int b_pad_zero = 0;
    float* dW = nullptr;       // may be NULL when K == 0
    int64_t ldw = 0;           // leading dimension of a group's K x N block of dW (0: N, dense)
    float* dbias = nullptr;    // may be NULL
    float* dbias2 = nullptr;   // optional second copy of the column sums (slice-encoding gradient)
    int* fault = nullptr;      // device status word; NULL: CUDA-core path
};
int64_t wgrad_scratch_bytes(int64_t M, int groups, int K, int N);
int64_t tc_wgrad_scratch_bytes(const WgradArgs& a);
bool tc_wgrad_masks_in_producer(const WgradArgs& a);   // the same question for a.b_mask, one launch
bool wgrad_masks_in_producer(const WgradArgs& a);      // ... for wgrad_run, which may cut dW into column blocks
// bias_done (optional): set when the column sums (dbias / dbias2) were produced as well
slicegcn_status_t tc_wgrad_run(const WgradArgs& a, void* scratch, int64_t scratch_bytes, cudaStream_t st, bool* bias_done = nullptr);
slicegcn_status_t wgrad_run(const WgradArgs& a, void* scratch, int64_t scratch_bytes, cudaStream_t st);

// ---- small kernels ----------------------------------------------------------------------------
// Slices of X (p column ranges of width w at starts[]) copied side by side at multiples of w_pad, padding zeroed
slicegcn_status_t repack_slices_run(int64_t n, int p, const int* starts, int w, int w_pad, const void* X, int64_t x_ld, int dtype,
                                    void* out, int64_t out_ld, cudaStream_t st);
// Parameter (or gradient) tensors copied between the caller's layout and the padded internal one: tensor e is
// `blocks` blocks of r x c floats at element offset `outer` of the caller's buffer and of rp x cp (rp >= r, cp >= c) at
// offset `inner` of the internal buffer.  pad: caller -> internal, padding written as zeros; else internal -> caller.
struct PadEntry {
    int64_t outer, inner;
    int blocks, r, c, rp, cp;
};
struct PadTable {
    int count = 0;
    PadEntry e[48];
};
slicegcn_status_t pad_params_run(const PadTable& t, bool pad, const float* src, float* dst, cudaStream_t st);
// Dropout in place: data[r, c] = mask[r, mc] ? data[r, c] * scale : 0 over n x cols (fp32 or bf16).  The data may keep
// every block of h_s columns padded to hp columns (hp >= h_s; padding untouched); the mask is dense in blocks of h_s.
slicegcn_status_t dropout_apply_run(int64_t n, int cols, void* data, int64_t ld, int dtype, const uint8_t* mask, int64_t mask_ld,
                                    int h_s, int hp, float scale, cudaStream_t st);
// out = in * mask (fp32, row-major with leading dimensions)
slicegcn_status_t mask_mul_run(int64_t M, int N, const float* in, int64_t ld_in, const uint8_t* mask, int64_t ld_mask,
                               float* out, int64_t ld_out, cudaStream_t st);
// Softmax cross entropy (Eq. 10) over the training rows: writes dlogits = (softmax - onehot)/n_train
// (rows outside the training set are zeroed) and the mean loss.  row_loss: scratch [n_train] floats.
// dlogits has leading dimension ld_d >= C; columns C..ld_d-1 of every row are written as zeros.
// A label outside [0, C) or a training index outside [0, n) is skipped, never dereferenced; `fault` (the graph's status
// word, may be NULL) then receives kStatusBadLabel.
constexpr int kStatusBadLabel = SLICEGCN_DEVSTATUS_BAD_LABEL;
slicegcn_status_t softmax_ce_run(int64_t n, int C, const float* logits, const int32_t* labels, const int32_t* train_idx,
                                 int64_t n_train, float* dlogits, int64_t ld_d, float* row_loss, float* loss_out,
                                 int* fault, cudaStream_t st);
// Adam with bias correction; `step` is 1-based.
slicegcn_status_t adam_run(int64_t count, float* theta, const float* grad, float* m1, float* m2, float lr, float beta1,
                           float beta2, float eps, float weight_decay, int step, cudaStream_t st);

}  // namespace sgcn
