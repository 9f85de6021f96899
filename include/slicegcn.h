/*
 * slicegcn.h -- C ABI of the B200 (sm_100a) SliceGCN hot-path library.
 *
 * SliceGCN (arXiv 2408.11500) trains a full-graph GCN on p column slices of the
 * node-feature matrix; the slices never interact during message passing and are
 * concatenated before the classifier.  Here every slice lives on ONE GPU as a
 * column block of one row-major matrix.
 *
 * Conventions
 *   - Every function returns slicegcn_status_t (0 = success).  No exception crosses
 *     the boundary; slicegcn_last_error() returns a thread-local message for the last
 *     failing call of the calling thread.
 *   - Pointers marked [host] are host memory, [device] are device memory of the
 *     current CUDA device.  Handles (slicegcn_graph, slicegcn_model) are opaque and
 *     owned by the library (create/destroy).  All tensors are caller-owned; the
 *     library never keeps a pointer after a call returns and never frees caller memory.
 *   - Matrices are row-major with an explicit leading dimension in ELEMENTS.
 *   - `stream` is a cudaStream_t passed as void* (NULL = the default stream).  Compute
 *     calls are asynchronous on that stream; graph construction and the export calls
 *     synchronise it.
 *   - Compute calls (spmm, layer_forward/backward, train_epoch) allocate nothing; scratch
 *     memory comes from the caller, sized by the *_bytes queries.  (One exception takes no scratch
 *     argument at all: slicegcn_spmm_static_scratch uses a buffer compiled into the library.)
 *   - dtype: storage type of features / activations.  Accumulation is always fp32;
 *     parameters, gradients and logits are always fp32.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with
 *     SLICEGCN_ERR_CUDA.
 */
#ifndef SLICEGCN_H_
#define SLICEGCN_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int32_t slicegcn_status_t;
enum {
    SLICEGCN_OK = 0,
    SLICEGCN_ERR_INVALID_ARG = 1,   /* null pointer, non-positive size, inconsistent description */
    SLICEGCN_ERR_OUT_OF_RANGE = 2,  /* a node id or label outside its range */
    SLICEGCN_ERR_OVERFLOW = 3,      /* n or nnz does not fit int32 indexing */
    SLICEGCN_ERR_ALLOC = 4,         /* device/host allocation failed, or caller scratch too small */
    SLICEGCN_ERR_CUDA = 5,          /* a CUDA runtime call or kernel launch failed */
    SLICEGCN_ERR_UNSUPPORTED = 6    /* valid request outside what the kernels implement */
};

enum { SLICEGCN_F32 = 0, SLICEGCN_BF16 = 1 };                 /* dtype */
enum { SLICEGCN_ORDER_AUTO = 0, SLICEGCN_AGG_FIRST = 1, SLICEGCN_XFORM_FIRST = 2 };
enum { SLICEGCN_RULE_CEIL = 0, SLICEGCN_RULE_FLOOR_PLUS_1 = 1 };
enum {                                                          /* graph_create flags */
    SLICEGCN_SYMMETRIZE = 1u,       /* also store (v,u) for every input pair (u,v) */
    SLICEGCN_ADD_SELF_LOOPS = 2u,   /* set every diagonal entry (an input self-loop is not doubled) */
    SLICEGCN_INPUT_ON_DEVICE = 4u,  /* src/dst (or rowptr/colidx) are device pointers */
    /* Aggregator.  Default (neither flag): the normalisation of Eq. 1, A_hat = D^-1/2 A D^-1/2.  The paper defines
     * only that one; its closing section points at other GNN layers, whose aggregators share every kernel here:
     * mean over the neighbor set, A_hat = D^-1 A, and plain sum, A_hat = A.  At most one of the two. */
    SLICEGCN_NORM_MEAN = 8u,
    SLICEGCN_NORM_SUM = 16u
};
#define SLICEGCN_MAX_SLICES 64

typedef struct slicegcn_graph slicegcn_graph;
typedef struct slicegcn_model slicegcn_model;

/* Message of the last failing call on this thread ("" if none).  Never NULL. */
const char* slicegcn_last_error(void);

/* ---------------------------------------------------------------------------------------------
 * Slice strategy -- Algorithm 1 ("Slice Strategy Generation") and Eq. 3.
 *   slice_size = ceil(in_d/p) (RULE_CEIL, the algorithm as printed) or floor(in_d/p)+1
 *   (RULE_FLOOR_PLUS_1, the width the text gives for W_FF); slice i starts at i*slice_size and
 *   spans int(slice_size*scale) columns; a slice that would end past in_d is shifted left so
 *   that it ends at in_d.  Pure host integer arithmetic.
 *   starts/ends [host, p entries each] receive 0-based half-open column ranges.
 * Errors: INVALID_ARG if in_d < 1, p < 1, p > SLICEGCN_MAX_SLICES, a null pointer, or the scaled
 *   width is outside [1, in_d].
 */
slicegcn_status_t slicegcn_slice_strategy(int32_t in_d, int32_t p, double scale, int32_t rule,
                                          int32_t* starts, int32_t* ends, int32_t* slice_size);

/* ---------------------------------------------------------------------------------------------
 * Graph -- Section III-A (adjacency A in {0,1}^{n x n}, neighbor sets N(v)) and the
 * normalisation of Eq. 1: 1/c_ij = 1/(sqrt|N(v_i)| sqrt|N(v_j)|), |N(v)| = stored entries of row v
 * (counted after the optional self-loop).
 *
 * slicegcn_graph_create: edge list -> canonical CSR on the device (columns ascending inside each
 *   row, repeated pairs merged), degree vector, dinv = 1/sqrt(deg) in IEEE fp32 (0 for an empty
 *   row) and, when the pattern is not symmetric, the CSR of the transpose for the backward pass.
 *   An input pair (src[e], dst[e]) stores column dst[e] in row src[e].
 *   n: number of nodes (1 <= n < 2^31).  n_edges >= 0.  src/dst: int32 [n_edges], host unless
 *   SLICEGCN_INPUT_ON_DEVICE; never modified.  *out receives a handle owned by the library.
 * slicegcn_graph_create_from_csr: same from rowptr int32 [n+1] / colidx int32 [rowptr[n]]
 *   (columns need not be sorted or unique); the same flags apply.
 * Errors: INVALID_ARG (also: both NORM flags), OUT_OF_RANGE (an id outside [0,n)), OVERFLOW (stored entries >= 2^31),
 *   ALLOC, CUDA.  On error *out is NULL.  Both calls synchronise `stream`.
 */
slicegcn_status_t slicegcn_graph_create(int64_t n, int64_t n_edges, const int32_t* src, const int32_t* dst,
                                        uint32_t flags, void* stream, slicegcn_graph** out);
slicegcn_status_t slicegcn_graph_create_from_csr(int64_t n, const int32_t* rowptr, const int32_t* colidx,
                                                 uint32_t flags, void* stream, slicegcn_graph** out);
/* Sizes of a graph: n, nnz (stored entries), whether the pattern is symmetric, and the number of
 * long-row segments the SpMM splits hub rows into (any pointer may be NULL). */
slicegcn_status_t slicegcn_graph_info(const slicegcn_graph* g, int64_t* n, int64_t* nnz, int32_t* is_symmetric,
                                      int64_t* n_segments);
/* Copies the canonical CSR out for inspection: rowptr [host, n+1], colidx [host, nnz],
 * deg [host, n], dinv [host, n] (any may be NULL).  Synchronises the device. */
slicegcn_status_t slicegcn_graph_export(const slicegcn_graph* g, int32_t* rowptr, int32_t* colidx, int32_t* deg,
                                        float* dinv);
/* Device-side status word of the graph.  Kernels that wait on asynchronous copies bound every wait;
 * a wait that runs out sets this word instead of hanging (values 1..31), and the loss kernel sets it to
 * SLICEGCN_DEVSTATUS_BAD_LABEL when it meets a label or a training index outside its range (that node is
 * skipped: it adds nothing to the loss or the gradients, and nothing is read through the bad value).
 * Synchronises the device; *status is 0 when no kernel working on this graph ever reported anything.
 * Errors: INVALID_ARG, CUDA. */
enum { SLICEGCN_DEVSTATUS_BAD_LABEL = 32 };
slicegcn_status_t slicegcn_graph_device_status(const slicegcn_graph* g, int32_t* status);
/* Frees the handle and its device memory (NULL is accepted). */
slicegcn_status_t slicegcn_graph_destroy(slicegcn_graph* g);

/* ---------------------------------------------------------------------------------------------
 * Normalised sparse aggregation -- the neighbor sum of Eq. 1 / Eq. 6:
 *   Y[i, 0:width] = sum_{j in N(v_i)} X[j, 0:width] / c_ij          (transpose = 0)
 *   Y = A_hat^T X                                                    (transpose = 1, backward pass)
 * (A_hat as fixed at graph creation: Eq. 1's normalisation unless a NORM flag chose the mean or the sum.)
 * X [device, n x width, leading dimension ldx], Y [device, n x width, ldy]; X and Y must not
 * overlap.  in_dtype / out_dtype: SLICEGCN_F32 or SLICEGCN_BF16 (fp32 accumulation); the pairs fp32 -> fp32,
 * bf16 -> bf16 and bf16 -> fp32 are supported (fp32 -> bf16: UNSUPPORTED).
 * workspace [device]: at least slicegcn_spmm_workspace_bytes(g, width) bytes (partial sums of the
 * split hub rows and one counter per such row; may be NULL when that size is 0; two calls that may
 * overlap on the GPU need separate workspaces).  Deterministic: no floating-point atomics.
 * Errors: INVALID_ARG, UNSUPPORTED, ALLOC (workspace too small), CUDA.
 */
slicegcn_status_t slicegcn_spmm_workspace_bytes(const slicegcn_graph* g, int32_t width, int64_t* bytes);
slicegcn_status_t slicegcn_spmm(const slicegcn_graph* g, int32_t transpose, int32_t in_dtype, int32_t out_dtype,
                                const void* X, int64_t ldx, void* Y, int64_t ldy, int32_t width,
                                void* workspace, int64_t workspace_bytes, void* stream);

/* The same aggregation for callers that cannot allocate device memory.  (The paper has no counterpart:
 * this entry point exists for the embedding, not for the method.)
 *
 * Some callers may not call cudaMalloc: code running inside a stream capture, a host with a fixed memory
 * plan handed out at start-up, a plugin that must not touch the allocator of the process it lives in.  For
 * them the scratch the split hub rows need (their partial sums) comes from a buffer compiled into the
 * library: 8 MiB of device memory that every GPU loading the library holds until the process exits.
 * The call allocates nothing on the host or the device and frees nothing; X and Y are still the caller's.
 *   - Limit: slicegcn_spmm_workspace_bytes(g, width) must be <= 8 MiB (8,388,608 bytes); otherwise the call
 *     fails with SLICEGCN_ERR_UNSUPPORTED and a message giving both numbers, and nothing is launched.
 *   - The first call on a device looks the buffer's device address up (once per device, with that device
 *     current -- the device of `g` must be current, as for every call).  Make that first call outside any
 *     stream capture.
 *   - All calls share the one buffer, which keeps whatever the last call left in it.  Nothing in it needs to
 *     start at zero (a call only reads partial sums it wrote itself), but two calls whose kernels overlap on
 *     the GPU -- different streams, or different threads -- race on it: serialise them.
 *   - Not counted by slicegcn_profile_begin/end.
 * Arguments, results and the other errors are those of slicegcn_spmm. */
slicegcn_status_t slicegcn_spmm_static_scratch(const slicegcn_graph* g, int32_t transpose, int32_t in_dtype,
                                               int32_t out_dtype, const void* X, int64_t ldx, void* Y, int64_t ldy,
                                               int32_t width, void* stream);

/* ---------------------------------------------------------------------------------------------
 * One sliced GCN layer -- Eq. 6 (and Eq. 7-8 when E is given):
 *   for slice i:  M_i = b_i + (A_hat H_in[:, in_starts[i] : in_starts[i]+in_width]) W_agg_i
 *                 H_out[:, i*h_s : (i+1)*h_s] = ReLU(M_i) + H_in[:, ...] W_self_i (+ b_self_i) (+ E_i)
 * num_slices = 1, W_self = NULL, E = NULL gives the plain GCN layer of Eq. 1.  Writing the slices
 * as adjacent column blocks of H_out IS the concatenation of Eq. 8.
 */
typedef struct slicegcn_layer_desc {
    int32_t num_slices;        /* p, 1..SLICEGCN_MAX_SLICES */
    const int32_t* in_starts;  /* [host, p] first input column of each slice (ranges may overlap) */
    int32_t in_width;          /* columns per slice (Algorithm 1 gives every slice the same width) */
    int32_t in_cols;           /* number of columns of H_in that hold data (>= max start + in_width) */
    int64_t in_ld;             /* leading dimension of H_in */
    int32_t h_s;               /* output columns per slice */
    int64_t out_ld;            /* leading dimension of H_out (>= p*h_s) */
    int32_t dtype;             /* storage type of H_in, H_out and the saved intermediate */
    int32_t order;             /* AUTO: aggregate at the narrower of the input / output widths */
    const float* W_agg;        /* [device] p x in_width x h_s, slice-major, row-major blocks */
    const float* W_self;       /* [device] same shape, or NULL (no self term) */
    const float* b;            /* [device] p x h_s (bias inside the ReLU) */
    const float* b_self;       /* [device] p x h_s or NULL */
    const float* E;            /* [device] p x h_s slice-encoding rows (Eq. 7) or NULL */
} slicegcn_layer_desc;

/* Bytes of `saved` (kept from forward to backward: the aggregated or transformed intermediate
 * and the ReLU mask) and of `workspace` (scratch, contents undefined afterwards). */
slicegcn_status_t slicegcn_layer_saved_bytes(const slicegcn_graph* g, const slicegcn_layer_desc* d, int64_t* bytes);
slicegcn_status_t slicegcn_layer_workspace_bytes(const slicegcn_graph* g, const slicegcn_layer_desc* d,
                                                 int64_t* bytes);
/* Where things lie inside `saved` after slicegcn_layer_forward, for inspection (tests read the ReLU decisions the
 * forward pass took): the intermediate (A_hat H_in for an aggregate-first layer, H_in W_agg for a transform-first
 * one; d->dtype, row-major) starts at byte *zt_offset with leading dimension *zt_ld elements and *zt_cols columns;
 * the ReLU mask of Eq. 6 -- one byte per unit, 1 where b + aggregation > 0 -- starts at byte *mask_offset with
 * leading dimension *mask_ld bytes and p*h_s columns.  Any output pointer may be NULL. */
slicegcn_status_t slicegcn_layer_saved_layout(const slicegcn_graph* g, const slicegcn_layer_desc* d, int64_t* zt_offset,
                                              int64_t* zt_ld, int32_t* zt_cols, int64_t* mask_offset, int64_t* mask_ld);
/* Forward.  H_in [device, n x in_cols], H_out [device, n x p*h_s], both of d->dtype.
 * Errors: INVALID_ARG, ALLOC (buffers too small), UNSUPPORTED, CUDA. */
slicegcn_status_t slicegcn_layer_forward(const slicegcn_graph* g, const slicegcn_layer_desc* d, const void* H_in,
                                         void* H_out, void* saved, int64_t saved_bytes, void* workspace,
                                         int64_t workspace_bytes, void* stream);
/* Backward of the same layer (the paper leaves it implicit: the last step of the epoch loop of
 * Algorithm 3 only names it).  dH_out [device, fp32, n x p*h_s, leading dimension dout_ld] is the gradient of the
 * loss w.r.t. H_out and is not modified.  Outputs (all fp32, OVERWRITTEN, each may be NULL to skip):
 *   dH_in  [device, n x in_cols, leading dimension din_ld] -- contributions of overlapping slices add;
 *   dW_agg, dW_self [p x in_width x h_s]; db, db_self, dE [p x h_s].
 * ReLU'(0) = 0.  With dtype SLICEGCN_BF16 one intermediate gradient is kept in bf16 as well: dZ = dM W_agg^T of an
 * aggregate-first layer whose slices read disjoint columns (the operand of the transposed aggregation); sums are
 * accumulated in fp32 on both sides of it. */
slicegcn_status_t slicegcn_layer_backward(const slicegcn_graph* g, const slicegcn_layer_desc* d, const void* H_in,
                                          const void* saved, const float* dH_out, int64_t dout_ld, float* dH_in,
                                          int64_t din_ld, float* dW_agg, float* dW_self, float* db, float* db_self,
                                          float* dE, void* workspace, int64_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Model and training epoch -- Algorithm 3 ("Training Process of Slice-GCN"), Eq. 4-10.
 *   [feature fusion: X_ff = ReLU(X W1 + b1) W2 + b2, one MLP d' -> d' -> slice_size whose output
 *    feeds every slice]  ->  L sliced layers (Eq. 6)  ->  slice encoding (Eq. 7)  ->  concat (Eq. 8)
 *   ->  classifier ReLU(H Wc1 + bc1) Wc2 + bc2 (Eq. 9)  ->  mean cross entropy over the training
 *   nodes (Eq. 10)  ->  backward  ->  Adam step with cosine-annealed learning rate.
 * Per-slice hidden width h_s = ceil(hidden / p); classifier hidden width = hidden.
 */
typedef struct slicegcn_model_desc {
    int32_t in_d;              /* d' */
    int32_t hidden;
    int32_t num_layers;        /* L >= 1 */
    int32_t num_classes;
    int32_t num_slices;        /* p */
    double slice_size_scale;   /* Algorithm 1; 1.0 = default */
    int32_t slice_rule;        /* SLICEGCN_RULE_* */
    int32_t use_ff;            /* feature fusion on/off */
    int32_t use_se;            /* slice encoding on/off */
    int32_t use_self;          /* W_self term of Eq. 6 (0: plain GCN, Eq. 1) */
    int32_t use_b_self;        /* second bias per layer */
    int32_t dtype;             /* storage type of X and of every activation (bf16: also of dZ, see slicegcn_layer_backward);
                                  parameters, their gradients, logits and loss are always fp32 */
    int32_t order;             /* SLICEGCN_ORDER_AUTO or a forced order for every layer */
    int32_t cache_input_aggregate;  /* 1: keep A_hat X of the first layer across calls (see slicegcn_train_epoch) */
} slicegcn_model_desc;

typedef struct slicegcn_opt_desc {
    double lr0;                /* initial learning rate */
    double beta1, beta2, eps, weight_decay;
    int32_t epoch;             /* 0-based index of this epoch; lr = lr0 * (1 + cos(pi*epoch/total))/2 */
    int32_t total_epochs;
} slicegcn_opt_desc;

/* Validates the description, runs Algorithm 1 and fixes the parameter layout.  Host only. */
slicegcn_status_t slicegcn_model_create(const slicegcn_model_desc* desc, slicegcn_model** out);
slicegcn_status_t slicegcn_model_destroy(slicegcn_model* m);
/* Number of learnable scalars (the closed form behind Table III). */
slicegcn_status_t slicegcn_model_param_count(const slicegcn_model* m, int64_t* count);
/* All parameters live in ONE fp32 buffer of slicegcn_model_param_elems() elements (tensors are
 * padded to 16-byte boundaries; padding is ignored and kept zero by the optimiser).  Tensor t
 * (0 <= t < num_tensors) has a name ("ff_W1", "ff_b1", "ff_W2", "ff_b2", "W_agg.<l>", "W_self.<l>",
 * "b.<l>", "b_self.<l>", "E", "Wc1", "bc1", "Wc2", "bc2"), an element offset and dims
 * (d0 x d1 x d2, unused dims = 1; per-layer tensors are slice-major p x rows x cols). */
slicegcn_status_t slicegcn_model_param_elems(const slicegcn_model* m, int64_t* elems);
slicegcn_status_t slicegcn_model_num_tensors(const slicegcn_model* m, int32_t* count);
slicegcn_status_t slicegcn_model_tensor_info(const slicegcn_model* m, int32_t t, char name[32], int64_t* offset,
                                             int32_t dims[3]);
/* Slice table of the model (Algorithm 1 applied to in_d): starts/ends [host, p], slice_size, h_s. */
slicegcn_status_t slicegcn_model_slices(const slicegcn_model* m, int32_t* starts, int32_t* ends,
                                        int32_t* slice_size, int32_t* h_s);
/* Order chosen for layer l (SLICEGCN_AGG_FIRST / SLICEGCN_XFORM_FIRST). */
slicegcn_status_t slicegcn_model_layer_order(const slicegcn_model* m, int32_t layer, int32_t* order);
/* Scratch bytes one epoch needs on graph g. */
slicegcn_status_t slicegcn_train_workspace_bytes(const slicegcn_model* m, const slicegcn_graph* g, int64_t* bytes);

/* One iteration of the epoch loop of Algorithm 3: forward, loss, backward and (if opt != NULL)
 * one Adam update with the cosine-annealed rate of epoch opt->epoch.
 *   X        [device, n x in_d of m's dtype, leading dimension x_ld]   (not modified)
 *   labels   [device, int32 n], each in [0, num_classes); a training node whose label is outside that range is
 *            skipped and reported through slicegcn_graph_device_status (SLICEGCN_DEVSTATUS_BAD_LABEL)
 *   train_idx[device, int32 n_train] or NULL = every node is a training node (then n_train is ignored); an index
 *            outside [0, n) is skipped and reported the same way
 *   params   [device, fp32 param_elems]  updated in place when opt != NULL
 *   grads    [device, fp32 param_elems]  overwritten with dLoss/dparams
 *   adam_m, adam_v [device, fp32 param_elems]  optimiser state (zero before the first epoch); may be
 *            NULL when opt == NULL
 *   logits_out [device, fp32 n x num_classes, dense] or NULL
 *   loss_out [device, one float] or NULL: mean cross entropy BEFORE the update
 *   workspace [device], workspace_bytes >= slicegcn_train_workspace_bytes()
 * Input aggregate cache (desc.cache_input_aggregate = 1): Algorithm 3 slices the features once, outside the epoch
 * loop, so what depends on X alone is the same in every epoch: with direct slicing and an aggregate-first first layer
 * its aggregate A_hat X^i (Eq. 6, l = 1), and any aligned / padded copy of X the kernels work from.  With the flag set
 * the library keeps these in `workspace` and skips recomputing them whenever X, x_ld, the graph, `workspace` and
 * `stream` are those of the previous call on this model.  The caller
 * then promises that the CONTENTS of X and of `workspace` do not change between such calls; after changing them, call
 * slicegcn_model_invalidate_caches().  The host-buffer entry points copy X anew every epoch and never use the cache.
 * Asynchronous on `stream`.  The model object keeps host-side bookkeeping of the converted weight operands it
 * has placed in `workspace` (they are converted again, in one launch, at the start of every call): calls on ONE model
 * must not run concurrently, and the contents of `workspace` are only meaningful to the library.
 * Errors: INVALID_ARG, ALLOC, UNSUPPORTED, CUDA. */
slicegcn_status_t slicegcn_train_epoch(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                       const int32_t* labels, const int32_t* train_idx, int64_t n_train,
                                       float* params, float* grads, float* adam_m, float* adam_v,
                                       const slicegcn_opt_desc* opt, float* logits_out, float* loss_out,
                                       void* workspace, int64_t workspace_bytes, void* stream);

/* The same iteration with dropout between the layers.  Table II of the paper lists a dropout rate per dataset; the
 * text never says where it acts, so the placement is this library's choice (and the oracle's): the output of every
 * sliced layer but the last is multiplied by a 0/1 mask and by 1/(1 - rate) before the next layer reads it, forward
 * and backward.  The masks are the caller's: the library draws no random numbers.
 *   rate      in [0, 1)
 *   masks     [host array of num_layers - 1 pointers]; masks[l] [device, n x (p*h_s) bytes, leading dimension mask_ld
 *             bytes]: 0 drops the unit, anything else keeps it; it acts on the output of layer l (0-based)
 * drop == NULL is slicegcn_train_epoch.  Errors: INVALID_ARG (rate outside [0,1), NULL mask, mask_ld < p*h_s), and
 * those of slicegcn_train_epoch. */
typedef struct slicegcn_dropout_desc {
    double rate;
    const uint8_t* const* masks;
    int64_t mask_ld;
} slicegcn_dropout_desc;
slicegcn_status_t slicegcn_train_epoch_dropout(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                               const int32_t* labels, const int32_t* train_idx, int64_t n_train,
                                               float* params, float* grads, float* adam_m, float* adam_v,
                                               const slicegcn_opt_desc* opt, const slicegcn_dropout_desc* drop,
                                               float* logits_out, float* loss_out, void* workspace, int64_t workspace_bytes,
                                               void* stream);

/* The paper's own placement (Section IV-A, Eq. 8): slice i of the features lives on its own device, the graph is
 * replicated, nothing is exchanged during message passing, and the slices' outputs H^i meet once, for the
 * concatenation in front of the classifier.  One process per GPU calls this entry point with the SAME model, graph,
 * X, labels and parameter buffers' contents, and its own range [slice_begin, slice_end) of the p slices: the sliced
 * layers (Eq. 6, 7) run for those slices only; the fusion MLP (Eq. 4), the classifier (Eq. 9), the loss and the Adam
 * step run on every rank with identical inputs, so the parameters stay replicas without being sent.  The library
 * does no communication itself; at three points it calls `exchange` (on the host, work queued on `stream` so far is
 * the caller's to order against):
 *   SLICEGCN_EXCHANGE_GATHER_H   buf [device, m's dtype, rows x (p*h_s), leading dimension ld]: columns
 *                                [col0, col0 + cols) hold this rank's slice outputs; on return every column must
 *                                hold its owner's values (an all-gather of column blocks: Eq. 8)
 *   SLICEGCN_EXCHANGE_SUM_DXFF   (feature-fusion models) buf [device, fp32, rows x cols, leading dimension ld]: this
 *                                rank's part of the gradient of the fused input X_ff, which every slice reads; on
 *                                return the sum over ranks
 *   SLICEGCN_EXCHANGE_SUM_GRADS  buf = grads [device, fp32, `rows` elements, ld = cols = 1]: per-slice tensors hold
 *                                this rank's slices (zeros elsewhere), replicated tensors are non-zero on the rank with
 *                                slice_begin == 0 only; on return the sum over ranks
 * `exchange` returns SLICEGCN_OK or an error code, which ends the call with that code (nothing is updated then).
 * With slice_begin = 0, slice_end = p and exchange = NULL this is slicegcn_train_epoch.  Not combined with dropout,
 * the input aggregate cache or per-slice widths that need the padded internal layout (UNSUPPORTED).
 * Errors: INVALID_ARG (empty or out-of-range slice range, exchange NULL for a partial range), and those of
 * slicegcn_train_epoch. */
#define SLICEGCN_EXCHANGE_GATHER_H 1
#define SLICEGCN_EXCHANGE_SUM_DXFF 2
#define SLICEGCN_EXCHANGE_SUM_GRADS 3
typedef slicegcn_status_t (*slicegcn_exchange_fn)(void* ctx, int32_t what, void* buf, int64_t rows, int64_t ld, int32_t col0,
                                                  int32_t cols, int32_t dtype, void* stream);
slicegcn_status_t slicegcn_train_epoch_sliced(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                              const int32_t* labels, const int32_t* train_idx, int64_t n_train,
                                              float* params, float* grads, float* adam_m, float* adam_v,
                                              const slicegcn_opt_desc* opt, int32_t slice_begin, int32_t slice_end,
                                              slicegcn_exchange_fn exchange, void* exchange_ctx, float* logits_out,
                                              float* loss_out, void* workspace, int64_t workspace_bytes, void* stream);

/* Forgets what the model object remembers about earlier calls (the input aggregate cache above).  Host only. */
slicegcn_status_t slicegcn_model_invalidate_caches(const slicegcn_model* m);

/* Evaluation pass: the forward half of the iteration above (Eq. 4-9) with the current parameters; writes the logits
 * [device, fp32 n x num_classes, dense] and nothing else a caller can see.  Same workspace as slicegcn_train_epoch.
 * Asynchronous on `stream`.  Errors: INVALID_ARG, ALLOC, UNSUPPORTED, CUDA. */
slicegcn_status_t slicegcn_forward_logits(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                          const float* params, float* logits_out, void* workspace, int64_t workspace_bytes,
                                          void* stream);

/* The same iteration for callers whose inputs live in host memory (the paper's training loop,
 * Algorithm 3, starts from the dataset in host memory): copies the feature matrix and the labels to
 * the caller's device staging buffers, runs slicegcn_train_epoch on them, copies the loss back and
 * waits for `stream`.
 *   X_host      [host, n rows of in_d values of m's dtype, row pitch x_ld elements]
 *   labels_host [host, int32 n]
 *   X_stage     [device, n * x_ld elements of m's dtype], labels_stage [device, int32 n]: staging
 *               owned by the caller, overwritten
 *   loss_host   [host, one float] or NULL
 *   loss_dev    [device, one float]: where the step leaves the loss before it is copied back
 *   every other argument as for slicegcn_train_epoch (device memory).
 * Host buffers should be page-locked: pageable memory works but the copies are slower and not
 * asynchronous.  Synchronous: returns after the stream has drained.  The labels are checked on the host before
 * anything is copied: OUT_OF_RANGE if one is outside [0, num_classes).  Other errors as above. */
slicegcn_status_t slicegcn_train_epoch_host(const slicegcn_model* m, const slicegcn_graph* g, const void* X_host, int64_t x_ld,
                                            const int32_t* labels_host, void* X_stage, int32_t* labels_stage,
                                            const int32_t* train_idx, int64_t n_train, float* params, float* grads,
                                            float* adam_m, float* adam_v, const slicegcn_opt_desc* opt, float* loss_dev,
                                            float* loss_host, void* workspace, int64_t workspace_bytes, void* stream);

/* num_epochs consecutive iterations of the loop of Algorithm 3 from host memory, epochs
 * opt->epoch, opt->epoch + 1, ...  Every epoch copies the feature matrix and the labels from the
 * host again (the caller may rewrite them between calls, not during one); the copy for epoch e+1
 * runs on a second stream into the other staging buffer while epoch e computes, so in steady state
 * the transfer is hidden behind the kernels.  Each epoch's loss is copied to losses_host[e] as
 * soon as it exists.
 *   X_stage0/1 [device, n * x_ld elements each], labels_stage0/1 [device, int32 n each]
 *   losses_dev [device, num_epochs floats], losses_host [host, num_epochs floats] or NULL
 *   opt        required (the epoch index advances inside the call)
 * Creates and destroys one stream and four events per call.  Synchronous.  OUT_OF_RANGE for a label outside
 * [0, num_classes) (checked on the host before the first copy); other errors as above. */
slicegcn_status_t slicegcn_train_epochs_host(const slicegcn_model* m, const slicegcn_graph* g, const void* X_host, int64_t x_ld,
                                             const int32_t* labels_host, void* X_stage0, void* X_stage1, int32_t* labels_stage0,
                                             int32_t* labels_stage1, const int32_t* train_idx, int64_t n_train, float* params,
                                             float* grads, float* adam_m, float* adam_v, const slicegcn_opt_desc* opt,
                                             int32_t num_epochs, float* losses_dev, float* losses_host, void* workspace,
                                             int64_t workspace_bytes, void* stream);

/* ---------------------------------------------------------------------------------------------
 * Instrumentation for benchmarks (the paper reports only end-to-end epochs per second, Table IV;
 * this splits out the aggregation kernel).  Between profile_begin and profile_end every SpMM call
 * is bracketed by CUDA events on its stream and kernel launches are counted.  profile_end
 * synchronises the device and returns: total SpMM device time [ms], number of SpMM calls, their
 * algorithmic bytes (CSR indices + degree vector + operand read once + result written once), and the
 * number of kernels the library launched.  Any output pointer may be NULL.  Not thread-safe.
 */
slicegcn_status_t slicegcn_profile_begin(void);
/* The same, bracketing only every stride-th SpMM call (stride >= 1): an event pair costs the stream a few
 * microseconds, which a benchmark that also reports whole-step time wants to keep small.  With a stride
 * coprime to the number of SpMM calls per step every call site is sampled equally often. */
slicegcn_status_t slicegcn_profile_begin_sampled(int32_t stride);
slicegcn_status_t slicegcn_profile_end(double* spmm_ms, int64_t* spmm_calls, double* spmm_bytes,
                                       int64_t* kernel_launches);

#ifdef __cplusplus
}
#endif
#endif /* SLICEGCN_H_ */
