// Host orchestration: slice strategy (Algorithm 1), one sliced layer forward / backward (Eq. 6-8),
// the model's parameter layout and one training epoch (Algorithm 3).  Everything here is launch
// sequencing on the caller's stream; all arithmetic on tensors happens in the kernels.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "kernels.cuh"

namespace sgcn {
namespace {

inline int64_t align_up(int64_t v, int64_t a) { return (v + a - 1) / a * a; }
inline int esize(int dtype) { return dtype == SLICEGCN_BF16 ? 2 : 4; }

// Bump allocator over caller scratch; with base == nullptr it only measures.
// Row order of the streaming products.  Consecutive kernels that stream the same N x width tensor find none of it in
// L2 when both walk the rows upwards (the tensor is larger than L2, the first reader's tail evicts its head); a
// consumer that walks downwards starts with what the producer left behind.  The products marked `reverse` below are the
// ones where that measured a gain on the benchmark workload (42 us per epoch in all): the fused layer product after
// the aggregation that wrote Z, the accumulating self product after the aggregation that wrote dH_in, dZ, the gated
// classifier product and the logits product after the kernels that wrote or read their operands upwards.

struct Bump {
    char* base = nullptr;
    int64_t off = 0;
    void* take(int64_t bytes) {
        off = align_up(off, 256);
        void* p = base ? base + off : nullptr;
        off += bytes;
        return p;
    }
};

slicegcn_status_t slice_strategy(int in_d, int p, double scale, int rule, int* starts, int* ends, int* slice_size) {
    if (in_d < 1 || p < 1 || p > SLICEGCN_MAX_SLICES || !starts || !ends || !slice_size)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "slice_strategy: need in_d >= 1, 1 <= p <= %d, non-NULL outputs",
                  SLICEGCN_MAX_SLICES);
    int size;
    if (rule == SLICEGCN_RULE_CEIL)
        size = (in_d + p - 1) / p;
    else if (rule == SLICEGCN_RULE_FLOOR_PLUS_1)
        size = in_d / p + 1;
    else
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "slice_strategy: unknown rule %d", rule);
    const double scaled = (double)size * scale;
    if (!(scaled >= 1.0) || scaled > (double)in_d + 0.5) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "slice_strategy: scaled width outside [1, in_d]");
    const int width = (int)scaled;   // truncation toward zero, as int() in the algorithm
    if (width < 1 || width > in_d) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "slice_strategy: scaled width outside [1, in_d]");
    for (int i = 0; i < p; ++i) {
        int s = i * size, e = s + width;
        if (e > in_d) {   // the last slice(s) are shifted left to end at in_d
            s -= e - in_d;
            e = in_d;
        }
        if (s < 0) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "slice_strategy: slice %d does not fit", i);
        starts[i] = s;
        ends[i] = e;
    }
    *slice_size = size;
    return SLICEGCN_OK;
}

// ------------------------------------------------------------------------------------------ layer
struct LayerPlan {
    int p = 0, in_width = 0, in_cols = 0, h_s = 0, out_cols = 0;
    int64_t in_ld = 0, out_ld = 0;
    int dtype = 0, order = 0, esz = 4;
    int in_starts[SLICEGCN_MAX_SLICES];
    bool disjoint_cover = false;   // slices tile [0, in_cols) without overlap or gap
    int zt_cols = 0;               // columns of the saved intermediate (Z: in_cols, T: out_cols)
    int64_t zt_ld = 0, mask_ld = 0, zt_bytes = 0, mask_bytes = 0;
    int64_t n = 0;
    // set by callers that keep the padding columns (up to the leading dimension) of H_in / the saved
    // intermediate at zero: lets 16-byte loads run over widths that are not multiples of 8
    bool in_pad_zero = false, zt_pad_zero = false;
    // backward may write zeros into the columns of dH_in between in_cols and the next multiple of 4 (internal buffers
    // of the training step only; never set for the layer-level calls, whose dH_in belongs to the caller)
    bool din_pad_write = false;
};

slicegcn_status_t make_plan(const slicegcn_graph* g, const slicegcn_layer_desc* d, LayerPlan* pl) {
    if (!g || !d) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: NULL graph or description");
    if (d->num_slices < 1 || d->num_slices > SLICEGCN_MAX_SLICES || !d->in_starts || d->in_width < 1 || d->h_s < 1)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: bad slice description");
    if (d->dtype != SLICEGCN_F32 && d->dtype != SLICEGCN_BF16) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: bad dtype");
    if (!d->W_agg) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: W_agg is NULL");
    LayerPlan& L = *pl;
    L.n = g->n;
    L.p = d->num_slices;
    L.in_width = d->in_width;
    L.in_cols = d->in_cols;
    L.h_s = d->h_s;
    L.out_cols = L.p * L.h_s;
    L.in_ld = d->in_ld;
    L.out_ld = d->out_ld;
    L.dtype = d->dtype;
    L.esz = esize(d->dtype);
    if (L.in_ld < L.in_cols || L.out_ld < L.out_cols) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: leading dimension too small");
    std::vector<int> cover(L.in_cols > 0 ? L.in_cols : 0, 0);
    bool disjoint = true;
    for (int i = 0; i < L.p; ++i) {
        const int s = d->in_starts[i];
        if (s < 0 || s + L.in_width > L.in_cols) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: slice %d outside [0, in_cols)", i);
        L.in_starts[i] = s;
        for (int c = s; c < s + L.in_width; ++c)
            if (cover[c]++) disjoint = false;
    }
    for (int c = 0; c < L.in_cols; ++c)
        if (!cover[c]) disjoint = false;
    L.disjoint_cover = disjoint;
    L.order = d->order;
    if (L.order == SLICEGCN_ORDER_AUTO) L.order = (L.in_cols <= L.out_cols) ? SLICEGCN_AGG_FIRST : SLICEGCN_XFORM_FIRST;
    if (L.order != SLICEGCN_AGG_FIRST && L.order != SLICEGCN_XFORM_FIRST) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer: bad order");
    L.zt_cols = L.order == SLICEGCN_AGG_FIRST ? L.in_cols : L.out_cols;
    L.zt_ld = align_up(L.zt_cols, 8);
    L.mask_ld = align_up(L.out_cols, 16);
    L.zt_bytes = align_up(L.n * L.zt_ld * L.esz, 256);
    L.mask_bytes = align_up(L.n * L.mask_ld, 256);
    return SLICEGCN_OK;
}

// scratch for the prepared weight images of the tensor-core GEMMs of one layer (forward and dgrad shapes)
int64_t layer_tc_img(const LayerPlan& L) {
    // forward may run the aggregation and self products in one pass: two images
    return std::max(2 * tc_image_bytes(L.p, L.in_width, L.h_s), tc_image_bytes(L.p, L.h_s, L.in_width));
}

int64_t layer_fwd_ws_bytes(const slicegcn_graph* g, const LayerPlan& L) {
    Bump b;
    b.take(layer_tc_img(L));
    b.take(spmm_partial_bytes(g, L.zt_cols));
    return align_up(b.off, 256);
}

int64_t layer_wgrad_scratch(const LayerPlan& L) {
    int64_t a = wgrad_scratch_bytes(L.n, L.p, L.in_width, L.h_s);
    int64_t b = wgrad_scratch_bytes(L.n, L.p, 0, L.h_s);
    return a > b ? a : b;
}

int64_t layer_bwd_ws_bytes(const slicegcn_graph* g, const LayerPlan& L) {
    Bump b;
    b.take(layer_tc_img(L));
    b.take(layer_wgrad_scratch(L));
    b.take(spmm_partial_bytes(g, L.zt_cols));
    b.take(L.n * align_up(L.out_cols, 8) * 4);   // dM = dH * mask
    b.take(L.n * L.zt_ld * 4);                   // dZ (aggregate-first) or dT (transform-first)
    return align_up(b.off, 256);
}

// Runs a grouped GEMM either as one launch (groups in grid.z) or, when the groups' output
// columns overlap, one group after the other.
slicegcn_status_t gemm_groups(const GemmArgs& a, bool sequential, cudaStream_t st) {
    if (!sequential || a.groups == 1) return gemm_run(a, st);
    for (int g = 0; g < a.groups; ++g) {
        GemmArgs s = a;
        s.groups = 1;
        s.a_start[0] = a.a_start[g];
        s.c_start[0] = a.c_start[g];
        s.B = a.B + (int64_t)g * a.b_gstride;
        if (a.bias) s.bias = a.bias + g * a.N;
        if (a.post1) s.post1 = a.post1 + g * a.N;
        if (a.post2) s.post2 = a.post2 + g * a.N;
        SGCN_TRY(gemm_run(s, st));
    }
    return SLICEGCN_OK;
}

// aggregate_cached: the saved intermediate already holds A_hat H_in from an earlier call (aggregate-first layers only)
slicegcn_status_t layer_forward_impl(const slicegcn_graph* g, const slicegcn_layer_desc* d, const LayerPlan& L,
                                     const void* H_in, void* H_out, void* saved, void* ws, int64_t ws_bytes,
                                     cudaStream_t st, bool aggregate_cached = false) {
    char* zt = static_cast<char*>(saved);
    uint8_t* mask = reinterpret_cast<uint8_t*>(zt + L.zt_bytes);
    if (ws_bytes < layer_fwd_ws_bytes(g, L)) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "layer_forward: workspace too small");
    Bump fb;
    fb.base = static_cast<char*>(ws);
    const int64_t img_bytes = layer_tc_img(L);
    void* img = fb.take(img_bytes);
    const int64_t part_bytes = spmm_partial_bytes(g, L.zt_cols);
    void* part = fb.take(part_bytes);
    const bool has_post = d->W_self || d->b_self || d->E;

    GemmArgs self;   // H_out = H_in W_self + b_self + E

    self.fault = g->fault;
    self.b_image = img;
    self.b_image_bytes = img_bytes;
    self.M = L.n;
    self.groups = L.p;
    self.K = d->W_self ? L.in_width : 0;
    self.N = L.h_s;
    self.A = H_in;
    self.lda = L.in_ld;
    self.a_dtype = L.dtype;
    self.B = d->W_self;
    self.b_gstride = (int64_t)L.in_width * L.h_s;
    self.ldb = L.h_s;
    self.C = H_out;
    self.ldc = L.out_ld;
    self.c_dtype = L.dtype;
    self.post1 = d->b_self;
    self.post2 = d->E;
    self.a_pad_zero = L.in_pad_zero ? 1 : 0;
    for (int i = 0; i < L.p; ++i) {
        self.a_start[i] = L.in_starts[i];
        self.c_start[i] = i * L.h_s;
    }

    if (L.order == SLICEGCN_AGG_FIRST) {
        // Z = A_hat H_in over every input column once; slices then read their column ranges of Z
        if (!aggregate_cached)
            SGCN_TRY(spmm_run(g, false, L.dtype, L.dtype, H_in, L.in_ld, zt, L.zt_ld, L.in_cols, nullptr, part, part_bytes, st));
        if (d->W_self) {
            // one pass: H_out = ReLU(Z W_agg + b) + H_in W_self + b_self + E (two accumulators)
            GemmArgs both = self;
            both.K = L.in_width;
            both.A = zt;
            both.lda = L.zt_ld;
            both.a_pad_zero = L.zt_pad_zero ? 1 : 0;
            both.B = d->W_agg;
            both.bias = d->b;
            both.relu = 1;
            both.mask_out = mask;
            both.mask_ld = L.mask_ld;
            both.A2 = H_in;
            both.lda2 = L.in_ld;
            both.a2_pad_zero = L.in_pad_zero ? 1 : 0;
            both.B2 = d->W_self;
            both.b2_gstride = self.b_gstride;
            both.K2 = L.in_width;
            for (int i = 0; i < L.p; ++i) both.a2_start[i] = L.in_starts[i];
            both.reverse = 1;   // Z was just written upwards by the aggregation
            const slicegcn_status_t rc = gemm_run(both, st);
            if (rc == SLICEGCN_OK) return SLICEGCN_OK;
            if (rc != SLICEGCN_ERR_UNSUPPORTED) return rc;
            SGCN_TRY(gemm_run(self, st));
        }
        GemmArgs agg = self;   // H_out = ReLU(Z W_agg + b) (+ H_out | + b_self + E)
        agg.K = L.in_width;
        agg.A = zt;
        agg.lda = L.zt_ld;
        agg.a_pad_zero = L.zt_pad_zero ? 1 : 0;
        agg.B = d->W_agg;
        agg.bias = d->b;
        agg.relu = 1;
        agg.mask_out = mask;
        agg.mask_ld = L.mask_ld;
        if (d->W_self) {
            agg.post1 = agg.post2 = nullptr;
            agg.accumulate = 1;
        }
        SGCN_TRY(gemm_run(agg, st));
    } else {
        GemmArgs tr = self;    // T = H_in W_agg
        tr.K = L.in_width;
        tr.B = d->W_agg;
        tr.C = zt;
        tr.ldc = L.zt_ld;
        tr.post1 = tr.post2 = nullptr;
        SGCN_TRY(gemm_run(tr, st));
        if (has_post) SGCN_TRY(gemm_run(self, st));
        SpmmEpilogue epi;      // H_out = ReLU(A_hat T + b) (+ H_out)
        epi.bias = d->b;
        epi.relu = 1;
        epi.mask = mask;
        epi.mask_ld = L.mask_ld;
        epi.accumulate = has_post ? 1 : 0;
        SGCN_TRY(spmm_run(g, false, L.dtype, L.dtype, zt, L.zt_ld, H_out, L.out_ld, L.out_cols, &epi, part, part_bytes, st));
    }
    return SLICEGCN_OK;
}

slicegcn_status_t layer_backward_impl(const slicegcn_graph* g, const slicegcn_layer_desc* d, const LayerPlan& L,
                                      const void* H_in, const void* saved, const float* dH_out, int64_t dout_ld,
                                      float* dH_in, int64_t din_ld, float* dW_agg, float* dW_self, float* db,
                                      float* db_self, float* dE, void* ws, int64_t ws_bytes, cudaStream_t st) {
    if (ws_bytes < layer_bwd_ws_bytes(g, L)) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "layer_backward: workspace too small");
    const char* zt = static_cast<const char*>(saved);
    const uint8_t* mask = reinterpret_cast<const uint8_t*>(zt + L.zt_bytes);
    Bump b;
    b.base = static_cast<char*>(ws);
    const int64_t img_bytes = layer_tc_img(L);
    void* img = b.take(img_bytes);
    const int64_t wg_bytes = layer_wgrad_scratch(L);
    void* wg = b.take(wg_bytes);
    const int64_t part_bytes = spmm_partial_bytes(g, L.zt_cols);
    void* part = b.take(part_bytes);
    const bool seq = !L.disjoint_cover;

    // self branch: dW_self = H_in^T dH, db_self = dE = colsum(dH)
    if ((d->W_self && dW_self) || db_self || dE) {
        WgradArgs w;
        w.fault = g->fault;
        w.M = L.n;
        w.groups = L.p;
        w.K = (d->W_self && dW_self) ? L.in_width : 0;
        w.N = L.h_s;
        w.A = H_in;
        w.lda = L.in_ld;
        w.a_dtype = L.dtype;
        w.a_pad_zero = L.in_pad_zero ? 1 : 0;
        w.B = dH_out;
        w.ldb = dout_ld;
        w.dW = dW_self;
        w.dbias = db_self;
        w.dbias2 = dE;
        for (int i = 0; i < L.p; ++i) {
            w.a_start[i] = L.in_starts[i];
            w.b_start[i] = i * L.h_s;
        }
        SGCN_TRY(wgrad_run(w, wg, wg_bytes, st));
    }

    GemmArgs dself;   // dH_in (+)= dH W_self^T

    dself.fault = g->fault;
    dself.b_image = img;
    dself.b_image_bytes = img_bytes;
    dself.M = L.n;
    dself.groups = L.p;
    dself.K = L.h_s;
    dself.N = L.in_width;
    dself.A = dH_out;
    dself.lda = dout_ld;
    dself.a_dtype = SLICEGCN_F32;
    dself.B = d->W_self;
    dself.b_gstride = (int64_t)L.in_width * L.h_s;
    dself.ldb = L.h_s;
    dself.b_trans = 1;
    dself.C = dH_in;
    dself.ldc = din_ld;
    dself.c_dtype = SLICEGCN_F32;
    for (int i = 0; i < L.p; ++i) {
        dself.a_start[i] = i * L.h_s;
        dself.c_start[i] = L.in_starts[i];
    }

    // All slices read the same input columns (fused input): the input gradient sums over the slices, which is ONE
    // product over the concatenated slice gradients with the slices' weight blocks stacked along K.
    bool shared_in = L.p > 1;
    for (int i = 1; i < L.p; ++i) shared_in = shared_in && L.in_starts[i] == L.in_starts[0];
    auto stacked = [&](GemmArgs a) {   // a: grouped product with one K block per slice -> single group, K = p * h_s
        a.groups = 1;
        a.K = L.p * L.h_s;
        a.b_kstack = L.h_s;
        a.a_start[0] = 0;
        a.c_start[0] = L.in_starts[0];
        a.c_pad_write = 1;   // the gradient buffers keep their rows padded to 8 columns
        return a;
    };

    if (L.order == SLICEGCN_AGG_FIRST) {
        // dM = dH * mask feeds the weight gradient, the bias gradient and dZ.  Where the tensor-core kernels
        // apply the byte mask in their producers (a mask tile travels next to every slab), dM is never
        // written; otherwise it is materialised once.
        const int64_t dm_ld = align_up(L.out_cols, 8);
        float* dM = static_cast<float*>(b.take(L.n * dm_ld * 4));
        WgradArgs w;      // dW_agg = Z^T dM, db = colsum(dM)
        w.fault = g->fault;
        w.M = L.n;
        w.groups = L.p;
        w.K = dW_agg ? L.in_width : 0;
        w.N = L.h_s;
        w.A = zt;
        w.lda = L.zt_ld;
        w.a_dtype = L.dtype;
        w.a_pad_zero = L.zt_pad_zero ? 1 : 0;
        w.dW = dW_agg;
        w.dbias = db;
        for (int i = 0; i < L.p; ++i) {
            w.a_start[i] = L.in_starts[i];
            w.b_start[i] = i * L.h_s;
        }
        GemmArgs dz = dself;   // dZ = dM W_agg^T
        dz.B = d->W_agg;
        // bf16 models store dZ -- the operand of the transposed aggregation, gathered deg times -- in bf16 like the
        // activations (fp32 accumulation on both sides); the fused input's narrow dZ stays fp32
        const bool dz_bf16 = L.dtype == SLICEGCN_BF16 && !shared_in && !seq && L.zt_ld % 8 == 0;
        if (dz_bf16) dz.c_dtype = SLICEGCN_BF16;
        const bool need_w = dW_agg || db;
        WgradArgs wm = w;
        wm.B = dH_out;
        wm.ldb = dout_ld;
        wm.b_mask = mask;
        wm.b_mask_ld = L.mask_ld;
        GemmArgs dzm = dz;
        dzm.A = dH_out;
        dzm.lda = dout_ld;
        dzm.a_mask = mask;
        dzm.a_mask_ld = L.mask_ld;
        // (a fused input shared by all slices: its dZ is ONE product over the stacked weight blocks, which takes the mask
        // like any other single-group product)
        bool dz_masked_ok = true;
        if (dH_in) {
            if (shared_in) {
                GemmArgs probe = stacked(dzm);
                probe.ldc = L.zt_ld;
                dz_masked_ok = tc_gemm_masks_in_producer(probe);
            } else {
                dz_masked_ok = !seq && tc_gemm_masks_in_producer(dzm);
            }
        }
        const bool in_producers = (!need_w || (dW_agg && wgrad_masks_in_producer(wm))) && dz_masked_ok;
        if (in_producers) {
            w = wm;
            dz = dzm;
        } else {
            SGCN_TRY(mask_mul_run(L.n, L.out_cols, dH_out, dout_ld, mask, L.mask_ld, dM, dm_ld, st));
            w.B = dM;
            w.ldb = dm_ld;
            dz.A = dM;
            dz.lda = dm_ld;
        }
        if (need_w) SGCN_TRY(wgrad_run(w, wg, wg_bytes, st));
        if (dH_in) {
            float* dZ = static_cast<float*>(b.take(L.n * L.zt_ld * 4));
            dz.C = dZ;
            dz.ldc = L.zt_ld;
            if (shared_in) {
                // whatever kernel takes the product, dZ's padding columns must be zero when they are aggregated below
                if (L.din_pad_write) SGCN_CUDA(cudaMemsetAsync(dZ, 0, L.n * L.zt_ld * 4, st));
                SGCN_TRY(gemm_run(stacked(dz), st));
            } else {
                if (seq) {
                    SGCN_CUDA(cudaMemsetAsync(dZ, 0, L.n * L.zt_ld * 4, st));
                    dz.accumulate = 1;
                }
                dz.reverse = 1;
                SGCN_TRY(gemm_groups(dz, seq, st));
            }
            // the stacked product left zeros in dZ's padding columns: aggregating them too keeps dH_in's padding at zero
            int sp_w = L.in_cols;
            if (shared_in && L.din_pad_write && align_up(L.in_cols, 4) <= std::min(L.zt_ld, din_ld)) sp_w = (int)align_up(L.in_cols, 4);
            SGCN_TRY(spmm_run(g, true, dz_bf16 ? SLICEGCN_BF16 : SLICEGCN_F32, SLICEGCN_F32, dZ, L.zt_ld, dH_in, din_ld, sp_w,
                              nullptr, part, part_bytes, st));
            if (d->W_self) {   // added by the GEMM's epilogue (an accumulating epilogue in the SpMM measured slower:
                               // its rows would wait for the old value at every row end)
                dself.accumulate = 1;
                dself.reverse = 1;   // dH_in was just written upwards by the aggregation
                if (shared_in) SGCN_TRY(gemm_run(stacked(dself), st));
                else SGCN_TRY(gemm_groups(dself, seq, st));
            }
        }
    } else {
        float* dM = static_cast<float*>(b.take(L.n * L.zt_ld * 4));
        float* dT = static_cast<float*>(b.take(L.n * L.zt_ld * 4));
        SGCN_TRY(mask_mul_run(L.n, L.out_cols, dH_out, dout_ld, mask, L.mask_ld, dM, L.zt_ld, st));
        if (db) {
            WgradArgs w;
            w.fault = g->fault;
            w.M = L.n;
            w.groups = L.p;
            w.K = 0;
            w.N = L.h_s;
            w.B = dM;
            w.ldb = L.zt_ld;
            w.dbias = db;
            for (int i = 0; i < L.p; ++i) w.b_start[i] = i * L.h_s;
            SGCN_TRY(wgrad_run(w, wg, wg_bytes, st));
        }
        if (dW_agg || dH_in) {   // dT = A_hat^T dM
            SGCN_TRY(spmm_run(g, true, SLICEGCN_F32, SLICEGCN_F32, dM, L.zt_ld, dT, L.zt_ld, L.out_cols, nullptr, part,
                              part_bytes, st));
        }
        if (dW_agg) {
            WgradArgs w;
            w.fault = g->fault;
            w.M = L.n;
            w.groups = L.p;
            w.K = L.in_width;
            w.N = L.h_s;
            w.A = H_in;
            w.lda = L.in_ld;
            w.a_dtype = L.dtype;
            w.a_pad_zero = L.in_pad_zero ? 1 : 0;
            w.B = dT;
            w.ldb = L.zt_ld;
            w.dW = dW_agg;
            for (int i = 0; i < L.p; ++i) {
                w.a_start[i] = L.in_starts[i];
                w.b_start[i] = i * L.h_s;
            }
            SGCN_TRY(wgrad_run(w, wg, wg_bytes, st));
        }
        if (dH_in) {
            GemmArgs dt = dself;   // dH_in = dT W_agg^T
            dt.A = dT;
            dt.lda = L.zt_ld;
            dt.B = d->W_agg;
            if (seq) {
                SGCN_CUDA(cudaMemset2DAsync(dH_in, din_ld * 4, 0, (size_t)L.in_cols * 4, L.n, st));
                dt.accumulate = 1;
            }
            bool done = false;
            if (d->W_self && !seq) {   // both products in one pass: dH_in = dT W_agg^T + dH W_self^T
                GemmArgs both = dt;
                both.A2 = dH_out;
                both.lda2 = dout_ld;
                both.B2 = d->W_self;
                both.b2_gstride = dself.b_gstride;
                both.K2 = L.h_s;
                for (int i = 0; i < L.p; ++i) both.a2_start[i] = i * L.h_s;
                const slicegcn_status_t rc = gemm_run(both, st);
                if (rc == SLICEGCN_OK) done = true;
                else if (rc != SLICEGCN_ERR_UNSUPPORTED) return rc;
            }
            if (!done) {
                SGCN_TRY(gemm_groups(dt, seq, st));
                if (d->W_self) {
                    dself.accumulate = 1;
                    SGCN_TRY(gemm_groups(dself, seq, st));
                }
            }
        }
    }
    return SLICEGCN_OK;
}

}  // namespace
}  // namespace sgcn

// ------------------------------------------------------------------------------------------ model
struct slicegcn_model {
    slicegcn_model_desc desc;
    int starts[SLICEGCN_MAX_SLICES], ends[SLICEGCN_MAX_SLICES];
    int slice_size = 0, slice_width = 0, h_s = 0;
    struct Tensor {
        std::string name;
        int64_t offset;
        int dims[3];
    };
    std::vector<Tensor> tensors;
    int64_t param_count = 0, param_elems = 0;
    // offsets into the flat parameter buffer (-1: absent)
    int64_t ff_W1 = -1, ff_b1 = -1, ff_W2 = -1, ff_b2 = -1, E = -1, Wc1 = -1, bc1 = -1, Wc2 = -1, bc2 = -1;
    std::vector<int64_t> W_agg, W_self, b, b_self;
    std::vector<int> order;   // resolved per layer
    // weight images of the tensor-core GEMMs, kept across the epochs of a training run (host bookkeeping only;
    // the images live in the caller's workspace).  Makes training calls on one model non-reentrant.
    mutable sgcn::TcImageCache* image_cache = nullptr;
    // input aggregate cache: what the first layer's saved A_hat X in the caller's workspace was computed from
    struct InputAggregateKey {
        const void* X = nullptr;
        int64_t x_ld = 0;
        const void* graph = nullptr;
        const void* workspace = nullptr;
        const void* stream = nullptr;
        bool valid = false;
    };
    mutable InputAggregateKey zkey;
    // Per-slice hidden widths that are not a multiple of 4 (fp32) / 8 (bf16) columns -- the paper's own p = 3:
    // ceil(512/3) = 171 -- run on an internal copy of the model whose slices are padded to the next multiple of 8.
    // The padded units have zero weights and biases, so they stay zero through every layer and take no gradient; the
    // caller's parameter layout is unchanged (parameters are copied in, gradients copied out, once per epoch each).
    slicegcn_model* inner = nullptr;
    sgcn::PadTable pad_table;
    int caller_h_s = 0;   // per-slice width of the caller's layout (= h_s unless this is a padded internal model)
    ~slicegcn_model() {
        sgcn::tc_image_cache_destroy(image_cache);
        delete inner;
    }

    int64_t add(const std::string& name, int d0, int d1, int d2) {
        const int64_t off = param_elems;
        tensors.push_back({name, off, {d0, d1, d2}});
        const int64_t cnt = (int64_t)d0 * d1 * d2;
        param_count += cnt;
        param_elems = sgcn::align_up(off + cnt, 4);
        return off;
    }
    int layer_in_width(int l) const { return l == 0 ? (desc.use_ff ? slice_size : slice_width) : h_s; }
    int layer_in_cols(int l) const { return l == 0 ? (desc.use_ff ? slice_size : desc.in_d) : desc.num_slices * h_s; }
    // Direct slicing with slices that are not 8-column aligned, or that overlap (Algorithm 1's shifted last slice):
    // the first layer reads a repacked copy of X -- slices side by side at multiples of repack_pad(), zero padding --
    // so that every kernel sees aligned, disjoint column blocks.  The copy is remade every epoch (X is an argument).
    bool repack_input() const {
        if (desc.use_ff) return false;
        bool need = slice_width % 8 != 0;
        for (int i = 0; i < desc.num_slices; ++i) {
            need = need || starts[i] % 8 != 0;
            if (i > 0) need = need || starts[i] < ends[i - 1];
        }
        return need;
    }
    int repack_pad() const { return (slice_width + 7) / 8 * 8; }
    // Feature fusion reads all of X: when its rows are not 16-byte aligned (or in_d is no multiple of 8) the fusion
    // MLP reads a copy with rows padded to 8 columns, zero padding.
    bool repack_ff_input(int64_t x_ld) const {
        const int64_t esz = desc.dtype == SLICEGCN_BF16 ? 2 : 4;
        return desc.use_ff && ((x_ld * esz) % 16 != 0 || desc.in_d % 8 != 0);
    }
    void layer_in_starts(int l, int* out) const {
        for (int i = 0; i < desc.num_slices; ++i) out[i] = l == 0 ? (desc.use_ff ? 0 : starts[i]) : i * h_s;
    }
};

namespace sgcn {
namespace {

struct EpochLayout {
    // element leading dimensions
    int64_t ld_h = 0, ld_x0 = 0, ld_ffact = 0, ld_cls = 0, ld_grad = 0, ld_dlog = 0;
    int64_t total = 0;
    // pointers (valid when built with a base)
    void* ff_act = nullptr;
    void* xff = nullptr;
    void* xrep = nullptr;        // repacked first-layer input (see slicegcn_model::repack_input)
    int64_t ld_xrep = 0;
    std::vector<void*> H;        // H[l+1], l = 0..L-1
    std::vector<void*> saved;
    std::vector<int64_t> saved_bytes;
    void* cls_act = nullptr;
    // ReLU byte masks of the two MLP hidden layers, used as the gates of their backward products when the
    // activations are far larger than L2 (on smaller problems the activation itself was just read by the preceding
    // weight gradient and gates from L2: measured faster than the mask from DRAM)
    uint8_t* cls_mask = nullptr;
    uint8_t* ff_mask = nullptr;
    int64_t ld_clsm = 0, ld_ffm = 0;
    bool cls_masks = false, ff_masks = false;   // the ReLU of the classifier / of the fusion MLP leaves a byte mask
    float* logits = nullptr;
    float* dlogits = nullptr;
    float* row_loss = nullptr;
    float* dA = nullptr;
    float* dH[2] = {nullptr, nullptr};
    float* dff = nullptr;
    void* ws = nullptr;
    int64_t ws_bytes = 0;
    void* tc_img = nullptr;      // weight images of the dense heads' tensor-core GEMMs
    int64_t tc_img_bytes = 0;
    void* img_cache = nullptr;   // region of the epoch's image cache
    int64_t img_cache_bytes = 0;
};

slicegcn_status_t layer_desc_for(const slicegcn_model* m, int l, const float* params, int64_t x_ld, int* starts_buf,
                                 slicegcn_layer_desc* d) {
    const slicegcn_model_desc& D = m->desc;
    m->layer_in_starts(l, starts_buf);
    d->num_slices = D.num_slices;
    d->in_starts = starts_buf;
    d->in_width = m->layer_in_width(l);
    d->in_cols = m->layer_in_cols(l);
    d->in_ld = l == 0 ? (D.use_ff ? align_up(m->slice_size, 8) : x_ld) : align_up((int64_t)D.num_slices * m->h_s, 8);
    if (l == 0 && m->repack_input()) {   // the first layer reads the repacked copy of X
        const int pad = m->repack_pad();
        for (int i = 0; i < D.num_slices; ++i) starts_buf[i] = i * pad;
        d->in_cols = D.num_slices * pad;
        d->in_ld = (int64_t)D.num_slices * pad;
    }
    d->h_s = m->h_s;
    d->out_ld = align_up((int64_t)D.num_slices * m->h_s, 8);
    d->dtype = D.dtype;
    d->order = m->order[l];
    d->W_agg = params ? params + m->W_agg[l] : reinterpret_cast<const float*>(16);
    d->W_self = D.use_self ? (params ? params + m->W_self[l] : reinterpret_cast<const float*>(16)) : nullptr;
    d->b = params ? params + m->b[l] : nullptr;
    d->b_self = D.use_b_self ? (params ? params + m->b_self[l] : reinterpret_cast<const float*>(16)) : nullptr;
    d->E = (D.use_se && l == D.num_layers - 1) ? (params ? params + m->E : reinterpret_cast<const float*>(16)) : nullptr;
    return SLICEGCN_OK;
}

slicegcn_status_t build_layout(const slicegcn_model* m, const slicegcn_graph* g, int64_t x_ld, char* base,
                               EpochLayout* out) {
    const slicegcn_model_desc& D = m->desc;
    const int64_t n = g->n;
    const int esz = esize(D.dtype);
    const int p = D.num_slices, L = D.num_layers;
    EpochLayout& E = *out;
    Bump b;
    b.base = base;
    E.ld_h = align_up((int64_t)p * m->h_s, 8);
    E.ld_cls = align_up(D.hidden, 8);
    E.ld_ffact = align_up(D.in_d, 8);
    E.ld_x0 = align_up(m->slice_size, 8);
    int64_t gw = E.ld_h;
    if (D.use_ff) gw = std::max(gw, std::max(E.ld_x0, E.ld_ffact));
    E.ld_grad = gw;
    E.ld_clsm = align_up(D.hidden, 16);
    E.ld_ffm = align_up(D.in_d, 16);
    // The ReLUs of the classifier and of the fusion MLP leave a byte mask; their backward products are stored ungated
    // and the consumers multiply by the mask in their producers (see the classifier's backward below).  Without the
    // masks (SLICEGCN_GATE_MASKS=0: the tests reach both forms) the products are gated by the activation in their epilogue.
    // That pays where the consumers' kernels take a mask (probed here with the shapes and leading dimensions of this
    // model; the pointers are aligned stand-ins that nothing dereferences); elsewhere a byte mask is still cheaper
    // to read back than the activation once the activation is far larger than the L2.
    {
        void* const fake = reinterpret_cast<void*>(static_cast<uintptr_t>(1) << 20);
        const bool big = n * E.ld_cls * esz >= ((int64_t)512 << 20);
        WgradArgs w1;   // dWc1 = H^T (dA * mask)
        w1.fault = static_cast<int*>(fake);
        w1.M = n;
        w1.K = p * m->h_s;
        w1.N = D.hidden;
        w1.A = fake;
        w1.lda = E.ld_h;
        w1.a_dtype = D.dtype;
        w1.B = static_cast<const float*>(fake);
        w1.ldb = E.ld_cls;
        w1.dW = static_cast<float*>(fake);
        w1.dbias = static_cast<float*>(fake);
        w1.b_mask = static_cast<const uint8_t*>(fake);
        w1.b_mask_ld = E.ld_clsm;
        GemmArgs h;     // dH = (dA * mask) Wc1^T
        h.fault = static_cast<int*>(fake);
        h.b_image = fake;
        h.b_image_bytes = (int64_t)1 << 60;
        h.M = n;
        h.K = D.hidden;
        h.N = p * m->h_s;
        h.A = fake;
        h.lda = E.ld_cls;
        h.B = static_cast<const float*>(fake);
        h.ldb = D.hidden;
        h.b_trans = 1;
        h.C = fake;
        h.ldc = gw;
        h.a_mask = static_cast<const uint8_t*>(fake);
        h.a_mask_ld = E.ld_clsm;
        E.cls_masks = big || (wgrad_masks_in_producer(w1) && tc_gemm_masks_in_producer(h));
        WgradArgs f1;   // dW1 = X^T (dact * mask) of the fusion MLP
        f1.fault = static_cast<int*>(fake);
        f1.M = n;
        f1.K = D.in_d;
        f1.N = D.in_d;
        f1.A = fake;
        f1.lda = m->repack_ff_input(x_ld) ? align_up(D.in_d, 8) : x_ld;
        f1.a_dtype = D.dtype;
        f1.B = static_cast<const float*>(fake);
        f1.ldb = gw;
        f1.dW = static_cast<float*>(fake);
        f1.dbias = static_cast<float*>(fake);
        f1.b_mask = static_cast<const uint8_t*>(fake);
        f1.b_mask_ld = E.ld_ffm;
        E.ff_masks = D.use_ff && (big || wgrad_masks_in_producer(f1));
        if (const char* force = getenv("SLICEGCN_GATE_MASKS")) E.cls_masks = E.ff_masks = atoi(force) != 0;
    }
    if (D.use_ff) {
        E.ff_act = b.take(n * E.ld_ffact * esz);
        if (E.ff_masks) E.ff_mask = static_cast<uint8_t*>(b.take(n * E.ld_ffm));
        E.xff = b.take(n * E.ld_x0 * esz);
    }
    if (m->repack_input()) {
        E.ld_xrep = (int64_t)p * m->repack_pad();
        E.xrep = b.take(n * E.ld_xrep * esz);
    } else if (m->repack_ff_input(x_ld)) {
        E.ld_xrep = align_up(D.in_d, 8);
        E.xrep = b.take(n * E.ld_xrep * esz);
    }
    int64_t ws_need = 0;
    E.H.resize(L);
    E.saved.resize(L);
    E.saved_bytes.resize(L);
    for (int l = 0; l < L; ++l) {
        int starts[SLICEGCN_MAX_SLICES];
        slicegcn_layer_desc d;
        layer_desc_for(m, l, nullptr, x_ld, starts, &d);
        LayerPlan pl;
        SGCN_TRY(make_plan(g, &d, &pl));
        E.H[l] = b.take(n * E.ld_h * esz);
        E.saved_bytes[l] = pl.zt_bytes + pl.mask_bytes;
        E.saved[l] = b.take(E.saved_bytes[l]);
        ws_need = std::max(ws_need, std::max(layer_fwd_ws_bytes(g, pl), layer_bwd_ws_bytes(g, pl)));
    }
    E.cls_act = b.take(n * E.ld_cls * esz);
    if (E.cls_masks) E.cls_mask = static_cast<uint8_t*>(b.take(n * E.ld_clsm));
    E.logits = static_cast<float*>(b.take(n * (int64_t)D.num_classes * 4));
    E.ld_dlog = align_up(D.num_classes, 4);
    E.dlogits = static_cast<float*>(b.take(n * E.ld_dlog * 4));
    E.row_loss = static_cast<float*>(b.take(n * 4));
    E.dA = static_cast<float*>(b.take(n * E.ld_cls * 4));
    E.dH[0] = static_cast<float*>(b.take(n * E.ld_grad * 4));
    E.dH[1] = static_cast<float*>(b.take(n * E.ld_grad * 4));
    // scratch of the dense heads (weight gradients)
    ws_need = std::max(ws_need, wgrad_scratch_bytes(n, 1, D.hidden, D.num_classes));
    ws_need = std::max(ws_need, wgrad_scratch_bytes(n, 1, p * m->h_s, D.hidden));
    if (D.use_ff) {
        ws_need = std::max(ws_need, wgrad_scratch_bytes(n, 1, D.in_d, m->slice_size));
        ws_need = std::max(ws_need, wgrad_scratch_bytes(n, 1, D.in_d, D.in_d));
    }
    E.ws_bytes = align_up(ws_need, 256);
    E.ws = b.take(E.ws_bytes);
    {
        const int HW = p * m->h_s;
        int64_t img = std::max(tc_image_bytes(1, HW, D.hidden), tc_image_bytes(1, D.hidden, HW));
        img = std::max(img, std::max(tc_image_bytes(1, D.hidden, D.num_classes), tc_image_bytes(1, D.num_classes, D.hidden)));
        if (D.use_ff) {
            img = std::max(img, tc_image_bytes(1, D.in_d, D.in_d));
            img = std::max(img, std::max(tc_image_bytes(1, D.in_d, m->slice_size), tc_image_bytes(1, m->slice_size, D.in_d)));
        }
        E.tc_img_bytes = align_up(img, 256);
        E.tc_img = b.take(E.tc_img_bytes);
        // every distinct weight operand of an epoch once: two heads forward and backward, FF, and per layer the two
        // forward and two backward operands (each at most one image of a layer's size)
        int64_t cache = 4 * E.tc_img_bytes;
        for (int l = 0; l < L; ++l) {
            const int in_w = m->layer_in_width(l);
            cache += 4 * align_up(std::max(tc_image_bytes(p, in_w, m->h_s), tc_image_bytes(p, m->h_s, in_w)), 256);
        }
        if (D.use_ff) cache += 4 * E.tc_img_bytes;
        E.img_cache_bytes = cache;
        E.img_cache = b.take(cache);
    }
    E.total = align_up(b.off, 256);
    return SLICEGCN_OK;
}

}  // namespace
}  // namespace sgcn

using namespace sgcn;

extern "C" {

slicegcn_status_t slicegcn_slice_strategy(int32_t in_d, int32_t p, double scale, int32_t rule, int32_t* starts,
                                          int32_t* ends, int32_t* slice_size) {
    return sgcn::slice_strategy(in_d, p, scale, rule, starts, ends, slice_size);
}

slicegcn_status_t slicegcn_layer_saved_bytes(const slicegcn_graph* g, const slicegcn_layer_desc* d, int64_t* bytes) {
    if (!bytes) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "bytes is NULL");
    LayerPlan pl;
    SGCN_TRY(make_plan(g, d, &pl));
    *bytes = pl.zt_bytes + pl.mask_bytes;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_layer_saved_layout(const slicegcn_graph* g, const slicegcn_layer_desc* d, int64_t* zt_offset,
                                              int64_t* zt_ld, int32_t* zt_cols, int64_t* mask_offset, int64_t* mask_ld) {
    LayerPlan pl;
    SGCN_TRY(make_plan(g, d, &pl));
    if (zt_offset) *zt_offset = 0;
    if (zt_ld) *zt_ld = pl.zt_ld;
    if (zt_cols) *zt_cols = pl.zt_cols;
    if (mask_offset) *mask_offset = pl.zt_bytes;
    if (mask_ld) *mask_ld = pl.mask_ld;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_layer_workspace_bytes(const slicegcn_graph* g, const slicegcn_layer_desc* d, int64_t* bytes) {
    if (!bytes) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "bytes is NULL");
    LayerPlan pl;
    SGCN_TRY(make_plan(g, d, &pl));
    *bytes = std::max(layer_fwd_ws_bytes(g, pl), layer_bwd_ws_bytes(g, pl));
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_layer_forward(const slicegcn_graph* g, const slicegcn_layer_desc* d, const void* H_in,
                                         void* H_out, void* saved, int64_t saved_bytes, void* workspace,
                                         int64_t workspace_bytes, void* stream) {
    LayerPlan pl;
    SGCN_TRY(make_plan(g, d, &pl));
    if (!H_in || !H_out || !saved) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer_forward: NULL tensor");
    if (saved_bytes < pl.zt_bytes + pl.mask_bytes) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "layer_forward: saved buffer too small");
    if (workspace_bytes < layer_fwd_ws_bytes(g, pl) || (!workspace && layer_fwd_ws_bytes(g, pl) > 0))
        SGCN_FAIL(SLICEGCN_ERR_ALLOC, "layer_forward: workspace too small");
    return layer_forward_impl(g, d, pl, H_in, H_out, saved, workspace, workspace_bytes, (cudaStream_t)stream);
}

slicegcn_status_t slicegcn_layer_backward(const slicegcn_graph* g, const slicegcn_layer_desc* d, const void* H_in,
                                          const void* saved, const float* dH_out, int64_t dout_ld, float* dH_in,
                                          int64_t din_ld, float* dW_agg, float* dW_self, float* db, float* db_self,
                                          float* dE, void* workspace, int64_t workspace_bytes, void* stream) {
    LayerPlan pl;
    SGCN_TRY(make_plan(g, d, &pl));
    if (!H_in || !saved || !dH_out || !workspace) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer_backward: NULL tensor");
    if (dout_ld < pl.out_cols || (dH_in && din_ld < pl.in_cols)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "layer_backward: leading dimension too small");
    return layer_backward_impl(g, d, pl, H_in, saved, dH_out, dout_ld, dH_in, din_ld, dW_agg, dW_self, db, db_self, dE,
                               workspace, workspace_bytes, (cudaStream_t)stream);
}

static slicegcn_status_t model_create_impl(const slicegcn_model_desc* desc, int h_s_override, slicegcn_model** out);

slicegcn_status_t slicegcn_model_create(const slicegcn_model_desc* desc, slicegcn_model** out) {
    SGCN_TRY(model_create_impl(desc, 0, out));
    slicegcn_model* m = *out;
    const int unit = m->desc.dtype == SLICEGCN_BF16 ? 8 : 4;
    if (m->h_s % unit == 0) return SLICEGCN_OK;
    // padded internal model: same tensors in the same order, every h_s-sized dimension widened to a multiple of 8
    const int hp = (m->h_s + 7) / 8 * 8;
    slicegcn_model* in = nullptr;
    slicegcn_status_t s = model_create_impl(desc, hp, &in);
    if (s != SLICEGCN_OK || in->tensors.size() != m->tensors.size() || m->tensors.size() > 48) {
        delete in;
        delete m;
        *out = nullptr;
        if (s == SLICEGCN_OK) SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED, "model: too many parameter tensors for the padded layout");
        return s;
    }
    m->inner = in;
    const int p = m->desc.num_slices;
    for (size_t t = 0; t < m->tensors.size(); ++t) {
        const auto& a = m->tensors[t];
        const auto& b = in->tensors[t];
        sgcn::PadEntry e;
        e.outer = a.offset;
        e.inner = b.offset;
        if (a.name == "Wc1") {   // (p*h_s) x hidden: p blocks of h_s rows
            e.blocks = p; e.r = m->h_s; e.c = a.dims[1]; e.rp = hp; e.cp = b.dims[1];
        } else {                 // d0 blocks (slices, or 1) of d1 x d2
            e.blocks = a.dims[0]; e.r = a.dims[1]; e.c = a.dims[2]; e.rp = b.dims[1]; e.cp = b.dims[2];
            if (a.dims[2] == 1 && b.dims[2] == 1 && a.dims[0] == p && b.dims[0] == p && a.name != "ff_b1" && a.name != "ff_b2" &&
                a.name != "bc1" && a.name != "bc2") {   // per-slice vectors p x h_s: one row of h_s columns per slice
                e.r = 1; e.rp = 1; e.c = a.dims[1]; e.cp = b.dims[1];
            }
        }
        m->pad_table.e[m->pad_table.count++] = e;
    }
    return SLICEGCN_OK;
}

static slicegcn_status_t model_create_impl(const slicegcn_model_desc* desc, int h_s_override, slicegcn_model** out) {
    if (!out) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (!desc) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "desc is NULL");
    const slicegcn_model_desc& D = *desc;
    if (D.in_d < 1 || D.hidden < 1 || D.num_layers < 1 || D.num_classes < 1 || D.num_slices < 1 ||
        D.num_slices > SLICEGCN_MAX_SLICES)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "model: sizes must be positive and num_slices <= %d", SLICEGCN_MAX_SLICES);
    if (D.dtype != SLICEGCN_F32 && D.dtype != SLICEGCN_BF16) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "model: bad dtype");
    if (D.order != SLICEGCN_ORDER_AUTO && D.order != SLICEGCN_AGG_FIRST && D.order != SLICEGCN_XFORM_FIRST)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "model: bad order");
    slicegcn_model* m = new (std::nothrow) slicegcn_model();
    if (!m) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "host allocation failed");
    m->desc = D;
    slicegcn_status_t s = sgcn::slice_strategy(D.in_d, D.num_slices, D.slice_size_scale, D.slice_rule, m->starts, m->ends,
                                               &m->slice_size);
    if (s != SLICEGCN_OK) {
        delete m;
        return s;
    }
    m->slice_width = m->ends[0] - m->starts[0];
    m->h_s = (D.hidden + D.num_slices - 1) / D.num_slices;   // each layer scaled down in proportion to p
    m->caller_h_s = m->h_s;
    if (h_s_override > 0) m->h_s = h_s_override;
    const int p = D.num_slices;
    if (D.use_ff) {
        m->ff_W1 = m->add("ff_W1", D.in_d, D.in_d, 1);
        m->ff_b1 = m->add("ff_b1", D.in_d, 1, 1);
        m->ff_W2 = m->add("ff_W2", D.in_d, m->slice_size, 1);
        m->ff_b2 = m->add("ff_b2", m->slice_size, 1, 1);
    }
    for (int l = 0; l < D.num_layers; ++l) {
        const int w_in = m->layer_in_width(l);
        const std::string sfx = "." + std::to_string(l);
        m->W_agg.push_back(m->add("W_agg" + sfx, p, w_in, m->h_s));
        m->W_self.push_back(D.use_self ? m->add("W_self" + sfx, p, w_in, m->h_s) : -1);
        m->b.push_back(m->add("b" + sfx, p, m->h_s, 1));
        m->b_self.push_back(D.use_b_self ? m->add("b_self" + sfx, p, m->h_s, 1) : -1);
        int order = D.order;
        if (order == SLICEGCN_ORDER_AUTO)
            order = m->layer_in_cols(l) <= p * m->h_s ? SLICEGCN_AGG_FIRST : SLICEGCN_XFORM_FIRST;
        m->order.push_back(order);
    }
    if (D.use_se) m->E = m->add("E", p, m->h_s, 1);
    m->Wc1 = m->add("Wc1", p * m->h_s, D.hidden, 1);
    m->bc1 = m->add("bc1", D.hidden, 1, 1);
    m->Wc2 = m->add("Wc2", D.hidden, D.num_classes, 1);
    m->bc2 = m->add("bc2", D.num_classes, 1, 1);
    *out = m;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_destroy(slicegcn_model* m) {
    delete m;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_invalidate_caches(const slicegcn_model* m) {
    if (!m) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "model is NULL");
    m->zkey.valid = false;
    if (m->inner) m->inner->zkey.valid = false;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_param_count(const slicegcn_model* m, int64_t* count) {
    if (!m || !count) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "NULL argument");
    *count = m->param_count;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_param_elems(const slicegcn_model* m, int64_t* elems) {
    if (!m || !elems) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "NULL argument");
    *elems = m->param_elems;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_num_tensors(const slicegcn_model* m, int32_t* count) {
    if (!m || !count) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "NULL argument");
    *count = (int32_t)m->tensors.size();
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_tensor_info(const slicegcn_model* m, int32_t t, char name[32], int64_t* offset,
                                             int32_t dims[3]) {
    if (!m || t < 0 || t >= (int32_t)m->tensors.size()) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "bad tensor index");
    const auto& T = m->tensors[t];
    if (name) {
        std::strncpy(name, T.name.c_str(), 31);
        name[31] = 0;
    }
    if (offset) *offset = T.offset;
    if (dims)
        for (int i = 0; i < 3; ++i) dims[i] = T.dims[i];
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_slices(const slicegcn_model* m, int32_t* starts, int32_t* ends, int32_t* slice_size,
                                        int32_t* h_s) {
    if (!m) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "model is NULL");
    for (int i = 0; i < m->desc.num_slices; ++i) {
        if (starts) starts[i] = m->starts[i];
        if (ends) ends[i] = m->ends[i];
    }
    if (slice_size) *slice_size = m->slice_size;
    if (h_s) *h_s = m->h_s;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_model_layer_order(const slicegcn_model* m, int32_t layer, int32_t* order) {
    if (!m || !order || layer < 0 || layer >= m->desc.num_layers) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "bad argument");
    *order = (m->inner ? m->inner : m)->order[layer];   // the order that actually runs
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_train_workspace_bytes(const slicegcn_model* m, const slicegcn_graph* g, int64_t* bytes) {
    if (!m || !g || !bytes) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "NULL argument");
    EpochLayout E;
    SGCN_TRY(build_layout(m->inner ? m->inner : m, g, m->desc.in_d, nullptr, &E));
    *bytes = E.total;
    if (m->inner) *bytes += 2 * align_up(m->inner->param_elems * (int64_t)sizeof(float), 256);   // padded parameters and gradients
    return SLICEGCN_OK;
}

// The slices this process computes and how their outputs meet the other processes' (slicegcn_train_epoch_sliced).
struct SliceRange {
    int begin, end;
    slicegcn_exchange_fn exchange;
    void* ctx;
};

// forward_only: stops after the logits (evaluation pass); labels, grads and the optimiser arguments are not used.
static slicegcn_status_t epoch_impl(bool forward_only, const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                    const int32_t* labels, const int32_t* train_idx, int64_t n_train, float* params,
                                    float* grads, float* adam_m, float* adam_v, const slicegcn_opt_desc* opt,
                                    float* logits_out, float* loss_out, void* workspace, int64_t workspace_bytes,
                                    void* stream, const slicegcn_dropout_desc* drop = nullptr, const SliceRange* sr = nullptr) {
    if (!m || !g || !X || !params || !workspace || (!forward_only && (!labels || !grads)))
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: NULL argument");
    if (sr && (m->inner || drop || forward_only))
        SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED, "train_epoch_sliced: not with dropout or per-slice widths that need the padded layout");
    if (m->inner) {
        // padded internal model: parameters in, the whole iteration on the padded shapes, gradients out, then the update
        // on the caller's buffers
        if (opt && (!adam_m || !adam_v)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: optimiser state is NULL");
        if (opt && (opt->total_epochs < 1 || opt->epoch < 0)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: bad epoch");
        cudaStream_t st = (cudaStream_t)stream;
        const int64_t pbytes = align_up(m->inner->param_elems * (int64_t)sizeof(float), 256);
        if (workspace_bytes < 2 * pbytes) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "train_epoch: workspace too small");
        float* pin = static_cast<float*>(workspace);
        float* gin = reinterpret_cast<float*>(static_cast<char*>(workspace) + pbytes);
        void* iws = static_cast<char*>(workspace) + 2 * pbytes;
        SGCN_TRY(pad_params_run(m->pad_table, true, params, pin, st));
        SGCN_TRY(epoch_impl(forward_only, m->inner, g, X, x_ld, labels, train_idx, n_train, pin, gin, nullptr, nullptr, nullptr,
                            logits_out, loss_out, iws, workspace_bytes - 2 * pbytes, stream, drop));
        if (forward_only) return SLICEGCN_OK;
        SGCN_CUDA(cudaMemsetAsync(grads, 0, sizeof(float) * m->param_elems, st));
        SGCN_TRY(pad_params_run(m->pad_table, false, gin, grads, st));
        if (opt) {
            const double kPi = 3.14159265358979323846;
            const double lr = opt->lr0 * 0.5 * (1.0 + std::cos(kPi * (double)opt->epoch / (double)opt->total_epochs));
            SGCN_TRY(adam_run(m->param_elems, params, grads, adam_m, adam_v, (float)lr, (float)opt->beta1, (float)opt->beta2,
                              (float)opt->eps, (float)opt->weight_decay, opt->epoch + 1, st));
        }
        return SLICEGCN_OK;
    }
    const slicegcn_model_desc& D = m->desc;
    if (x_ld < D.in_d) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: x_ld < in_d");
    if (opt && (!adam_m || !adam_v)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: optimiser state is NULL");
    if (opt && (opt->total_epochs < 1 || opt->epoch < 0)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: bad epoch");
    if (train_idx && n_train < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: empty training set");
    float drop_scale = 1.f;
    if (drop) {
        if (!(drop->rate >= 0.0 && drop->rate < 1.0)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: dropout rate outside [0, 1)");
        if (D.num_layers > 1 && (!drop->masks || drop->mask_ld < (int64_t)D.num_slices * m->caller_h_s))
            SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: dropout masks missing or mask_ld too small");
        for (int l = 0; l + 1 < D.num_layers; ++l)
            if (!drop->masks[l]) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch: dropout mask %d is NULL", l);
        drop_scale = (float)(1.0 / (1.0 - drop->rate));
    }
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n = g->n;
    const int p = D.num_slices, L = D.num_layers, C = D.num_classes;
    // the slices computed here: all of them, or this process's range (Section IV-A's placement)
    const int s0 = sr ? sr->begin : 0, s1 = sr ? sr->end : p, pl = s1 - s0;
    if (s0 < 0 || s1 > p || pl < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch_sliced: slice range outside [0, p)");
    const bool partial = pl != p;
    if (partial && !sr->exchange) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch_sliced: a partial range needs an exchange function");
    EpochLayout E;
    SGCN_TRY(build_layout(m, g, x_ld, static_cast<char*>(workspace), &E));
    if (workspace_bytes < E.total)
        SGCN_FAIL(SLICEGCN_ERR_ALLOC, "train_epoch: workspace too small (%lld < %lld)", (long long)workspace_bytes,
                  (long long)E.total);
    if (!forward_only) SGCN_CUDA(cudaMemsetAsync(grads, 0, sizeof(float) * m->param_elems, st));
    // weight images: everything recorded by earlier epochs of this run is converted now, in one launch
    if (!m->image_cache) m->image_cache = tc_image_cache_create();
    struct CacheScope {
        ~CacheScope() { tc_image_cache_end(); }
    } cache_scope;
    SGCN_TRY(tc_image_cache_begin(m->image_cache, E.img_cache, E.img_cache_bytes, params, m->param_elems, st));

    // ---------------- forward
    const void* h0 = X;
    int64_t ld0 = x_ld;
    if (D.use_ff && (m->slice_size % 8) != 0)
        SGCN_CUDA(cudaMemsetAsync(E.xff, 0, n * E.ld_x0 * esize(D.dtype), st));
    // the hidden activation of the fusion MLP is narrower than its rows: keep the padding columns at zero so that the
    // aligned kernels can read it (it is rewritten below, padding excluded)
    const bool ffact_pad = D.use_ff && (D.in_d % 8) != 0;
    if (ffact_pad) SGCN_CUDA(cudaMemsetAsync(E.ff_act, 0, n * E.ld_ffact * esize(D.dtype), st));
    const void* xin = X;          // what the fusion MLP reads
    int64_t xin_ld = x_ld;
    // What a caller who set cache_input_aggregate promises not to change between calls: X (and the workspace).  When
    // this call sees the X, graph, workspace and stream of the previous one, everything computed from X alone is still
    // in the workspace: the padded copy of X below, the repacked slices and the first layer's aggregate further down.
    const bool x_unchanged = !sr && D.cache_input_aggregate && m->zkey.valid && m->zkey.X == X && m->zkey.x_ld == x_ld && m->zkey.graph == g &&
                             m->zkey.workspace == workspace && m->zkey.stream == stream;
    m->zkey.valid = false;   // until this call has queued the first layer
    const bool ff_repacked = m->repack_ff_input(x_ld);
    if (ff_repacked) {
        const int zero = 0;
        if (!x_unchanged)
            SGCN_TRY(repack_slices_run(n, 1, &zero, D.in_d, (int)E.ld_xrep, X, x_ld, D.dtype, E.xrep, E.ld_xrep, st));
        xin = E.xrep;
        xin_ld = E.ld_xrep;
    }
    if (D.use_ff) {   // X_ff = ReLU(X W1 + b1) W2 + b2  (Eq. 4 / Algorithm 3)
        GemmArgs a;
        a.fault = g->fault;
        a.b_image = E.tc_img;
        a.b_image_bytes = E.tc_img_bytes;
        a.M = n;
        a.K = D.in_d;
        a.N = D.in_d;
        a.A = xin;
        a.lda = xin_ld;
        a.a_pad_zero = ff_repacked ? 1 : 0;
        a.a_dtype = D.dtype;
        a.B = params + m->ff_W1;
        a.ldb = D.in_d;
        a.bias = params + m->ff_b1;
        a.relu = 1;
        if (E.ff_masks) {
            a.mask_out = E.ff_mask;
            a.mask_ld = E.ld_ffm;
        }
        a.C = E.ff_act;
        a.ldc = E.ld_ffact;
        a.c_dtype = D.dtype;
        SGCN_TRY(gemm_run(a, st));
        GemmArgs c;
        c.fault = g->fault;
        c.b_image = E.tc_img;
        c.b_image_bytes = E.tc_img_bytes;
        c.M = n;
        c.K = D.in_d;
        c.N = m->slice_size;
        c.A = E.ff_act;
        c.lda = E.ld_ffact;
        c.a_pad_zero = ffact_pad ? 1 : 0;
        c.a_dtype = D.dtype;
        c.B = params + m->ff_W2;
        c.ldb = m->slice_size;
        c.bias = params + m->ff_b2;
        c.C = E.xff;
        c.ldc = E.ld_x0;
        c.c_dtype = D.dtype;
        c.c_pad_write = 1;   // an odd slice width (13 columns): the tile's padding columns are stored too, as zeros
        SGCN_TRY(gemm_run(c, st));
        h0 = E.xff;
        ld0 = E.ld_x0;
    }
    // Input aggregate cache: with direct slicing the first layer's A_hat X does not change from epoch to epoch
    // (Algorithm 3 slices outside the epoch loop); reuse what the previous call left in the workspace.
    const bool z_cacheable = D.cache_input_aggregate && !D.use_ff && m->order[0] == SLICEGCN_AGG_FIRST;
    const bool z_cached = z_cacheable && x_unchanged;
    const bool repacked = m->repack_input();
    if (repacked && x_unchanged) {   // the repacked copy is still in the workspace as well
        h0 = E.xrep;
        ld0 = E.ld_xrep;
    } else if (repacked) {   // slicing (Algorithm 2) as a copy: slices side by side at aligned starts, zero padding
        SGCN_TRY(repack_slices_run(n, p, m->starts, m->slice_width, m->repack_pad(), X, x_ld, D.dtype, E.xrep, E.ld_xrep, st));
        h0 = E.xrep;
        ld0 = E.ld_xrep;
    }
    std::vector<slicegcn_layer_desc> descs(L);
    std::vector<LayerPlan> plans(L);
    std::vector<std::vector<int>> starts(L, std::vector<int>(SLICEGCN_MAX_SLICES));
    std::vector<int> win(L, 0);   // first input column of each layer's window (0 unless this process computes a range of the slices)
    const void* hin = h0;
    for (int l = 0; l < L; ++l) {
        layer_desc_for(m, l, params, x_ld, starts[l].data(), &descs[l]);
        if (l == 0) descs[l].in_ld = ld0;
        if (partial) {   // this process's slices: their blocks of the per-slice tensors, and as the layer's input the
                         // window of columns they read (so that the layer sees slices tiling its input, as always)
            slicegcn_layer_desc& d = descs[l];
            const int64_t wblock = (int64_t)d.in_width * d.h_s;
            int lo = starts[l][s0], hi = starts[l][s0] + d.in_width;
            for (int i = s0; i < s1; ++i) {
                lo = std::min(lo, starts[l][i]);
                hi = std::max(hi, starts[l][i] + d.in_width);
            }
            for (int i = 0; i < pl; ++i) starts[l][i] = starts[l][s0 + i] - lo;
            win[l] = lo;
            d.in_cols = hi - lo;
            d.num_slices = pl;
            d.W_agg += s0 * wblock;
            if (d.W_self) d.W_self += s0 * wblock;
            if (d.b) d.b += s0 * d.h_s;
            if (d.b_self) d.b_self += s0 * d.h_s;
            if (d.E) d.E += s0 * d.h_s;
        }
        SGCN_TRY(make_plan(g, &descs[l], &plans[l]));
        if (l == 0 && repacked) {
            // padding columns of the copy are zero, and so are those of its aggregate
            plans[l].in_pad_zero = true;
            if (plans[l].order == SLICEGCN_AGG_FIRST) plans[l].zt_pad_zero = true;
        }
        if (l == 0 && D.use_ff) plans[l].din_pad_write = true;   // dX_ff lives in the step's own gradient buffer
        if (l == 0 && D.use_ff && (m->slice_size % 8) != 0) {
            // the fused input is narrower than its leading dimension: keep the padding columns of X_ff and of
            // the saved intermediate at zero (both buffers are fully rewritten below, padding excluded)
            plans[l].in_pad_zero = true;
            if (plans[l].order == SLICEGCN_AGG_FIRST) {
                plans[l].zt_pad_zero = true;
                SGCN_CUDA(cudaMemsetAsync(E.saved[l], 0, plans[l].zt_bytes, st));
            }
        }
        // (a partial range writes its own column block of the layer's output; the layers below the last never read
        // another process's columns)
        SGCN_TRY(layer_forward_impl(g, &descs[l], plans[l], static_cast<const char*>(hin) + (int64_t)win[l] * esize(D.dtype),
                                    static_cast<char*>(E.H[l]) + (int64_t)s0 * m->h_s * esize(D.dtype),
                                    E.saved[l], E.ws, E.ws_bytes, st, l == 0 && z_cached));
        if (l == 0 && D.cache_input_aggregate && !sr) {
            m->zkey.X = X;
            m->zkey.x_ld = x_ld;
            m->zkey.graph = g;
            m->zkey.workspace = workspace;
            m->zkey.stream = stream;
            m->zkey.valid = true;
        }
        if (drop && l + 1 < L)   // dropout on what the next layer reads (placement: see slicegcn_train_epoch_dropout)
            SGCN_TRY(dropout_apply_run(n, p * m->h_s, E.H[l], E.ld_h, D.dtype, drop->masks[l], drop->mask_ld, m->caller_h_s, m->h_s,
                                       drop_scale, st));
        hin = E.H[l];
    }
    const int HW = p * m->h_s;
    if (partial)   // Eq. 8: the one exchange of the forward pass -- every process ends up with all slices' outputs
        SGCN_TRY(sr->exchange(sr->ctx, SLICEGCN_EXCHANGE_GATHER_H, E.H[L - 1], n, E.ld_h, s0 * m->h_s, pl * m->h_s, D.dtype, stream));
    float* logits = logits_out ? logits_out : E.logits;
    {   // classifier (Eq. 9)
        GemmArgs a;
        a.fault = g->fault;
        a.b_image = E.tc_img;
        a.b_image_bytes = E.tc_img_bytes;
        a.M = n;
        a.K = HW;
        a.N = D.hidden;
        a.A = hin;
        a.lda = E.ld_h;
        a.a_dtype = D.dtype;
        a.B = params + m->Wc1;
        a.ldb = D.hidden;
        a.bias = params + m->bc1;
        a.relu = 1;
        if (E.cls_masks) {
            a.mask_out = E.cls_mask;
            a.mask_ld = E.ld_clsm;
        }
        a.C = E.cls_act;
        a.ldc = E.ld_cls;
        a.c_dtype = D.dtype;
        SGCN_TRY(gemm_run(a, st));
        GemmArgs c;
        c.fault = g->fault;
        c.b_image = E.tc_img;
        c.b_image_bytes = E.tc_img_bytes;
        c.M = n;
        c.K = D.hidden;
        c.N = C;
        c.A = E.cls_act;
        c.lda = E.ld_cls;
        c.a_dtype = D.dtype;
        c.B = params + m->Wc2;
        c.ldb = C;
        c.bias = params + m->bc2;
        c.C = logits;
        c.ldc = C;
        c.c_dtype = SLICEGCN_F32;
        c.reverse = 1;   // the hidden activation was just written upwards
        SGCN_TRY(gemm_run(c, st));
    }
    if (forward_only) return SLICEGCN_OK;
    // ---------------- loss (Eq. 10) and its gradient
    SGCN_TRY(softmax_ce_run(n, C, logits, labels, train_idx, n_train, E.dlogits, E.ld_dlog, E.row_loss, loss_out, g->fault, st));

    // ---------------- backward
    {
        WgradArgs w;
        w.fault = g->fault;
        w.M = n;
        w.K = D.hidden;
        w.N = C;
        w.A = E.cls_act;
        w.lda = E.ld_cls;
        w.a_dtype = D.dtype;
        w.B = E.dlogits;
        w.ldb = E.ld_dlog;
        w.b_pad_zero = 1;
        w.dW = grads + m->Wc2;
        w.dbias = grads + m->bc2;
        SGCN_TRY(wgrad_run(w, E.ws, E.ws_bytes, st));
        GemmArgs a;   // dA = (dlogits Wc2^T) * (cls_act > 0)
        a.fault = g->fault;
        a.b_image = E.tc_img;
        a.b_image_bytes = E.tc_img_bytes;
        a.M = n;
        a.K = C;
        a.N = D.hidden;
        a.A = E.dlogits;
        a.lda = E.ld_dlog;
        a.a_pad_zero = 1;
        a.B = params + m->Wc2;
        a.ldb = C;
        a.b_trans = 1;
        a.C = E.dA;
        a.ldc = E.ld_cls;
        a.mul_pos = E.cls_act;
        a.mul_pos_ld = E.ld_cls;
        a.mul_pos_dtype = D.dtype;
        if (E.cls_masks) {   // the byte mask of the forward ReLU: a quarter (bf16: half) of the activation's bytes
            a.mul_pos = E.cls_mask;
            a.mul_pos_ld = E.ld_clsm;
            a.mul_pos_dtype = kGateBytes;
        }
        a.reverse = 1;
        WgradArgs w1;
        w1.fault = g->fault;
        w1.M = n;
        w1.K = HW;
        w1.N = D.hidden;
        w1.A = hin;
        w1.lda = E.ld_h;
        w1.a_dtype = D.dtype;
        w1.B = E.dA;
        w1.ldb = E.ld_cls;
        w1.dW = grads + m->Wc1;
        w1.dbias = grads + m->bc1;
        GemmArgs h;   // dH = dA Wc1^T
        h.fault = g->fault;
        h.b_image = E.tc_img;
        h.b_image_bytes = E.tc_img_bytes;
        h.M = n;
        h.K = D.hidden;
        h.N = HW;
        h.A = E.dA;
        h.lda = E.ld_cls;
        h.B = params + m->Wc1;
        h.ldb = D.hidden;
        h.b_trans = 1;
        h.C = E.dH[0];
        h.ldc = E.ld_grad;
        if (E.cls_masks) {
            // A gate read in the epilogue costs that product two thirds of its time (its loads queue behind the
            // epilogue's own stores: 421 us with the gate against 140 us without, on a fifth of the largest
            // workload).  Both consumers of dA can multiply by the byte mask on their operand's way to the tensor
            // cores instead (a mask tile travels next to every slab), so dA is stored ungated.
            WgradArgs w1m = w1;
            w1m.b_mask = E.cls_mask;
            w1m.b_mask_ld = E.ld_clsm;
            GemmArgs hm = h;
            hm.a_mask = E.cls_mask;
            hm.a_mask_ld = E.ld_clsm;
            if (wgrad_masks_in_producer(w1m) && tc_gemm_masks_in_producer(hm)) {
                a.mul_pos = nullptr;
                w1 = w1m;
                h = hm;
            }
        }
        SGCN_TRY(gemm_run(a, st));
        SGCN_TRY(wgrad_run(w1, E.ws, E.ws_bytes, st));
        SGCN_TRY(gemm_run(h, st));
    }
    int cur = 0;
    for (int l = L - 1; l >= 0; --l) {
        const void* lin = l == 0 ? h0 : E.H[l - 1];
        const bool need_din = l > 0 || D.use_ff;
        if (drop && l + 1 < L)   // the gradient passes the same mask and scale on its way into the layer
            SGCN_TRY(dropout_apply_run(n, p * m->h_s, E.dH[cur], E.ld_grad, SLICEGCN_F32, drop->masks[l], drop->mask_ld, m->caller_h_s,
                                       m->h_s, drop_scale, st));
        // (s0 = 0 unless this process computes a range of the slices: then its column block of the incoming
        // gradient and its blocks of the per-slice gradient tensors)
        const int64_t wb = (int64_t)s0 * descs[l].in_width * m->h_s, vb = (int64_t)s0 * m->h_s;
        SGCN_TRY(layer_backward_impl(g, &descs[l], plans[l], static_cast<const char*>(lin) + (int64_t)win[l] * esize(D.dtype), E.saved[l],
                                     E.dH[cur] + vb, E.ld_grad, need_din ? E.dH[cur ^ 1] + win[l] : nullptr, E.ld_grad,
                                     grads + m->W_agg[l] + wb,
                                     D.use_self ? grads + m->W_self[l] + wb : nullptr, grads + m->b[l] + vb,
                                     D.use_b_self ? grads + m->b_self[l] + vb : nullptr,
                                     (D.use_se && l == L - 1) ? grads + m->E + vb : nullptr, E.ws, E.ws_bytes, st));
        cur ^= 1;
    }
    if (D.use_ff) {   // backward of the fusion MLP from dX_ff (sum over slices already formed)
        float* dxff = E.dH[cur];
        if (partial)   // every slice reads X_ff: the other processes' slices contribute too
            SGCN_TRY(sr->exchange(sr->ctx, SLICEGCN_EXCHANGE_SUM_DXFF, dxff, n, E.ld_grad, 0, m->slice_size, SLICEGCN_F32, stream));
        // aggregate-first first layer: its backward kept the padding columns of dX_ff at zero (see din_pad_write)
        const bool dxff_pad = plans[0].order == SLICEGCN_AGG_FIRST && pl > 1 && align_up(m->slice_size, 4) <= E.ld_grad &&
                              align_up(m->slice_size, 4) <= plans[0].zt_ld;
        WgradArgs w;
        w.fault = g->fault;
        w.M = n;
        w.K = D.in_d;
        w.N = m->slice_size;
        w.A = E.ff_act;
        w.lda = E.ld_ffact;
        w.a_pad_zero = ffact_pad ? 1 : 0;
        w.a_dtype = D.dtype;
        w.B = dxff;
        w.ldb = E.ld_grad;
        w.b_pad_zero = dxff_pad ? 1 : 0;
        w.dW = grads + m->ff_W2;
        w.dbias = grads + m->ff_b2;
        SGCN_TRY(wgrad_run(w, E.ws, E.ws_bytes, st));
        float* dact = E.dH[cur ^ 1];
        GemmArgs a;
        a.fault = g->fault;
        a.b_image = E.tc_img;
        a.b_image_bytes = E.tc_img_bytes;
        a.M = n;
        a.K = m->slice_size;
        a.N = D.in_d;
        a.A = dxff;
        a.lda = E.ld_grad;
        a.a_pad_zero = dxff_pad ? 1 : 0;
        a.B = params + m->ff_W2;
        a.ldb = m->slice_size;
        a.b_trans = 1;
        a.C = dact;
        a.ldc = E.ld_grad;
        a.mul_pos = E.ff_act;
        a.mul_pos_ld = E.ld_ffact;
        a.mul_pos_dtype = D.dtype;
        if (E.ff_masks) {
            a.mul_pos = E.ff_mask;
            a.mul_pos_ld = E.ld_ffm;
            a.mul_pos_dtype = kGateBytes;
        }
        WgradArgs w1;
        w1.fault = g->fault;
        w1.M = n;
        w1.K = D.in_d;
        w1.N = D.in_d;
        w1.A = xin;
        w1.lda = xin_ld;
        w1.a_pad_zero = ff_repacked ? 1 : 0;
        w1.a_dtype = D.dtype;
        w1.B = dact;
        w1.ldb = E.ld_grad;
        w1.dW = grads + m->ff_W1;
        w1.dbias = grads + m->ff_b1;
        if (E.ff_masks) {   // as for the classifier: the one consumer of this gradient applies the mask itself
            WgradArgs w1m = w1;
            w1m.b_mask = E.ff_mask;
            w1m.b_mask_ld = E.ld_ffm;
            if (wgrad_masks_in_producer(w1m)) {
                a.mul_pos = nullptr;
                w1 = w1m;
            }
        }
        SGCN_TRY(gemm_run(a, st));
        SGCN_TRY(wgrad_run(w1, E.ws, E.ws_bytes, st));
    }
    if (partial) {
        // The replicated tensors (fusion MLP, classifier) got the same gradient on every process: all but the one with
        // the first slice clear theirs, so that the sum over processes is the full gradient everywhere.
        if (s0 != 0)
            for (const auto& t : m->tensors)
                if (t.name.rfind("ff_", 0) == 0 || t.name == "Wc1" || t.name == "bc1" || t.name == "Wc2" || t.name == "bc2")
                    SGCN_CUDA(cudaMemsetAsync(grads + t.offset, 0, sizeof(float) * (size_t)t.dims[0] * t.dims[1] * t.dims[2], st));
        SGCN_TRY(sr->exchange(sr->ctx, SLICEGCN_EXCHANGE_SUM_GRADS, grads, m->param_elems, 1, 0, 1, SLICEGCN_F32, stream));
    }
    // ---------------- update: Adam, cosine-annealed learning rate, one step per epoch
    if (opt) {
        const double kPi = 3.14159265358979323846;
        const double lr = opt->lr0 * 0.5 * (1.0 + std::cos(kPi * (double)opt->epoch / (double)opt->total_epochs));
        SGCN_TRY(adam_run(m->param_elems, params, grads, adam_m, adam_v, (float)lr, (float)opt->beta1, (float)opt->beta2,
                          (float)opt->eps, (float)opt->weight_decay, opt->epoch + 1, st));
    }
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_train_epoch(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                       const int32_t* labels, const int32_t* train_idx, int64_t n_train, float* params,
                                       float* grads, float* adam_m, float* adam_v, const slicegcn_opt_desc* opt,
                                       float* logits_out, float* loss_out, void* workspace, int64_t workspace_bytes,
                                       void* stream) {
    return epoch_impl(false, m, g, X, x_ld, labels, train_idx, n_train, params, grads, adam_m, adam_v, opt, logits_out, loss_out,
                      workspace, workspace_bytes, stream);
}

slicegcn_status_t slicegcn_train_epoch_sliced(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                              const int32_t* labels, const int32_t* train_idx, int64_t n_train,
                                              float* params, float* grads, float* adam_m, float* adam_v,
                                              const slicegcn_opt_desc* opt, int32_t slice_begin, int32_t slice_end,
                                              slicegcn_exchange_fn exchange, void* exchange_ctx, float* logits_out,
                                              float* loss_out, void* workspace, int64_t workspace_bytes, void* stream) {
    const SliceRange sr{slice_begin, slice_end, exchange, exchange_ctx};
    return epoch_impl(false, m, g, X, x_ld, labels, train_idx, n_train, params, grads, adam_m, adam_v, opt, logits_out, loss_out,
                      workspace, workspace_bytes, stream, nullptr, &sr);
}

slicegcn_status_t slicegcn_train_epoch_dropout(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                               const int32_t* labels, const int32_t* train_idx, int64_t n_train,
                                               float* params, float* grads, float* adam_m, float* adam_v,
                                               const slicegcn_opt_desc* opt, const slicegcn_dropout_desc* drop,
                                               float* logits_out, float* loss_out, void* workspace, int64_t workspace_bytes,
                                               void* stream) {
    return epoch_impl(false, m, g, X, x_ld, labels, train_idx, n_train, params, grads, adam_m, adam_v, opt, logits_out, loss_out,
                      workspace, workspace_bytes, stream, drop);
}

slicegcn_status_t slicegcn_forward_logits(const slicegcn_model* m, const slicegcn_graph* g, const void* X, int64_t x_ld,
                                          const float* params, float* logits_out, void* workspace, int64_t workspace_bytes,
                                          void* stream) {
    if (!logits_out) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "forward_logits: logits_out is NULL");
    return epoch_impl(true, m, g, X, x_ld, nullptr, nullptr, 0, const_cast<float*>(params), nullptr, nullptr, nullptr, nullptr,
                      logits_out, nullptr, workspace, workspace_bytes, stream);
}

// The labels of the host-buffer entry points are readable here: every one must name a class.
static slicegcn_status_t check_labels_host(const int32_t* labels, int64_t n, int C, const char* who) {
    for (int64_t i = 0; i < n; ++i)
        if (labels[i] < 0 || labels[i] >= C)
            SGCN_FAIL(SLICEGCN_ERR_OUT_OF_RANGE, "%s: label %d of node %lld is outside [0, %d)", who, labels[i], (long long)i, C);
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_train_epoch_host(const slicegcn_model* m, const slicegcn_graph* g, const void* X_host, int64_t x_ld,
                                            const int32_t* labels_host, void* X_stage, int32_t* labels_stage,
                                            const int32_t* train_idx, int64_t n_train, float* params, float* grads,
                                            float* adam_m, float* adam_v, const slicegcn_opt_desc* opt, float* loss_dev,
                                            float* loss_host, void* workspace, int64_t workspace_bytes, void* stream) {
    if (!m || !g || !X_host || !labels_host || !X_stage || !labels_stage || !loss_dev)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch_host: NULL argument");
    if (x_ld < m->desc.in_d) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epoch_host: x_ld < in_d");
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n = g->n;
    SGCN_TRY(check_labels_host(labels_host, n, m->desc.num_classes, "train_epoch_host"));
    slicegcn_model_invalidate_caches(m);   // X is copied anew: nothing computed from the staging buffer's old contents may be reused
    SGCN_CUDA(cudaMemcpyAsync(X_stage, X_host, (size_t)(n * x_ld) * esize(m->desc.dtype), cudaMemcpyHostToDevice, st));
    SGCN_CUDA(cudaMemcpyAsync(labels_stage, labels_host, (size_t)n * sizeof(int32_t), cudaMemcpyHostToDevice, st));
    SGCN_TRY(slicegcn_train_epoch(m, g, X_stage, x_ld, labels_stage, train_idx, n_train, params, grads, adam_m, adam_v, opt, nullptr,
                                  loss_dev, workspace, workspace_bytes, stream));
    if (loss_host) SGCN_CUDA(cudaMemcpyAsync(loss_host, loss_dev, sizeof(float), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_train_epochs_host(const slicegcn_model* m, const slicegcn_graph* g, const void* X_host, int64_t x_ld,
                                             const int32_t* labels_host, void* X_stage0, void* X_stage1, int32_t* labels_stage0,
                                             int32_t* labels_stage1, const int32_t* train_idx, int64_t n_train, float* params,
                                             float* grads, float* adam_m, float* adam_v, const slicegcn_opt_desc* opt,
                                             int32_t num_epochs, float* losses_dev, float* losses_host, void* workspace,
                                             int64_t workspace_bytes, void* stream) {
    if (!m || !g || !X_host || !labels_host || !X_stage0 || !X_stage1 || !labels_stage0 || !labels_stage1 || !losses_dev || !opt)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epochs_host: NULL argument");
    if (x_ld < m->desc.in_d) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epochs_host: x_ld < in_d");
    if (num_epochs < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "train_epochs_host: num_epochs < 1");
    cudaStream_t st = (cudaStream_t)stream;
    const int64_t n = g->n;
    SGCN_TRY(check_labels_host(labels_host, n, m->desc.num_classes, "train_epochs_host"));
    const size_t x_bytes = (size_t)(n * x_ld) * esize(m->desc.dtype), y_bytes = (size_t)n * sizeof(int32_t);
    void* xs[2] = {X_stage0, X_stage1};
    int32_t* ys[2] = {labels_stage0, labels_stage1};
    cudaStream_t copy = nullptr;
    cudaEvent_t ready[2] = {nullptr, nullptr}, done[2] = {nullptr, nullptr};
    slicegcn_status_t rc = SLICEGCN_OK;
    auto cleanup = [&]() {
        for (int i = 0; i < 2; ++i) {
            if (ready[i]) cudaEventDestroy(ready[i]);
            if (done[i]) cudaEventDestroy(done[i]);
        }
        if (copy) cudaStreamDestroy(copy);
    };
    auto run = [&]() -> slicegcn_status_t {
        SGCN_CUDA(cudaStreamCreateWithFlags(&copy, cudaStreamNonBlocking));
        for (int i = 0; i < 2; ++i) {
            SGCN_CUDA(cudaEventCreateWithFlags(&ready[i], cudaEventDisableTiming));
            SGCN_CUDA(cudaEventCreateWithFlags(&done[i], cudaEventDisableTiming));
        }
        // the copies may not start before work already queued on the caller's stream has finished
        // with the staging buffers
        SGCN_CUDA(cudaEventRecord(done[0], st));
        SGCN_CUDA(cudaStreamWaitEvent(copy, done[0], 0));
        auto stage = [&](int b) -> slicegcn_status_t {
            SGCN_CUDA(cudaMemcpyAsync(xs[b], X_host, x_bytes, cudaMemcpyHostToDevice, copy));
            SGCN_CUDA(cudaMemcpyAsync(ys[b], labels_host, y_bytes, cudaMemcpyHostToDevice, copy));
            SGCN_CUDA(cudaEventRecord(ready[b], copy));
            return SLICEGCN_OK;
        };
        SGCN_TRY(stage(0));
        for (int e = 0; e < num_epochs; ++e) {
            const int b = e & 1;
            if (e + 1 < num_epochs) {
                // buffer b^1 was read by epoch e-1, which the caller's stream has been told to mark as done
                if (e >= 1) SGCN_CUDA(cudaStreamWaitEvent(copy, done[b ^ 1], 0));
                SGCN_TRY(stage(b ^ 1));
            }
            SGCN_CUDA(cudaStreamWaitEvent(st, ready[b], 0));
            slicegcn_opt_desc o = *opt;
            o.epoch = opt->epoch + e;
            slicegcn_model_invalidate_caches(m);   // the staging buffer holds a fresh copy of X
            SGCN_TRY(slicegcn_train_epoch(m, g, xs[b], x_ld, ys[b], train_idx, n_train, params, grads, adam_m, adam_v, &o, nullptr,
                                          losses_dev + e, workspace, workspace_bytes, stream));
            SGCN_CUDA(cudaEventRecord(done[b], st));
            if (losses_host)
                SGCN_CUDA(cudaMemcpyAsync(losses_host + e, losses_dev + e, sizeof(float), cudaMemcpyDeviceToHost, st));
        }
        SGCN_CUDA(cudaStreamSynchronize(st));
        SGCN_CUDA(cudaStreamSynchronize(copy));
        return SLICEGCN_OK;
    };
    rc = run();
    if (rc != SLICEGCN_OK) {   // drain whatever was queued before the events and the stream go away
        cudaStreamSynchronize(st);
        if (copy) cudaStreamSynchronize(copy);
    }
    cleanup();
    return rc;
}

}  // extern "C"
