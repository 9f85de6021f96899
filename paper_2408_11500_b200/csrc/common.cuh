// Shared internals of the SliceGCN CUDA library (not part of the C ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <cstdarg>
#include <cstdio>

#include "../../include/slicegcn.h"

namespace sgcn {

// ---- error reporting -------------------------------------------------------------------------
void set_error(const char* fmt, ...);

#define SGCN_FAIL(code, ...)           \
    do {                               \
        ::sgcn::set_error(__VA_ARGS__); \
        return (code);                 \
    } while (0)

#define SGCN_CUDA(expr)                                                                             \
    do {                                                                                            \
        cudaError_t _e = (expr);                                                                    \
        if (_e != cudaSuccess) {                                                                    \
            ::sgcn::set_error("%s failed: %s (%s:%d)", #expr, cudaGetErrorString(_e), __FILE__, __LINE__); \
            return (_e == cudaErrorMemoryAllocation) ? SLICEGCN_ERR_ALLOC : SLICEGCN_ERR_CUDA;      \
        }                                                                                           \
    } while (0)

#define SGCN_TRY(expr)                       \
    do {                                     \
        slicegcn_status_t _s = (expr);       \
        if (_s != SLICEGCN_OK) return _s;    \
    } while (0)

// after a kernel launch
#define SGCN_LAUNCH_CHECK() SGCN_CUDA(cudaGetLastError())

const char* last_error();

// ---- launch accounting (for the benchmark's launch count and SpMM timing) ---------------------
void count_launch(int n = 1);
long long launches();
void reset_launches();

// ---- CSR view used by the SpMM ----------------------------------------------------------------
// Rows with more than kLongRow stored entries are split into segments of kSegment entries; each
// segment is reduced by one warp into a partial row, and the partial rows of a long row are summed
// in a fixed order afterwards (deterministic, no floating-point atomics).
constexpr int kLongRow = 64;
constexpr int kSegment = 128;
// The remaining rows are dealt out in row-aligned chunks of about kChunk stored entries: chunk c
// owns every row whose first entry index lies in [c*kChunk, (c+1)*kChunk), so each lane group gets
// the same amount of gather work whatever the degree distribution.
constexpr int kChunk = 64;

struct CsrView {
    const int32_t* rowptr = nullptr;   // [n+1]
    const int32_t* colidx = nullptr;   // [nnz]
    int32_t n_long = 0;                // rows with deg > kLongRow
    const int32_t* long_rows = nullptr;  // [n_long] row ids
    const int32_t* seg_ptr = nullptr;    // [n_long+1] first segment of each long row
    int32_t n_seg = 0;
    const int32_t* seg_row = nullptr;    // [n_seg] index into long_rows
    const int32_t* seg_order = nullptr;  // [n_seg] segments sorted by their first column index (processing order)
    int32_t n_chunks = 0;
    const int32_t* chunk_row = nullptr;  // [n_chunks+1] first row of each chunk
    // A_hat_ij = row_scale[i] * col_scale[j] for every stored entry (no per-entry value array)
    const float* row_scale = nullptr;
    const float* col_scale = nullptr;
};

}  // namespace sgcn

struct slicegcn_graph {
    int64_t n = 0;
    int64_t nnz = 0;
    bool symmetric = false;
    int32_t* rowptr = nullptr;
    int32_t* colidx = nullptr;
    int32_t* deg = nullptr;
    float* dinv = nullptr;
    // aggregators other than Eq. 1's: 1/deg (0 for an empty row) and a vector of ones; norm 0 sym, 1 mean, 2 sum
    float* invdeg = nullptr;
    float* ones = nullptr;
    int norm = 0;
    int* fault = nullptr;   // device status word: non-zero once a bounded wait in a kernel ran out
    // transpose pattern (only when !symmetric)
    int32_t* rowptr_t = nullptr;
    int32_t* colidx_t = nullptr;
    // long-row tables (forward pattern and transpose pattern)
    int32_t* long_rows[2] = {nullptr, nullptr};
    int32_t* seg_ptr[2] = {nullptr, nullptr};
    int32_t* seg_row[2] = {nullptr, nullptr};
    int32_t* seg_order[2] = {nullptr, nullptr};
    int32_t n_long[2] = {0, 0};
    int32_t n_seg[2] = {0, 0};
    int32_t* chunk_row[2] = {nullptr, nullptr};
    int32_t n_chunks[2] = {0, 0};

    sgcn::CsrView view(bool transpose) const {
        sgcn::CsrView v;
        int t = (transpose && !symmetric) ? 1 : 0;
        v.rowptr = t ? rowptr_t : rowptr;
        v.colidx = t ? colidx_t : colidx;
        v.n_long = n_long[t];
        v.long_rows = long_rows[t];
        v.seg_ptr = seg_ptr[t];
        v.n_seg = n_seg[t];
        v.seg_row = seg_row[t];
        v.seg_order = seg_order[t];
        v.n_chunks = n_chunks[t];
        v.chunk_row = chunk_row[t];
        // sym: D^-1/2 A D^-1/2 either way; mean: D^-1 A forward, A^T D^-1 transposed; sum: A
        v.row_scale = norm == 0 ? dinv : (norm == 1 && !transpose ? invdeg : ones);
        v.col_scale = norm == 0 ? dinv : (norm == 1 && transpose ? invdeg : ones);
        return v;
    }
    int32_t max_segments() const { return n_seg[0] > n_seg[1] ? n_seg[0] : n_seg[1]; }
};
