// Graph construction: edge list / CSR -> canonical device CSR, degrees, 1/sqrt(deg), transpose
// pattern when needed, and the long-row segment tables the SpMM uses.
// Section III-A (A in {0,1}^{n x n}, neighbor sets) and the normalisation of Eq. 1.
// Sorting / compaction / scans use CUB device primitives; this is set-up work, outside the epoch.
#include <cub/cub.cuh>

#include <cstring>
#include <new>
#include <vector>

#include "common.cuh"

namespace sgcn {

static thread_local char g_err[512] = "";
static long long g_launches = 0;

void set_error(const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}
const char* last_error() { return g_err; }
void count_launch(int n) { g_launches += n; }
long long launches() { return g_launches; }
void reset_launches() { g_launches = 0; }

namespace {

// device buffer freed on scope exit unless released
struct DevBuf {
    void* p = nullptr;
    ~DevBuf() {
        if (p) cudaFree(p);
    }
    cudaError_t alloc(size_t bytes) { return cudaMalloc(&p, bytes ? bytes : 16); }
    template <typename T>
    T* as() {
        return static_cast<T*>(p);
    }
    template <typename T>
    T* release() {
        T* r = static_cast<T*>(p);
        p = nullptr;
        return r;
    }
};

__global__ void check_range_kernel(const int32_t* a, const int32_t* b, int64_t m, int32_t n, int* bad) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < m; i += stride) {
        int32_t u = a[i], v = b[i];
        if (u < 0 || u >= n || v < 0 || v >= n) *bad = 1;
    }
}

// keys: (row << 32) | col for every stored entry candidate
__global__ void make_keys_kernel(const int32_t* src, const int32_t* dst, int64_t m, int64_t n, bool sym, bool loops,
                                 uint64_t* keys) {
    int64_t total = m * (sym ? 2 : 1) + (loops ? n : 0);
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < total; i += stride) {
        uint64_t r, c;
        if (i < m) {
            r = (uint32_t)src[i];
            c = (uint32_t)dst[i];
        } else if (sym && i < 2 * m) {
            r = (uint32_t)dst[i - m];
            c = (uint32_t)src[i - m];
        } else {
            r = c = (uint64_t)(i - m * (sym ? 2 : 1));
        }
        keys[i] = (r << 32) | c;
    }
}

__global__ void swap_halves_kernel(const uint64_t* in, int64_t m, uint64_t* out) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < m; i += stride) {
        uint64_t k = in[i];
        out[i] = (k << 32) | (k >> 32);
    }
}

__global__ void split_keys_kernel(const uint64_t* keys, int64_t nnz, int32_t* colidx, int32_t* deg) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < nnz; i += stride) {
        uint64_t k = keys[i];
        colidx[i] = (int32_t)(k & 0xffffffffu);
        if (deg) atomicAdd(&deg[(int32_t)(k >> 32)], 1);   // integer atomics: order-independent result
    }
}

__global__ void compare_keys_kernel(const uint64_t* a, const uint64_t* b, int64_t m, int* differ) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < m; i += stride)
        if (a[i] != b[i]) *differ = 1;
}

__global__ void dinv_kernel(const int32_t* deg, int64_t n, float* dinv) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n) {
        int32_t d = deg[i];
        // IEEE-rounded sqrt and division so that the value is reproducible bit for bit on a host
        dinv[i] = d > 0 ? __fdiv_rn(1.0f, __fsqrt_rn((float)d)) : 0.0f;
    }
}

__global__ void invdeg_ones_kernel(const int32_t* deg, int64_t n, float* invdeg, float* ones) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n) {
        int32_t d = deg[i];
        invdeg[i] = d > 0 ? __fdiv_rn(1.0f, (float)d) : 0.0f;
        ones[i] = 1.0f;
    }
}

__global__ void expand_rows_kernel(const int32_t* rowptr, int64_t n, int32_t* rows) {
    // one warp per row
    int64_t warp = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    int lane = threadIdx.x & 31;
    int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    for (int64_t r = warp; r < n; r += nwarps)
        for (int32_t k = rowptr[r] + lane; k < rowptr[r + 1]; k += 32) rows[k] = (int32_t)r;
}

__global__ void check_rowptr_kernel(const int32_t* rowptr, int64_t n, int* bad) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i < n && rowptr[i + 1] < rowptr[i]) *bad = 1;
    if (i == 0 && rowptr[0] != 0) *bad = 1;
}

struct IsLong {
    const int32_t* rowptr;
    __device__ bool operator()(int32_t r) const { return rowptr[r + 1] - rowptr[r] > kLongRow; }
};

__global__ void seg_count_kernel(const int32_t* rowptr, const int32_t* long_rows, int32_t n_long, int32_t* cnt) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n_long) {
        int32_t r = long_rows[i];
        cnt[i] = (rowptr[r + 1] - rowptr[r] + kSegment - 1) / kSegment;
    }
    if (i == n_long) cnt[i] = 0;
}

__global__ void seg_fill_kernel(const int32_t* seg_ptr, int32_t n_long, int32_t* seg_row) {
    int i = blockIdx.x;
    if (i < n_long)
        for (int32_t s = seg_ptr[i] + threadIdx.x; s < seg_ptr[i + 1]; s += blockDim.x) seg_row[s] = i;
}

// Row r opens a new chunk when its first entry index falls into another kChunk-sized window than
// its predecessor's, or when it or its predecessor is a long row (long rows sit alone in a chunk, so
// a chunk is either one long row or a run of short rows with contiguous entries).
struct IsChunkStart {
    const int32_t* rowptr;
    __device__ bool is_long(int32_t r) const { return rowptr[r + 1] - rowptr[r] > kLongRow; }
    __device__ bool operator()(int32_t r) const {
        if (r == 0) return true;
        if (rowptr[r] / kChunk != rowptr[r - 1] / kChunk) return true;
        return is_long(r) || is_long(r - 1);
    }
};

inline int grid_for(int64_t work, int block = 256) {
    int64_t g = (work + block - 1) / block;
    if (g < 1) g = 1;
    if (g > 148 * 32) g = 148 * 32;
    return (int)g;
}

slicegcn_status_t rowptr_from_deg(const int32_t* deg, int64_t n, int32_t* rowptr, cudaStream_t st) {
    // rowptr[0..n] = exclusive scan of deg (with a trailing total)
    size_t tmp_bytes = 0;
    SGCN_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, tmp_bytes, deg, rowptr, (int)(n + 1), st));
    DevBuf tmp;
    SGCN_CUDA(tmp.alloc(tmp_bytes));
    SGCN_CUDA(cub::DeviceScan::ExclusiveSum(tmp.p, tmp_bytes, deg, rowptr, (int)(n + 1), st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    return SLICEGCN_OK;
}

// Builds the long-row tables of one CSR pattern.
// key of a segment = the column index of its first entry
__global__ void seg_first_col_kernel(const int32_t* rowptr, const int32_t* colidx, const int32_t* long_rows, const int32_t* seg_ptr,
                                     const int32_t* seg_row, int32_t n_seg, int32_t* key, int32_t* id) {
    const int32_t s = blockIdx.x * blockDim.x + threadIdx.x;
    if (s >= n_seg) return;
    const int32_t li = seg_row[s];
    key[s] = colidx[rowptr[long_rows[li]] + (s - seg_ptr[li]) * kSegment];
    id[s] = s;
}

slicegcn_status_t build_long_tables(slicegcn_graph* g, int t, const int32_t* rowptr, const int32_t* colidx, cudaStream_t st) {
    int64_t n = g->n;
    DevBuf ids, sel, cnt, tmp;
    SGCN_CUDA(ids.alloc(sizeof(int32_t) * n));
    SGCN_CUDA(sel.alloc(sizeof(int32_t) * n));
    SGCN_CUDA(cnt.alloc(sizeof(int32_t)));
    size_t tmp_bytes = 0;
    cub::CountingInputIterator<int32_t> it(0);
    IsLong pred{rowptr};
    SGCN_CUDA(cub::DeviceSelect::If(nullptr, tmp_bytes, it, sel.as<int32_t>(), cnt.as<int32_t>(), (int)n, pred, st));
    SGCN_CUDA(tmp.alloc(tmp_bytes));
    SGCN_CUDA(cub::DeviceSelect::If(tmp.p, tmp_bytes, it, sel.as<int32_t>(), cnt.as<int32_t>(), (int)n, pred, st));
    int32_t n_long = 0;
    SGCN_CUDA(cudaMemcpyAsync(&n_long, cnt.p, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    g->n_long[t] = n_long;
    g->n_seg[t] = 0;
    {
        DevBuf starts, ccnt, ctmp;
        SGCN_CUDA(starts.alloc(sizeof(int32_t) * (n + 1)));
        SGCN_CUDA(ccnt.alloc(sizeof(int32_t)));
        IsChunkStart cpred{rowptr};
        size_t ctb = 0;
        SGCN_CUDA(cub::DeviceSelect::If(nullptr, ctb, it, starts.as<int32_t>(), ccnt.as<int32_t>(), (int)n, cpred, st));
        SGCN_CUDA(ctmp.alloc(ctb));
        SGCN_CUDA(cub::DeviceSelect::If(ctmp.p, ctb, it, starts.as<int32_t>(), ccnt.as<int32_t>(), (int)n, cpred, st));
        int32_t n_chunks = 0;
        SGCN_CUDA(cudaMemcpyAsync(&n_chunks, ccnt.p, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
        SGCN_CUDA(cudaStreamSynchronize(st));
        DevBuf cr;
        SGCN_CUDA(cr.alloc(sizeof(int32_t) * (n_chunks + 1)));
        SGCN_CUDA(cudaMemcpyAsync(cr.p, starts.p, sizeof(int32_t) * n_chunks, cudaMemcpyDeviceToDevice, st));
        const int32_t n32 = (int32_t)n;
        SGCN_CUDA(cudaMemcpyAsync(cr.as<int32_t>() + n_chunks, &n32, sizeof(int32_t), cudaMemcpyHostToDevice, st));
        SGCN_CUDA(cudaStreamSynchronize(st));
        g->n_chunks[t] = n_chunks;
        g->chunk_row[t] = cr.release<int32_t>();
    }
    if (n_long == 0) return SLICEGCN_OK;
    DevBuf lr, counts, sp, tmp2;
    SGCN_CUDA(lr.alloc(sizeof(int32_t) * n_long));
    SGCN_CUDA(cudaMemcpyAsync(lr.p, sel.p, sizeof(int32_t) * n_long, cudaMemcpyDeviceToDevice, st));
    SGCN_CUDA(counts.alloc(sizeof(int32_t) * (n_long + 1)));
    SGCN_CUDA(sp.alloc(sizeof(int32_t) * (n_long + 1)));
    seg_count_kernel<<<(n_long + 1 + 255) / 256, 256, 0, st>>>(rowptr, lr.as<int32_t>(), n_long, counts.as<int32_t>());
    SGCN_LAUNCH_CHECK();
    size_t tb2 = 0;
    SGCN_CUDA(cub::DeviceScan::ExclusiveSum(nullptr, tb2, counts.as<int32_t>(), sp.as<int32_t>(), n_long + 1, st));
    SGCN_CUDA(tmp2.alloc(tb2));
    SGCN_CUDA(cub::DeviceScan::ExclusiveSum(tmp2.p, tb2, counts.as<int32_t>(), sp.as<int32_t>(), n_long + 1, st));
    int32_t n_seg = 0;
    SGCN_CUDA(cudaMemcpyAsync(&n_seg, sp.as<int32_t>() + n_long, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    DevBuf sr;
    SGCN_CUDA(sr.alloc(sizeof(int32_t) * n_seg));
    seg_fill_kernel<<<n_long, 128, 0, st>>>(sp.as<int32_t>(), n_long, sr.as<int32_t>());
    SGCN_LAUNCH_CHECK();
    // Processing order of the segments: by first column index.  Columns are sorted inside a row, so segments that
    // start at similar columns gather from the same stretch of the operand; run next to each other they find it in L2
    // (in row order every long row sweeps the whole operand again).
    DevBuf key, id, key2, so, stmp;
    SGCN_CUDA(key.alloc(sizeof(int32_t) * n_seg));
    SGCN_CUDA(id.alloc(sizeof(int32_t) * n_seg));
    SGCN_CUDA(key2.alloc(sizeof(int32_t) * n_seg));
    SGCN_CUDA(so.alloc(sizeof(int32_t) * n_seg));
    seg_first_col_kernel<<<(n_seg + 255) / 256, 256, 0, st>>>(rowptr, colidx, lr.as<int32_t>(), sp.as<int32_t>(), sr.as<int32_t>(), n_seg,
                                                             key.as<int32_t>(), id.as<int32_t>());
    SGCN_LAUNCH_CHECK();
    size_t stb = 0;
    SGCN_CUDA(cub::DeviceRadixSort::SortPairs(nullptr, stb, key.as<int32_t>(), key2.as<int32_t>(), id.as<int32_t>(), so.as<int32_t>(), n_seg,
                                              0, 32, st));
    SGCN_CUDA(stmp.alloc(stb));
    SGCN_CUDA(cub::DeviceRadixSort::SortPairs(stmp.p, stb, key.as<int32_t>(), key2.as<int32_t>(), id.as<int32_t>(), so.as<int32_t>(), n_seg,
                                              0, 32, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    g->n_seg[t] = n_seg;
    g->seg_order[t] = so.release<int32_t>();
    g->long_rows[t] = lr.release<int32_t>();
    g->seg_ptr[t] = sp.release<int32_t>();
    g->seg_row[t] = sr.release<int32_t>();
    return SLICEGCN_OK;
}

slicegcn_status_t sort_unique(DevBuf& keys, int64_t total, int end_bit, int64_t* n_unique, cudaStream_t st) {
    // sorts `keys` (uint64[total]) and removes repeats in place (keys is replaced)
    DevBuf alt, tmp, cnt;
    SGCN_CUDA(alt.alloc(sizeof(uint64_t) * total));
    SGCN_CUDA(cnt.alloc(sizeof(int64_t)));
    if (total >= (int64_t)1 << 31) SGCN_FAIL(SLICEGCN_ERR_OVERFLOW, "edge list too long: %lld candidates", (long long)total);
    cub::DoubleBuffer<uint64_t> db(keys.as<uint64_t>(), alt.as<uint64_t>());
    size_t tb = 0;
    SGCN_CUDA(cub::DeviceRadixSort::SortKeys(nullptr, tb, db, (int)total, 0, end_bit, st));
    SGCN_CUDA(tmp.alloc(tb));
    SGCN_CUDA(cub::DeviceRadixSort::SortKeys(tmp.p, tb, db, (int)total, 0, end_bit, st));
    uint64_t* sorted = db.Current();
    uint64_t* other = db.Alternate();
    size_t tb2 = 0;
    SGCN_CUDA(cub::DeviceSelect::Unique(nullptr, tb2, sorted, other, cnt.as<int64_t>(), (int)total, st));
    DevBuf tmp2;
    SGCN_CUDA(tmp2.alloc(tb2));
    SGCN_CUDA(cub::DeviceSelect::Unique(tmp2.p, tb2, sorted, other, cnt.as<int64_t>(), (int)total, st));
    SGCN_CUDA(cudaMemcpyAsync(n_unique, cnt.p, sizeof(int64_t), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    if (other != keys.as<uint64_t>()) {   // result sits in `alt`: swap ownership
        void* t = keys.p;
        keys.p = alt.p;
        alt.p = t;
    }
    return SLICEGCN_OK;
}

slicegcn_status_t create_impl(int64_t n, int64_t m, const int32_t* d_src, const int32_t* d_dst, uint32_t flags,
                              cudaStream_t st, slicegcn_graph** out) {
    const bool sym = flags & SLICEGCN_SYMMETRIZE, loops = flags & SLICEGCN_ADD_SELF_LOOPS;
    if ((flags & SLICEGCN_NORM_MEAN) && (flags & SLICEGCN_NORM_SUM))
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "graph_create: NORM_MEAN and NORM_SUM exclude each other");
    DevBuf flag;
    SGCN_CUDA(flag.alloc(sizeof(int)));
    SGCN_CUDA(cudaMemsetAsync(flag.p, 0, sizeof(int), st));
    if (m > 0) {
        check_range_kernel<<<grid_for(m), 256, 0, st>>>(d_src, d_dst, m, (int32_t)n, flag.as<int>());
        SGCN_LAUNCH_CHECK();
    }
    int bad = 0;
    SGCN_CUDA(cudaMemcpyAsync(&bad, flag.p, sizeof(int), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    if (bad) SGCN_FAIL(SLICEGCN_ERR_OUT_OF_RANGE, "edge list holds a node id outside [0, %lld)", (long long)n);

    int64_t total = m * (sym ? 2 : 1) + (loops ? n : 0);
    if (total >= (int64_t)1 << 31) SGCN_FAIL(SLICEGCN_ERR_OVERFLOW, "too many stored entries: %lld", (long long)total);
    int bits = 1;
    while (((int64_t)1 << bits) < n) ++bits;

    slicegcn_graph* g = new (std::nothrow) slicegcn_graph();
    if (!g) SGCN_FAIL(SLICEGCN_ERR_ALLOC, "host allocation failed");
    struct Guard {
        slicegcn_graph* g;
        ~Guard() {
            if (g) slicegcn_graph_destroy(g);
        }
    } guard{g};
    g->n = n;

    DevBuf keys;
    SGCN_CUDA(keys.alloc(sizeof(uint64_t) * (total ? total : 1)));
    int64_t nnz = 0;
    if (total > 0) {
        make_keys_kernel<<<grid_for(total), 256, 0, st>>>(d_src, d_dst, m, n, sym, loops, keys.as<uint64_t>());
        SGCN_LAUNCH_CHECK();
        SGCN_TRY(sort_unique(keys, total, 32 + bits, &nnz, st));
    }
    g->nnz = nnz;
    DevBuf rowptr, colidx, deg, dinv;
    SGCN_CUDA(rowptr.alloc(sizeof(int32_t) * (n + 1)));
    SGCN_CUDA(colidx.alloc(sizeof(int32_t) * (nnz ? nnz : 1)));
    SGCN_CUDA(deg.alloc(sizeof(int32_t) * (n + 1)));
    SGCN_CUDA(dinv.alloc(sizeof(float) * n));
    SGCN_CUDA(cudaMemsetAsync(deg.p, 0, sizeof(int32_t) * (n + 1), st));
    if (nnz > 0) {
        split_keys_kernel<<<grid_for(nnz), 256, 0, st>>>(keys.as<uint64_t>(), nnz, colidx.as<int32_t>(), deg.as<int32_t>());
        SGCN_LAUNCH_CHECK();
    }
    SGCN_TRY(rowptr_from_deg(deg.as<int32_t>(), n, rowptr.as<int32_t>(), st));
    dinv_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>(deg.as<int32_t>(), n, dinv.as<float>());
    SGCN_LAUNCH_CHECK();

    // symmetry of the pattern; transpose CSR if it is not symmetric
    bool symmetric = true;
    if (!sym && nnz > 0) {
        DevBuf tkeys;
        SGCN_CUDA(tkeys.alloc(sizeof(uint64_t) * nnz));
        swap_halves_kernel<<<grid_for(nnz), 256, 0, st>>>(keys.as<uint64_t>(), nnz, tkeys.as<uint64_t>());
        SGCN_LAUNCH_CHECK();
        int64_t nnz_t = 0;
        SGCN_TRY(sort_unique(tkeys, nnz, 32 + bits, &nnz_t, st));
        SGCN_CUDA(cudaMemsetAsync(flag.p, 0, sizeof(int), st));
        compare_keys_kernel<<<grid_for(nnz), 256, 0, st>>>(keys.as<uint64_t>(), tkeys.as<uint64_t>(), nnz, flag.as<int>());
        SGCN_LAUNCH_CHECK();
        int differ = 0;
        SGCN_CUDA(cudaMemcpyAsync(&differ, flag.p, sizeof(int), cudaMemcpyDeviceToHost, st));
        SGCN_CUDA(cudaStreamSynchronize(st));
        if (differ) {
            symmetric = false;
            DevBuf rp_t, ci_t, deg_t;
            SGCN_CUDA(rp_t.alloc(sizeof(int32_t) * (n + 1)));
            SGCN_CUDA(ci_t.alloc(sizeof(int32_t) * nnz));
            SGCN_CUDA(deg_t.alloc(sizeof(int32_t) * (n + 1)));
            SGCN_CUDA(cudaMemsetAsync(deg_t.p, 0, sizeof(int32_t) * (n + 1), st));
            split_keys_kernel<<<grid_for(nnz), 256, 0, st>>>(tkeys.as<uint64_t>(), nnz, ci_t.as<int32_t>(), deg_t.as<int32_t>());
            SGCN_LAUNCH_CHECK();
            SGCN_TRY(rowptr_from_deg(deg_t.as<int32_t>(), n, rp_t.as<int32_t>(), st));
            g->rowptr_t = rp_t.release<int32_t>();
            g->colidx_t = ci_t.release<int32_t>();
        }
    }
    g->symmetric = symmetric;
    {
        DevBuf fl;
        SGCN_CUDA(fl.alloc(sizeof(int)));
        SGCN_CUDA(cudaMemsetAsync(fl.p, 0, sizeof(int), st));
        g->fault = fl.release<int>();
    }
    g->rowptr = rowptr.release<int32_t>();
    g->colidx = colidx.release<int32_t>();
    g->deg = deg.release<int32_t>();
    g->dinv = dinv.release<float>();
    g->norm = (flags & SLICEGCN_NORM_MEAN) ? 1 : (flags & SLICEGCN_NORM_SUM) ? 2 : 0;
    if (g->norm != 0) {
        DevBuf inv, one;
        SGCN_CUDA(inv.alloc(sizeof(float) * n));
        SGCN_CUDA(one.alloc(sizeof(float) * n));
        invdeg_ones_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>(g->deg, n, inv.as<float>(), one.as<float>());
        SGCN_LAUNCH_CHECK();
        g->invdeg = inv.release<float>();
        g->ones = one.release<float>();
    }
    SGCN_TRY(build_long_tables(g, 0, g->rowptr, g->colidx, st));
    if (!symmetric) SGCN_TRY(build_long_tables(g, 1, g->rowptr_t, g->colidx_t, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    guard.g = nullptr;
    *out = g;
    return SLICEGCN_OK;
}

}  // namespace
}  // namespace sgcn

using namespace sgcn;

extern "C" {

const char* slicegcn_last_error(void) { return sgcn::last_error(); }

slicegcn_status_t slicegcn_graph_create(int64_t n, int64_t n_edges, const int32_t* src, const int32_t* dst,
                                        uint32_t flags, void* stream, slicegcn_graph** out) {
    if (!out) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (n < 1 || n_edges < 0) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "n must be >= 1 and n_edges >= 0");
    if (n >= ((int64_t)1 << 31)) SGCN_FAIL(SLICEGCN_ERR_OVERFLOW, "n does not fit int32");
    if (n_edges > 0 && (!src || !dst)) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "src/dst is NULL");
    cudaStream_t st = (cudaStream_t)stream;
    DevBuf ds, dd;
    const int32_t *d_src = src, *d_dst = dst;
    if (!(flags & SLICEGCN_INPUT_ON_DEVICE) && n_edges > 0) {
        SGCN_CUDA(ds.alloc(sizeof(int32_t) * n_edges));
        SGCN_CUDA(dd.alloc(sizeof(int32_t) * n_edges));
        SGCN_CUDA(cudaMemcpyAsync(ds.p, src, sizeof(int32_t) * n_edges, cudaMemcpyHostToDevice, st));
        SGCN_CUDA(cudaMemcpyAsync(dd.p, dst, sizeof(int32_t) * n_edges, cudaMemcpyHostToDevice, st));
        d_src = ds.as<int32_t>();
        d_dst = dd.as<int32_t>();
    }
    return create_impl(n, n_edges, d_src, d_dst, flags, st, out);
}

slicegcn_status_t slicegcn_graph_create_from_csr(int64_t n, const int32_t* rowptr, const int32_t* colidx,
                                                 uint32_t flags, void* stream, slicegcn_graph** out) {
    if (!out) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "out is NULL");
    *out = nullptr;
    if (n < 1 || !rowptr) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "n must be >= 1 and rowptr non-NULL");
    if (n >= ((int64_t)1 << 31)) SGCN_FAIL(SLICEGCN_ERR_OVERFLOW, "n does not fit int32");
    cudaStream_t st = (cudaStream_t)stream;
    const bool on_dev = flags & SLICEGCN_INPUT_ON_DEVICE;
    DevBuf drp, dci, rows, flag;
    const int32_t* d_rp = rowptr;
    if (!on_dev) {
        SGCN_CUDA(drp.alloc(sizeof(int32_t) * (n + 1)));
        SGCN_CUDA(cudaMemcpyAsync(drp.p, rowptr, sizeof(int32_t) * (n + 1), cudaMemcpyHostToDevice, st));
        d_rp = drp.as<int32_t>();
    }
    SGCN_CUDA(flag.alloc(sizeof(int)));
    SGCN_CUDA(cudaMemsetAsync(flag.p, 0, sizeof(int), st));
    check_rowptr_kernel<<<(int)((n + 255) / 256), 256, 0, st>>>(d_rp, n, flag.as<int>());
    SGCN_LAUNCH_CHECK();
    int bad = 0;
    int32_t m32 = 0;
    SGCN_CUDA(cudaMemcpyAsync(&bad, flag.p, sizeof(int), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaMemcpyAsync(&m32, d_rp + n, sizeof(int32_t), cudaMemcpyDeviceToHost, st));
    SGCN_CUDA(cudaStreamSynchronize(st));
    if (bad || m32 < 0) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "rowptr must start at 0 and be non-decreasing");
    int64_t m = m32;
    if (m > 0 && !colidx) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "colidx is NULL");
    const int32_t* d_ci = colidx;
    if (!on_dev && m > 0) {
        SGCN_CUDA(dci.alloc(sizeof(int32_t) * m));
        SGCN_CUDA(cudaMemcpyAsync(dci.p, colidx, sizeof(int32_t) * m, cudaMemcpyHostToDevice, st));
        d_ci = dci.as<int32_t>();
    }
    SGCN_CUDA(rows.alloc(sizeof(int32_t) * (m ? m : 1)));
    if (m > 0) {
        expand_rows_kernel<<<grid_for(n * 32), 256, 0, st>>>(d_rp, n, rows.as<int32_t>());
        SGCN_LAUNCH_CHECK();
    }
    return create_impl(n, m, rows.as<int32_t>(), d_ci, flags, st, out);
}

slicegcn_status_t slicegcn_graph_info(const slicegcn_graph* g, int64_t* n, int64_t* nnz, int32_t* is_symmetric,
                                      int64_t* n_segments) {
    if (!g) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "graph is NULL");
    if (n) *n = g->n;
    if (nnz) *nnz = g->nnz;
    if (is_symmetric) *is_symmetric = g->symmetric ? 1 : 0;
    if (n_segments) *n_segments = g->max_segments();
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_graph_export(const slicegcn_graph* g, int32_t* rowptr, int32_t* colidx, int32_t* deg,
                                        float* dinv) {
    if (!g) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "graph is NULL");
    SGCN_CUDA(cudaDeviceSynchronize());
    if (rowptr) SGCN_CUDA(cudaMemcpy(rowptr, g->rowptr, sizeof(int32_t) * (g->n + 1), cudaMemcpyDeviceToHost));
    if (colidx && g->nnz) SGCN_CUDA(cudaMemcpy(colidx, g->colidx, sizeof(int32_t) * g->nnz, cudaMemcpyDeviceToHost));
    if (deg) SGCN_CUDA(cudaMemcpy(deg, g->deg, sizeof(int32_t) * g->n, cudaMemcpyDeviceToHost));
    if (dinv) SGCN_CUDA(cudaMemcpy(dinv, g->dinv, sizeof(float) * g->n, cudaMemcpyDeviceToHost));
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_graph_device_status(const slicegcn_graph* g, int32_t* status) {
    if (!g || !status) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "NULL argument");
    SGCN_CUDA(cudaDeviceSynchronize());
    int v = 0;
    SGCN_CUDA(cudaMemcpy(&v, g->fault, sizeof(int), cudaMemcpyDeviceToHost));
    *status = v;
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_graph_destroy(slicegcn_graph* g) {
    if (!g) return SLICEGCN_OK;
    cudaFree(g->rowptr);
    cudaFree(g->colidx);
    cudaFree(g->deg);
    cudaFree(g->dinv);
    cudaFree(g->invdeg);
    cudaFree(g->ones);
    cudaFree(g->fault);
    cudaFree(g->rowptr_t);
    cudaFree(g->colidx_t);
    for (int t = 0; t < 2; ++t) {
        cudaFree(g->long_rows[t]);
        cudaFree(g->seg_ptr[t]);
        cudaFree(g->seg_row[t]);
        cudaFree(g->seg_order[t]);
        cudaFree(g->chunk_row[t]);
    }
    delete g;
    return SLICEGCN_OK;
}

}  // extern "C"
