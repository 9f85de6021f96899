// Dense kernels of the layer: grouped (per-slice) row-panel GEMM with the fused epilogues of
// Eq. 6-7, grouped weight gradients with a deterministic two-stage reduction, the cross-entropy
// of Eq. 10 and the Adam update.  This file holds the CUDA-core (FFMA) implementations.
#include <algorithm>
#include <cstdlib>

#include "common.cuh"
#include "kernels.cuh"

namespace sgcn {
namespace {

__device__ __forceinline__ float ldf(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------ grouped GEMM
constexpr int GM = 128;   // rows per CTA
constexpr int GK = 32;    // reduction slab

template <typename TA, typename TC, int BN, int TM, int TN>
__global__ void __launch_bounds__(256) gemm_kernel(const GemmArgs a) {
    static_assert((GM / TM) * (BN / TN) == 256, "thread tiling must cover the CTA tile");
    __shared__ float As[GK][GM + 4];
    __shared__ float Bs[GK][BN];
    const int g = blockIdx.z;
    const int64_t row0 = (int64_t)blockIdx.x * GM;
    const int n0 = blockIdx.y * BN;
    const int tid = threadIdx.x;
    const int tx = tid % (BN / TN), ty = tid / (BN / TN);
    const TA* A = static_cast<const TA*>(a.A) + a.a_start[g];
    const uint8_t* am = a.a_mask ? a.a_mask + a.a_start[g] : nullptr;
    const float* B = a.B + (int64_t)g * a.b_gstride;
    float acc[TM][TN];
#pragma unroll
    for (int i = 0; i < TM; ++i)
#pragma unroll
        for (int j = 0; j < TN; ++j) acc[i][j] = 0.f;

    for (int k0 = 0; k0 < a.K; k0 += GK) {
        // A slab: 128 rows x 32 k, one warp reads 32 consecutive k of a row
        {
            const int kk = tid & 31;
            const int k = k0 + kk;
#pragma unroll
            for (int i = 0; i < GM / 8; ++i) {
                const int r = (tid >> 5) + 8 * i;
                const int64_t row = row0 + r;
                float v = 0.f;
                if (row < a.M && k < a.K) {
                    v = ldf(A + row * a.lda + k);
                    if (am) v *= (float)am[row * a.a_mask_ld + k];
                }
                As[kk][r] = v;
            }
        }
        // B slab: 32 k x BN
        for (int e = tid; e < GK * BN; e += 256) {
            const int kk = e / BN, nn = e % BN;
            const int k = k0 + kk, n = n0 + nn;
            float v = 0.f;
            if (k < a.K && n < a.N) {
                const float* Bq = B;
                int kj = k;
                if (a.b_kstack > 0) {
                    Bq = B + (int64_t)(k / a.b_kstack) * a.b_gstride;
                    kj = k % a.b_kstack;
                }
                v = a.b_trans ? __ldg(Bq + (int64_t)n * a.ldb + kj) : __ldg(Bq + (int64_t)kj * a.ldb + n);
            }
            Bs[kk][nn] = v;
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < GK; ++kk) {
            float av[TM], bv[TN];
#pragma unroll
            for (int i = 0; i < TM; i += 4) {
                const float4 t = *reinterpret_cast<const float4*>(&As[kk][ty * TM + i]);
                av[i] = t.x; av[i + 1] = t.y; av[i + 2] = t.z; av[i + 3] = t.w;
            }
#pragma unroll
            for (int j = 0; j < TN; ++j) bv[j] = Bs[kk][tx * TN + j];
#pragma unroll
            for (int i = 0; i < TM; ++i)
#pragma unroll
                for (int j = 0; j < TN; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }

    TC* C = static_cast<TC*>(a.C);
    const int cs = a.c_start[g];
#pragma unroll
    for (int i = 0; i < TM; ++i) {
        const int64_t row = row0 + ty * TM + i;
        if (row >= a.M) continue;
#pragma unroll
        for (int j = 0; j < TN; ++j) {
            const int n = n0 + tx * TN + j;
            if (n >= a.N) continue;
            const int col = cs + n;
            float x = acc[i][j];
            if (a.bias) x += __ldg(a.bias + g * a.N + n);
            if (a.relu) {
                if (a.mask_out) a.mask_out[row * a.mask_ld + col] = x > 0.f ? 1 : 0;
                x = fmaxf(x, 0.f);
            }
            if (a.post1) x += __ldg(a.post1 + g * a.N + n);
            if (a.post2) x += __ldg(a.post2 + g * a.N + n);
            if (a.mul_pos) {
                const float pv = a.mul_pos_dtype == SLICEGCN_F32
                                     ? static_cast<const float*>(a.mul_pos)[row * a.mul_pos_ld + col]
                                     : a.mul_pos_dtype == kGateBytes
                                           ? (float)static_cast<const uint8_t*>(a.mul_pos)[row * a.mul_pos_ld + col]
                                           : __bfloat162float(static_cast<const __nv_bfloat16*>(a.mul_pos)[row * a.mul_pos_ld + col]);
                x = pv > 0.f ? x : 0.f;
            }
            if (a.accumulate) x += ldf(C + row * a.ldc + col);
            stf(C + row * a.ldc + col, x);
        }
    }
}

template <typename TA, typename TC>
slicegcn_status_t gemm_dispatch(const GemmArgs& a, cudaStream_t st) {
    const unsigned gx = (unsigned)((a.M + GM - 1) / GM);
    if (a.N <= 16) {
        dim3 grid(gx, 1, a.groups);
        gemm_kernel<TA, TC, 16, 4, 2><<<grid, 256, 0, st>>>(a);
    } else if (a.N <= 32) {
        dim3 grid(gx, 1, a.groups);
        gemm_kernel<TA, TC, 32, 4, 4><<<grid, 256, 0, st>>>(a);
    } else {
        dim3 grid(gx, (a.N + 63) / 64, a.groups);
        gemm_kernel<TA, TC, 64, 8, 4><<<grid, 256, 0, st>>>(a);
    }
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

// ------------------------------------------------------------------------------ weight gradient
constexpr int WT = 64;    // tile of dW (k and n)
constexpr int WR = 32;    // rows per smem slab

template <typename TA>
__global__ void __launch_bounds__(256) wgrad_partial_kernel(const WgradArgs a, float* scratch, int n_chunks,
                                                            int64_t rows_per_chunk, int Kext) {
    __shared__ float As[WR][WT];
    __shared__ float Bs[WR][WT];
    const int g = blockIdx.z;
    const int tiles_n = (a.N + WT - 1) / WT;
    const int k0 = (blockIdx.y / tiles_n) * WT, n0 = (blockIdx.y % tiles_n) * WT;
    const int chunk = blockIdx.x;
    const int64_t r_begin = chunk * rows_per_chunk;
    const int64_t r_end = min(a.M, r_begin + rows_per_chunk);
    const int tid = threadIdx.x;
    const int tx = tid & 15, ty = tid >> 4;
    const TA* A = static_cast<const TA*>(a.A) + a.a_start[g];
    const float* B = a.B + a.b_start[g];
    const uint8_t* bm = a.b_mask ? a.b_mask + a.b_start[g] : nullptr;
    float acc[4][4];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.f;
    for (int64_t rb = r_begin; rb < r_end; rb += WR) {
        const int c = tid & 63;
#pragma unroll
        for (int i = 0; i < WR / 4; ++i) {
            const int r = (tid >> 6) + 4 * i;
            const int64_t row = rb + r;
            float av = 0.f, bv = 0.f;
            if (row < r_end) {
                const int k = k0 + c, n = n0 + c;
                if (k < a.K)
                    av = ldf(A + row * a.lda + k);
                else if (k == a.K && Kext > a.K)
                    av = 1.f;   // the extra row of ones yields the bias gradient (column sums)
                if (n < a.N) {
                    bv = __ldg(B + row * a.ldb + n);
                    if (bm) bv *= (float)bm[row * a.b_mask_ld + n];
                }
            }
            As[r][c] = av;
            Bs[r][c] = bv;
        }
        __syncthreads();
#pragma unroll 8
        for (int r = 0; r < WR; ++r) {
            const float4 a4 = *reinterpret_cast<const float4*>(&As[r][ty * 4]);
            const float4 b4 = *reinterpret_cast<const float4*>(&Bs[r][tx * 4]);
            const float av[4] = {a4.x, a4.y, a4.z, a4.w};
            const float bv[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
        }
        __syncthreads();
    }
    float* out = scratch + ((int64_t)chunk * a.groups + g) * Kext * a.N;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int k = k0 + ty * 4 + i;
        if (k >= Kext) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int n = n0 + tx * 4 + j;
            if (n < a.N) out[(int64_t)k * a.N + n] = acc[i][j];
        }
    }
}

__global__ void wgrad_reduce_kernel(const float* scratch, int n_chunks, int groups, int K, int Kext, int N, float* dW,
                                    float* dbias, float* dbias2) {
    const int64_t per = (int64_t)groups * Kext * N;
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= per) return;
    float s = 0.f;
    for (int c = 0; c < n_chunks; ++c) s += scratch[c * per + i];   // fixed order
    const int g = (int)(i / ((int64_t)Kext * N));
    const int rem = (int)(i % ((int64_t)Kext * N));
    const int k = rem / N, n = rem % N;
    if (k < K) {
        if (dW) dW[((int64_t)g * K + k) * N + n] = s;
    } else {
        if (dbias) dbias[g * N + n] = s;
        if (dbias2) dbias2[g * N + n] = s;
    }
}

// Column sums of a (masked) row-major fp32 matrix: partial sums per row chunk, then a fixed-order
// reduction (deterministic).  Used for the bias and slice-encoding gradients.
__global__ void __launch_bounds__(256) colsum_partial_kernel(const WgradArgs a, int total_cols, int64_t rows_per_chunk,
                                                             float* scratch) {
    // blockDim = (32 columns) x (8 row lanes); grid = (column blocks, row chunks)
    __shared__ float sm[8][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
    const int c = blockIdx.x * 32 + tx;
    const int64_t r0 = blockIdx.y * rows_per_chunk, r1 = min(a.M, r0 + rows_per_chunk);
    float s = 0.f;
    if (c < total_cols) {
        const float* B = a.B + a.b_start[0] + c;
        const uint8_t* bm = a.b_mask ? a.b_mask + a.b_start[0] + c : nullptr;
        int64_t r = r0 + ty;
        for (; r + 56 < r1; r += 64) {   // eight independent loads in flight, summed in row order
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                v[q] = __ldg(B + (r + 8 * q) * a.ldb);
                if (bm) v[q] = bm[(r + 8 * q) * a.b_mask_ld] ? v[q] : 0.f;
            }
#pragma unroll
            for (int q = 0; q < 8; ++q) s += v[q];
        }
        for (; r < r1; r += 8) {
            float v = __ldg(B + r * a.ldb);
            if (bm) v = bm[r * a.b_mask_ld] ? v : 0.f;
            s += v;
        }
    }
    sm[ty][tx] = s;
    __syncthreads();
    if (ty == 0 && c < total_cols) {
        float t = 0.f;
#pragma unroll
        for (int i = 0; i < 8; ++i) t += sm[i][tx];
        scratch[(int64_t)blockIdx.y * total_cols + c] = t;
    }
}

__global__ void colsum_reduce_kernel(const float* scratch, int n_chunks, int total_cols, float* out1, float* out2) {
    const int c = blockIdx.x * blockDim.x + threadIdx.x;
    if (c >= total_cols) return;
    float s = 0.f;
    for (int i = 0; i < n_chunks; ++i) s += scratch[(int64_t)i * total_cols + c];
    if (out1) out1[c] = s;
    if (out2) out2[c] = s;
}

void wgrad_plan(int64_t M, int groups, int K, int N, bool bias, int* n_chunks, int64_t* rows_per_chunk, int* Kext) {
    *Kext = K + (bias ? 1 : 0);
    int tiles = ((*Kext + WT - 1) / WT) * ((N + WT - 1) / WT) * groups;
    if (tiles < 1) tiles = 1;
    int64_t want = (148 * 4 + tiles - 1) / tiles;
    int64_t max_chunks = (M + 1023) / 1024;
    if (want > max_chunks) want = max_chunks;
    if (want < 1) want = 1;
    int64_t rpc = (M + want - 1) / want;
    rpc = (rpc + WR - 1) / WR * WR;
    *rows_per_chunk = rpc;
    *n_chunks = (int)((M + rpc - 1) / rpc);
}

// ------------------------------------------------------------------------------ small kernels
__global__ void mask_mul_kernel(int64_t M, int N, const float* in, int64_t ld_in, const uint8_t* mask, int64_t ld_mask,
                                float* out, int64_t ld_out) {
    const int64_t total = M * N;
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < total; i += stride) {
        const int64_t r = i / N;
        const int c = (int)(i % N);
        out[r * ld_out + c] = mask[r * ld_mask + c] ? in[r * ld_in + c] : 0.f;
    }
}

// same, four columns per thread (all leading dimensions and N multiples of 4, 16-byte aligned rows)
__global__ void mask_mul4_kernel(int64_t M, int N4, const float4* in, int64_t ld_in4, const uint32_t* mask, int64_t ld_mask4,
                                 float4* out, int64_t ld_out4) {
    const int64_t total = M * N4;
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    for (; i < total; i += stride) {
        const int64_t r = i / N4;
        const int c = (int)(i - r * N4);
        float4 v = __ldg(in + r * ld_in4 + c);
        const uint32_t m = __ldg(mask + r * ld_mask4 + c);
        if (!(m & 0x000000FFu)) v.x = 0.f;
        if (!(m & 0x0000FF00u)) v.y = 0.f;
        if (!(m & 0x00FF0000u)) v.z = 0.f;
        if (!(m & 0xFF000000u)) v.w = 0.f;
        out[r * ld_out4 + c] = v;
    }
}

// LG lanes per training row (a warp holds 32/LG rows): few classes would leave most of a warp idle.
// A training index outside [0, n) or a label outside [0, C) is never dereferenced: the row is skipped (loss 0, zero
// gradient) and the status word receives kStatusBadLabel.
template <int LG>
__global__ void softmax_ce_kernel(int64_t n, int C, const float* logits, const int32_t* labels, const int32_t* train_idx,
                                  int64_t n_train, float inv_n, float* dlogits, int64_t ld_d, float* row_loss, int* fault) {
    const int lane = threadIdx.x & 31;
    const int sub = lane / LG, sl = lane % LG;
    const int64_t t = ((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5) * (32 / LG) + sub;
    const bool in_set = t < n_train;   // idle groups stay for the shuffles
    int64_t r = in_set ? (train_idx ? (int64_t)train_idx[t] : t) : 0;
    const bool row_ok = r >= 0 && r < n;
    if (!row_ok) r = 0;
    const int y = (in_set && row_ok) ? labels[r] : 0;
    const bool live = in_set && row_ok && y >= 0 && y < C;
    if (in_set && !live && sl == 0) {
        if (fault) atomicExch(fault, kStatusBadLabel);
        row_loss[t] = 0.f;
    }
    const float* z = logits + r * C;
    float mx = -INFINITY;
    if (live)
        for (int c = sl; c < C; c += LG) mx = fmaxf(mx, z[c]);
#pragma unroll
    for (int o = LG / 2; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o, LG));
    float s = 0.f;
    if (live)
        for (int c = sl; c < C; c += LG) s += expf(z[c] - mx);
#pragma unroll
    for (int o = LG / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o, LG);
    if (!in_set || !row_ok) return;
    if (!live) {   // a bad label on a valid row: the row contributes nothing
        for (int c = sl; c < ld_d; c += LG) dlogits[r * ld_d + c] = 0.f;
        return;
    }
    const float lse = mx + logf(s);
    if (sl == 0) row_loss[t] = lse - z[y];
    const float inv_s = 1.f / s;
    for (int c = sl; c < ld_d; c += LG) {
        float v = 0.f;   // padding columns stay zero
        if (c < C) v = (expf(z[c] - mx) * inv_s - (c == y ? 1.f : 0.f)) * inv_n;
        dlogits[r * ld_d + c] = v;
    }
}

// single CTA, fixed summation order: thread t sums elements t, t+1024, ...; then a tree in smem
__global__ void __launch_bounds__(1024) mean_reduce_kernel(const float* v, int64_t n, float scale, float* out) {
    __shared__ float sm[1024];
    float s = 0.f;
    for (int64_t i = threadIdx.x; i < n; i += 1024) s += v[i];
    sm[threadIdx.x] = s;
    __syncthreads();
    for (int o = 512; o > 0; o >>= 1) {
        if (threadIdx.x < o) sm[threadIdx.x] += sm[threadIdx.x + o];
        __syncthreads();
    }
    if (threadIdx.x == 0) *out = sm[0] * scale;
}

__global__ void adam_kernel(int64_t count, float* theta, const float* grad, float* m1, float* m2, float lr, float b1,
                            float b2, float eps, float wd, float c1, float c2) {
    int64_t i = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (i >= count) return;
    const float th = theta[i];
    const float g = grad[i] + wd * th;
    const float m = b1 * m1[i] + (1.f - b1) * g;
    const float v = b2 * m2[i] + (1.f - b2) * g * g;
    m1[i] = m;
    m2[i] = v;
    theta[i] = th - lr * (m / c1) / (sqrtf(v / c2) + eps);
}

// Slices of X copied side by side at aligned starts: out[r, i*w_pad + c] = X[r, start_i + c] for c < w, zero for the
// padding columns (and for the columns between p*w_pad and out_ld).  Overlapping slices get their columns twice.
struct RepackStarts {
    int start[SLICEGCN_MAX_SLICES];
};
template <typename T>
__global__ void repack_slices_kernel(int64_t n, int p, const RepackStarts st, int w, int w_pad, const T* X, int64_t x_ld, T* out,
                                     int64_t out_ld) {
    const int64_t total = n * out_ld;
    for (int64_t e = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = e / out_ld;
        const int c = (int)(e - r * out_ld);
        const int i = c / w_pad, cc = c - i * w_pad;
        T v = T(0.f);
        if (i < p && cc < w) v = X[r * x_ld + st.start[i] + cc];
        out[e] = v;
    }
}

}  // namespace

slicegcn_status_t gemm_run(const GemmArgs& a, cudaStream_t st) {
    if (a.M < 1 || a.groups < 1 || a.groups > SLICEGCN_MAX_SLICES || a.N < 1 || a.K < 0)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "gemm: bad shape");
    static const bool no_tc = getenv("SLICEGCN_NO_TC") != nullptr;   // CUDA-core kernels only (for A/B checks)
    if (a.A2) {   // two products in one pass: tensor-core path only, the caller splits it otherwise
        if (no_tc || !a.fault || !a.b_image || a.K < 1) return SLICEGCN_ERR_UNSUPPORTED;
        return tc_gemm_run(a, st);
    }
    if (!no_tc && a.fault && a.b_image && a.K >= 1 && a.b_image_bytes >= tc_image_bytes(a.groups, a.K, a.N))
        return tc_gemm_run(a, st);
    const bool abf = a.a_dtype == SLICEGCN_BF16, cbf = a.c_dtype == SLICEGCN_BF16;
    if (!abf && !cbf) return gemm_dispatch<float, float>(a, st);
    if (abf && cbf) return gemm_dispatch<__nv_bfloat16, __nv_bfloat16>(a, st);
    if (abf && !cbf) return gemm_dispatch<__nv_bfloat16, float>(a, st);
    return gemm_dispatch<float, __nv_bfloat16>(a, st);
}

int64_t wgrad_scratch_bytes(int64_t M, int groups, int K, int N) {
    // the tensor-core kernel keeps one 128 x (<= 256) partial tile per (row chunk, column tile)
    const int64_t m_tiles = std::max<int64_t>(groups, (K + 127) / 128);
    int64_t best = (148 * 3 + m_tiles) * 128 * 256 * (int64_t)sizeof(float);
    for (int bias = 0; bias < 2; ++bias) {
        int n_chunks, Kext;
        int64_t rpc;
        wgrad_plan(M, groups, K, N, bias != 0, &n_chunks, &rpc, &Kext);
        const int64_t b = (int64_t)n_chunks * groups * Kext * N * (int64_t)sizeof(float);
        if (b > best) best = b;
    }
    return best;
}

// Width of the column blocks wgrad_run cuts a single group's dW into (0: it is not cut).
static int wgrad_col_block(const WgradArgs& a) {
    if (!a.fault || a.K < 1 || !a.dW || a.groups != 1 || a.N % 4 != 0 || a.ldw != 0) return 0;
    if (a.N > 256) return 256;
    if (a.b_mask && a.N > 128 && a.N % 16 == 0 && !tc_wgrad_masks_in_producer(a)) {
        WgradArgs s = a;
        s.N = 128;
        s.ldw = a.N;
        if (tc_wgrad_masks_in_producer(s)) return 128;
    }
    return 0;
}

// Groups per launch when a masked grouped product is too wide for one launch with the mask in the producer but
// fits as several launches over runs of consecutive groups (0: no such split).
static WgradArgs wgrad_group_run(const WgradArgs& a, int g0, int gb) {
    WgradArgs s = a;
    s.groups = gb;
    for (int g = 0; g < gb; ++g) {
        s.a_start[g] = a.a_start[g0 + g];
        s.b_start[g] = a.b_start[g0 + g];
    }
    s.dW = a.dW + (int64_t)g0 * a.K * a.N;
    s.dbias = a.dbias ? a.dbias + g0 * a.N : nullptr;
    s.dbias2 = a.dbias2 ? a.dbias2 + g0 * a.N : nullptr;
    return s;
}

static int wgrad_mask_group_block(const WgradArgs& a) {
    if (!a.fault || !a.b_mask || a.K < 1 || !a.dW || a.groups < 2 || a.ldw != 0 || tc_wgrad_masks_in_producer(a)) return 0;
    for (int gb = a.groups / 2; gb >= 1; gb /= 2) {
        if (a.groups % gb) continue;
        bool ok = true;
        for (int g0 = 0; g0 < a.groups && ok; g0 += gb) ok = tc_wgrad_masks_in_producer(wgrad_group_run(a, g0, gb));
        if (ok) return gb;
    }
    return 0;
}

bool wgrad_masks_in_producer(const WgradArgs& a) {
    if (tc_wgrad_masks_in_producer(a)) return true;
    static const bool no_tc = getenv("SLICEGCN_NO_TC") != nullptr;
    if (no_tc || !a.b_mask) return false;
    return (a.N <= 256 && wgrad_col_block(a) == 128) || wgrad_mask_group_block(a) > 0;
}

slicegcn_status_t wgrad_run(const WgradArgs& a, void* scratch, int64_t scratch_bytes, cudaStream_t st) {
    if (a.M < 1 || a.groups < 1 || a.groups > SLICEGCN_MAX_SLICES || a.N < 1 || a.K < 0)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "wgrad: bad shape");
    const bool bias = a.dbias || a.dbias2;
    if (a.K == 0 && !bias) return SLICEGCN_OK;
    static const bool no_tc = getenv("SLICEGCN_NO_TC") != nullptr;
    // bias-only request over contiguous groups: plain column sums
    if (a.K == 0 && bias) {
        bool contiguous = true;
        for (int g = 0; g < a.groups; ++g) contiguous = contiguous && (a.b_start[g] == a.b_start[0] + g * a.N);
        const int total_cols = a.groups * a.N;
        int64_t rpc = (a.M + 147) / 148;
        rpc = (rpc + 7) / 8 * 8;
        const int n_chunks = (int)((a.M + rpc - 1) / rpc);
        if (contiguous && scratch && scratch_bytes >= (int64_t)n_chunks * total_cols * (int64_t)sizeof(float)) {
            dim3 grid((total_cols + 31) / 32, n_chunks);
            colsum_partial_kernel<<<grid, 256, 0, st>>>(a, total_cols, rpc, static_cast<float*>(scratch));
            SGCN_LAUNCH_CHECK();
            colsum_reduce_kernel<<<(total_cols + 255) / 256, 256, 0, st>>>(static_cast<const float*>(scratch), n_chunks,
                                                                           total_cols, a.dbias, a.dbias2);
            SGCN_LAUNCH_CHECK();
            count_launch(2);
            return SLICEGCN_OK;
        }
    }
    // one group wider than a tensor-core tile (256 result columns; 128 when B carries a byte mask, whose tiles share
    // the kernel's shared memory): column blocks of dW, one launch each
    const int col_block = wgrad_col_block(a);
    if (!no_tc && col_block > 0) {
        bool all = true;
        for (int c0 = 0; c0 < a.N; c0 += col_block) {
            WgradArgs s = a;
            s.N = std::min(col_block, a.N - c0);
            s.b_start[0] = a.b_start[0] + c0;
            s.dW = a.dW + c0;
            s.ldw = a.N;
            s.dbias = a.dbias ? a.dbias + c0 : nullptr;
            s.dbias2 = a.dbias2 ? a.dbias2 + c0 : nullptr;
            bool done_c = false;
            const slicegcn_status_t rc = tc_wgrad_run(s, scratch, scratch_bytes, st, &done_c);
            if (rc == SLICEGCN_ERR_UNSUPPORTED && c0 == 0) {
                all = false;   // nothing was launched: the general path below takes the whole product
                break;
            }
            if (rc != SLICEGCN_OK) return rc;
            if (bias && !done_c) {
                WgradArgs b = s;
                b.K = 0;
                b.dW = nullptr;
                b.fault = nullptr;
                SGCN_TRY(wgrad_run(b, scratch, scratch_bytes, st));
            }
        }
        if (all) return SLICEGCN_OK;
    }
    if (const int gb = no_tc ? 0 : wgrad_mask_group_block(a)) {   // masked, too wide for one launch: runs of gb groups
        for (int g0 = 0; g0 < a.groups; g0 += gb) {
            const WgradArgs s = wgrad_group_run(a, g0, gb);
            bool done_g = false;
            SGCN_TRY(tc_wgrad_run(s, scratch, scratch_bytes, st, &done_g));
            if (bias && !done_g) {
                WgradArgs b = s;
                b.K = 0;
                b.dW = nullptr;
                b.fault = nullptr;
                SGCN_TRY(wgrad_run(b, scratch, scratch_bytes, st));
            }
        }
        return SLICEGCN_OK;
    }
    if (!no_tc && a.fault && a.K >= 1 && a.dW) {
        bool bias_done = false;
        const slicegcn_status_t rc = tc_wgrad_run(a, scratch, scratch_bytes, st, &bias_done);
        if (rc == SLICEGCN_OK) {
            if (!bias || bias_done) return SLICEGCN_OK;
            WgradArgs b = a;     // column sums only
            b.K = 0;
            b.dW = nullptr;
            b.fault = nullptr;
            return wgrad_run(b, scratch, scratch_bytes, st);
        }
        if (rc != SLICEGCN_ERR_UNSUPPORTED) return rc;
        // grouped shapes the tensor-core plan does not take as one launch (slices wider than a tile, widths that
        // need their zero padding): one launch per group
        if (a.groups > 1) {
            bool all = true;
            for (int g = 0; g < a.groups && all; ++g) {
                WgradArgs s = a;
                s.groups = 1;
                s.a_start[0] = a.a_start[g];
                s.b_start[0] = a.b_start[g];
                s.dW = a.dW + (int64_t)g * a.K * a.N;
                s.dbias = a.dbias ? a.dbias + g * a.N : nullptr;
                s.dbias2 = a.dbias2 ? a.dbias2 + g * a.N : nullptr;
                bool done_g = false;
                const slicegcn_status_t rg = tc_wgrad_run(s, scratch, scratch_bytes, st, &done_g);
                if (rg == SLICEGCN_ERR_UNSUPPORTED) {
                    all = false;   // same shape for every group: the first one decides, nothing was launched
                    break;
                }
                if (rg != SLICEGCN_OK) return rg;
                if (bias && !done_g) {
                    WgradArgs b = s;
                    b.K = 0;
                    b.dW = nullptr;
                    b.fault = nullptr;
                    SGCN_TRY(wgrad_run(b, scratch, scratch_bytes, st));
                }
            }
            if (all) return SLICEGCN_OK;
        }
    }
    if (a.ldw != 0 && a.ldw != a.N) SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED, "wgrad: a column block of dW needs the tensor-core path");
    int n_chunks, Kext;
    int64_t rpc;
    wgrad_plan(a.M, a.groups, a.K, a.N, bias, &n_chunks, &rpc, &Kext);
    const int64_t need = (int64_t)n_chunks * a.groups * Kext * a.N * (int64_t)sizeof(float);
    if (!scratch || scratch_bytes < need)
        SGCN_FAIL(SLICEGCN_ERR_ALLOC, "wgrad: scratch too small (%lld < %lld)", (long long)scratch_bytes, (long long)need);
    dim3 grid(n_chunks, ((Kext + WT - 1) / WT) * ((a.N + WT - 1) / WT), a.groups);
    if (a.a_dtype == SLICEGCN_BF16)
        wgrad_partial_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(a, static_cast<float*>(scratch), n_chunks, rpc, Kext);
    else
        wgrad_partial_kernel<float><<<grid, 256, 0, st>>>(a, static_cast<float*>(scratch), n_chunks, rpc, Kext);
    SGCN_LAUNCH_CHECK();
    const int64_t per = (int64_t)a.groups * Kext * a.N;
    wgrad_reduce_kernel<<<(unsigned)((per + 255) / 256), 256, 0, st>>>(static_cast<const float*>(scratch), n_chunks,
                                                                      a.groups, a.K, Kext, a.N, a.dW, a.dbias, a.dbias2);
    SGCN_LAUNCH_CHECK();
    count_launch(2);
    return SLICEGCN_OK;
}

slicegcn_status_t repack_slices_run(int64_t n, int p, const int* starts, int w, int w_pad, const void* X, int64_t x_ld, int dtype,
                                    void* out, int64_t out_ld, cudaStream_t st) {
    RepackStarts rs;
    for (int i = 0; i < SLICEGCN_MAX_SLICES; ++i) rs.start[i] = i < p ? starts[i] : 0;
    const int64_t total = n * out_ld;
    const unsigned blocks = (unsigned)std::min<int64_t>((total + 255) / 256, 148 * 32);
    if (dtype == SLICEGCN_BF16)
        repack_slices_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(n, p, rs, w, w_pad, static_cast<const __nv_bfloat16*>(X), x_ld,
                                                                    static_cast<__nv_bfloat16*>(out), out_ld);
    else
        repack_slices_kernel<float><<<blocks, 256, 0, st>>>(n, p, rs, w, w_pad, static_cast<const float*>(X), x_ld, static_cast<float*>(out),
                                                            out_ld);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

// Parameter tensors between the caller's layout (blocks of r x c) and the padded internal one (blocks of rp x cp, the
// extra rows and columns zero).  One launch covers every tensor: blockIdx.y picks the table entry.
template <bool PAD>
__global__ void pad_params_kernel(const PadTable t, const float* src, float* dst) {
    const PadEntry e = t.e[blockIdx.y];
    // PAD: every element of the padded tensor is written (padding as zero); else: every element of the caller's tensor
    const int64_t total = (int64_t)e.blocks * (PAD ? (int64_t)e.rp * e.cp : (int64_t)e.r * e.c);
    for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < total; k += (int64_t)gridDim.x * blockDim.x) {
        const int cols = PAD ? e.cp : e.c, rows = PAD ? e.rp : e.r;
        const int64_t per = (int64_t)rows * cols;
        const int64_t blk = k / per, rem = k - blk * per;
        const int i = (int)(rem / cols), j = (int)(rem - (int64_t)i * cols);
        if (PAD) {
            float v = 0.f;
            if (i < e.r && j < e.c) v = src[e.outer + (blk * e.r + i) * e.c + j];
            dst[e.inner + k] = v;
        } else {
            dst[e.outer + k] = src[e.inner + (blk * e.rp + i) * e.cp + j];
        }
    }
}

slicegcn_status_t pad_params_run(const PadTable& t, bool pad, const float* src, float* dst, cudaStream_t st) {
    if (t.count < 1) return SLICEGCN_OK;
    dim3 grid(64, t.count);
    if (pad)
        pad_params_kernel<true><<<grid, 256, 0, st>>>(t, src, dst);
    else
        pad_params_kernel<false><<<grid, 256, 0, st>>>(t, src, dst);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

template <typename T>
__global__ void dropout_apply_kernel(int64_t n, int cols, T* data, int64_t ld, const uint8_t* mask, int64_t mask_ld, int h_s,
                                     int hp, float scale) {
    const int64_t total = n * cols;
    for (int64_t k = blockIdx.x * (int64_t)blockDim.x + threadIdx.x; k < total; k += (int64_t)gridDim.x * blockDim.x) {
        const int64_t r = k / cols;
        const int c = (int)(k - r * cols);
        const int blk = c / hp, j = c - blk * hp;
        if (j >= h_s) continue;   // padding column of the internal layout
        T* d = data + r * ld + c;
        const float v = mask[r * mask_ld + blk * h_s + j] ? (float)*d * scale : 0.f;
        *d = (T)v;
    }
}

slicegcn_status_t dropout_apply_run(int64_t n, int cols, void* data, int64_t ld, int dtype, const uint8_t* mask, int64_t mask_ld,
                                    int h_s, int hp, float scale, cudaStream_t st) {
    const unsigned blocks = (unsigned)std::min<int64_t>((n * cols + 255) / 256, 148 * 32);
    if (dtype == SLICEGCN_BF16)
        dropout_apply_kernel<__nv_bfloat16><<<blocks, 256, 0, st>>>(n, cols, static_cast<__nv_bfloat16*>(data), ld, mask, mask_ld, h_s, hp, scale);
    else
        dropout_apply_kernel<float><<<blocks, 256, 0, st>>>(n, cols, static_cast<float*>(data), ld, mask, mask_ld, h_s, hp, scale);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

slicegcn_status_t mask_mul_run(int64_t M, int N, const float* in, int64_t ld_in, const uint8_t* mask, int64_t ld_mask,
                               float* out, int64_t ld_out, cudaStream_t st) {
    int64_t blocks = (M * N + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    const bool vec = N % 4 == 0 && ld_in % 4 == 0 && ld_out % 4 == 0 && ld_mask % 4 == 0 && (uintptr_t)in % 16 == 0 &&
                     (uintptr_t)out % 16 == 0 && (uintptr_t)mask % 4 == 0;
    if (vec)
        mask_mul4_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N / 4, reinterpret_cast<const float4*>(in), ld_in / 4,
                                                           reinterpret_cast<const uint32_t*>(mask), ld_mask / 4,
                                                           reinterpret_cast<float4*>(out), ld_out / 4);
    else
        mask_mul_kernel<<<(unsigned)blocks, 256, 0, st>>>(M, N, in, ld_in, mask, ld_mask, out, ld_out);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

slicegcn_status_t softmax_ce_run(int64_t n, int C, const float* logits, const int32_t* labels, const int32_t* train_idx,
                                 int64_t n_train, float* dlogits, int64_t ld_d, float* row_loss, float* loss_out,
                                 int* fault, cudaStream_t st) {
    if (train_idx) SGCN_CUDA(cudaMemsetAsync(dlogits, 0, sizeof(float) * n * ld_d, st));
    const int64_t cnt = train_idx ? n_train : n;
    if (cnt < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "empty training set");
    if (C <= 64)
        softmax_ce_kernel<8><<<(unsigned)((cnt + 31) / 32), 256, 0, st>>>(n, C, logits, labels, train_idx, cnt, 1.0f / (float)cnt,
                                                                          dlogits, ld_d, row_loss, fault);
    else
        softmax_ce_kernel<32><<<(unsigned)((cnt + 7) / 8), 256, 0, st>>>(n, C, logits, labels, train_idx, cnt, 1.0f / (float)cnt,
                                                                         dlogits, ld_d, row_loss, fault);
    SGCN_LAUNCH_CHECK();
    count_launch();
    if (loss_out) {
        mean_reduce_kernel<<<1, 1024, 0, st>>>(row_loss, cnt, 1.0f / (float)cnt, loss_out);
        SGCN_LAUNCH_CHECK();
        count_launch();
    }
    return SLICEGCN_OK;
}

slicegcn_status_t adam_run(int64_t count, float* theta, const float* grad, float* m1, float* m2, float lr, float beta1,
                           float beta2, float eps, float weight_decay, int step, cudaStream_t st) {
    const float c1 = (float)(1.0 - pow((double)beta1, (double)step));
    const float c2 = (float)(1.0 - pow((double)beta2, (double)step));
    adam_kernel<<<(unsigned)((count + 255) / 256), 256, 0, st>>>(count, theta, grad, m1, m2, lr, beta1, beta2, eps,
                                                                  weight_decay, c1, c2);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

}  // namespace sgcn
