// Tensor-core (tcgen05) versions of the dense kernels of the layer: the grouped row-panel GEMM with
// the fused epilogues of Eq. 6-7 and the grouped weight gradient.
//
// fp32 operands use the tf32 path three times (hi*hi + lo*hi + hi*lo with hi = the value rounded to
// 10 mantissa bits, lo = value - hi), which keeps ~21 mantissa bits -- single-pass tf32 would miss the
// 1e-4 parity bound.  bf16 operands use one kind::f16 pass per weight part.  Accumulators live in
// tensor memory (TMEM) and come back through tcgen05.ld for the epilogue.
//
// Two generations of kernels share the contracts in kernels.cuh:
//   * tc_gemm_ts_kernel / tc_wgrad_ts_kernel (fp32 and bf16 activations): slabs arrive by tensor copy
//     (TMA), the activation operand (split into hi / lo when fp32) is written to TMEM with tcgen05.st
//     and the MMAs read it from there; only the small weight operand (a prepared image) or the B slab
//     of the weight gradient is an operand tile in shared memory.
//   * tc_gemm_ws_kernel / tc_gemm_kernel / tc_wgrad_ws_kernel / tc_wgrad_kernel: both operands staged in
//     shared memory in the canonical swizzled layouts that a tcgen05 matrix descriptor reads, written
//     with ordinary stores followed by a proxy fence (unaligned operands, odd output widths, masks
//     the first generation does not take).
// Every wait on an mbarrier is bounded; a wait that runs out sets the caller's status word.
#include <cuda.h>

#include <algorithm>
#include <cstdlib>
#include <type_traits>
#include <vector>

#include "common.cuh"
#include "kernels.cuh"

namespace sgcn {

constexpr int kMaxPrepJobs = 40;
struct PrepJob {            // one weight operand to convert: the B-side fields of a GemmArgs plus where the image goes
    const float* B;
    int64_t b_gstride;
    int ldb, b_trans, K, N, n_pad, n_slabs, n_tiles, groups, bf16, kstack;
    unsigned char* image;
    int block0;             // first block of this job in a batched launch
};


// Weight images of one model, kept across the GEMMs and the epochs of a training run.  A GEMM that
// finds its weight operand here skips the conversion; slicegcn_train_epoch converts every image
// recorded so far in ONE launch when the epoch starts (the weights change once per epoch) instead of
// one small launch in front of every GEMM.  Entries are keyed by the exact weight pointer and shape
// and live in a region of the caller's workspace; a different region, or weights outside the
// current parameter buffer, drop the entry.  Not thread-safe (one training run per model).
struct TcImageCache {
    unsigned char* region = nullptr;
    int64_t region_bytes = 0, used = 0;
    struct Entry {
        PrepJob job;
        bool fresh;
    };
    std::vector<Entry> entries;
};

namespace {

constexpr int kWaitSpins = 1 << 22;

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ bool mbar_test(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t ok;   // may suspend the thread for a short, hardware-bounded time before returning
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up (returns false) after kWaitSpins attempts or about two seconds.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    if (mbar_test(bar, parity)) return true;
    const long long t0 = clock64();
    for (int i = 0; i < kWaitSpins; ++i) {
        if (mbar_try(bar, parity)) return true;
        if ((i & 63) == 63 && clock64() - t0 > 4000000000LL) break;   // (a spinning warp shares its issue slots with working ones)
    }
    return false;
}

__device__ __forceinline__ void tmem_alloc(uint32_t* dst_smem, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(dst_smem)), "r"(ncols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// D[tmem] (+)= A[smem desc] * B[smem desc]
template <bool BF16>
__device__ __forceinline__ void umma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    if (BF16) {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    } else {
        asm volatile(
            "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
            "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}" ::"r"(d_tmem),
            "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
            : "memory");
    }
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// contiguous global -> shared copy by the bulk-copy engine; completion is counted on the mbarrier
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst)),
                 "l"(src), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
__device__ __forceinline__ void umma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
// 32 lanes x 32 columns of fp32: thread t of the warp receives row (lane base + t), columns col..col+31
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

// The same load without the wait, so that several can be in flight; tmem_ld_wait() before the values are used.
__device__ __forceinline__ void tmem_ld32_issue(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]),
          "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]),
          "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
// 32 lanes x 16 columns, registers r[OFF..OFF+15] -> TMEM: thread t of the warp writes row (lane base + t),
// columns col..col+15
template <int OFF>
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};" ::"r"(taddr),
        "r"(r[OFF + 0]), "r"(r[OFF + 1]), "r"(r[OFF + 2]), "r"(r[OFF + 3]), "r"(r[OFF + 4]), "r"(r[OFF + 5]), "r"(r[OFF + 6]),
        "r"(r[OFF + 7]), "r"(r[OFF + 8]), "r"(r[OFF + 9]), "r"(r[OFF + 10]), "r"(r[OFF + 11]), "r"(r[OFF + 12]), "r"(r[OFF + 13]),
        "r"(r[OFF + 14]), "r"(r[OFF + 15])
        : "memory");
}
// 32 lanes x 16 columns of fp32, added onto x[OFF..OFF+15]
template <int OFF>
__device__ __forceinline__ void tmem_ld16_add(uint32_t taddr, float (&x)[32]) {
    uint32_t r[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) x[OFF + i] += __uint_as_float(r[i]);
}
// two loads of 32 lanes x 16 columns in flight, both added onto x[OFF..OFF+15]
template <int OFF>
__device__ __forceinline__ void tmem_ld16x2_add(uint32_t taddr0, uint32_t taddr1, float (&x)[32]) {
    uint32_t r[16], q[16];
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
          "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr0));
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
        : "=r"(q[0]), "=r"(q[1]), "=r"(q[2]), "=r"(q[3]), "=r"(q[4]), "=r"(q[5]), "=r"(q[6]), "=r"(q[7]), "=r"(q[8]), "=r"(q[9]),
          "=r"(q[10]), "=r"(q[11]), "=r"(q[12]), "=r"(q[13]), "=r"(q[14]), "=r"(q[15])
        : "r"(taddr1));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) x[OFF + i] += __uint_as_float(r[i]) + __uint_as_float(q[i]);
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// the same for 16-bit operands (bf16): two K values per TMEM column
__device__ __forceinline__ void umma_ts_f16(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// D[tmem] (+)= A[tmem] * B[smem desc], tf32: A's row i sits in TMEM lane i, its K values in consecutive columns
__device__ __forceinline__ void umma_ts_tf32(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n\t}" ::"r"(d_tmem),
        "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// One box of a 2-D tensor map, global -> shared, by the tensor copy engine; completion (bytes) is
// counted on the mbarrier.  x (the contiguous coordinate) times the element size must be a multiple
// of 16 bytes; rows or columns outside the tensor arrive as zeros.
__device__ __forceinline__ void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];" ::"r"(
                     smem_u32(dst)),
                 "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar))
                 : "memory");
}

// K-major, 128-byte swizzle: rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t smem_desc(const void* tile) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_u32(tile) >> 4) & 0x3FFF);   // start address
    d |= (uint64_t)1 << 16;                            // leading byte offset (unused with swizzle): 1
    d |= (uint64_t)(1024 >> 4) << 32;                  // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;                            // descriptor version
    d |= (uint64_t)2 << 61;                            // SWIZZLE_128B
    return d;
}
// byte offset of 4-byte element (row, k) [k < 32] or 2-byte element [k < 64] inside a swizzled tile
__device__ __forceinline__ uint32_t sw_off(int row, int byte_in_row) {
    const int chunk = (byte_in_row >> 4) ^ (row & 7);
    return (uint32_t)(row * 128 + (chunk << 4) + (byte_in_row & 15));
}
__device__ __forceinline__ uint32_t idesc_f32acc(int M, int N, bool bf16) {
    const uint32_t fmt = bf16 ? 1u : 2u;   // BF16 : TF32
    return (1u << 4) | (fmt << 7) | (fmt << 10) | ((uint32_t)(N >> 3) << 17) | ((uint32_t)(M >> 4) << 24);
}

__device__ __forceinline__ float ld_as_f(const float* p) { return __ldg(p); }
__device__ __forceinline__ float ld_as_f(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// nearest value with a 10-bit mantissa (what the tf32 path keeps)
__device__ __forceinline__ float tf32_hi(float v) {
    // round half up in magnitude on the 13 dropped bits; Inf stays Inf, NaN stays NaN
    return __uint_as_float((__float_as_uint(v) + 0x1000u) & 0xFFFFE000u);
}
// stores one fp32 operand value into the hi / lo tiles (tf32 split) or one bf16 value
__device__ __forceinline__ void put_f32(unsigned char* hi, unsigned char* lo, int row, int k, float v) {
    const float h = tf32_hi(v);
    const uint32_t off = sw_off(row, k * 4);
    *reinterpret_cast<float*>(hi + off) = h;
    *reinterpret_cast<float*>(lo + off) = v - h;
}
__device__ __forceinline__ void put_bf16(unsigned char* t, int row, int k, float v) {
    *reinterpret_cast<__nv_bfloat16*>(t + sw_off(row, k * 2)) = __float2bfloat16_rn(v);
}
// fp32 weight as two bf16 values (hi + lo keeps ~16 mantissa bits); the activation operand is exact in bf16
__device__ __forceinline__ void put_bf16x2(unsigned char* hi, unsigned char* lo, int row, int k, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    const uint32_t off = sw_off(row, k * 2);
    *reinterpret_cast<__nv_bfloat16*>(hi + off) = h;
    *reinterpret_cast<__nv_bfloat16*>(lo + off) = __float2bfloat16_rn(v - __bfloat162float(h));
}

// ------------------------------------------------------------------------------ weight images
// The B operand (a small weight block) is the same for every row tile, so it is converted once per
// GEMM into the exact bytes a shared-memory tile holds -- K-major rows of 128 bytes, swizzled, split
// into hi and lo -- and every CTA then pulls a slab's image with one bulk copy.
// Image of (group g, n tile nt, K slab s): [hi: n_pad rows x 128 B][lo: n_pad rows x 128 B].
// One quarter (part) of the image of (group g, n tile nt, K slab s).
template <bool BF16>
__device__ __forceinline__ void prep_image_block(const PrepJob& j, int s, int part, int nt, int g) {
    constexpr int KS = BF16 ? 64 : 32;
    const float* B = j.B + (int64_t)g * j.b_gstride;
    unsigned char* hi = j.image + ((((int64_t)g * j.n_tiles + nt) * j.n_slabs + s) * 2) * ((int64_t)j.n_pad * 128);
    unsigned char* lo = hi + (int64_t)j.n_pad * 128;
    const int n0 = nt * j.n_pad, k0 = s * KS;
    const int per = (j.n_pad * KS + 3) / 4;   // this block's quarter of the tile's elements
    for (int e = part * per + threadIdx.x; e < min((part + 1) * per, j.n_pad * KS); e += 128) {
        int n, kk;
        if (j.b_trans) {
            kk = e % KS;
            n = e / KS;
        } else {
            n = e % j.n_pad;
            kk = e / j.n_pad;
        }
        const int k = k0 + kk, col = n0 + n;
        float v = 0.f;
        if (col < j.N && k < j.K) {
            const float* Bq = B;
            int kj = k;
            if (j.kstack > 0) {   // K stacked over weight blocks
                Bq = B + (int64_t)(k / j.kstack) * j.b_gstride;
                kj = k % j.kstack;
            }
            v = j.b_trans ? __ldg(Bq + (int64_t)col * j.ldb + kj) : __ldg(Bq + (int64_t)kj * j.ldb + col);
        }
        if (BF16)
            put_bf16x2(hi, lo, n, kk, v);
        else
            put_f32(hi, lo, n, kk, v);
    }
}

template <bool BF16>
__global__ void __launch_bounds__(128) tc_prep_b_kernel(const PrepJob j) {
    prep_image_block<BF16>(j, blockIdx.x / 4, blockIdx.x % 4, blockIdx.y, blockIdx.z);
}

// All images of a training epoch in one launch: block b belongs to the job with block0 <= b < next block0.
struct PrepBatch {
    PrepJob job[kMaxPrepJobs];
    int count;
};
__global__ void __launch_bounds__(128) tc_prep_batch_kernel(const __grid_constant__ PrepBatch batch) {
    int ji = 0;
    while (ji + 1 < batch.count && (int)blockIdx.x >= batch.job[ji + 1].block0) ++ji;
    const PrepJob& j = batch.job[ji];
    int b = (int)blockIdx.x - j.block0;
    const int per_g = j.n_slabs * 4 * j.n_tiles;
    const int g = b / per_g;
    b -= g * per_g;
    const int nt = b / (j.n_slabs * 4);
    b -= nt * (j.n_slabs * 4);
    if (j.bf16)
        prep_image_block<true>(j, b / 4, b % 4, nt, g);
    else
        prep_image_block<false>(j, b / 4, b % 4, nt, g);
}

// ------------------------------------------------------------------------------ row-panel GEMM
// Persistent CTAs (128 threads) walk work items (128-row tile, n tile of up to 256 columns, group).
// K is walked in slabs of one swizzle row (32 fp32 / 64 bf16 values).  Per slab: the weight image
// arrives by bulk copy into one of two buffers; the activation slab, fetched into registers one step
// ahead, is split and stored to shared memory; one elected thread issues the MMAs.  The global loads
// of the next slab (or next item) are in flight while the MMAs run and while the finished item's
// accumulators go TMEM -> registers -> per-warp staging tile -> global memory in whole 128-byte rows.
constexpr int kTcThreads = 128;
constexpr int kStagePitch = 36;   // floats per staged row: 16-byte aligned rows, few bank conflicts either way

template <typename TA, typename TC, bool BF16, bool VEC>
__global__ void __launch_bounds__(kTcThreads) tc_gemm_kernel(const GemmArgs a, const int n_pad, const int n_tiles,
                                                             const unsigned char* image, int* fault) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int KS = BF16 ? 64 : 32;          // K values per slab
    constexpr int UK = BF16 ? 16 : 8;           // K values per MMA
    constexpr int EPC = BF16 ? 8 : 4;           // elements per 16-byte chunk
    constexpr int NLD = VEC ? 8 : (BF16 ? 64 : 32);   // register slots of the prefetched slab
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // the swizzled tiles need 1024-byte alignment; the launch reserves the slack
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    unsigned char* A_hi = base;
    unsigned char* A_lo = base + 16384;
    unsigned char* Bbuf = base + (BF16 ? 16384 : 32768);           // two buffers of [hi | lo]
    const uint32_t slab_bytes = 2u * (uint32_t)n_pad * 128u;
    float* stage = reinterpret_cast<float*>(Bbuf + 2 * slab_bytes) + warp * (32 * kStagePitch);
    unsigned char* tail = Bbuf + 2 * slab_bytes + 4 * 32 * kStagePitch * 4;
    uint64_t* mbar_mma = reinterpret_cast<uint64_t*>(tail);
    uint64_t* mbar_b = reinterpret_cast<uint64_t*>(tail + 8);      // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 24);
    const int n_mma_max = n_pad;
    uint32_t ncols = 32;
    while ((int)ncols < n_mma_max) ncols <<= 1;
    if (tid == 0) {
        mbar_init(mbar_mma, 1);
        mbar_init(&mbar_b[0], 1);
        mbar_init(&mbar_b[1], 1);
    }
    if (warp == 0) tmem_alloc(tmem_slot, ncols);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int n_slabs = (a.K + KS - 1) / KS;
    const int64_t row_tiles = (a.M + 127) / 128;
    const int64_t n_items = row_tiles * a.groups * n_tiles;
    // item -> (row tile, group, n tile): groups and n tiles of one row tile are adjacent
    auto decode = [&](int64_t item, int64_t& row0, int& g, int& nt) {
        nt = (int)(item % n_tiles);
        g = (int)((item / n_tiles) % a.groups);
        row0 = (item / ((int64_t)n_tiles * a.groups)) * 128;
    };
    // prefetch of one activation slab into registers
    uint4 pre[VEC ? 8 : 1];
    float pres[VEC ? 1 : NLD];
    auto prefetch = [&](int64_t row0, int g, int s) {
        const TA* A = static_cast<const TA*>(a.A) + a.a_start[g];
        const uint8_t* am = a.a_mask ? a.a_mask + a.a_start[g] : nullptr;
        const int k0 = s * KS;
        if (VEC) {
            const int c = tid & 7;
            const int k = k0 + c * EPC;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int64_t row = row0 + (tid >> 3) + 16 * i;
                uint4 raw = make_uint4(0, 0, 0, 0);
                if (row < a.M && k < a.K) {
                    raw = __ldg(reinterpret_cast<const uint4*>(A + row * a.lda + k));
                    if (am) {
                        if (BF16) {
                            const uint2 m8 = *reinterpret_cast<const uint2*>(am + row * a.a_mask_ld + k);
                            uint32_t* w = reinterpret_cast<uint32_t*>(&raw);
                            const uint32_t mm[2] = {m8.x, m8.y};
#pragma unroll
                            for (int q = 0; q < 4; ++q) {
                                const uint32_t b0 = (mm[q >> 1] >> (16 * (q & 1))) & 0xFFu;
                                const uint32_t b1 = (mm[q >> 1] >> (16 * (q & 1) + 8)) & 0xFFu;
                                w[q] &= (b0 ? 0x0000FFFFu : 0u) | (b1 ? 0xFFFF0000u : 0u);
                            }
                        } else {
                            const uint32_t m4 = *reinterpret_cast<const uint32_t*>(am + row * a.a_mask_ld + k);
                            if (!(m4 & 0x000000FFu)) raw.x = 0;
                            if (!(m4 & 0x0000FF00u)) raw.y = 0;
                            if (!(m4 & 0x00FF0000u)) raw.z = 0;
                            if (!(m4 & 0xFF000000u)) raw.w = 0;
                        }
                    }
                }
                pre[i] = raw;
            }
        } else {
            // any alignment: warp w takes rows w, w+4, ...; a warp reads one row's KS values
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                const int64_t row = row0 + warp + 4 * i;
#pragma unroll
                for (int q = 0; q < KS / 32; ++q) {
                    const int k = k0 + lane + 32 * q;
                    float v = 0.f;
                    if (row < a.M && k < a.K) {
                        v = ld_as_f(A + row * a.lda + k);
                        if (am) v = am[row * a.a_mask_ld + k] ? v : 0.f;
                    }
                    pres[i * (KS / 32) + q] = v;
                }
            }
        }
    };
    auto store_slab = [&]() {
        if (VEC) {
            const int c = tid & 7;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = (tid >> 3) + 16 * i;
                const uint32_t off = sw_off(r, c * 16);
                if (BF16) {
                    *reinterpret_cast<uint4*>(A_hi + off) = pre[i];
                } else {
                    const float v0 = __uint_as_float(pre[i].x), v1 = __uint_as_float(pre[i].y);
                    const float v2 = __uint_as_float(pre[i].z), v3 = __uint_as_float(pre[i].w);
                    const float h0 = tf32_hi(v0), h1 = tf32_hi(v1), h2 = tf32_hi(v2), h3 = tf32_hi(v3);
                    *reinterpret_cast<float4*>(A_hi + off) = make_float4(h0, h1, h2, h3);
                    *reinterpret_cast<float4*>(A_lo + off) = make_float4(v0 - h0, v1 - h1, v2 - h2, v3 - h3);
                }
            }
        } else {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
#pragma unroll
                for (int q = 0; q < KS / 32; ++q) {
                    const float v = pres[i * (KS / 32) + q];
                    if (BF16)
                        put_bf16(A_hi, warp + 4 * i, lane + 32 * q, v);
                    else
                        put_f32(A_hi, A_lo, warp + 4 * i, lane + 32 * q, v);
                }
            }
        }
    };
    auto image_of = [&](int g, int nt, int s) {
        return image + ((((int64_t)g * n_tiles + nt) * n_slabs + s)) * (int64_t)slab_bytes;
    };

    uint32_t mma_phase = 0, b_phase = 0;   // b_phase: bit i = parity of weight buffer i
    bool ok = true;
    int64_t item = blockIdx.x;
    int64_t row0 = 0;
    int g = 0, nt = 0;
    int bsel = 0;   // weight buffer of the slab about to run
    if (item < n_items) {
        decode(item, row0, g, nt);
        if (tid == 0) {
            mbar_expect_tx(&mbar_b[0], slab_bytes);
            bulk_g2s(Bbuf, image_of(g, nt, 0), slab_bytes, &mbar_b[0]);
        }
        prefetch(row0, g, 0);
    }
    while (item < n_items && ok) {
        const int n0 = nt * n_pad;
        const int nn = min(n_pad, a.N - n0);
        const int n_mma = (nn + 15) & ~15;
        const uint32_t idesc = idesc_f32acc(128, n_mma, BF16);
        // the item after this one (its first slab is prefetched during this item's last slab)
        const int64_t nitem = item + gridDim.x;
        int64_t nrow0 = 0;
        int ng = 0, nnt = 0;
        if (nitem < n_items) decode(nitem, nrow0, ng, nnt);
        for (int s = 0; s < n_slabs && ok; ++s) {
            store_slab();
            proxy_fence();          // generic-proxy stores -> visible to the tensor core's async proxy
            tc_fence_before();
            __syncthreads();
            if (tid == 0) {
                if (mbar_wait(&mbar_b[bsel], (b_phase >> bsel) & 1u)) {
                    tc_fence_after();
                    unsigned char* B_hi = Bbuf + bsel * slab_bytes;
                    const uint64_t da_hi = smem_desc(A_hi), da_lo = smem_desc(A_lo);
                    const uint64_t db_hi = smem_desc(B_hi), db_lo = smem_desc(B_hi + n_pad * 128);
#pragma unroll
                    for (int ks = 0; ks < KS / UK; ++ks) {
                        const uint64_t adv = (uint64_t)((ks * 32) >> 4);   // 32 bytes per MMA along K
                        const uint32_t first = (s == 0 && ks == 0) ? 0u : 1u;
                        umma<BF16>(tmem, da_hi + adv, db_hi + adv, idesc, first);
                        if (!BF16) umma<BF16>(tmem, da_lo + adv, db_hi + adv, idesc, 1u);
                        umma<BF16>(tmem, da_hi + adv, db_lo + adv, idesc, 1u);
                    }
                } else {
                    atomicExch(fault, 3);
                }
                umma_commit(mbar_mma);   // arrives when the MMAs above have read smem and written TMEM
                // weight image of the next slab into the other buffer (its last reader finished before
                // this slab's stores began)
                const bool more = (s + 1 < n_slabs) || (nitem < n_items);
                if (more) {
                    const unsigned char* src = (s + 1 < n_slabs) ? image_of(g, nt, s + 1) : image_of(ng, nnt, 0);
                    mbar_expect_tx(&mbar_b[bsel ^ 1], slab_bytes);
                    bulk_g2s(Bbuf + (bsel ^ 1) * slab_bytes, src, slab_bytes, &mbar_b[bsel ^ 1]);
                }
            }
            b_phase ^= (1u << bsel);
            bsel ^= 1;
            // global loads of the next slab fly while the MMAs run
            if (s + 1 < n_slabs)
                prefetch(row0, g, s + 1);
            else if (nitem < n_items)
                prefetch(nrow0, ng, 0);
            ok = mbar_wait(mbar_mma, mma_phase);
            mma_phase ^= 1u;
            tc_fence_after();
        }
        if (!ok) break;
        // epilogue: warp w owns TMEM lanes 32w..32w+31 = rows row0+32w..; staged so that every global
        // access is one whole row segment (32 consecutive columns)
        TC* C = static_cast<TC*>(a.C);
        const int cs = a.c_start[g] + n0;
        for (int c0 = 0; c0 < n_mma; c0 += 32) {
            float v[32];
            tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
            for (int j = 0; j < 32; ++j) stage[lane * kStagePitch + j] = v[j];
            __syncwarp();
            const int n = c0 + lane;          // this lane's column within the tile
            const bool col_ok = n < nn;
            const int col = cs + n;
            float bias = 0.f, post = 0.f;
            if (col_ok) {
                if (a.bias) bias = __ldg(a.bias + g * a.N + n0 + n);
                if (a.post1) post += __ldg(a.post1 + g * a.N + n0 + n);
                if (a.post2) post += __ldg(a.post2 + g * a.N + n0 + n);
            }
            // operands the epilogue reads back (previous C, ReLU gate): all 32 rows requested up front
            float cold[32], gate[32];
            if (a.accumulate) {
#pragma unroll
                for (int r = 0; r < 32; ++r) {
                    const int64_t row = row0 + warp * 32 + r;
                    cold[r] = (row < a.M && col_ok) ? ld_as_f(C + row * a.ldc + col) : 0.f;
                }
            }
            if (a.mul_pos) {
#pragma unroll
                for (int r = 0; r < 32; ++r) {
                    const int64_t row = row0 + warp * 32 + r;
                    float pv = 1.f;
                    if (row < a.M && col_ok)
                        pv = a.mul_pos_dtype == SLICEGCN_F32
                                 ? __ldg(static_cast<const float*>(a.mul_pos) + row * a.mul_pos_ld + col)
                                 : a.mul_pos_dtype == kGateBytes
                                       ? (float)__ldg(static_cast<const uint8_t*>(a.mul_pos) + row * a.mul_pos_ld + col)
                                       : __bfloat162float(static_cast<const __nv_bfloat16*>(a.mul_pos)[row * a.mul_pos_ld + col]);
                    gate[r] = pv;
                }
            }
#pragma unroll
            for (int r = 0; r < 32; ++r) {
                const int64_t row = row0 + warp * 32 + r;
                if (row >= a.M || !col_ok) continue;
                float x = stage[r * kStagePitch + lane] + bias;
                if (a.relu) {
                    if (a.mask_out) a.mask_out[row * a.mask_ld + col] = x > 0.f ? 1 : 0;
                    x = fmaxf(x, 0.f);
                }
                x += post;
                if (a.mul_pos) x = gate[r] > 0.f ? x : 0.f;
                if (a.accumulate) x += cold[r];
                if (sizeof(TC) == 4)
                    reinterpret_cast<float*>(C)[row * a.ldc + col] = x;
                else
                    reinterpret_cast<__nv_bfloat16*>(C)[row * a.ldc + col] = __float2bfloat16_rn(x);
            }
            __syncwarp();
        }
        tc_fence_before();   // TMEM reads done before the next item's first MMA overwrites the accumulator
        item = nitem;
        row0 = nrow0;
        g = ng;
        nt = nnt;
    }
    if (!ok && tid == 0) atomicExch(fault, 3);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, ncols);
}

// Cursor over a CTA's work items (item = first + i * stride; the host keeps the item count below
// 2^31): row tile, group and column tile follow by additions, so nothing on the per-step paths of
// the persistent kernels divides.
struct ItemCursor {
    uint32_t rt, rem, dq, dr, per_row;
    int n_tiles, g, nt;
    int flip = -1;   // >= 0: row tiles are visited from the last one (index flip) down
    __device__ void init(uint32_t first, uint32_t stride, int groups, int n_tiles_) {
        n_tiles = n_tiles_;
        per_row = (uint32_t)(n_tiles * groups);
        rt = first / per_row;
        rem = first - rt * per_row;
        dq = stride / per_row;
        dr = stride - dq * per_row;
        split();
    }
    __device__ void split() {
        if (n_tiles == 1) {
            g = (int)rem;
            nt = 0;
        } else {
            g = (int)(rem / (uint32_t)n_tiles);
            nt = (int)(rem - (uint32_t)g * (uint32_t)n_tiles);
        }
    }
    __device__ void next() {
        rem += dr;
        rt += dq;
        if (rem >= per_row) {
            rem -= per_row;
            ++rt;
        }
        split();
    }
    __device__ int64_t row0() const { return (int64_t)(flip >= 0 ? (uint32_t)flip - rt : rt) * 128; }
};


// ------------------------------------------------------------------------------ row-panel GEMM, warp-specialised
// The same contract as tc_gemm_kernel, for 16-byte-aligned, unmasked operands.  One persistent CTA per
// SM, nine warps in three roles connected by mbarriers (every wait is bounded):
//   warps 0-3  producers: stream the activation slab of up to D-1 future steps into the stage ring
//              with cp.async (16-byte chunks, written straight into the swizzled tile), and, for the
//              step that has landed, split each fp32 chunk into its tf32 hi part (in place) and lo
//              part; thread 0 also requests the step's weight image by bulk copy into the same stage;
//   warp  4    MMA: one thread waits for a full stage, issues the tcgen05.mma chain into one of two
//              TMEM accumulators and commits -- to the stage's "free" barrier after every slab, to
//              the accumulator's "full" barrier after an item's last slab;
//   warps 5-8  epilogue: drain a finished accumulator (tcgen05.ld), hand it back, then apply the
//              fused epilogue and write whole 128-byte row segments.
// Loads, MMAs and the epilogue of neighbouring items therefore overlap inside one CTA, and the
// bytes in flight are set by the ring depth, not by the register file.
constexpr int kWsThreads = 288;
constexpr int kWsVecFloats = 1024;   // bias / post vectors up to this many floats are staged in shared memory

template <typename TA, typename TC, bool BF16>
__global__ void __launch_bounds__(kWsThreads, 1) tc_gemm_ws_kernel(const GemmArgs a, const int n_pad, const int n_tiles,
                                                                   const int D, const unsigned char* image,
                                                                   const unsigned char* image2, int* fault) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int KS = BF16 ? 64 : 32;
    constexpr int UK = BF16 ? 16 : 8;
    constexpr int EPC = BF16 ? 8 : 4;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    const uint32_t slab_bytes = 2u * (uint32_t)n_pad * 128u;                  // weight image [hi | lo]
    const uint32_t a_bytes = BF16 ? 16384u : 32768u;                          // activation tile(s) of a stage
    const uint32_t stage_bytes = a_bytes + slab_bytes;
    const bool fused = a.A2 != nullptr;     // second product: its accumulator sits next to the first
    float* stage_out = reinterpret_cast<float*>(base + (uint32_t)D * stage_bytes);   // 4 (8 if fused) x 32 x kStagePitch floats
    unsigned char* tail = reinterpret_cast<unsigned char*>(stage_out) + (fused ? 8 : 4) * 32 * kStagePitch * 4;
    uint64_t* full = reinterpret_cast<uint64_t*>(tail);            // [D]   128 producer arrivals + weight bytes
    uint64_t* freeb = full + 8;                                     // [D]   MMAs of the stage have completed
    uint64_t* tfull = freeb + 8;                                    // [2]   accumulator complete
    uint64_t* tfree = tfull + 2;                                    // [2]   accumulator drained (128 arrivals)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfree + 2);
    uint32_t half_cols = 32;
    while ((int)half_cols < n_pad) half_cols <<= 1;
    const uint32_t acc_cols = fused ? 2 * half_cols : half_cols;
    const uint32_t ncols = 2 * acc_cols;
    if (tid == 0) {
        for (int i = 0; i < D; ++i) {
            mbar_init(&full[i], 129);
            mbar_init(&freeb[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&tfull[i], 1);
            mbar_init(&tfree[i], 128);
        }
    }
    if (warp == 4) tmem_alloc(tmem_slot, ncols);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int ns1 = (a.K + KS - 1) / KS;                     // K slabs of the first product
    const int ns2 = fused ? (a.K2 + KS - 1) / KS : 0;        // and of the second
    const int n_slabs = ns1 + ns2;
    const int64_t row_tiles = (a.M + 127) / 128;
    const int64_t n_items = row_tiles * a.groups * n_tiles;
    const int64_t my_items = n_items > blockIdx.x ? (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t my_steps = my_items * n_slabs;
    if (warp < 4) {
        // ------------------------------------------------------------ producers
        const int c = tid & 7;          // 16-byte chunk of the 128-byte row
        const int rbase = tid >> 3;     // rows rbase + 16 i
        uint32_t offs[8];               // swizzled byte offsets of this thread's eight chunks
#pragma unroll
        for (int i = 0; i < 8; ++i) offs[i] = sw_off(rbase + 16 * i, c * 16);
        // steps requested ahead of the one being finished; with D >= 3 the stage a new request goes to
        // was last used two steps back, so the producer never waits for the MMAs it has just fed
        const int L = D >= 3 ? D - 2 : 1;
        // issue cursor: the step whose loads are requested next -> (stage, ring pass) and (item, slab)
        int i_st = 0, i_s = 0;
        uint32_t i_pass = 0;
        ItemCursor i_it;
        i_it.init(blockIdx.x, gridDim.x, a.groups, n_tiles);
        auto issue = [&]() {   // requests the next step's activation slab (and weight image)
            const int st = i_st;
            bool okw = true;
            if (i_pass >= 1) okw = mbar_wait(&freeb[st], (i_pass - 1) & 1);
            if (!okw) {
                if (lane == 0) atomicExch(fault, 5);
                return false;
            }
            const int64_t row0 = i_it.row0();
            const int g = i_it.g, nt = i_it.nt;
            int s = i_s;
            if (++i_st == D) {
                i_st = 0;
                ++i_pass;
            }
            if (++i_s == n_slabs) {
                i_s = 0;
                i_it.next();
            }
            const bool second = s >= ns1;     // this step belongs to the second product
            if (second) s -= ns1;
            unsigned char* stg = base + (uint32_t)st * stage_bytes;
            if (tid == 0) {
                const unsigned char* img = second ? image2 + ((((int64_t)g * n_tiles + nt) * ns2 + s)) * (int64_t)slab_bytes
                                                  : image + ((((int64_t)g * n_tiles + nt) * ns1 + s)) * (int64_t)slab_bytes;
                mbar_expect_tx(&full[st], slab_bytes);
                bulk_g2s(stg + a_bytes, img, slab_bytes, &full[st]);
            }
            const int k = s * KS + c * EPC;
            const int64_t ld = second ? a.lda2 : a.lda;
            const TA* src0 = (second ? static_cast<const TA*>(a.A2) + a.a2_start[g] : static_cast<const TA*>(a.A) + a.a_start[g]) +
                             (row0 + rbase) * ld + k;
            const int64_t row_step = 16 * ld;
            const uint32_t dst0 = smem_u32(stg);
            const int rows_left = (int)min((int64_t)128, a.M - row0) - rbase;   // rows rbase + 16 i < rows of the tile
            const bool k_in = k < (second ? a.K2 : a.K);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const bool in = k_in && 16 * i < rows_left;
                const TA* src = in ? (src0 + i * row_step) : static_cast<const TA*>(a.A);
                const int sz = in ? 16 : 0;   // zero-fill outside the matrix
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst0 + offs[i]), "l"(src), "r"(sz) : "memory");
            }
            return true;
        };
        bool okp = true;
        for (int64_t j = 0; j < L && okp; ++j) {   // exactly L groups, empty past the end, so the count below holds
            if (j < my_steps) okp = issue();
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        int st = 0;   // stage of the step being finished
        for (int64_t j = 0; j < my_steps && okp; ++j) {
            // L + j groups so far: step j (this thread's own copies) has landed once at most L-1 are pending
            if (L == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
            else asm volatile("cp.async.wait_group 0;" ::: "memory");
            unsigned char* stg = base + (uint32_t)st * stage_bytes;
            if (!BF16) {
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const float4 v = *reinterpret_cast<const float4*>(stg + offs[i]);
                    const float h0 = tf32_hi(v.x), h1 = tf32_hi(v.y), h2 = tf32_hi(v.z), h3 = tf32_hi(v.w);
                    *reinterpret_cast<float4*>(stg + offs[i]) = make_float4(h0, h1, h2, h3);
                    *reinterpret_cast<float4*>(stg + 16384 + offs[i]) = make_float4(v.x - h0, v.y - h1, v.z - h2, v.w - h3);
                }
            }
            proxy_fence();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&full[st])) : "memory");
            if (++st == D) st = 0;
            if (j + L < my_steps) okp = issue();
            asm volatile("cp.async.commit_group;" ::: "memory");   // one group per step, empty or not
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool okm = true;
            ItemCursor m_it;
            m_it.init(blockIdx.x, gridDim.x, a.groups, n_tiles);
            int st = 0;
            uint32_t pass = 0;
            for (int64_t it = 0; it < my_items && okm; ++it) {
                const int acc = (int)(it & 1);
                const int64_t use = it >> 1;
                if (use >= 1) okm = mbar_wait(&tfree[acc], (uint32_t)((use - 1) & 1));
                if (!okm) break;
                tc_fence_after();
                const int nt = m_it.nt;
                m_it.next();
                const int nn = min(n_pad, a.N - nt * n_pad);
                const int n_mma = (nn + 15) & ~15;
                const uint32_t idesc = idesc_f32acc(128, n_mma, BF16);
                const uint32_t d_tmem0 = tmem + (uint32_t)acc * acc_cols;
                for (int s = 0; s < n_slabs && okm; ++s) {
                    const uint32_t d_tmem = d_tmem0 + (s >= ns1 ? half_cols : 0u);   // second product: own columns
                    okm = mbar_wait(&full[st], pass & 1);
                    if (!okm) break;
                    tc_fence_after();
                    unsigned char* stg = base + (uint32_t)st * stage_bytes;
                    const uint64_t da_hi = smem_desc(stg), da_lo = smem_desc(stg + 16384);
                    const uint64_t db_hi = smem_desc(stg + a_bytes), db_lo = smem_desc(stg + a_bytes + n_pad * 128);
#pragma unroll
                    for (int ks = 0; ks < KS / UK; ++ks) {
                        const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                        umma<BF16>(d_tmem, da_hi + adv, db_hi + adv, idesc, ((s == 0 || s == ns1) && ks == 0) ? 0u : 1u);
                        if (!BF16) umma<BF16>(d_tmem, da_lo + adv, db_hi + adv, idesc, 1u);
                        umma<BF16>(d_tmem, da_hi + adv, db_lo + adv, idesc, 1u);
                    }
                    umma_commit(&freeb[st]);
                    if (++st == D) {
                        st = 0;
                        ++pass;
                    }
                }
                if (okm) umma_commit(&tfull[acc]);
            }
            if (!okm) atomicExch(fault, 6);
        }
    } else {
        // ------------------------------------------------------------ epilogue
        // lane: column quad cq (4 consecutive columns) of rows sub, sub+4, ...: every global access of a
        // warp covers four whole 128-byte row segments
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        float* stage = stage_out + q * (32 * kStagePitch);
        float* stage2 = stage_out + (4 + q) * (32 * kStagePitch);   // only there (and used) when fused
        const int cq = lane & 7, sub = lane >> 3;
        unsigned char* Cb = static_cast<unsigned char*>(a.C);
        // bias and post-activation vectors of all groups, staged once (a load from global memory per
        // item would sit on the critical path of every tile)
        float* sbias = reinterpret_cast<float*>(tail + 256);
        float* spost = sbias + kWsVecFloats;
        const bool vec_staged = a.groups * a.N <= kWsVecFloats;
        if (vec_staged) {
            for (int i = tid - 160; i < a.groups * a.N; i += 128) {
                sbias[i] = a.bias ? __ldg(a.bias + i) : 0.f;
                float pv = a.post1 ? __ldg(a.post1 + i) : 0.f;
                if (a.post2) pv += __ldg(a.post2 + i);
                spost[i] = pv;
            }
            asm volatile("bar.sync 1, 128;" ::: "memory");
        }
        bool oke = true;
        ItemCursor e_it;
        e_it.init(blockIdx.x, gridDim.x, a.groups, n_tiles);
        for (int64_t it = 0; it < my_items && oke; ++it) {
            const int acc = (int)(it & 1);
            oke = mbar_wait(&tfull[acc], (uint32_t)((it >> 1) & 1));
            if (!oke) break;
            tc_fence_after();
            const int64_t row0 = e_it.row0();
            const int g = e_it.g, nt = e_it.nt;
            e_it.next();
            const int n0 = nt * n_pad;
            const int nn = min(n_pad, a.N - n0);
            const int n_mma = (nn + 15) & ~15;
            const int cs = a.c_start[g] + n0;
            const uint32_t d_tmem = tmem + (uint32_t)acc * acc_cols + ((uint32_t)(q * 32) << 16);
            const int rows_here = (int)min((int64_t)32, a.M - (row0 + q * 32));   // valid rows of this warp's quarter
            for (int c0 = 0; c0 < n_mma; c0 += 32) {
                float v[32];
                if (fused) {   // the second product's columns first, into the second staging tile
                    tmem_ld32(d_tmem + half_cols + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        *reinterpret_cast<float4*>(stage2 + lane * kStagePitch + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
                tmem_ld32(d_tmem + (uint32_t)c0, v);
                if (c0 + 32 >= n_mma) {   // last read of this accumulator: hand it back to the MMA warp
                    tc_fence_before();
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&tfree[acc])) : "memory");
                }
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(stage + lane * kStagePitch + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                __syncwarp();
                const int n = c0 + cq * 4;            // first of this lane's four columns within the tile
                const bool col_ok = n < nn;           // nn is a multiple of 4 on this path
                const int col = cs + n;
                float4 bias = make_float4(0.f, 0.f, 0.f, 0.f), post = bias;
                if (col_ok && vec_staged) {
                    bias = *reinterpret_cast<const float4*>(sbias + g * a.N + n0 + n);
                    post = *reinterpret_cast<const float4*>(spost + g * a.N + n0 + n);
                } else if (col_ok) {
                    if (a.bias) bias = __ldg(reinterpret_cast<const float4*>(a.bias + g * a.N + n0 + n));
                    if (a.post1) post = __ldg(reinterpret_cast<const float4*>(a.post1 + g * a.N + n0 + n));
                    if (a.post2) {
                        const float4 p2 = __ldg(reinterpret_cast<const float4*>(a.post2 + g * a.N + n0 + n));
                        post = make_float4(post.x + p2.x, post.y + p2.y, post.z + p2.z, post.w + p2.w);
                    }
                }
                const int64_t rfirst = row0 + q * 32 + sub;
                float4 cold[8], gate[8];
                if (a.accumulate) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        cold[i] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (col_ok && 4 * i + sub < rows_here) {
                            if (sizeof(TC) == 4) {
                                cold[i] = *reinterpret_cast<const float4*>(Cb + ((rfirst + 4 * i) * a.ldc + col) * 4);
                            } else {
                                const uint2 h = *reinterpret_cast<const uint2*>(Cb + ((rfirst + 4 * i) * a.ldc + col) * 2);
                                cold[i] = make_float4(__uint_as_float(h.x << 16), __uint_as_float(h.x & 0xffff0000u),
                                                      __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xffff0000u));
                            }
                        }
                    }
                }
                if (a.mul_pos) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        gate[i] = make_float4(1.f, 1.f, 1.f, 1.f);
                        if (col_ok && 4 * i + sub < rows_here) {
                            if (a.mul_pos_dtype == SLICEGCN_F32) {
                                gate[i] = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(a.mul_pos) +
                                                                                (rfirst + 4 * i) * a.mul_pos_ld + col));
                            } else if (a.mul_pos_dtype == kGateBytes) {   // four mask bytes
                                const uint32_t mb = __ldg(reinterpret_cast<const uint32_t*>(
                                    static_cast<const uint8_t*>(a.mul_pos) + (rfirst + 4 * i) * a.mul_pos_ld + col));
                                // the bytes as float BIT PATTERNS (1 -> a positive denormal): the test below is "> 0", and an
                                // integer-to-float conversion per element would cost more than the load saves
                                gate[i] = make_float4(__uint_as_float(mb & 0xffu), __uint_as_float((mb >> 8) & 0xffu),
                                                      __uint_as_float((mb >> 16) & 0xffu), __uint_as_float(mb >> 24));
                            } else {
                                const uint2 h = __ldg(reinterpret_cast<const uint2*>(
                                    static_cast<const __nv_bfloat16*>(a.mul_pos) + (rfirst + 4 * i) * a.mul_pos_ld + col));
                                gate[i] = make_float4(__uint_as_float(h.x << 16), __uint_as_float(h.x & 0xffff0000u),
                                                      __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xffff0000u));
                            }
                        }
                    }
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + sub;
                    if (!col_ok || rr >= rows_here) continue;
                    const int64_t row = rfirst + 4 * i;
                    const float4 t = *reinterpret_cast<const float4*>(stage + rr * kStagePitch + cq * 4);
                    float x[4] = {t.x + bias.x, t.y + bias.y, t.z + bias.z, t.w + bias.w};
                    if (a.relu) {
                        if (a.mask_out) {
                            const uint32_t m = (x[0] > 0.f ? 1u : 0u) | (x[1] > 0.f ? 0x100u : 0u) | (x[2] > 0.f ? 0x10000u : 0u) |
                                               (x[3] > 0.f ? 0x1000000u : 0u);
                            *reinterpret_cast<uint32_t*>(a.mask_out + row * a.mask_ld + col) = m;
                        }
#pragma unroll
                        for (int e = 0; e < 4; ++e) x[e] = fmaxf(x[e], 0.f);
                    }
                    x[0] += post.x; x[1] += post.y; x[2] += post.z; x[3] += post.w;
                    if (a.mul_pos) {
                        x[0] = gate[i].x > 0.f ? x[0] : 0.f;
                        x[1] = gate[i].y > 0.f ? x[1] : 0.f;
                        x[2] = gate[i].z > 0.f ? x[2] : 0.f;
                        x[3] = gate[i].w > 0.f ? x[3] : 0.f;
                    }
                    if (a.accumulate) {
                        x[0] += cold[i].x; x[1] += cold[i].y; x[2] += cold[i].z; x[3] += cold[i].w;
                    }
                    if (fused) {
                        const float4 t2 = *reinterpret_cast<const float4*>(stage2 + rr * kStagePitch + cq * 4);
                        x[0] += t2.x; x[1] += t2.y; x[2] += t2.z; x[3] += t2.w;
                    }
                    if (sizeof(TC) == 4) {
                        *reinterpret_cast<float4*>(Cb + (row * a.ldc + col) * 4) = make_float4(x[0], x[1], x[2], x[3]);
                    } else {
                        const __nv_bfloat162 lo2 = __floats2bfloat162_rn(x[0], x[1]), hi2 = __floats2bfloat162_rn(x[2], x[3]);
                        uint2 pk;
                        pk.x = *reinterpret_cast<const uint32_t*>(&lo2);
                        pk.y = *reinterpret_cast<const uint32_t*>(&hi2);
                        *reinterpret_cast<uint2*>(Cb + (row * a.ldc + col) * 2) = pk;
                    }
                }
                __syncwarp();
            }
        }
        if (!oke && lane == 0) atomicExch(fault, 7);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, ncols);
}

// ------------------------------------------------------------------------------ row-panel GEMM, activation operand in TMEM
// The kernel for the sliced layers proper: fp32 operands, narrow outputs per group (n_pad <= 64, or
// <= 32 with the fused second product).  What limits the kernel above on these shapes is shared
// memory traffic -- every activation byte is written by the copy, read and written twice by the
// hi/lo split and read three times by the MMAs -- so here the activation operand never returns to
// shared memory:
//   warp 5      loader.  One thread keeps a ring of kTsRing raw slabs (128 rows x 32 values, 128-byte
//               swizzle) filled, one tensor copy (TMA) per step; rows past the matrix arrive as zeros.
//   warps 0-3   producers.  Warp w owns rows 32w..32w+31 of every tile: it reads the landed slab one
//               row per lane, splits it in registers and writes hi and lo into a TMEM stage with
//               tcgen05.st (row = TMEM lane, K along the columns -- the form the MMA takes its A
//               operand in).  Thread 0 also requests the step's weight image.  A K slab that runs past
//               a group's K columns brings the neighbouring columns along; the weight image holds zeros
//               there, so they do not contribute.
//   warp 4      MMA issuer.  Per K slab two chains instead of three: A_hi x [B_hi | B_lo] (the image
//               holds hi and lo back to back, so they form one operand of 2 n_pad rows) into
//               accumulator columns [0, 2 n_pad), then A_lo x B_hi onto columns [0, n_pad).
//   warps 8-15  epilogue, two groups of four that take alternate items (one per accumulator):
//               the halves (and the second product) are summed in registers in the row-per-lane
//               form, bias / ReLU / post are applied there, and only the finished tile (plus the
//               ReLU mask bytes) goes through a per-warp staging tile to be written in whole
//               128-byte row segments.
// TMEM columns: [accumulator 0][accumulator 1] (accw each) then kTsStages x 64 (A hi | A lo).
constexpr int kTsThreads = 512;
constexpr int kTsRing = 6;     // raw slabs in flight or being read
constexpr int kTsStages = 3;   // TMEM operand stages (with their weight images in shared memory)
constexpr int kTsMaskPitch = 48;

// MASKED: the activation operand is multiplied by the byte mask a.a_mask on its way to TMEM (fp32 only).
// ABF16: activations stored as bf16 -- a K slab is 64 values, they go to TMEM as they are (two per column) and the
// MMAs are kind::f16 against the bf16 hi / lo weight image: A x [B_hi | B_lo], one chain.  TC: float or bf16 result.
template <bool MASKED, bool ABF16, typename TC>
__global__ void __launch_bounds__(kTsThreads, 1) tc_gemm_ts_kernel(const GemmArgs a, const int n_pad, const int n_tiles, const int R,
                                                                   const unsigned char* image, const unsigned char* image2,
                                                                   int* fault, const __grid_constant__ CUtensorMap map_a,
                                                                   const __grid_constant__ CUtensorMap map_a2,
                                                                   const __grid_constant__ CUtensorMap map_m) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int S = kTsStages;
    const bool concat = n_pad <= 64;   // [B_hi | B_lo] as one operand; wider tiles take three chains per slab
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    const uint32_t slab_bytes = 2u * (uint32_t)n_pad * 128u;                  // weight image [hi | lo]
    const bool fused = a.A2 != nullptr;
    unsigned char* wring = base;                                              // [S] weight images
    // [R] raw activation slabs, 128 rows x 128 B, swizzled; with an operand mask (a.a_mask) each is followed by
    // its 128 x 32 mask bytes
    constexpr bool masked = MASKED;
    constexpr uint32_t raw_slot = MASKED ? 16384u + 4096u : 16384u;
    unsigned char* raw = wring + (uint32_t)S * slab_bytes;
    float* stage_out = reinterpret_cast<float*>(raw + R * raw_slot);          // [8 warps] 32 x kStagePitch floats
    unsigned char* stage_mask = reinterpret_cast<unsigned char*>(stage_out + 8 * 32 * kStagePitch);   // [8] 32 x kTsMaskPitch
    float* sbias = reinterpret_cast<float*>(stage_mask + 8 * 32 * kTsMaskPitch);
    float* spost = sbias + kWsVecFloats + 64;
    uint64_t* afull = reinterpret_cast<uint64_t*>(spost + kWsVecFloats + 64);   // [S] 128 producer arrivals + weight bytes
    uint64_t* afree = afull + S;                                              // [S] MMAs of the stage have completed
    uint64_t* tfull = afree + S;                                              // [2] accumulator complete
    uint64_t* tfree = tfull + 2;                                              // [2] accumulator drained (128 arrivals)
    uint64_t* rfull = tfree + 2;                                              // [R] raw slab landed (bytes)
    uint64_t* rfree = rfull + R;                                              // [R] raw slab read by the four producer warps
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(rfree + R);
    const uint32_t prodw = (concat ? 2u : 1u) * (uint32_t)n_pad;   // columns of one product: [hi*hi + lo*hi | hi*lo]
    const uint32_t accw = fused ? 2 * prodw : prodw;        // columns of one accumulator
    const uint32_t a_col0 = 2 * accw;                       // first column of the operand stages
    if (tid == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&afull[i], 129);
            mbar_init(&afree[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(&tfull[i], 1);
            mbar_init(&tfree[i], 128);
        }
        for (int i = 0; i < R; ++i) {
            mbar_init(&rfull[i], 1);
            mbar_init(&rfree[i], 4);
        }
    }
    if (warp == 4) tmem_alloc(tmem_slot, 512);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    constexpr int KS = ABF16 ? 64 : 32;                      // K values per slab (one 128-byte row)
    const int ns1 = (a.K + KS - 1) / KS;                     // K slabs of the first product
    const int ns2 = fused ? (a.K2 + KS - 1) / KS : 0;        // and of the second
    const int n_slabs = ns1 + ns2;
    const int64_t row_tiles = (a.M + 127) / 128;
    const int64_t n_items = row_tiles * a.groups * n_tiles;
    const int64_t my_items = n_items > blockIdx.x ? (n_items - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    const int64_t my_steps = my_items * n_slabs;

    if (warp < 4) {
        // ------------------------------------------------------------ producers
        // lane reads row 32 warp + lane of the landed slab: 16-byte chunk cc sits at (cc ^ (row & 7)) * 16
        const uint32_t roff = (uint32_t)((32 * warp + lane) * 128);
        int rs = 0, ts = 0, c_s = 0;
        uint32_t pass = 0, rpass = 0;
        ItemCursor c_it;
        c_it.init(blockIdx.x, gridDim.x, a.groups, n_tiles);
        c_it.flip = a.reverse ? (int)((a.M + 127) / 128) - 1 : -1;
        bool okp = true;
        for (int64_t j = 0; j < my_steps; ++j) {
            okp = mbar_wait(&rfull[rs], rpass & 1);
            if (okp && pass >= 1) okp = mbar_wait(&afree[ts], (pass - 1) & 1);
            if (!okp) break;
            if (tid == 0) {
                int s = c_s;
                const bool second = s >= ns1;
                if (second) s -= ns1;
                const int g = c_it.g, nt = c_it.nt;
                const unsigned char* img = second ? image2 + ((((int64_t)g * n_tiles + nt) * ns2 + s)) * (int64_t)slab_bytes
                                                  : image + ((((int64_t)g * n_tiles + nt) * ns1 + s)) * (int64_t)slab_bytes;
                mbar_expect_tx(&afull[ts], slab_bytes);
                bulk_g2s(wring + (uint32_t)ts * slab_bytes, img, slab_bytes, &afull[ts]);
                if (++c_s == n_slabs) {
                    c_s = 0;
                    c_it.next();
                }
            }
            __syncwarp();
            tc_fence_after();
            const unsigned char* slot = raw + rs * raw_slot + roff;
            const uint32_t t_hi = tmem + ((uint32_t)(32 * warp) << 16) + a_col0 + (uint32_t)ts * 64u;
            uint32_t mw[8];
            if (masked) {   // the row's 32 mask bytes: word ch covers the four values of 16-byte chunk ch
                const uint4* mrow = reinterpret_cast<const uint4*>(raw + rs * raw_slot + 16384 + (32 * warp + lane) * 32);
                const uint4 m0 = mrow[0], m1 = mrow[1];
                mw[0] = m0.x; mw[1] = m0.y; mw[2] = m0.z; mw[3] = m0.w;
                mw[4] = m1.x; mw[5] = m1.y; mw[6] = m1.z; mw[7] = m1.w;
            }
            if (ABF16) {   // 64 bf16 values of the row, unchanged, into 32 columns
                uint32_t u[32];
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    const uint4 v = *reinterpret_cast<const uint4*>(slot + ((ch ^ (lane & 7)) << 4));
                    u[4 * ch + 0] = v.x;
                    u[4 * ch + 1] = v.y;
                    u[4 * ch + 2] = v.z;
                    u[4 * ch + 3] = v.w;
                }
                __syncwarp();
                if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rfree[rs])) : "memory");
                __syncwarp();
                tmem_st16<0>(t_hi, u);
                tmem_st16<16>(t_hi + 16u, u);
            }
#pragma unroll
            for (int half = 0; half < (ABF16 ? 0 : 2); ++half) {   // 16 K values at a time keeps the register count down
                uint32_t h[32];                      // [0,16): hi of K 16 half..; [16,32): lo of the same
#pragma unroll
                for (int cc = 0; cc < 4; ++cc) {
                    const int ch = half * 4 + cc;
                    float4 v = *reinterpret_cast<const float4*>(slot + ((ch ^ (lane & 7)) << 4));
                    if (masked) {
                        const uint32_t m = mw[ch];
                        v.x = (m & 0xffu) ? v.x : 0.f;
                        v.y = (m & 0xff00u) ? v.y : 0.f;
                        v.z = (m & 0xff0000u) ? v.z : 0.f;
                        v.w = (m & 0xff000000u) ? v.w : 0.f;
                    }
                    const float h0 = tf32_hi(v.x), h1 = tf32_hi(v.y), h2 = tf32_hi(v.z), h3 = tf32_hi(v.w);
                    h[4 * cc + 0] = __float_as_uint(h0);
                    h[4 * cc + 1] = __float_as_uint(h1);
                    h[4 * cc + 2] = __float_as_uint(h2);
                    h[4 * cc + 3] = __float_as_uint(h3);
                    h[16 + 4 * cc + 0] = __float_as_uint(v.x - h0);
                    h[16 + 4 * cc + 1] = __float_as_uint(v.y - h1);
                    h[16 + 4 * cc + 2] = __float_as_uint(v.z - h2);
                    h[16 + 4 * cc + 3] = __float_as_uint(v.w - h3);
                }
                if (half == 1) {   // the slab is in registers: hand the slot back to the loader
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rfree[rs])) : "memory");
                    __syncwarp();
                }
                tmem_st16<0>(t_hi + 16u * half, h);
                tmem_st16<16>(t_hi + 32u + 16u * half, h);
            }
            tmem_st_wait();
            tc_fence_before();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&afull[ts])) : "memory");
            if (++rs == R) {
                rs = 0;
                ++rpass;
            }
            if (++ts == S) {
                ts = 0;
                ++pass;
            }
        }
        if (!okp && lane == 0) atomicExch(fault, 5);
    } else if (warp == 5) {
        // ------------------------------------------------------------ loader: one tensor copy per step
        if (lane == 0) {
            int rs = 0, l_s = 0;
            uint32_t rpass = 0;
            ItemCursor l_it;
            l_it.init(blockIdx.x, gridDim.x, a.groups, n_tiles);
            l_it.flip = a.reverse ? (int)((a.M + 127) / 128) - 1 : -1;
            for (int64_t j = 0; j < my_steps; ++j) {
                if (rpass >= 1 && !mbar_wait(&rfree[rs], (rpass - 1) & 1)) {
                    atomicExch(fault, 8);
                    break;
                }
                int s = l_s;
                const bool second = s >= ns1;
                if (second) s -= ns1;
                const int x = (second ? a.a2_start[l_it.g] : a.a_start[l_it.g]) + s * KS;
                const bool with_mask = masked && !second;
                mbar_expect_tx(&rfull[rs], with_mask ? 16384u + 4096u : 16384u);
                tma_load_2d(raw + rs * raw_slot, second ? &map_a2 : &map_a, x, (int)l_it.row0(), &rfull[rs]);
                if (with_mask) tma_load_2d(raw + rs * raw_slot + 16384, &map_m, x, (int)l_it.row0(), &rfull[rs]);
                if (++l_s == n_slabs) {
                    l_s = 0;
                    l_it.next();
                }
                if (++rs == R) {
                    rs = 0;
                    ++rpass;
                }
            }
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            bool okm = true;
            const uint32_t idesc_wide = idesc_f32acc(128, 2 * n_pad, ABF16);   // A_hi x [B_hi | B_lo]
            const uint32_t idesc_hi = idesc_f32acc(128, n_pad, ABF16);         // A_lo x B_hi
            int ts = 0;
            uint32_t pass = 0;
            for (int64_t it = 0; it < my_items && okm; ++it) {
                const int acc = (int)(it & 1);
                const int64_t use = it >> 1;
                if (use >= 1) okm = mbar_wait(&tfree[acc], (uint32_t)((use - 1) & 1));
                if (!okm) break;
                tc_fence_after();
                const uint32_t d_tmem0 = tmem + (uint32_t)acc * accw;
                if (fused && concat && ns1 == 1 && ns2 == 1) {
                    // One slab per product (the sliced layers' 32-wide blocks): MMAs into one accumulator range depend
                    // on each other and such small ones are bound by that latency, so the two products' chains -- they
                    // fill different column ranges -- are issued alternately (measured: 12-14 % off the kernel's time).  (Pairing two
                    // consecutive one-slab items the same way measured slower: the second item's producers and the first
                    // item's epilogue then wait for each other.)
                    const int ts2 = (ts + 1 == S) ? 0 : ts + 1;
                    const uint32_t pass2 = (ts + 1 == S) ? pass + 1 : pass;
                    okm = mbar_wait(&afull[ts], pass & 1);
                    if (okm) okm = mbar_wait(&afull[ts2], pass2 & 1);
                    if (!okm) break;
                    tc_fence_after();
                    const uint32_t a1 = tmem + a_col0 + (uint32_t)ts * 64u, a2 = tmem + a_col0 + (uint32_t)ts2 * 64u;
                    const uint64_t db1 = smem_desc(wring + (uint32_t)ts * slab_bytes), db2 = smem_desc(wring + (uint32_t)ts2 * slab_bytes);
                    if (ABF16) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                            umma_ts_f16(d_tmem0, a1 + 8u * ks, db1 + adv, idesc_wide, ks == 0 ? 0u : 1u);
                            umma_ts_f16(d_tmem0 + prodw, a2 + 8u * ks, db2 + adv, idesc_wide, ks == 0 ? 0u : 1u);
                        }
                    } else {   // fp32: A_hi x [B_hi | B_lo] of both products, then A_lo x B_hi of both
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                            umma_ts_tf32(d_tmem0, a1 + 8u * ks, db1 + adv, idesc_wide, ks == 0 ? 0u : 1u);
                            umma_ts_tf32(d_tmem0 + prodw, a2 + 8u * ks, db2 + adv, idesc_wide, ks == 0 ? 0u : 1u);
                        }
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                            umma_ts_tf32(d_tmem0, a1 + 32u + 8u * ks, db1 + adv, idesc_hi, 1u);
                            umma_ts_tf32(d_tmem0 + prodw, a2 + 32u + 8u * ks, db2 + adv, idesc_hi, 1u);
                        }
                    }
                    umma_commit(&afree[ts]);
                    umma_commit(&afree[ts2]);
                    ts = (ts2 + 1 == S) ? 0 : ts2 + 1;
                    pass = (ts2 + 1 == S) ? pass2 + 1 : pass2;
                    umma_commit(&tfull[acc]);
                    continue;
                }
                for (int s = 0; s < n_slabs && okm; ++s) {
                    const uint32_t d_tmem = d_tmem0 + (s >= ns1 ? prodw : 0u);   // second product: own columns
                    okm = mbar_wait(&afull[ts], pass & 1);
                    if (!okm) break;
                    tc_fence_after();
                    const uint32_t a_hi = tmem + a_col0 + (uint32_t)ts * 64u, a_lo = a_hi + 32u;
                    const uint64_t db = smem_desc(wring + (uint32_t)ts * slab_bytes);
                    if (ABF16) {   // bf16 activations: exact, so only the weight has a lo part
                        const uint64_t db_lo = smem_desc(wring + (uint32_t)ts * slab_bytes + n_pad * 128);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                            const uint32_t first = ((s == 0 || s == ns1) && ks == 0) ? 0u : 1u;
                            if (concat) {
                                umma_ts_f16(d_tmem, a_hi + 8u * ks, db + adv, idesc_wide, first);
                            } else {
                                umma_ts_f16(d_tmem, a_hi + 8u * ks, db + adv, idesc_hi, first);
                                umma_ts_f16(d_tmem, a_hi + 8u * ks, db_lo + adv, idesc_hi, 1u);
                            }
                        }
                    } else if (concat) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_ts_tf32(d_tmem, a_hi + 8u * ks, db + (uint64_t)((ks * 32) >> 4), idesc_wide,
                                         ((s == 0 || s == ns1) && ks == 0) ? 0u : 1u);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)
                            umma_ts_tf32(d_tmem, a_lo + 8u * ks, db + (uint64_t)((ks * 32) >> 4), idesc_hi, 1u);
                    } else {
                        const uint64_t db_lo = smem_desc(wring + (uint32_t)ts * slab_bytes + n_pad * 128);
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                            umma_ts_tf32(d_tmem, a_hi + 8u * ks, db + adv, idesc_hi, (s == 0 && ks == 0) ? 0u : 1u);
                            umma_ts_tf32(d_tmem, a_lo + 8u * ks, db + adv, idesc_hi, 1u);
                            umma_ts_tf32(d_tmem, a_hi + 8u * ks, db_lo + adv, idesc_hi, 1u);
                        }
                    }
                    umma_commit(&afree[ts]);
                    if (++ts == S) {
                        ts = 0;
                        ++pass;
                    }
                }
                if (okm) umma_commit(&tfull[acc]);
            }
            if (!okm) atomicExch(fault, 6);
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ epilogue
        // Group e takes items e, e+2, ... (accumulator e).  Phase 1, one row per lane: sum the partial
        // accumulators, apply bias / ReLU / post, park the tile (and the mask bytes) in the warp's
        // staging tiles.  Phase 2, lane = (column quad cq, row sub): gate, add the old C, store -- every
        // global access of a warp covers four whole 128-byte row segments.
        const int ew = warp - 8;                      // 0..7
        const int e = ew >> 2;                        // group = accumulator
        const int q = warp & 3;                       // TMEM lane quarter this warp may read
        float* stage = stage_out + ew * (32 * kStagePitch);
        unsigned char* mstage = stage_mask + ew * (32 * kTsMaskPitch);
        const int cq = lane & 7, sub = lane >> 3;
        float* Cf = static_cast<float*>(a.C);               // fp32 result
        unsigned char* Cb = static_cast<unsigned char*>(a.C);   // bf16 result (no accumulation, no gate)
        const bool wmask = a.relu && a.mask_out;
        const bool has_vec = a.bias || a.post1 || a.post2;   // otherwise the staged vectors are all zero
        const int nvec = a.groups * a.N;   // (with padding columns written: zeros up to the padded width)
        for (int i = tid - 256; i < (a.c_pad_write ? ((nvec + 3) & ~3) : nvec); i += 256) {
            const bool in = i < nvec;
            sbias[i] = (in && a.bias) ? __ldg(a.bias + i) : 0.f;
            float pv = (in && a.post1) ? __ldg(a.post1 + i) : 0.f;
            if (in && a.post2) pv += __ldg(a.post2 + i);
            spost[i] = pv;
        }
        // an fp32 result whose rows do not allow 16-byte stores (47 classes): element-wise stores, every other step alike
        const bool ragged = ((a.N & 3) && !a.c_pad_write) || (a.ldc & 3) || ((uintptr_t)a.C & 15);
        asm volatile("bar.sync 1, 256;" ::: "memory");
        bool oke = true;
        ItemCursor e_it;
        e_it.init(blockIdx.x + (uint32_t)e * gridDim.x, 2 * gridDim.x, a.groups, n_tiles);
        e_it.flip = a.reverse ? (int)((a.M + 127) / 128) - 1 : -1;
        for (int64_t it = e; it < my_items && oke; it += 2) {
            const int64_t row0 = e_it.row0();
            const int g = e_it.g, nt = e_it.nt;
            e_it.next();
            const int n0 = nt * n_pad;
            const int n_all = a.c_pad_write ? ((a.N + 3) & ~3) : a.N;   // padding columns of C are written too (zeros)
            const int nn = min(n_pad, n_all - n0);
            const int cs = a.c_start[g] + n0;
            const int rows_here = (int)min((int64_t)32, a.M - (row0 + q * 32));   // valid rows of this warp's quarter
            const int64_t rfirst = row0 + q * 32 + sub;
            if (a.mul_pos && it + 2 < my_items && cq == 0) {
                // the group's next item: ask for the lines of the gate it will read
                const int64_t nrow = e_it.row0() + q * 32 + sub;
                const int ncol0 = a.c_start[e_it.g] + e_it.nt * n_pad;
                const int nnn = min(n_pad, a.N - e_it.nt * n_pad);
                for (int i = 0; i < 8; ++i) {
                    if (nrow + 4 * i >= a.M) break;
                    for (int cc = 0; cc < nnn; cc += 32) {
                        asm volatile("prefetch.global.L2 [%0];" ::"l"(static_cast<const char*>(a.mul_pos) +
                                                                          ((nrow + 4 * i) * a.mul_pos_ld + ncol0 + cc) *
                                                                              (a.mul_pos_dtype == SLICEGCN_F32 ? 4 : a.mul_pos_dtype == kGateBytes ? 1 : 2)));
                    }
                }
            }
            oke = mbar_wait(&tfull[e], (uint32_t)((it >> 1) & 1));
            if (!oke) break;
            tc_fence_after();
            const uint32_t d_tmem = tmem + (uint32_t)e * accw + ((uint32_t)(q * 32) << 16);
            for (int c0 = 0; c0 < nn; c0 += 32) {
                const int n = c0 + cq * 4;            // first of this lane's four columns in phase 2
                const bool col_ok = n < nn;           // (nn is a multiple of 4 unless the result is ragged)
                const int col = cs + n;
                // ---- phase 1
                float x[32];
                if (concat) {   // both halves requested before the one wait
                    uint32_t u[32], v[32];
                    tmem_ld32_issue(d_tmem + (uint32_t)c0, u);
                    tmem_ld32_issue(d_tmem + (uint32_t)(n_pad + c0), v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j) x[j] = __uint_as_float(u[j]) + __uint_as_float(v[j]);
                } else {
                    tmem_ld32(d_tmem + (uint32_t)c0, x);
                }
                // gate values of phase 2: requested as soon as the accumulator halves are summed (their lines were
                // asked into L2 an item earlier), used after the tile has been staged
                float4 gate[8];
                if (a.mul_pos) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        gate[i] = make_float4(1.f, 1.f, 1.f, 1.f);
                        if (col_ok && 4 * i + sub < rows_here) {
                            if (a.mul_pos_dtype == SLICEGCN_F32) {
                                gate[i] = __ldg(reinterpret_cast<const float4*>(static_cast<const float*>(a.mul_pos) +
                                                                                (rfirst + 4 * i) * a.mul_pos_ld + col));
                            } else if (a.mul_pos_dtype == kGateBytes) {   // four mask bytes
                                const uint32_t mb = __ldg(reinterpret_cast<const uint32_t*>(
                                    static_cast<const uint8_t*>(a.mul_pos) + (rfirst + 4 * i) * a.mul_pos_ld + col));
                                // the bytes as float BIT PATTERNS (1 -> a positive denormal): the test below is "> 0", and an
                                // integer-to-float conversion per element would cost more than the load saves
                                gate[i] = make_float4(__uint_as_float(mb & 0xffu), __uint_as_float((mb >> 8) & 0xffu),
                                                      __uint_as_float((mb >> 16) & 0xffu), __uint_as_float(mb >> 24));
                            } else {
                                const uint2 hq = __ldg(reinterpret_cast<const uint2*>(
                                    static_cast<const __nv_bfloat16*>(a.mul_pos) + (rfirst + 4 * i) * a.mul_pos_ld + col));
                                gate[i] = make_float4(__uint_as_float(hq.x << 16), __uint_as_float(hq.x & 0xffff0000u),
                                                      __uint_as_float(hq.y << 16), __uint_as_float(hq.y & 0xffff0000u));
                            }
                        }
                    }
                }
                const float* bvec = sbias + g * a.N + n0 + c0;
                const float* pvec = spost + g * a.N + n0 + c0;
                uint32_t mword[8];   // the ReLU mask bytes of columns 4q .. 4q+3, one word per column quad
                if (a.relu) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 b4 = *reinterpret_cast<const float4*>(bvec + j);
                        const float4 p4 = *reinterpret_cast<const float4*>(pvec + j);
                        x[j] += b4.x; x[j + 1] += b4.y; x[j + 2] += b4.z; x[j + 3] += b4.w;
                        mword[j >> 2] = (x[j] > 0.f ? 1u : 0u) | (x[j + 1] > 0.f ? 0x100u : 0u) | (x[j + 2] > 0.f ? 0x10000u : 0u) |
                                        (x[j + 3] > 0.f ? 0x1000000u : 0u);
                        x[j] = fmaxf(x[j], 0.f) + p4.x;
                        x[j + 1] = fmaxf(x[j + 1], 0.f) + p4.y;
                        x[j + 2] = fmaxf(x[j + 2], 0.f) + p4.z;
                        x[j + 3] = fmaxf(x[j + 3], 0.f) + p4.w;
                    }
                } else if (has_vec) {
#pragma unroll
                    for (int j = 0; j < 32; j += 4) {
                        const float4 b4 = *reinterpret_cast<const float4*>(bvec + j);
                        const float4 p4 = *reinterpret_cast<const float4*>(pvec + j);
                        x[j] = (x[j] + b4.x) + p4.x;
                        x[j + 1] = (x[j + 1] + b4.y) + p4.y;
                        x[j + 2] = (x[j + 2] + b4.z) + p4.z;
                        x[j + 3] = (x[j + 3] + b4.w) + p4.w;
                    }
                }
                if (fused) {   // the second product's halves, 16 columns of each per wait
                    tmem_ld16x2_add<0>(d_tmem + prodw + (uint32_t)c0, d_tmem + prodw + (uint32_t)(n_pad + c0), x);
                    tmem_ld16x2_add<16>(d_tmem + prodw + (uint32_t)(c0 + 16), d_tmem + prodw + (uint32_t)(n_pad + c0 + 16), x);
                }
                if (c0 + 32 >= nn) {   // last read of this accumulator: hand it back to the MMA warp
                    tc_fence_before();
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&tfree[e])) : "memory");
                }
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    *reinterpret_cast<float4*>(stage + lane * kStagePitch + j) = make_float4(x[j], x[j + 1], x[j + 2], x[j + 3]);
                if (wmask) {   // (wmask implies a.relu: mword is set)
                    *reinterpret_cast<uint4*>(mstage + lane * kTsMaskPitch) = make_uint4(mword[0], mword[1], mword[2], mword[3]);
                    *reinterpret_cast<uint4*>(mstage + lane * kTsMaskPitch + 16) = make_uint4(mword[4], mword[5], mword[6], mword[7]);
                }
                __syncwarp();
                // ---- phase 2
                if (rows_here == 32 && col_ok && !a.mul_pos && !a.accumulate && !ragged) {
                    // whole tile, plain store (every forward product): no per-row tests, addresses by repeated addition
                    unsigned char* cp = Cb + (rfirst * a.ldc + col) * (int64_t)sizeof(TC);
                    uint8_t* mp = wmask ? a.mask_out + rfirst * a.mask_ld + col : nullptr;
                    const int64_t cstep = 4 * a.ldc * (int64_t)sizeof(TC), mstep = 4 * a.mask_ld;
                    const float* sp = stage + sub * kStagePitch + cq * 4;
                    const unsigned char* msp = mstage + sub * kTsMaskPitch + cq * 4;
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        const float4 t = *reinterpret_cast<const float4*>(sp + 4 * i * kStagePitch);
                        if (wmask) {
                            *reinterpret_cast<uint32_t*>(mp) = *reinterpret_cast<const uint32_t*>(msp + 4 * i * kTsMaskPitch);
                            mp += mstep;
                        }
                        if (sizeof(TC) == 4) {
                            *reinterpret_cast<float4*>(cp) = t;
                        } else {
                            const __nv_bfloat162 lo2 = __floats2bfloat162_rn(t.x, t.y), hi2 = __floats2bfloat162_rn(t.z, t.w);
                            uint2 pk;
                            pk.x = *reinterpret_cast<const uint32_t*>(&lo2);
                            pk.y = *reinterpret_cast<const uint32_t*>(&hi2);
                            *reinterpret_cast<uint2*>(cp) = pk;
                        }
                        cp += cstep;
                    }
                    __syncwarp();
                    continue;
                }
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    const int rr = 4 * i + sub;
                    if (!col_ok || rr >= rows_here) continue;
                    const int64_t row = rfirst + 4 * i;
                    float4 t = *reinterpret_cast<const float4*>(stage + rr * kStagePitch + cq * 4);
                    if (wmask)
                        *reinterpret_cast<uint32_t*>(a.mask_out + row * a.mask_ld + col) =
                            *reinterpret_cast<const uint32_t*>(mstage + rr * kTsMaskPitch + cq * 4);
                    if (a.mul_pos) {
                        t.x = gate[i].x > 0.f ? t.x : 0.f;
                        t.y = gate[i].y > 0.f ? t.y : 0.f;
                        t.z = gate[i].z > 0.f ? t.z : 0.f;
                        t.w = gate[i].w > 0.f ? t.w : 0.f;
                    }
                    if (a.accumulate) {
                        // C += t at the L2: every element receives exactly one addition per launch, so the
                        // result does not depend on the order, and the old value never travels to the SM
                        asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(Cf + row * a.ldc + col), "f"(t.x),
                                     "f"(t.y), "f"(t.z), "f"(t.w)
                                     : "memory");
                    } else if (ragged) {
                        float* cp = Cf + row * a.ldc + col;
                        cp[0] = t.x;
                        if (n + 1 < nn) cp[1] = t.y;
                        if (n + 2 < nn) cp[2] = t.z;
                        if (n + 3 < nn) cp[3] = t.w;
                    } else if (sizeof(TC) == 4) {
                        *reinterpret_cast<float4*>(Cf + row * a.ldc + col) = t;
                    } else {
                        const __nv_bfloat162 lo2 = __floats2bfloat162_rn(t.x, t.y), hi2 = __floats2bfloat162_rn(t.z, t.w);
                        uint2 pk;
                        pk.x = *reinterpret_cast<const uint32_t*>(&lo2);
                        pk.y = *reinterpret_cast<const uint32_t*>(&hi2);
                        *reinterpret_cast<uint2*>(Cb + (row * a.ldc + col) * 2) = pk;
                    }
                }
                __syncwarp();
            }
        }
        if (!oke && lane == 0) atomicExch(fault, 7);
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// Tensor map over a row-major fp32 (elem_bytes = 2: bf16, 1: byte) matrix for boxes of box_rows x box_cols values (default: one
// activation slab of 128 rows x 32 columns), written to shared memory with the 128-byte swizzle or plain.  `cols` bounds the columns a box may read
// (beyond it: zeros).  The encoder is a driver entry point, looked up once; false if unavailable.
typedef CUresult (*TensorMapEncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
bool make_slab_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_cols = 32, int box_rows = 128,
                   bool swizzle128 = true, int elem_bytes = 4) {
    static TensorMapEncodeFn encode = [] {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q = cudaDriverEntryPointSymbolNotFound;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess || q != cudaDriverEntryPointSuccess)
            fn = nullptr;
        return reinterpret_cast<TensorMapEncodeFn>(fn);
    }();
    if (!encode || rows < 1 || cols < 1) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * (cuuint64_t)elem_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return encode(map, elem_bytes == 1 ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : elem_bytes == 2 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                  swizzle128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

thread_local TcImageCache* t_image_cache = nullptr;

// The image for job j (image pointer filled in): from the cache when one is active, else nullptr.
// *fresh tells whether it already holds this epoch's weights.
unsigned char* cached_image(PrepJob& j, int64_t bytes, bool* fresh) {
    TcImageCache* c = t_image_cache;
    *fresh = false;
    if (!c || !c->region) return nullptr;
    for (auto& e : c->entries) {
        const PrepJob& k = e.job;
        if (k.B == j.B && k.b_gstride == j.b_gstride && k.ldb == j.ldb && k.b_trans == j.b_trans && k.K == j.K && k.N == j.N &&
            k.n_pad == j.n_pad && k.groups == j.groups && k.bf16 == j.bf16 && k.kstack == j.kstack) {
            *fresh = e.fresh;
            e.fresh = true;   // the caller converts it now if it was not
            j.image = k.image;
            return k.image;
        }
    }
    const int64_t need = (bytes + 255) & ~(int64_t)255;
    if ((int)c->entries.size() >= kMaxPrepJobs || c->used + need > c->region_bytes) return nullptr;
    j.image = c->region + c->used;
    c->used += need;
    c->entries.push_back({j, true});
    return j.image;
}

// fp32 products that tc_gemm_ts_kernel takes (n_pad as chosen by tc_gemm_launch): 16-byte aligned
// operands and result, up to 128 output columns per tile (32 with the fused second product), bias /
// post vectors that fit the staging arrays; an operand mask only without a second product and with
// 16-byte aligned mask rows and slice starts (it travels by tensor copy next to the slab).
bool ts_gemm_ok(const GemmArgs& a, int n_pad, int n_tiles) {
    static const bool off = getenv("SLICEGCN_NO_TS") != nullptr || getenv("SLICEGCN_NO_WS") != nullptr;
    const bool abf = a.a_dtype == SLICEGCN_BF16, cbf = a.c_dtype == SLICEGCN_BF16;
    if (off) return false;
    if (abf && (a.a_mask || a.accumulate || a.mul_pos)) return false;   // forward products only
    if (!abf && cbf && (a.accumulate || a.mul_pos || a.c_pad_write || a.A2)) return false;   // a bf16 result is stored, never added to
    const bool fused = a.A2 != nullptr;
    const int epc = abf ? 8 : 4;   // elements per 16 bytes of the activation operand
    bool ok = ((uintptr_t)a.A % 16 == 0) && (a.lda % epc == 0) && (a.K % epc == 0 || a.a_pad_zero);
    if (fused) ok = ok && ((uintptr_t)a.A2 % 16 == 0) && (a.lda2 % epc == 0) && (a.K2 % epc == 0 || a.a2_pad_zero);
    for (int g = 0; g < a.groups; ++g) {
        ok = ok && (a.a_start[g] % epc == 0) && (a.c_start[g] % 4 == 0);
        if (fused) ok = ok && (a.a2_start[g] % epc == 0);
    }
    const bool pad_write = a.c_pad_write && !a.mask_out && !a.mul_pos && a.groups == 1 && a.c_start[0] + ((a.N + 3) & ~3) <= a.ldc;
    // an fp32 result with rows that do not allow 16-byte stores is written element by element (one group, plain store)
    const bool ragged_ok = !cbf && !a.c_pad_write && a.groups == 1 && !a.mask_out && !a.mul_pos && !a.accumulate && !fused;
    ok = ok && (((a.N % 4 == 0 || pad_write) && (a.ldc % 4 == 0) && ((uintptr_t)a.C % 16 == 0)) || ragged_ok);
    if (a.mask_out) ok = ok && (a.mask_ld % 4 == 0) && ((uintptr_t)a.mask_out % 4 == 0);
    if (a.mul_pos) ok = ok && (a.mul_pos_ld % 4 == 0) && ((uintptr_t)a.mul_pos % 16 == 0);   // (a byte mask would do with 4)
    if (a.a_mask) {
        ok = ok && !fused && ((uintptr_t)a.a_mask % 16 == 0) && (a.a_mask_ld % 16 == 0);
        for (int g = 0; g < a.groups; ++g) ok = ok && (a.a_start[g] % 16 == 0);
    }
    const int64_t items = ((a.M + 127) / 128) * a.groups * n_tiles;
    return ok && n_pad <= (fused ? 32 : 128) && a.groups * a.N <= kWsVecFloats && items < ((int64_t)1 << 31) && a.M < ((int64_t)1 << 31);
}

int tc_n_pad(int N) { return N <= 256 ? ((N + 15) & ~15) : 256; }

template <typename TA, typename TC, bool BF16>
slicegcn_status_t tc_gemm_launch(const GemmArgs& a, void* image, int64_t image_bytes, int* fault, cudaStream_t st) {
    constexpr int KS = BF16 ? 64 : 32;
    constexpr int EPC = BF16 ? 8 : 4;
    int n_pad = tc_n_pad(a.N);
    const bool fused = a.A2 != nullptr;
    // N = 256 in fp32: two column tiles of 128 suit the kernel with the activation operand in TMEM
    // (two accumulators and the operand stages have to share the 512 TMEM columns); same image bytes
    if (!fused && a.N == 256 && a.groups * a.N <= kWsVecFloats && getenv("SLICEGCN_NO_TS") == nullptr)
        n_pad = 128;
    const int n_tiles = (a.N + n_pad - 1) / n_pad;
    const int n_slabs = (a.K + KS - 1) / KS;
    const int64_t need = (int64_t)a.groups * n_tiles * n_slabs * 2 * n_pad * 128;
    const int n_slabs2 = fused ? (a.K2 + KS - 1) / KS : 0;
    const int64_t need2 = (int64_t)a.groups * n_tiles * n_slabs2 * 2 * n_pad * 128;
    if (!image || image_bytes < need + need2) {
        if (fused) return SLICEGCN_ERR_UNSUPPORTED;   // the caller falls back to two separate products
        SGCN_FAIL(SLICEGCN_ERR_ALLOC, "tc_gemm: weight image scratch too small");
    }
    unsigned char* image2 = static_cast<unsigned char*>(image) + need;
    if (fused) {
        // everything the fused form needs is checked before anything is launched
        bool ok2 = ((uintptr_t)a.A % 16 == 0) && (a.lda % EPC == 0) && (a.K % EPC == 0 || a.a_pad_zero) &&
                   ((uintptr_t)a.A2 % 16 == 0) && (a.lda2 % EPC == 0) && (a.K2 % EPC == 0 || a.a2_pad_zero) && a.K2 >= 1 &&
                   !a.a_mask && !a.accumulate && n_pad <= 128 && a.N % 4 == 0 && a.ldc % 4 == 0 && ((uintptr_t)a.C % 16 == 0) &&
                   getenv("SLICEGCN_NO_WS") == nullptr;
        for (int g = 0; g < a.groups; ++g) ok2 = ok2 && a.a_start[g] % EPC == 0 && a.a2_start[g] % EPC == 0 && a.c_start[g] % 4 == 0;
        if (a.mask_out) ok2 = ok2 && (a.mask_ld % 4 == 0) && ((uintptr_t)a.mask_out % 4 == 0);
        if (a.mul_pos) ok2 = false;
        if (a.bias) ok2 = ok2 && ((uintptr_t)a.bias % 16 == 0);
        if (a.post1) ok2 = ok2 && ((uintptr_t)a.post1 % 16 == 0);
        if (a.post2) ok2 = ok2 && ((uintptr_t)a.post2 % 16 == 0);
        const int stage_b2 = (BF16 ? 16384 : 32768) + 2 * n_pad * 128;
        ok2 = ok2 && (220 * 1024 - (8 * 32 * kStagePitch * 4 + 256 + 1024 + 2 * kWsVecFloats * 4)) / stage_b2 >= 2;
        if (!ok2) return SLICEGCN_ERR_UNSUPPORTED;
    }
    const int smem_bytes = (BF16 ? 16384 : 32768) + 4 * n_pad * 128 + 4 * 32 * kStagePitch * 4 + 64 + 1024;
    static bool configured = false;
    if (!configured) {
        const int mx = 32768 + 4 * 256 * 128 + 4 * 32 * kStagePitch * 4 + 64 + 1024;
        SGCN_CUDA(cudaFuncSetAttribute(tc_gemm_kernel<TA, TC, BF16, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx));
        SGCN_CUDA(cudaFuncSetAttribute(tc_gemm_kernel<TA, TC, BF16, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx));
        configured = true;
    }
    {   // weight image(s): from the epoch's cache when there is one, else converted here into the scratch
        PrepJob j{a.B, a.b_gstride, a.ldb, a.b_trans, a.K, a.N, n_pad, n_slabs, n_tiles, a.groups, BF16 ? 1 : 0, a.b_kstack, nullptr, 0};
        bool fresh = false;
        unsigned char* cimg = cached_image(j, need, &fresh);
        if (cimg) image = cimg;
        else j.image = static_cast<unsigned char*>(image);
        if (!fresh) {
            dim3 pgrid(n_slabs * 4, n_tiles, a.groups);
            tc_prep_b_kernel<BF16><<<pgrid, 128, 0, st>>>(j);
            SGCN_LAUNCH_CHECK();
            count_launch();
        }
        if (fused) {
            PrepJob j2{a.B2, a.b2_gstride, a.ldb, a.b_trans, a.K2, a.N, n_pad, n_slabs2, n_tiles, a.groups, BF16 ? 1 : 0, 0, nullptr, 0};
            bool fresh2 = false;
            unsigned char* cimg2 = cached_image(j2, need2, &fresh2);
            if (cimg2) image2 = cimg2;
            else j2.image = image2;
            if (!fresh2) {
                dim3 pgrid2(n_slabs2 * 4, n_tiles, a.groups);
                tc_prep_b_kernel<BF16><<<pgrid2, 128, 0, st>>>(j2);
                SGCN_LAUNCH_CHECK();
                count_launch();
            }
        }
    }
    // 16-byte loads of the activation need aligned slices
    bool vec = ((uintptr_t)a.A % 16 == 0) && (a.lda % EPC == 0) && (a.K % EPC == 0 || a.a_pad_zero);
    for (int g = 0; g < a.groups; ++g) vec = vec && (a.a_start[g] % EPC == 0);
    if (a.a_mask) vec = vec && ((uintptr_t)a.a_mask % 8 == 0) && (a.a_mask_ld % 8 == 0);
    static const bool no_ws = getenv("SLICEGCN_NO_WS") != nullptr;
    // the warp-specialised kernel also writes (and re-reads) C, the ReLU mask and the gate in 4-element pieces
    const int ces = sizeof(TC);
    bool cvec = (a.N % 4 == 0) && (a.ldc % 4 == 0) && ((uintptr_t)a.C % 16 == 0);
    for (int g = 0; g < a.groups; ++g) cvec = cvec && (a.c_start[g] % 4 == 0);
    if (a.mask_out) cvec = cvec && (a.mask_ld % 4 == 0) && ((uintptr_t)a.mask_out % 4 == 0);
    if (a.mul_pos) cvec = cvec && (a.mul_pos_ld % 4 == 0) && ((uintptr_t)a.mul_pos % 16 == 0);
    if (a.bias) cvec = cvec && ((uintptr_t)a.bias % 16 == 0);
    if (a.post1) cvec = cvec && ((uintptr_t)a.post1 % 16 == 0);
    if (a.post2) cvec = cvec && ((uintptr_t)a.post2 % 16 == 0);
    (void)ces;
    const int64_t all_items = ((a.M + 127) / 128) * a.groups * n_tiles;
    {
        // the kernel that keeps the activation operand in TMEM (fp32 -> fp32 / bf16, bf16 -> bf16 / fp32)
        if (ts_gemm_ok(a, n_pad, n_tiles)) {
            constexpr int eb = BF16 ? 2 : 4;       // bytes per activation element; a slab row is 128 bytes either way
            // columns the slabs may touch: up to the end of the last group (the rest reads as zeros)
            int cols1 = 0, cols2 = 0;
            for (int g = 0; g < a.groups; ++g) {
                cols1 = std::max(cols1, a.a_start[g] + a.K);
                if (fused) cols2 = std::max(cols2, a.a2_start[g] + a.K2);
            }
            CUtensorMap map_a, map_a2, map_m;
            bool maps_ok = make_slab_map(&map_a, a.A, a.M, std::min<int64_t>(cols1, a.lda), a.lda, 128 / eb, 128, true, eb);
            if (maps_ok && fused)
                maps_ok = make_slab_map(&map_a2, a.A2, a.M, std::min<int64_t>(cols2, a.lda2), a.lda2, 128 / eb, 128, true, eb);
            if (maps_ok && !fused) map_a2 = map_a;
            if (maps_ok && a.a_mask)
                maps_ok = make_slab_map(&map_m, a.a_mask, a.M, std::min<int64_t>(cols1, a.a_mask_ld), a.a_mask_ld, 32, 128, false, 1);
            if (maps_ok && !a.a_mask) map_m = map_a;
            if (maps_ok) {
            // as many raw slabs as fit next to the weight images and the staging tiles (wider images leave fewer)
            const int raw_slot = a.a_mask ? 20480 : 16384;
            const int ts_fixed = kTsStages * 2 * n_pad * 128 + 8 * 32 * kStagePitch * 4 + 8 * 32 * kTsMaskPitch + 2 * (kWsVecFloats + 64) * 4 + 256 + 1024;
            const int ring = std::min(kTsRing, (225 * 1024 - ts_fixed) / raw_slot);
            const int ts_smem = ts_fixed + ring * raw_slot;
            static bool ts_configured = false;
            if (!ts_configured) {
                SGCN_CUDA(cudaFuncSetAttribute(tc_gemm_ts_kernel<false, BF16, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
                if (!BF16)
                    SGCN_CUDA(cudaFuncSetAttribute(tc_gemm_ts_kernel<!BF16, BF16, TC>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
                ts_configured = true;
            }
            int64_t tgrid = 148;
            if (tgrid > all_items) tgrid = all_items;
            if (!BF16 && a.a_mask)
                tc_gemm_ts_kernel<!BF16, BF16, TC><<<(unsigned)tgrid, kTsThreads, ts_smem, st>>>(a, n_pad, n_tiles, ring, static_cast<unsigned char*>(image),
                                                                                                 image2, fault, map_a, map_a2, map_m);
            else
                tc_gemm_ts_kernel<false, BF16, TC><<<(unsigned)tgrid, kTsThreads, ts_smem, st>>>(a, n_pad, n_tiles, ring, static_cast<unsigned char*>(image),
                                                                                                 image2, fault, map_a, map_a2, map_m);
            SGCN_LAUNCH_CHECK();
            count_launch();
            return SLICEGCN_OK;
            }
        }
    }
    if (vec && cvec && !a.a_mask && !no_ws && all_items < ((int64_t)1 << 31)) {
        // warp-specialised kernel: one CTA per SM, ring depth from what fits in shared memory
        const int a_bytes = BF16 ? 16384 : 32768;
        const int stage_b = a_bytes + 2 * n_pad * 128;
        const int fixed = (fused ? 8 : 4) * 32 * kStagePitch * 4 + 256 + 1024 + 2 * kWsVecFloats * 4;
        int D = (220 * 1024 - fixed) / stage_b;
        if (D > 4) D = 4;
        if (D >= 2) {
            const int ws_smem = D * stage_b + fixed;
            static bool ws_configured = false;
            if (!ws_configured) {
                SGCN_CUDA(cudaFuncSetAttribute(tc_gemm_ws_kernel<TA, TC, BF16>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
                ws_configured = true;
            }
            const int64_t items = ((a.M + 127) / 128) * a.groups * n_tiles;
            int64_t wgrid = 148;
            if (wgrid > items) wgrid = items;
            tc_gemm_ws_kernel<TA, TC, BF16><<<(unsigned)wgrid, kWsThreads, ws_smem, st>>>(a, n_pad, n_tiles, D, static_cast<unsigned char*>(image), image2, fault);
            SGCN_LAUNCH_CHECK();
            count_launch();
            return SLICEGCN_OK;
        }
    }
    if (fused) return SLICEGCN_ERR_UNSUPPORTED;   // not reachable: the fused form was vetted above
    // persistent grid: as many CTAs as fit at once (shared memory and 512 TMEM columns per SM)
    int ncols = 32;
    while (ncols < n_pad) ncols <<= 1;
    int per_sm = (227 * 1024) / (smem_bytes + 1024);
    if (per_sm > 512 / ncols) per_sm = 512 / ncols;
    if (per_sm > 8) per_sm = 8;
    if (per_sm < 1) per_sm = 1;
    const int64_t n_items = ((a.M + 127) / 128) * a.groups * n_tiles;
    int64_t grid = (int64_t)148 * per_sm;
    if (grid > n_items) grid = n_items;
    if (vec)
        tc_gemm_kernel<TA, TC, BF16, true><<<(unsigned)grid, kTcThreads, smem_bytes, st>>>(a, n_pad, n_tiles, static_cast<unsigned char*>(image), fault);
    else
        tc_gemm_kernel<TA, TC, BF16, false><<<(unsigned)grid, kTcThreads, smem_bytes, st>>>(a, n_pad, n_tiles, static_cast<unsigned char*>(image), fault);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

// ------------------------------------------------------------------------------ weight gradient
// dW = A^T B with the reduction running over the rows (nodes).  One CTA owns a 128-wide tile of A's
// columns (the MMA's M), the matching columns of B (the MMA's N: for grouped layers only the groups
// of that tile, so the block-diagonal structure is not wasted twice) and a chunk of rows.  Every 32
// rows form one K slab: both operands are read with 16-byte loads, transposed in registers (4x4
// micro-tiles) and stored K-major; the next slab's loads are in flight while the current slab's MMAs
// run (two shared-memory stages).  The CTA's partial product leaves TMEM once, at the end, into the
// scratch buffer; a second kernel sums the chunks in a fixed order.
constexpr int kWgThreads = 256;

struct WgTcPlan {
    int m_tiles;        // tiles of 128 A-columns
    int n_t;            // B columns per tile (MMA N, multiple of 16)
    int n_valid;        // valid B columns per tile
    int a_col0, b_col0; // first column of A / B
    int a_cols;         // total A columns (all groups)
    int b_cols_per_tile;
    int a_tile_cols;    // A columns between consecutive tiles (128 unless the narrow grouped plan is used)
    int a_box;          // A columns fetched per tile (multiple of 32, <= 128)
    int n_chunks;
    int64_t rows_per_chunk;
    int stages;
};

template <typename TA, int STAGES>
__global__ void __launch_bounds__(kWgThreads, STAGES == 1 ? 2 : 1) tc_wgrad_kernel(const WgradArgs a, const WgTcPlan pl,
                                                                                    float* scratch, int* fault) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int mt = blockIdx.y, chunk = blockIdx.x;
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    const uint32_t a_bytes = 16384, b_bytes = (uint32_t)pl.n_t * 128u;
    const uint32_t stage_bytes = 2 * a_bytes + 2 * b_bytes;
    unsigned char* tail = base + STAGES * stage_bytes;
    uint64_t* mbar_done = reinterpret_cast<uint64_t*>(tail);   // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tail + 16);
    uint32_t ncols = 32;
    while ((int)ncols < pl.n_t) ncols <<= 1;
    if (tid == 0) {
        mbar_init(&mbar_done[0], 1);
        mbar_init(&mbar_done[1], 1);
    }
    if (warp == 0) tmem_alloc(tmem_slot, ncols);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int64_t r_begin = (int64_t)chunk * pl.rows_per_chunk;
    const int64_t r_end = min(a.M, r_begin + pl.rows_per_chunk);
    const int n_slabs = (int)((r_end - r_begin + 31) / 32);
    // this thread's 4x4 micro-tiles: rows 4*rq .. 4*rq+3 of the slab, column quad cq of the operand
    const int rq = lane & 7;
    const int a_cq = warp * 4 + (lane >> 3);                 // 32 column quads of A (128 columns)
    const int a_col = mt * 128 + a_cq * 4;                   // column inside A's range
    const bool a_ok = a_col < pl.a_cols;
    const TA* Ap = static_cast<const TA*>(a.A) + pl.a_col0 + a_col;
    const int b_quads = pl.n_t / 4;                          // column quads of B in this tile (<= 64)
    const float* Bp = a.B + pl.b_col0 + mt * pl.b_cols_per_tile;
    const uint8_t* Mp = a.b_mask ? a.b_mask + pl.b_col0 + mt * pl.b_cols_per_tile : nullptr;

    float4 ra[4];
    float4 rb[2][4];
    auto load = [&](int s) {
        const int64_t rr = r_begin + (int64_t)s * 32 + rq * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            const int64_t row = rr + i;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            if (a_ok && row < r_end) {
                if (sizeof(TA) == 4) {
                    v = __ldg(reinterpret_cast<const float4*>(reinterpret_cast<const float*>(Ap) + row * a.lda));
                } else {
                    const uint2 h = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const __nv_bfloat16*>(Ap) + row * a.lda));
                    v = make_float4(__uint_as_float(h.x << 16), __uint_as_float(h.x & 0xffff0000u),
                                    __uint_as_float(h.y << 16), __uint_as_float(h.y & 0xffff0000u));
                }
            }
            ra[i] = v;
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                const int cq = warp * 4 + (lane >> 3) + 32 * j;
                float4 w = make_float4(0.f, 0.f, 0.f, 0.f);
                if (cq < b_quads && cq * 4 < pl.n_valid && row < r_end) {
                    w = __ldg(reinterpret_cast<const float4*>(Bp + row * a.ldb + cq * 4));
                    if (Mp) {
                        const uint32_t m4 = *reinterpret_cast<const uint32_t*>(Mp + row * a.b_mask_ld + cq * 4);
                        if (!(m4 & 0x000000FFu)) w.x = 0.f;
                        if (!(m4 & 0x0000FF00u)) w.y = 0.f;
                        if (!(m4 & 0x00FF0000u)) w.z = 0.f;
                        if (!(m4 & 0xFF000000u)) w.w = 0.f;
                    }
                }
                rb[j][i] = w;
            }
        }
    };
    // element (column c of the quad, rows 4*rq..+3) -> tile row (quad*4 + c), 16-byte chunk rq
    auto put_quad = [&](unsigned char* hi, unsigned char* lo, int quad, const float4 (&r)[4]) {
        const float e[4][4] = {{r[0].x, r[1].x, r[2].x, r[3].x},
                               {r[0].y, r[1].y, r[2].y, r[3].y},
                               {r[0].z, r[1].z, r[2].z, r[3].z},
                               {r[0].w, r[1].w, r[2].w, r[3].w}};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            const uint32_t off = sw_off(quad * 4 + c, rq * 16);
            const float h0 = tf32_hi(e[c][0]), h1 = tf32_hi(e[c][1]), h2 = tf32_hi(e[c][2]), h3 = tf32_hi(e[c][3]);
            *reinterpret_cast<float4*>(hi + off) = make_float4(h0, h1, h2, h3);
            *reinterpret_cast<float4*>(lo + off) = make_float4(e[c][0] - h0, e[c][1] - h1, e[c][2] - h2, e[c][3] - h3);
        }
    };
    const uint32_t idesc = idesc_f32acc(128, pl.n_t, false);
    uint32_t done_phase = 0;   // bit i: parity to wait for on mbar_done[i]
    int pending[2] = {0, 0};   // commits on each stage not yet waited for
    bool ok = true;
    if (n_slabs > 0) load(0);
    for (int s = 0; s < n_slabs && ok; ++s) {
        const int st = STAGES == 1 ? 0 : (s & 1);
        unsigned char* A_hi = base + st * stage_bytes;
        unsigned char* A_lo = A_hi + a_bytes;
        unsigned char* B_hi = A_lo + a_bytes;
        unsigned char* B_lo = B_hi + b_bytes;
        if (pending[st]) {   // the MMAs of slab s-2 must have finished reading this stage
            ok = mbar_wait(&mbar_done[st], (done_phase >> st) & 1u);
            done_phase ^= (1u << st);
            pending[st] = 0;
            if (!ok) break;
        }
        put_quad(A_hi, A_lo, a_cq, ra);
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int cq = warp * 4 + (lane >> 3) + 32 * j;
            if (cq < b_quads) put_quad(B_hi, B_lo, cq, rb[j]);
        }
        if (s + 1 < n_slabs) load(s + 1);   // in flight while this slab's MMAs run
        proxy_fence();
        tc_fence_before();
        __syncthreads();
        if (tid == 0) {
            tc_fence_after();
            const uint64_t da_hi = smem_desc(A_hi), da_lo = smem_desc(A_lo);
            const uint64_t db_hi = smem_desc(B_hi), db_lo = smem_desc(B_lo);
#pragma unroll
            for (int ks = 0; ks < 4; ++ks) {
                const uint64_t adv = (uint64_t)((ks * 32) >> 4);
                umma<false>(tmem, da_hi + adv, db_hi + adv, idesc, (s == 0 && ks == 0) ? 0u : 1u);
                if (sizeof(TA) == 4) umma<false>(tmem, da_lo + adv, db_hi + adv, idesc, 1u);   // bf16 values have no lo part
                umma<false>(tmem, da_hi + adv, db_lo + adv, idesc, 1u);
            }
            umma_commit(&mbar_done[st]);
        }
        pending[st] = 1;
    }
    // drain the commits still outstanding (at most one per stage)
    for (int st = 0; st < 2; ++st)
        if (ok && pending[st]) ok = mbar_wait(&mbar_done[st], (done_phase >> st) & 1u);
    tc_fence_after();
    float* out = scratch + ((int64_t)chunk * pl.m_tiles + mt) * 128 * pl.n_t;
    if (ok && warp < 4) {
        if (n_slabs > 0) {
            for (int c0 = 0; c0 < pl.n_t; c0 += 32) {
                float v[32];
                tmem_ld32(tmem + ((uint32_t)(warp * 32) << 16) + (uint32_t)c0, v);
                float* o = out + (int64_t)(warp * 32 + lane) * pl.n_t + c0;
#pragma unroll
                for (int j = 0; j < 32; j += 4)
                    if (c0 + j < pl.n_t) *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
            }
        } else {
            float* o = out + (int64_t)(warp * 32 + lane) * pl.n_t;
            for (int j = 0; j < pl.n_t; ++j) o[j] = 0.f;
        }
    }
    if (!ok && tid == 0) atomicExch(fault, 4);
    tc_fence_before();
    __syncthreads();
    if (warp == 0) tmem_dealloc(tmem, ncols);
}

// ------------------------------------------------------------------------------ weight gradient, warp-specialised
// Same product, for unmasked fp32 operands.  Both operands of dW = A^T B are read in their natural
// row-major form: a slab of 32 rows is, for the MMA, a K=32 slice whose M (resp. N) index runs along
// the contiguous columns -- the "MN-major" operand form -- so the slab goes from global memory into
// the swizzled tile by cp.async without any transposition, and the producers only split it into hi
// and lo parts in place.  One CTA per SM: 4 producer warps keep a ring of D stages filled, one thread
// of warp 4 issues the MMAs (one accumulation chain per CTA), warps 5-8 write the partial tile out at
// the end.  Tile layout (the one MN-major tf32 operands must use, "128-byte swizzle with 32-byte
// base"): atoms of 4 K-rows x 128 bytes (32 columns), the 32-byte chunk index XORed with the K-row;
// atom (K atom ka, column block mb) at ((ka * blocks + mb) * 512) bytes.
__device__ __forceinline__ uint64_t smem_desc_mn(const void* tile, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_u32(tile) >> 4) & 0x3FFF);
    d |= (uint64_t)((lbo_bytes >> 4) & 0x3FFF) << 16;   // between column blocks (MN direction)
    d |= (uint64_t)((sbo_bytes >> 4) & 0x3FFF) << 32;   // between 8-row K blocks
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)1 << 61;                             // SWIZZLE_128B with 32-byte base
    return d;
}

template <bool WIDE>   // WIDE: more than 32 column quads in the B tile
__global__ void __launch_bounds__(kWsThreads, 1) tc_wgrad_ws_kernel(const WgradArgs a, const WgTcPlan pl, const int D,
                                                                    float* scratch, int* fault) {
    extern __shared__ __align__(1024) unsigned char smem[];
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int mt = blockIdx.y, chunk = blockIdx.x;
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    const int nbk = (pl.n_t + 31) / 32;                      // column blocks of the B tile
    const uint32_t b_bytes = 4u * (uint32_t)nbk * 1024u;     // one B tile (hi or lo)
    const uint32_t stage_bytes = 32768u + 2u * b_bytes;      // A hi | A lo | B hi | B lo
    unsigned char* tail = base + (uint32_t)D * stage_bytes;
    uint64_t* full = reinterpret_cast<uint64_t*>(tail);      // [D] 128 producer arrivals
    uint64_t* freeb = full + 4;                              // [D] MMAs of the stage completed
    uint64_t* tfull = freeb + 4;                             // accumulator complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfull + 1);
    uint32_t ncols = 32;
    while ((int)ncols < pl.n_t) ncols <<= 1;
    if (tid == 0) {
        for (int i = 0; i < D; ++i) {
            mbar_init(&full[i], 128);
            mbar_init(&freeb[i], 1);
        }
        mbar_init(tfull, 1);
    }
    if (warp == 4) tmem_alloc(tmem_slot, ncols);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int64_t r_begin = (int64_t)chunk * pl.rows_per_chunk;
    const int64_t r_end = min(a.M, r_begin + pl.rows_per_chunk);
    const int n_slabs = r_end > r_begin ? (int)((r_end - r_begin + 31) / 32) : 0;

    if (warp < 4) {
        // ------------------------------------------------------------ producers
        // A: thread t copies 16-byte column chunk (t % 32) of rows t/32 + 4 i; B: chunk (t % 32) of the same
        // rows, or (WIDE) chunk (t % 64) of rows t/64 + 2 i
        const int acc_c = tid & 31, a_r0 = tid >> 5;
        const int b_cc = WIDE ? (tid & 63) : (tid & 31), b_r0 = WIDE ? (tid >> 6) : (tid >> 5);
        constexpr int BI = WIDE ? 16 : 8, BSTEP = WIDE ? 2 : 4;
        const int a_col = mt * 128 + acc_c * 4;
        const bool a_ok = a_col < pl.a_cols;
        const int nq = pl.n_t / 4;
        const bool b_ok = b_cc < nq && b_cc * 4 < pl.n_valid;
        const float* Ap = static_cast<const float*>(a.A) + pl.a_col0 + a_col;
        const float* Bp = a.B + pl.b_col0 + mt * pl.b_cols_per_tile + b_cc * 4;
        // (row r of the slab, 16-byte column chunk cc) -> byte offset inside the tile
        auto a_off = [&](int r) {
            return (uint32_t)((((r >> 2) * 4 + (acc_c >> 3)) << 9) + ((r & 3) << 7) + (((((acc_c & 7) >> 1) ^ (r & 3))) << 5) + ((acc_c & 1) << 4));
        };
        auto b_off = [&](int r) {
            return (uint32_t)((((r >> 2) * nbk + (b_cc >> 3)) << 9) + ((r & 3) << 7) + (((((b_cc & 7) >> 1) ^ (r & 3))) << 5) + ((b_cc & 1) << 4));
        };
        const int L = D >= 3 ? D - 1 : 1;
        int i_st = 0;            // issue cursor: stage and ring pass of the slab requested next
        uint32_t i_pass = 0;
        auto issue = [&](int j) {
            const int st = i_st;
            if (i_pass >= 1 && !mbar_wait(&freeb[st], (i_pass - 1) & 1)) {
                if (lane == 0) atomicExch(fault, 8);
                return false;
            }
            if (++i_st == D) {
                i_st = 0;
                ++i_pass;
            }
            unsigned char* stg = base + (uint32_t)st * stage_bytes;
            const uint32_t dA = smem_u32(stg), dB = smem_u32(stg + 32768);
            const int64_t rr = r_begin + (int64_t)j * 32;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int r = a_r0 + 4 * i;
                const bool in = a_ok && rr + r < r_end;
                const float* src = in ? Ap + (rr + r) * a.lda : static_cast<const float*>(a.A);
                const int sz = in ? 16 : 0;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dA + a_off(r)), "l"(src), "r"(sz) : "memory");
            }
            if (b_cc < nq) {
#pragma unroll
                for (int i = 0; i < BI; ++i) {
                    const int r = b_r0 + BSTEP * i;
                    const bool in = b_ok && rr + r < r_end;
                    const float* src = in ? Bp + (rr + r) * a.ldb : a.B;
                    const int sz = in ? 16 : 0;
                    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dB + b_off(r)), "l"(src), "r"(sz) : "memory");
                }
            }
            return true;
        };
        bool okp = true;
        for (int j = 0; j < L && okp; ++j) {
            if (j < n_slabs) okp = issue(j);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        int st = 0;
        for (int j = 0; j < n_slabs && okp; ++j) {
            if (L == 2) asm volatile("cp.async.wait_group 1;" ::: "memory");
            else asm volatile("cp.async.wait_group 0;" ::: "memory");
            unsigned char* stg = base + (uint32_t)st * stage_bytes;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const uint32_t off = a_off(a_r0 + 4 * i);
                const float4 v = *reinterpret_cast<const float4*>(stg + off);
                const float h0 = tf32_hi(v.x), h1 = tf32_hi(v.y), h2 = tf32_hi(v.z), h3 = tf32_hi(v.w);
                *reinterpret_cast<float4*>(stg + off) = make_float4(h0, h1, h2, h3);
                *reinterpret_cast<float4*>(stg + 16384 + off) = make_float4(v.x - h0, v.y - h1, v.z - h2, v.w - h3);
            }
            if (b_cc < nq) {
#pragma unroll
                for (int i = 0; i < BI; ++i) {
                    const uint32_t off = b_off(b_r0 + BSTEP * i);
                    const float4 v = *reinterpret_cast<const float4*>(stg + 32768 + off);
                    const float h0 = tf32_hi(v.x), h1 = tf32_hi(v.y), h2 = tf32_hi(v.z), h3 = tf32_hi(v.w);
                    *reinterpret_cast<float4*>(stg + 32768 + off) = make_float4(h0, h1, h2, h3);
                    *reinterpret_cast<float4*>(stg + 32768 + b_bytes + off) = make_float4(v.x - h0, v.y - h1, v.z - h2, v.w - h3);
                }
            }
            proxy_fence();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&full[st])) : "memory");
            if (++st == D) st = 0;
            if (j + L < n_slabs) okp = issue(j + L);
            asm volatile("cp.async.commit_group;" ::: "memory");
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // M = 128 A-columns, N = n_t B-columns, both operands MN-major
            const uint32_t idesc = idesc_f32acc(128, pl.n_t, false) | (1u << 15) | (1u << 16);
            bool okm = true;
            int st = 0;
            uint32_t pass = 0;
            for (int j = 0; j < n_slabs && okm; ++j) {
                okm = mbar_wait(&full[st], pass & 1);
                if (!okm) break;
                tc_fence_after();
                unsigned char* stg = base + (uint32_t)st * stage_bytes;
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    // one MMA covers 8 K-rows = two K atoms; column blocks are 512 bytes apart
                    const uint64_t da_hi = smem_desc_mn(stg + kb * 4096, 512, 2048);
                    const uint64_t da_lo = smem_desc_mn(stg + 16384 + kb * 4096, 512, 2048);
                    const uint64_t db_hi = smem_desc_mn(stg + 32768 + kb * nbk * 1024, 512, nbk * 512);
                    const uint64_t db_lo = smem_desc_mn(stg + 32768 + b_bytes + kb * nbk * 1024, 512, nbk * 512);
                    umma<false>(tmem, da_hi, db_hi, idesc, (j == 0 && kb == 0) ? 0u : 1u);
                    umma<false>(tmem, da_lo, db_hi, idesc, 1u);
                    umma<false>(tmem, da_hi, db_lo, idesc, 1u);
                }
                umma_commit(&freeb[st]);
                if (++st == D) {
                    st = 0;
                    ++pass;
                }
            }
            if (okm) umma_commit(tfull);
            else atomicExch(fault, 9);
        }
    } else {
        // ------------------------------------------------------------ epilogue: partial tile -> scratch
        const int q = warp & 3;
        float* out = scratch + ((int64_t)chunk * pl.m_tiles + mt) * 128 * pl.n_t + (int64_t)(q * 32 + lane) * pl.n_t;
        if (n_slabs > 0) {
            if (mbar_wait(tfull, 0)) {
                tc_fence_after();
                for (int c0 = 0; c0 < pl.n_t; c0 += 32) {
                    float v[32];
                    tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, v);
#pragma unroll
                    for (int j = 0; j < 32; j += 4)
                        if (c0 + j < pl.n_t) *reinterpret_cast<float4*>(out + c0 + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                }
            } else if (lane == 0) {
                atomicExch(fault, 10);
            }
        } else {
            for (int j = 0; j < pl.n_t; ++j) out[j] = 0.f;
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, ncols);
}

// ------------------------------------------------------------------------------ weight gradient, A^T operand in TMEM
// dW = A^T B for fp32 operands and B tiles of at most 128 columns (the sliced layers).  Same tiling and
// partial-sum scratch as the kernels above; what changes is the path of the operands, along the lines
// of the TS GEMM:
//   warp 5     loader: per slab of 32 rows one tensor copy of the A tile (32 x 128 values) and one of
//              the B tile (32 x n_t), unswizzled, into a ring of raw slots; rows past the end
//              of the matrix and columns past its width arrive as zeros.
//   warps 0-3  A producers: lane m of warp w reads column 32w + m of the raw A slab (32 values down the
//              rows -- consecutive lanes, consecutive words), splits them and writes hi and lo into a
//              TMEM stage with tcgen05.st: A^T in the K-major form, M index = TMEM lane.  After the last
//              slab they drain the accumulator into the scratch tile.
//   warps 8-15 B producers (they carry the most work per slab -- measured, they set the kernel's pace -- hence eight
//              warps): split the B slab (times its byte mask, if any) into the MN-major operand
//              tile ("128-byte swizzle, 32-byte base"; per K atom the hi column blocks are followed by
//              the lo column blocks, so [hi | lo] is one operand of 2 n_t columns) and keep the column
//              sums of B (the bias gradient).
//   warp 4     MMA issuer: per 8 rows A_hi x [B_hi | B_lo] and A_lo x B_hi.
// TMEM columns: accumulator [hi*hi + lo*hi | hi*lo] (64 nbk), then two stages of 64 (A hi | A lo).
constexpr int kWtThreads = 512;

// WIDE: B tiles of 129..256 columns -- no room for [hi | lo] in one operand (three chains per slab) and
// only two raw slots.  ABF16: A is stored as bf16 -- exact in tf32, so it has no lo part and a slab takes
// one chain less.
template <bool WIDE, bool ABF16>
__global__ void __launch_bounds__(kWtThreads, 1) tc_wgrad_ts_kernel(const WgradArgs a, const WgTcPlan pl, float* scratch, float* colsum,
                                                                    int* fault, const __grid_constant__ CUtensorMap map_a,
                                                                    const __grid_constant__ CUtensorMap map_b,
                                                                    const __grid_constant__ CUtensorMap map_bm) {
    extern __shared__ __align__(1024) unsigned char smem[];
    constexpr int R = WIDE ? 2 : 4, S = 2;   // raw slots; operand stages (TMEM A + shared-memory B)
    constexpr uint32_t kARaw = ABF16 ? 8192u : 16384u;   // raw A slab: 32 rows x 128 columns
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int mt = blockIdx.y, chunk = blockIdx.x;
    unsigned char* base = smem + ((1024u - (smem_u32(smem) & 1023u)) & 1023u);
    const int nbk = (pl.n_t + 31) / 32;                      // column blocks of the B tile
    const uint32_t b_raw_bytes = 32u * (uint32_t)pl.n_t * 4u;
    const bool masked = a.b_mask != nullptr;                 // B is multiplied by a byte mask on the way
    const uint32_t b_raw_pad = (b_raw_bytes + 1023u) & ~1023u;
    const uint32_t m_raw_bytes = 32u * (uint32_t)pl.n_t;
    const uint32_t slot_bytes = kARaw + b_raw_pad + (masked ? ((m_raw_bytes + 1023u) & ~1023u) : 0u);   // raw A | raw B | mask
    const uint32_t op_bytes = (uint32_t)nbk * 8192u;         // B operand stage: 8 K atoms x (nbk hi + nbk lo) x 512 B
    unsigned char* ops = base;                               // [S]
    unsigned char* raw = ops + S * op_bytes;                 // [R]
    float* csum_s = reinterpret_cast<float*>(raw + kARaw);   // [8][n_t] (wide: [4][n_t]) column-sum partials: reuse the B part of raw slot 0 after the last slab
    uint64_t* afull = reinterpret_cast<uint64_t*>(raw + R * slot_bytes);   // [S] 128 producer arrivals
    uint64_t* afree = afull + S;                             // [S] MMAs of the stage completed
    uint64_t* rfull = afree + S;                             // [R] raw slab landed
    uint64_t* rfree = rfull + R;                             // [R] raw slab read by the four producer warps
    uint64_t* tfull = rfree + R;                             // accumulator complete
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfull + 1);
    const uint32_t accw = (WIDE ? 32u : 64u) * (uint32_t)nbk;   // accumulator columns
    if (tid == 0) {
        for (int i = 0; i < S; ++i) {
            mbar_init(&afull[i], 128 + 256);
            mbar_init(&afree[i], 1);
        }
        for (int i = 0; i < R; ++i) {
            mbar_init(&rfull[i], 1);
            mbar_init(&rfree[i], 4 + 8);
        }
        mbar_init(tfull, 1);
    }
    if (warp == 4) tmem_alloc(tmem_slot, 512);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *tmem_slot;

    const int64_t r_begin = (int64_t)chunk * pl.rows_per_chunk;
    const int64_t r_end = min(a.M, r_begin + pl.rows_per_chunk);
    const int n_slabs = r_end > r_begin ? (int)((r_end - r_begin + 31) / 32) : 0;

    if (warp < 4) {
        // ------------------------------------------------------------ A producers (and, at the end, epilogue)
        int rs = 0, ts = 0;
        uint32_t pass = 0, rpass = 0;
        bool okp = true;
        for (int j = 0; j < n_slabs; ++j) {
            okp = mbar_wait(&rfull[rs], rpass & 1);
            if (okp && pass >= 1) okp = mbar_wait(&afree[ts], (pass - 1) & 1);
            if (!okp) break;
            tc_fence_after();
            const unsigned char* slot = raw + rs * slot_bytes;
            // column 32 warp + lane of the slab, 32 values down the rows
            const bool a_live = 32 * warp + lane < pl.a_box;   // columns past the fetched width stay zero
            const float* acol = reinterpret_cast<const float*>(slot) + (a_live ? 32 * warp + lane : 0);
            const uint16_t* acol16 = reinterpret_cast<const uint16_t*>(slot) + (a_live ? 32 * warp + lane : 0);
            const uint32_t t_hi = tmem + ((uint32_t)(32 * warp) << 16) + accw + (uint32_t)ts * 64u;
#pragma unroll
            for (int half = 0; half < 2; ++half) {
                uint32_t h[32];   // [0,16): hi of rows 16 half ..; [16,32): lo of the same
#pragma unroll
                for (int k = 0; k < 16; ++k) {
                    if (ABF16) {
                        h[k] = a_live ? (uint32_t)acol16[(16 * half + k) * pl.a_box] << 16 : 0u;
                        h[16 + k] = 0u;
                    } else {
                        const float v = a_live ? acol[(16 * half + k) * pl.a_box] : 0.f;
                        const float hv = tf32_hi(v);
                        h[k] = __float_as_uint(hv);
                        h[16 + k] = __float_as_uint(v - hv);
                    }
                }
                if (half == 1) {   // the slab is in registers: this warp is done with the raw slot
                    __syncwarp();
                    if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rfree[rs])) : "memory");
                    __syncwarp();
                }
                tmem_st16<0>(t_hi + 16u * half, h);
                if (!ABF16) tmem_st16<16>(t_hi + 32u + 16u * half, h);
            }
            tmem_st_wait();
            tc_fence_before();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&afull[ts])) : "memory");
            if (++rs == R) {
                rs = 0;
                ++rpass;
            }
            if (++ts == S) {
                ts = 0;
                ++pass;
            }
        }
        if (!okp && lane == 0) atomicExch(fault, 8);
        // epilogue: partial tile -> scratch (row = A column 32 warp + lane of the tile)
        float* out = scratch + ((int64_t)chunk * pl.m_tiles + mt) * 128 * pl.n_t + (int64_t)(warp * 32 + lane) * pl.n_t;
        if (n_slabs > 0 && okp) {
            if (mbar_wait(tfull, 0)) {
                tc_fence_after();
                const uint32_t d_tmem = tmem + ((uint32_t)(warp * 32) << 16);
                for (int c0 = 0; c0 < pl.n_t; c0 += 16) {
                    float x[32];
#pragma unroll
                    for (int jx = 0; jx < 16; ++jx) x[jx] = 0.f;
                    tmem_ld16_add<0>(d_tmem + (uint32_t)c0, x);
                    if (!WIDE) tmem_ld16_add<0>(d_tmem + (uint32_t)(32 * nbk + c0), x);
#pragma unroll
                    for (int jx = 0; jx < 16; jx += 4)
                        *reinterpret_cast<float4*>(out + c0 + jx) = make_float4(x[jx], x[jx + 1], x[jx + 2], x[jx + 3]);
                }
            } else if (lane == 0) {
                atomicExch(fault, 10);
            }
        } else if (n_slabs == 0) {
            for (int jx = 0; jx < pl.n_t; ++jx) out[jx] = 0.f;
        }
    } else if (warp >= 8) {
        // ------------------------------------------------------------ B producers: split (and mask) the B slab into the
        // operand tile, keep its column sums.  16-byte column chunk b_cc of rows b_r0 + BSTEP i.
        const int tb = tid - 256;
        const int b_cc = WIDE ? (tb & 63) : (tb & 31), b_r0 = WIDE ? (tb >> 6) : (tb >> 5);   // 256 threads
        constexpr int BI = WIDE ? 8 : 4, BSTEP = WIDE ? 4 : 8;
        const int nq = pl.n_t / 4;
        const bool b_mine = b_cc < nq;
        float4 csum = make_float4(0.f, 0.f, 0.f, 0.f);
        int rs = 0, ts = 0;
        uint32_t pass = 0, rpass = 0;
        bool okp = true;
        for (int j = 0; j < n_slabs; ++j) {
            okp = mbar_wait(&rfull[rs], rpass & 1);
            if (okp && pass >= 1) okp = mbar_wait(&afree[ts], (pass - 1) & 1);
            if (!okp) break;
            const unsigned char* slot = raw + rs * slot_bytes;
            if (b_mine) {
                const unsigned char* braw = slot + kARaw + b_cc * 16;
                const unsigned char* mraw = slot + kARaw + b_raw_pad + b_cc * 4;
                unsigned char* op = ops + ts * op_bytes;
#pragma unroll
                for (int i = 0; i < BI; ++i) {
                    const int r = b_r0 + BSTEP * i;
                    float4 v = *reinterpret_cast<const float4*>(braw + r * (pl.n_t * 4));
                    if (masked) {
                        const uint32_t m = *reinterpret_cast<const uint32_t*>(mraw + r * pl.n_t);
                        v.x = (m & 0xffu) ? v.x : 0.f;
                        v.y = (m & 0xff00u) ? v.y : 0.f;
                        v.z = (m & 0xff0000u) ? v.z : 0.f;
                        v.w = (m & 0xff000000u) ? v.w : 0.f;
                    }
                    const float h0 = tf32_hi(v.x), h1 = tf32_hi(v.y), h2 = tf32_hi(v.z), h3 = tf32_hi(v.w);
                    const uint32_t off = (uint32_t)((((r >> 2) * 2 * nbk + (b_cc >> 3)) << 9) + ((r & 3) << 7) +
                                                    (((((b_cc & 7) >> 1) ^ (r & 3))) << 5) + ((b_cc & 1) << 4));
                    *reinterpret_cast<float4*>(op + off) = make_float4(h0, h1, h2, h3);
                    *reinterpret_cast<float4*>(op + off + nbk * 512) = make_float4(v.x - h0, v.y - h1, v.z - h2, v.w - h3);
                    csum.x += v.x; csum.y += v.y; csum.z += v.z; csum.w += v.w;
                }
            }
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&rfree[rs])) : "memory");
            proxy_fence();
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&afull[ts])) : "memory");
            if (++rs == R) {
                rs = 0;
                ++rpass;
            }
            if (++ts == S) {
                ts = 0;
                ++pass;
            }
        }
        if (!okp && lane == 0) atomicExch(fault, 8);
        // column sums of this chunk's rows: the row groups of each column chunk, added in a fixed order
        if (colsum && (pl.b_cols_per_tile > 0 || mt == 0)) {
            asm volatile("bar.sync 1, 256;" ::: "memory");   // every B producer has read its last raw slab
            if (b_mine) *reinterpret_cast<float4*>(csum_s + b_r0 * pl.n_t + b_cc * 4) = csum;   // (inside the slot's B part: 128 n_t bytes)
            asm volatile("bar.sync 1, 256;" ::: "memory");
            for (int cidx = tb; cidx < pl.n_t; cidx += 256) {
                float sum = 0.f;   // the row groups' partial sums in a fixed order
#pragma unroll
                for (int rg = 0; rg < (WIDE ? 4 : 8); ++rg) sum += csum_s[rg * pl.n_t + cidx];
                colsum[((int64_t)chunk * pl.m_tiles + mt) * pl.n_t + cidx] = cidx < pl.n_valid ? sum : 0.f;
            }
        }
    } else if (warp == 4) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            // M = 128 A-columns (K-major, from TMEM), N = B-columns (MN-major, from shared memory)
            const uint32_t idesc_wide = idesc_f32acc(128, WIDE ? 32 * nbk : 64 * nbk, false) | (1u << 16);
            const uint32_t idesc_hi = idesc_f32acc(128, 32 * nbk, false) | (1u << 16);
            bool okm = true;
            int ts = 0;
            uint32_t pass = 0;
            for (int j = 0; j < n_slabs && okm; ++j) {
                okm = mbar_wait(&afull[ts], pass & 1);
                if (!okm) break;
                tc_fence_after();
                const unsigned char* op = ops + ts * op_bytes;
                const uint32_t a_hi = tmem + accw + (uint32_t)ts * 64u, a_lo = a_hi + 32u;
#pragma unroll
                for (int kb = 0; kb < 4; ++kb) {
                    // one MMA covers 8 rows = two K atoms; column blocks are 512 bytes apart
                    const uint64_t db = smem_desc_mn(op + kb * 2 * (2 * nbk * 512), 512, 2 * nbk * 512);
                    if (WIDE) {
                        const uint64_t db_lo = smem_desc_mn(op + kb * 2 * (2 * nbk * 512) + nbk * 512, 512, 2 * nbk * 512);
                        umma_ts_tf32(tmem, a_hi + 8u * kb, db, idesc_hi, (j == 0 && kb == 0) ? 0u : 1u);
                        if (!ABF16) umma_ts_tf32(tmem, a_lo + 8u * kb, db, idesc_hi, 1u);
                        umma_ts_tf32(tmem, a_hi + 8u * kb, db_lo, idesc_hi, 1u);
                    } else {
                        umma_ts_tf32(tmem, a_hi + 8u * kb, db, idesc_wide, (j == 0 && kb == 0) ? 0u : 1u);
                        if (!ABF16) umma_ts_tf32(tmem, a_lo + 8u * kb, db, idesc_hi, 1u);
                    }
                }
                umma_commit(&afree[ts]);
                if (++ts == S) {
                    ts = 0;
                    ++pass;
                }
            }
            if (okm) umma_commit(tfull);
            else atomicExch(fault, 9);
        }
    } else if (warp == 5) {
        // ------------------------------------------------------------ loader
        if (lane == 0) {
            int rs = 0;
            uint32_t rpass = 0;
            const int ax = pl.a_col0 + mt * pl.a_tile_cols, bx = pl.b_col0 + mt * pl.b_cols_per_tile;
            for (int j = 0; j < n_slabs; ++j) {
                if (rpass >= 1 && !mbar_wait(&rfree[rs], (rpass - 1) & 1)) {
                    atomicExch(fault, 11);
                    break;
                }
                unsigned char* slot = raw + rs * slot_bytes;
                const int y = (int)(r_begin + (int64_t)j * 32);
                mbar_expect_tx(&rfull[rs], (ABF16 ? 64u : 128u) * (uint32_t)pl.a_box + b_raw_bytes + (masked ? m_raw_bytes : 0u));
                tma_load_2d(slot, &map_a, ax, y, &rfull[rs]);
                tma_load_2d(slot + kARaw, &map_b, bx, y, &rfull[rs]);
                if (masked) tma_load_2d(slot + kARaw + b_raw_pad, &map_bm, bx, y, &rfull[rs]);
                if (++rs == R) {
                    rs = 0;
                    ++rpass;
                }
            }
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 4) tmem_dealloc(tmem, 512);
}

// dW[g][k][n] = sum over chunks of the partial tiles (fixed order).  A block owns 32 consecutive
// elements; its eight warps each sum every eighth chunk (a handful of independent loads, so the
// kernel is not one long dependent chain per element) and the eight partial sums are added in
// warp order.
// Blocks past the dW elements (when colsum != NULL) reduce the column-sum partials into dbias / dbias2 the same way.
__global__ void __launch_bounds__(256) tc_wgrad_reduce_kernel(const float* scratch, const WgTcPlan pl, int groups, int K, int N,
                                                              int groups_per_tile, float* dW, const float* colsum = nullptr,
                                                              float* dbias = nullptr, float* dbias2 = nullptr, int64_t ldw = 0) {
    __shared__ float part[8][32];
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int64_t total = (int64_t)groups * K * N;
    const int64_t w_blocks = (total + 31) / 32;
    if ((int64_t)blockIdx.x >= w_blocks) {   // bias part: element = (group, column)
        const int i = (int)((blockIdx.x - w_blocks) * 32) + lane;
        float s = 0.f;
        if (i < groups * N) {
            const int g = i / N, n = i % N;
            int mt = 0, c = n;
            if (groups_per_tile > 0) {
                mt = g / groups_per_tile;
                c = (g % groups_per_tile) * N + n;
            } else if (groups_per_tile < 0) {
                c = g * N + n;
            }
            const float* p = colsum + (int64_t)mt * pl.n_t + c;
            const int64_t stride = (int64_t)pl.m_tiles * pl.n_t;
            for (int ch = w; ch < pl.n_chunks; ch += 8) s += __ldg(p + ch * stride);
        }
        part[w][lane] = s;
        __syncthreads();
        if (w == 0 && i < groups * N) {
            float t = part[0][lane];
#pragma unroll
            for (int q = 1; q < 8; ++q) t += part[q][lane];
            if (dbias) dbias[i] = t;
            if (dbias2) dbias2[i] = t;
        }
        return;
    }
    const int64_t i = blockIdx.x * (int64_t)32 + lane;
    float s = 0.f;
    int64_t o = i;                  // where element i goes: rows of ldw floats when dW is a column block of a wider matrix
    if (i < total) {
        const int g = (int)(i / ((int64_t)K * N));
        const int k = (int)((i / N) % K), n = (int)(i % N);
        if (ldw > 0) o = ((int64_t)g * K + k) * ldw + n;
        int mt, f, c;
        if (groups_per_tile > 0) {   // grouped: tile mt holds groups mt*gpt .. ; block (g % gpt)
            mt = g / groups_per_tile;
            const int gl = g % groups_per_tile;
            f = gl * K + k;
            c = gl * N + n;
        } else if (groups_per_tile < 0) {   // all groups share A: tiles over K, group g in columns g*N ..
            mt = k / 128;
            f = k % 128;
            c = g * N + n;
        } else {                     // one group: tiles over K
            mt = k / 128;
            f = k % 128;
            c = n;
        }
        const float* p = scratch + ((int64_t)mt * 128 + f) * pl.n_t + c;
        const int64_t stride = (int64_t)pl.m_tiles * 128 * pl.n_t;
        int ch = w;
        for (; ch + 24 < pl.n_chunks; ch += 32) {   // four loads in flight, summed in chunk order
            float v[4];
#pragma unroll
            for (int q = 0; q < 4; ++q) v[q] = __ldg(p + (ch + 8 * q) * stride);
#pragma unroll
            for (int q = 0; q < 4; ++q) s += v[q];
        }
        for (; ch < pl.n_chunks; ch += 8) s += __ldg(p + ch * stride);
    }
    part[w][lane] = s;
    __syncthreads();
    if (w == 0 && i < total) {
        float t = part[0][lane];
#pragma unroll
        for (int q = 1; q < 8; ++q) t += part[q][lane];
        dW[o] = t;
    }
}

// narrow: grouped layers take fewer groups per tile so that a tile's B columns stay within 128 (the TMEM-operand
// kernel then runs its two-chain form with two operand stages, and may apply a mask); tiles of fewer than 128 A columns
// follow each other at a_tile_cols.
bool wgrad_tc_plan(const WgradArgs& a, WgTcPlan* pl, int* groups_per_tile, int force_per_sm = 0, bool narrow = false) {
    if (a.K < 1 || !a.dW) return false;
    bool shared_a = a.groups > 1;   // every group reads the same A columns (fused input feeding all slices)
    for (int g = 0; g < a.groups; ++g) shared_a = shared_a && (a.a_start[g] == a.a_start[0]);
    for (int g = 0; g < a.groups; ++g) {
        if (!shared_a && a.a_start[g] != a.a_start[0] + g * a.K) return false;
        if (a.b_start[g] != a.b_start[0] + g * a.N) return false;
    }
    // 4-element loads: aligned starts; widths either multiples of 4 or followed by zero padding
    if ((uintptr_t)a.A % 16 || a.lda % 4 || a.a_start[0] % 4) return false;
    if ((uintptr_t)a.B % 16 || a.ldb % 4 || a.b_start[0] % 4) return false;
    const bool a_single = a.groups == 1 || shared_a;
    if (a.K % 4 && !(a.a_pad_zero && a_single)) return false;
    if (a.N % 4 && !(a.b_pad_zero && a.groups == 1)) return false;
    if (a.b_mask && ((uintptr_t)a.b_mask % 4 || a.b_mask_ld % 4)) return false;
    WgTcPlan P{};
    P.a_tile_cols = 128;
    P.a_col0 = a.a_start[0];
    P.b_col0 = a.b_start[0];
    P.a_cols = shared_a ? a.K : a.groups * a.K;
    if (shared_a) {
        if (a.groups * a.N > 256) return false;
        P.m_tiles = (a.K + 127) / 128;
        P.n_valid = a.groups * a.N;
        P.b_cols_per_tile = 0;
        *groups_per_tile = -1;   // reduce: row k of tile k/128, column g*N + n
    } else if (a.groups > 1) {
        if (128 % a.K != 0) return false;
        int gpt = 128 / a.K;
        if (gpt > a.groups) gpt = a.groups;
        if (a.groups % gpt != 0) return false;
        if (narrow)
            while (gpt * a.N > 128 && gpt % 2 == 0) gpt /= 2;
        if (gpt * a.N > 256) return false;
        P.a_tile_cols = gpt * a.K;
        P.m_tiles = a.groups / gpt;
        P.n_valid = gpt * a.N;
        P.b_cols_per_tile = gpt * a.N;
        *groups_per_tile = gpt;
    } else {
        if (a.N > 256) return false;
        P.m_tiles = (a.K + 127) / 128;
        P.n_valid = a.N;
        P.b_cols_per_tile = 0;   // every tile multiplies the same B columns
        *groups_per_tile = 0;
    }
    P.n_t = (P.n_valid + 15) & ~15;
    P.a_box = std::min(128, (P.a_tile_cols + 31) & ~31);
    // single-stage CTAs are small enough for two or three per SM, which overlap each other
    P.stages = 1;
    const int per_sm = force_per_sm > 0 ? force_per_sm : (P.n_t <= 128 ? 3 : 2);
    int64_t want = (148 * per_sm + P.m_tiles - 1) / P.m_tiles;
    int64_t rpc = (a.M + want - 1) / want;
    rpc = (rpc + 31) / 32 * 32;
    if (rpc < 32) rpc = 32;
    P.rows_per_chunk = rpc;
    P.n_chunks = (int)((a.M + rpc - 1) / rpc);
    *pl = P;
    return true;
}

// Weight gradients that tc_wgrad_ts_kernel takes under plan pl (fp32, one CTA per SM): B tiles of up to
// 256 columns; a mask on B only for tiles of up to 128 columns (shared memory) with 16-byte aligned
// mask rows and tile starts.
bool wgrad_ts_ok(const WgradArgs& a, const WgTcPlan& pl) {
    const int nbk = (pl.n_t + 31) / 32;
    if (nbk > 8 || a.M >= ((int64_t)1 << 31)) return false;
    if (a.a_dtype == SLICEGCN_BF16 && (a.lda % 8 || pl.a_col0 % 8 || pl.a_tile_cols % 8)) return false;   // 16-byte tensor copies
    if (a.b_mask) {   // (the mask tiles of a wide B fit the shared memory only next to the half-size raw slabs of a bf16 A)
        if (nbk > (a.a_dtype == SLICEGCN_BF16 ? 8 : 4) || (uintptr_t)a.b_mask % 16 || a.b_mask_ld % 16 || pl.b_col0 % 16 ||
            pl.b_cols_per_tile % 16)
            return false;
    }
    return true;
}

}  // namespace

TcImageCache* tc_image_cache_create() { return new TcImageCache(); }
void tc_image_cache_destroy(TcImageCache* c) { delete c; }

slicegcn_status_t tc_image_cache_begin(TcImageCache* c, void* region, int64_t bytes, const float* params, int64_t param_elems,
                                       cudaStream_t st) {
    if (!c) return SLICEGCN_OK;
    if (c->region != region || c->region_bytes != bytes) {   // another workspace: nothing recorded is valid
        c->entries.clear();
        c->used = 0;
        c->region = static_cast<unsigned char*>(region);
        c->region_bytes = bytes;
    }
    // keep what still points into this call's parameter buffer, convert all of it in one launch
    std::vector<TcImageCache::Entry> keep;
    for (auto& e : c->entries)
        if (e.job.B >= params && e.job.B < params + param_elems) keep.push_back(e);
    if (keep.size() != c->entries.size()) {   // a hole would waste space: start over
        c->entries.clear();
        c->used = 0;
        keep.clear();
    }
    if (!keep.empty()) {
        PrepBatch batch;
        batch.count = (int)keep.size();
        int blocks = 0;
        for (int i = 0; i < batch.count; ++i) {
            batch.job[i] = keep[i].job;
            batch.job[i].block0 = blocks;
            blocks += keep[i].job.n_slabs * 4 * keep[i].job.n_tiles * keep[i].job.groups;
        }
        tc_prep_batch_kernel<<<blocks, 128, 0, st>>>(batch);
        SGCN_LAUNCH_CHECK();
        count_launch();
        for (auto& e : c->entries) e.fresh = true;
    }
    t_image_cache = c;
    return SLICEGCN_OK;
}
void tc_image_cache_end() { t_image_cache = nullptr; }

bool tc_wgrad_masks_in_producer(const WgradArgs& a) {
    static const bool off = getenv("SLICEGCN_NO_TS") != nullptr || getenv("SLICEGCN_NO_WS") != nullptr;
    WgTcPlan pl;
    int gpt = 0;
    if (off || !a.b_mask || !a.fault || !wgrad_tc_plan(a, &pl, &gpt, 1, true)) return false;
    return wgrad_ts_ok(a, pl);
}

bool tc_gemm_masks_in_producer(const GemmArgs& a) {
    if (!a.a_mask || !a.fault || !a.b_image || a.K < 1 || a.A2) return false;
    int n_pad = tc_n_pad(a.N);
    if (a.N == 256 && a.groups * a.N <= kWsVecFloats) n_pad = 128;
    const int n_tiles = (a.N + n_pad - 1) / n_pad;
    return ts_gemm_ok(a, n_pad, n_tiles) && a.b_image_bytes >= tc_image_bytes(a.groups, a.K, a.N);
}

int64_t tc_image_bytes(int groups, int K, int N) {
    const int n_pad = tc_n_pad(N);
    const int n_tiles = (N + n_pad - 1) / n_pad;
    const int n_slabs = (K + 31) / 32;   // fp32 slabs (the bf16 path needs half as many)
    return (int64_t)groups * n_tiles * n_slabs * 2 * n_pad * 128;
}

int64_t tc_wgrad_scratch_bytes(const WgradArgs& a) {
    WgTcPlan pl;
    int gpt;
    if (!wgrad_tc_plan(a, &pl, &gpt)) return 0;
    return (int64_t)pl.n_chunks * pl.m_tiles * 128 * pl.n_t * (int64_t)sizeof(float);
}

// Tensor-core weight gradient (dW only; bias sums stay with the CUDA-core kernel).  Returns
// SLICEGCN_ERR_UNSUPPORTED when the shapes / alignments do not fit and nothing was launched.
slicegcn_status_t tc_wgrad_run(const WgradArgs& a, void* scratch, int64_t scratch_bytes, cudaStream_t st, bool* bias_done) {
    WgTcPlan pl;
    int gpt = 0;
    if (bias_done) *bias_done = false;
    if (!a.fault || !wgrad_tc_plan(a, &pl, &gpt)) return SLICEGCN_ERR_UNSUPPORTED;
    static const bool no_ws = getenv("SLICEGCN_NO_WS") != nullptr;
    if (!no_ws) {
        // warp-specialised variants: one CTA per SM
        WgTcPlan pw;
        int gw = 0;
        {   // first choice: the TMEM-operand kernel under the narrow plan
            WgTcPlan pn;
            int gn = 0;
            if (wgrad_tc_plan(a, &pn, &gn, 1, true)) {
            const int nbk = (pn.n_t + 31) / 32;
            static const bool no_ts = getenv("SLICEGCN_NO_TS") != nullptr;
            const int64_t need_ts = (int64_t)pn.n_chunks * pn.m_tiles * 128 * pn.n_t * (int64_t)sizeof(float);
            const int64_t need_cs = (int64_t)pn.n_chunks * pn.m_tiles * pn.n_t * (int64_t)sizeof(float);
            if (!no_ts && wgrad_ts_ok(a, pn) && scratch && scratch_bytes >= need_ts) {
                // the kernel that keeps A^T in TMEM (and sums B's columns on the way)
                const bool wide = nbk > 4;
                const int b_total = a.groups * a.N;
                CUtensorMap map_a, map_b;
                CUtensorMap map_bm;
                bool maps_ok = make_slab_map(&map_a, a.A, a.M, std::min<int64_t>(pn.a_col0 + pn.a_cols, a.lda), a.lda, pn.a_box, 32, false,
                                             a.a_dtype == SLICEGCN_BF16 ? 2 : 4) &&
                               make_slab_map(&map_b, a.B, a.M, std::min<int64_t>(pn.b_col0 + b_total, a.ldb), a.ldb, pn.n_t, 32, false);
                if (maps_ok && a.b_mask)
                    maps_ok = make_slab_map(&map_bm, a.b_mask, a.M, std::min<int64_t>(pn.b_col0 + b_total, a.b_mask_ld), a.b_mask_ld, pn.n_t, 32,
                                            false, 1);
                if (maps_ok && !a.b_mask) map_bm = map_b;
                if (maps_ok) {
                    const bool want_bias = (a.dbias || a.dbias2) && scratch_bytes >= need_ts + need_cs;
                    float* colsum = want_bias ? static_cast<float*>(scratch) + need_ts / sizeof(float) : nullptr;
                    const int slot_b = (a.a_dtype == SLICEGCN_BF16 ? 8192 : 16384) + ((32 * pn.n_t * 4 + 1023) & ~1023) +
                                       (a.b_mask ? ((32 * pn.n_t + 1023) & ~1023) : 0);
                    const int ts_smem = 2 * nbk * 8192 + (wide ? 2 : 4) * slot_b + 256 + 1024;
                    if (ts_smem > 227 * 1024) return SLICEGCN_ERR_UNSUPPORTED;   // (wgrad_ts_ok rules these shapes out)
                    static bool ts_configured = false;
                    if (!ts_configured) {
                        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ts_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
                        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ts_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
                        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ts_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
                        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ts_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024));
                        ts_configured = true;
                    }
                    dim3 tgrid(pn.n_chunks, pn.m_tiles);
                    float* sc = static_cast<float*>(scratch);
                    const bool abf = a.a_dtype == SLICEGCN_BF16;
                    if (wide && abf) tc_wgrad_ts_kernel<true, true><<<tgrid, kWtThreads, ts_smem, st>>>(a, pn, sc, colsum, a.fault, map_a, map_b, map_bm);
                    else if (wide) tc_wgrad_ts_kernel<true, false><<<tgrid, kWtThreads, ts_smem, st>>>(a, pn, sc, colsum, a.fault, map_a, map_b, map_bm);
                    else if (abf) tc_wgrad_ts_kernel<false, true><<<tgrid, kWtThreads, ts_smem, st>>>(a, pn, sc, colsum, a.fault, map_a, map_b, map_bm);
                    else tc_wgrad_ts_kernel<false, false><<<tgrid, kWtThreads, ts_smem, st>>>(a, pn, sc, colsum, a.fault, map_a, map_b, map_bm);
                    SGCN_LAUNCH_CHECK();
                    const int64_t total_w = (int64_t)a.groups * a.K * a.N;
                    const unsigned red_blocks = (unsigned)((total_w + 31) / 32) + (want_bias ? (unsigned)((b_total + 31) / 32) : 0u);
                    tc_wgrad_reduce_kernel<<<red_blocks, 256, 0, st>>>(static_cast<const float*>(scratch), pn, a.groups, a.K, a.N, gn, a.dW,
                                                                         colsum, a.dbias, a.dbias2, a.ldw);
                    SGCN_LAUNCH_CHECK();
                    if (want_bias && bias_done) *bias_done = true;
                    count_launch(2);
                    return SLICEGCN_OK;
                }
            }
            }
        }
        if (wgrad_tc_plan(a, &pw, &gw, 1)) {
            const int nbk = (pw.n_t + 31) / 32;
            const int stage_b = 32768 + 2 * 4 * nbk * 1024;
            int D = (220 * 1024) / stage_b;
            if (D > 3) D = 3;
            if (a.b_mask || a.a_dtype != SLICEGCN_F32) D = 0;   // the shared-memory-operand variant takes fp32 operands without a mask
            const int64_t need_w = (int64_t)pw.n_chunks * pw.m_tiles * 128 * pw.n_t * (int64_t)sizeof(float);
            if (D >= 2 && scratch && scratch_bytes >= need_w) {
                const int ws_smem = D * stage_b + 256 + 1024;
                static bool ws_configured = false;
                if (!ws_configured) {
                    SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ws_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
                    SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_ws_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 225 * 1024));
                    ws_configured = true;
                }
                dim3 wgrid(pw.n_chunks, pw.m_tiles);
                if (pw.n_t / 4 > 32)
                    tc_wgrad_ws_kernel<true><<<wgrid, kWsThreads, ws_smem, st>>>(a, pw, D, static_cast<float*>(scratch), a.fault);
                else
                    tc_wgrad_ws_kernel<false><<<wgrid, kWsThreads, ws_smem, st>>>(a, pw, D, static_cast<float*>(scratch), a.fault);
                SGCN_LAUNCH_CHECK();
                const int64_t total_w = (int64_t)a.groups * a.K * a.N;
                tc_wgrad_reduce_kernel<<<(unsigned)((total_w + 31) / 32), 256, 0, st>>>(static_cast<const float*>(scratch), pw,
                                                                                         a.groups, a.K, a.N, gw, a.dW, nullptr, nullptr, nullptr, a.ldw);
                SGCN_LAUNCH_CHECK();
                count_launch(2);
                return SLICEGCN_OK;
            }
        }
    }
    const int64_t need = (int64_t)pl.n_chunks * pl.m_tiles * 128 * pl.n_t * (int64_t)sizeof(float);
    if (!scratch || scratch_bytes < need) return SLICEGCN_ERR_UNSUPPORTED;
    const int smem_bytes = pl.stages * (2 * 16384 + 2 * pl.n_t * 128) + 64 + 1024;
    static bool configured = false;
    if (!configured) {
        const int mx = (2 * 16384 + 2 * 256 * 128) + 64 + 1024;
        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_kernel<float, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx));
        SGCN_CUDA(cudaFuncSetAttribute(tc_wgrad_kernel<__nv_bfloat16, 1>, cudaFuncAttributeMaxDynamicSharedMemorySize, mx));
        configured = true;
    }
    dim3 grid(pl.n_chunks, pl.m_tiles);
    if (a.a_dtype == SLICEGCN_BF16)
        tc_wgrad_kernel<__nv_bfloat16, 1><<<grid, kWgThreads, smem_bytes, st>>>(a, pl, static_cast<float*>(scratch), a.fault);
    else
        tc_wgrad_kernel<float, 1><<<grid, kWgThreads, smem_bytes, st>>>(a, pl, static_cast<float*>(scratch), a.fault);
    SGCN_LAUNCH_CHECK();
    const int64_t total = (int64_t)a.groups * a.K * a.N;
    tc_wgrad_reduce_kernel<<<(unsigned)((total + 31) / 32), 256, 0, st>>>(static_cast<const float*>(scratch), pl, a.groups,
                                                                           a.K, a.N, gpt, a.dW, nullptr, nullptr, nullptr, a.ldw);
    SGCN_LAUNCH_CHECK();
    count_launch(2);
    return SLICEGCN_OK;
}

// Tensor-core grouped GEMM; same contract as gemm_run().
slicegcn_status_t tc_gemm_run(const GemmArgs& a, cudaStream_t st) {
    if (a.M < 1 || a.groups < 1 || a.groups > SLICEGCN_MAX_SLICES || a.N < 1 || a.K < 1)
        SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "tc_gemm: bad shape");
    const bool abf = a.a_dtype == SLICEGCN_BF16, cbf = a.c_dtype == SLICEGCN_BF16;
    // operands that are bf16 in memory run the bf16 tensor path; fp32 operands the 3x tf32 path
    if (abf && cbf) return tc_gemm_launch<__nv_bfloat16, __nv_bfloat16, true>(a, a.b_image, a.b_image_bytes, a.fault, st);
    if (abf && !cbf) return tc_gemm_launch<__nv_bfloat16, float, true>(a, a.b_image, a.b_image_bytes, a.fault, st);
    if (!abf && cbf) return tc_gemm_launch<float, __nv_bfloat16, false>(a, a.b_image, a.b_image_bytes, a.fault, st);
    return tc_gemm_launch<float, float, false>(a, a.b_image, a.b_image_bytes, a.fault, st);
}

}  // namespace sgcn
