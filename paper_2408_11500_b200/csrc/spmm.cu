// Normalised sparse aggregation  Y = A_hat X  (Eq. 1 / Eq. 6 neighbor sum; A_hat^T X in backward).
//
// Row-parallel CSR over row-aligned chunks of ~kChunk stored entries (common.cuh).  A group of L lanes streams one
// chunk; each lane keeps C 16-byte chunks of the output row in registers, so one 128-bit load per lane per chunk covers
// a neighbor's slice row.  No per-edge value array exists:  A_hat_ij = row_scale_i * col_scale_j.  Rows longer than
// kLongRow are cut into kSegment-entry segments, one warp each (same launch); a row of one segment is finished by that
// warp, the others leave partial rows that are summed in segment order -- deterministic, no floating-point atomics.
// Two gather loops share this structure:
//   - the staged kernel (rows of 512 bytes and more, a whole warp per chunk): column indices and the neighbor's scale
//     are read coalesced a batch at a time, parked in a per-warp shared-memory slot and read back as one broadcast
//     load per neighbor, row metadata handed out by shuffles; the warp that arrives last at a split row's counter
//     (an integer atomic) sums its partial rows, so there is no second launch;
//   - the direct kernel (rows of at most 256 bytes, 32/L chunks per warp): every lane group walks its chunk with plain
//     loads and no cooperation inside the warp; a small second launch sums the partial rows.
#include <vector>

#include "common.cuh"
#include "kernels.cuh"

namespace sgcn {
namespace {

template <typename T>
struct Vec;
template <>
struct Vec<float> {
    static constexpr int V = 4;
    static __device__ __forceinline__ void unpack(const uint4& r, float (&f)[4]) {
        f[0] = __uint_as_float(r.x);
        f[1] = __uint_as_float(r.y);
        f[2] = __uint_as_float(r.z);
        f[3] = __uint_as_float(r.w);
    }
    static __device__ __forceinline__ void store(float* p, const float (&f)[4]) {
        __stcs(reinterpret_cast<float4*>(p), make_float4(f[0], f[1], f[2], f[3]));   // streaming: keep X in L2
    }
};
template <>
struct Vec<__nv_bfloat16> {
    static constexpr int V = 8;
    static __device__ __forceinline__ void unpack(const uint4& r, float (&f)[8]) {
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            f[2 * i] = __uint_as_float(w[i] << 16);
            f[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
        uint4 r;
        uint32_t* w = reinterpret_cast<uint32_t*>(&r);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        __stcs(reinterpret_cast<uint4*>(p), r);
    }
};

__device__ __forceinline__ float to_f(float v) { return v; }
__device__ __forceinline__ float to_f(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T>
__device__ __forceinline__ T from_f(float v);
template <>
__device__ __forceinline__ float from_f<float>(float v) { return v; }
template <>
__device__ __forceinline__ __nv_bfloat16 from_f<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

struct SpmmParams {
    int64_t n;
    const int32_t* rowptr;
    const int32_t* colidx;
    const float* rs;   // row scale (1/sqrt(deg_i) for Eq. 1's normalisation)
    const float* cs;   // column scale (1/sqrt(deg_j))
    const void* X;
    int64_t ldx;
    void* Y;
    int64_t ldy;
    int32_t width;   // columns
    int32_t nch;     // 16-byte chunks per row = ceil(width / V)
    // long rows
    int32_t n_long, n_seg;
    const int32_t* long_rows;
    const int32_t* seg_ptr;
    const int32_t* seg_row;
    const int32_t* seg_order;   // processing order of the segments (by first column index)
    float* partial;  // [n_seg][nch*V]
    int32_t* seg_done;   // [n_long] segments of each long row that have left their partial row (zeroed before the launch)
    int32_t n_chunks;
    const int32_t* chunk_row;
    // epilogue (transform-first layers):  y = act(dinv_i*acc + bias) (+ previous y)
    const float* bias;
    uint8_t* mask;
    int64_t mask_ld;
    int32_t relu;
    int32_t accumulate;
};

template <typename TO, int V, bool EPI>
__device__ __forceinline__ void finish_chunk(const SpmmParams& p, int64_t row, int chunk, float di, float (&o)[V]) {
    TO* Y = static_cast<TO*>(p.Y) + row * p.ldy;
    const int col0 = chunk * V;
#pragma unroll
    for (int e = 0; e < V; ++e) o[e] *= di;
    if (EPI) {
#pragma unroll
        for (int e = 0; e < V; ++e) {
            const int col = col0 + e;
            if (col < p.width) {
                float x = o[e] + (p.bias ? __ldg(p.bias + col) : 0.f);
                if (p.relu) {
                    if (p.mask) p.mask[row * p.mask_ld + col] = x > 0.f ? 1 : 0;
                    x = fmaxf(x, 0.f);
                }
                if (p.accumulate) x += to_f(Y[col]);
                o[e] = x;
            }
        }
    }
    bool stored = false;
    if constexpr (V == Vec<TO>::V) {
        if (col0 + V <= p.width) {
            Vec<TO>::store(Y + col0, o);
            stored = true;
        }
    } else if constexpr (V == 8 && Vec<TO>::V == 4) {   // bf16 operand, fp32 result: two 16-byte stores
        if (col0 + V <= p.width) {
            const float lo[4] = {o[0], o[1], o[2], o[3]}, hi[4] = {o[4], o[5], o[6], o[7]};
            Vec<TO>::store(Y + col0, lo);
            Vec<TO>::store(Y + col0 + 4, hi);
            stored = true;
        }
    }
    if (!stored) {
#pragma unroll
        for (int e = 0; e < V; ++e)
            if (col0 + e < p.width) Y[col0 + e] = from_f<TO>(o[e]);
    }
}

// One lane group per row-aligned chunk of about kChunk stored entries (see common.cuh): a run of
// short rows whose entries are contiguous.  The group streams the chunk's entries a batch (L or 2 L
// entries) at a time; a row ends where the running entry index meets the row's end, at which point the
// accumulators are scaled, stored and cleared.  Short rows therefore share one stream of gathers (many
// loads in flight even for degree-1 rows) and every group does the same amount of work.  Row ends and
// 1/sqrt(deg) of a batch of consecutive rows are fetched by the L lanes at once and handed out by
// shuffles; the column indices of the next batch are requested before the current batch is gathered.
// Chunks that consist of one long row are left to the segment kernels.
constexpr int kRowsWarps = 1;   // warps per CTA of the row kernel: a finished warp frees its slot at once (measured best)
// Occupancy and neighbors gathered per round.  Measured on B200: for rows of 256 bytes and more what
// pays is resident warps (32 per SM, i.e. at most 64 registers) rather than loads per lane -- they run
// fastest with four 16-byte loads in flight per lane; the widest ones (three or four chunks per lane)
// keep eight loads per lane at 20 warps per SM.  (One-warp CTAs cap an SM at 32 warps; two-warp CTAs
// at 40-48 warps per SM need 40-48 registers, which this loop only reaches with spills: -5 % for
// 512-byte fp32 rows, +4..12 % for bf16 rows -- not adopted.  Five to eight loads per lane at 28-20
// warps per SM: 8-37 % slower.)
template <int L, int C>
constexpr bool kDenseWarps = C <= 2;
template <int L, int C>
constexpr int kGatherRound = kDenseWarps<L, C> ? (C == 2 ? 2 : 4) : ((8 / C) < 2 ? 2 : (8 / C));
template <int L, int C>
constexpr int kRowsBlocksPerSm = (kDenseWarps<L, C> ? 32 : 20) / kRowsWarps;
// Column indices a lane fetches per batch.  (The loop is written for any lane-group width L; only L = 32 is
// instantiated -- rows narrower than 512 bytes take the direct kernel -- so a batch is 32 entries, one per lane.)
template <int L>
constexpr int kIdxPerLane = L >= 32 ? 1 : 2;
template <int L>
constexpr int kBatch = kIdxPerLane<L> * L;
// shared-memory slots per warp: (column index, 1/sqrt(deg) bits) of every group's current batch; one
// slot of padding per group keeps the groups' broadcast reads on different banks
template <int L>
constexpr int kSlotStride = kBatch<L> + (L < 32 ? 1 : 0);
template <int L>
constexpr int kSlotsPerWarp = (32 / L) * kSlotStride<L>;

template <typename TI, typename TO, int L, int C, bool EPI>
__device__ __forceinline__ void spmm_rows_block(const SpmmParams& p, const int64_t vblock) {
    constexpr int V = Vec<TI>::V;
    constexpr int RPW = 32 / L;
    constexpr int NB = kIdxPerLane<L>;
    constexpr int BT = kBatch<L>;
    constexpr int U = kGatherRound<L, C>;   // neighbors gathered per round: U*C 16-byte loads per lane
    const int lane = threadIdx.x & 31;
    const int sub = lane / L, sl = lane % L;
    const int64_t warp = (vblock * (int64_t)blockDim.x + threadIdx.x) >> 5;
    const int64_t chunk = warp * RPW + sub;
    if (chunk >= p.n_chunks) return;
    const unsigned gmask = (L == 32) ? 0xffffffffu : (((1u << L) - 1u) << (sub * L));
    const int r0 = __ldg(p.chunk_row + chunk);
    const int r1 = __ldg(p.chunk_row + chunk + 1);
    if (r0 >= r1) return;
    int kk = __ldg(p.rowptr + r0);             // next entry to consume
    const int k1 = __ldg(p.rowptr + r1);       // end of the chunk's entries
    // row metadata (row end, 1/sqrt(deg)) of BT rows at a time: lane sl holds rows rbase + sl + i*L
    int rbase = r0;
    int rp_l[NB];
    float di_l[NB];
    auto load_meta = [&]() {
#pragma unroll
        for (int i = 0; i < NB; ++i) {
            const int r = rbase + sl + i * L;
            rp_l[i] = (r < r1) ? __ldg(p.rowptr + r + 1) : k1;
            di_l[i] = (r < r1) ? __ldg(p.rs + r) : 0.f;
        }
    };
    auto meta_end = [&](int idx) {   // idx is the same in every lane of the group
        int v = rp_l[0];
#pragma unroll
        for (int i = 1; i < NB; ++i) v = (idx / L == i) ? rp_l[i] : v;
        return __shfl_sync(gmask, v, idx % L, L);
    };
    auto meta_dinv = [&](int idx) {
        float v = di_l[0];
#pragma unroll
        for (int i = 1; i < NB; ++i) v = (idx / L == i) ? di_l[i] : v;
        return __shfl_sync(gmask, v, idx % L, L);
    };
    load_meta();
    int row = r0;
    int row_end = meta_end(0);
    if (row_end - kk > kLongRow) return;       // a long row sits alone in its chunk
    // per-lane column pointers (lanes past the last chunk re-read it; they never store)
    const uint32_t row16 = (uint32_t)((p.ldx * (int64_t)sizeof(TI)) >> 4);
    const uint4* xl[C];
#pragma unroll
    for (int c = 0; c < C; ++c) xl[c] = static_cast<const uint4*>(p.X) + min(sl + c * L, p.nch - 1);
    __shared__ int2 slots[kRowsWarps][kSlotsPerWarp<L>];
    int2* nb = &slots[threadIdx.x >> 5][sub * kSlotStride<L>];
    float acc[C][V];
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
    int jn[NB];
    float djn[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) jn[i] = (kk + sl + i * L < k1) ? __ldg(p.colidx + kk + sl + i * L) : 0;
#pragma unroll
    for (int i = 0; i < NB; ++i) djn[i] = (kk + sl + i * L < k1) ? __ldg(p.cs + jn[i]) : 0.f;

    auto close_row = [&]() {   // scale, store and clear the finished row; step to the next one
        const float di = meta_dinv(row - rbase);
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const int ch = sl + c * L;
            if (ch < p.nch) finish_chunk<TO, V, EPI>(p, row, ch, di, acc[c]);
#pragma unroll
            for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
        }
        ++row;
        if (row < r1) {
            if (row - rbase == BT) {
                rbase = row;
                load_meta();
            }
            row_end = meta_end(row - rbase);
        } else {
            row_end = -1;   // no further row: never matches an entry index
        }
    };

    for (;;) {
        while (kk == row_end) close_row();   // rows ending here, rows without entries included
        if (row >= r1) return;
        // one batch of up to BT entries starting at kk
        const int cnt = min(BT, k1 - kk);
        __syncwarp(gmask);
#pragma unroll
        for (int i = 0; i < NB; ++i) nb[sl + i * L] = make_int2(jn[i], __float_as_int(djn[i]));
        __syncwarp(gmask);
        const int nk = kk + cnt;
#pragma unroll
        for (int i = 0; i < NB; ++i)   // requested now, used by the next batch
            if (nk + sl + i * L < k1) jn[i] = __ldg(p.colidx + nk + sl + i * L);
        for (int t = 0; t < cnt;) {
            uint4 raw[U][C];
            int2 meta[U];
            if (L >= 16 && t + U <= cnt && row_end - kk >= U) {
                // fast round: U entries of the current row, no row end among them
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    meta[u] = nb[t + u];
#pragma unroll
                    for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)meta[u].x * row16);
                }
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const float dd = __int_as_float(meta[u].y);
#pragma unroll
                    for (int c = 0; c < C; ++c) {
                        float f[V];
                        Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                        for (int e = 0; e < V; ++e) acc[c][e] = fmaf(dd, f[e], acc[c][e]);
                    }
                }
                kk += U;
                t += U;
                continue;
            }
            // general round: up to U entries, rows may end in between
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (t + u < cnt) {
                    meta[u] = nb[t + u];
#pragma unroll
                    for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)meta[u].x * row16);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (t + u >= cnt) break;
                while (kk == row_end) close_row();   // a row ends inside the batch
                const float dd = __int_as_float(meta[u].y);
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float f[V];
                    Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] = fmaf(dd, f[e], acc[c][e]);
                }
                ++kk;
            }
            t += U;
        }
#pragma unroll
        for (int i = 0; i < NB; ++i)   // the indices have arrived by now
            if (nk + sl + i * L < k1) djn[i] = __ldg(p.cs + jn[i]);
    }
}

// One warp per segment of a long row; each of the 32/L lane groups takes a contiguous part of the
// segment and the groups are combined with a butterfly (fixed order).  A row that fits one segment is
// finished here; of the others the last warp to arrive sums the partial rows.
template <typename TI, typename TO, int L, int C, bool EPI>
__device__ __forceinline__ void spmm_segment_block(const SpmmParams& p, const int64_t vblock) {
    constexpr int V = Vec<TI>::V;
    constexpr int RPW = 32 / L;
    constexpr int GS = kSegment / RPW;                               // entries of a segment per lane group
    constexpr int BT = kBatch<L> < GS ? kBatch<L> : GS;              // entries per batch
    constexpr int NB = BT / L;
    static_assert(GS % L == 0 && BT % L == 0 && NB >= 1, "segment split");
    const int lane = threadIdx.x & 31;
    const int sub = lane / L, sl = lane % L;
    const int vseg = (int)((vblock * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (vseg >= p.n_seg) return;
    const int seg = __ldg(p.seg_order + vseg);
    const unsigned gmask = (L == 32) ? 0xffffffffu : (((1u << L) - 1u) << (sub * L));
    const int li = __ldg(p.seg_row + seg);
    const int row = __ldg(p.long_rows + li);
    const int start = __ldg(p.rowptr + row) + (seg - __ldg(p.seg_ptr + li)) * kSegment;
    const int end_seg = min(__ldg(p.rowptr + row + 1), start + kSegment);
    int base = start + sub * GS;                                      // this group's part: [base, end)
    const int end = min(end_seg, base + GS);
    constexpr int U = kGatherRound<L, C>;   // neighbors gathered per round
    __shared__ int2 slots[kRowsWarps][kSlotsPerWarp<L>];
    int2* nb = &slots[threadIdx.x >> 5][sub * kSlotStride<L>];
    const uint32_t row16 = (uint32_t)((p.ldx * (int64_t)sizeof(TI)) >> 4);
    const uint4* xl[C];
#pragma unroll
    for (int c = 0; c < C; ++c) xl[c] = static_cast<const uint4*>(p.X) + min(sl + c * L, p.nch - 1);
    float acc[C][V];
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
    int jn[NB];
    float djn[NB];
#pragma unroll
    for (int i = 0; i < NB; ++i) jn[i] = (base + sl + i * L < end) ? __ldg(p.colidx + base + sl + i * L) : 0;
#pragma unroll
    for (int i = 0; i < NB; ++i) djn[i] = (base + sl + i * L < end) ? __ldg(p.cs + jn[i]) : 0.f;
    for (; base < end; base += BT) {
        const int cnt = min(BT, end - base);
        __syncwarp(gmask);
#pragma unroll
        for (int i = 0; i < NB; ++i) nb[sl + i * L] = make_int2(jn[i], __float_as_int(djn[i]));
        __syncwarp(gmask);
        const int nbase = base + BT;
#pragma unroll
        for (int i = 0; i < NB; ++i)   // requested now, used by the next batch
            if (nbase + sl + i * L < end) jn[i] = __ldg(p.colidx + nbase + sl + i * L);
        int t = 0;
        for (; t + U <= cnt; t += U) {   // no row ends inside a segment: plain rounds
            uint4 raw[U][C];
            int2 meta[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                meta[u] = nb[t + u];
#pragma unroll
                for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)meta[u].x * row16);
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const float dd = __int_as_float(meta[u].y);
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float f[V];
                    Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] = fmaf(dd, f[e], acc[c][e]);
                }
            }
        }
        if (t < cnt) {                   // ragged end of the row's last segment
            uint4 raw[U][C];
            int2 meta[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (t + u < cnt) {
                    meta[u] = nb[t + u];
#pragma unroll
                    for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)meta[u].x * row16);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                if (t + u >= cnt) break;
                const float dd = __int_as_float(meta[u].y);
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float f[V];
                    Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] = fmaf(dd, f[e], acc[c][e]);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < NB; ++i)   // the indices have arrived by now
            if (nbase + sl + i * L < end) djn[i] = __ldg(p.cs + jn[i]);
    }
    __syncwarp();
#pragma unroll
    for (int off = L; off < 32; off <<= 1)
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[c][e] += __shfl_xor_sync(0xffffffffu, acc[c][e], off);
    const bool single = __ldg(p.seg_ptr + li + 1) - __ldg(p.seg_ptr + li) == 1;
    if (single) {
        if (sub == 0) {
            const float di = __ldg(p.rs + row);
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const int chunk = sl + c * L;
                if (chunk < p.nch) finish_chunk<TO, V, EPI>(p, row, chunk, di, acc[c]);
            }
        }
    } else {
        // several segments: leave the partial row; the warp that arrives last at the row's counter sums the row's
        // partial rows in segment order (whichever warp that is, the order of the additions is the same)
        const int pstride = p.nch * V;
        if (sub == 0) {
            float* out = p.partial + (int64_t)seg * pstride;
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const int chunk = sl + c * L;
                if (chunk < p.nch) {
#pragma unroll
                    for (int e = 0; e < V; e += 4)
                        *reinterpret_cast<float4*>(out + chunk * V + e) =
                            make_float4(acc[c][e], acc[c][e + 1], acc[c][e + 2], acc[c][e + 3]);
                }
            }
        }
        if (p.seg_done == nullptr) return;   // (no counters given: a second launch sums the partial rows)
        const int s0 = __ldg(p.seg_ptr + li), s1 = __ldg(p.seg_ptr + li + 1);
        int last = 0;
        __syncwarp();          // every lane's stores are ordered before lane 0's fence ...
        if (lane == 0) {
            __threadfence();   // ... which makes the whole partial row visible device-wide before the counter moves
            last = atomicAdd(p.seg_done + li, 1) == s1 - s0 - 1;
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
            // lane group g sums segments s0 + g, s0 + g + 32/L, ... in that order; the groups are then combined
            // with the same butterfly as above
            __threadfence();
#pragma unroll
            for (int c = 0; c < C; ++c)
#pragma unroll
                for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
#pragma unroll 4
            for (int s = s0 + sub; s < s1; s += RPW) {
                const float* src = p.partial + (int64_t)s * pstride;
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const int chunk = min(sl + c * L, p.nch - 1);
#pragma unroll
                    for (int e = 0; e < V; e += 4) {
                        const float4 v = __ldcg(reinterpret_cast<const float4*>(src + chunk * V + e));   // written by other SMs
                        acc[c][e] += v.x;
                        acc[c][e + 1] += v.y;
                        acc[c][e + 2] += v.z;
                        acc[c][e + 3] += v.w;
                    }
                }
            }
            __syncwarp();
#pragma unroll
            for (int off = L; off < 32; off <<= 1)
#pragma unroll
                for (int c = 0; c < C; ++c)
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] += __shfl_xor_sync(0xffffffffu, acc[c][e], off);
            if (sub == 0) {
                const float di = __ldg(p.rs + row);
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    const int chunk = sl + c * L;
                    if (chunk < p.nch) finish_chunk<TO, V, EPI>(p, row, chunk, di, acc[c]);
                }
            }
        }
    }
}

// The direct kernel: L lanes per row-aligned chunk (32/L chunks per warp), each lane C 16-byte chunks of the row, and NO
// cooperation between the lane groups of a warp -- every group walks its own chunk with plain loads (the lanes of a
// group read the same index and scale, which the load unit broadcasts), a few neighbors requested before they are
// accumulated, rows closed where the running entry index meets the row's end.  The staged kernel above parks indices
// in shared memory and hands row metadata around by shuffles; measured, its per-batch bookkeeping costs more than it
// saves wherever this kernel is used (see launch_direct).
template <int C>
constexpr int kDirectRound = C == 1 ? 4 : 2;   // neighbors requested per round: four 16-byte loads per lane in flight

// The 128-entry segments of the long rows: the 32/L lane groups of a warp take consecutive parts of the segment, each
// with plain loads as above, and are combined by a butterfly in a fixed order; a row of one segment is finished here,
// the others leave their partial row to spmm_long_finish_kernel.
template <typename TI, typename TO, int L, int C, bool EPI>
__device__ __forceinline__ void spmm_direct_segment(const SpmmParams& p, const int vseg) {
    constexpr int V = Vec<TI>::V;
    constexpr int U = kDirectRound<C>;
    constexpr int GS = kSegment / (32 / L);   // entries of a segment per lane group
    const int lane = threadIdx.x & 31;
    const int sub = lane / L, sl = lane % L;
    const int seg = __ldg(p.seg_order + vseg);
    const int li = __ldg(p.seg_row + seg);
    const int row = __ldg(p.long_rows + li);
    const int start = __ldg(p.rowptr + row) + (seg - __ldg(p.seg_ptr + li)) * kSegment;
    const int end_seg = min(__ldg(p.rowptr + row + 1), start + kSegment);
    const int base = start + sub * GS;
    const int end = min(end_seg, base + GS);
    const uint32_t row16 = (uint32_t)((p.ldx * (int64_t)sizeof(TI)) >> 4);
    const uint4* xl[C];
#pragma unroll
    for (int c = 0; c < C; ++c) xl[c] = static_cast<const uint4*>(p.X) + min(sl + c * L, p.nch - 1);
    float acc[C][V];
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
    for (int k = base; k < end; k += U) {
        const int cnt = min(U, end - k);
        int j[U];
        float d[U];
        uint4 raw[U][C];
#pragma unroll
        for (int u = 0; u < U; ++u) j[u] = u < cnt ? __ldg(p.colidx + k + u) : 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            d[u] = u < cnt ? __ldg(p.cs + j[u]) : 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)j[u] * row16);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (u < cnt) {   // (slots past the end loaded row 0: never accumulated, whatever it holds)
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float f[V];
                    Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] = fmaf(d[u], f[e], acc[c][e]);
                }
            }
        }
    }
    __syncwarp();
#pragma unroll
    for (int off = L; off < 32; off <<= 1)
#pragma unroll
        for (int c = 0; c < C; ++c)
#pragma unroll
            for (int e = 0; e < V; ++e) acc[c][e] += __shfl_xor_sync(0xffffffffu, acc[c][e], off);
    if (sub != 0) return;
    const bool single = __ldg(p.seg_ptr + li + 1) - __ldg(p.seg_ptr + li) == 1;
    const float di = single ? __ldg(p.rs + row) : 0.f;
#pragma unroll
    for (int c = 0; c < C; ++c) {
        const int ch = sl + c * L;
        if (ch >= p.nch) continue;
        if (single) {
            finish_chunk<TO, V, EPI>(p, row, ch, di, acc[c]);
        } else {
            float* out = p.partial + (int64_t)seg * (p.nch * V) + ch * V;
#pragma unroll
            for (int e = 0; e < V; e += 4)
                *reinterpret_cast<float4*>(out + e) = make_float4(acc[c][e], acc[c][e + 1], acc[c][e + 2], acc[c][e + 3]);
        }
    }
}

// One launch: the first seg_blocks CTAs (four warps, one segment each) take the long rows' segments, the others the chunks.
template <typename TI, typename TO, int L, int C, bool EPI>
__global__ void __launch_bounds__(128, 8) spmm_direct_kernel(const SpmmParams p, const int seg_blocks) {
    constexpr int V = Vec<TI>::V;
    constexpr int U = kDirectRound<C>;
    const int lane = threadIdx.x & 31;
    const int sub = lane / L, sl = lane % L;
    if ((int)blockIdx.x < seg_blocks) {
        const int vseg = (int)blockIdx.x * 4 + (threadIdx.x >> 5);
        if (vseg < p.n_seg) spmm_direct_segment<TI, TO, L, C, EPI>(p, vseg);
        return;
    }
    const int64_t chunk = ((((int64_t)blockIdx.x - seg_blocks) * (int64_t)blockDim.x + threadIdx.x) >> 5) * (32 / L) + sub;
    if (chunk >= p.n_chunks) return;
    const int r0 = __ldg(p.chunk_row + chunk);
    const int r1 = __ldg(p.chunk_row + chunk + 1);
    if (r0 >= r1) return;
    int k = __ldg(p.rowptr + r0);
    const int k1 = __ldg(p.rowptr + r1);
    int row = r0;
    int row_end = __ldg(p.rowptr + r0 + 1);
    if (row_end - k > kLongRow) return;   // a long row sits alone in its chunk: left to its segments
    const uint32_t row16 = (uint32_t)((p.ldx * (int64_t)sizeof(TI)) >> 4);
    const uint4* xl[C];
#pragma unroll
    for (int c = 0; c < C; ++c) xl[c] = static_cast<const uint4*>(p.X) + min(sl + c * L, p.nch - 1);
    float acc[C][V];
#pragma unroll
    for (int c = 0; c < C; ++c)
#pragma unroll
        for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
    auto close_row = [&]() {
        const float di = __ldg(p.rs + row);
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const int ch = sl + c * L;
            if (ch < p.nch) finish_chunk<TO, V, EPI>(p, row, ch, di, acc[c]);
#pragma unroll
            for (int e = 0; e < V; ++e) acc[c][e] = 0.f;
        }
        ++row;
        row_end = row < r1 ? __ldg(p.rowptr + row + 1) : -1;
    };
    while (k < k1) {
        const int cnt = min(U, k1 - k);
        int j[U];
        float d[U];
        uint4 raw[U][C];
#pragma unroll
        for (int u = 0; u < U; ++u) j[u] = u < cnt ? __ldg(p.colidx + k + u) : 0;
#pragma unroll
        for (int u = 0; u < U; ++u) {
            d[u] = u < cnt ? __ldg(p.cs + j[u]) : 0.f;
#pragma unroll
            for (int c = 0; c < C; ++c) raw[u][c] = __ldg(xl[c] + (uint64_t)(uint32_t)j[u] * row16);
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (u < cnt) {
                while (k == row_end) close_row();   // rows ending here, rows without entries included
#pragma unroll
                for (int c = 0; c < C; ++c) {
                    float f[V];
                    Vec<TI>::unpack(raw[u][c], f);
#pragma unroll
                    for (int e = 0; e < V; ++e) acc[c][e] = fmaf(d[u], f[e], acc[c][e]);
                }
                ++k;
            }
        }
    }
    while (row < r1 && k == row_end) close_row();
}

// One launch for both kinds of work: the first seg_blocks CTAs reduce the segments of the long rows
// (they are the heaviest items, so they start first), the others the row chunks.
template <typename TI, typename TO, int L, int C, bool EPI>
__global__ void __launch_bounds__(kRowsWarps * 32, kRowsBlocksPerSm<L, C>) spmm_rows_kernel(const SpmmParams p, const int seg_blocks) {
    if ((int)blockIdx.x < seg_blocks)
        spmm_segment_block<TI, TO, L, C, EPI>(p, blockIdx.x);
    else
        spmm_rows_block<TI, TO, L, C, EPI>(p, (int64_t)blockIdx.x - seg_blocks);
}

// After the direct kernel (see launch_direct): sums the partial rows of each long row in segment order, then scales / applies
// the epilogue.
// One warp per (long row, block of 32 columns): the hub rows with dozens of segments set the
// kernel's duration, so their columns are spread over many warps.
template <typename TO, bool EPI>
__global__ void __launch_bounds__(256) spmm_long_finish_kernel(const SpmmParams p, int pstride) {
    const int lane = threadIdx.x & 31;
    const int li = (int)((blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5);
    if (li >= p.n_long) return;
    const int col = blockIdx.y * 32 + lane;
    if (col >= p.width) return;
    const int64_t row = __ldg(p.long_rows + li);
    const int s0 = __ldg(p.seg_ptr + li), s1 = __ldg(p.seg_ptr + li + 1);
    if (s1 - s0 == 1) return;   // finished by its segment's warp
    const float di = __ldg(p.rs + row);
    TO* Y = static_cast<TO*>(p.Y) + row * p.ldy;
    {
        float a = 0.f;
        int s = s0;
        for (; s + 8 <= s1; s += 8) {   // eight loads in flight, summed in segment order
            float v[8];
#pragma unroll
            for (int q = 0; q < 8; ++q) v[q] = p.partial[(int64_t)(s + q) * pstride + col];
#pragma unroll
            for (int q = 0; q < 8; ++q) a += v[q];
        }
        for (; s < s1; ++s) a += p.partial[(int64_t)s * pstride + col];
        float x = a * di;
        if (EPI) {
            x += p.bias ? __ldg(p.bias + col) : 0.f;
            if (p.relu) {
                if (p.mask) p.mask[row * p.mask_ld + col] = x > 0.f ? 1 : 0;
                x = fmaxf(x, 0.f);
            }
            if (p.accumulate) x += to_f(Y[col]);
        }
        Y[col] = from_f<TO>(x);
    }
}

// Fallback for operands that do not allow 128-bit access (odd leading dimension / alignment):
// one warp per row, lanes over columns, scalar loads.  Handles long rows too (slow path).
template <typename TI, typename TO, bool EPI>
__global__ void __launch_bounds__(256) spmm_scalar_kernel(const SpmmParams p) {
    const int lane = threadIdx.x & 31;
    const int64_t row = (blockIdx.x * (int64_t)blockDim.x + threadIdx.x) >> 5;
    if (row >= p.n) return;
    const TI* X = static_cast<const TI*>(p.X);
    TO* Y = static_cast<TO*>(p.Y) + row * p.ldy;
    const int start = __ldg(p.rowptr + row), end = __ldg(p.rowptr + row + 1);
    const float di = __ldg(p.rs + row);
    for (int col = lane; col < p.width; col += 32) {
        float a = 0.f;
        for (int k = start; k < end; ++k) {
            const int j = __ldg(p.colidx + k);
            a = fmaf(__ldg(p.cs + j), to_f(X[(int64_t)j * p.ldx + col]), a);
        }
        float x = a * di;
        if (EPI) {
            x += p.bias ? __ldg(p.bias + col) : 0.f;
            if (p.relu) {
                if (p.mask) p.mask[row * p.mask_ld + col] = x > 0.f ? 1 : 0;
                x = fmaxf(x, 0.f);
            }
            if (p.accumulate) x += to_f(Y[col]);
        }
        Y[col] = from_f<TO>(x);
    }
}

// Rows of at most 256 bytes (up to sixteen 16-byte chunks): the direct kernel, then one small launch that sums the
// partial rows of the split long rows.  Measured against the staged kernel at the same widths: 9-27 % faster
// (co-purchase graph: 16-wide bf16 1.62 -> 1.35 ms, 16-wide fp32 2.21 -> 1.62 ms, 64-wide fp32 4.59 -> 4.01 ms), with
// bit-identical results.  At 512 bytes and more the staged kernel wins where the operand is near the L2's size
// (citation graph, 256 bf16: 167 us against 178 us) and loses 2-4 % where DRAM binds anyway; it keeps those widths.
template <typename TI, typename TO, int L>
slicegcn_status_t launch_direct(const SpmmParams& p, bool epi, cudaStream_t st) {
    constexpr int RPW = 32 / L;
    const int64_t warps = ((int64_t)p.n_chunks + RPW - 1) / RPW;
    SpmmParams q = p;
    q.seg_done = nullptr;   // split rows are summed by the second launch
    const int seg_blocks = (q.n_seg + 3) / 4;
    const unsigned blocks = (unsigned)((warps + 3) / 4) + (unsigned)seg_blocks;
    if (epi)
        spmm_direct_kernel<TI, TO, L, 1, true><<<blocks, 128, 0, st>>>(q, seg_blocks);
    else
        spmm_direct_kernel<TI, TO, L, 1, false><<<blocks, 128, 0, st>>>(q, seg_blocks);
    SGCN_LAUNCH_CHECK();
    count_launch();
    if (q.n_seg > 0) {
        const int pstride = q.nch * Vec<TI>::V;
        if (epi)
            spmm_long_finish_kernel<TO, true><<<dim3((q.n_long + 7) / 8, (q.width + 31) / 32), 256, 0, st>>>(q, pstride);
        else
            spmm_long_finish_kernel<TO, false><<<dim3((q.n_long + 7) / 8, (q.width + 31) / 32), 256, 0, st>>>(q, pstride);
        SGCN_LAUNCH_CHECK();
        count_launch();
    }
    return SLICEGCN_OK;
}

// Rows of 512 bytes and more: the staged kernel, a whole warp per chunk (L = 32), C chunks per lane.  Rows with several
// segments are finished by the last of their segment warps to arrive (its fence and counter update, ~1 us, are small
// next to a segment's gathers at these widths): no second launch.
template <typename TI, typename TO, int C>
slicegcn_status_t launch_staged(const SpmmParams& p, bool epi, cudaStream_t st) {
    const int64_t blocks = ((int64_t)p.n_chunks + kRowsWarps - 1) / kRowsWarps;
    const int seg_blocks = (p.n_seg + kRowsWarps - 1) / kRowsWarps;
    if (p.n_seg > 0) SGCN_CUDA(cudaMemsetAsync(p.seg_done, 0, sizeof(int32_t) * (size_t)p.n_long, st));
    if (epi)
        spmm_rows_kernel<TI, TO, 32, C, true><<<(unsigned)(blocks + seg_blocks), kRowsWarps * 32, 0, st>>>(p, seg_blocks);
    else
        spmm_rows_kernel<TI, TO, 32, C, false><<<(unsigned)(blocks + seg_blocks), kRowsWarps * 32, 0, st>>>(p, seg_blocks);
    SGCN_LAUNCH_CHECK();
    count_launch();
    return SLICEGCN_OK;
}

template <typename TI, typename TO>
slicegcn_status_t launch_vec(const SpmmParams& p, bool epi, int* fault, cudaStream_t st) {
    const int nch = p.nch;
    (void)fault;
    if (nch <= 2) return launch_direct<TI, TO, 2>(p, epi, st);
    if (nch <= 4) return launch_direct<TI, TO, 4>(p, epi, st);
    if (nch <= 8) return launch_direct<TI, TO, 8>(p, epi, st);
    if (nch <= 16) return launch_direct<TI, TO, 16>(p, epi, st);
    if (nch <= 32) return launch_staged<TI, TO, 1>(p, epi, st);
    if (nch <= 64) return launch_staged<TI, TO, 2>(p, epi, st);
    if (nch <= 96) return launch_staged<TI, TO, 3>(p, epi, st);
    return launch_staged<TI, TO, 4>(p, epi, st);
}

template <typename TI, typename TO>
slicegcn_status_t launch_typed(SpmmParams p, bool vec_ok, bool epi, int* fault, cudaStream_t st) {
    constexpr int V = Vec<TI>::V;
    if (!vec_ok) {
        const int64_t blocks = (p.n + 7) / 8;
        if (epi)
            spmm_scalar_kernel<TI, TO, true><<<(unsigned)blocks, 256, 0, st>>>(p);
        else
            spmm_scalar_kernel<TI, TO, false><<<(unsigned)blocks, 256, 0, st>>>(p);
        SGCN_LAUNCH_CHECK();
        count_launch();
        return SLICEGCN_OK;
    }
    // column blocks of at most 128 chunks (32 lanes x 4 chunks)
    const int total = p.width;
    const int block_cols = 128 * V;
    const TI* X = static_cast<const TI*>(p.X);
    TO* Y = static_cast<TO*>(p.Y);
    for (int c0 = 0; c0 < total; c0 += block_cols) {
        SpmmParams q = p;
        q.width = min(block_cols, total - c0);
        q.nch = (q.width + V - 1) / V;
        q.X = X + c0;
        q.Y = Y + c0;
        if (q.bias) q.bias += c0;
        if (q.mask) q.mask += c0;
        SGCN_TRY((launch_vec<TI, TO>(q, epi, fault, st)));
    }
    return SLICEGCN_OK;
}

}  // namespace

// ---- instrumentation ---------------------------------------------------------------------------
namespace {
struct Profiler {
    bool on = false;
    std::vector<cudaEvent_t> ev;   // pairs
    size_t used = 0;
    int64_t calls = 0;
    double bytes = 0.0;
    int64_t seen = 0;              // SpMM calls since begin
    int stride = 1;                // every stride-th call is bracketed by events
} g_prof;
}  // namespace

static int64_t partial_rows_bytes(const slicegcn_graph* g, int width) {
    // enough for either dtype: chunks of 8 elements, at most 128 chunks per column block
    int64_t w = width < 1024 ? width : 1024;
    int64_t padded = (w + 7) / 8 * 8;
    return (int64_t)g->max_segments() * padded * (int64_t)sizeof(float);
}

int64_t spmm_partial_bytes(const slicegcn_graph* g, int width) {
    // partial rows of the segments, then one counter per long row
    if (g->max_segments() == 0) return 0;
    const int64_t n_long = g->n_long[0] > g->n_long[1] ? g->n_long[0] : g->n_long[1];
    return partial_rows_bytes(g, width) + (n_long * (int64_t)sizeof(int32_t) + 15) / 16 * 16;
}

slicegcn_status_t spmm_run(const slicegcn_graph* g, bool transpose, int in_dtype, int out_dtype, const void* X,
                           int64_t ldx, void* Y, int64_t ldy, int width, const SpmmEpilogue* epi, void* ws,
                           int64_t ws_bytes, cudaStream_t st, bool instrument) {
    if (!g || !X || !Y) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm: NULL argument");
    if (width < 1 || ldx < width || ldy < width) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm: bad width / leading dimension");
    if (in_dtype != SLICEGCN_F32 && in_dtype != SLICEGCN_BF16) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm: bad dtype");
    if (out_dtype != SLICEGCN_F32 && out_dtype != SLICEGCN_BF16) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm: bad dtype");
    if (in_dtype == SLICEGCN_F32 && out_dtype == SLICEGCN_BF16)
        SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED, "spmm: an fp32 operand with a bf16 result is not supported");
    const CsrView v = g->view(transpose);
    SpmmParams p{};
    p.n = g->n;
    p.rowptr = v.rowptr;
    p.colidx = v.colidx;
    p.rs = v.row_scale;
    p.cs = v.col_scale;
    p.X = X;
    p.ldx = ldx;
    p.Y = Y;
    p.ldy = ldy;
    p.width = width;
    const int V = in_dtype == SLICEGCN_F32 ? 4 : 8;
    const int64_t esz = in_dtype == SLICEGCN_F32 ? 4 : 2;
    const int64_t osz = out_dtype == SLICEGCN_F32 ? 4 : 2;
    p.nch = (width + V - 1) / V;
    const bool vec_ok = ((uintptr_t)X % 16 == 0) && ((uintptr_t)Y % 16 == 0) && (ldx * esz) % 16 == 0 &&
                        (ldy * osz) % 16 == 0 && (int64_t)p.nch * V <= ldx;
    p.n_chunks = v.n_chunks;
    p.chunk_row = v.chunk_row;
    if (vec_ok) {
        p.n_long = v.n_long;
        p.n_seg = v.n_seg;
        p.long_rows = v.long_rows;
        p.seg_ptr = v.seg_ptr;
        p.seg_row = v.seg_row;
        p.seg_order = v.seg_order;
        p.partial = static_cast<float*>(ws);
        p.seg_done = ws ? reinterpret_cast<int32_t*>(static_cast<unsigned char*>(ws) + partial_rows_bytes(g, width)) : nullptr;
        if (v.n_seg > 0 && (!ws || ws_bytes < spmm_partial_bytes(g, width)))
            SGCN_FAIL(SLICEGCN_ERR_ALLOC, "spmm: workspace too small (%lld < %lld bytes)", (long long)ws_bytes,
                      (long long)spmm_partial_bytes(g, width));
    }
    cudaEvent_t ev_stop = nullptr;
    if (g_prof.on && instrument && (g_prof.seen++ % g_prof.stride) == 0) {
        if (g_prof.used + 2 > g_prof.ev.size()) {
            for (int i = 0; i < 2; ++i) {
                cudaEvent_t e;
                SGCN_CUDA(cudaEventCreate(&e));
                g_prof.ev.push_back(e);
            }
        }
        SGCN_CUDA(cudaEventRecord(g_prof.ev[g_prof.used], st));
        ev_stop = g_prof.ev[g_prof.used + 1];
        g_prof.used += 2;
        g_prof.calls += 1;
        g_prof.bytes += 4.0 * (double)g->nnz + 4.0 * (double)(g->n + 1) + 4.0 * (double)g->n +
                        (double)g->n * (double)width * (double)(esz + osz);
    }
    bool has_epi = false;
    if (epi) {
        p.bias = epi->bias;
        p.mask = epi->mask;
        p.mask_ld = epi->mask_ld;
        p.relu = epi->relu;
        p.accumulate = epi->accumulate;
        has_epi = true;
    }
    slicegcn_status_t rc = in_dtype == SLICEGCN_F32
                               ? launch_typed<float, float>(p, vec_ok, has_epi, g->fault, st)
                               : out_dtype == SLICEGCN_BF16
                                     ? launch_typed<__nv_bfloat16, __nv_bfloat16>(p, vec_ok, has_epi, g->fault, st)
                                     : launch_typed<__nv_bfloat16, float>(p, vec_ok, has_epi, g->fault, st);
    if (ev_stop) SGCN_CUDA(cudaEventRecord(ev_stop, st));
    return rc;
}

// ---- fixed scratch for callers that cannot allocate ------------------------------------------
// Lives in the library image: every GPU that loads the library holds these bytes until the process
// exits.  In host code the array's name is only a stand-in for the symbol, never a device address;
// the address a kernel may use comes from cudaGetSymbolAddress, once per device.
constexpr int64_t kStaticScratchBytes = 8ll << 20;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];
static void* g_static_scratch_ptr[64] = {nullptr};   // per device ordinal, filled on first use

static slicegcn_status_t static_scratch_for_current_device(void** out) {
    int dev = -1;
    SGCN_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED, "device ordinal %d outside the supported range", dev);
    if (!g_static_scratch_ptr[dev]) {
        void* p = nullptr;
        SGCN_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        g_static_scratch_ptr[dev] = p;
    }
    *out = g_static_scratch_ptr[dev];
    return SLICEGCN_OK;
}

}  // namespace sgcn

extern "C" {

slicegcn_status_t slicegcn_spmm_static_scratch(const slicegcn_graph* g, int32_t transpose, int32_t in_dtype,
                                               int32_t out_dtype, const void* X, int64_t ldx, void* Y, int64_t ldy,
                                               int32_t width, void* stream) {
    using namespace sgcn;
    if (!g || width < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm_static_scratch: bad argument");
    const int64_t need = spmm_partial_bytes(g, width);
    if (need > kStaticScratchBytes)
        SGCN_FAIL(SLICEGCN_ERR_UNSUPPORTED,
                  "spmm_static_scratch: this graph and width need %lld bytes of scratch, the built-in buffer holds %lld; "
                  "use slicegcn_spmm with a caller-provided workspace",
                  (long long)need, (long long)kStaticScratchBytes);
    void* scratch = nullptr;
    SGCN_TRY(static_scratch_for_current_device(&scratch));
    // nothing in the buffer has to start at zero: every partial row a call reads was written by that call
    return spmm_run(g, transpose != 0, in_dtype, out_dtype, X, ldx, Y, ldy, width, nullptr, scratch, kStaticScratchBytes,
                    (cudaStream_t)stream, /*instrument=*/false);
}

slicegcn_status_t slicegcn_profile_begin_sampled(int32_t stride) {
    using namespace sgcn;
    if (stride < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "profile_begin_sampled: stride < 1");
    g_prof.stride = stride;
    g_prof.seen = 0;
    g_prof.on = true;
    g_prof.used = 0;
    g_prof.calls = 0;
    g_prof.bytes = 0.0;
    reset_launches();
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_profile_begin(void) { return slicegcn_profile_begin_sampled(1); }

slicegcn_status_t slicegcn_profile_end(double* spmm_ms, int64_t* spmm_calls, double* spmm_bytes,
                                       int64_t* kernel_launches) {
    using namespace sgcn;
    g_prof.on = false;
    SGCN_CUDA(cudaDeviceSynchronize());
    double ms = 0.0;
    for (size_t i = 0; i + 1 < g_prof.used; i += 2) {
        float t = 0.f;
        SGCN_CUDA(cudaEventElapsedTime(&t, g_prof.ev[i], g_prof.ev[i + 1]));
        ms += t;
    }
    if (spmm_ms) *spmm_ms = ms;
    if (spmm_calls) *spmm_calls = g_prof.calls;
    if (spmm_bytes) *spmm_bytes = g_prof.bytes;
    if (kernel_launches) *kernel_launches = launches();
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_spmm_workspace_bytes(const slicegcn_graph* g, int32_t width, int64_t* bytes) {
    if (!g || !bytes || width < 1) SGCN_FAIL(SLICEGCN_ERR_INVALID_ARG, "spmm_workspace_bytes: bad argument");
    *bytes = sgcn::spmm_partial_bytes(g, width);
    return SLICEGCN_OK;
}

slicegcn_status_t slicegcn_spmm(const slicegcn_graph* g, int32_t transpose, int32_t in_dtype, int32_t out_dtype,
                                const void* X, int64_t ldx, void* Y, int64_t ldy, int32_t width, void* workspace,
                                int64_t workspace_bytes, void* stream) {
    return sgcn::spmm_run(g, transpose != 0, in_dtype, out_dtype, X, ldx, Y, ldy, width, nullptr, workspace,
                          workspace_bytes, (cudaStream_t)stream);
}

}  // extern "C"
