// Full-graph neighbour aggregation of one message-passing round (Eq. 1):
// GCN symmetric-normalised sum, GraphSAGE mean (+ self concat), and the fused
// GAT edge-score / segment-softmax / weighted-sum pass, over a CSR graph.
//
// The work is a gather-reduce bound by the memory system, not a dense
// contraction: neighbour rows are streamed with the widest aligned vector
// loads, several rows in flight per lane, sums kept in registers.  Work is
// handed out warp by warp from one counter (a persistent grid), so a power-law
// degree distribution does not leave SMs idle: rows of kHeavyDegree entries or
// more are cut into segments of kSegLen entries that are handed out first,
// each segment's partial sum goes to scratch, and a second kernel adds a row's
// segments in order.  Nothing depends on which warp ran what, so results are
// the same bits on every call.
#include "common.cuh"

namespace retexo {

constexpr int kHeavyDegree = 4096;     // rows at least this long are cut into segments
constexpr int kSegLen = 2048;          // entries per segment
constexpr int kAggThreads = 256;
constexpr int kAggWarps = kAggThreads / kWarp;
constexpr int kUnroll = 4;             // neighbour rows in flight per lane and column chunk

// Upper bound on the number of segments of a graph with n_edges entries.
static inline int64_t max_segments(int64_t n_edges) { return n_edges / kSegLen + n_edges / kHeavyDegree + 1; }

// ---------------------------------------------------------------- pre-pass
// coef[v]: GCN (deg+1)^-1/2, SAGE 1/deg (0 for isolated nodes).  Also lists
// the heavy rows and their segments (list order is arbitrary; no result
// depends on it).
__global__ void prep_rows_kernel(int64_t n, const int64_t* __restrict__ rowptr, int mode,
                                 float* __restrict__ coef, int32_t* __restrict__ heavy_list,
                                 int32_t* __restrict__ heavy_seg_base, int32_t* __restrict__ seg_slot,
                                 int32_t* __restrict__ counters /* [0] heavy rows, [1] segments, [2] work */) {
    int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (v >= n) return;
    int64_t deg = rowptr[v + 1] - rowptr[v];
    float c;
    if (mode == RETEXO_GCN) c = 1.0f / sqrtf((float)deg + 1.0f);
    else c = deg > 0 ? 1.0f / (float)deg : 0.0f;
    coef[v] = c;
    if (deg >= kHeavyDegree) {
        const int32_t slot = atomicAdd(counters + 0, 1);
        const int32_t nseg = (int32_t)((deg + kSegLen - 1) / kSegLen);
        const int32_t base = atomicAdd(counters + 1, nseg);
        heavy_list[slot] = (int32_t)v;
        heavy_seg_base[slot] = base;
        for (int32_t i = 0; i < nseg; ++i) seg_slot[base + i] = slot;
    }
}

// ---------------------------------------------------------------- vectors
template <int VEC> struct VecT;
template <> struct VecT<4> { using type = float4; };
template <> struct VecT<2> { using type = float2; };
template <> struct VecT<1> { using type = float; };

template <int VEC>
__device__ __forceinline__ void vec_zero(typename VecT<VEC>::type& a);
template <> __device__ __forceinline__ void vec_zero<4>(float4& a) { a = make_float4(0.f, 0.f, 0.f, 0.f); }
template <> __device__ __forceinline__ void vec_zero<2>(float2& a) { a = make_float2(0.f, 0.f); }
template <> __device__ __forceinline__ void vec_zero<1>(float& a) { a = 0.f; }

__device__ __forceinline__ void vec_fma(float4& a, float w, const float4& x) {
    a.x = fmaf(w, x.x, a.x); a.y = fmaf(w, x.y, a.y); a.z = fmaf(w, x.z, a.z); a.w = fmaf(w, x.w, a.w);
}
__device__ __forceinline__ void vec_fma(float2& a, float w, const float2& x) {
    a.x = fmaf(w, x.x, a.x); a.y = fmaf(w, x.y, a.y);
}
__device__ __forceinline__ void vec_fma(float& a, float w, const float& x) { a = fmaf(w, x, a); }
__device__ __forceinline__ void vec_add(float4& a, const float4& x) { a.x += x.x; a.y += x.y; a.z += x.z; a.w += x.w; }
__device__ __forceinline__ void vec_add(float2& a, const float2& x) { a.x += x.x; a.y += x.y; }
__device__ __forceinline__ void vec_add(float& a, const float& x) { a += x; }

__device__ __forceinline__ void vec_max(float4& a, const float4& x) {
    a.x = fmaxf(a.x, x.x); a.y = fmaxf(a.y, x.y); a.z = fmaxf(a.z, x.z); a.w = fmaxf(a.w, x.w);
}
__device__ __forceinline__ void vec_max(float2& a, const float2& x) { a.x = fmaxf(a.x, x.x); a.y = fmaxf(a.y, x.y); }
__device__ __forceinline__ void vec_max(float& a, const float& x) { a = fmaxf(a, x); }

// What a row's accumulator does with a neighbour row: plain sum (SAGE mean),
// sum weighted by coef[u] (GCN), or element-wise maximum (SAGE max-pooling).
constexpr int kOpSum = 0, kOpGcn = 1, kOpMax = 2;

template <int VEC, int OP>
__device__ __forceinline__ void vec_init(typename VecT<VEC>::type& a) {
    if constexpr (OP != kOpMax) vec_zero<VEC>(a);
    else if constexpr (VEC == 4) a = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    else if constexpr (VEC == 2) a = make_float2(-INFINITY, -INFINITY);
    else a = -INFINITY;
}

template <int VEC>
__device__ __forceinline__ float vec_get(const typename VecT<VEC>::type& a, int i);
template <> __device__ __forceinline__ float vec_get<4>(const float4& a, int i) {
    return i == 0 ? a.x : i == 1 ? a.y : i == 2 ? a.z : a.w;
}
template <> __device__ __forceinline__ float vec_get<2>(const float2& a, int i) { return i == 0 ? a.x : a.y; }
template <> __device__ __forceinline__ float vec_get<1>(const float& a, int) { return a; }

struct AggArgs {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* q;
    int64_t ldq;
    int32_t dim;
    const float* coef;
    float* out;             // may be null
    int64_t ldout;
    __nv_bfloat16* out16;   // may be null
    int64_t ldout16;
    int32_t concat_self;    // SAGE
    const int32_t* heavy_list;       // [heavy rows] node id
    const int32_t* heavy_seg_base;   // [heavy rows] first segment of the row
    const int32_t* seg_slot;         // [segments] index into heavy_list
    int32_t* counters;               // [0] heavy rows, [1] segments, [2] next work item
    float* seg_partial;              // [segments x round_up(dim, 4)] raw sums
    int64_t ld_partial;
    float hub_coef;                  // GCN, matrix larger than L2: rows of nodes with coef <= hub_coef (hubs) are
                                     // loaded "evict last", all others "evict first"; 0 = no hints
};

// L2 eviction priorities for the gathers of a matrix that does not fit the cache: a power-law graph
// reads its hubs' rows again and again, every other row a few times; left to itself the cache keeps
// neither.  The hints change nothing but which lines stay resident.
__device__ __forceinline__ uint64_t l2_policy_evict_last() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ uint64_t l2_policy_evict_first() {
    uint64_t p;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
    return p;
}
__device__ __forceinline__ float4 ldg_hinted(const float4* ptr, uint64_t policy) {
    float4 v;
    asm volatile("ld.global.nc.L2::cache_hint.v4.f32 {%0, %1, %2, %3}, [%4], %5;"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(ptr), "l"(policy));
    return v;
}

// Adds the neighbour rows of CSR entries [beg, end) into acc, in order, for the
// column vectors this lane owns in pass `pass`.  GCN weighs each row by coef[u].
template <int VEC, int CH, int OP>
__device__ __forceinline__ void accumulate_range(const AggArgs& a, int64_t beg, int64_t end, int lane,
                                                 int vec0, int nvec,
                                                 typename VecT<VEC>::type (&acc)[CH]) {
    using V = typename VecT<VEC>::type;
    const int64_t ldv = a.ldq / VEC;
    const V* __restrict__ qv = reinterpret_cast<const V*>(a.q);
    constexpr bool kCanHint = OP == kOpGcn && VEC == 4;
    [[maybe_unused]] uint64_t keep = 0, pass = 0;
    [[maybe_unused]] const bool hinting = kCanHint && a.hub_coef > 0.f;
    if constexpr (kCanHint) {
        if (hinting) { keep = l2_policy_evict_last(); pass = l2_policy_evict_first(); }
    }
    for (int64_t e0 = beg; e0 < end; e0 += kWarp) {
        const int cnt = (int)min((int64_t)kWarp, end - e0);
        int my_u = 0;
        float my_w = 0.f;
        if (lane < cnt) {
            my_u = __ldg(a.colidx + e0 + lane);
            if (OP == kOpGcn) my_w = __ldg(a.coef + my_u);
        }
        int j = 0;
        for (; j + kUnroll <= cnt; j += kUnroll) {
            V x[kUnroll][CH];
            float w[kUnroll];
#pragma unroll
            for (int t = 0; t < kUnroll; ++t) {
                const int u = __shfl_sync(0xffffffffu, my_u, j + t);
                if (OP == kOpGcn) w[t] = __shfl_sync(0xffffffffu, my_w, j + t);
                const V* row = qv + (int64_t)u * ldv;
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int vi = vec0 + c * kWarp + lane;
                    if (vi < nvec) {
                        if constexpr (kCanHint) {
                            if (hinting) x[t][c] = ldg_hinted(row + vi, w[t] <= a.hub_coef ? keep : pass);
                            else x[t][c] = __ldg(row + vi);
                        } else {
                            x[t][c] = __ldg(row + vi);
                        }
                    } else vec_zero<VEC>(x[t][c]);
                }
            }
#pragma unroll
            for (int t = 0; t < kUnroll; ++t)
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    if (OP == kOpGcn) vec_fma(acc[c], w[t], x[t][c]);
                    else if (OP == kOpMax) vec_max(acc[c], x[t][c]);
                    else vec_add(acc[c], x[t][c]);
                }
        }
        for (; j < cnt; ++j) {
            const int u = __shfl_sync(0xffffffffu, my_u, j);
            float w = 0.f;
            if (OP == kOpGcn) w = __shfl_sync(0xffffffffu, my_w, j);
            const V* row = qv + (int64_t)u * ldv;
#pragma unroll
            for (int c = 0; c < CH; ++c) {
                const int vi = vec0 + c * kWarp + lane;
                if (vi < nvec) {
                    V x = __ldg(row + vi);
                    if (OP == kOpGcn) vec_fma(acc[c], w, x);
                    else if (OP == kOpMax) vec_max(acc[c], x);
                    else vec_add(acc[c], x);
                }
            }
        }
    }
}

__device__ __forceinline__ void store_elem(const AggArgs& a, int64_t v, int col, float val) {
    if (a.out) a.out[v * a.ldout + col] = val;
    if (a.out16) a.out16[v * a.ldout16 + col] = f32_to_bf16(val);
}

// Finishes row v for the column vectors of this lane: GCN adds the self term
// and scales, SAGE divides by the degree and (optionally) copies the self row.
template <int VEC, int CH, int OP>
__device__ __forceinline__ void finish_row(const AggArgs& a, int64_t v, int lane, int vec0, int nvec,
                                           typename VecT<VEC>::type (&acc)[CH]) {
    using V = typename VecT<VEC>::type;
    const V* __restrict__ self = reinterpret_cast<const V*>(a.q) + v * (a.ldq / VEC);
    const float cv = a.coef[v];
    const int64_t deg = a.rowptr[v + 1] - a.rowptr[v];
#pragma unroll
    for (int c = 0; c < CH; ++c) {
        const int vi = vec0 + c * kWarp + lane;
        if (vi >= nvec) continue;
        const V s = self[vi];
#pragma unroll
        for (int i = 0; i < VEC; ++i) {
            const int col = vi * VEC + i;
            if (col >= a.dim) continue;
            const float sv = vec_get<VEC>(s, i);
            const float av = vec_get<VEC>(acc[c], i);
            if (OP == kOpGcn) {
                store_elem(a, v, col, cv * fmaf(cv, sv, av));
            } else {
                const float mean = deg <= 0 ? 0.0f : OP == kOpMax ? av : av / (float)deg;
                if (a.concat_self) {
                    store_elem(a, v, col, sv);
                    store_elem(a, v, a.dim + col, mean);
                } else {
                    store_elem(a, v, col, mean);
                }
            }
        }
    }
}

// Persistent kernel: each warp draws work items from one counter.  Items
// [0, n_seg) are segments of heavy rows (their raw sums go to scratch), items
// [n_seg, n_seg + n) are whole rows (heavy ones are skipped: their segments
// cover them).
template <int VEC, int CH, int OP>
__global__ void __launch_bounds__(kAggThreads) agg_rows_kernel(AggArgs a) {
    using V = typename VecT<VEC>::type;
    const int lane = threadIdx.x & 31;
    const int nvec = (a.dim + VEC - 1) / VEC;
    const int64_t n_seg = a.counters[1];
    const int64_t total = n_seg + a.n;
    for (;;) {
        int64_t item = 0;
        if (lane == 0) item = atomicAdd(reinterpret_cast<unsigned int*>(a.counters + 2), 1u);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item >= total) break;
        if (item < n_seg) {
            const int32_t slot = a.seg_slot[item];
            const int64_t v = a.heavy_list[slot];
            const int64_t i = item - a.heavy_seg_base[slot];
            const int64_t beg = a.rowptr[v] + i * kSegLen;
            const int64_t end = min(a.rowptr[v + 1], beg + kSegLen);
            for (int vec0 = 0; vec0 < nvec; vec0 += CH * kWarp) {
                V acc[CH];
#pragma unroll
                for (int c = 0; c < CH; ++c) vec_init<VEC, OP>(acc[c]);
                accumulate_range<VEC, CH, OP>(a, beg, end, lane, vec0, nvec, acc);
                float* dst = a.seg_partial + item * a.ld_partial;
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int vi = vec0 + c * kWarp + lane;
                    if (vi >= nvec) continue;
#pragma unroll
                    for (int k = 0; k < VEC; ++k) dst[vi * VEC + k] = vec_get<VEC>(acc[c], k);
                }
            }
        } else {
            const int64_t v = item - n_seg;
            const int64_t beg = a.rowptr[v], end = a.rowptr[v + 1];
            if (end - beg >= kHeavyDegree) continue;
            for (int vec0 = 0; vec0 < nvec; vec0 += CH * kWarp) {
                V acc[CH];
#pragma unroll
                for (int c = 0; c < CH; ++c) vec_init<VEC, OP>(acc[c]);
                accumulate_range<VEC, CH, OP>(a, beg, end, lane, vec0, nvec, acc);
                finish_row<VEC, CH, OP>(a, v, lane, vec0, nvec, acc);
            }
        }
    }
}

// One warp per heavy row: adds the row's segment sums in segment order and
// finishes the row.
template <int VEC, int CH, int OP>
__global__ void __launch_bounds__(kAggThreads) agg_combine_kernel(AggArgs a) {
    using V = typename VecT<VEC>::type;
    const int lane = threadIdx.x & 31;
    const int nvec = (a.dim + VEC - 1) / VEC;
    const int n_heavy = a.counters[0];
    for (int h = blockIdx.x * kAggWarps + (threadIdx.x >> 5); h < n_heavy; h += gridDim.x * kAggWarps) {
        const int64_t v = a.heavy_list[h];
        const int64_t deg = a.rowptr[v + 1] - a.rowptr[v];
        const int nseg = (int)((deg + kSegLen - 1) / kSegLen);
        const float* src = a.seg_partial + (int64_t)a.heavy_seg_base[h] * a.ld_partial;
        for (int vec0 = 0; vec0 < nvec; vec0 += CH * kWarp) {
            V acc[CH];
#pragma unroll
            for (int c = 0; c < CH; ++c) vec_init<VEC, OP>(acc[c]);
            for (int i = 0; i < nseg; ++i) {
#pragma unroll
                for (int c = 0; c < CH; ++c) {
                    const int vi = vec0 + c * kWarp + lane;
                    if (vi >= nvec) continue;
                    float t[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int k = 0; k < VEC; ++k) t[k] = src[(int64_t)i * a.ld_partial + vi * VEC + k];
                    V x;
                    if constexpr (VEC == 4) x = make_float4(t[0], t[1], t[2], t[3]);
                    else if constexpr (VEC == 2) x = make_float2(t[0], t[1]);
                    else x = t[0];
                    if (OP == kOpMax) vec_max(acc[c], x);
                    else vec_add(acc[c], x);
                }
            }
            finish_row<VEC, CH, OP>(a, v, lane, vec0, nvec, acc);
        }
    }
}

// ---------------------------------------------------------------- column slabs
// Variant for matrices that do not fit the L2 cache while a slab of their columns does.  The
// columns are cut into slabs of LPR float4 vectors; work items are ordered slab by slab, so that at
// any time the whole grid gathers from the same N x (LPR x 16 bytes) slab, which stays in L2: the
// neighbour rows then come from L2 instead of HBM, at the price of reading the index array once per
// slab (streamed with evict-first loads).  A warp takes 32 / LPR entries of a row at a time: lane
// group g = lane / LPR adds entries g, g + G, g + 2G, ... in CSR order, and the groups' sums are
// added in a fixed tree at the end, so results are still the same bits on every call.
#ifndef SLAB_U
#define SLAB_U 8
#define SLAB_TAIL_U 4
#define SLAB_BLOCKS 3
#define SLAB_MIN_MB 192
#endif
constexpr int kSlabUnroll = SLAB_U;                  // neighbour rows in flight per lane (full trips of 32 entries)
constexpr int kSlabTailUnroll = SLAB_TAIL_U;         // ... in the ragged last trip of a row
constexpr int kSlabBlocksPerSm = SLAB_BLOCKS;        // resident blocks the register budget is cut for
// Measured on B200 (126 MB of L2), 233 k rows: 256-byte gathers out of an L2-resident slab deliver
// 15-17 TB/s, while the plain variant runs at the HBM rate divided by (1 - L2 hit rate): 9 TB/s for a
// 561 MB matrix (30 % hits), 13 TB/s for 239 MB (50 %), and the L2 rate itself once the matrix fits.
constexpr size_t kSlabMinMatrixBytes = (size_t)SLAB_MIN_MB << 20;   // (1.5 x L2) smaller matrices are left to the cache as they are
#ifndef SLAB_MB
#define SLAB_MB 64
#endif
constexpr size_t kSlabBytes = (size_t)SLAB_MB << 20;             // a slab of all rows may take this much of L2

template <int LPR, int OP>
__global__ void __launch_bounds__(kAggThreads, kSlabBlocksPerSm) agg_slab_kernel(AggArgs a, int n_slabs) {
    constexpr int G = kWarp / LPR;                   // entries of a row taken per step
    constexpr int U = G * kSlabUnroll > kWarp ? kWarp / G : kSlabUnroll;              // steps in flight: at most one trip
    constexpr int UT = G * kSlabTailUnroll > kWarp ? kWarp / G : kSlabTailUnroll;
    const int lane = threadIdx.x & 31;
    const int g = lane / LPR, c = lane % LPR;
    const int nvec = (a.dim + 3) / 4;
    const int64_t n_seg = a.counters[1];
    const int64_t per_slab = n_seg + a.n;
    const int64_t total = per_slab * n_slabs;
    const int64_t ldv = a.ldq / 4;
    const float4* __restrict__ qv = reinterpret_cast<const float4*>(a.q);
    for (;;) {
        int64_t item = 0;
        if (lane == 0) item = atomicAdd(reinterpret_cast<unsigned long long*>(a.counters + 2), 1ull);
        item = __shfl_sync(0xffffffffu, item, 0);
        if (item >= total) break;
        const int slab = (int)(item / per_slab);
        const int64_t r = item % per_slab;
        int64_t v, beg, end;
        if (r < n_seg) {
            const int32_t slot = a.seg_slot[r];
            v = a.heavy_list[slot];
            beg = a.rowptr[v] + (r - a.heavy_seg_base[slot]) * kSegLen;
            end = min(a.rowptr[v + 1], beg + kSegLen);
        } else {
            v = r - n_seg;
            beg = a.rowptr[v]; end = a.rowptr[v + 1];
            if (end - beg >= kHeavyDegree) continue;
        }
        const int vi = slab * LPR + c;
        const bool active = vi < nvec;
        const float4* __restrict__ col = qv + (active ? vi : nvec - 1);
        float4 acc[1];
        vec_init<4, OP>(acc[0]);
        for (int64_t e0 = beg; e0 < end; e0 += kWarp) {
            const int cnt = (int)min((int64_t)kWarp, end - e0);
            int my_u = 0;
            float my_w = 0.f;
            if (lane < cnt) {
                my_u = __ldcs(a.colidx + e0 + lane);
                if (OP == kOpGcn) my_w = __ldg(a.coef + my_u);
            }
            if (cnt == kWarp) {
                // full trip: no predicates; a lane beyond the last column vector loads the last one and
                // its sum is dropped at the end
#pragma unroll 1
                for (int j = 0; j < kWarp; j += G * U) {
                    float4 x[U];
                    float w[U];
#pragma unroll
                    for (int t = 0; t < U; ++t) {
                        const int u = __shfl_sync(0xffffffffu, my_u, j + t * G + g);
                        if (OP == kOpGcn) w[t] = __shfl_sync(0xffffffffu, my_w, j + t * G + g);
                        x[t] = __ldg(col + (int64_t)u * ldv);
                    }
#pragma unroll
                    for (int t = 0; t < U; ++t) {
                        if (OP == kOpGcn) vec_fma(acc[0], w[t], x[t]);
                        else if (OP == kOpMax) vec_max(acc[0], x[t]);
                        else vec_add(acc[0], x[t]);
                    }
                }
                continue;
            }
            for (int j = 0; j < cnt; j += G * UT) {      // ragged last trip of the row
                float4 x[UT];
                float w[UT];
                bool on[UT];
#pragma unroll
                for (int t = 0; t < UT; ++t) {
                    const int idx = j + t * G + g;
                    const int u = __shfl_sync(0xffffffffu, my_u, idx & 31);
                    if (OP == kOpGcn) w[t] = __shfl_sync(0xffffffffu, my_w, idx & 31);
                    on[t] = active && idx < cnt;
                    if (on[t]) x[t] = __ldg(qv + (int64_t)u * ldv + vi);
                }
#pragma unroll
                for (int t = 0; t < UT; ++t) {
                    if (!on[t]) continue;
                    if (OP == kOpGcn) vec_fma(acc[0], w[t], x[t]);
                    else if (OP == kOpMax) vec_max(acc[0], x[t]);
                    else vec_add(acc[0], x[t]);
                }
            }
        }
        // the lane groups' sums, added in a fixed order (group 0 ends up with the total)
#pragma unroll
        for (int o = kWarp / 2; o >= LPR; o >>= 1) {
            float4 y;
            y.x = __shfl_xor_sync(0xffffffffu, acc[0].x, o); y.y = __shfl_xor_sync(0xffffffffu, acc[0].y, o);
            y.z = __shfl_xor_sync(0xffffffffu, acc[0].z, o); y.w = __shfl_xor_sync(0xffffffffu, acc[0].w, o);
            if (OP == kOpMax) vec_max(acc[0], y);
            else vec_add(acc[0], y);
        }
        const int nvec_slab = min(nvec, slab * LPR + LPR);       // lanes of the other groups fall outside
        if (r < n_seg) {
            if (g == 0 && active) {
                float* dst = a.seg_partial + r * a.ld_partial + vi * 4;
                dst[0] = acc[0].x; dst[1] = acc[0].y; dst[2] = acc[0].z; dst[3] = acc[0].w;
            }
        } else {
            finish_row<4, 1, OP>(a, v, lane, slab * LPR, nvec_slab, acc);
        }
    }
}

template <int LPR>
static int launch_slab(int op, const AggArgs& a, int n_sm, cudaStream_t st) {
    const int nvec = (a.dim + 3) / 4;
    const int n_slabs = (nvec + LPR - 1) / LPR;
    auto go = [&](auto kernel) {
        int per_sm = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kernel, kAggThreads, 0) != cudaSuccess || per_sm < 1) {
            (void)cudaGetLastError();
            per_sm = 1;
        }
        kernel<<<n_sm * per_sm, kAggThreads, 0, st>>>(a, n_slabs);
    };
    if (op == kOpGcn) go(agg_slab_kernel<LPR, kOpGcn>);
    else if (op == kOpMax) go(agg_slab_kernel<LPR, kOpMax>);
    else go(agg_slab_kernel<LPR, kOpSum>);
    // heavy rows: their segments' sums are added over the full width as in the plain variant
    if (op == kOpGcn) agg_combine_kernel<4, 1, kOpGcn><<<n_sm, kAggThreads, 0, st>>>(a);
    else if (op == kOpMax) agg_combine_kernel<4, 1, kOpMax><<<n_sm, kAggThreads, 0, st>>>(a);
    else agg_combine_kernel<4, 1, kOpSum><<<n_sm, kAggThreads, 0, st>>>(a);
    return launch_status();
}

// Lanes per neighbour row of the slab variant for an N x dim fp32 matrix, or 0 where the plain
// variant is the better choice (the matrix fits L2 as it is, or no slab of all rows would).
static int slab_lanes(int64_t n, int32_t dim) {
    if ((size_t)n * (size_t)dim * 4 < kSlabMinMatrixBytes) return 0;
    for (int lpr = 32; lpr >= 8; lpr >>= 1)      // (64-byte gathers out of slabs of 4 vectors measured far slower)
        if ((size_t)n * (size_t)lpr * 16 <= kSlabBytes) return lpr * 4 < dim ? lpr : 0;
    return 0;
}

template <int VEC, int CH, int OP>
static int launch_agg(const AggArgs& a, int n_sm, cudaStream_t st) {
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, agg_rows_kernel<VEC, CH, OP>, kAggThreads, 0) !=
            cudaSuccess || per_sm < 1) {
        (void)cudaGetLastError();
        per_sm = 1;
    }
    agg_rows_kernel<VEC, CH, OP><<<n_sm * per_sm, kAggThreads, 0, st>>>(a);
    agg_combine_kernel<VEC, CH, OP><<<n_sm, kAggThreads, 0, st>>>(a);
    return launch_status();
}

template <int VEC, int OP>
static int dispatch_ch(const AggArgs& a, int n_sm, cudaStream_t st) {
    const int nvec = (a.dim + VEC - 1) / VEC;
    const int need = (nvec + kWarp - 1) / kWarp;      // column chunks for one pass
    if (need <= 1) return launch_agg<VEC, 1, OP>(a, n_sm, st);
    if (need <= 2) return launch_agg<VEC, 2, OP>(a, n_sm, st);
    if (need <= 3) return launch_agg<VEC, 3, OP>(a, n_sm, st);
    if (need <= 4) return launch_agg<VEC, 4, OP>(a, n_sm, st);
    if (need <= 5) return launch_agg<VEC, 5, OP>(a, n_sm, st);
    return launch_agg<VEC, 6, OP>(a, n_sm, st);      // wider rows: several passes of 6 chunks
}

template <int VEC>
static int dispatch_op(int op, const AggArgs& a, int n_sm, cudaStream_t st) {
    if (op == kOpGcn) return dispatch_ch<VEC, kOpGcn>(a, n_sm, st);
    if (op == kOpMax) return dispatch_ch<VEC, kOpMax>(a, n_sm, st);
    return dispatch_ch<VEC, kOpSum>(a, n_sm, st);
}

// ---------------------------------------------------------------- GAT
constexpr int kGatMaxHeads = 8;

struct GatArgs {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* p;
    int64_t ldp;
    int32_t heads, head_dim, dim;
    const float* a_src;
    const float* a_dst;
    float slope;
    int32_t self_loop;
    float* s;               // [n x heads] scratch
    float* t;
    float* out;
    int64_t ldout;
    __nv_bfloat16* out16;
    int64_t ldout16;
    int32_t* hub_list;      // rows a whole block takes, listed by gat_scores_kernel (order arbitrary; no result depends on it)
    int32_t* hub_count;
};

constexpr int kGatHubEntries = 128;     // rows with at least this many entries are taken by a whole block

// s_u = <a_src, p_u>, t_u = <a_dst, p_u> per head; one warp per node.  The warp also lists its node
// if the node's row is long enough for a whole block.
__global__ void __launch_bounds__(kAggThreads) gat_scores_kernel(GatArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t u = blockIdx.x * (int64_t)kAggWarps + (threadIdx.x >> 5);
    if (u >= a.n) return;
    if (lane == 0 && a.rowptr[u + 1] - a.rowptr[u] + (a.self_loop ? 1 : 0) >= kGatHubEntries)
        a.hub_list[atomicAdd(a.hub_count, 1)] = (int32_t)u;
    const float* row = a.p + u * a.ldp;
    for (int h = 0; h < a.heads; ++h) {
        float ss = 0.f, tt = 0.f;
        for (int j = lane; j < a.head_dim; j += kWarp) {
            const float x = row[h * a.head_dim + j];
            ss = fmaf(a.a_src[h * a.head_dim + j], x, ss);
            tt = fmaf(a.a_dst[h * a.head_dim + j], x, tt);
        }
        ss = warp_sum(ss);
        tt = warp_sum(tt);
        if (lane == 0) {
            a.s[u * a.heads + h] = ss;
            a.t[u * a.heads + h] = tt;
        }
    }
}

// The running soft-max state and weighted sum of one warp over the entries [e0, e0 + 32) of row v, for
// e0 = e_first, e_first + e_step, ...  (entry `deg`, if any, is the self loop).  Entries are taken 32 at
// a time: lane j scores entry j for every head, the chunk maximum and the rescale of the running
// soft-max state are warp reductions (one exp per entry and head in total), then all lanes add the
// weighted neighbour rows for the columns they own.
template <int NC>
__device__ __forceinline__ void gat_accumulate(const GatArgs& a, int64_t v, int64_t beg, int64_t deg, int64_t total,
                                               int64_t e_first, int64_t e_step, int lane, int warp,
                                               float (*p_s)[kWarp][kGatMaxHeads], const float (&tv)[kGatMaxHeads],
                                               const int (&head_of)[NC], float (&m)[kGatMaxHeads],
                                               float (&l)[kGatMaxHeads], float (&acc)[NC]) {
    for (int64_t e0 = e_first; e0 < total; e0 += e_step) {
        const int cnt = (int)min((int64_t)kWarp, total - e0);
        int my_u = 0;
        float e[kGatMaxHeads];
        const bool valid = lane < cnt;
        if (valid) my_u = (e0 + lane < deg) ? __ldg(a.colidx + beg + e0 + lane) : (int)v;
#pragma unroll
        for (int h = 0; h < kGatMaxHeads; ++h) {
            e[h] = -INFINITY;
            if (valid && h < a.heads) {
                const float z = a.s[(int64_t)my_u * a.heads + h] + tv[h];
                e[h] = z > 0.f ? z : a.slope * z;
            }
        }
        float scale[kGatMaxHeads];
#pragma unroll
        for (int h = 0; h < kGatMaxHeads; ++h) {
            scale[h] = 1.f;
            if (h < a.heads) {
                const float mn = fmaxf(m[h], warp_max(e[h]));     // finite: cnt >= 1
                scale[h] = expf(m[h] - mn);                       // exp(-inf) = 0 on the first chunk
                const float pj = valid ? expf(e[h] - mn) : 0.f;
                l[h] = l[h] * scale[h] + warp_sum(pj);
                m[h] = mn;
                p_s[warp][lane][h] = pj;
            }
        }
        __syncwarp();
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            float sc = 1.f;
#pragma unroll
            for (int h = 0; h < kGatMaxHeads; ++h) if (h == head_of[c]) sc = scale[h];
            acc[c] *= sc;
        }
        // several neighbour rows in flight per lane (a hub's row is otherwise one dependent load after
        // another); the products are still added in entry order
        constexpr int U = NC <= 2 ? 8 : (NC <= 4 ? 4 : 2);
        int j = 0;
        for (; j + U <= cnt; j += U) {
            float x[U][NC];
#pragma unroll
            for (int t = 0; t < U; ++t) {
                const int u = __shfl_sync(0xffffffffu, my_u, j + t);
                const float* row = a.p + (int64_t)u * a.ldp;
#pragma unroll
                for (int c = 0; c < NC; ++c) {
                    const int col = c * kWarp + lane;
                    x[t][c] = col < a.dim ? __ldg(row + col) : 0.f;
                }
            }
#pragma unroll
            for (int t = 0; t < U; ++t)
#pragma unroll
                for (int c = 0; c < NC; ++c) acc[c] = fmaf(p_s[warp][j + t][head_of[c]], x[t][c], acc[c]);
        }
        for (; j < cnt; ++j) {
            const int u = __shfl_sync(0xffffffffu, my_u, j);
            const float* row = a.p + (int64_t)u * a.ldp;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int col = c * kWarp + lane;
                if (col < a.dim) acc[c] = fmaf(p_s[warp][j][head_of[c]], __ldg(row + col), acc[c]);
            }
        }
        __syncwarp();
    }
}

// Blocks [0, hub_blocks): one block per listed hub row at a time.  Warp w takes the trips w, w + 8, ...
// of the row with a soft-max state of its own; the eight states are then merged in warp order
//   M = max m_w,  L = sum l_w e^(m_w - M),  Z = sum acc_w e^(m_w - M) / L,
// so the result does not depend on scheduling (it differs from the one-warp order only in rounding).
// Blocks from hub_blocks on: one warp per destination v, rows of fewer than kGatHubEntries entries.
// The hub blocks come first in launch order, so the longest rows start ahead of the short ones.
template <int NC>
__global__ void __launch_bounds__(kAggThreads) gat_rows_kernel(GatArgs a, int hub_blocks) {
    __shared__ float p_s[kAggWarps][kWarp][kGatMaxHeads];
    __shared__ float sm_m[kAggWarps][kGatMaxHeads], sm_l[kAggWarps][kGatMaxHeads];
    __shared__ float sm_acc[kAggWarps][NC * kWarp];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const bool hub_block = (int)blockIdx.x < hub_blocks;
    const int n_hubs = hub_block ? *a.hub_count : 0;
    int hub = blockIdx.x;
    int64_t v = hub_block ? -1 : (int64_t)(blockIdx.x - hub_blocks) * kAggWarps + warp;
    if (!hub_block && v >= a.n) return;

    float m[kGatMaxHeads], l[kGatMaxHeads], tv[kGatMaxHeads];
    float acc[NC];
    int head_of[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int col = c * kWarp + lane;
        head_of[c] = col < a.dim ? col / a.head_dim : 0;
    }

    if (!hub_block) {
        const int64_t beg = a.rowptr[v];
        const int64_t deg = a.rowptr[v + 1] - beg;
        const int64_t total = deg + (a.self_loop ? 1 : 0);
        if (total >= kGatHubEntries) return;                 // a hub block takes this row
#pragma unroll
        for (int h = 0; h < kGatMaxHeads; ++h) {
            m[h] = -INFINITY;
            l[h] = 0.f;
            tv[h] = h < a.heads ? a.t[v * a.heads + h] : 0.f;
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[c] = 0.f;
        gat_accumulate<NC>(a, v, beg, deg, total, 0, kWarp, lane, warp, p_s, tv, head_of, m, l, acc);
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int col = c * kWarp + lane;
            if (col < a.dim) {
                float val = 0.f;
                if (total > 0) {
                    float lh = 1.f;
#pragma unroll
                    for (int h = 0; h < kGatMaxHeads; ++h) if (h == head_of[c]) lh = l[h];
                    val = acc[c] / lh;
                }
                if (a.out) a.out[v * a.ldout + col] = val;
                if (a.out16) a.out16[v * a.ldout16 + col] = f32_to_bf16(val);
            }
        }
        return;
    }

    for (; hub < n_hubs; hub += hub_blocks) {
        v = a.hub_list[hub];
        const int64_t beg = a.rowptr[v];
        const int64_t deg = a.rowptr[v + 1] - beg;
        const int64_t total = deg + (a.self_loop ? 1 : 0);
#pragma unroll
        for (int h = 0; h < kGatMaxHeads; ++h) {
            m[h] = -INFINITY;
            l[h] = 0.f;
            tv[h] = h < a.heads ? a.t[v * a.heads + h] : 0.f;
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) acc[c] = 0.f;
        gat_accumulate<NC>(a, v, beg, deg, total, (int64_t)warp * kWarp, (int64_t)kAggWarps * kWarp, lane, warp, p_s, tv,
                           head_of, m, l, acc);
        if (lane < kGatMaxHeads) {
            float mm = -INFINITY, ll = 0.f;
#pragma unroll
            for (int h = 0; h < kGatMaxHeads; ++h) if (h == lane) { mm = m[h]; ll = l[h]; }
            sm_m[warp][lane] = mm;
            sm_l[warp][lane] = ll;
        }
#pragma unroll
        for (int c = 0; c < NC; ++c) sm_acc[warp][c * kWarp + lane] = acc[c];
        __syncthreads();
        for (int col = threadIdx.x; col < a.dim; col += kAggThreads) {
            const int h = col / a.head_dim;
            float big = -INFINITY;
            for (int w = 0; w < kAggWarps; ++w) big = fmaxf(big, sm_m[w][h]);
            float den = 0.f, num = 0.f;
            for (int w = 0; w < kAggWarps; ++w) {
                const float f = sm_m[w][h] == -INFINITY ? 0.f : expf(sm_m[w][h] - big);     // (a warp without trips)
                den = fmaf(sm_l[w][h], f, den);
                num = fmaf(sm_acc[w][col], f, num);
            }
            const float val = num / den;
            if (a.out) a.out[v * a.ldout + col] = val;
            if (a.out16) a.out16[v * a.ldout16 + col] = f32_to_bf16(val);
        }
        __syncthreads();
    }
}

}  // namespace retexo

using namespace retexo;

extern "C" size_t retexo_aggregate_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t type,
                                                  int32_t dim, int32_t heads) {
    Sizer s;
    if (n_nodes < 0) return 0;
    if (type == RETEXO_GAT) {
        s.take<float>((size_t)n_nodes * (size_t)(heads > 0 ? heads : 1));
        s.take<float>((size_t)n_nodes * (size_t)(heads > 0 ? heads : 1));
        s.take<int32_t>((size_t)n_nodes);                                 // hub rows
        s.take<int32_t>(64);                                              // their count
    } else {
        s.take<float>((size_t)n_nodes);                                   // coef
        s.take<int32_t>((size_t)(n_edges / kHeavyDegree + 1));            // heavy rows
        s.take<int32_t>((size_t)(n_edges / kHeavyDegree + 1));            // their first segment
        s.take<int32_t>((size_t)max_segments(n_edges));                   // segment -> heavy row
        s.take<int32_t>(64);                                              // counters
        s.take<float>((size_t)max_segments(n_edges) * (size_t)((dim + 3) / 4 * 4));   // segment sums
    }
    return s.off + kAlign;
}

extern "C" int retexo_aggregate(const retexo_csr* g, int32_t type, const float* q, int64_t ldq, int32_t dim,
                                const retexo_gat_params* gat, float* out, int64_t ldout,
                                int32_t concat_self, void* out_bf16, int64_t ldout_bf16,
                                void* workspace, size_t workspace_bytes, void* stream) {
    if (!g || g->n_nodes < 0 || g->n_edges < 0 || g->n_nodes > INT32_MAX) return RETEXO_ERR_INVALID_ARG;
    if (type != RETEXO_GCN && type != RETEXO_SAGE_MEAN && type != RETEXO_GAT && type != RETEXO_SAGE_MAX)
        return RETEXO_ERR_INVALID_ARG;
    if (dim <= 0 || ldq < dim) return RETEXO_ERR_INVALID_ARG;
    if (g->n_nodes == 0) return RETEXO_OK;                      // nothing to aggregate
    if (!out && !out_bf16) return RETEXO_ERR_INVALID_ARG;
    if (!g->rowptr || !q || (g->n_edges > 0 && !g->colidx)) return RETEXO_ERR_INVALID_ARG;
    const bool sage = type == RETEXO_SAGE_MEAN || type == RETEXO_SAGE_MAX;
    const int64_t width = (sage && concat_self) ? 2 * (int64_t)dim : dim;
    if (out && ldout < width) return RETEXO_ERR_INVALID_ARG;
    if (out_bf16 && ldout_bf16 < width) return RETEXO_ERR_INVALID_ARG;
    if (dim > 4096) return RETEXO_ERR_UNSUPPORTED;
    if (type == RETEXO_GAT) {
        if (!gat || gat->heads <= 0 || gat->head_dim <= 0 || !gat->a_src || !gat->a_dst) return RETEXO_ERR_INVALID_ARG;
        if ((int64_t)gat->heads * gat->head_dim != dim) return RETEXO_ERR_INVALID_ARG;
        if (gat->heads > kGatMaxHeads || dim > 256) return RETEXO_ERR_UNSUPPORTED;
    }
    const size_t need = retexo_aggregate_workspace_size(g->n_nodes, g->n_edges, type, dim, gat ? gat->heads : 0);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_sm = sm_count();
    if (n_sm <= 0) return RETEXO_ERR_CUDA;
    Arena ws(workspace, workspace_bytes);
    const int64_t n = g->n_nodes;

    if (type == RETEXO_GAT) {
        GatArgs a;
        a.n = n; a.rowptr = g->rowptr; a.colidx = g->colidx; a.p = q; a.ldp = ldq;
        a.heads = gat->heads; a.head_dim = gat->head_dim; a.dim = dim;
        a.a_src = gat->a_src; a.a_dst = gat->a_dst; a.slope = gat->negative_slope;
        a.self_loop = gat->add_self_loop ? 1 : 0;
        a.s = ws.take<float>((size_t)n * gat->heads);
        a.t = ws.take<float>((size_t)n * gat->heads);
        a.hub_list = ws.take<int32_t>((size_t)n);
        a.hub_count = ws.take<int32_t>(64);
        RETEXO_CUDA_TRY(cudaMemsetAsync(a.hub_count, 0, sizeof(int32_t), st));
        a.out = out; a.ldout = ldout;
        a.out16 = static_cast<__nv_bfloat16*>(out_bf16); a.ldout16 = ldout_bf16;
        const unsigned blocks = (unsigned)((n + kAggWarps - 1) / kAggWarps);
        gat_scores_kernel<<<blocks, kAggThreads, 0, st>>>(a);
        const int nc = (dim + kWarp - 1) / kWarp;
        const int hub_blocks = 3 * n_sm;       // as many as are resident at once; those without a row leave at once
        const unsigned grid = blocks + (unsigned)hub_blocks;
        if (nc <= 1) gat_rows_kernel<1><<<grid, kAggThreads, 0, st>>>(a, hub_blocks);
        else if (nc <= 2) gat_rows_kernel<2><<<grid, kAggThreads, 0, st>>>(a, hub_blocks);
        else if (nc <= 4) gat_rows_kernel<4><<<grid, kAggThreads, 0, st>>>(a, hub_blocks);
        else gat_rows_kernel<8><<<grid, kAggThreads, 0, st>>>(a, hub_blocks);
        return launch_status();
    }

    AggArgs a;
    a.n = n; a.rowptr = g->rowptr; a.colidx = g->colidx; a.q = q; a.ldq = ldq; a.dim = dim;
    float* coef = ws.take<float>((size_t)n);
    const int64_t e = g->n_edges;
    int32_t* heavy_list = ws.take<int32_t>((size_t)(e / kHeavyDegree + 1));
    int32_t* heavy_seg_base = ws.take<int32_t>((size_t)(e / kHeavyDegree + 1));
    int32_t* seg_slot = ws.take<int32_t>((size_t)max_segments(e));
    int32_t* counters = ws.take<int32_t>(64);
    a.ld_partial = (dim + 3) / 4 * 4;
    a.seg_partial = ws.take<float>((size_t)max_segments(e) * (size_t)a.ld_partial);
    a.coef = coef; a.heavy_list = heavy_list; a.heavy_seg_base = heavy_seg_base; a.seg_slot = seg_slot;
    // hubs = nodes of at least four times the mean degree; hinted only where the matrix is larger than L2
    a.hub_coef = 0.f;
    if (type == RETEXO_GCN && (size_t)n * (size_t)dim * 4 >= kSlabMinMatrixBytes && n > 0)
        a.hub_coef = (float)(1.0 / sqrt(4.0 * (double)e / (double)n + 1.0));
    a.counters = counters;
    a.out = out; a.ldout = ldout;
    a.out16 = static_cast<__nv_bfloat16*>(out_bf16); a.ldout16 = ldout_bf16;
    a.concat_self = concat_self ? 1 : 0;
    RETEXO_CUDA_TRY(cudaMemsetAsync(counters, 0, 64 * sizeof(int32_t), st));
    prep_rows_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(n, g->rowptr, type, coef, heavy_list,
                                                                  heavy_seg_base, seg_slot, counters);

    const int op = type == RETEXO_GCN ? kOpGcn : type == RETEXO_SAGE_MAX ? kOpMax : kOpSum;
    const bool v4 = aligned_to(q, 16) && ldq % 4 == 0 && ldq >= (dim + 3) / 4 * 4;
    const bool v2 = aligned_to(q, 8) && ldq % 2 == 0 && ldq >= (dim + 1) / 2 * 2;
    if (v4) {
        const int lpr = slab_lanes(n, dim);
        if (lpr == 32) return launch_slab<32>(op, a, n_sm, st);
        if (lpr == 16) return launch_slab<16>(op, a, n_sm, st);
        if (lpr == 8) return launch_slab<8>(op, a, n_sm, st);
        return dispatch_op<4>(op, a, n_sm, st);
    }
    if (v2) return dispatch_op<2>(op, a, n_sm, st);
    return dispatch_op<1>(op, a, n_sm, st);
}
