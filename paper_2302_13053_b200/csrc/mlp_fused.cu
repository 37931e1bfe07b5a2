// The row-local middle of one training iteration of the per-node model (Section 3.1: f_theta = Linear +
// ReLU, temporary classifier C_theta = Linear) in one kernel on sm_100a.  For every tile of 128 batch rows:
//   logits = Hd W2 + b2                     tcgen05.mma, Hd tile and W2 resident in shared memory
//   loss_i = CE(softmax(logits_i), y_i),  dL = (softmax - onehot) / n     in registers, two threads per row
//   dHd    = (dL W2^T) .* [Hd > 0]          a second tcgen05.mma whose A operand is the dL tile just written
//                                           to shared memory; the gate is one bit per hidden unit, written by
//                                           the forward product next to Hd
// Hd is read from global memory once, the logits never leave the SM, and dL and dHd go out row-major (the
// weight-gradient products read them as they lie).  One copy of W2^T in shared memory serves both products:
// K-major (reduction over the hidden units) for the logits, MN-major (reduction over the classes) for dHd.
//
// Roles: warp 0 loads (TMA), warp 1 issues the MMAs and owns tensor memory, warps 2-9 turn logits into loss
// and dL (two threads per row), warps 10-17 gate dHd and send it out.  An Hd tile is held only from its load to
// the end of the logits product (64 KB each, two of them), the logits are double-buffered in tensor memory, and
// the gate role stages its output in blocks of its own, so the three roles work on different tiles at once.
// Every wait is bounded: one that runs out sets *status and the block tears down in order.
#include <string.h>

#include "gemm_tc.h"
#include "tc_common.cuh"

namespace retexo {

constexpr int kHbThreads = 576;
constexpr int kHbLossWarp0 = 2, kHbLossWarps = 8, kHbGateWarp0 = 10, kHbGateWarps = 8;
constexpr uint32_t kHbPanelBytes = 128 * 128;       // [128 rows x 64 bf16], 128-byte swizzle
constexpr uint32_t kHbW2PanelBytes = 64 * 128;      // [64 classes x 64 hidden units]
constexpr uint32_t kHbSlabBytes = 32 * 128;         // one warp's 32 rows of a panel
constexpr uint32_t kHbLogitCols = 64, kHbGradCol0 = 256;

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

struct HbArgs {
    int64_t n_all, n_train;
    int32_t H, O, np;                  // np = panels of 64 hidden units
    const float* b2;
    const int32_t* y; const int32_t* y_eval;
    float inv_rows, gate_scale;
    const uint32_t* gate_bits; int64_t ld_bits;      // bit j of word [row][j / 32]: hidden unit j of the row is positive
    float* loss_partial;               // [4 x tiles]: one per tile and warp of the loss role
    unsigned long long* correct;
    int32_t* status;
};

enum HbBarrier { HB_W2_FULL = 0, HB_HD_FULL = 1, HB_HD_EMPTY = 3, HB_D1_FULL = 5, HB_D1_EMPTY = 7, HB_DL_FULL = 9,
                 HB_DL_EMPTY = 11, HB_D2_FULL = 13, HB_D2_EMPTY = 14, HB_N_BARRIERS = 15 };

__global__ void __launch_bounds__(kHbThreads, 1)
head_backward_kernel(const __grid_constant__ CUtensorMap map_hd, const __grid_constant__ CUtensorMap map_w2,
                     const __grid_constant__ CUtensorMap map_dl, const __grid_constant__ CUtensorMap map_dhd, HbArgs g) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* base = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int np = g.np;
    const uint32_t hd_bytes = (uint32_t)np * kHbPanelBytes;
    uint8_t* hd_buf = base;                                         // [2][np panels]
    uint8_t* w2_s = base + 2 * hd_bytes;                            // [np panels of 64 classes x 64 units]
    uint8_t* dl_buf = w2_s + (uint32_t)np * kHbW2PanelBytes;        // [128 rows x 64 classes]
    uint8_t* out_stage = dl_buf + kHbPanelBytes;                // [8 gate warps][32 rows x 64 units]
    uint64_t* bars = reinterpret_cast<uint64_t*>(out_stage + kHbGateWarps * kHbSlabBytes);
    float* bias_s = reinterpret_cast<float*>(bars + 16);            // [64]
    float* xch = bias_s + 64;                                       // exchange between the two threads of a row: 4 x [4][2][32]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(xch + 4 * 4 * 2 * 32);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tiles = (g.n_all + 127) / 128;
    const int64_t nt = (int64_t)blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        mbar_init(bars + HB_W2_FULL, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bars + HB_HD_FULL + b, 1);
            mbar_init(bars + HB_HD_EMPTY + b, 1);
            mbar_init(bars + HB_D1_FULL + b, 1);
            mbar_init(bars + HB_D1_EMPTY + b, kHbLossWarps);
            mbar_init(bars + HB_DL_FULL + b, 4);
            mbar_init(bars + HB_DL_EMPTY + b, 1);
        }
        mbar_init(bars + HB_D2_FULL, 1);
        mbar_init(bars + HB_D2_EMPTY, kHbGateWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {      // all of tensor memory: two logit accumulators of 64 columns, one gradient accumulator of 256
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
    }
    grid_dependency_wait();          // everything from here on may read what the previous kernel wrote
    grid_dependency_release();
    if (threadIdx.x >= 64 && threadIdx.x < 128) {
        const int c = threadIdx.x - 64;
        bias_s[c] = (g.b2 && c < g.O) ? g.b2[c] : 0.f;
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = *tmem_slot;

    if (warp == 0) {
        if (lane == 0 && nt > 0) {
            mbar_expect_tx(bars + HB_W2_FULL, (uint32_t)np * kHbW2PanelBytes);
            for (int p = 0; p < np; ++p) tma_load_2d(w2_s + p * kHbW2PanelBytes, &map_w2, 64 * p, 0, bars + HB_W2_FULL);
            int64_t issued = 0;
            for (int64_t i = 0; i < nt; ++i) {
                const int b = (int)(i & 1);
                const uint32_t u = (uint32_t)(i >> 1) & 1;
                if (!mbar_wait(bars + HB_HD_EMPTY + b, u ^ 1, g.status, abort_flag)) break;
                const int64_t tile = blockIdx.x + i * gridDim.x;
                mbar_expect_tx(bars + HB_HD_FULL + b, hd_bytes);
                for (int p = 0; p < np; ++p)
                    tma_load_2d(hd_buf + b * hd_bytes + p * kHbPanelBytes, &map_hd, 64 * p, (int32_t)(tile * 128),
                                bars + HB_HD_FULL + b);
                // The buffer of the tile after this one is freed about one tile's time from now; its rows are
                // asked into L2 already, so that the load then issued finds them there.
                if (i + 1 < nt)
                    for (int p = 0; p < np; ++p) tma_prefetch_2d(&map_hd, 64 * p, (int32_t)((tile + gridDim.x) * 128));
                issued = i + 1;
            }
            if (*abort_flag) {      // await (bounded) what was issued, so that nothing lands after the block has left
                for (uint32_t w = 0; w < (1u << 20); ++w) if (mbar_try_wait(bars + HB_W2_FULL, 0)) break;
                for (int64_t i = issued > 2 ? issued - 2 : 0; i < issued; ++i)
                    for (uint32_t w = 0; w < (1u << 20); ++w)
                        if (mbar_try_wait(bars + HB_HD_FULL + (i & 1), (uint32_t)(i >> 1) & 1)) break;
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && nt > 0) {
            const uint32_t idesc_logits = make_idesc((int)kHbLogitCols);
            const uint32_t idesc_grad = make_idesc(64 * np, false, true);
            const uint32_t w2_addr = smem_u32(w2_s);
            const uint64_t w2_desc = make_smem_desc(w2_addr), w2_desc_mn = make_smem_desc_mn(w2_addr, kHbW2PanelBytes);
            bool ok = mbar_wait(bars + HB_W2_FULL, 0, g.status, abort_flag);
            // logits of tile i: A = the Hd tile (K-major panels), B = W2^T (K-major panels), K = hidden units
            auto issue_logits = [&](int64_t i) -> bool {
                const int b = (int)(i & 1);
                const uint32_t u = (uint32_t)(i >> 1) & 1;
                if (!mbar_wait(bars + HB_HD_FULL + b, u, g.status, abort_flag)) return false;
                if (!mbar_wait(bars + HB_D1_EMPTY + b, u ^ 1, g.status, abort_flag)) return false;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // (descriptor arithmetic in 16-byte units: a panel further on, or 32 bytes = 16 hidden units along K)
                const uint64_t adesc = make_smem_desc(smem_u32(hd_buf + b * hd_bytes));
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    if (p < np) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            umma_bf16(tmem + (uint32_t)b * kHbLogitCols, adesc + (uint64_t)(p * (kHbPanelBytes >> 4) + 2 * j),
                                      w2_desc + (uint64_t)(p * (kHbW2PanelBytes >> 4) + 2 * j), idesc_logits, (p | j) ? 1u : 0u);
                    }
                }
                umma_commit(bars + HB_D1_FULL + b);
                umma_commit(bars + HB_HD_EMPTY + b);      // the Hd tile is free again once these MMAs have read it
                return true;
            };
            if (ok) ok = issue_logits(0);
            for (int64_t i = 0; i < nt && ok; ++i) {
                // The logits of tile i + 1 go first only if their Hd tile has already arrived: waiting for it
                // here would hold the gradient product of tile i (whose inputs may be ready) behind a load.
                bool next_issued = i + 1 >= nt;
                if (!next_issued && mbar_try_wait(bars + HB_HD_FULL + ((i + 1) & 1), (uint32_t)((i + 1) >> 1) & 1) &&
                    mbar_try_wait(bars + HB_D1_EMPTY + ((i + 1) & 1), ((uint32_t)((i + 1) >> 1) & 1) ^ 1)) {
                    ok = issue_logits(i + 1);
                    if (!ok) break;
                    next_issued = true;
                }
                if (!mbar_wait(bars + HB_DL_FULL, (uint32_t)(i & 1), g.status, abort_flag)) break;
                if (!mbar_wait(bars + HB_D2_EMPTY, (uint32_t)(i & 1) ^ 1, g.status, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // dHd of tile i: A = the dL tile (K-major, K = classes), B = the same W2^T panels read MN-major
                const uint64_t dl_desc = make_smem_desc(smem_u32(dl_buf));
#pragma unroll
                for (int j = 0; j < 4; ++j)      // 16 classes along K: 32 bytes of a dL line, two 1024-byte atoms of W2^T
                    umma_bf16(tmem + kHbGradCol0, dl_desc + (uint64_t)(2 * j), w2_desc_mn + (uint64_t)(128 * j), idesc_grad, j ? 1u : 0u);
                umma_commit(bars + HB_D2_FULL);
                umma_commit(bars + HB_DL_EMPTY);
                if (!next_issued) ok = issue_logits(i + 1);
            }
        }
    } else if (warp < kHbGateWarp0) {
        // ---- loss role: two threads share a row of logits, in two warps of the same tensor-memory lane quarter
        // (warp w and w + 4): the classes are cut into groups of eight, the first half of the groups goes to
        // the one, the rest to the other; row maximum, sum and the label's logit are exchanged through shared
        // memory.  Every reduction is a tree, so that a warp finds independent instructions to issue.
        const int q = warp & 3, part = (warp - kHbLossWarp0) >> 2;
        const int ng = (g.O + 7) >> 3, g_split = (ng + 1) >> 1;
        const int g_first = part ? g_split : 0, g_count = part ? ng - g_split : g_split;      // this thread's groups (<= 4)
        const int pair_bar = 1 + q;                                                            // named barrier of the two warps
        float* x_max = xch + (q * 2) * 32, *x_sum = xch + (8 + q * 2) * 32, *x_ly = xch + (16 + q * 2) * 32;
        int* x_best = reinterpret_cast<int*>(xch + (24 + q * 2) * 32);
        for (int64_t i = 0; i < nt; ++i) {
            const int b = (int)(i & 1);
            const uint32_t u = (uint32_t)(i >> 1) & 1;
            const int64_t tile = blockIdx.x + i * gridDim.x;
            const int64_t row0 = tile * 128 + q * 32, row = row0 + lane;
            const bool train = row < g.n_train;
            const bool eval = !train && row < g.n_all && g.y_eval != nullptr;
            const int32_t label = train ? g.y[row] : (eval ? g.y_eval[row - g.n_train] : -1);
            if (!mbar_wait(bars + HB_D1_FULL + b, u, g.status, abort_flag)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float v[32];
            {
                uint32_t r[32];
                tmem_ld_issue(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)b * kHbLogitCols + (uint32_t)(8 * g_first), r);
                tmem_ld_wait(r);
#pragma unroll
                for (int gi = 0; gi < 4; ++gi) {
                    if (gi < g_count) {
                        const int c0 = 8 * (g_first + gi);
                        const float4 b0 = *reinterpret_cast<const float4*>(bias_s + c0);
                        const float4 b1 = *reinterpret_cast<const float4*>(bias_s + c0 + 4);
                        const float bb[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
#pragma unroll
                        for (int k = 0; k < 8; ++k)
                            v[8 * gi + k] = c0 + k < g.O ? __uint_as_float(r[8 * gi + k]) + bb[k] : -INFINITY;
                    }
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_D1_EMPTY + b)) : "memory");
            float mx = -INFINITY;
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {
                if (gi < g_count) {
                    const float m01 = fmaxf(v[8 * gi], v[8 * gi + 1]), m23 = fmaxf(v[8 * gi + 2], v[8 * gi + 3]);
                    const float m45 = fmaxf(v[8 * gi + 4], v[8 * gi + 5]), m67 = fmaxf(v[8 * gi + 6], v[8 * gi + 7]);
                    mx = fmaxf(mx, fmaxf(fmaxf(m01, m23), fmaxf(m45, m67)));
                }
            }
            const bool has_eval = g.correct && row0 + 32 > g.n_train;      // evaluated rows among this warp's
            if (has_eval) {      // arg-max: the lowest index that reaches this thread's maximum
                int best = 0;
#pragma unroll
                for (int gi = 3; gi >= 0; --gi) {
                    if (gi < g_count) {
#pragma unroll
                        for (int k = 7; k >= 0; --k) best = v[8 * gi + k] == mx ? 8 * (g_first + gi) + k : best;
                    }
                }
                x_best[part * 32 + lane] = best;
            }
            x_max[part * 32 + lane] = mx;
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            const float m0 = x_max[lane], m1 = x_max[32 + lane];
            mx = fmaxf(m0, m1);
            if (has_eval && part == 0) {      // the lower classes win ties
                const int arg = m1 > m0 ? x_best[32 + lane] : x_best[lane];
                const unsigned hits = __ballot_sync(0xffffffffu, eval && arg == label);
                if (lane == 0 && hits) atomicAdd(g.correct, (unsigned long long)__popc(hits));
            }
            // exp(v - mx) as one multiply-add and one exponential per column; the label's logit is picked up on the way
            const float kLog2e = 1.4426950408889634f;
            const float shift = -mx * kLog2e;
            float den = 0.f, ly = 0.f;
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {
                if (gi < g_count) {
                    float e[8];
#pragma unroll
                    for (int k = 0; k < 8; ++k) {
                        ly = 8 * (g_first + gi) + k == label ? v[8 * gi + k] : ly;
                        e[k] = fast_exp2(fmaf(v[8 * gi + k], kLog2e, shift));      // columns beyond the last class hold -inf: 0
                        v[8 * gi + k] = e[k];
                    }
                    den += ((e[0] + e[1]) + (e[2] + e[3])) + ((e[4] + e[5]) + (e[6] + e[7]));
                }
            }
            x_sum[part * 32 + lane] = den;
            x_ly[part * 32 + lane] = ly;
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            den = x_sum[lane] + x_sum[32 + lane];
            ly = x_ly[lane] + x_ly[32 + lane];
            const float scale = train ? g.inv_rows / den : 0.f;
            const float hot = train ? g.inv_rows : 0.f;
            // the dL tile of the previous tile has been read by its MMA and by its store
            if (!mbar_wait(bars + HB_DL_EMPTY, (uint32_t)(i & 1) ^ 1, g.status, abort_flag)) break;
            if (part == 0 && lane == 0) bulk_wait_read_all();
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            uint8_t* slab = dl_buf + q * kHbSlabBytes;
#pragma unroll
            for (int gi = 0; gi < 4; ++gi) {      // one 16-byte piece of the row's line per group of eight classes
                const int piece = part ? g_split + gi : gi;      // part 1 also clears the pieces beyond the last class
                if (piece < 8 && (part || gi < g_split)) {
                    uint32_t pk[4] = {0u, 0u, 0u, 0u};
                    if (gi < g_count) {
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int c = 8 * piece + 2 * k;
                            const float lo = fmaf(v[8 * gi + 2 * k], scale, c == label ? -hot : 0.f);
                            const float hi = fmaf(v[8 * gi + 2 * k + 1], scale, c + 1 == label ? -hot : 0.f);
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                            pk[k] = *reinterpret_cast<uint32_t*>(&b2);
                        }
                    }
                    *reinterpret_cast<uint4*>(slab + lane * 128 + ((piece ^ (lane & 7)) * 16)) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                }
            }
            if (part == 1) {      // pieces that neither thread's four groups reach (few classes): zeros
                for (int piece = g_split + 4; piece < 8; ++piece)
                    *reinterpret_cast<uint4*>(slab + lane * 128 + ((piece ^ (lane & 7)) * 16)) = make_uint4(0u, 0u, 0u, 0u);
            }
            fence_proxy_async_smem();
            asm volatile("bar.sync %0, 64;" ::"r"(pair_bar) : "memory");
            if (part == 0) {
                if (lane == 0) {
                    if (row0 < g.n_train) { tma_store_2d(&map_dl, slab, 0, (int32_t)row0); bulk_commit(); }
                    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_DL_FULL)) : "memory");
                }
                const float loss = warp_sum(train ? (mx + __logf(den)) - ly : 0.f);
                if (lane == 0 && g.loss_partial) g.loss_partial[tile * 4 + q] = loss;
            }
        }
        if (lane == 0) bulk_wait_all();
    } else {
        // ---- gate role: dHd = accumulator where the unit's ReLU bit is set, staged per warp and sent out
        const int q = warp & 3, h = (warp - kHbGateWarp0) >> 2;
        uint8_t* stage = out_stage + (warp - kHbGateWarp0) * kHbSlabBytes;
        const bool scaled = g.gate_scale != 1.f;      // (dropout: the kept units' factor)
        for (int64_t i = 0; i < nt; ++i) {
            const int64_t tile = blockIdx.x + i * gridDim.x;
            const int64_t row0 = tile * 128 + q * 32, row = row0 + lane;
            // this row's ReLU bits for the (up to two) panels of 64 units this warp takes: p = h and h + 2
            uint2 bits[2] = {make_uint2(0u, 0u), make_uint2(0u, 0u)};
            if (row < g.n_train) {
#pragma unroll
                for (int k = 0; k < 2; ++k)
                    if (h + 2 * k < np) bits[k] = __ldg(reinterpret_cast<const uint2*>(g.gate_bits + row * g.ld_bits + 2 * (h + 2 * k)));
            }
            if (!mbar_wait(bars + HB_D2_FULL, (uint32_t)(i & 1), g.status, abort_flag)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int p = h + 2 * k;
                if (p < np) {
                    uint32_t ra[32], rb[32];
                    const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + kHbGradCol0 + (uint32_t)(64 * p);
                    tmem_ld_issue(taddr, ra);
                    tmem_ld_issue(taddr + 32u, rb);
                    tmem_ld_wait(ra);
                    tmem_ld_wait(rb);
                    // A unit whose bit is clear gives zero: the accumulator's bits are ANDed with 0 - bit.  Everything
                    // is packed in registers first, so that the wait for the staging block comes after the arithmetic.
                    uint32_t o[32];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t word = (j < 4 ? bits[k].x : bits[k].y) >> (8 * (j & 3));
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int c = 8 * (j & 3) + 2 * e;
                            const uint32_t x0 = (j < 4 ? ra[c] : rb[c]) & (0u - ((word >> (2 * e)) & 1u));
                            const uint32_t x1 = (j < 4 ? ra[c + 1] : rb[c + 1]) & (0u - ((word >> (2 * e + 1)) & 1u));
                            float lo = __uint_as_float(x0), hi = __uint_as_float(x1);
                            if (scaled) { lo *= g.gate_scale; hi *= g.gate_scale; }
                            __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                            o[4 * j + e] = *reinterpret_cast<uint32_t*>(&b2);
                        }
                    }
                    if (lane == 0) bulk_wait_read_all();      // the store of the previous panel has read the staging block
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<uint4*>(stage + lane * 128 + ((j ^ (lane & 7)) * 16)) = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
                if (k == 1 || p + 2 >= np) {      // this warp's last read of the accumulator for this tile
                    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
                    __syncwarp();
                    if (lane == 0 && (k == 1 || p >= np || p + 2 >= np))
                        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_D2_EMPTY)) : "memory");
                }
                if (p < np) {
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0 && row0 < g.n_train) { tma_store_2d(&map_dhd, stage, 64 * p, (int32_t)row0); bulk_commit(); }
                }
                if (p + 2 >= np) break;
            }
        }
        if (lane == 0) bulk_wait_all();
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512));
    }
}

bool head_backward_supported(const HeadBackward& h) {
    if (h.hidden < 1 || h.hidden > 256 || h.n_classes < 1 || h.n_classes > 64) return false;
    if (h.n_train < 1 || h.n_all < h.n_train || h.n_all > INT32_MAX - 256) return false;
    if (!h.hd || !h.w2t || !h.dl || !h.dhd || !h.y || h.ld_dl != 64) return false;
    if (!h.gate_bits || h.ld_bits < 2 * ((h.hidden + 63) / 64) || h.ld_bits % 2 != 0 || !aligned_to(h.gate_bits, 8)) return false;
    if (h.ld_hd < h.hidden || h.ld_w2t < h.hidden || h.ld_dhd < h.hidden) return false;
    if (h.ld_hd % 8 != 0 || h.ld_w2t % 8 != 0 || h.ld_dhd % 8 != 0) return false;
    return aligned_to(h.hd, 16) && aligned_to(h.w2t, 16) && aligned_to(h.dl, 16) && aligned_to(h.dhd, 16);
}

int head_backward_launch(const HeadBackward& h, cudaStream_t st) {
    if (!head_backward_supported(h)) return RETEXO_ERR_UNSUPPORTED;
    const int np = (h.hidden + 63) / 64;
    CUtensorMap m_hd, m_w2, m_dl, m_dhd;
    if (!tc_make_map_2d(&m_hd, h.hd, h.n_all, h.hidden, h.ld_hd, 128, 64, 128, true)) return RETEXO_ERR_CUDA;
    if (!tc_make_map_2d(&m_w2, h.w2t, h.n_classes, h.hidden, h.ld_w2t, 64, 64, 128, true)) return RETEXO_ERR_CUDA;
    if (!tc_make_map_2d(&m_dl, h.dl, h.n_train, 64, h.ld_dl, 32, 64, 128, false)) return RETEXO_ERR_CUDA;
    if (!tc_make_map_2d(&m_dhd, h.dhd, h.n_train, h.hidden, h.ld_dhd, 32, 64, 128, false)) return RETEXO_ERR_CUDA;
    const size_t smem = 1024 + (size_t)2 * np * kHbPanelBytes + (size_t)np * kHbW2PanelBytes + kHbPanelBytes +
                        kHbGateWarps * kHbSlabBytes + 1024 + 4096;
    if (cudaFuncSetAttribute(head_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    HbArgs g{};
    g.n_all = h.n_all; g.n_train = h.n_train; g.H = h.hidden; g.O = h.n_classes; g.np = np;
    g.b2 = h.b2; g.y = h.y; g.y_eval = h.y_eval;
    g.inv_rows = h.inv_rows; g.gate_scale = h.gate_scale != 0.f ? h.gate_scale : 1.f;
    g.gate_bits = h.gate_bits; g.ld_bits = h.ld_bits;
    g.loss_partial = h.loss_partial; g.correct = h.correct; g.status = h.status;
    const int64_t n_tiles = (h.n_all + 127) / 128;
    const int n_sm = sm_count();
    if (n_sm <= 0) return RETEXO_ERR_CUDA;
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);
    OverlapLaunch ol(dim3(grid), dim3(kHbThreads), smem, st);
    if (cudaLaunchKernelEx(&ol.cfg, head_backward_kernel, m_hd, m_w2, m_dl, m_dhd, g) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace retexo
