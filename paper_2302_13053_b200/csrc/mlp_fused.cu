// The row-local middle of one training iteration of the per-node model (Section 3.1: f_theta = Linear +
// ReLU, temporary classifier C_theta = Linear) in one kernel on sm_100a.  For every tile of 128 batch rows:
//   logits = Hd W2 + b2                     tcgen05.mma, Hd tile and W2 resident in shared memory
//   loss_i = CE(softmax(logits_i), y_i),  dL = (softmax - onehot) / n     in registers, one thread per row
//   dHd    = (dL W2^T) .* [Hd > 0]          a second tcgen05.mma whose A operand is the dL tile just written
//                                           to shared memory; the gate is the Hd tile still resident there
// Hd is read from global memory once, the logits never leave the SM, and dL and dHd go out row-major (the
// weight-gradient products read them as they lie).  One copy of W2^T in shared memory serves both products:
// K-major (reduction over the hidden units) for the logits, MN-major (reduction over the classes) for dHd.
//
// Roles: warp 0 loads (TMA), warp 1 issues the MMAs and owns tensor memory, warps 2-5 turn logits into loss
// and dL (one thread per row), warps 6-13 gate dHd and send it out.  The Hd tile, the logits and the dL tile
// are double-buffered, so the loss warps work on tile i + 1 while the gate warps finish tile i.
// Every wait is bounded: one that runs out sets *status and the block tears down in order.
#include <string.h>

#include "gemm_tc.h"
#include "tc_common.cuh"

namespace retexo {

constexpr int kHbThreads = 448;
constexpr int kHbLossWarp0 = 2, kHbGateWarp0 = 6, kHbGateWarps = 8;
constexpr uint32_t kHbPanelBytes = 128 * 128;       // [128 rows x 64 bf16], 128-byte swizzle
constexpr uint32_t kHbW2PanelBytes = 64 * 128;      // [64 classes x 64 hidden units]
constexpr uint32_t kHbSlabBytes = 32 * 128;         // one warp's 32 rows of a panel
constexpr uint32_t kHbLogitCols = 64, kHbGradCol0 = 256;

struct HbArgs {
    int64_t n_all, n_train;
    int32_t H, O, np;                  // np = panels of 64 hidden units
    const float* b2;
    const int32_t* y; const int32_t* y_eval;
    float inv_rows, gate_scale;
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
    uint8_t* dl_buf = w2_s + (uint32_t)np * kHbW2PanelBytes;        // [2][128 rows x 64 classes]
    uint64_t* bars = reinterpret_cast<uint64_t*>(dl_buf + 2 * kHbPanelBytes);
    float* bias_s = reinterpret_cast<float*>(bars + 16);            // [64]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bias_s + 64);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_tiles = (g.n_all + 127) / 128;
    const int64_t nt = (int64_t)blockIdx.x < n_tiles ? (n_tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;

    if (threadIdx.x == 0) {
        mbar_init(bars + HB_W2_FULL, 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(bars + HB_HD_FULL + b, 1);
            mbar_init(bars + HB_HD_EMPTY + b, kHbGateWarps);
            mbar_init(bars + HB_D1_FULL + b, 1);
            mbar_init(bars + HB_D1_EMPTY + b, 4);
            mbar_init(bars + HB_DL_FULL + b, 4);
            mbar_init(bars + HB_DL_EMPTY + b, 1);
        }
        mbar_init(bars + HB_D2_FULL, 1);
        mbar_init(bars + HB_D2_EMPTY, kHbGateWarps);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (threadIdx.x >= 64 && threadIdx.x < 128) {
        const int c = threadIdx.x - 64;
        bias_s[c] = (g.b2 && c < g.O) ? g.b2[c] : 0.f;
    }
    if (warp == 1) {      // all of tensor memory: two logit accumulators of 64 columns, one gradient accumulator of 256
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512));
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
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
            bool ok = mbar_wait(bars + HB_W2_FULL, 0, g.status, abort_flag);
            // logits of tile i: A = the Hd tile (K-major panels), B = W2^T (K-major panels), K = hidden units
            auto issue_logits = [&](int64_t i) -> bool {
                const int b = (int)(i & 1);
                const uint32_t u = (uint32_t)(i >> 1) & 1;
                if (!mbar_wait(bars + HB_HD_FULL + b, u, g.status, abort_flag)) return false;
                if (!mbar_wait(bars + HB_D1_EMPTY + b, u ^ 1, g.status, abort_flag)) return false;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_addr = smem_u32(hd_buf + b * hd_bytes);
                for (int kk = 0; kk < 4 * np; ++kk) {
                    const uint32_t p = (uint32_t)kk >> 2, j = (uint32_t)kk & 3;
                    umma_bf16(tmem + (uint32_t)b * kHbLogitCols, make_smem_desc(a_addr + p * kHbPanelBytes + j * 32),
                              make_smem_desc(w2_addr + p * kHbW2PanelBytes + j * 32), idesc_logits, kk > 0 ? 1u : 0u);
                }
                umma_commit(bars + HB_D1_FULL + b);
                return true;
            };
            if (ok) ok = issue_logits(0);
            for (int64_t i = 0; i < nt && ok; ++i) {
                if (i + 1 < nt) { ok = issue_logits(i + 1); if (!ok) break; }
                const int b = (int)(i & 1);
                const uint32_t u = (uint32_t)(i >> 1) & 1;
                if (!mbar_wait(bars + HB_DL_FULL + b, u, g.status, abort_flag)) break;
                if (!mbar_wait(bars + HB_D2_EMPTY, (uint32_t)(i & 1) ^ 1, g.status, abort_flag)) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // dHd of tile i: A = the dL tile (K-major, K = classes), B = the same W2^T panels read MN-major
                const uint32_t a_addr = smem_u32(dl_buf + b * kHbPanelBytes);
                for (uint32_t j = 0; j < 4; ++j)
                    umma_bf16(tmem + kHbGradCol0, make_smem_desc(a_addr + j * 32), make_smem_desc_mn(w2_addr + j * 2048, kHbW2PanelBytes),
                              idesc_grad, j > 0 ? 1u : 0u);
                umma_commit(bars + HB_D2_FULL);
                umma_commit(bars + HB_DL_EMPTY + b);
            }
        }
    } else if (warp < kHbGateWarp0) {
        // ---- loss role: one thread per row holds the whole row of logits
        const int q = warp & 3;
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
            float v[64];
            {
                uint32_t ra[32], rb[32];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)b * kHbLogitCols;
                tmem_ld_issue(taddr, ra);
                tmem_ld_issue(taddr + 32u, rb);
                tmem_ld_wait(ra);
                tmem_ld_wait(rb);
#pragma unroll
                for (int c = 0; c < 32; ++c) {
                    v[c] = c < g.O ? __uint_as_float(ra[c]) + bias_s[c] : -INFINITY;
                    v[32 + c] = 32 + c < g.O ? __uint_as_float(rb[c]) + bias_s[32 + c] : -INFINITY;
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_D1_EMPTY + b)) : "memory");
            float mx = v[0];
            int best = 0;
#pragma unroll
            for (int c = 1; c < 64; ++c) if (v[c] > mx) { mx = v[c]; best = c; }      // strict: lowest index on ties
            float den = 0.f, ly = 0.f;
#pragma unroll
            for (int c = 0; c < 64; ++c) {
                ly = c == label ? v[c] : ly;
                v[c] = c < g.O ? __expf(v[c] - mx) : 0.f;
                den += v[c];
            }
            const float scale = train ? g.inv_rows / den : 0.f;
            uint32_t pk[32];
#pragma unroll
            for (int k = 0; k < 32; ++k) {
                const float lo = v[2 * k] * scale - ((train && 2 * k == label) ? g.inv_rows : 0.f);
                const float hi = v[2 * k + 1] * scale - ((train && 2 * k + 1 == label) ? g.inv_rows : 0.f);
                __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                pk[k] = *reinterpret_cast<uint32_t*>(&b2);
            }
            // the dL tile written two tiles ago has been read by its MMA and by this warp's own store
            if (!mbar_wait(bars + HB_DL_EMPTY + b, u ^ 1, g.status, abort_flag)) break;
            if (lane == 0) bulk_wait_read_all();
            __syncwarp();
            uint8_t* slab = dl_buf + b * kHbPanelBytes + q * kHbSlabBytes;
#pragma unroll
            for (int ch = 0; ch < 8; ++ch)
                *reinterpret_cast<uint4*>(slab + lane * 128 + ((ch ^ (lane & 7)) * 16)) =
                    make_uint4(pk[4 * ch], pk[4 * ch + 1], pk[4 * ch + 2], pk[4 * ch + 3]);
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                if (row0 < g.n_train) { tma_store_2d(&map_dl, slab, 0, (int32_t)row0); bulk_commit(); }
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_DL_FULL + b)) : "memory");
            }
            const float loss = warp_sum(train ? (mx + __logf(den)) - ly : 0.f);
            if (lane == 0 && g.loss_partial) g.loss_partial[tile * 4 + q] = loss;
            if (g.correct && row0 + 32 > g.n_train) {      // evaluated rows among this warp's
                const unsigned hits = __ballot_sync(0xffffffffu, eval && best == label);
                if (lane == 0 && hits) atomicAdd(g.correct, (unsigned long long)__popc(hits));
            }
        }
        if (lane == 0) bulk_wait_all();
    } else {
        // ---- gate role: dHd = accumulator where the resident Hd entry is positive, written over that entry
        const int q = warp & 3, h = (warp - kHbGateWarp0) >> 2;
        for (int64_t i = 0; i < nt; ++i) {
            const int b = (int)(i & 1);
            const int64_t tile = blockIdx.x + i * gridDim.x;
            const int64_t row0 = tile * 128 + q * 32;
            if (!mbar_wait(bars + HB_D2_FULL, (uint32_t)(i & 1), g.status, abort_flag)) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            for (int p = h; p < np; p += 2) {
                uint32_t ra[32], rb[32];
                const uint32_t taddr = tmem + ((uint32_t)(q * 32) << 16) + kHbGradCol0 + (uint32_t)(64 * p);
                tmem_ld_issue(taddr, ra);
                tmem_ld_issue(taddr + 32u, rb);
                uint8_t* line = hd_buf + b * hd_bytes + p * kHbPanelBytes + (q * 32 + lane) * 128;
                tmem_ld_wait(ra);
                tmem_ld_wait(rb);
#pragma unroll
                for (int ch = 0; ch < 8; ++ch) {
                    uint4* slot = reinterpret_cast<uint4*>(line + ((ch ^ (lane & 7)) * 16));
                    const uint4 gate = *slot;
                    const __nv_bfloat16* gv = reinterpret_cast<const __nv_bfloat16*>(&gate);
                    uint32_t o[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int c = 8 * ch + 2 * e;
                        const float a0 = __uint_as_float(c < 32 ? ra[c & 31] : rb[c & 31]);
                        const float a1 = __uint_as_float(c + 1 < 32 ? ra[(c + 1) & 31] : rb[(c + 1) & 31]);
                        const float lo = __bfloat162float(gv[2 * e]) > 0.f ? a0 * g.gate_scale : 0.f;
                        const float hi = __bfloat162float(gv[2 * e + 1]) > 0.f ? a1 * g.gate_scale : 0.f;
                        __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                        o[e] = *reinterpret_cast<uint32_t*>(&b2);
                    }
                    *slot = make_uint4(o[0], o[1], o[2], o[3]);
                }
            }
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) {
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_D2_EMPTY)) : "memory");
                if (row0 < g.n_train) {
                    for (int p = h; p < np; p += 2)
                        tma_store_2d(&map_dhd, hd_buf + b * hd_bytes + p * kHbPanelBytes + q * kHbSlabBytes, 64 * p, (int32_t)row0);
                    bulk_commit();
                    bulk_wait_read_all();      // the stores have read the tile: the loader may refill it
                }
                asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bars + HB_HD_EMPTY + b)) : "memory");
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
    const size_t smem = 1024 + (size_t)2 * np * kHbPanelBytes + (size_t)np * kHbW2PanelBytes + 2 * kHbPanelBytes + 1024;
    if (cudaFuncSetAttribute(head_backward_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    HbArgs g{};
    g.n_all = h.n_all; g.n_train = h.n_train; g.H = h.hidden; g.O = h.n_classes; g.np = np;
    g.b2 = h.b2; g.y = h.y; g.y_eval = h.y_eval;
    g.inv_rows = h.inv_rows; g.gate_scale = h.gate_scale != 0.f ? h.gate_scale : 1.f;
    g.loss_partial = h.loss_partial; g.correct = h.correct; g.status = h.status;
    const int64_t n_tiles = (h.n_all + 127) / 128;
    const int n_sm = sm_count();
    if (n_sm <= 0) return RETEXO_ERR_CUDA;
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);
    head_backward_kernel<<<grid, kHbThreads, smem, st>>>(m_hd, m_w2, m_dl, m_dhd, g);
    return launch_status();
}

}  // namespace retexo
