// Tensor-core GEMM for the dense products of the per-node model on sm_100a:
//   C[M x N] = A[M x K] * B[N x K]^T,  A and B bf16 with K contiguous, or (the split-K weight-gradient
//   products, whose reduction runs over the batch) C = A^T B with A [K x M] and B [K x N] row-major;
//   fp32 accumulation in tensor memory (tcgen05.mma, cta_group::1, M = 128).
// Operand tiles are brought in by TMA (128-byte swizzle) through a ring of
// shared-memory stages guarded by mbarriers; one thread issues the MMAs; eight
// or sixteen warps drain the accumulators with tcgen05.ld and apply the fused
// epilogue (bias / ReLU / bf16 down-cast, soft-max loss, gate, split-K partial).
// Every wait is bounded: a wait that runs out sets *status and the block
// tears down in order (outstanding copies awaited, tensor memory freed).
#include <string.h>

#include "gemm_tc.h"
#include "tc_common.cuh"

namespace retexo {

// Threads: warp 0 TMA, warp 1 MMA + tensor-memory owner, then EW epilogue warps (8 or 16).  The epilogues
// are chains of dependent instructions, so their speed is set by how many warps share an SM's schedulers:
// with 16 warps a tile's columns are cut four ways (BN >= 128), or (BN = 64, where a row of logits is
// shared by two threads) two groups of 8 warps take alternate tiles out of four accumulators.
#ifndef TC256_EW
#define TC256_EW 8
#define TC256_STAGES 4
#endif
#ifndef TC128_EW
#define TC128_EW 16
#define TC128_STAGES 4
#endif
#ifndef TC64_EW
#define TC64_EW 16
#define TC64_STAGES 5
#endif

// One block of the counter-based generator Philox4x32-10 (Salmon et al., SC'11), from its definition:
// ten rounds of (c0,c1,c2,c3) <- (hi(M1 c2)^c1^k0, lo(M1 c2), hi(M0 c0)^c3^k1, lo(M0 c0)), the key raised
// by (W0, W1) between rounds.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&out)[4]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint32_t hi0 = __umulhi(0xD2511F53u, c0), lo0 = 0xD2511F53u * c0;
        const uint32_t hi1 = __umulhi(0xCD9E8D57u, c2), lo1 = 0xCD9E8D57u * c2;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

struct TcKernelArgs {
    int64_t M, N;
    int32_t k_blocks_total;       // ceil(K / 64)
    int32_t k_blocks_per_split;
    int32_t splits;
    int mode, relu;
    const float* bias;
    float* out_f32; int64_t ld_f32;
    __nv_bfloat16* out_bf16; int64_t ld_bf16;
    int ones_col;
    uint32_t* relu_bits; int64_t ld_bits;
    const __nv_bfloat16* mask; int64_t ld_mask;
    float gate_scale;
    uint32_t drop_thresh, drop_step, drop_key0, drop_key1; float drop_scale; int64_t drop_rows;
    const unsigned long long* drop_step_dev;
    float* partial;
    const int32_t* y; float inv_rows; float* loss_partial;
    int32_t* pred; unsigned long long* correct;
    int64_t n_train; const int32_t* y_eval;       // SOFTMAX_CE: rows >= n_train are evaluated, not trained on
    int32_t* status;
    int tma_rows;                 // out_bf16 leaves through bulk tensor stores (map_rows)
};

// Per-warp staging of one 32 x 32 bf16 block: 32 lines of 64 bytes, a line being one output row.  The four
// 16-byte pieces of a line are XOR-swizzled with the line index so that both the fill (one thread per row)
// and the drain (eight lines of 64 contiguous bytes per instruction) are free of bank conflicts.
// This is also the 64-byte swizzle of a tensor map (address bits 4-5 XOR bits 7-8), so a block staged in a
// 1024-byte aligned buffer can leave as one bulk tensor store.  Every warp owns two such blocks (the gated
// epilogue alternates between them, so that one can be filled while the other's store is in flight).
constexpr int kStageBlockBytes = 32 * 64;
constexpr int kStageBytesPerWarp = 2 * kStageBlockBytes;
__device__ __forceinline__ int stage_piece(int line, int piece) { return piece ^ ((line >> 1) & 3); }

// Drains the staged block: line L goes to dst + L * stride (elements), 64 contiguous bytes each.
__device__ __forceinline__ void drain_stage(const uint8_t* stage, __nv_bfloat16* dst, int64_t stride, int64_t n_lines,
                                            int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int line = (lane >> 2) + 8 * i, piece = lane & 3;
        if (line < n_lines)
            *reinterpret_cast<uint4*>(dst + line * stride + piece * 8) =
                *reinterpret_cast<const uint4*>(stage + line * 64 + stage_piece(line, piece) * 16);
    }
}

// Row-major store without a tensor map: out[row][col0 .. col0+32); a full, aligned block of columns goes through the staging
// block, anything else through guarded element stores.  Rows beyond M are dropped.
__device__ __forceinline__ void store_block_rows(__nv_bfloat16* out, int64_t ld, int64_t col0, int64_t n_cols, int64_t row0,
                                                 int64_t M, const float (&v)[32], uint8_t* stage, int lane) {
    if (col0 + 32 <= n_cols && (ld & 7) == 0 && aligned16(out)) {
#pragma unroll
        for (int p = 0; p < 4; ++p) {         // line = this lane's row; four 16-byte pieces of 8 columns
            __nv_bfloat162 a = __floats2bfloat162_rn(v[8 * p], v[8 * p + 1]), b = __floats2bfloat162_rn(v[8 * p + 2], v[8 * p + 3]);
            __nv_bfloat162 c = __floats2bfloat162_rn(v[8 * p + 4], v[8 * p + 5]), d = __floats2bfloat162_rn(v[8 * p + 6], v[8 * p + 7]);
            uint4 pk;
            pk.x = *reinterpret_cast<uint32_t*>(&a); pk.y = *reinterpret_cast<uint32_t*>(&b);
            pk.z = *reinterpret_cast<uint32_t*>(&c); pk.w = *reinterpret_cast<uint32_t*>(&d);
            *reinterpret_cast<uint4*>(stage + lane * 64 + stage_piece(lane, p) * 16) = pk;
        }
        __syncwarp();
        const int64_t n_lines = M - row0 < 32 ? M - row0 : 32;
        drain_stage(stage, out + row0 * ld + col0, ld, n_lines, lane);
        __syncwarp();
    } else if (row0 + lane < M) {
        __nv_bfloat16* dst = out + (row0 + lane) * ld + col0;
#pragma unroll
        for (int j = 0; j < 32; ++j) if (col0 + j < n_cols) dst[j] = __float2bfloat16_rn(v[j]);
    }
}

// Bulk-store core: p[k] holds columns col0 + 2k (low half) and col0 + 2k + 1 (high half) of this lane's row as bf16.
// The block is staged row-major and leaves as one bulk tensor store, clipped to the map's extents (the caller
// guarantees row0 and col0 inside them).  ready_block (optional): a staging block the caller has already made
// sure no bulk store is reading; it is used instead of the warp's own block and nothing is waited for.
// Warp-uniform arguments except p.
__device__ __forceinline__ void store_block_packed(const uint32_t (&p)[16], uint8_t* stage, int lane, int64_t col0, int64_t row0,
                                                   const CUtensorMap* rows_map, uint8_t* ready_block = nullptr) {
    uint8_t* rows_block = stage + kStageBlockBytes;
    if (ready_block) {
        rows_block = ready_block;
    } else {
        if (lane == 0) bulk_wait_read_all();      // the previous block's store has read the staging block
        __syncwarp();
    }
    uint8_t* line = rows_block + lane * 64;
#pragma unroll
    for (int q = 0; q < 4; ++q)
        *reinterpret_cast<uint4*>(line + stage_piece(lane, q) * 16) = make_uint4(p[4 * q], p[4 * q + 1], p[4 * q + 2], p[4 * q + 3]);
    fence_proxy_async_smem();
    __syncwarp();
    if (lane == 0) {
        tma_store_2d(rows_map, rows_block, (int32_t)col0, (int32_t)row0);
        bulk_commit();
    }
}

// Stores a warp's 32 x 32 block (lane = row, v[j] = column col0 + j) as bf16, row-major, into out: through a
// bulk tensor store where the output has a tensor map, else through store_block_rows.  Warp-uniform
// arguments except v.
__device__ __forceinline__ void store_block(const float (&v)[32], uint8_t* stage, int lane, int64_t col0, int64_t n_cols,
                                            int64_t row0, int64_t M, __nv_bfloat16* out, int64_t ld,
                                            const CUtensorMap* rows_map) {
    if (!rows_map) {
        store_block_rows(out, ld, col0, n_cols, row0, M, v, stage + kStageBlockBytes, lane);
        return;
    }
    uint32_t p[16];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        __nv_bfloat162 b2 = __floats2bfloat162_rn(v[2 * k], v[2 * k + 1]);
        p[k] = *reinterpret_cast<uint32_t*>(&b2);
    }
    store_block_packed(p, stage, lane, col0, row0, rows_map);
}

// Copies a [32 x 32] bf16 block (rows row0.., columns col0..; full and aligned columns, guaranteed by the
// caller) into a staging block in 64-byte runs; rows beyond M are filled with zeros.  Afterwards lane L
// finds piece q (columns 8q .. 8q+7) of row L at block + L * 64 + stage_piece(L, q) * 16.
__device__ __forceinline__ void stage_block_from_global(const __nv_bfloat16* src, int64_t ld, int64_t col0, int64_t row0,
                                                        int64_t M, uint8_t* block, int lane) {
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int line = (lane >> 2) + 8 * i, piece = lane & 3;
        uint4 pk = make_uint4(0u, 0u, 0u, 0u);
        if (row0 + line < M) pk = __ldg(reinterpret_cast<const uint4*>(src + (row0 + line) * ld + col0 + piece * 8));
        *reinterpret_cast<uint4*>(block + line * 64 + stage_piece(line, piece) * 16) = pk;
    }
    __syncwarp();
}

// MODE (a TcEpilogue value) is a template parameter so that every instantiation carries the registers of
// its own epilogue only.
template <int BN, int STAGES, int MODE, int EW, bool PAIR = false>
__global__ void __launch_bounds__(64 + 32 * EW, 1)
tc_gemm_kernel(const __grid_constant__ CUtensorMap map_a, const __grid_constant__ CUtensorMap map_b,
               const __grid_constant__ CUtensorMap map_rows, TcKernelArgs g) {
    // Persistent: the block walks over output tiles t = blockIdx.x, blockIdx.x + gridDim.x, ...  The
    // stage ring runs on across tiles and the accumulator is multi-buffered in tensor memory, so
    // the loads and MMAs of the next tile(s) overlap the epilogue of the current one.
    constexpr int TG = (BN == 64 && EW == 16) ? 2 : 1;      // groups of epilogue warps that take alternate tiles
    constexpr int CP = EW / 4 / TG;                         // column parts a tile is cut into
    constexpr int NACC = 2 * TG;                            // accumulators in tensor memory
    static_assert(BN % (32 * CP) == 0 && NACC * BN <= 512, "tile split");
    extern __shared__ uint8_t smem_raw[];
    // PAIR: the block is one of a pair (cluster of two) that shares 256-row tiles: it holds its own 128 rows of A
    // and its own half of the B tile (BN / 2 rows), so a stage is a third smaller and every B tile crosses the
    // L2 -> SM path once per 256 rows instead of once per 128.
    constexpr uint32_t kABytes = kTcBM * kTcBK * 2, kBBytes = (PAIR ? BN / 2 : BN) * kTcBK * 2, kStageBytes = kABytes + kBBytes;
    constexpr int kTileRows = PAIR ? 2 * kTcBM : kTcBM;
    static_assert(!PAIR || (MODE != TC_EPI_PARTIAL && BN == 256 && TG == 1), "pairs: K-major 256-column tiles");
    const uint32_t pair_rank = PAIR ? cluster_rank() : 0u;
    const int64_t tile_first = PAIR ? (int64_t)(blockIdx.x >> 1) : (int64_t)blockIdx.x;
    const int64_t tile_stride = PAIR ? (int64_t)(gridDim.x >> 1) : (int64_t)gridDim.x;
    // The split-K products reduce over the batch, and their operands (activations and gradients, one batch row
    // per line) are read as they lie in memory: M and N are the contiguous dimensions ("MN-major" operands).
    constexpr bool kMnMajor = MODE == TC_EPI_PARTIAL;
    constexpr uint32_t kMnBoxBytes = kTcBK * 64 * 2;      // one box: 64 reduction rows of 64 elements
    uint8_t* tiles = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    uint64_t* full = reinterpret_cast<uint64_t*>(tiles + STAGES * kStageBytes);
    uint64_t* empty = full + STAGES;
    uint64_t* acc_full = empty + STAGES;          // [NACC] accumulator b holds a finished tile
    uint64_t* acc_empty = acc_full + NACC;        // [NACC] accumulator b has been drained
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(acc_empty + NACC);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    float* warp_loss_all = reinterpret_cast<float*>(tmem_slot + 2);              // [TG][4]
    // staging blocks: EW x kStageBytesPerWarp, 1024 bytes behind the barrier area (so 1024-byte aligned)
    uint8_t* stage_base = tiles + STAGES * kStageBytes + 1024;
    float (*xch_all)[2][128] = reinterpret_cast<float (*)[2][128]>(stage_base + EW * kStageBytesPerWarp);   // [TG][4][2][128]

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t n_m = (g.M + kTileRows - 1) / kTileRows, n_n = (g.N + BN - 1) / BN;
    const int64_t per_split = n_m * n_n;
    const int64_t n_tiles = per_split * g.splits;

    if (threadIdx.x == 0) {
        for (int s = 0; s < STAGES; ++s) { mbar_init(full + s, 1); mbar_init(empty + s, 1); }
        // the arg-max epilogue lets one thread own a whole row of logits: it uses four of the eight warps
        const bool row_owner = BN == 64 && MODE == TC_EPI_ARGMAX;
        // (pairs: the even block's "accumulator drained" barrier collects the epilogue warps of both blocks)
        for (int b = 0; b < NACC; ++b) { mbar_init(acc_full + b, 1); mbar_init(acc_empty + b, row_owner ? 4 : (PAIR ? 2 : 1) * EW / TG); }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {      // tensor memory: NACC accumulators of BN fp32 columns x 128 lanes
        if constexpr (PAIR) {
            asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(NACC * BN));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;");
        } else {
            asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(NACC * BN));
            asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;");
        }
    }
    grid_dependency_wait();          // everything from here on may read what the previous kernel wrote
    grid_dependency_release();
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();      // both blocks' barriers exist before either signals the other's
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            int64_t it = 0;                       // k-blocks issued so far, over all tiles
            bool ok = true;
            for (int64_t t = tile_first; t < n_tiles && ok; t += tile_stride) {
                const int64_t z = t / per_split, rem = t % per_split;
                const int32_t m0 = (int32_t)((rem % n_m) * kTileRows + pair_rank * kTcBM), n0 = (int32_t)((rem / n_m) * BN);
                const int32_t kb0 = (int32_t)z * g.k_blocks_per_split;
                const int32_t kb1 = min(g.k_blocks_total, kb0 + g.k_blocks_per_split);
                for (int32_t kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = (int)(it % STAGES);
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1;
                    if (!mbar_wait(empty + s, ph ^ 1, g.status, abort_flag)) { ok = false; break; }
                    uint8_t* a_dst = tiles + s * kStageBytes;
                    if constexpr (PAIR) {
                        // the even block's barrier counts the bytes of both blocks' loads
                        if (pair_rank == 0) mbar_expect_tx(full + s, 2 * kStageBytes);
                        tma_load_2d_pair(a_dst, &map_a, kb * kTcBK, m0, full + s);
                        tma_load_2d_pair(a_dst + kABytes, &map_b, kb * kTcBK, n0 + (int32_t)pair_rank * (BN / 2), full + s);
                        continue;
                    }
                    mbar_expect_tx(full + s, kStageBytes);
                    if constexpr (kMnMajor) {
                        // operands stored [reduction index][M or N]: boxes of 64 reduction rows x 64 elements
#pragma unroll
                        for (int i = 0; i < kTcBM / 64; ++i)
                            tma_load_2d(a_dst + i * kMnBoxBytes, &map_a, m0 + 64 * i, kb * kTcBK, full + s);
#pragma unroll
                        for (int i = 0; i < BN / 64; ++i)
                            tma_load_2d(a_dst + kABytes + i * kMnBoxBytes, &map_b, n0 + 64 * i, kb * kTcBK, full + s);
                    } else {
                        tma_load_2d(a_dst, &map_a, kb * kTcBK, m0, full + s);
                        tma_load_2d(a_dst + kABytes, &map_b, kb * kTcBK, n0, full + s);
                    }
                }
            }
            if (*abort_flag && !(PAIR && pair_rank != 0)) {    // await (bounded) what was issued and not consumed, so nothing lands after exit
                for (int64_t i = it > STAGES ? it - STAGES : 0; i < it; ++i) {
                    const int s = (int)(i % STAGES);
                    const uint32_t ph = (uint32_t)(i / STAGES) & 1;
                    for (uint32_t w = 0; w < (1u << 20); ++w) if (mbar_try_wait(full + s, ph)) break;
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && pair_rank == 0) {        // (of a pair, the even block issues the MMAs for both)
            constexpr uint32_t idesc = make_idesc(BN, kMnMajor, kMnMajor, kTileRows);
            int64_t it = 0, lt = 0;               // k-blocks consumed, tiles done by this block
            bool ok = true;
            for (int64_t t = tile_first; t < n_tiles && ok; t += tile_stride, ++lt) {
                const int64_t z = t / per_split;
                const int32_t kb0 = (int32_t)z * g.k_blocks_per_split;
                const int32_t kb1 = min(g.k_blocks_total, kb0 + g.k_blocks_per_split);
                const int b = (int)(lt % NACC);
                const uint32_t pb = (uint32_t)(lt / NACC) & 1;
                ok = mbar_wait(acc_empty + b, pb ^ 1, g.status, abort_flag);      // drained by the epilogue
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t acc_addr = tmem_acc + (uint32_t)(b * BN);
                for (int32_t kb = kb0; kb < kb1; ++kb, ++it) {
                    const int s = (int)(it % STAGES);
                    const uint32_t ph = (uint32_t)(it / STAGES) & 1;
                    ok = mbar_wait(full + s, ph, g.status, abort_flag);
                    if (!ok) break;
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                    const uint32_t a_addr = smem_u32(tiles + s * kStageBytes);
                    if constexpr (kMnMajor) {
                        const uint64_t adesc = make_smem_desc_mn(a_addr, kMnBoxBytes);
                        const uint64_t bdesc = make_smem_desc_mn(a_addr + kABytes, kMnBoxBytes);
#pragma unroll
                        for (int k = 0; k < kTcBK / 16; ++k)      // 16 reduction rows = two 1024-byte atoms: +128 in 16-byte units
                            umma_bf16(acc_addr, adesc + 128 * k, bdesc + 128 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    } else if constexpr (PAIR) {
                        // one MMA over both blocks' shared memory (same offsets in either) and tensor memory
                        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kTcBK / 16; ++k)
                            umma_bf16_pair(acc_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    } else {
                        const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(a_addr + kABytes);
#pragma unroll
                        for (int k = 0; k < kTcBK / 16; ++k)      // 16 bf16 = 32 bytes per MMA along K: +2 in 16-byte units
                            umma_bf16(acc_addr, adesc + 2 * k, bdesc + 2 * k, idesc, (kb > kb0 || k > 0) ? 1u : 0u);
                    }
                    if constexpr (PAIR) umma_commit_pair(empty + s);      // frees the stage in both blocks
                    else umma_commit(empty + s);              // frees the stage once these MMAs have read it
                }
                if (ok) {                                     // accumulator complete (at once for an empty K range)
                    if constexpr (PAIR) umma_commit_pair(acc_full + b);
                    else umma_commit(acc_full + b);
                }
            }
        }
    } else {
        const int q = warp & 3;                           // tensor-memory lane quarter this warp may read
        const int ew = warp - 2;
        const int gi = TG == 2 ? ew >> 3 : 0;             // tile group of this warp
        const int half = (ew >> 2) % CP;                  // which part of the tile's columns this warp drains
        constexpr int kPartCols = BN / CP;
        float* warp_loss = warp_loss_all + gi * 4;
        float (*xch)[2][128] = xch_all + gi * 4;
        uint8_t* stage = stage_base + ew * kStageBytesPerWarp;      // this warp's two staging blocks
        int flip = 0;
        const CUtensorMap* rows_map = g.tma_rows ? &map_rows : nullptr;
        const bool row_owner = BN == 64 && MODE == TC_EPI_ARGMAX;
        constexpr bool kGated = MODE == TC_EPI_MASK;
        // soft-max epilogue: this warp's 32 bias values never change (its columns are the same in every tile)
        float ce_bias_lane = 0.f;
        if constexpr (BN == 64 && MODE == TC_EPI_SOFTMAX_CE)
            ce_bias_lane = (g.bias && half * 32 + lane < g.N) ? __ldg(g.bias + half * 32 + lane) : 0.f;
        // gated epilogue: the gate block of the next chunk is fetched while the current chunk is processed
        uint4 gate_next[4];
        bool gate_have = false;
        [[maybe_unused]] auto gate_prefetch = [&](int64_t tile, int c0) {
            gate_have = false;
            if (tile >= n_tiles) return;
            const int64_t rem = tile % per_split;
            const int64_t r0 = (rem % n_m) * kTcBM + q * 32, cc0 = (rem / n_m) * BN + c0;
            if (!rows_map || r0 >= g.M || cc0 + 32 > g.N || (g.ld_mask & 7) != 0 || !aligned16(g.mask)) return;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int line = (lane >> 2) + 8 * i, piece = lane & 3;
                gate_next[i] = make_uint4(0u, 0u, 0u, 0u);
                if (r0 + line < g.M)
                    gate_next[i] = __ldg(reinterpret_cast<const uint4*>(g.mask + (r0 + line) * g.ld_mask + cc0 + piece * 8));
            }
            gate_have = true;
        };
        if constexpr (kGated) gate_prefetch(tile_first + (int64_t)gi * tile_stride, half * kPartCols);
        int64_t lt = gi;
        for (int64_t t = tile_first + (int64_t)gi * tile_stride; t < n_tiles && !(row_owner && half == 1);
             t += (int64_t)TG * tile_stride, lt += TG) {
            const int64_t z = t / per_split, rem = t % per_split;
            const int64_t mt = rem % n_m;
            const int64_t m0 = mt * kTileRows + (int64_t)pair_rank * kTcBM, n0 = (rem / n_m) * BN;
            const int32_t kb0 = (int32_t)z * g.k_blocks_per_split;
            const int32_t n_kb = min(g.k_blocks_total, kb0 + g.k_blocks_per_split) - kb0;
            const int b = (int)(lt % NACC);
            const uint32_t pb = (uint32_t)(lt / NACC) & 1;
            const uint32_t acc_addr = tmem_acc + (uint32_t)(b * BN);
            const int64_t row0 = m0 + q * 32;
            const int64_t row = row0 + lane;
            int32_t ce_label = -1;          // soft-max epilogue: fetched before the wait so that its latency is hidden
            if constexpr (BN == 64 && MODE == TC_EPI_SOFTMAX_CE)
                ce_label = (row < g.M && row < g.n_train && g.y) ? g.y[row] : -1;
            const bool ok = mbar_wait(acc_full + b, pb, g.status, abort_flag);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            if (!ok) break;
            if constexpr (BN == 64 && MODE == TC_EPI_SOFTMAX_CE) {
                // Two threads share a row of logits: warp q takes columns [0, 32), warp q + 4 columns
                // [32, 64); row maximum, sum and the label's logit are exchanged through shared memory.
                const int cb = half * 32;
                const int slot = q * 32 + lane;                          // this row's slot in the exchange arrays
                float v[32];
                {
                    uint32_t r[32];
                    if (n_kb > 0) { tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16) + (uint32_t)cb, r); tmem_ld_wait(r); }
                    else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = 0u;
                    }
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        v[j] = cb + j < g.N ? __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, ce_bias_lane, j) : -INFINITY;
                }
                const bool is_eval = row >= g.n_train;
                const bool live = row < g.M && !is_eval;
                const int32_t yi = live ? ce_label : -1;
                float mx = v[0];
                int best = 0;
#pragma unroll
                for (int j = 1; j < 32; ++j) if (v[j] > mx) { mx = v[j]; best = j; }      // strict: lowest index on ties
                xch[0][half][slot] = mx;
                xch[1][half][slot] = __int_as_float(cb + best);
                asm volatile("bar.sync %0, 256;" ::"r"(1 + gi) : "memory");
                const float m0v = xch[0][0][slot], m1v = xch[0][1][slot];
                if (g.n_train < g.M && m0 + kTcBM > g.n_train && half == 0) {
                    // evaluation rows in this tile: arg-max over both halves (the lower half wins ties)
                    const int arg = m1v > m0v ? __float_as_int(xch[1][1][slot]) : __float_as_int(xch[1][0][slot]);
                    const bool hit = is_eval && row < g.M && arg == g.y_eval[row - g.n_train];
                    const unsigned hits = __ballot_sync(0xffffffffu, hit);
                    if (lane == 0 && hits) atomicAdd(g.correct, (unsigned long long)__popc(hits));
                }
                mx = fmaxf(m0v, m1v);
                float den = 0.f, ly = 0.f;
#pragma unroll
                for (int j = 0; j < 32; ++j) {
                    ly = cb + j == yi ? v[j] : ly;
                    v[j] = cb + j < g.N ? __expf(v[j] - mx) : 0.f;
                    den += v[j];
                }
                xch[2][half][slot] = den;
                xch[3][half][slot] = ly;
                asm volatile("bar.sync %0, 256;" ::"r"(1 + gi) : "memory");
                den = xch[2][0][slot] + xch[2][1][slot];
                ly = xch[3][0][slot] + xch[3][1][slot];
                const float scale = g.inv_rows / den;
#pragma unroll
                for (int j = 0; j < 32; ++j) v[j] = cb + j < g.N ? (v[j] * scale - (cb + j == yi ? g.inv_rows : 0.f)) : 0.f;
                // dL row-major (clipped to the trained rows, padding columns zero)
                if (rows_map && g.out_bf16 && row0 < g.n_train && cb < g.ld_bf16)
                    store_block(v, stage, lane, cb, g.N, row0, g.n_train, g.out_bf16, g.ld_bf16, rows_map);
                if (!rows_map && live && g.out_bf16) {       // this thread's columns, 16 bytes at a time
                    __nv_bfloat16* dst = g.out_bf16 + row * g.ld_bf16 + cb;
#pragma unroll
                    for (int c = 0; c < 32; c += 8) {
                        if (cb + c >= g.ld_bf16) break;
                        __nv_bfloat162 p0 = __floats2bfloat162_rn(v[c], v[c + 1]), p1 = __floats2bfloat162_rn(v[c + 2], v[c + 3]);
                        __nv_bfloat162 p2 = __floats2bfloat162_rn(v[c + 4], v[c + 5]), p3 = __floats2bfloat162_rn(v[c + 6], v[c + 7]);
                        uint4 pk;
                        pk.x = *reinterpret_cast<uint32_t*>(&p0); pk.y = *reinterpret_cast<uint32_t*>(&p1);
                        pk.z = *reinterpret_cast<uint32_t*>(&p2); pk.w = *reinterpret_cast<uint32_t*>(&p3);
                        *reinterpret_cast<uint4*>(dst + c) = pk;
                    }
                }
                if (half == 0) {
                    float loss = live ? (mx + __logf(den)) - ly : 0.f;
                    loss = warp_sum(loss);
                    if (lane == 0) warp_loss[q] = loss;
                }
                asm volatile("bar.sync %0, 256;" ::"r"(1 + gi) : "memory");
                if ((ew & 7) == 0 && lane == 0 && g.loss_partial)
                    g.loss_partial[mt] = ((warp_loss[0] + warp_loss[1]) + warp_loss[2]) + warp_loss[3];
                // (the exchange arrays and warp_loss are next written after the following tile's first
                //  barrier-protected phase: every warp passes two more barriers before reusing them)
            } else if constexpr (BN == 64 && MODE == TC_EPI_ARGMAX) {
                // one thread owns the whole row of logits (four of the eight warps take part)
                float v[64];
                if (ok) {
                    uint32_t ra[32], rb[32];
                    if (n_kb > 0) {       // both halves of the row in flight together
                        tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16), ra);
                        tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16) + 32u, rb);
                        tmem_ld_wait(ra);
                        tmem_ld_wait(rb);
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) { ra[j] = 0u; rb[j] = 0u; }
                    }
                    const float bias_a = (g.bias && lane < g.N) ? __ldg(g.bias + lane) : 0.f;
                    const float bias_b = (g.bias && 32 + lane < g.N) ? __ldg(g.bias + 32 + lane) : 0.f;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        v[j] = j < g.N ? __uint_as_float(ra[j]) + __shfl_sync(0xffffffffu, bias_a, j) : -INFINITY;
                        v[32 + j] = 32 + j < g.N ? __uint_as_float(rb[j]) + __shfl_sync(0xffffffffu, bias_b, j) : -INFINITY;
                    }
                } else {
#pragma unroll
                    for (int c = 0; c < 64; ++c) v[c] = 0.f;
                }
                const bool live = ok && row < g.M;
                const int32_t yi = (live && g.y) ? g.y[row] : -1;
                int best = 0;
                float bv = v[0];
#pragma unroll
                for (int c = 1; c < 64; ++c) if (v[c] > bv) { bv = v[c]; best = c; }   // strict: lowest index wins ties
                if (live) {
                    if (g.pred) g.pred[row] = best;
                    if (g.out_f32) {
#pragma unroll
                        for (int c = 0; c < 64; ++c) if (c < g.N) g.out_f32[row * g.ld_f32 + c] = v[c];
                    }
                }
                if (g.correct) {
                    const unsigned hits = __ballot_sync(0xffffffffu, live && best == yi);
                    if (lane == 0 && hits) atomicAdd(g.correct, (unsigned long long)__popc(hits));
                }
            } else if (ok) {
                // the accumulator load of chunk c + 1 is in flight while chunk c is processed (gated modes
                // spend those registers on the gate block of chunk c + 1 instead)
                [[maybe_unused]] uint32_t nxt[32];
                const int c_begin = half * kPartCols, c_end = c_begin + kPartCols;
                if constexpr (!kGated) {
                    if (n_kb > 0) tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16) + (uint32_t)c_begin, nxt);
                    else {
#pragma unroll
                        for (int j = 0; j < 32; ++j) nxt[j] = 0u;
                    }
                }
#pragma unroll 1
                for (int c0 = c_begin; c0 < c_end; c0 += 32) {
                    uint32_t r[32];
                    if constexpr (!kGated) {
                        if (n_kb > 0) tmem_ld_wait(nxt);
#pragma unroll
                        for (int j = 0; j < 32; ++j) r[j] = nxt[j];
                        if (n_kb > 0 && c0 + 32 < c_end)
                            tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16) + (uint32_t)(c0 + 32), nxt);
                    } else {
                        if (n_kb > 0) tmem_ld_issue(acc_addr + ((uint32_t)(q * 32) << 16) + (uint32_t)c0, r);
                        else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) r[j] = 0u;
                        }
                    }
                    const int64_t col0 = n0 + c0;
                    if (col0 >= g.N) {
                        if constexpr (kGated) { if (n_kb > 0) tmem_ld_wait(r); }
                        continue;
                    }
                    if constexpr (MODE == TC_EPI_PARTIAL) {
                        if (row >= g.M) continue;
                        float* dst = g.partial + ((int64_t)z * g.M + row) * g.N + col0;
                        if (col0 + 32 <= g.N && (g.N & 3) == 0 && aligned16(g.partial)) {
#pragma unroll
                            for (int j = 0; j < 32; j += 4)
                                *reinterpret_cast<float4*>(dst + j) = make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                                                                                  __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
                        } else {
#pragma unroll
                            for (int j = 0; j < 32; ++j) if (col0 + j < g.N) dst[j] = __uint_as_float(r[j]);
                        }
                    } else if constexpr (MODE == TC_EPI_MASK) {
                        const CUtensorMap* out_map = rows_map;
                        const bool gate_runs = col0 + 32 <= g.N && (g.ld_mask & 7) == 0 && aligned16(g.mask);
                        // this chunk's gate block (if it was fetched ahead), then the fetch for the next chunk
                        uint4 gate_cur[4];
                        const bool have_gate = gate_have;
#pragma unroll
                        for (int i = 0; i < 4; ++i) gate_cur[i] = gate_next[i];
                        if (c0 + 32 < c_end) gate_prefetch(t, c0 + 32);
                        else gate_prefetch(t + (int64_t)TG * tile_stride, c_begin);
                        if (gate_runs && out_map) {
                            // the two staging blocks take turns: the bulk store issued two chunks ago has read this one
                            flip ^= 1;
                            uint8_t* blk = stage + flip * kStageBlockBytes;
                            if (lane == 0) bulk_wait_read_but_one();
                            __syncwarp();
                            if (have_gate) {      // 64-byte runs from global memory, one row per lane out of the block
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const int line = (lane >> 2) + 8 * i, piece = lane & 3;
                                    *reinterpret_cast<uint4*>(blk + line * 64 + stage_piece(line, piece) * 16) = gate_cur[i];
                                }
                                __syncwarp();
                            } else {
                                stage_block_from_global(g.mask, g.ld_mask, col0, row0, g.M, blk, lane);
                            }
                            if (n_kb > 0) tmem_ld_wait(r);
                            if (g.gate_scale != 1.f) {      // (dropout: the kept units' factor)
#pragma unroll
                                for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * g.gate_scale);
                            }
                            uint32_t p[16];
#pragma unroll
                            for (int qd = 0; qd < 4; ++qd) {
                                const uint4 mk = *reinterpret_cast<const uint4*>(blk + lane * 64 + stage_piece(lane, qd) * 16);
                                const __nv_bfloat16* mv = reinterpret_cast<const __nv_bfloat16*>(&mk);
#pragma unroll
                                for (int i = 0; i < 4; ++i) {
                                    const float lo = __bfloat162float(mv[2 * i]) > 0.f ? __uint_as_float(r[8 * qd + 2 * i]) : 0.f;
                                    const float hi = __bfloat162float(mv[2 * i + 1]) > 0.f ? __uint_as_float(r[8 * qd + 2 * i + 1]) : 0.f;
                                    __nv_bfloat162 b2 = __floats2bfloat162_rn(lo, hi);
                                    p[4 * qd + i] = *reinterpret_cast<uint32_t*>(&b2);
                                }
                            }
                            __syncwarp();         // every lane has read its gate row: the block may take the output
                            if (row0 < g.M)
                                store_block_packed(p, stage, lane, col0, row0, rows_map, blk);
                        } else {
                            if (n_kb > 0) tmem_ld_wait(r);
                            float v[32];
                            if (row < g.M) {
                                const __nv_bfloat16* mrow = g.mask + row * g.ld_mask + col0;
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    v[j] = (col0 + j < g.N && __bfloat162float(mrow[j]) > 0.f) ? __uint_as_float(r[j]) * g.gate_scale : 0.f;
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) v[j] = 0.f;
                            }
                            if (row0 < g.M)
                                store_block(v, stage, lane, col0, g.N, row0, g.M, g.out_bf16, g.ld_bf16, rows_map);
                        }
                    } else {
                        float v[32];
                        // one coalesced bias load per chunk, handed round by shuffles (32 same-address loads per
                        // thread cost more than the rest of the epilogue together)
                        const float bias_lane = (g.bias && col0 + lane < g.N) ? __ldg(g.bias + col0 + lane) : 0.f;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            float x = __uint_as_float(r[j]) + __shfl_sync(0xffffffffu, bias_lane, j);
                            if (g.relu) x = fmaxf(x, 0.f);
                            v[j] = x;
                        }
                        if constexpr (MODE == TC_EPI_BIAS_DROP) {
                            if (row < g.drop_rows) {      // training rows only; col0 is a multiple of 32
                                const uint32_t update = g.drop_step_dev ? (uint32_t)__ldg(g.drop_step_dev) + 1u : g.drop_step;
#pragma unroll
                                for (int j4 = 0; j4 < 8; ++j4) {
                                    uint32_t w[4];
                                    philox4x32_10((uint32_t)row, (uint32_t)((col0 >> 2) + j4), update, 0u, g.drop_key0,
                                                  g.drop_key1, w);
#pragma unroll
                                    for (int t = 0; t < 4; ++t)
                                        v[4 * j4 + t] = w[t] >= g.drop_thresh ? v[4 * j4 + t] * g.drop_scale : 0.f;
                                }
                            }
                        }
                        if (g.relu_bits && row < g.M) {      // one bit per unit: is the value that goes out positive?
                            uint32_t word = 0u;
#pragma unroll
                            for (int j = 0; j < 32; ++j) word |= (v[j] > 0.f ? 1u : 0u) << j;
                            g.relu_bits[row * g.ld_bits + (col0 >> 5)] = word;
                        }
                        if (g.out_f32 && row < g.M) {
                            float* dst = g.out_f32 + row * g.ld_f32 + col0;
                            if (col0 + 32 <= g.N && (g.ld_f32 & 3) == 0 && aligned16(g.out_f32)) {
#pragma unroll
                                for (int j = 0; j < 32; j += 4)
                                    *reinterpret_cast<float4*>(dst + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                            } else {
#pragma unroll
                                for (int j = 0; j < 32; ++j) if (col0 + j < g.N) dst[j] = v[j];
                            }
                        }
                        if (row0 < g.M && g.out_bf16)
                            store_block(v, stage, lane, col0, g.N, row0, g.M, g.out_bf16, g.ld_bf16, rows_map);
                        // the column of ones behind the last output column (it makes the bias gradient one more
                        // row of the weight-gradient product that reads this matrix)
                        if (g.out_bf16 && g.ones_col && col0 == 0 && row < g.M)
                            g.out_bf16[row * g.ld_bf16 + g.N] = __float2bfloat16_rn(1.0f);
                    }
                }
            }
            // hand the accumulator back to the MMA thread
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
                if constexpr (PAIR) mbar_arrive_even_block(acc_empty + b);      // the MMA thread lives in the even block
                else asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(acc_empty + b)) : "memory");
            }
        }
        if (lane == 0) bulk_wait_all();       // this thread's bulk stores have reached global memory
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if constexpr (PAIR) cluster_sync_all();   // neither block leaves while the other may still signal it or use its tensor memory
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if constexpr (PAIR) asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(NACC * BN));
        else asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(NACC * BN));
    }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Tensor map of a 2-D bf16 matrix [rows x cols], cols contiguous, row stride ld elements, for boxes of
// [box_rows x box_cols] with the given swizzle width in bytes (128 or 64; box_cols * 2 must equal it).
bool tc_make_map_2d(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows, int box_cols,
                    int swizzle_bytes, bool l2_promote) {
    EncodeTiledFn fn = encode_fn();
    if (!fn || !base || rows <= 0 || cols <= 0 || !aligned_to(base, 16) || ld % 8 != 0 || ld < cols) return false;
    if (rows > INT32_MAX || cols > INT32_MAX || box_cols * 2 != swizzle_bytes || box_rows < 1 || box_rows > 256) return false;
    cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    cuuint32_t box[2] = {(cuuint32_t)box_cols, (cuuint32_t)box_rows};
    cuuint32_t estr[2] = {1, 1};
    return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B,
              l2_promote ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Operand tile loads: box = [box_rows x 64], 128-byte swizzle.
static bool make_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows) {
    return tc_make_map_2d(map, base, rows, cols, ld, box_rows, kTcBK, 128, true);
}

// Tensor map of a bf16 output matrix [rows x cols] (row stride ld elements) for [32 x 32] stores with the
// 64-byte swizzle of the staging blocks.  Returns false where the layout does not allow one.
static bool make_store_map(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld) {
    return tc_make_map_2d(map, base, rows, cols, ld, 32, 32, 64, false);
}

template <int BN, int STAGES, int MODE, int EW>
static int launch_tc_mode(const TcGemm& t, const CUtensorMap& ma, const CUtensorMap& mb, cudaStream_t st) {
    // stage ring + alignment slack + barrier area + staging blocks (+ the soft-max exchange arrays)
    constexpr size_t smem = (size_t)STAGES * (kTcBM * kTcBK * 2 + BN * kTcBK * 2) + 1024 + 1024 + EW * kStageBytesPerWarp +
                            (BN == 64 ? (EW / 8) * 4 * 2 * 128 * 4 : 0);
    static_assert(smem <= 227 * 1024, "shared memory budget");
    // (the attribute belongs to the current device's copy of the kernel: set on every launch, which is cheap,
    //  instead of remembered per process)
    if (cudaFuncSetAttribute(tc_gemm_kernel<BN, STAGES, MODE, EW>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
        cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    TcKernelArgs g{};
    g.M = t.M; g.N = t.N;
    g.k_blocks_total = (int32_t)((t.K + kTcBK - 1) / kTcBK);
    const int splits = t.mode == TC_EPI_PARTIAL ? (t.splits > 0 ? t.splits : 1) : 1;
    g.k_blocks_per_split = (g.k_blocks_total + splits - 1) / splits;
    g.splits = splits;
    g.mode = t.mode; g.relu = t.relu; g.bias = t.bias;
    g.out_f32 = t.out_f32; g.ld_f32 = t.ld_f32; g.out_bf16 = t.out_bf16; g.ld_bf16 = t.ld_bf16;
    g.ones_col = (t.ones_col && t.out_bf16 && t.ld_bf16 > t.N) ? 1 : 0;
    g.relu_bits = t.relu_bits; g.ld_bits = t.ld_bits;
    g.mask = t.mask; g.ld_mask = t.ld_mask;
    g.gate_scale = t.gate_scale != 0.f ? t.gate_scale : 1.f;
    g.drop_thresh = t.drop_thresh; g.drop_step = t.drop_step; g.drop_key0 = t.drop_key[0]; g.drop_key1 = t.drop_key[1];
    g.drop_scale = t.drop_scale; g.drop_rows = t.drop_rows; g.drop_step_dev = t.drop_step_dev;
    g.partial = t.partial; g.status = t.status;
    g.y = t.y; g.inv_rows = t.inv_rows; g.loss_partial = t.loss_partial; g.pred = t.pred; g.correct = t.correct;
    g.n_train = (t.mode == TC_EPI_SOFTMAX_CE && t.eval_from > 0 && t.eval_from < t.M) ? t.eval_from : t.M;
    g.y_eval = t.y_eval;
    // bf16 outputs leave through bulk tensor stores where their layout allows it
    CUtensorMap m_rows;
    memset(&m_rows, 0, sizeof(m_rows));
    const bool ce = t.mode == TC_EPI_SOFTMAX_CE;
    const bool bias_like = t.mode == TC_EPI_BIAS || t.mode == TC_EPI_BIAS_DROP;
    // (with a column of ones behind an output whose width is not a whole number of 16-byte pieces, the store of
    //  the last piece and the plain store of the ones would meet in one piece: such shapes take plain stores)
    if (t.out_bf16 && (bias_like || t.mode == TC_EPI_MASK || ce) && !(g.ones_col && t.N % 8 != 0))
        g.tma_rows = make_store_map(&m_rows, t.out_bf16, ce ? g.n_train : t.M, ce ? t.ld_bf16 : t.N, t.ld_bf16) ? 1 : 0;
    const int64_t n_tiles = ((t.M + kTcBM - 1) / kTcBM) * ((t.N + BN - 1) / BN) * splits;
    const int n_sm = sm_count();
    if (n_sm <= 0) return RETEXO_ERR_CUDA;
    const unsigned grid = (unsigned)(n_tiles < n_sm ? n_tiles : n_sm);      // one persistent block per SM
    OverlapLaunch ol(dim3(grid), dim3(64 + 32 * EW), smem, st);
    if (cudaLaunchKernelEx(&ol.cfg, tc_gemm_kernel<BN, STAGES, MODE, EW>, ma, mb, m_rows, g) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

// The forward products in pairs of thread blocks (clusters of two): 256-row tiles, each block loading its own
// rows of A and half of the B tile.  `t`'s epilogue arguments are those of launch_tc_mode.
template <int MODE>
static int launch_tc_pair(const TcGemm& t, cudaStream_t st) {
    constexpr int BN = 256, EW = 8, STAGES = 6;
    constexpr size_t smem = (size_t)STAGES * (kTcBM * kTcBK * 2 + (BN / 2) * kTcBK * 2) + 1024 + 1024 + EW * kStageBytesPerWarp;
    static_assert(smem <= 227 * 1024, "shared memory budget");
    auto kernel = tc_gemm_kernel<BN, STAGES, MODE, EW, true>;
    if (cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    CUtensorMap ma, mb, m_rows;
    memset(&m_rows, 0, sizeof(m_rows));
    if (!make_map(&ma, t.A, t.M, t.K, t.lda, kTcBM)) return RETEXO_ERR_CUDA;
    if (!make_map(&mb, t.B, t.N, t.K, t.ldb, BN / 2)) return RETEXO_ERR_CUDA;
    TcKernelArgs g{};
    g.M = t.M; g.N = t.N;
    g.k_blocks_total = (int32_t)((t.K + kTcBK - 1) / kTcBK);
    g.k_blocks_per_split = g.k_blocks_total;
    g.splits = 1;
    g.mode = t.mode; g.relu = t.relu; g.bias = t.bias;
    g.out_f32 = t.out_f32; g.ld_f32 = t.ld_f32; g.out_bf16 = t.out_bf16; g.ld_bf16 = t.ld_bf16;
    g.ones_col = (t.ones_col && t.out_bf16 && t.ld_bf16 > t.N) ? 1 : 0;
    g.relu_bits = t.relu_bits; g.ld_bits = t.ld_bits;
    g.drop_thresh = t.drop_thresh; g.drop_step = t.drop_step; g.drop_key0 = t.drop_key[0]; g.drop_key1 = t.drop_key[1];
    g.drop_scale = t.drop_scale; g.drop_rows = t.drop_rows; g.drop_step_dev = t.drop_step_dev;
    g.status = t.status; g.n_train = t.M;
    if (t.out_bf16 && !(g.ones_col && t.N % 8 != 0)) g.tma_rows = make_store_map(&m_rows, t.out_bf16, t.M, t.N, t.ld_bf16) ? 1 : 0;
    const int64_t n_tiles = ((t.M + 2 * kTcBM - 1) / (2 * kTcBM)) * ((t.N + BN - 1) / BN);
    OverlapLaunch ol(dim3(2), dim3(64 + 32 * EW), smem, st, 2);
    cudaLaunchConfig_t& cfg = ol.cfg;
    // as many pairs as can be resident at once (persistent blocks), found once per device
    static int max_pairs[64] = {};
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return RETEXO_ERR_CUDA;
    if (max_pairs[dev] == 0) {
        cfg.gridDim = dim3(2 * (unsigned)sm_count(), 1, 1);
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kernel, &cfg) != cudaSuccess || n <= 0) {
            (void)cudaGetLastError();
            return RETEXO_ERR_UNSUPPORTED;
        }
        max_pairs[dev] = n;
    }
    const int64_t pairs = n_tiles < max_pairs[dev] ? n_tiles : max_pairs[dev];
    cfg.gridDim = dim3((unsigned)(2 * pairs), 1, 1);
    if (cudaLaunchKernelEx(&cfg, kernel, ma, mb, m_rows, g) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

template <int BN, int STAGES, int EW>
static int launch_tc(const TcGemm& t, const CUtensorMap& ma, const CUtensorMap& mb, cudaStream_t st) {
    switch (t.mode) {
        case TC_EPI_BIAS: return launch_tc_mode<BN, STAGES, TC_EPI_BIAS, EW>(t, ma, mb, st);
        case TC_EPI_BIAS_DROP: return launch_tc_mode<BN, STAGES, TC_EPI_BIAS_DROP, EW>(t, ma, mb, st);
        case TC_EPI_PARTIAL: return launch_tc_mode<BN, STAGES, TC_EPI_PARTIAL, EW>(t, ma, mb, st);
        case TC_EPI_MASK: return launch_tc_mode<BN, STAGES, TC_EPI_MASK, EW>(t, ma, mb, st);
        case TC_EPI_SOFTMAX_CE:
            if constexpr (BN == 64) return launch_tc_mode<BN, STAGES, TC_EPI_SOFTMAX_CE, EW>(t, ma, mb, st);
            break;
        case TC_EPI_ARGMAX:
            if constexpr (BN == 64) return launch_tc_mode<BN, STAGES, TC_EPI_ARGMAX, EW>(t, ma, mb, st);
            break;
        default: break;
    }
    return RETEXO_ERR_UNSUPPORTED;
}

bool tc_gemm_supported(const TcGemm& t) {
    if (t.M <= 0 || t.N <= 0 || t.K <= 0) return false;
    if (t.mode == TC_EPI_MASK && (!t.mask || !t.out_bf16)) return false;
    if (t.mode == TC_EPI_PARTIAL && !t.partial) return false;
    if ((t.mode == TC_EPI_SOFTMAX_CE || t.mode == TC_EPI_ARGMAX) && t.N > 64) return false;
    if (t.mode == TC_EPI_SOFTMAX_CE && (!t.y || (t.out_bf16 && (t.ld_bf16 % 8 != 0 || t.ld_bf16 > 64)))) return false;
    if (!aligned_to(t.A, 16) || !aligned_to(t.B, 16) || t.lda % 8 != 0 || t.ldb % 8 != 0) return false;
    if (t.M > INT32_MAX || t.N > INT32_MAX || t.K > INT32_MAX - 64) return false;
    if ((t.M + kTcBM - 1) / kTcBM > 2147483647LL || (t.N + 63) / 64 > 65535) return false;
    return encode_fn() != nullptr;
}

int tc_gemm_launch(const TcGemm& t, cudaStream_t st) {
    if (!tc_gemm_supported(t)) return RETEXO_ERR_UNSUPPORTED;
    int bn = t.N > 128 ? 256 : (t.N > 64 ? 128 : 64);
    // the gated products have a short reduction and a heavy epilogue: tiles of 128 columns put sixteen
    // epilogue warps on them (measured: the 256 x 153757 x 41 product itself is level with 256-column
    // tiles, the whole training iteration 1 % shorter)
    if (t.mode == TC_EPI_MASK && bn == 256) bn = 128;
    // wide forward products over many rows go to pairs of thread blocks: the B tile (the weights) is then
    // fetched once per 256 rows, which is what bounds these products on the L2 -> SM path
    if (bn == 256 && t.M >= 4096 && (t.mode == TC_EPI_BIAS || t.mode == TC_EPI_BIAS_DROP)) {
        const int rc = t.mode == TC_EPI_BIAS ? launch_tc_pair<TC_EPI_BIAS>(t, st) : launch_tc_pair<TC_EPI_BIAS_DROP>(t, st);
        if (rc != RETEXO_ERR_UNSUPPORTED) return rc;
    }
    CUtensorMap ma, mb;
    if (t.mode == TC_EPI_PARTIAL) {      // A [K x M], B [K x N] as they lie in memory: boxes of 64 reduction rows x 64 elements
        if (!make_map(&ma, t.A, t.K, t.M, t.lda, kTcBK)) return RETEXO_ERR_CUDA;
        if (!make_map(&mb, t.B, t.K, t.N, t.ldb, kTcBK)) return RETEXO_ERR_CUDA;
    } else {
        if (!make_map(&ma, t.A, t.M, t.K, t.lda, kTcBM)) return RETEXO_ERR_CUDA;
        if (!make_map(&mb, t.B, t.N, t.K, t.ldb, bn)) return RETEXO_ERR_CUDA;
    }
    if (bn == 256) return launch_tc<256, TC256_STAGES, TC256_EW>(t, ma, mb, st);
    if (bn == 128) return launch_tc<128, TC128_STAGES, TC128_EW>(t, ma, mb, st);
    return launch_tc<64, TC64_STAGES, TC64_EW>(t, ma, mb, st);
}

}  // namespace retexo
