// Kernels of the per-node model (Section 3.1) beside its tensor-core products: batch packing and the fused
// gradient-reduce + optimiser update.
#pragma once
#include "common.cuh"
#include "launch_overlap.cuh"

namespace retexo {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------- packing
// dst[i][c] = bf16(src[idx ? idx[i] : i][c]); dst_t[c][i] likewise.  Padding
// columns of both outputs are written as zero.  With ones, dst gets one more
// column (index dim) and dst_t one more row (index dim) holding 1 for every
// batch row: the all-ones vector that makes the bias gradient one more output
// row of the weight-gradient product.
template <bool SRC_BF16>
__global__ void __launch_bounds__(256) pack_rows_kernel(const void* __restrict__ src, int64_t ld_src, int32_t dim,
                                                        const int32_t* __restrict__ idx, int64_t n_rows,
                                                        bf16* __restrict__ dst, int64_t ld_dst,
                                                        bf16* __restrict__ dst_t, int64_t ld_t, int ones) {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;     // 32 x 8
    const int64_t r0 = blockIdx.x * 32ll;
    const int64_t c0 = blockIdx.y * 32ll;
    for (int i = ty; i < 32; i += 8) {
        const int64_t r = r0 + i, c = c0 + tx;
        float v = 0.f;
        if (r < n_rows && c < dim) {
            const int64_t sr = idx ? idx[r] : r;
            v = SRC_BF16 ? bf16_to_f32(static_cast<const bf16*>(src)[sr * ld_src + c])
                         : static_cast<const float*>(src)[sr * ld_src + c];
        }
        tile[i][tx] = v;
        if (dst && r < n_rows && c < ld_dst) dst[r * ld_dst + c] = f32_to_bf16((ones && c == dim) ? 1.0f : v);
    }
    if (!dst_t) return;
    __syncthreads();
    for (int i = ty; i < 32; i += 8) {
        const int64_t c = c0 + i, r = r0 + tx;
        if (c < dim && r < ld_t) dst_t[c * ld_t + r] = f32_to_bf16(tile[tx][i]);
    }
    if (ones && blockIdx.y == 0 && ty == 0) {
        const int64_t r = r0 + tx;
        if (r < ld_t) dst_t[(int64_t)dim * ld_t + r] = f32_to_bf16(r < n_rows ? 1.0f : 0.0f);
    }
}

// ---------------------------------------------------------------- optimiser
struct GradSeg {
    int64_t size;              // parameters in this segment
    const float* partial;      // [count x size], summed in index order
    int64_t count;
};
struct UpdateArgs {
    GradSeg seg[3];            // [W1 | b1], (hidden > 0) [W2 | b2] and (normalisation) [gamma | beta], each laid out like theta
    // batch normalisation (optional): [r_mean | r_var] behind [gamma | beta] in theta are state, not parameters:
    // r <- (1 - bn_momentum) r + bn_momentum s with s the batch's mean / its variance x bn_unbias (bn_batch holds
    // mean | biased variance); their gradient entries are 0 and the optimiser's moments stay untouched
    const float* bn_batch; float bn_momentum, bn_unbias;
    int n_seg;
    float* theta;
    float* m;
    float* v;
    float* grad_out;           // may be null
    int optimizer;
    float lr, beta1, beta2, eps, corr1, corr2;     // corr = 1 - beta^step
    const float* loss_partial; int64_t n_loss; float inv_rows; float* loss_out;
    const int32_t* status;     // non-zero: a kernel of this step gave up on a bounded wait -> loss = NaN
    int32_t* status_out;       // (optional) receives *status
    // bf16 copies of the updated weights in the orientations the next products read (optional)
    bf16* w1t16; int64_t ld_k;       // W1^T [out1 x ld_k]
    bf16* w1r16; int64_t ld_o1;      // W1   [d_in x ld_o1]
    bf16* w2t16; int64_t ld_h;       // W2^T [n_classes x ld_h]
    bf16* w2p16; int64_t ld_dl;      // W2   [hidden x ld_dl]
    int32_t d_in, out1, hidden, n_classes;
    // keep-the-best snapshot of theta as it is before this update (optional, see EvalTail)
    unsigned long long* snap_cur; unsigned long long* snap_best; int32_t* snap_have;
    float* theta_best;
    int32_t* snap_decision;          // (optional) receives whether this launch copied theta to theta_best
    // bookkeeping of the validation count by the last block to finish (optional, see EvalTail)
    unsigned long long* done; int32_t rec_iter; int32_t* rec_best_iter; unsigned long long* rec_history_slot;
    // iteration state on the device (optional, see DeviceIter; needs `done`): with s = *step_dev updates applied
    // so far, this launch applies update s + 1, writes its loss to loss_base[s], books the validation count
    // as iteration s's into history_base[s - 1], and its last block leaves *step_dev = s + 1
    unsigned long long* step_dev; float* loss_base; unsigned long long* history_base;
};

// base^e for a whole exponent by repeated squaring (a handful of double multiplications: the library
// power function costs microseconds on a part with few double-precision units).
__host__ __device__ __forceinline__ double pow_whole(double base, unsigned long long e) {
    double r = 1.0;
    while (e) {
        if (e & 1ull) r *= base;
        base *= base;
        e >>= 1;
    }
    return r;
}

// Sum of one parameter's split-K partials in index order.  BATCH loads are in flight before the first addition
// waits for one (warps issue in order, so a loop of small batches would pay the memory latency once per batch;
// a larger batch costs registers, and with them the blocks an SM holds at once: the launcher picks 16 where
// that covers the largest layer's partials in one go, else 32).
template <int BATCH>
__device__ __forceinline__ float sum_partials(const float* __restrict__ src, int32_t count, int64_t stride) {
    float g = 0.f;
    for (int32_t z = 0; z < count; z += BATCH) {
        float x[BATCH];
        const float* s = src;
#pragma unroll
        for (int i = 0; i < BATCH; ++i) {
            x[i] = z + i < count ? __ldcs(s) : 0.f;      // read once: streamed
            s += stride;
        }
#pragma unroll
        for (int i = 0; i < BATCH; ++i) g += x[i];
        src = s;
    }
    return g;
}

// Sums each parameter's split-K partials in index order, applies the optimiser, and refreshes
// the bf16 weight copies.  Block 0 also reduces the loss (fixed order: per-lane strided sums,
// then a shuffle tree).  With u.done set, the last block to arrive does the validation bookkeeping.
// The kernel sits between two products on the critical path of an iteration and moves little
// data, so it is laid out for latency: every load that depends on nothing (the iteration state,
// the partials, the parameter and its moments) is issued before anything waits.
template <int BATCH>
__global__ void __launch_bounds__(256, BATCH == 16 ? 4 : 2) reduce_update_kernel(UpdateArgs u) {
    // A block owns a 16 x 16 tile of one segment's (inputs + 1) x outputs matrix (the last row is the
    // bias): 64-byte runs of each partial on the way in, and whole 32-byte sectors of the transposed
    // bf16 copy on the way out (a 2-byte store per parameter into a row of its own has every store
    // read-modify-write a sector that fifteen other blocks are writing too).
    const int32_t rows0 = u.d_in + 1, cols0 = u.out1;
    const int32_t tc0 = (cols0 + 15) >> 4, tiles0 = ((rows0 + 15) >> 4) * tc0;
    const int32_t tiles1 = u.n_seg > 1 ? ((u.hidden + 1 + 15) >> 4) * ((u.n_classes + 15) >> 4) : 0;
    // (the third segment, a layer norm's [gamma ; beta], is a 2 x hidden matrix: one row of tiles)
    const int sidx = (int32_t)blockIdx.x < tiles0 ? 0 : ((int32_t)blockIdx.x < tiles0 + tiles1 ? 1 : 2);
    const int32_t rows = sidx == 0 ? rows0 : (sidx == 1 ? u.hidden + 1 : (u.bn_batch ? 4 : 2)), cols = sidx == 0 ? cols0 : (sidx == 1 ? u.n_classes : u.hidden);
    const int32_t tcs = (cols + 15) >> 4;
    const int32_t tile = (int32_t)blockIdx.x - (sidx == 0 ? 0 : (sidx == 1 ? tiles0 : tiles0 + tiles1));
    const int32_t row0 = (tile / tcs) << 4, col0 = (tile % tcs) << 4;
    const int32_t row = row0 + ((int32_t)threadIdx.x >> 4), col = col0 + ((int32_t)threadIdx.x & 15);
    const int64_t size = (int64_t)rows * cols;
    const int64_t q = (int64_t)row * cols + col;
    const int64_t p = q + (sidx == 0 ? 0 : (sidx == 1 ? u.seg[0].size : u.seg[0].size + u.seg[1].size));
    const bool live = row < rows && col < cols;
    const bool adam = u.optimizer != RETEXO_SGD;
    const bool state = sidx == 2 && row >= 2;      // a running statistic of batch normalisation

    grid_dependency_wait();
    grid_dependency_release();
    // ---- loads with no dependence
    unsigned long long step_now = 0, snap_cur = 0, snap_best = 0;
    int32_t snap_have = 1;
    if (u.step_dev) step_now = *u.step_dev;
    if (u.snap_cur) { snap_have = *u.snap_have; snap_cur = *u.snap_cur; snap_best = *u.snap_best; }
    float theta = 0.f, m = 0.f, v = 0.f, g = 0.f;
    if (live) {
        theta = u.theta[p];
        if (state) {
            g = u.bn_batch[q - 2 * (int64_t)cols] * (row == 3 ? u.bn_unbias : 1.f);      // the statistic it moves towards
        } else {
            if (adam) { m = u.m[p]; v = u.v[p]; }
            g = sum_partials<BATCH>(u.seg[sidx].partial + q, (int32_t)u.seg[sidx].count, sidx == 2 ? 2 * (int64_t)cols : size);      // (a partial of the third segment holds its two trained rows)
        }
    }

    float corr1 = u.corr1, corr2 = u.corr2;
    float* loss_out = u.loss_out;
    if (u.step_dev) {      // the iteration number lives on the device: bias corrections and slots follow from it
        __shared__ float corr_s[2];
        if (threadIdx.x == 0) corr_s[0] = (float)(1.0 - pow_whole((double)u.beta1, step_now + 1));
        if (threadIdx.x == 32) corr_s[1] = (float)(1.0 - pow_whole((double)u.beta2, step_now + 1));
        __syncthreads();
        corr1 = corr_s[0]; corr2 = corr_s[1];
        loss_out = u.loss_base ? u.loss_base + step_now : nullptr;
    }
    // keep-the-best: are the weights as they stand (validated in this iteration's forward pass) the best so far?
    const bool snapshot = u.theta_best && (!snap_have || snap_cur > snap_best);
    if (u.done) {
        // Once every block has read the validation state and the iteration number (signalled here, before
        // the block's own stores, so the fence has nothing to wait for), the last block to arrive books
        // the count and moves the state on, while the others are already updating their parameters.
        __syncthreads();
        if (threadIdx.x == 0) {
            __threadfence();
            if (atomicAdd(u.done, 1ull) == (unsigned long long)gridDim.x - 1ull) {
                __threadfence();
                if (u.snap_decision) *u.snap_decision = snapshot ? 1 : 0;
                if (u.snap_cur) {
                    unsigned long long* slot = u.step_dev ? (u.history_base && step_now > 0 ? u.history_base + (step_now - 1) : nullptr)
                                                          : u.rec_history_slot;
                    if (slot) *slot = snap_cur;
                    if (!snap_have || snap_cur > snap_best) {
                        *u.snap_best = snap_cur;
                        if (u.rec_best_iter) *u.rec_best_iter = u.step_dev ? (int32_t)step_now : u.rec_iter;
                        *u.snap_have = 1;
                    }
                    *u.snap_cur = 0ull;
                }
                if (u.step_dev) *u.step_dev = step_now + 1;
                *u.done = 0ull;
            }
        }
    }
    if (blockIdx.x == 0 && threadIdx.x >= 224 && loss_out) {      // the block's last warp: not the one that signals
        const int lane = threadIdx.x - 224;
        float s = 0.f;
        for (int64_t i = lane; i < u.n_loss; i += 32) s += u.loss_partial[i];
        s = warp_sum(s);
        if (lane == 0) *loss_out = (u.status && *u.status) ? __int_as_float(0x7fc00000) : s * u.inv_rows;
    }
    if (blockIdx.x == 0 && threadIdx.x == 64 && u.status_out && u.status) *u.status_out = *u.status;

    bf16 t16 = f32_to_bf16(0.f);
    if (live) {
        if (u.grad_out) u.grad_out[p] = state ? 0.f : g;
        if (snapshot) u.theta_best[p] = theta;
        float t;
        if (state) {
            t = (1.f - u.bn_momentum) * theta + u.bn_momentum * g;
        } else if (!adam) {
            t = theta - u.lr * g;
        } else {
            m = u.beta1 * m + (1.f - u.beta1) * g;
            v = u.beta2 * v + (1.f - u.beta2) * g * g;
            u.m[p] = m;
            u.v[p] = v;
            t = theta - u.lr * (m / corr1) / (sqrtf(v / corr2) + u.eps);
        }
        u.theta[p] = t;
        t16 = f32_to_bf16(t);
        if (row < rows - 1) {                   // the weights (not the bias row), as the products read them
            if (sidx == 0) { if (u.w1r16) u.w1r16[(int64_t)row * u.ld_o1 + col] = t16; }
            else if (sidx == 1 && u.w2p16) u.w2p16[(int64_t)row * u.ld_dl + col] = t16;
        }
    }
    bf16* wt = sidx == 0 ? u.w1t16 : (sidx == 1 ? u.w2t16 : nullptr);
    if (wt) {                                   // uniform over the block
        __shared__ bf16 tile16[16][18];
        tile16[threadIdx.x >> 4][threadIdx.x & 15] = t16;
        __syncthreads();
        const int32_t trow = row0 + ((int32_t)threadIdx.x & 15), tcol = col0 + ((int32_t)threadIdx.x >> 4);
        if (trow < rows - 1 && tcol < cols)
            wt[(int64_t)tcol * (sidx == 0 ? u.ld_k : u.ld_h) + trow] = tile16[threadIdx.x & 15][threadIdx.x >> 4];
    }
}

}  // namespace retexo
