// Batch normalisation inside f_theta (Section 2.2 names batch and layer normalisation among the parts of f_theta):
//     z = x W1 + b1,   zhat = (z - mean) / sqrt(var + eps)   per hidden unit,   Hd = ReLU(gamma .* zhat + beta)
// with mean and the biased variance taken over the rows of the training batch while training and from the
// running statistics at evaluation.  The product leaves z in fp32; the kernels here are the rest.  Unlike layer
// normalisation the statistics span the batch, so the forward pass is column sums (two passes: the mean, then
// the mean squared deviation from it), a one-block-per-32-units kernel that adds the per-block sums in block
// order, and a row-local kernel; the backward pass has the same shape.  A warp owns a row, lane l the units
// l, l + 32, ..., so every access of a warp is one contiguous run; nothing is added atomically, so the bits do
// not depend on scheduling.
#include "batch_norm.h"

#include "common.cuh"
#include "launch_overlap.cuh"

namespace retexo {

constexpr int kBnThreads = 256, kBnWarps = kBnThreads / 32;
constexpr int kBnPerLane = kBnMaxHidden / 32;

int64_t bn_blocks(int64_t n_rows) {
    const int64_t want = (n_rows + kBnWarps - 1) / kBnWarps;
    return want < 1 ? 1 : (want < kBnBlocks ? want : kBnBlocks);
}

// MODE 0: sum z.  MODE 1: sum (z - mean)^2.  MODE 2: sum dy zhat and sum dy.
// partial[block][j] (and partial[block][H + j] in mode 2).  Rows are dealt to warps round-robin, every warp adds
// its rows in ascending order, the block adds its warps' sums in warp order.
template <int MODE>
__global__ void __launch_bounds__(kBnThreads) bn_colsum_kernel(const float* __restrict__ z, int64_t ld_z, int64_t n_rows,
                                                               int32_t H, const float* __restrict__ batch,
                                                               const __nv_bfloat16* __restrict__ dy, int64_t ld_dy,
                                                               float* __restrict__ partial) {
    grid_dependency_wait();
    grid_dependency_release();
    __shared__ float red[kBnWarps][(MODE == 2 ? 2 : 1) * kBnMaxHidden];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float mean[kBnPerLane], rstd[kBnPerLane], acc0[kBnPerLane], acc1[kBnPerLane];
#pragma unroll
    for (int i = 0; i < kBnPerLane; ++i) {
        const int j = lane + 32 * i;
        mean[i] = (MODE >= 1 && j < H) ? batch[j] : 0.f;
        rstd[i] = (MODE == 2 && j < H) ? batch[2 * H + j] : 0.f;
        acc0[i] = acc1[i] = 0.f;
    }
    for (int64_t row = (int64_t)blockIdx.x * kBnWarps + warp; row < n_rows; row += (int64_t)gridDim.x * kBnWarps) {
        const float* zr = z + row * ld_z;
#pragma unroll
        for (int i = 0; i < kBnPerLane; ++i) {
            const int j = lane + 32 * i;
            if (j < H) {
                const float v = zr[j];
                if (MODE == 0) acc0[i] += v;
                if (MODE == 1) { const float d = v - mean[i]; acc0[i] += d * d; }
                if (MODE == 2) {
                    const float g = bf16_to_f32(dy[row * ld_dy + j]);
                    acc0[i] += g * ((v - mean[i]) * rstd[i]);
                    acc1[i] += g;
                }
            }
        }
    }
#pragma unroll
    for (int i = 0; i < kBnPerLane; ++i) {
        const int j = lane + 32 * i;
        red[warp][j] = acc0[i];
        if (MODE == 2) red[warp][kBnMaxHidden + j] = acc1[i];
    }
    __syncthreads();
    const int n_out = (MODE == 2 ? 2 : 1) * H;
    for (int j = threadIdx.x; j < n_out; j += kBnThreads) {
        const int col = j < H ? j : kBnMaxHidden + (j - H);
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kBnWarps; ++w) s += red[w][col];
        partial[(int64_t)blockIdx.x * n_out + j] = s;
    }
}

// Adds the per-block sums: a block takes 32 columns, its eight warps the blocks g, g + 8, ... in ascending order,
// and their eight sums are added in warp order.  MODE as above: 0 writes the mean, 1 the biased variance and
// 1 / sqrt(var + eps), 2 the two sums as they are.
template <int MODE>
__global__ void __launch_bounds__(kBnThreads) bn_finalize_kernel(const float* __restrict__ partial, int64_t n_blocks, int32_t H,
                                                                 float inv_rows, float eps, float* __restrict__ batch,
                                                                 float* __restrict__ sums) {
    grid_dependency_wait();
    grid_dependency_release();
    __shared__ float red[kBnWarps][32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int n_out = (MODE == 2 ? 2 : 1) * H;
    const int j = (int)blockIdx.x * 32 + lane;
    float s = 0.f;
    if (j < n_out)
        for (int64_t b = warp; b < n_blocks; b += kBnWarps) s += partial[b * n_out + j];
    red[warp][lane] = s;
    __syncthreads();
    if (warp == 0 && j < n_out) {
        float t = 0.f;
#pragma unroll
        for (int w = 0; w < kBnWarps; ++w) t += red[w][lane];
        if (MODE == 0) batch[j] = t * inv_rows;
        if (MODE == 1) {
            const float var = t * inv_rows;
            batch[H + j] = var;
            batch[2 * H + j] = 1.0f / sqrtf(var + eps);
        }
        if (MODE == 2) sums[j] = t;
    }
}

__global__ void __launch_bounds__(kBnThreads) bn_forward_kernel(BnForward a) {
    grid_dependency_wait();
    grid_dependency_release();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kBnWarps + (threadIdx.x >> 5);
    if (row >= a.n_rows) return;
    const bool in_batch = row < a.n_batch;      // (uniform over the warp)
    const float* z = a.z + row * a.ld_z;
#pragma unroll
    for (int i = 0; i < kBnPerLane; ++i) {
        const int j = lane + 32 * i;
        if (32 * i >= a.H) break;
        float y = 0.f;
        if (j < a.H) {
            const float mean = in_batch ? a.batch[j] : a.r_mean[j];
            const float rstd = in_batch ? a.batch[2 * a.H + j] : 1.0f / sqrtf(a.r_var[j] + a.eps);
            y = fmaxf(a.gamma[j] * ((z[j] - mean) * rstd) + a.beta[j], 0.f);
        }
        const unsigned word = __ballot_sync(0xffffffffu, y > 0.f);
        if (a.bits && lane == 0) a.bits[row * a.ld_bits + i] = word;
        if (j < a.H) {
            if (a.out_bf16) a.out_bf16[row * a.ld_bf16 + j] = f32_to_bf16(y);
            if (a.out_f32) a.out_f32[row * a.ld_f32 + j] = y;
        }
    }
    if (a.out_bf16)      // the rest of the row: the column of ones behind the hidden units (or a zero), then zeros
        for (int64_t j = a.H + lane; j < a.ld_bf16; j += 32)
            a.out_bf16[row * a.ld_bf16 + j] = f32_to_bf16((a.ones && j == a.H) ? 1.f : 0.f);
    if (a.bits && lane == 0)
        for (int64_t w = (a.H + 31) / 32; w < a.ld_bits; ++w) a.bits[row * a.ld_bits + w] = 0u;
}

__global__ void __launch_bounds__(kBnThreads) bn_backward_kernel(const float* __restrict__ z, int64_t ld_z, int64_t n_rows,
                                                                 int32_t H, const float* __restrict__ gamma,
                                                                 const float* __restrict__ batch, const float* __restrict__ sums,
                                                                 float inv_rows, __nv_bfloat16* __restrict__ dy, int64_t ld_dy) {
    grid_dependency_wait();
    grid_dependency_release();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kBnWarps + (threadIdx.x >> 5);
    if (row >= n_rows) return;
#pragma unroll
    for (int i = 0; i < kBnPerLane; ++i) {
        const int j = lane + 32 * i;
        if (j < H) {
            const float rstd = batch[2 * H + j];
            const float zh = (z[row * ld_z + j] - batch[j]) * rstd;
            const float g = bf16_to_f32(dy[row * ld_dy + j]);
            dy[row * ld_dy + j] = f32_to_bf16(gamma[j] * rstd * (g - sums[H + j] * inv_rows - zh * (sums[j] * inv_rows)));
        }
    }
}

template <typename... Params, typename... Args>
static int bn_launch(void (*kernel)(Params...), int64_t blocks, cudaStream_t st, Args... args) {
    OverlapLaunch ol(dim3((unsigned)blocks), dim3(kBnThreads), 0, st);
    if (cudaLaunchKernelEx(&ol.cfg, kernel, static_cast<Params>(args)...) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

int bn_batch_stats_launch(const float* z, int64_t ld_z, int64_t n_rows, int32_t H, float eps, const BnScratch& s,
                          cudaStream_t st) {
    if (H < 1 || H > kBnMaxHidden || !z || n_rows < 1 || !s.partial || !s.batch) return RETEXO_ERR_INVALID_ARG;
    const int64_t nb = bn_blocks(n_rows), fb = (H + 31) / 32;
    const float inv = 1.0f / (float)n_rows;
    const __nv_bfloat16* none = nullptr;
    RETEXO_TRY(bn_launch(bn_colsum_kernel<0>, nb, st, z, ld_z, n_rows, H, (const float*)s.batch, none, (int64_t)0, s.partial));
    RETEXO_TRY(bn_launch(bn_finalize_kernel<0>, fb, st, (const float*)s.partial, nb, H, inv, eps, s.batch, s.sums));
    RETEXO_TRY(bn_launch(bn_colsum_kernel<1>, nb, st, z, ld_z, n_rows, H, (const float*)s.batch, none, (int64_t)0, s.partial));
    return bn_launch(bn_finalize_kernel<1>, fb, st, (const float*)s.partial, nb, H, inv, eps, s.batch, s.sums);
}

int bn_forward_launch(const BnForward& a, cudaStream_t st) {
    if (a.H < 1 || a.H > kBnMaxHidden || !a.z || !a.gamma || !a.beta || a.n_rows < 0 || a.n_batch < 0) return RETEXO_ERR_INVALID_ARG;
    if (a.n_batch > 0 && !a.batch) return RETEXO_ERR_INVALID_ARG;
    if (a.n_batch < a.n_rows && (!a.r_mean || !a.r_var)) return RETEXO_ERR_INVALID_ARG;
    if (a.n_rows == 0) return RETEXO_OK;
    return bn_launch(bn_forward_kernel, (a.n_rows + kBnWarps - 1) / kBnWarps, st, a);
}

int bn_backward_launch(const float* z, int64_t ld_z, int64_t n_rows, int32_t H, const float* gamma,
                       __nv_bfloat16* dy, int64_t ld_dy, const BnScratch& s, cudaStream_t st) {
    if (H < 1 || H > kBnMaxHidden || !z || !gamma || !dy || n_rows < 1 || !s.partial || !s.batch || !s.sums)
        return RETEXO_ERR_INVALID_ARG;
    const int64_t nb = bn_blocks(n_rows);
    const float inv = 1.0f / (float)n_rows;
    RETEXO_TRY(bn_launch(bn_colsum_kernel<2>, nb, st, z, ld_z, n_rows, H, (const float*)s.batch, (const __nv_bfloat16*)dy, ld_dy,
                         s.partial));
    RETEXO_TRY(bn_launch(bn_finalize_kernel<2>, (2 * (int64_t)H + 31) / 32, st, (const float*)s.partial, nb, H, inv, 0.f, s.batch,
                         s.sums));
    return bn_launch(bn_backward_kernel, (n_rows + kBnWarps - 1) / kBnWarps, st, z, ld_z, n_rows, H, gamma,
                     (const float*)s.batch, (const float*)s.sums, inv, dy, ld_dy);
}

}  // namespace retexo
