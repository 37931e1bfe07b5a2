// Layer normalisation inside f_theta (Section 2.2 lists normalisation layers among the parts of f_theta):
//     z = x W1 + b1,   zhat = (z - mean(z)) / sqrt(var(z) + eps)   (over the hidden units of a row, biased variance)
//     Hd = ReLU(gamma .* zhat + beta)
// The product leaves z in fp32; the two kernels here are the row-local rest, forward and backward.  They are
// bound by HBM (one pass over z each way): a warp owns a row, lane l the units l, l + 32, ..., so every access
// of a warp is one contiguous run, and the row statistics are two shuffle reductions over registers.
#include "layer_norm.h"

#include "common.cuh"
#include "launch_overlap.cuh"

namespace retexo {

constexpr int kLnThreads = 256, kLnWarps = kLnThreads / 32;
constexpr int kLnPerLane = kLnMaxHidden / 32;

__device__ __forceinline__ float ln_warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

__global__ void __launch_bounds__(kLnThreads) ln_forward_kernel(LnForward a) {
    grid_dependency_wait();
    grid_dependency_release();
    const int lane = threadIdx.x & 31;
    const int64_t row = (int64_t)blockIdx.x * kLnWarps + (threadIdx.x >> 5);
    if (row >= a.n_rows) return;
    const float* z = a.z + row * a.ld_z;
    float v[kLnPerLane];
    float s = 0.f;
#pragma unroll
    for (int i = 0; i < kLnPerLane; ++i) {
        const int j = lane + 32 * i;
        v[i] = j < a.H ? z[j] : 0.f;
        s += v[i];
    }
    const float mean = ln_warp_sum(s) / (float)a.H;
    float q = 0.f;
#pragma unroll
    for (int i = 0; i < kLnPerLane; ++i) {
        const int j = lane + 32 * i;
        const float d = j < a.H ? v[i] - mean : 0.f;
        q += d * d;
    }
    const float rstd = 1.0f / sqrtf(ln_warp_sum(q) / (float)a.H + a.eps);
    if (a.stats && lane == 0) a.stats[row] = make_float2(mean, rstd);
#pragma unroll
    for (int i = 0; i < kLnPerLane; ++i) {
        const int j = lane + 32 * i;
        if (32 * i >= a.H) break;                       // (uniform over the warp)
        float y = 0.f;
        if (j < a.H) y = fmaxf(a.gamma[j] * ((v[i] - mean) * rstd) + a.beta[j], 0.f);
        const unsigned word = __ballot_sync(0xffffffffu, y > 0.f);
        if (a.bits && lane == 0) a.bits[row * a.ld_bits + i] = word;
        if (j < a.H) {
            if (a.out_bf16) a.out_bf16[row * a.ld_bf16 + j] = f32_to_bf16(y);
            if (a.out_f32) a.out_f32[row * a.ld_f32 + j] = y;
        }
    }
    if (a.out_bf16) {
        // the rest of the row: the column of ones behind the hidden units (or a zero), then zeros
        for (int64_t j = a.H + lane; j < a.ld_bf16; j += 32)
            a.out_bf16[row * a.ld_bf16 + j] = f32_to_bf16((a.ones && j == a.H) ? 1.f : 0.f);
    }
    if (a.bits && lane == 0)
        for (int64_t w = (a.H + 31) / 32; w < a.ld_bits; ++w) a.bits[row * a.ld_bits + w] = 0u;
}

// dy (the gated gradient at the normalisation's output, bf16) -> dz (bf16, in place) and this block's sums of
// d gamma = dy .* zhat and d beta = dy over its rows.  Rows are dealt to warps round-robin, every warp adds
// its rows in ascending order, and the block adds its warps' sums in warp order: the result does not depend
// on timing.
__global__ void __launch_bounds__(kLnThreads) ln_backward_kernel(LnBackward a) {
    grid_dependency_wait();
    grid_dependency_release();
    __shared__ float red[kLnWarps][2 * kLnMaxHidden];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    float gam[kLnPerLane], acc_g[kLnPerLane], acc_b[kLnPerLane];
#pragma unroll
    for (int i = 0; i < kLnPerLane; ++i) {
        const int j = lane + 32 * i;
        gam[i] = j < a.H ? a.gamma[j] : 0.f;
        acc_g[i] = acc_b[i] = 0.f;
    }
    for (int64_t row = (int64_t)blockIdx.x * kLnWarps + warp; row < a.n_rows; row += (int64_t)gridDim.x * kLnWarps) {
        const float2 st = a.stats[row];
        const float* z = a.z + row * a.ld_z;
        __nv_bfloat16* d = a.dy + row * a.ld_dy;
        float zh[kLnPerLane], dzh[kLnPerLane];
        float s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int i = 0; i < kLnPerLane; ++i) {
            const int j = lane + 32 * i;
            zh[i] = dzh[i] = 0.f;
            if (j < a.H) {
                const float dy = bf16_to_f32(d[j]);
                zh[i] = (z[j] - st.x) * st.y;
                dzh[i] = dy * gam[i];
                acc_g[i] += dy * zh[i];
                acc_b[i] += dy;
                s1 += dzh[i];
                s2 += dzh[i] * zh[i];
            }
        }
        const float m1 = ln_warp_sum(s1) / (float)a.H, m2 = ln_warp_sum(s2) / (float)a.H;
#pragma unroll
        for (int i = 0; i < kLnPerLane; ++i) {
            const int j = lane + 32 * i;
            if (j < a.H) d[j] = f32_to_bf16(st.y * (dzh[i] - m1 - zh[i] * m2));
        }
    }
#pragma unroll
    for (int i = 0; i < kLnPerLane; ++i) {
        const int j = lane + 32 * i;
        red[warp][j] = acc_g[i];
        red[warp][kLnMaxHidden + j] = acc_b[i];
    }
    __syncthreads();
    for (int j = threadIdx.x; j < 2 * a.H; j += kLnThreads) {
        const int col = j < a.H ? j : kLnMaxHidden + (j - a.H);
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kLnWarps; ++w) s += red[w][col];
        a.partial[(int64_t)blockIdx.x * 2 * a.H + j] = s;
    }
}

int ln_forward_launch(const LnForward& a, cudaStream_t st) {
    if (a.H < 1 || a.H > kLnMaxHidden || !a.z || !a.gamma || !a.beta || a.n_rows < 0) return RETEXO_ERR_INVALID_ARG;
    if (a.n_rows == 0) return RETEXO_OK;
    OverlapLaunch ol(dim3((unsigned)((a.n_rows + kLnWarps - 1) / kLnWarps)), dim3(kLnThreads), 0, st);
    if (cudaLaunchKernelEx(&ol.cfg, ln_forward_kernel, a) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

int64_t ln_backward_blocks(int64_t n_rows) {
    const int64_t want = (n_rows + kLnWarps - 1) / kLnWarps;
    return want < 1 ? 1 : (want < kLnBackwardBlocks ? want : kLnBackwardBlocks);
}

int ln_backward_launch(const LnBackward& a, cudaStream_t st) {
    if (a.H < 1 || a.H > kLnMaxHidden || !a.z || !a.gamma || !a.dy || !a.stats || !a.partial || a.n_rows < 1)
        return RETEXO_ERR_INVALID_ARG;
    OverlapLaunch ol(dim3((unsigned)ln_backward_blocks(a.n_rows)), dim3(kLnThreads), 0, st);
    if (cudaLaunchKernelEx(&ol.cfg, ln_backward_kernel, a) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

}  // namespace retexo
