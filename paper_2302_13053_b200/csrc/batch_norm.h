// Internal: the kernels of batch normalisation inside f_theta (see batch_norm.cu).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "retexo.h"

namespace retexo {

constexpr int kBnMaxHidden = 512;           // hidden units (a lane holds 16 of them)
constexpr int64_t kBnBlocks = 592;          // blocks (and partial column sums) of the column-sum kernels: 148 SMs x 4

int64_t bn_blocks(int64_t n_rows);

// Scratch of one training iteration (all fp32):
//   partial [bn_blocks(n_rows)][2 H]   per-block column sums (one or two sums per unit)
//   batch   [3 H]                      mean | biased variance | 1 / sqrt(var + eps)   of the training rows
//   sums    [2 H]                      sum_rows dy zhat | sum_rows dy   ( = d gamma | d beta )
struct BnScratch {
    float* partial;
    float* batch;
    float* sums;
};

// Column statistics of z over rows [0, n_rows): two passes (mean, then the mean of squared deviations), each a
// column-sum kernel and a one-block kernel that adds the per-block sums in block order.
int bn_batch_stats_launch(const float* z, int64_t ld_z, int64_t n_rows, int32_t H, float eps, const BnScratch& s,
                          cudaStream_t st);

struct BnForward {
    const float* z; int64_t ld_z;           // [n_rows x ld_z] fp32, x W1 + b1
    const float* gamma; const float* beta;  // [H]
    int32_t H;
    int64_t n_rows;
    int64_t n_batch;                        // rows [0, n_batch) are normalised with `batch` (mean | var | rstd),
    const float* batch;                     //   rows [n_batch, n_rows) with the running statistics
    const float* r_mean; const float* r_var; float eps;
    __nv_bfloat16* out_bf16; int64_t ld_bf16;   // (optional) ReLU(gamma zhat + beta); columns [H, ld_bf16) zero-filled,
    int32_t ones;                               //   column H with 1 if `ones` (needs ld_bf16 > H)
    float* out_f32; int64_t ld_f32;             // (optional) the same in fp32
    uint32_t* bits; int64_t ld_bits;            // (optional) bit j & 31 of word [row][j / 32] = [output j > 0]
};
int bn_forward_launch(const BnForward& a, cudaStream_t st);

// dy (the gated gradient at the normalisation's output, bf16, rows [0, n_rows)) becomes the gradient at z in
// place:  dz = gamma rstd (dy - s1 / n - zhat s2 / n),  s1 = sum_rows dy,  s2 = sum_rows dy zhat;  s.sums is
// left holding [s2 | s1], which are d gamma and d beta.
int bn_backward_launch(const float* z, int64_t ld_z, int64_t n_rows, int32_t H, const float* gamma,
                       __nv_bfloat16* dy, int64_t ld_dy, const BnScratch& s, cudaStream_t st);

}  // namespace retexo
