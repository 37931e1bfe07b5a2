// Internal: the row-local kernels of layer normalisation inside f_theta (see layer_norm.cu).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "retexo.h"

namespace retexo {

constexpr int kLnMaxHidden = 512;           // hidden units a row may have (a lane holds 16 of them)
constexpr int64_t kLnBackwardBlocks = 592;  // blocks (and partial sums of d gamma / d beta) of the backward kernel: 148 SMs x 4

struct LnForward {
    const float* z; int64_t ld_z;           // [n_rows x ld_z] fp32, x W1 + b1
    const float* gamma; const float* beta;  // [H]
    float eps;
    int32_t H;
    int64_t n_rows;
    __nv_bfloat16* out_bf16; int64_t ld_bf16;   // (optional) ReLU(gamma zhat + beta); columns [H, ld_bf16) are zero-filled,
    int32_t ones;                               //   column H with 1 if `ones` (needs ld_bf16 > H)
    float* out_f32; int64_t ld_f32;             // (optional) the same in fp32
    uint32_t* bits; int64_t ld_bits;            // (optional) bit j & 31 of word [row][j / 32] = [output j > 0]
    float2* stats;                              // (optional) [n_rows] (mean, 1 / sqrt(var + eps)), for the backward pass
};
int ln_forward_launch(const LnForward& a, cudaStream_t st);

struct LnBackward {
    const float* z; int64_t ld_z;
    const float2* stats;
    const float* gamma;
    int32_t H;
    int64_t n_rows;
    __nv_bfloat16* dy; int64_t ld_dy;       // in: gated gradient at the normalisation's output; out: gradient at z
    float* partial;                         // [ln_backward_blocks(n_rows)][2 H]: per block, d gamma then d beta
};
int64_t ln_backward_blocks(int64_t n_rows);
int ln_backward_launch(const LnBackward& a, cudaStream_t st);

}  // namespace retexo
