// Internal: shapes, scratch layout and launch entry points of the per-node
// model, shared by the single-call API and the K-round driver.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "retexo.h"

namespace retexo {

constexpr int64_t kTargetBlocks = 592;      // 148 SMs x 4: block count the split-K and row-loop grids aim for

struct MlpPlan {
    int32_t d_in, hidden, n_classes, out1;  // out1 = width of the first linear layer's output
    int64_t n_rows, nt;                     // nt = parameters in theta
    int64_t ld_dl;                          // row stride of the bf16 dL (classes rounded up to 8)
    int64_t sm_blocks;                      // softmax blocks = number of loss / db partials
    int64_t tiles_m;                        // 64-row tiles of the batch
    int64_t split_w1, split_w2;             // split-K factors of the weight-gradient products (CUDA-core path)
    int64_t tc_split_w1;                    // split-K factor of the tensor-core dW1 product
    int64_t ld_k;                           // row stride of the transposed bf16 W1 (d_in rounded up to 8)
    int64_t ld_n;                           // row stride of transposed per-row gradients (n_rows rounded up to 8)
};

struct MlpBuffers {
    __nv_bfloat16* theta16;
    __nv_bfloat16* hd16;
    float* logits;
    __nv_bfloat16* dl16;
    __nv_bfloat16* dhd16;
    float* loss_partial;
    float* dlsum_partial;
    float* dhdsum_partial;
    float* pw1;
    float* pw2;
    __nv_bfloat16* w1t16;                   // W1^T, [out1 x ld_k]
    __nv_bfloat16* gradt16;                 // (dHd or dL)^T, [out1 x ld_n]
    int32_t* status;                        // raised by a tensor-core kernel whose bounded wait gave up
};

MlpPlan make_plan(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows);

int mlp_train_step_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model,
                          const __nv_bfloat16* x, int64_t ldx, const __nv_bfloat16* x_t, int64_t ld_xt,
                          const int32_t* y, float* loss_out, float* grad_out, cudaStream_t st);

int mlp_embed_launch(const retexo_mlp* model, __nv_bfloat16* theta16, __nv_bfloat16* hd16_ws, float* logits_ws,
                     __nv_bfloat16* w1t16, int32_t* status, const __nv_bfloat16* x, int64_t ldx, const int32_t* row_idx, int64_t n_rows,
                     float* hidden_out, int64_t ld_hidden, __nv_bfloat16* hidden_out_bf16, int64_t ld_hidden_bf16,
                     float* logits_out, int64_t ld_logits, int32_t* pred_out, const int32_t* y,
                     unsigned long long* correct_out, cudaStream_t st);

// out[M x N] (fp32, row stride ld_out) = A[M x K] (bf16) * B[K x N] (bf16), no bias.
int project_rows_launch(const __nv_bfloat16* A, int64_t lda, const __nv_bfloat16* B, int64_t ldb, int64_t M, int64_t N,
                        int64_t K, float* out, int64_t ld_out, cudaStream_t st);
int convert_f32_to_bf16_launch(const float* src, __nv_bfloat16* dst, int64_t n, cudaStream_t st);

}  // namespace retexo
