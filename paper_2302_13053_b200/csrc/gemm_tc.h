// Internal interface of the tcgen05 tensor-core GEMM (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace retexo {

enum TcEpilogue { TC_EPI_BIAS = 0, TC_EPI_PARTIAL = 1, TC_EPI_MASK_T = 2 };

// C[M x N] = A[M x K] * B[N x K]^T with A and B bf16, K contiguous (row strides
// lda / ldb elements, multiples of 8; bases 16-byte aligned).
//   TC_EPI_BIAS   : out = acc + bias[n] (bias optional), optional ReLU, written as
//                   fp32 (out_f32, ld_f32) and/or bf16 (out_bf16, ld_bf16).
//                   out_bf16_t (optional): the same values transposed, bf16 [N x ld_t];
//                   with ones_row_t its row N is set to 1 for the M valid columns (the
//                   all-ones row that turns a bias gradient into one more output row of
//                   the weight-gradient product).
//   TC_EPI_PARTIAL: K is cut into `splits` ranges; partial[z][M][N] (fp32) receives
//                   the raw sum of range z (zeros for an empty range).
//   TC_EPI_MASK_T : out_bf16_t[n][m] = acc[m][n] where mask[m][n] > 0 (bf16, row stride
//                   ld_mask), else 0: the ReLU gate applied to a back-propagated gradient,
//                   stored transposed.
// status: device word that receives RETEXO_ERR_TIMEOUT if a bounded wait gives up.
struct TcGemm {
    const __nv_bfloat16* A; int64_t lda;
    const __nv_bfloat16* B; int64_t ldb;
    int64_t M, N, K;
    int mode, relu, splits;
    const float* bias;
    float* out_f32; int64_t ld_f32;
    __nv_bfloat16* out_bf16; int64_t ld_bf16;
    __nv_bfloat16* out_bf16_t; int64_t ld_t; int ones_row_t;
    const __nv_bfloat16* mask; int64_t ld_mask;
    float* partial;
    int32_t* status;
};

bool tc_gemm_supported(const TcGemm& t);
int tc_gemm_launch(const TcGemm& t, cudaStream_t st);

}  // namespace retexo
