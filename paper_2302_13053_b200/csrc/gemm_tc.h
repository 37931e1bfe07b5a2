// Internal interface of the tcgen05 tensor-core GEMM (sm_100a).
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace retexo {

enum TcEpilogue { TC_EPI_BIAS = 0, TC_EPI_PARTIAL = 1, TC_EPI_SOFTMAX_CE = 3, TC_EPI_ARGMAX = 4,
                  TC_EPI_MASK = 5, TC_EPI_BIAS_DROP = 6 };

// C[M x N] = A[M x K] * B[N x K]^T with A and B bf16, K contiguous (row strides
// lda / ldb elements, multiples of 8; bases 16-byte aligned).
//   TC_EPI_BIAS   : out = acc + bias[n] (bias optional), optional ReLU, written as
//                   fp32 (out_f32, ld_f32) and/or bf16 (out_bf16, ld_bf16).  With ones_col
//                   (needs ld_bf16 > N) column N of out_bf16 is set to 1 in every row: the
//                   all-ones column that turns a bias gradient into one more output row of
//                   the weight-gradient product that reads this matrix.  relu_bits (optional)
//                   receives one bit per element, set where the value written is positive.
//   TC_EPI_PARTIAL: C = A^T B with the operands as they lie in memory, A [K x lda] holding M
//                   columns and B [K x ldb] holding N columns (the reduction runs over the rows,
//                   i.e. over the batch; no transposed copy is needed).  K is cut into `splits`
//                   ranges; partial[z][M][N] (fp32) receives the raw sum of range z (zeros for
//                   an empty range).
//   TC_EPI_MASK   : out_bf16[m][n] = acc[m][n] where mask[m][n] > 0 (bf16, row stride ld_mask), else 0:
//                   the ReLU gate applied to a back-propagated gradient.
//   TC_EPI_SOFTMAX_CE (N <= 64): logits = acc + bias; per row the softmax cross-entropy against
//                   label y[m] and its gradient dL = (softmax - onehot) * inv_rows, written as bf16
//                   row-major (out_bf16, ld_bf16 a multiple of 8, padding columns zero);
//                   loss_partial[blockIdx.x] = sum of the block's row losses.  The logits never
//                   leave the SM.
//   TC_EPI_ARGMAX (N <= 64): logits = acc + bias; pred[m] = arg-max (lowest index on ties),
//                   *correct += number of rows with pred == y[m]; optional fp32 logits (out_f32).
// status: device word that receives RETEXO_ERR_TIMEOUT if a bounded wait gives up.
struct TcGemm {
    const __nv_bfloat16* A; int64_t lda;
    const __nv_bfloat16* B; int64_t ldb;
    int64_t M, N, K;
    int mode, relu, splits;
    const float* bias;
    float* out_f32; int64_t ld_f32;
    __nv_bfloat16* out_bf16; int64_t ld_bf16;
    int ones_col;
    // TC_EPI_BIAS / TC_EPI_BIAS_DROP (optional): one bit per output element, bit n & 31 of word [m][n / 32] = [out > 0]
    uint32_t* relu_bits; int64_t ld_bits;
    const __nv_bfloat16* mask; int64_t ld_mask;
    float gate_scale;          // TC_EPI_MASK: factor on the gated values (0 is read as 1)
    // TC_EPI_BIAS_DROP: as TC_EPI_BIAS, then dropout on rows [0, drop_rows): element (m, n) is kept iff word
    // (n mod 4) of Philox4x32-10(counter = (m, n / 4, drop_step, 0), key = drop_key) >= drop_thresh, and a
    // kept element is multiplied by drop_scale; rows from drop_rows on (evaluation rows) are left as they are.
    // drop_step_dev (optional): the update number is *drop_step_dev + 1 instead of drop_step.
    uint32_t drop_thresh, drop_step, drop_key[2]; float drop_scale; int64_t drop_rows;
    const unsigned long long* drop_step_dev;
    float* partial;
    const int32_t* y; float inv_rows; float* loss_partial;      // TC_EPI_SOFTMAX_CE / TC_EPI_ARGMAX
    // TC_EPI_SOFTMAX_CE only: rows [eval_from, M) are not trained on but only evaluated: their arg-max is
    // compared with y_eval[row - eval_from] and the hits are added to *correct (0 = no such rows)
    int64_t eval_from; const int32_t* y_eval;
    int32_t* pred; unsigned long long* correct;                  // TC_EPI_ARGMAX (both optional)
    int32_t* status;
};

bool tc_gemm_supported(const TcGemm& t);
int tc_gemm_launch(const TcGemm& t, cudaStream_t st);

// Tensor map of a 2-D bf16 matrix [rows x cols] (cols contiguous, row stride ld elements, base 16-byte aligned,
// ld a multiple of 8) for boxes of [box_rows x box_cols]; swizzle_bytes is 128 or 64 and equals box_cols * 2.
// Returns false where the layout does not allow one or the driver entry point is missing.
bool tc_make_map_2d(CUtensorMap* map, const void* base, int64_t rows, int64_t cols, int64_t ld, int box_rows, int box_cols,
                    int swizzle_bytes, bool l2_promote);

// The class product, the soft-max cross-entropy and the gated back-propagation of one training iteration in
// one kernel (hidden <= 256, n_classes <= 64); see mlp_fused.cu.
struct HeadBackward {
    const __nv_bfloat16* hd; int64_t ld_hd;         // Hd [n_all x ld_hd], hidden columns
    const uint32_t* gate_bits; int64_t ld_bits;     // [n_train x ld_bits] words: bit j & 31 of word j / 32 = [Hd[row][j] > 0]
    const __nv_bfloat16* w2t; int64_t ld_w2t;       // W2^T [n_classes x ld_w2t]
    const float* b2;
    int32_t hidden, n_classes;
    int64_t n_train, n_all;                         // rows [n_train, n_all) are only evaluated
    const int32_t* y; const int32_t* y_eval;
    float inv_rows, gate_scale;
    __nv_bfloat16* dl; int64_t ld_dl;               // dL  [n_train x ld_dl], ld_dl = 64
    __nv_bfloat16* dhd; int64_t ld_dhd;             // dHd [n_train x ld_dhd]
    float* loss_partial;                            // one per 128-row tile
    unsigned long long* correct;                    // hits of the evaluated rows (may be null)
    int32_t* status;
};
bool head_backward_supported(const HeadBackward& h);
int head_backward_launch(const HeadBackward& h, cudaStream_t st);

}  // namespace retexo
