// Internal: shapes, scratch layout and launch entry points of the per-node
// model, shared by the single-call API and the K-round driver.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "retexo.h"

namespace retexo {

constexpr int64_t kTargetBlocks = 592;      // 148 SMs x 4: block count row-loop grids aim for
constexpr int64_t kSmCountTarget = 148;     // one tensor-core block per SM

struct MlpPlan {
    int32_t d_in, hidden, n_classes, out1;  // out1 = width of the first linear layer's output
    int64_t n_rows, nt;                     // training rows; nt = parameters in theta
    int64_t n_eval;                         // rows after the training rows that are only evaluated (validation)
    int64_t ld_dl;                          // row stride of bf16 dL and of the padded W2 (classes rounded up to 64)
    int64_t ld_h;                           // row stride of bf16 dHd and of W2^T (hidden rounded up to 64)
    int64_t ld_h1;                          // row stride of [Hd | 1] (hidden + 1 rounded up to 64)
    int64_t ld_bits;                        // words per row of the ReLU bits (two per 64 hidden units)
    int64_t ld_k;                           // row stride of W1^T (d_in rounded up to 64)
    int64_t ld_o1;                          // row stride of the bf16 copy of W1 (out1 rounded up to 64)
    int64_t ld_x1;                          // row stride of the workspace copy [X | 1] (d_in + 1 rounded up to 64)
    int64_t sm_blocks;                      // loss partials the workspace has room for
    int64_t split_w1, split_w2;             // split-K factors of the two weight-gradient products
    int32_t norm;                           // retexo_norm (0 where hidden == 0): f_theta = Linear -> norm -> ReLU; theta ends in
                                            //   [gamma | beta] (layer) or [gamma | beta | r_mean | r_var] (batch)
    int64_t ln_blocks;                      // layer norm: partial sums of [d gamma | d beta] the backward kernel leaves
    int64_t bn_blocks;                      // batch norm: per-block column sums of its column-sum kernels
};

struct MlpBuffers {
    __nv_bfloat16* w1t16;                   // W1^T            [out1 x ld_k]
    __nv_bfloat16* w1r16;                   // W1              [d_in x ld_o1]  (may be null: retexo_embed does not need it)
    __nv_bfloat16* w2t16;                   // W2^T            [n_classes x ld_h]
    __nv_bfloat16* w2p16;                   // W2, padded rows [hidden x ld_dl]
    __nv_bfloat16* x1;                      // [X | 1]         [n x ld_x1]  (only when the caller's batch has no column of ones)
    __nv_bfloat16* hd16;                    // [Hd | 1]        [n x ld_h1]
    float* logits;                          //                 [n x n_classes]  (retexo_embed only)
    __nv_bfloat16* dl16;                    // dL              [n x ld_dl]
    __nv_bfloat16* dhd16;                   // dHd             [n x ld_h]
    uint32_t* gate_bits;                    // [Hd > 0], a bit per unit   [n x ld_bits]
    float* loss_partial;
    float* pw1;                             // [split_w1 x (d_in+1) x out1]   partials of [dW1 ; db1]
    float* pw2;                             // [split_w2 x (hidden+1) x n_classes]   partials of [dW2 ; db2]
    int32_t* status;                        // raised by a tensor-core kernel whose bounded wait gave up
    float* z1;                              // layer / batch norm: x W1 + b1 in fp32   [n x hidden]
    float2* ln_stats;                       // layer norm: (mean, 1 / sqrt(var + eps)) per row   [n]
    float* pln;                             // layer norm: [ln_blocks x 2 hidden] partials of [d gamma | d beta]
    float* bn_partial;                      // batch norm: [bn_blocks x 2 hidden] per-block column sums
    float* bn_batch;                        // batch norm: [3 hidden] mean | biased variance | 1 / sqrt(var + eps) of the batch
    float* bn_sums;                         // batch norm: [2 hidden] d gamma | d beta
};

// Split-K factor the library uses for a weight-gradient product C[M x N] = A^T B reduced over K rows.
int64_t gemm_split(int64_t M, int64_t N, int64_t K);

MlpPlan make_plan(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows, int64_t n_eval = 0,
                  int32_t norm = RETEXO_NORM_NONE);
size_t mlp_step_workspace_size(const MlpPlan& p);

// Validation folded into a training iteration: the batch holds p.n_eval more rows after the
// training rows; the forward pass covers them too, the loss epilogue counts their hits into
// *correct (weights as they are before this iteration's update), and the update kernel first
// copies theta to theta_best if that count beats *best (or nothing was kept yet).
// With `done` set, the update kernel's last block also does the bookkeeping of that validation
// count: history_slot receives it, best / have_best / best_iter are brought up to date for
// iteration `iter`, and *correct is cleared for the next iteration (so the caller clears it once
// per round, not once per iteration).  *done must be zero before the first launch; the kernel
// leaves it zero.
struct EvalTail {
    const int32_t* y_eval;
    unsigned long long* correct;
    unsigned long long* best;
    int32_t* have_best;
    float* theta_best;
    unsigned long long* done = nullptr;
    int32_t iter = 0;
    int32_t* best_iter = nullptr;
    unsigned long long* history_slot = nullptr;
    // (optional, with `done`) receives 1 if this launch copied theta to theta_best, else 0: a caller that keeps
    // further parameters next to theta (a trained aggregator) takes the same decision from it
    int32_t* decision = nullptr;
};

// Iteration state kept on the device, so that every iteration of a round is the same launch sequence
// with the same arguments (which lets the K-round driver record it once as a CUDA graph and replay it).
// With s = *step updates applied so far, a step launched with this state applies update s + 1 (Adam's bias
// corrections follow from s), writes its loss to loss_base[s], books the validation count that rode along
// as iteration s's (history_base[s - 1], best_iter) and leaves *step = s + 1.  *step and *done are cleared
// by the caller once per round.
struct DeviceIter {
    unsigned long long* step;
    unsigned long long* done;
    float* loss_base;
    unsigned long long* history_base;
};

// Lays the step's scratch buffers out over a workspace of retexo_mlp_train_step_workspace_size bytes.
void mlp_step_buffers(const MlpPlan& p, void* workspace, size_t bytes, MlpBuffers* out);

// One training iteration.  shadows_ready: the bf16 weight copies in `b` already hold the
// current theta (the previous iteration's update refreshed them), so they are not rebuilt.
// On return they hold the updated theta.
// x_has_ones: column d_in of x holds 1 in every row (ldx > d_in); otherwise the batch is first copied into
// the workspace with that column added.
int mlp_train_step_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model,
                          const __nv_bfloat16* x, int64_t ldx, bool x_has_ones,
                          const int32_t* y, float* loss_out, float* grad_out, bool shadows_ready,
                          const EvalTail* tail, cudaStream_t st, const DeviceIter* dev = nullptr,
                          float* dx_out = nullptr, int64_t ld_dx = 0);      // dx_out: fp32 [n_rows x ld_dx], dLoss / dX

// Forward + arg-max + hit count over a dense batch with the weight copies in `b` (which must
// hold model->theta): what validation needs after every iteration.  hd_ws: bf16 [n_rows x p.ld_h];
// z_ws: fp32 [n_rows x hidden], needed with a normalisation only.
int mlp_count_hits_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model,
                          const __nv_bfloat16* x, int64_t ldx, int64_t n_rows, __nv_bfloat16* hd_ws,
                          const int32_t* y, unsigned long long* correct, cudaStream_t st, float* z_ws = nullptr);

// One linear layer theta = [W | b] (W [d_in x out], row-major) of a jointly trained model: sums the `splits`
// partials of [dW ; db] = [X | 1]^T dZ (each (d_in + 1) x out, fp32) in index order, applies update number `step`
// of the optimiser, writes the gradient to grad_out (optional) and refreshes the bf16 copies W^T [out x ld_k] and
// W [d_in x ld_o1] (either may be null).  linear_shadows_launch builds those copies from theta.
int linear_update_launch(int32_t d_in, int32_t out, float* theta, float* adam_m, float* adam_v, const float* partial,
                         int64_t splits, int optimizer, float lr, float beta1, float beta2, float eps, int64_t step,
                         __nv_bfloat16* wt16, int64_t ld_k, __nv_bfloat16* wr16, int64_t ld_o1, float* grad_out,
                         cudaStream_t st);
int linear_shadows_launch(int32_t d_in, int32_t out, const float* theta, __nv_bfloat16* wt16, int64_t ld_k,
                          __nv_bfloat16* wr16, int64_t ld_o1, cudaStream_t st);


}  // namespace retexo
