// Host side of the per-node model calls: argument checks, workspace layout and
// the launch sequence of one training iteration / one embedding pass.
//
// Every matrix product of an iteration runs on the tensor cores.  Activations and
// gradients are kept row-major only (one batch row per line): the forward products
// read them with the reduction dimension contiguous, the weight-gradient products,
// whose reduction runs over the batch, read the same arrays with M / N contiguous.
//   forward   [Hd | 1] = ReLU(X W1 + b1)                 gemm_tc.cu, A = X, B = W1^T
//   middle    L = Hd W2 + b2, loss, dL,                  mlp_fused.cu: one kernel, Hd read once,
//             dHd = (dL W2^T) .* [Hd > 0]                the logits never leave the SM
//   backward  [dW2 ; db2] = [Hd | 1]^T dL                gemm_tc.cu, split over the batch
//             [dW1 ; db1] = [X | 1]^T dHd                gemm_tc.cu, split over the batch
// (hidden > 256: the middle runs as two products of gemm_tc.cu instead.)
// The column of ones behind X and Hd turns each bias gradient into one more output
// row, so the partial sums come out laid out exactly like theta = [W1 | b1 | W2 | b2].
#include "gemm_tc.h"
#include "batch_norm.h"
#include "layer_norm.h"
#include "mlp_kernels.cuh"
#include "mlp_plan.h"

using namespace retexo;

namespace retexo {

// Leading dimension of a bf16 matrix: rows start on 128-byte lines, so that no 128-byte row of a
// tensor-map box straddles two lines.
static inline int64_t pad_ld(int64_t x) { return (x + 63) / 64 * 64; }

// rows of a gathered batch that retexo_embed packs and multiplies at a time (bounds the scratch it needs for them)
constexpr int64_t kEmbedGatherRows = 32768;


// Split-K factor of a tensor-core weight-gradient product: one block per SM.
static int64_t tc_split(int64_t M, int64_t N, int64_t K) {
    const int64_t bn = N > 128 ? 256 : (N > 64 ? 128 : 64);
    const int64_t tiles = ((M + 127) / 128) * ((N + bn - 1) / bn);
    int64_t s = kSmCountTarget / tiles;
    const int64_t kb = (K + 63) / 64;
    if (s > kb) s = kb;
    if (s > 64) s = 64;
    if (s < 1) s = 1;
    return s;
}

int64_t gemm_split(int64_t M, int64_t N, int64_t K) { return tc_split(M, N, K); }

MlpPlan make_plan(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows, int64_t n_eval, int32_t norm) {
    MlpPlan p{};
    p.d_in = d_in; p.hidden = hidden; p.n_classes = n_classes; p.n_rows = n_rows; p.n_eval = n_eval;
    p.out1 = hidden > 0 ? hidden : n_classes;
    p.norm = hidden > 0 ? norm : RETEXO_NORM_NONE;
    p.ln_blocks = p.norm == RETEXO_NORM_LAYER ? ln_backward_blocks(n_rows) : 0;
    p.bn_blocks = p.norm == RETEXO_NORM_BATCH ? bn_blocks(n_rows) : 0;
    p.nt = retexo_theta_size_norm(d_in, hidden, n_classes, p.norm);
    p.ld_dl = pad_ld(n_classes);                           // 64: classes padded with zero columns
    p.ld_h = pad_ld(hidden > 0 ? hidden : 1);
    p.ld_h1 = pad_ld(hidden > 0 ? hidden + 1 : 1);
    p.ld_bits = hidden > 0 ? 2 * (((int64_t)hidden + 63) / 64) : 2;
    p.ld_k = pad_ld(d_in);
    p.ld_o1 = pad_ld(p.out1);
    p.ld_x1 = pad_ld((int64_t)d_in + 1);
    p.sm_blocks = 4 * ((n_rows + n_eval + 127) / 128);     // up to four loss partials per 128-row tile
    p.split_w1 = tc_split((int64_t)d_in + 1, p.out1, n_rows);
    p.split_w2 = hidden > 0 ? tc_split((int64_t)hidden + 1, n_classes, n_rows) : 0;
    return p;
}

template <typename Taker>
static void layout(const MlpPlan& p, Taker& t, MlpBuffers* out) {
    MlpBuffers b{};
    const size_t n = (size_t)p.n_rows;
    const size_t n_all = (size_t)(p.n_rows + p.n_eval);
    const bool h = p.hidden > 0;
    b.w1t16 = t.template take<bf16>((size_t)p.out1 * p.ld_k);
    b.w1r16 = t.template take<bf16>((size_t)p.d_in * p.ld_o1);
    b.w2t16 = t.template take<bf16>(h ? (size_t)p.n_classes * p.ld_h : 1);
    b.w2p16 = t.template take<bf16>(h ? (size_t)p.hidden * p.ld_dl : 1);
    b.x1 = t.template take<bf16>(n_all * p.ld_x1);
    b.hd16 = t.template take<bf16>(h ? n_all * p.ld_h1 : 1);
    b.dl16 = t.template take<bf16>(n * p.ld_dl);
    b.dhd16 = t.template take<bf16>(h ? n * p.ld_h : 1);
    b.gate_bits = t.template take<uint32_t>(h ? n_all * (size_t)p.ld_bits : 1);
    b.loss_partial = t.template take<float>((size_t)p.sm_blocks);
    b.pw1 = t.template take<float>((size_t)p.split_w1 * (p.d_in + 1) * p.out1);
    b.pw2 = t.template take<float>(h ? (size_t)p.split_w2 * (p.hidden + 1) * p.n_classes : 1);
    b.status = t.template take<int32_t>(64);
    if (p.norm) {
        b.z1 = t.template take<float>(n_all * (size_t)p.hidden);
        if (p.norm == RETEXO_NORM_LAYER) {
            b.ln_stats = t.template take<float2>(n_all);
            b.pln = t.template take<float>((size_t)p.ln_blocks * 2 * p.hidden);
        } else {
            b.bn_partial = t.template take<float>((size_t)p.bn_blocks * 2 * p.hidden);
            b.bn_batch = t.template take<float>(3 * (size_t)p.hidden);
            b.bn_sums = t.template take<float>(2 * (size_t)p.hidden);
        }
    }
    if (out) *out = b;
}

void mlp_step_buffers(const MlpPlan& p, void* workspace, size_t bytes, MlpBuffers* out) {
    Arena ws(workspace, bytes);
    layout(p, ws, out);
}

struct NullTaker {
    Sizer s;
    template <typename T> T* take(size_t count) { s.take<T>(count); return nullptr; }
};

size_t mlp_step_workspace_size(const MlpPlan& p) {
    NullTaker t;
    layout(p, t, nullptr);
    return t.s.off + kAlign;
}

static int check_model(const retexo_mlp* m) {
    if (!m || m->d_in <= 0 || m->hidden < 0 || m->n_classes <= 0 || !m->theta) return RETEXO_ERR_INVALID_ARG;
    if (m->n_classes > 64 || m->hidden > 512) return RETEXO_ERR_UNSUPPORTED;
    if (!(m->dropout >= 0.f && m->dropout < 1.f)) return RETEXO_ERR_INVALID_ARG;
    if (m->norm != RETEXO_NORM_NONE && m->norm != RETEXO_NORM_LAYER && m->norm != RETEXO_NORM_BATCH) return RETEXO_ERR_INVALID_ARG;
    if (m->norm && m->hidden > 0) {
        if (!(m->norm_eps > 0.f)) return RETEXO_ERR_INVALID_ARG;
        if (m->norm == RETEXO_NORM_BATCH && !(m->bn_momentum >= 0.f && m->bn_momentum <= 1.f)) return RETEXO_ERR_INVALID_ARG;
        if (m->hidden > kLnMaxHidden || m->dropout > 0.f) return RETEXO_ERR_UNSUPPORTED;
    }
    return RETEXO_OK;
}

static int32_t norm_of(const retexo_mlp* m) { return m->hidden > 0 ? m->norm : RETEXO_NORM_NONE; }

// bf16 shadows of the weights in the orientations the products need.
static int build_weight_shadows(const MlpPlan& p, const MlpBuffers& b, const float* theta, cudaStream_t st) {
    const int32_t d_in = p.d_in, H = p.hidden, O = p.n_classes, out1 = p.out1;
    RETEXO_TRY(retexo_pack_rows(theta, 0, out1, out1, nullptr, d_in, b.w1r16, b.w1r16 ? p.ld_o1 : 0, b.w1t16, p.ld_k, 0, st));
    if (H > 0) {
        const float* w2 = theta + (int64_t)d_in * out1 + out1;
        RETEXO_TRY(retexo_pack_rows(w2, 0, O, O, nullptr, H, b.w2p16, p.ld_dl, b.w2t16, p.ld_h, 0, st));
    }
    return RETEXO_OK;
}

static TcGemm tc_base(const bf16* A, int64_t lda, const bf16* B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                      int32_t* status) {
    TcGemm t{};
    t.A = A; t.lda = lda; t.B = B; t.ldb = ldb; t.M = M; t.N = N; t.K = K; t.status = status;
    t.mode = TC_EPI_BIAS;
    return t;
}

}  // namespace retexo

extern "C" int64_t retexo_theta_size(int32_t d_in, int32_t hidden, int32_t n_classes) {
    if (hidden > 0) return (int64_t)d_in * hidden + hidden + (int64_t)hidden * n_classes + n_classes;
    return (int64_t)d_in * n_classes + n_classes;
}

extern "C" int64_t retexo_theta_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes, int32_t norm) {
    if (hidden <= 0 || norm == RETEXO_NORM_NONE) return retexo_theta_size(d_in, hidden, n_classes);
    return retexo_theta_size(d_in, hidden, n_classes) + (norm == RETEXO_NORM_BATCH ? 4 : 2) * (int64_t)hidden;
}

extern "C" int retexo_pack_rows(const void* src, int32_t src_is_bf16, int64_t ld_src, int32_t dim,
                                const int32_t* idx, int64_t n_rows, void* dst, int64_t ld_dst,
                                void* dst_t, int64_t ld_t, int32_t ones, void* stream) {
    if (!src || dim <= 0 || ld_src < dim || n_rows < 0 || (!dst && !dst_t)) return RETEXO_ERR_INVALID_ARG;
    if (dst && ld_dst < dim + (ones ? 1 : 0)) return RETEXO_ERR_INVALID_ARG;
    if (dst_t && ld_t < n_rows) return RETEXO_ERR_INVALID_ARG;
    const int64_t rows_cover = dst_t ? (ld_t > n_rows ? ld_t : n_rows) : n_rows;
    const int64_t cols_cover = dst ? ld_dst : dim;
    if (rows_cover == 0) return RETEXO_OK;
    dim3 grid((unsigned)((rows_cover + 31) / 32), (unsigned)((cols_cover + 31) / 32));
    if (grid.y > 65535) return RETEXO_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (src_is_bf16)
        pack_rows_kernel<true><<<grid, 256, 0, st>>>(src, ld_src, dim, idx, n_rows, static_cast<bf16*>(dst), ld_dst,
                                                     static_cast<bf16*>(dst_t), ld_t, ones ? 1 : 0);
    else
        pack_rows_kernel<false><<<grid, 256, 0, st>>>(src, ld_src, dim, idx, n_rows, static_cast<bf16*>(dst), ld_dst,
                                                      static_cast<bf16*>(dst_t), ld_t, ones ? 1 : 0);
    return launch_status();
}

extern "C" size_t retexo_mlp_train_step_workspace_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes,
                                                          int64_t n_rows, int32_t norm) {
    if (d_in <= 0 || hidden < 0 || n_classes <= 0 || n_rows <= 0) return 0;
    return mlp_step_workspace_size(make_plan(d_in, hidden, n_classes, n_rows, 0, norm));
}

extern "C" size_t retexo_mlp_train_step_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes,
                                                       int64_t n_rows) {
    return retexo_mlp_train_step_workspace_size_norm(d_in, hidden, n_classes, n_rows, 0);
}

extern "C" int retexo_mlp_train_step(retexo_mlp* model, const void* x, int64_t ldx, int32_t x_has_ones,
                                     const int32_t* y, int64_t n_rows, float* loss_out, float* grad_out,
                                     float* dx_out, int64_t ld_dx,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    RETEXO_TRY(check_model(model));
    if (!x || !y || n_rows <= 0 || ldx < model->d_in) return RETEXO_ERR_INVALID_ARG;
    if (model->optimizer != RETEXO_SGD && model->optimizer != RETEXO_ADAM) return RETEXO_ERR_INVALID_ARG;
    if (model->optimizer == RETEXO_ADAM && (!model->adam_m || !model->adam_v)) return RETEXO_ERR_INVALID_ARG;
    if (x_has_ones && ldx < (int64_t)model->d_in + 1) return RETEXO_ERR_INVALID_ARG;
    if (dx_out && ld_dx < model->d_in) return RETEXO_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || ldx % 8 != 0) return RETEXO_ERR_ALIGNMENT;
    const size_t need = retexo_mlp_train_step_workspace_size_norm(model->d_in, model->hidden, model->n_classes, n_rows,
                                                                  norm_of(model));
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const MlpPlan p = make_plan(model->d_in, model->hidden, model->n_classes, n_rows, 0, norm_of(model));
    Arena ws(workspace, workspace_bytes);
    MlpBuffers b{};
    layout(p, ws, &b);
    RETEXO_TRY(mlp_train_step_launch(p, b, model, static_cast<const bf16*>(x), ldx, x_has_ones != 0, y, loss_out, grad_out,
                                     false, nullptr, st, nullptr, dx_out, ld_dx));
    model->step += 1;
    return RETEXO_OK;
}

namespace retexo {

// The launch sequence of one iteration; `model->step` is the count of updates
// already applied.
int mlp_train_step_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model,
                          const bf16* x, int64_t ldx, bool x_has_ones, const int32_t* y,
                          float* loss_out, float* grad_out, bool shadows_ready, const EvalTail* tail,
                          cudaStream_t st, const DeviceIter* dev, float* dx_out, int64_t ld_dx) {
    const int64_t n = p.n_rows;
    const int64_t n_all = n + (tail ? p.n_eval : 0);          // evaluation rows ride along in the forward pass
    const int32_t d_in = p.d_in, H = p.hidden, O = p.n_classes, out1 = p.out1;
    const float* theta = model->theta;
    const float* b1 = theta + (int64_t)d_in * out1;
    const float* b2 = b1 + out1 + (int64_t)H * O;
    // (a caller that chains iterations clears the status word once: a give-up then marks every later loss)
    if (!shadows_ready) {
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.status, 0, sizeof(int32_t), st));
        RETEXO_TRY(build_weight_shadows(p, b, theta, st));
    }
    if (!x_has_ones) {      // no column of ones behind the caller's batch: copy it with one (one more pass over X per call)
        RETEXO_TRY(retexo_pack_rows(x, 1, ldx, d_in, nullptr, n_all, b.x1, p.ld_x1, nullptr, 0, 1, st));
        x = b.x1;
        ldx = p.ld_x1;
    }

    // ---- forward
    if (tail && !tail->done) RETEXO_CUDA_TRY(cudaMemsetAsync(tail->correct, 0, sizeof(unsigned long long), st));
    TcGemm fwd = tc_base(x, ldx, b.w1t16, p.ld_k, n_all, out1, d_in, b.status);
    fwd.bias = b1;
    const bool dropping = H > 0 && model->dropout > 0.f;
    const float keep_scale = dropping ? (float)(1.0 / (1.0 - (double)model->dropout)) : 1.f;
    const bf16* grad1 = b.dl16;      // gradient at the first layer's output, one batch row per line
    int64_t ld_grad1 = p.ld_dl;
    int64_t n_loss = (n_all + 127) / 128;
    const bool ln = p.norm == RETEXO_NORM_LAYER, bn = p.norm == RETEXO_NORM_BATCH;
    const float* ln_gamma = theta + retexo_theta_size(d_in, H, O);      // (normalisation) [gamma | beta (| r_mean | r_var)] end theta
    const BnScratch bns{b.bn_partial, b.bn_batch, b.bn_sums};
    if (bn && n < 2) return RETEXO_ERR_INVALID_ARG;                     // (the unbiased variance of the running statistics)
    if (H > 0) {
        if (ln || bn) {
            // the product leaves z = X W1 + b1 in fp32; the normalisation's kernel applies the ReLU and
            // writes [Hd | 1] and the gate bits as the plain forward epilogue would
            fwd.out_f32 = b.z1; fwd.ld_f32 = H;
        } else {
            fwd.relu = 1; fwd.out_bf16 = b.hd16; fwd.ld_bf16 = p.ld_h1; fwd.ones_col = 1;
            fwd.relu_bits = b.gate_bits; fwd.ld_bits = p.ld_bits;
        }
        if (dropping) {
            fwd.mode = TC_EPI_BIAS_DROP;
            fwd.drop_thresh = (uint32_t)floor((double)model->dropout * 4294967296.0);
            fwd.drop_step = (uint32_t)(model->step + 1);
            fwd.drop_step_dev = dev ? dev->step : nullptr;      // (iteration state on the device: read there)
            fwd.drop_key[0] = (uint32_t)(model->dropout_seed & 0xffffffffu);
            fwd.drop_key[1] = (uint32_t)(model->dropout_seed >> 32);
            fwd.drop_scale = keep_scale;
            fwd.drop_rows = n;
        }
        RETEXO_TRY(tc_gemm_launch(fwd, st));
        if (ln) {
            LnForward lf{};
            lf.z = b.z1; lf.ld_z = H; lf.gamma = ln_gamma; lf.beta = ln_gamma + H; lf.eps = model->norm_eps; lf.H = H;
            lf.n_rows = n_all; lf.out_bf16 = b.hd16; lf.ld_bf16 = p.ld_h1; lf.ones = 1;
            lf.bits = b.gate_bits; lf.ld_bits = p.ld_bits; lf.stats = b.ln_stats;
            RETEXO_TRY(ln_forward_launch(lf, st));
        }
        if (bn) {      // training rows: the batch's own statistics; rows riding along for validation: the running ones
            RETEXO_TRY(bn_batch_stats_launch(b.z1, H, n, H, model->norm_eps, bns, st));
            BnForward bf{};
            bf.z = b.z1; bf.ld_z = H; bf.gamma = ln_gamma; bf.beta = ln_gamma + H; bf.H = H; bf.n_rows = n_all; bf.n_batch = n;
            bf.batch = b.bn_batch; bf.r_mean = ln_gamma + 2 * H; bf.r_var = ln_gamma + 3 * H; bf.eps = model->norm_eps;
            bf.out_bf16 = b.hd16; bf.ld_bf16 = p.ld_h1; bf.ones = 1; bf.bits = b.gate_bits; bf.ld_bits = p.ld_bits;
            RETEXO_TRY(bn_forward_launch(bf, st));
        }
        // ---- class product, loss and gated back-propagation
        HeadBackward hb{};
        hb.hd = b.hd16; hb.ld_hd = p.ld_h1; hb.gate_bits = b.gate_bits; hb.ld_bits = p.ld_bits; hb.w2t = b.w2t16; hb.ld_w2t = p.ld_h; hb.b2 = b2;
        hb.hidden = H; hb.n_classes = O; hb.n_train = n; hb.n_all = n_all;
        hb.y = y; hb.y_eval = tail ? tail->y_eval : nullptr;
        hb.inv_rows = 1.0f / (float)n; hb.gate_scale = keep_scale;      // a dropped unit has Hd = 0: the gate holds the mask
        hb.dl = b.dl16; hb.ld_dl = p.ld_dl; hb.dhd = b.dhd16; hb.ld_dhd = p.ld_h;
        hb.loss_partial = b.loss_partial; hb.correct = tail ? tail->correct : nullptr; hb.status = b.status;
        if (head_backward_supported(hb)) {
            RETEXO_TRY(head_backward_launch(hb, st));
            n_loss *= 4;
        } else {      // wide hidden layers: the same three steps as two products
            TcGemm head = tc_base(b.hd16, p.ld_h1, b.w2t16, p.ld_h, n_all, O, H, b.status);
            head.bias = b2;
            head.mode = TC_EPI_SOFTMAX_CE; head.y = y; head.inv_rows = 1.0f / (float)n; head.loss_partial = b.loss_partial;
            head.out_bf16 = b.dl16; head.ld_bf16 = p.ld_dl;
            if (tail) { head.eval_from = n; head.y_eval = tail->y_eval; head.correct = tail->correct; }
            RETEXO_TRY(tc_gemm_launch(head, st));
            TcGemm bk = tc_base(b.dl16, p.ld_dl, b.w2p16, p.ld_dl, n, H, O, b.status);
            bk.mode = TC_EPI_MASK; bk.mask = b.hd16; bk.ld_mask = p.ld_h1; bk.out_bf16 = b.dhd16; bk.ld_bf16 = p.ld_h;
            bk.gate_scale = keep_scale;
            RETEXO_TRY(tc_gemm_launch(bk, st));
        }
        // ---- [dW2 ; db2] = [Hd | 1]^T dL
        TcGemm g2 = tc_base(b.hd16, p.ld_h1, b.dl16, p.ld_dl, (int64_t)H + 1, O, n, b.status);
        g2.mode = TC_EPI_PARTIAL; g2.splits = (int)p.split_w2; g2.partial = b.pw2;
        RETEXO_TRY(tc_gemm_launch(g2, st));
        if (ln) {      // through the normalisation: dHd (in place) becomes the gradient at z; partials of d gamma, d beta
            LnBackward lb{};
            lb.z = b.z1; lb.ld_z = H; lb.stats = b.ln_stats; lb.gamma = ln_gamma; lb.H = H; lb.n_rows = n;
            lb.dy = b.dhd16; lb.ld_dy = p.ld_h; lb.partial = b.pln;
            RETEXO_TRY(ln_backward_launch(lb, st));
        }
        if (bn) RETEXO_TRY(bn_backward_launch(b.z1, H, n, H, ln_gamma, b.dhd16, p.ld_h, bns, st));
        grad1 = b.dhd16;
        ld_grad1 = p.ld_h;
    } else {
        // last round: the single linear layer ends in the loss
        fwd.mode = TC_EPI_SOFTMAX_CE; fwd.y = y; fwd.inv_rows = 1.0f / (float)n; fwd.loss_partial = b.loss_partial;
        fwd.out_bf16 = b.dl16; fwd.ld_bf16 = p.ld_dl;
        if (tail) { fwd.eval_from = n; fwd.y_eval = tail->y_eval; fwd.correct = tail->correct; }
        RETEXO_TRY(tc_gemm_launch(fwd, st));
    }
    // ---- dX = grad1 W1^T, for a caller that trains what produced X (an aggregator with parameters)
    if (dx_out) {
        TcGemm dxg = tc_base(grad1, ld_grad1, b.w1r16, p.ld_o1, n, d_in, out1, b.status);
        dxg.out_f32 = dx_out; dxg.ld_f32 = ld_dx;
        RETEXO_TRY(tc_gemm_launch(dxg, st));
    }
    // ---- [dW1 ; db1] = [X | 1]^T grad1
    TcGemm g1 = tc_base(x, ldx, grad1, ld_grad1, (int64_t)d_in + 1, out1, n, b.status);
    g1.mode = TC_EPI_PARTIAL; g1.splits = (int)p.split_w1; g1.partial = b.pw1;
    RETEXO_TRY(tc_gemm_launch(g1, st));

    // ---- reduce the partials and update
    UpdateArgs u{};
    u.n_seg = H > 0 ? 2 : 1;
    u.seg[0] = {((int64_t)d_in + 1) * out1, b.pw1, p.split_w1};
    if (H > 0) u.seg[1] = {((int64_t)H + 1) * O, b.pw2, p.split_w2};
    if (ln) { u.n_seg = 3; u.seg[2] = {2 * (int64_t)H, b.pln, p.ln_blocks}; }
    if (bn) {      // [d gamma | d beta] arrive summed; the running statistics behind them move towards the batch's
        u.n_seg = 3; u.seg[2] = {2 * (int64_t)H, b.bn_sums, 1};
        u.bn_batch = b.bn_batch; u.bn_momentum = model->bn_momentum; u.bn_unbias = (float)((double)n / (double)(n - 1));
    }
    u.theta = model->theta; u.m = model->adam_m; u.v = model->adam_v; u.grad_out = grad_out;
    u.optimizer = model->optimizer; u.lr = model->lr; u.beta1 = model->beta1; u.beta2 = model->beta2;
    u.eps = model->eps;
    const double t = (double)(model->step + 1);
    u.corr1 = (float)(1.0 - pow((double)model->beta1, t));
    u.corr2 = (float)(1.0 - pow((double)model->beta2, t));
    u.loss_partial = b.loss_partial; u.n_loss = n_loss;      // the partials this launch's loss kernel wrote
    u.inv_rows = 1.0f / (float)n; u.loss_out = loss_out;
    u.status = b.status;
    u.w1t16 = b.w1t16; u.ld_k = p.ld_k; u.w1r16 = b.w1r16; u.ld_o1 = p.ld_o1; u.w2t16 = H > 0 ? b.w2t16 : nullptr; u.ld_h = p.ld_h;
    u.w2p16 = H > 0 ? b.w2p16 : nullptr; u.ld_dl = p.ld_dl;
    u.d_in = d_in; u.out1 = out1; u.hidden = H; u.n_classes = O;
    if (tail) {
        u.snap_decision = tail->decision;
        u.snap_cur = tail->correct; u.snap_best = tail->best; u.snap_have = tail->have_best; u.theta_best = tail->theta_best;
        u.done = tail->done; u.rec_iter = tail->iter; u.rec_best_iter = tail->best_iter; u.rec_history_slot = tail->history_slot;
    }
    if (dev) {
        u.step_dev = dev->step; u.done = dev->done; u.loss_base = dev->loss_base; u.history_base = dev->history_base;
        u.loss_out = nullptr;
    }
    const int64_t tiles = (((int64_t)d_in + 16) / 16) * ((out1 + 15) / 16) + (H > 0 ? (((int64_t)H + 16) / 16) * ((O + 15) / 16) : 0) +
                          ((ln || bn) ? ((int64_t)H + 15) / 16 : 0);      // (a normalisation's segment has 2 or 4 rows of hidden entries)
    u.status_out = model->status_out;
    OverlapLaunch ol(dim3((unsigned)tiles), dim3(256), 0, st);
    if (cudaLaunchKernelEx(&ol.cfg, p.split_w1 <= 16 ? reduce_update_kernel<16> : reduce_update_kernel<32>, u) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

// Update of one linear layer theta = [W | b] (W [d_in x out]) from the split-K partials of [X | 1]^T dZ; see mlp_plan.h.
int linear_update_launch(int32_t d_in, int32_t out, float* theta, float* adam_m, float* adam_v, const float* partial,
                         int64_t splits, int optimizer, float lr, float beta1, float beta2, float eps, int64_t step,
                         bf16* wt16, int64_t ld_k, bf16* wr16, int64_t ld_o1, float* grad_out, cudaStream_t st) {
    UpdateArgs u{};
    u.n_seg = 1;
    u.seg[0] = {((int64_t)d_in + 1) * out, partial, splits};
    u.theta = theta; u.m = adam_m; u.v = adam_v; u.grad_out = grad_out;
    u.optimizer = optimizer; u.lr = lr; u.beta1 = beta1; u.beta2 = beta2; u.eps = eps;
    u.corr1 = (float)(1.0 - pow((double)beta1, (double)step));
    u.corr2 = (float)(1.0 - pow((double)beta2, (double)step));
    u.w1t16 = wt16; u.ld_k = ld_k; u.w1r16 = wr16; u.ld_o1 = ld_o1;
    u.d_in = d_in; u.out1 = out; u.hidden = 0; u.n_classes = out;
    const int64_t tiles = (((int64_t)d_in + 16) / 16) * ((out + 15) / 16);
    OverlapLaunch ol(dim3((unsigned)tiles), dim3(256), 0, st);
    if (cudaLaunchKernelEx(&ol.cfg, splits <= 16 ? reduce_update_kernel<16> : reduce_update_kernel<32>, u) != cudaSuccess) {
        (void)cudaGetLastError();
        return RETEXO_ERR_CUDA;
    }
    return launch_status();
}

int linear_shadows_launch(int32_t d_in, int32_t out, const float* theta, bf16* wt16, int64_t ld_k, bf16* wr16, int64_t ld_o1,
                          cudaStream_t st) {
    return retexo_pack_rows(theta, 0, out, out, nullptr, d_in, wr16, wr16 ? ld_o1 : 0, wt16, ld_k, 0, st);
}

// Hd = ReLU(norm(z)) for rows whose z = x W1 + b1 the forward product has left in fp32 (evaluation: batch
// normalisation uses its running statistics).
static int normalise_rows(const retexo_mlp* model, const float* z, int64_t n_rows, bf16* hd16, int64_t ld16,
                          float* hidden_out, int64_t ld_hidden, cudaStream_t st) {
    const int32_t H = model->hidden;
    const float* gamma = model->theta + retexo_theta_size(model->d_in, H, model->n_classes);
    if (model->norm == RETEXO_NORM_BATCH) {
        BnForward bf{};
        bf.z = z; bf.ld_z = H; bf.gamma = gamma; bf.beta = gamma + H; bf.H = H; bf.n_rows = n_rows; bf.n_batch = 0;
        bf.r_mean = gamma + 2 * H; bf.r_var = gamma + 3 * H; bf.eps = model->norm_eps;
        bf.out_bf16 = hd16; bf.ld_bf16 = ld16; bf.out_f32 = hidden_out; bf.ld_f32 = ld_hidden;
        return bn_forward_launch(bf, st);
    }
    LnForward lf{};
    lf.z = z; lf.ld_z = H; lf.gamma = gamma; lf.beta = gamma + H; lf.eps = model->norm_eps; lf.H = H; lf.n_rows = n_rows;
    lf.out_bf16 = hd16; lf.ld_bf16 = ld16; lf.out_f32 = hidden_out; lf.ld_f32 = ld_hidden;
    return ln_forward_launch(lf, st);
}

int mlp_count_hits_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model, const bf16* x, int64_t ldx,
                          int64_t n_rows, bf16* hd_ws, const int32_t* y, unsigned long long* correct, cudaStream_t st,
                          float* z_ws) {
    const int32_t d_in = p.d_in, H = p.hidden, O = p.n_classes, out1 = p.out1;
    const float* b1 = model->theta + (int64_t)d_in * out1;
    const float* b2 = b1 + out1 + (int64_t)H * O;
    RETEXO_CUDA_TRY(cudaMemsetAsync(correct, 0, sizeof(unsigned long long), st));
    if (n_rows == 0) return RETEXO_OK;
    TcGemm fwd = tc_base(x, ldx, b.w1t16, p.ld_k, n_rows, out1, d_in, b.status);
    fwd.bias = b1;
    if (H > 0) {
        if (p.norm) {
            if (!z_ws) return RETEXO_ERR_WORKSPACE;
            fwd.out_f32 = z_ws; fwd.ld_f32 = H;
            RETEXO_TRY(tc_gemm_launch(fwd, st));
            RETEXO_TRY(normalise_rows(model, z_ws, n_rows, hd_ws, p.ld_h, nullptr, 0, st));
        } else {
            fwd.relu = 1; fwd.out_bf16 = hd_ws; fwd.ld_bf16 = p.ld_h;
            RETEXO_TRY(tc_gemm_launch(fwd, st));
        }
        TcGemm l2 = tc_base(hd_ws, p.ld_h, b.w2t16, p.ld_h, n_rows, O, H, b.status);
        l2.bias = b2; l2.mode = TC_EPI_ARGMAX; l2.y = y; l2.correct = correct;
        return tc_gemm_launch(l2, st);
    }
    fwd.mode = TC_EPI_ARGMAX; fwd.y = y; fwd.correct = correct;
    return tc_gemm_launch(fwd, st);
}

}  // namespace retexo

extern "C" size_t retexo_embed_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows) {
    return retexo_embed_workspace_size_norm(d_in, hidden, n_classes, n_rows, 0);
}

extern "C" size_t retexo_embed_workspace_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows,
                                                 int32_t norm) {
    if (d_in <= 0 || hidden < 0 || n_classes <= 0 || n_rows < 0) return 0;
    Sizer s;
    const size_t out1 = hidden > 0 ? hidden : n_classes;
    s.take<bf16>(out1 * (size_t)pad_ld(d_in));                                   // W1^T
    s.take<bf16>(hidden > 0 ? (size_t)n_classes * pad_ld(hidden) : 1);           // W2^T
    s.take<bf16>(hidden > 0 ? (size_t)hidden * pad_ld(n_classes) : 1);           // W2 padded (unused here)
    s.take<bf16>((size_t)(n_rows < kEmbedGatherRows ? n_rows : kEmbedGatherRows) * pad_ld(d_in));   // gathered rows, a chunk
    s.take<bf16>(hidden > 0 ? (size_t)n_rows * pad_ld(hidden) : 1);              // Hd
    s.take<float>((size_t)n_rows * n_classes);                                      // logits
    s.take<int32_t>(64);
    if (norm && hidden > 0) s.take<float>((size_t)n_rows * hidden);           // z = x W1 + b1 before the normalisation
    return s.off + kAlign;
}

extern "C" int retexo_embed(const retexo_mlp* model, const void* x, int64_t ldx, const int32_t* row_idx,
                            int64_t n_rows, float* hidden_out, int64_t ld_hidden, void* hidden_out_bf16,
                            int64_t ld_hidden_bf16, float* logits_out, int64_t ld_logits, int32_t* pred_out,
                            const int32_t* y, uint64_t* correct_out, void* workspace, size_t workspace_bytes,
                            void* stream) {
    RETEXO_TRY(check_model(model));
    if (!x || n_rows < 0 || ldx < model->d_in) return RETEXO_ERR_INVALID_ARG;
    const int32_t H = model->hidden, O = model->n_classes, d_in = model->d_in;
    const int32_t out1 = H > 0 ? H : O;
    if ((hidden_out || hidden_out_bf16) && H == 0) return RETEXO_ERR_INVALID_ARG;
    if (hidden_out && ld_hidden < H) return RETEXO_ERR_INVALID_ARG;
    if (hidden_out_bf16 && ld_hidden_bf16 < H) return RETEXO_ERR_INVALID_ARG;
    if (logits_out && ld_logits < O) return RETEXO_ERR_INVALID_ARG;
    if (correct_out && !y) return RETEXO_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || ldx % 8 != 0) return RETEXO_ERR_ALIGNMENT;
    const bool ln = norm_of(model) != RETEXO_NORM_NONE;
    const size_t need = retexo_embed_workspace_size_norm(d_in, H, O, n_rows, norm_of(model));
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Arena ws(workspace, workspace_bytes);
    MlpPlan p = make_plan(d_in, H, O, n_rows > 0 ? n_rows : 1);
    MlpBuffers b{};
    b.w1t16 = ws.take<bf16>((size_t)out1 * p.ld_k);
    b.w2t16 = ws.take<bf16>(H > 0 ? (size_t)O * p.ld_h : 1);
    b.w2p16 = ws.take<bf16>(H > 0 ? (size_t)H * p.ld_dl : 1);
    bf16* xg = ws.take<bf16>((size_t)(n_rows < kEmbedGatherRows ? n_rows : kEmbedGatherRows) * p.ld_k);      // gathered rows, a chunk
    b.hd16 = ws.take<bf16>(H > 0 ? (size_t)n_rows * p.ld_h : 1);
    b.logits = ws.take<float>((size_t)n_rows * O);
    b.status = ws.take<int32_t>(64);
    float* z_ws = ln ? ws.take<float>((size_t)n_rows * H) : nullptr;
    unsigned long long* correct = reinterpret_cast<unsigned long long*>(correct_out);

    if (correct) RETEXO_CUDA_TRY(cudaMemsetAsync(correct, 0, sizeof(unsigned long long), st));
    if (n_rows == 0) return RETEXO_OK;
    RETEXO_CUDA_TRY(cudaMemsetAsync(b.status, 0, sizeof(int32_t), st));
    const float* theta = model->theta;
    const float* b1 = theta + (int64_t)d_in * out1;
    const float* b2 = b1 + out1 + (int64_t)H * O;
    const bool want_logits = logits_out || pred_out || correct;

    RETEXO_TRY(build_weight_shadows(p, b, theta, st));
    // One pass of the tensor-core path over `rows` dense rows xd; `off` is their position in the outputs.
    auto dense = [&](const bf16* xd, int64_t ldxd, int64_t rows, int64_t off) -> int {
        float* hid = hidden_out ? hidden_out + off * ld_hidden : nullptr;
        bf16* hid16 = hidden_out_bf16 ? static_cast<bf16*>(hidden_out_bf16) + off * ld_hidden_bf16 : nullptr;
        float* lgo = logits_out ? logits_out + off * ld_logits : nullptr;
        int32_t* pred = pred_out ? pred_out + off : nullptr;
        const int32_t* yy = y ? y + off : nullptr;
        TcGemm fwd = tc_base(xd, ldxd, b.w1t16, p.ld_k, rows, out1, d_in, b.status);
        fwd.bias = b1;
        if (H > 0) {
            // the logits product reads Hd through TMA, so it wants an aligned copy with a stride of 8 elements
            const bool user16_ok = hid16 && aligned_to(hid16, 16) && ld_hidden_bf16 % 8 == 0;
            bf16* h16 = user16_ok ? hid16 : b.hd16 + off * p.ld_h;
            const int64_t ld16 = user16_ok ? ld_hidden_bf16 : p.ld_h;
            if (ln) {
                float* z = z_ws + off * H;
                fwd.out_f32 = z; fwd.ld_f32 = H;
                RETEXO_TRY(tc_gemm_launch(fwd, st));
                RETEXO_TRY(normalise_rows(model, z, rows, (want_logits || hid16) ? h16 : nullptr, ld16, hid, ld_hidden, st));
            } else {
                fwd.relu = 1; fwd.out_f32 = hid; fwd.ld_f32 = ld_hidden;
                fwd.out_bf16 = (want_logits || hid16) ? h16 : nullptr; fwd.ld_bf16 = ld16;
                RETEXO_TRY(tc_gemm_launch(fwd, st));
            }
            if (hid16 && !user16_ok)      // odd layout asked for: a second, plain copy
                RETEXO_TRY(retexo_pack_rows(hid ? (const void*)hid : (const void*)h16, hid ? 0 : 1, hid ? ld_hidden : p.ld_h, H,
                                            nullptr, rows, hid16, ld_hidden_bf16, nullptr, 0, 0, st));
            if (want_logits) {
                TcGemm l2 = tc_base(h16, ld16, b.w2t16, p.ld_h, rows, O, H, b.status);
                l2.bias = b2; l2.mode = TC_EPI_ARGMAX; l2.out_f32 = lgo; l2.ld_f32 = ld_logits;
                l2.pred = pred; l2.y = yy; l2.correct = correct;
                RETEXO_TRY(tc_gemm_launch(l2, st));
            }
        } else if (want_logits) {
            fwd.mode = TC_EPI_ARGMAX; fwd.out_f32 = lgo; fwd.ld_f32 = ld_logits;
            fwd.pred = pred; fwd.y = yy; fwd.correct = correct;
            RETEXO_TRY(tc_gemm_launch(fwd, st));
        }
        return RETEXO_OK;
    };
    if (row_idx) {
        // gathered rows: packed into a dense batch a chunk at a time, so that these products run on the tensor cores too
        for (int64_t off = 0; off < n_rows; off += kEmbedGatherRows) {
            const int64_t rows = n_rows - off < kEmbedGatherRows ? n_rows - off : kEmbedGatherRows;
            RETEXO_TRY(retexo_pack_rows(x, 1, ldx, d_in, row_idx + off, rows, xg, p.ld_k, nullptr, 0, 0, st));
            RETEXO_TRY(dense(xg, p.ld_k, rows, off));
        }
    } else {
        RETEXO_TRY(dense(static_cast<const bf16*>(x), ldx, n_rows, 0));
    }
    if (model->status_out)
        RETEXO_CUDA_TRY(cudaMemcpyAsync(model->status_out, b.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return launch_status();
}
