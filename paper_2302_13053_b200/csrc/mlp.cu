// Host side of the per-node model calls: argument checks, workspace layout and
// the launch sequence of one training iteration / one embedding pass.
#include "gemm_tc.h"
#include "mlp_kernels.cuh"
#include "mlp_plan.h"

using namespace retexo;

namespace retexo {

static int launch_gemm(const GemmArgs& g, bool a_t, bool b_t, int64_t splits, cudaStream_t st) {
    if (g.M <= 0 || g.N <= 0) return RETEXO_OK;
    dim3 grid((unsigned)((g.N + kBN - 1) / kBN), (unsigned)((g.M + kBM - 1) / kBM), (unsigned)splits);
    if (a_t && b_t) gemm_bf16_kernel<true, true><<<grid, kGemmThreads, 0, st>>>(g);
    else if (a_t) gemm_bf16_kernel<true, false><<<grid, kGemmThreads, 0, st>>>(g);
    else if (b_t) gemm_bf16_kernel<false, true><<<grid, kGemmThreads, 0, st>>>(g);
    else gemm_bf16_kernel<false, false><<<grid, kGemmThreads, 0, st>>>(g);
    return launch_status();
}

static GemmArgs gemm_base(int64_t M, int64_t N, int64_t K, const bf16* A, int64_t lda, const bf16* B, int64_t ldb) {
    GemmArgs g{};
    g.M = M; g.N = N; g.K = K; g.A = A; g.lda = lda; g.B = B; g.ldb = ldb;
    g.a_row_idx = nullptr; g.k_chunk = (K + kBK - 1) / kBK * kBK; if (g.k_chunk == 0) g.k_chunk = kBK;
    g.mode = EPI_BIAS;
    return g;
}

int project_rows_launch(const bf16* A, int64_t lda, const bf16* B, int64_t ldb, int64_t M, int64_t N, int64_t K,
                        float* out, int64_t ld_out, cudaStream_t st) {
    GemmArgs g = gemm_base(M, N, K, A, lda, B, ldb);
    g.mode = EPI_BIAS; g.relu = 0; g.bias = nullptr; g.out_f32 = out; g.ld_f32 = ld_out;
    return launch_gemm(g, false, false, 1, st);
}

int convert_f32_to_bf16_launch(const float* src, bf16* dst, int64_t n, cudaStream_t st) {
    if (n > 0) f32_to_bf16_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(src, dst, n);
    return launch_status();
}

static int64_t split_count(int64_t M, int64_t N, int64_t K) {
    const int64_t tiles = ((M + kBM - 1) / kBM) * ((N + kBN - 1) / kBN);
    int64_t s = (kTargetBlocks + tiles - 1) / tiles;
    const int64_t max_s = (K + 255) / 256;
    if (s > max_s) s = max_s;
    if (s < 1) s = 1;
    if (s > 64) s = 64;
    return s;
}

MlpPlan make_plan(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows) {
    MlpPlan p{};
    p.d_in = d_in; p.hidden = hidden; p.n_classes = n_classes; p.n_rows = n_rows;
    p.out1 = hidden > 0 ? hidden : n_classes;
    p.nt = retexo_theta_size(d_in, hidden, n_classes);
    p.ld_dl = (n_classes + 7) / 8 * 8;
    p.sm_blocks = (n_rows + 7) / 8 < kTargetBlocks ? (n_rows + 7) / 8 : kTargetBlocks;
    if (p.sm_blocks < 1) p.sm_blocks = 1;
    p.tiles_m = (n_rows + kBM - 1) / kBM;
    p.split_w1 = split_count(d_in, p.out1, n_rows);
    p.split_w2 = hidden > 0 ? split_count(hidden, n_classes, n_rows) : 0;
    {   // tensor-core dW1: 128 x {64,128,256} tiles, one block per SM
        const int64_t bn = p.out1 > 128 ? 256 : (p.out1 > 64 ? 128 : 64);
        const int64_t tiles = ((d_in + 127) / 128) * ((p.out1 + bn - 1) / bn);
        int64_t s = 148 / tiles;
        const int64_t kb = (n_rows + 63) / 64;
        if (s > kb) s = kb;
        if (s > 64) s = 64;
        if (s < 1) s = 1;
        p.tc_split_w1 = s;
    }
    p.ld_k = (d_in + 7) / 8 * 8;
    p.ld_n = (n_rows + 7) / 8 * 8;
    return p;
}

template <typename Taker>
static void layout(const MlpPlan& p, Taker& t, MlpBuffers* b) {
    bf16* theta16 = t.template take<bf16>((size_t)p.nt);
    bf16* hd16 = t.template take<bf16>(p.hidden > 0 ? (size_t)p.n_rows * p.hidden : 1);
    float* logits = t.template take<float>((size_t)p.n_rows * p.n_classes);
    bf16* dl16 = t.template take<bf16>((size_t)p.n_rows * p.ld_dl);
    bf16* dhd16 = t.template take<bf16>(p.hidden > 0 ? (size_t)p.n_rows * p.hidden : 1);
    float* loss_partial = t.template take<float>((size_t)p.sm_blocks);
    float* dlsum_partial = t.template take<float>((size_t)p.sm_blocks * p.n_classes);
    float* dhdsum_partial = t.template take<float>(p.hidden > 0 ? (size_t)p.tiles_m * p.hidden : 1);
    const int64_t s1 = p.split_w1 > p.tc_split_w1 ? p.split_w1 : p.tc_split_w1;
    float* pw1 = t.template take<float>((size_t)s1 * p.d_in * p.out1);
    float* pw2 = t.template take<float>(p.hidden > 0 ? (size_t)p.split_w2 * p.hidden * p.n_classes : 1);
    bf16* w1t16 = t.template take<bf16>((size_t)p.out1 * p.ld_k);
    bf16* gradt16 = t.template take<bf16>((size_t)p.out1 * p.ld_n);
    int32_t* status = t.template take<int32_t>(64);
    if (b) {
        b->w1t16 = w1t16; b->gradt16 = gradt16; b->status = status;
        b->theta16 = theta16; b->hd16 = hd16; b->logits = logits; b->dl16 = dl16; b->dhd16 = dhd16;
        b->loss_partial = loss_partial; b->dlsum_partial = dlsum_partial; b->dhdsum_partial = dhdsum_partial;
        b->pw1 = pw1; b->pw2 = pw2;
    }
}

struct NullTaker {
    Sizer s;
    template <typename T> T* take(size_t count) { s.take<T>(count); return nullptr; }
};

static int check_model(const retexo_mlp* m) {
    if (!m || m->d_in <= 0 || m->hidden < 0 || m->n_classes <= 0 || !m->theta) return RETEXO_ERR_INVALID_ARG;
    if (m->n_classes > 64 || m->hidden > 512) return RETEXO_ERR_UNSUPPORTED;
    return RETEXO_OK;
}

}  // namespace retexo

extern "C" int64_t retexo_theta_size(int32_t d_in, int32_t hidden, int32_t n_classes) {
    if (hidden > 0) return (int64_t)d_in * hidden + hidden + (int64_t)hidden * n_classes + n_classes;
    return (int64_t)d_in * n_classes + n_classes;
}

extern "C" int retexo_pack_rows(const void* src, int32_t src_is_bf16, int64_t ld_src, int32_t dim,
                                const int32_t* idx, int64_t n_rows, void* dst, int64_t ld_dst,
                                void* dst_t, int64_t ld_t, void* stream) {
    if (!src || dim <= 0 || ld_src < dim || n_rows < 0 || (!dst && !dst_t)) return RETEXO_ERR_INVALID_ARG;
    if (dst && ld_dst < dim) return RETEXO_ERR_INVALID_ARG;
    if (dst_t && ld_t < n_rows) return RETEXO_ERR_INVALID_ARG;
    const int64_t rows_cover = dst_t ? (ld_t > n_rows ? ld_t : n_rows) : n_rows;
    const int64_t cols_cover = dst ? ld_dst : dim;
    if (rows_cover == 0) return RETEXO_OK;
    dim3 grid((unsigned)((rows_cover + 31) / 32), (unsigned)((cols_cover + 31) / 32));
    if (grid.y > 65535) return RETEXO_ERR_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (src_is_bf16)
        pack_rows_kernel<true><<<grid, 256, 0, st>>>(src, ld_src, dim, idx, n_rows, static_cast<bf16*>(dst), ld_dst,
                                                     static_cast<bf16*>(dst_t), ld_t);
    else
        pack_rows_kernel<false><<<grid, 256, 0, st>>>(src, ld_src, dim, idx, n_rows, static_cast<bf16*>(dst), ld_dst,
                                                      static_cast<bf16*>(dst_t), ld_t);
    return launch_status();
}

extern "C" size_t retexo_mlp_train_step_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes,
                                                       int64_t n_rows) {
    if (d_in <= 0 || hidden < 0 || n_classes <= 0 || n_rows <= 0) return 0;
    MlpPlan p = make_plan(d_in, hidden, n_classes, n_rows);
    NullTaker t;
    layout(p, t, nullptr);
    return t.s.off + kAlign;
}

extern "C" int retexo_mlp_train_step(retexo_mlp* model, const void* x, int64_t ldx, const void* x_t, int64_t ld_xt,
                                     const int32_t* y, int64_t n_rows, float* loss_out, float* grad_out,
                                     void* workspace, size_t workspace_bytes, void* stream) {
    RETEXO_TRY(check_model(model));
    if (!x || !y || n_rows <= 0 || ldx < model->d_in) return RETEXO_ERR_INVALID_ARG;
    if (model->optimizer != RETEXO_SGD && model->optimizer != RETEXO_ADAM) return RETEXO_ERR_INVALID_ARG;
    if (model->optimizer == RETEXO_ADAM && (!model->adam_m || !model->adam_v)) return RETEXO_ERR_INVALID_ARG;
    if (x_t && ld_xt < n_rows) return RETEXO_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || ldx % 8 != 0) return RETEXO_ERR_ALIGNMENT;
    if (x_t && (!aligned_to(x_t, 16) || ld_xt % 8 != 0)) return RETEXO_ERR_ALIGNMENT;
    const size_t need = retexo_mlp_train_step_workspace_size(model->d_in, model->hidden, model->n_classes, n_rows);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);

    const MlpPlan p = make_plan(model->d_in, model->hidden, model->n_classes, n_rows);
    Arena ws(workspace, workspace_bytes);
    MlpBuffers b{};
    layout(p, ws, &b);
    RETEXO_TRY(mlp_train_step_launch(p, b, model, static_cast<const bf16*>(x), ldx,
                                     static_cast<const bf16*>(x_t), ld_xt, y, loss_out, grad_out, st));
    model->step += 1;
    return RETEXO_OK;
}

namespace retexo {

// The launch sequence of one iteration; `model->step` is the count of updates
// already applied.  Shared with the K-round driver.
int mlp_train_step_launch(const MlpPlan& p, const MlpBuffers& b, const retexo_mlp* model,
                          const bf16* x, int64_t ldx, const bf16* x_t, int64_t ld_xt, const int32_t* y,
                          float* loss_out, float* grad_out, cudaStream_t st) {
    const int64_t n = p.n_rows;
    const int32_t d_in = p.d_in, H = p.hidden, O = p.n_classes, out1 = p.out1;
    const float* theta = model->theta;
    RETEXO_CUDA_TRY(cudaMemsetAsync(b.status, 0, sizeof(int32_t), st));
    f32_to_bf16_kernel<<<(unsigned)((p.nt + 255) / 256), 256, 0, st>>>(theta, b.theta16, p.nt);
    const bf16* w1 = b.theta16;
    const float* b1 = theta + (int64_t)d_in * out1;
    const bf16* w2 = b.theta16 + (int64_t)d_in * out1 + out1;
    const float* b2 = b1 + out1 + (int64_t)H * O;

    // The two large products (X W1 and X^T dHd) go to the tensor cores when their operands meet
    // the TMA alignment rules; both operands must then have the reduction dimension contiguous,
    // hence the transposed copies W1^T, X^T (given by the caller) and dHd^T / dL^T.
    TcGemm fwd{};
    fwd.A = x; fwd.lda = ldx; fwd.B = b.w1t16; fwd.ldb = p.ld_k; fwd.M = n; fwd.N = out1; fwd.K = d_in;
    fwd.mode = TC_EPI_BIAS; fwd.relu = H > 0 ? 1 : 0; fwd.bias = b1; fwd.status = b.status;
    if (H > 0) { fwd.out_bf16 = b.hd16; fwd.ld_bf16 = H; } else { fwd.out_f32 = b.logits; fwd.ld_f32 = O; }
    const bool tc_fwd = tc_gemm_supported(fwd);
    TcGemm wg{};
    wg.A = x_t; wg.lda = ld_xt; wg.B = b.gradt16; wg.ldb = p.ld_n; wg.M = d_in; wg.N = out1; wg.K = n;
    wg.mode = TC_EPI_PARTIAL; wg.splits = (int)p.tc_split_w1; wg.partial = b.pw1; wg.status = b.status;
    const bool tc_wg = x_t != nullptr && tc_gemm_supported(wg);
    if (tc_fwd)
        RETEXO_TRY(retexo_pack_rows(theta, 0, out1, out1, nullptr, d_in, nullptr, 0, b.w1t16, p.ld_k, st));

    if (H > 0) {
        // Hd = ReLU(X W1 + b1)
        if (tc_fwd) {
            RETEXO_TRY(tc_gemm_launch(fwd, st));
        } else {
            GemmArgs g = gemm_base(n, H, d_in, x, ldx, w1, H);
            g.mode = EPI_BIAS; g.relu = 1; g.bias = b1; g.out_bf16 = b.hd16; g.ld_bf16 = H;
            RETEXO_TRY(launch_gemm(g, false, false, 1, st));
        }
        // L = Hd W2 + b2
        GemmArgs g = gemm_base(n, O, H, b.hd16, H, w2, O);
        g.mode = EPI_BIAS; g.relu = 0; g.bias = b2; g.out_f32 = b.logits; g.ld_f32 = O;
        RETEXO_TRY(launch_gemm(g, false, false, 1, st));
    } else if (tc_fwd) {
        RETEXO_TRY(tc_gemm_launch(fwd, st));
    } else {
        GemmArgs g = gemm_base(n, O, d_in, x, ldx, w1, O);
        g.mode = EPI_BIAS; g.relu = 0; g.bias = b1; g.out_f32 = b.logits; g.ld_f32 = O;
        RETEXO_TRY(launch_gemm(g, false, false, 1, st));
    }
    softmax_ce_kernel<<<(unsigned)p.sm_blocks, kSmThreads, 0, st>>>(b.logits, O, y, n, O, b.dl16, p.ld_dl,
                                                                    (H == 0 && tc_wg) ? b.gradt16 : nullptr, p.ld_n,
                                                                    b.loss_partial, b.dlsum_partial);
    int64_t w1_parts = p.split_w1;
    if (H > 0) {
        // dHd = (dL W2^T) .* [Hd > 0]   (+ column sums for db1)
        GemmArgs g = gemm_base(n, H, O, b.dl16, p.ld_dl, w2, O);
        g.mode = EPI_MASK; g.mask = b.hd16; g.ld_mask = H; g.colsum = b.dhdsum_partial;
        if (tc_wg) { g.out_bf16_t = b.gradt16; g.ld_t = p.ld_n; }
        else { g.out_bf16 = b.dhd16; g.ld_bf16 = H; }
        RETEXO_TRY(launch_gemm(g, false, true, 1, st));
        // dW2 = Hd^T dL
        g = gemm_base(H, O, n, b.hd16, H, b.dl16, p.ld_dl);
        g.mode = EPI_PARTIAL; g.partial = b.pw2;
        g.k_chunk = ((n + p.split_w2 - 1) / p.split_w2 + kBK - 1) / kBK * kBK;
        RETEXO_TRY(launch_gemm(g, true, false, p.split_w2, st));
    }
    // dW1 = X^T dHd   (last round: X^T dL)
    if (tc_wg) {
        RETEXO_TRY(tc_gemm_launch(wg, st));
        w1_parts = p.tc_split_w1;
    } else {
        GemmArgs g = H > 0 ? gemm_base(d_in, H, n, x, ldx, b.dhd16, H) : gemm_base(d_in, O, n, x, ldx, b.dl16, p.ld_dl);
        g.mode = EPI_PARTIAL; g.partial = b.pw1;
        g.k_chunk = ((n + p.split_w1 - 1) / p.split_w1 + kBK - 1) / kBK * kBK;
        RETEXO_TRY(launch_gemm(g, true, false, p.split_w1, st));
    }

    UpdateArgs u{};
    if (H > 0) {
        u.n_seg = 4;
        u.seg[0] = {(int64_t)d_in * H, b.pw1, w1_parts};
        u.seg[1] = {(int64_t)H, b.dhdsum_partial, p.tiles_m};
        u.seg[2] = {(int64_t)H * O, b.pw2, p.split_w2};
        u.seg[3] = {(int64_t)O, b.dlsum_partial, p.sm_blocks};
    } else {
        u.n_seg = 2;
        u.seg[0] = {(int64_t)d_in * O, b.pw1, w1_parts};
        u.seg[1] = {(int64_t)O, b.dlsum_partial, p.sm_blocks};
    }
    u.theta = model->theta; u.m = model->adam_m; u.v = model->adam_v; u.grad_out = grad_out;
    u.optimizer = model->optimizer; u.lr = model->lr; u.beta1 = model->beta1; u.beta2 = model->beta2;
    u.eps = model->eps;
    const double t = (double)(model->step + 1);
    u.corr1 = (float)(1.0 - pow((double)model->beta1, t));
    u.corr2 = (float)(1.0 - pow((double)model->beta2, t));
    u.loss_partial = b.loss_partial; u.n_loss = p.sm_blocks; u.inv_rows = 1.0f / (float)n; u.loss_out = loss_out; u.status = b.status;
    reduce_update_kernel<<<(unsigned)((p.nt + 255) / 256), 256, 0, st>>>(u);
    return launch_status();
}

}  // namespace retexo

extern "C" size_t retexo_embed_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows) {
    if (d_in <= 0 || hidden < 0 || n_classes <= 0 || n_rows < 0) return 0;
    Sizer s;
    s.take<bf16>((size_t)retexo_theta_size(d_in, hidden, n_classes));
    s.take<bf16>(hidden > 0 ? (size_t)n_rows * hidden : 1);
    s.take<float>((size_t)n_rows * n_classes);
    s.take<bf16>((size_t)(hidden > 0 ? hidden : n_classes) * (size_t)((d_in + 7) / 8 * 8));
    s.take<int32_t>(64);
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
    if ((hidden_out || hidden_out_bf16) && H == 0) return RETEXO_ERR_INVALID_ARG;
    if (hidden_out && ld_hidden < H) return RETEXO_ERR_INVALID_ARG;
    if (hidden_out_bf16 && ld_hidden_bf16 < H) return RETEXO_ERR_INVALID_ARG;
    if (logits_out && ld_logits < O) return RETEXO_ERR_INVALID_ARG;
    if (correct_out && !y) return RETEXO_ERR_INVALID_ARG;
    if (!aligned_to(x, 16) || ldx % 8 != 0) return RETEXO_ERR_ALIGNMENT;
    const size_t need = retexo_embed_workspace_size(d_in, H, O, n_rows);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Arena ws(workspace, workspace_bytes);
    const int64_t nt = retexo_theta_size(d_in, H, O);
    bf16* theta16 = ws.take<bf16>((size_t)nt);
    bf16* hd16 = ws.take<bf16>(H > 0 ? (size_t)n_rows * H : 1);
    float* logits_ws = ws.take<float>((size_t)n_rows * O);
    bf16* w1t16 = ws.take<bf16>((size_t)(H > 0 ? H : O) * (size_t)((d_in + 7) / 8 * 8));
    int32_t* status = ws.take<int32_t>(64);
    return mlp_embed_launch(model, theta16, hd16, logits_ws, w1t16, status, static_cast<const bf16*>(x), ldx, row_idx, n_rows,
                            hidden_out, ld_hidden, static_cast<bf16*>(hidden_out_bf16), ld_hidden_bf16,
                            logits_out, ld_logits, pred_out, y, reinterpret_cast<unsigned long long*>(correct_out), st);
}

namespace retexo {

int mlp_embed_launch(const retexo_mlp* model, bf16* theta16, bf16* hd16_ws, float* logits_ws, bf16* w1t16,
                     int32_t* status, const bf16* x, int64_t ldx, const int32_t* row_idx, int64_t n_rows,
                     float* hidden_out, int64_t ld_hidden, bf16* hidden_out_bf16, int64_t ld_hidden_bf16,
                     float* logits_out, int64_t ld_logits, int32_t* pred_out, const int32_t* y,
                     unsigned long long* correct_out, cudaStream_t st) {
    const int32_t H = model->hidden, O = model->n_classes, d_in = model->d_in;
    const int32_t out1 = H > 0 ? H : O;
    const int64_t nt = retexo_theta_size(d_in, H, O);
    if (correct_out) RETEXO_CUDA_TRY(cudaMemsetAsync(correct_out, 0, sizeof(unsigned long long), st));
    if (n_rows == 0) return RETEXO_OK;
    f32_to_bf16_kernel<<<(unsigned)((nt + 255) / 256), 256, 0, st>>>(model->theta, theta16, nt);
    const bf16* w1 = theta16;
    const float* b1 = model->theta + (int64_t)d_in * out1;
    const bf16* w2 = theta16 + (int64_t)d_in * out1 + out1;
    const float* b2 = b1 + out1 + (int64_t)H * O;
    const bool want_logits = logits_out || pred_out || correct_out;
    float* lg = logits_out ? logits_out : logits_ws;
    const int64_t ld_lg = logits_out ? ld_logits : O;
    const int64_t ld_k = (d_in + 7) / 8 * 8;
    TcGemm fwd{};
    fwd.A = x; fwd.lda = ldx; fwd.B = w1t16; fwd.ldb = ld_k; fwd.M = n_rows; fwd.N = out1; fwd.K = d_in;
    fwd.mode = TC_EPI_BIAS; fwd.relu = H > 0 ? 1 : 0; fwd.bias = b1; fwd.status = status;
    const bool tc_fwd = row_idx == nullptr && tc_gemm_supported(fwd);
    if (tc_fwd) {
        RETEXO_CUDA_TRY(cudaMemsetAsync(status, 0, sizeof(int32_t), st));
        RETEXO_TRY(retexo_pack_rows(model->theta, 0, out1, out1, nullptr, d_in, nullptr, 0, w1t16, ld_k, st));
    }
    if (H > 0) {
        bf16* h16 = hidden_out_bf16 ? hidden_out_bf16 : hd16_ws;
        const int64_t ld16 = hidden_out_bf16 ? ld_hidden_bf16 : H;
        bf16* h16_out = (want_logits || hidden_out_bf16) ? h16 : nullptr;
        if (tc_fwd) {
            fwd.out_f32 = hidden_out; fwd.ld_f32 = ld_hidden; fwd.out_bf16 = h16_out; fwd.ld_bf16 = ld16;
            RETEXO_TRY(tc_gemm_launch(fwd, st));
        } else {
            GemmArgs g = gemm_base(n_rows, H, d_in, x, ldx, w1, H);
            g.a_row_idx = row_idx;
            g.mode = EPI_BIAS; g.relu = 1; g.bias = b1;
            g.out_f32 = hidden_out; g.ld_f32 = ld_hidden;
            g.out_bf16 = h16_out; g.ld_bf16 = ld16;
            RETEXO_TRY(launch_gemm(g, false, false, 1, st));
        }
        if (want_logits) {
            GemmArgs g = gemm_base(n_rows, O, H, h16, ld16, w2, O);
            g.mode = EPI_BIAS; g.relu = 0; g.bias = b2; g.out_f32 = lg; g.ld_f32 = ld_lg;
            RETEXO_TRY(launch_gemm(g, false, false, 1, st));
        }
    } else if (want_logits) {
        if (tc_fwd) {
            fwd.out_f32 = lg; fwd.ld_f32 = ld_lg;
            RETEXO_TRY(tc_gemm_launch(fwd, st));
        } else {
            GemmArgs g = gemm_base(n_rows, O, d_in, x, ldx, w1, O);
            g.a_row_idx = row_idx;
            g.mode = EPI_BIAS; g.relu = 0; g.bias = b1; g.out_f32 = lg; g.ld_f32 = ld_lg;
            RETEXO_TRY(launch_gemm(g, false, false, 1, st));
        }
    }
    if (pred_out || correct_out)
        argmax_kernel<<<(unsigned)((n_rows + 255) / 256), 256, 0, st>>>(lg, ld_lg, n_rows, O, pred_out, y, correct_out);
    return launch_status();
}

}  // namespace retexo
