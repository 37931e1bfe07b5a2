// Standard (end-to-end) training of the K-layer GNN (Section 2.3), the scheme lazy message passing is compared
// with, on the kernels of the lazy path: every iteration runs the aggregations forward, the last layer with its
// loss as the per-node model's training step (which also returns the gradient with respect to its batch), and
// carries that gradient back through the transposed aggregations and the hidden layers.
//   forward   X^m = AGGR(H^{m-1})  (retexo_aggregate, bf16 out with a column of ones behind it),
//             H^m = ReLU(X^m W_m + b_m)  (tensor-core product over all nodes; fp32 out and one gate bit per unit)
//   last      batch = rows [train | val] of X^K; mlp_train_step_launch with hidden = 0 (loss, dX, update of W_K,
//             validation of the previous iterate riding along, keep-the-best decision)
//   backward  G^K = dX scattered to node order; for m = K-1 .. 1:
//               dH^m = AGGR^T(G^{m+1})   GCN: the aggregation itself (the matrix is symmetric);
//                                        SAGE: g_self + deg .* mean(g_mean ./ deg)  (A symmetric, so the transpose of
//                                        D^-1 A is A D^-1: scale, aggregate with the mean kernel, undo its division)
//               dZ^m = bf16(dH^m .* gate),  [dW_m ; db_m] = [X^m | 1]^T dZ^m  (split over the nodes),
//               G^m = dZ^m W_m^T  (m > 1),  update of layer m.
// X^1 = AGGR(F) is computed once.  No kernel adds floating-point values atomically: results repeat bit for bit.
#include <vector>

#include "common.cuh"
#include "gemm_tc.h"
#include "mlp_plan.h"

using namespace retexo;

namespace retexo {

typedef __nv_bfloat16 bf16;

static inline int64_t std_round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

static __global__ void std_gather_i32_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ idx, int64_t n,
                                             int32_t* __restrict__ dst) {
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < n) dst[i] = src[idx[i]];
}
// x[row][col] = 1 for every row: the all-ones column behind an aggregated matrix (the aggregation kernels write
// the columns of the matrix only, so it stays).
static __global__ void std_ones_column_kernel(bf16* __restrict__ x, int64_t ld, int64_t n, int64_t col) {
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < n) x[i * ld + col] = f32_to_bf16(1.f);
}
// g[idx[i]][0 .. dim) = dx[i][0 .. dim): the batch-ordered input gradient goes to node order (g cleared before).
static __global__ void std_scatter_rows_kernel(const float* __restrict__ dx, int64_t ld_dx, const int32_t* __restrict__ idx,
                                               int64_t n_rows, int32_t dim, float* __restrict__ g, int64_t ld_g) {
    const int64_t t = blockIdx.x * 256ll + threadIdx.x;
    const int64_t i = t / dim;
    const int32_t c = (int32_t)(t % dim);
    if (i < n_rows) g[(int64_t)idx[i] * ld_g + c] = dx[i * ld_dx + c];
}
// s[v][j] = g[v][off + j] / deg v (0 where deg v = 0): the mean half of a SAGE gradient, scaled for the transposed mean.
static __global__ void std_prescale_kernel(const float* __restrict__ g, int64_t ld_g, int32_t off, int32_t dim,
                                           const int64_t* __restrict__ rowptr, int64_t n, float* __restrict__ s, int64_t ld_s) {
    const int64_t t = blockIdx.x * 256ll + threadIdx.x;
    const int64_t v = t / dim;
    const int32_t j = (int32_t)(t % dim);
    if (v >= n) return;
    const int64_t deg = rowptr[v + 1] - rowptr[v];
    s[v * ld_s + j] = deg > 0 ? g[v * ld_g + off + j] / (float)deg : 0.f;
}
// dz[v][j] = bf16(dH[v][j]) where unit j of row v passed the ReLU, else 0, with
//   dH = a[v][j]                         (self == nullptr: GCN, a = AGGR(G))
//   dH = self[v][j] + deg v * a[v][j]    (SAGE: a = mean over N(v) of the scaled gradient rows)
static __global__ void std_gate_kernel(const float* __restrict__ a, int64_t ld_a, const float* __restrict__ self, int64_t ld_self,
                                       const int64_t* __restrict__ rowptr, const uint32_t* __restrict__ bits, int64_t ld_bits,
                                       int64_t n, int32_t dim, bf16* __restrict__ dz, int64_t ld_dz) {
    const int64_t t = blockIdx.x * 256ll + threadIdx.x;
    const int64_t v = t / dim;
    const int32_t j = (int32_t)(t % dim);
    if (v >= n) return;
    float d = a[v * ld_a + j];
    if (self) d = self[v * ld_self + j] + (float)(rowptr[v + 1] - rowptr[v]) * d;
    const bool open = (bits[v * ld_bits + (j >> 5)] >> (j & 31)) & 1u;
    dz[v * ld_dz + j] = f32_to_bf16(open ? d : 0.f);
}
static __global__ void std_copy_if_kernel(const int32_t* decision, const float* src, float* dst, int64_t n) {
    if (!*decision) return;
    const int64_t p = blockIdx.x * 256ll + threadIdx.x;
    if (p < n) dst[p] = src[p];
}
static __global__ void std_snapshot_if_better_kernel(const unsigned long long* cur, const unsigned long long* best,
                                                     const int32_t* have_best, const float* theta, float* theta_best, int64_t nt) {
    if (*have_best && *cur <= *best) return;
    const int64_t p = blockIdx.x * 256ll + threadIdx.x;
    if (p < nt) theta_best[p] = theta[p];
}
static __global__ void std_record_validation_kernel(const unsigned long long* cur, unsigned long long* best, int32_t* have_best,
                                                    int32_t iter, int32_t* best_iter, unsigned long long* history_slot) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    *history_slot = *cur;
    if (!*have_best || *cur > *best) {
        *best = *cur;
        *best_iter = iter;
        *have_best = 1;
    }
}

constexpr int kStdMaxLayers = 8;

struct StdLayer {
    int32_t rep, d, out;        // width of H^{m-1}, of X^m, of the layer's output
    int64_t ldx, ld_k, ld_o1, nt, splits;
    bf16* x;                    // X^m [n x ldx], column d holds ones, the rest of the padding zeros
    float* theta; float* am; float* av; float* best;
    // hidden layers only
    float* h; int64_t ld_h32;   // H^m [n x ld_h32] fp32
    uint32_t* bits; int64_t ld_bits;
    bf16* wt16; bf16* wr16;     // W^T [out x ld_k], W [d x ld_o1]
    float* partial;             // [splits x (d + 1) x out]
};

struct StdBuffers {
    StdLayer L[kStdMaxLayers];
    float* g; int64_t ld_g;     // gradient at an aggregated matrix X^m, node order [n x ld_g]
    float* a; int64_t ld_a;     // result of a transposed aggregation [n x ld_a]
    float* s;                   // SAGE: scaled mean half [n x ld_a]
    bf16* dz; int64_t ld_dz;    // gated gradient [n x ld_dz]
    bf16* xb; int64_t ld_xb;    // batch [train | val] (later: test) rows of X^K with the column of ones
    float* dx; int64_t ld_dx;   // dLoss / d batch rows [n_train x ld_dx]
    int32_t* batch_idx;         // [n_train + n_val]
    int32_t* y_tr; int32_t* y_val; int32_t* y_te;
    unsigned long long* counters;   // cur, done, best
    int32_t* have_best; int32_t* decision; int32_t* best_iter;
    void* ws_step; size_t ws_step_bytes;
    void* ws_agg; size_t ws_agg_bytes;
    void* ws_embed; size_t ws_embed_bytes;
};

static int std_check(const retexo_standard_config* c) {
    if (!c || c->K < 1 || c->R < 1 || c->d0 < 1 || c->n_classes < 1) return RETEXO_ERR_INVALID_ARG;
    if (c->K > kStdMaxLayers) return RETEXO_ERR_UNSUPPORTED;
    if (c->K > 1 && c->hidden < 1) return RETEXO_ERR_INVALID_ARG;
    if (c->aggr != RETEXO_GCN && c->aggr != RETEXO_SAGE_MEAN) return RETEXO_ERR_UNSUPPORTED;
    if (c->n_classes > 64 || c->hidden > 512) return RETEXO_ERR_UNSUPPORTED;
    if (c->optimizer != RETEXO_SGD && c->optimizer != RETEXO_ADAM) return RETEXO_ERR_INVALID_ARG;
    return RETEXO_OK;
}

static void std_dims(const retexo_standard_config& c, int m, StdLayer* l) {
    const int mult = c.aggr == RETEXO_SAGE_MEAN ? 2 : 1;
    l->rep = m == 0 ? c.d0 : c.hidden;
    l->d = l->rep * mult;
    l->out = m < c.K - 1 ? c.hidden : c.n_classes;
    l->ldx = std_round_up((int64_t)l->d + 1, 64);
    l->ld_k = std_round_up(l->d, 64);
    l->ld_o1 = std_round_up(l->out, 64);
    l->nt = ((int64_t)l->d + 1) * l->out;
}

template <typename Taker>
static void std_layout(const retexo_standard_config& c, int64_t n, int64_t e, int64_t n_tr, int64_t n_val, int64_t n_te,
                       Taker& t, StdBuffers* out) {
    StdBuffers b{};
    int32_t max_d = 1, max_rep = 1;
    for (int m = 0; m < c.K; ++m) {
        StdLayer& l = b.L[m];
        std_dims(c, m, &l);
        l.x = t.template take<bf16>((size_t)n * l.ldx);
        l.theta = t.template take<float>((size_t)l.nt);
        l.am = t.template take<float>((size_t)l.nt);
        l.av = t.template take<float>((size_t)l.nt);
        l.best = t.template take<float>((size_t)l.nt);
        if (m < c.K - 1) {
            l.ld_h32 = std_round_up(c.hidden, 32);
            l.ld_bits = 2 * (((int64_t)c.hidden + 63) / 64);
            l.h = t.template take<float>((size_t)n * l.ld_h32);
            l.bits = t.template take<uint32_t>((size_t)n * l.ld_bits);
            l.wt16 = t.template take<bf16>((size_t)l.out * l.ld_k);
            l.wr16 = t.template take<bf16>((size_t)l.d * l.ld_o1);
            l.splits = gemm_split((int64_t)l.d + 1, l.out, n);
            l.partial = t.template take<float>((size_t)l.splits * (l.d + 1) * l.out);
        }
        if (m > 0 && l.d > max_d) max_d = l.d;
        if (l.rep > max_rep && m > 0) max_rep = l.rep;
    }
    const StdLayer& last = b.L[c.K - 1];
    b.ld_g = std_round_up(max_d, 32);
    b.ld_a = std_round_up(c.K > 1 ? c.hidden : 1, 32);
    b.ld_dz = std_round_up(c.K > 1 ? c.hidden : 1, 64);
    b.g = t.template take<float>(c.K > 1 ? (size_t)n * b.ld_g : 1);
    b.a = t.template take<float>(c.K > 1 ? (size_t)n * b.ld_a : 1);
    b.s = t.template take<float>((c.K > 1 && c.aggr == RETEXO_SAGE_MEAN) ? (size_t)n * b.ld_a : 1);
    b.dz = t.template take<bf16>(c.K > 1 ? (size_t)n * b.ld_dz : 1);
    const int64_t n_batch = n_tr + n_val > n_te ? n_tr + n_val : n_te;
    b.ld_xb = last.ldx;
    b.xb = t.template take<bf16>((size_t)n_batch * b.ld_xb);
    b.ld_dx = std_round_up(last.d, 32);
    b.dx = t.template take<float>((size_t)n_tr * b.ld_dx);
    b.batch_idx = t.template take<int32_t>((size_t)(n_tr + n_val));
    b.y_tr = t.template take<int32_t>((size_t)n_tr);
    b.y_val = t.template take<int32_t>(n_val > 0 ? (size_t)n_val : 1);
    b.y_te = t.template take<int32_t>(n_te > 0 ? (size_t)n_te : 1);
    b.counters = t.template take<unsigned long long>(8);
    b.have_best = t.template take<int32_t>(8);
    b.decision = b.have_best + 1;
    b.best_iter = b.have_best + 2;
    b.ws_step_bytes = mlp_step_workspace_size(make_plan(last.d, 0, c.n_classes, n_tr, n_val));
    b.ws_step = t.template take<uint8_t>(b.ws_step_bytes);
    size_t agg = 0;
    for (int m = 0; m < c.K; ++m) {
        const size_t s = retexo_aggregate_workspace_size(n, e, c.aggr, b.L[m].rep, 0);
        if (s > agg) agg = s;
    }
    b.ws_agg_bytes = agg;
    b.ws_agg = t.template take<uint8_t>(agg);
    b.ws_embed_bytes = retexo_embed_workspace_size(last.d, 0, c.n_classes, n);
    b.ws_embed = t.template take<uint8_t>(b.ws_embed_bytes);
    if (out) *out = b;
}

struct StdNullTaker {
    Sizer s;
    template <typename T> T* take(size_t count) { s.take<T>(count); return nullptr; }
};

}  // namespace retexo

extern "C" size_t retexo_standard_workspace_size(const retexo_standard_config* cfg, int64_t n_nodes, int64_t n_edges,
                                                 int64_t n_train, int64_t n_val, int64_t n_test) {
    if (std_check(cfg) != RETEXO_OK || n_nodes < 1 || n_edges < 0 || n_train < 1 || n_val < 0 || n_test < 0) return 0;
    StdNullTaker t;
    std_layout(*cfg, n_nodes, n_edges, n_train, n_val, n_test, t, nullptr);
    return t.s.off + kAlign;
}

extern "C" int retexo_standard_train(const retexo_standard_config* cfg, const retexo_lmp_inputs* in,
                                     const retexo_standard_outputs* out, void* workspace, size_t workspace_bytes,
                                     void* stream) {
    RETEXO_TRY(std_check(cfg));
    if (!in || !out || !in->graph.rowptr || !in->graph.colidx || !in->features || !in->labels || !in->train_idx ||
        !in->theta0 || !out->loss_history)
        return RETEXO_ERR_INVALID_ARG;
    const retexo_standard_config c = *cfg;
    const int64_t n = in->graph.n_nodes, e = in->graph.n_edges;
    const int64_t n_tr = in->n_train, n_val = in->n_val, n_te = in->n_test;
    if (n < 1 || e < 0 || n_tr < 1 || n_val < 0 || n_te < 0 || in->ld_features < c.d0) return RETEXO_ERR_INVALID_ARG;
    if ((n_val > 0 && (!in->val_idx || !out->val_correct)) || (n_te > 0 && !in->test_idx)) return RETEXO_ERR_INVALID_ARG;
    for (int m = 0; m < c.K; ++m)
        if (!in->theta0[m]) return RETEXO_ERR_INVALID_ARG;
    const size_t need = retexo_standard_workspace_size(cfg, n, e, n_tr, n_val, n_te);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    Arena ws(workspace, workspace_bytes);
    StdBuffers b{};
    std_layout(c, n, e, n_tr, n_val, n_te, ws, &b);
    const retexo_csr& g = in->graph;
    const bool sage = c.aggr == RETEXO_SAGE_MEAN;
    const int K = c.K;
    StdLayer& last = b.L[K - 1];

    // ---- set-up: parameters, labels, batch order, the aggregated matrices' padding and column of ones, X^1
    for (int m = 0; m < K; ++m) {
        StdLayer& l = b.L[m];
        RETEXO_CUDA_TRY(cudaMemcpyAsync(l.theta, in->theta0[m], sizeof(float) * (size_t)l.nt, cudaMemcpyDeviceToDevice, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(l.am, 0, sizeof(float) * (size_t)l.nt, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(l.av, 0, sizeof(float) * (size_t)l.nt, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(l.x, 0, sizeof(bf16) * (size_t)n * l.ldx, st));
        std_ones_column_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(l.x, l.ldx, n, l.d);
        if (m < K - 1) RETEXO_TRY(linear_shadows_launch(l.d, l.out, l.theta, l.wt16, l.ld_k, l.wr16, l.ld_o1, st));
    }
    if (K > 1) RETEXO_CUDA_TRY(cudaMemsetAsync(b.dz, 0, sizeof(bf16) * (size_t)n * b.ld_dz, st));
    RETEXO_CUDA_TRY(cudaMemcpyAsync(b.batch_idx, in->train_idx, sizeof(int32_t) * (size_t)n_tr, cudaMemcpyDeviceToDevice, st));
    std_gather_i32_kernel<<<(unsigned)((n_tr + 255) / 256), 256, 0, st>>>(in->labels, in->train_idx, n_tr, b.y_tr);
    if (n_val) {
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.batch_idx + n_tr, in->val_idx, sizeof(int32_t) * (size_t)n_val,
                                        cudaMemcpyDeviceToDevice, st));
        std_gather_i32_kernel<<<(unsigned)((n_val + 255) / 256), 256, 0, st>>>(in->labels, in->val_idx, n_val, b.y_val);
    }
    if (n_te) std_gather_i32_kernel<<<(unsigned)((n_te + 255) / 256), 256, 0, st>>>(in->labels, in->test_idx, n_te, b.y_te);
    RETEXO_CUDA_TRY(cudaMemsetAsync(b.counters, 0, 8 * sizeof(unsigned long long), st));
    RETEXO_CUDA_TRY(cudaMemsetAsync(b.have_best, 0, 8 * sizeof(int32_t), st));
    RETEXO_TRY(launch_status());
    RETEXO_TRY(retexo_aggregate(&g, c.aggr, in->features, in->ld_features, c.d0, nullptr, nullptr, 0, sage ? 1 : 0,
                                b.L[0].x, b.L[0].ldx, b.ws_agg, b.ws_agg_bytes, st));

    const MlpPlan plan = make_plan(last.d, 0, c.n_classes, n_tr, n_val);
    MlpBuffers sb{};
    mlp_step_buffers(plan, b.ws_step, b.ws_step_bytes, &sb);
    retexo_mlp model{};
    model.d_in = last.d; model.hidden = 0; model.n_classes = c.n_classes;
    model.theta = last.theta; model.adam_m = last.am; model.adam_v = last.av;
    model.optimizer = c.optimizer; model.lr = c.lr; model.beta1 = c.beta1; model.beta2 = c.beta2; model.eps = c.eps;
    model.step = 0;
    retexo_mlp best = model;
    best.theta = last.best;

    // Forward of the hidden layers over all nodes with the weights as they stand; leaves X^K in last.x.
    auto forward_hidden = [&]() -> int {
        for (int m = 0; m < K - 1; ++m) {
            StdLayer& l = b.L[m];
            TcGemm f{};
            f.A = l.x; f.lda = l.ldx; f.B = l.wt16; f.ldb = l.ld_k; f.M = n; f.N = l.out; f.K = l.d; f.mode = TC_EPI_BIAS;
            f.bias = l.theta + (int64_t)l.d * l.out; f.relu = 1; f.out_f32 = l.h; f.ld_f32 = l.ld_h32;
            f.relu_bits = l.bits; f.ld_bits = l.ld_bits; f.status = sb.status;
            RETEXO_TRY(tc_gemm_launch(f, st));
            StdLayer& nx = b.L[m + 1];
            RETEXO_TRY(retexo_aggregate(&g, c.aggr, l.h, l.ld_h32, c.hidden, nullptr, nullptr, 0, sage ? 1 : 0, nx.x, nx.ldx,
                                        b.ws_agg, b.ws_agg_bytes, st));
        }
        return RETEXO_OK;
    };
    EvalTail tail{b.y_val, b.counters, b.counters + 2, b.have_best, last.best};
    tail.done = b.counters + 1;
    tail.best_iter = b.best_iter;
    tail.decision = b.decision;

    int pending_it = 0;       // iteration whose weights still await their validation count
    for (int it = 1; it <= c.R; ++it) {
        RETEXO_TRY(forward_hidden());
        RETEXO_TRY(retexo_pack_rows(last.x, 1, last.ldx, last.d, b.batch_idx, n_tr + n_val, b.xb, b.ld_xb, nullptr, 0, 1, st));
        // last layer: loss, dX of the train rows, its own update; the validation rows ride along and count the hits of
        // the weights as they stand, i.e. of iteration it - 1, which the update kernel keeps if they are the best so far
        tail.iter = pending_it;
        tail.history_slot = reinterpret_cast<unsigned long long*>(out->val_correct) + (pending_it > 0 ? pending_it - 1 : 0);
        const EvalTail* riding = pending_it ? &tail : nullptr;
        if (!riding) RETEXO_CUDA_TRY(cudaMemsetAsync(b.decision, 0, sizeof(int32_t), st));
        const bool want_grad = out->grad_last && it == c.R;
        RETEXO_TRY(mlp_train_step_launch(plan, sb, &model, b.xb, b.ld_xb, true, b.y_tr, out->loss_history + (it - 1),
                                         want_grad ? out->grad_last[K - 1] : nullptr, it > 1, riding, st, nullptr,
                                         K > 1 ? b.dx : nullptr, b.ld_dx));
        model.step += 1;
        if (K > 1) {
            RETEXO_CUDA_TRY(cudaMemsetAsync(b.g, 0, sizeof(float) * (size_t)n * b.ld_g, st));
            std_scatter_rows_kernel<<<(unsigned)((n_tr * last.d + 255) / 256), 256, 0, st>>>(b.dx, b.ld_dx, in->train_idx, n_tr,
                                                                                              last.d, b.g, b.ld_g);
        }
        for (int m = K - 2; m >= 0; --m) {
            StdLayer& l = b.L[m];
            const int32_t H = c.hidden;
            // the hidden layers' kept copies follow the last layer's decision (their weights are still iteration it - 1's)
            std_copy_if_kernel<<<(unsigned)((l.nt + 255) / 256), 256, 0, st>>>(b.decision, l.theta, l.best, l.nt);
            // dH^m = AGGR^T(G^{m+1})
            const unsigned eb = (unsigned)((n * H + 255) / 256);
            if (sage) {
                std_prescale_kernel<<<eb, 256, 0, st>>>(b.g, b.ld_g, H, H, g.rowptr, n, b.s, b.ld_a);
                RETEXO_TRY(retexo_aggregate(&g, RETEXO_SAGE_MEAN, b.s, b.ld_a, H, nullptr, b.a, b.ld_a, 0, nullptr, 0, b.ws_agg,
                                            b.ws_agg_bytes, st));
                std_gate_kernel<<<eb, 256, 0, st>>>(b.a, b.ld_a, b.g, b.ld_g, g.rowptr, l.bits, l.ld_bits, n, H, b.dz, b.ld_dz);
            } else {
                RETEXO_TRY(retexo_aggregate(&g, RETEXO_GCN, b.g, b.ld_g, H, nullptr, b.a, b.ld_a, 0, nullptr, 0, b.ws_agg,
                                            b.ws_agg_bytes, st));
                std_gate_kernel<<<eb, 256, 0, st>>>(b.a, b.ld_a, nullptr, 0, g.rowptr, l.bits, l.ld_bits, n, H, b.dz, b.ld_dz);
            }
            // [dW_m ; db_m] = [X^m | 1]^T dZ^m, reduced over the nodes
            TcGemm gw{};
            gw.A = l.x; gw.lda = l.ldx; gw.B = b.dz; gw.ldb = b.ld_dz; gw.M = (int64_t)l.d + 1; gw.N = l.out; gw.K = n;
            gw.mode = TC_EPI_PARTIAL; gw.splits = (int)l.splits; gw.partial = l.partial; gw.status = sb.status;
            RETEXO_TRY(tc_gemm_launch(gw, st));
            if (m > 0) {      // G^m = dZ^m W_m^T, the gradient at X^m (the first layer's input is the data: no gradient needed)
                TcGemm gx{};
                gx.A = b.dz; gx.lda = b.ld_dz; gx.B = l.wr16; gx.ldb = l.ld_o1; gx.M = n; gx.N = l.d; gx.K = l.out;
                gx.mode = TC_EPI_BIAS; gx.out_f32 = b.g; gx.ld_f32 = b.ld_g; gx.status = sb.status;
                RETEXO_TRY(tc_gemm_launch(gx, st));
            }
            RETEXO_TRY(linear_update_launch(l.d, l.out, l.theta, l.am, l.av, l.partial, l.splits, c.optimizer, c.lr, c.beta1,
                                            c.beta2, c.eps, it, l.wt16, l.ld_k, l.wr16, l.ld_o1,
                                            want_grad ? out->grad_last[m] : nullptr, st));
        }
        pending_it = (n_val && it < c.R) ? it : 0;
    }
    // ---- the last iterate has no next iteration to ride on: one more forward pass
    RETEXO_TRY(forward_hidden());
    if (n_val) {
        RETEXO_TRY(retexo_pack_rows(last.x, 1, last.ldx, last.d, in->val_idx, n_val, b.xb, b.ld_xb, nullptr, 0, 0, st));
        RETEXO_TRY(mlp_count_hits_launch(plan, sb, &model, b.xb, b.ld_xb, n_val, nullptr, b.y_val, b.counters, st));
        for (int m = 0; m < K; ++m)
            std_snapshot_if_better_kernel<<<(unsigned)((b.L[m].nt + 255) / 256), 256, 0, st>>>(
                b.counters, b.counters + 2, b.have_best, b.L[m].theta, b.L[m].best, b.L[m].nt);
        std_record_validation_kernel<<<1, 32, 0, st>>>(b.counters, b.counters + 2, b.have_best, c.R, b.best_iter,
                                                       reinterpret_cast<unsigned long long*>(out->val_correct) + (c.R - 1));
    } else {
        for (int m = 0; m < K; ++m)
            RETEXO_CUDA_TRY(cudaMemcpyAsync(b.L[m].best, b.L[m].theta, sizeof(float) * (size_t)b.L[m].nt,
                                            cudaMemcpyDeviceToDevice, st));
        const int32_t r_last = c.R;
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.best_iter, &r_last, sizeof(int32_t), cudaMemcpyHostToDevice, st));
    }
    if (out->best_val_correct)
        RETEXO_CUDA_TRY(cudaMemcpyAsync(out->best_val_correct, b.counters + 2, sizeof(uint64_t), cudaMemcpyDeviceToDevice, st));
    if (out->best_iter)
        RETEXO_CUDA_TRY(cudaMemcpyAsync(out->best_iter, b.best_iter, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));

    // ---- test hits of the last iterate (its X^K is in place), then the kept weights: test hits, logits of all nodes
    if (out->test_correct_last) {
        if (n_te) {
            RETEXO_TRY(retexo_pack_rows(last.x, 1, last.ldx, last.d, in->test_idx, n_te, b.xb, b.ld_xb, nullptr, 0, 0, st));
            RETEXO_TRY(retexo_embed(&model, b.xb, b.ld_xb, nullptr, n_te, nullptr, 0, nullptr, 0, nullptr, 0, nullptr, b.y_te,
                                    out->test_correct_last, b.ws_embed, b.ws_embed_bytes, st));
        } else {
            RETEXO_CUDA_TRY(cudaMemsetAsync(out->test_correct_last, 0, sizeof(uint64_t), st));
        }
    }
    for (int m = 0; m < K - 1; ++m) {
        StdLayer& l = b.L[m];
        RETEXO_CUDA_TRY(cudaMemcpyAsync(l.theta, l.best, sizeof(float) * (size_t)l.nt, cudaMemcpyDeviceToDevice, st));
        RETEXO_TRY(linear_shadows_launch(l.d, l.out, l.theta, l.wt16, l.ld_k, nullptr, 0, st));
    }
    RETEXO_TRY(forward_hidden());
    if (out->test_correct) {
        if (n_te) {
            RETEXO_TRY(retexo_pack_rows(last.x, 1, last.ldx, last.d, in->test_idx, n_te, b.xb, b.ld_xb, nullptr, 0, 0, st));
            RETEXO_TRY(retexo_embed(&best, b.xb, b.ld_xb, nullptr, n_te, nullptr, 0, nullptr, 0, nullptr, 0, nullptr, b.y_te,
                                    out->test_correct, b.ws_embed, b.ws_embed_bytes, st));
        } else {
            RETEXO_CUDA_TRY(cudaMemsetAsync(out->test_correct, 0, sizeof(uint64_t), st));
        }
    }
    if (out->final_logits || out->final_pred)
        RETEXO_TRY(retexo_embed(&best, last.x, last.ldx, nullptr, n, nullptr, 0, nullptr, 0, out->final_logits, out->ld_logits,
                                out->final_pred, nullptr, nullptr, b.ws_embed, b.ws_embed_bytes, st));
    if (out->theta_best)
        for (int m = 0; m < K; ++m)
            if (out->theta_best[m])
                RETEXO_CUDA_TRY(cudaMemcpyAsync(out->theta_best[m], b.L[m].best, sizeof(float) * (size_t)b.L[m].nt,
                                                cudaMemcpyDeviceToDevice, st));
    if (out->status)
        RETEXO_CUDA_TRY(cudaMemcpyAsync(out->status, sb.status, sizeof(int32_t), cudaMemcpyDeviceToDevice, st));
    return launch_status();
}
