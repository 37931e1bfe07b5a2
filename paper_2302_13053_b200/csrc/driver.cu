// The K-round lazy-message-passing loop (Section 3.1) run from one host call:
// per round one aggregation, R training iterations with validation and
// best-iterate tracking on the device (no host round trips inside the loop),
// then the emission of the next representations.
#include <vector>

#include "common.cuh"
#include "gemm_tc.h"
#include "mlp_plan.h"

using namespace retexo;

namespace retexo {

typedef __nv_bfloat16 bf16;

static inline int64_t round_up(int64_t x, int64_t a) { return (x + a - 1) / a * a; }

__global__ void gather_i32_kernel(const int32_t* __restrict__ src, const int32_t* __restrict__ idx, int64_t n,
                                  int32_t* __restrict__ dst) {
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < n) dst[i] = src[idx[i]];
}

// Keeps the iterate with the most validation hits, earliest on ties.  Every
// thread takes the same decision from (cur, best); the bookkeeping kernel that
// follows then updates best.
__global__ void snapshot_if_better_kernel(const unsigned long long* cur, const unsigned long long* best,
                                          const int32_t* have_best, const float* theta, float* theta_best,
                                          int64_t nt) {
    if (*have_best && *cur <= *best) return;
    const int64_t p = blockIdx.x * 256ll + threadIdx.x;
    if (p < nt) theta_best[p] = theta[p];
}
__global__ void record_validation_kernel(const unsigned long long* cur, unsigned long long* best, int32_t* have_best,
                                         int32_t iter, int32_t* best_iter, unsigned long long* history_slot) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    *history_slot = *cur;
    if (!*have_best || *cur > *best) {
        *best = *cur;
        *best_iter = iter;
        *have_best = 1;
    }
}
// dz[idx[i]][0 .. dim) = dx[i][0 .. dim): the batch-ordered input gradient goes back to node order.
__global__ void scatter_rows_kernel(const float* __restrict__ dx, int64_t ld_dx, const int32_t* __restrict__ idx,
                                    int64_t n_rows, int32_t dim, float* __restrict__ dz, int64_t ld_dz) {
    const int64_t t = blockIdx.x * 256ll + threadIdx.x;
    const int64_t i = t / dim;
    const int32_t c = (int32_t)(t % dim);
    if (i < n_rows) dz[(int64_t)idx[i] * ld_dz + c] = dx[i * ld_dx + c];
}
// dst = src if *decision is set (the trained aggregator's parameters follow theta into the kept copy).
__global__ void copy_if_kernel(const int32_t* decision, const float* src, float* dst, int64_t n) {
    if (!*decision) return;
    const int64_t p = blockIdx.x * 256ll + threadIdx.x;
    if (p < n) dst[p] = src[p];
}
// One optimiser update of the aggregator's parameters [W_att | a_src | a_dst]: the gradient of W_att is the
// sum of split-K partials (added in index order), those of the attention vectors come ready-made.
// `step` is the 1-based number of this update, read on the device.
__device__ __forceinline__ double whole_power(double base, unsigned long long e) {      // base^e by repeated squaring
    double r = 1.0;
    for (; e; e >>= 1, base *= base) if (e & 1ull) r *= base;
    return r;
}
struct AttUpdateArgs {
    float *att, *m, *v;
    const float* partial; int64_t n_w, splits;
    const float* da; int64_t n_att;
    int optimizer; float lr, beta1, beta2, eps;
    const unsigned long long* step;
    float* grad_out;      // optional
};
__global__ void att_update_kernel(AttUpdateArgs a) {
    const int64_t p = blockIdx.x * 256ll + threadIdx.x;
    if (p >= a.n_att) return;
    float g = 0.f;
    if (p < a.n_w) for (int64_t z = 0; z < a.splits; ++z) g += a.partial[z * a.n_w + p];
    else g = a.da[p - a.n_w];
    if (a.grad_out) a.grad_out[p] = g;
    if (a.optimizer == RETEXO_SGD) { a.att[p] -= a.lr * g; return; }
    const unsigned long long t = *a.step;
    const float c1 = (float)(1.0 - whole_power((double)a.beta1, t)), c2 = (float)(1.0 - whole_power((double)a.beta2, t));
    const float m = a.beta1 * a.m[p] + (1.f - a.beta1) * g;
    const float v = a.beta2 * a.v[p] + (1.f - a.beta2) * g * g;
    a.m[p] = m;
    a.v[p] = v;
    a.att[p] -= a.lr * (m / c1) / (sqrtf(v / c2) + a.eps);
}
// Keeps the first non-zero status of the run.
__global__ void merge_status_kernel(int32_t* run, const int32_t* a, const int32_t* b) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    if (*run == 0 && a && *a != 0) *run = *a;
    if (*run == 0 && b && *b != 0) *run = *b;
}
__global__ void fill_u64_kernel(unsigned long long* p, int64_t n, unsigned long long v) {
    const int64_t i = blockIdx.x * 256ll + threadIdx.x;
    if (i < n) p[i] = v;
}
__global__ void pack_counts_kernel(const uint64_t* cross, const uint64_t* pairs, const uint64_t* total,
                                   const uint64_t* per_round, int K, uint64_t* out) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    out[0] = *cross; out[1] = *pairs; out[2] = *total;
    out[3] = *total == UINT64_MAX ? UINT64_MAX : 2 * *total;
    for (int m = 0; m < K; ++m) out[4 + m] = per_round[m];
}

// A stream of the library's own for the duration of one call, ordered after everything the caller
// has enqueued and joined back into the caller's stream at the end: the iteration loop is recorded
// as a CUDA graph, which the legacy default stream does not allow.  Falls back to the caller's stream.
struct WorkStream {
    cudaStream_t caller, s;
    cudaEvent_t ev = nullptr;
    bool own = false;
    explicit WorkStream(cudaStream_t c) : caller(c), s(c) {
        cudaStream_t ns = nullptr;
        if (cudaStreamCreateWithFlags(&ns, cudaStreamNonBlocking) == cudaSuccess) {
            if (cudaEventCreateWithFlags(&ev, cudaEventDisableTiming) == cudaSuccess &&
                cudaEventRecord(ev, caller) == cudaSuccess && cudaStreamWaitEvent(ns, ev, 0) == cudaSuccess) {
                s = ns;
                own = true;
            } else {
                if (ev) { (void)cudaEventDestroy(ev); ev = nullptr; }
                (void)cudaStreamDestroy(ns);
            }
        }
        (void)cudaGetLastError();
    }
    // Orders the caller's stream after the work enqueued here so far.
    int join() {
        if (!own) return RETEXO_OK;
        if (cudaEventRecord(ev, s) != cudaSuccess || cudaStreamWaitEvent(caller, ev, 0) != cudaSuccess) {
            (void)cudaGetLastError();
            return RETEXO_ERR_CUDA;
        }
        return RETEXO_OK;
    }
    ~WorkStream() {
        if (!own) return;
        (void)join();
        (void)cudaEventDestroy(ev);
        (void)cudaStreamDestroy(s);      // (work already enqueued still runs to completion)
    }
    WorkStream(const WorkStream&) = delete;
    WorkStream& operator=(const WorkStream&) = delete;
};

constexpr int kGraphIterations = 8;      // iterations replayed by one launch of the chunk graph

// Owns an executable graph of one round's training iterations.
struct IterationGraph {
    cudaGraphExec_t exec = nullptr;
    void reset() { if (exec) { (void)cudaGraphExecDestroy(exec); exec = nullptr; } }
    ~IterationGraph() { reset(); }
};

struct RoundDims { int32_t rep_dim, agg_dim, d_in, hidden; };

static RoundDims round_dims(const retexo_lmp_config& c, int m /*1-based*/) {
    RoundDims r;
    r.rep_dim = m == 1 ? c.d0 : c.hidden;
    if (c.aggr == RETEXO_GAT) { r.agg_dim = c.gat_heads * c.gat_head_dim; r.d_in = r.agg_dim; }
    else if (c.aggr == RETEXO_SAGE_MEAN || c.aggr == RETEXO_SAGE_MAX) { r.agg_dim = r.rep_dim; r.d_in = 2 * r.rep_dim; }
    else { r.agg_dim = r.rep_dim; r.d_in = r.rep_dim; }
    r.hidden = m < c.K ? c.hidden : 0;
    return r;
}

struct LmpBuffers {
    // staged inputs (host mode only)
    int64_t* rowptr; int32_t* colidx; float* features; int32_t* labels;
    int32_t *train_idx, *val_idx, *test_idx, *part;
    // representations
    float* q[2];
    bf16* x16; bf16* q16; float* proj; bf16* watt_t16;
    float *att, *att_m, *att_v, *att_best, *att_partial, *da, *dx, *dz; bf16* dp16; int32_t* decision; int32_t* status;
    int64_t att_splits; void* ws_gatbwd; size_t ws_gatbwd_bytes;
    bf16 *xtr16, *xval16;
    int32_t *y_tr, *y_val, *y_test;
    float *theta, *adam_m, *adam_v, *theta_best;
    unsigned long long *cur_correct, *best_correct, *scratch_u64;
    int32_t *have_best, *best_iter_cur, *run_status;
    // device copies of the outputs
    float* loss_history; unsigned long long* val_history;
    unsigned long long *best_val, *test_best, *test_last; int32_t* best_iter;
    uint64_t* counts; uint64_t* count_raw;
    float* final_logits; int32_t* final_pred;
    void *ws_step, *ws_embed, *ws_agg, *ws_count;
    size_t ws_step_bytes, ws_embed_bytes, ws_agg_bytes, ws_count_bytes;
};

template <typename Taker>
static void lmp_layout(const retexo_lmp_config& c, int64_t n, int64_t e, int64_t n_tr, int64_t n_val, int64_t n_te,
                       int32_t n_parts, Taker& t, LmpBuffers* b) {
    LmpBuffers l{};
    const bool host = c.memory_is_host != 0;
    int32_t max_din = 0, max_rep = 0;
    int64_t max_nt = 0;
    size_t step_b = 0, embed_b = 0, agg_b = 0;
    for (int m = 1; m <= c.K; ++m) {
        const RoundDims r = round_dims(c, m);
        if (r.d_in > max_din) max_din = r.d_in;
        if (r.rep_dim > max_rep) max_rep = r.rep_dim;
        const int64_t nt = retexo_theta_size_norm(r.d_in, r.hidden, c.n_classes, c.norm);
        if (nt > max_nt) max_nt = nt;
        size_t s = mlp_step_workspace_size(make_plan(r.d_in, r.hidden, c.n_classes, n_tr, n_val, c.norm));
        if (s > step_b) step_b = s;
        s = retexo_embed_workspace_size_norm(r.d_in, r.hidden, c.n_classes, n, c.norm);
        if (s > embed_b) embed_b = s;
        s = retexo_aggregate_workspace_size(n, e, c.aggr, r.agg_dim, c.gat_heads);
        if (s > agg_b) agg_b = s;
    }
    const int64_t ld16 = round_up(max_din, 64);      // bf16 rows start on 128-byte lines
    l.features = t.template take<float>((size_t)n * round_up(c.d0, 32));   // 128-byte-row copy of the features
    if (host) {
        l.rowptr = t.template take<int64_t>((size_t)n + 1);
        l.colidx = t.template take<int32_t>((size_t)e);
        l.labels = t.template take<int32_t>((size_t)n);
        l.train_idx = t.template take<int32_t>((size_t)n_tr);
        l.val_idx = t.template take<int32_t>((size_t)n_val);
        l.test_idx = t.template take<int32_t>((size_t)n_te);
        l.part = t.template take<int32_t>(n_parts > 0 ? (size_t)n : 1);
    }
    const size_t qsz = c.K > 1 ? (size_t)n * round_up(c.hidden, 32) : 1;
    l.q[0] = t.template take<float>(qsz);
    l.q[1] = t.template take<float>(c.K > 2 ? qsz : 1);
    l.x16 = t.template take<bf16>((size_t)n * ld16);
    if (c.aggr == RETEXO_GAT) {
        const int32_t hd = c.gat_heads * c.gat_head_dim;
        const size_t n_att = (size_t)max_rep * hd + 2 * (size_t)hd;
        l.q16 = t.template take<bf16>((size_t)n * round_up(max_rep, 64));
        l.proj = t.template take<float>((size_t)n * round_up(hd, 32));
        l.watt_t16 = t.template take<bf16>((size_t)hd * round_up(max_rep, 64));
        l.att = t.template take<float>(n_att);
        l.att_m = t.template take<float>(n_att);
        l.att_v = t.template take<float>(n_att);
        l.att_best = t.template take<float>(n_att);
        l.att_splits = gemm_split((int64_t)max_rep, hd, n);
        l.att_partial = t.template take<float>((size_t)l.att_splits * (size_t)max_rep * hd);
        l.da = t.template take<float>((size_t)2 * hd);
        l.dx = t.template take<float>((size_t)n_tr * round_up(hd, 32));
        l.dz = t.template take<float>((size_t)n * round_up(hd, 32));
        l.dp16 = t.template take<bf16>((size_t)n * round_up(hd, 64));
        l.decision = t.template take<int32_t>(64);
        l.status = t.template take<int32_t>(64);
        l.ws_gatbwd_bytes = retexo_gat_backward_workspace_size(n, e, c.gat_heads, hd);
        l.ws_gatbwd = t.template take<char>(l.ws_gatbwd_bytes);
    }
    // training rows, then validation rows, each followed by a column of ones (it carries the bias gradient
    // through the weight-gradient product); after the round's last iteration the test rows take their place
    l.xtr16 = t.template take<bf16>((size_t)(n_tr + n_val > n_te ? n_tr + n_val : n_te) * (size_t)round_up(max_din + 1, 64));
    l.xval16 = nullptr;
    l.y_tr = t.template take<int32_t>((size_t)n_tr);
    l.y_val = t.template take<int32_t>((size_t)(n_val > 0 ? n_val : 1));
    l.y_test = t.template take<int32_t>((size_t)(n_te > 0 ? n_te : 1));
    l.theta = t.template take<float>((size_t)max_nt);
    l.adam_m = t.template take<float>((size_t)max_nt);
    l.adam_v = t.template take<float>((size_t)max_nt);
    l.theta_best = t.template take<float>((size_t)max_nt);
    l.cur_correct = t.template take<unsigned long long>(4);
    l.best_correct = t.template take<unsigned long long>(4);
    l.scratch_u64 = t.template take<unsigned long long>(4);
    l.have_best = t.template take<int32_t>(4);
    l.best_iter_cur = t.template take<int32_t>(4);
    l.run_status = t.template take<int32_t>(4);
    l.loss_history = t.template take<float>((size_t)c.K * c.R);
    l.val_history = t.template take<unsigned long long>((size_t)c.K * c.R);
    l.best_val = t.template take<unsigned long long>((size_t)c.K);
    l.test_best = t.template take<unsigned long long>((size_t)c.K);
    l.test_last = t.template take<unsigned long long>((size_t)c.K);
    l.best_iter = t.template take<int32_t>((size_t)c.K);
    l.counts = t.template take<uint64_t>((size_t)4 + c.K);
    l.count_raw = t.template take<uint64_t>((size_t)4 + c.K);
    if (host) {
        l.final_logits = t.template take<float>((size_t)n * c.n_classes);
        l.final_pred = t.template take<int32_t>((size_t)n);
    }
    l.ws_step_bytes = step_b; l.ws_embed_bytes = embed_b; l.ws_agg_bytes = agg_b;
    l.ws_count_bytes = n_parts > 0 ? retexo_cross_partition_workspace_size(n, e, n_parts) : 0;
    l.ws_step = t.template take<char>(step_b);
    l.ws_embed = t.template take<char>(embed_b);
    l.ws_agg = t.template take<char>(agg_b);
    l.ws_count = t.template take<char>(l.ws_count_bytes ? l.ws_count_bytes : 1);
    if (b) *b = l;
}

struct NullTaker2 {
    Sizer s;
    template <typename T> T* take(size_t count) { s.take<T>(count); return nullptr; }
};

static int check_cfg(const retexo_lmp_config* c) {
    if (!c) return RETEXO_ERR_INVALID_ARG;
    if (c->K < 1 || c->K > 8 || c->R < 1 || c->d0 <= 0 || c->n_classes <= 0) return RETEXO_ERR_INVALID_ARG;
    if (c->K > 1 && c->hidden <= 0) return RETEXO_ERR_INVALID_ARG;
    if (c->aggr != RETEXO_GCN && c->aggr != RETEXO_SAGE_MEAN && c->aggr != RETEXO_GAT && c->aggr != RETEXO_SAGE_MAX)
        return RETEXO_ERR_INVALID_ARG;
    if (c->aggr == RETEXO_GAT && (c->gat_heads <= 0 || c->gat_head_dim <= 0)) return RETEXO_ERR_INVALID_ARG;
    if (c->eval_every < 1) return RETEXO_ERR_INVALID_ARG;
    if (!(c->dropout >= 0.f && c->dropout < 1.f)) return RETEXO_ERR_INVALID_ARG;
    if (c->n_classes > 64 || c->hidden > 512) return RETEXO_ERR_UNSUPPORTED;
    if (c->norm != RETEXO_NORM_NONE && c->norm != RETEXO_NORM_LAYER && c->norm != RETEXO_NORM_BATCH) return RETEXO_ERR_INVALID_ARG;
    if (c->norm && !(c->norm_eps > 0.f)) return RETEXO_ERR_INVALID_ARG;
    if (c->norm == RETEXO_NORM_BATCH && !(c->bn_momentum >= 0.f && c->bn_momentum <= 1.f)) return RETEXO_ERR_INVALID_ARG;
    if (c->norm && c->dropout > 0.f) return RETEXO_ERR_UNSUPPORTED;
    return RETEXO_OK;
}

}  // namespace retexo

extern "C" size_t retexo_lmp_workspace_size(const retexo_lmp_config* cfg, int64_t n_nodes, int64_t n_edges,
                                            int64_t n_train, int64_t n_val, int64_t n_test, int32_t n_parts) {
    if (check_cfg(cfg) != RETEXO_OK || n_nodes <= 0 || n_edges < 0 || n_train <= 0 || n_val < 0 || n_test < 0) return 0;
    NullTaker2 t;
    lmp_layout(*cfg, n_nodes, n_edges, n_train, n_val, n_test, n_parts, t, nullptr);
    return t.s.off + kAlign;
}

extern "C" int retexo_lmp_train(const retexo_lmp_config* cfg, const retexo_lmp_inputs* in,
                                const retexo_lmp_outputs* out, void* workspace, size_t workspace_bytes,
                                void* stream) {
    RETEXO_TRY(check_cfg(cfg));
    if (!in || !out) return RETEXO_ERR_INVALID_ARG;
    const retexo_lmp_config& c = *cfg;
    const int64_t n = in->graph.n_nodes, e = in->graph.n_edges;
    if (n <= 0 || e < 0 || n > INT32_MAX || !in->graph.rowptr || (e > 0 && !in->graph.colidx)) return RETEXO_ERR_INVALID_ARG;
    if (!in->features || in->ld_features < c.d0 || !in->labels) return RETEXO_ERR_INVALID_ARG;
    if (!in->train_idx || in->n_train <= 0 || in->n_val < 0 || in->n_test < 0) return RETEXO_ERR_INVALID_ARG;
    if ((in->n_val > 0 && !in->val_idx) || (in->n_test > 0 && !in->test_idx)) return RETEXO_ERR_INVALID_ARG;
    if (!in->theta0 || (c.aggr == RETEXO_GAT && !in->gat_w)) return RETEXO_ERR_INVALID_ARG;
    for (int m = 0; m < c.K; ++m) {
        if (!in->theta0[m]) return RETEXO_ERR_INVALID_ARG;
        if (c.aggr == RETEXO_GAT && !in->gat_w[m]) return RETEXO_ERR_INVALID_ARG;
    }
    if (in->part && in->n_parts <= 0) return RETEXO_ERR_INVALID_ARG;
    if (out->final_logits && out->ld_logits < c.n_classes) return RETEXO_ERR_INVALID_ARG;
    const int32_t n_parts = in->part ? in->n_parts : 0;
    const size_t need = retexo_lmp_workspace_size(cfg, n, e, in->n_train, in->n_val, in->n_test, n_parts);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    WorkStream work(static_cast<cudaStream_t>(stream));
    cudaStream_t st = work.s;
    IterationGraph iteration, chunk;
    const bool host = c.memory_is_host != 0;
    const cudaMemcpyKind in_kind = host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice;
    const cudaMemcpyKind out_kind = host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice;

    Arena ws(workspace, workspace_bytes);
    LmpBuffers b{};
    lmp_layout(c, n, e, in->n_train, in->n_val, in->n_test, n_parts, ws, &b);
    const int64_t n_tr = in->n_train, n_val = in->n_val, n_te = in->n_test;

    // ---- inputs
    retexo_csr g = in->graph;
    const float* feat = in->features;
    int64_t ld_feat = in->ld_features;
    const int32_t *labels = in->labels, *train_idx = in->train_idx, *val_idx = in->val_idx, *test_idx = in->test_idx;
    const int32_t* part = in->part;
    if (host) {
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.rowptr, g.rowptr, sizeof(int64_t) * (size_t)(n + 1), in_kind, st));
        if (e > 0) RETEXO_CUDA_TRY(cudaMemcpyAsync(b.colidx, g.colidx, sizeof(int32_t) * (size_t)e, in_kind, st));
        const int64_t ldp = round_up(c.d0, 32);
        if (ldp != c.d0) RETEXO_CUDA_TRY(cudaMemsetAsync(b.features, 0, sizeof(float) * (size_t)n * ldp, st));
        RETEXO_CUDA_TRY(cudaMemcpy2DAsync(b.features, sizeof(float) * ldp, feat, sizeof(float) * ld_feat,
                                          sizeof(float) * c.d0, (size_t)n, in_kind, st));
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.labels, labels, sizeof(int32_t) * (size_t)n, in_kind, st));
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.train_idx, train_idx, sizeof(int32_t) * (size_t)n_tr, in_kind, st));
        if (n_val) RETEXO_CUDA_TRY(cudaMemcpyAsync(b.val_idx, val_idx, sizeof(int32_t) * (size_t)n_val, in_kind, st));
        if (n_te) RETEXO_CUDA_TRY(cudaMemcpyAsync(b.test_idx, test_idx, sizeof(int32_t) * (size_t)n_te, in_kind, st));
        if (part) RETEXO_CUDA_TRY(cudaMemcpyAsync(b.part, part, sizeof(int32_t) * (size_t)n, in_kind, st));
        g.rowptr = b.rowptr; g.colidx = b.colidx; feat = b.features; ld_feat = ldp;
        labels = b.labels; train_idx = b.train_idx; val_idx = b.val_idx; test_idx = b.test_idx;
        if (part) part = b.part;
    } else if (ld_feat % 4 != 0 || !aligned_to(feat, 16)) {
        // rows that do not start on 16-byte boundaries would force narrow loads on the dominant
        // gather of round 1: re-lay them once with rows of whole 128-byte lines
        const int64_t ldp = round_up(c.d0, 32);
        if (ldp != c.d0) RETEXO_CUDA_TRY(cudaMemsetAsync(b.features, 0, sizeof(float) * (size_t)n * ldp, st));
        RETEXO_CUDA_TRY(cudaMemcpy2DAsync(b.features, sizeof(float) * ldp, feat, sizeof(float) * ld_feat,
                                          sizeof(float) * c.d0, (size_t)n, cudaMemcpyDeviceToDevice, st));
        feat = b.features;
        ld_feat = ldp;
    }
    gather_i32_kernel<<<(unsigned)((n_tr + 255) / 256), 256, 0, st>>>(labels, train_idx, n_tr, b.y_tr);
    if (n_val) gather_i32_kernel<<<(unsigned)((n_val + 255) / 256), 256, 0, st>>>(labels, val_idx, n_val, b.y_val);
    if (n_te) gather_i32_kernel<<<(unsigned)((n_te + 255) / 256), 256, 0, st>>>(labels, test_idx, n_te, b.y_test);
    fill_u64_kernel<<<(unsigned)(((int64_t)c.K * c.R + 255) / 256), 256, 0, st>>>(b.val_history, (int64_t)c.K * c.R,
                                                                                  ~0ull);
    RETEXO_CUDA_TRY(cudaMemsetAsync(b.run_status, 0, sizeof(int32_t), st));

    // ---- messages and bytes across the partition, all rounds
    if (part) {
        int32_t dims[8];
        for (int m = 1; m <= c.K; ++m) dims[m - 1] = round_dims(c, m).rep_dim;
        RETEXO_TRY(retexo_cross_partition_bytes(&g, part, n_parts, c.K, dims, 4, b.count_raw, b.count_raw + 1,
                                                b.count_raw + 4, b.count_raw + 2, nullptr, nullptr, b.ws_count,
                                                b.ws_count_bytes, st));
        pack_counts_kernel<<<1, 32, 0, st>>>(b.count_raw, b.count_raw + 1, b.count_raw + 2, b.count_raw + 4, c.K,
                                             b.counts);
    }

    {   // padding columns of the bf16 inputs are never read as data, but keep them defined
        int32_t max_din = 0;
        for (int m = 1; m <= c.K; ++m) if (round_dims(c, m).d_in > max_din) max_din = round_dims(c, m).d_in;
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.x16, 0, sizeof(bf16) * (size_t)n * (size_t)round_up(max_din, 64), st));
    }
    const float* q = feat;
    int64_t ldq = ld_feat;
    for (int m = 1; m <= c.K; ++m) {
        const RoundDims r = round_dims(c, m);
        const int64_t ld16 = round_up(r.d_in, 64);
        const int64_t nt = retexo_theta_size_norm(r.d_in, r.hidden, c.n_classes, c.norm);

        // ---- one message-passing round: X = COMBINE(Q, AGGR(Q)), emitted in bf16 for the model
        const bool gat = c.aggr == RETEXO_GAT;
        const bool gat_train = gat && !c.gat_freeze_attention;      // the round trains the aggregator too
        const int32_t hd = gat ? r.agg_dim : 0;
        const int64_t ldq16 = round_up(r.rep_dim, 64), ldp = round_up(hd > 0 ? hd : 1, 32);
        const int64_t n_att = (int64_t)r.rep_dim * hd + 2 * (int64_t)hd;
        // GAT: P = Q W_att on the tensor cores (a bias-free product), then scores, soft-max and weighted sum in
        // one pass, with the projection and attention vectors at `att` = [W_att | a_src | a_dst]
        auto gat_forward = [&](const float* att) -> int {
            RETEXO_TRY(retexo_pack_rows(att, 0, hd, hd, nullptr, r.rep_dim, nullptr, 0, b.watt_t16, ldq16, 0, st));
            TcGemm pr{};
            pr.A = b.q16; pr.lda = ldq16; pr.B = b.watt_t16; pr.ldb = ldq16; pr.M = n; pr.N = hd; pr.K = r.rep_dim;
            pr.mode = TC_EPI_BIAS; pr.out_f32 = b.proj; pr.ld_f32 = ldp; pr.status = b.status;
            RETEXO_TRY(tc_gemm_launch(pr, st));
            retexo_gat_params gp;
            gp.heads = c.gat_heads; gp.head_dim = c.gat_head_dim; gp.a_src = att + (int64_t)r.rep_dim * hd;
            gp.a_dst = gp.a_src + hd; gp.negative_slope = c.gat_negative_slope; gp.add_self_loop = 1;
            return retexo_aggregate(&g, RETEXO_GAT, b.proj, ldp, hd, &gp, nullptr, 0, 0, b.x16, ld16, b.ws_agg,
                                    b.ws_agg_bytes, st);
        };
        if (gat) {
            RETEXO_CUDA_TRY(cudaMemcpyAsync(b.att, in->gat_w[m - 1], sizeof(float) * (size_t)n_att, cudaMemcpyDefault, st));
            RETEXO_CUDA_TRY(cudaMemcpyAsync(b.att_best, b.att, sizeof(float) * (size_t)n_att, cudaMemcpyDeviceToDevice, st));
            RETEXO_CUDA_TRY(cudaMemsetAsync(b.status, 0, sizeof(int32_t), st));
            RETEXO_TRY(retexo_pack_rows(q, 0, ldq, r.rep_dim, nullptr, n, b.q16, ldq16, nullptr, 0, 0, st));
            if (gat_train) {
                RETEXO_CUDA_TRY(cudaMemsetAsync(b.att_m, 0, sizeof(float) * (size_t)n_att, st));
                RETEXO_CUDA_TRY(cudaMemsetAsync(b.att_v, 0, sizeof(float) * (size_t)n_att, st));
                RETEXO_CUDA_TRY(cudaMemsetAsync(b.dz, 0, sizeof(float) * (size_t)n * (size_t)ldp, st));
                RETEXO_CUDA_TRY(cudaMemsetAsync(b.decision, 0, sizeof(int32_t), st));
            } else {
                RETEXO_TRY(gat_forward(b.att));
            }
        } else {
            RETEXO_TRY(retexo_aggregate(&g, c.aggr, q, ldq, r.agg_dim, nullptr, nullptr, 0, 1, b.x16, ld16, b.ws_agg,
                                        b.ws_agg_bytes, st));
        }

        // ---- the round's batches and model state
        const int64_t ld_tr = round_up(r.d_in + 1, 64);
        bf16* xval16 = b.xtr16 + (size_t)n_tr * ld_tr;
        // the training rows (followed by their column of ones), then the validation rows; a round that trains
        // its aggregator packs them anew after every local aggregation
        auto pack_batches = [&]() -> int {
            RETEXO_TRY(retexo_pack_rows(b.x16, 1, ld16, r.d_in, train_idx, n_tr, b.xtr16, ld_tr, nullptr, 0, 1, st));
            if (n_val) RETEXO_TRY(retexo_pack_rows(b.x16, 1, ld16, r.d_in, val_idx, n_val, xval16, ld_tr, nullptr, 0, 0, st));
            return RETEXO_OK;
        };
        if (!gat_train) RETEXO_TRY(pack_batches());
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.theta, in->theta0[m - 1], sizeof(float) * (size_t)nt, cudaMemcpyDefault, st));
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.theta_best, b.theta, sizeof(float) * (size_t)nt, cudaMemcpyDeviceToDevice, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.adam_m, 0, sizeof(float) * (size_t)nt, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.adam_v, 0, sizeof(float) * (size_t)nt, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.best_correct, 0, sizeof(unsigned long long), st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.have_best, 0, sizeof(int32_t), st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.best_iter_cur, 0, sizeof(int32_t), st));

        retexo_mlp model{};
        model.d_in = r.d_in; model.hidden = r.hidden; model.n_classes = c.n_classes;
        model.theta = b.theta; model.adam_m = b.adam_m; model.adam_v = b.adam_v;
        model.optimizer = c.optimizer; model.lr = c.lr; model.beta1 = c.beta1; model.beta2 = c.beta2;
        model.eps = c.eps; model.step = 0;
        model.dropout = c.dropout; model.dropout_seed = c.dropout_seed + (uint64_t)(m - 1);
        model.status_out = nullptr;
        model.norm = c.norm; model.norm_eps = c.norm_eps; model.bn_momentum = c.bn_momentum;
        retexo_mlp best = model;
        best.theta = b.theta_best;

        // ---- R training iterations; validation and best-iterate tracking stay on the device
        const MlpPlan plan = make_plan(r.d_in, r.hidden, c.n_classes, n_tr, n_val, c.norm);
        MlpBuffers sb{};
        mlp_step_buffers(plan, b.ws_step, b.ws_step_bytes, &sb);
        bf16* val_hd = reinterpret_cast<bf16*>(b.ws_embed);      // [n_val x ld_h] scratch of a stand-alone validation forward
        // (normalisation: its fp32 pre-normalisation rows [n_val x hidden] sit behind it; the embedding workspace
        //  is sized for all n >= n_val rows of both)
        float* val_z = reinterpret_cast<float*>(reinterpret_cast<uint8_t*>(b.ws_embed) +
                                                round_up((int64_t)sizeof(bf16) * n_val * plan.ld_h, 256));
        // cur_correct[0]: hits of the validation rows riding along; cur_correct[1]: the update kernel's
        // count of finished blocks.  Both are cleared here once and left clear by the update kernel.
        // cur_correct[2]: updates applied so far in this round (the iteration number lives on the device).
        RETEXO_CUDA_TRY(cudaMemsetAsync(b.cur_correct, 0, 3 * sizeof(unsigned long long), st));
        EvalTail tail{b.y_val, b.cur_correct, b.best_correct, b.have_best, b.theta_best};
        tail.done = b.cur_correct + 1;
        tail.best_iter = b.best_iter_cur;
        const DeviceIter dev{b.cur_correct + 2, b.cur_correct + 1, b.loss_history + (size_t)(m - 1) * c.R,
                             b.val_history + (size_t)(m - 1) * c.R};
        // With validation every iteration (or none) all iterations from the second on are the same six
        // launches with the same arguments: the second one is recorded as a graph, the rest replay it.
        const bool uniform = work.own && c.R > 3 && (n_val == 0 || c.eval_every == 1);
        tail.decision = gat_train ? b.decision : nullptr;
        const int64_t ld_dx = ldp;
        // What a round that trains its aggregator adds to an iteration (Section 3.1: after the round's exchange
        // everything an iteration needs is local, so the aggregation is redone with the current parameters):
        // before the step, projection + aggregation + batches; after it, the kept copy follows theta's, the
        // input gradient goes back through the attention, and [W_att | a_src | a_dst] take their update.
        auto gat_backward_and_update = [&]() -> int {
            copy_if_kernel<<<(unsigned)((n_att + 255) / 256), 256, 0, st>>>(b.decision, b.att, b.att_best, n_att);
            scatter_rows_kernel<<<(unsigned)((n_tr * hd + 255) / 256), 256, 0, st>>>(b.dx, ld_dx, train_idx, n_tr, hd, b.dz, ldp);
            retexo_gat_params gp;
            gp.heads = c.gat_heads; gp.head_dim = c.gat_head_dim; gp.a_src = b.att + (int64_t)r.rep_dim * hd;
            gp.a_dst = gp.a_src + hd; gp.negative_slope = c.gat_negative_slope; gp.add_self_loop = 1;
            RETEXO_TRY(retexo_gat_backward(&g, b.proj, ldp, &gp, b.dz, ldp, nullptr, 0, b.dp16, round_up(hd, 64), b.da,
                                           b.da + hd, b.ws_gatbwd, b.ws_gatbwd_bytes, st));
            TcGemm gw{};      // dW_att = Q^T dP, reduced over the nodes
            gw.A = b.q16; gw.lda = ldq16; gw.B = b.dp16; gw.ldb = round_up(hd, 64); gw.M = r.rep_dim; gw.N = hd; gw.K = n;
            gw.mode = TC_EPI_PARTIAL; gw.splits = (int)gemm_split(r.rep_dim, hd, n); gw.partial = b.att_partial;
            gw.status = b.status;
            RETEXO_TRY(tc_gemm_launch(gw, st));
            AttUpdateArgs au{};
            au.att = b.att; au.m = b.att_m; au.v = b.att_v; au.partial = b.att_partial; au.n_w = (int64_t)r.rep_dim * hd;
            au.splits = gw.splits; au.da = b.da; au.n_att = n_att; au.optimizer = c.optimizer; au.lr = c.lr;
            au.beta1 = c.beta1; au.beta2 = c.beta2; au.eps = c.eps; au.step = b.cur_correct + 2;      // (already advanced)
            att_update_kernel<<<(unsigned)((n_att + 255) / 256), 256, 0, st>>>(au);
            return launch_status();
        };
        iteration.reset();
        chunk.reset();
        bool graphs_ok = true;
        int pending_it = 0;       // iteration whose weights still await their validation count
        for (int it = 1; it <= c.R; ++it) {
            int done_now = 1;     // iterations this pass of the loop enqueues
            float* loss_slot = b.loss_history + (size_t)(m - 1) * c.R + (it - 1);
            // The weights of iteration it-1 are validated inside this iteration's forward pass (the
            // validation rows ride along; the update kernel keeps them if they are the best so far).
            // The update of iteration it-1 also left bf16 copies of the current weights behind.
            // (its count is recorded as iteration pending_it's by the update kernel's last block)
            tail.iter = pending_it;
            tail.history_slot = b.val_history + (size_t)(m - 1) * c.R + (pending_it > 0 ? pending_it - 1 : 0);
            const EvalTail* riding = pending_it ? &tail : nullptr;
            // one iteration's launches (with a trained aggregator: projection, aggregation and batches before the
            // per-node model's step, the attention's backward pass and update after it)
            auto enqueue = [&](bool shadows_ready) -> int {
                if (!gat_train)
                    return mlp_train_step_launch(plan, sb, &model, b.xtr16, ld_tr, true, b.y_tr, loss_slot, nullptr,
                                                 shadows_ready, riding, st, &dev);
                RETEXO_TRY(gat_forward(b.att));
                RETEXO_TRY(pack_batches());
                if (!riding) RETEXO_CUDA_TRY(cudaMemsetAsync(b.decision, 0, sizeof(int32_t), st));
                RETEXO_TRY(mlp_train_step_launch(plan, sb, &model, b.xtr16, ld_tr, true, b.y_tr, loss_slot, nullptr,
                                                 shadows_ready, riding, st, &dev, b.dx, ld_dx));
                return gat_backward_and_update();
            };
            if (uniform && it >= 2) {
                // Iterations 2..R are the same launches (their iteration-dependent state lives on the device), so
                // they are replayed from graphs: a chunk of kGraphIterations while that many remain (inside a
                // graph consecutive kernels overlap their set-up with the predecessor's tail, across graph
                // launches they do not), a single iteration for the rest.
                auto record = [&](IterationGraph& gr, int count) -> bool {
                    bool recorded = false;
                    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeRelaxed) == cudaSuccess) {
                        int rc = RETEXO_OK;
                        for (int i = 0; i < count && rc == RETEXO_OK; ++i) rc = enqueue(true);
                        cudaGraph_t graph = nullptr;
                        const cudaError_t ended = cudaStreamEndCapture(st, &graph);
                        if (rc == RETEXO_OK && ended == cudaSuccess && graph &&
                            cudaGraphInstantiate(&gr.exec, graph, 0) == cudaSuccess)
                            recorded = true;
                        if (graph) (void)cudaGraphDestroy(graph);
                    }
                    (void)cudaGetLastError();
                    if (!recorded) gr.reset();
                    return recorded;
                };
                const int remaining = c.R - it + 1;
                if (graphs_ok && remaining >= kGraphIterations && (chunk.exec || record(chunk, kGraphIterations))) {
                    RETEXO_CUDA_TRY(cudaGraphLaunch(chunk.exec, st));
                    done_now = kGraphIterations;
                } else if (graphs_ok && (iteration.exec || record(iteration, 1))) {
                    RETEXO_CUDA_TRY(cudaGraphLaunch(iteration.exec, st));
                } else {      // no graph on this stream: plain launches
                    graphs_ok = false;
                    RETEXO_TRY(enqueue(true));
                }
            } else {
                RETEXO_TRY(enqueue(it > 1));
            }
            it += done_now - 1;
            model.step += done_now - 1;
            model.step += 1;
            const bool want = n_val && (it % c.eval_every == 0 || it == c.R);
            pending_it = (want && it < c.R) ? it : 0;
            if (want && it == c.R) {      // the last iterate has no next iteration to ride on
                if (gat_train) {
                    RETEXO_TRY(gat_forward(b.att));
                    RETEXO_TRY(pack_batches());
                }
                RETEXO_TRY(mlp_count_hits_launch(plan, sb, &model, xval16, ld_tr, n_val, val_hd, b.y_val,
                                                 b.cur_correct, st, val_z));
                snapshot_if_better_kernel<<<(unsigned)((nt + 255) / 256), 256, 0, st>>>(
                    b.cur_correct, b.best_correct, b.have_best, b.theta, b.theta_best, nt);
                if (gat_train)
                    snapshot_if_better_kernel<<<(unsigned)((n_att + 255) / 256), 256, 0, st>>>(
                        b.cur_correct, b.best_correct, b.have_best, b.att, b.att_best, n_att);
                record_validation_kernel<<<1, 32, 0, st>>>(b.cur_correct, b.best_correct, b.have_best, it,
                                                           b.best_iter_cur,
                                                           b.val_history + (size_t)(m - 1) * c.R + (it - 1));
            }
        }
        if (!n_val) {   // nothing to select on: keep the last iterate
            if (gat_train)
                RETEXO_CUDA_TRY(cudaMemcpyAsync(b.att_best, b.att, sizeof(float) * (size_t)n_att, cudaMemcpyDeviceToDevice, st));
            RETEXO_CUDA_TRY(cudaMemcpyAsync(b.theta_best, b.theta, sizeof(float) * (size_t)nt, cudaMemcpyDeviceToDevice, st));
            const int32_t last = c.R;
            RETEXO_CUDA_TRY(cudaMemcpyAsync(b.best_iter_cur, &last, sizeof(int32_t), cudaMemcpyHostToDevice, st));
        }
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.best_val + (m - 1), b.best_correct, sizeof(unsigned long long),
                                        cudaMemcpyDeviceToDevice, st));
        RETEXO_CUDA_TRY(cudaMemcpyAsync(b.best_iter + (m - 1), b.best_iter_cur, sizeof(int32_t),
                                        cudaMemcpyDeviceToDevice, st));

        // ---- test accuracy of the kept and of the last iterate
        if (n_te) {
            // the test rows are gathered once into a dense batch (the training batch is no longer needed),
            // so both forward passes run on the tensor cores
            bf16* xte16 = b.xtr16;
            if (gat_train) RETEXO_TRY(gat_forward(b.att));           // the last iterate's own aggregation
            RETEXO_TRY(retexo_pack_rows(b.x16, 1, ld16, r.d_in, test_idx, n_te, xte16, ld16, nullptr, 0, 0, st));
            RETEXO_TRY(retexo_embed(&model, xte16, ld16, nullptr, n_te, nullptr, 0, nullptr, 0, nullptr, 0, nullptr,
                                    b.y_test, reinterpret_cast<uint64_t*>(b.test_last + (m - 1)), b.ws_embed,
                                    b.ws_embed_bytes, st));
            if (gat_train) {                                          // the kept iterate's: x16 then stays for the emission
                RETEXO_TRY(gat_forward(b.att_best));
                RETEXO_TRY(retexo_pack_rows(b.x16, 1, ld16, r.d_in, test_idx, n_te, xte16, ld16, nullptr, 0, 0, st));
            }
            RETEXO_TRY(retexo_embed(&best, xte16, ld16, nullptr, n_te, nullptr, 0, nullptr, 0, nullptr, 0, nullptr,
                                    b.y_test, reinterpret_cast<uint64_t*>(b.test_best + (m - 1)), b.ws_embed,
                                    b.ws_embed_bytes, st));
        } else {
            RETEXO_CUDA_TRY(cudaMemsetAsync(b.test_best + (m - 1), 0, sizeof(unsigned long long), st));
            RETEXO_CUDA_TRY(cudaMemsetAsync(b.test_last + (m - 1), 0, sizeof(unsigned long long), st));
            if (gat_train) RETEXO_TRY(gat_forward(b.att_best));
        }
        if (gat && out->gat_best && out->gat_best[m - 1])
            RETEXO_CUDA_TRY(cudaMemcpyAsync(out->gat_best[m - 1], b.att_best, sizeof(float) * (size_t)n_att,
                                            cudaMemcpyDefault, st));
        if (out->theta_best && out->theta_best[m - 1])
            RETEXO_CUDA_TRY(cudaMemcpyAsync(out->theta_best[m - 1], b.theta_best, sizeof(float) * (size_t)nt,
                                            cudaMemcpyDefault, st));

        merge_status_kernel<<<1, 32, 0, st>>>(b.run_status, sb.status, c.aggr == RETEXO_GAT ? b.status : nullptr);
        // ---- emit Q^m (classifier dropped) or the final logits
        if (m < c.K) {
            float* qn = b.q[(m - 1) & 1];
            const int64_t ldn = round_up(c.hidden, 32);
            RETEXO_TRY(retexo_embed(&best, b.x16, ld16, nullptr, n, qn, ldn, nullptr, 0, nullptr, 0, nullptr, nullptr,
                                    nullptr, b.ws_embed, b.ws_embed_bytes, st));
            q = qn;
            ldq = ldn;
        } else if (out->final_logits || out->final_pred) {
            float* lg = host ? b.final_logits : out->final_logits;
            const int64_t ldl = host ? c.n_classes : out->ld_logits;
            int32_t* pr = host ? b.final_pred : out->final_pred;
            RETEXO_TRY(retexo_embed(&best, b.x16, ld16, nullptr, n, nullptr, 0, nullptr, 0,
                                    out->final_logits ? lg : nullptr, ldl, out->final_pred ? pr : nullptr, nullptr,
                                    nullptr, b.ws_embed, b.ws_embed_bytes, st));
        }
    }

    // ---- results
    const size_t kr = (size_t)c.K * c.R;
    if (out->loss_history) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->loss_history, b.loss_history, sizeof(float) * kr, out_kind, st));
    if (out->val_correct) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->val_correct, b.val_history, sizeof(uint64_t) * kr, out_kind, st));
    if (out->best_val_correct) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->best_val_correct, b.best_val, sizeof(uint64_t) * c.K, out_kind, st));
    if (out->best_iter) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->best_iter, b.best_iter, sizeof(int32_t) * c.K, out_kind, st));
    if (out->test_correct) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->test_correct, b.test_best, sizeof(uint64_t) * c.K, out_kind, st));
    if (out->test_correct_last) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->test_correct_last, b.test_last, sizeof(uint64_t) * c.K, out_kind, st));
    if (out->status) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->status, b.run_status, sizeof(int32_t), out_kind, st));
    if (out->counts && part) RETEXO_CUDA_TRY(cudaMemcpyAsync(out->counts, b.counts, sizeof(uint64_t) * (4 + c.K), out_kind, st));
    if (host) {
        if (out->final_logits)
            RETEXO_CUDA_TRY(cudaMemcpy2DAsync(out->final_logits, sizeof(float) * out->ld_logits, b.final_logits,
                                              sizeof(float) * c.n_classes, sizeof(float) * c.n_classes, (size_t)n,
                                              out_kind, st));
        if (out->final_pred)
            RETEXO_CUDA_TRY(cudaMemcpyAsync(out->final_pred, b.final_pred, sizeof(int32_t) * (size_t)n, out_kind, st));
        RETEXO_CUDA_TRY(cudaStreamSynchronize(st));
    }
    return launch_status();
}
