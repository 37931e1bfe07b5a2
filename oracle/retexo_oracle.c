/*
 * CPU checker for the on-device hot path of lazy message passing
 * ("Scalable Neural Network Training over Distributed Graphs", Retexo).
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is a plain, slow restatement of the
 * paper's definitions, used only by the tests, by the smoke check and as the
 * timed CPU baseline.  The CUDA library never calls it and shares no source,
 * header, table or helper with it.
 *
 * Conventions
 *   - graph: symmetric CSR (both directions of every undirected edge stored),
 *     no self loops, no duplicate entries (Section 2.1: "the graphs are
 *     undirected"); rowptr is int64, colidx int32.
 *   - features / representations are fp32 in memory; every sum is carried in
 *     double and rounded to fp32 once at the end.
 *   - counts are exact uint64.
 *   - OpenMP is used only over independent output rows (or over fixed chunks
 *     that are combined in index order), so no result depends on the number
 *     of threads.
 *
 * Parity status: every function here is pinned by tests/test_oracle_*.py
 * (dense brute force, closed forms, invariants, library special cases).  What
 * cannot be pinned is agreement with the paper's printed accuracy and timing
 * tables, which need the public datasets: parity unpinned for those.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define ORACLE_OK 0
#define ORACLE_BAD_ARG 1
#define ORACLE_NO_MEM 2

/* ------------------------------------------------------------------ */
/* bf16 operand rounding (round to nearest, ties to even, of the top   */
/* 16 bits of an IEEE-754 binary32; NaN stays NaN)                      */
/* ------------------------------------------------------------------ */
static float bf16_round(float x)
{
    uint32_t u;
    memcpy(&u, &x, 4);
    if ((u & 0x7f800000u) == 0x7f800000u) {       /* inf / nan: truncate, keep nan */
        if (u & 0x007fffffu) u |= 0x00400000u;
        u &= 0xffff0000u;
    } else {
        uint32_t lsb = (u >> 16) & 1u;
        u += 0x7fffu + lsb;
        u &= 0xffff0000u;
    }
    memcpy(&x, &u, 4);
    return x;
}

float oracle_bf16_round(float x) { return bf16_round(x); }

static double opnd(double x, int round_bf16)
{
    return round_bf16 ? (double)bf16_round((float)x) : x;
}

/* ================================================================== */
/* Aggregation, Eq. 1:  AGGR over u in N(v) of Q^{m-1}_u               */
/* `rows` selects destination nodes (NULL = all); output row i belongs */
/* to node rows[i].                                                    */
/* ================================================================== */

/* GCN: Z = D^-1/2 (A + I) D^-1/2 Q with D = degree + 1 (the self loop is
 * implicit).  Section 2.2 names the GCN aggregator; the symmetric
 * normalisation is that of the cited GCN layer.  Isolated node: Z_v = Q_v. */
int oracle_aggregate_gcn(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                         const float *q, int64_t ldq, int32_t dim,
                         float *out, int64_t ldout,
                         const int64_t *rows, int64_t n_rows)
{
    if (n < 0 || dim < 0 || ldq < dim || ldout < dim) return ORACLE_BAD_ARG;
    int64_t cnt = rows ? n_rows : n;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < cnt; ++i) {
        int64_t v = rows ? rows[i] : i;
        double *acc = (double *)calloc((size_t)(dim > 0 ? dim : 1), sizeof(double));
        if (!acc) { failed = 1; continue; }
        double nv = 1.0 / sqrt((double)(rowptr[v + 1] - rowptr[v]) + 1.0);
        for (int32_t j = 0; j < dim; ++j) acc[j] = nv * (double)q[v * ldq + j];
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            int64_t u = colidx[e];
            double nu = 1.0 / sqrt((double)(rowptr[u + 1] - rowptr[u]) + 1.0);
            for (int32_t j = 0; j < dim; ++j) acc[j] += nu * (double)q[u * ldq + j];
        }
        for (int32_t j = 0; j < dim; ++j) out[i * ldout + j] = (float)(nv * acc[j]);
        free(acc);
    }
    return failed ? ORACLE_NO_MEM : ORACLE_OK;
}

/* GraphSAGE mean with COMBINE = concatenation (Section 2.2): columns [0,dim)
 * are the node's own row, columns [dim,2dim) the mean over N(v) (v itself
 * excluded); a node without neighbours gets a zero mean. */
int oracle_aggregate_sage_mean(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                               const float *q, int64_t ldq, int32_t dim,
                               float *out, int64_t ldout,
                               const int64_t *rows, int64_t n_rows)
{
    if (n < 0 || dim < 0 || ldq < dim || ldout < 2 * (int64_t)dim) return ORACLE_BAD_ARG;
    int64_t cnt = rows ? n_rows : n;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < cnt; ++i) {
        int64_t v = rows ? rows[i] : i;
        double *acc = (double *)calloc((size_t)(dim > 0 ? dim : 1), sizeof(double));
        if (!acc) { failed = 1; continue; }
        int64_t deg = rowptr[v + 1] - rowptr[v];
        for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
            int64_t u = colidx[e];
            for (int32_t j = 0; j < dim; ++j) acc[j] += (double)q[u * ldq + j];
        }
        for (int32_t j = 0; j < dim; ++j) {
            out[i * ldout + j] = q[v * ldq + j];
            out[i * ldout + dim + j] = deg > 0 ? (float)(acc[j] / (double)deg) : 0.0f;
        }
        free(acc);
    }
    return failed ? ORACLE_NO_MEM : ORACLE_OK;
}

/* GraphSAGE with the max-pooling aggregator named in Section 2.2, COMBINE =
 * concatenation: columns [0,dim) are the node's own row, column dim+j the
 * largest q[u][j] over u in N(v) (v itself excluded); a node without
 * neighbours gets zeros.  The pooling layer's own transform is not part of
 * this function: q is taken as already transformed. */
int oracle_aggregate_sage_max(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                              const float *q, int64_t ldq, int32_t dim,
                              float *out, int64_t ldout,
                              const int64_t *rows, int64_t n_rows)
{
    if (n < 0 || dim < 0 || ldq < dim || ldout < 2 * (int64_t)dim) return ORACLE_BAD_ARG;
    int64_t cnt = rows ? n_rows : n;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < cnt; ++i) {
        int64_t v = rows ? rows[i] : i;
        for (int32_t j = 0; j < dim; ++j) {
            float best = 0.0f;
            for (int64_t e = rowptr[v]; e < rowptr[v + 1]; ++e) {
                float x = q[(int64_t)colidx[e] * ldq + j];
                if (e == rowptr[v] || x > best) best = x;
            }
            out[i * ldout + j] = q[v * ldq + j];
            out[i * ldout + dim + j] = best;
        }
    }
    return ORACLE_OK;
}

/* GAT (cited in Section 2.2; formula of the cited layer).  p holds the
 * already projected rows, heads*head_dim wide, head k in columns
 * [k*head_dim, (k+1)*head_dim).  For destination v and head k:
 *   s_u = <a_src[k], p_u^k>,  t_v = <a_dst[k], p_v^k>
 *   e_uv = LeakyReLU_slope(s_u + t_v)  for u in N(v) (and u = v if
 *                                      add_self_loop)
 *   alpha_uv = softmax over those u of e_uv
 *   Z_v^k = sum_u alpha_uv p_u^k
 * A node whose softmax set is empty gets zeros.
 * alpha_edge [n_edges x heads] and alpha_self [n x heads] (both optional,
 * only with rows == NULL) receive the attention weights. */
int oracle_aggregate_gat(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                         const float *p, int64_t ldp, int32_t heads, int32_t head_dim,
                         const float *a_src, const float *a_dst, double slope,
                         int32_t add_self_loop,
                         float *out, int64_t ldout,
                         const int64_t *rows, int64_t n_rows,
                         double *alpha_edge, double *alpha_self)
{
    int32_t dim = heads * head_dim;
    if (n < 0 || heads <= 0 || head_dim <= 0 || ldp < dim || ldout < dim) return ORACLE_BAD_ARG;
    if (rows && (alpha_edge || alpha_self)) return ORACLE_BAD_ARG;
    double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * heads);
    double *t = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1) * heads);
    if (!s || !t) { free(s); free(t); return ORACLE_NO_MEM; }
#pragma omp parallel for
    for (int64_t u = 0; u < n; ++u)
        for (int32_t k = 0; k < heads; ++k) {
            double ss = 0.0, tt = 0.0;
            for (int32_t j = 0; j < head_dim; ++j) {
                double x = (double)p[u * ldp + k * head_dim + j];
                ss += (double)a_src[k * head_dim + j] * x;
                tt += (double)a_dst[k * head_dim + j] * x;
            }
            s[u * heads + k] = ss;
            t[u * heads + k] = tt;
        }
    int64_t cnt = rows ? n_rows : n;
    int failed = 0;
#pragma omp parallel for schedule(dynamic, 64)
    for (int64_t i = 0; i < cnt; ++i) {
        int64_t v = rows ? rows[i] : i;
        int64_t deg = rowptr[v + 1] - rowptr[v];
        int64_t m = deg + (add_self_loop ? 1 : 0);
        double *e = (double *)malloc(sizeof(double) * (size_t)(m > 0 ? m : 1));
        double *acc = (double *)malloc(sizeof(double) * (size_t)head_dim);
        if (!e || !acc) { free(e); free(acc); failed = 1; continue; }
        for (int32_t k = 0; k < heads; ++k) {
            for (int64_t a = 0; a < m; ++a) {
                int64_t u = a < deg ? (int64_t)colidx[rowptr[v] + a] : v;
                double z = s[u * heads + k] + t[v * heads + k];
                e[a] = z > 0.0 ? z : slope * z;
            }
            double mx = -INFINITY, den = 0.0;
            for (int64_t a = 0; a < m; ++a) if (e[a] > mx) mx = e[a];
            for (int64_t a = 0; a < m; ++a) { e[a] = exp(e[a] - mx); den += e[a]; }
            for (int32_t j = 0; j < head_dim; ++j) acc[j] = 0.0;
            for (int64_t a = 0; a < m; ++a) {
                int64_t u = a < deg ? (int64_t)colidx[rowptr[v] + a] : v;
                double alpha = e[a] / den;
                if (a < deg) { if (alpha_edge) alpha_edge[(rowptr[v] + a) * heads + k] = alpha; }
                else if (alpha_self) alpha_self[v * heads + k] = alpha;
                for (int32_t j = 0; j < head_dim; ++j)
                    acc[j] += alpha * (double)p[u * ldp + k * head_dim + j];
            }
            for (int32_t j = 0; j < head_dim; ++j)
                out[i * ldout + k * head_dim + j] = m > 0 ? (float)acc[j] : 0.0f;
        }
        free(e);
        free(acc);
    }
    free(s);
    free(t);
    return failed ? ORACLE_NO_MEM : ORACLE_OK;
}

/* Backward of the GAT aggregation above (Section 2.2: "AGGR may have
 * trainable parameters"; Section 3.1: the whole layer, AGGR included, is what a
 * round trains).  dz [n x heads*head_dim] is the gradient of the loss with
 * respect to the aggregation's output Z (zero rows for nodes outside the loss).
 * With e_uv = LeakyReLU(z_uv), z_uv = s_u + t_v, alpha = softmax_u(e_uv),
 * Z_v = sum_u alpha_uv p_u, the chain rule gives, per head,
 *   dalpha_uv = <dz_v, p_u>
 *   de_uv     = alpha_uv (dalpha_uv - sum_w alpha_wv dalpha_wv)
 *   dz_uv     = de_uv * (z_uv > 0 ? 1 : slope)
 *   ds_u = sum_v dz_uv,  dt_v = sum_u dz_uv
 *   dp_u = sum_v alpha_uv dz_v + ds_u a_src + dt_u a_dst
 *   da_src = sum_u ds_u p_u,  da_dst = sum_v dt_v p_v
 * (the sums over v run over the destinations that attend over u, u itself
 * included with the self loop).  Everything is carried in double; dp
 * [n x heads*head_dim], da_src and da_dst [heads x head_dim] are outputs. */
int oracle_gat_backward(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                        const float *p, int64_t ldp, int32_t heads, int32_t head_dim,
                        const float *a_src, const float *a_dst, double slope, int32_t add_self_loop,
                        const double *dz, double *dp, double *da_src, double *da_dst)
{
    int32_t dim = heads * head_dim;
    if (n < 0 || heads <= 0 || head_dim <= 0 || ldp < dim || !dz || !dp || !da_src || !da_dst) return ORACLE_BAD_ARG;
    size_t nh = (size_t)(n > 0 ? n : 1) * heads;
    double *s = (double *)malloc(sizeof(double) * nh), *t = (double *)malloc(sizeof(double) * nh);
    double *ds = (double *)calloc(nh, sizeof(double)), *dt = (double *)calloc(nh, sizeof(double));
    if (!s || !t || !ds || !dt) { free(s); free(t); free(ds); free(dt); return ORACLE_NO_MEM; }
    for (int64_t u = 0; u < n; ++u)
        for (int32_t k = 0; k < heads; ++k) {
            double ss = 0.0, tt = 0.0;
            for (int32_t j = 0; j < head_dim; ++j) {
                double x = (double)p[u * ldp + k * head_dim + j];
                ss += (double)a_src[k * head_dim + j] * x;
                tt += (double)a_dst[k * head_dim + j] * x;
            }
            s[u * heads + k] = ss;
            t[u * heads + k] = tt;
        }
    for (int64_t i = 0; i < n * (int64_t)dim; ++i) dp[i] = 0.0;
    for (int32_t i = 0; i < dim; ++i) { da_src[i] = 0.0; da_dst[i] = 0.0; }
    int failed = 0;
    for (int64_t v = 0; v < n && !failed; ++v) {
        int64_t deg = rowptr[v + 1] - rowptr[v];
        int64_t m = deg + (add_self_loop ? 1 : 0);
        if (m == 0) continue;
        double *alpha = (double *)malloc(sizeof(double) * (size_t)m);
        double *dalpha = (double *)malloc(sizeof(double) * (size_t)m);
        if (!alpha || !dalpha) { free(alpha); free(dalpha); failed = 1; break; }
        for (int32_t k = 0; k < heads; ++k) {
            const double *g = dz + v * dim + k * head_dim;
            double mx = -INFINITY, den = 0.0, c = 0.0;
            for (int64_t a = 0; a < m; ++a) {
                int64_t u = a < deg ? (int64_t)colidx[rowptr[v] + a] : v;
                double z = s[u * heads + k] + t[v * heads + k];
                alpha[a] = z > 0.0 ? z : slope * z;
                if (alpha[a] > mx) mx = alpha[a];
            }
            for (int64_t a = 0; a < m; ++a) { alpha[a] = exp(alpha[a] - mx); den += alpha[a]; }
            for (int64_t a = 0; a < m; ++a) {
                int64_t u = a < deg ? (int64_t)colidx[rowptr[v] + a] : v;
                alpha[a] /= den;
                double d = 0.0;
                for (int32_t j = 0; j < head_dim; ++j) d += g[j] * (double)p[u * ldp + k * head_dim + j];
                dalpha[a] = d;
                c += alpha[a] * d;
            }
            for (int64_t a = 0; a < m; ++a) {
                int64_t u = a < deg ? (int64_t)colidx[rowptr[v] + a] : v;
                double z = s[u * heads + k] + t[v * heads + k];
                double dzz = alpha[a] * (dalpha[a] - c) * (z > 0.0 ? 1.0 : slope);
                ds[u * heads + k] += dzz;
                dt[v * heads + k] += dzz;
                for (int32_t j = 0; j < head_dim; ++j) dp[u * dim + k * head_dim + j] += alpha[a] * g[j];
            }
        }
        free(alpha);
        free(dalpha);
    }
    for (int64_t x = 0; x < n && !failed; ++x)
        for (int32_t k = 0; k < heads; ++k)
            for (int32_t j = 0; j < head_dim; ++j) {
                double px = (double)p[x * ldp + k * head_dim + j];
                dp[x * dim + k * head_dim + j] += ds[x * heads + k] * (double)a_src[k * head_dim + j] +
                                                  dt[x * heads + k] * (double)a_dst[k * head_dim + j];
                da_src[k * head_dim + j] += ds[x * heads + k] * px;
                da_dst[k * head_dim + j] += dt[x * heads + k] * px;
            }
    free(s); free(t); free(ds); free(dt);
    return failed ? ORACLE_NO_MEM : ORACLE_OK;
}

/* ================================================================== */
/* Per-node model of one round (Section 3.1): f_theta = Linear+ReLU,   */
/* temporary classifier C_theta = Linear; last round: one Linear.      */
/* theta is one flat double array:                                     */
/*   hidden > 0 : [ W1 (d_in x hidden) | b1 (hidden) |                 */
/*                  W2 (hidden x n_classes) | b2 (n_classes) ]         */
/*   hidden == 0: [ W1 (d_in x n_classes) | b1 (n_classes) ]           */
/* matrices row-major [in x out].                                       */
/* round_bf16 != 0: both operands of every matrix product are rounded  */
/* to bf16 first ("bf16 inputs, wider accumulate"); sums, biases,      */
/* softmax and the optimiser stay in double.  A bias gradient is the   */
/* product of the all-ones vector with the layer's output gradient, so */
/* it sums the rounded gradient like any other product.                */
/* ================================================================== */

int64_t oracle_theta_size(int32_t d_in, int32_t hidden, int32_t n_classes)
{
    if (hidden > 0)
        return (int64_t)d_in * hidden + hidden + (int64_t)hidden * n_classes + n_classes;
    return (int64_t)d_in * n_classes + n_classes;
}

/* Layer normalisation inside f_theta (Section 2.2 lists normalisation layers among its parts; the
 * configurations use none).  Reading taken here: it sits between the fully-connected layer and the ReLU,
 *   z = x W1 + b1,  zhat = (z - mean(z)) / sqrt(var(z) + ln_eps)  (mean and biased variance over the
 *   hidden units of the row),  Hd = ReLU(gamma .* zhat + beta),
 * with trainable gamma and beta appended to theta: [ W1 | b1 | W2 | b2 | gamma (hidden) | beta (hidden) ].
 * In rounded mode the normalisation is computed wide, forward and backward; the gated gradient that enters
 * its backward pass is rounded to bf16 first (it is handed on in the format the products read), and the
 * gradient that leaves it is an operand of the weight-gradient products and rounded there like any other. */
int64_t oracle_theta_size_ln(int32_t d_in, int32_t hidden, int32_t n_classes, int32_t layer_norm)
{
    return oracle_theta_size(d_in, hidden, n_classes) + ((layer_norm && hidden > 0) ? 2 * (int64_t)hidden : 0);
}

/* Batch normalisation inside f_theta (the other normalisation Section 2.2 names).  Reading taken here, the
 * usual one of the framework the paper's code is written in: between the fully-connected layer and the ReLU,
 *   training:   zhat = (z - mean_b) / sqrt(var_b + eps), mean_b and the biased variance var_b taken per hidden
 *               unit over the rows of the (full) training batch;  Hd = ReLU(gamma .* zhat + beta);
 *               running statistics  r_mean <- (1 - mom) r_mean + mom mean_b,
 *                                   r_var  <- (1 - mom) r_var  + mom var_b n / (n - 1)   (unbiased);
 *   evaluation: zhat = (z - r_mean) / sqrt(r_var + eps)  (validation, test, emission of Q^m);
 * theta = [ W1 | b1 | W2 | b2 | gamma | beta | r_mean | r_var ]: gamma, beta trained, the running statistics
 * state that the optimiser does not touch (their gradient entries are 0).  `norm`: 0 none, 1 layer
 * normalisation, 2 batch normalisation.  Rounded mode: as for layer normalisation (wide inside, the gated
 * gradient enters the backward pass rounded to bf16). */
int64_t oracle_theta_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes, int32_t norm)
{
    int64_t extra = (hidden > 0 && norm == 1) ? 2 * (int64_t)hidden : ((hidden > 0 && norm == 2) ? 4 * (int64_t)hidden : 0);
    return oracle_theta_size(d_in, hidden, n_classes) + extra;
}

/* ------------------------------------------------------------------ */
/* Dropout (Appendix B lists dropout rates among the hyper-parameters; */
/* the configurations use none).  The random bits come from the        */
/* counter-based generator Philox4x32-10 (Salmon, Moraes, Dror, Shaw:   */
/* "Parallel random numbers: as easy as 1, 2, 3", SC'11), written out   */
/* here from its definition: ten rounds of                              */
/*   (c0,c1,c2,c3) <- (hi(M1 c2)^c1^k0, lo(M1 c2), hi(M0 c0)^c3^k1, lo(M0 c0)) */
/* with the key raised by (W0, W1) between rounds.                      */
/* ------------------------------------------------------------------ */
void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3], k0 = key[0], k1 = key[1];
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0, n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1, n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += W0; k1 += W1;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Unit j of batch row i is kept in update number `step` iff word (j mod 4) of
 * Philox(counter = (i, j / 4, step, 0), key = seed) is >= floor(p 2^32); a kept
 * unit is scaled by 1 / (1 - p).  keep[j] receives that factor or 0. */
static void dropout_row(int64_t i, int64_t step, int32_t hidden, double p, uint64_t seed, double *keep)
{
    const uint32_t thresh = (uint32_t)floor(p * 4294967296.0);
    const double scale = 1.0 / (1.0 - p);
    const uint32_t key[2] = {(uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32)};
    for (int32_t j0 = 0; j0 < hidden; j0 += 4) {
        const uint32_t ctr[4] = {(uint32_t)i, (uint32_t)(j0 >> 2), (uint32_t)step, 0u};
        uint32_t w[4];
        oracle_philox4x32_10(ctr, key, w);
        for (int32_t t = 0; t < 4 && j0 + t < hidden; ++t) keep[j0 + t] = w[t] >= thresh ? scale : 0.0;
    }
}

/* The keep factors of one row, for tests: keep_out[j] = 1/(1-p) or 0. */
int oracle_dropout_mask(int64_t row, int64_t step, int32_t hidden, double p, uint64_t seed, double *keep_out)
{
    if (hidden <= 0 || p < 0.0 || p >= 1.0 || !keep_out) return ORACLE_BAD_ARG;
    dropout_row(row, step, hidden, p, seed, keep_out);
    return ORACLE_OK;
}

/* forward for one input row; a1 = pre-activation (hidden wide, may be NULL
 * when hidden == 0), logits = n_classes wide.  keep (optional, training with
 * dropout only): factor applied to each hidden unit after the ReLU. */
static void forward_row_ln(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                           int round_bf16, const float *xrow, const double *w1r, const double *w2r,
                           double *a1, double *logits, const double *keep,
                           const double *ln_gamma, const double *ln_beta, double ln_eps,
                           double *zhat_out, double *rstd_out, const double *bn_mean, const double *bn_rstd);

static void forward_row(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                        int round_bf16, const float *xrow, const double *w1r, const double *w2r,
                        double *a1, double *logits, const double *keep)
{
    forward_row_ln(d_in, hidden, n_classes, theta, round_bf16, xrow, w1r, w2r, a1, logits, keep,
                   NULL, NULL, 0.0, NULL, NULL, NULL, NULL);
}

/* ln_gamma != NULL: layer normalisation between the first linear layer and the ReLU; a1 then holds the
 * normalised, scaled and shifted pre-activation, zhat_out (hidden wide) the normalised values and *rstd_out
 * 1 / sqrt(var + eps) of the row. */
static void forward_row_ln(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                           int round_bf16, const float *xrow, const double *w1r, const double *w2r,
                           double *a1, double *logits, const double *keep,
                           const double *ln_gamma, const double *ln_beta, double ln_eps,
                           double *zhat_out, double *rstd_out, const double *bn_mean, const double *bn_rstd)
{
    /* bn_mean != NULL (with ln_gamma, ln_beta): batch normalisation with the given per-unit mean and
     * 1 / sqrt(var + eps) instead of the row's own statistics */
    if (hidden > 0) {
        const double *b1 = theta + (int64_t)d_in * hidden;
        const double *b2 = b1 + hidden + (int64_t)hidden * n_classes;
        for (int32_t j = 0; j < hidden; ++j) a1[j] = 0.0;
        for (int32_t k = 0; k < d_in; ++k) {
            double xv = opnd((double)xrow[k], round_bf16);
            if (xv == 0.0) continue;
            const double *wrow = w1r + (int64_t)k * hidden;
            for (int32_t j = 0; j < hidden; ++j) a1[j] += xv * wrow[j];
        }
        for (int32_t j = 0; j < hidden; ++j) a1[j] += b1[j];
        if (ln_gamma && bn_mean) {
            for (int32_t j = 0; j < hidden; ++j) {
                double zh = (a1[j] - bn_mean[j]) * bn_rstd[j];
                if (zhat_out) zhat_out[j] = zh;
                a1[j] = ln_gamma[j] * zh + ln_beta[j];
            }
        } else if (ln_gamma) {
            double mean = 0.0, var = 0.0;
            for (int32_t j = 0; j < hidden; ++j) mean += a1[j];
            mean /= (double)hidden;
            for (int32_t j = 0; j < hidden; ++j) var += (a1[j] - mean) * (a1[j] - mean);
            var /= (double)hidden;
            double rstd = 1.0 / sqrt(var + ln_eps);
            for (int32_t j = 0; j < hidden; ++j) {
                double zh = (a1[j] - mean) * rstd;
                if (zhat_out) zhat_out[j] = zh;
                a1[j] = ln_gamma[j] * zh + ln_beta[j];
            }
            if (rstd_out) *rstd_out = rstd;
        }
        for (int32_t c = 0; c < n_classes; ++c) logits[c] = 0.0;
        for (int32_t j = 0; j < hidden; ++j) {
            double h = a1[j] > 0.0 ? a1[j] : 0.0;
            if (keep) h *= keep[j];
            h = opnd(h, round_bf16);
            if (h == 0.0) continue;
            const double *wrow = w2r + (int64_t)j * n_classes;
            for (int32_t c = 0; c < n_classes; ++c) logits[c] += h * wrow[c];
        }
        for (int32_t c = 0; c < n_classes; ++c) logits[c] += b2[c];
    } else {
        const double *b1 = theta + (int64_t)d_in * n_classes;
        for (int32_t c = 0; c < n_classes; ++c) logits[c] = 0.0;
        for (int32_t k = 0; k < d_in; ++k) {
            double xv = opnd((double)xrow[k], round_bf16);
            if (xv == 0.0) continue;
            const double *wrow = w1r + (int64_t)k * n_classes;
            for (int32_t c = 0; c < n_classes; ++c) logits[c] += xv * wrow[c];
        }
        for (int32_t c = 0; c < n_classes; ++c) logits[c] += b1[c];
    }
}

/* copies of the weight matrices with the operand rounding applied */
static int rounded_weights(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                           int round_bf16, double **w1r, double **w2r)
{
    int32_t out1 = hidden > 0 ? hidden : n_classes;
    int64_t n1 = (int64_t)d_in * out1;
    *w1r = (double *)malloc(sizeof(double) * (size_t)(n1 > 0 ? n1 : 1));
    *w2r = NULL;
    if (!*w1r) return ORACLE_NO_MEM;
    for (int64_t i = 0; i < n1; ++i) (*w1r)[i] = opnd(theta[i], round_bf16);
    if (hidden > 0) {
        int64_t n2 = (int64_t)hidden * n_classes;
        const double *w2 = theta + n1 + hidden;
        *w2r = (double *)malloc(sizeof(double) * (size_t)(n2 > 0 ? n2 : 1));
        if (!*w2r) { free(*w1r); return ORACLE_NO_MEM; }
        for (int64_t i = 0; i < n2; ++i) (*w2r)[i] = opnd(w2[i], round_bf16);
    }
    return ORACLE_OK;
}

/* The optimiser update alone: SGD (theta -= lr g) or Adam (bias-corrected,
 * eps outside the root, no weight decay); `step` is the 1-based count of this
 * update.  Also callable on its own, e.g. with a gradient computed elsewhere. */
int oracle_apply_update(int64_t nt, double *theta, double *adam_m, double *adam_v, const double *grad,
                        int32_t optimizer, double lr, double beta1, double beta2, double eps, int64_t step)
{
    if (optimizer == 0) {
        for (int64_t p = 0; p < nt; ++p) theta[p] -= lr * grad[p];
        return ORACLE_OK;
    }
    if (!adam_m || !adam_v || step < 1) return ORACLE_BAD_ARG;
    double c1 = 1.0 - pow(beta1, (double)step), c2 = 1.0 - pow(beta2, (double)step);
    for (int64_t p = 0; p < nt; ++p) {
        adam_m[p] = beta1 * adam_m[p] + (1.0 - beta1) * grad[p];
        adam_v[p] = beta2 * adam_v[p] + (1.0 - beta2) * grad[p] * grad[p];
        double mh = adam_m[p] / c1, vh = adam_v[p] / c2;
        theta[p] -= lr * mh / (sqrt(vh) + eps);
    }
    return ORACLE_OK;
}

#define GRAD_CHUNKS 64

/* One full-batch training step (Section 2.3: forward, loss, backward, update;
 * one worker, so the gradient average at the master is the identity).
 *   loss = mean_i CE(softmax(logits_i), y_i)
 * Batch row i is x[row_idx ? row_idx[i] : i]; y[i] is its label.
 * optimizer: 0 = SGD (theta -= lr g), 1 = Adam (bias-corrected, eps outside
 * the root, no weight decay); `step` is the 1-based count of this update.
 * grad_out (optional) receives the gradient, laid out like theta. */
static int train_step_impl(int32_t d_in, int32_t hidden, int32_t n_classes,
                           double *theta, double *adam_m, double *adam_v,
                           int32_t optimizer, double lr, double beta1, double beta2, double eps,
                           int64_t step, int32_t round_bf16,
                           const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                           const int32_t *y, double *loss_out, double *grad_out,
                           double drop_p, uint64_t drop_seed, double *dx_out,
                           int32_t layer_norm /* 0 none, 1 layer, 2 batch normalisation */, double ln_eps,
                           double bn_momentum)
{
    if (d_in <= 0 || n_classes <= 0 || hidden < 0 || n_rows <= 0 || ldx < d_in) return ORACLE_BAD_ARG;
    if (drop_p < 0.0 || drop_p >= 1.0) return ORACLE_BAD_ARG;
    if (layer_norm && (hidden <= 0 || ln_eps <= 0.0)) return ORACLE_BAD_ARG;
    const int batch_norm = layer_norm == 2;
    if (batch_norm && (n_rows < 2 || bn_momentum < 0.0 || bn_momentum > 1.0)) return ORACLE_BAD_ARG;
    const int dropping = drop_p > 0.0 && hidden > 0;
    if (optimizer == 1 && (!adam_m || !adam_v || step < 1)) return ORACLE_BAD_ARG;
    int64_t nt = oracle_theta_size_norm(d_in, hidden, n_classes, layer_norm);
    int32_t out1 = hidden > 0 ? hidden : n_classes;
    /* layer normalisation: gamma and beta sit behind [W1 | b1 | W2 | b2] */
    const double *ln_gamma = layer_norm ? theta + oracle_theta_size(d_in, hidden, n_classes) : NULL;
    const double *ln_beta = layer_norm ? ln_gamma + hidden : NULL;
    /* per row: the normalised values and the (bf16-rounded, in rounded mode) gated gradient, for d gamma / d beta */
    double *zh_all = layer_norm ? (double *)malloc(sizeof(double) * (size_t)n_rows * hidden) : NULL;
    double *dy_all = layer_norm ? (double *)malloc(sizeof(double) * (size_t)n_rows * hidden) : NULL;
    if (layer_norm && (!zh_all || !dy_all)) { free(zh_all); free(dy_all); return ORACLE_NO_MEM; }
    double *w1r, *w2r;
    if (rounded_weights(d_in, hidden, n_classes, theta, round_bf16, &w1r, &w2r)) { free(zh_all); free(dy_all); return ORACLE_NO_MEM; }
    /* batch normalisation: the statistics of z = x W1 + b1 over the whole batch come first */
    double *bn_mean = NULL, *bn_var = NULL, *bn_rstd = NULL;
    if (batch_norm) {
        bn_mean = (double *)calloc((size_t)hidden, sizeof(double));
        bn_var = (double *)calloc((size_t)hidden, sizeof(double));
        bn_rstd = (double *)calloc((size_t)hidden, sizeof(double));
        double *z_all = (double *)malloc(sizeof(double) * (size_t)n_rows * hidden);
        if (!bn_mean || !bn_var || !bn_rstd || !z_all) {
            free(bn_mean); free(bn_var); free(bn_rstd); free(z_all); free(w1r); free(w2r); free(zh_all); free(dy_all);
            return ORACLE_NO_MEM;
        }
#pragma omp parallel
        {
            double *lg0 = (double *)malloc(sizeof(double) * (size_t)n_classes);
#pragma omp for schedule(static)
            for (int64_t i = 0; i < n_rows; ++i) {
                int64_t r = row_idx ? row_idx[i] : i;
                forward_row(d_in, hidden, n_classes, theta, round_bf16, x + r * ldx, w1r, w2r, z_all + i * hidden, lg0, NULL);
            }
            free(lg0);
        }
        for (int64_t i = 0; i < n_rows; ++i)
            for (int32_t j = 0; j < hidden; ++j) bn_mean[j] += z_all[i * hidden + j];
        for (int32_t j = 0; j < hidden; ++j) bn_mean[j] /= (double)n_rows;
        for (int64_t i = 0; i < n_rows; ++i)
            for (int32_t j = 0; j < hidden; ++j) {
                double d = z_all[i * hidden + j] - bn_mean[j];
                bn_var[j] += d * d;
            }
        for (int32_t j = 0; j < hidden; ++j) {
            bn_var[j] /= (double)n_rows;
            bn_rstd[j] = 1.0 / sqrt(bn_var[j] + ln_eps);
        }
        free(z_all);
    }

    /* per-row results of the forward/backward through the row-local part */
    double *d1 = (double *)malloc(sizeof(double) * (size_t)n_rows * out1);       /* grad wrt first linear output */
    double *hd = hidden > 0 ? (double *)malloc(sizeof(double) * (size_t)n_rows * hidden) : NULL;
    double *dl = hidden > 0 ? (double *)malloc(sizeof(double) * (size_t)n_rows * n_classes) : NULL;
    double *row_loss = (double *)malloc(sizeof(double) * (size_t)n_rows);
    double *grad = (double *)calloc((size_t)nt, sizeof(double));
    int bad_label = 0;
    if (!d1 || (hidden > 0 && (!hd || !dl)) || !row_loss || !grad) {
        free(w1r); free(w2r); free(d1); free(hd); free(dl); free(row_loss); free(grad); free(zh_all); free(dy_all);
        return ORACLE_NO_MEM;
    }

#pragma omp parallel
    {
        double *a1 = (double *)malloc(sizeof(double) * (size_t)(hidden > 0 ? hidden : 1));
        double *lg = (double *)malloc(sizeof(double) * (size_t)n_classes);
        double *keep = dropping ? (double *)malloc(sizeof(double) * (size_t)hidden) : NULL;
#pragma omp for schedule(static)
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t r = row_idx ? row_idx[i] : i;
            if (keep) dropout_row(i, step, hidden, drop_p, drop_seed, keep);
            double rstd = 0.0;
            forward_row_ln(d_in, hidden, n_classes, theta, round_bf16, x + r * ldx, w1r, w2r, a1, lg, keep,
                           ln_gamma, ln_beta, ln_eps, layer_norm ? zh_all + i * hidden : NULL, &rstd, bn_mean, bn_rstd);
            int32_t yi = y[i];
            if (yi < 0 || yi >= n_classes) { bad_label = 1; yi = 0; }
            double mx = lg[0];
            for (int32_t c = 1; c < n_classes; ++c) if (lg[c] > mx) mx = lg[c];
            double den = 0.0;
            for (int32_t c = 0; c < n_classes; ++c) den += exp(lg[c] - mx);
            row_loss[i] = (mx + log(den)) - lg[yi];
            double *g = hidden > 0 ? dl + i * n_classes : d1 + i * out1;
            for (int32_t c = 0; c < n_classes; ++c)
                g[c] = (exp(lg[c] - mx) / den - (c == yi ? 1.0 : 0.0)) / (double)n_rows;
            if (hidden > 0) {
                for (int32_t j = 0; j < hidden; ++j) {
                    double h = a1[j] > 0.0 ? a1[j] : 0.0;
                    if (keep) h *= keep[j];
                    hd[i * hidden + j] = h;
                    double acc = 0.0;
                    if (a1[j] > 0.0 && (!keep || keep[j] != 0.0)) {
                        const double *wrow = w2r + (int64_t)j * n_classes;
                        for (int32_t c = 0; c < n_classes; ++c) acc += opnd(g[c], round_bf16) * wrow[c];
                        if (keep) acc *= keep[j];
                    }
                    d1[i * hidden + j] = acc;
                }
                if (batch_norm) {
                    /* the column sums its backward pass needs span the batch: keep the (rounded) gated gradient */
                    for (int32_t j = 0; j < hidden; ++j) dy_all[i * hidden + j] = opnd(d1[i * hidden + j], round_bf16);
                } else if (layer_norm) {
                    /* backward through the normalisation: with dy the gated gradient at its output,
                     *   dzhat = dy .* gamma,  dz = rstd (dzhat - mean(dzhat) - zhat mean(dzhat .* zhat)) */
                    const double *zh = zh_all + i * hidden;
                    double *dy = dy_all + i * hidden;
                    double m1 = 0.0, m2 = 0.0;
                    for (int32_t j = 0; j < hidden; ++j) {
                        dy[j] = opnd(d1[i * hidden + j], round_bf16);
                        double dzh = dy[j] * ln_gamma[j];
                        m1 += dzh;
                        m2 += dzh * zh[j];
                    }
                    m1 /= (double)hidden;
                    m2 /= (double)hidden;
                    for (int32_t j = 0; j < hidden; ++j)
                        d1[i * hidden + j] = rstd * (dy[j] * ln_gamma[j] - m1 - zh[j] * m2);
                }
            }
        }
        free(a1);
        free(lg);
        free(keep);
    }

    double loss = 0.0;
    for (int64_t i = 0; i < n_rows; ++i) loss += row_loss[i];
    loss /= (double)n_rows;

    if (batch_norm) {
        /* backward through the batch normalisation: with dy the gated gradient at its output, per unit j
         *   s1 = sum_rows dy,  s2 = sum_rows dy zhat,
         *   dz = gamma rstd (dy - s1 / n - zhat s2 / n)                                   */
        double *s1 = (double *)calloc((size_t)hidden, sizeof(double));
        double *s2 = (double *)calloc((size_t)hidden, sizeof(double));
        if (s1 && s2) {
            for (int64_t i = 0; i < n_rows; ++i)
                for (int32_t j = 0; j < hidden; ++j) {
                    s1[j] += dy_all[i * hidden + j];
                    s2[j] += dy_all[i * hidden + j] * zh_all[i * hidden + j];
                }
            for (int64_t i = 0; i < n_rows; ++i)
                for (int32_t j = 0; j < hidden; ++j)
                    d1[i * hidden + j] = ln_gamma[j] * bn_rstd[j] *
                                         (dy_all[i * hidden + j] - s1[j] / (double)n_rows - zh_all[i * hidden + j] * s2[j] / (double)n_rows);
        }
        free(s1); free(s2);
    }

    /* gradient with respect to the batch itself, dX = d1 W1^T (needed when what produces X is trained too,
     * e.g. an aggregator with parameters): one more matrix product, operands d1 and W1 rounded like the others */
    if (dx_out) {
#pragma omp parallel for schedule(static)
        for (int64_t i = 0; i < n_rows; ++i)
            for (int32_t k = 0; k < d_in; ++k) {
                double acc = 0.0;
                const double *wrow = w1r + (int64_t)k * out1;
                for (int32_t j = 0; j < out1; ++j) acc += opnd(d1[i * out1 + j], round_bf16) * wrow[j];
                dx_out[i * d_in + k] = acc;
            }
    }

    /* weight gradients: sums over batch rows, taken in fixed chunks of rows
     * that are then added in chunk order */
    double *part = (double *)calloc((size_t)GRAD_CHUNKS * (size_t)nt, sizeof(double));
    if (!part) {
        free(w1r); free(w2r); free(d1); free(hd); free(dl); free(row_loss); free(grad); free(zh_all); free(dy_all);
        return ORACLE_NO_MEM;
    }
#pragma omp parallel for schedule(dynamic, 1)
    for (int ch = 0; ch < GRAD_CHUNKS; ++ch) {
        int64_t lo = n_rows * ch / GRAD_CHUNKS, hi = n_rows * (ch + 1) / GRAD_CHUNKS;
        double *g = part + (int64_t)ch * nt;
        double *gw1 = g, *gb1 = g + (int64_t)d_in * out1;
        double *gw2 = gb1 + out1, *gb2 = gw2 + (int64_t)hidden * n_classes;
        for (int64_t i = lo; i < hi; ++i) {
            int64_t r = row_idx ? row_idx[i] : i;
            const float *xrow = x + r * ldx;
            const double *d1row = d1 + i * out1;
            /* dW1 = X^T d1,  db1 = 1^T d1 */
            for (int32_t k = 0; k < d_in; ++k) {
                double xv = opnd((double)xrow[k], round_bf16);
                if (xv == 0.0) continue;
                double *grow = gw1 + (int64_t)k * out1;
                for (int32_t j = 0; j < out1; ++j) grow[j] += xv * opnd(d1row[j], round_bf16);
            }
            for (int32_t j = 0; j < out1; ++j) gb1[j] += opnd(d1row[j], round_bf16);
            if (hidden > 0) {
                /* dW2 = Hd^T dL,  db2 = 1^T dL */
                const double *dlrow = dl + i * n_classes;
                for (int32_t j = 0; j < hidden; ++j) {
                    double h = opnd(hd[i * hidden + j], round_bf16);
                    if (h == 0.0) continue;
                    double *grow = gw2 + (int64_t)j * n_classes;
                    for (int32_t c = 0; c < n_classes; ++c) grow[c] += h * opnd(dlrow[c], round_bf16);
                }
                for (int32_t c = 0; c < n_classes; ++c) gb2[c] += opnd(dlrow[c], round_bf16);
            }
            if (layer_norm) {
                /* d gamma = sum_rows dy .* zhat,  d beta = sum_rows dy */
                double *gg = gb2 + n_classes, *gbt = gg + hidden;
                for (int32_t j = 0; j < hidden; ++j) {
                    gg[j] += dy_all[i * hidden + j] * zh_all[i * hidden + j];
                    gbt[j] += dy_all[i * hidden + j];
                }
            }
        }
    }
    for (int ch = 0; ch < GRAD_CHUNKS; ++ch)
        for (int64_t p = 0; p < nt; ++p) grad[p] += part[(int64_t)ch * nt + p];
    free(part);

    oracle_apply_update(nt, theta, adam_m, adam_v, grad, optimizer, lr, beta1, beta2, eps, step);
    if (batch_norm) {      /* running statistics: state, moved towards this batch's (gradient entries are 0) */
        double *r_mean = theta + oracle_theta_size(d_in, hidden, n_classes) + 2 * (int64_t)hidden, *r_var = r_mean + hidden;
        for (int32_t j = 0; j < hidden; ++j) {
            r_mean[j] = (1.0 - bn_momentum) * r_mean[j] + bn_momentum * bn_mean[j];
            r_var[j] = (1.0 - bn_momentum) * r_var[j] + bn_momentum * bn_var[j] * (double)n_rows / (double)(n_rows - 1);
        }
    }
    free(bn_mean); free(bn_var); free(bn_rstd);
    if (loss_out) *loss_out = loss;
    if (grad_out) memcpy(grad_out, grad, sizeof(double) * (size_t)nt);
    free(w1r); free(w2r); free(d1); free(hd); free(dl); free(row_loss); free(grad); free(zh_all); free(dy_all);
    return bad_label ? ORACLE_BAD_ARG : ORACLE_OK;
}

int oracle_mlp_train_step(int32_t d_in, int32_t hidden, int32_t n_classes,
                          double *theta, double *adam_m, double *adam_v,
                          int32_t optimizer, double lr, double beta1, double beta2, double eps,
                          int64_t step, int32_t round_bf16,
                          const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                          const int32_t *y, double *loss_out, double *grad_out)
{
    return train_step_impl(d_in, hidden, n_classes, theta, adam_m, adam_v, optimizer, lr, beta1, beta2, eps, step,
                           round_bf16, x, ldx, row_idx, n_rows, y, loss_out, grad_out, 0.0, 0, NULL, 0, 0.0, 0.0);
}

/* The same step, also returning dX [n_rows x d_in], the gradient of the loss with respect to the batch
 * rows (taken with the weights as they are before the update). */
int oracle_mlp_train_step_dx(int32_t d_in, int32_t hidden, int32_t n_classes,
                             double *theta, double *adam_m, double *adam_v,
                             int32_t optimizer, double lr, double beta1, double beta2, double eps,
                             int64_t step, int32_t round_bf16,
                             const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                             const int32_t *y, double *loss_out, double *grad_out, double *dx_out)
{
    return train_step_impl(d_in, hidden, n_classes, theta, adam_m, adam_v, optimizer, lr, beta1, beta2, eps, step,
                           round_bf16, x, ldx, row_idx, n_rows, y, loss_out, grad_out, 0.0, 0, dx_out, 0, 0.0, 0.0);
}

/* The same step with dropout on the hidden units: Hd = ReLU(X W1 + b1) .* keep,
 * keep = 1/(1-p) with probability 1-p, else 0 (see dropout_row); the classifier,
 * the loss and the backward pass see the masked, scaled Hd. */
int oracle_mlp_train_step_dropout(int32_t d_in, int32_t hidden, int32_t n_classes,
                                  double *theta, double *adam_m, double *adam_v,
                                  int32_t optimizer, double lr, double beta1, double beta2, double eps,
                                  int64_t step, int32_t round_bf16,
                                  const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                                  const int32_t *y, double *loss_out, double *grad_out,
                                  double drop_p, uint64_t drop_seed)
{
    return train_step_impl(d_in, hidden, n_classes, theta, adam_m, adam_v, optimizer, lr, beta1, beta2, eps, step,
                           round_bf16, x, ldx, row_idx, n_rows, y, loss_out, grad_out, drop_p, drop_seed, NULL, 0, 0.0, 0.0);
}

/* The same step with layer normalisation inside f_theta (see oracle_theta_size_ln for the reading and the
 * layout of theta, adam_m, adam_v and grad_out); dx_out optional. */
int oracle_mlp_train_step_ln(int32_t d_in, int32_t hidden, int32_t n_classes,
                             double *theta, double *adam_m, double *adam_v,
                             int32_t optimizer, double lr, double beta1, double beta2, double eps,
                             int64_t step, int32_t round_bf16,
                             const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                             const int32_t *y, double *loss_out, double *grad_out, double *dx_out, double ln_eps)
{
    return train_step_impl(d_in, hidden, n_classes, theta, adam_m, adam_v, optimizer, lr, beta1, beta2, eps, step,
                           round_bf16, x, ldx, row_idx, n_rows, y, loss_out, grad_out, 0.0, 0, dx_out, 1, ln_eps, 0.0);
}

/* The same step with batch normalisation inside f_theta (see oracle_theta_size_norm for the reading and the
 * layout of theta, adam_m, adam_v and grad_out); dx_out optional. */
int oracle_mlp_train_step_bn(int32_t d_in, int32_t hidden, int32_t n_classes,
                             double *theta, double *adam_m, double *adam_v,
                             int32_t optimizer, double lr, double beta1, double beta2, double eps,
                             int64_t step, int32_t round_bf16,
                             const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                             const int32_t *y, double *loss_out, double *grad_out, double *dx_out, double bn_eps,
                             double bn_momentum)
{
    return train_step_impl(d_in, hidden, n_classes, theta, adam_m, adam_v, optimizer, lr, beta1, beta2, eps, step,
                           round_bf16, x, ldx, row_idx, n_rows, y, loss_out, grad_out, 0.0, 0, dx_out, 2, bn_eps,
                           bn_momentum);
}

/* Forward of the trained per-node model over a set of rows.
 *   hidden > 0: hidden_out = ReLU(x W1 + b1)  — the representation Q^m that
 *               the next round aggregates, the classifier being dropped
 *               (Section 3.1) — and/or logits = hidden W2 + b2;
 *   hidden == 0: logits = x W1 + b1 (hidden_out must be NULL).
 * pred = argmax of the fp32-rounded logits, lowest index on ties;
 * correct = number of rows with pred == y[i] (y optional). */
static int embed_impl(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                      int32_t round_bf16,
                      const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                      float *hidden_out, int64_t ld_hidden,
                      float *logits_out, int64_t ld_logits,
                      int32_t *pred_out, const int32_t *y, uint64_t *correct_out,
                      int32_t layer_norm, double ln_eps)
{
    if (d_in <= 0 || n_classes <= 0 || hidden < 0 || n_rows < 0 || ldx < d_in) return ORACLE_BAD_ARG;
    if (hidden == 0 && hidden_out) return ORACLE_BAD_ARG;
    if (layer_norm && (hidden <= 0 || ln_eps <= 0.0)) return ORACLE_BAD_ARG;
    const double *ln_gamma = layer_norm ? theta + oracle_theta_size(d_in, hidden, n_classes) : NULL;
    const double *ln_beta = layer_norm ? ln_gamma + hidden : NULL;
    /* batch normalisation (2): evaluation uses the running statistics kept in theta */
    const double *bn_mean = layer_norm == 2 ? ln_beta + hidden : NULL;
    double *bn_rstd = NULL;
    if (layer_norm == 2) {
        bn_rstd = (double *)malloc(sizeof(double) * (size_t)hidden);
        if (!bn_rstd) return ORACLE_NO_MEM;
        for (int32_t j = 0; j < hidden; ++j) bn_rstd[j] = 1.0 / sqrt(bn_mean[hidden + j] + ln_eps);
    }
    double *w1r, *w2r;
    if (rounded_weights(d_in, hidden, n_classes, theta, round_bf16, &w1r, &w2r)) { free(bn_rstd); return ORACLE_NO_MEM; }
    uint64_t correct = 0;
#pragma omp parallel reduction(+ : correct)
    {
        double *a1 = (double *)malloc(sizeof(double) * (size_t)(hidden > 0 ? hidden : 1));
        double *lg = (double *)malloc(sizeof(double) * (size_t)n_classes);
#pragma omp for schedule(static)
        for (int64_t i = 0; i < n_rows; ++i) {
            int64_t r = row_idx ? row_idx[i] : i;
            forward_row_ln(d_in, hidden, n_classes, theta, round_bf16, x + r * ldx, w1r, w2r, a1, lg, NULL,
                           ln_gamma, ln_beta, ln_eps, NULL, NULL, bn_mean, bn_rstd);
            if (hidden_out)
                for (int32_t j = 0; j < hidden; ++j)
                    hidden_out[i * ld_hidden + j] = (float)(a1[j] > 0.0 ? a1[j] : 0.0);
            if (logits_out)
                for (int32_t c = 0; c < n_classes; ++c) logits_out[i * ld_logits + c] = (float)lg[c];
            int32_t best = 0;
            for (int32_t c = 1; c < n_classes; ++c)
                if ((float)lg[c] > (float)lg[best]) best = c;
            if (pred_out) pred_out[i] = best;
            if (y && best == y[i]) correct += 1;
        }
        free(a1);
        free(lg);
    }
    if (correct_out) *correct_out = correct;
    free(w1r);
    free(w2r);
    free(bn_rstd);
    return ORACLE_OK;
}

int oracle_embed(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                 int32_t round_bf16,
                 const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                 float *hidden_out, int64_t ld_hidden,
                 float *logits_out, int64_t ld_logits,
                 int32_t *pred_out, const int32_t *y, uint64_t *correct_out)
{
    return embed_impl(d_in, hidden, n_classes, theta, round_bf16, x, ldx, row_idx, n_rows, hidden_out, ld_hidden,
                      logits_out, ld_logits, pred_out, y, correct_out, 0, 0.0);
}

/* The same with batch normalisation in evaluation mode (running statistics; theta as oracle_theta_size_norm says). */
int oracle_embed_bn(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                    int32_t round_bf16,
                    const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                    float *hidden_out, int64_t ld_hidden,
                    float *logits_out, int64_t ld_logits,
                    int32_t *pred_out, const int32_t *y, uint64_t *correct_out, double bn_eps)
{
    return embed_impl(d_in, hidden, n_classes, theta, round_bf16, x, ldx, row_idx, n_rows, hidden_out, ld_hidden,
                      logits_out, ld_logits, pred_out, y, correct_out, 2, bn_eps);
}

/* The same with layer normalisation inside f_theta: hidden_out = ReLU(gamma .* zhat + beta), theta laid out as
 * oracle_theta_size_ln says. */
int oracle_embed_ln(int32_t d_in, int32_t hidden, int32_t n_classes, const double *theta,
                    int32_t round_bf16,
                    const float *x, int64_t ldx, const int32_t *row_idx, int64_t n_rows,
                    float *hidden_out, int64_t ld_hidden,
                    float *logits_out, int64_t ld_logits,
                    int32_t *pred_out, const int32_t *y, uint64_t *correct_out, double ln_eps)
{
    return embed_impl(d_in, hidden, n_classes, theta, round_bf16, x, ldx, row_idx, n_rows, hidden_out, ld_hidden,
                      logits_out, ld_logits, pred_out, y, correct_out, 1, ln_eps);
}

/* ================================================================== */
/* Messages and bytes that cross a given node partition in one lazy    */
/* message-passing round (Section 2.1 boundary nodes; Appendix A.1).   */
/*   cross_edges    = #{CSR entries (u,v): part[u] != part[v]}         */
/*   boundary_pairs = #{distinct (u, part[v]) over those entries}      */
/*                  = sum over workers i of B_i (its boundary nodes)   */
/*   send_per_part[p] = pairs whose node u lives in p                  */
/*   recv_per_part[p] = pairs whose destination partition is p  (=B_p) */
/*   bytes_per_round[m] = boundary_pairs * dims[m] * elem_bytes        */
/*   bytes_total = sum_m bytes_per_round[m]; the appendix' DV^lazy_lt  */
/*   counts every message at sender and receiver, i.e. 2 * bytes_total */
/* ================================================================== */
static int cmp_i32(const void *a, const void *b)
{
    int32_t x = *(const int32_t *)a, y = *(const int32_t *)b;
    return (x > y) - (x < y);
}

int oracle_cross_partition(int64_t n, const int64_t *rowptr, const int32_t *colidx,
                           const int32_t *part, int32_t n_parts,
                           int32_t K, const int32_t *dims, int32_t elem_bytes,
                           uint64_t *cross_edges, uint64_t *boundary_pairs,
                           uint64_t *bytes_per_round, uint64_t *bytes_total,
                           uint64_t *send_per_part, uint64_t *recv_per_part)
{
    if (n < 0 || n_parts <= 0 || K < 0 || elem_bytes <= 0) return ORACLE_BAD_ARG;
    for (int64_t v = 0; v < n; ++v)
        if (part[v] < 0 || part[v] >= n_parts) return ORACLE_BAD_ARG;
    uint64_t ce = 0, bp = 0;
    if (send_per_part) memset(send_per_part, 0, sizeof(uint64_t) * (size_t)n_parts);
    if (recv_per_part) memset(recv_per_part, 0, sizeof(uint64_t) * (size_t)n_parts);
    for (int64_t u = 0; u < n; ++u) {
        int64_t deg = rowptr[u + 1] - rowptr[u];
        if (deg == 0) continue;
        int32_t *dst = (int32_t *)malloc(sizeof(int32_t) * (size_t)deg);
        if (!dst) return ORACLE_NO_MEM;
        int64_t m = 0;
        for (int64_t e = rowptr[u]; e < rowptr[u + 1]; ++e) {
            int64_t v = colidx[e];
            if (part[v] != part[u]) dst[m++] = part[v];
        }
        ce += (uint64_t)m;
        qsort(dst, (size_t)m, sizeof(int32_t), cmp_i32);
        for (int64_t a = 0; a < m; ++a) {
            if (a > 0 && dst[a] == dst[a - 1]) continue;
            bp += 1;
            if (send_per_part) send_per_part[part[u]] += 1;
            if (recv_per_part) recv_per_part[dst[a]] += 1;
        }
        free(dst);
    }
    uint64_t tot = 0;
    for (int32_t m = 0; m < K; ++m) {
        uint64_t b = bp * (uint64_t)dims[m] * (uint64_t)elem_bytes;
        if (bytes_per_round) bytes_per_round[m] = b;
        tot += b;
    }
    if (cross_edges) *cross_edges = ce;
    if (boundary_pairs) *boundary_pairs = bp;
    if (bytes_total) *bytes_total = tot;
    return ORACLE_OK;
}
