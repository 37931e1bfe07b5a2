/*
 * retexo.h — C ABI of the on-device hot path of lazy message passing (LMP),
 * the layer-by-layer GNN training order of "Scalable Neural Network Training
 * over Distributed Graphs" (Retexo).
 *
 * One LMP round m = 1..K (Section 3.1) is, on the device:
 *   1. one full-graph neighbour aggregation of the previous representations
 *      Q^{m-1} (Eq. 1: AGGR + COMBINE)                   -> retexo_aggregate
 *   2. R full-batch training iterations of the per-node model
 *      (f_theta = Linear+ReLU, temporary classifier C_theta = Linear; the last
 *      round is a single Linear)                          -> retexo_mlp_train_step
 *   3. emission of Q^m = ReLU(X W1 + b1) with the classifier dropped, or of
 *      logits / predictions / accuracy                    -> retexo_embed
 * and, once per graph + partition, the number of boundary-node messages and
 * bytes one round sends across the partition (Section 2.1, Appendix A.1)
 *                                                         -> retexo_cross_partition_bytes
 * retexo_lmp_train runs the whole K-round loop on the device.
 *
 * General rules
 *   - Plain C, no exceptions.  Every function returns a retexo_status
 *     (RETEXO_OK = 0); retexo_status_string names it.
 *   - Unless a parameter says "host", every array pointer is a DEVICE pointer
 *     owned by the caller.  The library never allocates or frees device
 *     memory: scratch comes from the caller's `workspace` (size from the
 *     matching *_workspace_size query, 256-byte aligned).
 *   - Work is enqueued on the caller's stream (`stream` is a cudaStream_t
 *     passed as void*, NULL = default stream) without synchronising, except
 *     where stated.  Scalar results go to caller-provided device memory.
 *   - Arguments are validated on the host first; a call that returns an error
 *     other than RETEXO_ERR_CUDA has launched nothing.  Inputs are never
 *     modified.  There is no CPU fallback: without a CUDA device every
 *     compute call fails with RETEXO_ERR_CUDA.
 *   - Results are deterministic: no floating-point atomics are used, so the
 *     same inputs give the same bits on every call.
 *   - Graphs are symmetric CSR (both directions of each undirected edge
 *     stored; Section 2.1: graphs are undirected), without self loops or
 *     duplicate entries, column indices ascending inside a row.
 */
#ifndef RETEXO_H
#define RETEXO_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum retexo_status {
    RETEXO_OK = 0,
    RETEXO_ERR_INVALID_ARG = 1,   /* null pointer, negative size, bad enum, ld too small */
    RETEXO_ERR_BAD_GRAPH = 2,     /* reported by retexo_validate_csr */
    RETEXO_ERR_ALIGNMENT = 3,     /* a pointer / leading dimension breaks a stated alignment rule */
    RETEXO_ERR_WORKSPACE = 4,     /* workspace NULL, misaligned or too small */
    RETEXO_ERR_UNSUPPORTED = 5,   /* shape outside what the kernels cover (stated per call) */
    RETEXO_ERR_CUDA = 6,          /* a CUDA runtime call or launch failed / no device */
    RETEXO_ERR_TIMEOUT = 7        /* a bounded device-side wait gave up (status word set) */
} retexo_status;

const char* retexo_status_string(int status);
/* Library version, major*10000 + minor*100 + patch. */
int retexo_version(void);

/* ------------------------------------------------------------------ graph */
typedef struct retexo_csr {
    int64_t n_nodes;
    int64_t n_edges;          /* = rowptr[n_nodes]; directed count = 2 |E_undirected| */
    const int64_t* rowptr;    /* device, [n_nodes + 1] */
    const int32_t* colidx;    /* device, [n_edges] */
} retexo_csr;

/* Checks rowptr[0] == 0, rowptr monotone, rowptr[n] == n_edges, 0 <= colidx < n,
 * no self loop, strictly ascending columns inside a row.  Writes to
 * status_out (device, int64[2]): [0] = number of violations found,
 * [1] = index (row or edge) of one of them (-1 if none).  Host reads it after
 * synchronising.  Needs no workspace. */
int retexo_validate_csr(const retexo_csr* g, int64_t* status_out, void* stream);

/* ------------------------------------------------------------ aggregation */
typedef enum retexo_aggr { RETEXO_GCN = 0, RETEXO_SAGE_MEAN = 1, RETEXO_GAT = 2, RETEXO_SAGE_MAX = 3 } retexo_aggr;

typedef struct retexo_gat_params {
    int32_t heads, head_dim;        /* dim must equal heads * head_dim; heads <= 8 */
    const float* a_src;             /* device, [heads x head_dim], applied to the neighbour u */
    const float* a_dst;             /* device, [heads x head_dim], applied to the destination v */
    float negative_slope;           /* LeakyReLU slope of the edge score */
    int32_t add_self_loop;          /* 1: v attends over N(v) and itself */
} retexo_gat_params;

size_t retexo_aggregate_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t type, int32_t dim,
                                       int32_t heads);

/* One message-passing round over the whole graph: the AGGR (+ COMBINE) of
 * Eq. 1 applied to q = Q^{m-1} (fp32, row-major, row stride ldq >= dim).
 *   RETEXO_GCN       out[v] = n_v ( n_v q[v] + sum_{u in N(v)} n_u q[u] ),
 *                    n_x = (deg x + 1)^-1/2  (symmetric normalisation with an
 *                    implicit self loop); out is [n x dim].
 *   RETEXO_SAGE_MEAN mean[v] = (1/deg v) sum_{u in N(v)} q[u], zeros if
 *                    deg v = 0.  concat_self = 1: out is [n x 2 dim] with
 *                    q[v] in columns [0,dim) and the mean in [dim, 2 dim)
 *                    (COMBINE = concatenation); concat_self = 0: out is
 *                    [n x dim], the mean only.
 *   RETEXO_SAGE_MAX  the max-pooling aggregator Section 2.2 names for
 *                    GraphSAGE: max[v][j] = max_{u in N(v)} q[u][j], zeros
 *                    if deg v = 0; the pooling layer's own transform is not
 *                    applied here (q is taken as already transformed).  Same
 *                    output layout and concat_self rule as RETEXO_SAGE_MEAN.
 *                    Exact (no rounding) for finite q.
 *   RETEXO_GAT       q holds already projected rows, head k in columns
 *                    [k*head_dim, (k+1)*head_dim).  Per head:
 *                    e_uv = LeakyReLU(<a_src,q_u> + <a_dst,q_v>),
 *                    alpha = softmax over u in N(v) (+ v), out[v] = sum alpha q[u];
 *                    scores, softmax and weighted sum happen in one pass.
 *                    Rows with an empty softmax set give zeros.  dim <= 256.
 * out      fp32 [n x ldout], may be NULL if out_bf16 is given.
 * out_bf16 optional bf16 (round-to-nearest-even) copy of the same matrix,
 *          row stride ldout_bf16 elements; NULL if not wanted.
 * Sums are taken in CSR order per row in fp32; rows of at least 4096 entries
 * are cut into segments of 2048 entries whose sums are added in segment order.
 * 128-bit loads are used when q is 16-byte aligned, ldq % 4 == 0 and
 * ldq >= round_up(dim, 4); 64-bit loads under the analogous rule; otherwise
 * scalar loads.  Nothing is an error for being unaligned.
 * dim <= 4096.  Errors: INVALID_ARG, WORKSPACE, UNSUPPORTED. */
int retexo_aggregate(const retexo_csr* g, int32_t type,
                     const float* q, int64_t ldq, int32_t dim,
                     const retexo_gat_params* gat,
                     float* out, int64_t ldout, int32_t concat_self,
                     void* out_bf16, int64_t ldout_bf16,
                     void* workspace, size_t workspace_bytes, void* stream);

size_t retexo_gat_backward_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t heads, int32_t dim);

/* Backward of RETEXO_GAT, for rounds that train the aggregator as well (Section 2.2: "AGGR may have
 * trainable parameters"; Section 3.1: a round trains the whole layer): given dz = dLoss / dOut
 * (fp32 [n x lddz]; rows of nodes outside the loss are zero) and the same p and parameters the forward
 * pass took, computes
 *   dp      fp32 [n x lddp] and / or bf16 [n x lddp_bf16] (either may be NULL, not both): dLoss / dp,
 *           through the weighted sum and through both score terms;
 *   da_src, da_dst  fp32 [heads x head_dim]: gradients of the attention vectors.
 * Scores, soft-max and every sum are fp32; sums run in CSR order per row, the parameter gradients are
 * summed per thread block and then in block order (deterministic).  The graph must be symmetric (the rows
 * that attend over u are read off u's own row).  heads <= 8, heads * head_dim <= 256.
 * Errors: INVALID_ARG, WORKSPACE, UNSUPPORTED. */
int retexo_gat_backward(const retexo_csr* g, const float* p, int64_t ldp, const retexo_gat_params* gat,
                        const float* dz, int64_t lddz, float* dp, int64_t lddp, void* dp_bf16, int64_t lddp_bf16,
                        float* da_src, float* da_dst, void* workspace, size_t workspace_bytes, void* stream);

/* --------------------------------------------------------- per-node model */
typedef enum retexo_optimizer { RETEXO_SGD = 0, RETEXO_ADAM = 1 } retexo_optimizer;

/* The trainable part of round m (Section 3.1).  theta is one flat fp32
 * device array, matrices row-major [in x out]:
 *   hidden > 0 : [ W1 (d_in x hidden) | b1 (hidden) | W2 (hidden x n_classes) | b2 (n_classes) ]
 *   hidden == 0: [ W1 (d_in x n_classes) | b1 (n_classes) ]       (last round)
 * adam_m / adam_v have the same length (NULL for SGD).  `step` counts the
 * updates already applied; retexo_mlp_train_step increments it.
 * Every matrix product takes both operands rounded to bf16 and accumulates in
 * fp32 on the tensor cores (a bias gradient is the product of the all-ones
 * vector with the layer's output gradient and follows the same rule); biases,
 * softmax, loss and the optimiser are fp32.  A device-side wait that runs out
 * (it never should) makes the reported loss NaN. */
typedef enum retexo_norm { RETEXO_NORM_NONE = 0, RETEXO_NORM_LAYER = 1, RETEXO_NORM_BATCH = 2 } retexo_norm;

typedef struct retexo_mlp {
    int32_t d_in, hidden, n_classes;
    float* theta;
    float* adam_m;
    float* adam_v;
    int32_t optimizer;              /* retexo_optimizer */
    float lr, beta1, beta2, eps;    /* Adam: bias-corrected, eps outside the root, no weight decay */
    int64_t step;
    /* Dropout on the hidden units while training (Appendix B lists dropout rates among the
     * hyper-parameters): unit j of batch row i is dropped in update number s = step + 1 iff word (j mod 4)
     * of Philox4x32-10(counter = (i, j / 4, s, 0), key = (low, high word of dropout_seed)) is below
     * floor(dropout * 2^32); kept units are scaled by 1 / (1 - dropout).  0 <= dropout < 1; 0 = none.
     * retexo_embed (evaluation) never drops. */
    float dropout;
    uint64_t dropout_seed;
    /* Optional device int32.  Every device-side wait of the tensor-core kernels is bounded; one that runs out
     * (it never should) makes its block give up in order and raises a status word.  After the kernels of a
     * retexo_mlp_train_step / retexo_embed call the word is copied here: RETEXO_OK, or RETEXO_ERR_TIMEOUT
     * (the loss of that step is then NaN and its outputs are not to be used).  Read it after synchronising. */
    int32_t* status_out;
    /* Normalisation inside f_theta (Section 2.2 names batch and layer normalisation among its parts; the
     * paper's configurations use none).  With norm != RETEXO_NORM_NONE and hidden > 0 (ignored when hidden == 0):
     *   z = X W1 + b1,  Hd = ReLU(gamma .* zhat + beta),  gamma and beta trained;
     * RETEXO_NORM_LAYER: zhat = (z - mean z) / sqrt(var z + norm_eps) over the hidden units of a row (biased
     *   variance); theta = [W1 | b1 | W2 | b2 | gamma | beta].
     * RETEXO_NORM_BATCH: per hidden unit over the rows of the batch.  retexo_mlp_train_step uses the batch's own
     *   mean and biased variance and then moves the running statistics kept in theta,
     *   r_mean <- (1 - bn_momentum) r_mean + bn_momentum mean,  r_var likewise with the unbiased variance
     *   (n_rows >= 2); retexo_embed (evaluation, emission) normalises with the running statistics;
     *   theta = [W1 | b1 | W2 | b2 | gamma | beta | r_mean | r_var]; the running statistics are state: the
     *   optimiser does not touch them and their entries of grad_out are 0.
     * theta, adam_m, adam_v, grad_out hold retexo_theta_size_norm entries.  The normalisation is computed in fp32,
     * forward and backward; hidden <= 512; not combined with dropout (UNSUPPORTED).  Workspaces: the
     * *_workspace_size_norm functions. */
    int32_t norm;                   /* retexo_norm */
    float norm_eps;
    float bn_momentum;
} retexo_mlp;

int64_t retexo_theta_size(int32_t d_in, int32_t hidden, int32_t n_classes);
int64_t retexo_theta_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes, int32_t norm);

/* Gathers rows of a matrix into a dense bf16 batch: dst[i] = bf16(src[idx ? idx[i] : i]).
 * src is fp32 (src_is_bf16 = 0) or bf16 (1), row stride ld_src elements;
 * dst is bf16 [n_rows x ld_dst], ld_dst >= dim; columns [dim, ld_dst) are
 * zero-filled.  dst_t (optional) receives the transpose, bf16 [dim x ld_t],
 * ld_t >= n_rows, columns [n_rows, ld_t) zero-filled.  With ones = 1 the batch
 * carries the all-ones vector as well: column `dim` of dst holds 1 in every row
 * (ld_dst > dim required) and dst_t has one more row (index dim) that holds 1
 * for every batch row; the form retexo_mlp_train_step takes with
 * x_has_ones = 1.  dst may be NULL if only the transpose is wanted.
 * Needs no workspace. */
int retexo_pack_rows(const void* src, int32_t src_is_bf16, int64_t ld_src, int32_t dim,
                     const int32_t* idx, int64_t n_rows,
                     void* dst, int64_t ld_dst, void* dst_t, int64_t ld_t, int32_t ones, void* stream);

size_t retexo_mlp_train_step_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes,
                                            int64_t n_rows);
size_t retexo_mlp_train_step_workspace_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes,
                                               int64_t n_rows, int32_t norm);

/* One full-batch training iteration (Section 2.3: forward, loss, backward,
 * update; with a single worker the gradient average is the identity):
 *   hidden > 0 : Hd = ReLU(X W1 + b1), L = Hd W2 + b2
 *   hidden == 0: L = X W1 + b1
 *   loss = mean_i CE(softmax(L_i), y_i), gradients by back-propagation,
 *   then one SGD / Adam update of theta in place.
 * x     bf16 [n_rows x ldx]: the batch, one training node per row
 *       (retexo_pack_rows builds it once per round); ldx % 8 == 0 and x
 *       16-byte aligned.  The weight-gradient products read it as it lies,
 *       reducing over the rows.
 * x_has_ones  1: column d_in of x holds 1 in every row (ldx > d_in;
 *       retexo_pack_rows with ones = 1 writes it).  That column makes the bias
 *       gradient one more output row of the weight-gradient product.  0: the
 *       call first copies x into its workspace with that column added, at the
 *       price of one more pass over x per call.
 * y     int32 [n_rows] labels in [0, n_classes).
 * loss_out  device float, the loss before the update (may be NULL).
 * grad_out  optional device fp32 array shaped like theta: the gradient.
 * dx_out    optional device fp32 [n_rows x ld_dx], ld_dx >= d_in: dLoss / dx, the gradient with respect
 *           to the batch rows themselves (one more product, dHd W1^T).  A round whose aggregator has
 *           parameters (Section 2.2) passes it on to retexo_gat_backward.
 * Increments model->step (host struct).  n_classes <= 64, hidden <= 512.
 * Errors: INVALID_ARG, ALIGNMENT, WORKSPACE, UNSUPPORTED. */
int retexo_mlp_train_step(retexo_mlp* model,
                          const void* x, int64_t ldx, int32_t x_has_ones,
                          const int32_t* y, int64_t n_rows,
                          float* loss_out, float* grad_out, float* dx_out, int64_t ld_dx,
                          void* workspace, size_t workspace_bytes, void* stream);

size_t retexo_embed_workspace_size(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows);
size_t retexo_embed_workspace_size_norm(int32_t d_in, int32_t hidden, int32_t n_classes, int64_t n_rows,
                                      int32_t norm);

/* Forward of the per-node model over rows x[row_idx ? row_idx[i] : i]
 * (x bf16, row stride ldx, 16-byte aligned, ldx % 8 == 0):
 *   hidden_out / hidden_out_bf16 : ReLU(x W1 + b1), i.e. the representation
 *       Q^m handed to the next round once the classifier is dropped
 *       (requires hidden > 0); fp32 [n_rows x ld_hidden] and/or bf16
 *       [n_rows x ld_hidden_bf16];
 *   logits_out : fp32 [n_rows x ld_logits];
 *   pred_out   : int32 [n_rows], argmax of the fp32 logits, lowest class on ties;
 *   correct_out: uint64, number of rows with pred == y[i] (y: int32 [n_rows]).
 * Every output pointer may be NULL.  With hidden > 0 and only hidden outputs
 * requested the classifier is not evaluated. */
int retexo_embed(const retexo_mlp* model,
                 const void* x, int64_t ldx, const int32_t* row_idx, int64_t n_rows,
                 float* hidden_out, int64_t ld_hidden,
                 void* hidden_out_bf16, int64_t ld_hidden_bf16,
                 float* logits_out, int64_t ld_logits,
                 int32_t* pred_out, const int32_t* y, uint64_t* correct_out,
                 void* workspace, size_t workspace_bytes, void* stream);

/* Packs rows of a fp32 matrix for the one exchange of a round (Section 3.4, sync_embeddings): dst[i] = src[idx[i]],
 * dim columns each (idx: device, row indices into src; ld_src, ld_dst >= dim).  A worker of a sharded run calls it
 * once per peer with the list of its owned rows that peer aggregates over, hands the packed rows to the transport
 * (an all-to-all with per-peer counts), and aggregates over [owned rows | received rows] with retexo_aggregate on
 * its local CSR.  Needs no workspace.  Errors: INVALID_ARG, CUDA. */
int retexo_gather_rows(const float* src, int64_t ld_src, int32_t dim, const int32_t* idx, int64_t n_rows,
                       float* dst, int64_t ld_dst, void* stream);

/* ------------------------------------------------ cross-partition traffic */
size_t retexo_cross_partition_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t n_parts);

/* Messages and bytes one LMP round sends across a given node partition.
 * A message is one (node u, destination partition p) pair with p != part[u]
 * and some neighbour of u living in p: u is a boundary node of worker p
 * (Section 2.1) and its representation crosses once per round (Appendix A.1).
 *   cross_edges     = #{CSR entries (u,v) : part[u] != part[v]}
 *   boundary_pairs  = number of distinct such pairs = sum over workers of B_i
 *   bytes_per_round[m] = boundary_pairs * dims[m] * elem_bytes, m = 0..K-1,
 *                        dims[m] = width of the representation sent in round m+1
 *   bytes_total     = sum over rounds; the appendix' DV^lazy_lt counts each
 *                     message at sender and receiver, i.e. 2 * bytes_total
 *   send_per_part[p] = pairs whose node lives in p; recv_per_part[p] = pairs
 *                     destined to p (= B_p).  Optional, uint64 [n_parts].
 * part: int32 [n_nodes] with values in [0, n_parts) (a value outside that range
 * sets every scalar output to UINT64_MAX); dims: HOST int32 [K].
 * All outputs are device uint64, exact.  Errors: INVALID_ARG, WORKSPACE. */
int retexo_cross_partition_bytes(const retexo_csr* g, const int32_t* part, int32_t n_parts,
                                 int32_t K, const int32_t* dims, int32_t elem_bytes,
                                 uint64_t* cross_edges, uint64_t* boundary_pairs,
                                 uint64_t* bytes_per_round, uint64_t* bytes_total,
                                 uint64_t* send_per_part, uint64_t* recv_per_part,
                                 void* workspace, size_t workspace_bytes, void* stream);

/* The same count for callers that cannot allocate device memory at all: code
 * running inside a framework that owns the allocator, a plug-in loaded into a
 * process whose memory budget is fixed up front, a latency-critical loop where
 * cudaMalloc's implicit synchronisation is not acceptable.  (The paper has no
 * counterpart of this call; it is a convenience of this library.)
 * It needs no workspace argument: its scratch is a fixed 4 MiB array inside
 * the library image (retexo_cross_partition_static_scratch_bytes), which every
 * GPU that loads the library holds until the process exits.  The call itself
 * calls no cudaMalloc / cudaFree and no allocating library routine.
 *   - Limit: a problem whose scratch need
 *     (retexo_cross_partition_workspace_size) exceeds that array is rejected
 *     with RETEXO_ERR_UNSUPPORTED and nothing is launched.  Up to 8192
 *     partitions the need is about 1 KiB whatever the graph's size; beyond
 *     that it grows as 4 n_nodes + 18.5 n_parts bytes (+ 1 KiB).
 *   - The first call on a device looks the array's device address up
 *     (one-time set-up, per device, with that device current); make that first
 *     call before any stream capture.
 *   - All calls on a device share the one array: two calls whose kernels may
 *     overlap on the GPU (different streams, no ordering) race and give wrong
 *     counts.  Calls ordered on one stream are fine; each call clears the
 *     counters it uses.
 * Arguments, outputs and errors otherwise as retexo_cross_partition_bytes. */
size_t retexo_cross_partition_static_scratch_bytes(void);
int retexo_cross_partition_bytes_static(const retexo_csr* g, const int32_t* part, int32_t n_parts,
                                        int32_t K, const int32_t* dims, int32_t elem_bytes,
                                        uint64_t* cross_edges, uint64_t* boundary_pairs,
                                        uint64_t* bytes_per_round, uint64_t* bytes_total,
                                        uint64_t* send_per_part, uint64_t* recv_per_part, void* stream);

/* ------------------------------------------- analytical data volume */
typedef struct retexo_data_volume_result {
    double lazy_lt;             /* DV^{lazy}_{lt}:     one exchange of H_0..H_{K-1} per boundary row, both ways */
    double standard_lt;         /* DV^{standard}_{lt}: 2 R exchanges of H_1..H_{K-1} + the cached features */
    double lazy_reduce;         /* DV^{lazy}_{reduce}: 2 n R (M + sum of the temporary classifiers C_m) */
    double standard_reduce;     /* DV^{standard}_{reduce}: 2 n R M */
    double gamma;               /* Eq. 2: (standard_lt + standard_reduce) / (lazy_lt + lazy_reduce) */
    double model_size;          /* M = sum of L */
} retexo_data_volume_result;

/* The closed-form network data volumes of Section 3.3 / Appendix A.1, in
 * elements, and their ratio gamma (Eq. 2).  Host arithmetic only: no device
 * is touched.  H (host) holds the K + 1 representation widths H_0..H_K, L
 * (host) the K layer sizes L_1..L_K; n_workers > 0, B >= 0 boundary nodes per
 * worker, R > 0 training iterations.  C_m = H_m x H_K for m < K.  With
 * n_workers * B set to the boundary_pairs counted by
 * retexo_cross_partition_bytes, lazy_lt equals that call's 2 x bytes_total at
 * elem_bytes = 1.  Errors: INVALID_ARG. */
int retexo_data_volume(int32_t K, const int64_t* H, const int64_t* L, double n_workers, double B, double R,
                       retexo_data_volume_result* out);

/* -------------------------------------------------- the K-round LMP loop */
typedef struct retexo_lmp_config {
    int32_t aggr;                   /* retexo_aggr */
    int32_t K;                      /* rounds = GNN layers, 1..8 */
    int32_t R;                      /* training iterations per round */
    int32_t d0;                     /* feature width */
    int32_t hidden;                 /* width of Q^1..Q^{K-1} */
    int32_t n_classes;
    int32_t optimizer;
    float lr, beta1, beta2, eps;
    int32_t eval_every;             /* validate every this many iterations (and at the last) */
    int32_t gat_heads, gat_head_dim;
    float gat_negative_slope;
    int32_t memory_is_host;         /* 0: every input array below is on the device;
                                       1: every input array is in HOST memory and is copied to the
                                          device inside the call; results are also written to host */
    float dropout;                  /* dropout rate of the hidden units while training (see retexo_mlp); 0 = none */
    uint64_t dropout_seed;          /* round m = 1..K draws its masks with the key dropout_seed + (m - 1) */
    int32_t gat_freeze_attention;   /* RETEXO_GAT only.  0 (default): the round trains the whole layer, i.e. the
                                       projection W_att and the attention vectors together with the per-node model
                                       (Section 2.2: AGGR may have trainable parameters; Section 3.1), re-aggregating
                                       locally in every iteration.  1: they stay at the values given in gat_w and the
                                       aggregation runs once per round */
    int32_t norm;                   /* retexo_norm: normalisation inside f_theta in the rounds that have a hidden layer
                                       (see retexo_mlp): theta0[m], theta_best[m] then hold retexo_theta_size_norm
                                       entries (batch normalisation: theta0 carries the initial running statistics,
                                       theta_best those of the kept iterate) */
    float norm_eps;
    float bn_momentum;
} retexo_lmp_config;

typedef struct retexo_lmp_inputs {
    retexo_csr graph;
    const float* features; int64_t ld_features;       /* fp32 [n x ld] */
    const int32_t* labels;                            /* [n] */
    const int32_t* train_idx; int64_t n_train;
    const int32_t* val_idx;   int64_t n_val;
    const int32_t* test_idx;  int64_t n_test;
    const int32_t* part; int32_t n_parts;             /* may be NULL: skip the count */
    const float* const* theta0;    /* HOST array of K pointers to the initial theta of each round
                                      (pointees: device or host memory, like the other inputs) */
    const float* const* gat_w;     /* GAT only: HOST array of K pointers, each to
                                      [W_att (rep_dim x heads*head_dim) | a_src | a_dst] fp32: the initial
                                      (gat_freeze_attention = 1: the fixed) parameters of each round's aggregator */
} retexo_lmp_inputs;

typedef struct retexo_lmp_outputs {
    float* loss_history;            /* [K*R] loss of every iteration */
    uint64_t* val_correct;          /* [K*R] validation hits per iteration (UINT64_MAX where not evaluated) */
    uint64_t* best_val_correct;     /* [K] */
    int32_t* best_iter;             /* [K] 1-based iteration whose model was kept */
    uint64_t* test_correct;         /* [K] test hits of the kept model of each round */
    uint64_t* test_correct_last;    /* [K] test hits of the last iterate */
    uint64_t* counts;               /* [4 + K]: cross_edges, boundary_pairs, bytes_total, 2*bytes_total,
                                       then bytes_per_round; untouched if part == NULL */
    float* final_logits; int64_t ld_logits;   /* [n x ld] logits of the last round's kept model; may be NULL */
    int32_t* final_pred;            /* [n]; may be NULL */
    float* const* theta_best;       /* HOST array of K pointers receiving each round's kept theta; may be NULL */
    float* const* gat_best;         /* GAT only: HOST array of K pointers receiving each round's kept
                                       [W_att | a_src | a_dst]; may be NULL */
    int32_t* status;                /* optional, one int32 (device, or host with memory_is_host): RETEXO_OK, or
                                       RETEXO_ERR_TIMEOUT if a bounded device-side wait ran out in any round
                                       (the results are then not to be used) */
} retexo_lmp_outputs;

size_t retexo_lmp_workspace_size(const retexo_lmp_config* cfg, int64_t n_nodes, int64_t n_edges,
                                 int64_t n_train, int64_t n_val, int64_t n_test, int32_t n_parts);

/* Lazy message passing (Section 3.1), entirely on the device: for m = 1..K
 * { aggregate Q^{m-1} once; train the round's per-node model for R iterations
 *   from theta0[m]; every eval_every iterations measure validation accuracy
 *   and keep the iterate with the most hits (earliest on ties); emit Q^m from
 *   the kept model (last round: logits, predictions, test accuracy) }.
 * GAT: P = Q^{m-1} W_att, then scores, soft-max and weighted sum.  By default the
 * aggregator's parameters are trained with the per-node model: every iteration
 * recomputes P and the aggregation with the current parameters (all local once the
 * round's exchange has delivered Q^{m-1}), back-propagates through the attention
 * (retexo_gat_backward) and updates [W_att | a_src | a_dst] with the same optimiser;
 * the iterate kept on validation keeps its aggregator parameters with it.  With
 * gat_freeze_attention = 1 they stay fixed and the aggregation runs once.
 * With memory_is_host = 0 the call only enqueues work (outputs are device
 * memory); with 1 it copies inputs in, runs, copies outputs to the host
 * arrays and synchronises the stream before returning.
 * Streams: the work is ordered after everything already enqueued on `stream`, and whatever is
 * enqueued on `stream` after the call is ordered after the work.  In between it runs on a stream the
 * call creates and releases itself, because the R iterations of a round (the same launches with the
 * same arguments once the iteration number is kept on the device) are recorded once as a CUDA graph
 * and replayed, which the legacy default stream does not allow.  If no stream or graph can be had
 * the launches go to `stream` one by one.  Do not call it while `stream` is being captured. */
int retexo_lmp_train(const retexo_lmp_config* cfg, const retexo_lmp_inputs* in,
                     const retexo_lmp_outputs* out,
                     void* workspace, size_t workspace_bytes, void* stream);

/* ---------------------------------------------- standard (end-to-end) training */
/* The scheme lazy message passing is compared with (Section 2.3): one model of K layers,
 *   H^0 = F,  X^m = COMBINE(H^{m-1}, AGGR(H^{m-1}))  (Eq. 1),  H^m = ReLU(X^m W_m + b_m) for m < K,
 *   logits = X^K W_K + b_K,
 * trained jointly: every iteration runs the aggregations forward and carries the gradient back through them
 * (the transposed aggregation; on the symmetric graphs this library takes, GCN's is the aggregation itself and
 * SAGE-mean's is dH[u] = g_self[u] + sum_{v in N(u)} g_mean[v] / deg v).  X^1 = AGGR(F) does not change and is
 * computed once, so an iteration runs K - 1 forward and K - 1 transposed aggregations: the exchanges of
 * H^1 .. H^{K-1} and of as many gradients that Appendix A.1 counts for standard training.
 * aggr: RETEXO_GCN or RETEXO_SAGE_MEAN (others: UNSUPPORTED).  Layer m has theta_m = [W_m | b_m],
 * W_m [d_m x out_m] row-major, d_m the width of X^m (d0 or hidden; twice that for SAGE), out_m = hidden for
 * m < K and n_classes for m = K; hidden <= 512, n_classes <= 64.  Loss: mean soft-max cross-entropy over the
 * train rows, full batch.  Validation after every iteration, the iterate with the most hits kept (earliest on
 * ties).  Operand precision as in retexo_mlp (both operands of every product rounded to bf16, sums fp32). */
typedef struct retexo_standard_config {
    int32_t aggr, K, R, d0, hidden, n_classes, optimizer;
    float lr, beta1, beta2, eps;
} retexo_standard_config;

typedef struct retexo_standard_outputs {
    float* loss_history;            /* [R] loss of every iteration (before its update) */
    uint64_t* val_correct;          /* [R] validation hits after every iteration */
    uint64_t* best_val_correct;     /* [1] */
    int32_t* best_iter;             /* [1] 1-based iteration whose weights were kept */
    uint64_t* test_correct;         /* [1] test hits of the kept weights */
    uint64_t* test_correct_last;    /* [1] test hits of the last iterate */
    float* final_logits; int64_t ld_logits;   /* [n x ld] logits of the kept weights over all nodes; may be NULL */
    int32_t* final_pred;            /* [n]; may be NULL */
    float* const* theta_best;       /* HOST array of K device pointers receiving the kept theta_m; may be NULL */
    float* const* grad_last;        /* HOST array of K device pointers receiving the gradients [dW_m | db_m] of the
                                       last iteration run; may be NULL */
    int32_t* status;                /* optional, one int32: RETEXO_OK, or RETEXO_ERR_TIMEOUT if a bounded device-side
                                       wait ran out (the results are then not to be used) */
} retexo_standard_outputs;

size_t retexo_standard_workspace_size(const retexo_standard_config* cfg, int64_t n_nodes, int64_t n_edges,
                                      int64_t n_train, int64_t n_val, int64_t n_test);

/* Runs R iterations from in->theta0[m] (K device arrays; in->part, in->gat_w are ignored; all of `in` and `out`
 * is device memory except the two pointer arrays).  Only enqueues work on `stream`; nothing synchronises.
 * Errors: INVALID_ARG, UNSUPPORTED, WORKSPACE, CUDA. */
int retexo_standard_train(const retexo_standard_config* cfg, const retexo_lmp_inputs* in,
                          const retexo_standard_outputs* out,
                          void* workspace, size_t workspace_bytes, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* RETEXO_H */
