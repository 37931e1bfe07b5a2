// Backward of the GAT aggregation (Section 2.2: AGGR may have trainable parameters; Section 3.1: a round
// trains the whole layer).  With z_uv = s_u + t_v, e = LeakyReLU(z), alpha = softmax over u in N(v) (+ v),
// Z_v = sum_u alpha_uv p_u and dz = dLoss/dZ:
//   dalpha_uv = <dz_v, p_u>             de_uv = alpha_uv (dalpha_uv - c_v),  c_v = sum_w alpha_wv dalpha_wv
//   dzz_uv    = de_uv (z_uv > 0 ? 1 : slope)
//   dt_v = sum_u dzz_uv                 ds_u = sum_v dzz_uv
//   dp_u = sum_v alpha_uv dz_v + ds_u a_src + dt_u a_dst
//   da_src = sum_u ds_u p_u             da_dst = sum_v dt_v p_v
// Two passes over the same CSR (the graph is symmetric, so the rows that attend over u are u's own row):
// one warp per destination v computes the soft-max statistics, c_v and dt_v; one warp per source u then walks
// the destinations v that attend over it and accumulates ds_u and dp_u in CSR order.  No floating-point
// atomics: the parameter gradients are summed per block and the block sums in block order.
#include "common.cuh"

namespace retexo {

constexpr int kGbThreads = 256, kGbWarps = kGbThreads / kWarp, kGbMaxHeads = 8;

struct GatBwdArgs {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const float* p; int64_t ldp;
    int32_t heads, head_dim, dim;
    const float* a_src; const float* a_dst;
    float slope; int32_t self_loop;
    const float* dz; int64_t lddz;
    float* s; float* t;              // [n x heads]
    float4* stats;                   // [n x heads]: (row maximum, 1 / soft-max sum (0 = dz_v is zero), c_v, dt_v)
    float* dp; int64_t lddp;
    __nv_bfloat16* dp16; int64_t lddp16;
    float* partial;                  // [blocks x 2 x dim]: per-block sums of ds_u p_u and dt_u p_u
    // rows of kGbHubEntries entries or more ("hub rows") are listed by the score kernel and taken by whole blocks
    int32_t* hub_count; int32_t* hub_list;      // how many, which (in the order the score kernel met them)
    int32_t* hub_pos;                           // [n]: position in the list, -1 for every other row
    float* hub_sum;                             // [hubs x 72]: per hub row the 64 column sums of its source pass, then ds per head
};

constexpr int kGbHubEntries = 128;   // a warp takes 32 entries per trip: rows this long keep one warp busy while the grid drains
constexpr int kGbHubBlocks = 296;    // blocks of the hub kernels (they loop over the list)

__global__ void __launch_bounds__(kGbThreads) gat_bwd_scores_kernel(GatBwdArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t u = blockIdx.x * (int64_t)kGbWarps + (threadIdx.x >> 5);
    if (u >= a.n) return;
    const float* row = a.p + u * a.ldp;
    for (int h = 0; h < a.heads; ++h) {
        float ss = 0.f, tt = 0.f;
        for (int j = lane; j < a.head_dim; j += kWarp) {
            const float x = row[h * a.head_dim + j];
            ss = fmaf(a.a_src[h * a.head_dim + j], x, ss);
            tt = fmaf(a.a_dst[h * a.head_dim + j], x, tt);
        }
        ss = warp_sum(ss);
        tt = warp_sum(tt);
        if (lane == 0) { a.s[u * a.heads + h] = ss; a.t[u * a.heads + h] = tt; }
    }
    if (a.hub_pos && lane == 0) {
        const int64_t total = a.rowptr[u + 1] - a.rowptr[u] + (a.self_loop ? 1 : 0);
        int32_t pos = -1;
        if (total >= kGbHubEntries) {      // (the list's order varies from run to run; no result depends on it)
            pos = atomicAdd(a.hub_count, 1);
            a.hub_list[pos] = (int32_t)u;
        }
        a.hub_pos[u] = pos;
    }
}

// <x, y> restricted to each head's columns, summed over the warp: every lane ends up with all heads' values.
template <int NC>
__device__ __forceinline__ void head_dots(const float (&x)[NC], const float (&y)[NC], const int (&head_of)[NC], int heads,
                                          float (&out)[kGbMaxHeads]) {
#pragma unroll
    for (int h = 0; h < kGbMaxHeads; ++h) {
        out[h] = 0.f;
        if (h < heads) {
            float part = 0.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) part = head_of[c] == h ? fmaf(x[c], y[c], part) : part;
            out[h] = warp_sum(part);
        }
    }
}

// Pass over destinations: one warp per v.  Lane L owns the columns L, L + 32, ...
template <int NC>
__global__ void __launch_bounds__(kGbThreads) gat_bwd_dst_kernel(GatBwdArgs a) {
    const int lane = threadIdx.x & 31;
    const int64_t v = blockIdx.x * (int64_t)kGbWarps + (threadIdx.x >> 5);
    if (v >= a.n) return;
    int head_of[NC];
    float g[NC];
    bool any = false;
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int col = c * kWarp + lane;
        head_of[c] = col < a.dim ? col / a.head_dim : -1;
        g[c] = col < a.dim ? a.dz[v * a.lddz + col] : 0.f;
        any = any || g[c] != 0.f;
    }
    const int64_t beg = a.rowptr[v];
    const int64_t deg = a.rowptr[v + 1] - beg;
    const int64_t total = deg + (a.self_loop ? 1 : 0);
    if (!__any_sync(0xffffffffu, any) || total == 0) {       // outside the loss: nothing flows back through this row
        if (lane < a.heads) a.stats[v * a.heads + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    float tv[kGbMaxHeads], m[kGbMaxHeads], den[kGbMaxHeads];
#pragma unroll
    for (int h = 0; h < kGbMaxHeads; ++h) {
        tv[h] = h < a.heads ? a.t[v * a.heads + h] : 0.f;
        m[h] = -INFINITY;
        den[h] = 0.f;
    }
    // sweep 1: row maximum and soft-max sum per head, 32 entries at a time (lane j scores entry j)
    for (int64_t e0 = 0; e0 < total; e0 += kWarp) {
        const bool valid = e0 + lane < total;
        const int64_t u = !valid ? v : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : v);
#pragma unroll
        for (int h = 0; h < kGbMaxHeads; ++h) {
            if (h < a.heads) {
                const float z = a.s[u * a.heads + h] + tv[h];
                const float e = valid ? (z > 0.f ? z : a.slope * z) : -INFINITY;
                const float mn = fmaxf(m[h], warp_max(e));
                den[h] = den[h] * expf(m[h] - mn) + warp_sum(valid ? expf(e - mn) : 0.f);
                m[h] = mn;
            }
        }
    }
    // sweep 2: c_v = sum alpha dalpha, and the two sums that give dt_v = sum alpha (dalpha - c_v) g'
    float csum[kGbMaxHeads], a1[kGbMaxHeads], a2[kGbMaxHeads];
#pragma unroll
    for (int h = 0; h < kGbMaxHeads; ++h) { csum[h] = 0.f; a1[h] = 0.f; a2[h] = 0.f; }
    for (int64_t e = 0; e < total; ++e) {
        const int64_t u = e < deg ? (int64_t)__ldg(a.colidx + beg + e) : v;
        float x[NC], dalpha[kGbMaxHeads];
#pragma unroll
        for (int c = 0; c < NC; ++c) {
            const int col = c * kWarp + lane;
            x[c] = col < a.dim ? __ldg(a.p + u * a.ldp + col) : 0.f;
        }
        head_dots<NC>(g, x, head_of, a.heads, dalpha);
#pragma unroll
        for (int h = 0; h < kGbMaxHeads; ++h) {
            if (h < a.heads) {
                const float z = a.s[u * a.heads + h] + tv[h];
                const float alpha = expf((z > 0.f ? z : a.slope * z) - m[h]) / den[h];
                const float gp = z > 0.f ? 1.f : a.slope;
                csum[h] = fmaf(alpha, dalpha[h], csum[h]);
                a1[h] = fmaf(alpha * gp, dalpha[h], a1[h]);
                a2[h] = fmaf(alpha, gp, a2[h]);
            }
        }
    }
#pragma unroll
    for (int h = 0; h < kGbMaxHeads; ++h)
        if (h < a.heads && lane == h) a.stats[v * a.heads + h] = make_float4(m[h], 1.f / den[h], csum[h], a1[h] - csum[h] * a2[h]);
}

// Pass over sources: one warp per u walks the destinations that attend over u (its own row, and itself).
template <int NC>
__global__ void __launch_bounds__(kGbThreads) gat_bwd_src_kernel(GatBwdArgs a) {
    __shared__ float sm_part[kGbWarps][2][NC * kWarp];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t u = blockIdx.x * (int64_t)kGbWarps + warp;
    int head_of[NC];
    float px[NC], acc[NC];
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int col = c * kWarp + lane;
        head_of[c] = col < a.dim ? col / a.head_dim : -1;
        px[c] = (u < a.n && col < a.dim) ? a.p[u * a.ldp + col] : 0.f;
        acc[c] = 0.f;
    }
    float ds[kGbMaxHeads], dtu[kGbMaxHeads], su[kGbMaxHeads];
#pragma unroll
    for (int h = 0; h < kGbMaxHeads; ++h) { ds[h] = 0.f; dtu[h] = 0.f; su[h] = 0.f; }
    if (u < a.n) {
#pragma unroll
        for (int h = 0; h < kGbMaxHeads; ++h) {
            if (h < a.heads) {
                su[h] = a.s[u * a.heads + h];
                dtu[h] = a.stats[u * a.heads + h].w;
            }
        }
        const int64_t beg = a.rowptr[u];
        const int64_t deg = a.rowptr[u + 1] - beg;
        const int64_t total = deg + (a.self_loop ? 1 : 0);
        for (int64_t e = 0; e < total; ++e) {
            const int64_t v = e < deg ? (int64_t)__ldg(a.colidx + beg + e) : u;
            if (a.stats[v * a.heads].y == 0.f) continue;      // dz_v is zero (the same for every lane)
            float g[NC], dalpha[kGbMaxHeads], alpha[kGbMaxHeads];
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int col = c * kWarp + lane;
                g[c] = col < a.dim ? __ldg(a.dz + v * a.lddz + col) : 0.f;
            }
            head_dots<NC>(g, px, head_of, a.heads, dalpha);
#pragma unroll
            for (int h = 0; h < kGbMaxHeads; ++h) {
                alpha[h] = 0.f;
                if (h < a.heads) {
                    const float4 st = a.stats[v * a.heads + h];
                    const float z = su[h] + a.t[v * a.heads + h];
                    alpha[h] = expf((z > 0.f ? z : a.slope * z) - st.x) * st.y;
                    ds[h] = fmaf(alpha[h] * (z > 0.f ? 1.f : a.slope), dalpha[h] - st.z, ds[h]);
                }
            }
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                float al = 0.f;
#pragma unroll
                for (int h = 0; h < kGbMaxHeads; ++h) al = head_of[c] == h ? alpha[h] : al;
                acc[c] = fmaf(al, g[c], acc[c]);
            }
        }
    }
#pragma unroll
    for (int c = 0; c < NC; ++c) {
        const int col = c * kWarp + lane;
        float dsc = 0.f, dtc = 0.f;
#pragma unroll
        for (int h = 0; h < kGbMaxHeads; ++h) { dsc = head_of[c] == h ? ds[h] : dsc; dtc = head_of[c] == h ? dtu[h] : dtc; }
        if (u < a.n && col < a.dim) {
            const float val = acc[c] + dsc * a.a_src[col] + dtc * a.a_dst[col];
            if (a.dp) a.dp[u * a.lddp + col] = val;
            if (a.dp16) a.dp16[u * a.lddp16 + col] = f32_to_bf16(val);
        }
        sm_part[warp][0][c * kWarp + lane] = dsc * px[c];       // (zero beyond the last node / column)
        sm_part[warp][1][c * kWarp + lane] = dtc * px[c];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * a.dim; i += kGbThreads) {
        const int which = i / a.dim, col = i % a.dim;
        float sum = 0.f;
        for (int w = 0; w < kGbWarps; ++w) sum += sm_part[w][which][col];
        a.partial[((int64_t)blockIdx.x * 2 + which) * a.dim + col] = sum;
    }
}

// da_src / da_dst: one block per column sums the per-block partials, each thread its share in index order,
// then the 256 shares in thread order.
__global__ void __launch_bounds__(256) gat_bwd_reduce_kernel(const float* partial, int64_t n_blocks, int32_t dim,
                                                             float* da_src, float* da_dst) {
    __shared__ float share[256];
    const int which = blockIdx.x / dim, col = blockIdx.x % dim;
    float sum = 0.f;
    for (int64_t b = threadIdx.x; b < n_blocks; b += 256) sum += partial[(b * 2 + which) * dim + col];
    share[threadIdx.x] = sum;
    __syncthreads();
    if (threadIdx.x == 0) {
        float total = 0.f;
        for (int t = 0; t < 256; ++t) total += share[t];
        (which ? da_dst : da_src)[col] = total;
    }
}

// ---- rows of up to 64 columns, head width a power of two (the shapes of the paper's RetexoGAT): one lane per
// entry.  A lane fetches its entry's whole row (16-byte loads, all independent) and takes the per-head dot
// products by itself against the warp's own row, which sits in shared memory; nothing is exchanged between
// lanes until the row is done, so a row of several hundred entries is a few dozen trips of 32.
constexpr int kGb64Warps = 4, kGb64Threads = kGb64Warps * kWarp;

template <int HD>
__global__ void __launch_bounds__(kGb64Threads) gat_bwd_dst64_kernel(GatBwdArgs a) {
    __shared__ __align__(16) float g_s[kGb64Warps][64];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t v = blockIdx.x * (int64_t)kGb64Warps + warp;
    if (v >= a.n) return;
    const int nv = a.dim >> 2;                      // float4 pieces per row
    bool any = false;
    for (int c = lane; c < 64; c += kWarp) {
        const float x = c < a.dim ? a.dz[v * a.lddz + c] : 0.f;
        g_s[warp][c] = x;
        any = any || x != 0.f;
    }
    const int64_t beg = a.rowptr[v];
    const int64_t deg = a.rowptr[v + 1] - beg;
    const int64_t total = deg + (a.self_loop ? 1 : 0);
    if (total >= kGbHubEntries) return;             // a hub row: gat_bwd_dst64_hub_kernel's
    if (!__any_sync(0xffffffffu, any) || total == 0) {
        if (lane < a.heads) a.stats[v * a.heads + lane] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    __syncwarp();
    constexpr int NH = 64 / HD;                     // heads at most
    float tv[NH], m[NH], den[NH], csum[NH], a1[NH], a2[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        tv[h] = h < a.heads ? a.t[v * a.heads + h] : 0.f;
        m[h] = -INFINITY; den[h] = 0.f; csum[h] = 0.f; a1[h] = 0.f; a2[h] = 0.f;
    }
    for (int64_t e0 = 0; e0 < total; e0 += kWarp) {
        const bool valid = e0 + lane < total;
        const int64_t u = !valid ? v : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : v);
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            if (h < a.heads) {
                const float z = a.s[u * a.heads + h] + tv[h];
                const float e = valid ? (z > 0.f ? z : a.slope * z) : -INFINITY;
                const float mn = fmaxf(m[h], warp_max(e));
                den[h] = den[h] * expf(m[h] - mn) + warp_sum(valid ? expf(e - mn) : 0.f);
                m[h] = mn;
            }
        }
    }
    for (int64_t e0 = 0; e0 < total; e0 += kWarp) {
        const bool valid = e0 + lane < total;
        const int64_t u = !valid ? v : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : v);
        float dalpha[NH];
#pragma unroll
        for (int h = 0; h < NH; ++h) dalpha[h] = 0.f;
        const float4* row = reinterpret_cast<const float4*>(a.p + u * a.ldp);
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            if (i < nv) {
                const float4 x = valid ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 gg = *reinterpret_cast<const float4*>(&g_s[warp][4 * i]);
                dalpha[(4 * i) / HD] += (x.x * gg.x + x.y * gg.y) + (x.z * gg.z + x.w * gg.w);
            }
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            if (h < a.heads && valid) {
                const float z = a.s[u * a.heads + h] + tv[h];
                const float alpha = expf((z > 0.f ? z : a.slope * z) - m[h]) / den[h];
                const float gp = z > 0.f ? 1.f : a.slope;
                csum[h] = fmaf(alpha, dalpha[h], csum[h]);
                a1[h] = fmaf(alpha * gp, dalpha[h], a1[h]);
                a2[h] = fmaf(alpha, gp, a2[h]);
            }
        }
    }
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        if (h < a.heads) {
            const float c = warp_sum(csum[h]), s1 = warp_sum(a1[h]), s2 = warp_sum(a2[h]);
            if (lane == 0) a.stats[v * a.heads + h] = make_float4(m[h], 1.f / den[h], c, s1 - c * s2);
        }
    }
}

template <int HD>
__global__ void __launch_bounds__(kGb64Threads, 5) gat_bwd_src64_kernel(GatBwdArgs a) {
    __shared__ __align__(16) float p_s[kGb64Warps][64];
    __shared__ float red[kGb64Warps][kWarp][65];
    __shared__ float sm_part[kGb64Warps][2][64];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int64_t u = blockIdx.x * (int64_t)kGb64Warps + warp;
    const int nv = a.dim >> 2;
    constexpr int NH = 64 / HD;
    // A lane's 64 column sums live in its own row of `red` (stride 65: no two lanes of a warp meet in a bank), not
    // in registers: the registers go to the sixteen loads in flight, and more warps fit on an SM.
    float* mine = red[warp][lane];
    float ds[NH], su[NH];
#pragma unroll
    for (int h = 0; h < NH; ++h) { ds[h] = 0.f; su[h] = 0.f; }
    for (int c = lane; c < 64; c += kWarp) p_s[warp][c] = (u < a.n && c < a.dim) ? a.p[u * a.ldp + c] : 0.f;
    __syncwarp();
    bool first = true;                              // nothing stored in `mine` yet
    if (u < a.n) {
#pragma unroll
        for (int h = 0; h < NH; ++h) if (h < a.heads) su[h] = a.s[u * a.heads + h];
        const int64_t beg = a.rowptr[u];
        const int64_t deg = a.rowptr[u + 1] - beg;
        int64_t total = deg + (a.self_loop ? 1 : 0);
        if (total >= kGbHubEntries) {               // a hub row: its sums come from gat_bwd_src64_hub_kernel
            const float* hs = a.hub_sum + (int64_t)a.hub_pos[u] * 72;
#pragma unroll 8
            for (int c = 0; c < 64; ++c) mine[c] = lane == 0 ? hs[c] : 0.f;
            if (lane == 0) {
#pragma unroll
                for (int h = 0; h < NH; ++h) ds[h] = hs[64 + h];
            }
            first = false;
            total = 0;
        }
        for (int64_t e0 = 0; e0 < total; e0 += kWarp) {
            const bool valid = e0 + lane < total;
            const int64_t v = !valid ? u : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : u);
            const bool live = valid && a.stats[v * a.heads].y != 0.f;      // dz_v is zero otherwise
            float4 g[16];
            float dalpha[NH], alpha[NH];
#pragma unroll
            for (int h = 0; h < NH; ++h) { dalpha[h] = 0.f; alpha[h] = 0.f; }
            const float4* row = reinterpret_cast<const float4*>(a.dz + v * a.lddz);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                g[i] = (live && i < nv) ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 pp = *reinterpret_cast<const float4*>(&p_s[warp][4 * i]);
                dalpha[(4 * i) / HD] += (g[i].x * pp.x + g[i].y * pp.y) + (g[i].z * pp.z + g[i].w * pp.w);
            }
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < a.heads && live) {
                    const float4 st = a.stats[v * a.heads + h];
                    const float z = su[h] + a.t[v * a.heads + h];
                    alpha[h] = expf((z > 0.f ? z : a.slope * z) - st.x) * st.y;
                    ds[h] = fmaf(alpha[h] * (z > 0.f ? 1.f : a.slope), dalpha[h] - st.z, ds[h]);
                }
            }
            if (first) {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float al = alpha[(4 * i) / HD];
                    mine[4 * i] = al * g[i].x; mine[4 * i + 1] = al * g[i].y;
                    mine[4 * i + 2] = al * g[i].z; mine[4 * i + 3] = al * g[i].w;
                }
                first = false;
            } else {
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const float al = alpha[(4 * i) / HD];
                    mine[4 * i] = fmaf(al, g[i].x, mine[4 * i]); mine[4 * i + 1] = fmaf(al, g[i].y, mine[4 * i + 1]);
                    mine[4 * i + 2] = fmaf(al, g[i].z, mine[4 * i + 2]); mine[4 * i + 3] = fmaf(al, g[i].w, mine[4 * i + 3]);
                }
            }
        }
    }
    if (first) {
#pragma unroll 8
        for (int c = 0; c < 64; ++c) mine[c] = 0.f;
    }
    // the lanes' partial rows are added in lane order; the lanes' ds in a shuffle tree
#pragma unroll
    for (int h = 0; h < NH; ++h) ds[h] = warp_sum(ds[h]);
    __syncwarp();
    for (int c = lane; c < 64; c += kWarp) {
        float sum = 0.f;
        for (int l = 0; l < kWarp; ++l) sum += red[warp][l][c];
        float dsc = 0.f, dtc = 0.f;
#pragma unroll
        for (int h = 0; h < NH; ++h) if (h == c / HD) dsc = ds[h];
        if (u < a.n && c < a.dim) {
            dtc = a.stats[u * a.heads + c / HD].w;
            const float val = sum + dsc * a.a_src[c] + dtc * a.a_dst[c];
            if (a.dp) a.dp[u * a.lddp + c] = val;
            if (a.dp16) a.dp16[u * a.lddp16 + c] = f32_to_bf16(val);
        } else {
            dsc = 0.f;
        }
        sm_part[warp][0][c] = dsc * p_s[warp][c];
        sm_part[warp][1][c] = dtc * p_s[warp][c];
    }
    __syncthreads();
    for (int i = threadIdx.x; i < 2 * a.dim; i += kGb64Threads) {
        const int which = i / a.dim, col = i % a.dim;
        float sum = 0.f;
        for (int w = 0; w < kGb64Warps; ++w) sum += sm_part[w][which][col];
        a.partial[((int64_t)blockIdx.x * 2 + which) * a.dim + col] = sum;
    }
}

// ---- hub rows: one block per listed row, its warps taking the trips w, w + W, ...; per-warp results are merged in
// warp order, so the bits depend neither on timing nor on the list's order.
constexpr int kGbHubWarps = 8, kGbHubThreads = kGbHubWarps * kWarp;

template <int HD>
__global__ void __launch_bounds__(kGbHubThreads) gat_bwd_dst64_hub_kernel(GatBwdArgs a) {
    constexpr int NH = 64 / HD;
    __shared__ __align__(16) float g_s[64];
    __shared__ float st_m[kGbHubWarps][NH], st_den[kGbHubWarps][NH], part[kGbHubWarps][NH][3];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nv = a.dim >> 2;
    const int32_t count = *a.hub_count;
    for (int32_t item = blockIdx.x; item < count; item += gridDim.x) {
        const int64_t v = a.hub_list[item];
        __syncthreads();                                 // the previous row's shared values are done with
        bool any = false;
        if (threadIdx.x < 64) {
            const float x = (int)threadIdx.x < a.dim ? a.dz[v * a.lddz + threadIdx.x] : 0.f;
            g_s[threadIdx.x] = x;
            any = x != 0.f;
        }
        if (!__syncthreads_or(any)) {
            if ((int)threadIdx.x < a.heads) a.stats[v * a.heads + threadIdx.x] = make_float4(0.f, 0.f, 0.f, 0.f);
            continue;
        }
        const int64_t beg = a.rowptr[v];
        const int64_t deg = a.rowptr[v + 1] - beg;
        const int64_t total = deg + (a.self_loop ? 1 : 0);
        float tv[NH], m[NH], den[NH], csum[NH], a1[NH], a2[NH];
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            tv[h] = h < a.heads ? a.t[v * a.heads + h] : 0.f;
            m[h] = -INFINITY; den[h] = 0.f; csum[h] = 0.f; a1[h] = 0.f; a2[h] = 0.f;
        }
        for (int64_t e0 = (int64_t)warp * kWarp; e0 < total; e0 += kGbHubThreads) {
            const bool valid = e0 + lane < total;
            const int64_t u = !valid ? v : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : v);
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < a.heads) {
                    const float z = a.s[u * a.heads + h] + tv[h];
                    const float e = valid ? (z > 0.f ? z : a.slope * z) : -INFINITY;
                    const float mn = fmaxf(m[h], warp_max(e));
                    den[h] = den[h] * expf(m[h] - mn) + warp_sum(valid ? expf(e - mn) : 0.f);
                    m[h] = mn;
                }
            }
        }
        if (lane == 0) {
#pragma unroll
            for (int h = 0; h < NH; ++h) { st_m[warp][h] = m[h]; st_den[warp][h] = den[h]; }
        }
        __syncthreads();
#pragma unroll
        for (int h = 0; h < NH; ++h) {                   // every thread merges the warps' states in warp order
            float mm = -INFINITY, dd = 0.f;
            for (int w = 0; w < kGbHubWarps; ++w) mm = fmaxf(mm, st_m[w][h]);
            for (int w = 0; w < kGbHubWarps; ++w)
                if (st_den[w][h] > 0.f) dd += st_den[w][h] * expf(st_m[w][h] - mm);
            m[h] = mm; den[h] = dd;
        }
        for (int64_t e0 = (int64_t)warp * kWarp; e0 < total; e0 += kGbHubThreads) {
            const bool valid = e0 + lane < total;
            const int64_t u = !valid ? v : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : v);
            float dalpha[NH];
#pragma unroll
            for (int h = 0; h < NH; ++h) dalpha[h] = 0.f;
            const float4* row = reinterpret_cast<const float4*>(a.p + u * a.ldp);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                if (i < nv) {
                    const float4 x = valid ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                    const float4 gg = *reinterpret_cast<const float4*>(&g_s[4 * i]);
                    dalpha[(4 * i) / HD] += (x.x * gg.x + x.y * gg.y) + (x.z * gg.z + x.w * gg.w);
                }
            }
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < a.heads && valid) {
                    const float z = a.s[u * a.heads + h] + tv[h];
                    const float alpha = expf((z > 0.f ? z : a.slope * z) - m[h]) / den[h];
                    const float gp = z > 0.f ? 1.f : a.slope;
                    csum[h] = fmaf(alpha, dalpha[h], csum[h]);
                    a1[h] = fmaf(alpha * gp, dalpha[h], a1[h]);
                    a2[h] = fmaf(alpha, gp, a2[h]);
                }
            }
        }
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const float c = warp_sum(csum[h]), s1 = warp_sum(a1[h]), s2 = warp_sum(a2[h]);
            if (lane == 0) { part[warp][h][0] = c; part[warp][h][1] = s1; part[warp][h][2] = s2; }
        }
        __syncthreads();
        if ((int)threadIdx.x < a.heads && (int)threadIdx.x < NH) {
            const int h = threadIdx.x;
            float c = 0.f, s1 = 0.f, s2 = 0.f, mm = -INFINITY, dd = 0.f;
            for (int w = 0; w < kGbHubWarps; ++w) { c += part[w][h][0]; s1 += part[w][h][1]; s2 += part[w][h][2]; }
            for (int w = 0; w < kGbHubWarps; ++w) mm = fmaxf(mm, st_m[w][h]);
            for (int w = 0; w < kGbHubWarps; ++w)
                if (st_den[w][h] > 0.f) dd += st_den[w][h] * expf(st_m[w][h] - mm);
            a.stats[v * a.heads + h] = make_float4(mm, 1.f / dd, c, s1 - c * s2);
        }
    }
}

// The source pass of a hub row u: the entry sums only (sum_v alpha_uv dz_v per column and ds_u per head); the row's
// own epilogue (dp_u, the parameter-gradient partials) stays with gat_bwd_src64_kernel, which picks the sums up.
template <int HD>
__global__ void __launch_bounds__(kGb64Threads) gat_bwd_src64_hub_kernel(GatBwdArgs a) {
    constexpr int NH = 64 / HD;
    __shared__ __align__(16) float p_s[64];
    __shared__ float red[kGb64Warps][kWarp][65];
    __shared__ float rows[kGb64Warps][64], dsw[kGb64Warps][NH];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int nv = a.dim >> 2;
    const int32_t count = *a.hub_count;
    for (int32_t item = blockIdx.x; item < count; item += gridDim.x) {
        const int64_t u = a.hub_list[item];
        __syncthreads();
        if (threadIdx.x < 64) p_s[threadIdx.x] = (int)threadIdx.x < a.dim ? a.p[u * a.ldp + threadIdx.x] : 0.f;
        __syncthreads();
        float acc[64], ds[NH], su[NH];
#pragma unroll
        for (int c = 0; c < 64; ++c) acc[c] = 0.f;
#pragma unroll
        for (int h = 0; h < NH; ++h) { ds[h] = 0.f; su[h] = h < a.heads ? a.s[u * a.heads + h] : 0.f; }
        const int64_t beg = a.rowptr[u];
        const int64_t deg = a.rowptr[u + 1] - beg;
        const int64_t total = deg + (a.self_loop ? 1 : 0);
        for (int64_t e0 = (int64_t)warp * kWarp; e0 < total; e0 += kGb64Threads) {
            const bool valid = e0 + lane < total;
            const int64_t v = !valid ? u : (e0 + lane < deg ? (int64_t)__ldg(a.colidx + beg + e0 + lane) : u);
            const bool live = valid && a.stats[v * a.heads].y != 0.f;      // dz_v is zero otherwise
            float4 g[16];
            float dalpha[NH], alpha[NH];
#pragma unroll
            for (int h = 0; h < NH; ++h) { dalpha[h] = 0.f; alpha[h] = 0.f; }
            const float4* row = reinterpret_cast<const float4*>(a.dz + v * a.lddz);
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                g[i] = (live && i < nv) ? __ldg(row + i) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 pp = *reinterpret_cast<const float4*>(&p_s[4 * i]);
                dalpha[(4 * i) / HD] += (g[i].x * pp.x + g[i].y * pp.y) + (g[i].z * pp.z + g[i].w * pp.w);
            }
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                if (h < a.heads && live) {
                    const float4 st = a.stats[v * a.heads + h];
                    const float z = su[h] + a.t[v * a.heads + h];
                    alpha[h] = expf((z > 0.f ? z : a.slope * z) - st.x) * st.y;
                    ds[h] = fmaf(alpha[h] * (z > 0.f ? 1.f : a.slope), dalpha[h] - st.z, ds[h]);
                }
            }
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const float al = alpha[(4 * i) / HD];
                acc[4 * i] = fmaf(al, g[i].x, acc[4 * i]);
                acc[4 * i + 1] = fmaf(al, g[i].y, acc[4 * i + 1]);
                acc[4 * i + 2] = fmaf(al, g[i].z, acc[4 * i + 2]);
                acc[4 * i + 3] = fmaf(al, g[i].w, acc[4 * i + 3]);
            }
        }
        // lanes in lane order, then warps in warp order
#pragma unroll
        for (int c = 0; c < 64; ++c) red[warp][lane][c] = acc[c];
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const float d = warp_sum(ds[h]);
            if (lane == 0) dsw[warp][h] = d;
        }
        __syncwarp();
        for (int c = lane; c < 64; c += kWarp) {
            float sum = 0.f;
            for (int l = 0; l < kWarp; ++l) sum += red[warp][l][c];
            rows[warp][c] = sum;
        }
        __syncthreads();
        float* hs = a.hub_sum + (int64_t)item * 72;
        if (threadIdx.x < 64) {
            float sum = 0.f;
            for (int w = 0; w < kGb64Warps; ++w) sum += rows[w][threadIdx.x];
            hs[threadIdx.x] = sum;
        } else if ((int)threadIdx.x - 64 < NH) {
            const int h = threadIdx.x - 64;
            float sum = 0.f;
            for (int w = 0; w < kGb64Warps; ++w) sum += dsw[w][h];
            hs[64 + h] = sum;
        }
    }
}

template <int HD>
static int launch_bwd64(const GatBwdArgs& a, float* da_src, float* da_dst, cudaStream_t st) {
    const unsigned blocks = (unsigned)((a.n + kGb64Warps - 1) / kGb64Warps);
    gat_bwd_dst64_kernel<HD><<<blocks, kGb64Threads, 0, st>>>(a);
    gat_bwd_dst64_hub_kernel<HD><<<kGbHubBlocks, kGbHubThreads, 0, st>>>(a);
    gat_bwd_src64_hub_kernel<HD><<<kGbHubBlocks, kGb64Threads, 0, st>>>(a);
    gat_bwd_src64_kernel<HD><<<blocks, kGb64Threads, 0, st>>>(a);
    gat_bwd_reduce_kernel<<<(unsigned)(2 * a.dim), 256, 0, st>>>(a.partial, blocks, a.dim, da_src, da_dst);
    return launch_status();
}

template <int NC>
static int launch_bwd(const GatBwdArgs& a, unsigned blocks, float* da_src, float* da_dst, cudaStream_t st) {
    gat_bwd_dst_kernel<NC><<<blocks, kGbThreads, 0, st>>>(a);
    gat_bwd_src_kernel<NC><<<blocks, kGbThreads, 0, st>>>(a);
    gat_bwd_reduce_kernel<<<(unsigned)(2 * a.dim), 256, 0, st>>>(a.partial, blocks, a.dim, da_src, da_dst);
    return launch_status();
}

}  // namespace retexo

using namespace retexo;

// rows of kGbHubEntries entries or more a graph can hold at most (with the self loop counted as an entry)
static inline int64_t max_hub_rows(int64_t n_nodes, int64_t n_edges) { return (n_edges + n_nodes) / kGbHubEntries + 1; }

extern "C" size_t retexo_gat_backward_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t heads, int32_t dim) {
    if (n_nodes < 0 || n_edges < 0 || heads <= 0 || dim <= 0) return 0;
    Sizer s;
    s.take<float>((size_t)n_nodes * heads);
    s.take<float>((size_t)n_nodes * heads);
    s.take<float4>((size_t)n_nodes * heads);
    s.take<float>((size_t)((n_nodes + kGb64Warps - 1) / kGb64Warps + 1) * 2 * (size_t)dim);
    s.take<int32_t>(64);
    s.take<int32_t>((size_t)max_hub_rows(n_nodes, n_edges));
    s.take<int32_t>((size_t)n_nodes);
    s.take<float>((size_t)max_hub_rows(n_nodes, n_edges) * 72);
    return s.off + kAlign;
}

extern "C" int retexo_gat_backward(const retexo_csr* g, const float* p, int64_t ldp, const retexo_gat_params* gat,
                                   const float* dz, int64_t lddz, float* dp, int64_t lddp, void* dp_bf16,
                                   int64_t lddp_bf16, float* da_src, float* da_dst, void* workspace,
                                   size_t workspace_bytes, void* stream) {
    if (!g || g->n_nodes < 0 || g->n_edges < 0 || g->n_nodes > INT32_MAX) return RETEXO_ERR_INVALID_ARG;
    if (!gat || gat->heads <= 0 || gat->head_dim <= 0 || !gat->a_src || !gat->a_dst) return RETEXO_ERR_INVALID_ARG;
    const int32_t dim = gat->heads * gat->head_dim;
    if (gat->heads > kGbMaxHeads || dim > 256) return RETEXO_ERR_UNSUPPORTED;
    if (!da_src || !da_dst || (!dp && !dp_bf16)) return RETEXO_ERR_INVALID_ARG;
    if (ldp < dim || lddz < dim || (dp && lddp < dim) || (dp_bf16 && lddp_bf16 < dim)) return RETEXO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (g->n_nodes == 0) {
        RETEXO_CUDA_TRY(cudaMemsetAsync(da_src, 0, sizeof(float) * dim, st));
        RETEXO_CUDA_TRY(cudaMemsetAsync(da_dst, 0, sizeof(float) * dim, st));
        return RETEXO_OK;
    }
    if (!g->rowptr || !p || !dz || (g->n_edges > 0 && !g->colidx)) return RETEXO_ERR_INVALID_ARG;
    const size_t need = retexo_gat_backward_workspace_size(g->n_nodes, g->n_edges, gat->heads, dim);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    const int64_t n = g->n_nodes;
    Arena ws(workspace, workspace_bytes);
    GatBwdArgs a;
    a.n = n; a.rowptr = g->rowptr; a.colidx = g->colidx; a.p = p; a.ldp = ldp;
    a.heads = gat->heads; a.head_dim = gat->head_dim; a.dim = dim;
    a.a_src = gat->a_src; a.a_dst = gat->a_dst; a.slope = gat->negative_slope; a.self_loop = gat->add_self_loop ? 1 : 0;
    a.dz = dz; a.lddz = lddz;
    a.s = ws.take<float>((size_t)n * gat->heads);
    a.t = ws.take<float>((size_t)n * gat->heads);
    a.stats = ws.take<float4>((size_t)n * gat->heads);
    const unsigned blocks = (unsigned)((n + kGbWarps - 1) / kGbWarps);
    a.partial = ws.take<float>((size_t)((n + kGb64Warps - 1) / kGb64Warps + 1) * 2 * (size_t)dim);
    a.dp = dp; a.lddp = lddp; a.dp16 = static_cast<__nv_bfloat16*>(dp_bf16); a.lddp16 = lddp_bf16;
    int32_t* hub_count = ws.take<int32_t>(64);
    int32_t* hub_list = ws.take<int32_t>((size_t)max_hub_rows(n, g->n_edges));
    int32_t* hub_pos = ws.take<int32_t>((size_t)n);
    float* hub_sum = ws.take<float>((size_t)max_hub_rows(n, g->n_edges) * 72);
    // rows of up to 64 columns in whole 16-byte pieces, head width 8 / 16 / 32 / 64: one lane per entry, hub rows by blocks
    const int hdw = gat->head_dim;
    const bool lane_per_entry = dim <= 64 && dim % 4 == 0 && ldp % 4 == 0 && lddz % 4 == 0 && aligned_to(p, 16) && aligned_to(dz, 16) &&
                                (hdw == 8 || hdw == 16 || hdw == 32 || hdw == 64);
    a.hub_count = nullptr; a.hub_list = nullptr; a.hub_pos = nullptr; a.hub_sum = nullptr;
    if (lane_per_entry) {
        a.hub_count = hub_count; a.hub_list = hub_list; a.hub_pos = hub_pos; a.hub_sum = hub_sum;
        RETEXO_CUDA_TRY(cudaMemsetAsync(hub_count, 0, sizeof(int32_t), st));
    }
    gat_bwd_scores_kernel<<<blocks, kGbThreads, 0, st>>>(a);
    if (lane_per_entry) {
        if (hdw == 8) return launch_bwd64<8>(a, da_src, da_dst, st);
        if (hdw == 16) return launch_bwd64<16>(a, da_src, da_dst, st);
        if (hdw == 32) return launch_bwd64<32>(a, da_src, da_dst, st);
        return launch_bwd64<64>(a, da_src, da_dst, st);
    }
    const int nc = (dim + kWarp - 1) / kWarp;
    if (nc <= 1) return launch_bwd<1>(a, blocks, da_src, da_dst, st);
    if (nc <= 2) return launch_bwd<2>(a, blocks, da_src, da_dst, st);
    if (nc <= 4) return launch_bwd<4>(a, blocks, da_src, da_dst, st);
    return launch_bwd<8>(a, blocks, da_src, da_dst, st);
}
