// Exact count of the boundary-node messages (and bytes) one lazy
// message-passing round sends across a node partition (Section 2.1,
// Appendix A.1), plus the CSR validator.  Integer work only; all tallies use
// integer atomics, whose result does not depend on the order they land in.
#include <mutex>

#include "common.cuh"

namespace retexo {

constexpr int kCntThreads = 256;
constexpr int kCntWarps = kCntThreads / kWarp;
constexpr int kBitmapParts = 8192;                  // per-warp shared bitmap covers this many partitions
constexpr int kBitmapWords = kBitmapParts / 32;
constexpr int kHashSlots = 1024;                    // per-warp shared hash set
constexpr int kHashMaxDeg = 512;                    // rows up to this length use it
constexpr int kHashWarps = 4;
constexpr int kBigRowBlocks = 148;                  // blocks (and global bitmaps) of the long-row pass
constexpr int kBlockRowDeg = 4096;                  // rows longer than this go to the long-row pass at once
constexpr int32_t kCrossCounted = INT32_MIN;        // list flag: the row's cross edges are already tallied

struct CountArgs {
    int64_t n;
    const int64_t* rowptr;
    const int32_t* colidx;
    const int32_t* part;
    int32_t n_parts;
    unsigned long long* cross_edges;      // accumulators (zeroed before launch)
    unsigned long long* pairs;
    unsigned long long* send;             // may be null
    unsigned long long* recv;             // may be null
    int32_t* big_list;                    // rows deferred to the long-row pass
    int32_t* big_count;
    uint32_t* big_bitmaps;                // kBigRowBlocks x words_per_bitmap, all zero between rows
    int64_t words_per_bitmap;
    unsigned long long* bad_part;         // set to 1 if a partition id is out of range
    unsigned long long* next_row;         // work counter (zeroed before launch): rows are handed out in batches
    int32_t row_batch;                    // rows per draw from the counter
};

// Rows are drawn from one counter, row_batch at a time, so that a power-law degree distribution
// does not leave warps with a fixed share of hub rows behind the others.  Returns the first row
// of this warp's next batch (>= n when the rows have run out).
__device__ __forceinline__ int64_t next_rows(const CountArgs& a, int lane) {
    unsigned long long u = 0;
    if (lane == 0) u = atomicAdd(a.next_row, (unsigned long long)a.row_batch);
    return (int64_t)__shfl_sync(0xffffffffu, u, 0);
}

// Partition id of node x; an id outside [0, n_parts) raises the flag and is
// replaced by 0 so that every table access stays in bounds.
__device__ __forceinline__ int32_t part_of(const CountArgs& a, int64_t x) {
    const int32_t p = __ldg(a.part + x);
    if ((uint32_t)p >= (uint32_t)a.n_parts) {
        *a.bad_part = 1ull;
        return 0;
    }
    return p;
}

__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Partition count <= kBitmapParts: one warp per row, the set of destination
// partitions already seen is a bitmap in shared memory.
__global__ void __launch_bounds__(kCntThreads) count_bitmap_kernel(CountArgs a) {
    __shared__ uint32_t bm[kCntWarps][kBitmapWords];
    // per-partition receive tally of this block (only when asked for: n_parts words of dynamic shared
    // memory), added to the global one once at the end: one global atomic per message would serialise
    // on the few hundred addresses
    extern __shared__ uint32_t recv_block[];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = lane; i < kBitmapWords; i += kWarp) bm[warp][i] = 0u;
    if (a.recv) {
        for (int i = threadIdx.x; i < a.n_parts; i += kCntThreads) recv_block[i] = 0u;
        __syncthreads();
    }
    __syncwarp();
    unsigned long long my_cross = 0, my_pairs = 0;
    for (int64_t u0 = next_rows(a, lane); u0 < a.n; u0 = next_rows(a, lane))
    for (int64_t u = u0; u < min(a.n, u0 + a.row_batch); ++u) {
        const int64_t beg = a.rowptr[u], end = a.rowptr[u + 1];
        if (beg == end) continue;
        const int32_t pu = part_of(a, u);
        unsigned row_new = 0;
        // four chunks of 32 entries per trip: the index loads, then the partition-id gathers, are
        // issued together, so a trip costs two memory latencies instead of eight
        for (int64_t e0 = beg; e0 < end; e0 += 4 * kWarp) {
            int32_t nb[4], pv[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int64_t e = e0 + t * kWarp + lane;
                nb[t] = e < end ? __ldg(a.colidx + e) : -1;
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) pv[t] = nb[t] >= 0 ? part_of(a, nb[t]) : pu;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const bool cross = pv[t] != pu;
                bool is_new = false;
                if (cross) {
                    const uint32_t bit = 1u << (pv[t] & 31);
                    const uint32_t old = atomicOr(&bm[warp][pv[t] >> 5], bit);
                    is_new = !(old & bit);
                    if (is_new && a.recv) atomicAdd(&recv_block[pv[t]], 1u);
                }
                my_cross += cross ? 1ull : 0ull;
                row_new += __popc(__ballot_sync(0xffffffffu, is_new));
            }
        }
        __syncwarp();
        // clear the touched words again
        if (end - beg >= kBitmapWords) {
            for (int i = lane; i < kBitmapWords; i += kWarp) bm[warp][i] = 0u;
        } else {
            for (int64_t e = beg + lane; e < end; e += kWarp) {
                const int32_t pv = part_of(a, __ldg(a.colidx + e));
                bm[warp][pv >> 5] = 0u;
            }
        }
        __syncwarp();
        if (lane == 0) {
            my_pairs += row_new;
            if (a.send && row_new) atomicAdd(a.send + pu, (unsigned long long)row_new);
        }
    }
    my_cross = warp_sum_u64(my_cross);
    if (lane == 0) {
        if (my_cross) atomicAdd(a.cross_edges, my_cross);
        if (my_pairs) atomicAdd(a.pairs, my_pairs);
    }
    if (a.recv) {
        __syncthreads();
        for (int i = threadIdx.x; i < a.n_parts; i += kCntThreads)
            if (recv_block[i]) atomicAdd(a.recv + i, (unsigned long long)recv_block[i]);
    }
}

__device__ __forceinline__ uint32_t hash32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du; x ^= x >> 15; x *= 0x846ca68bu; x ^= x >> 16;
    return x;
}

// Any partition count: one warp per row.
//  1. If the destination partitions come in non-decreasing order along the row
//     (true for node-level and for range partitions, the columns being
//     sorted), equal ones are adjacent and a compare with the previous entry
//     finds the distinct ones.
//  2. Otherwise rows of up to kHashMaxDeg entries use a hash set in shared
//     memory; longer ones are listed for the long-row pass.
__global__ void __launch_bounds__(kHashWarps * kWarp) count_general_kernel(CountArgs a) {
    __shared__ int32_t tab[kHashWarps][kHashSlots];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int i = lane; i < kHashSlots; i += kWarp) tab[warp][i] = -1;
    __syncwarp();
    unsigned long long my_cross = 0, my_pairs = 0;
    for (int64_t u0 = next_rows(a, lane); u0 < a.n; u0 = next_rows(a, lane))
    for (int64_t u = u0; u < min(a.n, u0 + a.row_batch); ++u) {
        const int64_t beg = a.rowptr[u], end = a.rowptr[u + 1];
        if (beg == end) continue;
        const int32_t pu = part_of(a, u);
        if (end - beg > kBlockRowDeg) {     // a whole block takes this row (a single warp would be a long tail)
            if (lane == 0) {
                const int32_t slot = atomicAdd(a.big_count, 1);
                a.big_list[slot] = (int32_t)u;
            }
            continue;
        }
        // pass 1: order check + adjacent-distinct count, four chunks of 32 entries per trip
        bool mono = true;
        unsigned n_cross = 0, n_new = 0;
        int32_t carry = -1;
        for (int64_t e0 = beg; e0 < end; e0 += 4 * kWarp) {
            int32_t nb[4], pvs[4];
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int64_t e = e0 + t * kWarp + lane;
                nb[t] = e < end ? __ldg(a.colidx + e) : -1;
            }
#pragma unroll
            for (int t = 0; t < 4; ++t) pvs[t] = nb[t] >= 0 ? part_of(a, nb[t]) : INT32_MAX;
#pragma unroll
            for (int t = 0; t < 4; ++t) {
                const int32_t pv = pvs[t];
                const bool valid = nb[t] >= 0;
                int32_t prev = __shfl_up_sync(0xffffffffu, pv, 1);
                if (lane == 0) prev = carry;
                mono = mono && __all_sync(0xffffffffu, pv >= prev);
                const bool cross = valid && pv != pu;
                n_cross += __popc(__ballot_sync(0xffffffffu, cross));
                n_new += __popc(__ballot_sync(0xffffffffu, cross && pv != prev));
                carry = __shfl_sync(0xffffffffu, pv, kWarp - 1);
            }
        }
        if (lane == 0) my_cross += n_cross;
        if (n_cross == 0) continue;
        if (mono) {
            if (a.recv) {
                carry = -1;
                for (int64_t e0 = beg; e0 < end; e0 += kWarp) {
                    const int64_t e = e0 + lane;
                    const bool valid = e < end;
                    const int32_t pv = valid ? part_of(a, __ldg(a.colidx + e)) : INT32_MAX;
                    int32_t prev = __shfl_up_sync(0xffffffffu, pv, 1);
                    if (lane == 0) prev = carry;
                    if (valid && pv != pu && pv != prev) atomicAdd(a.recv + pv, 1ull);
                    carry = __shfl_sync(0xffffffffu, pv, kWarp - 1);
                }
            }
        } else if (end - beg <= kHashMaxDeg) {
            n_new = 0;
            for (int64_t e0 = beg; e0 < end; e0 += kWarp) {
                const int64_t e = e0 + lane;
                bool is_new = false;
                if (e < end) {
                    const int32_t pv = part_of(a, __ldg(a.colidx + e));
                    if (pv != pu) {
                        uint32_t h = hash32((uint32_t)pv) & (kHashSlots - 1);
                        for (int probe = 0; probe < kHashSlots; ++probe) {      // table is never full
                            const int32_t old = atomicCAS(&tab[warp][h], -1, pv);
                            if (old == -1) { is_new = true; break; }
                            if (old == pv) break;
                            h = (h + 1) & (kHashSlots - 1);
                        }
                        if (is_new && a.recv) atomicAdd(a.recv + pv, 1ull);
                    }
                }
                n_new += __popc(__ballot_sync(0xffffffffu, is_new));
            }
            __syncwarp();
            for (int i = lane; i < kHashSlots; i += kWarp) tab[warp][i] = -1;
            __syncwarp();
        } else {
            if (lane == 0) {
                const int32_t slot = atomicAdd(a.big_count, 1);
                a.big_list[slot] = (int32_t)u | kCrossCounted;
            }
            continue;      // pairs of this row are counted by the long-row pass
        }
        if (lane == 0) {
            my_pairs += n_new;
            if (a.send && n_new) atomicAdd(a.send + pu, (unsigned long long)n_new);
        }
    }
    if (lane == 0) {
        if (my_cross) atomicAdd(a.cross_edges, my_cross);
        if (my_pairs) atomicAdd(a.pairs, my_pairs);
    }
}

// Long unordered rows with many partitions: one block per row, the seen-set is
// a bitmap in global memory owned by the block (all zero on entry and exit).
__global__ void __launch_bounds__(kCntThreads) count_big_rows_kernel(CountArgs a) {
    __shared__ unsigned int block_new, block_cross;
    uint32_t* bm = a.big_bitmaps + (int64_t)blockIdx.x * a.words_per_bitmap;
    const int n_big = *a.big_count;
    for (int r = blockIdx.x; r < n_big; r += gridDim.x) {
        const int32_t entry = a.big_list[r];
        const bool cross_counted = (entry & kCrossCounted) != 0;      // a warp already found it unordered
        const int64_t u = entry & INT32_MAX;
        const int64_t beg = a.rowptr[u], end = a.rowptr[u + 1];
        const int32_t pu = part_of(a, u);
        if (threadIdx.x == 0) { block_new = 0; block_cross = 0; }
        __syncthreads();
        if (!cross_counted) {
            // ordered rows (node-level or range partitions): compare every entry with its predecessor
            bool mono = true;
            unsigned n_cross = 0, n_adj = 0;
            for (int64_t e0 = beg + threadIdx.x; e0 < end; e0 += 4 * kCntThreads) {
                int32_t nb[4], pb[4], pv[4], pp[4];
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    const int64_t e = e0 + (int64_t)t * kCntThreads;
                    nb[t] = e < end ? __ldg(a.colidx + e) : -1;
                    pb[t] = (e < end && e > beg) ? __ldg(a.colidx + e - 1) : -1;
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    pv[t] = nb[t] >= 0 ? part_of(a, nb[t]) : INT32_MAX;
                    pp[t] = pb[t] >= 0 ? part_of(a, pb[t]) : -1;
                }
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    if (nb[t] < 0) continue;
                    mono = mono && pv[t] >= pp[t];
                    if (pv[t] != pu) { ++n_cross; if (pv[t] != pp[t]) ++n_adj; }
                }
            }
            if (n_cross) atomicAdd(&block_cross, n_cross);
            const int all_mono = __syncthreads_and(mono ? 1 : 0);
            if (threadIdx.x == 0 && block_cross) atomicAdd(a.cross_edges, (unsigned long long)block_cross);
            if (all_mono) {
                if (n_adj) atomicAdd(&block_new, n_adj);
                if (a.recv) {
                    for (int64_t e = beg + threadIdx.x; e < end; e += kCntThreads) {
                        const int32_t pv = part_of(a, __ldg(a.colidx + e));
                        const int32_t pp = e > beg ? part_of(a, __ldg(a.colidx + e - 1)) : -1;
                        if (pv != pu && pv != pp) atomicAdd(a.recv + pv, 1ull);
                    }
                }
                __syncthreads();
                if (threadIdx.x == 0 && block_new) {
                    atomicAdd(a.pairs, (unsigned long long)block_new);
                    if (a.send) atomicAdd(a.send + pu, (unsigned long long)block_new);
                }
                __syncthreads();
                continue;
            }
        }
        unsigned mine = 0;
        for (int64_t e = beg + threadIdx.x; e < end; e += kCntThreads) {
            const int32_t pv = part_of(a, __ldg(a.colidx + e));
            if (pv == pu) continue;
            const uint32_t bit = 1u << (pv & 31);
            const uint32_t old = atomicOr(bm + (pv >> 5), bit);
            if (!(old & bit)) {
                ++mine;
                if (a.recv) atomicAdd(a.recv + pv, 1ull);
            }
        }
        if (mine) atomicAdd(&block_new, mine);
        __syncthreads();
        for (int64_t e = beg + threadIdx.x; e < end; e += kCntThreads) {
            const int32_t pv = part_of(a, __ldg(a.colidx + e));
            bm[pv >> 5] = 0u;
        }
        __syncthreads();
        if (threadIdx.x == 0 && block_new) {
            atomicAdd(a.pairs, (unsigned long long)block_new);
            if (a.send) atomicAdd(a.send + pu, (unsigned long long)block_new);
        }
        __syncthreads();
    }
}

// The widths of the K rounds travel in the kernel's arguments (K <= 64), so the call makes no copy from the
// caller's host array that could outlive it.
struct RoundDimsArg { int32_t d[64]; };

__global__ void count_finalize_kernel(const unsigned long long* cross_acc, const unsigned long long* pairs_acc,
                                      const unsigned long long* bad_part, int32_t K, const RoundDimsArg dims, int32_t elem_bytes,
                                      uint64_t* cross_edges, uint64_t* boundary_pairs,
                                      uint64_t* bytes_per_round, uint64_t* bytes_total) {
    if (blockIdx.x != 0 || threadIdx.x != 0) return;
    if (*bad_part) {          // a partition id was out of range: poison the results
        if (cross_edges) *cross_edges = UINT64_MAX;
        if (boundary_pairs) *boundary_pairs = UINT64_MAX;
        for (int m = 0; m < K; ++m) if (bytes_per_round) bytes_per_round[m] = UINT64_MAX;
        if (bytes_total) *bytes_total = UINT64_MAX;
        return;
    }
    const uint64_t bp = *pairs_acc;
    if (cross_edges) *cross_edges = *cross_acc;
    if (boundary_pairs) *boundary_pairs = bp;
    uint64_t tot = 0;
    for (int m = 0; m < K; ++m) {
        const uint64_t b = bp * (uint64_t)dims.d[m] * (uint64_t)elem_bytes;
        if (bytes_per_round) bytes_per_round[m] = b;
        tot += b;
    }
    if (bytes_total) *bytes_total = tot;
}

// ---------------------------------------------------------------- validator
__global__ void validate_csr_kernel(int64_t n, int64_t n_edges, const int64_t* rowptr, const int32_t* colidx,
                                    unsigned long long* bad, long long* where) {
    const int64_t v = blockIdx.x * (int64_t)blockDim.x + threadIdx.x;
    if (v > n) return;
    bool wrong = false;
    if (v == 0 && rowptr[0] != 0) wrong = true;
    if (v == n) {
        if (rowptr[n] != n_edges) wrong = true;
    } else {
        const int64_t beg = rowptr[v], end = rowptr[v + 1];
        if (beg > end || beg < 0 || end > n_edges) wrong = true;
        else {
            int64_t prev = -1;
            for (int64_t e = beg; e < end; ++e) {
                const int64_t c = colidx[e];
                if (c < 0 || c >= n || c == v || c <= prev) { wrong = true; break; }
                prev = c;
            }
        }
    }
    if (wrong) {
        atomicAdd(bad, 1ull);
        atomicMax(where, (long long)v);
    }
}

}  // namespace retexo

using namespace retexo;

extern "C" int retexo_validate_csr(const retexo_csr* g, int64_t* status_out, void* stream) {
    if (!g || !status_out || g->n_nodes < 0 || g->n_edges < 0) return RETEXO_ERR_INVALID_ARG;
    if (!g->rowptr || (g->n_edges > 0 && !g->colidx)) return RETEXO_ERR_INVALID_ARG;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const long long init[2] = {0, -1};
    RETEXO_CUDA_TRY(cudaMemcpyAsync(status_out, init, sizeof(init), cudaMemcpyHostToDevice, st));
    const int64_t threads = g->n_nodes + 1;
    validate_csr_kernel<<<(unsigned)((threads + 255) / 256), 256, 0, st>>>(
        g->n_nodes, g->n_edges, g->rowptr, g->colidx,
        reinterpret_cast<unsigned long long*>(status_out), reinterpret_cast<long long*>(status_out + 1));
    return launch_status();
}

extern "C" size_t retexo_cross_partition_workspace_size(int64_t n_nodes, int64_t n_edges, int32_t n_parts) {
    (void)n_edges;
    if (n_nodes < 0 || n_parts <= 0) return 0;
    Sizer s;
    s.take<unsigned long long>(32);                       // accumulators
    if (n_parts > kBitmapParts) {
        s.take<int32_t>((size_t)n_nodes);                 // long-row list
        s.take<int32_t>(64);
        s.take<uint32_t>((size_t)kBigRowBlocks * (size_t)((n_parts + 31) / 32));
    }
    return s.off + kAlign;
}

extern "C" int retexo_cross_partition_bytes(const retexo_csr* g, const int32_t* part, int32_t n_parts,
                                            int32_t K, const int32_t* dims, int32_t elem_bytes,
                                            uint64_t* cross_edges, uint64_t* boundary_pairs,
                                            uint64_t* bytes_per_round, uint64_t* bytes_total,
                                            uint64_t* send_per_part, uint64_t* recv_per_part,
                                            void* workspace, size_t workspace_bytes, void* stream) {
    if (!g || g->n_nodes < 0 || g->n_edges < 0 || g->n_nodes > INT32_MAX) return RETEXO_ERR_INVALID_ARG;
    if (n_parts <= 0 || K < 0 || K > 64 || elem_bytes <= 0 || (K > 0 && !dims)) return RETEXO_ERR_INVALID_ARG;
    if (g->n_nodes > 0 && (!g->rowptr || !part || (g->n_edges > 0 && !g->colidx))) return RETEXO_ERR_INVALID_ARG;
    for (int m = 0; m < K; ++m) if (dims[m] < 0) return RETEXO_ERR_INVALID_ARG;
    const size_t need = retexo_cross_partition_workspace_size(g->n_nodes, g->n_edges, n_parts);
    if (!workspace || !aligned_to(workspace, kAlign) || workspace_bytes < need) return RETEXO_ERR_WORKSPACE;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const int n_sm = sm_count();
    if (n_sm <= 0) return RETEXO_ERR_CUDA;

    Arena ws(workspace, workspace_bytes);
    unsigned long long* acc = ws.take<unsigned long long>(32);
    RoundDimsArg dims_arg{};
    for (int m = 0; m < K; ++m) dims_arg.d[m] = dims[m];
    CountArgs a;
    a.n = g->n_nodes; a.rowptr = g->rowptr; a.colidx = g->colidx; a.part = part; a.n_parts = n_parts;
    a.cross_edges = acc; a.pairs = acc + 1; a.bad_part = acc + 2; a.next_row = acc + 4;
    a.row_batch = 1;
    a.send = reinterpret_cast<unsigned long long*>(send_per_part);
    a.recv = reinterpret_cast<unsigned long long*>(recv_per_part);
    a.big_list = nullptr; a.big_count = nullptr; a.big_bitmaps = nullptr; a.words_per_bitmap = 0;

    RETEXO_CUDA_TRY(cudaMemsetAsync(acc, 0, 32 * sizeof(unsigned long long), st));
    if (send_per_part) RETEXO_CUDA_TRY(cudaMemsetAsync(send_per_part, 0, sizeof(uint64_t) * (size_t)n_parts, st));
    if (recv_per_part) RETEXO_CUDA_TRY(cudaMemsetAsync(recv_per_part, 0, sizeof(uint64_t) * (size_t)n_parts, st));

    if (a.n > 0) {
        if (n_parts <= kBitmapParts) {
            const int64_t want = (a.n + kCntWarps - 1) / kCntWarps;
            const unsigned blocks = (unsigned)(want < (int64_t)n_sm * 8 ? want : (int64_t)n_sm * 8);
            // ~16 draws per warp: fine enough to balance hub rows, coarse enough for the counter
            const int64_t batch = a.n / ((int64_t)blocks * kCntWarps * 16);
            a.row_batch = (int32_t)(batch < 1 ? 1 : batch > 64 ? 64 : batch);
            const size_t tally = a.recv ? sizeof(uint32_t) * (size_t)n_parts : 0;      // <= 32 KB
            count_bitmap_kernel<<<blocks, kCntThreads, tally, st>>>(a);
        } else {
            a.big_list = ws.take<int32_t>((size_t)a.n);
            a.big_count = ws.take<int32_t>(64);
            a.words_per_bitmap = (n_parts + 31) / 32;
            a.big_bitmaps = ws.take<uint32_t>((size_t)kBigRowBlocks * (size_t)a.words_per_bitmap);
            RETEXO_CUDA_TRY(cudaMemsetAsync(a.big_count, 0, sizeof(int32_t), st));
            RETEXO_CUDA_TRY(cudaMemsetAsync(a.big_bitmaps, 0,
                                            sizeof(uint32_t) * (size_t)kBigRowBlocks * (size_t)a.words_per_bitmap, st));
            const int64_t want = (a.n + kHashWarps - 1) / kHashWarps;
            const unsigned blocks = (unsigned)(want < (int64_t)n_sm * 32 ? want : (int64_t)n_sm * 32);
            const int64_t batch = a.n / ((int64_t)blocks * kHashWarps * 16);
            a.row_batch = (int32_t)(batch < 1 ? 1 : batch > 64 ? 64 : batch);
            count_general_kernel<<<blocks, kHashWarps * kWarp, 0, st>>>(a);
            count_big_rows_kernel<<<kBigRowBlocks, kCntThreads, 0, st>>>(a);
        }
    }
    count_finalize_kernel<<<1, 32, 0, st>>>(acc, acc + 1, acc + 2, K, dims_arg, elem_bytes, cross_edges, boundary_pairs,
                                            bytes_per_round, bytes_total);
    return launch_status();
}

// ---------------------------------------------------------------- no-allocation variant
namespace retexo {

// Scratch of the allocation-free entry point.  It lives in the library image, so
// every GPU that loads the library holds these 4 MiB until the process exits.
constexpr size_t kStaticScratchBytes = size_t(4) << 20;
static __device__ __align__(256) unsigned char g_static_count_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
static std::mutex g_static_scratch_mutex;
static void* g_static_scratch_addr[kMaxDevices] = {};

// In host code the array's name is only a handle for the runtime, not a device
// address: the address is looked up once per device, with that device current.
static int static_scratch_address(void** out) {
    int dev = 0;
    RETEXO_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return RETEXO_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_addr[dev]) {
        void* ptr = nullptr;
        RETEXO_CUDA_TRY(cudaGetSymbolAddress(&ptr, g_static_count_scratch));
        g_static_scratch_addr[dev] = ptr;
    }
    *out = g_static_scratch_addr[dev];
    return RETEXO_OK;
}

}  // namespace retexo

extern "C" size_t retexo_cross_partition_static_scratch_bytes(void) { return kStaticScratchBytes; }

extern "C" int retexo_cross_partition_bytes_static(const retexo_csr* g, const int32_t* part, int32_t n_parts,
                                                   int32_t K, const int32_t* dims, int32_t elem_bytes,
                                                   uint64_t* cross_edges, uint64_t* boundary_pairs,
                                                   uint64_t* bytes_per_round, uint64_t* bytes_total,
                                                   uint64_t* send_per_part, uint64_t* recv_per_part, void* stream) {
    if (!g || g->n_nodes < 0 || g->n_edges < 0 || n_parts <= 0) return RETEXO_ERR_INVALID_ARG;
    const size_t need = retexo_cross_partition_workspace_size(g->n_nodes, g->n_edges, n_parts);
    if (need == 0) return RETEXO_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return RETEXO_ERR_UNSUPPORTED;     // beyond the built-in scratch
    void* scratch = nullptr;
    RETEXO_TRY(static_scratch_address(&scratch));
    // The counters and lists inside the scratch are cleared by the call below before use, so
    // what an earlier call left there does not matter.
    return retexo_cross_partition_bytes(g, part, n_parts, K, dims, elem_bytes, cross_edges, boundary_pairs,
                                        bytes_per_round, bytes_total, send_per_part, recv_per_part, scratch,
                                        kStaticScratchBytes, stream);
}
