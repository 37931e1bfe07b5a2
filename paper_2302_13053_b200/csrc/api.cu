// Status strings and version of the retexo C ABI.
#include "common.cuh"

extern "C" const char* retexo_status_string(int status) {
    switch (status) {
        case RETEXO_OK: return "ok";
        case RETEXO_ERR_INVALID_ARG: return "invalid argument";
        case RETEXO_ERR_BAD_GRAPH: return "malformed CSR graph";
        case RETEXO_ERR_ALIGNMENT: return "pointer or leading dimension breaks an alignment rule";
        case RETEXO_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case RETEXO_ERR_UNSUPPORTED: return "shape not supported";
        case RETEXO_ERR_CUDA: return "CUDA runtime error or no CUDA device";
        case RETEXO_ERR_TIMEOUT: return "bounded device-side wait gave up";
        default: return "unknown status";
    }
}

extern "C" int retexo_version(void) { return 100; }

// Closed forms of Section 3.3 / Appendix A.1 (host arithmetic).
extern "C" int retexo_data_volume(int32_t K, const int64_t* H, const int64_t* L, double n_workers, double B, double R,
                                  retexo_data_volume_result* out) {
    if (K < 1 || !H || !L || !out || !(n_workers > 0.0) || !(B >= 0.0) || !(R > 0.0)) return RETEXO_ERR_INVALID_ARG;
    double hidden_sum = 0.0, model = 0.0, classifiers = 0.0;
    for (int32_t m = 0; m <= K; ++m) if (H[m] < 0) return RETEXO_ERR_INVALID_ARG;
    for (int32_t m = 1; m < K; ++m) {
        hidden_sum += (double)H[m];
        classifiers += (double)H[m] * (double)H[K];
    }
    for (int32_t m = 0; m < K; ++m) {
        if (L[m] < 0) return RETEXO_ERR_INVALID_ARG;
        model += (double)L[m];
    }
    const double pairs = 2.0 * n_workers * B;                  // boundary rows sent plus received
    out->lazy_lt = pairs * (hidden_sum + (double)H[0]);
    out->standard_lt = pairs * (2.0 * R * hidden_sum + (double)H[0]);
    out->standard_reduce = 2.0 * n_workers * R * model;
    out->lazy_reduce = 2.0 * n_workers * R * (model + classifiers);
    out->model_size = model;
    const double den = out->lazy_lt + out->lazy_reduce;
    out->gamma = den > 0.0 ? (out->standard_lt + out->standard_reduce) / den : 0.0;
    return RETEXO_OK;
}

// dst[i][0 .. dim) = src[idx[i]][0 .. dim): the owned rows a peer needs, packed for the round's one exchange.
// A warp moves a row; 16-byte pieces where both sides allow.
__global__ void __launch_bounds__(256) gather_rows_f32_kernel(const float* __restrict__ src, int64_t ld_src, int32_t dim,
                                                              const int32_t* __restrict__ idx, int64_t n_rows,
                                                              float* __restrict__ dst, int64_t ld_dst, int vec) {
    const int lane = threadIdx.x & 31;
    const int64_t i = blockIdx.x * 8ll + (threadIdx.x >> 5);
    if (i >= n_rows) return;
    const float* s = src + (int64_t)idx[i] * ld_src;
    float* d = dst + i * ld_dst;
    if (vec) {
        for (int c = lane; c < dim / 4; c += 32) reinterpret_cast<float4*>(d)[c] = __ldg(reinterpret_cast<const float4*>(s) + c);
    } else {
        for (int c = lane; c < dim; c += 32) d[c] = s[c];
    }
}

extern "C" int retexo_gather_rows(const float* src, int64_t ld_src, int32_t dim, const int32_t* idx, int64_t n_rows,
                                  float* dst, int64_t ld_dst, void* stream) {
    if (n_rows < 0 || dim <= 0 || ld_src < dim || ld_dst < dim) return RETEXO_ERR_INVALID_ARG;
    if (n_rows == 0) return RETEXO_OK;
    if (!src || !idx || !dst) return RETEXO_ERR_INVALID_ARG;
    const int vec = dim % 4 == 0 && ld_src % 4 == 0 && ld_dst % 4 == 0 && retexo::aligned_to(src, 16) && retexo::aligned_to(dst, 16);
    gather_rows_f32_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, static_cast<cudaStream_t>(stream)>>>(src, ld_src, dim, idx, n_rows,
                                                                                                      dst, ld_dst, vec);
    return retexo::launch_status();
}
