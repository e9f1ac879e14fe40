// matq_gemm_multi: multi-precision dense forward (Eq. 7).  Not built yet.
#include "common.cuh"

extern "C" size_t matq_gemm_multi_workspace_bytes(int src_kind, int64_t M, int64_t N, int64_t K, int n_r) {
    (void)src_kind; (void)M; (void)N; (void)K; (void)n_r;
    return 0;
}

extern "C" int matq_gemm_multi(int, const void*, int64_t, int64_t, int, float*, float*, int,
                               const int32_t*, const uint16_t*, const void*, int64_t, int64_t,
                               const int*, int, float* const*, int64_t, void*, size_t, int32_t*, void*) {
    return MATQ_ERR_UNSUPPORTED;
}
