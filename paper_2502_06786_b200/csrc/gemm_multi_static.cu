// matq_gemm_multi_static: the multi-precision dense forward for callers that cannot hand the library any scratch.
//
// Some users of this library run where device memory cannot be obtained at call time: a serving loop whose memory
// was carved up once at start-up and which must not call cudaMalloc on the request path (it synchronises the whole
// device and may fail once memory is fragmented), or a plug-in living inside another framework's allocator that has
// no way to ask it for more.  matq_gemm_multi needs a workspace for the codes, the per-precision bf16 planes and
// the row sums of X; this entry point supplies that workspace itself, from an array that is part of the library's
// device image, so the caller passes inputs and outputs only and nothing is allocated by anyone.
//
// The array is a fixed kStaticScratchBytes (16 MiB) per GPU that loads the library, held until the process exits.
// Problems whose workspace would be larger are refused with MATQ_ERR_WORKSPACE before anything is launched.
// All calls on a GPU share the one array and it keeps whatever the previous call left in it.  Nothing in it has to
// start at zero (every byte a kernel reads is written earlier in the same call), so no clearing is done; but two
// calls that overlap on the GPU (different streams, or different host threads) would overwrite each other's
// planes: callers must order them.
//
// The array's name is only meaningful in device code.  Host code must not pass it to a kernel as if it were a
// pointer; it asks the runtime for the array's device address (cudaGetSymbolAddress) once per device, with that
// device current, and passes that address on.  This happens in the first call made on each device, which for that
// reason should be made before any stream capture is started.
#include <atomic>

#include "common.cuh"

namespace matq {
namespace {

constexpr size_t kStaticScratchBytes = 16u << 20;
constexpr int kMaxDevices = 64;

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

std::atomic<void*> g_scratch_addr[kMaxDevices];

// Device address of the array on the current device; resolved on first use per device.
int static_scratch(void** out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return MATQ_ERR_CUDA;
    void* p = g_scratch_addr[dev].load(std::memory_order_acquire);
    if (!p) {
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return MATQ_ERR_CUDA;
        }
        g_scratch_addr[dev].store(p, std::memory_order_release);   // racing threads store the same value
    }
    *out = p;
    return MATQ_OK;
}

}  // namespace
}  // namespace matq

extern "C" size_t matq_gemm_multi_static_max_bytes(void) { return matq::kStaticScratchBytes; }

extern "C" int matq_gemm_multi_static(int src_kind, const void* Wsrc, int64_t N, int64_t K, int c,
                                      float* alpha, float* zero, int extra_precision,
                                      const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                                      const void* X, int64_t M, int64_t ldx,
                                      const int* rs, int n_r, float* const* Y, int64_t ldy,
                                      int32_t* dev_status, void* stream) {
    using namespace matq;
    if (M < 0 || N < 0 || K <= 0 || n_r < 1 || n_r > 3) return MATQ_ERR_INVALID_ARG;
    // an empty problem needs no scratch, whatever N * K says: it behaves exactly like matq_gemm_multi
    if (M == 0 || N == 0)
        return matq_gemm_multi(src_kind, Wsrc, N, K, c, alpha, zero, extra_precision, ovf_row_ptr, ovf_col, X, M, ldx,
                               rs, n_r, Y, ldy, nullptr, 0, dev_status, stream);
    // size check next: a problem that does not fit the built-in array is refused without touching the GPU
    const size_t need = matq_gemm_multi_workspace_bytes(src_kind, M, N, K, n_r);
    if (need == 0) return MATQ_ERR_INVALID_ARG;
    if (need > kStaticScratchBytes) return MATQ_ERR_WORKSPACE;
    void* scratch = nullptr;
    const int st = static_scratch(&scratch);
    if (st != MATQ_OK) return st;
    return matq_gemm_multi(src_kind, Wsrc, N, K, c, alpha, zero, extra_precision, ovf_row_ptr, ovf_col, X, M, ldx,
                           rs, n_r, Y, ldy, scratch, kStaticScratchBytes, dev_status, stream);
}
