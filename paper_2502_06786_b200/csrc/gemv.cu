// matq_gemv: host-side validation and kernel selection for the decode GEMV.
#include "common.cuh"
#include "gemv_cuda_core.cuh"
#include "gemv_tensor.cuh"
#include "gemv_tcgen05.cuh"
#include "gemv_imma.cuh"
#include "gemv_stream.cuh"
#include "gemv_stream_batch.cuh"

namespace {

// The integer kernel at the (m-tiles per warp, K split) the caller chose.
template <int R>
int launch_imma_split(int mt, int sk, const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                      const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                      float* y, int64_t ldy, bool pdl, cudaStream_t s) {
    using namespace matq::imma;
#define MATQ_IMMA(MT, SK, W) launch<R, MT, SK, W>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
    if (sk == 32) return MATQ_IMMA(1, 32, 32);
    if (sk == 16) return MATQ_IMMA(1, 16, 16);
    if (mt == 2) return sk == 8 ? MATQ_IMMA(2, 8, 8) : sk == 4 ? MATQ_IMMA(2, 4, 8) : sk == 2 ? MATQ_IMMA(2, 2, 8) : MATQ_IMMA(2, 1, 8);
    return sk == 8 ? MATQ_IMMA(1, 8, 8) : sk == 4 ? MATQ_IMMA(1, 4, 8) : sk == 2 ? MATQ_IMMA(1, 2, 8) : MATQ_IMMA(1, 1, 8);
#undef MATQ_IMMA
}

constexpr long long kStreamWaitCycles = 4000000000ll;         // limit of its waits: about two seconds of SM clock
constexpr long long kStallWaitCycles = 2000000ll;            // the same under MATQ_GEMV_TEST_STALL: about a millisecond

}  // namespace

extern "C" int matq_gemv_grouped(const matq_gemv_problem* problems, int n_problems, int c, unsigned flags,
                                 int32_t* dev_status, void* stream) {
    using namespace matq;
    if (n_problems < 0 || (n_problems > 0 && !problems)) return MATQ_ERR_INVALID_ARG;
    if (flags & ~(unsigned)(MATQ_GEMV_PDL | MATQ_GEMV_TEST_STALL)) return MATQ_ERR_INVALID_ARG;
    const bool stall = (flags & MATQ_GEMV_TEST_STALL) != 0;
    if (c != kCodeBits) return MATQ_ERR_UNSUPPORTED;
    static_assert(sizeof(gstream::HostProblem) == sizeof(matq_gemv_problem), "descriptor layouts must agree");
    bool any_batch = false;
    for (int i = 0; i < n_problems; ++i) {
        const matq_gemv_problem& q = problems[i];
        if (q.N < 0 || q.K <= 0 || q.B < 0 || q.B > 16 || !q.x || (q.N > 0 && (!q.packed || !q.alpha || !q.zero || !q.y))) return MATQ_ERR_INVALID_ARG;
        if ((q.ovf_row_ptr == nullptr) != (q.ovf_col == nullptr)) return MATQ_ERR_INVALID_ARG;
        if (!(q.r == 8 || q.r == 4 || q.r == 2)) return MATQ_ERR_UNSUPPORTED;
        if (q.B > 1 && q.ovf_row_ptr) return MATQ_ERR_UNSUPPORTED;       // lists with several vectors: matq_gemv per matrix
        if (q.K % 128 != 0 || q.K > imma::kMaxK || q.N >= (1ll << 31) - 16) return MATQ_ERR_SHAPE;
        if (q.B > 1 && q.r == 2 && q.K % 256 != 0) return MATQ_ERR_SHAPE;
        if ((q.N > 0 && !aligned16(q.packed)) || !aligned16(q.x)) return MATQ_ERR_ALIGNMENT;
        any_batch = any_batch || q.B > 1;
    }
    const bool pdl = (flags & MATQ_GEMV_PDL) != 0;
    const long long wait = stall ? kStallWaitCycles : kStreamWaitCycles;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const gstream::HostProblem* hp = reinterpret_cast<const gstream::HostProblem*>(problems);
    if (!any_batch) return gstream::launch(hp, n_problems, pdl, wait, stall, dev_status, s);
    // Single vectors and batches take different kernels: two sublists, in the order given (problems are independent).
    // A batch larger than one launch can stage becomes several problems that share the plane.
    std::vector<gstream::HostProblem> one, many;
    std::vector<int> many_b;
    for (int i = 0; i < n_problems; ++i) {
        if (hp[i].B <= 1) { one.push_back(hp[i]); continue; }
        const int st = gstream::split_batch(hp[i], one, many, many_b);
        if (st != MATQ_OK) return st;
    }
    for (const gstream::HostProblem& q : one)
        if (q.N != 0 && !gstream::eligible(q.N, q.K, q.r)) return MATQ_ERR_SHAPE;          // before anything is launched
    for (size_t i = 0; i < many.size(); ++i)
        if (many[i].N != 0 && !gstream::eligible_batch(many[i].N, many[i].K, many[i].r, many_b[i])) return MATQ_ERR_SHAPE;
    if (!one.empty()) {
        const int st = gstream::launch(one.data(), (int)one.size(), pdl, wait, stall, dev_status, s);
        if (st != MATQ_OK) return st;
    }
    return gstream::launch_batch(many.data(), many_b.data(), (int)many.size(), pdl, wait, stall, dev_status, s);
}

extern "C" int matq_gemv_grouped_launches(const matq_gemv_problem* problems, int n_problems) {
    using namespace matq;
    if (n_problems < 0 || (n_problems > 0 && !problems)) return -1;
    const gstream::HostProblem* hp = reinterpret_cast<const gstream::HostProblem*>(problems);
    std::vector<gstream::HostProblem> one, many;
    std::vector<int> many_b;
    for (int i = 0; i < n_problems; ++i) {
        if (hp[i].N == 0) continue;
        if (hp[i].B <= 1) { one.push_back(hp[i]); continue; }
        if (gstream::split_batch(hp[i], one, many, many_b) != MATQ_OK) return -1;
    }
    int launches = 0;
    const size_t per = one.size() <= (size_t)gstream::kSmallList ? gstream::kSmallList : gstream::kLargeList;
    for (size_t i = 0; i < one.size(); i += per) {
        bool lists = false;
        for (size_t j = i; j < std::min(one.size(), i + per); ++j) lists = lists || one[j].ovf_row_ptr != nullptr;
        launches += lists ? 2 : 1;                                  // ep_rowsum + the persistent kernel
    }
    return launches + gstream::count_batch_launches(many.data(), many_b.data(), (int)many.size());
}

extern "C" size_t matq_gemv_workspace_bytes(int64_t N, int64_t K, int r, int B) {
    (void)N; (void)K; (void)r; (void)B;
    return 0;   // the K-split is reduced inside warps / CTAs; no scratch is needed
}

extern "C" int matq_gemv(const uint8_t* packed, int64_t N, int64_t K, int c, int r,
                         const float* alpha, const float* zero,
                         const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                         const void* x, int B, int64_t ldx, float* y, int64_t ldy,
                         void* workspace, size_t workspace_bytes, unsigned flags,
                         int32_t* dev_status, void* stream) {
    using namespace matq;
    (void)workspace; (void)workspace_bytes;
    if (N < 0 || K <= 0 || B < 1 || B > 16 || !x || (N > 0 && (!packed || !alpha || !zero || !y))) return MATQ_ERR_INVALID_ARG;
    if ((ovf_row_ptr == nullptr) != (ovf_col == nullptr)) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits || !(r == 8 || r == 4 || r == 2)) return MATQ_ERR_UNSUPPORTED;
    if (K % 128 != 0 || ldx < K || ldx % 8 != 0 || ldy < N) return MATQ_ERR_SHAPE;
    if (ovf_row_ptr && K > 65536) return MATQ_ERR_SHAPE;
    if ((N > 0 && !aligned16(packed)) || !aligned16(x)) return MATQ_ERR_ALIGNMENT;
    const unsigned path = flags & MATQ_GEMV_PATH_MASK;
    if (path > MATQ_GEMV_STREAM || (flags & ~(MATQ_GEMV_PATH_MASK | MATQ_GEMV_PDL))) return MATQ_ERR_INVALID_ARG;
    if (N == 0) return MATQ_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool pdl = (flags & MATQ_GEMV_PDL) != 0;
    if (path == MATQ_GEMV_CUDA_CORE) {
        if (r == 8) launch_gemv_cuda_core<8>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        else if (r == 4) launch_gemv_cuda_core<4>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        else launch_gemv_cuda_core<2>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        return launch_status();
    }
    if (path == MATQ_GEMV_TCGEN05) {   // opt-in: correct, but its per-CTA set-up still costs more than it saves at decode sizes
        int st5;
        if (r == 8) st5 = t5::launch<8>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, dev_status, pdl, s);
        else if (r == 4) st5 = t5::launch<4>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, dev_status, pdl, s);
        else st5 = t5::launch<2>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, dev_status, pdl, s);
        if (st5 != MATQ_ERR_SHAPE) return st5;     // a K too long for one cluster's shared memory falls through
    }
    // Extra precision at B = 1: the list kernel of the persistent path (eight lanes per row, whole CTA on long lists)
    // replaces the few threads per row of the per-matrix kernels, which take milliseconds on rows whose codes all sit
    // in the extra bucket (heavy-tailed weights under plain min-max).
    const bool ep_stream = path == MATQ_GEMV_AUTO && B == 1 && ovf_row_ptr && gstream::eligible(N, K, r);
    if (path == MATQ_GEMV_STREAM && B > 1) {
        // batches in the persistent kernel: dense rows of x and y, no lists, at most 8 vectors per problem
        if (ovf_row_ptr) return MATQ_ERR_UNSUPPORTED;
        if (ldx != K || ldy != N) return MATQ_ERR_SHAPE;
        const gstream::HostProblem q = {packed, N, K, r, alpha, zero, nullptr, nullptr, x, y, B};
        std::vector<gstream::HostProblem> one, many;
        std::vector<int> many_b;
        int st = gstream::split_batch(q, one, many, many_b);
        if (st != MATQ_OK) return st;
        if (!one.empty() && !gstream::eligible(N, K, r)) return MATQ_ERR_SHAPE;
        if (!one.empty() && (st = gstream::launch(one.data(), (int)one.size(), pdl, kStreamWaitCycles, false, dev_status, s)) != MATQ_OK) return st;
        return gstream::launch_batch(many.data(), many_b.data(), (int)many.size(), pdl || !one.empty(), kStreamWaitCycles, false, dev_status, s);
    }
    if (path == MATQ_GEMV_STREAM || ep_stream) {
        if (B != 1 || !gstream::eligible(N, K, r)) return MATQ_ERR_SHAPE;
        const gstream::HostProblem hp = {packed, N, K, r, alpha, zero, ovf_row_ptr, ovf_col, x, y, 1};
        return gstream::launch(&hp, 1, pdl, kStreamWaitCycles, false, dev_status, s);
    }
    // Warp tile: 16*MT rows x K/SK; the SK warps of a row tile sit in one CTA.  The split aims at ONE wave of CTAs
    // (a second, partly filled wave costs up to 40 %; measured on B200 for 4-26 MB planes):
    //   * few, long rows (at most one or two 16-row tiles per SM): one tile per CTA of 32 or 16 warps, SK = 32 / 16;
    //   * otherwise CTAs of 8 warps with two m-tiles per warp (the staged activations are reused twice; two such
    //     CTAs fit an SM) and the finest K split (8, 4, 2 or 1) that still fits one wave; if none does, SK = 8 and
    //     several waves.
    const int sms = sm_count();
    const int64_t n_qc = (K * r / 8 + 63) / 64;
    const int64_t tiles16 = (N + 15) / 16;
    int mt = 1, sk = 1;
    if (tiles16 <= sms && n_qc >= 16) sk = 32;
    else if (tiles16 <= 2 * sms && n_qc >= 8) sk = 16;
    else if (tiles16 <= 2 * sms) {                       // few short rows: as many warps as there are chunks
        while (sk < 8 && n_qc / (2 * sk) >= 1) sk *= 2;
    } else {
        mt = 2;
        const int64_t tiles32 = (N + 31) / 32;
        sk = 8;                                          // CTAs = tiles32 / (8 / sk): halve sk until they fit one wave
        while (sk > 1 && (tiles32 * sk + 7) / 8 > 2 * sms) sk /= 2;
        if ((tiles32 * sk + 7) / 8 > 2 * sms) sk = 8;     // not even SK = 1 fits: several waves of the finest split
        while (sk > 1 && n_qc < sk) sk /= 2;
    }
    int st = MATQ_ERR_SHAPE;
    // A single activation vector goes to the integer tensor path (twice the weights per MMA, one mask per four
    // weights, no offset to remove, exact sums); it declines (MATQ_ERR_SHAPE) what it does not take (B > 1,
    // K > 32768) and the bf16 kernel below runs instead.  Measured on B200 it wins or ties on every decode shape
    // (1.2-1.7x on 25-50 MB planes).
    const bool int8_auto = B == 1;
    if ((path == MATQ_GEMV_AUTO && int8_auto) || path == MATQ_GEMV_TENSOR_INT8) {
        st = (r == 8) ? launch_imma_split<8>(mt, sk, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
           : (r == 4) ? launch_imma_split<4>(mt, sk, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
                      : launch_imma_split<2>(mt, sk, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        if (st == MATQ_OK) return launch_status();
        if (st != MATQ_ERR_SHAPE) return st;
    }
#define MATQ_GEMV_T(RR, MT, NT, SK) launch_gemv_tensor<RR, MT, NT, SK>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
#define MATQ_GEMV_W(RR, NT, W) launch_gemv_tensor<RR, 1, NT, W, W>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
#define MATQ_GEMV_S(RR, MT, NT) ((sk == 8) ? MATQ_GEMV_T(RR, MT, NT, 8) : (sk == 4) ? MATQ_GEMV_T(RR, MT, NT, 4) : (sk == 2) ? MATQ_GEMV_T(RR, MT, NT, 2) : MATQ_GEMV_T(RR, MT, NT, 1))
#define MATQ_GEMV_R(MT, NT) ((r == 8) ? MATQ_GEMV_S(8, MT, NT) : (r == 4) ? MATQ_GEMV_S(4, MT, NT) : MATQ_GEMV_S(2, MT, NT))
#define MATQ_GEMV_RW(NT, W) ((r == 8) ? MATQ_GEMV_W(8, NT, W) : (r == 4) ? MATQ_GEMV_W(4, NT, W) : MATQ_GEMV_W(2, NT, W))
    const bool wide = mt == 2 && sk == 8 && B > 4 && B <= 8 && ((N + 31) / 32 + 1) / 2 <= sms;
    // Batches of four or more on long rows: a cluster of 4 CTAs takes four times the rows and splits K four ways, so
    // each CTA stages a quarter of the B activation columns (same number of CTAs, same work per warp).  Measured on
    // B200: 3584 x 14336 at B = 8 33.5 -> 16.9 us, 3584 x 4096 at B = 16 19.4 -> 11.1 us; shapes with so few rows that
    // a row tile has a whole CTA of 32 warps (2304 x 9216) lose with clusters (10.4 -> 14.3 us) and keep the plain kernel.
    if (B >= 4 && n_qc >= 32 && (B >= 8 || n_qc >= 56) && (wide || sk == 16 || (mt == 2 && sk == 8))) {
#define MATQ_GEMV_C(RR, MT, NT, SK, W) launch_gemv_tensor<RR, MT, NT, SK, W, 4>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
#define MATQ_GEMV_CR(MT, NT, SK, W) ((r == 8) ? MATQ_GEMV_C(8, MT, NT, SK, W) : (r == 4) ? MATQ_GEMV_C(4, MT, NT, SK, W) : MATQ_GEMV_C(2, MT, NT, SK, W))
        if (wide) st = MATQ_GEMV_CR(2, 1, 2, 16);
        else if (sk == 16) st = B <= 8 ? MATQ_GEMV_CR(1, 1, 4, 16) : MATQ_GEMV_CR(1, 2, 4, 16);
        else st = B <= 8 ? MATQ_GEMV_CR(2, 1, 2, 8) : MATQ_GEMV_CR(2, 2, 2, 8);
#undef MATQ_GEMV_CR
#undef MATQ_GEMV_C
        if (st == MATQ_OK) return launch_status();
        if (st != MATQ_ERR_SHAPE) return st;
    }
    if (wide) {                    // a batch: 16-warp CTAs (two row tiles) halve the staging of x' per SM (measured 4-12 %)
        st = (r == 8) ? launch_gemv_tensor<8, 2, 1, 8, 16>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
           : (r == 4) ? launch_gemv_tensor<4, 2, 1, 8, 16>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s)
                      : launch_gemv_tensor<2, 2, 1, 8, 16>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
    } else
    if (sk >= 16) {                // few, long rows: one 16-row tile per CTA, K split over 16 or 32 warps
        if (B <= 8) st = (sk == 32) ? MATQ_GEMV_RW(1, 32) : MATQ_GEMV_RW(1, 16);
        else st = (sk == 32) ? MATQ_GEMV_RW(2, 32) : MATQ_GEMV_RW(2, 16);
    } else if (B <= 8) st = (mt == 2) ? MATQ_GEMV_R(2, 1) : MATQ_GEMV_R(1, 1);
    else st = (mt == 2) ? MATQ_GEMV_R(2, 2) : MATQ_GEMV_R(1, 2);
#undef MATQ_GEMV_RW
#undef MATQ_GEMV_R
#undef MATQ_GEMV_S
#undef MATQ_GEMV_W
#undef MATQ_GEMV_T
    if (st == MATQ_ERR_SHAPE) {   // the staged activations of this call do not fit in shared memory: FMA path
        if (r == 8) launch_gemv_cuda_core<8>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        else if (r == 4) launch_gemv_cuda_core<4>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        else launch_gemv_cuda_core<2>(packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, x, B, ldx, y, ldy, pdl, s);
        return launch_status();
    }
    if (st != MATQ_OK) return st;
    return launch_status();
}
