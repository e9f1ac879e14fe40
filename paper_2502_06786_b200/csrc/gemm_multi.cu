// matq_gemm_multi: the multi-precision dense forward of MatQuant co-training (Eq. 7): for every r in rs,
//   Y_r[m,n] = alpha_n * ( 2^(c-r) * sum_k X[m,k] k_r[n,k]  -  z_n * sum_k X[m,k] ),   k_r = S(q, r) / 2^(c-r).
//
// The contraction runs on the fifth-generation tensor cores.  The integer fields k_r (0 .. 2^r, at most 256) are
// exact in bf16 and the activations are bf16, so every product is exact in fp32 and only the fp32 accumulation
// rounds; alpha, the power of two and the zero-point term z_n * sum_k x are applied per channel after accumulation.
//
// Stages of one call (all on the caller's stream, scratch in the caller's workspace):
//   1. MATQ_SRC_BF16 only: Eq. 1 (matq_quantize) -> codes in the workspace, alpha / zero to the caller.
//   2. expand: codes (or a packed plane + overflow list) -> one bf16 plane of fields per precision in the workspace.
//   3. rowsum: sx[m] = sum_k X[m,k] in fp32.
//   4. GEMM: one CTA per 128 x 128 output tile computes ALL precisions from one pass over its X tiles:
//        warp 0   TMA producer: per 64-wide k block one 128 x 64 box of X and one of every plane, 128-byte swizzle,
//                 into a ring of shared-memory stages (mbarrier full / empty pairs);
//        warp 1   issues tcgen05.mma (M = 128, N = 128, K = 16; A and B from shared-memory descriptors), one fp32
//                 accumulator of 128 TMEM columns per precision; tcgen05.commit releases a stage;
//        warps 2-5 epilogue: tcgen05.ld the accumulators, apply alpha / 2^sh / z * sx, store fp32 rows.
//      Every copy goes to the loading CTA only; no clusters.  Every wait on an mbarrier is bounded and reports MATQ_ERR_TIMEOUT.
#include <cuda.h>

#include "common.cuh"

namespace matq {
namespace gm {

constexpr int kBM = 128, kBN = 128, kBK = 64;
constexpr int kThreads = 192;
constexpr int kMaxR = 3;
constexpr int kMaxStages = 8;
constexpr int kTileBytes = kBM * kBK * 2;          // 16 KB: one 128 x 64 bf16 box
constexpr long long kWaitCycles = 4000000000ll;     // SM clock cycles after which a wait on an mbarrier gives up: about two seconds
constexpr long long kStallWaitCycles = 2000000ll;   // the same under matq_gemm_multi_test_stall: about a millisecond

struct Params {
    const float* alpha;
    const float* zero;
    const float* sx;
    float* Y[kMaxR];
    int sh[kMaxR];
    int64_t M, N, K, ldy;
    int n_r, stages;
    int wide;      // one plane only: the CTA takes 256 channels as two adjacent 128-row tiles (n_r is then 2)
    const float* Yt;      // loss mode: target [M, N] (row stride ldt); outputs are not stored
    int64_t ldt;
    float* loss_part;     // loss mode: [CTAs][kMaxR] sums of squared errors
    int teacher[kMaxR];   // loss mode, per precision: -1 target only, j another precision's output as the target, 256 + j both
    int32_t* dev_status;
    long long wait_cycles;   // limit of every wait on an mbarrier
    int hold;                // tests of the error path: the producer issues no copies
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

// Bounded in SM clock cycles (the clock is read once per 64 polls; the first reading starts the count).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, long long limit) {
    uint32_t done = 0;
    long long t0 = 0;
    for (uint32_t it = 0; !done; ++it) {
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        if (!done && (it & 63u) == 63u) {
            const long long now = clock64();
            if (t0 == 0) t0 = now;
            else if (now - t0 > limit) break;
        }
    }
    return done != 0;
}

// K-major operand tile written by TMA with 128-byte swizzle: rows of 128 bytes, 8-row atoms 1024 bytes apart.
__device__ __forceinline__ uint64_t sw128_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | (1ull << 16) | ((uint64_t)(1024 >> 4) << 32) | (1ull << 46) | (2ull << 61);
}
// 32 consecutive fp32 columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t addr, uint32_t (&d)[32]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
                 "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]),
                   "=r"(d[8]), "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15]),
                   "=r"(d[16]), "=r"(d[17]), "=r"(d[18]), "=r"(d[19]), "=r"(d[20]), "=r"(d[21]), "=r"(d[22]), "=r"(d[23]),
                   "=r"(d[24]), "=r"(d[25]), "=r"(d[26]), "=r"(d[27]), "=r"(d[28]), "=r"(d[29]), "=r"(d[30]), "=r"(d[31])
                 : "r"(addr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// kind::f16, D = fp32, A = B = bf16, both K-major, N = 128, M = 128
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBN >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);
// the same with N = 256: two adjacent plane tiles in one instruction
constexpr uint32_t kIdesc2 = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)((2 * kBN) >> 3) << 17) | ((uint32_t)(kBM >> 4) << 24);

__global__ void __launch_bounds__(kThreads, 1)
gemm_multi_kernel(const __grid_constant__ CUtensorMap tm_x, const __grid_constant__ CUtensorMap tm_b0,
                  const __grid_constant__ CUtensorMap tm_b1, const __grid_constant__ CUtensorMap tm_b2, const Params P) {
    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_full[kMaxStages], s_empty[kMaxStages], s_acc;
    __shared__ uint32_t s_tmem;
    __shared__ float s_alpha[2 * kBN], s_az[2 * kBN];      // alpha_n and alpha_n * z_n of this tile's columns
    __shared__ int s_timeout;
    __shared__ float s_loss[4][kMaxR];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // blockIdx.x walks the token tiles: CTAs that run together share one 128-channel slab of the planes (3 x 1 MB,
    // read from HBM once) and differ in their X tiles, and all of X stays in the L2.  The other order re-streams the
    // planes from HBM once per token tile.
    const int64_t m0 = (int64_t)blockIdx.x * kBM, n0 = (int64_t)blockIdx.y * (P.wide ? 2 * kBN : kBN);
    const int nkb = (int)(P.K / kBK);
    const int stage_bytes = (1 + P.n_r) * kTileBytes;
    const int tmem_cols = P.n_r == 1 ? 128 : (P.n_r == 2 ? 256 : 512);
    // dynamic shared memory is only guaranteed 16-byte aligned: round the ring up to the 1024 bytes the swizzle needs
    unsigned char* ring = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);

    if (tid == 0) {
        for (int s = 0; s < P.stages; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_full[s])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_empty[s])));
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_acc)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_timeout = 0;
    }
    if (warp == 2) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    if (warp >= 2) {
        for (int c = tid - 64; c < (P.wide ? 2 * kBN : kBN); c += kBN) {   // a column of this tile
            const int64_t n = n0 + c;
            const float a = n < P.N ? P.alpha[n] : 0.f, z = n < P.N ? P.zero[n] : 0.f;
            s_alpha[c] = a;
            s_az[c] = a * z;
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    if (warp == 0) {
        // ---------------- TMA producer
        if (lane == 0) {
            const CUtensorMap* tmb[kMaxR] = {&tm_b0, &tm_b1, &tm_b2};
            for (int kb = 0; kb < nkb && !P.hold; ++kb) {
                const int s = kb % P.stages;
                const uint32_t ph = (uint32_t)(kb / P.stages) & 1u;
                if (!mbar_wait(smem_u32(&s_empty[s]), ph ^ 1u, P.wait_cycles)) { s_timeout = 1; break; }
                const uint32_t bar = smem_u32(&s_full[s]);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(stage_bytes) : "memory");
                unsigned char* st = ring + (size_t)s * stage_bytes;
                const int k0 = kb * kBK;
                asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                             ::"r"(smem_u32(st)), "l"(&tm_x), "r"(k0), "r"((int)m0), "r"(bar) : "memory");
                for (int r = 0; r < P.n_r; ++r)
                    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                                 ::"r"(smem_u32(st + (size_t)(1 + r) * kTileBytes)), "l"(tmb[P.wide ? 0 : r]), "r"(k0),
                                   "r"((int)n0 + (P.wide ? r * kBN : 0)), "r"(bar) : "memory");
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer
        if (lane == 0) {
            bool ok = true;
            for (int kb = 0; kb < nkb && ok; ++kb) {
                const int s = kb % P.stages;
                const uint32_t ph = (uint32_t)(kb / P.stages) & 1u;
                if (!mbar_wait(smem_u32(&s_full[s]), ph, P.wait_cycles)) {
                    s_timeout = 1;                            // visible to the epilogue before the arrival below
                    __threadfence_block();
                    ok = false;
                    break;
                }
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t a_base = smem_u32(ring + (size_t)s * stage_bytes);
#pragma unroll
                for (int kk = 0; kk < kBK / 16; ++kk) {
                    const uint64_t ad = sw128_desc(a_base + kk * 32);
                    // The tiles of the first two planes are adjacent in the stage (rows 0..255 of one K-major operand) and
                    // so are their accumulators in TMEM: one N = 256 MMA covers both and reads the X tile once for them.
                    const uint32_t accumulate = (kb > 0 || kk > 0) ? 1u : 0u;
                    for (int r = 0; r < P.n_r; ++r) {
                        const bool pair = (r == 0 && P.n_r >= 2);
                        const uint64_t bd = sw128_desc(a_base + (1 + r) * kTileBytes + kk * 32);
                        asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p; }"
                                     ::"r"(tmem + r * kBN), "l"(ad), "l"(bd), "r"(pair ? kIdesc2 : kIdesc), "r"(accumulate) : "memory");
                        if (pair) ++r;
                    }
                }
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_empty[s])) : "memory");
            }
            // arrives when every MMA above has retired (also on the give-up path, so the epilogue never hangs)
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_acc)) : "memory");
        }
    } else {
        // ---------------- epilogue: thread = one output row (TMEM lane), 32 columns at a time
        const int quad = warp & 3;
        const int64_t m = m0 + quad * 32 + lane;
        // whole warps agree on the outcome: the reads of tensor memory below are warp-wide
        // (the arrival also comes when the MMA warp gave up: the accumulators are then incomplete and are not used)
        const bool done = __all_sync(0xffffffffu, mbar_wait(smem_u32(&s_acc), 0, P.wait_cycles)) && *(volatile int*)&s_timeout == 0;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        if (!done) s_timeout = 1;                           // gave up: report it, read and store nothing
        const float sx = (m < P.M) ? P.sx[m] : 0.f;
        float lacc[kMaxR] = {0.f, 0.f, 0.f};               // loss mode: this thread's squared errors per precision
        for (int r = 0; r < (done ? P.n_r : 0); ++r) {
            const int pr = P.wide ? 0 : r;                    // which precision this accumulator belongs to
            const int64_t nb = n0 + (P.wide ? r * kBN : 0);     // first channel of this accumulator
            const float* al = s_alpha + (P.wide ? r * kBN : 0);
            const float* az = s_az + (P.wide ? r * kBN : 0);
            const float scale = (float)(1 << P.sh[pr]);
            float* yrow = P.Yt ? nullptr : P.Y[pr] + m * P.ldy + nb;
            for (int c0 = 0; c0 < kBN; c0 += 32) {
                uint32_t d[32];
                // loss mode: the thread's 128 bytes of the target row are requested before the accumulators are read
                const float* trow = P.Yt ? P.Yt + m * P.ldt + nb + c0 : nullptr;
                const bool tvec = P.Yt && m < P.M && (nb + c0 + 32 <= P.N) && ((reinterpret_cast<uintptr_t>(trow) & 15u) == 0);
                float4 t4[8];
                if (tvec) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) t4[j] = __ldg(reinterpret_cast<const float4*>(trow) + j);
                }
                const uint32_t addr = tmem + ((uint32_t)(quad * 32) << 16) + r * kBN + c0;
                tmem_ld32(addr, d);
                if (P.Yt) {                                   // Eq. 7's loss instead of the outputs
                    const int code = P.teacher[pr];
                    const bool vs_target = code < 0 || code >= 256;
                    const int tj = code >= 0 ? (code & 255) : -1;    // co-distillation: precision tj's output is a target too
                    uint32_t dt[32];
                    float scale_t = 0.f;
                    if (tj >= 0) {                                // warp-uniform
                        tmem_ld32(tmem + ((uint32_t)(quad * 32) << 16) + tj * kBN + c0, dt);
                        scale_t = (float)(1 << P.sh[tj]);
                    }
                    if (m < P.M) {
                        float acc = 0.f;
                        if (vs_target && tvec) {                  // the common case: a whole, aligned chunk of the target
#pragma unroll
                            for (int j = 0; j < 8; ++j) {
                                const float tv[4] = {t4[j].x, t4[j].y, t4[j].z, t4[j].w};
#pragma unroll
                                for (int u = 0; u < 4; ++u) {
                                    const int cc = c0 + 4 * j + u;
                                    const float e = al[cc] * scale * __uint_as_float(d[4 * j + u]) - az[cc] * sx - tv[u];
                                    acc = fmaf(e, e, acc);
                                }
                            }
                        } else if (vs_target) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (nb + c0 + j < P.N) {
                                    const float e = al[c0 + j] * scale * __uint_as_float(d[j]) - az[c0 + j] * sx - trow[j];
                                    acc = fmaf(e, e, acc);
                                }
                        }
                        if (tj >= 0) {
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                if (nb + c0 + j < P.N) {          // alpha z sum(x) is common to both outputs
                                    const float e = al[c0 + j] * (scale_t * __uint_as_float(dt[j]) - scale * __uint_as_float(d[j]));
                                    acc = fmaf(e, e, acc);
                                }
                        }
                        lacc[pr] += acc;
                    }
                } else if (m < P.M) {
                    const bool vec = (nb + c0 + 32 <= P.N) && ((reinterpret_cast<uintptr_t>(yrow + c0) & 15u) == 0);
                    if (vec) {
#pragma unroll
                        for (int j = 0; j < 32; j += 4) {
                            float4 o;
                            o.x = al[c0 + j] * scale * __uint_as_float(d[j]) - az[c0 + j] * sx;
                            o.y = al[c0 + j + 1] * scale * __uint_as_float(d[j + 1]) - az[c0 + j + 1] * sx;
                            o.z = al[c0 + j + 2] * scale * __uint_as_float(d[j + 2]) - az[c0 + j + 2] * sx;
                            o.w = al[c0 + j + 3] * scale * __uint_as_float(d[j + 3]) - az[c0 + j + 3] * sx;
                            *reinterpret_cast<float4*>(yrow + c0 + j) = o;
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (nb + c0 + j < P.N)
                                yrow[c0 + j] = al[c0 + j] * scale * __uint_as_float(d[j]) - az[c0 + j] * sx;
                    }
                }
            }
        }
        if (P.Yt) {                                           // warp sums in a fixed order, one slot per epilogue warp
#pragma unroll
            for (int i = 0; i < kMaxR; ++i) {
                float v = lacc[i];
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
                if (lane == 0) s_loss[quad][i] = v;
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (P.Yt && tid < kMaxR)
        P.loss_part[((size_t)blockIdx.y * gridDim.x + blockIdx.x) * kMaxR + tid] =
            (s_loss[0][tid] + s_loss[1][tid]) + (s_loss[2][tid] + s_loss[3][tid]);
    if (tid == 0 && s_timeout) report(P.dev_status, MATQ_ERR_TIMEOUT);
    if (warp == 2)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(tmem_cols) : "memory");
}

// ---------------------------------------------------------------- small helper kernels

// codes -> one bf16 plane of fields per precision.  One thread = 16 codes.
struct ExpandArgs {
    __nv_bfloat16* plane[kMaxR];
    int r[kMaxR];
    int n_r, extra_precision;
};

__global__ void __launch_bounds__(256)
expand_codes(const uint4* __restrict__ q, int64_t nchunks, ExpandArgs A) {
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < nchunks; i += stride) {
        const uint4 v = ld_stream_u4(q + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        for (int t = 0; t < A.n_r; ++t) {
            const int r = A.r[t], sh = kCodeBits - r;
            const uint32_t kmax = (1u << r) - 1u;
            uint32_t out[8];
#pragma unroll
            for (int j = 0; j < 16; j += 2) {
                uint32_t f[2];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint32_t code = (w[(j + h) >> 2] >> (8 * ((j + h) & 3))) & 0xffu;
                    uint32_t k = sh ? ((code + (1u << (sh - 1))) >> sh) : code;
                    if (!A.extra_precision && k > kmax) k = kmax;
                    f[h] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn((float)k));
                }
                out[j >> 1] = f[0] | (f[1] << 16);
            }
            uint4* dst = reinterpret_cast<uint4*>(A.plane[t]) + 2 * i;
            dst[0] = make_uint4(out[0], out[1], out[2], out[3]);
            dst[1] = make_uint4(out[4], out[5], out[6], out[7]);
        }
    }
}

// packed r-bit plane -> bf16 plane of fields.  One thread = 16 bytes of the plane (128 / r fields), written as
// 16-byte stores of eight bf16 each.
template <int R>
__global__ void __launch_bounds__(256)
expand_packed(const uint4* __restrict__ packed, int64_t nvec, __nv_bfloat16* __restrict__ plane) {
    constexpr int kPerWord = 32 / R;
    constexpr uint32_t kMask = (1u << R) - 1u;
    const int64_t stride = (int64_t)gridDim.x * 256;
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < nvec; i += stride) {
        const uint4 v = ld_stream_u4(packed + i);
        const uint32_t w[4] = {v.x, v.y, v.z, v.w};
        uint4* dst = reinterpret_cast<uint4*>(plane + i * (4 * kPerWord));
#pragma unroll
        for (int t = 0; t < (4 * kPerWord) / 8; ++t) {         // eight fields per 16-byte store
            uint32_t o[4];
#pragma unroll
            for (int h = 0; h < 4; ++h) {
                const int e0 = 8 * t + 2 * h, e1 = e0 + 1;
                const uint32_t lo = (w[e0 / kPerWord] >> ((e0 % kPerWord) * R)) & kMask;
                const uint32_t hi = (w[e1 / kPerWord] >> ((e1 % kPerWord) * R)) & kMask;
                o[h] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn((float)lo)) |
                       ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn((float)hi)) << 16);
            }
            dst[t] = make_uint4(o[0], o[1], o[2], o[3]);
        }
    }
}

// extra precision from a list: the listed fields are one higher than the stored, clamped ones
__global__ void __launch_bounds__(256)
add_overflow(const int32_t* __restrict__ row_ptr, const uint16_t* __restrict__ col, int64_t N, int64_t K,
             __nv_bfloat16* __restrict__ plane) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t n = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); n < N; n += warps)
        for (int32_t p = row_ptr[n] + lane; p < row_ptr[n + 1]; p += 32) {
            __nv_bfloat16* e = plane + n * K + col[p];
            *e = __float2bfloat16_rn(__bfloat162float(*e) + 1.0f);
        }
}

// sx[m] = sum_k X[m,k], one warp per row, fp32
__global__ void __launch_bounds__(256)
rowsum_x(const __nv_bfloat16* __restrict__ X, int64_t M, int64_t K, int64_t ldx, float* __restrict__ sx) {
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * 8;
    for (int64_t m = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5); m < M; m += warps) {
        const uint4* row = reinterpret_cast<const uint4*>(X + m * ldx);
        float s = 0.f;
        for (int64_t i = lane; i < K / 8; i += 32) {
            const uint4 v = row[i];
            const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int j = 0; j < 4; ++j) s += __uint_as_float(w[j] << 16) + __uint_as_float(w[j] & 0xffff0000u);
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (lane == 0) sx[m] = s;
    }
}

// ---------------------------------------------------------------- host side

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 [rows, K] with row stride ld elements; box = 64 (k) x 128 (rows), 128-byte swizzle, out-of-range reads as zero
inline bool make_map(CUtensorMap* tm, const void* base, int64_t rows, int64_t K, int64_t ld) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)K, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, (cuuint32_t)kBM};
    const cuuint32_t estr[2] = {1, 1};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

struct Layout {
    size_t codes_off, plane_off, plane_bytes, sx_off, total;
};

// Sums the per-CTA squared errors in double precision and in a fixed order: thread t adds the CTAs t, t + 256, ...
// and the 256 thread sums are folded by a tree.  loss[i] = L_{rs[i]}, loss[n_r] = sum_i lambda_i L_i.
struct LossArgs {
    float lambda[kMaxR];
    int n_r;
};
__global__ void __launch_bounds__(256) loss_reduce(const float* __restrict__ part, int64_t n_cta, LossArgs A, double* __restrict__ loss) {
    __shared__ double s[256];
    double total = 0.0;
    for (int i = 0; i < A.n_r; ++i) {
        double v = 0.0;
        for (int64_t c = threadIdx.x; c < n_cta; c += 256) v += (double)part[c * kMaxR + i];
        s[threadIdx.x] = v;
        __syncthreads();
        for (int o = 128; o > 0; o >>= 1) {
            if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
            __syncthreads();
        }
        if (threadIdx.x == 0) { loss[i] = s[0]; total += (double)A.lambda[i] * s[0]; }
        __syncthreads();
    }
    if (threadIdx.x == 0) loss[A.n_r] = total;
}

inline Layout layout(int src_kind, int64_t M, int64_t N, int64_t K, int n_r) {
    Layout L;
    size_t off = 0;
    L.codes_off = off;
    if (src_kind == MATQ_SRC_BF16) off += align_up((size_t)N * K, 1024);
    L.plane_off = off;
    L.plane_bytes = align_up((size_t)N * K * 2, 1024);
    off += L.plane_bytes * (size_t)n_r;
    L.sx_off = off;
    off += align_up((size_t)M * sizeof(float), 1024);
    L.total = off;
    return L;
}

}  // namespace gm
}  // namespace matq

extern "C" size_t matq_gemm_multi_workspace_bytes(int src_kind, int64_t M, int64_t N, int64_t K, int n_r) {
    if (M < 0 || N < 0 || K <= 0 || n_r < 1 || n_r > matq::gm::kMaxR || src_kind < MATQ_SRC_BF16 || src_kind > MATQ_SRC_PACKED)
        return 0;
    return matq::gm::layout(src_kind, M, N, K, n_r).total;
}

namespace matq {
namespace gm {
// Loss partials live behind the forward's workspace, 256-byte aligned.
inline size_t loss_part_off(const Layout& L) { return (L.total + 255) / 256 * 256; }
inline int64_t cta_count(int64_t M, int64_t N, int n_r) {
    const int64_t cta_n = (n_r == 1 && N > kBN) ? 2 * kBN : kBN;
    return ((M + kBM - 1) / kBM) * ((N + cta_n - 1) / cta_n);
}
}  // namespace gm
}  // namespace matq

// Tests of the error path (matq_gemm_multi_test_stall): process-wide, read when a call builds its launch.
static std::atomic<int> g_test_stall{0};

extern "C" int matq_gemm_multi_test_stall(int on) { return g_test_stall.exchange(on ? 1 : 0); }

// The forward (Y != NULL, Yt == NULL) or the loss (Yt != NULL, loss_part != NULL; nothing is stored to Y).
static int gemm_multi_impl(int src_kind, const void* Wsrc, int64_t N, int64_t K, int c,
                           float* alpha, float* zero, int extra_precision,
                           const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                           const void* X, int64_t M, int64_t ldx,
                           const int* rs, int n_r, float* const* Y, int64_t ldy,
                           const float* Yt, int64_t ldt, float* loss_part, const int* teacher,
                           void* workspace, size_t workspace_bytes,
                           int32_t* dev_status, void* stream) {
    using namespace matq;
    using namespace matq::gm;
    if (M < 0 || N < 0 || K <= 0 || !rs || (!Y && !Yt) || n_r < 1 || n_r > kMaxR) return MATQ_ERR_INVALID_ARG;
    if (src_kind < MATQ_SRC_BF16 || src_kind > MATQ_SRC_PACKED) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits) return MATQ_ERR_UNSUPPORTED;
    for (int i = 0; i < n_r; ++i) {
        if (rs[i] < 1 || rs[i] > c) return MATQ_ERR_UNSUPPORTED;
        for (int j = 0; j < i; ++j) if (rs[j] == rs[i]) return MATQ_ERR_INVALID_ARG;
    }
    if (src_kind == MATQ_SRC_PACKED) {
        if (n_r != 1) return MATQ_ERR_INVALID_ARG;
        if (!(rs[0] == 8 || rs[0] == 4 || rs[0] == 2)) return MATQ_ERR_UNSUPPORTED;
        if ((ovf_row_ptr == nullptr) != (ovf_col == nullptr)) return MATQ_ERR_INVALID_ARG;
    }
    if (K % kBK != 0 || N % 8 != 0 || ldx < K || ldx % 8 != 0 || (Y && ldy < N) || (Yt && ldt < N)) return MATQ_ERR_SHAPE;
    if (M == 0 || N == 0) return MATQ_OK;
    if (!Wsrc || !alpha || !zero || !X) return MATQ_ERR_INVALID_ARG;
    if (Y) for (int i = 0; i < n_r; ++i) if (!Y[i]) return MATQ_ERR_INVALID_ARG;
    if (!aligned16(Wsrc) || !aligned16(X)) return MATQ_ERR_ALIGNMENT;
    const Layout L = layout(src_kind, M, N, K, n_r);
    if (!workspace || workspace_bytes < L.total) return MATQ_ERR_WORKSPACE;
    if ((reinterpret_cast<uintptr_t>(workspace) & 255u) != 0) return MATQ_ERR_ALIGNMENT;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    unsigned char* ws = static_cast<unsigned char*>(workspace);
    const int sms = sm_count();

    // 1. codes
    const uint8_t* codes = nullptr;
    if (src_kind == MATQ_SRC_BF16) {
        uint8_t* q = ws + L.codes_off;
        const int st = matq_quantize(Wsrc, N, K, K, c, q, alpha, zero, dev_status, stream);
        if (st != MATQ_OK) return st;
        codes = q;
    } else if (src_kind == MATQ_SRC_CODES8) {
        codes = static_cast<const uint8_t*>(Wsrc);
    }

    // 2. bf16 planes of fields
    ExpandArgs EA;
    EA.n_r = n_r;
    EA.extra_precision = extra_precision ? 1 : 0;
    for (int i = 0; i < kMaxR; ++i) {
        EA.plane[i] = reinterpret_cast<__nv_bfloat16*>(ws + L.plane_off + (size_t)(i < n_r ? i : 0) * L.plane_bytes);
        EA.r[i] = rs[i < n_r ? i : 0];
    }
    if (codes) {
        const int64_t nchunks = N * K / 16;                  // K % 64 == 0
        int64_t blocks = (nchunks + 255) / 256;
        if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
        expand_codes<<<(unsigned)blocks, 256, 0, s>>>(reinterpret_cast<const uint4*>(codes), nchunks, EA);
    } else {
        const int64_t nvec = N * K * rs[0] / 128;            // K % 64 == 0: rows are whole 16-byte pieces for r = 8, 4, 2
        int64_t blocks = (nvec + 255) / 256;
        if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
        const uint4* pk = static_cast<const uint4*>(Wsrc);
        if (rs[0] == 8) expand_packed<8><<<(unsigned)blocks, 256, 0, s>>>(pk, nvec, EA.plane[0]);
        else if (rs[0] == 4) expand_packed<4><<<(unsigned)blocks, 256, 0, s>>>(pk, nvec, EA.plane[0]);
        else expand_packed<2><<<(unsigned)blocks, 256, 0, s>>>(pk, nvec, EA.plane[0]);
        if (extra_precision && ovf_row_ptr) {
            int64_t b2 = (N + 7) / 8;
            if (b2 > (int64_t)sms * 16) b2 = (int64_t)sms * 16;
            add_overflow<<<(unsigned)b2, 256, 0, s>>>(ovf_row_ptr, ovf_col, N, K, EA.plane[0]);
        }
    }

    // 3. row sums of X
    float* sx = reinterpret_cast<float*>(ws + L.sx_off);
    {
        int64_t blocks = (M + 7) / 8;
        if (blocks > (int64_t)sms * 16) blocks = (int64_t)sms * 16;
        rowsum_x<<<(unsigned)blocks, 256, 0, s>>>(static_cast<const __nv_bfloat16*>(X), M, K, ldx, sx);
    }
    if (launch_status() != MATQ_OK) return MATQ_ERR_CUDA;

    // 4. GEMM
    CUtensorMap tm_x, tm_b[kMaxR];
    if (!make_map(&tm_x, X, M, K, ldx)) return MATQ_ERR_CUDA;
    for (int i = 0; i < kMaxR; ++i)
        if (!make_map(&tm_b[i], EA.plane[i], N, K, K)) return MATQ_ERR_CUDA;
    Params P;
    P.alpha = alpha; P.zero = zero; P.sx = sx;
    for (int i = 0; i < kMaxR; ++i) { P.Y[i] = Y ? Y[i < n_r ? i : 0] : nullptr; P.sh[i] = c - rs[i < n_r ? i : 0]; }
    P.Yt = Yt; P.ldt = ldt; P.loss_part = loss_part;
    for (int i = 0; i < kMaxR; ++i) P.teacher[i] = (teacher && i < n_r) ? teacher[i] : -1;
    P.M = M; P.N = N; P.K = K; P.ldy = ldy; P.n_r = n_r;
    P.dev_status = dev_status;
    P.hold = g_test_stall.load(std::memory_order_relaxed) ? 1 : 0;
    P.wait_cycles = P.hold ? kStallWaitCycles : kWaitCycles;
    // A single plane would leave every MMA at N = 128 (shared-memory bound); the CTA then takes 256 channels as two
    // adjacent tiles of the same plane so that one N = 256 instruction covers them.
    P.wide = (n_r == 1 && N > kBN) ? 1 : 0;
    if (P.wide) { P.n_r = 2; tm_b[1] = tm_b[0]; n_r = 2; }
    const int cta_n = P.wide ? 2 * kBN : kBN;
    const int stage_bytes = (1 + n_r) * kTileBytes;
    int stages = (200 * 1024) / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    P.stages = stages;
    const size_t smem = (size_t)stages * stage_bytes + 1024;
    static std::atomic<unsigned long long> smem_ok{0};
    if (!matq::opt_in_max_smem(gemm_multi_kernel, smem_ok)) return MATQ_ERR_CUDA;
    const dim3 grid((unsigned)((M + kBM - 1) / kBM), (unsigned)((N + cta_n - 1) / cta_n), 1);
    gemm_multi_kernel<<<grid, kThreads, smem, s>>>(tm_x, tm_b[0], tm_b[1], tm_b[2], P);
    return launch_status();
}

extern "C" int matq_gemm_multi(int src_kind, const void* Wsrc, int64_t N, int64_t K, int c,
                               float* alpha, float* zero, int extra_precision,
                               const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                               const void* X, int64_t M, int64_t ldx,
                               const int* rs, int n_r, float* const* Y, int64_t ldy,
                               void* workspace, size_t workspace_bytes,
                               int32_t* dev_status, void* stream) {
    if (!Y) return MATQ_ERR_INVALID_ARG;
    return gemm_multi_impl(src_kind, Wsrc, N, K, c, alpha, zero, extra_precision, ovf_row_ptr, ovf_col, X, M, ldx, rs, n_r,
                           Y, ldy, nullptr, 0, nullptr, nullptr, workspace, workspace_bytes, dev_status, stream);
}

extern "C" size_t matq_gemm_multi_loss_workspace_bytes(int src_kind, int64_t M, int64_t N, int64_t K, int n_r) {
    using namespace matq::gm;
    if (M < 0 || N < 0 || K <= 0 || n_r < 1 || n_r > kMaxR || src_kind < MATQ_SRC_BF16 || src_kind > MATQ_SRC_PACKED)
        return 0;
    return loss_part_off(layout(src_kind, M, N, K, n_r)) + (size_t)cta_count(M, N, n_r) * kMaxR * sizeof(float);
}

extern "C" int matq_gemm_multi_loss(int src_kind, const void* Wsrc, int64_t N, int64_t K, int c,
                                    float* alpha, float* zero, int extra_precision,
                                    const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                                    const void* X, int64_t M, int64_t ldx,
                                    const int* rs, int n_r, const float* lambda, const int* teacher,
                                    const float* Yt, int64_t ldt, double* loss,
                                    void* workspace, size_t workspace_bytes,
                                    int32_t* dev_status, void* stream) {
    using namespace matq;
    using namespace matq::gm;
    if (!lambda || !loss || !Yt || n_r < 1 || n_r > kMaxR || M < 0 || N < 0 || K <= 0) return MATQ_ERR_INVALID_ARG;
    if (src_kind < MATQ_SRC_BF16 || src_kind > MATQ_SRC_PACKED) return MATQ_ERR_INVALID_ARG;
    if (teacher)
        for (int i = 0; i < n_r; ++i) {
            const int j = teacher[i] >= 256 ? teacher[i] - 256 : teacher[i];
            if (teacher[i] < -1 || j >= n_r || j == i) return MATQ_ERR_INVALID_ARG;
        }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (M == 0 || N == 0)                                        // nothing to compare: every loss is zero
        return cudaMemsetAsync(loss, 0, (size_t)(n_r + 1) * sizeof(double), s) == cudaSuccess ? MATQ_OK : MATQ_ERR_CUDA;
    const size_t need = matq_gemm_multi_loss_workspace_bytes(src_kind, M, N, K, n_r);
    if (!workspace || workspace_bytes < need) return MATQ_ERR_WORKSPACE;
    const Layout L = layout(src_kind, M, N, K, n_r);
    float* part = reinterpret_cast<float*>(static_cast<unsigned char*>(workspace) + loss_part_off(L));
    const int st = gemm_multi_impl(src_kind, Wsrc, N, K, c, alpha, zero, extra_precision, ovf_row_ptr, ovf_col, X, M, ldx,
                                   rs, n_r, nullptr, 0, Yt, ldt, part, teacher, workspace, L.total, dev_status, stream);
    if (st != MATQ_OK) return st;
    LossArgs A;
    A.n_r = n_r;
    for (int i = 0; i < kMaxR; ++i) A.lambda[i] = i < n_r ? lambda[i] : 0.f;
    loss_reduce<<<1, 256, 0, s>>>(part, cta_count(M, N, n_r), A, loss);
    return launch_status();
}
