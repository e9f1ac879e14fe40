// matq_quantize: per-output-channel MinMax quantisation (Eq. 1).
//
// One CTA owns one row at a time.  The row is read from HBM once: while its
// 16-byte chunks stream in they are parked in shared memory and folded into
// the running min / max; after a block reduction every thread forms alpha and
// z and the codes are produced from the shared-memory copy.  Traffic is the
// algorithmic 2 bytes read + 1 byte written per weight.
//
// The arithmetic of Eq. 1 is pinned to IEEE binary32 with one correctly
// rounded operation per step (__fdiv_rn / __fadd_rn / __fsub_rn are never
// contracted into FMAs), so the codes are reproducible bit for bit.  The
// register-resident kernel reaches the same bits through a sequence of fused
// multiply-adds that reproduces each of those roundings (see RowFast).
#include "common.cuh"

namespace matq {
namespace {

constexpr int kQuantThreads = 256;

__device__ __forceinline__ float code_from_weight(float w, float a, float z) {
    const float t = __fdiv_rn(w, a);
    const float u = __fadd_rn(t, z);
    const float fl = floorf(u);
    const float frac = __fsub_rn(u, fl);          // exact for |u| < 2^23
    float r = (frac >= 0.5f) ? __fadd_rn(fl, 1.0f) : fl;   // round half up
    r = fminf(fmaxf(r, 0.0f), 255.0f);
    return r;
}

struct RowRange {
    float mn, mx;
    int bad;
};

// Block-wide min / max / any(non-finite); result valid in every thread.
__device__ __forceinline__ RowRange block_range(float mn, float mx, int bad) {
    __shared__ float s_mn[kQuantThreads / 32], s_mx[kQuantThreads / 32];
    __shared__ int s_bad[kQuantThreads / 32];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        bad |= __shfl_xor_sync(0xffffffffu, bad, o);
    }
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    __syncthreads();                              // previous row's readers are done with s_*
    if (lane == 0) { s_mn[warp] = mn; s_mx[warp] = mx; s_bad[warp] = bad; }
    __syncthreads();
    RowRange r{s_mn[0], s_mx[0], s_bad[0]};
#pragma unroll
    for (int w = 1; w < kQuantThreads / 32; ++w) {
        r.mn = fminf(r.mn, s_mn[w]);
        r.mx = fmaxf(r.mx, s_mx[w]);
        r.bad |= s_bad[w];
    }
    return r;
}

// alpha and z of Eq. 3 from the row's extremes and its clipping scales (g = b = 1 is Eq. 1 exactly: the products
// are then exact).  One correctly rounded operation per step, in the order the header states.
__device__ __forceinline__ void scale_zero(const RowRange& rr, float g, float b, float& a, float& z) {
    const float hi = __fmul_rn(g, rr.mx), lo = __fmul_rn(b, rr.mn);
    const float range = __fsub_rn(hi, lo);
    a = (range > 0.0f) ? __fdiv_rn(range, 255.0f) : 1.0f;
    z = __fdiv_rn(-lo, a);
}

// Clipping scales of row n (absent = 1); a non-finite scale marks the row bad like a non-finite weight.
__device__ __forceinline__ void row_scales(const float* __restrict__ gamma, const float* __restrict__ beta, int64_t n,
                                           float& g, float& b, int& bad) {
    g = gamma ? gamma[n] : 1.0f;
    b = beta ? beta[n] : 1.0f;
    bad |= !(fabsf(g) <= 3.4e38f) | !(fabsf(b) <= 3.4e38f);
}

__device__ __forceinline__ void fold_word(uint32_t w, float& mn, float& mx, int& bad) {
    const float lo = __uint_as_float(w << 16);
    const float hi = __uint_as_float(w & 0xffff0000u);
    mn = fminf(mn, fminf(lo, hi));
    mx = fmaxf(mx, fmaxf(lo, hi));
    bad |= ((w & 0x7f80u) == 0x7f80u) | ((w & 0x7f800000u) == 0x7f800000u);
}

__device__ __forceinline__ uint32_t codes_from_words(uint32_t w0, uint32_t w1, float a, float z) {
    const uint32_t c0 = (uint32_t)code_from_weight(__uint_as_float(w0 << 16), a, z);
    const uint32_t c1 = (uint32_t)code_from_weight(__uint_as_float(w0 & 0xffff0000u), a, z);
    const uint32_t c2 = (uint32_t)code_from_weight(__uint_as_float(w1 << 16), a, z);
    const uint32_t c3 = (uint32_t)code_from_weight(__uint_as_float(w1 & 0xffff0000u), a, z);
    return c0 | (c1 << 8) | (c2 << 16) | (c3 << 24);
}

// ---- the same codes without the special-function pipe ---------------------------------------------------------
// Per element the pinned arithmetic needs a division, a floor and a float->int conversion, all of which issue on
// the quarter-rate special-function pipe and bound the kernel.  The fast path below produces the SAME codes with
// fused multiply-adds only, by reproducing every rounding of the pinned sequence:
//   t = RN(w / alpha) from ra = RN(1 / alpha) (once per row) by two residual corrections
//         q0 = RN(w ra),  r0 = w - q0 alpha (exact in an FMA),  q1 = RN(q0 + r0 ra)     (q1 is a faithful quotient)
//         r1 = w - q1 alpha (exact),  t = RN(q1 + r1 ra)
//       which is the correctly rounded quotient (Markstein's theorem: a faithful quotient corrected once with the
//       exact residual and a correctly rounded reciprocal rounds correctly; rows whose alpha has an all-ones
//       significand, the theorem's one exception, take the pinned path).  An FMA residual is only inexact when it
//       underflows, i.e. for |w| below 2^-100: such a t is too small to move u = RN(t + z) across a rounding boundary.
//   u = RN(t + z), exactly the pinned u.
//   m = RN(u + 1.5 * 2^23) holds u rounded to the nearest-even integer in its low mantissa bits; u - (m - 1.5 * 2^23)
//       is exact, and it equals +1/2 exactly when u was a tie that nearest-even rounded DOWN: round half up (the
//       pinned rule) then gives one more.  Inside [0, 255] the code is the low byte of m's bit pattern, and u lies
//       in [-2^-16, 255 + 2^-7] by construction of alpha and z, so no clamp and no conversion are needed.
// Unlike a guard-band scheme this has no data-dependent fallback: with bf16 weights 0.2 % of the elements sit
// exactly on a tie, enough to send a third of all warps down a divergent slow path.
struct RowFast {
    float a, z, ra;
    bool ok;        // false: the row is outside the fast path's domain and takes the pinned sequence
};

__device__ __forceinline__ RowFast row_fast(float a, float z, float mn, float mx, int bad) {
    RowFast f{a, z, 0.f, false};
    const float big = fmaxf(fabsf(mn), fabsf(mx));
    if (!bad && a > 1e-30f && a < 1e30f && fabsf(z) < 1048576.0f && big < 1e30f &&
        (__float_as_uint(a) & 0x007fffffu) != 0x007fffffu) {
        f.ra = __frcp_rn(a);
        f.ok = big * f.ra * 1.0001f + fabsf(z) < 2097152.0f;      // |u| < 2^21: the rounding trick is exact
    }
    return f;
}

// Two fp32 lanes per instruction (sm_100 packed arithmetic; each lane rounds exactly like the scalar instruction).
__device__ __forceinline__ uint64_t f2_pack(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void f2_unpack(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t f2_fma(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t f2_mul(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_add(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ uint64_t f2_sub(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Eight codes of one 16-byte piece by the fast sequence, the two bf16 halves of a word side by side.  CLIP: Eq. 3's
// scales can put u outside [0, 255]; rounding is monotone, so clamping u first gives the clamped code.
template <bool CLIP>
__device__ __forceinline__ uint2 codes8_fast(const uint4& v, const RowFast& f) {
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
    const uint64_t ra2 = f2_pack(f.ra, f.ra), na2 = f2_pack(-f.a, -f.a), z2 = f2_pack(f.z, f.z);
    const uint64_t c2 = f2_pack(12582912.0f, 12582912.0f);               // 1.5 * 2^23
    uint32_t mb[8];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint64_t x = f2_pack(__uint_as_float(w[j] << 16), __uint_as_float(w[j] & 0xffff0000u));
        uint64_t q = f2_mul(x, ra2);
        q = f2_fma(f2_fma(q, na2, x), ra2, q);
        const uint64_t t = f2_fma(f2_fma(q, na2, x), ra2, q);            // = RN(x / alpha)
        uint64_t u = f2_add(t, z2);
        if (CLIP) {
            float u0, u1;
            f2_unpack(u, u0, u1);
            u = f2_pack(fminf(fmaxf(u0, 0.0f), 255.0f), fminf(fmaxf(u1, 0.0f), 255.0f));
        }
        const uint64_t m = f2_add(u, c2);
        const uint64_t d = f2_sub(u, f2_sub(m, c2));
        float m0, m1, d0, d1;
        f2_unpack(m, m0, m1);
        f2_unpack(d, d0, d1);
        mb[2 * j] = __float_as_uint(m0) + (d0 == 0.5f ? 1u : 0u);
        mb[2 * j + 1] = __float_as_uint(m1) + (d1 == 0.5f ? 1u : 0u);
    }
    const uint32_t lo = __byte_perm(__byte_perm(mb[0], mb[1], 0x0040), __byte_perm(mb[2], mb[3], 0x0040), 0x5410);
    const uint32_t hi = __byte_perm(__byte_perm(mb[4], mb[5], 0x0040), __byte_perm(mb[6], mb[7], 0x0040), 0x5410);
    return make_uint2(lo, hi);
}

// Fast path: K % 16 == 0, rows 16-byte aligned.  Dynamic shared memory: K * 2 bytes.
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_vec(const uint16_t* __restrict__ W, int64_t N, int K, int64_t ldw,
                  const float* __restrict__ gamma, const float* __restrict__ beta,
                  uint8_t* __restrict__ q, float* __restrict__ alpha, float* __restrict__ zero,
                  int32_t* dev_status) {
    extern __shared__ uint4 row_s[];
    const int nvec = K >> 3;
    for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
        const uint4* src = reinterpret_cast<const uint4*>(W + n * ldw);
        float mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);
        int bad = 0;
        for (int i = threadIdx.x; i < nvec; i += kQuantThreads) {
            const uint4 v = ld_stream_u4(src + i);
            row_s[i] = v;
            fold_word(v.x, mn, mx, bad);
            fold_word(v.y, mn, mx, bad);
            fold_word(v.z, mn, mx, bad);
            fold_word(v.w, mn, mx, bad);
        }
        RowRange rr = block_range(mn, mx, bad);         // its barriers also publish row_s
        float a, z, g, b;
        row_scales(gamma, beta, n, g, b, rr.bad);
        scale_zero(rr, g, b, a, z);
        if (threadIdx.x == 0) {
            if (rr.bad) report(dev_status, MATQ_ERR_NONFINITE);
            alpha[n] = a;
            zero[n] = z;
        }
        if (q) {
            uint4* dst = reinterpret_cast<uint4*>(q + n * (int64_t)K);
            for (int i = threadIdx.x; i < (nvec >> 1); i += kQuantThreads) {
                const uint4 v0 = row_s[2 * i], v1 = row_s[2 * i + 1];
                uint4 o;
                o.x = codes_from_words(v0.x, v0.y, a, z);
                o.y = codes_from_words(v0.z, v0.w, a, z);
                o.z = codes_from_words(v1.x, v1.y, a, z);
                o.w = codes_from_words(v1.z, v1.w, a, z);
                dst[i] = o;
            }
        }
        __syncthreads();                           // row_s is reused by the next row
    }
}

// Range of two bf16 values at a time: packed min / max that PROPAGATE NaN, so a NaN anywhere ends up in the running
// pair and an Inf is the extreme itself: non-finite weights are detected once per thread from the four folded
// values instead of once per weight.
__device__ __forceinline__ void fold_word2(uint32_t w, uint32_t& mn2, uint32_t& mx2) {
    asm("min.NaN.bf16x2 %0, %0, %1;" : "+r"(mn2) : "r"(w));
    asm("max.NaN.bf16x2 %0, %0, %1;" : "+r"(mx2) : "r"(w));
}

// Register-resident path (K <= 16384, K % 8 == 0): a team of 32 * WPR threads owns a row and keeps it in registers
// (NV 16-byte pieces per thread), so the row is read once, never touches shared memory, and every thread both
// folds the range and emits codes.  A CTA of 8 warps works on 8 / WPR rows at a time.
template <int NV, int WARPS, bool CLIP>
__global__ void __launch_bounds__(WARPS * 32, (NV <= 5 ? 32 : NV <= 9 ? 24 : 16) / WARPS)
quantize_rows_reg(const uint16_t* __restrict__ W, int64_t N, int K, int64_t ldw, int wpr,
                  const float* __restrict__ gamma, const float* __restrict__ beta,
                  uint8_t* __restrict__ q, float* __restrict__ alpha, float* __restrict__ zero,
                  int32_t* dev_status) {
    __shared__ float s_mn[WARPS], s_mx[WARPS];
    __shared__ int s_bad[WARPS];
    let_next_kernel_start();
    after_previous_kernel();
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int rows_per_cta = (WARPS) / wpr;
    const int team = warp / wpr, team_tid = (warp % wpr) * 32 + lane, team_threads = 32 * wpr;
    const int nvec = K >> 3;
    for (int64_t n_base = (int64_t)blockIdx.x * rows_per_cta; n_base < N; n_base += (int64_t)gridDim.x * rows_per_cta) {
        const int64_t n = n_base + team;
        const bool live = n < N;
        uint4 v[NV];
        uint32_t mn2 = 0x7f807f80u, mx2 = 0xff80ff80u;                // +Inf / -Inf pairs
        if (live) {
            const uint4* src = reinterpret_cast<const uint4*>(W + n * ldw);
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                const int i = team_tid + j * team_threads;
                if (i < nvec) v[j] = ld_stream_u4(src + i);
            }
#pragma unroll
            for (int j = 0; j < NV; ++j) {
                const int i = team_tid + j * team_threads;
                if (i < nvec) {
                    fold_word2(v[j].x, mn2, mx2);
                    fold_word2(v[j].y, mn2, mx2);
                    fold_word2(v[j].z, mn2, mx2);
                    fold_word2(v[j].w, mn2, mx2);
                }
            }
        }
        // a thread that folded at least one piece (team_tid < nvec) sees +-Inf or NaN here only from a weight
        const float mn_a = __uint_as_float(mn2 << 16), mn_b = __uint_as_float(mn2 & 0xffff0000u);
        const float mx_a = __uint_as_float(mx2 << 16), mx_b = __uint_as_float(mx2 & 0xffff0000u);
        float mn = fminf(mn_a, mn_b);
        float mx = fmaxf(mx_a, mx_b);
        int bad = live && team_tid < nvec && (!(fabsf(mn_a) <= 3.4e38f) | !(fabsf(mn_b) <= 3.4e38f) | !(fabsf(mx_a) <= 3.4e38f) | !(fabsf(mx_b) <= 3.4e38f));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
            mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
            bad |= __shfl_xor_sync(0xffffffffu, bad, o);
        }
        if (wpr > 1) {                                    // uniform over the CTA
            __syncthreads();                              // the previous round's readers are done
            if (lane == 0) { s_mn[warp] = mn; s_mx[warp] = mx; s_bad[warp] = bad; }
            __syncthreads();
            for (int w = 0; w < wpr; ++w) {
                mn = fminf(mn, s_mn[team * wpr + w]);
                mx = fmaxf(mx, s_mx[team * wpr + w]);
                bad |= s_bad[team * wpr + w];
            }
        }
        if (!live) continue;
        float a, z, g, b;
        row_scales(gamma, beta, n, g, b, bad);
        RowRange rr{mn, mx, bad};
        scale_zero(rr, g, b, a, z);
        if (team_tid == 0) {
            if (bad) report(dev_status, MATQ_ERR_NONFINITE);
            alpha[n] = a;
            zero[n] = z;
        }
        if (q) {
            uint2* dst = reinterpret_cast<uint2*>(q + n * (int64_t)K);
            const RowFast f = row_fast(a, z, mn, mx, bad);
            if (f.ok) {                                       // uniform over the row's team
#pragma unroll
                for (int j = 0; j < NV; ++j) {
                    const int i = team_tid + j * team_threads;
                    if (i < nvec) dst[i] = codes8_fast<CLIP>(v[j], f);
                }
            } else {
#pragma unroll 1
                for (int i = team_tid; i < nvec; i += team_threads) {    // rare: re-read the row, pinned sequence
                    const uint4 wv = ld_stream_u4(reinterpret_cast<const uint4*>(W + n * ldw) + i);
                    dst[i] = make_uint2(codes_from_words(wv.x, wv.y, a, z), codes_from_words(wv.z, wv.w, a, z));
                }
            }
        }
    }
}

// Any K, ldw, alignment: scalar loads, the row is read twice (second pass usually from L2).
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_generic(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw,
                      const float* __restrict__ gamma, const float* __restrict__ beta,
                      uint8_t* __restrict__ q, float* __restrict__ alpha, float* __restrict__ zero,
                      int32_t* dev_status) {
    for (int64_t n = blockIdx.x; n < N; n += gridDim.x) {
        const uint16_t* src = W + n * ldw;
        float mn = __int_as_float(0x7f800000), mx = __int_as_float(0xff800000);
        int bad = 0;
        for (int64_t k = threadIdx.x; k < K; k += kQuantThreads) {
            const uint32_t b = src[k];
            const float w = __uint_as_float(b << 16);
            mn = fminf(mn, w);
            mx = fmaxf(mx, w);
            bad |= ((b & 0x7f80u) == 0x7f80u);
        }
        RowRange rr = block_range(mn, mx, bad);
        float a, z, g, b;
        row_scales(gamma, beta, n, g, b, rr.bad);
        scale_zero(rr, g, b, a, z);
        if (threadIdx.x == 0) {
            if (rr.bad) report(dev_status, MATQ_ERR_NONFINITE);
            alpha[n] = a;
            zero[n] = z;
        }
        if (q)
            for (int64_t k = threadIdx.x; k < K; k += kQuantThreads)
                q[n * K + k] = (uint8_t)code_from_weight(__uint_as_float((uint32_t)src[k] << 16), a, z);
    }
}

}  // namespace
}  // namespace matq

extern "C" int matq_quantize(const void* W, int64_t N, int64_t K, int64_t ldw, int c,
                             uint8_t* q, float* alpha, float* zero,
                             int32_t* dev_status, void* stream) {
    return matq_quantize_clip(W, N, K, ldw, c, nullptr, nullptr, q, alpha, zero, dev_status, stream);
}

extern "C" int matq_quantize_clip(const void* W, int64_t N, int64_t K, int64_t ldw, int c,
                                  const float* gamma, const float* beta,
                                  uint8_t* q, float* alpha, float* zero,
                                  int32_t* dev_status, void* stream) {
    using namespace matq;
    const bool clip = gamma != nullptr || beta != nullptr;
    if (N < 0 || K <= 0 || ldw < K || (N > 0 && (!W || !alpha || !zero))) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits) return MATQ_ERR_UNSUPPORTED;
    if (N == 0) return MATQ_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int sms = sm_count();
    const uint16_t* Wb = static_cast<const uint16_t*>(W);
    const bool reg = aligned16(W) && (K % 8 == 0) && (ldw % 8 == 0) && K <= 16384 &&
                     (q == nullptr || (reinterpret_cast<uintptr_t>(q) & 7u) == 0);
    const bool fast = aligned16(W) && (K % 16 == 0) && (ldw % 8 == 0) && K <= 65536 &&
                      (q == nullptr || aligned16(q));
    if (reg) {
        const int nvec = (int)(K / 8);
        int wpr = 1;
        while (wpr < 8 && (nvec + 32 * wpr - 1) / (32 * wpr) > 9) wpr *= 2;
        const int nv = (nvec + 32 * wpr - 1) / (32 * wpr);
        // CTAs of 4 warps when a row's team fits (measured 5 % faster than 8: more CTAs per SM in different phases)
        const int warps = wpr <= 4 ? 4 : 8;
        const int rows_per_cta = warps / wpr;
        int64_t grid = (N + rows_per_cta - 1) / rows_per_cta;
        if (grid > (int64_t)sms * 32) grid = (int64_t)sms * 32;
#define MATQ_QUANT_REG(NV) do { \
        if (clip) { \
            if (warps == 4) launch_overlapped(quantize_rows_reg<NV, 4, true>, dim3((unsigned)grid), dim3(128), 0, s, Wb, N, (int)K, ldw, wpr, gamma, beta, q, alpha, zero, dev_status); \
            else launch_overlapped(quantize_rows_reg<NV, 8, true>, dim3((unsigned)grid), dim3(256), 0, s, Wb, N, (int)K, ldw, wpr, gamma, beta, q, alpha, zero, dev_status); \
        } else { \
            if (warps == 4) launch_overlapped(quantize_rows_reg<NV, 4, false>, dim3((unsigned)grid), dim3(128), 0, s, Wb, N, (int)K, ldw, wpr, gamma, beta, q, alpha, zero, dev_status); \
            else launch_overlapped(quantize_rows_reg<NV, 8, false>, dim3((unsigned)grid), dim3(256), 0, s, Wb, N, (int)K, ldw, wpr, gamma, beta, q, alpha, zero, dev_status); \
        } } while (0)
        if (nv <= 2) MATQ_QUANT_REG(2);
        else if (nv <= 3) MATQ_QUANT_REG(3);
        else if (nv <= 4) MATQ_QUANT_REG(4);
        else if (nv <= 5) MATQ_QUANT_REG(5);
        else if (nv <= 7) MATQ_QUANT_REG(7);
        else MATQ_QUANT_REG(9);
#undef MATQ_QUANT_REG
    } else if (fast) {
        const size_t smem = (size_t)K * 2;
        static std::atomic<unsigned long long> smem_ok{0};
        if (smem > 40 * 1024 &&   // the 48 KB default counts static shared memory too
            !opt_in_max_smem(quantize_rows_vec, smem_ok))
            return MATQ_ERR_CUDA;
        int per_sm = (int)((200u * 1024u) / (smem + 1024));
        per_sm = per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm);
        const int64_t grid = N < (int64_t)sms * per_sm ? N : (int64_t)sms * per_sm;
        quantize_rows_vec<<<(unsigned)grid, kQuantThreads, smem, s>>>(Wb, N, (int)K, ldw, gamma, beta, q, alpha, zero, dev_status);
    } else {
        const int64_t grid = N < (int64_t)sms * 8 ? N : (int64_t)sms * 8;
        quantize_rows_generic<<<(unsigned)grid, kQuantThreads, 0, s>>>(Wb, N, K, ldw, gamma, beta, q, alpha, zero, dev_status);
    }
    return launch_status();
}
