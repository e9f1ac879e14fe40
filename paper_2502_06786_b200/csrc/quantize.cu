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
// contracted into FMAs), so the codes are reproducible bit for bit.
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

__device__ __forceinline__ void scale_zero(const RowRange& rr, float& a, float& z) {
    const float range = __fsub_rn(rr.mx, rr.mn);
    a = (range > 0.0f) ? __fdiv_rn(range, 255.0f) : 1.0f;
    z = __fdiv_rn(-rr.mn, a);
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

// Fast path: K % 16 == 0, rows 16-byte aligned.  Dynamic shared memory: K * 2 bytes.
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_vec(const uint16_t* __restrict__ W, int64_t N, int K, int64_t ldw,
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
        const RowRange rr = block_range(mn, mx, bad);   // its barriers also publish row_s
        float a, z;
        scale_zero(rr, a, z);
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

// Any K, ldw, alignment: scalar loads, the row is read twice (second pass usually from L2).
__global__ void __launch_bounds__(kQuantThreads)
quantize_rows_generic(const uint16_t* __restrict__ W, int64_t N, int64_t K, int64_t ldw,
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
        const RowRange rr = block_range(mn, mx, bad);
        float a, z;
        scale_zero(rr, a, z);
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
    using namespace matq;
    if (N < 0 || K <= 0 || ldw < K || (N > 0 && (!W || !alpha || !zero))) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits) return MATQ_ERR_UNSUPPORTED;
    if (N == 0) return MATQ_OK;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const bool fast = aligned16(W) && (K % 16 == 0) && (ldw % 8 == 0) && K <= 65536 &&
                      (q == nullptr || aligned16(q));
    const int sms = sm_count();
    if (fast) {
        const size_t smem = (size_t)K * 2;
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(quantize_rows_vec, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
            return MATQ_ERR_CUDA;
        int per_sm = (int)((200u * 1024u) / (smem + 1024));
        per_sm = per_sm < 1 ? 1 : (per_sm > 8 ? 8 : per_sm);
        const int64_t grid = N < (int64_t)sms * per_sm ? N : (int64_t)sms * per_sm;
        quantize_rows_vec<<<(unsigned)grid, kQuantThreads, smem, s>>>(
            static_cast<const uint16_t*>(W), N, (int)K, ldw, q, alpha, zero, dev_status);
    } else {
        const int64_t grid = N < (int64_t)sms * 8 ? N : (int64_t)sms * 8;
        quantize_rows_generic<<<(unsigned)grid, kQuantThreads, 0, s>>>(
            static_cast<const uint16_t*>(W), N, K, ldw, q, alpha, zero, dev_status);
    }
    return launch_status();
}
