// Decode GEMV on the fp32 FMA pipes: y[b,n] = alpha_n (2^sh sum_k x[b,k] k_r[n,k] - z_n sum_k x[b,k]).
//
// One warp owns two rows at a time and strides over K in 16-byte chunks of the
// packed plane (128/r weights per lane and load).  Fields are unpacked with
// shifts and masks, converted to fp32 and accumulated with FMAs; the per-lane
// partial sums (and the partial sums of x for the zero-point term) are
// combined by a warp-shuffle tree, i.e. the split over K lives inside a warp
// and needs no scratch memory.  Extra-precision overflow columns add x[b,j]
// once more (their field is one higher than the stored, clamped one).
#pragma once
#include "common.cuh"

namespace matq {

constexpr int kGemvCcThreads = 256;
constexpr int kGemvCcRows = 2;

template <int R, int BT>
__global__ void __launch_bounds__(kGemvCcThreads)
gemv_cuda_core(const uint8_t* __restrict__ packed, int64_t N, int64_t K,
               const float* __restrict__ alpha, const float* __restrict__ zero,
               const int32_t* __restrict__ ovf_row_ptr, const uint16_t* __restrict__ ovf_col,
               const __nv_bfloat16* __restrict__ x, int B, int64_t ldx,
               float* __restrict__ y, int64_t ldy, bool pdl) {
    constexpr int kPerWord = 32 / R;            // fields per 32-bit word
    constexpr int kPerChunk = 4 * kPerWord;     // weights per 16-byte load
    constexpr uint32_t kMask = (1u << R) - 1u;
    constexpr int sh = kCodeBits - R;
    const int lane = threadIdx.x & 31;
    const int64_t chunks = K / kPerChunk;
    const int64_t row_bytes = K * R / 8;
    const int64_t warps = (int64_t)gridDim.x * (kGemvCcThreads / 32);
    if (pdl) {
        asm volatile("griddepcontrol.launch_dependents;");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    for (int b0 = 0; b0 < B; b0 += BT) {
        for (int64_t n0 = ((int64_t)blockIdx.x * (kGemvCcThreads / 32) + (threadIdx.x >> 5)) * kGemvCcRows; n0 < N;
             n0 += warps * kGemvCcRows) {
            float acc[kGemvCcRows][BT];
            float xs[BT];
#pragma unroll
            for (int b = 0; b < BT; ++b) {
                xs[b] = 0.f;
#pragma unroll
                for (int rr = 0; rr < kGemvCcRows; ++rr) acc[rr][b] = 0.f;
            }
            for (int64_t i = lane; i < chunks; i += 32) {
                uint32_t w[kGemvCcRows][4];
#pragma unroll
                for (int rr = 0; rr < kGemvCcRows; ++rr) {
                    uint4 v = make_uint4(0, 0, 0, 0);
                    if (n0 + rr < N) v = ld_stream_u4(packed + (n0 + rr) * row_bytes + i * 16);
                    w[rr][0] = v.x; w[rr][1] = v.y; w[rr][2] = v.z; w[rr][3] = v.w;
                }
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int64_t k0 = i * kPerChunk + j * kPerWord;
#pragma unroll
                    for (int b = 0; b < BT; ++b) {
                        const int bb = (b0 + b < B) ? b0 + b : B - 1;
                        const __nv_bfloat16* xp = x + bb * ldx + k0;
                        float xv[kPerWord];
#pragma unroll
                        for (int f = 0; f < kPerWord; f += 2) {
                            const uint32_t pr = *reinterpret_cast<const uint32_t*>(xp + f);
                            xv[f] = __uint_as_float(pr << 16);
                            xv[f + 1] = __uint_as_float(pr & 0xffff0000u);
                            xs[b] += xv[f] + xv[f + 1];
                        }
#pragma unroll
                        for (int rr = 0; rr < kGemvCcRows; ++rr)
#pragma unroll
                            for (int f = 0; f < kPerWord; ++f)
                                acc[rr][b] = fmaf((float)((w[rr][j] >> (f * R)) & kMask), xv[f], acc[rr][b]);
                    }
                }
            }
            if (ovf_row_ptr) {
#pragma unroll
                for (int rr = 0; rr < kGemvCcRows; ++rr) {
                    if (n0 + rr >= N) continue;
                    const int32_t e = ovf_row_ptr[n0 + rr + 1];
                    for (int32_t p = ovf_row_ptr[n0 + rr] + lane; p < e; p += 32) {
                        const int col = ovf_col[p];
#pragma unroll
                        for (int b = 0; b < BT; ++b) {
                            const int bb = (b0 + b < B) ? b0 + b : B - 1;
                            acc[rr][b] += __bfloat162float(x[bb * ldx + col]);
                        }
                    }
                }
            }
#pragma unroll
            for (int b = 0; b < BT; ++b) {
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    xs[b] += __shfl_xor_sync(0xffffffffu, xs[b], o);
#pragma unroll
                    for (int rr = 0; rr < kGemvCcRows; ++rr)
                        acc[rr][b] += __shfl_xor_sync(0xffffffffu, acc[rr][b], o);
                }
            }
            if (lane == 0) {
#pragma unroll
                for (int rr = 0; rr < kGemvCcRows; ++rr) {
                    if (n0 + rr >= N) continue;
                    const float a = alpha[n0 + rr], z = zero[n0 + rr];
#pragma unroll
                    for (int b = 0; b < BT; ++b)
                        if (b0 + b < B)
                            y[(int64_t)(b0 + b) * ldy + n0 + rr] = a * (acc[rr][b] * (float)(1 << sh) - z * xs[b]);
                }
            }
        }
    }
}

template <int R>
inline void launch_gemv_cuda_core(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                                  const int32_t* ovf_row_ptr, const uint16_t* ovf_col,
                                  const void* x, int B, int64_t ldx, float* y, int64_t ldy, bool pdl, cudaStream_t s) {
    const int warps_per_block = kGemvCcThreads / 32;
    int64_t blocks = (N + kGemvCcRows * warps_per_block - 1) / (kGemvCcRows * warps_per_block);
    const int64_t cap = (int64_t)sm_count() * 8;
    if (blocks > cap) blocks = cap;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3(kGemvCcThreads);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    const __nv_bfloat16* xb = static_cast<const __nv_bfloat16*>(x);
    if (B == 1) cudaLaunchKernelEx(&cfg, gemv_cuda_core<R, 1>, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, xb, B, ldx, y, ldy, pdl);
    else if (B == 2) cudaLaunchKernelEx(&cfg, gemv_cuda_core<R, 2>, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, xb, B, ldx, y, ldy, pdl);
    else cudaLaunchKernelEx(&cfg, gemv_cuda_core<R, 4>, packed, N, K, alpha, zero, ovf_row_ptr, ovf_col, xb, B, ldx, y, ldy, pdl);
}

}  // namespace matq
