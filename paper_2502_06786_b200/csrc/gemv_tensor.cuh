// Decode GEMV with the multiply-accumulates on the tensor pipe (warp-level
// mma.m16n8k16, bf16 x bf16 -> fp32) so that unpacking costs well under one
// issue slot per weight and a batch of up to 16 activations rides for free.
//
// Operand roles: A = 16 output channels x 16 weights, B = 16 weights x 8
// batch columns, D = fp32 [16 channels x 8 batch].  A dot product does not care
// in which order its terms are added, so the 16 "k slots" of an MMA are mapped
// to whatever weights a thread happens to hold in its 16-byte load:
//
//   * thread (g = lane/4, t = lane%4) loads 16 bytes of rows g and g+8 (per
//     m-tile) at byte offset qc*64 + t*16 of the row ("qc" = 64-byte quad chunk);
//   * a 32-bit word w of packed fields is turned into bf16x2 registers with one
//     LOP3 each:  ((w >> s) & mask) | 0x43004300.  0x4300 is bf16 128.0 whose
//     mantissa LSB weighs 1, so a field placed at mantissa bit 2i reads as
//     128 + field * 4^i.  For r = 2 fields at bit offsets 0, 2, 4 are used in
//     place (s in {0, 6, 12}), which needs 2 shifts + 8 LOP3 per 16 weights;
//     the 4^i is undone by pre-scaling the matching activation by 4^-i (exact).
//     For r = 4 the field sits at bit 0 after a shift by 4p.  r = 8 codes are
//     read as two nibbles, the high one paired with 16 * x.
//   * the constant 128 adds 128 * sum(x') to every accumulator; it is removed
//     in the epilogue with the separately computed sum of the pre-scaled
//     activations x'.
//
// The activations are staged once per CTA into shared memory as x' in exactly
// the order the B fragments are consumed, so a thread fetches the B registers
// of two MMAs with one conflict-free 128-bit load and reuses them for all of
// its m-tiles.
//
// Work split: a CTA owns kRows = 16*MT*WARPS_M output channels and one slice of
// K; its WARPS_K warp groups interleave over the slice's chunks and are summed
// through shared memory.  Slices of K (grid.y) form a thread-block cluster and
// are summed through distributed shared memory in rank order, so the result is
// deterministic and no global scratch is used.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace matq {
namespace cg = cooperative_groups;

struct GemvTensorParams {
    const uint8_t* packed;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const __nv_bfloat16* x;
    float* y;
    int64_t N, K, ldx, ldy;
    int64_t row_bytes;
    int B;        // batch columns in use
    int bpad;     // batch columns staged: 1, 2, 4, 8 or 16
    int n_qc;     // 64-byte chunks per row (last one may be partial)
    int qc_per_split;
    int pdl;
};

template <int R> struct GemvFmt;
template <> struct GemvFmt<2> { static constexpr int kWeightsPerWord = 16, kPairs = 8; };
template <> struct GemvFmt<4> { static constexpr int kWeightsPerWord = 8, kPairs = 4; };
template <> struct GemvFmt<8> { static constexpr int kWeightsPerWord = 4, kPairs = 4; };

// bf16x2 register of pair p of word w: two fields riding on the mantissa of 128.0
template <int R>
__device__ __forceinline__ uint32_t field_pair(uint32_t w, int p) {
    if (R == 2) {
        const int s = 6 * (p / 3), i = p % 3;
        return ((w >> s) & (0x00030003u << (2 * i))) | 0x43004300u;
    }
    return ((w >> (4 * p)) & 0x000f000fu) | 0x43004300u;
}

// Which weights of a word pair p holds (offsets inside the word's k range) and the factor its activation carries.
template <int R>
__device__ __forceinline__ void pair_slots(int p, int& f_lo, int& f_hi, float& scale) {
    if (R == 2) { f_lo = p; f_hi = p + 8; scale = (p % 3 == 0) ? 1.0f : (p % 3 == 1 ? 0.25f : 0.0625f); }
    else if (R == 4) { f_lo = p; f_hi = p + 4; scale = 1.0f; }
    else { f_lo = p >> 1; f_hi = (p >> 1) + 2; scale = (p & 1) ? 16.0f : 1.0f; }
}

// sum over the virtual weights of one k of the factor carried by its activation
template <int R>
__device__ __forceinline__ float slot_scale_sum(int64_t k) {
    if (R == 2) { const int m = (int)(k & 7) % 3; return m == 0 ? 1.0f : (m == 1 ? 0.25f : 0.0625f); }
    if (R == 4) return 1.0f;
    return 17.0f;
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int R, int MT, int NT, int WARPS_M, int WARPS_K>
__global__ void __launch_bounds__(32 * WARPS_M * WARPS_K)
gemv_tensor(const GemvTensorParams P) {
    using Fmt = GemvFmt<R>;
    constexpr int kThreads = 32 * WARPS_M * WARPS_K;
    constexpr int kRows = 16 * MT * WARPS_M;
    constexpr int kPairs = Fmt::kPairs;
    constexpr int kPG = kPairs / 4;                       // 128-bit B loads per word
    constexpr int kWq = 16 * Fmt::kWeightsPerWord;        // weights per 64-byte chunk of a row
    constexpr int sh = kCodeBits - R;
    constexpr int kMaxB = 8 * NT;

    extern __shared__ __align__(16) unsigned char smem_raw[];
    __shared__ float s_sumx[kMaxB], s_sumxp[kMaxB];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int wm = warp % WARPS_M, wk = warp / WARPS_M;
    const int split = blockIdx.y, n_split = gridDim.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const int qc0 = split * P.qc_per_split;
    const int nq = min(P.qc_per_split, P.n_qc - qc0);      // chunks of this CTA (>= 1 by construction)
    const int bpad = P.bpad;

    // shared memory: x' fragments, then the partial-result tile
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);
    const int xs_vec = nq * 4 * kPG * bpad * 4;            // uint4 elements
    float* part = reinterpret_cast<float*>(smem_raw + (size_t)P.qc_per_split * 4 * kPG * bpad * 4 * 16);
    // part[wk][row_local][kMaxB]

    // ---- weights of the first chunk are requested before anything that depends on the previous kernel
    const int64_t warp_row0 = row0 + (int64_t)wm * 16 * MT;
    auto load_chunk = [&](int qi, uint4 (&dst)[2 * MT]) {
        const int64_t off = (int64_t)(qc0 + qi) * 64 + t * 16;
#pragma unroll
        for (int h = 0; h < 2 * MT; ++h) {
            const int64_t row = warp_row0 + (h >> 1) * 16 + (h & 1) * 8 + g;
            dst[h] = make_uint4(0, 0, 0, 0);
            if (qi < nq && row < P.N && off < P.row_bytes) dst[h] = ld_stream_u4(P.packed + row * P.row_bytes + off);
        }
    };
    uint4 cur[2 * MT], nxt[2 * MT];
    load_chunk(wk, cur);
    load_chunk(wk + WARPS_K, nxt);

    if (P.pdl) {
        asm volatile("griddepcontrol.launch_dependents;");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    // ---- stage x' (pre-scaled activations in B-fragment order) and the two sums per batch column
    {
        const int total = xs_vec * 4;                      // bf16x2 elements
        uint32_t* xs32 = reinterpret_cast<uint32_t*>(xs);
        for (int e = tid; e < total; e += kThreads) {
            int idx = e;
            const int pl = idx & 3; idx >>= 2;
            const int tt = idx & 3; idx >>= 2;
            const int gg = idx % bpad; idx /= bpad;
            const int pg = idx % kPG; idx /= kPG;
            const int j = idx & 3; idx >>= 2;
            const int qi = idx;
            int f_lo, f_hi; float scale;
            pair_slots<R>(pg * 4 + pl, f_lo, f_hi, scale);
            const int64_t kb = (int64_t)(qc0 + qi) * kWq + tt * (kWq / 4) + j * Fmt::kWeightsPerWord;
            uint32_t v = 0;
            if (gg < P.B && kb < P.K) {                     // K % (weights per word) == 0: a word is inside or outside
                const __nv_bfloat16* xr = P.x + (int64_t)gg * P.ldx + kb;
                const float lo = __bfloat162float(xr[f_lo]) * scale, hi = __bfloat162float(xr[f_hi]) * scale;
                v = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(lo)) |
                    ((uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(hi)) << 16);
            }
            xs32[e] = v;
        }
        // sums: warp w takes batch columns w, w + warps, ...
        const int64_t k_lo = (int64_t)qc0 * kWq;
        const int64_t k_hi = min((int64_t)(qc0 + nq) * kWq, P.K);
        for (int b = warp; b < kMaxB; b += kThreads / 32) {
            float sx = 0.f, sxp = 0.f;
            if (b < P.B) {
                const __nv_bfloat16* xr = P.x + (int64_t)b * P.ldx;
                for (int64_t k = k_lo + lane; k < k_hi; k += 32) {
                    const float v = __bfloat162float(xr[k]);
                    sx += v;
                    sxp += v * slot_scale_sum<R>(k);
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    sx += __shfl_xor_sync(0xffffffffu, sx, o);
                    sxp += __shfl_xor_sync(0xffffffffu, sxp, o);
                }
            }
            if (lane == 0) { s_sumx[b] = sx; s_sumxp[b] = sxp; }
        }
    }
    __syncthreads();

    // ---- main loop: this warp group's chunks wk, wk + WARPS_K, ...
    float acc[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[mt][nt][i] = 0.f;

    for (int qi = wk; qi < nq; qi += WARPS_K) {
        uint4 nn[2 * MT];
        load_chunk(qi + 2 * WARPS_K, nn);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
#pragma unroll
            for (int pg = 0; pg < kPG; ++pg) {
                uint4 xb[NT];
#pragma unroll
                for (int nt = 0; nt < NT; ++nt) {
                    xb[nt] = make_uint4(0, 0, 0, 0);
                    const int gb = g + 8 * nt;
                    if (gb < bpad) xb[nt] = xs[(((qi * 4 + j) * kPG + pg) * bpad + gb) * 4 + t];
                }
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int p = pg * 4 + 2 * u;
#pragma unroll
                    for (int mt = 0; mt < MT; ++mt) {
                        const uint32_t w_lo = (j == 0 ? cur[2 * mt].x : j == 1 ? cur[2 * mt].y : j == 2 ? cur[2 * mt].z : cur[2 * mt].w);
                        const uint32_t w_hi = (j == 0 ? cur[2 * mt + 1].x : j == 1 ? cur[2 * mt + 1].y : j == 2 ? cur[2 * mt + 1].z : cur[2 * mt + 1].w);
                        const uint32_t a0 = field_pair<R>(w_lo, p), a1 = field_pair<R>(w_hi, p);
                        const uint32_t a2 = field_pair<R>(w_lo, p + 1), a3 = field_pair<R>(w_hi, p + 1);
#pragma unroll
                        for (int nt = 0; nt < NT; ++nt) {
                            const uint32_t b0 = u ? xb[nt].z : xb[nt].x, b1 = u ? xb[nt].w : xb[nt].y;
                            mma_bf16_16816(acc[mt][nt], a0, a1, a2, a3, b0, b1);
                        }
                    }
                }
            }
        }
#pragma unroll
        for (int h = 0; h < 2 * MT; ++h) { cur[h] = nxt[h]; nxt[h] = nn[h]; }
    }

    // ---- partial tile to shared memory: value = 2^sh (acc - 128 sum x') per (row, batch); z term added at the end
    {
        float* mine = part + (size_t)wk * kRows * kMaxB;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int rl = wm * 16 * MT + mt * 16 + g + (i >> 1) * 8;
                    const int b = nt * 8 + 2 * t + (i & 1);
                    mine[rl * kMaxB + b] = acc[mt][nt][i];
                }
    }
    __syncthreads();

    // ---- fold the warp groups, remove the 128 offset, add the extra-precision columns: one thread per (row, batch)
    for (int e = tid; e < kRows * kMaxB; e += kThreads) {
        const int rl = e / kMaxB, b = e % kMaxB;
        float v = part[e];
#pragma unroll
        for (int w = 1; w < WARPS_K; ++w) v += part[(size_t)w * kRows * kMaxB + e];
        if (b < P.B) v -= 128.0f * s_sumxp[b];
        const int64_t row = row0 + rl;
        if (P.ovf_row_ptr && row < P.N && b < P.B) {
            // entries split, split + n_split, ... of the row's ascending list belong to this CTA
            const int32_t pe = P.ovf_row_ptr[row + 1];
            const __nv_bfloat16* xr = P.x + (int64_t)b * P.ldx;
            float ev = 0.f;
            for (int32_t p = P.ovf_row_ptr[row] + split; p < pe; p += n_split) ev += __bfloat162float(xr[P.ovf_col[p]]);
            v += ev;
        }
        part[e] = v;
    }

    // ---- sum the K slices across the cluster in rank order and write y
    if (n_split > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        const int rows_per = (kRows + n_split - 1) / n_split;
        const int r_lo = split * rows_per, r_hi = min(kRows, r_lo + rows_per);
        for (int e = r_lo * kMaxB + tid; e < r_hi * kMaxB; e += kThreads) {
            const int rl = e / kMaxB, b = e % kMaxB;
            const int64_t row = row0 + rl;
            if (row >= P.N || b >= P.B) continue;
            float v = 0.f, sx = 0.f;
            for (int s = 0; s < n_split; ++s) {
                v += cluster.map_shared_rank(part, s)[e];
                sx += cluster.map_shared_rank(s_sumx, s)[b];
            }
            P.y[(int64_t)b * P.ldy + row] = P.alpha[row] * (v * (float)(1 << sh) - P.zero[row] * sx);
        }
        cluster.sync();                                   // peers may still be reading this CTA's tile
    } else {
        __syncthreads();
        for (int e = tid; e < kRows * kMaxB; e += kThreads) {
            const int rl = e / kMaxB, b = e % kMaxB;
            const int64_t row = row0 + rl;
            if (row >= P.N || b >= P.B) continue;
            P.y[(int64_t)b * P.ldy + row] = P.alpha[row] * (part[e] * (float)(1 << sh) - P.zero[row] * s_sumx[b]);
        }
    }
}

// Host side: geometry and launch.
struct GemvTensorPlan {
    int n_qc, qc_per_split, n_split, bpad;
    size_t smem;
    dim3 grid;
};

template <int R, int MT, int NT, int WARPS_M, int WARPS_K>
inline int launch_gemv_tensor(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                              const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                              float* y, int64_t ldy, bool pdl, cudaStream_t s) {
    using Fmt = GemvFmt<R>;
    constexpr int kRows = 16 * MT * WARPS_M, kThreads = 32 * WARPS_M * WARPS_K, kMaxB = 8 * NT;
    constexpr int kPG = Fmt::kPairs / 4;
    GemvTensorParams P;
    P.packed = packed; P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y; P.N = N; P.K = K; P.ldx = ldx; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    P.B = B;
    P.bpad = B <= 1 ? 1 : B <= 2 ? 2 : B <= 4 ? 4 : B <= 8 ? 8 : 16;
    P.n_qc = (int)((P.row_bytes + 63) / 64);
    P.pdl = pdl ? 1 : 0;
    const int64_t row_blocks = (N + kRows - 1) / kRows;
    // enough CTAs to fill the machine about twice, at most 8 K slices (portable cluster size), each at least one chunk
    const int sms = sm_count();
    int want = (int)((2 * (int64_t)sms + row_blocks - 1) / row_blocks);
    if (want > 8) want = 8;
    if (want > P.n_qc) want = P.n_qc;
    if (want < 1) want = 1;
    P.qc_per_split = (P.n_qc + want - 1) / want;
    const size_t part_bytes = (size_t)WARPS_K * kRows * kMaxB * sizeof(float);
    auto xs_bytes = [&](int qps) { return (size_t)qps * 4 * kPG * P.bpad * 4 * 16; };
    while (xs_bytes(P.qc_per_split) + part_bytes > 200 * 1024 && P.qc_per_split > 1) --P.qc_per_split;
    int n_split = (P.n_qc + P.qc_per_split - 1) / P.qc_per_split;
    if (n_split > 8) return MATQ_ERR_SHAPE;   // K too long for one cluster's shared memory at this batch size
    const size_t smem = xs_bytes(P.qc_per_split) + part_bytes;
    auto kern = gemv_tensor<R, MT, NT, WARPS_M, WARPS_K>;
    if (smem > 48 * 1024 &&
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return MATQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)row_blocks, (unsigned)n_split, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (n_split > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = 1; attr[na].val.clusterDim.y = (unsigned)n_split; attr[na].val.clusterDim.z = 1;
        ++na;
    }
    if (pdl) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    if (cudaLaunchKernelEx(&cfg, kern, P) != cudaSuccess) { cudaGetLastError(); return MATQ_ERR_CUDA; }
    return MATQ_OK;
}

}  // namespace matq
