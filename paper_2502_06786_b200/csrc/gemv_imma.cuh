// Decode GEMV for the smallest batches (B = 1, 2) on the integer tensor path:
// warp-level mma.m16n8k32, u8 x s8 -> s32.
//
// Why integers.  A warp-level MMA consumes one A fragment per instruction,
// whatever the batch is, so the rate at which packed weights can be multiplied
// is (weights per A fragment) x (MMA issue rate).  A bf16 fragment holds 256
// weights, an 8-bit fragment 512, and an r-bit field becomes an 8-bit operand
// with ONE mask per four weights and no shift (r = 8: nothing at all): a field
// left where it sits in its byte reads as field * 2^s, which is still an
// unsigned 8-bit integer, and the matching activation is divided by 2^s when it
// is turned into an integer.  There is no offset to remove afterwards, and the
// accumulators are 32-bit integers.
//
// The activations are bf16 and have to become 8-bit operands too.  Per batch
// column the kernel takes e = exponent of max |x|, scales the column by the
// power of two 2^(29 - e - s) (s = bit offset of the field the activation
// meets, 0 <= s <= 6), rounds to an integer v with |v| < 2^30 and writes v in
// balanced base 256: v = 2^24 t0 + 2^16 t1 + 2^8 t2 + t3, every digit in
// [-128, 127].  Each digit is one column of the MMA's 8-wide B operand, so a
// batch column costs four of the 8 columns and the products are summed exactly;
// the digits are recombined in a 64-bit integer in the epilogue and scaled back
// once.  bf16 has 8 significant bits, so every activation within 2^(-22+s) of
// the column's largest is represented exactly and the rest to an absolute
// 2^(-30+s) of it: a column with an outlier thousands of times its typical
// entry still comes out at fp32 accuracy.  (Columns whose largest magnitude is
// below 2^-97 are scaled as if it were 2^-97.)
//
// Fragment mapping (k slots of an MMA may be any weights as long as A and B
// agree): thread (g = lane / 4, t = lane % 4) loads 16 bytes of rows g and g + 8
// of an m-tile at byte offset qc * 64 + t * 16 ("qc" = 64-byte chunk of a row).
//   r = 8: word j is an A register as it stands; an MMA takes words (2u, 2u+1).
//   r = 4: w & 0x0f0f0f0f (even fields) and w & 0xf0f0f0f0 (odd fields, times 16)
//          are the two A registers of a row; one MMA per word.
//   r = 2: w & (0x03030303 << 2i) holds fields i, i+4, i+8, i+12 times 4^i; two MMAs per word.
// The activations are staged once per CTA in shared memory as 16-byte units in
// exactly that order (the B registers of two MMAs per unit), one unit per
// (16 weights, digit column, t), so the inner loop reads them with one
// conflict-free 128-bit load per two MMAs.
//
// Everything else follows the bf16 kernel: register streaming of the rows
// three chunks ahead, the first chunks requested before the programmatic
// dependency wait, the K split over the warps of a CTA summed in a fixed order
// through shared memory (deterministic, no global scratch), extra-precision
// lists walked by a few threads per row during the staging.
#pragma once
#include "common.cuh"
#include "gemv_tensor.cuh"

namespace matq {
namespace imma {

constexpr int kCols = 8;                     // columns of the B operand
constexpr int kMaxB = 2;                     // largest batch this kernel takes (four digit columns each)
constexpr int kTerms = 4;                    // base-256 digits per activation
constexpr int kP = 29;                       // activations become integers below 2^(kP+1)

struct Params {
    const uint8_t* packed;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const __nv_bfloat16* x;
    float* y;
    int64_t N, K, ldx, ldy;
    int64_t row_bytes;
    int B;            // batch columns
    int ncp;          // digit columns staged: 4 (B = 1) or 8
    int n_qc;         // 64-byte chunks per row (the last one may be half full at r = 2)
    int qc_pass;      // chunks whose activations are staged at a time
    int pdl;
};

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// element of the 16 consecutive activations that lands in byte p of a staged unit
template <int R>
__host__ __device__ constexpr int unit_src(int p) {
    return R == 8 ? p : R == 4 ? (p & 8) + 2 * (p & 3) + ((p >> 2) & 1) : 4 * (p & 3) + (p >> 2);
}

template <int R, int MT, int SK, int WARPS, bool EP>
__global__ void __launch_bounds__(WARPS * 32, (MT == 1 ? 32 : 16) / WARPS)
gemv_imma(const Params P) {
    constexpr int kThreads = WARPS * 32;
    constexpr int kTileRows = 16 * MT;                    // rows of a warp
    constexpr int kTiles = WARPS / SK;                    // row tiles of a CTA
    constexpr int kRows = kTileRows * kTiles;
    constexpr int kWpp = 128 / R;                         // weights per 16-byte piece of a row
    constexpr int kM2 = kWpp / 16;                        // staged units (pairs of MMAs) per piece
    constexpr int sh = kCodeBits - R;
    constexpr int kSets = (MT >= 2) ? 1 : 2;              // independent accumulator sets per m-tile

    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ uint32_t s_rmax[WARPS][kMaxB];
    __shared__ float s_rsum[WARPS][kMaxB];
    __shared__ float s_ep[EP ? kRows : 1][kMaxB];
    __shared__ float s_alpha[kRows], s_zero[kRows];
    constexpr int kRowThreads = kThreads / kRows;         // = 2 SK / MT consecutive threads per row of the CTA
    constexpr int kTPR = kRowThreads > 32 ? 32 : kRowThreads;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int tile = warp / SK, ks = warp % SK;
    const int64_t row0 = (int64_t)blockIdx.x * kRows + (int64_t)tile * kTileRows;
    int pass_lo = 0, pass_hi = min(P.qc_pass, P.n_qc);
    int q_lo, q_hi;
    auto set_slice = [&]() {
        const int per_warp = (pass_hi - pass_lo + SK - 1) / SK;
        q_lo = pass_lo + ks * per_warp;
        q_hi = min(q_lo + per_warp, pass_hi);
    };
    set_slice();
    const int ncp = P.ncp;
    constexpr int terms = kTerms;

    // shared memory: staged digit units of one pass | partial tiles [warp][kTileRows][kCols]
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);
    int* part = reinterpret_cast<int*>(smem_raw + (size_t)min(P.qc_pass, P.n_qc) * kM2 * ncp * 64);

    // ---- weights of the first chunks are requested before anything that depends on the previous kernel.
    // Rows past N are clamped to the last row (never stored); a piece that would start past the end of a half-full
    // last chunk is clamped to the row's last 16 bytes and meets activations staged as zeros.
    const uint8_t* wrow[2 * MT];
#pragma unroll
    for (int h = 0; h < 2 * MT; ++h) {
        const int64_t row = row0 + (h >> 1) * 16 + (h & 1) * 8 + g;
        wrow[h] = P.packed + (row < P.N ? row : P.N - 1) * P.row_bytes;
    }
    const int max_off = (int)P.row_bytes - 16;
    auto load_chunk = [&](int q, uint4 (&dst)[2 * MT]) {
        if (q < q_hi) {                                   // warp-uniform
            const int off = min(q * 64 + t * 16, max_off);
#pragma unroll
            for (int h = 0; h < 2 * MT; ++h) dst[h] = ld_stream_u4(wrow[h] + off);
        }
    };
    uint4 wbuf[kGemvDepth][2 * MT];
#pragma unroll
    for (int d = 0; d < kGemvDepth; ++d) load_chunk(q_lo + d, wbuf[d]);

    for (int rl = tid; rl < kRows; rl += kThreads) {
        const int64_t row = (int64_t)blockIdx.x * kRows + rl;
        s_alpha[rl] = row < P.N ? P.alpha[row] : 0.f;
        s_zero[rl] = row < P.N ? P.zero[row] : 0.f;
    }

    // Extra precision (Errata, Eq. 8): an overflow column's field is one higher than the stored, clamped one, so
    // its activation is added once more, in fp32 from the bf16 activations themselves.
    const int ep_row = tid / kRowThreads, ep_j = tid % kRowThreads;
    int ep_p = 0, ep_hi = 0, ep_c0 = 0;
    if (EP && ep_j < kTPR) {
        const int64_t row = (int64_t)blockIdx.x * kRows + ep_row;
        if (row < P.N) {
            ep_p = P.ovf_row_ptr[row] + ep_j;
            ep_hi = P.ovf_row_ptr[row + 1];
            if (ep_p < ep_hi) ep_c0 = P.ovf_col[ep_p];
        }
    }

    if (P.pdl) {
        asm volatile("griddepcontrol.launch_dependents;");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    float ep_x0 = 0.f;
    if (EP && ep_p < ep_hi) ep_x0 = __bfloat162float(P.x[ep_c0]);

    // ---- per batch column: largest magnitude (as a bf16 bit pattern, which orders like the value) and fp32 sum
    uint32_t cmax[kMaxB];
    float csum[kMaxB];
    {
        const int n8 = (int)(P.K >> 3);
#pragma unroll
        for (int b = 0; b < kMaxB; ++b) {
            uint32_t mx = 0;
            float sm = 0.f;
            if (b < P.B) {
                const __nv_bfloat16* xr = P.x + (int64_t)b * P.ldx;
                for (int i = tid; i < n8; i += kThreads) {
                    const uint4 v = ld_x4(xr + 8 * i);
                    mx = __vmaxu2(mx, v.x & 0x7fff7fffu); mx = __vmaxu2(mx, v.y & 0x7fff7fffu);
                    mx = __vmaxu2(mx, v.z & 0x7fff7fffu); mx = __vmaxu2(mx, v.w & 0x7fff7fffu);
                    sm += ((bf_lo(v.x) + bf_hi(v.x)) + (bf_lo(v.y) + bf_hi(v.y))) +
                          ((bf_lo(v.z) + bf_hi(v.z)) + (bf_lo(v.w) + bf_hi(v.w)));
                }
                mx = max(mx & 0xffffu, mx >> 16);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    sm += __shfl_xor_sync(0xffffffffu, sm, o);
                }
                if (lane == 0) { s_rmax[warp][b] = mx; s_rsum[warp][b] = sm; }
            }
            cmax[b] = 0; csum[b] = 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int b = 0; b < kMaxB; ++b) {
            if (b < P.B) {
                uint32_t mx = lane < WARPS ? s_rmax[lane][b] : 0u;
                float sm = lane < WARPS ? s_rsum[lane][b] : 0.f;
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) {
                    mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    sm += __shfl_xor_sync(0xffffffffu, sm, o);
                }
                cmax[b] = mx; csum[b] = sm;
            }
        }
    }
    // biased exponent of the column's largest magnitude, kept where both 2^(P - e) and 2^(e - P) are normal floats
    int cexp[kMaxB];
#pragma unroll
    for (int b = 0; b < kMaxB; ++b) cexp[b] = min(max((int)(cmax[b] >> 7), kP + 1), 254);

    int acc[kSets][MT][4];
#pragma unroll
    for (int c = 0; c < kSets; ++c)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[c][mt][i] = 0;

    for (;;) {
        // ---- stage the digit units of this pass.  Item = (chunk, unit of the piece, batch column, t): 16 consecutive
        // activations, scaled, rounded, split into digits, bytes permuted into fragment order.
        {
            const int n_items = (pass_hi - pass_lo) * kM2 * P.B * 4;
            for (int it = tid; it < n_items; it += kThreads) {
                const int tt = it & 3;
                const int rest = it >> 2;
                const int b = rest % P.B;
                const int qm = rest / P.B;                // (chunk of the pass) * kM2 + unit
                const int ql = qm / kM2, m2 = qm % kM2;
                const int k0 = ((pass_lo + ql) * 4 + tt) * kWpp + m2 * 16;
                uint32_t digit[4][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}};
                if (k0 < (int)P.K) {                      // K % 128 == 0: a unit lies inside or outside
                    int e = cexp[0];
#pragma unroll
                    for (int bb = 1; bb < kMaxB; ++bb) if (b == bb) e = cexp[bb];
                    // multiplier of the activations that meet a field at bit offset R * cls of its byte
                    float mult[8 / R];
#pragma unroll
                    for (int cls = 0; cls < 8 / R; ++cls) mult[cls] = __uint_as_float((uint32_t)(254 + kP - e - R * cls) << 23);
                    const __nv_bfloat16* xp = P.x + (int64_t)b * P.ldx + k0;
                    const uint4 va = ld_x4(xp), vb = ld_x4(xp + 8);
                    const uint32_t raw[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                    int v[16];
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        v[2 * i] = __float2int_rn(bf_lo(raw[i]) * mult[(2 * i) % (8 / R)]);
                        v[2 * i + 1] = __float2int_rn(bf_hi(raw[i]) * mult[(2 * i + 1) % (8 / R)]);
                    }
#pragma unroll
                    for (int p = 0; p < 16; ++p) {
                        int val = v[unit_src<R>(p)];
                        // balanced base 256, least significant digit first; digit d goes to column terms-1-d
                        const uint32_t d0 = (uint32_t)val & 0xffu;  val = (val + 128) >> 8;
                        const uint32_t d1 = (uint32_t)val & 0xffu;  val = (val + 128) >> 8;
                        const uint32_t d2 = (uint32_t)val & 0xffu;  val = (val + 128) >> 8;
                        const uint32_t d3 = (uint32_t)val & 0xffu;
                        digit[0][p >> 2] |= d0 << (8 * (p & 3));
                        digit[1][p >> 2] |= d1 << (8 * (p & 3));
                        digit[2][p >> 2] |= d2 << (8 * (p & 3));
                        digit[3][p >> 2] |= d3 << (8 * (p & 3));
                    }
                }
                uint4* dst = xs + ((size_t)qm * ncp + b * terms) * 4 + tt;
                dst[0] = make_uint4(digit[3][0], digit[3][1], digit[3][2], digit[3][3]);
                dst[4] = make_uint4(digit[2][0], digit[2][1], digit[2][2], digit[2][3]);
                dst[8] = make_uint4(digit[1][0], digit[1][1], digit[1][2], digit[1][3]);
                dst[12] = make_uint4(digit[0][0], digit[0][1], digit[0][2], digit[0][3]);
            }
        }
        if (EP && pass_lo == 0) {                             // uniform over the CTA
            for (int b = 0; b < P.B; ++b) {
                const __nv_bfloat16* xr = P.x + (int64_t)b * P.ldx;
                float ev = b == 0 ? ep_x0 : (ep_p < ep_hi ? __bfloat162float(xr[ep_c0]) : 0.f);
                for (int p = ep_p + kTPR; p < ep_hi; p += 4 * kTPR) {      // lists longer than kTPR entries
                    int col[4];
#pragma unroll
                    for (int u = 0; u < 4; ++u) col[u] = p + u * kTPR < ep_hi ? (int)P.ovf_col[p + u * kTPR] : -1;
#pragma unroll
                    for (int u = 0; u < 4; ++u)
                        if (col[u] >= 0) ev += __bfloat162float(xr[col[u]]);
                }
#pragma unroll
                for (int o = kTPR / 2; o > 0; o >>= 1) ev += __shfl_xor_sync(0xffffffffu, ev, o);
                if (ep_j == 0) s_ep[ep_row][b] = ev;
            }
        }
        const bool last_pass = pass_hi >= P.n_qc;            // uniform over the CTA
        __syncthreads();

        // ---- this warp's chunks of the pass
        for (int q0 = q_lo; q0 < q_hi; q0 += kGemvDepth) {
#pragma unroll
            for (int d = 0; d < kGemvDepth; ++d) {
                const int q = q0 + d;
                if (q < q_hi) {                               // warp-uniform
                    uint4 wv[2 * MT];
#pragma unroll
                    for (int h = 0; h < 2 * MT; ++h) wv[h] = wbuf[d][h];
                    load_chunk(q + kGemvDepth, wbuf[d]);
#pragma unroll
                    for (int m2 = 0; m2 < kM2; ++m2) {
                        uint4 xb = make_uint4(0, 0, 0, 0);
                        if (g < ncp) xb = xs[((size_t)(q - pass_lo) * kM2 + m2) * ncp * 4 + g * 4 + t];
#pragma unroll
                        for (int sub = 0; sub < 2; ++sub) {
                            const uint32_t b0 = sub ? xb.z : xb.x, b1 = sub ? xb.w : xb.y;
#pragma unroll
                            for (int mt = 0; mt < MT; ++mt) {
                                uint32_t a0, a1, a2, a3;
                                if (R == 8) {
                                    a0 = sub ? wv[2 * mt].z : wv[2 * mt].x;          a2 = sub ? wv[2 * mt].w : wv[2 * mt].y;
                                    a1 = sub ? wv[2 * mt + 1].z : wv[2 * mt + 1].x;  a3 = sub ? wv[2 * mt + 1].w : wv[2 * mt + 1].y;
                                } else {
                                    const int j = R == 4 ? 2 * m2 + sub : m2;
                                    const uint32_t w_lo = (j == 0 ? wv[2 * mt].x : j == 1 ? wv[2 * mt].y : j == 2 ? wv[2 * mt].z : wv[2 * mt].w);
                                    const uint32_t w_hi = (j == 0 ? wv[2 * mt + 1].x : j == 1 ? wv[2 * mt + 1].y : j == 2 ? wv[2 * mt + 1].z : wv[2 * mt + 1].w);
                                    if (R == 4) {
                                        a0 = w_lo & 0x0f0f0f0fu;  a2 = w_lo & 0xf0f0f0f0u;
                                        a1 = w_hi & 0x0f0f0f0fu;  a3 = w_hi & 0xf0f0f0f0u;
                                    } else {
                                        a0 = w_lo & (0x03030303u << (4 * sub));  a2 = w_lo & (0x0c0c0c0cu << (4 * sub));
                                        a1 = w_hi & (0x03030303u << (4 * sub));  a3 = w_hi & (0x0c0c0c0cu << (4 * sub));
                                    }
                                }
                                mma_u8s8(acc[sub % kSets][mt], a0, a1, a2, a3, b0, b1);
                            }
                        }
                    }
                }
            }
        }
        if (last_pass) break;
        // ---- next pass: request its first chunks, then wait until every warp is done with the staged activations
        pass_lo = pass_hi;
        pass_hi = min(pass_lo + P.qc_pass, P.n_qc);
        set_slice();
#pragma unroll
        for (int d = 0; d < kGemvDepth; ++d) load_chunk(q_lo + d, wbuf[d]);
        __syncthreads();
    }
    if (kSets == 2) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[0][mt][i] += acc[1][mt][i];
    }

    // ---- epilogue.  Accumulator i of thread (g, t): row g + 8*(i>>1) of the m-tile, digit column 2t + (i&1).
    {
        int* mine = part + (size_t)warp * kTileRows * kCols;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            *reinterpret_cast<int2*>(mine + (mt * 16 + g) * kCols + 2 * t) = make_int2(acc[0][mt][0], acc[0][mt][1]);
            *reinterpret_cast<int2*>(mine + (mt * 16 + g + 8) * kCols + 2 * t) = make_int2(acc[0][mt][2], acc[0][mt][3]);
        }
    }
    __syncthreads();
    // Output o = (row of the CTA) * kMaxB + batch column: the SK partial sums of each digit column are added as
    // integers in a fixed order, the digits recombined in 64 bits, converted once and scaled back.
    for (int o = tid; o < kRows * kMaxB; o += kThreads) {
        const int b = o % kMaxB, row_l = o / kMaxB;
        const int64_t row = (int64_t)blockIdx.x * kRows + row_l;
        if (b >= P.B || row >= P.N) continue;
        const int* src = part + ((size_t)(row_l / kTileRows) * SK * kTileRows + row_l % kTileRows) * kCols + b * terms;
        long long tot = 0;
        for (int d = 0; d < terms; ++d) {
            int sd = src[d];
#pragma unroll
            for (int sidx = 1; sidx < SK; ++sidx) sd += src[(size_t)sidx * kTileRows * kCols + d];
            tot = tot * 256 + sd;
        }
        int e = cexp[0];
        float sx = csum[0];
#pragma unroll
        for (int bb = 1; bb < kMaxB; ++bb) if (b == bb) { e = cexp[bb]; sx = csum[bb]; }
        float v = __ll2float_rn(tot) * __uint_as_float((uint32_t)(e - kP) << 23);
        if (EP) v += s_ep[row_l][b];
        P.y[(int64_t)b * P.ldy + row] = s_alpha[row_l] * (v * (float)(1 << sh) - s_zero[row_l] * sx);
    }
}

// Host side: geometry and launch.
template <int R, int MT, int SK, int WARPS = 8>
inline int launch(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                  const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                  float* y, int64_t ldy, bool pdl, cudaStream_t s) {
    constexpr int kThreads = WARPS * 32;
    constexpr int kRows = 16 * MT * (WARPS / SK);
    constexpr int kM2 = (128 / R) / 16;
    if (B < 1 || B > kMaxB) return MATQ_ERR_SHAPE;
    Params P;
    P.packed = packed; P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y;
    P.N = N; P.K = K; P.ldx = ldx; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    if (K > 65536) return MATQ_ERR_SHAPE;                  // 255 * 128 * K must stay below 2^31 (240 * 128 * K at r = 4)
    P.B = B;
    P.ncp = B * kTerms;
    P.n_qc = (int)((P.row_bytes + 63) / 64);
    P.pdl = pdl ? 1 : 0;
    // Shared memory: the staged units of one pass (64 * kM2 * ncp bytes per chunk) + the partial tiles.
    const size_t part_bytes = (size_t)WARPS * 16 * MT * kCols * sizeof(int);
    const size_t chunk_bytes = (size_t)kM2 * P.ncp * 64;
    const int fit = (int)((150 * 1024 - part_bytes) / chunk_bytes);
    const int passes = (P.n_qc + fit - 1) / fit;
    P.qc_pass = (P.n_qc + passes - 1) / passes;
    const size_t smem = (size_t)P.qc_pass * chunk_bytes + part_bytes;
    auto kern = ovf_row_ptr ? gemv_imma<R, MT, SK, WARPS, true> : gemv_imma<R, MT, SK, WARPS, false>;
    if (smem > 16 * 1024 &&   // the 48 KB default counts static shared memory too
        cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return MATQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + kRows - 1) / kRows), 1, 1);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, P) != cudaSuccess) { cudaGetLastError(); return MATQ_ERR_CUDA; }
    return MATQ_OK;
}

}  // namespace imma
}  // namespace matq
