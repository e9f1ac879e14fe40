// Decode GEMV for a single activation vector (B = 1) on the integer tensor
// path: warp-level mma.m16n8k32, u8 x u8 -> s32.
//
// Why integers.  A warp-level MMA consumes one A fragment per instruction,
// whatever the batch is, so the rate at which packed weights can be multiplied
// is (weights per A fragment) x (MMA issue rate).  A bf16 fragment holds 256
// weights, an 8-bit fragment 512, and an r-bit field becomes an 8-bit operand
// with ONE mask per four weights and no shift (r = 8: nothing at all): a field
// left where it sits in its byte reads as field * 2^s, which is still an
// unsigned 8-bit integer, and the matching activation is divided by 2^s when it
// is turned into an integer.  The accumulators are 32-bit integers, so the
// weights side and every sum are exact.
//
// The activations are bf16 and have to become 8-bit operands too.  The kernel
// takes e = exponent of max |x|, scales x[k] by the power of two 2^(29 - e - s)
// (s = bit offset of the field that x[k] meets, 0 <= s <= 6), rounds to an
// integer v[k] with |v[k]| < 2^(30-s) and adds 2^(30-s): the result is a
// non-negative 32-bit integer whose four BYTES are four columns of the MMA's
// 8-wide B operand (byte d weighs 256^d).  A fifth column holds the constants
// 2^(smax - s) and so returns 2^smax * (sum of the row's fields), which removes
// the added offsets exactly:
//   sum_k f 2^s (v + 2^(30-s)) = sum_k f 2^s v + 2^30 sum_k f.
// The five column sums are recombined in a 64-bit integer in the epilogue and
// scaled back once.  bf16 has 8 significant bits, so every activation within
// 2^(-22+s) of the largest is represented exactly and the rest to an absolute
// 2^(-30+s) of it: a vector with an outlier thousands of times its typical
// entry still comes out at fp32 accuracy.  (A vector whose largest magnitude
// is below 2^-97 is scaled as if it were 2^-97.)
//
// Fragment mapping (k slots of an MMA may be any weights as long as A and B
// agree): thread (g = lane / 4, t = lane % 4) loads 16 bytes of rows g and g + 8
// of an m-tile at byte offset qc * 64 + t * 16 ("qc" = 64-byte chunk of a row).
//   r = 8: word j is an A register as it stands; an MMA takes words (2u, 2u+1).
//   r = 4: w & 0x0f0f0f0f (even fields) and w & 0xf0f0f0f0 (odd fields, times 16)
//          are the two A registers of a row; one MMA per word.
//   r = 2: w & (0x03030303 << 2i) holds fields i, i+4, i+8, i+12 times 4^i; two MMAs per word.
// The activation bytes are staged once per CTA in shared memory as 16-byte
// units in exactly that order (the B registers of two MMAs per unit), one unit
// per (16 weights, byte column, t), so the inner loop reads them with one
// conflict-free 128-bit load per two MMAs; a 4 x 4 byte transpose (8 byte
// permutes) turns four converted activations into one word of each column.
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
constexpr int kBytes = 4;                    // byte columns of an activation (column 4 is the constant one)
constexpr int kP = 29;                       // activations become integers below 2^(kP+1)
constexpr int64_t kMaxK = 32768;             // 255 * 255 * K must stay below 2^31

struct Params {
    const uint8_t* packed;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const __nv_bfloat16* x;
    float* y;
    int64_t N, K, ldy;
    int64_t row_bytes;
    int n_qc;         // 64-byte chunks per row (the last one may be half full at r = 2)
    int qc_pass;      // chunks whose activations are staged at a time
    int pdl;
};

__device__ __forceinline__ void mma_u8u8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.u8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// element of the 16 consecutive activations that lands in byte p of a staged unit
template <int R>
__host__ __device__ constexpr int unit_src(int p) {
    return R == 8 ? p : R == 4 ? (p & 8) + 2 * (p & 3) + ((p >> 2) & 1) : 4 * (p & 3) + (p >> 2);
}

// B registers of the constant column for MMA `sub` of a unit: 2^(smax - s) in every byte, s = bit offset of the
// field that the byte's k slot holds (b0 meets the A register a0, b1 meets a2)
template <int R>
__device__ __forceinline__ uint32_t ones_b0(int sub) { return R == 8 ? 0x01010101u : R == 4 ? 0x10101010u : (sub ? 0x04040404u : 0x40404040u); }
template <int R>
__device__ __forceinline__ uint32_t ones_b1(int sub) { return R == 2 ? (sub ? 0x01010101u : 0x10101010u) : 0x01010101u; }

template <int R, int MT, int SK, int WARPS, bool EP>
__global__ void __launch_bounds__(WARPS * 32, (MT == 1 ? 32 : 16) / WARPS)
gemv_imma(const Params P) {
    constexpr int kThreads = WARPS * 32;
    constexpr int kTileRows = 16 * MT;                    // rows of a warp
    constexpr int kTiles = WARPS / SK;                    // row tiles of a CTA
    constexpr int kRows = kTileRows * kTiles;
    constexpr int kWpp = 128 / R;                         // weights per 16-byte piece of a row
    constexpr int kM2 = kWpp / 16;                        // staged units (pairs of MMAs) per piece
    constexpr int sh = kCodeBits - R;                     // also the largest bit offset of a field in its byte
    constexpr int kSets = (MT >= 2) ? 1 : 2;              // independent accumulator sets per m-tile

    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ uint32_t s_rmax[WARPS];
    __shared__ float s_rsum[WARPS];
    __shared__ float s_ep[EP ? kRows : 1];
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

    // shared memory: staged byte units of one pass [chunk][unit][byte column][t] | partial tiles [warp][kTileRows][kCols]
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);
    int* part = reinterpret_cast<int*>(smem_raw + (size_t)min(P.qc_pass, P.n_qc) * kM2 * kBytes * 64);

    // ---- weights of the first chunks are requested before anything that depends on the previous kernel.
    // Rows past N are clamped to the last row (never stored); a piece that would start past the end of a half-full
    // last chunk is clamped to the row's last 16 bytes and meets zeros in every column of B.
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

    // ---- largest magnitude (as a bf16 bit pattern, which orders like the value) and fp32 sum of the activations
    uint32_t xmax = 0;
    float xsum = 0.f;
    {
        const int n8 = (int)(P.K >> 3);
        for (int i = tid; i < n8; i += kThreads) {
            const uint4 v = ld_x4(P.x + 8 * i);
            xmax = __vmaxu2(xmax, v.x & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.y & 0x7fff7fffu);
            xmax = __vmaxu2(xmax, v.z & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.w & 0x7fff7fffu);
            xsum += ((bf_lo(v.x) + bf_hi(v.x)) + (bf_lo(v.y) + bf_hi(v.y))) + ((bf_lo(v.z) + bf_hi(v.z)) + (bf_lo(v.w) + bf_hi(v.w)));
        }
        xmax = max(xmax & 0xffffu, xmax >> 16);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
            xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
        }
        if (lane == 0) { s_rmax[warp] = xmax; s_rsum[warp] = xsum; }
        __syncthreads();
        xmax = lane < WARPS ? s_rmax[lane] : 0u;
        xsum = lane < WARPS ? s_rsum[lane] : 0.f;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
            xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
        }
    }
    // biased exponent of the largest magnitude, kept where both 2^(P - e - s) and 2^(e - P) are normal floats
    const int xexp = min(max((int)(xmax >> 7), kP + 1), 254);

    int acc[kSets][MT][4];
#pragma unroll
    for (int c = 0; c < kSets; ++c)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) acc[c][mt][i] = 0;

    for (;;) {
        // ---- stage the byte units of this pass.  Item = (chunk, unit of the piece, t): 16 consecutive activations,
        // scaled, rounded, made non-negative; 4 x 4 byte transposes put byte d of four of them into one word of column d.
        {
            const int n_items = (pass_hi - pass_lo) * kM2 * 4;
            // multiplier and offset of the activations that meet a field at bit offset R * cls of its byte
            float mult[8 / R];
#pragma unroll
            for (int cls = 0; cls < 8 / R; ++cls) mult[cls] = __uint_as_float((uint32_t)(254 + kP - xexp - R * cls) << 23);
            for (int it = tid; it < n_items; it += kThreads) {
                const int tt = it & 3;
                const int qm = it >> 2;                   // (chunk of the pass) * kM2 + unit
                const int ql = qm / kM2, m2 = qm % kM2;
                const int k0 = ((pass_lo + ql) * 4 + tt) * kWpp + m2 * 16;
                uint32_t col[kBytes][4] = {{0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}, {0, 0, 0, 0}};
                if (k0 < (int)P.K) {                      // K % 128 == 0: a unit lies inside or outside
                    const uint4 va = ld_x4(P.x + k0), vb = ld_x4(P.x + k0 + 8);
                    const uint32_t raw[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                    uint32_t v[16];
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const int cls = i % (8 / R);
                        const float xf = (i & 1) ? bf_hi(raw[i >> 1]) : bf_lo(raw[i >> 1]);
                        v[i] = (uint32_t)(__float2int_rn(xf * mult[cls]) + (1 << (kP + 1 - R * cls)));
                    }
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const uint32_t e0 = v[unit_src<R>(4 * w)], e1 = v[unit_src<R>(4 * w + 1)];
                        const uint32_t e2 = v[unit_src<R>(4 * w + 2)], e3 = v[unit_src<R>(4 * w + 3)];
                        const uint32_t t0 = __byte_perm(e0, e1, 0x5140), t1 = __byte_perm(e2, e3, 0x5140);
                        const uint32_t t2 = __byte_perm(e0, e1, 0x7362), t3 = __byte_perm(e2, e3, 0x7362);
                        col[0][w] = __byte_perm(t0, t1, 0x5410);  col[1][w] = __byte_perm(t0, t1, 0x7632);
                        col[2][w] = __byte_perm(t2, t3, 0x5410);  col[3][w] = __byte_perm(t2, t3, 0x7632);
                    }
                }
                uint4* dst = xs + (size_t)qm * kBytes * 4 + tt;
#pragma unroll
                for (int d = 0; d < kBytes; ++d) dst[4 * d] = make_uint4(col[d][0], col[d][1], col[d][2], col[d][3]);
            }
        }
        if (EP && pass_lo == 0) {                             // uniform over the CTA
            float ev = ep_x0;
            for (int p = ep_p + kTPR; p < ep_hi; p += 4 * kTPR) {      // lists longer than kTPR entries
                int col[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) col[u] = p + u * kTPR < ep_hi ? (int)P.ovf_col[p + u * kTPR] : -1;
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (col[u] >= 0) ev += __bfloat162float(P.x[col[u]]);
            }
#pragma unroll
            for (int o = kTPR / 2; o > 0; o >>= 1) ev += __shfl_xor_sync(0xffffffffu, ev, o);
            if (ep_j == 0) s_ep[ep_row] = ev;
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
                    const bool piece_ok = q * 64 + t * 16 <= max_off;      // else: the clamped piece of a half-full chunk
#pragma unroll
                    for (int m2 = 0; m2 < kM2; ++m2) {
                        uint4 xb = make_uint4(0, 0, 0, 0);
                        if (g < kBytes) xb = xs[((size_t)(q - pass_lo) * kM2 + m2) * kBytes * 4 + g * 4 + t];
                        else if (g == kBytes && piece_ok) xb = make_uint4(ones_b0<R>(0), ones_b1<R>(0), ones_b0<R>(1), ones_b1<R>(1));
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
                                mma_u8u8(acc[sub % kSets][mt], a0, a1, a2, a3, b0, b1);
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

    // ---- epilogue.  Accumulator i of thread (g, t): row g + 8*(i>>1) of the m-tile, column 2t + (i&1).
    {
        int* mine = part + (size_t)warp * kTileRows * kCols;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            *reinterpret_cast<int2*>(mine + (mt * 16 + g) * kCols + 2 * t) = make_int2(acc[0][mt][0], acc[0][mt][1]);
            *reinterpret_cast<int2*>(mine + (mt * 16 + g + 8) * kCols + 2 * t) = make_int2(acc[0][mt][2], acc[0][mt][3]);
        }
    }
    __syncthreads();
    // One thread per (row, column): the SK partial sums of a column are added as integers in a fixed order; the
    // five columns of a row sit in neighbouring lanes and are recombined in 64 bits by the first of them, the
    // offsets removed with the constant column, one conversion, one scaling back.  kRows * kCols is a multiple of
    // 32, so whole warps take part in the shuffles.
    for (int o = tid; o < kRows * kCols; o += kThreads) {
        const int col = o % kCols, row_l = o / kCols;
        const int64_t row = (int64_t)blockIdx.x * kRows + row_l;
        const int* src = part + ((size_t)(row_l / kTileRows) * SK * kTileRows + row_l % kTileRows) * kCols + col;
        int sd = 0;
        if (col <= kBytes) {
            sd = src[0];
#pragma unroll
            for (int sidx = 1; sidx < SK; ++sidx) sd += src[(size_t)sidx * kTileRows * kCols];
        }
        const int s1 = __shfl_down_sync(0xffffffffu, sd, 1, kCols), s2 = __shfl_down_sync(0xffffffffu, sd, 2, kCols);
        const int s3 = __shfl_down_sync(0xffffffffu, sd, 3, kCols), s4 = __shfl_down_sync(0xffffffffu, sd, 4, kCols);
        if (col != 0 || row >= P.N) continue;
        // sum_k f 2^s v = sum_d 256^d D_d - 2^30 sum_k f, and column 4 holds 2^sh sum_k f
        const long long tot = (((long long)s3 * 256 + s2) * 256 + s1) * 256 + sd - ((long long)s4 << (kP + 1 - sh));
        float v = __ll2float_rn(tot) * __uint_as_float((uint32_t)(xexp - kP) << 23);
        if (EP) v += s_ep[row_l];
        P.y[row] = s_alpha[row_l] * (v * (float)(1 << sh) - s_zero[row_l] * xsum);
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
    (void)ldx;
    if (B != 1 || K > kMaxK) return MATQ_ERR_SHAPE;
    Params P;
    P.packed = packed; P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y;
    P.N = N; P.K = K; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    P.n_qc = (int)((P.row_bytes + 63) / 64);
    P.pdl = pdl ? 1 : 0;
    // Shared memory: the staged units of one pass (64 * kM2 * kBytes bytes per chunk) + the partial tiles.
    const size_t part_bytes = (size_t)WARPS * 16 * MT * kCols * sizeof(int);
    const size_t chunk_bytes = (size_t)kM2 * kBytes * 64;
    const int fit = (int)((150 * 1024 - part_bytes) / chunk_bytes);
    const int passes = (P.n_qc + fit - 1) / fit;
    P.qc_pass = (P.n_qc + passes - 1) / passes;
    const size_t smem = (size_t)P.qc_pass * chunk_bytes + part_bytes;
    auto kern = ovf_row_ptr ? gemv_imma<R, MT, SK, WARPS, true> : gemv_imma<R, MT, SK, WARPS, false>;
    static std::atomic<unsigned long long> smem_ok[2] = {{0}, {0}};     // one per kernel of this template instance
    if (smem > 16 * 1024 &&   // the 48 KB default counts static shared memory too
        !opt_in_max_smem(kern, smem_ok[ovf_row_ptr ? 1 : 0]))
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
