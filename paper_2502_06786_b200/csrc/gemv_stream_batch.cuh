// Decode GEMV for small batches (2 <= B <= 8 activation vectors per problem) in the persistent kernel of
// gemv_stream.cuh: the same list, the same partition into (16-row tile x 64-byte chunk) items, the same producer warp
// and ring; what differs is what the multiplying warps do with a unit.
//
// Columns.  The integer MMA (m16n8k32, u8 x u8 -> s32) has eight B columns.  For a single vector gemv_stream uses
// five: the four bytes of a 30-bit block-scaled activation and a constant column.  Here a GROUP of columns serves TWO
// activation vectors: three bytes each of a 22-bit block-scaled activation (every vector with its own power-of-two
// scale, taken from its largest magnitude) and the constant column, seven of the eight.  A batch of B vectors is
// G = ceil(B / 2) groups.  A fragment of weights (the plane's bytes masked in place, nested masks as in
// gemv_stream) is loaded and masked ONCE and multiplied with the G groups' B fragments, so the shared-memory loads
// of the plane, the mask instructions and, above all, the HBM traffic of the plane do not grow with B; the MMAs and
// the B-fragment loads do (G per fragment of weights).
//   22 bits: an activation is rounded to 2^-22 of the largest magnitude of its vector, an error of about
//   2^-23 max|x| / rms(x) of rms(y), far below the tolerance of the batched paths (1e-2 rms(y)) and of the
//   bf16 inputs themselves (8 significant bits).
//
// Accumulators.  The eight accumulator sets of a warp are split over the groups (8 / G sets each); the MMAs of one
// fragment go to G different sets and successive fragments rotate through a group's sets, so the same set is used
// again after eight MMAs, as in the single-vector kernel.
//
// Staging.  The activations of the current problem are kept in shared memory as byte units in B-fragment order, one
// region per group: per (chunk, 16-weight unit) six column blocks of 64 bytes (bytes 0-2 of the first vector, 0-2 of
// the second; the constant column is held in registers by the lanes of column 6).  A CTA converts only the problems
// its share of the list touches (one or two when a call covers a whole decoder stack), which is what makes batches
// affordable here: a kernel per matrix has every CTA convert all B vectors for every matrix.
//
// Not here: extra-precision lists with B > 1 (those calls keep the bf16 kernel of gemv_tensor.cuh), r = 2 planes
// whose K is not a multiple of 256.  Batches above 8, or above what the staged activations of a long row leave room
// for, are cut into problems that share the plane; the later ones find it in the L2.
//
// Quad groups.  At r = 8 and r = 4, batches of three or more vectors use a second column layout (further down): four
// vectors per group as two signed digits each, a u8 x s8 MMA, no constant column; half the MMAs and fragment loads
// for the same vectors, up to 16 vectors per problem, 15-bit activations instead of 22-bit ones.
#pragma once
#include <vector>

#include "gemv_stream.cuh"

namespace matq {
namespace gstream {

constexpr int kP2 = 21;                      // batched activations become integers below 2^(kP2 + 1)
constexpr int kPairCols = 7;                 // columns of a group: 3 + 3 bytes and the constant column
constexpr int kPairUnit = (kPairCols - 1) * 64;   // bytes of a staged (chunk, unit) block: the six byte columns (the constant column lives in registers)
constexpr int kMaxBatch = 8;                 // vectors of a problem in pair groups (4 groups of 2)
constexpr int kP4 = 14;                      // quad groups: activations become integers of magnitude below 2^(kP4 + 1)
constexpr int kQuadUnit = 8 * 64;            // bytes of a staged (chunk, unit) block of a quad group: two signed digits of four vectors
constexpr int kMaxVec = 16;                  // vectors of a problem in quad groups (4 groups of 4)
constexpr int kWideFit = 7;                  // stages a problem's own shapes must leave room for to share a launch with the short rows

// Staged bytes of one group for a problem (all chunks of a row).
inline size_t xs_group_bytes_of(const Geo& g, int r, bool quad = false) { return (size_t)g.n_qc * ((128 / r) / 16) * (quad ? kQuadUnit : kPairUnit); }

// Converts 16 consecutive activations of the two vectors of a group and stores their byte units: column blocks 0-2
// (first vector) and 3-5 (second).  `dst` points at this item's 16 bytes of column block 0.
template <int R>
__device__ __forceinline__ void stage_item_pair(const uint32_t (&rawa)[8], const uint32_t (&rawb)[8], const float (&multa)[8 / R],
                                                const float (&multb)[8 / R], uint4* dst) {
    constexpr int kF = 8 / R;
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        int V[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const uint32_t w = half ? rawb[i >> 1] : rawa[i >> 1];
            const float xf = (i & 1) ? bf_hi(w) : bf_lo(w);
            V[i] = __float2int_rn(xf * (half ? multb[i % kF] : multa[i % kF]));
        }
        uint32_t v[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int cls = i % kF;
            const int y = cls == kF - 1 ? V[i] : V[i] - V[i + 1 < 16 ? i + 1 : i];
            v[i] = (uint32_t)y + (1u << (kP2 + 2 - R * cls));
        }
        uint32_t col[3][4];
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint32_t e0 = v[imma::unit_src<R>(4 * w)], e1 = v[imma::unit_src<R>(4 * w + 1)];
            const uint32_t e2 = v[imma::unit_src<R>(4 * w + 2)], e3 = v[imma::unit_src<R>(4 * w + 3)];
            const uint32_t t0 = __byte_perm(e0, e1, 0x5140), t1 = __byte_perm(e2, e3, 0x5140);
            const uint32_t t2 = __byte_perm(e0, e1, 0x7362), t3 = __byte_perm(e2, e3, 0x7362);
            col[0][w] = __byte_perm(t0, t1, 0x5410);  col[1][w] = __byte_perm(t0, t1, 0x7632);
            col[2][w] = __byte_perm(t2, t3, 0x5410);
        }
#pragma unroll
        for (int d = 0; d < 3; ++d) dst[4 * (3 * half + d)] = make_uint4(col[d][0], col[d][1], col[d][2], col[d][3]);
    }
}

// Stages the B vectors of a problem (rows of x, K apart): per vector the largest magnitude and the fp32 sum, reduced
// over the CTA (s_xexp / s_xsum: biased exponent of the scale and the sum, per vector), then the byte units of every
// group.  Three named barriers; the first also separates the previous problem's multiplies from the restaging.
template <int R, int G>
__device__ __forceinline__ void stage_activations_pair(const __nv_bfloat16* x, int K, int B, int n_qc, unsigned char* xs, size_t group_bytes,
                                                       int ctid, int nthr, int W, uint32_t (*s_cmax)[kMaxBatch], float (*s_csum)[kMaxBatch],
                                                       int* s_xexp, float* s_xsum) {
    constexpr int kWpp = 128 / R;
    constexpr int kM2 = kWpp / 16;
    constexpr int kF = 8 / R;
    const int lane = ctid & 31, warp = ctid >> 5;
    const int n_items = n_qc * kM2 * 4;
    auto k0_of = [&](int it) {
        const int tt = it & 3, qm = it >> 2;
        return ((qm / kM2) * 4 + tt) * kWpp + (qm % kM2) * 16;
    };
    for (int c = 0; c < 2 * G; ++c) {
        uint32_t xmax = 0;
        float xsum = 0.f;
        if (c < B) {
            const __nv_bfloat16* xc = x + (size_t)c * K;
            for (int it = ctid; it < n_items; it += nthr) {
                const int k0 = k0_of(it);
                if (k0 >= K) continue;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 v = ld_x4(xc + k0 + 8 * h);
                    xmax = __vmaxu2(xmax, v.x & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.y & 0x7fff7fffu);
                    xmax = __vmaxu2(xmax, v.z & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.w & 0x7fff7fffu);
                }
            }
            // the sum in an order that does not depend on the number of consumer warps (see stage_activations)
            if (ctid < kSumThreads)
                for (int it = ctid; it < n_items; it += kSumThreads) {
                    const int k0 = k0_of(it);
                    if (k0 >= K) continue;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint4 v = ld_x4(xc + k0 + 8 * h);
                        xsum += ((bf_lo(v.x) + bf_hi(v.x)) + (bf_lo(v.y) + bf_hi(v.y))) + ((bf_lo(v.z) + bf_hi(v.z)) + (bf_lo(v.w) + bf_hi(v.w)));
                    }
                }
        }
        xmax = max(xmax & 0xffffu, xmax >> 16);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
            xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
        }
        if (lane == 0) { s_cmax[warp][c] = xmax; s_csum[warp][c] = xsum; }
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
    if (ctid < 2 * G) {
        uint32_t xmax = 0;
        float xsum = 0.f;
        for (int w = 0; w < W; ++w) xmax = max(xmax, s_cmax[w][ctid]);
        for (int w = 0; w < kSumThreads / 32; ++w) xsum += s_csum[w][ctid];
        s_xexp[ctid] = min(max((int)(xmax >> 7), kP2 + 1), 254);
        s_xsum[ctid] = xsum;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
#pragma unroll 1
    for (int g = 0; g < G; ++g) {
        const int ca = 2 * g, cb = 2 * g + 1;
        float multa[kF], multb[kF];
#pragma unroll
        for (int cls = 0; cls < kF; ++cls) {
            multa[cls] = __uint_as_float((uint32_t)(254 + kP2 - s_xexp[ca] - R * cls) << 23);
            multb[cls] = __uint_as_float((uint32_t)(254 + kP2 - s_xexp[cb] - R * cls) << 23);
        }
        const __nv_bfloat16* xa = x + (size_t)ca * K;
        const __nv_bfloat16* xb = x + (size_t)cb * K;
        uint4* xg = reinterpret_cast<uint4*>(xs + (size_t)g * group_bytes);
        for (int it = ctid; it < n_items; it += nthr) {
            uint4* dst = xg + (size_t)(it >> 2) * (kPairUnit / 16) + (it & 3);
            const int k0 = k0_of(it);
            uint32_t rawa[8] = {0, 0, 0, 0, 0, 0, 0, 0}, rawb[8] = {0, 0, 0, 0, 0, 0, 0, 0};
            if (k0 < K && ca < B) {
                const uint4 va = ld_x4(xa + k0), vb = ld_x4(xa + k0 + 8);
                rawa[0] = va.x; rawa[1] = va.y; rawa[2] = va.z; rawa[3] = va.w; rawa[4] = vb.x; rawa[5] = vb.y; rawa[6] = vb.z; rawa[7] = vb.w;
            }
            if (k0 < K && cb < B) {
                const uint4 va = ld_x4(xb + k0), vb = ld_x4(xb + k0 + 8);
                rawb[0] = va.x; rawb[1] = va.y; rawb[2] = va.z; rawb[3] = va.w; rawb[4] = vb.x; rawb[5] = vb.y; rawb[6] = vb.z; rawb[7] = vb.w;
            }
            if (k0 < K) {
                stage_item_pair<R>(rawa, rawb, multa, multb, dst);
            } else {
#pragma unroll
                for (int d = 0; d < 6; ++d) dst[4 * d] = make_uint4(0, 0, 0, 0);      // past the end of the row: no offsets either
            }
        }
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
}

// One (tile, chunk) item against the G groups.  `x_sa`: shared address of this lane's 16 bytes in column block
// (lane >> 2) of the chunk's first unit in group 0; the next unit kPairUnit further, the next group `xg_bytes`.
// Fragment f of the item goes, for group g, to accumulator set g * (kSets / G) + (F0 + f) % (kSets / G).
template <int R, int G, int F0>
__device__ __forceinline__ void multiply_item_pair(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, uint32_t xg_bytes, int col_lane,
                                                   const uint4& cz, int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kS = kSets / G;
    const uint4 wl = *reinterpret_cast<const uint4*>(wl_p);
    const uint4 wh = *reinterpret_cast<const uint4*>(wh_p);
#pragma unroll
    for (int m2 = 0; m2 < kM2; ++m2) {
        uint4 xb[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            xb[g] = cz;
            lds128_if(xb[g], x_sa + (uint32_t)g * xg_bytes + m2 * kPairUnit, col_lane);
        }
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            uint32_t a0, a1, a2, a3;
            if (R == 8) {
                a0 = sub ? wl.z : wl.x;  a2 = sub ? wl.w : wl.y;
                a1 = sub ? wh.z : wh.x;  a3 = sub ? wh.w : wh.y;
            } else {
                const int j = R == 4 ? 2 * m2 + sub : m2;
                const uint32_t w_lo = j == 0 ? wl.x : j == 1 ? wl.y : j == 2 ? wl.z : wl.w;
                const uint32_t w_hi = j == 0 ? wh.x : j == 1 ? wh.y : j == 2 ? wh.z : wh.w;
                if (R == 4) {
                    a0 = w_lo & 0x0f0f0f0fu;  a2 = w_lo;
                    a1 = w_hi & 0x0f0f0f0fu;  a3 = w_hi;
                } else if (sub == 0) {
                    a0 = w_lo & 0x03030303u;  a2 = w_lo & 0x0f0f0f0fu;
                    a1 = w_hi & 0x03030303u;  a3 = w_hi & 0x0f0f0f0fu;
                } else {
                    a0 = w_lo & 0x3f3f3f3fu;  a2 = w_lo;
                    a1 = w_hi & 0x3f3f3f3fu;  a3 = w_hi;
                }
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint32_t b0 = sub ? xb[g].z : xb[g].x, b1 = sub ? xb[g].w : xb[g].y;
                imma::mma_u8u8(acc[g * kS + (F0 + 2 * m2 + sub) % kS], a0, a1, a2, a3, b0, b1);
            }
        }
    }
}

// All chunks of one unit's tile panel against the G groups.
template <int R, int G>
__device__ __forceinline__ void multiply_unit_pair(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, int xq_bytes, uint32_t xg_bytes,
                                                   int col_lane, const uint4& cz, int n_chunks, int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kFrag = 2 * kM2;                                   // fragments of an item
    constexpr int kS = kSets / G;
    constexpr int kU = kS > kFrag ? kS / kFrag : (R == 8 ? 2 : 1);   // items per round: a round uses every set of a group; at r = 8 at least
                                                                     // two, so that the loads of the second item are in flight during the first's MMAs
#define MATQ_PITEM(I) multiply_item_pair<R, G, ((I) * kFrag) % kS>(wl_p + (c + (I)) * 64, wh_p + (c + (I)) * 64, x_sa + (uint32_t)((c + (I)) * xq_bytes), xg_bytes, col_lane, cz, acc)
    int c = 0;
#pragma unroll 1
    for (; c + kU <= n_chunks; c += kU) {
        MATQ_PITEM(0);
        if (kU >= 2) MATQ_PITEM(1);
        if (kU >= 4) { MATQ_PITEM(2); MATQ_PITEM(3); }
    }
#pragma unroll 1
    for (; c < n_chunks; ++c) MATQ_PITEM(0);
#undef MATQ_PITEM
}

// Finishes one tile for the two vectors of a group.  Accumulator a_i of thread (g, t) holds row g + 8 (i >> 1), column
// 2t + (i & 1): columns 0-2 are the bytes of the first vector's sum, 3-5 of the second's, 6 the constant column.  The
// lanes t = 0 gather a row's seven columns and recombine them in 64 bits; `scales`: alpha of row (lane) in lanes 0-15,
// zero of row (lane - 16) in lanes 16-31.  `yb` is null when the group has one vector.  Called by whole warps.
__device__ __noinline__ void finish_tile_pair(float* __restrict__ ya, float* __restrict__ yb, int N, int sh, int xexp_a, int xexp_b, float xsum_a,
                                              float xsum_b, long long row0, int a0, int a1, int a2, int a3, float scales, int lane, bool store) {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int c0 = h ? a2 : a0, c1 = h ? a3 : a1;
        const int c2 = __shfl_down_sync(0xffffffffu, c0, 1), c3 = __shfl_down_sync(0xffffffffu, c1, 1);
        const int c4 = __shfl_down_sync(0xffffffffu, c0, 2), c5 = __shfl_down_sync(0xffffffffu, c1, 2);
        const int c6 = __shfl_down_sync(0xffffffffu, c0, 3);
        const float al = __shfl_sync(0xffffffffu, scales, g + 8 * h), ze = __shfl_sync(0xffffffffu, scales, 16 + g + 8 * h);
        const long long row = row0 + g + 8 * h;
        if (t != 0 || row >= N || !store) continue;
        const long long off = (long long)c6 << (kP2 + 2 - sh);
        const long long ta = (((long long)c2 * 256 + c1) * 256 + c0) - off;
        const float va = __ll2float_rn(ta) * __uint_as_float((uint32_t)(xexp_a - kP2) << 23);
        ya[row] = al * (va * (float)(1 << sh) - ze * xsum_a);
        if (yb) {
            const long long tb = (((long long)c5 * 256 + c4) * 256 + c3) - off;
            const float vb = __ll2float_rn(tb) * __uint_as_float((uint32_t)(xexp_b - kP2) << 23);
            yb[row] = al * (vb * (float)(1 << sh) - ze * xsum_b);
        }
    }
}


// ---------------------------------------------------------------------------------------------------------------
// Quad groups (r = 8 and r = 4, three or more vectors): the eight B columns of a group are TWO SIGNED digits (base 256,
// each in [-128, 127]) of FOUR vectors; the MMA is u8 x s8, there is no offset and no constant column, and column
// 2v + d of the result is digit d of vector v's sum, so thread (g, t) of the accumulator fragment holds both digits of
// vector t for its two rows.  Half the MMAs and B-fragment loads of pair groups for the same vectors.  An activation
// is rounded to an integer of magnitude at most 2^15 - 256 (15 bits and the sign: 2^-14 of the power of two at or
// below the vector's largest magnitude, one bit less when that magnitude's significand is all ones).  At r = 4 the
// upper field is shifted down instead of being left in place, so both fields meet activations of the same scale.

__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
    uint4 v;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// 16 consecutive activations of one vector as two signed digits: `dst` points at this item's 16 bytes of the vector's
// low-digit column block, the high-digit block follows it.
template <int R>
__device__ __forceinline__ void stage_item_quad(const uint32_t (&raw)[8], float mult, uint4* dst) {
    uint32_t u[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const uint32_t w = raw[i >> 1];
        const int V = __float2int_rn(((i & 1) ? bf_hi(w) : bf_lo(w)) * mult);
        u[i] = (uint32_t)(V + ((V & 0x80) << 1));             // low byte as a signed digit: the high byte takes the carry
    }
    uint32_t col[2][4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const uint32_t e0 = u[imma::unit_src<R>(4 * w)], e1 = u[imma::unit_src<R>(4 * w + 1)];
        const uint32_t e2 = u[imma::unit_src<R>(4 * w + 2)], e3 = u[imma::unit_src<R>(4 * w + 3)];
        const uint32_t t0 = __byte_perm(e0, e1, 0x5140), t1 = __byte_perm(e2, e3, 0x5140);
        col[0][w] = __byte_perm(t0, t1, 0x5410);  col[1][w] = __byte_perm(t0, t1, 0x7632);
    }
    dst[0] = make_uint4(col[0][0], col[0][1], col[0][2], col[0][3]);
    dst[4] = make_uint4(col[1][0], col[1][1], col[1][2], col[1][3]);
}

// As stage_activations_pair, for G groups of four vectors.
template <int R, int G>
__device__ __forceinline__ void stage_activations_quad(const __nv_bfloat16* x, int K, int B, int n_qc, unsigned char* xs, size_t group_bytes,
                                                       int ctid, int nthr, int W, uint32_t (*s_cmax)[kMaxVec], float (*s_csum)[kMaxVec],
                                                       int* s_xexp, float* s_xsum) {
    constexpr int kWpp = 128 / R;
    constexpr int kM2 = kWpp / 16;
    const int lane = ctid & 31, warp = ctid >> 5;
    const int n_items = n_qc * kM2 * 4;
    auto k0_of = [&](int it) {
        const int tt = it & 3, qm = it >> 2;
        return ((qm / kM2) * 4 + tt) * kWpp + (qm % kM2) * 16;
    };
    for (int c = 0; c < 4 * G; ++c) {
        uint32_t xmax = 0;
        float xsum = 0.f;
        if (c < B) {
            const __nv_bfloat16* xc = x + (size_t)c * K;
            for (int it = ctid; it < n_items; it += nthr) {
                const int k0 = k0_of(it);
                if (k0 >= K) continue;
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const uint4 v = ld_x4(xc + k0 + 8 * h);
                    xmax = __vmaxu2(xmax, v.x & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.y & 0x7fff7fffu);
                    xmax = __vmaxu2(xmax, v.z & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.w & 0x7fff7fffu);
                }
            }
            if (ctid < kSumThreads)                                // fixed order: see stage_activations
                for (int it = ctid; it < n_items; it += kSumThreads) {
                    const int k0 = k0_of(it);
                    if (k0 >= K) continue;
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint4 v = ld_x4(xc + k0 + 8 * h);
                        xsum += ((bf_lo(v.x) + bf_hi(v.x)) + (bf_lo(v.y) + bf_hi(v.y))) + ((bf_lo(v.z) + bf_hi(v.z)) + (bf_lo(v.w) + bf_hi(v.w)));
                    }
                }
        }
        xmax = max(xmax & 0xffffu, xmax >> 16);
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
            xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
        }
        if (lane == 0) { s_cmax[warp][c] = xmax; s_csum[warp][c] = xsum; }
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
    if (ctid < 4 * G) {
        uint32_t xmax = 0;
        float xsum = 0.f;
        for (int w = 0; w < W; ++w) xmax = max(xmax, s_cmax[w][ctid]);
        for (int w = 0; w < kSumThreads / 32; ++w) xsum += s_csum[w][ctid];
        // biased exponent of the scale; a largest magnitude with an all-ones significand would round to 2^15 - 128, one
        // more than two signed digits hold, and takes the next power of two
        const int e = (int)(xmax >> 7) + ((xmax & 0x7fu) == 0x7fu ? 1 : 0);
        s_xexp[ctid] = min(max(e, kP4 + 1), 254);
        s_xsum[ctid] = xsum;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
#pragma unroll 1
    for (int c = 0; c < 4 * G; ++c) {
        const float mult = __uint_as_float((uint32_t)(254 + kP4 - s_xexp[c]) << 23);
        const __nv_bfloat16* xc = x + (size_t)c * K;
        uint4* xg = reinterpret_cast<uint4*>(xs + (size_t)(c >> 2) * group_bytes) + 8 * (c & 3);      // column blocks 2v, 2v + 1
        for (int it = ctid; it < n_items; it += nthr) {
            uint4* dst = xg + (size_t)(it >> 2) * (kQuadUnit / 16) + (it & 3);
            const int k0 = k0_of(it);
            if (k0 < K && c < B) {
                const uint4 va = ld_x4(xc + k0), vb = ld_x4(xc + k0 + 8);
                const uint32_t raw[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
                stage_item_quad<R>(raw, mult, dst);
            } else {
                dst[0] = make_uint4(0, 0, 0, 0);                  // past the end of the row, or no such vector
                dst[4] = make_uint4(0, 0, 0, 0);
            }
        }
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
}

// One (tile, chunk) item against the G quad groups; arguments as for multiply_item_pair, every lane loads its column.
template <int R, int G, int F0>
__device__ __forceinline__ void multiply_item_quad(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, uint32_t xg_bytes,
                                                   int (&acc)[kSets][4]) {
    static_assert(R == 8 || R == 4, "quad groups serve r = 8 and r = 4");
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kS = kSets / G;
    const uint4 wl = *reinterpret_cast<const uint4*>(wl_p);
    const uint4 wh = *reinterpret_cast<const uint4*>(wh_p);
#pragma unroll
    for (int m2 = 0; m2 < kM2; ++m2) {
        uint4 xb[G];
#pragma unroll
        for (int g = 0; g < G; ++g) xb[g] = lds128(x_sa + (uint32_t)g * xg_bytes + m2 * kQuadUnit);
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            uint32_t a0, a1, a2, a3;
            if (R == 8) {
                a0 = sub ? wl.z : wl.x;  a2 = sub ? wl.w : wl.y;
                a1 = sub ? wh.z : wh.x;  a3 = sub ? wh.w : wh.y;
            } else {
                const int j = 2 * m2 + sub;
                const uint32_t w_lo = j == 0 ? wl.x : j == 1 ? wl.y : j == 2 ? wl.z : wl.w;
                const uint32_t w_hi = j == 0 ? wh.x : j == 1 ? wh.y : j == 2 ? wh.z : wh.w;
                a0 = w_lo & 0x0f0f0f0fu;  a2 = (w_lo >> 4) & 0x0f0f0f0fu;
                a1 = w_hi & 0x0f0f0f0fu;  a3 = (w_hi >> 4) & 0x0f0f0f0fu;
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const uint32_t b0 = sub ? xb[g].z : xb[g].x, b1 = sub ? xb[g].w : xb[g].y;
                mma_u8s8(acc[g * kS + (F0 + 2 * m2 + sub) % kS], a0, a1, a2, a3, b0, b1);
            }
        }
    }
}

template <int R, int G>
__device__ __forceinline__ void multiply_unit_quad(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, int xq_bytes, uint32_t xg_bytes,
                                                   int n_chunks, int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kFrag = 2 * kM2;
    constexpr int kS = kSets / G;
    constexpr int kU = kS > kFrag ? kS / kFrag : (R == 8 ? 2 : 1);   // as in multiply_unit_pair
#define MATQ_QITEM(I) multiply_item_quad<R, G, ((I) * kFrag) % kS>(wl_p + (c + (I)) * 64, wh_p + (c + (I)) * 64, x_sa + (uint32_t)((c + (I)) * xq_bytes), xg_bytes, acc)
    int c = 0;
#pragma unroll 1
    for (; c + kU <= n_chunks; c += kU) {
        MATQ_QITEM(0);
        if (kU >= 2) MATQ_QITEM(1);
        if (kU >= 4) { MATQ_QITEM(2); MATQ_QITEM(3); }
    }
#pragma unroll 1
    for (; c < n_chunks; ++c) MATQ_QITEM(0);
#undef MATQ_QITEM
}

// Finishes one tile for the (up to four) vectors of a quad group.  Thread (g, t) holds, for rows g and g + 8, the low
// and the high digit of vector t's sum; `yq`: y of the group's first vector, `xexp` / `xsum`: the group's entries of the
// per-vector scale exponents and sums (shared memory), `nvec`: vectors the group really has.  Called by whole warps.
__device__ __noinline__ void finish_tile_quad(float* __restrict__ yq, int N, int nvec, int sh, const int* xexp, const float* xsum, long long row0,
                                              int a0, int a1, int a2, int a3, float scales, int lane, bool store) {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        const int lo = h ? a2 : a0, hi = h ? a3 : a1;
        const float al = __shfl_sync(0xffffffffu, scales, g + 8 * h), ze = __shfl_sync(0xffffffffu, scales, 16 + g + 8 * h);
        const long long row = row0 + g + 8 * h;
        if (t >= nvec || row >= N || !store) continue;
        const long long tot = (long long)hi * 256 + lo;
        const float v = __ll2float_rn(tot) * __uint_as_float((uint32_t)(xexp[t] - kP4) << 23);
        yq[(size_t)t * N + row] = al * (v * (float)(1 << sh) - ze * xsum[t]);
    }
}

// Q: quad groups (see above) instead of pair groups; the problems of such a launch are all at r = 8 or r = 4.
template <int NP, int G, bool Q>
__global__ void __launch_bounds__((kMaxW + 1) * 32, 1)
gemv_stream_batch(const __grid_constant__ Params<NP> P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_full[kMaxSlots], s_empty[kMaxSlots];
    __shared__ int s_tile[kTileSlots][G][16][imma::kCols];     // sums of tiles whose panels are spread over warps
    __shared__ int s_tile_cnt[kTileSlots];
    constexpr int kVec = Q ? kMaxVec : kMaxBatch;
    __shared__ uint32_t s_cmax[kMaxW][kVec];
    __shared__ float s_csum[kMaxW][kVec];
    __shared__ int s_xexp[kVec];
    __shared__ float s_xsum[kVec];
    __shared__ int s_abort;
    constexpr int kS = kSets / G;

    const int W = P.W;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthr = W * 32;
    unsigned char* xs = smem_raw;
    unsigned char* ring = smem_raw + P.xs_bytes;
    volatile int* abort_flag = &s_abort;

    if (tid == 0) s_abort = 0;
    if (tid < P.slots) {
        mbar_init(smem_u32(&s_full[tid]), 1);
        mbar_init(smem_u32(&s_empty[tid]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < kTileSlots * G * 16 * imma::kCols; i += blockDim.x) (&s_tile[0][0][0][0])[i] = 0;
    if (tid < kTileSlots) s_tile_cnt[tid] = 0;
    __syncthreads();
    if (P.pdl) asm volatile("griddepcontrol.launch_dependents;");

    const long long lo = P.items * blockIdx.x / gridDim.x, hi = P.items * (blockIdx.x + 1) / gridDim.x;
    int p_first = 0;
    {
        int a = 0, b = P.n - 1;
        while (a < b) {
            const int m = (a + b + 1) >> 1;
            if (P.p[m].item0 <= lo) a = m; else b = m - 1;
        }
        p_first = a;
    }

    if (warp == W) {
        producer_warp(P, lo, hi, p_first, W, ring, s_full, s_empty, abort_flag, lane);
    } else {
        const int g = lane >> 2, t = lane & 3;
        const int ctid = tid;
        int it0 = 0, split_tiles = 0;
        int p = p_first, t_lo, t_hi, tail_lo = -1, tail_hi = 0, staged_p = -1;
        bool first = true;
        while (next_segment(P, lo, hi, p, t_lo, t_hi, tail_lo, tail_hi)) {
            const Problem& pr = P.p[p - 1];
            const Geo GE = geometry(pr.N, pr.K, pr.r, P.unit_row);
            const int R = pr.r;
            const int sh = kCodeBits - R;
            const int T = t_hi - t_lo;
            const int B = pr.B;
            const Plan pl = plan_of(GE, T, W);
            {
                // alpha and zero of this CTA's rows into the L2 (they do not depend on the previous kernel)
                const long long r0 = (long long)t_lo * 16, r1 = min((long long)t_hi * 16, (long long)pr.N);
                for (long long rr = r0 + (long long)ctid * 32; rr < r1; rr += (long long)nthr * 32) {
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(pr.alpha + rr));
                    asm volatile("prefetch.global.L2 [%0];" ::"l"(pr.zero + rr));
                }
            }
            if (first) {
                for (int i = ctid * 64; i < pr.K * B; i += nthr * 64) asm volatile("prefetch.global.L2 [%0];" ::"l"(pr.x + i));
                if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
            }
            first = false;

            const int kM2 = (128 / R) / 16;
            constexpr int kUnit = Q ? kQuadUnit : kPairUnit;
            const size_t group_bytes = (size_t)GE.n_qc * kM2 * kUnit;
            if (staged_p == p) {                                  // the second segment of a problem finds them staged
            } else if constexpr (Q) {
                if (R == 8) stage_activations_quad<8, G>(pr.x, pr.K, B, GE.n_qc, xs, group_bytes, ctid, nthr, W, (uint32_t (*)[kMaxVec])s_cmax, (float (*)[kMaxVec])s_csum, s_xexp, s_xsum);
                else stage_activations_quad<4, G>(pr.x, pr.K, B, GE.n_qc, xs, group_bytes, ctid, nthr, W, (uint32_t (*)[kMaxVec])s_cmax, (float (*)[kMaxVec])s_csum, s_xexp, s_xsum);
            } else if (R == 8) stage_activations_pair<8, G>(pr.x, pr.K, B, GE.n_qc, xs, group_bytes, ctid, nthr, W, (uint32_t (*)[kMaxBatch])s_cmax, (float (*)[kMaxBatch])s_csum, s_xexp, s_xsum);
            else if (R == 4) stage_activations_pair<4, G>(pr.x, pr.K, B, GE.n_qc, xs, group_bytes, ctid, nthr, W, (uint32_t (*)[kMaxBatch])s_cmax, (float (*)[kMaxBatch])s_csum, s_xexp, s_xsum);
            else stage_activations_pair<2, G>(pr.x, pr.K, B, GE.n_qc, xs, group_bytes, ctid, nthr, W, (uint32_t (*)[kMaxBatch])s_cmax, (float (*)[kMaxBatch])s_csum, s_xexp, s_xsum);
            staged_p = p;

            // this lane's B source: column block g of a unit; the lanes g = 6 hold the constant column in registers
            // (quad groups: every lane loads its column, there is no constant column)
            const int col_lane = (Q || g < kPairCols - 1) ? 1 : 0;
            const uint32_t x_sa0 = smem_u32(xs) + (uint32_t)(((Q || g < kPairCols - 1) ? g : 0) * 4 + t) * 16u;
            const int xq_bytes = kM2 * kUnit;
            uint4 cz = make_uint4(0, 0, 0, 0);
            if (!Q && g == kPairCols - 1) {
                if (R == 8) cz = make_uint4(imma::ones_b0<8>(0), imma::ones_b1<8>(0), imma::ones_b0<8>(1), imma::ones_b1<8>(1));
                else if (R == 4) cz = make_uint4(imma::ones_b0<4>(0), imma::ones_b1<4>(0), imma::ones_b0<4>(1), imma::ones_b1<4>(1));
                else cz = make_uint4(imma::ones_b0<2>(0), imma::ones_b1<2>(0), imma::ones_b0<2>(1), imma::ones_b1<2>(1));
            }

            auto multiply = [&](const unsigned char* tile_rows, int pn, int (&acc)[kSets][4]) {
                const int q0 = pn * GE.panel_qc, q1 = min(q0 + GE.panel_qc, GE.n_qc);
                const unsigned char* base = tile_rows + t * 16;
                const unsigned char* wl_p = base + (size_t)g * GE.stride;
                const unsigned char* wh_p = base + (size_t)(g + 8) * GE.stride;
                const uint32_t x_sa = x_sa0 + (uint32_t)(q0 * xq_bytes);
                if constexpr (Q) {
                    if (R == 8) multiply_unit_quad<8, G>(wl_p, wh_p, x_sa, xq_bytes, (uint32_t)group_bytes, q1 - q0, acc);
                    else multiply_unit_quad<4, G>(wl_p, wh_p, x_sa, xq_bytes, (uint32_t)group_bytes, q1 - q0, acc);
                } else if (R == 8) multiply_unit_pair<8, G>(wl_p, wh_p, x_sa, xq_bytes, (uint32_t)group_bytes, col_lane, cz, q1 - q0, acc);
                else if (R == 4) multiply_unit_pair<4, G>(wl_p, wh_p, x_sa, xq_bytes, (uint32_t)group_bytes, col_lane, cz, q1 - q0, acc);
                else multiply_unit_pair<2, G>(wl_p, wh_p, x_sa, xq_bytes, (uint32_t)group_bytes, col_lane, cz, q1 - q0, acc);
            };
            auto zero_acc = [&](int (&acc)[kSets][4]) {
#pragma unroll
                for (int c2 = 0; c2 < kSets; ++c2)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[c2][i] = 0;
            };
            // the sets of group gg summed into its first one
            auto fold = [&](int (&acc)[kSets][4]) {
#pragma unroll
                for (int gg = 0; gg < G; ++gg)
#pragma unroll
                    for (int c2 = 1; c2 < kS; ++c2)
#pragma unroll
                        for (int i = 0; i < 4; ++i) acc[gg * kS][i] += acc[gg * kS + c2][i];
            };
            int acc[kSets][4] = {};
            // scales and stores the 16 rows of a tile for every group (the sums of group gg in acc[gg * kS])
            auto finish = [&](long long row0) {
                const long long row = row0 + (lane & 15);
                float scales = 0.f;
                if (row < pr.N) scales = lane < 16 ? pr.alpha[row] : pr.zero[row];
                const bool store = !*abort_flag;
                if constexpr (Q) {
#pragma unroll
                    for (int gg = 0; gg < G; ++gg) {
                        if (4 * gg >= B) break;
                        finish_tile_quad(pr.y + (size_t)(4 * gg) * pr.N, pr.N, min(4, B - 4 * gg), sh, s_xexp + 4 * gg, s_xsum + 4 * gg, row0,
                                         acc[gg * kS][0], acc[gg * kS][1], acc[gg * kS][2], acc[gg * kS][3], scales, lane, store);
                    }
                    return;
                }
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    if (2 * gg >= B) break;
                    float* ya = pr.y + (size_t)(2 * gg) * pr.N;
                    float* yb = 2 * gg + 1 < B ? pr.y + (size_t)(2 * gg + 1) * pr.N : nullptr;
                    finish_tile_pair(ya, yb, pr.N, sh, s_xexp[2 * gg], s_xexp[2 * gg + 1], s_xsum[2 * gg], s_xsum[2 * gg + 1], row0,
                                     acc[gg * kS][0], acc[gg * kS][1], acc[gg * kS][2], acc[gg * kS][3], scales, lane, store);
                }
            };
            const int contributors = min(GE.n_panels, W);
            int cur = -1;
            // split mode: this warp's partial sums of tile `cur` go to the tile's accumulators in shared memory; the warp
            // that brings the last contribution takes the totals back into acc[gg * kS] and returns true
            auto merge_split = [&]() -> bool {
                fold(acc);
                const int ts = (split_tiles + cur) % kTileSlots;
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    atomicAdd(&s_tile[ts][gg][g][2 * t], acc[gg * kS][0]);
                    atomicAdd(&s_tile[ts][gg][g + 8][2 * t], acc[gg * kS][2]);
                    if (Q || t < 3) { atomicAdd(&s_tile[ts][gg][g][2 * t + 1], acc[gg * kS][1]); atomicAdd(&s_tile[ts][gg][g + 8][2 * t + 1], acc[gg * kS][3]); }
                }
                __threadfence_block();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(&s_tile_cnt[ts], 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev != contributors - 1) return false;
                __threadfence_block();
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {
                    acc[gg * kS][0] = s_tile[ts][gg][g][2 * t];          acc[gg * kS][2] = s_tile[ts][gg][g + 8][2 * t];
                    acc[gg * kS][1] = s_tile[ts][gg][g][2 * t + 1];      acc[gg * kS][3] = s_tile[ts][gg][g + 8][2 * t + 1];
                }
                __syncwarp();
#pragma unroll
                for (int gg = 0; gg < G; ++gg) {                       // leave the slot clean for the tile that reuses it
                    s_tile[ts][gg][g][2 * t] = 0;      s_tile[ts][gg][g + 8][2 * t] = 0;
                    s_tile[ts][gg][g][2 * t + 1] = 0;  s_tile[ts][gg][g + 8][2 * t + 1] = 0;
                }
                if (lane == 0) s_tile_cnt[ts] = 0;
                return true;
            };
            const int step_t = pl.split ? W / GE.n_panels : 0, step_p = pl.split ? W % GE.n_panels : 0;
            int tj = pl.split ? warp / GE.n_panels : warp * pl.tpu;
            int pn = pl.split ? warp % GE.n_panels : 0;
            int slot = (it0 + warp) % P.slots;
            uint32_t parity = (uint32_t)(((it0 + warp) / P.slots) & 1);
            for (int s = warp; s < pl.n_units; s += W) {
                const int n_tiles = tj < T ? min(pl.tpu, T - tj) : 0;
                if (pl.split) {
                    if (n_tiles && tj != cur) {
                        if (cur >= 0 && merge_split()) finish((long long)(t_lo + cur) * 16);
                        cur = tj;
                        zero_acc(acc);
                    }
                } else if (pn == 0) {
                    zero_acc(acc);
                }
                const bool landed = wait_phase(smem_u32(&s_full[slot]), parity, abort_flag, P.wait_cycles);
                const unsigned char* rows = ring + (size_t)slot * P.slot_bytes;
                const bool tile_done = !pl.split && pn == GE.n_panels - 1;
                for (int k = 0; k < n_tiles; ++k) {
                    if (k > 0) zero_acc(acc);
                    if (landed) multiply(rows + (size_t)k * 16 * GE.stride, pn, acc);
                    if (k == n_tiles - 1) {
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
                    }
                    if (tile_done) {
                        fold(acc);
                        finish((long long)(t_lo + tj + k) * 16);
                    }
                }
                if (n_tiles == 0) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
                }
                if (pl.split) {
                    tj += step_t; pn += step_p;
                    if (pn >= GE.n_panels) { pn -= GE.n_panels; ++tj; }
                } else if (++pn == GE.n_panels) { pn = 0; tj += W * pl.tpu; }
                slot += W;
                if (slot >= P.slots) { slot -= P.slots; parity ^= 1u; }
            }
            if (pl.split) {
                if (cur >= 0 && merge_split()) finish((long long)(t_lo + cur) * 16);
                split_tiles += T;
            }
            it0 += pl.n_units;
        }
    }
    __syncthreads();
    if (tid == 0 && s_abort) report(P.dev_status, MATQ_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------------------
// Host side

// static shared memory of the batched kernel with G groups, rounded up
inline int static_reserve_batch(int G) { return (10 + (G - 1) * 6) * 1024; }

// Quad groups (four vectors a group, 15-bit activations) serve r = 8 and r = 4 from three vectors up; pair groups (two
// vectors a group, 22-bit activations) everything else.
inline bool quad_mode(int r, int64_t B) { return r != 2 && B >= 3; }
inline int groups_of(int64_t B, bool quad) { return quad ? (B <= 4 ? 1 : B <= 8 ? 2 : 4) : (B <= 2 ? 1 : B <= 4 ? 2 : 4); }
inline long long batch_fit(const Geo& g, int r, int G, bool quad) {
    return ((long long)kSmemLimit - static_reserve_batch(G) - (long long)(G * xs_group_bytes_of(g, r, quad))) / slot_bytes_of(g);
}
// Stages a problem gets beside its staged activations.  Long rows leave few stages of the usual size (K = 9216, eight
// vectors: four); such problems run in launches of their own with units half as large (`narrow`), i.e. with twice
// the stages and warps.
inline long long batch_fit(int64_t N, int64_t K, int r, int G, bool quad, bool* narrow = nullptr) {
    const long long full = batch_fit(geometry((int)N, (int)K, r, kUnitRow), r, G, quad);
    if (narrow) *narrow = full < kWideFit;
    return full >= kWideFit ? full : batch_fit(geometry((int)N, (int)K, r, kUnitRow / 2), r, G, quad);
}

// Whether a problem with B vectors (2 <= B <= kMaxBatch) can take the batched path.
inline bool eligible_batch(int64_t N, int64_t K, int r, int64_t B) {
    const bool quad = quad_mode(r, B);
    if (B < 2 || B > (quad ? kMaxVec : kMaxBatch)) return false;
    if (!(r == 8 || r == 4 || r == 2) || K % 128 != 0 || (r == 2 && K % 256 != 0) || K > imma::kMaxK || N <= 0 || N >= (1ll << 31) - 16) return false;
    return batch_fit(N, K, r, groups_of(B, quad), quad) >= kMinW;
}

// One launch over a list of problems that all take the batched path (hb[i]: the vectors of problem i).
template <int NP, int G, bool Q>
inline int launch_list_batch(const HostProblem* hp, const int* hb, int n, int unit_row, bool pdl, long long wait_cycles, bool hold, int32_t* dev_status, cudaStream_t s) {
    static std::atomic<unsigned long long> smem_ok{0};
    Params<NP> P;
    long long items = 0, tiles = 0;
    for (int i = 0; i < n; ++i) {
        if (hp[i].N == 0) continue;
        const Geo g = geometry((int)hp[i].N, (int)hp[i].K, hp[i].r, unit_row);
        items += (long long)g.tiles * tile_cost(g, hp[i].r);
        tiles += g.tiles;
    }
    if (tiles == 0) return MATQ_OK;
    const int sms = sm_count();
    const int grid = (int)std::min<long long>(sms, tiles);
    size_t xs_bytes = 0;
    int slot_bytes = 0, m = 0;
    long long item0 = 0;
    for (int i = 0; i < n; ++i) {
        if (hp[i].N == 0) continue;
        Problem& q = P.p[m];
        q.packed = hp[i].packed; q.alpha = hp[i].alpha; q.zero = hp[i].zero;
        q.ovf_row_ptr = nullptr; q.ovf_col = nullptr;
        q.x = static_cast<const __nv_bfloat16*>(hp[i].x); q.y = hp[i].y;
        q.N = (int)hp[i].N; q.K = (int)hp[i].K; q.r = hp[i].r; q.B = hb[i];
        q.item0 = item0;
        const Geo g = geometry(q.N, q.K, q.r, unit_row);
        if (!g.contig && !make_plane_map(&P.tm[m], q.packed, q.N, g)) return MATQ_ERR_CUDA;
        item0 += (long long)g.tiles * tile_cost(g, q.r);
        xs_bytes = std::max(xs_bytes, (size_t)G * xs_group_bytes_of(g, q.r, Q));
        slot_bytes = std::max(slot_bytes, slot_bytes_of(g));
        ++m;
    }
    for (int i = m; i < NP; ++i) P.p[i] = Problem{};
    xs_bytes = (xs_bytes + 127) / 128 * 128;
    const long long room = (long long)kSmemLimit - static_reserve_batch(G) - (long long)xs_bytes;
    const int fit = (int)std::min<long long>(room / slot_bytes, kMaxSlots);
    int W = std::min(kFewW, fit);
    if (W < kMinW) return MATQ_ERR_SHAPE;
    W = pick_warps(W, fit);
    const int slots = fit / W * W;
    P.items = items; P.wait_cycles = wait_cycles; P.dev_status = dev_status; P.n = m; P.slots = slots; P.slot_bytes = slot_bytes;
    P.xs_bytes = (int)xs_bytes; P.W = W; P.pdl = pdl ? 1 : 0; P.unit_row = unit_row; P.hold = hold ? 1 : 0; P.pairs = 0;
    P.tails = 1;
    auto kern = gemv_stream_batch<NP, G, Q>;
    if (!opt_in_max_smem(kern, smem_ok)) return MATQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)((W + 1) * 32));
    cfg.dynamicSmemBytes = xs_bytes + (size_t)slots * slot_bytes;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, kern, P) != cudaSuccess) { cudaGetLastError(); return MATQ_ERR_CUDA; }
    return MATQ_OK;
}

template <int NP>
inline int launch_list_batch_g(int G, bool quad, const HostProblem* hp, const int* hb, int n, int unit_row, bool pdl, long long wait_cycles, bool hold, int32_t* dev_status, cudaStream_t s) {
    if (quad) {
        if (G == 1) return launch_list_batch<NP, 1, true>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
        if (G == 2) return launch_list_batch<NP, 2, true>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
        return launch_list_batch<NP, 4, true>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
    }
    if (G == 1) return launch_list_batch<NP, 1, false>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
    if (G == 2) return launch_list_batch<NP, 2, false>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
    return launch_list_batch<NP, 4, false>(hp, hb, n, unit_row, pdl, wait_cycles, hold, dev_status, s);
}

// The largest number of column groups (4, 2 or 1) whose staged activations leave room for at least kMinW stages; 0 when
// not even one group fits.
inline int max_groups(int64_t N, int64_t K, int r, bool quad) {
    // more groups only while they leave at least six stages (and warps): K = 14336 at r = 2 takes two vectors with seven
    // stages twice rather than four with four stages once
    for (int G = 4; G >= 1; G /= 2)
        if (batch_fit(N, K, r, G, quad) >= kWideFit - 1) return G;
    for (int G = 4; G >= 1; G /= 2)
        if (batch_fit(N, K, r, G, quad) >= kMinW) return G;
    return 0;
}

// A list of problems with batches (hb[i] >= 2 vectors each; the caller has cut them to what eligible_batch accepts).
// Problems with the same number of groups share a launch.
inline int launch_batch(const HostProblem* hp, const int* hb, int n, bool pdl, long long wait_cycles, bool hold, int32_t* dev_status, cudaStream_t s) {
    for (int i = 0; i < n; ++i)
        if (hp[i].N != 0 && !eligible_batch(hp[i].N, hp[i].K, hp[i].r, hb[i])) return MATQ_ERR_SHAPE;      // before anything is launched
    // Problems with the same number of groups share a launch, except that those whose staged activations would leave
    // the launch fewer than seven stages and warps (long rows) get a launch of their own: the number of warps is a
    // property of the launch, and the short rows of a stack should not run with four.
    std::vector<HostProblem> sel;
    std::vector<int> sel_b;
    for (int quad = 0; quad < 2; ++quad)
    for (int G = 1; G <= 4; G *= 2)
        for (int wide = 0; wide < 2; ++wide) {
            sel.clear(); sel_b.clear();
            for (int i = 0; i < n; ++i) {
                if (hp[i].N == 0 || quad_mode(hp[i].r, hb[i]) != (quad == 1) || groups_of(hb[i], quad == 1) != G) continue;
                bool narrow = false;
                batch_fit(hp[i].N, hp[i].K, hp[i].r, G, quad == 1, &narrow);
                if (narrow != (wide == 1)) continue;
                sel.push_back(hp[i]); sel_b.push_back(hb[i]);
            }
            for (size_t i = 0; i < sel.size(); i += kLargeList) {
                const int cnt = (int)std::min<size_t>(kLargeList, sel.size() - i);
                const int st = cnt <= kSmallList ? launch_list_batch_g<kSmallList>(G, quad == 1, sel.data() + i, sel_b.data() + i, cnt, wide ? kUnitRow / 2 : kUnitRow, pdl, wait_cycles, hold, dev_status, s)
                                                 : launch_list_batch_g<kLargeList>(G, quad == 1, sel.data() + i, sel_b.data() + i, cnt, wide ? kUnitRow / 2 : kUnitRow, pdl, wait_cycles, hold, dev_status, s);
                if (st != MATQ_OK) return st;
            }
        }
    return MATQ_OK;
}

// Number of launches launch_batch makes for these batch sizes and shapes.
inline int count_batch_launches(const HostProblem* hp, const int* hb, int n) {
    int launches = 0;
    for (int quad = 0; quad < 2; ++quad)
    for (int G = 1; G <= 4; G *= 2)
        for (int wide = 0; wide < 2; ++wide) {
            size_t cnt = 0;
            for (int i = 0; i < n; ++i) {
                if (hp[i].N == 0 || quad_mode(hp[i].r, hb[i]) != (quad == 1) || groups_of(hb[i], quad == 1) != G) continue;
                bool narrow = false;
                batch_fit(hp[i].N, hp[i].K, hp[i].r, G, quad == 1, &narrow);
                cnt += narrow == (wide == 1);
            }
            launches += (int)((cnt + kLargeList - 1) / kLargeList);
        }
    return launches;
}

// Cuts a problem with B >= 2 vectors into parts the kernels take: batches of at most 2 * max_groups vectors that share
// the plane (`many`, with their sizes in `many_b`), a single left-over vector as a problem of its own (`one`).
inline int split_batch(const HostProblem& q, std::vector<HostProblem>& one, std::vector<HostProblem>& many, std::vector<int>& many_b) {
    if (q.N == 0) return MATQ_OK;
    const bool quad = quad_mode(q.r, q.B);
    const int Gmax = max_groups(q.N, q.K, q.r, quad);
    if (Gmax == 0) return MATQ_ERR_SHAPE;
    const int64_t step = quad ? std::min<int64_t>(4 * Gmax, kMaxVec) : std::min<int64_t>(2 * Gmax, kMaxBatch);
    for (int64_t b0 = 0; b0 < q.B; b0 += step) {
        HostProblem part = q;
        const int64_t nb = std::min<int64_t>(step, q.B - b0);
        part.x = static_cast<const __nv_bfloat16*>(q.x) + b0 * q.K;
        part.y = q.y + b0 * q.N;
        part.B = nb;
        if (nb == 1) { one.push_back(part); continue; }
        many.push_back(part);
        many_b.push_back((int)nb);
    }
    return MATQ_OK;
}

}  // namespace gstream
}  // namespace matq
