// Decode GEMV with the multiply-accumulates on the tensor pipe (warp-level
// mma.m16n8k16, bf16 x bf16 -> fp32) so that unpacking costs about one issue
// slot per weight (less at r = 2) and a batch of up to 16 activations rides
// for free.
//
// Operand roles: A = 16 output channels x 16 weights, B = 16 weights x 8
// batch columns, D = fp32 [16 channels x 8 batch].  A dot product does not care
// in which order its terms are added, so the 16 "k slots" of an MMA are mapped
// to whatever weights a thread holds in a 16-byte piece of a row:
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
// Work split.  A warp owns 16*MT output channels and 1/SK of K; it streams its
// rows straight from global memory into registers with 128-bit loads, three
// chunks ahead of the MMAs, and the first chunks are requested BEFORE the
// kernel waits for its predecessor in the stream (programmatic dependent
// launch): a layer's weights are already in flight while the previous layer is
// still computing, only the activations depend on it.  With SK = 1 a warp
// finishes its outputs alone and writes y from its accumulators; with SK > 1
// the SK warps of a row tile are summed through shared memory in a fixed
// order.  No global scratch, no atomics: results are deterministic.  The
// extra-precision overflow lists are walked by a few threads per row in
// parallel with the staging of the activations.
//
// The activations are staged once per CTA into shared memory as x' in exactly
// the order the B fragments are consumed, so a thread fetches the B registers
// of two MMAs with one conflict-free 128-bit load and reuses them for all of
// its m-tiles; the sums of x and x' per batch column fall out of the same pass.
#pragma once
#include "common.cuh"

namespace matq {

constexpr int kGemvDepth = 3;               // chunks requested ahead of the one being multiplied

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
    int B;            // batch columns in use
    int bpad;         // batch columns staged: 1, 2, 4, 8 or 16
    int bpad_log2;
    int n_qc;         // 64-byte chunks per row (last one may be partial)
    int qc_pass;      // chunks whose activations are staged at a time (a multiple of nothing in particular; >= 1)
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

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// (lo = a.lo, hi = b.lo) and (lo = a.hi, hi = b.hi)
__device__ __forceinline__ uint32_t pack_lo(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x5410); }
__device__ __forceinline__ uint32_t pack_hi(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x7632); }
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
// exact power-of-two scaling of both bf16 halves with one packed multiply
__device__ __forceinline__ uint32_t scale2(uint32_t v, uint32_t s2) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s2));
    return r;
}

// Activations are written by the previous kernel of the stream while this one may already be resident, so they
// are read with plain (coherent) global loads after the dependency wait, never through the read-only path.
__device__ __forceinline__ uint4 ld_x4(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint2 ld_x2(const void* p) {
    uint2 v;
    asm volatile("ld.global.v2.u32 {%0,%1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
    return v;
}

// Stage the x' fragments of one packed word's worth of activations (starting at xw) for one batch column:
// writes kPairs/4 16-byte groups in B-fragment order and adds what it staged to sx (sum of x) and sxp (sum of x').
template <int R>
__device__ __forceinline__ void stage_word(const __nv_bfloat16* xw, uint4* dst, int dst_stride, float& sx, float& sxp) {
    if (R == 4) {                                   // 8 activations; pair p = (x[p], x[p+4])
        const uint4 v = ld_x4(xw);
        dst[0] = make_uint4(pack_lo(v.x, v.z), pack_hi(v.x, v.z), pack_lo(v.y, v.w), pack_hi(v.y, v.w));
        const float s = bf_lo(v.x) + bf_hi(v.x) + bf_lo(v.y) + bf_hi(v.y) + bf_lo(v.z) + bf_hi(v.z) + bf_lo(v.w) + bf_hi(v.w);
        sx += s; sxp += s;
    } else if (R == 8) {                            // 4 activations; pairs (x0,x2), 16(x0,x2), (x1,x3), 16(x1,x3)
        const uint2 v = ld_x2(xw);
        const uint32_t e = pack_lo(v.x, v.y), o = pack_hi(v.x, v.y);
        dst[0] = make_uint4(e, scale2(e, 0x41804180u), o, scale2(o, 0x41804180u));      // 0x4180 = bf16 16.0
        const float s = bf_lo(v.x) + bf_hi(v.x) + bf_lo(v.y) + bf_hi(v.y);
        sx += s; sxp += 17.0f * s;
    } else {                                        // 16 activations; pair p = (x[p], x[p+8]) * 4^-(p%3)
        const uint4 a = ld_x4(xw), b = ld_x4(xw + 8);
        uint32_t pr[8];
        pr[0] = pack_lo(a.x, b.x); pr[1] = pack_hi(a.x, b.x); pr[2] = pack_lo(a.y, b.y); pr[3] = pack_hi(a.y, b.y);
        pr[4] = pack_lo(a.z, b.z); pr[5] = pack_hi(a.z, b.z); pr[6] = pack_lo(a.w, b.w); pr[7] = pack_hi(a.w, b.w);
        float s0 = 0.f, s1 = 0.f, s2 = 0.f;         // sums of the pairs scaled by 1, 1/4, 1/16
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const float s = bf_lo(pr[p]) + bf_hi(pr[p]);
            if (p % 3 == 0) s0 += s; else if (p % 3 == 1) s1 += s; else s2 += s;
            if (p % 3 == 1) pr[p] = scale2(pr[p], 0x3e803e80u);        // 0x3e80 = bf16 0.25
            if (p % 3 == 2) pr[p] = scale2(pr[p], 0x3d803d80u);        // 0x3d80 = bf16 0.0625
        }
        sx += s0 + s1 + s2;
        sxp += s0 + 0.25f * s1 + 0.0625f * s2;
        dst[0] = make_uint4(pr[0], pr[1], pr[2], pr[3]);
        dst[dst_stride] = make_uint4(pr[4], pr[5], pr[6], pr[7]);
    }
}

// CL > 1: a thread-block cluster of CL CTAs shares a block of rows and splits K between its CTAs, so each CTA stages
// only 1/CL of the activations (the staging of B columns per CTA is what a batch costs); the per-CTA partial results
// (offset already removed) are summed by the cluster's first CTA through distributed shared memory.
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(const float* local, uint32_t rank) {
    uint32_t la = (uint32_t)__cvta_generic_to_shared(local), ra;
    float v;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(la), "r"(rank));
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
    return v;
}

template <int R, int MT, int NT, int SK, int WARPS, bool EP, int CL = 1>
__global__ void __launch_bounds__(WARPS * 32, (MT == 1 ? 32 : 16) / WARPS)   // MT = 1: 64 registers, a full SM of warps
gemv_tensor(const GemvTensorParams P) {
    constexpr int kGemvThreads = WARPS * 32, kGemvWarps = WARPS;
    using Fmt = GemvFmt<R>;
    constexpr int kTileRows = 16 * MT;                    // rows of a warp
    constexpr int kTiles = kGemvWarps / SK;               // row tiles of a CTA
    constexpr int kRows = kTileRows * kTiles;
    constexpr int kPG = Fmt::kPairs / 4;                  // 128-bit B loads per word
    constexpr int kWq = 16 * Fmt::kWeightsPerWord;        // weights per 64-byte chunk of a row
    constexpr int sh = kCodeBits - R;
    constexpr int kMaxB = 8 * NT;
    constexpr int kSets = (MT >= 2) ? 1 : 2;              // independent accumulator sets per m-tile

    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ float s_sumx[kMaxB], s_sumxp[kMaxB], s_grp[2][kGemvThreads / 4];
    __shared__ float s_ep[EP ? kRows : 1][kMaxB];         // extra-precision correction per row and batch column
    __shared__ float s_alpha[(SK > 1 || CL > 1) ? kRows : 1], s_zero[(SK > 1 || CL > 1) ? kRows : 1];
    constexpr int kRowThreads = kGemvThreads / kRows;     // = 2 SK / MT consecutive threads per row of the CTA
    constexpr int kTPR = kRowThreads > 32 ? 32 : kRowThreads;   // of which this many walk the row's overflow list

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int tile = warp / SK, ks = warp % SK;
    uint32_t crank = 0;                                   // this CTA's place in its cluster = its share of K
    if (CL > 1) asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(crank));
    const int64_t rblock = CL > 1 ? (int64_t)(blockIdx.x / CL) : (int64_t)blockIdx.x;   // block of kRows rows
    const int64_t row0 = rblock * kRows + (int64_t)tile * kTileRows;
    const int c_per = (P.n_qc + CL - 1) / CL;
    const int c_lo = min((int)crank * c_per, P.n_qc), c_hi = min(c_lo + c_per, P.n_qc);   // this CTA's chunks
    // K is walked in passes of qc_pass chunks (one pass unless the staged activations would not fit in shared memory);
    // inside a pass the SK warps of a row tile take consecutive slices of its chunks.
    int pass_lo = c_lo, pass_hi = min(c_lo + P.qc_pass, c_hi);
    int q_lo, q_hi;
    auto set_slice = [&]() {
        const int per_warp = (pass_hi - pass_lo + SK - 1) / SK;
        q_lo = pass_lo + ks * per_warp;
        q_hi = min(q_lo + per_warp, pass_hi);
    };
    set_slice();
    const int bpad = P.bpad;

    // shared memory: x' fragments for all of K | partial tiles [warp][kTileRows][kMaxB] (SK > 1 only)
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);
    float* part = reinterpret_cast<float*>(smem_raw + (size_t)min(P.qc_pass, P.n_qc) * 4 * kPG * bpad * 64);
    float* red = part + (size_t)kGemvWarps * kTileRows * kMaxB;     // CL > 1: [kRows][kMaxB] partial results + [kMaxB] sums of x

    // ---- weights of the first chunks are requested before anything that depends on the previous kernel
    // Rows past N are clamped to the last row (their results are never stored) and a lane whose piece would start
    // past the end of a ragged last chunk is clamped to the row's last 16 bytes (the matching activations are staged
    // as zeros and unpacked fields are always finite), so the loads need no predicates and no zero fill.
    const uint8_t* wrow[2 * MT];
    bool wok[2 * MT];
#pragma unroll
    for (int h = 0; h < 2 * MT; ++h) {
        const int64_t row = row0 + (h >> 1) * 16 + (h & 1) * 8 + g;
        wok[h] = row < P.N;
        wrow[h] = P.packed + (wok[h] ? row : P.N - 1) * P.row_bytes;
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

    // scale and zero point: with SK = 1 a thread finishes rows g and g+8 of every m-tile from its accumulators and
    // keeps them in registers; with SK > 1 the CTA's rows are parked in shared memory for the shared epilogue.
    float a_pre[2 * MT], z_pre[2 * MT];
    if (SK == 1 && CL == 1) {
#pragma unroll
        for (int h = 0; h < 2 * MT; ++h) {
            const int64_t row = row0 + (h >> 1) * 16 + (h & 1) * 8 + g;
            a_pre[h] = wok[h] ? P.alpha[row] : 0.f;
            z_pre[h] = wok[h] ? P.zero[row] : 0.f;
        }
    } else {
        for (int rl = tid; rl < kRows; rl += kGemvThreads) {
            const int64_t row = rblock * kRows + rl;
            s_alpha[rl] = row < P.N ? P.alpha[row] : 0.f;
            s_zero[rl] = row < P.N ? P.zero[row] : 0.f;
        }
    }

    // Extra precision (Errata, Eq. 8): an overflow column's field is one higher than the stored, clamped one, so its
    // activation is added once more.  kTPR threads share a row's list; the list (weights-side data) is read before
    // the dependency wait, the activations it points at right after it, and the sums land in s_ep before the
    // barrier that precedes the epilogue.
    const int ep_row = tid / kRowThreads, ep_j = tid % kRowThreads;
    int ep_p = 0, ep_hi = 0, ep_c0 = 0;
    if (EP && ep_j < kTPR && crank == 0) {
        const int64_t row = rblock * kRows + ep_row;
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

    // activation (batch column 0) of this thread's first overflow column: requested now, used after the staging
    float ep_x0 = 0.f;
    if (EP && ep_p < ep_hi) ep_x0 = __bfloat162float(P.x[ep_c0]);

    float acc[kSets][MT][NT][4];
#pragma unroll
    for (int c = 0; c < kSets; ++c)
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[c][mt][nt][i] = 0.f;

    float sx = 0.f, sxp = 0.f;                            // this thread's share of sum(x) and sum(x') of its column
    for (;;) {
        // ---- stage x' (pre-scaled activations in B-fragment order) of this pass and add to the two sums.
        // Item i = ((q*4 + j) * bpad + gg) * 4 + tt covers one packed word's worth of activations.  (i >> 2) % bpad
        // is the batch column and threads / 4 is a multiple of bpad, so every group of 4 lanes sees a single column.
        {
            // thread -> (tt, gg) is fixed; its items are qstep apart in (q*4 + j), so everything but two adds is hoisted
            const int n_qjl = (pass_hi - pass_lo) * 4;
            const int qstep = (kGemvThreads / 4) >> P.bpad_log2;
            const int tt = tid & 3, gg = (tid >> 2) & (bpad - 1);
            const bool col_ok = gg < P.B;
            const __nv_bfloat16* xrow = P.x + (int64_t)(col_ok ? gg : 0) * P.ldx;
            int qjl = (tid >> 2) >> P.bpad_log2;
            uint4* dst = xs + ((uint32_t)qjl * kPG * bpad + gg) * 4 + tt;
            const uint32_t dstep = (uint32_t)qstep * kPG * bpad * 4;
            const int kmax = (int)P.K;
            for (; qjl < n_qjl; qjl += qstep, dst += dstep) {
                const int qj = pass_lo * 4 + qjl;
                const int kb = Fmt::kWeightsPerWord * (16 * (qj >> 2) + 4 * tt + (qj & 3));
                if (col_ok && kb < kmax) {                    // K % 128 == 0: a word lies inside or outside
                    stage_word<R>(xrow + kb, dst, bpad * 4, sx, sxp);
                } else {
                    dst[0] = make_uint4(0, 0, 0, 0);
                    if (kPG == 2) dst[bpad * 4] = make_uint4(0, 0, 0, 0);
                }
            }
        }
        if (EP && pass_lo == 0 && crank == 0) {               // uniform over the CTA
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
        const bool last_pass = pass_hi >= c_hi;              // uniform over the CTA
        if (last_pass) {
            sx += __shfl_xor_sync(0xffffffffu, sx, 1);  sxp += __shfl_xor_sync(0xffffffffu, sxp, 1);
            sx += __shfl_xor_sync(0xffffffffu, sx, 2);  sxp += __shfl_xor_sync(0xffffffffu, sxp, 2);
            if (t == 0) { s_grp[0][tid >> 2] = sx; s_grp[1][tid >> 2] = sxp; }
        }
        __syncthreads();
        if (last_pass && warp == 0) {
            // entry h of s_grp belongs to batch column h % bpad (bpad divides 32): lanes congruent modulo bpad are summed
            float tx = 0.f, txp = 0.f;
#pragma unroll
            for (int h = 0; h < kGemvThreads / 4; h += 32) { tx += s_grp[0][h + lane]; txp += s_grp[1][h + lane]; }
            for (int o = 16; o >= bpad; o >>= 1) {
                tx += __shfl_xor_sync(0xffffffffu, tx, o);
                txp += __shfl_xor_sync(0xffffffffu, txp, o);
            }
            if (lane < kMaxB) {        // read after the barrier that precedes the epilogue
                s_sumx[lane] = lane < bpad ? tx : 0.f;
                s_sumxp[lane] = lane < bpad ? txp : 0.f;
            }
        }

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
                    for (int j = 0; j < 4; ++j) {
#pragma unroll
                        for (int pg = 0; pg < kPG; ++pg) {
                            uint4 xb[NT];
#pragma unroll
                            for (int nt = 0; nt < NT; ++nt) {
                                xb[nt] = make_uint4(0, 0, 0, 0);
                                const int gb = g + 8 * nt;
                                if (gb < bpad) xb[nt] = xs[(((size_t)(q - pass_lo) * 4 + j) * kPG + pg) * bpad * 4 + gb * 4 + t];
                            }
#pragma unroll
                            for (int u = 0; u < 2; ++u) {
                                const int p = pg * 4 + 2 * u;
#pragma unroll
                                for (int mt = 0; mt < MT; ++mt) {
                                    const uint32_t w_lo = (j == 0 ? wv[2 * mt].x : j == 1 ? wv[2 * mt].y : j == 2 ? wv[2 * mt].z : wv[2 * mt].w);
                                    const uint32_t w_hi = (j == 0 ? wv[2 * mt + 1].x : j == 1 ? wv[2 * mt + 1].y : j == 2 ? wv[2 * mt + 1].z : wv[2 * mt + 1].w);
                                    const uint32_t a0 = field_pair<R>(w_lo, p), a1 = field_pair<R>(w_hi, p);
                                    const uint32_t a2 = field_pair<R>(w_lo, p + 1), a3 = field_pair<R>(w_hi, p + 1);
#pragma unroll
                                    for (int nt = 0; nt < NT; ++nt) {
                                        const uint32_t b0 = u ? xb[nt].z : xb[nt].x, b1 = u ? xb[nt].w : xb[nt].y;
                                        mma_bf16_16816(acc[u % kSets][mt][nt], a0, a1, a2, a3, b0, b1);
                                    }
                                }
                            }
                        }
                    }
                }
            }
        }
        if (last_pass) break;
        // ---- next pass: request its first chunks, then wait until every warp is done with the staged activations
        pass_lo = pass_hi;
        pass_hi = min(pass_lo + P.qc_pass, c_hi);
        set_slice();
#pragma unroll
        for (int d = 0; d < kGemvDepth; ++d) load_chunk(q_lo + d, wbuf[d]);
        __syncthreads();
    }
    if (kSets == 2) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i) acc[0][mt][nt][i] += acc[kSets - 1][mt][nt][i];
    }

    // ---- epilogue.  Accumulator i of thread (g, t): row g + 8*(i>>1) of the m-tile, batch column 2t + (i&1).
    if (SK > 1 || CL > 1) {
        float* mine = part + (size_t)warp * kTileRows * kMaxB;
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt)
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    mine[(mt * 16 + g + (i >> 1) * 8) * kMaxB + nt * 8 + 2 * t + (i & 1)] = acc[0][mt][nt][i];
    }
    __syncthreads();                                      // publishes s_sumx / s_sumxp and the partial tiles
    if (CL > 1) {
        // this CTA's share of every output, offset removed (everything is linear in the K range), and of the sums of x
        for (int o = tid; o < kRows * kMaxB; o += kGemvThreads) {
            const int b = o % kMaxB, row_l = o / kMaxB;
            const float* src = part + ((size_t)(row_l / kTileRows) * SK * kTileRows + row_l % kTileRows) * kMaxB + b;
            float v = src[0];
#pragma unroll
            for (int sidx = 1; sidx < SK; ++sidx) v += src[(size_t)sidx * kTileRows * kMaxB];
            red[o] = v - 128.0f * s_sumxp[b];
        }
        if (tid < kMaxB) red[kRows * kMaxB + tid] = s_sumx[tid];
        cluster_sync_all();
        if (crank == 0) {
            for (int o = tid; o < kRows * kMaxB; o += kGemvThreads) {
                const int b = o % kMaxB, row_l = o / kMaxB;
                const int64_t row = rblock * kRows + row_l;
                if (b >= P.B || row >= P.N) continue;
                float v = red[o], sxa = red[kRows * kMaxB + b];
#pragma unroll
                for (uint32_t c = 1; c < (uint32_t)CL; ++c) {
                    v += ld_cluster_f32(red + o, c);
                    sxa += ld_cluster_f32(red + kRows * kMaxB + b, c);
                }
                if (EP) v += s_ep[row_l][b];
                P.y[(int64_t)b * P.ldy + row] = s_alpha[row_l] * (v * (float)(1 << sh) - s_zero[row_l] * sxa);
            }
        }
        cluster_sync_all();                               // the other CTAs' shared memory stays alive until it was read
        return;
    }
    if (SK > 1) {
        // Every thread finishes outputs: output o = (row of the CTA) * kMaxB + batch column sums its SK partials in
        // a fixed order and is scaled with the row's alpha / zero (parked in shared memory at the start).
        for (int o = tid; o < kRows * kMaxB; o += kGemvThreads) {
            const int b = o % kMaxB, row_l = o / kMaxB;
            const int64_t row = rblock * kRows + row_l;
            if (b >= P.B || row >= P.N) continue;
            const float* src = part + ((size_t)(row_l / kTileRows) * SK * kTileRows + row_l % kTileRows) * kMaxB + b;
            float v = src[0];
#pragma unroll
            for (int sidx = 1; sidx < SK; ++sidx) v += src[(size_t)sidx * kTileRows * kMaxB];
            v -= 128.0f * s_sumxp[b];
            if (EP) v += s_ep[row_l][b];
            P.y[(int64_t)b * P.ldy + row] = s_alpha[row_l] * (v * (float)(1 << sh) - s_zero[row_l] * s_sumx[b]);
        }
        return;
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int h = 2 * mt + (i >> 1);
                const int b = nt * 8 + 2 * t + (i & 1);
                const int64_t row = row0 + mt * 16 + g + (i >> 1) * 8;
                if (!wok[h] || b >= P.B) continue;
                float v = acc[0][mt][nt][i] - 128.0f * s_sumxp[b];
                if (EP) v += s_ep[tile * kTileRows + mt * 16 + g + (i >> 1) * 8][b];
                P.y[(int64_t)b * P.ldy + row] = a_pre[h] * (v * (float)(1 << sh) - z_pre[h] * s_sumx[b]);
            }
}

// Host side: geometry and launch.
template <int R, int MT, int NT, int SK, int WARPS = 8, int CL = 1>
inline int launch_gemv_tensor(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                              const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                              float* y, int64_t ldy, bool pdl, cudaStream_t s) {
    using Fmt = GemvFmt<R>;
    constexpr int kGemvThreads = WARPS * 32, kGemvWarps = WARPS;
    constexpr int kRows = 16 * MT * (kGemvWarps / SK), kMaxB = 8 * NT;
    constexpr int kPG = Fmt::kPairs / 4;
    GemvTensorParams P;
    P.packed = packed; P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y;
    P.N = N; P.K = K; P.ldx = ldx; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    if (P.row_bytes > 0x7fffffff) return MATQ_ERR_SHAPE;   // byte offsets inside a row are 32-bit
    P.B = B;
    P.bpad = B <= 1 ? 1 : B <= 2 ? 2 : B <= 4 ? 4 : B <= 8 ? 8 : 16;
    P.n_qc = (int)((P.row_bytes + 63) / 64);
    P.pdl = pdl ? 1 : 0;
    P.bpad_log2 = P.bpad == 1 ? 0 : P.bpad == 2 ? 1 : P.bpad == 4 ? 2 : P.bpad == 8 ? 3 : 4;
    // Shared memory: the staged activations of one pass (64 * 4 * kPG * bpad bytes per chunk) + the split-K partials.
    // Passes are as long as ~150 KB allow (one pass for all decode shapes up to K = 9216 at B = 8).
    const size_t part_bytes = (SK > 1 || CL > 1 ? (size_t)kGemvWarps * 16 * MT * kMaxB * sizeof(float) : 0) +
                              (CL > 1 ? (size_t)(kRows + 1) * kMaxB * sizeof(float) : 0);
    const size_t chunk_bytes = (size_t)4 * kPG * P.bpad * 64;
    const int fit = (int)((150 * 1024 - part_bytes) / chunk_bytes);
    const int c_per = (P.n_qc + CL - 1) / CL;             // chunks of one CTA of a cluster
    const int passes = (c_per + fit - 1) / fit;
    P.qc_pass = (c_per + passes - 1) / passes;
    const size_t smem = (size_t)P.qc_pass * chunk_bytes + part_bytes;
    auto kern = ovf_row_ptr ? gemv_tensor<R, MT, NT, SK, WARPS, true, CL> : gemv_tensor<R, MT, NT, SK, WARPS, false, CL>;
    static std::atomic<unsigned long long> smem_ok[2] = {{0}, {0}};     // one per kernel of this template instance
    if (smem > 16 * 1024 &&   // the 48 KB default counts static shared memory too
        !opt_in_max_smem(kern, smem_ok[ovf_row_ptr ? 1 : 0]))
        return MATQ_ERR_CUDA;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((N + kRows - 1) / kRows) * CL, 1, 1);
    cfg.blockDim = dim3(kGemvThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (CL > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = CL; attr[na].val.clusterDim.y = 1; attr[na].val.clusterDim.z = 1;
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
