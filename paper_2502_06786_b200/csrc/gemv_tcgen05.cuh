// Decode GEMV on the fifth-generation tensor cores (tcgen05.mma, accumulators and the A operand in tensor memory).
//
// Why not the warp-level MMA: on B200 one mma.sync.m16n8k16 occupies a sub-partition's legacy tensor pipe for
// about 32 cycles, so a decode GEMV (one batch column = 7/8 padding per MMA) is bound by that pipe well below the
// HBM roofline.  tcgen05.mma multiplies a 128 x 16 tile of A against 16 batch columns in a handful of cycles, which
// leaves the unpacking of the fields as the only per-weight work on the SM: well under one issue slot per weight.
//
// Roles.  A CTA owns 128 output channels (one per TMEM lane) and one slice of K.  A (M = 128 rows x K = 16 per
// instruction) is the unpacked weight tile and lives in TENSOR MEMORY: thread "row" turns 32-bit words of its own
// row into bf16x2 registers (one LOP3 each, see below) and stores them into a TMEM slot with tcgen05.st.  B (16
// k-slots x N = 16 batch columns) is the activation tile x' in shared memory, K-major without swizzle.  D (128 x 16
// fp32) accumulates in TMEM.
//
// Unpacking.  ((w >> s) & mask) | 0x43004300 puts two fields on the mantissas of two bf16 128.0: each half reads
// 128 + field * 4^i where 2i is the bit offset of the field inside its half.  r = 2 uses offsets 0, 2, 4 in place
// (2 shifts + 8 LOP3 per 16 weights) and the matching activations are pre-scaled by 4^-i; r = 4 uses offset 0 after
// a shift by 4p; r = 8 is read as two nibbles, the high one against 16 x.  A dot product does not care about the
// order of its terms, so the k-slot order of an instruction is simply the order in which the fields fall out of a
// word, and x' is staged in that same order.  The constant 128 contributes 128 * sum(x') to every row; it is removed
// in the epilogue with the separately accumulated sum.
//
// Data movement.  Every thread of the first four warps issues one bulk asynchronous copy (cp.async.bulk) for its
// row's slice of the packed plane, completion counted on one mbarrier per 32 rows; all of a CTA's bytes are in flight
// at once and are requested BEFORE the kernel waits for its predecessor in the stream (programmatic dependent
// launch), so a layer's weights stream in while the previous layer still computes.  TMEM is allocated before the
// dependents are released, so a waiting successor can never starve a predecessor of tensor memory.
//
// Four warpgroups take the 16-byte chunks of the slice round-robin, each with two TMEM slots (tcgen05.commit frees a
// slot when the MMAs that read it retire) and its own accumulator; the four accumulators are added in a fixed order.
// Slices of K (grid.y > 1) form a thread-block cluster and are summed through distributed shared memory in rank
// order.  No global scratch, no atomics: results are deterministic.
#pragma once
#include <cooperative_groups.h>

#include "common.cuh"

namespace matq {
namespace t5 {
namespace cg = cooperative_groups;

constexpr int kThreads = 512;
constexpr int kWarpgroups = 4;
constexpr int kRows = 128;                   // M of the MMA = TMEM lanes
constexpr int kNB = 16;                      // N of the MMA = batch columns (padded)
constexpr int kStepBytes = 512;              // x' bytes of one K = 16 instruction: [k-half][n-group][8 n][8 k] bf16
constexpr int kSlotCols = 16;                // TMEM columns of one A slot = two K = 16 instructions
constexpr int kTmemCols = 256;               // 4 accumulators x 16 + 4 warpgroups x 2 slots x 16 = 192 -> 256
constexpr int kAccCol = 0, kSlotCol = 64;
constexpr uint32_t kSpinLimit = 1u << 22;    // mbarrier polls before a wait gives up

struct Params {
    const uint8_t* packed;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const __nv_bfloat16* x;
    float* y;
    int32_t* dev_status;
    int64_t N, K, ldx, ldy;
    int64_t row_bytes;
    int B;
    int slice_bytes;     // bytes of a row handled by one CTA (multiple of 16; the last slice may be shorter)
    int tile_stride;     // bytes between rows of the shared-memory weight tile (16 mod 128)
    int pdl;
};

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

template <int R>
__device__ __forceinline__ uint32_t field_pair(uint32_t w, int p) {
    if (R == 2) {
        const int s = 6 * (p / 3), i = p % 3;
        return ((w >> s) & (0x00030003u << (2 * i))) | 0x43004300u;
    }
    return ((w >> (4 * p)) & 0x000f000fu) | 0x43004300u;
}

__device__ __forceinline__ uint32_t pack_lo(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x5410); }
__device__ __forceinline__ uint32_t pack_hi(uint32_t a, uint32_t b) { return __byte_perm(a, b, 0x7632); }
__device__ __forceinline__ float bf_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
__device__ __forceinline__ uint32_t scale2(uint32_t v, uint32_t s2) {
    uint32_t r;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(v), "r"(s2));
    return r;
}
// plain (coherent) loads: the activations are written by the previous kernel of the stream
__device__ __forceinline__ uint4 ld_x4(const void* p) {
    uint4 v;
    asm volatile("ld.global.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
    return v;
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    uint32_t done = 0;
    for (uint32_t it = 0; it < kSpinLimit && !done; ++it)
        asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                     : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    return done != 0;
}

// Shared-memory matrix descriptor of one x' step: K-major, no swizzle, 8 x 16-byte core matrices; the two k-halves
// are 256 bytes apart (leading byte offset), the two groups of 8 batch columns 128 bytes (stride byte offset).
__device__ __forceinline__ uint64_t b_desc(uint32_t smem_addr) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)(256 >> 4) << 16) | ((uint64_t)(128 >> 4) << 32) | (1ull << 46);
}
// kind::f16, D = fp32, A = B = bf16, both K-major, N = 16, M = 128
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kNB >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);

// Steps (K = 16 instructions) per 16-byte chunk of a row, and activations covered by one step.
template <int R> struct Fmt;
template <> struct Fmt<2> { static constexpr int kStepsPerChunk = 4, kKPerStep = 16; };
template <> struct Fmt<4> { static constexpr int kStepsPerChunk = 2, kKPerStep = 16; };
template <> struct Fmt<8> { static constexpr int kStepsPerChunk = 2, kKPerStep = 8; };

// The two 16-byte halves (k-slots 0..7 and 8..15) of one step's x' row for one batch column, in the slot order the
// unpacking produces, plus what they add to sum(x) and sum(x').
template <int R>
__device__ __forceinline__ void stage_step(const __nv_bfloat16* xk, uint4& h0, uint4& h1, float& sx, float& sxp) {
    if (R == 4) {            // two words of 8 fields: slots (2p, 2p+1) = fields (p, p+4) of each word
        const uint4 a = ld_x4(xk), b = ld_x4(xk + 8);
        h0 = make_uint4(pack_lo(a.x, a.z), pack_hi(a.x, a.z), pack_lo(a.y, a.w), pack_hi(a.y, a.w));
        h1 = make_uint4(pack_lo(b.x, b.z), pack_hi(b.x, b.z), pack_lo(b.y, b.w), pack_hi(b.y, b.w));
        const float s = bf_lo(a.x) + bf_hi(a.x) + bf_lo(a.y) + bf_hi(a.y) + bf_lo(a.z) + bf_hi(a.z) + bf_lo(a.w) + bf_hi(a.w) +
                        bf_lo(b.x) + bf_hi(b.x) + bf_lo(b.y) + bf_hi(b.y) + bf_lo(b.z) + bf_hi(b.z) + bf_lo(b.w) + bf_hi(b.w);
        sx += s; sxp += s;
    } else if (R == 8) {     // two words of 4 codes: slots (x0,x2), 16(x0,x2), (x1,x3), 16(x1,x3) per word
        const uint4 a = ld_x4(xk);
        const uint32_t e0 = pack_lo(a.x, a.y), o0 = pack_hi(a.x, a.y), e1 = pack_lo(a.z, a.w), o1 = pack_hi(a.z, a.w);
        h0 = make_uint4(e0, scale2(e0, 0x41804180u), o0, scale2(o0, 0x41804180u));     // 0x4180 = bf16 16.0
        h1 = make_uint4(e1, scale2(e1, 0x41804180u), o1, scale2(o1, 0x41804180u));
        const float s = bf_lo(a.x) + bf_hi(a.x) + bf_lo(a.y) + bf_hi(a.y) + bf_lo(a.z) + bf_hi(a.z) + bf_lo(a.w) + bf_hi(a.w);
        sx += s; sxp += 17.0f * s;
    } else {                 // one word of 16 fields: slots (2p, 2p+1) = fields (p, p+8) scaled by 4^-(p%3)
        const uint4 a = ld_x4(xk), b = ld_x4(xk + 8);
        uint32_t pr[8];
        pr[0] = pack_lo(a.x, b.x); pr[1] = pack_hi(a.x, b.x); pr[2] = pack_lo(a.y, b.y); pr[3] = pack_hi(a.y, b.y);
        pr[4] = pack_lo(a.z, b.z); pr[5] = pack_hi(a.z, b.z); pr[6] = pack_lo(a.w, b.w); pr[7] = pack_hi(a.w, b.w);
        float s0 = 0.f, s1 = 0.f, s2 = 0.f;
#pragma unroll
        for (int p = 0; p < 8; ++p) {
            const float s = bf_lo(pr[p]) + bf_hi(pr[p]);
            if (p % 3 == 0) s0 += s; else if (p % 3 == 1) s1 += s; else s2 += s;
            if (p % 3 == 1) pr[p] = scale2(pr[p], 0x3e803e80u);        // bf16 0.25
            if (p % 3 == 2) pr[p] = scale2(pr[p], 0x3d803d80u);        // bf16 0.0625
        }
        sx += s0 + s1 + s2;
        sxp += s0 + 0.25f * s1 + 0.0625f * s2;
        h0 = make_uint4(pr[0], pr[1], pr[2], pr[3]);
        h1 = make_uint4(pr[4], pr[5], pr[6], pr[7]);
    }
}

template <int R>
__global__ void __launch_bounds__(kThreads, 1)
gemv_tcgen05(const Params P) {
    constexpr int sh = kCodeBits - R;
    constexpr int kStepsPerChunk = Fmt<R>::kStepsPerChunk;
    constexpr int kKPerStep = Fmt<R>::kKPerStep;
    constexpr int kSlotBytes = 16 * 2 / kStepsPerChunk;       // row bytes unpacked into one slot (two steps)
    constexpr int kWordsPerSlot = kSlotBytes / 4;

    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_wbar[4];                 // weight rows of TMEM lane quadrant q have landed
    __shared__ __align__(8) uint64_t s_free[kWarpgroups][2];    // A slot may be overwritten
    __shared__ __align__(8) uint64_t s_done[kWarpgroups];       // accumulator of the warpgroup is final
    __shared__ uint32_t s_tmem;
    __shared__ float s_red[2][kThreads / 32][kNB];
    __shared__ float s_sumx[kNB], s_sumxp[kNB];
    __shared__ float s_part[kRows][kNB];                         // this CTA's partial outputs (cluster reduction)

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int wg = warp >> 2, quad = warp & 3;                  // warp may touch TMEM lanes [32*quad, 32*quad + 32)
    const int row_l = quad * 32 + lane;                         // the row this thread unpacks and finishes
    const int split = blockIdx.y, n_split = gridDim.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const int64_t slice_off = (int64_t)split * P.slice_bytes;
    const int my_bytes = (int)min((int64_t)P.slice_bytes, P.row_bytes - slice_off);    // multiple of 16, >= 16
    const int n_chunks = my_bytes / kSlotBytes;                 // slots to fill in this CTA
    const int n_steps = n_chunks * 2;
    const int rows_here = (int)min((int64_t)kRows, P.N - row0);

    unsigned char* wt = smem_raw;                               // [128][tile_stride]
    unsigned char* xs = smem_raw + (size_t)kRows * P.tile_stride;   // [steps][512]

    // ---- barriers, tensor memory, weight copies: nothing here depends on the previous kernel
    if (tid == 0) {
        for (int q = 0; q < 4; ++q) {
            const int rq = max(0, min(32, rows_here - q * 32));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_wbar[q])));
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(&s_wbar[q])), "r"(rq * my_bytes) : "memory");
        }
        for (int w = 0; w < kWarpgroups; ++w) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_free[w][0])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_free[w][1])));
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_done[w])));
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;

    if (tid < rows_here) {
        const uint8_t* src = P.packed + (row0 + tid) * P.row_bytes + slice_off;
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(smem_u32(wt + (size_t)tid * P.tile_stride)), "l"(src), "r"(my_bytes), "r"(smem_u32(&s_wbar[tid >> 5])) : "memory");
    }
    float a_pre = 0.f, z_pre = 0.f;
    if (wg == 0 && row0 + row_l < P.N) {
        a_pre = P.alpha[row0 + row_l];
        z_pre = P.zero[row0 + row_l];
    }

    if (P.pdl) {
        asm volatile("griddepcontrol.launch_dependents;");
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }

    // ---- activations: zero the x' tile, then write the rows of the batch columns in use; sums on the way
    {
        uint4* xz = reinterpret_cast<uint4*>(xs);
        for (int i = tid; i < n_steps * (kStepBytes / 16); i += kThreads) xz[i] = make_uint4(0, 0, 0, 0);
    }
    __syncthreads();
    {
        // item = (step, batch column); 512 threads cover 32 steps x 16 columns per pass, a thread keeps its column
        const int bcol = tid & (kNB - 1);
        const int64_t k_base = slice_off * 8 / R;               // first activation of the slice
        float sx = 0.f, sxp = 0.f;
        if (bcol < P.B) {
            for (int st = tid >> 4; st < n_steps; st += kThreads / kNB) {
                const int64_t k = k_base + (int64_t)st * kKPerStep;
                if (k < P.K) {
                    uint4 h0, h1;
                    stage_step<R>(P.x + (int64_t)bcol * P.ldx + k, h0, h1, sx, sxp);
                    unsigned char* base = xs + (size_t)st * kStepBytes + (bcol >> 3) * 128 + (bcol & 7) * 16;
                    *reinterpret_cast<uint4*>(base) = h0;
                    *reinterpret_cast<uint4*>(base + 256) = h1;
                }
            }
        }
        // lanes l and l + 16 hold the same column: fold, then one value per (warp, column)
        sx += __shfl_xor_sync(0xffffffffu, sx, 16);  sxp += __shfl_xor_sync(0xffffffffu, sxp, 16);
        if (lane < kNB) { s_red[0][warp][lane] = sx; s_red[1][warp][lane] = sxp; }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");     // x' was written with ordinary stores, the MMA reads it
    __syncthreads();
    if (tid < kNB) {
        float sx = 0.f, sxp = 0.f;
        for (int w = 0; w < kThreads / 32; ++w) { sx += s_red[0][w][tid]; sxp += s_red[1][w][tid]; }
        s_sumx[tid] = sx;
        s_sumxp[tid] = sxp;
    }

    // ---- main loop: warpgroup wg fills slots with chunks wg, wg + 4, ...; one thread issues the MMAs
    bool ok = mbar_wait(smem_u32(&s_wbar[quad]), 0);
    const unsigned char* my_row = wt + (size_t)row_l * P.tile_stride;
    const uint32_t acc_addr = tmem + kAccCol + wg * kNB;
    int it = 0;
    for (int c = wg; c < n_chunks; c += kWarpgroups, ++it) {
        const int slot = it & 1;
        if (it >= 2) ok &= mbar_wait(smem_u32(&s_free[wg][slot]), ((it >> 1) - 1) & 1);
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        uint32_t wv[4];
        if (kWordsPerSlot == 4) {
            const uint4 v = *reinterpret_cast<const uint4*>(my_row + (size_t)c * 16);
            wv[0] = v.x; wv[1] = v.y; wv[2] = v.z; wv[3] = v.w;
        } else {
            const uint2 v = *reinterpret_cast<const uint2*>(my_row + (size_t)c * 8);
            wv[0] = v.x; wv[1] = v.y; wv[2] = 0; wv[3] = 0;
        }
        uint32_t a[kSlotCols];
#pragma unroll
        for (int i = 0; i < kSlotCols; ++i) {
            constexpr int kPairsPerWord = kSlotCols / kWordsPerSlot;
            a[i] = field_pair<R>(wv[i / kPairsPerWord], i % kPairsPerWord);
        }
        const uint32_t slot_addr = tmem + ((uint32_t)(quad * 32) << 16) + kSlotCol + (wg * 2 + slot) * kSlotCols;
        asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16};"
                     ::"r"(slot_addr), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),
                       "r"(a[8]), "r"(a[9]), "r"(a[10]), "r"(a[11]), "r"(a[12]), "r"(a[13]), "r"(a[14]), "r"(a[15]) : "memory");
        asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
        asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
        asm volatile("bar.sync %0, 128;" ::"r"(1 + wg) : "memory");
        if ((tid & 127) == 0) {
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = tmem + kSlotCol + (wg * 2 + slot) * kSlotCols;
#pragma unroll
            for (int s = 0; s < 2; ++s) {
                const uint64_t bd = b_desc(smem_u32(xs + (size_t)(2 * c + s) * kStepBytes));
                const uint32_t accumulate = (it > 0 || s > 0) ? 1u : 0u;
                asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }"
                             ::"r"(acc_addr), "r"(a_addr + s * 8), "l"(bd), "r"(kIdesc), "r"(accumulate) : "memory");
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_free[wg][slot])) : "memory");
            if (c + kWarpgroups >= n_chunks)
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_done[wg])) : "memory");
        }
    }
    const int my_iters = it;                                     // chunks this warpgroup issued (may be 0)
    __syncthreads();                                             // s_sumx / s_sumxp visible; all MMAs issued

    // ---- epilogue: warpgroup 0 adds the four accumulators of its rows in a fixed order
    float v[kNB];
#pragma unroll
    for (int b = 0; b < kNB; ++b) v[b] = 0.f;
    if (wg == 0) {
        for (int w = 0; w < kWarpgroups; ++w) {
            const int iters_w = (n_chunks > w) ? (n_chunks - w + kWarpgroups - 1) / kWarpgroups : 0;
            if (iters_w == 0) continue;                          // that accumulator was never written
            ok &= mbar_wait(smem_u32(&s_done[w]), 0);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            uint32_t d[kNB];
            const uint32_t addr = tmem + ((uint32_t)(quad * 32) << 16) + kAccCol + w * kNB;
            asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                         : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]),
                           "=r"(d[8]), "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                         : "r"(addr) : "memory");
            asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
            for (int b = 0; b < kNB; ++b) v[b] += __uint_as_float(d[b]);
        }
        const int64_t row = row0 + row_l;
#pragma unroll
        for (int b = 0; b < kNB; ++b) {
            if (b >= P.B) continue;
            float val = v[b] - 128.0f * s_sumxp[b];
            if (P.ovf_row_ptr && row < P.N) {                    // extra-precision columns: their field is one higher
                const __nv_bfloat16* xr = P.x + (int64_t)b * P.ldx;
                const int32_t pe = P.ovf_row_ptr[row + 1];
                float ev = 0.f;
                for (int32_t p = P.ovf_row_ptr[row] + split; p < pe; p += n_split) ev += __bfloat162float(xr[P.ovf_col[p]]);
                val += ev;
            }
            if (n_split == 1) {
                if (row < P.N) P.y[(int64_t)b * P.ldy + row] = a_pre * (val * (float)(1 << sh) - z_pre * s_sumx[b]);
            } else {
                s_part[row_l][b] = val;
            }
        }
    }
    (void)my_iters;
    if (!ok && lane == 0) report(P.dev_status, MATQ_ERR_TIMEOUT);

    // ---- K slices: sum across the cluster in rank order
    if (n_split > 1) {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();
        const int rows_per = (kRows + n_split - 1) / n_split;
        const int r_lo = split * rows_per, r_hi = min(kRows, r_lo + rows_per);
        for (int e = r_lo * kNB + tid; e < r_hi * kNB; e += kThreads) {
            const int rl = e / kNB, b = e % kNB;
            const int64_t row = row0 + rl;
            if (row >= P.N || b >= P.B) continue;
            float sum = 0.f, sumx = 0.f;
            for (int s = 0; s < n_split; ++s) {
                sum += cluster.map_shared_rank(&s_part[0][0], s)[e];
                sumx += cluster.map_shared_rank(s_sumx, s)[b];
            }
            P.y[(int64_t)b * P.ldy + row] = P.alpha[row] * (sum * (float)(1 << sh) - P.zero[row] * sumx);
        }
        cluster.sync();                                          // peers may still be reading this CTA's tile
    }

    // ---- release tensor memory (all tcgen05 traffic of this CTA has been waited for above)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

// Host side.  Returns MATQ_ERR_SHAPE when the call does not fit this kernel (the caller then uses another path).
template <int R>
inline int launch(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                  const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                  float* y, int64_t ldy, int32_t* dev_status, bool pdl, cudaStream_t s) {
    constexpr int kSlotBytes = 16 * 2 / Fmt<R>::kStepsPerChunk;
    Params P;
    P.packed = packed; P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y; P.dev_status = dev_status;
    P.N = N; P.K = K; P.ldx = ldx; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    P.B = B;
    P.pdl = pdl ? 1 : 0;
    const int64_t row_blocks = (N + kRows - 1) / kRows;
    const int sms = sm_count();
    // shared memory per byte of row slice: 128 tile bytes + x' (512 bytes per step = per kSlotBytes / 2 row bytes)
    auto smem_for = [&](int64_t sb) {
        return (size_t)kRows * (size_t)(((sb + 127) / 128) * 128 + 16) + (size_t)(sb / kSlotBytes) * 2 * kStepBytes;
    };
    int n_split = (int)((sms + row_blocks - 1) / row_blocks);     // about one CTA per SM
    if (n_split < 1) n_split = 1;
    if (n_split > 8) n_split = 8;
    int64_t sb = 0;
    for (;; ++n_split) {
        if (n_split > 8) return MATQ_ERR_SHAPE;
        sb = ((P.row_bytes + n_split - 1) / n_split + 15) / 16 * 16;
        if (smem_for(sb) <= 200 * 1024) break;
    }
    n_split = (int)((P.row_bytes + sb - 1) / sb);
    P.slice_bytes = (int)sb;
    P.tile_stride = (int)(((sb + 127) / 128) * 128 + 16);          // 16 mod 128: conflict-free 16-byte reads down a column of rows
    // At least 80 KB per CTA keeps residency at two CTAs per SM, which is what the 512 TMEM columns allow
    // (2 x 256): tcgen05.alloc then never has to wait for another CTA.
    const size_t smem = smem_for(sb) < 80 * 1024 ? 80 * 1024 : smem_for(sb);
    auto kern = gemv_tcgen05<R>;
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

}  // namespace t5
}  // namespace matq
