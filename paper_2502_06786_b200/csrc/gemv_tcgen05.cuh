// Decode GEMV on the fifth-generation tensor cores (tcgen05.mma, accumulator and the A operand in tensor memory).
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
// Warp roles (13 warps):
//   warps 0-7   two "unpack" warpgroups.  Each owns two TMEM slots of 32 columns (4 instructions' worth of A) and
//               fills them round-robin from the shared-memory weight tile; an mbarrier per slot says "ready", the
//               tcgen05.commit of the instructions that read a slot says "free".  They start as soon as the weights
//               land, i.e. BEFORE the kernel's predecessor in the stream has finished.
//   warps 8-11  wait for the predecessor (programmatic dependent launch), stage x' and the two sums, signal "x ready".
//   warp 12     one lane issues the TMA copies of the weight tile (before the dependency wait) and later all MMAs,
//               always in slot order and round-robin over eight accumulators (a fixed assignment, so results are
//               reproducible); one accumulator alone would serialise the tiny N = 16 instructions on their latency.
//
// Data movement.  The CTA's slice of the packed plane is fetched as 128-byte x 128-row boxes of a 2-D tensor map over
// the plane (uint8, 128-byte swizzle so that 32 rows can be read 16 bytes at a time without bank conflicts; rows and
// bytes outside the matrix arrive as zeros); every copy goes to the loading CTA only.  TMEM is allocated before the dependents are released, so
// a waiting successor can never starve a predecessor of tensor memory.  Slices of K (grid.y > 1) form a thread-block
// cluster and are summed through distributed shared memory in rank order.  No global scratch, no atomics.
#pragma once
#include <cooperative_groups.h>
#include <cuda.h>

#include "common.cuh"

namespace matq {
namespace t5 {
namespace cg = cooperative_groups;

constexpr int kUnpackWarps = 8, kStageWarps = 4;
constexpr int kThreads = 32 * (kUnpackWarps + kStageWarps + 1);
constexpr int kRows = 128;                   // M of the MMA = TMEM lanes
constexpr int kNB = 16;                      // N of the MMA = batch columns (padded)
constexpr int kSlotCols = 32;                // TMEM columns of one A slot = four K = 16 instructions
constexpr int kSlots = 2;                    // slots per unpack warpgroup
constexpr int kAccs = 8;                     // independent accumulators: consecutive MMAs into ONE accumulator would
                                             // each wait out the previous one's full latency (N = 16 is a tiny instruction)
constexpr int kTmemCols = 256;               // 8 accumulators x 16 + 2 warpgroups x 2 slots x 32 = 256
constexpr int kAccCol = 0, kSlotCol = kAccs * kNB;
constexpr int kBoxBytes = 128 * kRows;       // one TMA box: 128 bytes of 128 rows
constexpr int kMaxBoxes = 8;
constexpr uint32_t kSpinLimit = 1u << 22;    // mbarrier polls before a wait gives up

struct Params {
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
    int slice_bytes;     // bytes of a row handled by one CTA (multiple of 128 except possibly the last slice)
    int step_bytes;      // x' bytes of one instruction: 256 (B <= 8: both column groups read the same 128 bytes) or 512
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

// Shared-memory matrix descriptor of one x' step: K-major, no swizzle, 8 x 16-byte core matrices.  The two k-halves
// are lbo bytes apart (leading byte offset), the two groups of 8 batch columns sbo bytes (stride byte offset; 0 makes
// columns 8..15 re-read columns 0..7, whose results are never used when B <= 8).
__device__ __forceinline__ uint64_t b_desc(uint32_t smem_addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((smem_addr >> 4) & 0x3fffu) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}
// kind::f16, D = fp32, A = B = bf16, both K-major, N = 16, M = 128
constexpr uint32_t kIdesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kNB >> 3) << 17) | ((uint32_t)(kRows >> 4) << 24);

template <int R>
__global__ void __launch_bounds__(kThreads, 2)
gemv_tcgen05(const __grid_constant__ CUtensorMap tm_w, const Params P) {
    constexpr int sh = kCodeBits - R;
    constexpr int kKPerStep = Fmt<R>::kKPerStep;
    constexpr int kSlotBytes = 16 * 4 / Fmt<R>::kStepsPerChunk;   // row bytes unpacked into one slot (four steps): 32 or 16
    constexpr int kWordsPerSlot = kSlotBytes / 4;
    constexpr int kPairsPerWord = kSlotCols / kWordsPerSlot;

    extern __shared__ __align__(1024) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_wbar[kMaxBoxes];          // box b of the weight tile has landed
    __shared__ __align__(8) uint64_t s_ready[2][kSlots];         // slot filled by all 128 threads of its warpgroup
    __shared__ __align__(8) uint64_t s_free[2][kSlots];          // the instructions that read the slot have retired
    __shared__ __align__(8) uint64_t s_xready, s_done;
    __shared__ uint32_t s_tmem;
    __shared__ float s_red[2][kStageWarps][kNB];
    __shared__ float s_sumx[kNB], s_sumxp[kNB];
    __shared__ float s_part[kRows][kNB];                         // this CTA's partial outputs (cluster reduction)
    __shared__ int s_timeout;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int split = blockIdx.y, n_split = gridDim.y;
    const int64_t row0 = (int64_t)blockIdx.x * kRows;
    const int64_t slice_off = (int64_t)split * P.slice_bytes;
    const int my_bytes = (int)min((int64_t)P.slice_bytes, P.row_bytes - slice_off);    // multiple of 16, >= 16
    const int n_boxes = (my_bytes + 127) / 128;
    const int n_slots = (my_bytes + kSlotBytes - 1) / kSlotBytes;
    const int n_steps = n_slots * 4;

    unsigned char* wt = smem_raw + ((1024 - (smem_u32(smem_raw) & 1023)) & 1023);      // [box][128 rows][128 B], swizzled
    unsigned char* xs = wt + (size_t)n_boxes * kBoxBytes;                              // [step][step_bytes]

    // ---- barriers, tensor memory, weight copies: nothing here depends on the previous kernel
    if (tid == 0) {
        for (int b = 0; b < kMaxBoxes; ++b) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_wbar[b])));
        for (int w = 0; w < 2; ++w)
            for (int sl = 0; sl < kSlots; ++sl) {
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 128;" ::"r"(smem_u32(&s_ready[w][sl])));
                asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_free[w][sl])));
            }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&s_xready)), "r"(32 * kStageWarps));
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&s_done)));
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        s_timeout = 0;
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&s_tmem)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem = s_tmem;
    if (P.pdl) asm volatile("griddepcontrol.launch_dependents;");

    if (warp < kUnpackWarps) {
        // ================= unpack warpgroups: weights -> bf16x2 -> TMEM slots; warpgroup 0 also finishes the rows
        const int wg = warp >> 2, quad = warp & 3;
        const int row_l = quad * 32 + lane;
        bool ok = true;
        float a_pre = 0.f, z_pre = 0.f;
        if (wg == 0 && row0 + row_l < P.N) { a_pre = P.alpha[row0 + row_l]; z_pre = P.zero[row0 + row_l]; }
        int landed = 0;                                          // boxes this thread has already waited for
        int it = 0;
        for (int s = wg; s < n_slots; s += 2, ++it) {
            const int slot = it % kSlots;
            if (it >= kSlots) ok &= mbar_wait(smem_u32(&s_free[wg][slot]), (uint32_t)(it / kSlots - 1) & 1u);
            const int off = s * kSlotBytes;
            const int box = off >> 7;
            while (landed <= box) { ok &= mbar_wait(smem_u32(&s_wbar[landed]), 0); ++landed; }
            const unsigned char* rowp = wt + (size_t)box * kBoxBytes + row_l * 128;
            const int j0 = (off & 127) >> 4;
            uint32_t wv[8];
            {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + ((j0 ^ (row_l & 7)) << 4));
                wv[0] = v.x; wv[1] = v.y; wv[2] = v.z; wv[3] = v.w;
            }
            if (kWordsPerSlot == 8) {
                const uint4 v = *reinterpret_cast<const uint4*>(rowp + (((j0 + 1) ^ (row_l & 7)) << 4));
                wv[4] = v.x; wv[5] = v.y; wv[6] = v.z; wv[7] = v.w;
            }
            uint32_t a[kSlotCols];
#pragma unroll
            for (int i = 0; i < kSlotCols; ++i) a[i] = field_pair<R>(wv[i / kPairsPerWord], i % kPairsPerWord);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t slot_addr = tmem + ((uint32_t)(quad * 32) << 16) + kSlotCol + (wg * kSlots + slot) * kSlotCols;
            asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
                         "{%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                         ::"r"(slot_addr), "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(a[4]), "r"(a[5]), "r"(a[6]), "r"(a[7]),
                           "r"(a[8]), "r"(a[9]), "r"(a[10]), "r"(a[11]), "r"(a[12]), "r"(a[13]), "r"(a[14]), "r"(a[15]),
                           "r"(a[16]), "r"(a[17]), "r"(a[18]), "r"(a[19]), "r"(a[20]), "r"(a[21]), "r"(a[22]), "r"(a[23]),
                           "r"(a[24]), "r"(a[25]), "r"(a[26]), "r"(a[27]), "r"(a[28]), "r"(a[29]), "r"(a[30]), "r"(a[31]) : "memory");
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&s_ready[wg][slot])) : "memory");
        }
        if (wg == 0) {
            // ---- epilogue: the accumulator of this thread's row
            ok &= mbar_wait(smem_u32(&s_done), 0);
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            float acc[kNB];
#pragma unroll
            for (int b = 0; b < kNB; ++b) acc[b] = 0.f;
            const int used = n_steps < kAccs ? n_steps : kAccs;  // accumulators that were written at all
            for (int a = 0; a < used; ++a) {                     // fixed order: results are reproducible
                uint32_t d[kNB];
                const uint32_t addr = tmem + ((uint32_t)(quad * 32) << 16) + kAccCol + a * kNB;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                             : "=r"(d[0]), "=r"(d[1]), "=r"(d[2]), "=r"(d[3]), "=r"(d[4]), "=r"(d[5]), "=r"(d[6]), "=r"(d[7]),
                               "=r"(d[8]), "=r"(d[9]), "=r"(d[10]), "=r"(d[11]), "=r"(d[12]), "=r"(d[13]), "=r"(d[14]), "=r"(d[15])
                             : "r"(addr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int b = 0; b < kNB; ++b) acc[b] += __uint_as_float(d[b]);
            }
            const int64_t row = row0 + row_l;
#pragma unroll
            for (int b = 0; b < kNB; ++b) {
                if (b >= P.B) continue;
                float val = acc[b] - 128.0f * s_sumxp[b];
                if (P.ovf_row_ptr && row < P.N) {                // extra-precision columns: their field is one higher
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
        if (!ok) s_timeout = 1;
    } else if (warp < kUnpackWarps + kStageWarps) {
        // ================= stage warps: the only readers of x; everything after this point depends on the predecessor
        if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
        const int st_tid = tid - 32 * kUnpackWarps;              // 0..127
        const int bcol = st_tid & (kNB - 1);
        const int64_t k_base = slice_off * 8 / R;
        const bool wide = P.step_bytes == 512;
        float sx = 0.f, sxp = 0.f;
        if (wide || bcol < 8) {
            for (int st = st_tid >> 4; st < n_steps; st += (32 * kStageWarps) / kNB) {
                const int64_t k = k_base + (int64_t)st * kKPerStep;
                uint4 h0 = make_uint4(0, 0, 0, 0), h1 = h0;
                if (bcol < P.B && k < P.K) stage_step<R>(P.x + (int64_t)bcol * P.ldx + k, h0, h1, sx, sxp);
                unsigned char* base = xs + (size_t)st * P.step_bytes + (wide ? (bcol >> 3) * 128 : 0) + (bcol & 7) * 16;
                *reinterpret_cast<uint4*>(base) = h0;
                *reinterpret_cast<uint4*>(base + (wide ? 256 : 128)) = h1;
            }
        }
        sx += __shfl_xor_sync(0xffffffffu, sx, 16);  sxp += __shfl_xor_sync(0xffffffffu, sxp, 16);
        const int sw = warp - kUnpackWarps;
        if (lane < kNB) { s_red[0][sw][lane] = sx; s_red[1][sw][lane] = sxp; }
        asm volatile("bar.sync 1, 128;" ::: "memory");           // the four stage warps
        if (st_tid < kNB) {
            float a = 0.f, b = 0.f;
            for (int w = 0; w < kStageWarps; ++w) { a += s_red[0][w][st_tid]; b += s_red[1][w][st_tid]; }
            s_sumx[st_tid] = a;
            s_sumxp[st_tid] = b;
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // x' was written with ordinary stores, the MMA reads it
        asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&s_xready)) : "memory");
    } else if (lane == 0) {
        // ================= control lane: weight copies now, all MMAs later (in slot order)
        for (int b = 0; b < n_boxes; ++b) {
            const uint32_t bar = smem_u32(&s_wbar[b]);
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(kBoxBytes) : "memory");
            asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                         ::"r"(smem_u32(wt + (size_t)b * kBoxBytes)), "l"(&tm_w), "r"((int)(slice_off + b * 128)), "r"((int)row0), "r"(bar) : "memory");
        }
        bool ok = mbar_wait(smem_u32(&s_xready), 0);
        const uint32_t lbo = P.step_bytes == 512 ? 256u : 128u, sbo = P.step_bytes == 512 ? 128u : 0u;
        // descriptor of step 0; later steps only move the start address (14-bit field in units of 16 bytes)
        uint64_t bd = b_desc(smem_u32(xs), lbo, sbo);
        const uint64_t bd_step = (uint64_t)(P.step_bytes >> 4);
        int n_mma = 0;                                            // MMA number n accumulates into accumulator n % kAccs
        for (int s = 0; s < n_slots && ok; ++s) {
            const int wg = s & 1, it = s >> 1, slot = it % kSlots;
            ok &= mbar_wait(smem_u32(&s_ready[wg][slot]), (uint32_t)(it / kSlots) & 1u);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t a_addr = tmem + kSlotCol + (wg * kSlots + slot) * kSlotCols;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                asm volatile("{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p; }"
                             ::"r"(tmem + kAccCol + (n_mma % kAccs) * kNB), "r"(a_addr + i * 8), "l"(bd), "r"(kIdesc),
                               "r"(n_mma >= kAccs ? 1u : 0u) : "memory");
                ++n_mma;
                bd += bd_step;
            }
            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_free[wg][slot])) : "memory");
        }
        // arrives when every MMA above has retired (also after a give-up, so the epilogue never waits in vain)
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(&s_done)) : "memory");
        if (!ok) s_timeout = 1;
    }

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

    // ---- release tensor memory (every tcgen05 operation of this CTA has been waited for above)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (tid == 0 && s_timeout) report(P.dev_status, MATQ_ERR_TIMEOUT);
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
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

// Returns MATQ_ERR_SHAPE when the call does not fit this kernel (the caller then uses another path).
template <int R>
inline int launch(const uint8_t* packed, int64_t N, int64_t K, const float* alpha, const float* zero,
                  const int32_t* ovf_row_ptr, const uint16_t* ovf_col, const void* x, int B, int64_t ldx,
                  float* y, int64_t ldy, int32_t* dev_status, bool pdl, cudaStream_t s) {
    constexpr int kSlotBytes = 16 * 4 / Fmt<R>::kStepsPerChunk;
    Params P;
    P.alpha = alpha; P.zero = zero; P.ovf_row_ptr = ovf_row_ptr; P.ovf_col = ovf_col;
    P.x = static_cast<const __nv_bfloat16*>(x); P.y = y; P.dev_status = dev_status;
    P.N = N; P.K = K; P.ldx = ldx; P.ldy = ldy;
    P.row_bytes = K * R / 8;
    P.B = B;
    P.step_bytes = B <= 8 ? 256 : 512;
    P.pdl = pdl ? 1 : 0;
    if (P.row_bytes % 16 != 0 || P.row_bytes >= (1ll << 31) || N >= (1ll << 31)) return MATQ_ERR_SHAPE;
    const int64_t row_blocks = (N + kRows - 1) / kRows;
    const int sms = sm_count();
    auto smem_for = [&](int64_t sb) {
        const int64_t boxes = (sb + 127) / 128, slots = (sb + kSlotBytes - 1) / kSlotBytes;
        return (size_t)(boxes * kBoxBytes + slots * 4 * P.step_bytes + 1024);
    };
    // slices of whole 128-byte boxes; about one CTA per SM, at most 8 slices (portable cluster), at most kMaxBoxes boxes
    const int64_t total_boxes = (P.row_bytes + 127) / 128;
    int n_split = (int)((sms + row_blocks - 1) / row_blocks);
    if (n_split < 1) n_split = 1;
    if (n_split > 8) n_split = 8;
    if (n_split > total_boxes) n_split = (int)total_boxes;
    int64_t sb = 0;
    for (;; ++n_split) {
        if (n_split > 8 || n_split > total_boxes) return MATQ_ERR_SHAPE;
        sb = ((total_boxes + n_split - 1) / n_split) * 128;
        if (sb / 128 <= kMaxBoxes && smem_for(sb) <= 200 * 1024) break;
    }
    n_split = (int)((P.row_bytes + sb - 1) / sb);
    P.slice_bytes = (int)sb;
    CUtensorMap tm;
    {
        EncodeTiledFn fn = encode_fn();
        if (!fn) return MATQ_ERR_CUDA;
        const cuuint64_t dims[2] = {(cuuint64_t)P.row_bytes, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)P.row_bytes};
        const cuuint32_t box[2] = {128, (cuuint32_t)kRows};
        const cuuint32_t estr[2] = {1, 1};
        if (fn(&tm, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, const_cast<uint8_t*>(packed), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return MATQ_ERR_SHAPE;
    }
    // At least 80 KB per CTA keeps residency at two CTAs per SM, which is what the 512 TMEM columns allow
    // (2 x 256): tcgen05.alloc then never has to wait for another CTA.
    const size_t smem = smem_for(sb) < 80 * 1024 ? 80 * 1024 : smem_for(sb);
    auto kern = gemv_tcgen05<R>;
    static std::atomic<unsigned long long> smem_ok{0};
    if (!opt_in_max_smem(kern, smem_ok)) return MATQ_ERR_CUDA;
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
    if (cudaLaunchKernelEx(&cfg, kern, tm, P) != cudaSuccess) { cudaGetLastError(); return MATQ_ERR_CUDA; }
    return MATQ_OK;
}

}  // namespace t5
}  // namespace matq
