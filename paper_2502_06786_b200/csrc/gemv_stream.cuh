// Decode GEMV for single activation vectors (B = 1) as ONE persistent kernel
// over a list of problems: the planes are streamed by the copy engine into a
// ring in shared memory, the multiplies are the integer warp MMAs of
// gemv_imma.cuh.
//
// Why.  A packed plane of a decoder layer is 2-50 MB, i.e. 0.4-8 us of HBM
// time, and a kernel per plane spends about 2 us per launch on a chain that no
// amount of tuning removes (dependency wait, activations, multiply, K-split
// sum, store, drain).  Here
//   * one CTA per SM stays resident for the whole list; each CTA owns a
//     contiguous share of the list's (16-row tile x 64-byte chunk) items, cut
//     at tile boundaries, so SMs are balanced to within one tile whatever the
//     shapes are, and a CTA prepares the activations only of the one to three
//     problems its share touches;
//   * one producer warp feeds a ring of stages (up to 18.5 KB each) with ONE copy per stage
//     (completion counted on an mbarrier).  A stage is one UNIT: rows of up to
//     1184 bytes are staged whole, 1 to 4 consecutive 16-row tiles being one
//     contiguous run of the plane (cp.async.bulk); longer rows are cut into K
//     panels of at most 1088 bytes and a unit is the 16 x panel box of a tensor
//     map over the plane (cp.async.bulk.tensor.2d; rows and columns past the
//     end arrive as zeros).  One copy per unit matters: the copy engine takes
//     about 55 ns per request whatever its size, so a copy per row segment
//     cannot reach the HBM rate.  150 KB and more per SM are in flight
//     independently of what the multiplying warps do, and with programmatic
//     dependent launch the ring is filled while the previous kernel of the
//     stream is still running;
//   * every unit is multiplied by ONE consumer warp (unit s of a CTA's share of
//     a problem goes to warp s mod W, and the number of stages is a multiple of
//     W, so a stage always serves the same warp and a warp never has to ask
//     whether an older use of its stage has completed): A fragments come from the stage with
//     128-bit loads, B fragments from the staged activation bytes exactly as in
//     gemv_imma, into eight independent accumulator sets.  Warps never wait for
//     one another while a problem is being multiplied:
//       - when the share has at least W tiles, the units are ordered so that a
//         warp receives all panels of "its" tiles; it keeps the sums in
//         registers and finishes the 16 outputs alone (three shuffles per row);
//         at r = 2 a unit holds two tiles and both are multiplied in one pass,
//         so that the activation fragments are loaded once for 32 rows;
//       - when it has fewer tiles than warps and rows of several panels, the
//         panels of a tile are spread over the warps; each adds its partial
//         sums to a small accumulator in shared memory with integer atomics and
//         the warp that arrives last finishes the tile.
//     Integer sums do not depend on their order, so the result is reproducible
//     and does not depend on how the list was cut or which warp came last.
// The arithmetic (fields masked in place as exact 8-bit operands, activations
// as the four bytes of a block-scaled integer, a constant column that removes
// the offsets) is that of gemv_imma.cuh and is described there; the masks are
// nested here (see stage_activations), which saves a quarter to a half of them.
//
// Extra precision (Errata, Eq. 8): a listed column's field is one bucket higher
// than the stored, clamped one, so its activation is added once more in fp32.
// That sparse term is a matrix-vector product with the lists as a CSR pattern of
// ones; it has nothing in common with the dense stream (two dependent
// global-memory round trips per row, 2-byte indices, gathers), so it runs as a
// kernel of its own (ep_rowsum: eight lanes per row, many rows in flight) that
// leaves sum_{j in list(n)} x_j in y[n]; the persistent kernel, launched as its
// programmatic dependent, picks the value up when it finishes row n.
//
// Every wait is bounded (a limit in clock cycles, about two seconds): a wait
// that gives up sets a flag in shared memory and MATQ_ERR_TIMEOUT in
// dev_status; from then on every wait returns at once, the control flow of all
// warps (trip counts, named barriers) stays the same, nothing more is stored,
// and the producer waits, bounded, for the copies it still has in flight before
// the CTA returns.
#pragma once
#include <algorithm>
#include <atomic>
#include <type_traits>

#include "common.cuh"
#include "gemv_imma.cuh"
#include "gemv_tcgen05.cuh"
#include "gemv_tensor.cuh"

namespace matq {
namespace gstream {

constexpr int kMaxSlots = 24;
constexpr int kUnitRow = 1184;                // bytes per row of the largest unit (16 rows)
constexpr int kMaxTpu = 4;                   // tiles per unit at most
constexpr int kMaxW = 11;                   // consumer warps at most (with the producer: 12 warps, 168 registers a thread)
constexpr int kPairs = 1;                    // units of an even number of tiles, two tiles multiplied per pass (see geometry())
constexpr int kFewW = 8;                    // ... on lists with little work per CTA and for batches: two per sub-partition
constexpr int kManyItems = 1000;            // items per CTA from which a list gets kMaxW warps: eleven warps measured 1-4 %
                                            // faster on whole decoder stacks and 8-12 % slower on a layer's three matrices
constexpr int kTileSlots = kMaxW;            // shared-memory accumulators of tiles whose panels are spread over warps
constexpr int kStaticReserve = 16 * 1024;    // static shared memory of the kernel, rounded up
constexpr int kSmallList = 8;
constexpr int kLargeList = 128;
constexpr int kSmemLimit = 227 * 1024;
constexpr int kSets = 8;                     // independent accumulator sets of a warp
constexpr unsigned kWaitHintNs = 2000;       // longest suspension of one probe of a stage by a multiplying warp
constexpr unsigned kProducerNapNs = 100;     // pause of the producer warp when it has nothing to issue

struct Problem {
    const uint8_t* packed;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const __nv_bfloat16* x;
    float* y;
    int N, K;
    int r;
    int B;                    // activation vectors (1 in gemv_stream; 2 .. 8 in gemv_stream_batch)
    long long item0;          // cost (tile_cost units) of the problems before this one
};

template <int NP>
struct Params {
    CUtensorMap tm[NP];       // over each plane as [N][row_bytes / 8] 64-bit words, box 16 x panel (only read for long rows)
    Problem p[NP];
    long long items;          // total cost of the list (tile_cost units: sixteenths of an item)
    long long wait_cycles;    // limit of a wait, in SM clock cycles
    int32_t* dev_status;
    int n;                    // problems
    int slots;                // ring stages in use
    int slot_bytes;
    int xs_bytes;             // staged activation bytes (largest problem)
    int W;                    // consumer warps
    int pdl;                  // 0: plain launch; 1: programmatic dependent of an unknown kernel (wait before x is read);
                              // 2: dependent of ep_rowsum, released after that kernel's own wait (wait before its sums are read)
    int tails;                // whether a share that is not a whole number of rounds is cut in two (see next_segment)
    int unit_row;             // bytes per row of the largest unit
    int hold;                 // diagnostics: the producer issues no copies, so every wait for a stage runs out
    int pairs;                // geometry with an even number of tiles per unit (see geometry())
};

// Shape of a problem's units.  Short rows are staged whole: `tpu` (1 to 4) consecutive tiles are one contiguous run of the
// plane, rows `row_bytes` apart in shared memory.  Longer rows are cut into `n_panels` panels of `panel_qc` 64-byte
// chunks (an odd number, so that rows are an odd multiple of 64 bytes apart and the 128-bit loads of a quarter warp fall
// into different banks; the last panel may be shorter), and a unit is the box of 16 tpu rows x one panel.
// `pairs` = 0: rows of up to `unit_row` (1184) bytes are whole, a box is one tile high (panels of up to 17 chunks).
// `pairs` = 1 (taken at r = 2 only): a unit always holds an even number of tiles, so that two tiles can be multiplied in
// one pass with one load of the activation fragments: rows of up to unit_row / 2 bytes are whole (2 or 4 tiles), boxes
// are two tiles high (panels of up to 9 chunks).  The bytes of a unit are the same either way.
struct Geo {
    int row_bytes, n_qc, tiles, n_panels, panel_qc, stride, contig, tpu;
};
__host__ __device__ inline Geo geometry(int N, int K, int r, int unit_row, int pairs = 0) {
    const int kUnitBytes = 16 * unit_row;
    Geo g;
    g.row_bytes = K / 8 * r;
    g.n_qc = (g.row_bytes + 63) / 64;
    g.tiles = (N + 15) / 16;
    // Pairs pay at r = 2 only (measured, whole planes: +1 % at K = 2304, +3 % at 3584, +10 % at 9216; at r = 4 and 8 the
    // narrower panels cost 2-7 % more than the shared fragment loads save).  r = 2 with K % 256 == 128: the half-full
    // last chunk is handled one tile at a time.
    if (r != 2 || (g.row_bytes & 63)) pairs = 0;
    if (16 * (pairs ? 2 : 1) * g.row_bytes <= kUnitBytes) {
        g.contig = 1;
        g.tpu = kUnitBytes / (16 * g.row_bytes);
        if (g.tpu > kMaxTpu) g.tpu = kMaxTpu;
        if (pairs) g.tpu &= ~1;
        g.n_panels = 1;
        g.panel_qc = g.n_qc;
        g.stride = g.row_bytes;
        return g;
    }
    g.contig = 0;
    g.tpu = pairs ? 2 : 1;
    const int max_qc = pairs ? (kUnitBytes / 32) / 64 : (kUnitBytes / 16) / 64 - 1;      // 9 : 17, both odd
    g.n_panels = (g.n_qc + max_qc - 1) / max_qc;
    g.panel_qc = (g.n_qc + g.n_panels - 1) / g.n_panels;
    g.panel_qc |= 1;
    g.n_panels = (g.n_qc + g.panel_qc - 1) / g.panel_qc;
    g.stride = g.panel_qc * 64;
    return g;
}

// What a tile of a problem counts for when the list is divided among the CTAs, in sixteenths of a (tile x chunk) item:
// the list is cut into shares of equal COST, not of equal bytes.  Rows of four or more K panels cost the multiplying
// warps an eighth more per byte at r = 4 and r = 2 (measured: 9216-wide rows run at 0.78 / 0.56 of the HBM rate where
// 2304-wide rows run at 0.89 / 0.64); at r = 8 every shape is bound by HBM and a byte is a byte.
__host__ __device__ inline int tile_cost(const Geo& g, int r) { return g.n_qc * ((g.n_panels >= 4 && r != 8) ? 18 : 16); }

// How a CTA's share of a problem (T tiles, i.e. ceil(T / tpu) groups of tiles) is laid out as a sequence of units.
// Unit s goes to warp s mod W; the sequence is padded with empty units to a multiple of W.
//   at least W groups, or single-panel rows: rounds of W groups; within a round panel-major, so warp w meets
//     (group g W + w, panel 0), (same group, panel 1), ...;
//   fewer tiles than warps and several panels: tile-major, the panels of a tile are spread over the warps.
struct Plan {
    int split, n_units, tpu;
};
__host__ __device__ inline Plan plan_of(const Geo& g, int T, int W) {
    Plan pl;
    pl.tpu = g.tpu;
    if (g.contig && T < W * pl.tpu) pl.tpu = T / W > 1 ? T / W : 1;      // a short share of whole rows: fewer tiles per unit rather than idle warps
    const int Tu = (T + pl.tpu - 1) / pl.tpu;
    pl.split = (Tu < W && g.n_panels > 1) ? 1 : 0;
    pl.n_units = pl.split ? (Tu * g.n_panels + W - 1) / W * W : (Tu + W - 1) / W * g.n_panels * W;
    return pl;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// one probe of a phase; the hardware may suspend the thread for up to `hint_ns` before it answers
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity, uint32_t hint_ns) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity), "r"(hint_ns) : "memory");
    return ok != 0;
}
// one probe of a phase that never suspends
__device__ __forceinline__ bool mbar_test_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// one contiguous run of global memory into this CTA's shared memory; completion is counted in bytes on `bar`
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

// the 16-row box of a tensor map that starts at (64-bit word x, row y) into this CTA's shared memory
__device__ __forceinline__ void tensor_g2s(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar) : "memory");
}

// Bounded wait for phase `parity` of an mbarrier.  Returns false (and raises the abort flag) when it gives up; returns
// false at once when another wait of this CTA already gave up.  The limit is in SM clock cycles (reading the clock
// costs a few cycles; the nanosecond timer costs about a microsecond).
__device__ __forceinline__ bool wait_phase(uint32_t bar, uint32_t parity, volatile int* abort_flag, long long limit_cycles) {
    if (mbar_try_wait(bar, parity, kWaitHintNs)) return true;
    if (*abort_flag) return false;
    const long long t0 = clock64();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity, kWaitHintNs)) return true;
        if (*abort_flag) return false;
        if (clock64() - t0 > limit_cycles) { *abort_flag = 1; return false; }
    }
}

// The next problem (from index p on) of which this CTA owns tiles, and which: [t_lo, t_hi).  A share of rows with
// several K panels that is not a whole number of rounds (W groups of tiles, one per warp) comes as two segments: the
// whole rounds, which the warps take a tile each, and the rest (`tail_lo`, `tail_hi`: state of the iteration, -1 = none),
// fewer groups than warps, whose panels plan_of() spreads over all warps; otherwise the last round would keep a few
// warps busy for a whole tile (K = 9216 at r = 8: 147 KB) while the others idle.  Problem p - 1 is the current one for
// both segments.
template <int NP>
__device__ __forceinline__ bool next_segment(const Params<NP>& P, long long lo, long long hi, int& p, int& t_lo, int& t_hi, int& tail_lo, int& tail_hi) {
    if (tail_lo >= 0) {
        t_lo = tail_lo; t_hi = tail_hi;
        tail_lo = -1;
        return true;
    }
    while (p < P.n) {
        const long long i0 = P.p[p].item0;
        if (i0 >= hi) return false;
        const Geo g = geometry(P.p[p].N, P.p[p].K, P.p[p].r, P.unit_row, P.pairs);
        const int tc = tile_cost(g, P.p[p].r);
        const long long a = lo > i0 ? (lo - i0 + tc - 1) / tc : 0;
        const long long b = (hi - i0 + tc - 1) / tc;
        ++p;
        t_lo = (int)(a < g.tiles ? a : g.tiles);
        t_hi = (int)(b < g.tiles ? b : g.tiles);
        if (t_lo < t_hi) {
            if (P.tails && g.n_panels > 1) {
                const int Tu = (t_hi - t_lo + g.tpu - 1) / g.tpu, rem = Tu % P.W;
                if (Tu > P.W && rem != 0 && rem <= P.W - 2) {
                    tail_lo = t_lo + (Tu - rem) * g.tpu; tail_hi = t_hi;
                    t_hi = tail_lo;
                }
            }
            return true;
        }
    }
    return false;
}

// 128-bit shared-memory load that only the lanes with `on` execute; the others keep what `v` held.
__device__ __forceinline__ void lds128_if(uint4& v, uint32_t addr, int on) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %5, 0;\n @p ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];\n}"
                 : "+r"(v.x), "+r"(v.y), "+r"(v.z), "+r"(v.w) : "r"(addr), "r"(on));
}

// One (tile, chunk) item: 16 rows x 64 bytes of plane from the stage, times the staged activation bytes.  B source:
// the lanes of byte column g < 4 (`col_lane`) load their column of the chunk's staged units from shared memory
// (`x_sa`: shared address of the first unit, the next one 256 bytes further); the lanes g = 4 hold the constant
// column in `xb` and keep it (the load is predicated off for them, which also halves the shared-memory wavefronts of
// the B loads); what the lanes g > 4 hold is irrelevant, columns 5-7 of the product are never read.
// The 2 * kM2 MMAs go to accumulator sets SET0, SET0 + 1, ...
template <int R, int SET0>
__device__ __forceinline__ void multiply_item(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, int col_lane,
                                              uint4 (&xb)[(128 / R) / 16], int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    const uint4 wl = *reinterpret_cast<const uint4*>(wl_p);
    const uint4 wh = *reinterpret_cast<const uint4*>(wh_p);
#pragma unroll
    for (int m2 = 0; m2 < kM2; ++m2) lds128_if(xb[m2], x_sa + m2 * 256, col_lane);
#pragma unroll
    for (int m2 = 0; m2 < kM2; ++m2) {
#pragma unroll
        for (int sub = 0; sub < 2; ++sub) {
            const uint32_t b0 = sub ? xb[m2].z : xb[m2].x, b1 = sub ? xb[m2].w : xb[m2].y;
            uint32_t a0, a1, a2, a3;
            if (R == 8) {
                a0 = sub ? wl.z : wl.x;  a2 = sub ? wl.w : wl.y;
                a1 = sub ? wh.z : wh.x;  a3 = sub ? wh.w : wh.y;
            } else {
                const int j = R == 4 ? 2 * m2 + sub : m2;
                const uint32_t w_lo = j == 0 ? wl.x : j == 1 ? wl.y : j == 2 ? wl.z : wl.w;
                const uint32_t w_hi = j == 0 ? wh.x : j == 1 ? wh.y : j == 2 ? wh.z : wh.w;
                // nested masks: operand i keeps fields 0 .. i of its byte (the last one is the byte as it stands)
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
            imma::mma_u8u8(acc[SET0 + 2 * m2 + sub], a0, a1, a2, a3, b0, b1);
        }
    }
}

// All chunks of one unit's tile panel.  `wl_p` / `wh_p`: this lane's 16 bytes of rows g and g + 8 in the first chunk;
// `x_sa`: shared address of its B source for that chunk, `xq_bytes` per chunk further for the next; `cz`: the
// constant column (lanes g = 4).  Four chunks (two at r = 2) are taken per round: their loads are issued together,
// and the eight accumulator sets are used in turn, so that neither the shared-memory latency nor the MMA latency
// sits between two MMAs of a warp.
template <int R>
__device__ __forceinline__ void multiply_unit(const unsigned char* wl_p, const unsigned char* wh_p, uint32_t x_sa, int xq_bytes, int col_lane,
                                              const uint4& cz, int n_chunks, int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kU = R == 2 ? 2 : 4;                    // chunks per round
    uint4 xb[kU][kM2];
#pragma unroll
    for (int i = 0; i < kU; ++i)
#pragma unroll
        for (int m2 = 0; m2 < kM2; ++m2) xb[i][m2] = cz;
#define MATQ_ITEM(I) multiply_item<R, ((I) * 2 * kM2) % kSets>(wl_p + (c + (I)) * 64, wh_p + (c + (I)) * 64, x_sa + (c + (I)) * xq_bytes, col_lane, xb[I], acc)
    int c = 0;
#pragma unroll 1
    for (; c + kU <= n_chunks; c += kU) {
        MATQ_ITEM(0);
        MATQ_ITEM(1);
        if (kU >= 4) { MATQ_ITEM(2); MATQ_ITEM(3); }
    }
#pragma unroll 1
    for (; c < n_chunks; ++c) MATQ_ITEM(0);
#undef MATQ_ITEM
}

// Two consecutive tiles of a unit in one pass: the B fragments of a chunk (a third to two thirds of the 128-bit
// shared-memory loads of an item, and such a load costs a sub-partition more issue time than an MMA) are loaded once
// and used for both tiles' weights.  Tile 0 accumulates in sets 0-3, tile 1 in sets 4-7; a set is used again after
// eight MMAs.  `wl_p` / `wh_p` belong to tile 0, tile 1 lies `tile_bytes` further.
template <int R>
__device__ __forceinline__ void multiply_two_tiles(const unsigned char* wl_p, const unsigned char* wh_p, int tile_bytes, uint32_t x_sa, int xq_bytes,
                                                   int col_lane, const uint4& cz, int n_chunks, int (&acc)[kSets][4]) {
    constexpr int kM2 = (128 / R) / 16;
    constexpr int kFrag = 2 * kM2;                       // fragments (MMAs per tile) of an item: 2, 4, 8
    constexpr int kU = kFrag >= 4 ? 1 : 2;               // items per round: at least four fragments, one per set of a tile
    uint4 xb[kU][kM2];
#pragma unroll
    for (int i = 0; i < kU; ++i)
#pragma unroll
        for (int m2 = 0; m2 < kM2; ++m2) xb[i][m2] = cz;
    auto round = [&](int c, auto n_items) {
        constexpr int kN = decltype(n_items)::value;
        uint4 wl[kN][2], wh[kN][2];
#pragma unroll
        for (int i = 0; i < kN; ++i) {
#pragma unroll
            for (int tile = 0; tile < 2; ++tile) {
                wl[i][tile] = *reinterpret_cast<const uint4*>(wl_p + tile * tile_bytes + (c + i) * 64);
                wh[i][tile] = *reinterpret_cast<const uint4*>(wh_p + tile * tile_bytes + (c + i) * 64);
            }
#pragma unroll
            for (int m2 = 0; m2 < kM2; ++m2) lds128_if(xb[i][m2], x_sa + (uint32_t)((c + i) * xq_bytes) + m2 * 256, col_lane);
        }
#pragma unroll
        for (int i = 0; i < kN; ++i)
#pragma unroll
            for (int m2 = 0; m2 < kM2; ++m2)
#pragma unroll
                for (int sub = 0; sub < 2; ++sub) {
                    const uint32_t b0 = sub ? xb[i][m2].z : xb[i][m2].x, b1 = sub ? xb[i][m2].w : xb[i][m2].y;
#pragma unroll
                    for (int tile = 0; tile < 2; ++tile) {
                        const uint4& l = wl[i][tile];
                        const uint4& h = wh[i][tile];
                        uint32_t a0, a1, a2, a3;
                        if (R == 8) {
                            a0 = sub ? l.z : l.x;  a2 = sub ? l.w : l.y;
                            a1 = sub ? h.z : h.x;  a3 = sub ? h.w : h.y;
                        } else {
                            const int j = R == 4 ? 2 * m2 + sub : m2;
                            const uint32_t w_lo = j == 0 ? l.x : j == 1 ? l.y : j == 2 ? l.z : l.w;
                            const uint32_t w_hi = j == 0 ? h.x : j == 1 ? h.y : j == 2 ? h.z : h.w;
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
                        imma::mma_u8u8(acc[4 * tile + (i * kFrag + 2 * m2 + sub) % 4], a0, a1, a2, a3, b0, b1);
                    }
                }
    };
    int c = 0;
#pragma unroll 1
    for (; c + kU <= n_chunks; c += kU) round(c, std::integral_constant<int, kU>{});
    if (kU > 1 && c < n_chunks) round(c, std::integral_constant<int, 1>{});
}

// Activation bytes of one problem in B-fragment order (all chunks of a row).  The byte layout is that of
// gemv_imma.cuh; the values differ in one respect that saves a quarter (r = 2) or half (r = 4) of the mask
// instructions of the multiply.  With V_i = round(x_i 2^(P - e - R i)) for the activation that meets field i of a
// byte, gemv_imma pairs V_i with the operand f_i 2^(R i) (one mask per field).  Here operand i is the byte masked
// to its fields 0 .. i, A_i = sum_{j <= i} f_j 2^(R j) (the last one needs no mask at all), paired with
// Y_i = V_i - V_{i+1} (Y of the last field = V):  sum_i A_i Y_i = sum_j f_j 2^(R j) sum_{i >= j} Y_i = sum_j f_j 2^(R j) V_j,
// the same exact integer.  |Y_i| < 1.25 * 2^(P + 1 - R i), so the offset that makes it a non-negative 32-bit
// integer is 2^(P + 2 - R i); the constant column (2^(smax - R i) per byte) returns sum_i A_i 2^(smax - R i), which
// removes sum_i A_i 2^(P + 2 - R i) exactly.
constexpr int kHeld = 4;     // staging items (16 activations each) a thread keeps in registers between the two passes
constexpr int kSumThreads = 128;   // threads that sum x: the smallest number of consumer threads a launch can have (kMinW warps)

// Convert one staging item (16 consecutive activations, raw bf16 pairs) and store its byte units.
template <int R>
__device__ __forceinline__ void stage_item(const uint32_t (&raw)[8], const float (&mult)[8 / R], uint4* dst) {
    constexpr int kF = 8 / R;                                  // fields per byte
    int V[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float xf = (i & 1) ? bf_hi(raw[i >> 1]) : bf_lo(raw[i >> 1]);
        V[i] = __float2int_rn(xf * mult[i % kF]);
    }
    uint32_t v[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const int cls = i % kF;                              // 16 consecutive activations start at a byte boundary
        const int y = cls == kF - 1 ? V[i] : V[i] - V[i + 1 < 16 ? i + 1 : i];
        v[i] = (uint32_t)y + (1u << (imma::kP + 2 - R * cls));
    }
    uint32_t col[imma::kBytes][4];
#pragma unroll
    for (int w = 0; w < 4; ++w) {
        const uint32_t e0 = v[imma::unit_src<R>(4 * w)], e1 = v[imma::unit_src<R>(4 * w + 1)];
        const uint32_t e2 = v[imma::unit_src<R>(4 * w + 2)], e3 = v[imma::unit_src<R>(4 * w + 3)];
        const uint32_t t0 = __byte_perm(e0, e1, 0x5140), t1 = __byte_perm(e2, e3, 0x5140);
        const uint32_t t2 = __byte_perm(e0, e1, 0x7362), t3 = __byte_perm(e2, e3, 0x7362);
        col[0][w] = __byte_perm(t0, t1, 0x5410);  col[1][w] = __byte_perm(t0, t1, 0x7632);
        col[2][w] = __byte_perm(t2, t3, 0x5410);  col[3][w] = __byte_perm(t2, t3, 0x7632);
    }
#pragma unroll
    for (int d = 0; d < imma::kBytes; ++d) dst[4 * d] = make_uint4(col[d][0], col[d][1], col[d][2], col[d][3]);
}

// Stages the activations of one problem: every thread of the W consumer warps reads its items ONCE (the first
// kHeld of them stay in registers across the reduction), the largest magnitude and the fp32 sum are reduced over the
// CTA, then the items are converted and stored.  Two named barriers; the first also separates the previous
// problem's multiplies from the restaging.  Returns the sum of x and the biased exponent of max |x|.
template <int R>
__device__ __forceinline__ void stage_activations(const __nv_bfloat16* x, int K, int n_qc, uint4* xs, int ctid, int nthr, int W,
                                                  uint32_t* s_rmax, float* s_rsum, float& xsum_out, int& xexp_out) {
    constexpr int kWpp = 128 / R;
    constexpr int kM2 = kWpp / 16;
    constexpr int kF = 8 / R;
    const int lane = ctid & 31, warp = ctid >> 5;
    const int n_items = n_qc * kM2 * 4;
    auto k0_of = [&](int it) {
        const int tt = it & 3, qm = it >> 2;
        return ((qm / kM2) * 4 + tt) * kWpp + (qm % kM2) * 16;
    };
    uint4 held[kHeld][2];
    uint32_t xmax = 0;
    float xsum = 0.f;
    auto fold = [&](const uint4& v) {
        xmax = __vmaxu2(xmax, v.x & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.y & 0x7fff7fffu);
        xmax = __vmaxu2(xmax, v.z & 0x7fff7fffu); xmax = __vmaxu2(xmax, v.w & 0x7fff7fffu);
    };
    auto sum8 = [](const uint4& v) {
        return ((bf_lo(v.x) + bf_hi(v.x)) + (bf_lo(v.y) + bf_hi(v.y))) + ((bf_lo(v.z) + bf_hi(v.z)) + (bf_lo(v.w) + bf_hi(v.w)));
    };
#pragma unroll
    for (int j = 0; j < kHeld; ++j) {
        const int it = ctid + j * nthr;
        const int k0 = it < n_items ? k0_of(it) : K;
        held[j][0] = held[j][1] = make_uint4(0, 0, 0, 0);
        if (k0 < K) { held[j][0] = ld_x4(x + k0); held[j][1] = ld_x4(x + k0 + 8); }
    }
    // The fp32 sum of x is taken by the first kSumThreads threads in an order that does not depend on the number of
    // consumer warps, so a problem gives the same bits in every list and launch shape (the integer sums do anyway).
    if (ctid < kSumThreads)
        for (int it = ctid; it < n_items; it += kSumThreads) {
            const int k0 = k0_of(it);
            if (k0 < K) { xsum += sum8(ld_x4(x + k0)); xsum += sum8(ld_x4(x + k0 + 8)); }
        }
#pragma unroll
    for (int j = 0; j < kHeld; ++j) { fold(held[j][0]); fold(held[j][1]); }
    for (int it = ctid + kHeld * nthr; it < n_items; it += nthr) {       // rows too long to hold: read again below
        const int k0 = k0_of(it);
        if (k0 < K) { fold(ld_x4(x + k0)); fold(ld_x4(x + k0 + 8)); }
    }
    xmax = max(xmax & 0xffffu, xmax >> 16);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
        xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
    }
    if (lane == 0) { s_rmax[warp] = xmax; s_rsum[warp] = xsum; }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
    xmax = lane < W ? s_rmax[lane] : 0u;
    xsum = lane < kSumThreads / 32 ? s_rsum[lane] : 0.f;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        xmax = max(xmax, __shfl_xor_sync(0xffffffffu, xmax, o));
        xsum += __shfl_xor_sync(0xffffffffu, xsum, o);
    }
    xsum_out = xsum;
    const int xexp = min(max((int)(xmax >> 7), imma::kP + 1), 254);
    xexp_out = xexp;
    float mult[kF];
#pragma unroll
    for (int cls = 0; cls < kF; ++cls) mult[cls] = __uint_as_float((uint32_t)(254 + imma::kP - xexp - R * cls) << 23);
#pragma unroll
    for (int j = 0; j < kHeld; ++j) {
        const int it = ctid + j * nthr;
        if (it < n_items) {
            uint4* dst = xs + (size_t)(it >> 2) * imma::kBytes * 4 + (it & 3);
            if (k0_of(it) < K) {
                const uint32_t raw[8] = {held[j][0].x, held[j][0].y, held[j][0].z, held[j][0].w, held[j][1].x, held[j][1].y, held[j][1].z, held[j][1].w};
                stage_item<R>(raw, mult, dst);
            } else {
#pragma unroll
                for (int d = 0; d < imma::kBytes; ++d) dst[4 * d] = make_uint4(0, 0, 0, 0);
            }
        }
    }
    for (int it = ctid + kHeld * nthr; it < n_items; it += nthr) {
        uint4* dst = xs + (size_t)(it >> 2) * imma::kBytes * 4 + (it & 3);
        const int k0 = k0_of(it);
        if (k0 < K) {
            const uint4 va = ld_x4(x + k0), vb = ld_x4(x + k0 + 8);
            const uint32_t raw[8] = {va.x, va.y, va.z, va.w, vb.x, vb.y, vb.z, vb.w};
            stage_item<R>(raw, mult, dst);
        } else {
#pragma unroll
            for (int d = 0; d < imma::kBytes; ++d) dst[4 * d] = make_uint4(0, 0, 0, 0);
        }
    }
    asm volatile("bar.sync 1, %0;" ::"r"(nthr) : "memory");
}

// Finishes one tile.  Accumulator a_i of thread (g, t) holds row g + 8 (i >> 1), column 2t + (i & 1); the five
// columns of a row are recombined in 64 bits by the lanes t = 0 and scaled back once.  `scales`: alpha of row
// (lane) in lanes 0-15, zero of row (lane - 16) in lanes 16-31; `ep_rows`: the extra-precision sum of row (lane) in
// lanes 0-15 (zero without lists).  Called by whole warps.  Everything is passed by value: a structure would live in
// local memory, and its first load would cost a trip to the L2 per launch.
__device__ __noinline__ void finish_tile(float* __restrict__ y, int N, int sh, int xexp, float xsum, long long row0,
                                         int a0, int a1, int a2, int a3, float scales, float ep_rows, int lane, bool store) {
    const int g = lane >> 2, t = lane & 3;
#pragma unroll
    for (int h = 0; h < 2; ++h) {                               // rows g and g + 8
        const int d0 = h ? a2 : a0, d1 = h ? a3 : a1;
        const int d2 = __shfl_down_sync(0xffffffffu, d0, 1), d3 = __shfl_down_sync(0xffffffffu, d1, 1);
        const int d4 = __shfl_down_sync(0xffffffffu, d0, 2);
        const float al = __shfl_sync(0xffffffffu, scales, g + 8 * h), ze = __shfl_sync(0xffffffffu, scales, 16 + g + 8 * h);
        const float ep = __shfl_sync(0xffffffffu, ep_rows, g + 8 * h);
        const long long row = row0 + g + 8 * h;
        if (t != 0 || row >= N || !store) continue;
        // sum_i A_i Y_i = sum_d 256^d D_d - sum_i A_i 2^(P + 2 - R i), and column 4 holds sum_i A_i 2^(sh - R i)
        const long long tot = (((long long)d3 * 256 + d2) * 256 + d1) * 256 + d0 - ((long long)d4 << (imma::kP + 2 - sh));
        const float v = __ll2float_rn(tot) * __uint_as_float((uint32_t)(xexp - imma::kP) << 23) + ep;
        y[row] = al * (v * (float)(1 << sh) - ze * xsum);
    }
}

// ---------------------------------------------------------------------------------------------------------------
// Extra precision: y[n] = sum of x over the listed columns of row n, for every problem of a list that has lists.

struct EpProblem {
    const int32_t* row_ptr;
    const uint16_t* col;
    const __nv_bfloat16* x;
    float* y;
    int N, K;
    long long row0;           // rows of the problems before this one
};
template <int NP>
struct EpParams {
    EpProblem p[NP];
    long long rows;           // total rows
    int n;
    int pdl;
};
constexpr int kEpThreads = 512;

constexpr int kEpLongList = 512;     // lists longer than this are summed by the whole CTA
constexpr int kEpMaxLong = 128;      // such rows a CTA remembers per problem (more are summed by their eight lanes)

// Sum of x over list entries [e0, e1) taken with stride `step` from e0 + `first`: a fixed partition of the list over the
// lanes and over four partial sums per lane.  Lists that no slice_pack produced (entries >= K) are wrapped, not trusted.
__device__ __forceinline__ float ep_partial(const uint16_t* __restrict__ col, const __nv_bfloat16* xs, int K, int e0, int e1, int first, int step) {
    auto xat = [&](int c) { return __bfloat162float(xs[c < K ? c : c % K]); };
    float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
    int e = e0 + first;
    for (; e + 3 * step < e1; e += 4 * step) {
        const int c0 = col[e], c1 = col[e + step], c2 = col[e + 2 * step], c3 = col[e + 3 * step];
        s0 += xat(c0); s1 += xat(c1); s2 += xat(c2); s3 += xat(c3);
    }
    for (; e < e1; e += step) s0 += xat(col[e]);
    return (s0 + s1) + (s2 + s3);
}

template <int NP>
__global__ void __launch_bounds__(kEpThreads)
ep_rowsum(const __grid_constant__ EpParams<NP> P) {
    extern __shared__ __align__(16) unsigned char ep_smem[];
    __shared__ int s_long[kEpMaxLong];
    __shared__ int s_nlong;
    __shared__ float s_wsum[kEpThreads / 32];
    __nv_bfloat16* xs = reinterpret_cast<__nv_bfloat16*>(ep_smem);      // the problem's activations
    const int tid = threadIdx.x, sub = tid & 7, grp = tid >> 3;          // eight lanes per row, 2 x 64 rows per pass
    const unsigned gmask = 0xffu << (tid & 24);
    // x may be written by the previous kernel.  The persistent kernel behind this one is released only after that
    // wait: once it runs, x is final, so it may stage x and multiply while these sums are still being taken, and it
    // waits for this kernel only before it reads the first sum.
    if (P.pdl) asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;");
    const long long lo = P.rows * blockIdx.x / gridDim.x, hi = P.rows * (blockIdx.x + 1) / gridDim.x;
    int p_first = 0;
    {
        int a = 0, b = P.n - 1;                                           // last problem that starts at or before lo
        while (a < b) {
            const int m = (a + b + 1) >> 1;
            if (P.p[m].row0 <= lo) a = m; else b = m - 1;
        }
        p_first = a;
    }
    for (int p = p_first; p < P.n && P.p[p].row0 < hi; ++p) {           // only the problems this CTA's rows belong to
        const EpProblem& pr = P.p[p];
        const long long a = lo > pr.row0 ? lo - pr.row0 : 0;
        const long long b = hi - pr.row0 < pr.N ? hi - pr.row0 : pr.N;
        if (a >= b) continue;
        __syncthreads();                                                  // the previous problem's gathers are done
        if (tid == 0) s_nlong = 0;
        for (int i = tid; i < (pr.K >> 3); i += kEpThreads) reinterpret_cast<uint4*>(xs)[i] = ld_x4(pr.x + 8 * i);
        __syncthreads();
        // Two rows per group and pass.  What a pass costs is dependent round trips to the L2 / HBM, so they are kept to
        // one: the list bounds of the NEXT pass are requested before this pass's columns, and the first four columns of
        // each lane (32 entries of a row; most rows have fewer) are requested together for both rows, predicated, before
        // any is used.  A row lists at most K columns: row_ptr values that say otherwise are cut short, so that every
        // loop ends.
        auto bounds = [&](long long r, bool on, int& lo_e, int& hi_e) {
            lo_e = on ? max(pr.row_ptr[r], 0) : 0;
            hi_e = on ? min(pr.row_ptr[r + 1], lo_e + pr.K) : 0;
        };
        auto xat = [&](int c) { return c < 0 ? 0.f : __bfloat162float(xs[c < pr.K ? c : c % pr.K]); };
        constexpr int kStride = 2 * (kEpThreads / 8);
        int e0, e1, f0, f1;
        bounds(a + grp, a + grp < b, e0, e1);
        bounds(a + grp + kEpThreads / 8, a + grp + kEpThreads / 8 < b, f0, f1);
        for (long long row = a + grp; row < b; row += kStride) {
            const long long row2 = row + kEpThreads / 8;
            const bool two = row2 < b;
            int ne0, ne1, nf0, nf1;                                        // the next pass's lists
            bounds(row + kStride, row + kStride < b, ne0, ne1);
            bounds(row2 + kStride, row2 + kStride < b, nf0, nf1);
            const bool long_a = e1 - e0 > kEpLongList, long_b = f1 - f0 > kEpLongList;
            bool defer_a = false, defer_b = false;
            if (long_a || long_b) {                                       // remembered for the CTA-wide pass below
                int slot_a = kEpMaxLong, slot_b = kEpMaxLong;
                if (sub == 0) {
                    if (long_a) slot_a = atomicAdd(&s_nlong, 1);
                    if (long_b) slot_b = atomicAdd(&s_nlong, 1);
                    if (slot_a < kEpMaxLong) s_long[slot_a] = (int)(row - a);
                    if (slot_b < kEpMaxLong) s_long[slot_b] = (int)(row2 - a);
                }
                slot_a = __shfl_sync(gmask, slot_a, tid & 24);
                slot_b = __shfl_sync(gmask, slot_b, tid & 24);
                defer_a = long_a && slot_a < kEpMaxLong;
                defer_b = long_b && slot_b < kEpMaxLong;
            }
            const int ea = defer_a ? e0 : e1, eb = (!two || defer_b) ? f0 : f1;   // an empty range for rows not summed here
            int ca[4], cb[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                ca[j] = e0 + sub + 8 * j < ea ? (int)pr.col[e0 + sub + 8 * j] : -1;
                cb[j] = f0 + sub + 8 * j < eb ? (int)pr.col[f0 + sub + 8 * j] : -1;
            }
            float sa = (xat(ca[0]) + xat(ca[1])) + (xat(ca[2]) + xat(ca[3]));
            float sb = (xat(cb[0]) + xat(cb[1])) + (xat(cb[2]) + xat(cb[3]));
            if (ea - e0 > 32) sa += ep_partial(pr.col, xs, pr.K, e0 + 32, ea, sub, 8);
            if (eb - f0 > 32) sb += ep_partial(pr.col, xs, pr.K, f0 + 32, eb, sub, 8);
            sa += __shfl_xor_sync(gmask, sa, 4);  sb += __shfl_xor_sync(gmask, sb, 4);   // the eight lanes of this group only: the
            sa += __shfl_xor_sync(gmask, sa, 2);  sb += __shfl_xor_sync(gmask, sb, 2);   // other groups of the warp may already have
            sa += __shfl_xor_sync(gmask, sa, 1);  sb += __shfl_xor_sync(gmask, sb, 1);   // left the loop
            if (sub == 0) {
                if (!defer_a) pr.y[row] = sa;
                if (two && !defer_b) pr.y[row2] = sb;
            }
            e0 = ne0; e1 = ne1; f0 = nf0; f1 = nf1;
        }
        __syncthreads();
        // long lists (a row whose codes all sit in the extra bucket lists K columns): all threads on one row at a time
        const int n_long = min(s_nlong, kEpMaxLong);
        for (int i = 0; i < n_long; ++i) {
            const long long row = a + s_long[i];
            const int e0 = max(pr.row_ptr[row], 0), e1 = min(pr.row_ptr[row + 1], e0 + pr.K);
            float v = ep_partial(pr.col, xs, pr.K, e0, e1, tid, kEpThreads);
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
            if ((tid & 31) == 0) s_wsum[tid >> 5] = v;
            __syncthreads();
            if (tid == 0) {
                float t = 0.f;
                for (int w = 0; w < kEpThreads / 32; ++w) t += s_wsum[w];
                pr.y[row] = t;
            }
            __syncthreads();
        }
    }
}

// The producer warp of a CTA: lane l < W feeds consumer warp l's stages with the units of this CTA's share [lo, hi), in
// the order plan_of() defines.  Shared by the kernels that consume the ring.
template <int NP>
__device__ __forceinline__ void producer_warp(const Params<NP>& P, long long lo, long long hi, int p_first, int W, unsigned char* ring,
                                              uint64_t* s_full, uint64_t* s_empty, volatile int* abort_flag, int lane) {
    // ------------------------------------------------------------------ producer warp: lane l < W feeds warp l's stages
    int it0 = 0;                                          // units of the segments before this one (a multiple of W)
    bool waited = P.pdl != 1;
    int p = p_first, t_lo, t_hi, tail_lo = -1, tail_hi = 0;
    bool ok = true;
    int last_it = -1;                                     // latest unit this lane issued a copy for
    while (ok && !P.hold && next_segment(P, lo, hi, p, t_lo, t_hi, tail_lo, tail_hi)) {
        const Problem& pr = P.p[p - 1];
        const Geo G = geometry(pr.N, pr.K, pr.r, P.unit_row, P.pairs);
        const int T = t_hi - t_lo;
        const Plan pl = plan_of(G, T, W);
        // Lane l feeds warp l: its units are l, l + W, ...; (tile, panel) and (stage, phase) move by fixed steps.  The
        // lanes advance independently: each probes ITS stage (without suspending) and issues its next copy as soon as
        // its warp has released the stage, so a slow consumer warp never holds back the copies of the others.
        const int step_t = pl.split ? W / G.n_panels : 0, step_p = pl.split ? W % G.n_panels : 0;
        int tj = pl.split ? lane / G.n_panels * pl.tpu : lane * pl.tpu;      // first tile of the unit, relative to t_lo
        int pn = pl.split ? lane % G.n_panels : 0;
        int slot = (it0 + lane) % P.slots;
        int use = (it0 + lane) / P.slots;                      // how often the stage has been used before
        int s = lane < W ? lane : pl.n_units;                  // this lane's next unit
        long long t_wait = 0;
        int spins = 0;
        while (__any_sync(0xffffffffu, s < pl.n_units)) {
            if (!waited && __any_sync(0xffffffffu, s < pl.n_units && use > 0)) {
                // The consumers only start after the previous kernel of the stream has finished; wait for it here
                // (a wait the stream itself bounds), so that the bounded waits below measure this CTA only.
                asm volatile("griddepcontrol.wait;" ::: "memory");
                waited = true;
            }
            bool progressed = false;
            if (s < pl.n_units && (use == 0 || mbar_test_wait(smem_u32(&s_empty[slot]), (uint32_t)((use - 1) & 1)))) {
                const uint32_t bar = smem_u32(&s_full[slot]);
                const uint32_t dst = smem_u32(ring + (size_t)slot * P.slot_bytes);
                if (tj >= T) {
                    mbar_arrive(bar);                           // padding: an empty unit
                } else if (G.contig) {
                    // the unit is one run of the plane; rows past the end of the matrix are not fetched
                    const long long row0 = (long long)(t_lo + tj) * 16;
                    const long long rows = min((long long)min(pl.tpu, T - tj) * 16, pr.N - row0);
                    const uint32_t bytes = (uint32_t)rows * (uint32_t)G.row_bytes;
                    mbar_arrive_expect_tx(bar, bytes);
                    bulk_g2s(dst, pr.packed + row0 * G.row_bytes, bytes, bar);
                    last_it = it0 + s;
                } else {
                    mbar_arrive_expect_tx(bar, (uint32_t)(16 * G.tpu * G.stride));     // the whole box, zeros included
                    tensor_g2s(dst, &P.tm[p - 1], pn * G.panel_qc * 8, (t_lo + tj) * 16, bar);
                    last_it = it0 + s;
                }
                if (pl.split) {
                    tj += step_t * pl.tpu; pn += step_p;
                    if (pn >= G.n_panels) { pn -= G.n_panels; tj += pl.tpu; }
                } else if (++pn == G.n_panels) { pn = 0; tj += W * pl.tpu; }
                slot += W;
                if (slot >= P.slots) { slot -= P.slots; ++use; }
                s += W;
                progressed = true;
            }
            // bounded: no lane made progress for the wait limit
            if (__any_sync(0xffffffffu, progressed)) { spins = 0; t_wait = 0; }
            else {
                __nanosleep(kProducerNapNs);                      // every stage is full: leave the issue slots to the multiplying warps
                if (++spins >= 64) {
                    spins = 0;
                    const long long now = clock64();
                    if (t_wait == 0) t_wait = now;
                    const bool give_up = *abort_flag || now - t_wait > P.wait_cycles;
                    if (__any_sync(0xffffffffu, give_up)) { *abort_flag = 1; ok = false; break; }
                }
            }
        }
        it0 += pl.n_units;
    }
    if (!ok && lane < W) {
        // gave up: copies already issued still write into this CTA's shared memory; wait for them (bounded).  A lane's
        // stages are its own, so the phase of a stage's latest use stays complete once its copy has landed.
        const long long t0 = clock64();
        for (int it = last_it; it >= 0 && it > last_it - P.slots; it -= W) {
            const uint32_t bar = smem_u32(&s_full[it % P.slots]);
            while (!mbar_try_wait(bar, (uint32_t)((it / P.slots) & 1), 1000) && clock64() - t0 < P.wait_cycles) {}
        }
    }
}

// RF: 0 = the problems of the list may differ in r; 8, 4, 2 = they are all at that precision, and only that precision's
// code is compiled into the variant.  The kernel is sensitive to its size (the warps of a CTA are at different places of
// it, "no instruction" is its most frequent stall): a variant per precision is 3-6 % faster than the one that holds all
// three.  The r = 2 variant uses pair units (geometry with pairs = 1): two tiles are multiplied per pass with one load
// of the activation fragments.  LISTS: whether any problem has extra-precision lists (the code that reads ep_rowsum's
// sums is compiled in only then).
template <int NP, int RF, bool LISTS>
__global__ void __launch_bounds__((kMaxW + 1) * 32, 1)
gemv_stream(const __grid_constant__ Params<NP> P) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    __shared__ __align__(8) uint64_t s_full[kMaxSlots], s_empty[kMaxSlots];
    __shared__ int s_tile[kTileSlots][2][16][imma::kCols];    // sums of tiles (pairs of tiles) whose panels are spread over warps
    __shared__ int s_tile_cnt[kTileSlots];
    __shared__ uint32_t s_rmax[kMaxW];
    __shared__ float s_rsum[kMaxW];
    __shared__ int s_abort;

    const int W = P.W;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nthr = W * 32;                                  // consumer threads
    uint4* xs = reinterpret_cast<uint4*>(smem_raw);
    unsigned char* ring = smem_raw + P.xs_bytes;
    volatile int* abort_flag = &s_abort;

    if (tid == 0) s_abort = 0;
    if (tid < P.slots) {
        mbar_init(smem_u32(&s_full[tid]), 1);
        mbar_init(smem_u32(&s_empty[tid]), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    for (int i = tid; i < kTileSlots * 2 * 16 * imma::kCols; i += blockDim.x) (&s_tile[0][0][0][0])[i] = 0;
    if (tid < kTileSlots) s_tile_cnt[tid] = 0;
    __syncthreads();
    if (P.pdl) asm volatile("griddepcontrol.launch_dependents;");

    // this CTA's share of the list: items [lo, hi), cut at tile boundaries (a tile belongs to the CTA its first item falls to)
    const long long lo = P.items * blockIdx.x / gridDim.x, hi = P.items * (blockIdx.x + 1) / gridDim.x;
    int p_first = 0;
    {
        int a = 0, b = P.n - 1;                               // last problem that starts at or before lo
        while (a < b) {
            const int m = (a + b + 1) >> 1;
            if (P.p[m].item0 <= lo) a = m; else b = m - 1;
        }
        p_first = a;
    }

    if (warp == W) {
        producer_warp(P, lo, hi, p_first, W, ring, s_full, s_empty, abort_flag, lane);
    } else {
        // ------------------------------------------------------------------ consumer warps
        const int g = lane >> 2, t = lane & 3;
        const int ctid = tid;                                  // warps 0 .. W-1
        int it0 = 0;                                           // units of the segments before this one (a multiple of W)
        int split_tiles = 0;                                   // split-mode tiles of earlier segments (a tile's slot = its count mod kTileSlots)
        int p = p_first, t_lo, t_hi, tail_lo = -1, tail_hi = 0, staged_p = -1;
        bool first = true;
        bool ep_ready = P.pdl != 2;                            // whether ep_rowsum's sums may be read yet
        Geo G;
        float xsum = 0.f;
        int xexp = 0;
        while (next_segment(P, lo, hi, p, t_lo, t_hi, tail_lo, tail_hi)) {
            const Problem& pr = P.p[p - 1];
            G = geometry(pr.N, pr.K, pr.r, P.unit_row, P.pairs);
            const int R = RF ? RF : pr.r;
            const int sh = kCodeBits - R;
            const int T = t_hi - t_lo;
            const Plan pl = plan_of(G, T, W);
            // alpha and zero of this warp's first tiles do not depend on the previous kernel: requested before anything else
            const int tpu0 = pl.tpu;
            float sc_first[kMaxTpu];
#pragma unroll
            for (int k = 0; k < kMaxTpu; ++k) {
                const int tn = pl.split ? warp / G.n_panels * tpu0 : warp * tpu0 + k;      // split mode: the first tile of the warp's first unit
                const long long row = (long long)(t_lo + tn) * 16 + (lane & 15);
                sc_first[k] = (k < tpu0 && tn < T && row < pr.N) ? (lane < 16 ? pr.alpha[row] : pr.zero[row]) : 0.f;
            }
            if (first) {
                // The activations may still be written by the previous kernel, so they are only READ after the dependency
                // wait; pulling their lines into the L2 earlier is harmless (the L2 is the point of coherence) and takes the
                // HBM latency of a cold vector off the critical path.
                for (int i = ctid * 64; i < pr.K; i += nthr * 64) asm volatile("prefetch.global.L2 [%0];" ::"l"(pr.x + i));
                if (P.pdl == 1) asm volatile("griddepcontrol.wait;" ::: "memory");
            }
            first = false;

            // ---- the activations of this problem as byte units in fragment order (all consumer warps together)
            // (the second segment of a problem finds them staged)
            if (staged_p == p) {}
            else if (R == 8) stage_activations<8>(pr.x, pr.K, G.n_qc, xs, ctid, nthr, W, s_rmax, s_rsum, xsum, xexp);
            else if (R == 4) stage_activations<4>(pr.x, pr.K, G.n_qc, xs, ctid, nthr, W, s_rmax, s_rsum, xsum, xexp);
            else stage_activations<2>(pr.x, pr.K, G.n_qc, xs, ctid, nthr, W, s_rmax, s_rsum, xsum, xexp);
            staged_p = p;

            const int kM2 = (128 / R) / 16;
            // this lane's B source: chunk q of byte column g starts at xs[q * kM2 * 16 + g * 4 + t]; the lanes g = 4 hold
            // the constant column (2^(smax - s) per byte, see gemv_imma.cuh) in registers
            const int col_lane = g < imma::kBytes ? 1 : 0;
            const uint32_t x_sa0 = smem_u32(xs) + (uint32_t)((g & 3) * 4 + t) * 16u;
            const int xq_bytes = kM2 * 256;
            uint4 cz = make_uint4(0, 0, 0, 0);
            if (g == imma::kBytes) {
                if (R == 8) cz = make_uint4(imma::ones_b0<8>(0), imma::ones_b1<8>(0), imma::ones_b0<8>(1), imma::ones_b1<8>(1));
                else if (R == 4) cz = make_uint4(imma::ones_b0<4>(0), imma::ones_b1<4>(0), imma::ones_b0<4>(1), imma::ones_b1<4>(1));
                else cz = make_uint4(imma::ones_b0<2>(0), imma::ones_b1<2>(0), imma::ones_b0<2>(1), imma::ones_b1<2>(1));
            }
            const bool half_tail = R == 2 && (G.row_bytes & 63) != 0;   // r = 2, K % 256 == 128: the last chunk is half full

            // panel `pn` of the tile whose rows start at `tile_rows` in a stage
            auto multiply = [&](const unsigned char* tile_rows, int pn, int (&acc)[kSets][4]) {
                const int q0 = pn * G.panel_qc, q1 = min(q0 + G.panel_qc, G.n_qc);
                const unsigned char* base = tile_rows + t * 16;
                const unsigned char* wl_p = base + (size_t)g * G.stride;
                const unsigned char* wh_p = base + (size_t)(g + 8) * G.stride;
                const uint32_t x_sa = x_sa0 + (uint32_t)(q0 * xq_bytes);
                int n_chunks = q1 - q0;
                const bool tail = half_tail && q1 == G.n_qc;
                if (tail) --n_chunks;
                if (R == 8) multiply_unit<8>(wl_p, wh_p, x_sa, xq_bytes, col_lane, cz, n_chunks, acc);
                else if (R == 4) multiply_unit<4>(wl_p, wh_p, x_sa, xq_bytes, col_lane, cz, n_chunks, acc);
                else multiply_unit<2>(wl_p, wh_p, x_sa, xq_bytes, col_lane, cz, n_chunks, acc);
                if (tail) {
                    // the pieces t >= 2 of the half-full chunk lie past the end of the row: their activation bytes
                    // were staged as zeros, and the constant column must be zero for them too
                    uint4 xt[4];
#pragma unroll
                    for (int m2 = 0; m2 < 4; ++m2) xt[m2] = t < 2 ? cz : make_uint4(0, 0, 0, 0);
                    multiply_item<2, 0>(wl_p + n_chunks * 64, wh_p + n_chunks * 64, x_sa + (uint32_t)(n_chunks * xq_bytes), col_lane, xt, acc);
                }
            };
            // two tiles of a unit per pass (see multiply_two_tiles); not with a half-full last chunk
            const bool pair_tiles = RF == 2 && kPairs && !half_tail;
            auto multiply2 = [&](const unsigned char* tile_rows, int pn, int (&acc)[kSets][4]) {
                const int q0 = pn * G.panel_qc, q1 = min(q0 + G.panel_qc, G.n_qc);
                const unsigned char* base = tile_rows + t * 16;
                const unsigned char* wl_p = base + (size_t)g * G.stride;
                const unsigned char* wh_p = base + (size_t)(g + 8) * G.stride;
                const uint32_t x_sa = x_sa0 + (uint32_t)(q0 * xq_bytes);
                multiply_two_tiles<2>(wl_p, wh_p, 16 * G.stride, x_sa, xq_bytes, col_lane, cz, q1 - q0, acc);
            };
            auto zero_acc = [&](int (&acc)[kSets][4]) {
#pragma unroll
                for (int c2 = 0; c2 < kSets; ++c2)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[c2][i] = 0;
            };
            // after a pass over two tiles: tile 0's sets summed into acc[0], tile 1's into acc[4]
            auto fold_two = [&](int (&acc)[kSets][4]) {
#pragma unroll
                for (int c2 = 1; c2 < 4; ++c2)
#pragma unroll
                    for (int i = 0; i < 4; ++i) { acc[0][i] += acc[c2][i]; acc[4][i] += acc[4 + c2][i]; }
            };
            auto fold = [&](int (&acc)[kSets][4]) {
#pragma unroll
                for (int c2 = 1; c2 < kSets; ++c2)
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[0][i] += acc[c2][i];
            };
            // alpha (lanes 0-15) and zero (lanes 16-31) of the 16 rows of a tile
            auto load_scales = [&](long long row0) -> float {
                const long long row = row0 + (lane & 15);
                if (row >= pr.N) return 0.f;
                return lane < 16 ? pr.alpha[row] : pr.zero[row];
            };

            // ---- this warp's units, in order.  One call site for the multiply and one for the finish keep the loop small
            // enough for the instruction cache (warps are at different places of it most of the time).
            int acc[kSets][4];
            const int contributors = min(G.n_panels, W);              // split mode: warps that hold a part of a tile
            int cur = -1;                                              // split mode: tile whose partial sums are in `acc`
            float sc[kMaxTpu], sc_next[kMaxTpu];
            float epv[kMaxTpu], epv_next[kMaxTpu];                    // extra precision: the sparse term of a tile's rows (lanes 0-15)
            const bool ep = LISTS && pr.ovf_row_ptr != nullptr;          // LISTS: some problem of the list has extra-precision lists
            // The sparse term is left in y by ep_rowsum (plain coherent loads).  Behind that kernel (pdl == 2) this one
            // starts before the sums are complete: it waits for them when it first needs one, and until then the loads a
            // round ahead are skipped (`epv_ok` / `epv_next_ok`: whether the registers hold loaded values).
            auto load_ep = [&](long long row0) -> float {
                const long long row = row0 + lane;
                float v = 0.f;
                if (lane < 16 && row < pr.N) asm volatile("ld.global.f32 %0, [%1];" : "=f"(v) : "l"(pr.y + row) : "memory");
                return v;
            };
            bool epv_ok = false, epv_next_ok = ep_ready;
#pragma unroll
            for (int k = 0; k < kMaxTpu; ++k) {
                sc[k] = 0.f; sc_next[k] = sc_first[k];                      // tile mode: the first unit's tiles
                epv[k] = 0.f;
                const int tn = warp * pl.tpu + k;
                epv_next[k] = (ep && ep_ready && !pl.split && k < pl.tpu && tn < T) ? load_ep((long long)(t_lo + tn) * 16) : 0.f;
            }
            auto await_ep = [&]() {
                if (!ep_ready) {
                    asm volatile("griddepcontrol.wait;" ::: "memory");
                    ep_ready = true;
                }
            };
            // split mode: the partial sums of tile `cur` go to its accumulator in shared memory; the warp that brings the
            // last of a tile's contributions finishes it (returns true for that warp, with the sums in acc[0])
            auto flush = [&]() -> bool {
                const bool both = pair_tiles && min(pl.tpu, T - cur) >= 2;      // the unit held two tiles: sums in sets 0-3 and 4-7
                if (both) fold_two(acc); else fold(acc);
                const int ts = (split_tiles + cur / pl.tpu) % kTileSlots;
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
                    if (tile == 1 && !both) break;
                    if (t < 3) {
                        atomicAdd(&s_tile[ts][tile][g][2 * t], acc[4 * tile][0]);
                        atomicAdd(&s_tile[ts][tile][g + 8][2 * t], acc[4 * tile][2]);
                        if (t < 2) { atomicAdd(&s_tile[ts][tile][g][2 * t + 1], acc[4 * tile][1]); atomicAdd(&s_tile[ts][tile][g + 8][2 * t + 1], acc[4 * tile][3]); }
                    }
                }
                __threadfence_block();
                __syncwarp();
                int prev = 0;
                if (lane == 0) prev = atomicAdd(&s_tile_cnt[ts], 1);
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev != contributors - 1) return false;
                __threadfence_block();                                 // last to arrive: every other contribution is visible
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) acc[4 * tile][i] = 0;
                    if (tile == 1 && !both) break;
                    if (t < 3) {
                        acc[4 * tile][0] = s_tile[ts][tile][g][2 * t];      acc[4 * tile][2] = s_tile[ts][tile][g + 8][2 * t];
                        if (t < 2) { acc[4 * tile][1] = s_tile[ts][tile][g][2 * t + 1];  acc[4 * tile][3] = s_tile[ts][tile][g + 8][2 * t + 1]; }
                    }
                }
                __syncwarp();
#pragma unroll
                for (int tile = 0; tile < 2; ++tile) {                 // leave the slot clean for the tiles that reuse it
                    if (tile == 1 && !both) break;
                    if (t < 3) {
                        s_tile[ts][tile][g][2 * t] = 0;  s_tile[ts][tile][g + 8][2 * t] = 0;
                        if (t < 2) { s_tile[ts][tile][g][2 * t + 1] = 0;  s_tile[ts][tile][g + 8][2 * t + 1] = 0; }
                    }
                }
                if (lane == 0) s_tile_cnt[ts] = 0;
                return true;
            };
            // unit s = warp, warp + W, ... without divisions in the loop: (tile, panel) and (stage, phase) move by fixed steps
            const int step_t = pl.split ? W / G.n_panels : 0, step_p = pl.split ? W % G.n_panels : 0;
            int tj = pl.split ? warp / G.n_panels * pl.tpu : warp * pl.tpu;   // first tile of the unit (relative to t_lo)
            int pn = pl.split ? warp % G.n_panels : 0;                    // its panel
            int slot = (it0 + warp) % P.slots;
            uint32_t parity = (uint32_t)(((it0 + warp) / P.slots) & 1);
            // split mode: the warp that completes a tile finishes it
            auto finish_split = [&](long long row0, float scales) {
                if (ep) await_ep();
                const float ep_rows = ep ? load_ep(row0) : 0.f;
                finish_tile(pr.y, pr.N, sh, xexp, xsum, row0, acc[0][0], acc[0][1], acc[0][2], acc[0][3], scales, ep_rows, lane, !*abort_flag);
                if (pair_tiles && min(pl.tpu, T - cur) >= 2) {             // the second tile of the pair
                    const float ep2 = ep ? load_ep(row0 + 16) : 0.f;
                    finish_tile(pr.y, pr.N, sh, xexp, xsum, row0 + 16, acc[4][0], acc[4][1], acc[4][2], acc[4][3], load_scales(row0 + 16), ep2, lane, !*abort_flag);
                }
            };
            for (int s = warp; s < pl.n_units; s += W) {
                const int n_tiles = tj < T ? min(pl.tpu, T - tj) : 0;     // 0: an empty unit (padding)
                if (pl.split) {
                    if (n_tiles && tj != cur) {
                        if (cur >= 0 && flush()) finish_split((long long)(t_lo + cur) * 16, sc[0]);
                        cur = tj;
                        sc[0] = s == warp ? sc_first[0] : load_scales((long long)(t_lo + tj) * 16);     // the first one was requested early
                        zero_acc(acc);
                    }
                } else if (pn == 0) {
#pragma unroll
                    for (int k = 0; k < kMaxTpu; ++k) {
                        sc[k] = sc_next[k];
                        epv[k] = epv_next[k];
                        const int tn = tj + W * pl.tpu + k;                  // the same warp's next group of tiles, a round ahead
                        if (k < pl.tpu && tn < T) {
                            sc_next[k] = load_scales((long long)(t_lo + tn) * 16);
                            if (ep && ep_ready) epv_next[k] = load_ep((long long)(t_lo + tn) * 16);
                        }
                    }
                    epv_ok = epv_next_ok;
                    epv_next_ok = ep_ready;
                    zero_acc(acc);
                }
                const bool landed = wait_phase(smem_u32(&s_full[slot]), parity, abort_flag, P.wait_cycles);
                const unsigned char* rows = ring + (size_t)slot * P.slot_bytes;
                const bool tile_done = !pl.split && pn == G.n_panels - 1;
                for (int k = 0; k < n_tiles; ++k) {
                    const bool two = pair_tiles && k + 1 < n_tiles;       // this tile and the next in one pass
                    if (k > 0) zero_acc(acc);
                    if (landed) {
                        if (two) multiply2(rows + (size_t)k * 16 * G.stride, pn, acc);
                        else multiply(rows + (size_t)k * 16 * G.stride, pn, acc);
                    }
                    if (k + (two ? 1 : 0) == n_tiles - 1) {               // the last read of the stage is done
                        __syncwarp();
                        if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
                    }
                    if (tile_done) {
                        if (two) fold_two(acc); else fold(acc);
                        if (ep && !epv_ok) {                                  // not loaded a round ahead: wait for the sums, load them now
                            await_ep();
#pragma unroll
                            for (int kk = 0; kk < kMaxTpu; ++kk)
                                if (kk < n_tiles) epv[kk] = load_ep((long long)(t_lo + tj + kk) * 16);
                            epv_ok = true;
                        }
                        finish_tile(pr.y, pr.N, sh, xexp, xsum, (long long)(t_lo + tj + k) * 16, acc[0][0], acc[0][1], acc[0][2], acc[0][3],
                                    k == 0 ? sc[0] : k == 1 ? sc[1] : k == 2 ? sc[2] : sc[3],
                                    k == 0 ? epv[0] : k == 1 ? epv[1] : k == 2 ? epv[2] : epv[3], lane, !*abort_flag);
                        if (two)
                            finish_tile(pr.y, pr.N, sh, xexp, xsum, (long long)(t_lo + tj + k + 1) * 16, acc[4][0], acc[4][1], acc[4][2], acc[4][3],
                                        k == 0 ? sc[1] : sc[3], k == 0 ? epv[1] : epv[3], lane, !*abort_flag);
                    }
                    if (two) ++k;                                         // the pass covered the next tile too
                }
                if (n_tiles == 0) {
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&s_empty[slot]));
                }
                // next unit of this warp
                if (pl.split) {
                    tj += step_t * pl.tpu; pn += step_p;
                    if (pn >= G.n_panels) { pn -= G.n_panels; tj += pl.tpu; }
                } else if (++pn == G.n_panels) { pn = 0; tj += W * pl.tpu; }
                slot += W;
                if (slot >= P.slots) { slot -= P.slots; parity ^= 1u; }
            }
            if (pl.split) {
                if (cur >= 0 && flush()) finish_split((long long)(t_lo + cur) * 16, sc[0]);
                split_tiles += (T + pl.tpu - 1) / pl.tpu;
            }
            it0 += pl.n_units;
        }
    }
    __syncthreads();
    if (tid == 0 && s_abort) report(P.dev_status, MATQ_ERR_TIMEOUT);
}

// ---------------------------------------------------------------------------------------------------------------
// Host side

struct HostProblem {
    const uint8_t* packed;
    int64_t N, K;
    int r;
    const float* alpha;
    const float* zero;
    const int32_t* ovf_row_ptr;
    const uint16_t* ovf_col;
    const void* x;
    float* y;
    int64_t B;
};

inline size_t xs_bytes_of(const Geo& g, int r) { return (size_t)g.n_qc * ((128 / r) / 16) * 256; }
inline int slot_bytes_of(const Geo& g) { return (16 * g.tpu * g.stride + 64 + 127) / 128 * 128; }   // a half-full last chunk is read 32 bytes past its row

// Consumer warps for a list whose largest problem stages `xs_bytes` of activations and needs `slot_bytes` per stage:
// as many as have a stage each (at most kMaxW); fewer than kMinW means the list does not fit this kernel.
constexpr int kMinW = 4;
inline int warps_for(size_t xs_bytes, int slot_bytes) {
    const long long fit = ((long long)kSmemLimit - kStaticReserve - (long long)xs_bytes) / slot_bytes;
    return (int)std::min<long long>(kMaxW, fit);
}

// W warps, or W - 1 when that puts more stages to use (the number of stages is a multiple of the number of warps: 14
// instead of 8, say): bytes in flight matter more than the last warp.  Fewer warps still were measured: five with two
// stages each win on K = 9216 at r = 8 and 4 and lose everywhere else.
inline int pick_warps(int W, int fit) {
    return (W > kMinW && fit / (W - 1) * (W - 1) > fit / W * W) ? W - 1 : W;
}

// Whether a problem can take this path at all (B = 1 is implied).
inline bool eligible(int64_t N, int64_t K, int r) {
    if (!(r == 8 || r == 4 || r == 2) || K % 128 != 0 || K > imma::kMaxK || N <= 0 || N >= (1ll << 31) - 16) return false;
    const Geo g = geometry((int)N, (int)K, r, kUnitRow);
    return warps_for(xs_bytes_of(g, r), slot_bytes_of(g)) >= kMinW;
}

// Tensor map over a plane as [N][row_bytes / 8] 64-bit words with a box of 16 tpu rows x one panel.
inline bool make_plane_map(CUtensorMap* tm, const uint8_t* packed, int64_t N, const Geo& g) {
    t5::EncodeTiledFn fn = t5::encode_fn();
    if (!fn) return false;
    const cuuint64_t dims[2] = {(cuuint64_t)(g.row_bytes / 8), (cuuint64_t)N};
    const cuuint64_t strides[1] = {(cuuint64_t)g.row_bytes};
    const cuuint32_t box[2] = {(cuuint32_t)(g.stride / 8), (cuuint32_t)(16 * g.tpu)};
    const cuuint32_t estr[2] = {1u, 1u};
    return fn(tm, CU_TENSOR_MAP_DATA_TYPE_UINT64, 2, const_cast<uint8_t*>(packed), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int NP>
inline int launch_list(const HostProblem* hp, int n, bool pdl, long long wait_cycles, bool hold, int32_t* dev_status, cudaStream_t s) {
    static std::atomic<unsigned long long> smem_ok[8] = {};
    Params<NP> P;
    // the precision the whole list is at (0: mixed) selects the kernel variant; lists at r = 2 get pair units
    int rf = -1;
    for (int i = 0; i < n; ++i)
        if (hp[i].N != 0) rf = rf < 0 ? hp[i].r : (rf == hp[i].r ? rf : 0);
    if (rf < 0) rf = 0;
    const int pairs = (rf == 2) ? kPairs : 0;
    long long items = 0, tiles = 0;
    for (int i = 0; i < n; ++i) {
        if (hp[i].N == 0) continue;
        if (!eligible(hp[i].N, hp[i].K, hp[i].r)) return MATQ_ERR_SHAPE;
        const Geo g = geometry((int)hp[i].N, (int)hp[i].K, hp[i].r, kUnitRow, pairs);
        items += (long long)g.tiles * tile_cost(g, hp[i].r);
        tiles += g.tiles;
    }
    if (tiles == 0) return MATQ_OK;
    const int sms = sm_count();
    const int grid = (int)std::min<long long>(sms, tiles);
    const int unit_row = kUnitRow;
    size_t xs_bytes = 0;
    int slot_bytes = 0;
    int m = 0;
    long long item0 = 0;
    for (int i = 0; i < n; ++i) {
        if (hp[i].N == 0) continue;
        Problem& q = P.p[m];
        q.packed = hp[i].packed; q.alpha = hp[i].alpha; q.zero = hp[i].zero;
        q.ovf_row_ptr = hp[i].ovf_row_ptr; q.ovf_col = hp[i].ovf_col;
        q.x = static_cast<const __nv_bfloat16*>(hp[i].x); q.y = hp[i].y;
        q.N = (int)hp[i].N; q.K = (int)hp[i].K; q.r = hp[i].r; q.B = 1;
        q.item0 = item0;
        const Geo g = geometry(q.N, q.K, q.r, unit_row, pairs);
        if (!g.contig && !make_plane_map(&P.tm[m], q.packed, q.N, g)) return MATQ_ERR_CUDA;
        item0 += (long long)g.tiles * tile_cost(g, q.r);
        xs_bytes = std::max(xs_bytes, xs_bytes_of(g, q.r));
        slot_bytes = std::max(slot_bytes, slot_bytes_of(g));
        ++m;
    }
    for (int i = m; i < NP; ++i) P.p[i] = Problem{};
    int W = std::min(warps_for(xs_bytes, slot_bytes), items / grid >= 16ll * kManyItems ? kMaxW : kFewW);
    if (W < kMinW) return MATQ_ERR_SHAPE;
    const int fit = std::min((int)((kSmemLimit - kStaticReserve - xs_bytes) / slot_bytes), kMaxSlots);
    // The number of stages is a multiple of W: a stage always serves the same warp.
    W = pick_warps(W, fit);
    const int slots = fit / W * W;
    bool behind_ep = false;
    // Extra precision: the sparse term of every problem with lists goes to its y first (see ep_rowsum); the persistent
    // kernel then runs as that kernel's programmatic dependent (it touches y only after its dependency wait).
    {
        static std::atomic<unsigned long long> ep_smem_ok{0};
        EpParams<NP> E;
        long long rows = 0;
        int me = 0, k_max = 0;
        for (int i = 0; i < m; ++i) {
            const Problem& q = P.p[i];
            if (!q.ovf_row_ptr) continue;
            E.p[me++] = EpProblem{q.ovf_row_ptr, q.ovf_col, q.x, q.y, q.N, q.K, rows};
            rows += q.N;
            k_max = std::max(k_max, q.K);
        }
        if (me > 0) {
            for (int i = me; i < NP; ++i) E.p[i] = EpProblem{};
            E.rows = rows; E.n = me; E.pdl = pdl ? 1 : 0;
            auto ek = ep_rowsum<NP>;
            if (!opt_in_max_smem(ek, ep_smem_ok)) return MATQ_ERR_CUDA;
            cudaLaunchConfig_t ec = {};
            int per_sm = 0;                                  // one wave: as many CTAs as are resident together
            if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, ek, kEpThreads, (size_t)2 * k_max) != cudaSuccess || per_sm < 1) per_sm = 1;
            ec.gridDim = dim3((unsigned)std::max<long long>(1, std::min<long long>((long long)per_sm * sms, (rows + 63) / 64)));
            ec.blockDim = dim3(kEpThreads);
            ec.dynamicSmemBytes = (size_t)2 * k_max;
            ec.stream = s;
            cudaLaunchAttribute ea[1];
            ea[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            ea[0].val.programmaticStreamSerializationAllowed = 1;
            ec.attrs = ea;
            ec.numAttrs = pdl ? 1 : 0;
            if (cudaLaunchKernelEx(&ec, ek, E) != cudaSuccess) { cudaGetLastError(); return MATQ_ERR_CUDA; }
            pdl = true;
            behind_ep = true;
        }
    }
    P.items = items; P.wait_cycles = wait_cycles; P.dev_status = dev_status; P.n = m; P.slots = slots; P.slot_bytes = slot_bytes;
    P.xs_bytes = (int)xs_bytes; P.W = W; P.pdl = behind_ep ? 2 : pdl ? 1 : 0; P.unit_row = unit_row; P.hold = hold ? 1 : 0;
    P.pairs = pairs;
    P.tails = 1;
    auto kern = behind_ep ? (rf == 8 ? gemv_stream<NP, 8, true> : rf == 4 ? gemv_stream<NP, 4, true> : rf == 2 ? gemv_stream<NP, 2, true> : gemv_stream<NP, 0, true>)
                          : (rf == 8 ? gemv_stream<NP, 8, false> : rf == 4 ? gemv_stream<NP, 4, false> : rf == 2 ? gemv_stream<NP, 2, false> : gemv_stream<NP, 0, false>);
    if (!opt_in_max_smem(kern, smem_ok[(behind_ep ? 4 : 0) + (rf == 8 ? 3 : rf == 4 ? 2 : rf == 2 ? 1 : 0)])) return MATQ_ERR_CUDA;
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

// A list longer than one launch's descriptor table is served by several launches.
inline int launch(const HostProblem* hp, int n, bool pdl, long long wait_cycles, bool hold, int32_t* dev_status, cudaStream_t s) {
    for (int i = 0; i < n; ++i)
        if (hp[i].N != 0 && !eligible(hp[i].N, hp[i].K, hp[i].r)) return MATQ_ERR_SHAPE;      // before anything is launched
    if (n <= kSmallList) return launch_list<kSmallList>(hp, n, pdl, wait_cycles, hold, dev_status, s);
    for (int i = 0; i < n; i += kLargeList) {
        const int st = launch_list<kLargeList>(hp + i, std::min(kLargeList, n - i), pdl, wait_cycles, hold, dev_status, s);
        if (st != MATQ_OK) return st;
    }
    return MATQ_OK;
}

}  // namespace gstream
}  // namespace matq
