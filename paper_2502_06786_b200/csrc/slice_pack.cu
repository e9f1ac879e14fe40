// matq_slice_pack: MSB slicing S(q, r) (Eq. 6), the un-clamped variant of the
// Errata (Eq. 8) as a sparse overflow list, and packing into r-bit planes.
//
// The pass is pure integer work bound by HBM: 1 byte read and r/8 bytes written
// per weight.  Four codes are sliced at once inside a 32-bit register:
//   a = (w >> sh) & fieldmask        top r bits of every byte
//   b = (w >> (sh-1)) & 0x01010101   the (r+1)-th most significant bit (Appendix A's rounding bit)
//   s = a + b                        <= 2^r per byte, never carries across bytes
//   ov = (s >> r) & 0x01010101       1 where rounding overflowed into bucket 2^r
//   k = s - ov                       the clamp of Eq. 6
// `ov` is exactly the extra bucket Eq. 8 keeps, so the extra-precision list is
// a by-product of the same arithmetic.
//
// Extra precision normally runs as one kernel (slice_pack_ep: pack, count,
// chained scan and list in a single pass over the codes).  Shapes it does not
// take (K not a multiple of 16, K > 16384, 2^31 codes or more, unaligned
// buffers) use three stream-ordered kernels: (1) pack + per-row overflow
// counts, (2) one-block exclusive scan of the counts into ovf_row_ptr,
// (3) one warp per row re-reads the codes and writes the ascending column
// list at its row's offset.
#include "common.cuh"

namespace matq {
namespace {

constexpr int kSliceThreads = 256;

struct Sliced {
    uint32_t k;   // four r-bit fields, one per byte
    uint32_t ov;  // bit 0 of each byte: Eq. 8 differs from Eq. 6 here
};

__device__ __forceinline__ Sliced slice4(uint32_t w, int r) {
    const int sh = kCodeBits - r;
    if (sh == 0) return {w, 0u};
    const uint32_t fieldmask = 0x01010101u * ((1u << r) - 1u);
    const uint32_t a = (w >> sh) & fieldmask;
    const uint32_t b = (w >> (sh - 1)) & 0x01010101u;
    const uint32_t s = a + b;
    const uint32_t ov = (s >> r) & 0x01010101u;
    return {s - ov, ov};
}

// Four one-byte fields -> 4*R contiguous bits, element 0 in the least significant bits.
template <int R>
__device__ __forceinline__ uint32_t pack4(uint32_t k) {
    if (R == 8) return k;
    if (R == 4) {
        const uint32_t t = (k | (k >> 4)) & 0x00ff00ffu;
        return (t | (t >> 8)) & 0xffffu;
    }
    const uint32_t t = (k | (k >> 6)) & 0x000f000fu;   // R == 2
    return (t | (t >> 12)) & 0xffu;
}

// r = 2 in one step: four codes -> the packed byte of their four clamped 2-bit fields and the 4-bit mask of the codes
// whose Eq. 8 value is one bucket higher.  With u = q >> 6 (bits 7, 6) and the rounding bit t = bit 5, Eq. 6 is
// min(u + t, 3), i.e. bit 1 = u1 | (u0 & t), bit 0 = (u0 ^ t) | (u1 & u0 & t), overflow = u1 & u0 & t: three
// bitwise functions of the word and its shifts by one and two, evaluated for all four bytes at once (only bits 7
// and 6 of each byte are kept, so what the shifts carry across byte borders never matters).  The multiplications
// gather bits 7, 6 of the four bytes into the top byte, and bit 7 of the four bytes into the top nibble; the partial
// products land on distinct bits, so nothing carries.
__device__ __forceinline__ void slice_pack4_r2(uint32_t w, uint32_t& byte, uint32_t& ovmask) {
    const uint32_t l1 = w << 1, l2 = w << 2, r1 = w >> 1;
    const uint32_t ovw = w & l1 & l2;
    const uint32_t k1 = w | (l1 & l2);
    const uint32_t k0 = (w ^ l1) | (r1 & w & l1);
    const uint32_t kk = (k1 & 0x80808080u) | (k0 & 0x40404040u);
    byte = (kk * 0x00041041u) >> 24;
    ovmask = ((ovw & 0x80808080u) * 0x00204081u) >> 28;
}

// bits 0, 8, 16, 24 -> bits 0..3
__device__ __forceinline__ uint32_t gather_byte_lsbs(uint32_t ov) { return ((ov * 0x01020408u) >> 24) & 0xfu; }

// Fast path: K % 16 == 0 and 16-byte aligned buffers.  One thread = 16 codes.
// PACK_R = 0: no packed output (any r, runtime); otherwise r == PACK_R.
template <int PACK_R>
__global__ void __launch_bounds__(kSliceThreads)
slice_pack_vec(const uint4* __restrict__ q, int64_t nchunks, int chunks_per_row, int r_runtime,
               uint8_t* __restrict__ packed, uint4* __restrict__ sliced, int32_t* __restrict__ row_count) {
    const int r = PACK_R ? PACK_R : r_runtime;
    const int sh = kCodeBits - r;
    const int64_t stride = (int64_t)gridDim.x * kSliceThreads;
    let_next_kernel_start();
    after_previous_kernel();
    for (int64_t i = (int64_t)blockIdx.x * kSliceThreads + threadIdx.x; i < nchunks; i += stride) {
        const uint4 v = ld_stream_u4(q + i);
        if (PACK_R == 2 && !sliced) {
            uint32_t b0, b1, b2, b3, m0, m1, m2, m3;
            slice_pack4_r2(v.x, b0, m0); slice_pack4_r2(v.y, b1, m1); slice_pack4_r2(v.z, b2, m2); slice_pack4_r2(v.w, b3, m3);
            reinterpret_cast<uint32_t*>(packed)[i] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
            if (row_count) {
                const int cnt = __popc(m0 | (m1 << 4) | (m2 << 8) | (m3 << 12));
                if (cnt) atomicAdd(row_count + (i / chunks_per_row), cnt);
            }
            continue;
        }
        const Sliced s0 = slice4(v.x, r), s1 = slice4(v.y, r), s2 = slice4(v.z, r), s3 = slice4(v.w, r);
        if (PACK_R == 8) {
            reinterpret_cast<uint4*>(packed)[i] = make_uint4(s0.k, s1.k, s2.k, s3.k);
        } else if (PACK_R == 4) {
            reinterpret_cast<uint2*>(packed)[i] =
                make_uint2(pack4<4>(s0.k) | (pack4<4>(s1.k) << 16), pack4<4>(s2.k) | (pack4<4>(s3.k) << 16));
        } else if (PACK_R == 2) {
            reinterpret_cast<uint32_t*>(packed)[i] =
                pack4<2>(s0.k) | (pack4<2>(s1.k) << 8) | (pack4<2>(s2.k) << 16) | (pack4<2>(s3.k) << 24);
        }
        if (sliced) sliced[i] = make_uint4(s0.k << sh, s1.k << sh, s2.k << sh, s3.k << sh);
        if (row_count) {
            const int cnt = __popc(s0.ov) + __popc(s1.ov) + __popc(s2.ov) + __popc(s3.ov);
            if (cnt) atomicAdd(row_count + (i / chunks_per_row), cnt);
        }
    }
}

// Any K / alignment: one thread = the codes of one packed byte (or one code when nothing is packed).
__global__ void __launch_bounds__(kSliceThreads)
slice_pack_generic(const uint8_t* __restrict__ q, int64_t N, int64_t K, int r, int per_byte,
                   uint8_t* __restrict__ packed, uint8_t* __restrict__ sliced, int32_t* __restrict__ row_count) {
    const int sh = kCodeBits - r;
    const int64_t groups = N * K / per_byte;
    const int64_t stride = (int64_t)gridDim.x * kSliceThreads;
    for (int64_t g = (int64_t)blockIdx.x * kSliceThreads + threadIdx.x; g < groups; g += stride) {
        uint32_t byte = 0;
        for (int i = 0; i < per_byte; ++i) {
            const int64_t e = g * per_byte + i;
            const Sliced s = slice4(q[e], r);
            byte |= (s.k & 0xffu) << (i * r);
            if (sliced) sliced[e] = (uint8_t)((s.k & 0xffu) << sh);
            if (row_count && (s.ov & 1u)) atomicAdd(row_count + e / K, 1);
        }
        if (packed) packed[g] = (uint8_t)byte;
    }
}

// row_ptr[n+1] holds row n's count on entry; on exit row_ptr is the exclusive scan.
// One CTA: every thread scans kScanItems consecutive rows in registers, the 1024 thread totals are scanned once
// through shared memory, and a running carry links passes of 1024 * kScanItems rows.
constexpr int kScanItems = 16;

__global__ void __launch_bounds__(1024)
ovf_scan(int32_t* __restrict__ row_ptr, int64_t N, int64_t capacity, int64_t* __restrict__ total_out,
         int32_t* dev_status) {
    __shared__ int64_t warp_sum[32];
    __shared__ int64_t carry_s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) { carry_s = 0; row_ptr[0] = 0; }
    __syncthreads();
    for (int64_t base = 0; base < N; base += 1024 * kScanItems) {
        const int64_t n0 = base + (int64_t)threadIdx.x * kScanItems;
        int32_t c[kScanItems];
        int64_t mine = 0;
#pragma unroll
        for (int i = 0; i < kScanItems; ++i) {
            c[i] = (n0 + i < N) ? row_ptr[n0 + i + 1] : 0;
            mine += c[i];
        }
        int64_t v = mine;                                   // inclusive scan of the thread totals
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int64_t t = __shfl_up_sync(0xffffffffu, v, o);
            if (lane >= o) v += t;
        }
        if (lane == 31) warp_sum[warp] = v;
        __syncthreads();
        if (warp == 0) {
            int64_t w = warp_sum[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int64_t t = __shfl_up_sync(0xffffffffu, w, o);
                if (lane >= o) w += t;
            }
            warp_sum[lane] = w;
        }
        __syncthreads();
        int64_t run = carry_s + (v - mine) + (warp ? warp_sum[warp - 1] : 0);   // sum of everything before row n0
#pragma unroll
        for (int i = 0; i < kScanItems; ++i) {
            run += c[i];
            if (n0 + i < N) row_ptr[n0 + i + 1] = (int32_t)(run > 0x7fffffff ? 0x7fffffff : run);
        }
        __syncthreads();
        if (threadIdx.x == 1023) carry_s = run;
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        const int64_t total = carry_s;
        *total_out = total;
        if (total > capacity || total > 0x7fffffff) report(dev_status, MATQ_ERR_CAPACITY);
    }
}

// One warp per row writes the ascending column indices of the overflow elements, one code per lane and step (rows
// whose length or alignment the vectorised variant below does not take).
__global__ void __launch_bounds__(kSliceThreads)
ovf_fill(const uint8_t* __restrict__ q, int64_t N, int64_t K, int r, const int32_t* __restrict__ row_ptr,
         const int64_t* __restrict__ total, int64_t capacity, uint16_t* __restrict__ ovf_col) {
    if (*total > capacity || *total > 0x7fffffff) return;   // lists are unspecified in that case (ovf_scan has reported it)
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (kSliceThreads / 32);
    for (int64_t n = (int64_t)blockIdx.x * (kSliceThreads / 32) + (threadIdx.x >> 5); n < N; n += warps) {
        int64_t out = row_ptr[n];
        if (row_ptr[n + 1] == out) continue;
        const uint8_t* row = q + n * K;
        for (int64_t k0 = 0; k0 < K; k0 += 32) {
            const int64_t k = k0 + lane;
            const uint32_t mask = k < K ? (slice4(row[k], r).ov & 1u) : 0u;
            const unsigned ballot = __ballot_sync(0xffffffffu, mask != 0);
            if (mask) ovf_col[out + __popc(ballot & ((1u << lane) - 1u))] = (uint16_t)k;
            out += __popc(ballot);
        }
    }
}

// The vectorised variant used in practice: the same warp-per-row walk, but eight 512-code pieces of the row are
// fetched at once (eight independent 16-byte loads per lane instead of a load -> scan -> store chain per piece), and
// the eight per-piece lane scans run as three packed scans (counts <= 16 per lane, so 10 bits per running sum).
__global__ void __launch_bounds__(kSliceThreads)
ovf_fill_batched(const uint8_t* __restrict__ q, int64_t N, int64_t K, int r, const int32_t* __restrict__ row_ptr,
                 const int64_t* __restrict__ total, int64_t capacity, uint16_t* __restrict__ ovf_col) {
    if (*total > capacity || *total > 0x7fffffff) return;
    const int lane = threadIdx.x & 31;
    const int64_t warps = (int64_t)gridDim.x * (kSliceThreads / 32);
    for (int64_t n = (int64_t)blockIdx.x * (kSliceThreads / 32) + (threadIdx.x >> 5); n < N; n += warps) {
        int64_t out = row_ptr[n];
        if (row_ptr[n + 1] == out) continue;
        const uint8_t* row = q + n * K;
        for (int64_t k0 = 0; k0 < K; k0 += 8 * 512) {
            uint32_t mask[8];
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const int64_t k = k0 + j * 512 + lane * 16;
                uint4 v = make_uint4(0, 0, 0, 0);
                if (k < K) v = ld_stream_u4(row + k);
                mask[j] = gather_byte_lsbs(slice4(v.x, r).ov) | (gather_byte_lsbs(slice4(v.y, r).ov) << 4) |
                          (gather_byte_lsbs(slice4(v.z, r).ov) << 8) | (gather_byte_lsbs(slice4(v.w, r).ov) << 12);
            }
            uint32_t pk[3];                                   // inclusive lane scans, three 10-bit fields per word
            pk[0] = __popc(mask[0]) | (__popc(mask[1]) << 10) | (__popc(mask[2]) << 20);
            pk[1] = __popc(mask[3]) | (__popc(mask[4]) << 10) | (__popc(mask[5]) << 20);
            pk[2] = __popc(mask[6]) | (__popc(mask[7]) << 10);
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
                for (int w = 0; w < 3; ++w) {
                    const uint32_t t = __shfl_up_sync(0xffffffffu, pk[w], o);
                    if (lane >= o) pk[w] += t;
                }
            }
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                const uint32_t incl = (pk[j / 3] >> (10 * (j % 3))) & 0x3ffu;
                const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
                uint32_t m = mask[j];
                int64_t pos = out + incl - __popc(m);
                const int kb = (int)(k0 + j * 512 + lane * 16);
                while (m) {
                    const int bpos = __ffs(m) - 1;
                    ovf_col[pos++] = (uint16_t)(kb + bpos);
                    m &= m - 1;
                }
                out += tot;
            }
        }
    }
}


// ---------------------------------------------------------------------------------------------------------------
// Extra precision in ONE pass (K % 16 == 0, K <= 16384, N * K < 2^31): pack, count, scan and list in the same kernel,
// so the codes are read from HBM once.
//
// A tile is T = warps * rows_per_warp consecutive rows, sized on the host so that the matrix is about one tile per
// SM.  Every warp slices and packs its rows, parks the 16-bit overflow mask of every 16-code chunk in shared memory
// and counts each row's overflow elements.  Warp 0 scans the T counts and finds the tile's place in the global list
// by a chained scan with look-back: the tile publishes its own total ("partial") at once, sums the partials of the
// tiles before it until it meets one that already knows its inclusive prefix, and finally replaces its own partial
// by its inclusive prefix.  With the place known every warp writes its rows' entries of ovf_row_ptr and their
// columns from the parked masks.  Few, large tiles keep the look-back short (at most a few hundred flags, fetched
// 128 at a time) while the other warps wait at a barrier without issuing anything.
//
// The scan state lives in ovf_row_ptr itself: the entry after a tile's last row is that tile's flag word,
//   0xffffffff (the memset before the launch)  nothing yet
//   0x80000000 | total of the tile             partial (a tile holds fewer than 2^30 elements)
//   value < 2^31                               inclusive prefix = the final content of that entry
//   0xc0000000                                 a wait gave up in this tile or before it
// so value and state travel in one 32-bit word and no ordering between separate words is needed.  CTAs are
// persistent and all resident (the grid is sized from the occupancy), tile t belongs to CTA t mod gridDim.x and only
// ever waits for tiles below t, so every wait ends; each one is bounded all the same, and a wait that gives up
// poisons the flags after it and reports MATQ_ERR_TIMEOUT instead of hanging.
constexpr uint32_t kEpNothing = 0xffffffffu, kEpPartial = 0x80000000u, kEpPoison = 0xc0000000u;
constexpr int kEpSpinLimit = 1 << 20;
constexpr int kEpStallSpinLimit = 1 << 8;    // under matq_slice_pack_test_stall
constexpr int kEpWindows = 4;              // look-back windows of 32 tiles fetched per round trip
constexpr size_t kEpSmemLimit = 160 * 1024;
constexpr int kEpBatch = 6;                // 16-byte loads a lane has in flight

__device__ __forceinline__ uint32_t ld_flag(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_flag(uint32_t* p, uint32_t v) {
    asm volatile("st.relaxed.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

__device__ __forceinline__ uint32_t chunk_mask(const Sliced& s0, const Sliced& s1, const Sliced& s2, const Sliced& s3) {
    return gather_byte_lsbs(s0.ov) | (gather_byte_lsbs(s1.ov) << 4) | (gather_byte_lsbs(s2.ov) << 8) |
           (gather_byte_lsbs(s3.ov) << 12);
}

// Sets every flag word to "nothing yet".  The one-pass kernel is launched as its programmatic dependent: it slices,
// packs and counts while this runs and only waits for it before it touches the first flag.
__global__ void __launch_bounds__(256) ep_init_flags(uint32_t* __restrict__ row_ptr, int64_t n) {
    // Launched as a dependent of whatever precedes it: it waits for that kernel FIRST and only then releases
    // slice_pack_ep, which reads the codes before its own wait (they may be that kernel's output).
    after_previous_kernel();
    asm volatile("griddepcontrol.launch_dependents;");
    for (int64_t i = (int64_t)blockIdx.x * 256 + threadIdx.x; i < n; i += (int64_t)gridDim.x * 256) row_ptr[i] = kEpNothing;
}

template <int PACK_R>
__global__ void __launch_bounds__(1024)
slice_pack_ep(const uint8_t* __restrict__ q, int64_t N, int K, int r_runtime, int rows_per_warp,
              uint8_t* __restrict__ packed, uint8_t* __restrict__ packed4, uint8_t* __restrict__ sliced, uint32_t* __restrict__ row_ptr,
              uint16_t* __restrict__ ovf_col, int64_t capacity, int64_t* __restrict__ total_out, int32_t* dev_status,
              int spin_limit, int hold) {
    // spin_limit: polls of a look-back before it gives up.  hold (tests of that path): the first tile never publishes
    // its prefix, so every later tile's look-back meets "nothing yet" until its limit, or the poison of a tile before it.
    extern __shared__ __align__(16) uint8_t ep_smem[];
    __shared__ uint32_t base_s, total_s;
    __shared__ int bad_s;
    let_next_kernel_start();            // every CTA of this grid is resident by now (one wave), so nothing started early can displace one
    const int r = PACK_R ? PACK_R : r_runtime;
    const int sh = kCodeBits - r;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const int T = nwarps * rows_per_warp;              // rows per tile
    const int cpr = K / 16;                            // 16-code chunks per row
    int* row_off = reinterpret_cast<int*>(ep_smem);    // [T] counts, then exclusive offsets within the tile
    uint16_t* ep_mask = reinterpret_cast<uint16_t*>(row_off + T);   // [T][cpr]
    const int64_t ntiles = (N + T - 1) / T;
    for (int64_t t = blockIdx.x; t < ntiles; t += gridDim.x) {
        const int64_t row0 = t * T;
        for (int i = 0; i < rows_per_warp; ++i) {
            const int lr = i * nwarps + warp;
            const int64_t n = row0 + lr;
            int cnt = 0;
            if (n < N) {
                const uint4* src = reinterpret_cast<const uint4*>(q + n * K);
                const int64_t c_row = n * cpr;
                uint16_t* mrow = ep_mask + (size_t)lr * cpr;
                for (int c0 = 0; c0 < cpr; c0 += kEpBatch * 32) {
                    uint4 v[kEpBatch];
#pragma unroll
                    for (int u = 0; u < kEpBatch; ++u) {
                        const int c = c0 + u * 32 + lane;
                        v[u] = make_uint4(0, 0, 0, 0);
                        if (c < cpr) v[u] = ld_stream_u4(src + c);
                    }
#pragma unroll
                    for (int u = 0; u < kEpBatch; ++u) {
                        const int c = c0 + u * 32 + lane;
                        if (c >= cpr) continue;
                        if (PACK_R == 2 && !sliced) {
                            uint32_t b0, b1, b2, b3, m0, m1, m2, m3;
                            slice_pack4_r2(v[u].x, b0, m0); slice_pack4_r2(v[u].y, b1, m1);
                            slice_pack4_r2(v[u].z, b2, m2); slice_pack4_r2(v[u].w, b3, m3);
                            reinterpret_cast<uint32_t*>(packed)[c_row + c] = b0 | (b1 << 8) | (b2 << 16) | (b3 << 24);
                            if (packed4) {                      // the int4 plane of the same codes from the same read (Eq. 6)
                                const uint32_t k0 = slice4(v[u].x, 4).k, k1 = slice4(v[u].y, 4).k, k2 = slice4(v[u].z, 4).k, k3 = slice4(v[u].w, 4).k;
                                reinterpret_cast<uint2*>(packed4)[c_row + c] =
                                    make_uint2(pack4<4>(k0) | (pack4<4>(k1) << 16), pack4<4>(k2) | (pack4<4>(k3) << 16));
                            }
                            const uint32_t m = m0 | (m1 << 4) | (m2 << 8) | (m3 << 12);
                            mrow[c] = (uint16_t)m;
                            cnt += __popc(m);
                            continue;
                        }
                        const Sliced s0 = slice4(v[u].x, r), s1 = slice4(v[u].y, r), s2 = slice4(v[u].z, r), s3 = slice4(v[u].w, r);
                        if (PACK_R == 4) {
                            reinterpret_cast<uint2*>(packed)[c_row + c] =
                                make_uint2(pack4<4>(s0.k) | (pack4<4>(s1.k) << 16), pack4<4>(s2.k) | (pack4<4>(s3.k) << 16));
                        } else if (PACK_R == 2) {
                            reinterpret_cast<uint32_t*>(packed)[c_row + c] =
                                pack4<2>(s0.k) | (pack4<2>(s1.k) << 8) | (pack4<2>(s2.k) << 16) | (pack4<2>(s3.k) << 24);
                        }
                        if (sliced) reinterpret_cast<uint4*>(sliced)[c_row + c] = make_uint4(s0.k << sh, s1.k << sh, s2.k << sh, s3.k << sh);
                        const uint32_t m = chunk_mask(s0, s1, s2, s3);
                        mrow[c] = (uint16_t)m;
                        cnt += __popc(m);
                    }
                }
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) cnt += __shfl_xor_sync(0xffffffffu, cnt, o);
            }
            if (lane == 0) row_off[lr] = cnt;
        }
        if (t == (int64_t)blockIdx.x) asm volatile("griddepcontrol.wait;" ::: "memory");   // the flags are initialised
        __syncthreads();
        if (warp == 0) {
            uint32_t tile_total = 0;                                     // counts -> exclusive offsets, 32 rows at a time
            for (int c0 = 0; c0 < T; c0 += 32) {
                const int v = c0 + lane < T ? row_off[c0 + lane] : 0;
                int incl = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    const int u = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= o) incl += u;
                }
                if (c0 + lane < T) row_off[c0 + lane] = (int)tile_total + incl - v;
                tile_total += (uint32_t)__shfl_sync(0xffffffffu, incl, 31);
            }
            const int64_t last_row = min(row0 + T - 1, N - 1);
            uint32_t base = 0;
            bool bad = false;
            if (t > 0) {
                if (lane == 0) st_flag(row_ptr + last_row + 1, kEpPartial | tile_total);
                int64_t look = t - 1;                  // lane l of window w looks at tile look - 32 w - l
                for (bool found = false; !found && !bad;) {
                    uint32_t f[kEpWindows];            // "tile -1" and below: inclusive prefix 0
                    int spins = 0;
                    for (;;) {                         // all windows are fetched at once: one L2 round trip for 128 tiles
                        bool nothing = false;
#pragma unroll
                        for (int w = 0; w < kEpWindows; ++w) {
                            const int64_t j = look - 32 * w - lane;
                            f[w] = j >= 0 ? ld_flag(row_ptr + (j + 1) * T) : 0u;   // tiles before t are full
                            nothing |= f[w] == kEpNothing;
                        }
                        if (!__any_sync(0xffffffffu, nothing)) break;
                        if (++spins > spin_limit) { bad = true; break; }
                        __nanosleep(40);
                    }
                    if (bad) break;
#pragma unroll
                    for (int w = 0; w < kEpWindows; ++w) {
                        if (found) continue;
                        if (__any_sync(0xffffffffu, f[w] == kEpPoison)) { bad = true; found = true; continue; }
                        const uint32_t have_incl = __ballot_sync(0xffffffffu, (f[w] & kEpPartial) == 0);
                        const int stop = have_incl ? __ffs(have_incl) - 1 : 31;   // nearest tile with an inclusive prefix
                        uint32_t part = lane <= stop ? (f[w] & 0x7fffffffu) : 0u;
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) part += __shfl_xor_sync(0xffffffffu, part, o);
                        base += part;
                        found = have_incl != 0;
                    }
                    look -= 32 * kEpWindows;
                }
            }
            if (lane == 0) {
                if (bad) {
                    st_flag(row_ptr + last_row + 1, kEpPoison);
                    report(dev_status, MATQ_ERR_TIMEOUT);
                    if (t == ntiles - 1) *total_out = 0;
                } else if (!(hold && t == 0)) {
                    st_flag(row_ptr + last_row + 1, base + tile_total);   // the thread that wrote the partial replaces it
                    if (t == 0) row_ptr[0] = 0;
                    if (t == ntiles - 1) {
                        const int64_t total = (int64_t)base + tile_total;
                        *total_out = total;
                        if (total > capacity) report(dev_status, MATQ_ERR_CAPACITY);
                    }
                }
                base_s = base; total_s = tile_total; bad_s = bad ? 1 : 0;
            }
        }
        __syncthreads();
        if (!bad_s) {
            const int64_t last_row = min(row0 + T - 1, N - 1);
            for (int i = 0; i < rows_per_warp; ++i) {
                const int lr = i * nwarps + warp;
                const int64_t n = row0 + lr;
                if (n >= N) break;
                const uint32_t excl = (uint32_t)row_off[lr];
                const uint32_t cnt = (lr + 1 < T ? (uint32_t)row_off[lr + 1] : total_s) - excl;
                if (lane == 0 && n < last_row) row_ptr[n + 1] = base_s + excl + cnt;
                if (cnt == 0) continue;
                const uint16_t* mrow = ep_mask + (size_t)lr * cpr;
                int64_t out = (int64_t)base_s + excl;
                for (int c0 = 0; c0 < cpr; c0 += 8 * 32) {
                    uint32_t mask[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const int c = c0 + j * 32 + lane;
                        mask[j] = c < cpr ? mrow[c] : 0u;
                    }
                    uint32_t pk[3];                               // inclusive lane scans, three 10-bit fields per word
                    pk[0] = __popc(mask[0]) | (__popc(mask[1]) << 10) | (__popc(mask[2]) << 20);
                    pk[1] = __popc(mask[3]) | (__popc(mask[4]) << 10) | (__popc(mask[5]) << 20);
                    pk[2] = __popc(mask[6]) | (__popc(mask[7]) << 10);
                    if (!__any_sync(0xffffffffu, (pk[0] | pk[1] | pk[2]) != 0)) continue;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
#pragma unroll
                        for (int w = 0; w < 3; ++w) {
                            const uint32_t v = __shfl_up_sync(0xffffffffu, pk[w], o);
                            if (lane >= o) pk[w] += v;
                        }
                    }
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const uint32_t incl = (pk[j / 3] >> (10 * (j % 3))) & 0x3ffu;
                        const uint32_t tot = __shfl_sync(0xffffffffu, incl, 31);
                        uint32_t m = mask[j];
                        int64_t pos = out + incl - __popc(m);
                        const int kb = (c0 + j * 32 + lane) * 16;
                        while (m) {
                            const int bpos = __ffs(m) - 1;
                            if (pos < capacity) ovf_col[pos] = (uint16_t)(kb + bpos);
                            ++pos;
                            m &= m - 1;
                        }
                        out += tot;
                    }
                }
            }
        }
        __syncthreads();                                      // masks, offsets and the base are reused by the next tile
    }
}

// Tests of the look-back's give-up path (matq_slice_pack_test_stall): process-wide, read when a call builds its launch.
static std::atomic<int> g_test_stall{0};

// Returns MATQ_ERR_SHAPE when no tile fits the shared-memory budget (the caller then uses the three-kernel chain).
template <int PACK_R>
int launch_ep(const uint8_t* q, int64_t N, int64_t K, int r, uint8_t* packed, uint8_t* sliced, int32_t* row_ptr,
              uint16_t* ovf_col, int64_t capacity, int64_t* total, int32_t* dev_status, cudaStream_t s, uint8_t* packed4 = nullptr) {
    const int sms = sm_count();
    const size_t row_smem = sizeof(int) + (size_t)(K / 16) * sizeof(uint16_t);
    int nwarps = 32, rpw = 1;
    for (;; nwarps >>= 1) {                                   // about one tile per SM, as many warps per tile as that allows
        rpw = (int)((N + (int64_t)nwarps * sms - 1) / ((int64_t)nwarps * sms));
        const int64_t rpw_fit = (int64_t)(kEpSmemLimit / (row_smem * nwarps));
        if (rpw > rpw_fit) rpw = (int)rpw_fit;
        if (nwarps == 8) break;
        if (rpw >= 1 && (N + (int64_t)nwarps * rpw - 1) / ((int64_t)nwarps * rpw) >= (int64_t)sms * 85 / 100) break;
    }
    if (rpw < 1) return MATQ_ERR_SHAPE;
    const int T = nwarps * rpw;
    const size_t smem = (size_t)T * row_smem;
    static std::atomic<unsigned long long> smem_ok{0};     // one per template instance
    if (smem > 40 * 1024 &&   // the 48 KB default counts static shared memory too
        !opt_in_max_smem(slice_pack_ep<PACK_R>, smem_ok))
        return MATQ_ERR_CUDA;
    int per_sm = 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, slice_pack_ep<PACK_R>, nwarps * 32, smem) != cudaSuccess ||
        per_sm < 1)
        return MATQ_ERR_CUDA;
    const int64_t ntiles = (N + T - 1) / T;
    int64_t blocks = (int64_t)sms * per_sm;                   // all resident: the look-back waits rely on it
    if (blocks > ntiles) blocks = ntiles;
    const int64_t init_blocks = (N + 1 + 255) / 256;
    launch_overlapped(ep_init_flags, dim3((unsigned)(init_blocks < 2 * sms ? init_blocks : 2 * sms)), dim3(256), 0, s, reinterpret_cast<uint32_t*>(row_ptr), (int64_t)(N + 1));
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)blocks);
    cfg.blockDim = dim3((unsigned)(nwarps * 32));
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    const int K32 = (int)K;
    uint32_t* flags = reinterpret_cast<uint32_t*>(row_ptr);
    const int hold = g_test_stall.load(std::memory_order_relaxed) ? 1 : 0;
    if (cudaLaunchKernelEx(&cfg, slice_pack_ep<PACK_R>, q, N, K32, r, rpw, packed, packed4, sliced, flags, ovf_col, capacity, total,
                           dev_status, hold ? kEpStallSpinLimit : kEpSpinLimit, hold) != cudaSuccess) {
        cudaGetLastError();
        return MATQ_ERR_CUDA;
    }
    return launch_status();
}

template <int PACK_R>
void launch_vec(const uint8_t* q, int64_t N, int64_t K, int r, uint8_t* packed, uint8_t* sliced,
                int32_t* row_count, cudaStream_t s) {
    const int64_t nchunks = N * K / 16;
    int64_t blocks = (nchunks + kSliceThreads - 1) / kSliceThreads;
    const int64_t cap = (int64_t)sm_count() * 32;
    if (blocks > cap) blocks = cap;
    launch_overlapped(slice_pack_vec<PACK_R>, dim3((unsigned)blocks), dim3(kSliceThreads), 0, s,
                      reinterpret_cast<const uint4*>(q), nchunks, (int)(K / 16), r, packed, reinterpret_cast<uint4*>(sliced), row_count);
}

}  // namespace
}  // namespace matq

extern "C" int matq_slice_pack_test_stall(int on) { return matq::g_test_stall.exchange(on ? 1 : 0); }

extern "C" int64_t matq_packed_row_bytes(int64_t K, int r) {
    if (!(r == 8 || r == 4 || r == 2) || K <= 0 || (K % (8 / r)) != 0) return -1;
    return K * r / 8;
}

extern "C" int matq_slice_pack(const uint8_t* q, int64_t N, int64_t K, int c, int r, int extra_precision,
                               uint8_t* packed, uint8_t* sliced_unpacked,
                               int32_t* ovf_row_ptr, uint16_t* ovf_col, int64_t ovf_capacity, int64_t* ovf_count,
                               int32_t* dev_status, void* stream) {
    using namespace matq;
    if (N < 0 || K <= 0 || (!q && N > 0)) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits || r < 1 || r > c) return MATQ_ERR_UNSUPPORTED;
    const bool packable = (r == 8 || r == 4 || r == 2);
    if (packed && !packable) return MATQ_ERR_UNSUPPORTED;
    const int per_byte = packed ? 8 / r : 1;
    if (packed && (K % per_byte) != 0) return MATQ_ERR_SHAPE;
    const bool want_ovf = extra_precision && r < c;
    if (want_ovf && (!ovf_row_ptr || !ovf_col || !ovf_count || ovf_capacity < 0)) return MATQ_ERR_INVALID_ARG;
    if (want_ovf && K > 65536) return MATQ_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (!want_ovf && ovf_count && cudaMemsetAsync(ovf_count, 0, sizeof(int64_t), s) != cudaSuccess) return MATQ_ERR_CUDA;
    if (N == 0) {
        if (want_ovf && (cudaMemsetAsync(ovf_row_ptr, 0, sizeof(int32_t), s) != cudaSuccess ||
                         cudaMemsetAsync(ovf_count, 0, sizeof(int64_t), s) != cudaSuccess)) return MATQ_ERR_CUDA;
        return MATQ_OK;
    }
    const bool vec = (K % 16 == 0) && aligned16(q) && (!packed || aligned16(packed)) &&
                     (!sliced_unpacked || aligned16(sliced_unpacked));
    if (want_ovf && vec && K <= 16384 && N * K < (int64_t(1) << 31)) {
        int st;
        if (!packed) st = launch_ep<0>(q, N, K, r, packed, sliced_unpacked, ovf_row_ptr, ovf_col, ovf_capacity, ovf_count, dev_status, s);
        else if (r == 4) st = launch_ep<4>(q, N, K, r, packed, sliced_unpacked, ovf_row_ptr, ovf_col, ovf_capacity, ovf_count, dev_status, s);
        else st = launch_ep<2>(q, N, K, r, packed, sliced_unpacked, ovf_row_ptr, ovf_col, ovf_capacity, ovf_count, dev_status, s);
        if (st != MATQ_ERR_SHAPE) return st;
    }
    int32_t* row_count = nullptr;
    if (want_ovf) {
        if (cudaMemsetAsync(ovf_row_ptr, 0, (size_t)(N + 1) * sizeof(int32_t), s) != cudaSuccess) return MATQ_ERR_CUDA;
        row_count = ovf_row_ptr + 1;
    }
    if (packed || sliced_unpacked || row_count) {
        if (vec) {
            if (!packed) launch_vec<0>(q, N, K, r, packed, sliced_unpacked, row_count, s);
            else if (r == 8) launch_vec<8>(q, N, K, r, packed, sliced_unpacked, row_count, s);
            else if (r == 4) launch_vec<4>(q, N, K, r, packed, sliced_unpacked, row_count, s);
            else launch_vec<2>(q, N, K, r, packed, sliced_unpacked, row_count, s);
        } else {
            const int64_t groups = N * K / per_byte;
            int64_t blocks = (groups + kSliceThreads - 1) / kSliceThreads;
            const int64_t cap = (int64_t)sm_count() * 32;
            if (blocks > cap) blocks = cap;
            slice_pack_generic<<<(unsigned)blocks, kSliceThreads, 0, s>>>(q, N, K, r, per_byte, packed, sliced_unpacked, row_count);
        }
        if (launch_status() != MATQ_OK) return MATQ_ERR_CUDA;
    }
    if (want_ovf) {
        ovf_scan<<<1, 1024, 0, s>>>(ovf_row_ptr, N, ovf_capacity, ovf_count, dev_status);
        const int warps_per_block = kSliceThreads / 32;
        int64_t blocks = (N + warps_per_block - 1) / warps_per_block;
        const int64_t cap = (int64_t)sm_count() * 32;
        if (blocks > cap) blocks = cap;
        if (vec) ovf_fill_batched<<<(unsigned)blocks, kSliceThreads, 0, s>>>(q, N, K, r, ovf_row_ptr, ovf_count, ovf_capacity, ovf_col);
        else ovf_fill<<<(unsigned)blocks, kSliceThreads, 0, s>>>(q, N, K, r, ovf_row_ptr, ovf_count, ovf_capacity, ovf_col);
    }
    return launch_status();
}

extern "C" int matq_slice_pack_nested(const uint8_t* q, int64_t N, int64_t K, int c, uint8_t* packed4, uint8_t* packed2, int extra_precision,
                                      int32_t* ovf_row_ptr, uint16_t* ovf_col, int64_t ovf_capacity, int64_t* ovf_count,
                                      int32_t* dev_status, void* stream) {
    using namespace matq;
    if (N < 0 || K <= 0 || (!q && N > 0) || !packed4 || !packed2) return MATQ_ERR_INVALID_ARG;
    if (c != kCodeBits) return MATQ_ERR_UNSUPPORTED;
    if (K % 4 != 0) return MATQ_ERR_SHAPE;
    if (extra_precision && (!ovf_row_ptr || !ovf_col || !ovf_count || ovf_capacity < 0)) return MATQ_ERR_INVALID_ARG;
    if (extra_precision && K > 65536) return MATQ_ERR_SHAPE;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // one pass over the codes when the one-pass extra-precision kernel takes the shape; two calls otherwise
    const bool vec = (K % 16 == 0) && aligned16(q) && aligned16(packed4) && aligned16(packed2);
    if (extra_precision && N > 0 && vec && K <= 16384 && N * K < (int64_t(1) << 31)) {
        const int st = launch_ep<2>(q, N, K, 2, packed2, nullptr, ovf_row_ptr, ovf_col, ovf_capacity, ovf_count, dev_status, s, packed4);
        if (st != MATQ_ERR_SHAPE) return st;
    }
    const int st = matq_slice_pack(q, N, K, c, 4, 0, packed4, nullptr, nullptr, nullptr, 0, nullptr, dev_status, stream);
    if (st != MATQ_OK) return st;
    return matq_slice_pack(q, N, K, c, 2, extra_precision, packed2, nullptr, ovf_row_ptr, ovf_col, ovf_capacity, ovf_count, dev_status, stream);
}
