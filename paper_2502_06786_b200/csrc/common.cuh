// Shared device/host helpers of the CUDA library (sm_100a only).
#pragma once

#include <atomic>

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "matq.h"

namespace matq {

constexpr int kCodeBits = 8;  // c: the only base width the paper trains (int8)

// First data-dependent error wins; never traps.
__device__ __forceinline__ void report(int32_t* dev_status, int code) {
    if (dev_status) atomicCAS(dev_status, 0, code);
}

__device__ __forceinline__ float bf16_bits_to_float(uint32_t b16) { return __uint_as_float(b16 << 16); }

// 128-bit read-only load that does not pollute L1 (weights are streamed once).
__device__ __forceinline__ uint4 ld_stream_u4(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

inline int launch_status() { return cudaGetLastError() == cudaSuccess ? MATQ_OK : MATQ_ERR_CUDA; }

// Number of SMs of the current device (148 on B200).
inline int sm_count() {
    int dev = 0, n = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) return 148;
    return n;
}

// Programmatic dependent launch that is safe behind ANY kernel: the launch may begin while the previous kernel of the
// stream is still running (its start-up then overlaps that kernel's tail), and the kernel calls after_previous_kernel()
// before its first access to global memory, so it neither reads what the predecessor has not written yet nor writes what
// it may still read.  let_next_kernel_start() lets a successor launched the same way begin its own start-up early.
__device__ __forceinline__ void after_previous_kernel() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void let_next_kernel_start() { asm volatile("griddepcontrol.launch_dependents;"); }

template <typename Kern, typename... Args>
inline cudaError_t launch_overlapped(Kern kern, dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, args...);
}

// Opts a kernel in, once per device, to the largest dynamic shared memory size an SM offers it (227 KB less the
// kernel's static shared memory).  The attribute belongs to the function, not to a launch: setting it to each call's
// size would let two host threads with different shapes undo one another between the setting and the launch.
// `done` holds one bit per device; give every kernel (every template instance) its own.
template <typename Kern>
inline bool opt_in_max_smem(Kern kern, std::atomic<unsigned long long>& done) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    const unsigned long long bit = 1ull << (dev & 63);
    if (done.load(std::memory_order_acquire) & bit) return true;
    cudaFuncAttributes attr;
    if (cudaFuncGetAttributes(&attr, kern) != cudaSuccess) { cudaGetLastError(); return false; }
    const int max_dynamic = 227 * 1024 - (int)attr.sharedSizeBytes;
    if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dynamic) != cudaSuccess) { cudaGetLastError(); return false; }
    done.fetch_or(bit, std::memory_order_release);
    return true;
}

}  // namespace matq
