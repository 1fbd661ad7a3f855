// Shared helpers of the lvlm kernels: argument checks, bf16 packing, order-preserving keys.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "lvlm.h"

namespace lvlm {

constexpr int kHeadDim = 128;
constexpr int kMaxSortN = 16384;      // kv_compress: one CTA (1024 threads, 16 entries each) holds at most this many keys
constexpr int kMaxGroup = 8;          // query heads per KV head supported by decode attention
// Opt-in limit of dynamic shared memory asked for every kernel that may exceed 48 KB.  The
// attribute is a property of the function, not of a launch, so it is always set to this one
// value: a launch recorded in a CUDA graph stays valid whatever size later calls use.
constexpr int kMaxDynSmem = 200 * 1024;

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
inline bool aligned256(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 255u) == 0; }
inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

#define LVLM_RETURN_IF_CUDA(expr)                      \
    do {                                               \
        cudaError_t e__ = (expr);                      \
        if (e__ != cudaSuccess) return LVLM_ERR_CUDA;  \
    } while (0)

inline lvlm_status launch_status() {
    return cudaGetLastError() == cudaSuccess ? LVLM_OK : LVLM_ERR_CUDA;
}

// ---- programmatic dependent launch ----------------------------------------------------------
// Every kernel of the library is launched so that it may be scheduled while the kernel before it
// in the stream is still draining (launch latency and the start-up of its CTAs overlap the tail
// of that kernel).  The contract inside a kernel: pdl_wait() comes before the first access to
// global memory that an earlier kernel may have written, or that an earlier kernel may still read
// while this one writes it; once it returns, everything enqueued before is complete and visible.
// pdl_launch_dependents() lets the next kernel start being scheduled; it comes right after the wait.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_enter() { pdl_wait(); pdl_launch_dependents(); }

bool pdl_enabled();            // lvlm.cu: true, except in the test build when its hook switched it off

// Launches `kernel` with programmatic stream serialisation and thread-block clusters of the given shape
// (1, 1, 1 = no clusters).
template <typename... KArgs, typename... Args>
inline lvlm_status launch_kernel_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                         cudaStream_t stream, dim3 cluster, Args... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    int na = 0;
    if (cluster.x * cluster.y * cluster.z > 1) {
        attr[na].id = cudaLaunchAttributeClusterDimension;
        attr[na].val.clusterDim.x = cluster.x;
        attr[na].val.clusterDim.y = cluster.y;
        attr[na].val.clusterDim.z = cluster.z;
        ++na;
    }
    if (pdl_enabled()) {
        attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[na].val.programmaticStreamSerializationAllowed = 1;
        ++na;
    }
    cfg.attrs = attr;
    cfg.numAttrs = na;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...) == cudaSuccess ? LVLM_OK : LVLM_ERR_CUDA;
}

// The same with clusters of cluster_x CTAs along x.
template <typename... KArgs, typename... Args>
inline lvlm_status launch_kernel(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem,
                                 cudaStream_t stream, int cluster_x, Args... args) {
    return launch_kernel_cluster(kernel, grid, block, smem, stream, dim3(cluster_x < 1 ? 1 : cluster_x, 1, 1),
                                 args...);
}

// ---- bf16 <-> fp32 on packed words -------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// ---- total order used by selection and eviction --------------------------------------
// Ascending order of the returned 32-bit value == DESCENDING order of the score; NaN maps to
// the largest value (sorted last); -0 and +0 map to the same value.
__device__ __forceinline__ uint32_t desc_key(float s, bool* nonfinite) {
    uint32_t u = __float_as_uint(s);
    if ((u & 0x7F800000u) == 0x7F800000u) *nonfinite = true;
    if ((u & 0x7FFFFFFFu) > 0x7F800000u) return 0xFFFFFFFFu;      // NaN
    if (u == 0x80000000u) u = 0;                                  // -0 -> +0
    uint32_t asc = (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    return ~asc;
}

// ---- small block-level primitives ----------------------------------------------------
__device__ __forceinline__ int warp_sum(int v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// Exclusive prefix sum of one int per thread over the block (blockDim.x <= 1024, a multiple
// of 32).  `scratch` holds 33 ints of shared memory.  Returns the exclusive prefix; *total
// receives the block sum.
__device__ __forceinline__ int block_exclusive_scan(int v, int* scratch, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nwarp = blockDim.x >> 5;
    int incl = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        int t = __shfl_up_sync(0xFFFFFFFFu, incl, o);
        if (lane >= o) incl += t;
    }
    __syncthreads();                      // scratch may still be read from a previous call
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        int w = lane < nwarp ? scratch[lane] : 0;
        int wi = w;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            int t = __shfl_up_sync(0xFFFFFFFFu, wi, o);
            if (lane >= o) wi += t;
        }
        scratch[lane] = wi - w;           // exclusive warp offsets
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    *total = scratch[32];
    return scratch[warp] + incl - v;
}

}  // namespace lvlm
