// In-place stable compaction of row sequences.  Every output row lies at or before its source
// row, so one CTA can walk a sequence tile by tile in increasing order: it stages the tile's
// source rows in shared memory, adds the merged (dropped) rows that sit in the tile's position
// range to fp32 accumulators, and only then overwrites those positions.
#include "compact.cuh"

namespace lvlm {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxC = 4;           // 16-byte column groups per thread (rows up to 16 KB)
constexpr int kCompactSmem = 96 * 1024;

struct InplaceArgs {
    char* base0; char* base1;
    int64_t stride_b, stride_g;
    int G, V, Nout, N, n, i0, merged_row, meta_stride, maps_per_g, R, CG, RL;
    int64_t map_stride;
    const int32_t* src_map; const float* wgt; const int32_t* meta; const int32_t* nout;
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_wait_all() {
    asm volatile("cp.async.wait_all;\n" ::: "memory");
}

__global__ void __launch_bounds__(kCompactThreads) inplace_compact_kernel(InplaceArgs a) {
    extern __shared__ __align__(16) uint4 tile[];
    const int which = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    char* base = (which ? a.base1 : a.base0) + (int64_t)b * a.stride_b + (int64_t)g * a.stride_g;
    uint4* rows = reinterpret_cast<uint4*>(base);
    const int m = a.maps_per_g == 1 ? b : b * a.G + g;
    const int32_t* src = a.src_map + (int64_t)m * a.map_stride;
    const int Nout = a.nout ? a.nout[m] : a.Nout;
    const int o_start = a.meta[m * a.meta_stride];
    const float* w = a.wgt ? a.wgt + (int64_t)b * a.n : nullptr;
    const int Nscan = w ? a.N : Nout;
    const int V = a.V, CG = a.CG, RL = a.RL, R = a.R;
    const int cg = threadIdx.x % CG, rl = threadIdx.x / CG;

    float acc[kCompactMaxC][8];
#pragma unroll
    for (int ci = 0; ci < kCompactMaxC; ++ci)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[ci][e] = 0.f;

    for (int t0 = o_start; t0 < Nscan; t0 += R) {
        for (int rr = rl; rr < R; rr += RL) {
            const int o = t0 + rr;
            if (o < Nout) {
                const int s = src[o];
                if (s >= 0 && s != o) {
#pragma unroll
                    for (int ci = 0; ci < kCompactMaxC; ++ci) {
                        const int c = cg + ci * CG;
                        if (c < V) cp_async16(&tile[rr * V + c], rows + (int64_t)s * V + c);
                    }
                }
            }
            if (w && o < Nscan && o >= a.i0 && o < a.i0 + a.n) {
                const float wj = w[o - a.i0];
                if (wj != 0.f) {
#pragma unroll
                    for (int ci = 0; ci < kCompactMaxC; ++ci) {
                        const int c = cg + ci * CG;
                        if (c < V) {
                            const uint4 x = rows[(int64_t)o * V + c];
                            acc[ci][0] = fmaf(wj, bf16_lo(x.x), acc[ci][0]); acc[ci][1] = fmaf(wj, bf16_hi(x.x), acc[ci][1]);
                            acc[ci][2] = fmaf(wj, bf16_lo(x.y), acc[ci][2]); acc[ci][3] = fmaf(wj, bf16_hi(x.y), acc[ci][3]);
                            acc[ci][4] = fmaf(wj, bf16_lo(x.z), acc[ci][4]); acc[ci][5] = fmaf(wj, bf16_hi(x.z), acc[ci][5]);
                            acc[ci][6] = fmaf(wj, bf16_lo(x.w), acc[ci][6]); acc[ci][7] = fmaf(wj, bf16_hi(x.w), acc[ci][7]);
                        }
                    }
                }
            }
        }
        cp_async_wait_all();
        __syncthreads();
        for (int rr = rl; rr < R; rr += RL) {
            const int o = t0 + rr;
            if (o < Nout) {
                const int s = src[o];
                if (s >= 0 && s != o) {
#pragma unroll
                    for (int ci = 0; ci < kCompactMaxC; ++ci) {
                        const int c = cg + ci * CG;
                        if (c < V) rows[(int64_t)o * V + c] = tile[rr * V + c];
                    }
                }
            }
        }
        __syncthreads();
    }
    if (!w) return;
    // merged row: add the row-lane partial sums in lane order, round once, store
    float* red = reinterpret_cast<float*>(tile);          // [RL][V*8]
#pragma unroll
    for (int ci = 0; ci < kCompactMaxC; ++ci) {
        const int c = cg + ci * CG;
        if (c < V) {
#pragma unroll
            for (int e = 0; e < 8; ++e) red[(rl * V + c) * 8 + e] = acc[ci][e];
        }
    }
    __syncthreads();
    for (int c = threadIdx.x; c < V; c += blockDim.x) {
        float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
        for (int l = 0; l < RL; ++l)
#pragma unroll
            for (int e = 0; e < 8; ++e) t[e] += red[(l * V + c) * 8 + e];
        uint4 o;
        o.x = pack_bf16(t[0], t[1]); o.y = pack_bf16(t[2], t[3]);
        o.z = pack_bf16(t[4], t[5]); o.w = pack_bf16(t[6], t[7]);
        rows[(int64_t)a.merged_row * V + c] = o;
    }
}

lvlm_status launch_inplace_compact(void* base0, void* base1, int64_t stride_b, int64_t stride_g,
                                   int B, int G, int V, int Nout, const int32_t* src_map,
                                   const float* wgt, const int32_t* meta, int N, int n, int i0,
                                   int merged_row, int meta_stride, cudaStream_t stream,
                                   int maps_per_g, int64_t map_stride, const int32_t* nout) {
    InplaceArgs a;
    a.base0 = static_cast<char*>(base0);
    a.base1 = static_cast<char*>(base1);
    a.stride_b = stride_b; a.stride_g = stride_g;
    a.G = G; a.V = V; a.Nout = Nout; a.N = N; a.n = n; a.i0 = i0; a.merged_row = merged_row;
    a.meta_stride = meta_stride; a.maps_per_g = maps_per_g;
    a.map_stride = map_stride < 0 ? N : map_stride;
    a.src_map = src_map; a.wgt = wgt; a.meta = meta; a.nout = nout;
    int CG = 1;
    while (CG * 2 <= V && CG * 2 <= kCompactThreads) CG *= 2;
    if ((V + CG - 1) / CG > kCompactMaxC) return LVLM_ERR_UNSUPPORTED;
    a.CG = CG; a.RL = kCompactThreads / CG;
    int R = kCompactSmem / (V * 16);
    R = R > 256 ? 256 : R;
    R = R / a.RL * a.RL;
    if (R < 2 * a.RL) R = 2 * a.RL;
    a.R = R;
    const size_t smem = (size_t)R * V * 16;
    if (smem > (size_t)kMaxDynSmem) return LVLM_ERR_UNSUPPORTED;
    LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(inplace_compact_kernel,
                                             cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem));
    dim3 grid(base1 ? 2 : 1, G, B);
    inplace_compact_kernel<<<grid, kCompactThreads, smem, stream>>>(a);
    return launch_status();
}

}  // namespace lvlm
