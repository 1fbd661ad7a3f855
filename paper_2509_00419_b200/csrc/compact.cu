// In-place stable compaction of row sequences.  Every output row lies at or before its source
// row, so a sequence can be rewritten from the front as long as nobody overwrites a row that
// somebody else still has to read.
//
// A sequence (or, for wide rows, one group of its columns: column groups never interact) is
// walked by one thread-block cluster in super-tiles of S x R consecutive positions, CTA `rank`
// owning R of them.  Per super-tile every CTA stages rows in shared memory (cp.async) - the source
// rows of its output positions, or, when rows are merged, its input rows themselves - and only after
// a cluster barrier, when every CTA has its rows on chip, writes: a row goes to its destination,
// a merged row is added to fp32 sums.  What the next super-tile needs lies beyond everything written
// so far, so it is fetched into a second buffer while the current one is being stored.
// With many independent sequences S is 1 and the barrier is a block barrier.
#include "compact.cuh"

namespace lvlm {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxC = 4;              // 16-byte column groups per thread
constexpr int kCompactBufBytes = 24 * 1024;  // one of the two staging buffers
constexpr int kCompactMaxCluster = 8;
constexpr int kCompactTargetCtas = 2 * 148;

struct InplaceArgs {
    char* base0; char* base1;
    int64_t stride_b, stride_g;
    int G, V, Vsub, S, Nout, N, n, i0, merged_row, meta_stride, maps_per_g, Rmax, CG, RL;
    int64_t map_stride;
    const int32_t* src_map; const int32_t* dst_map; const float* wgt; const int32_t* meta; const int32_t* nout;
};

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
    const uint32_t s = (uint32_t)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem) : "memory");
}
__device__ __forceinline__ void cp_async_commit_group() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait_group() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_barrier() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n"
                 "barrier.cluster.wait.acquire.aligned;\n" ::: "memory");
}
// Execution barrier only: nobody passes before everybody has arrived, but no memory is published.  Enough
// between "my rows are on chip" and "I overwrite rows": nobody reads what another CTA writes here.
__device__ __forceinline__ void cluster_barrier_exec() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;\n"
                 "barrier.cluster.wait.aligned;\n" ::: "memory");
}
__device__ __forceinline__ float ld_cluster_f32(const float* my_smem, uint32_t rank) {
    uint32_t local = (uint32_t)__cvta_generic_to_shared(my_smem), remote;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(local), "r"(rank));
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(remote) : "memory");
    return v;
}

// grid.x = column groups * S (clusters of S along x), grid.y = G (* 2 with a second tensor), grid.z = B
template <int MAXC>                                      // 16-byte column groups per thread
__global__ void __launch_bounds__(kCompactThreads) inplace_compact_kernel(const InplaceArgs a) {
    extern __shared__ __align__(16) uint4 tile[];
    pdl_enter();
    const int S = a.S;
    const int rank = (int)cluster_rank();
    const int col = blockIdx.x / S;
    const int which = blockIdx.y / a.G, g = blockIdx.y % a.G, b = blockIdx.z;
    char* base = (which ? a.base1 : a.base0) + (int64_t)b * a.stride_b + (int64_t)g * a.stride_g;
    const int V = a.V;
    const int c0 = col * a.Vsub;                         // my columns: [c0, c0 + vw) of V
    const int vw = min(a.Vsub, V - c0);
    uint4* rows = reinterpret_cast<uint4*>(base) + c0;
    const int m = a.maps_per_g == 1 ? b : b * a.G + g;
    const int32_t* src = a.src_map + (int64_t)m * a.map_stride;
    const int Nout = a.nout ? a.nout[m] : a.Nout;
    const int o_start = a.meta[m * a.meta_stride];
    const float* w = a.wgt ? a.wgt + (int64_t)b * a.n : nullptr;
    const int Nscan = w ? a.N : Nout;
    const int CG = a.CG, RL = a.RL;
    const int cg = threadIdx.x % CG, rl = threadIdx.x / CG;

    // rows per CTA per super-tile: everything that is left, shared out evenly, capped by the buffer
    int R = (max(Nscan - o_start, 1) + S - 1) / S;
    R = (R + RL - 1) / RL * RL;
    R = min(R, a.Rmax);
    const int Rc = R * S;
    uint4* buf[2] = {tile, tile + (size_t)a.Rmax * a.Vsub};
    // Two ways to walk a sequence.  Without merged rows (w == NULL) the walk is over OUTPUT positions: a
    // position's source row is staged (rows that are dropped are never read).  With merged rows the walk is
    // over INPUT positions: every row from the first change on is staged exactly once, in order, and then
    // either stored to its destination (at or before it) or added, times its weight, to the sums.
    // Per position of a super-tile: s_idx = row to copy from / to (-1: nothing, -2: merged row), s_wt = weight;
    // both are fetched two rounds ahead so that no copy ever waits for them.
    const bool by_input = w != nullptr;
    const int32_t* dst = by_input ? a.dst_map + (int64_t)b * a.map_stride : nullptr;
    int32_t* s_idx = reinterpret_cast<int32_t*>(tile + 2 * (size_t)a.Rmax * a.Vsub);     // [3][Rmax]
    float* s_wt = reinterpret_cast<float*>(s_idx + 3 * a.Rmax);                          // [3][Rmax]
    constexpr int kIdxPerThread = 2;                     // Rmax <= 2 * blockDim.x

    float acc[MAXC][8];
#pragma unroll
    for (int ci = 0; ci < MAXC; ++ci)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[ci][e] = 0.f;

    auto fetch_idx = [&](int t0, int* reg, float* regw) {
#pragma unroll
        for (int u = 0; u < kIdxPerThread; ++u) {
            const int rr = threadIdx.x + u * kCompactThreads;
            const int o = t0 + rank * R + rr;
            int v = -1;
            float wv = 0.f;
            if (rr < R) {
                if (!by_input) {
                    if (o < Nout) { v = src[o]; if (v == o) v = -1; }
                } else if (o < a.N) {
                    const int d = dst[o];                                  // two independent loads
                    wv = (o >= a.i0 && o < a.i0 + a.n) ? w[o - a.i0] : 0.f;
                    if (d >= 0) { v = d == o ? -1 : d; wv = 0.f; }
                    else v = wv != 0.f ? -2 : -1;
                }
            }
            reg[u] = v;
            regw[u] = wv;
        }
    };
    auto put_idx = [&](int slot, const int* reg, const float* regw) {
#pragma unroll
        for (int u = 0; u < kIdxPerThread; ++u) {
            const int rr = threadIdx.x + u * kCompactThreads;
            if (rr < R) { s_idx[slot * a.Rmax + rr] = reg[u]; s_wt[slot * a.Rmax + rr] = regw[u]; }
        }
    };
    auto load_tile = [&](int t0, int slot, uint4* dstbuf) {
        for (int rr = rl; rr < R; rr += RL) {
            const int v = s_idx[slot * a.Rmax + rr];
            if (v != -1) {
                const int64_t from = by_input ? (int64_t)(t0 + rank * R + rr) : (int64_t)v;
#pragma unroll
                for (int ci = 0; ci < MAXC; ++ci) {
                    const int c = cg + ci * CG;
                    if (c < vw) cp_async16(&dstbuf[rr * a.Vsub + c], rows + from * V + c);
                }
            }
        }
        cp_async_commit_group();
    };

    {
        int reg[kIdxPerThread];
        float regw[kIdxPerThread];
        fetch_idx(o_start, reg, regw);
        put_idx(0, reg, regw);
        fetch_idx(o_start + Rc, reg, regw);
        put_idx(1, reg, regw);
        __syncthreads();
    }
    load_tile(o_start, 0, buf[0]);
    int k = 0;
    for (int t0 = o_start; t0 < Nscan; t0 += Rc, ++k) {
        if (t0 + Rc < Nscan) load_tile(t0 + Rc, (k + 1) % 3, buf[(k + 1) & 1]);
        else cp_async_commit_group();
        int reg[kIdxPerThread];
        float regw[kIdxPerThread];
        fetch_idx(t0 + 2 * Rc, reg, regw);            // in flight while this round runs
        cp_async_wait_group<1>();                     // this super-tile's rows have landed
        __syncthreads();                              // ... for every thread of this CTA
        cluster_barrier_exec();                       // ... in every CTA of the cluster
        const uint4* cur = buf[k & 1];
        const int32_t* cur_idx = s_idx + (k % 3) * a.Rmax;
        const float* cur_wt = s_wt + (k % 3) * a.Rmax;
        for (int rr = rl; rr < R; rr += RL) {
            const int v = cur_idx[rr];
            if (v >= 0) {
                const int64_t to = by_input ? (int64_t)v : (int64_t)(t0 + rank * R + rr);
#pragma unroll
                for (int ci = 0; ci < MAXC; ++ci) {
                    const int c = cg + ci * CG;
                    if (c < vw) rows[to * V + c] = cur[rr * a.Vsub + c];
                }
            } else if (v == -2) {
                const float wj = cur_wt[rr];
#pragma unroll
                for (int ci = 0; ci < MAXC; ++ci) {
                    const int c = cg + ci * CG;
                    if (c < vw) {
                        const uint4 xv = cur[rr * a.Vsub + c];
                        acc[ci][0] = fmaf(wj, bf16_lo(xv.x), acc[ci][0]); acc[ci][1] = fmaf(wj, bf16_hi(xv.x), acc[ci][1]);
                        acc[ci][2] = fmaf(wj, bf16_lo(xv.y), acc[ci][2]); acc[ci][3] = fmaf(wj, bf16_hi(xv.y), acc[ci][3]);
                        acc[ci][4] = fmaf(wj, bf16_lo(xv.z), acc[ci][4]); acc[ci][5] = fmaf(wj, bf16_hi(xv.z), acc[ci][5]);
                        acc[ci][6] = fmaf(wj, bf16_lo(xv.w), acc[ci][6]); acc[ci][7] = fmaf(wj, bf16_hi(xv.w), acc[ci][7]);
                    }
                }
            }
        }
        put_idx((k + 2) % 3, reg, regw);
        __syncthreads();                              // buffer and index slot are reused in the next round
    }
    cp_async_wait_group<0>();
    if (!w) return;
    // merged row: row lanes added in lane order, CTAs in rank order, rounded once, stored by rank 0
    float* red = reinterpret_cast<float*>(tile);          // [RL][vw][8]
#pragma unroll
    for (int ci = 0; ci < MAXC; ++ci) {
        const int c = cg + ci * CG;
        if (c < vw) {
#pragma unroll
            for (int e = 0; e < 8; ++e) red[(rl * vw + c) * 8 + e] = acc[ci][e];
        }
    }
    __syncthreads();
    float* part = red + (size_t)RL * vw * 8;              // [vw][8] this CTA's sum
    for (int i = threadIdx.x; i < vw * 8; i += blockDim.x) {
        float t = 0.f;
        for (int l = 0; l < RL; ++l) t += red[l * vw * 8 + i];
        part[i] = t;
    }
    cluster_barrier();
    if (rank == 0) {
        for (int c = threadIdx.x; c < vw; c += blockDim.x) {
            float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
            for (int r = 0; r < S; ++r)
#pragma unroll
                for (int e = 0; e < 8; ++e) t[e] += ld_cluster_f32(part + c * 8 + e, r);
            uint4 o;
            o.x = pack_bf16(t[0], t[1]); o.y = pack_bf16(t[2], t[3]);
            o.z = pack_bf16(t[4], t[5]); o.w = pack_bf16(t[6], t[7]);
            rows[(int64_t)a.merged_row * V + c] = o;
        }
    }
    cluster_barrier();                                    // rank 0 has read everybody's sums
}

lvlm_status launch_inplace_compact(void* base0, void* base1, int64_t stride_b, int64_t stride_g,
                                   int B, int G, int V, int Nout, const int32_t* src_map,
                                   const float* wgt, const int32_t* meta, int N, int n, int i0,
                                   int merged_row, int meta_stride, cudaStream_t stream,
                                   int maps_per_g, int64_t map_stride, const int32_t* nout,
                                   const int32_t* dst_map) {
    InplaceArgs a;
    if (wgt && !dst_map) return LVLM_ERR_INVALID_ARG;      // merged rows need the destination map
    a.dst_map = dst_map;
    a.base0 = static_cast<char*>(base0);
    a.base1 = static_cast<char*>(base1);
    a.stride_b = stride_b; a.stride_g = stride_g;
    a.G = G; a.V = V; a.Nout = Nout; a.N = N; a.n = n; a.i0 = i0; a.merged_row = merged_row;
    a.meta_stride = meta_stride; a.maps_per_g = maps_per_g;
    a.map_stride = map_stride < 0 ? N : map_stride;
    a.src_map = src_map; a.wgt = wgt; a.meta = meta; a.nout = nout;

    // enough CTAs to fill the GPU: first a cluster per sequence, then column groups of wide rows
    const int64_t nseq = (int64_t)B * G * (base1 ? 2 : 1);
    int S = 1;
    while (S < kCompactMaxCluster && nseq * (2 * S) <= kCompactTargetCtas && N / (2 * S) >= 32) S *= 2;
    int Vsub = V;
    while (Vsub > 8 && nseq * S * ((V + Vsub - 1) / Vsub) < 2 * kCompactTargetCtas) Vsub = ((Vsub + 1) / 2 + 7) / 8 * 8;
    // rows wider than the per-thread budget are always split
    while (Vsub > kCompactMaxC * kCompactThreads) Vsub = ((Vsub + 1) / 2 + 7) / 8 * 8;
    const int ncol = (V + Vsub - 1) / Vsub;
    a.S = S; a.Vsub = Vsub;
    int CG = 1;
    while (CG * 2 <= Vsub && CG * 2 <= kCompactThreads) CG *= 2;
    if ((Vsub + CG - 1) / CG > kCompactMaxC) return LVLM_ERR_UNSUPPORTED;
    a.CG = CG; a.RL = kCompactThreads / CG;
    int R = kCompactBufBytes / (Vsub * 16);
    R = R > 2 * kCompactThreads ? 2 * kCompactThreads : R;
    R = R / a.RL * a.RL;
    if (R < a.RL) R = a.RL;
    a.Rmax = R;
    size_t smem = 2 * (size_t)R * Vsub * 16 + 6 * (size_t)R * 4;
    const size_t red = ((size_t)a.RL + 1) * Vsub * 32;
    if (red > smem) smem = red;
    if (smem > (size_t)kMaxDynSmem) return LVLM_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)(ncol * S), (unsigned)(G * (base1 ? 2 : 1)), (unsigned)B);
    const int chunks = (Vsub + CG - 1) / CG;
#define LVLM_COMPACT_CASE(MC)                                                                              \
    do {                                                                                                   \
        LVLM_RETURN_IF_CUDA(cudaFuncSetAttribute(inplace_compact_kernel<MC>,                               \
                                                 cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynSmem)); \
        return launch_kernel(inplace_compact_kernel<MC>, grid, dim3(kCompactThreads), smem, stream, S, a); \
    } while (0)
    if (chunks <= 1) LVLM_COMPACT_CASE(1);
    if (chunks <= 2) LVLM_COMPACT_CASE(2);
    LVLM_COMPACT_CASE(4);
#undef LVLM_COMPACT_CASE
}

}  // namespace lvlm
