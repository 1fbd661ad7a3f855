// In-place stable compaction of row sequences.  Every output row lies at or before its source
// row, so a sequence can be rewritten from the front as long as nobody overwrites a row that
// somebody else still has to read.
//
// A sequence (or, for wide rows, one group of its columns: column groups never interact) is
// walked by one thread-block cluster in super-tiles of S x R consecutive OUTPUT positions, CTA
// `rank` owning R of them.  Per super-tile every CTA stages the source rows of its positions in
// shared memory (16-byte cp.async per thread: the rows are 256 bytes or pieces of wider rows, too
// small for bulk copies to pay), and only after a cluster barrier, when every CTA has its rows on
// chip, writes them.  Rows that are dropped are never read; rows that stay where they are are never
// touched.  What the next super-tile needs lies beyond everything written so far, so it is fetched
// into a second buffer while the current one is being stored.  With many independent sequences S
// is 1 and the barrier is a block barrier.
//
// The merged row of lvlm_merge_compact is not computed here: the kernel that streams the rows
// before this one leaves fp32 partial sums, and the CTA that owns the merged position adds them in
// a fixed order and writes the row.
#include "compact.cuh"

namespace lvlm {

constexpr int kCompactThreads = 256;
constexpr int kCompactMaxC = 4;              // 16-byte column groups per thread
constexpr int kCompactMaxCluster = 8;
constexpr int kCompactTargetCtas = 2 * 148;
constexpr int kIdxPerThread = 2;             // positions of a super-tile per thread: Rmax <= 2 * blockDim.x

struct InplaceArgs {
    char* base0; char* base1;
    int64_t stride_b, stride_g, map_stride;
    int G, T, V, Vsub, S, Nout, meta_stride, maps_per_g, Rmax, CG, RL, merged_row, P, early;
    const int32_t* src_map; const int32_t* meta; const int32_t* nout; const float* partial;
    char* fin_base; int64_t fin_stride_b; int fin_row, fin_V, fin_P, fin_y; const float* fin_partial;
    uint32_t* side_dst[2]; const uint32_t* side_src[2];
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
// Execution barrier only: nobody passes before everybody has arrived, but no memory is published.  Enough
// between "my rows are on chip" and "I overwrite rows": nobody reads what another CTA writes here.
__device__ __forceinline__ void cluster_barrier_exec() {
    asm volatile("barrier.cluster.arrive.relaxed.aligned;\n"
                 "barrier.cluster.wait.aligned;\n" ::: "memory");
}

// Sum of P fp32 partial rows (pp[p*row_floats + c*8 ...], p = 0..P-1 in that order) for 16-byte group c, rounded once.
__device__ __forceinline__ uint4 sum_partials(const float* pp, int P, int64_t row_floats, int c) {
    float t[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    for (int p0 = 0; p0 < P; p0 += 4) {
        float4 x0[4], x1[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            x0[u] = x1[u] = make_float4(0.f, 0.f, 0.f, 0.f);
            if (p0 + u < P) {
                const float4* q = reinterpret_cast<const float4*>(pp + (int64_t)(p0 + u) * row_floats + c * 8);
                x0[u] = __ldcg(q); x1[u] = __ldcg(q + 1);
            }
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            t[0] += x0[u].x; t[1] += x0[u].y; t[2] += x0[u].z; t[3] += x0[u].w;
            t[4] += x1[u].x; t[5] += x1[u].y; t[6] += x1[u].z; t[7] += x1[u].w;
        }
    }
    uint4 o;
    o.x = pack_bf16(t[0], t[1]); o.y = pack_bf16(t[2], t[3]);
    o.z = pack_bf16(t[4], t[5]); o.w = pack_bf16(t[6], t[7]);
    return o;
}

// grid.x = column groups * S (clusters of S along x), grid.y = G * T (+ 1: the CTAs that finish the merged row of
// another tensor), grid.z = B
template <int MAXC>                                      // 16-byte column groups per thread
__global__ void __launch_bounds__(kCompactThreads) inplace_compact_kernel(const InplaceArgs a) {
    extern __shared__ __align__(16) uint4 tile[];
    if (!a.early) pdl_enter();
    if ((int)blockIdx.y == a.fin_y) {                    // merged row of the other tensor: the CTAs of this row share its columns
        if (a.early) pdl_enter();
        const int b = blockIdx.z;
        const float* pp = a.fin_partial + (int64_t)b * a.fin_P * a.fin_V * 8;
        uint4* out = reinterpret_cast<uint4*>(a.fin_base + (int64_t)b * a.fin_stride_b) + (int64_t)a.fin_row * a.fin_V;
        for (int c = blockIdx.x * kCompactThreads + threadIdx.x; c < a.fin_V; c += gridDim.x * kCompactThreads)
            out[c] = sum_partials(pp, a.fin_P, (int64_t)a.fin_V * 8, c);
        return;
    }
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
    const int CG = a.CG, RL = a.RL;
    const int cg = threadIdx.x % CG, rl = threadIdx.x / CG;

    // the small per-entry arrays the kernel before compacted out of place: copied back by the CTA of tensor `which`
    if (col == 0 && rank == 0 && which < 2 && a.side_dst[which]) {
        uint32_t* sd = a.side_dst[which] + (int64_t)m * a.map_stride;
        const uint32_t* ss = a.side_src[which] + (int64_t)m * a.map_stride;
        for (int o = o_start + threadIdx.x; o < Nout; o += kCompactThreads) sd[o] = ss[o];
    }
    // positions per CTA per super-tile: everything that is left, shared out evenly, capped by the buffer
    int R = (max(Nout - o_start, 1) + S - 1) / S;
    R = (R + RL - 1) / RL * RL;
    R = min(R, a.Rmax);
    const int Rc = R * S;
    uint4* buf[2] = {tile, tile + (size_t)a.Rmax * a.Vsub};
    // Per position of a super-tile: s_idx = row to copy from, -1 = nothing to do (past the end, the row stays
    // where it is, or it is the merged row); fetched two rounds ahead so that no copy ever waits for it.
    int32_t* s_idx = reinterpret_cast<int32_t*>(tile + 2 * (size_t)a.Rmax * a.Vsub);     // [3][Rmax]

    auto fetch_idx = [&](int t0, int* reg) {
#pragma unroll
        for (int u = 0; u < kIdxPerThread; ++u) {
            const int rr = threadIdx.x + u * kCompactThreads;
            const int o = t0 + rank * R + rr;
            int v = -1;
            if (rr < R && o < Nout) { v = src[o]; if (v == o) v = -1; }
            reg[u] = v;
        }
    };
    auto put_idx = [&](int slot, const int* reg) {
#pragma unroll
        for (int u = 0; u < kIdxPerThread; ++u) {
            const int rr = threadIdx.x + u * kCompactThreads;
            if (rr < R) s_idx[slot * a.Rmax + rr] = reg[u];
        }
    };
    auto load_tile = [&](int slot, uint4* dstbuf) {
        for (int rr = rl; rr < R; rr += RL) {
            const int v = s_idx[slot * a.Rmax + rr];
            if (v >= 0) {
#pragma unroll
                for (int ci = 0; ci < MAXC; ++ci) {
                    const int c = cg + ci * CG;
                    if (c < vw) cp_async16(&dstbuf[rr * a.Vsub + c], rows + (int64_t)v * V + c);
                }
            }
        }
        cp_async_commit_group();
    };

    {
        int reg[kIdxPerThread];
        fetch_idx(o_start, reg);
        put_idx(0, reg);
        fetch_idx(o_start + Rc, reg);
        put_idx(1, reg);
        __syncthreads();
    }
    load_tile(0, buf[0]);
    if (a.early) pdl_enter();                         // the partial rows and every write come after the kernel ahead
    int k = 0;
    for (int t0 = o_start; t0 < Nout; t0 += Rc, ++k) {
        if (t0 + Rc < Nout) load_tile((k + 1) % 3, buf[(k + 1) & 1]);
        else cp_async_commit_group();
        int reg[kIdxPerThread];
        fetch_idx(t0 + 2 * Rc, reg);                  // in flight while this round runs
        cp_async_wait_group<1>();                     // this super-tile's rows have landed
        __syncthreads();                              // ... for every thread of this CTA
        if (S > 1) cluster_barrier_exec();            // ... in every CTA of the cluster
        const uint4* cur = buf[k & 1];
        const int32_t* cur_idx = s_idx + (k % 3) * a.Rmax;
        const int lo = t0 + rank * R;
        for (int rr = rl; rr < R; rr += RL) {
            if (cur_idx[rr] >= 0) {
#pragma unroll
                for (int ci = 0; ci < MAXC; ++ci) {
                    const int c = cg + ci * CG;
                    if (c < vw) rows[(int64_t)(lo + rr) * V + c] = cur[rr * a.Vsub + c];
                }
            }
        }
        if (a.partial && a.merged_row >= lo && a.merged_row < lo + R && a.merged_row < Nout) {
            // the merged row: partial sums added in their order, rounded once
            const float* pp = a.partial + (int64_t)((b * a.G + g) * a.T + which) * a.P * V * 8 + (int64_t)c0 * 8;
            for (int c = threadIdx.x; c < vw; c += kCompactThreads)
                rows[(int64_t)a.merged_row * V + c] = sum_partials(pp, a.P, (int64_t)V * 8, c);
        }
        put_idx((k + 2) % 3, reg);
        __syncthreads();                              // buffer and index slot are reused in the next round
    }
    cp_async_wait_group<0>();
}

lvlm_status launch_inplace_compact(const CompactJob& j, cudaStream_t stream) {
    const bool fin = j.fin_base != nullptr;
    if (fin && (!j.fin_partial || j.fin_P <= 0 || j.fin_V <= 0 || j.B <= 0)) return LVLM_ERR_INVALID_ARG;
    InplaceArgs a = {};
    a.fin_base = static_cast<char*>(j.fin_base); a.fin_stride_b = j.fin_stride_b; a.fin_row = j.fin_row;
    a.fin_V = j.fin_V; a.fin_P = j.fin_P; a.fin_partial = j.fin_partial; a.fin_y = -1;
    if (!j.base0) {                                      // only the merged row of the other tensor
        if (!fin) return LVLM_ERR_INVALID_ARG;
        a.fin_y = 0; a.S = 1; a.G = 1; a.T = 1;
        const int ctas = (j.fin_V + kCompactThreads - 1) / kCompactThreads;
        return launch_kernel(inplace_compact_kernel<1>, dim3((unsigned)ctas, 1, (unsigned)j.B), dim3(kCompactThreads), 0,
                             stream, 1, a);
    }
    if (!j.src_map || !j.meta || j.B <= 0 || j.G <= 0 || j.V <= 0 || j.N <= 0) return LVLM_ERR_INVALID_ARG;
    if (j.partial && (j.P <= 0 || j.merged_row < 0)) return LVLM_ERR_INVALID_ARG;
    a.base0 = static_cast<char*>(j.base0);
    a.base1 = static_cast<char*>(j.base1);
    a.stride_b = j.stride_b; a.stride_g = j.stride_g;
    a.G = j.G; a.T = j.base1 ? 2 : 1; a.V = j.V; a.Nout = j.Nout;
    a.meta_stride = j.meta_stride; a.maps_per_g = j.maps_per_g;
    a.map_stride = j.map_stride > 0 ? j.map_stride : j.N;
    a.src_map = j.src_map; a.meta = j.meta; a.nout = j.nout;
    a.merged_row = j.merged_row; a.partial = j.partial; a.P = j.P;
    a.early = j.maps_ready && !j.side_dst[0] && !j.side_dst[1] ? 1 : 0;
    if (fin) a.fin_y = j.G * a.T;
    for (int i = 0; i < 2; ++i) {
        a.side_dst[i] = static_cast<uint32_t*>(j.side_dst[i]);
        a.side_src[i] = static_cast<const uint32_t*>(j.side_src[i]);
    }
    if (a.side_dst[1] && !j.base1) return LVLM_ERR_INVALID_ARG;   // the second array rides with the second tensor

    // enough CTAs to fill the GPU: first a cluster per sequence, then column groups of wide rows
    const int64_t nseq = (int64_t)j.B * j.G * a.T;
    int S = 1;
    while (S < kCompactMaxCluster && nseq * (2 * S) <= kCompactTargetCtas && j.N / (2 * S) >= 32) S *= 2;
    int Vsub = j.V;
    while (Vsub > 8 && nseq * S * ((j.V + Vsub - 1) / Vsub) < kCompactTargetCtas) Vsub = ((Vsub + 1) / 2 + 7) / 8 * 8;
    // rows wider than the per-thread budget are always split
    while (Vsub > kCompactMaxC * kCompactThreads) Vsub = ((Vsub + 1) / 2 + 7) / 8 * 8;
    const int ncol = (j.V + Vsub - 1) / Vsub;
    a.S = S; a.Vsub = Vsub;
    int CG = 1;
    while (CG * 2 <= Vsub && CG * 2 <= kCompactThreads) CG *= 2;
    if ((Vsub + CG - 1) / CG > kCompactMaxC) return LVLM_ERR_UNSUPPORTED;
    a.CG = CG; a.RL = kCompactThreads / CG;
    // staging buffers: as large as the number of CTAs per SM allows (one, two or four of them)
    // (clusters are placed inside one GPC: about 128 CTAs in clusters of 8 run at a time with one CTA per SM)
    const int64_t ctas = (nseq + (fin ? j.B : 0)) * S * ncol;
    const int per_wave = S > 1 ? 128 : 148;
    const int buf_bytes = ctas <= per_wave ? 96 * 1024 : (ctas <= 2 * per_wave ? 48 * 1024 : 24 * 1024);
    int R = buf_bytes / (Vsub * 16);
    R = R > kIdxPerThread * kCompactThreads ? kIdxPerThread * kCompactThreads : R;
    R = R / a.RL * a.RL;
    if (R < a.RL) R = a.RL;
    a.Rmax = R;
    const size_t smem = 2 * (size_t)R * Vsub * 16 + 3 * (size_t)R * 4;
    if (smem > (size_t)kMaxDynSmem) return LVLM_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)(ncol * S), (unsigned)(j.G * a.T + (fin ? 1 : 0)), (unsigned)j.B);
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
